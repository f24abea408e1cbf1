"""CPU-only checks of the CUDA library: it loads, exports what include/lq.h declares, validates
arguments, and its host-side mirror of Algorithm 1 agrees with the oracle (bookkeeping-only mode)."""
import os
import re

import numpy as np
import pytest

import oracle
from helpers import alg1_python
from paper_2503_19950_b200 import LQ_DEVICE_NONE, LogQuantCache, LogQuantError, binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module", autouse=True)
def _built():
    build.build()


def test_library_exports_every_declared_symbol():
    header = open(os.path.join(ROOT, "include", "lq.h")).read()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    declared = sorted(set(re.findall(r"\b(lq_[a-z_]+)\s*\(", header)))
    assert "lq_decode_attn" in declared and "lq_compress" in declared and len(declared) >= 9
    lib = binding.load_library()
    for name in declared:
        assert hasattr(lib, name), name
    assert sorted(binding.SYMBOLS) == declared


def test_status_strings():
    lib = binding.load_library()
    assert lib.lq_status_str(0) == b"ok"
    assert len({lib.lq_status_str(i) for i in range(8)}) == 8


def _dry(W=4, G=4, **kw):
    args = dict(n_layers=1, batch=1, n_q_heads=4, n_kv_heads=2, window=W, group=G, max_tokens=4096,
                device=LQ_DEVICE_NONE)
    args.update(kw)
    return LogQuantCache(**args)


@pytest.mark.parametrize("bad", [dict(group=16), dict(group=48, window=96), dict(head_dim=64),
                                 dict(bits=3), dict(bits=8),
                                 dict(n_q_heads=18, n_kv_heads=2), dict(window=1024)])
def test_unsupported_configurations(bad):
    with pytest.raises(LogQuantError) as e:
        _dry(W=bad.pop("window", 128), G=bad.pop("group", 32), **bad)
    assert e.value.status == binding.LQ_ERR_UNSUPPORTED


@pytest.mark.parametrize("bad", [dict(n_q_heads=5, n_kv_heads=2), dict(batch=0), dict(max_tokens=0), dict(n_layers=0)])
def test_invalid_configurations(bad):
    with pytest.raises(LogQuantError) as e:
        _dry(W=128, G=32, **bad)
    assert e.value.status == binding.LQ_ERR_INVALID_ARG


def test_no_gpu_means_no_compute():
    # without a CUDA device there is no fallback: creation on device 0 fails here, and the
    # bookkeeping-only mode refuses the compute calls
    import torch
    if not torch.cuda.is_available():
        with pytest.raises(LogQuantError):
            LogQuantCache(1, 1, 4, 2, 128, 32, 1024, device=0)
    c = _dry(W=128, G=32)
    c.append(0, None, None, n_tokens=10)
    with pytest.raises(LogQuantError) as e:
        c._check(c._lib.lq_decode_attn(c._h, 0, None, 0.0, None, 0, None))
    assert e.value.status == binding.LQ_ERR_UNSUPPORTED


def test_allocator_hooks_come_in_pairs():
    cfg = binding.lq_config_t(1, 1, 4, 2, 128, 128, 32, 2, 1024, 1, LQ_DEVICE_NONE, 0, 0, 0, 0,
                              binding.ALLOC_FN(lambda n, ctx: 0), binding.FREE_FN(0), None)
    import ctypes
    h = ctypes.c_void_p()
    assert binding.load_library().lq_cache_create(ctypes.byref(cfg), ctypes.byref(h)) == binding.LQ_ERR_INVALID_ARG


def test_padding_arguments_without_a_device():
    c = _dry(W=128, G=32, batch=3)
    c.set_padding([0, 5, 9])
    c.set_padding(None)
    with pytest.raises(LogQuantError) as e:
        c.set_padding([0, -2, 1])
    assert e.value.status == binding.LQ_ERR_INVALID_ARG
    with pytest.raises(ValueError):
        c.set_padding([1, 2])
    with pytest.raises(LogQuantError) as e:  # still no compute without a device
        c._check(c._lib.lq_decode_attn_fp_only(c._h, 0, None, 0.0, None, 0, None))
    assert e.value.status == binding.LQ_ERR_UNSUPPORTED


@pytest.mark.parametrize("W,G", [(32, 32), (64, 32), (128, 64), (256, 64)])
def test_host_mirror_of_algorithm1_matches_oracle(W, G):
    c = _dry(W=W, G=G, max_tokens=40 * W)
    n = 0
    rng = np.random.default_rng(W)
    while n < 30 * W:
        step = int(rng.integers(1, 2 * W))
        c.append(0, None, None, n_tokens=step)
        n += step
        kept, quant, ev = oracle.filter_ids(W, n)
        img = c.export(0, ids_only=True)
        inf = c.info(0)
        assert (inf.n_seen, inf.n_fp, inf.n_quant, inf.n_events) == (n, len(kept), len(quant), ev)
        assert img["kept_ids"].tolist() == kept.tolist()
        assert img["quant_ids"].tolist() == quant.tolist()
    A, Q = alg1_python(W, n)
    assert img["kept_ids"].tolist() == A and img["quant_ids"].tolist() == Q


@pytest.mark.parametrize("W,G", [(32, 32), (128, 64)])
def test_recent_window_comparator_keeps_exactly_the_newest_tokens(W, G):
    """LQ_FILTER_RECENT (comparator): the W oldest of the 3W full-precision tokens leave on overflow, so the
    kept set is always the newest n_fp tokens and the store order is the token order (closed form), in the
    host mirror and in the oracle alike."""
    c = _dry(W=W, G=G, max_tokens=20 * W, filter=binding.LQ_FILTER_RECENT)
    oc = oracle.OracleCache(1, 4, 2, 128, W, G, recent_only=True)
    n = 0
    rng = np.random.default_rng(W + 1)
    while n < 12 * W:
        step = int(rng.integers(1, 2 * W))
        c.append(0, None, None, n_tokens=step)
        oc.append(np.zeros((1, 2, step, 128), np.uint16), np.zeros((1, 2, step, 128), np.uint16))
        n += step
        inf = c.info(0)
        n_ev = 0 if n <= 3 * W else (n - 3 * W + W - 1) // W
        assert (inf.n_seen, inf.n_events, inf.n_quant, inf.n_fp) == (n, n_ev, n_ev * W, n - n_ev * W)
        img = c.export(0, ids_only=True)
        assert img["kept_ids"].tolist() == list(range(n_ev * W, n))
        assert img["quant_ids"].tolist() == list(range(n_ev * W))
        oimg = oc.export()
        assert oimg["kept_ids"].tolist() == img["kept_ids"].tolist()
        assert oimg["quant_ids"].tolist() == img["quant_ids"].tolist()
    with pytest.raises(LogQuantError):
        _dry(W=W, G=G, filter=7)


@pytest.mark.parametrize("W,G", [(42, 64), (85, 64), (100, 32), (21, 32)])
def test_host_mirror_with_key_groups_across_overflow_steps(W, G):
    """W not a multiple of G: removed tokens wait at full precision until G of them form a key group.  The
    host mirror must agree with the oracle (which is pinned against the filter's closed form) on every count
    and on both id lists, whatever the chunking of the appends."""
    c = _dry(W=W, G=G, max_tokens=40 * W + 64)
    oc = oracle.OracleCache(1, 4, 2, 128, W, G)
    rng = np.random.default_rng(W)
    n = 0
    while n < 30 * W:
        step = int(rng.integers(1, 2 * W))
        c.append(0, None, None, n_tokens=step)
        oc.append(np.zeros((1, 2, step, 128), np.uint16), np.zeros((1, 2, step, 128), np.uint16))
        n += step
        inf = c.info(0)
        assert (inf.n_seen, inf.n_fp, inf.n_quant, inf.n_events) == (n, oc.n_fp, oc.n_quant, oc.n_events)
        assert inf.n_quant % G == 0 and inf.n_fp <= 3 * W + G - 1
        img, oimg = c.export(0, ids_only=True), oc.export()
        assert img["kept_ids"].tolist() == oimg["kept_ids"].tolist()
        assert img["quant_ids"].tolist() == oimg["quant_ids"].tolist()


def test_manual_compress_state_rules():
    W, G = 32, 32
    c = _dry(W=W, G=G, auto_compress=False, n_layers=3)
    with pytest.raises(LogQuantError) as e:
        c.compress(0)
    assert e.value.status == binding.LQ_ERR_NOT_FULL
    c.append(0, None, None, n_tokens=3 * W)
    with pytest.raises(LogQuantError) as e:
        c.append(0, None, None, n_tokens=1)
    assert e.value.status == binding.LQ_ERR_WINDOW_FULL
    assert c.info(0).n_seen == 3 * W  # the failed call changed nothing
    ids = c.next_evicted_ids(0)
    assert ids.tolist() == list(range(1, 2 * W, 2))
    c.append(1, None, None, n_tokens=5)
    c.compress(-1)  # layer 0 is full, layers 1 and 2 are skipped
    assert (c.info(0).n_fp, c.info(0).n_quant, c.info(0).n_events) == (2 * W, W, 1)
    assert (c.info(1).n_fp, c.info(1).n_events, c.info(2).n_seen) == (5, 0, 0)
    c.append(0, None, None, n_tokens=W)
    ids2 = c.next_evicted_ids(0)
    A, _ = alg1_python(W, 4 * W)  # state right before the second event
    assert ids2.tolist() == A[1:2 * W:2]
    with pytest.raises(LogQuantError) as e:
        c.append(0, None, None, n_tokens=10 ** 6)
    assert e.value.status == binding.LQ_ERR_CAPACITY


def test_info_byte_accounting():
    c = _dry(W=128, G=32, batch=8, n_q_heads=32, n_kv_heads=8, max_tokens=9000)
    c.append(0, None, None, n_tokens=8193)
    inf = c.info(0)
    assert (inf.n_quant, inf.n_fp) == (7936, 257)
    assert inf.bytes_quant_per_token == 96
    assert inf.bytes_decode_step == 64 * (7936 * 96 + 257 * 512)  # 57.18 MB
    c2 = _dry(W=256, G=64, batch=4, n_q_heads=28, n_kv_heads=4, max_tokens=33000)
    c2.append(0, None, None, n_tokens=32769)
    inf = c2.info(0)
    assert (inf.n_quant, inf.n_fp, inf.bytes_quant_per_token) == (32256, 513, 80)
    c4 = _dry(W=128, G=32, batch=8, n_q_heads=32, n_kv_heads=8, max_tokens=9000, bits=4)
    c4.append(0, None, None, n_tokens=8193)
    inf = c4.info(0)
    assert (inf.n_quant, inf.n_fp, inf.bytes_quant_per_token) == (7936, 257, 160)
    assert inf.bytes_decode_step == 64 * (7936 * 160 + 257 * 512)


def test_new_entry_points_without_a_device():
    """Bookkeeping-only caches: guard check and status reset succeed trivially, the test hooks and lq_import refuse
    or do nothing; null handles are argument errors."""
    import numpy as np
    c = _dry(W=128, G=32)
    assert c.check_guards() == 0
    c.reset_kernel_status()
    c.debug_stall_next_decode()
    with pytest.raises(LogQuantError) as e:
        c.debug_bad_slot_next_append()   # only the index-check build of the library takes this hook
    assert e.value.status == binding.LQ_ERR_UNSUPPORTED
    img = dict(kept_ids=np.zeros(4, np.int32), quant_ids=np.zeros(0, np.int32))
    with pytest.raises(LogQuantError) as e:
        c.import_image(0, img, 4)
    assert e.value.status == binding.LQ_ERR_UNSUPPORTED
    lib = c._lib
    n = binding.C.c_int32(0)
    assert lib.lq_check_guards(None, binding.C.byref(n)) == binding.LQ_ERR_INVALID_ARG
    assert lib.lq_reset_kernel_status(None) == binding.LQ_ERR_INVALID_ARG
    assert lib.lq_debug_stall_next_decode(None) == binding.LQ_ERR_INVALID_ARG
    assert lib.lq_import(None, 0, None, 1, 0, 0) == binding.LQ_ERR_INVALID_ARG
    assert c.info(0).n_ctas_overlapped == 0


@pytest.mark.parametrize("W,G,recent", [(32, 32, False), (64, 32, False), (128, 64, False), (64, 64, True),
                                        (42, 64, False), (48, 32, False), (100, 64, True), (21, 32, False)])
def test_chunks_appended_to_a_layer_in_use_go_through_the_one_launch_plan(W, G, recent):
    """A chunk of at least 2 W tokens that makes a layer in use overflow is planned as ONE launch (sources of the new
    key groups, take-over lists, copy list).  Without a device the library plays that plan on token ids and checks
    that no slot is read by one thread and written by another, that each key group gathers its tokens in store
    order and that the store ends as its maps say (a failed check is an error status); here the counts and both id
    lists must also follow the oracle through every mix of first-chunk sizes and chunk lengths, with
    token-by-token steps (the overflow step's own slot rules) in between."""
    rng = np.random.default_rng(W + G + recent)
    for first in (1, W - 1, 2 * W - 3, 2 * W, 2 * W + 1, 3 * W - 1, 3 * W):
        c = _dry(W=W, G=G, max_tokens=80 * W, filter=binding.LQ_FILTER_RECENT if recent else 0)
        oc = oracle.OracleCache(1, 4, 2, 128, W, G, recent_only=recent)
        n = 0
        for step in [first] + [int(x) for x in rng.choice([1, 2, W, W + 1, 2 * W - 1, 2 * W, 3 * W, 3 * W + 5, 7 * W + 3],
                                                         size=14)]:
            c.append(0, None, None, n_tokens=step)
            oc.append(np.zeros((1, 2, step, 128), np.uint16), np.zeros((1, 2, step, 128), np.uint16))
            n += step
            inf = c.info(0)
            assert (inf.n_seen, inf.n_fp, inf.n_quant, inf.n_events) == (n, oc.n_fp, oc.n_quant, oc.n_events)
            img, oimg = c.export(0, ids_only=True), oc.export()
            assert img["kept_ids"].tolist() == oimg["kept_ids"].tolist()
            assert img["quant_ids"].tolist() == oimg["quant_ids"].tolist()
        c.close()
        oc.close()

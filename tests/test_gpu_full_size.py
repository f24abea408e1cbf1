"""GPU parity at the full sizes of the benchmark configurations (one layer cache each), default kernel and
library-chosen split count: bit-exact canonical image and attention within tolerance against the float64
oracle for every (batch row, head).  The first group of tests drives decode through lq_append + lq_decode_attn;
the `timed entry point` tests drive it through the calls bench.py times -- lq_append_decode_attn (append and
attention in one launch) and lq_decode_step_host (host buffers, pinned and pageable) -- over 128 and more
decode steps with one window overflow in the middle of the run."""
import numpy as np
import pytest
import torch

import oracle
from gpu_common import assert_images_equal, attn_tolerance
from paper_2503_19950_b200 import LogQuantCache, build, synth

pytestmark = pytest.mark.gpu
D = 128


@pytest.fixture(scope="module", autouse=True)
def _built():
    build.build()


def _run(B, Hq, Hkv, W, G, ctx, seed, n_steps, n_outliers=3, planted=False, image_stride=1, bits=2, pad=None):
    dev = "cuda"
    total = ctx + n_steps
    outl = synth.outlier_channels(seed, Hkv, D, n_outliers) if n_outliers else None
    u = synth.unit_vectors(seed, Hkv, D) if planted else None
    cache = LogQuantCache(1, B, Hq, Hkv, W, G, max_tokens=total + 8, bits=bits)
    oc = oracle.OracleCache(B, Hq, Hkv, D, W, G, bits=bits)
    if pad is not None:
        cache.set_padding(pad)
    chunk = 2048
    for t0 in list(range(0, ctx, chunk)) + [ctx + i for i in range(n_steps)]:
        n = min(chunk, ctx - t0) if t0 < ctx else 1
        k, v = synth.keys_values(seed, B, Hkv, n, D, dev, token_start=t0, token_total=total, outliers=outl)
        if u is not None:
            k = synth.plant_spikes(k, u, 16.0, t0, ctx)
        cache.append(0, k, v)
        oc.append(synth.bf16_bits(k), synth.bf16_bits(v))
        if t0 < ctx:
            continue
        step = t0 - ctx
        inf = cache.info(0)
        assert (inf.n_fp, inf.n_quant, inf.n_events) == (oc.n_fp, oc.n_quant, oc.n_events)
        if step % image_stride == 0:
            assert_images_equal(cache.export(0), oc.export())
        q = synth.queries(seed, B, Hq, D, step, dev)
        if u is not None:
            q = (q.float() + 4.0 * u.to(dev).repeat_interleave(Hq // Hkv, dim=0)[None]).to(torch.bfloat16)
        out = torch.full((B, Hq, D), float("nan"), device=dev)
        cache.decode_attn(0, q, out)
        torch.cuda.synchronize()
        if pad is not None:
            ref = oc.attention_subset(synth.bf16_bits(q), 1 / np.sqrt(D), pad=pad)
        else:
            ref = oc.attention(synth.bf16_bits(q), 1 / np.sqrt(D), n_threads=16)
        got = out.cpu().numpy().astype(np.float64)
        err, tol = float(np.abs(got - ref).max()), attn_tolerance(ref)
        assert np.isfinite(got).all() and err <= tol, f"step {step}: max|delta| {err:.3e} > {tol:.3e}"
    assert cache.kernel_status() == 0
    return cache.info(0)


def test_config2_llama3_8b_layer_8k():
    # 32 q / 8 kv heads, batch 8, context 8192, W=128, G=32: 61 overflow events in the prefill, the 62nd
    # on the first decode step
    inf = _run(B=8, Hq=32, Hkv=8, W=128, G=32, ctx=8192, seed=2, n_steps=2)
    assert (inf.n_quant, inf.n_fp) == (7936, 258)


def test_config3_batch16_4k():
    inf = _run(B=16, Hq=32, Hkv=8, W=128, G=32, ctx=4096, seed=3, n_steps=1)
    assert (inf.n_quant, inf.n_fp) == (3840, 257)


@pytest.mark.parametrize("B", [32, 64])
def test_config3_larger_batches_4k(B):
    # 256 and 512 (b, kv) pairs: one to three CTAs per pair, and at batch 64 a step of two launches
    inf = _run(B=B, Hq=32, Hkv=8, W=128, G=32, ctx=4096, seed=3, n_steps=1, image_stride=1)
    assert (inf.n_quant, inf.n_fp) == (3840, 257)


def test_config4_gqa7_32k_planted_spikes():
    # 28 q / 4 kv heads, W=256, G=64, keys with planted high-logit tokens at log-spaced distances
    inf = _run(B=4, Hq=28, Hkv=4, W=256, G=64, ctx=32768, seed=4, n_steps=1, n_outliers=0, planted=True)
    assert (inf.n_quant, inf.n_fp) == (32256, 513)


def test_config5_mha_128k_one_layer():
    inf = _run(B=1, Hq=32, Hkv=32, W=256, G=32, ctx=131072, seed=5, n_steps=1)
    assert (inf.n_quant, inf.n_fp) == (130560, 513)


def test_config4_with_four_bit_codes_at_group_64():
    # config 4 (GQA-7, W = 256, G = 64) at the paper's second precision and its own group size (Sec. 3.1, Table 3)
    inf = _run(B=4, Hq=28, Hkv=4, W=256, G=64, ctx=32768, seed=4, n_steps=2, bits=4)
    assert inf.bytes_quant_per_token == 144


def test_config2_with_four_bit_codes():
    # the llama3-8b-8k-int4 workload of bench.py: config 2 at the paper's second precision
    inf = _run(B=8, Hq=32, Hkv=8, W=128, G=32, ctx=8192, seed=2, n_steps=2, bits=4)
    assert inf.bytes_quant_per_token == 160


def test_config2_left_padded_batch():
    # config 2 as a ragged batch: prompts of 8192, 8191, 8000, 7169, 4096, 2049, 300 and 2 real tokens,
    # left-padded to 8192 positions
    pad = [0, 1, 192, 1023, 4096, 6143, 7892, 8190]
    inf = _run(B=8, Hq=32, Hkv=8, W=128, G=32, ctx=8192, seed=6, n_steps=2, pad=pad)
    assert (inf.n_quant, inf.n_fp) == (7936, 258)


def test_config4_left_padded_batch():
    inf = _run(B=4, Hq=28, Hkv=4, W=256, G=64, ctx=32768, seed=7, n_steps=1, n_outliers=0, planted=True,
               pad=[0, 31, 16385, 32700])
    assert (inf.n_quant, inf.n_fp) == (32256, 513)


# ---- the entry points bench.py times, at full size -------------------------------------------------
def _run_timed_entry(entry, B, Hq, Hkv, W, G, ctx, seed, check_steps, n_outliers=3, planted=False):
    """Prefill ctx tokens, then max(check_steps) decode steps through `entry`: "fused" = lq_append_decode_attn,
    "host_pinned" / "host_pageable" = lq_decode_step_host.  Steps are counted from 1; on the steps named in
    check_steps the image and the attention output are compared with the oracle, on the others only the
    bookkeeping (so that an overflow step in between is crossed by both sides)."""
    dev = "cuda"
    n_steps = max(check_steps)
    total = ctx + n_steps
    outl = synth.outlier_channels(seed, Hkv, D, n_outliers) if n_outliers else None
    u = synth.unit_vectors(seed, Hkv, D) if planted else None
    cache = LogQuantCache(1, B, Hq, Hkv, W, G, max_tokens=total + 8)
    oc = oracle.OracleCache(B, Hq, Hkv, D, W, G)
    chunk = 2048
    for t0 in range(0, ctx, chunk):
        n = min(chunk, ctx - t0)
        k, v = synth.keys_values(seed, B, Hkv, n, D, dev, token_start=t0, token_total=total, outliers=outl)
        if u is not None:
            k = synth.plant_spikes(k, u, 16.0, t0, ctx)
        cache.append(0, k, v)
        oc.append(synth.bf16_bits(k), synth.bf16_bits(v))
    events0 = oc.n_events
    host = entry.startswith("host")
    pin = (lambda t: t.cpu().pin_memory()) if entry == "host_pinned" else (lambda t: t.cpu())
    out = torch.full((B, Hq, D), float("nan"), device=dev)
    out_host = torch.full((B, Hq, D), float("nan"))
    if entry == "host_pinned":
        out_host = out_host.pin_memory()
    for step in range(1, n_steps + 1):
        k, v = synth.keys_values(seed, B, Hkv, 1, D, dev, token_start=ctx + step - 1, token_total=total, outliers=outl)
        q = synth.queries(seed, B, Hq, D, step, dev)
        if u is not None:
            q = (q.float() + 4.0 * u.to(dev).repeat_interleave(Hq // Hkv, dim=0)[None]).to(torch.bfloat16)
        if host:
            cache.decode_step_host(0, pin(k), pin(v), pin(q), out_host, sync=True)
            got = out_host.numpy().astype(np.float64)
        else:
            cache.append_decode_attn(0, k, v, q, out)
        oc.append(synth.bf16_bits(k), synth.bf16_bits(v))
        inf = cache.info(0)
        assert (inf.n_seen, inf.n_fp, inf.n_quant, inf.n_events) == (oc.n_seen, oc.n_fp, oc.n_quant, oc.n_events)
        if step not in check_steps:
            continue
        if not host:
            torch.cuda.synchronize()
            got = out.cpu().numpy().astype(np.float64)
        assert_images_equal(cache.export(0), oc.export())
        ref = oc.attention(synth.bf16_bits(q), 1 / np.sqrt(D), n_threads=16)
        err, tol = float(np.abs(got - ref).max()), attn_tolerance(ref)
        assert np.isfinite(got).all() and err <= tol, f"{entry} step {step}: max|delta| {err:.3e} > {tol:.3e}"
    assert cache.kernel_status() == 0
    return oc.n_events - events0


@pytest.mark.parametrize("entry", ["fused", "host_pinned", "host_pageable"])
def test_config2_timed_entry_points_over_128_steps(entry):
    # the prompt is W/2 tokens short of 8192, so the overflow step falls on decode step 65: steps 1, 2 and 64
    # come before it, 65 is the step that runs it, 128 well after it
    events = _run_timed_entry(entry, B=8, Hq=32, Hkv=8, W=128, G=32, ctx=8192 - 64, seed=2,
                              check_steps=[1, 2, 64, 65, 128])
    assert events == 1


def test_config2_fused_entry_point_overflow_on_the_first_step():
    # full 8192-token prompt: the bf16 window is exactly full, the first decode step runs the overflow step
    events = _run_timed_entry("fused", B=8, Hq=32, Hkv=8, W=128, G=32, ctx=8192, seed=2, check_steps=[1, 2, 64, 128])
    assert events == 1


@pytest.mark.parametrize("entry", ["fused", "host_pinned"])
def test_config4_timed_entry_points_across_an_overflow(entry):
    # W = 256: with the prompt W/2 short the overflow step falls on decode step 129
    events = _run_timed_entry(entry, B=4, Hq=28, Hkv=4, W=256, G=64, ctx=32768 - 128, seed=4,
                              check_steps=[1, 2, 64, 128, 129, 130], n_outliers=0, planted=True)
    assert events == 1


# ---- overlapped launches (LQ_FLAG_OVERLAP_DECODE), the configuration bench.py times ------------------
@pytest.mark.parametrize("entry", ["fused", "host_pinned"])
@pytest.mark.parametrize("cfg", [dict(B=8, Hq=32, Hkv=8, W=128, G=32, ctx=8192 - 3, seed=2, n_outliers=3),
                                 dict(B=4, Hq=28, Hkv=4, W=256, G=64, ctx=32768 - 3, seed=4, n_outliers=0),
                                 # launches of more than 192 MB: fused only because launches overlap
                                 dict(B=64, Hq=32, Hkv=8, W=128, G=32, ctx=4096 - 3, seed=3, n_outliers=3),
                                 dict(B=1, Hq=32, Hkv=32, W=256, G=32, ctx=131072 - 3, seed=5, n_outliers=3,
                                      entries=("fused",))],
                         ids=["llama3-8b-8k", "gqa7-32k", "llama3-8b-4k-b64", "mha-128k"])
def test_overlapped_launches_of_stacked_layers_at_full_size(entry, cfg):
    """Three layer caches with different contents, six decode steps enqueued layer after layer without any
    synchronisation in between (the fourth step overflows every window): every launch but the first of a chain
    overlaps the one before it, with a third of a wave per launch.  Every layer's output of every step and the
    final images must be the oracle's."""
    from paper_2503_19950_b200 import LQ_FLAG_OVERLAP_DECODE
    if entry not in cfg.get("entries", ("fused", "host_pinned")):
        pytest.skip("one entry point is enough at this size")
    B, Hq, Hkv, W, G, ctx, seed = (cfg[k] for k in ("B", "Hq", "Hkv", "W", "G", "ctx", "seed"))
    L, n_steps, dev = 3, 6, "cuda"
    total = ctx + n_steps
    cache = LogQuantCache(L, B, Hq, Hkv, W, G, max_tokens=total + 8, flags=LQ_FLAG_OVERLAP_DECODE)
    ocs = [oracle.OracleCache(B, Hq, Hkv, D, W, G) for _ in range(L)]
    outl = [synth.outlier_channels(seed + 10 * l, Hkv, D, cfg["n_outliers"]) if cfg["n_outliers"] else None for l in range(L)]
    for l in range(L):
        for t0 in range(0, ctx, 4096):
            n = min(4096, ctx - t0)
            k, v = synth.keys_values(seed + 10 * l, B, Hkv, n, D, dev, token_start=t0, token_total=total, outliers=outl[l])
            cache.append(l, k, v)
            ocs[l].append(synth.bf16_bits(k), synth.bf16_bits(v))
    launches0 = cache.info(0).n_kernel_launches
    pin = lambda t: t.cpu().pin_memory()
    outs = [[(torch.full((B, Hq, D), float("nan")).pin_memory() if entry == "host_pinned"
              else torch.full((B, Hq, D), float("nan"), device=dev)) for _ in range(L)] for _ in range(n_steps)]
    qs, keep = [], []
    for step in range(n_steps):          # everything is enqueued first ...
        qs.append([])
        for l in range(L):
            k, v = synth.keys_values(seed + 10 * l, B, Hkv, 1, D, dev, token_start=ctx + step, token_total=total,
                                     outliers=outl[l])
            q = synth.queries(seed + 10 * l, B, Hq, D, step, dev)
            qs[step].append(q)
            if entry == "host_pinned":
                hk, hv, hq = pin(k), pin(v), pin(q)
                keep.append((hk, hv, hq))
                cache.decode_step_host(l, hk, hv, hq, outs[step][l], sync=False)
            else:
                cache.append_decode_attn(l, k, v, q, outs[step][l])
            ocs[l].append(synth.bf16_bits(k), synth.bf16_bits(v))
    torch.cuda.synchronize()             # ... and checked afterwards, against oracles replayed step by step
    assert cache.kernel_status() == 0
    # one launch per layer and step, except in the step that overflows (overflow kernel, append, attention)
    if entry == "fused":
        assert cache.info(0).n_kernel_launches - launches0 == L * (n_steps - 1) + 3 * L
    replay = [oracle.OracleCache(B, Hq, Hkv, D, W, G) for _ in range(L)]
    for l in range(L):
        for t0 in range(0, ctx, 4096):
            n = min(4096, ctx - t0)
            k, v = synth.keys_values(seed + 10 * l, B, Hkv, n, D, dev, token_start=t0, token_total=total, outliers=outl[l])
            replay[l].append(synth.bf16_bits(k), synth.bf16_bits(v))
    for step in range(n_steps):
        for l in range(L):
            k, v = synth.keys_values(seed + 10 * l, B, Hkv, 1, D, dev, token_start=ctx + step, token_total=total,
                                     outliers=outl[l])
            replay[l].append(synth.bf16_bits(k), synth.bf16_bits(v))
            ref = replay[l].attention(synth.bf16_bits(qs[step][l]), 1 / np.sqrt(D), n_threads=16)
            got = outs[step][l].cpu().numpy().astype(np.float64)
            err, tol = float(np.abs(got - ref).max()), attn_tolerance(ref)
            assert np.isfinite(got).all() and err <= tol, f"step {step} layer {l}: max|delta| {err:.3e} > {tol:.3e}"
    for l in range(L):
        assert replay[l].n_events == ocs[l].n_events and ocs[l].n_events >= 1
        assert_images_equal(cache.export(l), ocs[l].export())
    cache.close()


def test_long_run_of_overlapped_fused_steps_over_32_layers():
    """The pattern bench.py times, for longer: 32 layer caches of configuration 2, 260 decode steps of fused
    append+attention launches enqueued without a pause (three overflow steps per layer on the way), every launch
    overlapping its predecessor except around the overflow steps.  Four of the layers are replayed in the oracle:
    their outputs of the last step and their final images must be the oracle's; every layer's output is finite."""
    from paper_2503_19950_b200 import LQ_FLAG_OVERLAP_DECODE
    B, Hq, Hkv, W, G, ctx, seed, L, n_steps, dev = 8, 32, 8, 128, 32, 8192, 2, 32, 260, "cuda"
    checked = (0, 1, 15, 31)
    total = ctx + n_steps
    cache = LogQuantCache(L, B, Hq, Hkv, W, G, max_tokens=total + 8, flags=LQ_FLAG_OVERLAP_DECODE)
    ocs = {l: oracle.OracleCache(B, Hq, Hkv, D, W, G) for l in checked}
    outl = [synth.outlier_channels(seed + 10 * l, Hkv, D, 3) for l in range(L)]
    for l in range(L):
        for t0 in range(0, ctx, 4096):
            k, v = synth.keys_values(seed + 10 * l, B, Hkv, 4096, D, dev, token_start=t0, token_total=total, outliers=outl[l])
            cache.append(l, k, v)
            if l in ocs:
                ocs[l].append(synth.bf16_bits(k), synth.bf16_bits(v))
    # a small rotation of inputs per layer (as in the benchmark), generated before the run
    R = 4
    kvq = [[(synth.keys_values(seed + 10 * l + 1000 * i, B, Hkv, 1, D, dev, outliers=outl[l]),
             synth.queries(seed + 10 * l, B, Hq, D, i, dev)) for i in range(R)] for l in range(L)]
    outs = [torch.full((B, Hq, D), float("nan"), device=dev) for _ in range(L)]
    torch.cuda.synchronize()
    before = cache.info(0)
    for step in range(n_steps):
        for l in range(L):
            (k, v), q = kvq[l][step % R]
            cache.append_decode_attn(l, k, v, q, outs[l])
    torch.cuda.synchronize()
    after = cache.info(0)
    assert cache.kernel_status() == 0
    # an overflow step takes three launches per layer (overflow kernel, append, attention), none of them overlapped
    n_ovf = after.n_events - before.n_events
    assert n_ovf >= 2
    assert after.n_kernel_launches - before.n_kernel_launches == L * n_steps + 2 * n_ovf * L
    assert after.n_launches_overlapped - before.n_launches_overlapped >= L * (n_steps - n_ovf) - 1 - n_ovf
    for l in range(L):
        assert bool(torch.isfinite(outs[l]).all()), l
    for l in checked:
        for step in range(n_steps):
            (k, v), q = kvq[l][step % R]
            ocs[l].append(synth.bf16_bits(k), synth.bf16_bits(v))
        (k, v), q = kvq[l][(n_steps - 1) % R]
        ref = ocs[l].attention(synth.bf16_bits(q), 1 / np.sqrt(D), n_threads=16)
        got = outs[l].cpu().numpy().astype(np.float64)
        err, tol = float(np.abs(got - ref).max()), attn_tolerance(ref)
        assert err <= tol, f"layer {l}: max|delta| {err:.3e} > {tol:.3e}"
        assert_images_equal(cache.export(l), ocs[l].export())
    cache.close()
    for oc in ocs.values():
        oc.close()

"""GPU parity: the CUDA library (through the C-ABI) against the CPU oracle on the same seeded inputs.
Packed codes, scale/zero bits, full-precision rows and index sets must match bit for bit; attention
outputs within max|delta| <= 2e-3*max|ref| + 1e-3."""
import numpy as np
import pytest
import torch

import oracle
from gpu_common import assert_images_equal, attn_tolerance, run_case
from paper_2503_19950_b200 import (LQ_KERNEL_AUTO, LQ_KERNEL_MMA, LQ_KERNEL_SCALAR, LogQuantCache, LogQuantError,
                                   binding, build, synth)

pytestmark = pytest.mark.gpu

KERNELS = [LQ_KERNEL_SCALAR, LQ_KERNEL_MMA]


@pytest.fixture(scope="module", autouse=True)
def _built():
    build.build()


def test_generator_is_bit_identical_on_cpu_and_gpu():
    for shape, ax in [((2, 3, 50, 128), 2), ((4, 8, 128), None)]:
        a = synth.tensor_f32(5, 17, shape, "cpu", ax, 11, 100)
        b = synth.tensor_f32(5, 17, shape, "cuda", ax, 11, 100)
        assert torch.equal(a, b.cpu())
    k0, v0 = synth.keys_values(3, 2, 2, 40, 128, "cpu", 5, 64, synth.outlier_channels(3, 2, 128, 3))
    k1, v1 = synth.keys_values(3, 2, 2, 40, 128, "cuda", 5, 64, synth.outlier_channels(3, 2, 128, 3))
    assert torch.equal(k0, k1.cpu()) and torch.equal(v0, v1.cpu())


@pytest.mark.parametrize("kernel", KERNELS)
def test_config1_tiny_decode(kernel):
    # 1 layer, batch 1, 8 q heads / 2 KV heads, W=128, G=32: prefill 1024 (5 overflow events), 16 decode
    # steps, the first of which triggers the sixth event.  Full parity at every step.
    worst = run_case(B=1, Hq=8, Hkv=2, W=128, G=32, n_prefill=1024, n_steps=16, seed=1, kernel=kernel, n_outliers=4)
    assert worst <= 1.0


@pytest.mark.parametrize("kernel", KERNELS)
@pytest.mark.parametrize("B,Hq,Hkv,W,G,n_prefill,n_steps", [
    (2, 8, 2, 32, 32, 0, 3),        # a cache of 1..3 tokens, nothing quantised
    (1, 4, 4, 32, 32, 95, 4),       # crosses the first overflow (MHA, r = 1)
    (2, 14, 2, 64, 64, 64 * 9 + 7, 3),   # GQA-7, G = 64, ragged fp tail
    (1, 16, 2, 64, 32, 64 * 6 + 33, 2),  # r = 8
    (3, 6, 2, 256, 64, 256 * 5 + 100, 2),  # W = 256, r = 3
    (1, 2, 1, 512, 64, 512 * 4 + 1, 2),  # largest window
])
def test_shapes_and_edge_cases(kernel, B, Hq, Hkv, W, G, n_prefill, n_steps):
    worst = run_case(B, Hq, Hkv, W, G, n_prefill, n_steps, seed=7, kernel=kernel)
    assert worst <= 1.0


@pytest.mark.parametrize("kernel", KERNELS)
@pytest.mark.parametrize("G", [32, 64])
@pytest.mark.parametrize("B,Hq,Hkv,W,n_prefill,n_steps,chunk", [
    (1, 8, 2, 128, 1024, 4, None),          # the tiny configuration at 4 bits, prompt ingested in one launch
    (2, 4, 4, 64, 64 * 2 + 63, 4, 40),      # r = 1, crosses the first overflow step by step
    (2, 14, 2, 64, 64 * 7 + 9, 3, None),    # GQA-7: two column blocks, fp16 p.v
    (1, 16, 2, 64, 64 * 11 + 5, 2, 100),    # r = 8
    (1, 8, 2, 85, 85 * 6 + 30, 3, 97),      # W % G != 0: waiting tokens
])
def test_four_bit_cache(kernel, G, B, Hq, Hkv, W, n_prefill, n_steps, chunk):
    """bits = 4 (16 levels, two codes per byte in the image; two 2-bit planes on the device): same bar, at both
    group sizes (G = 64 is the paper's own, Sec. 3.1; its 9 KB tiles take the larger stages of the kernel)."""
    worst = run_case(B, Hq, Hkv, W, G, n_prefill, n_steps, seed=13, kernel=kernel, bits=4, prefill_chunk=chunk)
    assert worst <= 1.0


def test_four_bit_is_closer_to_exact_attention_than_two_bit():
    B, Hq, Hkv, W, G, D, n = 2, 8, 2, 64, 32, 128, 64 * 12
    k, v = synth.keys_values(17, B, Hkv, n, D, "cuda", outliers=synth.outlier_channels(17, Hkv, D, 3))
    q = synth.queries(17, B, Hq, D, 0, "cuda")
    kf, vf = k.float().repeat_interleave(Hq // Hkv, 1), v.float().repeat_interleave(Hq // Hkv, 1)
    p = torch.softmax(torch.einsum("bhd,bhtd->bht", q.float(), kf) / D ** 0.5, -1)
    exact = torch.einsum("bht,bhtd->bhd", p, vf)
    err = {}
    for bits in (2, 4):
        c = LogQuantCache(1, B, Hq, Hkv, W, G, max_tokens=n + 8, bits=bits)
        c.append(0, k, v)
        out = torch.empty(B, Hq, D, device="cuda")
        c.decode_attn(0, q, out)
        err[bits] = float((out - exact).abs().max())
        assert c.info(0).bytes_quant_per_token == (96 if bits == 2 else 160)  # G = 32: 64 * bits / 2 + 32 bytes of scale and zero
        c.close()
    assert err[4] < err[2] / 2


@pytest.mark.parametrize("kernel", KERNELS)
@pytest.mark.parametrize("bits,chunk", [(2, None), (4, 50)])
def test_recent_window_comparator(kernel, bits, chunk):
    """LQ_FILTER_RECENT: same kernels, other removal list (prompt ingestion and step-by-step overflow)."""
    worst = run_case(2, 8, 2, 64, 32, 64 * 8 + 21, 3, seed=19, kernel=kernel, bits=bits, prefill_chunk=chunk,
                     recent_only=True)
    assert worst <= 1.0


@pytest.mark.parametrize("kernel", KERNELS)
@pytest.mark.parametrize("B,Hq,Hkv,W,G,bits,n_prefill,n_steps,chunk", [
    (2, 8, 2, 42, 64, 2, 42 * 9 + 5, 4, None),    # the paper's W = 42 (reserved length 128), G = 64; one-launch prompt
    (1, 14, 2, 85, 64, 2, 85 * 7 + 30, 3, 97),    # W = 85 (reserved length 256), GQA-7, step-by-step overflow
    (2, 4, 4, 100, 32, 2, 100 * 5 + 1, 3, 1),     # G = 32, r = 1, one token at a time
    (1, 8, 2, 50, 32, 4, 50 * 8 + 17, 50, 60),    # 4-bit codes; the decode steps cross an overflow
])
def test_window_not_a_multiple_of_the_group(kernel, B, Hq, Hkv, W, G, bits, n_prefill, n_steps, chunk):
    """W % G != 0: removed tokens wait at full precision until G of them form a key group."""
    worst = run_case(B, Hq, Hkv, W, G, n_prefill, n_steps, seed=29, kernel=kernel, bits=bits, prefill_chunk=chunk,
                     check_image_every=7 if n_steps > 10 else 1)
    assert worst <= 1.0


def test_window_not_a_multiple_of_the_group_manual_overflow_and_layers():
    """W % G != 0 with caller-driven overflow steps (auto_compress = 0), several layers in one lq_compress(-1)
    call, and the host-buffer step."""
    B, Hq, Hkv, W, G, D, L = 2, 8, 2, 42, 64, 128, 3
    assert run_case(B, Hq, Hkv, W, G, 42 * 6 + 3, 3, seed=31, kernel=LQ_KERNEL_MMA, auto_compress=False) <= 1.0
    cache = LogQuantCache(L, B, Hq, Hkv, W, G, max_tokens=12 * W, auto_compress=False)
    ocs = [oracle.OracleCache(B, Hq, Hkv, D, W, G) for _ in range(L)]
    for rnd in range(4):  # layers 0 and 1 enter every round with a full window; layer 2 stays short
        for l, n in enumerate((3 * W, 3 * W, 30) if rnd == 0 else (0, 0, 0)):
            if n:
                k, v = synth.keys_values(50 + rnd, B, Hkv, n, D, "cuda", layer=l)
                cache.append(l, k, v)
                ocs[l].append(synth.bf16_bits(k), synth.bf16_bits(v))
        cache.compress(-1)
        for l in range(L):  # the oracle runs the overflow step when the next token arrives: feed one
            k, v = synth.keys_values(60 + rnd, B, Hkv, 1, D, "cpu", layer=l)
            q = synth.queries(60 + rnd, B, Hq, D, 0, "cpu", layer=l)
            out = torch.empty(B, Hq, D, dtype=torch.float32)
            k, v, q, out = k.pin_memory(), v.pin_memory(), q.pin_memory(), out.pin_memory()
            if l < 2:
                cache.decode_step_host(l, k, v, q, out)
            else:
                cache.append(l, k.cuda(), v.cuda())
                o = torch.empty(B, Hq, D, device="cuda")
                cache.decode_attn(l, q.cuda(), o)
                out = o.cpu()
            ocs[l].append(synth.bf16_bits(k), synth.bf16_bits(v))
            assert_images_equal(cache.export(l), ocs[l].export())
            ref = ocs[l].attention(synth.bf16_bits(q), 1 / np.sqrt(D))
            assert np.abs(out.numpy() - ref).max() <= attn_tolerance(ref)
        for l in range(2):  # bring layers 0 and 1 back to W - 1 below full for the next round
            k, v = synth.keys_values(70 + rnd, B, Hkv, W - 1, D, "cuda", layer=l)
            cache.append(l, k, v)
            ocs[l].append(synth.bf16_bits(k), synth.bf16_bits(v))
    assert [cache.info(l).n_events for l in range(L)] == [4, 4, 0]
    assert cache.kernel_status() == 0
    cache.close()


@pytest.mark.parametrize("B,Hq,Hkv,W,G,n_prefill", [
    (64, 32, 8, 32, 32, 32 * 6 + 17),   # 512 pairs: one CTA for most pairs, two for the rest
    (75, 8, 8, 32, 32, 32 * 12 + 31),   # 600 pairs: more pairs than one wave of CTAs, r = 1
    (40, 56, 8, 64, 64, 64 * 7 + 3),    # 320 pairs, GQA-7
])
def test_more_pairs_than_ctas_per_wave(B, Hq, Hkv, W, G, n_prefill):
    """Many (b, kv) pairs: the grid degenerates to one or two CTAs per pair, or to several waves."""
    worst = run_case(B, Hq, Hkv, W, G, n_prefill, 2, seed=37, kernel=LQ_KERNEL_MMA)
    assert worst <= 1.0


def _random_cases(n, seed):
    rng = np.random.default_rng(seed)
    cases = []
    while len(cases) < n:
        G = int(rng.choice([32, 64]))
        W = int(rng.choice([32, 42, 64, 85, 96, 100, 128, 192, 256]))
        Hkv = int(rng.choice([1, 2, 4]))
        r = int(rng.choice([1, 2, 3, 4, 5, 7, 8]))
        bits = 4 if rng.random() < 0.3 else 2
        B = int(rng.integers(1, 4))
        n_prefill = int(rng.integers(1, 9 * W))
        chunk = None if rng.random() < 0.5 else int(rng.integers(1, 3 * W))
        cases.append((B, Hkv * r, Hkv, W, G, bits, n_prefill, chunk, bool(rng.random() < 0.2)))
    return cases


@pytest.mark.parametrize("B,Hq,Hkv,W,G,bits,n_prefill,chunk,recent", _random_cases(12, 2024))
def test_seeded_random_configurations(B, Hq, Hkv, W, G, bits, n_prefill, chunk, recent):
    """A seeded draw over head ratios, windows, groups, code widths, prompt lengths, chunkings and filters."""
    worst = run_case(B, Hq, Hkv, W, G, n_prefill, 2, seed=100 + n_prefill, kernel=LQ_KERNEL_MMA, bits=bits,
                     prefill_chunk=chunk, recent_only=recent, check_image_every=1)
    assert worst <= 1.0


@pytest.mark.parametrize("kernel", KERNELS)
def test_chunked_prefill_and_manual_compress_give_the_same_image(kernel):
    # a prompt appended in ragged chunks, with the caller driving lq_compress, equals n single appends
    worst = run_case(2, 8, 2, 64, 32, 64 * 7 + 19, 2, seed=9, kernel=kernel, prefill_chunk=37, auto_compress=False)
    assert worst <= 1.0


@pytest.mark.parametrize("kernel", KERNELS)
def test_spiky_attention_and_custom_scale(kernel):
    # large queries make the softmax nearly one-hot: exercises the running-max rescale path
    worst = run_case(1, 8, 2, 64, 32, 64 * 8 + 5, 3, seed=11, kernel=kernel, sm_scale=0.25, q_gain=3.0)
    assert worst <= 1.0


@pytest.mark.parametrize("kernel", KERNELS)
@pytest.mark.parametrize("n_splits", [1, 2, 7, 64])
def test_any_split_count_gives_the_same_answer(kernel, n_splits):
    worst = run_case(1, 8, 2, 64, 32, 64 * 12 + 3, 1, seed=13, kernel=kernel, n_splits=n_splits, check_image_every=0)
    assert worst <= 1.0


def test_bf16_output():
    worst = run_case(2, 8, 2, 64, 32, 64 * 5 + 3, 2, seed=15, kernel=LQ_KERNEL_AUTO, out_dtype=torch.bfloat16,
                     check_image_every=0)
    assert worst <= 1.0


def test_constant_and_degenerate_groups():
    # constant keys/values (scale = 0), signed zeros and a wide-range group, bit-exact against the oracle
    B, Hq, Hkv, W, G, D = 1, 4, 1, 32, 32, 128
    N = 3 * W + 1
    k, v = synth.keys_values(21, B, Hkv, N, D, "cuda")
    k[:, :, :, 0] = 1.5          # constant channel -> scale 0
    k[:, :, 1::2, 1] = -0.0      # signed zeros as the group minimum
    k[:, :, 0::2, 1] = 0.0
    k[:, :, :, 2] = k[:, :, :, 2] * 1000
    v[:, :, 3, :] = -2.25        # constant token -> all value groups have scale 0
    v[:, :, 5, :32] = 0.0
    cache = LogQuantCache(1, B, Hq, Hkv, W, G, max_tokens=N + 4)
    oc = oracle.OracleCache(B, Hq, Hkv, D, W, G)
    cache.append(0, k, v)
    oc.append(synth.bf16_bits(k), synth.bf16_bits(v))
    assert oc.n_events == 1
    assert_images_equal(cache.export(0), oc.export())
    q = synth.queries(21, B, Hq, D, 0, "cuda")
    out = torch.empty(B, Hq, D, device="cuda")
    cache.decode_attn(0, q, out)
    ref = oc.attention(synth.bf16_bits(q), 1 / np.sqrt(D))
    assert np.abs(out.cpu().numpy() - ref).max() <= attn_tolerance(ref)


def test_multi_layer_compress_all_and_independence():
    B, Hq, Hkv, W, G, D, L = 2, 8, 2, 32, 32, 128, 3
    cache = LogQuantCache(L, B, Hq, Hkv, W, G, max_tokens=8 * W, auto_compress=False)
    ocs = [oracle.OracleCache(B, Hq, Hkv, D, W, G) for _ in range(L)]
    lens = [3 * W, 3 * W, 40]
    for l in range(L):
        k, v = synth.keys_values(30, B, Hkv, lens[l], D, "cuda", layer=l)
        cache.append(l, k, v)
        ocs[l].append(synth.bf16_bits(k), synth.bf16_bits(v))
    cache.compress(-1)  # layers 0 and 1 overflow in one launch; layer 2 is skipped
    for l in range(L):
        k, v = synth.keys_values(31, B, Hkv, 1, D, "cuda", layer=l)
        cache.append(l, k, v)
        ocs[l].append(synth.bf16_bits(k), synth.bf16_bits(v))
        assert_images_equal(cache.export(l), ocs[l].export())
        q = synth.queries(30, B, Hq, D, 0, "cuda", layer=l)
        out = torch.empty(B, Hq, D, device="cuda")
        cache.decode_attn(l, q, out)
        ref = ocs[l].attention(synth.bf16_bits(q), 1 / np.sqrt(D))
        assert np.abs(out.cpu().numpy() - ref).max() <= attn_tolerance(ref)
    assert [cache.info(l).n_events for l in range(L)] == [1, 1, 0]


@pytest.mark.parametrize("W,G,n", [(32, 32, 3 * 32 + 1), (64, 32, 777), (128, 64, 2048 + 55)])
def test_prompt_ingestion_in_one_launch_equals_token_by_token(W, G, n):
    """A prompt appended to an empty layer goes through one kernel; the same tokens appended after a
    first single token go through the append / overflow kernels.  Both must leave the same image, the
    same physical stores (identical attention bits) and the oracle's image."""
    B, Hq, Hkv, D = 2, 8, 2, 128
    k, v = synth.keys_values(77, B, Hkv, n, D, "cuda", outliers=synth.outlier_channels(77, Hkv, D, 3))
    one = LogQuantCache(2, B, Hq, Hkv, W, G, max_tokens=n + 2 * W + 8)
    seq = LogQuantCache(1, B, Hq, Hkv, W, G, max_tokens=n + 2 * W + 8)
    before = one.info(1).n_kernel_launches
    one.append(1, k, v)
    assert one.info(1).n_kernel_launches == before + 1
    seq.append(0, k[:, :, :1].contiguous(), v[:, :, :1].contiguous())
    for t0 in range(1, n, 31):   # fewer than W tokens per call: the append and overflow kernels
        seq.append(0, k[:, :, t0:t0 + 31].contiguous(), v[:, :, t0:t0 + 31].contiguous())
    assert seq.info(0).n_kernel_launches > 2
    oc = oracle.OracleCache(B, Hq, Hkv, D, W, G)
    oc.append(synth.bf16_bits(k), synth.bf16_bits(v))
    a, b = one.export(1), seq.export(0)
    assert_images_equal(a, b)
    assert_images_equal(a, oc.export())
    i1, i2 = one.info(1), seq.info(0)
    assert (i1.n_seen, i1.n_fp, i1.n_quant, i1.n_events) == (i2.n_seen, i2.n_fp, i2.n_quant, i2.n_events)
    q = synth.queries(77, B, Hq, D, 0, "cuda")
    o1, o2 = torch.empty(B, Hq, D, device="cuda"), torch.empty(B, Hq, D, device="cuda")
    one.decode_attn(1, q, o1)
    seq.decode_attn(0, q, o2)
    torch.cuda.synchronize()
    # (same stores, same partition; the partials of a pair are summed in arrival order, hence not bit for bit)
    assert torch.allclose(o1, o2, rtol=0, atol=2e-6 * float(o2.abs().max()) + 1e-7)
    # the next overflow step removes the same tokens in both
    k2, v2 = synth.keys_values(78, B, Hkv, 2 * W, D, "cuda")
    one.append(1, k2, v2)
    seq.append(0, k2, v2)
    assert_images_equal(one.export(1), seq.export(0))
    assert one.kernel_status() == 0 and seq.kernel_status() == 0
    one.close(); seq.close(); oc.close()


@pytest.mark.parametrize("W,G,bits,recent,chunks", [
    (32, 32, 2, False, [1, 32, 100, 33, 64, 250, 32]),          # first call leaves 1 token: every later slot is new
    (32, 32, 2, False, [95, 97, 1, 1, 40, 500]),                # store almost full, then chunks and single tokens
    (64, 32, 2, False, [130, 64, 700, 65, 191]),                # two key groups per step; old rows above 2W move down
    (64, 64, 4, False, [3 * 64, 64, 3 * 64 + 7, 128]),          # full store first, 4-bit codes
    (128, 64, 2, False, [300, 1000, 129, 2048]),
    (32, 32, 2, True, [50, 60, 200, 32, 33]),                   # recent-window comparator
    (42, 64, 2, False, [100, 90, 300, 84, 1, 500]),             # W not a multiple of G: waiting tokens in the store
    (48, 32, 4, False, [140, 96, 97, 400]),                     # the same with 4-bit codes
    (21, 32, 2, True, [60, 42, 43, 200]),                       # W < G, recent-window comparator
])
def test_chunks_appended_to_a_layer_in_use_take_one_launch_each(W, G, bits, recent, chunks):
    """Chunked prefill: a chunk of at least 2 W tokens that makes a layer in use overflow goes through ONE launch,
    which gathers key groups from the old full-precision rows and from the chunk, lets rows take over the slots
    that lose their token, and writes the rest of the chunk.  After every chunk the image must be the oracle's bit
    for bit and attention must agree; single decode steps afterwards (overflow kernel, fused append) must find the
    store as they expect it."""
    B, Hq, Hkv, D = 2, 8, 2, 128
    total = sum(chunks) + 2 * W + 3
    k, v = synth.keys_values(91, B, Hkv, total, D, "cuda", outliers=synth.outlier_channels(91, Hkv, D, 3))
    cache = LogQuantCache(1, B, Hq, Hkv, W, G, max_tokens=total + 8, bits=bits, filter=1 if recent else 0)
    oc = oracle.OracleCache(B, Hq, Hkv, D, W, G, bits=bits, recent_only=recent)
    done = 0

    def check(step):
        inf = cache.info(0)
        assert (inf.n_seen, inf.n_fp, inf.n_quant, inf.n_events) == (oc.n_seen, oc.n_fp, oc.n_quant, oc.n_events)
        assert_images_equal(cache.export(0), oc.export())
        q = synth.queries(91, B, Hq, D, step, "cuda")
        out = torch.empty(B, Hq, D, device="cuda")
        cache.decode_attn(0, q, out)
        ref = oc.attention(synth.bf16_bits(q), 1 / np.sqrt(D))
        assert np.abs(out.cpu().numpy() - ref).max() <= attn_tolerance(ref)

    for i, n in enumerate(chunks):
        before = cache.info(0).n_kernel_launches
        in_use, kept = done > 0, cache.info(0).n_fp
        cache.append(0, k[:, :, done:done + n].contiguous(), v[:, :, done:done + n].contiguous())
        if in_use and n >= 2 * W and kept + n > 3 * W:
            assert cache.info(0).n_kernel_launches == before + 1, (i, n)
        oc.append(synth.bf16_bits(k[:, :, done:done + n]), synth.bf16_bits(v[:, :, done:done + n]))
        done += n
        check(i)
    for t in range(2 * W + 3):   # token by token across the next overflow steps
        kn, vn = k[:, :, done:done + 1].contiguous(), v[:, :, done:done + 1].contiguous()
        q = synth.queries(91, B, Hq, D, 100 + t, "cuda")
        out = torch.empty(B, Hq, D, device="cuda")
        cache.append_decode_attn(0, kn, vn, q, out)
        oc.append(synth.bf16_bits(kn), synth.bf16_bits(vn))
        done += 1
        if t % 16 == 0 or t == 2 * W + 2:
            ref = oc.attention(synth.bf16_bits(q), 1 / np.sqrt(D))
            assert np.abs(out.cpu().numpy() - ref).max() <= attn_tolerance(ref)
            assert_images_equal(cache.export(0), oc.export())
    assert cache.kernel_status() == 0
    cache.close(); oc.close()


@pytest.mark.parametrize("B,Hq,Hkv,W,G,bits,n0,pad", [
    (2, 8, 2, 32, 32, 2, 3 * 32 - 5, None),     # crosses an overflow step (falls back to the two calls there)
    (1, 14, 2, 64, 64, 2, 64 * 5 + 15, None),   # GQA-7; the new row opens a new 16-slot tile on the way
    (2, 8, 8, 32, 32, 4, 32 * 7 + 1, None),     # r = 1, 4-bit codes
    (2, 8, 2, 42, 64, 2, 42 * 5 + 11, None),    # W not a multiple of G: waiting tokens in the fp store
    (3, 8, 2, 32, 32, 2, 32 * 6 + 20, [150, 0, 33]),   # left-padded batch
    (2, 14, 2, 64, 64, 2, 64 * 4 + 60, [7, 200]),      # left-padded, GQA-7, crosses an overflow step
])
def test_append_and_attention_in_one_launch(B, Hq, Hkv, W, G, bits, n0, pad):
    """lq_append_decode_attn: same image, same attention bits as lq_append + lq_decode_attn, one launch."""
    D, n_steps = 128, 20
    k, v = synth.keys_values(23, B, Hkv, n0 + n_steps, D, "cuda")
    fused = LogQuantCache(1, B, Hq, Hkv, W, G, max_tokens=n0 + n_steps + 8, bits=bits)
    plain = LogQuantCache(1, B, Hq, Hkv, W, G, max_tokens=n0 + n_steps + 8, bits=bits)
    oc = oracle.OracleCache(B, Hq, Hkv, D, W, G, bits=bits)
    for c in (fused, plain):
        c.append(0, k[:, :, :n0].contiguous(), v[:, :, :n0].contiguous())
        if pad is not None:
            c.set_padding(pad)
    oc.append(synth.bf16_bits(k[:, :, :n0]), synth.bf16_bits(v[:, :, :n0]))
    single = 0
    for t in range(n_steps):
        k1, v1 = k[:, :, n0 + t:n0 + t + 1].contiguous(), v[:, :, n0 + t:n0 + t + 1].contiguous()
        q = synth.queries(23, B, Hq, D, t, "cuda")
        o1 = torch.full((B, Hq, D), float("nan"), device="cuda")
        o2 = torch.full((B, Hq, D), float("nan"), device="cuda")
        before = fused.info(0).n_kernel_launches
        fused.append_decode_attn(0, k1, v1, q, o1)
        single += fused.info(0).n_kernel_launches == before + 1
        plain.append(0, k1, v1)
        plain.decode_attn(0, q, o2)
        torch.cuda.synchronize()
        assert torch.allclose(o1, o2, rtol=0, atol=2e-6 * float(o2.abs().max()) + 1e-7), f"step {t}"  # arrival order
        oc.append(synth.bf16_bits(k1), synth.bf16_bits(v1))
        ref = oc.attention_subset(synth.bf16_bits(q), 1 / np.sqrt(D), pad=pad)
        assert np.abs(o1.cpu().numpy() - ref).max() <= attn_tolerance(ref)
        if t % 6 == 0 or t == n_steps - 1:
            assert_images_equal(fused.export(0), oc.export())
    assert single >= n_steps - 1  # every step but the one that had to run the overflow step in between
    # (caches above 192 MB per launch take the two calls as well; the full-size tests cover those sizes)
    assert fused.kernel_status() == 0
    fused.close(); plain.close(); oc.close()


@pytest.mark.parametrize("pinned", [True, False])
def test_decode_step_with_host_buffers(pinned):
    """Page-locked buffers are read and written by the kernels in place; pageable ones are copied."""
    B, Hq, Hkv, W, G, D = 2, 8, 2, 32, 32, 128
    N = 3 * W  # the first host step has to run the overflow itself, even with auto_compress = 0
    cache = LogQuantCache(1, B, Hq, Hkv, W, G, max_tokens=N + 8, auto_compress=False)
    oc = oracle.OracleCache(B, Hq, Hkv, D, W, G)
    k, v = synth.keys_values(40, B, Hkv, N, D, "cuda", token_total=N + 4)
    cache.append(0, k, v)
    oc.append(synth.bf16_bits(k), synth.bf16_bits(v))
    for step in range(3):
        k1, v1 = synth.keys_values(40, B, Hkv, 1, D, "cpu", token_start=N + step, token_total=N + 4)
        q = synth.queries(40, B, Hq, D, step, "cpu")
        out = torch.full((B, Hq, D), float("nan"), dtype=torch.float32)
        if pinned:
            k1, v1, q, out = k1.pin_memory(), v1.pin_memory(), q.pin_memory(), out.pin_memory()
        cache.decode_step_host(0, k1, v1, q, out)
        oc.append(synth.bf16_bits(k1), synth.bf16_bits(v1))
        ref = oc.attention(synth.bf16_bits(q), 1 / np.sqrt(D))
        assert np.abs(out.numpy() - ref).max() <= attn_tolerance(ref)
    assert_images_equal(cache.export(0), oc.export())


def test_argument_errors_on_device():
    cache = LogQuantCache(1, 1, 4, 2, 32, 32, max_tokens=64)
    q = torch.zeros(1, 4, 128, dtype=torch.bfloat16, device="cuda")
    out = torch.zeros(1, 4, 128, device="cuda")
    with pytest.raises(LogQuantError) as e:
        cache.decode_attn(0, q, out)  # empty cache
    assert e.value.status == binding.LQ_ERR_INVALID_ARG
    with pytest.raises(LogQuantError) as e:
        cache.decode_attn(3, q, out)
    assert e.value.status == binding.LQ_ERR_INVALID_ARG
    k = torch.zeros(1, 2, 65, 128, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(LogQuantError) as e:
        cache.append(0, k, k)
    assert e.value.status == binding.LQ_ERR_CAPACITY
    assert cache.info(0).n_seen == 0
    # the one-launch step: capacity and window errors leave the cache as it was
    k1 = torch.zeros(1, 2, 1, 128, dtype=torch.bfloat16, device="cuda")
    cache.append(0, k[:, :, :64].contiguous(), k[:, :, :64].contiguous())
    with pytest.raises(LogQuantError) as e:
        cache.append_decode_attn(0, k1, k1, q, out)
    assert e.value.status == binding.LQ_ERR_CAPACITY and cache.info(0).n_seen == 64
    with pytest.raises(LogQuantError) as e:
        cache.append_decode_attn(1, k1, k1, q, out)
    assert e.value.status == binding.LQ_ERR_INVALID_ARG
    manual = LogQuantCache(1, 1, 4, 2, 32, 32, max_tokens=256, auto_compress=False)
    manual.append(0, k[:, :, :64].contiguous(), k[:, :, :64].contiguous())
    manual.append(0, k[:, :, :32].contiguous(), k[:, :, :32].contiguous())
    with pytest.raises(LogQuantError) as e:
        manual.append_decode_attn(0, k1, k1, q, out)  # window full and the caller drives the overflow step
    assert e.value.status == binding.LQ_ERR_WINDOW_FULL and manual.info(0).n_seen == 96
    manual.compress(0)
    manual.append_decode_attn(0, k1, k1, q, out)
    assert manual.info(0).n_seen == 97 and torch.isfinite(out).all()
    manual.close()


# ---- left padding of a ragged batch, and attention over the full-precision store only ----------------
@pytest.mark.parametrize("kernel", KERNELS)
@pytest.mark.parametrize("B,Hq,Hkv,W,G,bits,n_prefill,n_steps,chunk,pad", [
    (3, 8, 2, 32, 32, 2, 500, 40, None, [0, 37, 300]),      # none / inside the first groups / whole leading groups
    (2, 14, 2, 64, 64, 2, 64 * 9 + 3, 70, 200, [129, 5]),   # GQA-7 (two column blocks), G = 64: two mask words
    (2, 8, 8, 32, 32, 4, 32 * 8 + 17, 20, None, [64, 201]), # r = 1, 4-bit codes
    (2, 8, 2, 42, 64, 2, 42 * 9 + 5, 50, None, [11, 260]),  # W not a multiple of G: waiting tokens may be padding
    (1, 4, 1, 32, 32, 2, 40, 70, None, [39]),               # padding still in the window; crosses the first overflow
    (80, 8, 8, 32, 32, 2, 150, 3, None, [(7 * i) % 120 for i in range(80)]),  # more (b, kv) pairs than one wave of CTAs
    (2, 8, 1, 32, 32, 2, 3000, 3, None, [0, 2900]),         # very unequal work: the CTAs go where the tokens are
])
def test_left_padded_batch(kernel, B, Hq, Hkv, W, G, bits, n_prefill, n_steps, chunk, pad):
    """Sequence b attends to tokens pad[b].. only; the stores are those of the unpadded run (same image)."""
    worst = run_case(B, Hq, Hkv, W, G, n_prefill, n_steps, 31, kernel, bits=bits, prefill_chunk=chunk, pad=pad,
                     check_image_every=9)
    assert worst <= 1.0


@pytest.mark.parametrize("kernel", KERNELS)
@pytest.mark.parametrize("B,Hq,Hkv,W,G,n_prefill,pad", [
    (2, 8, 2, 32, 32, 700, None), (2, 14, 2, 64, 64, 1000, None), (2, 8, 2, 32, 32, 700, [90, 0])])
def test_attention_over_the_full_precision_store_only(kernel, B, Hq, Hkv, W, G, n_prefill, pad):
    worst = run_case(B, Hq, Hkv, W, G, n_prefill, 12, 32, kernel, fp_only=True, pad=pad, check_image_every=0)
    assert worst <= 1.0


def test_padding_can_change_and_bad_padding_is_refused():
    B, Hq, Hkv, W, G, D, N = 2, 8, 2, 32, 32, 128, 400
    cache = LogQuantCache(1, B, Hq, Hkv, W, G, max_tokens=N + 16)
    oc = oracle.OracleCache(B, Hq, Hkv, D, W, G)
    k, v = synth.keys_values(33, B, Hkv, N, D, "cuda")
    cache.append(0, k, v)
    oc.append(synth.bf16_bits(k), synth.bf16_bits(v))
    q = synth.queries(33, B, Hq, D, 0, "cuda")
    out = torch.empty(B, Hq, D, device="cuda")

    def check(pad):
        cache.decode_attn(0, q, out)
        torch.cuda.synchronize()
        ref = oc.attention_subset(synth.bf16_bits(q), 1 / np.sqrt(D), pad=pad)
        assert np.abs(out.cpu().numpy() - ref).max() <= attn_tolerance(ref)
        return out.clone()

    plain = check(None)
    cache.set_padding([100, 0])
    padded = check([100, 0])
    # (sequence 1 is untouched up to summation order: the padded launch shares its CTAs out differently)
    assert not torch.allclose(padded[0], plain[0], atol=1e-3) and torch.allclose(padded[1], plain[1], atol=1e-3)
    cache.set_padding([0, 399])  # sequence 1 keeps its newest token only: the output is that token's value row
    one = check([0, 399])
    assert torch.allclose(one[1, 0], v[1, 0, 399].float(), atol=1e-5)
    cache.set_padding(None)
    assert torch.allclose(check(None), plain, rtol=0, atol=2e-6 * float(plain.abs().max()) + 1e-7)
    # the one-launch step on a padded batch
    cache.set_padding([7, 150])
    k1, v1 = synth.keys_values(34, B, Hkv, 1, D, "cuda")
    cache.append_decode_attn(0, k1, v1, q, out)
    torch.cuda.synchronize()
    oc.append(synth.bf16_bits(k1), synth.bf16_bits(v1))
    ref = oc.attention_subset(synth.bf16_bits(q), 1 / np.sqrt(D), pad=[7, 150])
    assert np.abs(out.cpu().numpy() - ref).max() <= attn_tolerance(ref)
    # refused: negative, or a sequence with nothing left
    with pytest.raises(LogQuantError) as e:
        cache.set_padding([-1, 0])
    assert e.value.status == binding.LQ_ERR_INVALID_ARG
    cache.set_padding([N + 1, 0])
    with pytest.raises(LogQuantError) as e:
        cache.decode_attn(0, q, out)
    assert e.value.status == binding.LQ_ERR_INVALID_ARG
    cache.set_padding([N, 0])  # N + 1 tokens appended: the newest one is left
    check([N, 0])
    assert cache.kernel_status() == 0
    cache.close(); oc.close()


@pytest.mark.parametrize("Hq,Hkv,G,W", [(8, 2, 32, 32), (14, 2, 64, 64), (12, 2, 32, 32)])
def test_large_value_magnitudes(Hq, Hkv, G, W):
    """Values of magnitude ~2000 (value scales of several hundred, far above what p * s_v would bear in fp16
    without the 2^-8 on the probabilities of the path for more than 4 query heads per KV head)."""
    B, D, N = 2, 128, W * 9 + 7
    k, v = synth.keys_values(51, B, Hkv, N, D, "cuda")
    v = (v.float() * 600.0).to(torch.bfloat16)
    cache = LogQuantCache(1, B, Hq, Hkv, W, G, max_tokens=N + 8)
    oc = oracle.OracleCache(B, Hq, Hkv, D, W, G)
    cache.append(0, k, v)
    oc.append(synth.bf16_bits(k), synth.bf16_bits(v))
    assert_images_equal(cache.export(0), oc.export())
    assert float(torch.from_numpy(oc.export()["v_scale"].astype(np.int32)).max()) > 0  # quantised tokens exist
    for step in range(3):
        q = synth.queries(51, B, Hq, D, step, "cuda")
        out = torch.full((B, Hq, D), float("nan"), device="cuda")
        cache.decode_attn(0, q, out)
        torch.cuda.synchronize()
        ref = oc.attention(synth.bf16_bits(q), 1 / np.sqrt(D))
        got = out.cpu().numpy().astype(np.float64)
        assert np.isfinite(got).all()
        assert np.abs(got - ref).max() <= attn_tolerance(ref)
    assert cache.kernel_status() == 0
    cache.close(); oc.close()


@pytest.mark.parametrize("k0_gain,pad0", [(0.0, 0), (-24.0, 0), (24.0, 0), (24.0, 1), (-40.0, 1)])
def test_partials_summed_on_arrival_and_the_record_fallback(k0_gain, pad0):
    """More than 12 CTAs per (b, kv) pair: the partials are added, scaled to the score of the token in slot 0, to
    one sum per pair.  A slot-0 score far below or above everything else (also as padding) drives the scale out
    of range, and the pair is merged from the records instead; either way the oracle's result comes out."""
    B, Hq, Hkv, W, G, D, N = 1, 4, 1, 32, 32, 128, 4600
    u = synth.unit_vectors(61, Hkv, D)
    k, v = synth.keys_values(61, B, Hkv, N, D, "cuda")
    k[:, :, 0] = (k[:, :, 0].float() + k0_gain * u.to("cuda")[None]).to(torch.bfloat16)
    cache = LogQuantCache(1, B, Hq, Hkv, W, G, max_tokens=N + 8, n_splits=16)
    oc = oracle.OracleCache(B, Hq, Hkv, D, W, G)
    cache.append(0, k, v)
    oc.append(synth.bf16_bits(k), synth.bf16_bits(v))
    assert cache.info(0).n_splits == 16
    pad = [pad0] if pad0 else None
    if pad:
        cache.set_padding(pad)
    for step in range(3):
        q = (synth.queries(61, B, Hq, D, step, "cuda").float() + 24.0 * u.to("cuda")[None]).to(torch.bfloat16)
        out = torch.full((B, Hq, D), float("nan"), device="cuda")
        cache.decode_attn(0, q, out)
        torch.cuda.synchronize()
        ref = oc.attention_subset(synth.bf16_bits(q), 1 / np.sqrt(D), pad=pad)
        got = out.cpu().numpy().astype(np.float64)
        assert np.isfinite(got).all()
        assert np.abs(got - ref).max() <= attn_tolerance(ref), (step, k0_gain, pad0)
    assert cache.kernel_status() == 0
    cache.close(); oc.close()


def test_caller_supplied_device_allocator():
    """Every device block of a cache can come from the caller (here torch's caching allocator); a failing
    allocator gives LQ_ERR_OOM and hands back what it had handed out."""
    B, Hq, Hkv, W, G, D, N = 2, 8, 2, 32, 32, 128, 300
    cache = LogQuantCache(2, B, Hq, Hkv, W, G, max_tokens=N + 8, allocator="torch")
    blocks = cache._blocks  # address -> tensor, filled and emptied by the hooks
    assert sum(t.numel() for t in blocks.values()) >= cache.info(0).bytes_device > 0
    n_blocks = len(blocks)
    oc = oracle.OracleCache(B, Hq, Hkv, D, W, G)
    k, v = synth.keys_values(71, B, Hkv, N, D, "cuda")
    cache.append(1, k, v)
    oc.append(synth.bf16_bits(k), synth.bf16_bits(v))
    assert_images_equal(cache.export(1), oc.export())
    q = synth.queries(71, B, Hq, D, 0, "cuda")
    out = torch.empty(B, Hq, D, device="cuda")
    cache.set_padding([10, 0])  # the masks are allocated through the same hook
    assert len(blocks) == n_blocks + 1
    cache.decode_attn(1, q, out)
    torch.cuda.synchronize()
    ref = oc.attention_subset(synth.bf16_bits(q), 1 / np.sqrt(D), pad=[10, 0])
    assert np.abs(out.cpu().numpy() - ref).max() <= attn_tolerance(ref)
    cache.close()
    assert not blocks  # every block went back through dev_free

    live, calls = {}, [0]

    def alloc(nbytes):
        calls[0] += 1
        if calls[0] > 3:
            return 0  # out of memory on the fourth block
        t = torch.empty(nbytes, dtype=torch.uint8, device="cuda")
        live[t.data_ptr()] = t
        return t.data_ptr()

    with pytest.raises(LogQuantError) as e:
        LogQuantCache(1, B, Hq, Hkv, W, G, max_tokens=N, allocator=(alloc, lambda ptr: live.pop(ptr)))
    assert e.value.status == binding.LQ_ERR_OOM and not live


def _random_padded_cases(n, seed):
    rng = np.random.default_rng(seed)
    cases = []
    for B, Hq, Hkv, W, G, bits, n_prefill, chunk, recent in _random_cases(n, seed):
        B = max(B, 2)
        pad = [int(rng.integers(0, n_prefill + 1)) if rng.random() < 0.75 else 0 for _ in range(B)]
        kernel = LQ_KERNEL_MMA if rng.random() < 0.75 else LQ_KERNEL_SCALAR
        cases.append((B, Hq, Hkv, W, G, bits, n_prefill, chunk, recent, pad, kernel, bool(rng.random() < 0.7)))
    return cases


@pytest.mark.parametrize("B,Hq,Hkv,W,G,bits,n_prefill,chunk,recent,pad,kernel,auto", _random_padded_cases(10, 4242))
def test_seeded_random_padded_configurations(B, Hq, Hkv, W, G, bits, n_prefill, chunk, recent, pad, kernel, auto):
    """A seeded draw like the one above with left padding, both kernels and caller-driven overflow steps."""
    worst = run_case(B, Hq, Hkv, W, G, n_prefill, 3, seed=200 + n_prefill, kernel=kernel, bits=bits, prefill_chunk=chunk,
                     recent_only=recent, pad=pad, auto_compress=auto, check_image_every=1)
    assert worst <= 1.0


def _overlap_ref(oc, q, D, pad):
    if pad is None:
        return oc.attention(synth.bf16_bits(q), 1 / np.sqrt(D))
    return oc.attention_subset(synth.bf16_bits(q), 1 / np.sqrt(D), pad=pad)


@pytest.mark.parametrize("L,fused,r,pad", [(4, True, 4, None), (4, False, 4, None), (2, True, 7, None), (3, False, 1, None),
                                           (4, True, 4, [0, 333]), (3, False, 7, [650, 17])])
def test_overlapped_decode_launches_of_different_layers(L, fused, r, pad):
    """LQ_FLAG_OVERLAP_DECODE: back-to-back decode launches of different layers start streaming before the launch
    in front of them has finished (and wait for it only before the shared workspace); every layer's output and
    image must still be the oracle's, step after step, also when a layer is visited twice in a row and when
    appends and an overflow step fall between the launches."""
    from paper_2503_19950_b200 import LQ_FLAG_OVERLAP_DECODE
    B, Hkv, W, G, D, n0, n_steps = 2, 2, 64, 32, 128, 64 * 10 + 50, 20
    Hq = Hkv * r
    cache = LogQuantCache(L, B, Hq, Hkv, W, G, max_tokens=n0 + n_steps + 8, kernel=LQ_KERNEL_MMA,
                          flags=LQ_FLAG_OVERLAP_DECODE)
    if pad is not None:   # a left-padded batch: the padded kernel variant and its own third-of-a-wave plan
        cache.set_padding(pad)
    ocs = [oracle.OracleCache(B, Hq, Hkv, D, W, G) for _ in range(L)]
    ks, vs = [], []
    for l in range(L):
        k, v = synth.keys_values(300 + l, B, Hkv, n0 + n_steps, D, "cuda", outliers=synth.outlier_channels(300 + l, Hkv, D, 3))
        ks.append(k); vs.append(v)
        cache.append(l, k[:, :, :n0].contiguous(), v[:, :, :n0].contiguous())
        ocs[l].append(synth.bf16_bits(k[:, :, :n0]), synth.bf16_bits(v[:, :, :n0]))
    outs = [torch.empty(B, Hq, D, device="cuda") for _ in range(L)]
    twice = torch.empty(B, Hq, D, device="cuda")
    for step in range(n_steps):   # the 14th step overflows the window of every layer
        t = n0 + step
        qs = [synth.queries(300 + l, B, Hq, D, step, "cuda") for l in range(L)]
        for l in range(L):        # all launches of a step are enqueued before anything is checked
            kt, vt = ks[l][:, :, t:t + 1].contiguous(), vs[l][:, :, t:t + 1].contiguous()
            if fused:
                cache.append_decode_attn(l, kt, vt, qs[l], outs[l])
            else:
                cache.append(l, kt, vt)
                cache.decode_attn(l, qs[l], outs[l])
                if l == L - 1:
                    cache.decode_attn(l, qs[l], twice)   # the same layer twice in a row
            ocs[l].append(synth.bf16_bits(kt), synth.bf16_bits(vt))
        if not fused:             # attention only, layer after layer: every launch but the first overlaps
            for l in range(L):
                cache.decode_attn(l, qs[l], outs[l])
        torch.cuda.synchronize()
        for l in range(L):
            ref = _overlap_ref(ocs[l], qs[l], D, pad)
            assert np.abs(outs[l].cpu().numpy() - ref).max() <= attn_tolerance(ref), (step, l)
        if not fused:   # (a launch that overlaps shares its pair's work out differently: equal up to summation order)
            ref = _overlap_ref(ocs[L - 1], qs[L - 1], D, pad)
            assert np.abs(twice.cpu().numpy() - ref).max() <= attn_tolerance(ref), step
    for l in range(L):
        assert_images_equal(cache.export(l), ocs[l].export())
    assert cache.kernel_status() == 0
    cache.close()


@pytest.mark.parametrize("W,G,bits", [(32, 32, 2), (64, 64, 2), (32, 32, 4), (64, 64, 4)])
def test_codes_at_the_rounding_boundaries(W, G, bits):
    """Groups whose quotients (x - min) / scale sit exactly on k + 1/2 (ties) and one bf16 step beside it, at
    exponents from the bf16 subnormal range up: the codes must be the oracle's, bit for bit.  Every group draws from
    {0 .. 2 top} * 2^e and the bf16 neighbours of the odd members, so that scale = 2 * 2^e whenever 0 and
    2 top are both drawn, and other nearby scales otherwise."""
    B, Hq, Hkv, D = 2, 4, 2, 128
    N = 5 * W + 1
    top = (1 << bits) - 1
    rng = np.random.default_rng(1234 + W + bits)
    base = np.arange(0, 2 * top + 1, dtype=np.float64)
    odd = base[1::2]
    ulp = 2.0 ** (np.floor(np.log2(odd)) - 7)            # bf16 spacing at the odd members
    cand = np.concatenate([base, odd + ulp, odd - ulp / np.where(odd == 2.0 ** np.floor(np.log2(odd)), 2, 1)])
    exps = np.array([-130.0, -40.0, -3.0, 0.0, 3.0])

    def draw(shape_groups, axis_len, axis):
        e = rng.choice(exps, size=shape_groups)
        idx = rng.integers(0, len(cand), size=shape_groups[:axis] + (axis_len,) + shape_groups[axis:])
        # bf16 subnormals (multiples of 2^-133) hold the integer members only
        idx = np.where(np.expand_dims(e, axis) < -126, idx % len(base), idx)
        vals = cand[idx] * np.expand_dims(2.0 ** e, axis)
        sign = rng.choice([1.0, -1.0], size=shape_groups)   # mirrored groups: the minimum is the negative end
        return (vals * np.expand_dims(sign, axis)).astype(np.float32)

    k = draw((B, Hkv, D), N, 2)                               # one exponent per channel: key groups run over tokens
    v = draw((B, Hkv, N, D // G), G, 4).reshape(B, Hkv, N, D)  # one exponent per (token, channel group)
    kt = torch.from_numpy(k).to(torch.bfloat16).cuda()
    vt = torch.from_numpy(v).to(torch.bfloat16).cuda()
    assert (kt.float().cpu().numpy() == k).all() and (vt.float().cpu().numpy() == v).all()  # representable
    for chunk in (N, 1):                                       # one ingestion launch, then token by token
        cache = LogQuantCache(1, B, Hq, Hkv, W, G, max_tokens=N + 4, bits=bits)
        oc = oracle.OracleCache(B, Hq, Hkv, D, W, G, bits=bits)
        for s in range(0, N, chunk):
            cache.append(0, kt[:, :, s:s + chunk].contiguous(), vt[:, :, s:s + chunk].contiguous())
        oc.append(synth.bf16_bits(kt), synth.bf16_bits(vt))
        want = oc.export()
        assert_images_equal(cache.export(0), want)
        for key in ("k_codes", "v_codes"):                      # every code value occurs (packed low bits first)
            seen = set()
            for sh in range(0, 8, bits):
                seen |= set(np.unique((want[key] >> sh) & top).tolist())
            assert seen == set(range(top + 1)), key
        assert cache.kernel_status() == 0
        cache.close()
        oc.close()


def test_chunks_at_the_largest_window_with_padding_and_stacked_layers():
    """Chunk ingestion at W = 512 (the largest window), G = 64, on a left-padded batch, on two layers of one cache
    in turn with overlapped decode launches in between: images bit-exact, attention (which leaves the padding out)
    within tolerance."""
    from paper_2503_19950_b200 import LQ_FLAG_OVERLAP_DECODE
    B, Hq, Hkv, D, W, G, L = 2, 8, 2, 128, 512, 64, 2
    pad = [700, 0]
    chunks = [900, 1024, 2 * W, 1500]
    total = sum(chunks)
    cache = LogQuantCache(L, B, Hq, Hkv, W, G, max_tokens=total + 8, flags=LQ_FLAG_OVERLAP_DECODE)
    cache.set_padding(pad)
    ocs = [oracle.OracleCache(B, Hq, Hkv, D, W, G) for _ in range(L)]
    done = 0
    for i, n in enumerate(chunks):
        outs = []
        for l in range(L):
            k, v = synth.keys_values(5, B, Hkv, n, D, "cuda", token_start=done, token_total=total, layer=l)
            cache.append(l, k, v)
            ocs[l].append(synth.bf16_bits(k), synth.bf16_bits(v))
        qs = [synth.queries(5, B, Hq, D, i, "cuda", layer=l) for l in range(L)]
        for l in range(L):   # back to back: the second launch overlaps the first
            outs.append(torch.empty(B, Hq, D, device="cuda"))
            cache.decode_attn(l, qs[l], outs[l])
        done += n
        for l in range(L):
            assert_images_equal(cache.export(l), ocs[l].export())
            ref = ocs[l].attention_subset(synth.bf16_bits(qs[l]), 1 / np.sqrt(D), pad=pad)
            assert np.abs(outs[l].cpu().numpy() - ref).max() <= attn_tolerance(ref), (i, l)
    assert cache.kernel_status() == 0
    cache.close()
    for oc in ocs:
        oc.close()


@pytest.mark.parametrize("L,expect_all", [(16, True), (3, False)])
def test_fused_steps_of_many_layers_overlap_without_a_wait_per_step(L, expect_all):
    """Steps of fused append+attention launches over the layers of one cache, back to back on one stream with
    LQ_FLAG_OVERLAP_DECODE.  The launch of layer l in step t+1 reads the row that the launch of layer l in step t
    wrote; it may overlap its predecessor only if that earlier launch is known to be complete, which the library
    derives from the CTAs launched in between (16 layers: enough, every launch after the first overlaps; 3 layers:
    not enough, the first launch of a step waits).  Outputs of every layer and step against the oracle, images at
    the end."""
    from paper_2503_19950_b200 import LQ_FLAG_OVERLAP_DECODE
    B, Hq, Hkv, D, W, G = 8, 32, 8, 128, 32, 32
    n0, steps = 128 * W + 5, 6
    cache = LogQuantCache(L, B, Hq, Hkv, W, G, max_tokens=n0 + steps + 8, flags=LQ_FLAG_OVERLAP_DECODE)
    ocs = [oracle.OracleCache(B, Hq, Hkv, D, W, G) for _ in range(L)]
    for l in range(L):
        k, v = synth.keys_values(61, B, Hkv, n0, D, "cuda", layer=l)
        cache.append(l, k, v)
        ocs[l].append(synth.bf16_bits(k), synth.bf16_bits(v))
    ins = [[(synth.keys_values(62 + t, B, Hkv, 1, D, "cuda", layer=l), synth.queries(62 + t, B, Hq, D, t, "cuda", layer=l))
            for l in range(L)] for t in range(steps)]
    outs = [[torch.empty(B, Hq, D, device="cuda") for _ in range(L)] for _ in range(steps)]
    torch.cuda.synchronize()
    before = cache.info(0).n_launches_overlapped
    for t in range(steps):          # nothing between the launches: this is the pattern bench.py times
        for l in range(L):
            (kn, vn), q = ins[t][l]
            cache.append_decode_attn(l, kn, vn, q, outs[t][l])
    torch.cuda.synchronize()
    inf = cache.info(0)
    overlapped = inf.n_launches_overlapped - before
    # CTAs of the L - 1 launches between two launches of a layer, against twice what the device can hold (4 per SM)
    grid = B * Hkv + inf.n_ctas_overlapped
    enough = (L - 1) * grid >= 2 * 4 * torch.cuda.get_device_properties(0).multi_processor_count
    assert enough == expect_all, (grid, L)
    assert overlapped == (steps * L - 1 if expect_all else steps * (L - 1))
    for t in range(steps):
        for l in range(L):
            (kn, vn), q = ins[t][l]
            ocs[l].append(synth.bf16_bits(kn), synth.bf16_bits(vn))
            if l % 5 == 0 or t == steps - 1:
                ref = ocs[l].attention(synth.bf16_bits(q), 1 / np.sqrt(D), n_threads=8)
                err = np.abs(outs[t][l].cpu().numpy() - ref).max()
                assert err <= attn_tolerance(ref), (t, l, err)
    for l in range(0, L, 5):
        assert_images_equal(cache.export(l), ocs[l].export())
    assert cache.kernel_status() == 0
    cache.close()
    for oc in ocs:
        oc.close()

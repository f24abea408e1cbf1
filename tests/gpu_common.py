"""Shared driver for the GPU parity tests: runs the CUDA library and the CPU oracle on the same
seeded inputs and compares them (bit-exact image, attention within the stated tolerance)."""
import numpy as np
import torch

import oracle
from paper_2503_19950_b200 import LogQuantCache, LogQuantError, synth
from paper_2503_19950_b200.binding import LQ_ERR_WINDOW_FULL

IMAGE_KEYS = ["kept_ids", "quant_ids", "k_codes", "v_codes", "k_scale", "k_zero", "v_scale", "v_zero", "fp_k", "fp_v"]


def attn_tolerance(ref: np.ndarray) -> float:
    """max |delta| <= 2e-3 * max|out_ref| + 1e-3 (fp32 result against the float64 oracle)."""
    return 2e-3 * float(np.abs(ref).max()) + 1e-3


def assert_images_equal(got: dict, want: dict):
    for key in IMAGE_KEYS:
        assert got[key].shape == want[key].shape, key
        if not np.array_equal(got[key], want[key]):
            bad = np.argwhere(got[key] != want[key])
            raise AssertionError(f"{key}: {len(bad)} mismatches, first at {bad[0].tolist()}: "
                                 f"got {got[key][tuple(bad[0])]} want {want[key][tuple(bad[0])]}")


def run_case(B, Hq, Hkv, W, G, n_prefill, n_steps, seed, kernel, n_outliers=3, check_image_every=1,
             sm_scale=0.0, n_splits=0, prefill_chunk=None, auto_compress=True, out_dtype=torch.float32,
             q_gain=1.0, bits=2, recent_only=False, pad=None, fp_only=False):
    """Prefill n_prefill tokens, then n_steps x (append 1 token, attention).  Returns max error ratio.
    pad: leading padding positions per sequence (set before the first token); fp_only: attention over the
    full-precision store only."""
    D = 128
    dev = "cuda"
    total = n_prefill + n_steps
    outl = synth.outlier_channels(seed, Hkv, D, n_outliers) if n_outliers else None
    cache = LogQuantCache(1, B, Hq, Hkv, W, G, max_tokens=total + 8, auto_compress=auto_compress, kernel=kernel,
                          n_splits=n_splits, bits=bits, filter=1 if recent_only else 0)
    oc = oracle.OracleCache(B, Hq, Hkv, D, W, G, bits=bits, recent_only=recent_only)
    if pad is not None:
        cache.set_padding(pad)

    def feed(start, n):
        k, v = synth.keys_values(seed, B, Hkv, n, D, dev, token_start=start, token_total=total, outliers=outl)
        if auto_compress:
            cache.append(0, k, v)
        else:
            for t in range(n):  # caller-driven overflow handling: append, and on "window full" compress and retry
                kt, vt = k[:, :, t:t + 1].contiguous(), v[:, :, t:t + 1].contiguous()
                try:
                    cache.append(0, kt, vt)
                except LogQuantError as err:
                    assert err.status == LQ_ERR_WINDOW_FULL
                    cache.compress(0)
                    cache.append(0, kt, vt)
        oc.append(synth.bf16_bits(k), synth.bf16_bits(v))

    done = 0
    chunk = prefill_chunk or max(n_prefill, 1)
    while done < n_prefill:
        n = min(chunk, n_prefill - done)
        feed(done, n)
        done += n
    worst = 0.0
    scale = sm_scale if sm_scale > 0 else 1.0 / np.sqrt(D)
    for step in range(n_steps):
        feed(n_prefill + step, 1)
        inf = cache.info(0)
        assert (inf.n_seen, inf.n_fp, inf.n_quant, inf.n_events) == (oc.n_seen, oc.n_fp, oc.n_quant, oc.n_events)
        if check_image_every and step % check_image_every == 0:
            assert_images_equal(cache.export(0), oc.export())
        q = (synth.queries(seed, B, Hq, D, step, dev).float() * q_gain).to(torch.bfloat16)
        out = torch.full((B, Hq, D), float("nan"), dtype=out_dtype, device=dev)
        if fp_only:
            cache.decode_attn_fp_only(0, q, out, sm_scale=sm_scale)
        else:
            cache.decode_attn(0, q, out, sm_scale=sm_scale)
        torch.cuda.synchronize()
        if fp_only or pad is not None:
            ref = oc.attention_subset(synth.bf16_bits(q), scale, fp_only=fp_only, pad=pad)
        else:
            ref = oc.attention(synth.bf16_bits(q), scale, n_threads=8)
        got = out.float().cpu().numpy().astype(np.float64)
        assert np.isfinite(got).all()
        tol = attn_tolerance(ref)
        if out_dtype == torch.bfloat16:
            tol += 2.0 ** -8 * float(np.abs(ref).max())
        err = float(np.abs(got - ref).max())
        assert err <= tol, f"step {step}: max|delta| {err:.3e} > tol {tol:.3e}"
        worst = max(worst, err / tol)
    assert cache.kernel_status() == 0
    cache.close()
    oc.close()
    return worst

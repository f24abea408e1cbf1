"""The allocation-free entry point lq_decode_attn_image_static.

Some callers of this library cannot allocate device memory (a server with a fixed start-up arena, code
under a foreign allocator policy, code called during stream capture), so they cannot use lq_cache_create.
They keep the cache as a canonical image in memory of their own and call this entry point, whose split-K
scratch is a fixed array inside the library.  The test feeds it the image exported from an ordinary cache
and checks, on two calls in a row (the second one finds the first one's leftovers in the shared scratch),
that the output agrees with lq_decode_attn on the same cache AND with the float64 CPU oracle fed the same
tokens, both within the tolerance of the parity tests.
Collected last on purpose: a run that stops at the first failure has run everything else before it."""
import numpy as np
import pytest
import torch

import oracle
from gpu_common import attn_tolerance
from paper_2503_19950_b200 import LogQuantCache, binding, build, decode_attn_image_static, synth

pytestmark = pytest.mark.gpu
D = 128


def _image_on_device(cache):
    img = cache.export(0)
    return {k: torch.from_numpy(v.view(np.int16) if v.dtype == np.uint16 else v).cuda()
            for k, v in img.items() if k not in ("kept_ids", "quant_ids")}


# (B, Hq, Hkv, W, G, n_tokens, bits): GQA 4, GQA 7 at G = 64, MHA below the first overflow, GQA 8, the paper's
# W = 42 with G = 64 (removed tokens that wait for a full key group sit among the bf16 rows), 4-bit codes, and
# B * Hq = 2048 heads with 2200 tokens, where the split count is clipped by the size of the scratch (4, not 5)
CASES = [(2, 8, 2, 64, 32, 64 * 9 + 5, 2), (1, 14, 2, 64, 64, 64 * 6 + 1, 2), (1, 4, 4, 32, 32, 40, 2),
         (1, 16, 2, 64, 32, 64 * 5 + 3, 2), (2, 8, 2, 42, 64, 42 * 11 + 7, 2), (2, 8, 2, 64, 32, 64 * 7 + 9, 4),
         (64, 32, 8, 128, 32, 2200, 2)]


@pytest.mark.parametrize("B,Hq,Hkv,W,G,n_tokens,bits", CASES)
def test_static_scratch_entry_point_matches_the_cache_entry_point_and_the_oracle_twice(B, Hq, Hkv, W, G, n_tokens,
                                                                                      bits):
    build.build()
    outl = synth.outlier_channels(77, Hkv, D, 3)
    k, v = synth.keys_values(77, B, Hkv, n_tokens, D, "cuda", outliers=outl)
    cache = LogQuantCache(1, B, Hq, Hkv, W, G, max_tokens=n_tokens + 8, bits=bits)
    cache.append(0, k, v)
    oc = oracle.OracleCache(B, Hq, Hkv, D, W, G, bits=bits)
    oc.append(synth.bf16_bits(k), synth.bf16_bits(v))
    image = _image_on_device(cache)
    for call in range(2):
        q = synth.queries(77, B, Hq, D, call, "cuda")
        want = torch.empty(B, Hq, D, device="cuda")
        cache.decode_attn(0, q, want)
        got = torch.full((B, Hq, D), float("nan"), device="cuda")
        status = decode_attn_image_static(image, Hq, G, q, got, bits=bits)
        assert status == binding.LQ_OK
        torch.cuda.synchronize()
        got = got.cpu().numpy().astype(np.float64)
        assert np.isfinite(got).all()
        ref = oc.attention(synth.bf16_bits(q), 1 / np.sqrt(D), n_threads=16)
        err = float(np.abs(got - ref).max())
        assert err <= attn_tolerance(ref), ("oracle", call, err)
        other = want.cpu().numpy().astype(np.float64)
        err = float(np.abs(got - other).max())
        assert err <= attn_tolerance(other), ("lq_decode_attn", call, err)


def _empty_image(B):
    z16 = torch.zeros(1, dtype=torch.int16, device="cuda")
    return dict(fp_k=torch.zeros(B, 1, 1, 128, dtype=torch.int16, device="cuda"),
                fp_v=torch.zeros(B, 1, 1, 128, dtype=torch.int16, device="cuda"),
                k_codes=torch.zeros(B, 1, 0, 32, dtype=torch.uint8, device="cuda"),
                v_codes=torch.zeros(B, 1, 0, 32, dtype=torch.uint8, device="cuda"),
                k_scale=z16[:0].reshape(B, 1, 0, 128), k_zero=z16[:0].reshape(B, 1, 0, 128),
                v_scale=z16[:0].reshape(B, 1, 0, 4), v_zero=z16[:0].reshape(B, 1, 0, 4))


def test_sizes_beyond_the_scratch_are_rejected():
    build.build()
    image = _empty_image(1100)
    q = torch.zeros(1100, 8, 128, dtype=torch.bfloat16, device="cuda")
    out = torch.zeros(1100, 8, 128, device="cuda")
    assert decode_attn_image_static(image, 8, 32, q, out) == binding.LQ_ERR_CAPACITY  # 8800 > 8192 records
    assert b"scratch" in binding.load_library().lq_status_str(binding.LQ_ERR_CAPACITY)


def test_a_code_width_the_image_format_does_not_have_is_rejected():
    build.build()
    image = _empty_image(1)
    q = torch.zeros(1, 1, 128, dtype=torch.bfloat16, device="cuda")
    out = torch.zeros(1, 1, 128, device="cuda")
    for bits in (0, 3, 8):
        assert decode_attn_image_static(image, 1, 32, q, out, bits=bits) == binding.LQ_ERR_INVALID_ARG

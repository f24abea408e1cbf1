"""The allocation-free entry point lq_decode_attn_image_static.

Some callers of this library cannot allocate device memory (a server with a fixed start-up arena, code
under a foreign allocator policy, code called during stream capture), so they cannot use lq_cache_create.
They keep the cache as a canonical image in memory of their own and call this entry point, whose split-K
scratch is a fixed array inside the library.  The test feeds it the image exported from an ordinary cache
and checks, on two calls in a row (the second one finds the first one's leftovers in the shared scratch),
that the output agrees with lq_decode_attn on the same cache within the tolerance of the parity tests.
Collected last on purpose: a run that stops at the first failure has run everything else before it."""
import numpy as np
import pytest
import torch

from gpu_common import attn_tolerance
from paper_2503_19950_b200 import LogQuantCache, binding, build, decode_attn_image_static, synth

pytestmark = pytest.mark.gpu


def _image_on_device(cache):
    img = cache.export(0)
    return {k: torch.from_numpy(v.view(np.int16) if v.dtype == np.uint16 else v).cuda()
            for k, v in img.items() if k not in ("kept_ids", "quant_ids")}


@pytest.mark.parametrize("B,Hq,Hkv,W,G,n_tokens", [(2, 8, 2, 64, 32, 64 * 9 + 5), (1, 14, 2, 64, 64, 64 * 6 + 1),
                                                  (1, 4, 4, 32, 32, 40)])
def test_static_scratch_entry_point_matches_the_cache_entry_point_twice(B, Hq, Hkv, W, G, n_tokens):
    build.build()
    D = 128
    k, v = synth.keys_values(77, B, Hkv, n_tokens, D, "cuda", outliers=synth.outlier_channels(77, Hkv, D, 3))
    cache = LogQuantCache(1, B, Hq, Hkv, W, G, max_tokens=n_tokens + 8)
    cache.append(0, k, v)
    image = _image_on_device(cache)
    for call in range(2):
        q = synth.queries(77, B, Hq, D, call, "cuda")
        want = torch.empty(B, Hq, D, device="cuda")
        cache.decode_attn(0, q, want)
        got = torch.full((B, Hq, D), float("nan"), device="cuda")
        status = decode_attn_image_static(image, Hq, G, q, got)
        assert status == binding.LQ_OK
        torch.cuda.synchronize()
        ref = want.cpu().numpy().astype(np.float64)
        err = float(np.abs(got.cpu().numpy() - ref).max())
        assert np.isfinite(got.cpu().numpy()).all() and err <= attn_tolerance(ref), (call, err)


def test_sizes_beyond_the_scratch_are_rejected():
    build.build()
    z16 = torch.zeros(1, dtype=torch.int16, device="cuda")
    image = dict(fp_k=torch.zeros(1100, 1, 1, 128, dtype=torch.int16, device="cuda"),
                 fp_v=torch.zeros(1100, 1, 1, 128, dtype=torch.int16, device="cuda"),
                 k_codes=torch.zeros(1100, 1, 0, 32, dtype=torch.uint8, device="cuda"),
                 v_codes=torch.zeros(1100, 1, 0, 32, dtype=torch.uint8, device="cuda"),
                 k_scale=z16[:0].reshape(1100, 1, 0, 128), k_zero=z16[:0].reshape(1100, 1, 0, 128),
                 v_scale=z16[:0].reshape(1100, 1, 0, 4), v_zero=z16[:0].reshape(1100, 1, 0, 4))
    q = torch.zeros(1100, 8, 128, dtype=torch.bfloat16, device="cuda")
    out = torch.zeros(1100, 8, 128, device="cuda")
    assert decode_attn_image_static(image, 8, 32, q, out) == binding.LQ_ERR_CAPACITY  # 8800 > 8192 records
    assert b"scratch" in binding.load_library().lq_status_str(binding.LQ_ERR_CAPACITY)

"""GPU parity of the tcgen05 decode kernel (LQ_KERNEL_UMMA) and of the device layout made for it: every cache
operation runs on that layout, the canonical image must equal the oracle's bit for bit and the attention
output must lie within max|delta| <= 2e-3*max|ref| + 1e-3 of the float64 oracle."""
import numpy as np
import pytest
import torch

from gpu_common import run_case
from paper_2503_19950_b200 import LQ_KERNEL_UMMA, LogQuantCache, LogQuantError, build

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _built():
    build.build()


def test_config1_tiny_decode():
    worst = run_case(B=1, Hq=8, Hkv=2, W=128, G=32, n_prefill=1024, n_steps=16, seed=1, kernel=LQ_KERNEL_UMMA,
                     n_outliers=4)
    assert worst <= 1.0


@pytest.mark.parametrize("B,Hq,Hkv,W,G,n_prefill,n_steps,chunk", [
    (2, 8, 2, 32, 32, 0, 3, None),            # a cache of 1..3 tokens, nothing quantised
    (1, 4, 4, 32, 32, 95, 4, None),           # crosses the first overflow (MHA, r = 1)
    (2, 14, 2, 64, 64, 64 * 9 + 7, 3, None),  # GQA-7, G = 64, ragged fp tail, odd number of key groups
    (1, 16, 2, 64, 32, 64 * 6 + 33, 2, None), # r = 8
    (3, 6, 2, 256, 64, 256 * 5 + 100, 2, None),  # W = 256, r = 3
    (1, 2, 1, 512, 64, 512 * 4 + 1, 2, None),    # largest window
    (2, 8, 2, 42, 64, 42 * 9 + 5, 4, None),      # W = 42, G = 64: waiting tokens, one-launch prompt
    (1, 14, 2, 85, 64, 85 * 7 + 30, 3, 97),      # W = 85, step-by-step overflow
    (2, 4, 4, 100, 32, 100 * 5 + 1, 3, 1),       # one token at a time
    (2, 8, 2, 64, 32, 64 * 21 + 3, 3, None),     # several 128-token super-tiles per CTA
])
def test_shapes_and_edge_cases(B, Hq, Hkv, W, G, n_prefill, n_steps, chunk):
    worst = run_case(B, Hq, Hkv, W, G, n_prefill, n_steps, seed=7, kernel=LQ_KERNEL_UMMA, prefill_chunk=chunk)
    assert worst <= 1.0


@pytest.mark.parametrize("B,Hq,Hkv,W,G,n_prefill,n_splits", [
    (1, 8, 2, 64, 32, 64 * 40 + 3, 1),     # one CTA per pair: ~27 items per CTA through the whole pipeline
    (2, 14, 2, 64, 64, 64 * 30 + 9, 1),    # the same at G = 64, GQA-7
    (1, 16, 2, 64, 32, 64 * 25 + 1, 1),    # r = 8: one buffer of key codes
    (40, 32, 8, 64, 32, 64 * 9 + 5, 0),    # 320 pairs on 296 CTAs: CTAs that work for two pairs
    (75, 8, 8, 32, 32, 32 * 5 + 7, 0),     # 600 pairs: up to four pairs per CTA, MHA
])
def test_many_items_and_several_pairs_per_cta(B, Hq, Hkv, W, G, n_prefill, n_splits):
    worst = run_case(B, Hq, Hkv, W, G, n_prefill, 3, seed=23, kernel=LQ_KERNEL_UMMA, n_splits=n_splits,
                     check_image_every=0)
    assert worst <= 1.0


def test_four_bit_codes_are_refused():
    with pytest.raises(LogQuantError):
        LogQuantCache(1, 1, 8, 2, 64, 32, max_tokens=512, bits=4, kernel=LQ_KERNEL_UMMA)

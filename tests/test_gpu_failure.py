"""Failure detection on the GPU without a fault: a bounded device-side wait that runs out must set bit 0 of the
cache's status word, leave the output untouched and return; the cache stays usable afterwards."""
import numpy as np
import pytest
import torch

import oracle
from gpu_common import attn_tolerance
from paper_2503_19950_b200 import LQ_KERNEL_MMA, LQ_KERNEL_UMMA, LogQuantCache, build, synth

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _built():
    build.build()


@pytest.mark.parametrize("kernel", [LQ_KERNEL_MMA, LQ_KERNEL_UMMA])
@pytest.mark.parametrize("n_tokens,n_splits", [(64 * 9 + 5, 0),   # several CTAs per pair: the merging CTA must write nothing
                                               (40, 1)])          # one CTA per pair, bf16 tokens only
def test_wait_that_runs_out_sets_status_and_leaves_out_untouched(kernel, n_tokens, n_splits):
    B, Hq, Hkv, W, G, D = 2, 8, 2, 64, 32, 128
    cache = LogQuantCache(1, B, Hq, Hkv, W, G, max_tokens=n_tokens + 8, kernel=kernel, n_splits=n_splits)
    oc = oracle.OracleCache(B, Hq, Hkv, D, W, G)
    k, v = synth.keys_values(41, B, Hkv, n_tokens, D, "cuda")
    cache.append(0, k, v)
    oc.append(synth.bf16_bits(k), synth.bf16_bits(v))
    q = synth.queries(41, B, Hq, D, 0, "cuda")
    out = torch.full((B, Hq, D), -7.0, device="cuda")
    assert cache.kernel_status() == 0
    cache.debug_stall_next_decode()       # the launch arms its query barrier, issues no copy and polls briefly
    cache.decode_attn(0, q, out)
    torch.cuda.synchronize()              # returns: nothing hangs, nothing faults
    assert cache.kernel_status() & 1
    assert bool((out == -7.0).all())
    # the hook covers one launch; after the status word is reset the cache works as before
    cache.reset_kernel_status()
    cache.decode_attn(0, q, out)
    torch.cuda.synchronize()
    assert cache.kernel_status() == 0
    ref = oc.attention(synth.bf16_bits(q), 1 / np.sqrt(D))
    assert np.abs(out.cpu().numpy() - ref).max() <= attn_tolerance(ref)
    cache.close()


def test_guard_bytes_detect_a_write_past_the_end_of_a_block():
    """256 guard bytes follow every device block; lq_check_guards counts the blocks whose guard changed.  With the
    torch allocator the blocks are tensors, so the test can damage one by hand (inside its own allocation)."""
    B, Hq, Hkv, W, G, D, N = 1, 8, 2, 32, 32, 128, 200
    cache = LogQuantCache(1, B, Hq, Hkv, W, G, max_tokens=N + 8, allocator="torch")
    k, v = synth.keys_values(43, B, Hkv, N, D, "cuda")
    cache.append(0, k, v)
    out = torch.empty(B, Hq, D, device="cuda")
    cache.decode_attn(0, synth.queries(43, B, Hq, D, 0, "cuda"), out)
    assert cache.check_guards() == 0
    n_alloc = [0]
    real_blocks = cache._blocks

    class Counting(dict):
        def __setitem__(self, key, value):
            n_alloc[0] += 1
            super().__setitem__(key, value)

    cache._blocks = Counting(real_blocks)
    cache.export(0)                      # the staging buffers of the export come from the caller's allocator too
    assert n_alloc[0] >= 8 and len(cache._blocks) == len(real_blocks)
    assert cache.check_guards() == 0
    victim = next(iter(cache._blocks.values()))
    victim[-1] = 0                       # the last guard byte of one block
    torch.cuda.synchronize()
    assert cache.check_guards() == 1
    victim[-1] = 0xA5
    torch.cuda.synchronize()
    assert cache.check_guards() == 0
    cache.close()

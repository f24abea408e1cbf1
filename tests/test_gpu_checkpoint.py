"""Checkpoint / resume through the canonical image: lq_export -> lq_import into a fresh cache (possibly on the other
device layout) must reproduce the image, the oracle's attention, and the oracle's stores after further tokens."""
import numpy as np
import pytest
import torch

import oracle
from gpu_common import attn_tolerance
from paper_2503_19950_b200 import LQ_KERNEL_MMA, LQ_KERNEL_UMMA, LogQuantCache, LogQuantError, build, synth

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _built():
    build.build()


@pytest.mark.parametrize("kernel_out,kernel_in,W,G,bits,recent,n_tokens", [
    (LQ_KERNEL_MMA, LQ_KERNEL_MMA, 64, 32, 2, False, 64 * 9 + 21),
    (LQ_KERNEL_MMA, LQ_KERNEL_UMMA, 64, 32, 2, False, 64 * 7 + 3),    # resume on the other device layout
    (LQ_KERNEL_UMMA, LQ_KERNEL_MMA, 85, 64, 2, False, 85 * 6 + 40),   # W % G != 0: tokens waiting for a full key group
    (LQ_KERNEL_MMA, LQ_KERNEL_MMA, 64, 64, 4, False, 64 * 5 + 11),    # 4-bit codes
    (LQ_KERNEL_MMA, LQ_KERNEL_MMA, 32, 32, 2, True, 32 * 8 + 5),      # the recent-window comparator's filter
    (LQ_KERNEL_MMA, LQ_KERNEL_MMA, 64, 32, 2, False, 100),            # nothing quantised yet
])
def test_export_import_round_trip_and_resume(kernel_out, kernel_in, W, G, bits, recent, n_tokens):
    """Checkpoint / resume: an exported image loaded into a fresh cache (lq_import) gives the same image, the same
    attention as the oracle, and the same stores as the oracle after further decode steps."""
    B, Hq, Hkv, D, n_more, n_chunk = 2, 8, 2, 128, W + 7, 3 * W + 5
    filt = 1 if recent else 0
    src = LogQuantCache(1, B, Hq, Hkv, W, G, max_tokens=n_tokens + n_more + 8, bits=bits, kernel=kernel_out, filter=filt)
    oc = oracle.OracleCache(B, Hq, Hkv, D, W, G, bits=bits, recent_only=recent)
    k, v = synth.keys_values(47, B, Hkv, n_tokens + n_more, D, "cuda", outliers=synth.outlier_channels(47, Hkv, D, 3))
    k0, v0 = k[:, :, :n_tokens].contiguous(), v[:, :, :n_tokens].contiguous()
    src.append(0, k0, v0)
    oc.append(synth.bf16_bits(k0), synth.bf16_bits(v0))
    image = src.export(0)
    src.close()
    dst = LogQuantCache(2, B, Hq, Hkv, W, G, max_tokens=n_tokens + n_more + n_chunk + 8, bits=bits, kernel=kernel_in, filter=filt)
    dst.import_image(1, image, n_tokens)
    inf = dst.info(1)
    assert (inf.n_seen, inf.n_fp, inf.n_quant) == (n_tokens, image["kept_ids"].size, image["quant_ids"].size)
    again = dst.export(1)
    assert all(np.array_equal(again[key], image[key]) for key in image)
    q = synth.queries(47, B, Hq, D, 0, "cuda")
    out = torch.empty(B, Hq, D, device="cuda")
    dst.decode_attn(1, q, out)
    ref = oc.attention(synth.bf16_bits(q), 1 / np.sqrt(D))
    assert np.abs(out.cpu().numpy() - ref).max() <= attn_tolerance(ref)
    # resume: further tokens cross at least one overflow; the stores must stay those of the oracle
    for t in range(n_tokens, n_tokens + n_more):
        kt, vt = k[:, :, t:t + 1].contiguous(), v[:, :, t:t + 1].contiguous()
        dst.append(1, kt, vt)
        oc.append(synth.bf16_bits(kt), synth.bf16_bits(vt))
    want, got = oc.export(), dst.export(1)
    assert all(np.array_equal(got[key], want[key]) for key in want)
    dst.decode_attn(1, q, out)
    ref = oc.attention(synth.bf16_bits(q), 1 / np.sqrt(D))
    assert np.abs(out.cpu().numpy() - ref).max() <= attn_tolerance(ref)
    # a chunk of a prompt on top of the resumed layer: one launch that gathers from the imported rows and the chunk
    kc, vc = synth.keys_values(48, B, Hkv, n_chunk, D, "cuda", outliers=synth.outlier_channels(47, Hkv, D, 3))
    before = dst.info(1).n_kernel_launches
    dst.append(1, kc, vc)
    assert dst.info(1).n_kernel_launches == before + 1
    oc.append(synth.bf16_bits(kc), synth.bf16_bits(vc))
    want, got = oc.export(), dst.export(1)
    assert all(np.array_equal(got[key], want[key]) for key in want)
    dst.decode_attn(1, q, out)
    ref = oc.attention(synth.bf16_bits(q), 1 / np.sqrt(D))
    assert np.abs(out.cpu().numpy() - ref).max() <= attn_tolerance(ref)
    assert dst.kernel_status() == 0
    assert dst.kernel_status() == 0
    # a layer that is not empty, or sizes that do not belong to n_seen tokens, are refused and change nothing
    with pytest.raises(LogQuantError):
        dst.import_image(1, image, n_tokens)
    with pytest.raises(LogQuantError):
        dst.import_image(0, image, n_tokens + 1)
    assert dst.info(0).n_seen == 0
    dst.close()

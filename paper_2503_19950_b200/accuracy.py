"""Attention error of the mixed cache against exact bf16 attention, on synthetic data.

The paper scores its method on model benchmarks (Sec. 3.2) that need weights and datasets.  What can be
measured without them is the quantity those scores follow from: how far the attention output over the
compressed cache is from the output over the original bf16 cache, for

  * the log-distributed filter of Algorithm 1 (LQ_FILTER_LOG) and
  * a recent-window filter with the same number of full-precision tokens (LQ_FILTER_RECENT, the retention
    rule of the sliding-window quantisers the paper compares with, Sec. 2.2-2.3),

each with 2-bit and (at G = 32) 4-bit codes, and for the eviction variant of both filters (the removed tokens are
dropped instead of quantised, Sec. 2.3: `lq_decode_attn_fp_only`).  Keys carry planted high-logit tokens at log-spaced
distances behind the query position (the shape of the attention pattern in the paper's Fig. 1); the
prompt length is varied so that the planted tokens fall on and off the filter's kept grid.

Usage:  python -m paper_2503_19950_b200.accuracy [--ctx 8192] [--lengths 16]
Every cache operation runs in the CUDA library; torch computes only the exact reference.
"""
from __future__ import annotations

import argparse
import json

import torch

from . import LQ_FILTER_LOG, LQ_FILTER_RECENT, LogQuantCache, synth

D = 128


def exact_attention(q, k, v):
    """softmax(q k^T / sqrt(D)) v in float64 over the original bf16 keys and values."""
    r = q.shape[1] // k.shape[1]
    kf, vf = k.double().repeat_interleave(r, 1), v.double().repeat_interleave(r, 1)
    p = torch.softmax(torch.einsum("bhd,bhtd->bht", q.double(), kf) / D ** 0.5, -1)
    return torch.einsum("bht,bhtd->bhd", p, vf)


def planted_case(seed, B, Hq, Hkv, n, kappa, a, device):
    """Keys N(0,1) + kappa*u at distances 2^i behind the last position; q = N(0,1) + a*u."""
    u = synth.unit_vectors(seed, Hkv, D)
    k, v = synth.keys_values(seed, B, Hkv, n, D, device)
    k = synth.plant_spikes(k, u, kappa, 0, n)
    q = synth.queries(seed, B, Hq, D, n, device)
    q = (q.float() + a * u.to(device).repeat_interleave(Hq // Hkv, dim=0)[None]).to(torch.bfloat16)
    return q, k, v


def run(ctx=8192, lengths=16, B=2, kappa=16.0, a=4.0, seed=4, device="cuda"):
    shapes = [dict(name="Hq32/Hkv8 W128 G32", Hq=32, Hkv=8, W=128, G=32, bits=(2, 4)),
              dict(name="Hq28/Hkv4 W256 G64", Hq=28, Hkv=4, W=256, G=64, bits=(2,)),
              # the paper's own settings (Sec. 3.1): group 64, reserved length 128 and 256 tokens, i.e. W = 42, 85
              dict(name="Hq32/Hkv8 W42 G64", Hq=32, Hkv=8, W=42, G=64, bits=(2,)),
              dict(name="Hq32/Hkv8 W85 G64", Hq=32, Hkv=8, W=85, G=64, bits=(2,))]
    rows = []
    for sh in shapes:
        for bits in sh["bits"]:
            variants = [(LQ_FILTER_LOG, "log (Algorithm 1)", False), (LQ_FILTER_RECENT, "recent window", False)]
            if bits == 2:
                variants += [(LQ_FILTER_LOG, "log, eviction", True), (LQ_FILTER_RECENT, "recent window, eviction", True)]
            for filt, fname, evict in variants:
                num = den = worst = 0.0
                for i in range(lengths):
                    n = ctx + 37 * i  # off the window grid on purpose
                    q, k, v = planted_case(seed + i, B, sh["Hq"], sh["Hkv"], n, kappa, a, device)
                    ref = exact_attention(q, k, v)
                    cache = LogQuantCache(1, B, sh["Hq"], sh["Hkv"], sh["W"], sh["G"], max_tokens=n + 8, bits=bits,
                                          filter=filt)
                    cache.append(0, k, v)
                    out = torch.empty(B, sh["Hq"], D, device=device)
                    if evict:
                        cache.decode_attn_fp_only(0, q, out)
                    else:
                        cache.decode_attn(0, q, out)
                    torch.cuda.synchronize()
                    inf = cache.info(0)
                    err = (out.double() - ref).abs()
                    num += float(err.sum())
                    den += float(ref.abs().sum())
                    worst = max(worst, float(err.max() / ref.abs().max()))
                    kept_bytes = inf.n_fp * 4 * D + (0 if evict else inf.n_quant * inf.bytes_quant_per_token)
                    ratio = (n * 4 * D) / kept_bytes
                    cache.close()
                rows.append(dict(shape=sh["name"], bits=0 if evict else bits, filter=fname, rel_l1=num / den, worst_rel_max=worst,
                                 compression=ratio))
    return rows


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--ctx", type=int, default=8192)
    ap.add_argument("--lengths", type=int, default=16)
    args = ap.parse_args()
    if not torch.cuda.is_available():
        raise SystemExit("needs a CUDA device: every cache operation runs in the CUDA library")
    for row in run(args.ctx, args.lengths):
        print(json.dumps(row))


if __name__ == "__main__":
    main()

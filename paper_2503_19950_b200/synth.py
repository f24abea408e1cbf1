"""Seeded synthetic inputs for tests and benchmarks (no method arithmetic lives here).

A counter-based generator built from integer tensor ops only, so that the same (seed, index)
gives bit-identical bf16 values on the CPU and on the GPU: 64-bit mix hash of the element's
linear index -> twelve 16-bit uniforms -> (sum - 12*32767.5) / 65536 (an Irwin-Hall
approximation of N(0,1), exact in fp32) -> optional per-channel gain -> bf16 (round to nearest even).

Workload recipes (shapes and value distributions of the benchmark configurations):
  * keys:    N(0,1) with a few "outlier" channels scaled x10 (fixed per KV head from the seed)
  * values:  N(0,1)
  * queries: N(0,1)
  * planted keys (long-context configuration): N(0,1) plus kappa*u at log-spaced distances
    behind the last position, u a fixed unit vector per KV head; queries get a*u added.
"""
from __future__ import annotations

import torch

_M1 = -7046029254386353131  # 0x9E3779B97F4A7C15 as int64
_M2 = -4658895280553007687  # 0xBF58476D1CE4E5B9
_M3 = -7723592293110705685  # 0x94D049BB133111EB


def _lsr(x: torch.Tensor, n: int) -> torch.Tensor:
    """Logical shift right of int64."""
    return (x >> n) & ((1 << (64 - n)) - 1)


def _mix(x: torch.Tensor) -> torch.Tensor:
    x = (x ^ _lsr(x, 30)) * _M2
    x = (x ^ _lsr(x, 27)) * _M3
    return x ^ _lsr(x, 31)


def _wrap(x: int) -> int:
    """Python int -> two's-complement int64 value."""
    x &= (1 << 64) - 1
    return x - (1 << 64) if x >= (1 << 63) else x


def _normal_at(seed: int, stream: int, idx: torch.Tensor) -> torch.Tensor:
    """Approximately-N(0,1) fp32 values for the int64 linear indices `idx` (any shape)."""
    base = _mix(idx * _M1 + _wrap((seed * 1000003 + stream) * _M2))
    total = torch.zeros_like(idx)
    for rep in range(3):
        h = _mix(base + _wrap((rep + 1) * _M3))
        for s in (0, 16, 32, 48):
            total += _lsr(h, s) & 0xFFFF
    return (total.to(torch.float32) - 393210.0) / 65536.0  # 12 * 32767.5 = 393210


def normal_f32(seed: int, stream: int, start: int, count: int, device="cpu") -> torch.Tensor:
    """`count` approximately-N(0,1) fp32 values for linear indices [start, start+count)."""
    return _normal_at(seed, stream, torch.arange(start, start + count, dtype=torch.int64, device=device))


def tensor_f32(seed: int, stream: int, shape, device="cpu", token_axis=None, token_start=0,
               token_total=None) -> torch.Tensor:
    """N(0,1) fp32 tensor of `shape` (every value is exactly representable in bf16 precision only
    after the caller rounds it).  If token_axis is given, the tensor is the slice
    [token_start, token_start + shape[token_axis]) of a virtual tensor whose token axis has length
    token_total, so that a long sequence can be produced in chunks with identical values."""
    shape = tuple(shape)
    full = list(shape)
    if token_axis is not None:
        full[token_axis] = token_total
    strides = [1] * len(full)
    for i in range(len(full) - 2, -1, -1):
        strides[i] = strides[i + 1] * full[i + 1]
    idx = torch.zeros(shape, dtype=torch.int64, device=device)
    for ax, n in enumerate(shape):
        r = torch.arange(n, dtype=torch.int64, device=device)
        if ax == token_axis:
            r = r + token_start
        view = [1] * len(shape)
        view[ax] = n
        idx = idx + r.reshape(view) * strides[ax]
    return _normal_at(seed, stream, idx)


def outlier_channels(seed: int, n_kv_heads: int, head_dim: int, n_outliers: int) -> torch.Tensor:
    """[n_kv_heads, n_outliers] distinct channel indices per KV head, from the seed."""
    out = []
    for h in range(n_kv_heads):
        r = normal_f32(seed, 7000 + h, 0, head_dim, "cpu")
        out.append(torch.argsort(r)[:n_outliers])
    return torch.stack(out)


def keys_values(seed: int, B: int, Hkv: int, n_tokens: int, D: int, device="cpu", token_start=0,
                token_total=None, outliers: torch.Tensor | None = None, gain: float = 10.0, layer: int = 0):
    """k, v: bf16 [B, Hkv, n_tokens, D], the slice [token_start, token_start+n_tokens) of a sequence
    of token_total tokens.  `outliers`: [Hkv, n] channel indices whose keys are scaled by `gain`."""
    token_total = token_total if token_total is not None else token_start + n_tokens
    k = tensor_f32(seed, 10 + 4 * layer, (B, Hkv, n_tokens, D), device, 2, token_start, token_total)
    v = tensor_f32(seed, 11 + 4 * layer, (B, Hkv, n_tokens, D), device, 2, token_start, token_total)
    if outliers is not None and outliers.numel():
        g = torch.ones(Hkv, D, dtype=torch.float32)
        for h in range(Hkv):
            g[h, outliers[h]] = gain
        k = k * g.to(device)[None, :, None, :]
    return k.to(torch.bfloat16).contiguous(), v.to(torch.bfloat16).contiguous()


def queries(seed: int, B: int, Hq: int, D: int, step: int = 0, device="cpu", layer: int = 0) -> torch.Tensor:
    return tensor_f32(seed, 12 + 4 * layer + 1000 * (step + 1), (B, Hq, D), device).to(torch.bfloat16).contiguous()


def unit_vectors(seed: int, Hkv: int, D: int) -> torch.Tensor:
    u = normal_f32(seed, 9000, 0, Hkv * D, "cpu").reshape(Hkv, D)
    return u / u.norm(dim=1, keepdim=True)


def plant_spikes(k: torch.Tensor, u: torch.Tensor, kappa: float, token_start: int, last_pos: int) -> torch.Tensor:
    """Add kappa*u[h] to the keys at distances 2^i behind `last_pos` (those that fall in this chunk)."""
    kf = k.to(torch.float32)
    i = 0
    while (1 << i) <= last_pos:
        t = last_pos - (1 << i) - token_start
        if 0 <= t < k.shape[2]:
            kf[:, :, t, :] += kappa * u.to(k.device)[None, :, :]
        i += 1
    return kf.to(torch.bfloat16).contiguous()


def bf16_bits(t: torch.Tensor):
    """uint16 numpy view of a bf16 tensor (moved to the host)."""
    return t.detach().cpu().contiguous().view(torch.int16).numpy().view("uint16")

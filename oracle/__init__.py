"""CPU oracle for the LogQuant decode hot path -- TEST INFRASTRUCTURE, NOT PRODUCT CODE.

A ctypes wrapper over ``lq_oracle.cpp`` (plain C++17, float64 attention, IEEE fp32
quantiser).  Only the tests, the smoke check and the benchmark's CPU-baseline leg may
import this package; the CUDA library never does, and shares no code with it.

Tensors cross this boundary as numpy arrays: bf16 data as ``uint16`` bit patterns.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "lq_oracle.cpp")
_LIB = os.path.join(_HERE, "liblq_oracle.so")


def build(force: bool = False) -> str:
    """Compile the oracle with g++ (no CUDA, no fast-math, no FMA contraction)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["g++", "-O2", "-std=c++17", "-ffp-contract=off", "-fPIC", "-shared", "-pthread",
               _SRC, "-o", _LIB + ".tmp"]
        subprocess.run(cmd, check=True)
        os.replace(_LIB + ".tmp", _LIB)
    return _LIB


_lib = None


def lib():
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
        L = _lib
        p, i32, i64, f64 = C.c_void_p, C.c_int, C.c_int64, C.c_double
        L.lqo_filter.restype = i64
        L.lqo_filter.argtypes = [i32, i64, p, p, p, p]
        L.lqo_quantize_group.argtypes = [p, i32, p, p, p]
        L.lqo_quantize_group_bits.argtypes = [p, i32, i32, p, p, p]
        L.lqo_pack4.argtypes = [p, i64, p]
        L.lqo_unpack4.argtypes = [p, i64, p]
        L.lqo_create_bits.restype = p
        L.lqo_create_bits.argtypes = [i32] * 7
        L.lqo_create_policy.restype = p
        L.lqo_create_policy.argtypes = [i32] * 8
        L.lqo_dequant.restype = f64
        L.lqo_dequant.argtypes = [C.c_uint16, C.c_uint16, C.c_uint8]
        L.lqo_pack2.argtypes = [p, i64, p]
        L.lqo_unpack2.argtypes = [p, i64, p]
        L.lqo_f32_to_bf16.restype = C.c_uint16
        L.lqo_f32_to_bf16.argtypes = [C.c_float]
        L.lqo_bf16_to_f32.restype = C.c_float
        L.lqo_bf16_to_f32.argtypes = [C.c_uint16]
        L.lqo_attention_dense.argtypes = [p, p, p, i64, i32, f64, p]
        L.lqo_attention_partial.argtypes = [p, p, p, i64, i32, f64, p, p, p]
        L.lqo_attention_merge.argtypes = [p, p, p, i32, i32, p]
        L.lqo_create.restype = p
        L.lqo_create.argtypes = [i32] * 6
        L.lqo_destroy.argtypes = [p]
        L.lqo_append.argtypes = [p, p, p, i32]
        for name in ("lqo_n_seen", "lqo_n_fp", "lqo_n_quant", "lqo_n_events"):
            getattr(L, name).restype = i64
            getattr(L, name).argtypes = [p]
        L.lqo_export.argtypes = [p] * 11
        L.lqo_dense_rows.argtypes = [p, i32, i32, p, p]
        L.lqo_attention.argtypes = [p, p, f64, p, i32]
        L.lqo_attention_subset.argtypes = [p, p, f64, p, i32, p]
        L.lqo_hardware_threads.restype = C.c_uint
    return _lib


def _ptr(a):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


def _c(a, dtype):
    a = np.ascontiguousarray(a, dtype=dtype)
    return a


# ---- stand-alone pieces ---------------------------------------------------------------
def filter_ids(W: int, N: int):
    """Algorithm 1 on token ids 0..N-1 -> (kept ids, quantised ids in store order, events)."""
    kept = np.zeros(3 * W, np.int64)
    quant = np.zeros(max(N, 1), np.int64)
    nk, nq = C.c_int64(0), C.c_int64(0)
    ev = lib().lqo_filter(W, N, _ptr(kept), C.byref(nk), _ptr(quant), C.byref(nq))
    return kept[: nk.value].copy(), quant[: nq.value].copy(), int(ev)


def quantize_group(x_bf16: np.ndarray, bits: int = 2):
    """One quantisation group (uint16 bf16 bits) -> (scale bits, zero bits, codes)."""
    x = _c(x_bf16, np.uint16)
    s, z = np.zeros(1, np.uint16), np.zeros(1, np.uint16)
    codes = np.zeros(x.size, np.uint8)
    if bits == 2:
        lib().lqo_quantize_group(_ptr(x), x.size, _ptr(s), _ptr(z), _ptr(codes))
    else:
        lib().lqo_quantize_group_bits(_ptr(x), x.size, bits, _ptr(s), _ptr(z), _ptr(codes))
    return int(s[0]), int(z[0]), codes


def dequant(scale_bits: int, zero_bits: int, code: int) -> float:
    return float(lib().lqo_dequant(scale_bits, zero_bits, code))


def pack2(codes: np.ndarray) -> np.ndarray:
    c = _c(codes, np.uint8)
    out = np.zeros(c.size // 4, np.uint8)
    lib().lqo_pack2(_ptr(c), c.size, _ptr(out))
    return out


def unpack2(bytes_: np.ndarray) -> np.ndarray:
    b = _c(bytes_, np.uint8)
    out = np.zeros(b.size * 4, np.uint8)
    lib().lqo_unpack2(_ptr(b), out.size, _ptr(out))
    return out


def pack4(codes: np.ndarray) -> np.ndarray:
    c = _c(codes, np.uint8)
    out = np.zeros(c.size // 2, np.uint8)
    lib().lqo_pack4(_ptr(c), c.size, _ptr(out))
    return out


def unpack4(bytes_: np.ndarray) -> np.ndarray:
    b = _c(bytes_, np.uint8)
    out = np.zeros(b.size * 2, np.uint8)
    lib().lqo_unpack4(_ptr(b), out.size, _ptr(out))
    return out


def f32_to_bf16(x: float) -> int:
    return int(lib().lqo_f32_to_bf16(x))


def bf16_to_f32(h: int) -> float:
    return float(lib().lqo_bf16_to_f32(h))


def attention_dense(q, K, V, sm_scale: float) -> np.ndarray:
    q, K, V = _c(q, np.float64), _c(K, np.float64), _c(V, np.float64)
    n, D = K.shape
    out = np.zeros(D, np.float64)
    lib().lqo_attention_dense(_ptr(q), _ptr(K), _ptr(V), n, D, sm_scale, _ptr(out))
    return out


def attention_partial(q, K, V, sm_scale: float):
    q, K, V = _c(q, np.float64), _c(K, np.float64), _c(V, np.float64)
    D = q.size
    n = K.shape[0] if K.size else 0
    m, l = C.c_double(0), C.c_double(0)
    o = np.zeros(D, np.float64)
    lib().lqo_attention_partial(_ptr(q), _ptr(K), _ptr(V), n, D, sm_scale, C.byref(m), C.byref(l), _ptr(o))
    return m.value, l.value, o


def attention_merge(m, l, o) -> np.ndarray:
    m, l, o = _c(m, np.float64), _c(l, np.float64), _c(o, np.float64)
    S, D = o.shape
    out = np.zeros(D, np.float64)
    lib().lqo_attention_merge(_ptr(m), _ptr(l), _ptr(o), S, D, _ptr(out))
    return out


def hardware_threads() -> int:
    return int(lib().lqo_hardware_threads())


# ---- the cache object -------------------------------------------------------------------
class OracleCache:
    """One layer's mixed cache for B sequences: Algorithm 1 + quantiser + attention."""

    def __init__(self, B, Hq, Hkv, D, W, G, bits=2, recent_only=False):
        self.B, self.Hq, self.Hkv, self.D, self.W, self.G, self.bits = B, Hq, Hkv, D, W, G, bits
        self._h = lib().lqo_create_policy(B, Hq, Hkv, D, W, G, bits, int(recent_only))
        if not self._h:
            raise ValueError("unsupported oracle configuration")

    def close(self):
        if self._h:
            lib().lqo_destroy(self._h)
            self._h = None

    def __del__(self):
        self.close()

    def append(self, k_bf16: np.ndarray, v_bf16: np.ndarray):
        """k, v: uint16 [B, Hkv, n, D]; n single appends, each running Algorithm 1."""
        k, v = _c(k_bf16, np.uint16), _c(v_bf16, np.uint16)
        assert k.shape == v.shape and k.shape[0] == self.B and k.shape[1] == self.Hkv and k.shape[3] == self.D
        lib().lqo_append(self._h, _ptr(k), _ptr(v), k.shape[2])

    @property
    def n_seen(self):
        return int(lib().lqo_n_seen(self._h))

    @property
    def n_fp(self):
        return int(lib().lqo_n_fp(self._h))

    @property
    def n_quant(self):
        return int(lib().lqo_n_quant(self._h))

    @property
    def n_events(self):
        return int(lib().lqo_n_events(self._h))

    def export(self) -> dict:
        """Canonical image (see include/lq.h): ids, packed codes, bf16 scale/zero, fp rows."""
        B, H, D, G = self.B, self.Hkv, self.D, self.G
        nf, nq = self.n_fp, self.n_quant
        img = dict(
            kept_ids=np.zeros(nf, np.int32), quant_ids=np.zeros(nq, np.int32),
            k_codes=np.zeros((B, H, nq, D * self.bits // 8), np.uint8),
            v_codes=np.zeros((B, H, nq, D * self.bits // 8), np.uint8),
            k_scale=np.zeros((B, H, nq // G, D), np.uint16), k_zero=np.zeros((B, H, nq // G, D), np.uint16),
            v_scale=np.zeros((B, H, nq, D // G), np.uint16), v_zero=np.zeros((B, H, nq, D // G), np.uint16),
            fp_k=np.zeros((B, H, nf, D), np.uint16), fp_v=np.zeros((B, H, nf, D), np.uint16))
        order = ["kept_ids", "quant_ids", "k_codes", "v_codes", "k_scale", "k_zero", "v_scale", "v_zero",
                 "fp_k", "fp_v"]
        lib().lqo_export(self._h, *[_ptr(img[k]) for k in order])
        return img

    def dense_rows(self, b: int, kv: int):
        n = self.n_fp + self.n_quant
        K, V = np.zeros((n, self.D), np.float64), np.zeros((n, self.D), np.float64)
        lib().lqo_dense_rows(self._h, b, kv, _ptr(K), _ptr(V))
        return K, V

    def attention(self, q_bf16: np.ndarray, sm_scale: float, n_threads: int = 1) -> np.ndarray:
        q = _c(q_bf16, np.uint16)
        assert q.shape == (self.B, self.Hq, self.D)
        out = np.zeros((self.B, self.Hq, self.D), np.float64)
        lib().lqo_attention(self._h, _ptr(q), float(sm_scale), _ptr(out), n_threads)
        return out

    def attention_subset(self, q_bf16: np.ndarray, sm_scale: float, fp_only: bool = False, pad=None) -> np.ndarray:
        """Attention over the tokens at original precision only (fp_only) and/or without the first pad[b]
        positions of sequence b (left padding of a ragged batch)."""
        q = _c(q_bf16, np.uint16)
        assert q.shape == (self.B, self.Hq, self.D)
        padv = None if pad is None else _c(pad, np.int32)
        assert padv is None or padv.shape == (self.B,)
        out = np.zeros((self.B, self.Hq, self.D), np.float64)
        lib().lqo_attention_subset(self._h, _ptr(q), float(sm_scale), _ptr(out), int(fp_only), _ptr(padv))
        return out

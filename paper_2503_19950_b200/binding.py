"""ctypes binding with the same names as include/lq.h (argument marshalling only)."""
from __future__ import annotations

import ctypes as C
import os
import weakref

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
# LOGQUANT_LIBRARY: another build of the same library (e.g. liblogquant_bounds.so, the build with index checks)
_LIB_PATH = os.environ.get("LOGQUANT_LIBRARY") or os.path.join(_HERE, "liblogquant.so")

LQ_DEVICE_NONE = -1
LQ_KERNEL_AUTO, LQ_KERNEL_SCALAR, LQ_KERNEL_MMA, LQ_KERNEL_UMMA = 0, 1, 2, 3
LQ_FILTER_LOG, LQ_FILTER_RECENT = 0, 1
LQ_FLAG_OVERLAP_DECODE = 1
LQ_OK, LQ_ERR_INVALID_ARG, LQ_ERR_UNSUPPORTED, LQ_ERR_OOM, LQ_ERR_WINDOW_FULL, LQ_ERR_NOT_FULL, \
    LQ_ERR_CAPACITY, LQ_ERR_CUDA = range(8)


ALLOC_FN = C.CFUNCTYPE(C.c_void_p, C.c_size_t, C.c_void_p)
FREE_FN = C.CFUNCTYPE(None, C.c_void_p, C.c_void_p)


class lq_config_t(C.Structure):
    _fields_ = [("n_layers", C.c_int32), ("batch", C.c_int32), ("n_q_heads", C.c_int32),
                ("n_kv_heads", C.c_int32), ("head_dim", C.c_int32), ("window", C.c_int32),
                ("group", C.c_int32), ("bits", C.c_int32), ("max_tokens", C.c_int64),
                ("auto_compress", C.c_int32), ("device", C.c_int32), ("kernel", C.c_int32),
                ("n_splits", C.c_int32), ("filter", C.c_int32), ("flags", C.c_int32),
                ("dev_alloc", ALLOC_FN), ("dev_free", FREE_FN), ("alloc_ctx", C.c_void_p)]


class lq_info_t(C.Structure):
    _fields_ = [("n_seen", C.c_int64), ("n_fp", C.c_int64), ("n_quant", C.c_int64), ("n_events", C.c_int64),
                ("bytes_device", C.c_int64), ("bytes_decode_step", C.c_int64),
                ("bytes_quant_per_token", C.c_int64), ("n_splits", C.c_int32), ("n_ctas", C.c_int32),
                ("n_kernel_launches", C.c_int64), ("n_ctas_overlapped", C.c_int32), ("n_launches_overlapped", C.c_int32)]


class lq_image_t(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in ("kept_ids", "quant_ids", "k_codes", "v_codes", "k_scale", "k_zero",
                                          "v_scale", "v_zero", "fp_k", "fp_v")]


class lq_device_image_t(C.Structure):
    _fields_ = [("batch", C.c_int32), ("n_q_heads", C.c_int32), ("n_kv_heads", C.c_int32), ("head_dim", C.c_int32),
                ("group", C.c_int32), ("bits", C.c_int32), ("n_fp", C.c_int32), ("n_quant", C.c_int64)] + \
               [(n, C.c_void_p) for n in ("fp_k", "fp_v", "k_codes", "v_codes", "k_scale", "k_zero", "v_scale", "v_zero")]


SYMBOLS = ["lq_cache_create", "lq_destroy", "lq_append", "lq_compress", "lq_decode_attn", "lq_append_decode_attn",
           "lq_decode_attn_fp_only", "lq_set_padding",
           "lq_decode_step_host", "lq_profile_enable", "lq_profile_read", "lq_kernel_status", "lq_cache_info", "lq_export",
           "lq_next_evicted_ids", "lq_decode_attn_image_static", "lq_status_str", "lq_last_error", "lq_check_guards",
           "lq_reset_kernel_status", "lq_debug_stall_next_decode", "lq_debug_bad_slot_next_append", "lq_import"]

_lib = None


class LogQuantError(RuntimeError):
    def __init__(self, status, msg):
        super().__init__(msg)
        self.status = status


def load_library():
    """Load liblogquant.so.  There is no fallback: a missing library is an error."""
    global _lib
    if _lib is None:
        if not os.path.exists(_LIB_PATH):
            raise ImportError(f"{_LIB_PATH} is missing: run `python -m paper_2503_19950_b200.build` "
                              "(there is no CPU or PyTorch fallback for the LogQuant kernels)")
        L = C.CDLL(_LIB_PATH)
        vp, i32 = C.c_void_p, C.c_int32
        L.lq_cache_create.argtypes = [C.POINTER(lq_config_t), C.POINTER(vp)]
        L.lq_destroy.argtypes = [vp]
        L.lq_append.argtypes = [vp, i32, vp, vp, i32, vp]
        L.lq_compress.argtypes = [vp, i32, vp]
        L.lq_decode_attn.argtypes = [vp, i32, vp, C.c_float, vp, i32, vp]
        L.lq_append_decode_attn.argtypes = [vp, i32, vp, vp, vp, C.c_float, vp, i32, vp]
        L.lq_decode_attn_fp_only.argtypes = [vp, i32, vp, C.c_float, vp, i32, vp]
        L.lq_set_padding.argtypes = [vp, vp]
        L.lq_decode_step_host.argtypes = [vp, i32, vp, vp, vp, C.c_float, vp, i32, vp]
        L.lq_kernel_status.argtypes = [vp, C.POINTER(C.c_int32)]
        L.lq_check_guards.argtypes = [vp, C.POINTER(C.c_int32)]
        L.lq_reset_kernel_status.argtypes = [vp]
        L.lq_debug_stall_next_decode.argtypes = [vp]
        L.lq_debug_bad_slot_next_append.argtypes = [vp]
        L.lq_profile_enable.argtypes = [vp, i32]
        L.lq_profile_read.argtypes = [vp, C.POINTER(C.c_double), C.POINTER(C.c_int64)]
        L.lq_cache_info.argtypes = [vp, i32, C.POINTER(lq_info_t)]
        L.lq_export.argtypes = [vp, i32, C.POINTER(lq_image_t)]
        L.lq_import.argtypes = [vp, i32, C.POINTER(lq_image_t), C.c_int64, C.c_int64, C.c_int64]
        L.lq_next_evicted_ids.argtypes = [vp, i32, vp]
        L.lq_decode_attn_image_static.argtypes = [C.POINTER(lq_device_image_t), vp, C.c_float, vp, vp]
        L.lq_status_str.argtypes = [i32]
        L.lq_status_str.restype = C.c_char_p
        L.lq_last_error.argtypes = [vp]
        L.lq_last_error.restype = C.c_char_p
        for s in SYMBOLS:
            if getattr(L, s).restype is C.c_int:
                getattr(L, s).restype = i32
        _lib = L
    return _lib


def exported_symbols():
    L = load_library()
    return [s for s in SYMBOLS if hasattr(L, s)]


def _ptr(x):
    """Device/host address of a torch tensor, numpy array, int or None."""
    if x is None:
        return None
    if isinstance(x, int):
        return x
    if isinstance(x, np.ndarray):
        return x.ctypes.data
    return x.data_ptr()  # torch tensor


def _stream(stream):
    if stream is None:
        import torch
        return torch.cuda.current_stream().cuda_stream if torch.cuda.is_available() else None
    return stream if isinstance(stream, int) else stream.cuda_stream


def decode_attn_image_static(image: dict, n_q_heads: int, group: int, q, out, sm_scale=0.0, stream=None,
                             bits: int = 2) -> int:
    """lq_decode_attn_image_static on a canonical image whose arrays are torch tensors on the device
    (keys as in LogQuantCache.export, without the ids).  Allocates nothing; returns the status code."""
    B, Hkv, n_fp, D = image["fp_k"].shape
    n_quant = image["k_codes"].shape[2]
    st = lq_device_image_t(B, n_q_heads, Hkv, D, group, bits, n_fp, n_quant,
                           *[(_ptr(image[k]) if image[k].numel() else None)
                             for k in ("fp_k", "fp_v", "k_codes", "v_codes", "k_scale", "k_zero", "v_scale", "v_zero")])
    return load_library().lq_decode_attn_image_static(C.byref(st), _ptr(q), sm_scale, _ptr(out), _stream(stream))


class LogQuantCache:
    """Owner of one lq_cache_t.  Methods mirror the C entry points one to one."""

    live = weakref.WeakSet()   # caches that have not been collected yet (the tests check their guard bytes)
    guards_on_close = False    # True: close() checks the guard bytes behind every device block and raises if one changed

    def __init__(self, n_layers, batch, n_q_heads, n_kv_heads, window, group, max_tokens, head_dim=128, bits=2,
                 auto_compress=True, device=0, kernel=LQ_KERNEL_AUTO, n_splits=0, filter=0, allocator=None, flags=0):
        """allocator: None (cudaMalloc / cudaFree), "torch" (every device block of the cache is a uint8 tensor from
        torch's caching allocator, kept alive until the cache is closed), or a pair of callables
        (alloc(bytes) -> device address or 0, free(address))."""
        self._lib = load_library()
        self._blocks = {}
        LogQuantCache.live.add(self)
        alloc_cb, free_cb = ALLOC_FN(0), FREE_FN(0)
        if allocator == "torch":
            import torch

            def _alloc(nbytes, _ctx):
                try:
                    t = torch.empty(max(int(nbytes), 1), dtype=torch.uint8, device=torch.device("cuda", device))
                except RuntimeError:
                    return 0
                self._blocks[t.data_ptr()] = t
                return t.data_ptr()

            def _free(ptr, _ctx):
                self._blocks.pop(ptr, None)

            alloc_cb, free_cb = ALLOC_FN(_alloc), FREE_FN(_free)
        elif allocator is not None:
            user_alloc, user_free = allocator
            alloc_cb = ALLOC_FN(lambda nbytes, _ctx: int(user_alloc(int(nbytes))) or 0)
            free_cb = FREE_FN(lambda ptr, _ctx: user_free(ptr))
        self._callbacks = (alloc_cb, free_cb)  # keep the trampolines alive as long as the cache
        self.cfg = lq_config_t(n_layers, batch, n_q_heads, n_kv_heads, head_dim, window, group, bits, max_tokens,
                               int(auto_compress), device, kernel, n_splits, filter, flags, alloc_cb, free_cb, None)
        self._h = C.c_void_p()
        self._check(self._lib.lq_cache_create(C.byref(self.cfg), C.byref(self._h)), create=True)

    def _check(self, status, create=False):
        if status != LQ_OK:
            msg = self._lib.lq_status_str(status).decode()
            if not create and status == LQ_ERR_CUDA:
                msg += ": " + self._lib.lq_last_error(self._h).decode()
            raise LogQuantError(status, msg)

    def close(self):
        if getattr(self, "_h", None):
            damaged = self.check_guards() if LogQuantCache.guards_on_close else 0
            self._lib.lq_destroy(self._h)
            self._h = None
            if damaged:
                raise LogQuantError(LQ_ERR_CUDA, "%d device block(s) of the cache were written past their end" % damaged)

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # -- the five calls -----------------------------------------------------------------
    def append(self, layer, k, v, n_tokens=None, stream=None):
        if n_tokens is None:
            n_tokens = k.shape[2]
        self._check(self._lib.lq_append(self._h, layer, _ptr(k), _ptr(v), n_tokens,
                                        None if self.cfg.device < 0 else _stream(stream)))

    def compress(self, layer=-1, stream=None):
        self._check(self._lib.lq_compress(self._h, layer, None if self.cfg.device < 0 else _stream(stream)))

    def append_decode_attn(self, layer, k, v, q, out, sm_scale=0.0, stream=None):
        """Append one token and run decode attention in one launch (k, v: [B, Hkv, 1, D] bf16)."""
        import torch
        assert k.shape[2] == 1 and v.shape == k.shape
        out_dtype = 1 if out.dtype == torch.bfloat16 else 0
        self._check(self._lib.lq_append_decode_attn(self._h, layer, _ptr(k), _ptr(v), _ptr(q), sm_scale, _ptr(out),
                                                    out_dtype, _stream(stream)))

    def decode_attn(self, layer, q, out, sm_scale=0.0, stream=None):
        import torch
        out_dtype = 1 if out.dtype == torch.bfloat16 else 0
        self._check(self._lib.lq_decode_attn(self._h, layer, _ptr(q), sm_scale, _ptr(out), out_dtype,
                                             _stream(stream)))

    def decode_attn_fp_only(self, layer, q, out, sm_scale=0.0, stream=None):
        import torch
        out_dtype = 1 if out.dtype == torch.bfloat16 else 0
        self._check(self._lib.lq_decode_attn_fp_only(self._h, layer, _ptr(q), sm_scale, _ptr(out), out_dtype,
                                                     _stream(stream)))

    def set_padding(self, pad):
        """pad: `batch` leading padding positions per sequence (any int sequence), or None to clear."""
        if pad is None:
            self._check(self._lib.lq_set_padding(self._h, None))
            return
        pad = [int(x) for x in pad]
        if len(pad) != self.cfg.batch:
            raise ValueError("one padding length per sequence of the batch")
        arr = (C.c_int32 * self.cfg.batch)(*pad)
        self._check(self._lib.lq_set_padding(self._h, C.cast(arr, C.c_void_p)))

    def decode_step_host(self, layer, k_host, v_host, q_host, out_host, sm_scale=0.0, sync=True, stream=None):
        self._check(self._lib.lq_decode_step_host(self._h, layer, _ptr(k_host), _ptr(v_host), _ptr(q_host),
                                                  sm_scale, _ptr(out_host), int(sync), _stream(stream)))

    def profile_enable(self, on=True):
        self._check(self._lib.lq_profile_enable(self._h, int(on)))

    def profile_read(self):
        ms, n = C.c_double(0), C.c_int64(0)
        self._check(self._lib.lq_profile_read(self._h, C.byref(ms), C.byref(n)))
        return ms.value, n.value

    # -- introspection --------------------------------------------------------------------
    def check_guards(self) -> int:
        """Number of device blocks whose guard bytes were overwritten (lq_check_guards; synchronises)."""
        n = C.c_int32(0)
        self._check(self._lib.lq_check_guards(self._h, C.byref(n)))
        return n.value

    def reset_kernel_status(self):
        self._check(self._lib.lq_reset_kernel_status(self._h))

    def debug_bad_slot_next_append(self):
        self._check(self._lib.lq_debug_bad_slot_next_append(self._h))

    def debug_stall_next_decode(self):
        self._check(self._lib.lq_debug_stall_next_decode(self._h))

    def kernel_status(self) -> int:
        w = C.c_int32(0)
        self._check(self._lib.lq_kernel_status(self._h, C.byref(w)))
        return w.value

    def info_fast(self, layer=0):
        """(n_quant, n_fp) of one layer."""
        inf = self.info(layer)
        return inf.n_quant, inf.n_fp

    def info(self, layer=0) -> lq_info_t:
        info = lq_info_t()
        self._check(self._lib.lq_cache_info(self._h, layer, C.byref(info)))
        return info

    def next_evicted_ids(self, layer=0) -> np.ndarray:
        ids = np.zeros(self.cfg.window, np.int32)
        self._check(self._lib.lq_next_evicted_ids(self._h, layer, ids.ctypes.data))
        return ids

    def export(self, layer=0, ids_only=False) -> dict:
        """Canonical image of one layer as numpy arrays (see include/lq.h)."""
        c, inf = self.cfg, self.info(layer)
        B, H, D, G, nf, nq = c.batch, c.n_kv_heads, c.head_dim, c.group, inf.n_fp, inf.n_quant
        img = dict(kept_ids=np.zeros(nf, np.int32), quant_ids=np.zeros(nq, np.int32))
        if not ids_only:
            img.update(
                k_codes=np.zeros((B, H, nq, D * self.cfg.bits // 8), np.uint8),
                v_codes=np.zeros((B, H, nq, D * self.cfg.bits // 8), np.uint8),
                k_scale=np.zeros((B, H, nq // G, D), np.uint16), k_zero=np.zeros((B, H, nq // G, D), np.uint16),
                v_scale=np.zeros((B, H, nq, D // G), np.uint16), v_zero=np.zeros((B, H, nq, D // G), np.uint16),
                fp_k=np.zeros((B, H, nf, D), np.uint16), fp_v=np.zeros((B, H, nf, D), np.uint16))
        st = lq_image_t(**{k: (v.ctypes.data if v.size else None) for k, v in img.items()})
        self._check(self._lib.lq_export(self._h, layer, C.byref(st)))
        return img

    def import_image(self, layer, img: dict, n_seen: int):
        """lq_import: load an image made by export() into an empty layer (sizes are taken from the arrays)."""
        arrs = {k: np.ascontiguousarray(v) for k, v in img.items()}
        st = lq_image_t(**{k: (v.ctypes.data if v.size else None) for k, v in arrs.items()})
        self._check(self._lib.lq_import(self._h, layer, C.byref(st), int(n_seen), int(arrs["kept_ids"].size),
                                        int(arrs["quant_ids"].size)))

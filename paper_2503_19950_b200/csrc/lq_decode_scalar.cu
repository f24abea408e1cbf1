// Plain fp32 decode attention over the mixed cache (LQ_KERNEL_SCALAR) and the split-K merge.
//
// The scalar kernel is the simplest possible CUDA statement of Eq. 2 on the device layout: one
// thread per token for q.k, one thread per channel for p.v, every element fetched through the
// layout's addressing functions and dequantised as zero + code*scale in fp32.  It exists as a
// slow, independent cross-check of the tensor-core kernel and is never the default.
#include <cuda_bf16.h>

#include "lq_kernels.cuh"

namespace lq {

namespace {

__device__ __forceinline__ float bf16f(uint16_t b) { return __uint_as_float(static_cast<uint32_t>(b) << 16); }

struct TokenRef {  // where token t of the unified index space [fp tokens | quantised tokens] lives
  const uint8_t* fp;    // head base of the fp store
  const uint8_t* quant; // head base of the 2-bit store
  int n_fp;
  int G;
  int P;  // 2-bit planes per code
  int layout;
};

__device__ __forceinline__ float load_k(const TokenRef& r, int64_t t, int d) {
  if (t < r.n_fp) return bf16f(*reinterpret_cast<const uint16_t*>(r.fp + fp_elem_off(r.layout, static_cast<int>(t), d)));
  const int64_t tq = t - r.n_fp;
  const uint8_t* tile = r.quant + (tq / r.G) * quant_tile_bytes(r.G, r.P);
  uint32_t code = 0;
  for (int pl = 0; pl < r.P; ++pl) {
    int off, bit;
    kcode_pos(r.layout, r.G, r.P, pl, static_cast<int>(tq % r.G), d, off, bit);
    code |= ((*reinterpret_cast<const uint32_t*>(tile + off) >> bit) & 3u) << (2 * pl);
  }
  const float s = bf16f(*reinterpret_cast<const uint16_t*>(tile + kscale_off(r.layout, r.G, d)));
  const float z = bf16f(*reinterpret_cast<const uint16_t*>(tile + kzero_off(r.layout, r.G, d)));
  return fmaf(static_cast<float>(code), s, z);
}

__device__ __forceinline__ float load_v(const TokenRef& r, int64_t t, int d) {
  if (t < r.n_fp)
    return bf16f(*reinterpret_cast<const uint16_t*>(r.fp + fp_v_delta(r.layout) + fp_elem_off(r.layout, static_cast<int>(t), d)));
  const int64_t tq = t - r.n_fp;
  const uint8_t* tile = r.quant + (tq / r.G) * quant_tile_bytes(r.G, r.P);
  const int tt = static_cast<int>(tq % r.G);
  uint32_t code = 0;
  for (int pl = 0; pl < r.P; ++pl) {
    int off, bit;
    vcode_pos(r.layout, r.G, r.P, pl, tt, d, off, bit);
    code |= ((*reinterpret_cast<const uint32_t*>(tile + off) >> bit) & 3u) << (2 * pl);
  }
  const int g = d / r.G;
  const float s = bf16f(*reinterpret_cast<const uint16_t*>(tile + vscale_off(r.layout, r.G, r.P, tt, g)));
  const float z = bf16f(*reinterpret_cast<const uint16_t*>(tile + vzero_off(r.layout, r.G, r.P, tt, g)));
  return fmaf(static_cast<float>(code), s, z);
}

}  // namespace

__global__ void __launch_bounds__(128) lq_decode_scalar_kernel(DecodeArgs a) {
  const CacheView& cv = a.cv;
  const int r = cv.Hq / cv.Hkv;
  const int S = a.S;
  const int64_t pair = blockIdx.x / S;
  const int s = blockIdx.x % S;
  const int b = static_cast<int>(pair / cv.Hkv), kv = static_cast<int>(pair % cv.Hkv);
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

  __shared__ float sq[kMaxRatio][kD];
  __shared__ float sp[kMaxRatio][128];
  __shared__ float red[4][kMaxRatio];

  const __nv_bfloat16* q = static_cast<const __nv_bfloat16*>(a.q);
  for (int j = 0; j < r; ++j)
    sq[j][tid] = __bfloat162float(q[(static_cast<int64_t>(b) * cv.Hq + kv * r + j) * kD + tid]) * a.scale_log2;
  __syncthreads();

  TokenRef ref;
  ref.fp = cv.fp + a.layer * cv.fp_layer_stride + pair * cv.fp_head_stride;
  ref.quant = cv.quant + a.layer * cv.quant_layer_stride + pair * cv.quant_head_stride;
  ref.n_fp = a.n_fp;
  ref.G = cv.G;
  ref.P = cv.planes;
  ref.layout = cv.layout;

  const int64_t T = a.n_fp + a.n_quant;
  const int64_t chunk = (T + S - 1) / S;
  const int64_t begin = s * chunk;
  const int64_t end = begin + chunk < T ? begin + chunk : T;

  float m[kMaxRatio], l[kMaxRatio], acc[kMaxRatio];
#pragma unroll
  for (int j = 0; j < kMaxRatio; ++j) { m[j] = -INFINITY; l[j] = 0.f; acc[j] = 0.f; }

  // left padding: bit set = attention leaves the token out
  const uint32_t* fpmask = a.fpmask ? a.fpmask + static_cast<int64_t>(b) * a.fpmask_words : nullptr;
  const uint32_t* qmask = a.qmask ? a.qmask + static_cast<int64_t>(b) * a.qmask_words : nullptr;
  auto is_padding = [&](int64_t t) {
    if (t < a.n_fp) return fpmask != nullptr && ((fpmask[t >> 5] >> (t & 31)) & 1u) != 0u;
    const int64_t tq = t - a.n_fp;
    return qmask != nullptr && ((qmask[tq >> 5] >> (tq & 31)) & 1u) != 0u;
  };

  for (int64_t t0 = begin; t0 < end; t0 += 128) {
    const int64_t t = t0 + tid;
    const bool valid = t < end && !is_padding(t);
    float sc[kMaxRatio];
#pragma unroll
    for (int j = 0; j < kMaxRatio; ++j) sc[j] = 0.f;
    if (valid) {
      for (int d = 0; d < kD; ++d) {
        const float kval = load_k(ref, t, d);
#pragma unroll
        for (int j = 0; j < kMaxRatio; ++j)
          if (j < r) sc[j] = fmaf(sq[j][d], kval, sc[j]);
      }
    }
    // block max per head
#pragma unroll
    for (int j = 0; j < kMaxRatio; ++j) {
      float v = valid ? sc[j] : -INFINITY;
      for (int o = 16; o; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xFFFFFFFFu, v, o));
      if (lane == 0) red[warp][j] = v;
    }
    __syncthreads();
    float corr[kMaxRatio];
#pragma unroll
    for (int j = 0; j < kMaxRatio; ++j) {
      const float bm = fmaxf(fmaxf(red[0][j], red[1][j]), fmaxf(red[2][j], red[3][j]));
      const float mn = fmaxf(m[j], bm);
      corr[j] = (m[j] == -INFINITY) ? 0.f : exp2f(m[j] - mn);
      m[j] = mn;
      sp[j][tid] = (valid && j < r) ? exp2f(sc[j] - mn) : 0.f;
    }
    __syncthreads();
    // p.v : thread tid owns channel d = tid
    const int nt = static_cast<int>(end - t0 < 128 ? end - t0 : 128);
    float add[kMaxRatio], lsum[kMaxRatio];
#pragma unroll
    for (int j = 0; j < kMaxRatio; ++j) { add[j] = 0.f; lsum[j] = 0.f; }
    for (int tt = 0; tt < nt; ++tt) {
      const float vv = load_v(ref, t0 + tt, tid);
#pragma unroll
      for (int j = 0; j < kMaxRatio; ++j)
        if (j < r) {
          const float p = sp[j][tt];
          add[j] = fmaf(p, vv, add[j]);
          lsum[j] += p;
        }
    }
#pragma unroll
    for (int j = 0; j < kMaxRatio; ++j) {
      acc[j] = acc[j] * corr[j] + add[j];
      l[j] = l[j] * corr[j] + lsum[j];
    }
    __syncthreads();
  }

  const int64_t rec = (pair * S + s) * r;
  for (int j = 0; j < r; ++j) {
    a.part_o[(rec + j) * kD + tid] = acc[j];
    if (tid == 0) {
      a.part_ml[(rec + j) * 2 + 0] = m[j];
      a.part_ml[(rec + j) * 2 + 1] = l[j];
    }
  }
}

cudaError_t launch_decode_scalar(const DecodeArgs& a, cudaStream_t st) {
  const int blocks = a.cv.B * a.cv.Hkv * a.S;
  lq_decode_scalar_kernel<<<blocks, 128, 0, st>>>(a);
  return cudaGetLastError();
}

// ---------------------------------------------------------------------------------------
// Split-K merge (second pass): m = max_s m_s, l = sum_s l_s 2^{m_s-m},
// out = sum_s o_s 2^{m_s-m} / l.  One CTA per (b, query head), one thread per channel.
// Partitions that saw no token carry l = 0 and are skipped.
// ---------------------------------------------------------------------------------------
__global__ void __launch_bounds__(128) lq_merge_kernel(DecodeArgs a) {
  const CacheView& cv = a.cv;
  const int r = cv.Hq / cv.Hkv;
  const int b = blockIdx.x / cv.Hq, h = blockIdx.x % cv.Hq;
  const int64_t pair = static_cast<int64_t>(b) * cv.Hkv + h / r;
  const int j = h % r;
  const int d = threadIdx.x;
  const int count = a.S;
  float M = -INFINITY;
  for (int s = 0; s < count; ++s) {
    const int64_t rec = (pair * a.S + s) * r + j;
    if (a.part_ml[rec * 2 + 1] > 0.f) M = fmaxf(M, a.part_ml[rec * 2]);
  }
  float L = 0.f, o = 0.f;
  for (int s = 0; s < count; ++s) {
    const int64_t rec = (pair * a.S + s) * r + j;
    const float ls = a.part_ml[rec * 2 + 1];
    if (ls > 0.f) {
      const float w = exp2f(a.part_ml[rec * 2] - M);
      L = fmaf(ls, w, L);
      o = fmaf(a.part_o[rec * kD + d], w, o);
    }
  }
  const float res = o / L;
  const int64_t oi = (static_cast<int64_t>(b) * cv.Hq + h) * kD + d;
  if (a.out_bf16)
    static_cast<__nv_bfloat16*>(a.out)[oi] = __float2bfloat16_rn(res);
  else
    static_cast<float*>(a.out)[oi] = res;
}

cudaError_t launch_merge(const DecodeArgs& a, cudaStream_t st) {
  lq_merge_kernel<<<a.cv.B * a.cv.Hq, 128, 0, st>>>(a);
  return cudaGetLastError();
}

}  // namespace lq

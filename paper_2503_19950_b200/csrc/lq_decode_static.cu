// Decode attention over a caller-owned cache image, with no allocation anywhere.
//
// Some users of this library are not allowed to allocate device memory: a serving process that
// carved its whole memory budget into a fixed arena at start-up, a plugin running inside someone
// else's allocator policy, or code that is called while a CUDA stream is being captured (where
// cudaMalloc is illegal).  lq_cache_create cannot serve them, because it allocates the stores and the
// split-K workspace.  This entry point takes the two stores as plain device arrays in the canonical
// image format of include/lq.h (wherever the caller keeps them) and keeps its only scratch -- the
// split-K partial results -- in a fixed array that is part of the library image itself.
//
// It is a variant of the plain fp32 split-K kernel (thread per token for q.k, thread per channel for
// p.v, dequantisation as zero + code * scale), reading the canonical layout instead of the private one.
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include "../../include/lq.h"

namespace {

constexpr int kD = 128;
constexpr int kMaxR = 8;
constexpr int kStaticMaxRecords = 8192;  // (batch row, query head, split) partials that fit the scratch
constexpr int kRecordFloats = kD + 2;    // o[128], m, l

// Split-K scratch.  Every GPU that loads the library holds these 4.06 MiB until the process exits.
// In host code this name is only a handle for cudaGetSymbolAddress, never a device address.
static __device__ __align__(256) float g_static_partials[kStaticMaxRecords * kRecordFloats];

struct ImageArgs {
  int B, Hq, Hkv, G, n_fp, S;
  int bits;  // 2 or 4: width of a code in k_codes / v_codes
  long long n_quant;
  const uint16_t *fp_k, *fp_v, *k_scale, *k_zero, *v_scale, *v_zero;
  const uint8_t *k_codes, *v_codes;
  const __nv_bfloat16* q;
  float scale_log2;
  float* partials;
  float* out;
};

__device__ __forceinline__ float bf16f(uint16_t b) { return __uint_as_float(static_cast<uint32_t>(b) << 16); }

// code of channel d of token row `row` in the canonical packing: 8 / bits codes per byte, channel (8/bits)*j + i of
// a token in bits [bits*i + bits - 1 : bits*i] of byte j
__device__ __forceinline__ uint32_t image_code(const uint8_t* codes, int bits, long long row, int d) {
  const int per_byte = 8 / bits;
  return (codes[row * (kD / per_byte) + d / per_byte] >> (bits * (d % per_byte))) & ((1u << bits) - 1u);
}

__device__ __forceinline__ float image_k(const ImageArgs& a, long long pair, long long t, int d) {
  if (t < a.n_fp) return bf16f(a.fp_k[(pair * a.n_fp + t) * kD + d]);
  const long long tq = t - a.n_fp;
  const uint32_t code = image_code(a.k_codes, a.bits, pair * a.n_quant + tq, d);
  const long long grp = (pair * (a.n_quant / a.G) + tq / a.G) * kD + d;
  return fmaf(static_cast<float>(code), bf16f(a.k_scale[grp]), bf16f(a.k_zero[grp]));
}

__device__ __forceinline__ float image_v(const ImageArgs& a, long long pair, long long t, int d) {
  if (t < a.n_fp) return bf16f(a.fp_v[(pair * a.n_fp + t) * kD + d]);
  const long long tq = t - a.n_fp;
  const uint32_t code = image_code(a.v_codes, a.bits, pair * a.n_quant + tq, d);
  const long long grp = (pair * a.n_quant + tq) * (kD / a.G) + d / a.G;
  return fmaf(static_cast<float>(code), bf16f(a.v_scale[grp]), bf16f(a.v_zero[grp]));
}

// One CTA per (b, kv head, split); partial record of query head h and split s at ((b*Hq + h)*S + s).
__global__ void __launch_bounds__(128) lq_image_split_kernel(ImageArgs a) {
  const int r = a.Hq / a.Hkv;
  const long long pair = blockIdx.x / a.S;
  const int s = blockIdx.x % a.S;
  const int b = static_cast<int>(pair / a.Hkv), kv = static_cast<int>(pair % a.Hkv);
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  __shared__ float sq[kMaxR][kD];
  __shared__ float sp[kMaxR][128];
  __shared__ float red[4][kMaxR];
  for (int j = 0; j < r; ++j)
    sq[j][tid] = __bfloat162float(a.q[(static_cast<long long>(b) * a.Hq + kv * r + j) * kD + tid]) * a.scale_log2;
  __syncthreads();
  const long long T = a.n_fp + a.n_quant;
  const long long chunk = (T + a.S - 1) / a.S;
  const long long begin = s * chunk;
  const long long end = begin + chunk < T ? begin + chunk : T;
  float m[kMaxR], l[kMaxR], acc[kMaxR];
#pragma unroll
  for (int j = 0; j < kMaxR; ++j) { m[j] = -INFINITY; l[j] = 0.f; acc[j] = 0.f; }
  for (long long t0 = begin; t0 < end; t0 += 128) {
    const long long t = t0 + tid;
    const bool valid = t < end;
    float sc[kMaxR];
#pragma unroll
    for (int j = 0; j < kMaxR; ++j) sc[j] = 0.f;
    if (valid)
      for (int d = 0; d < kD; ++d) {
        const float kval = image_k(a, pair, t, d);
#pragma unroll
        for (int j = 0; j < kMaxR; ++j)
          if (j < r) sc[j] = fmaf(sq[j][d], kval, sc[j]);
      }
#pragma unroll
    for (int j = 0; j < kMaxR; ++j) {
      float v = valid ? sc[j] : -INFINITY;
      for (int o = 16; o; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xFFFFFFFFu, v, o));
      if (lane == 0) red[warp][j] = v;
    }
    __syncthreads();
    float corr[kMaxR];
#pragma unroll
    for (int j = 0; j < kMaxR; ++j) {
      const float bm = fmaxf(fmaxf(red[0][j], red[1][j]), fmaxf(red[2][j], red[3][j]));
      const float mn = fmaxf(m[j], bm);
      corr[j] = (m[j] == -INFINITY) ? 0.f : exp2f(m[j] - mn);
      m[j] = mn;
      sp[j][tid] = (valid && j < r) ? exp2f(sc[j] - mn) : 0.f;
    }
    __syncthreads();
    const int nt = static_cast<int>(end - t0 < 128 ? end - t0 : 128);
    float add[kMaxR], lsum[kMaxR];
#pragma unroll
    for (int j = 0; j < kMaxR; ++j) { add[j] = 0.f; lsum[j] = 0.f; }
    for (int tt = 0; tt < nt; ++tt) {
      const float vv = image_v(a, pair, t0 + tt, tid);
#pragma unroll
      for (int j = 0; j < kMaxR; ++j)
        if (j < r) {
          add[j] = fmaf(sp[j][tt], vv, add[j]);
          lsum[j] += sp[j][tt];
        }
    }
#pragma unroll
    for (int j = 0; j < kMaxR; ++j) {
      acc[j] = acc[j] * corr[j] + add[j];
      l[j] = l[j] * corr[j] + lsum[j];
    }
    __syncthreads();
  }
  // every record of this call is written here before the merge reads it: nothing in the scratch
  // has to start at zero, and whatever the previous call left behind is simply overwritten
  for (int j = 0; j < r; ++j) {
    float* rec = a.partials + ((static_cast<long long>(b) * a.Hq + kv * r + j) * a.S + s) * kRecordFloats;
    rec[tid] = acc[j];
    if (tid == 0) { rec[kD] = m[j]; rec[kD + 1] = l[j]; }
  }
}

__global__ void __launch_bounds__(128) lq_image_merge_kernel(ImageArgs a) {
  const long long bh = blockIdx.x;
  const int d = threadIdx.x;
  const float* rec0 = a.partials + bh * a.S * kRecordFloats;
  float M = -INFINITY;
  for (int s = 0; s < a.S; ++s)
    if (rec0[s * kRecordFloats + kD + 1] > 0.f) M = fmaxf(M, rec0[s * kRecordFloats + kD]);
  float L = 0.f, o = 0.f;
  for (int s = 0; s < a.S; ++s) {
    const float ls = rec0[s * kRecordFloats + kD + 1];
    if (ls > 0.f) {
      const float w = exp2f(rec0[s * kRecordFloats + kD] - M);
      L = fmaf(ls, w, L);
      o = fmaf(rec0[s * kRecordFloats + d], w, o);
    }
  }
  a.out[bh * kD + d] = o / L;
}

// device address of the scratch, looked up once per device (index = CUDA device ordinal)
float* g_partials_ptr[64] = {};

}  // namespace

extern "C" lq_status_t lq_decode_attn_image_static(const lq_device_image_t* img, const void* q, float sm_scale,
                                                   float* out, void* stream) {
  if (!img || !q || !out) return LQ_ERR_INVALID_ARG;
  if (img->batch < 1 || img->n_q_heads < 1 || img->n_kv_heads < 1 || img->n_q_heads % img->n_kv_heads ||
      img->n_fp < 0 || img->n_quant < 0 || img->n_fp + img->n_quant < 1)
    return LQ_ERR_INVALID_ARG;
  if (img->bits != 2 && img->bits != 4) return LQ_ERR_INVALID_ARG;
  if (img->head_dim != kD || (img->group != 32 && img->group != 64) || img->n_q_heads / img->n_kv_heads > kMaxR ||
      img->n_quant % img->group)
    return LQ_ERR_UNSUPPORTED;
  if ((img->n_fp > 0 && (!img->fp_k || !img->fp_v)) ||
      (img->n_quant > 0 && (!img->k_codes || !img->v_codes || !img->k_scale || !img->k_zero || !img->v_scale || !img->v_zero)))
    return LQ_ERR_INVALID_ARG;

  // split count: about 512 tokens per partial, at most 16, and never more records than the scratch holds
  const long long heads = static_cast<long long>(img->batch) * img->n_q_heads;
  if (heads > kStaticMaxRecords) return LQ_ERR_CAPACITY;
  long long S = (img->n_fp + img->n_quant + 511) / 512;
  if (S > 16) S = 16;
  if (S > kStaticMaxRecords / heads) S = kStaticMaxRecords / heads;
  if (S < 1) S = 1;

  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return LQ_ERR_CUDA;
  if (!g_partials_ptr[dev]) {
    // first call on this device: resolve the device address of the scratch (the host-side name of a
    // __device__ array is not one).  Not legal during stream capture, hence "call once before".
    float* p = nullptr;
    if (cudaGetSymbolAddress(reinterpret_cast<void**>(&p), g_static_partials) != cudaSuccess || !p) {
      cudaGetLastError();
      return LQ_ERR_CUDA;
    }
    g_partials_ptr[dev] = p;
  }

  ImageArgs a;
  a.B = img->batch; a.Hq = img->n_q_heads; a.Hkv = img->n_kv_heads; a.G = img->group; a.bits = img->bits;
  a.n_fp = img->n_fp; a.n_quant = img->n_quant; a.S = static_cast<int>(S);
  a.fp_k = img->fp_k; a.fp_v = img->fp_v; a.k_codes = img->k_codes; a.v_codes = img->v_codes;
  a.k_scale = img->k_scale; a.k_zero = img->k_zero; a.v_scale = img->v_scale; a.v_zero = img->v_zero;
  a.q = static_cast<const __nv_bfloat16*>(q);
  if (!(sm_scale > 0.f)) sm_scale = 0.08838834764831845f;  // 1/sqrt(128)
  a.scale_log2 = sm_scale * 1.4426950408889634f;
  a.partials = g_partials_ptr[dev];
  a.out = out;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  lq_image_split_kernel<<<img->batch * img->n_kv_heads * a.S, 128, 0, st>>>(a);
  if (cudaGetLastError() != cudaSuccess) return LQ_ERR_CUDA;
  lq_image_merge_kernel<<<static_cast<unsigned>(heads), 128, 0, st>>>(a);
  if (cudaGetLastError() != cudaSuccess) return LQ_ERR_CUDA;
  return LQ_OK;
}

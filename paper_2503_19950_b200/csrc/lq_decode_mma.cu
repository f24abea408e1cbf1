// Tensor-core decode attention over the mixed cache (LQ_KERNEL_MMA): split-K first pass.
//
// One CTA = one (b, kv head, split); 4 warps, each with a private ring of shared-memory stages
// filled by 1-D bulk copies (cp.async.bulk + mbarrier, no multicast).  A warp walks its own
// contiguous range of "units" -- fp tiles (16 bf16 tokens, 8 KB) first, then quant units (one or
// two key groups) -- and keeps a private online-softmax state (m, l, o) that the CTA merges at
// the end into one split-K partial (Eq. 3 makes any visiting order legal).
//
// Contractions (mma.sync.m16n8k16, fp32 accumulate), r = query heads per KV head (<= 8):
//   q.k   tokens on M (16), query heads on N, channels on K.  Heads are handled in column blocks
//         of 4: column 2h' = "hi", 2h'+1 = "lo" of head 4cb+h'.
//         2-bit keys: the A fragment is the packed word masked at one code position -- a bf16
//         subnormal c*2^(p-133) -- so unpacking costs one AND per two codes.  The key scale is
//         folded into the query: q*s is split exactly into bf16 hi + lo with one packed multiply
//         and one packed fma (both have 8-bit significands), so q.k^ is exact up to fp32
//         accumulation.  The key zero contributes q.z per group, computed by 8 MMAs per group.
//         bf16 keys: ldmatrix fragments of the swizzled rows, bf16 x bf16 exact.
//   p.v   channels on M (16), heads on N (8), tokens on K.  2-bit values: fp16 subnormal codes
//         c*2^(p-24) times p*s_v rounded to fp16; the value zero goes through one extra MMA per
//         16 tokens.  bf16 values: ldmatrix.trans fragments times p split into bf16 hi + lo.
//   The softmax probabilities come out of q.k with (token, head) = (lane/4, lane%4) and are
//   moved to the (head, token pair) arrangement p.v needs with 4 warp shuffles per 16 tokens.
#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include "lq_kernels.cuh"

namespace lq {

namespace {

constexpr int kWarps = 4;
constexpr int kStageBytes = 8192;
constexpr int kStages = 2;
constexpr uint32_t kFull = 0xFFFFFFFFu;
constexpr int kSpinLimit = 1 << 22;

// ---- PTX wrappers ----------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ uint32_t mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok;
}
__device__ __forceinline__ void bulk_load(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst),
               "l"(src), "r"(bytes), "r"(bar)
               : "memory");
}
__device__ __forceinline__ void mma_bf16(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                         uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ void mma_f16(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                        uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ void ldmatrix_x4(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3)
               : "r"(addr));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2,
                                                  uint32_t& r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3)
               : "r"(addr));
}
__device__ __forceinline__ uint32_t bf16x2_mul(uint32_t a, uint32_t b) {
  uint32_t d;
  asm("mul.rn.bf16x2 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));
  return d;
}
__device__ __forceinline__ uint32_t bf16x2_fma(uint32_t a, uint32_t b, uint32_t c) {
  uint32_t d;
  asm("fma.rn.bf16x2 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(c));
  return d;
}
// pack two floats: `lo` into bits [15:0], `hi` into bits [31:16]
__device__ __forceinline__ uint32_t pack_f16x2(float lo, float hi) {
  uint32_t d;
  asm("cvt.rn.f16x2.f32 %0, %1, %2;" : "=r"(d) : "f"(hi), "f"(lo));
  return d;
}
__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
  uint32_t d;
  asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(d) : "f"(hi), "f"(lo));
  return d;
}
__device__ __forceinline__ float bf16lo_f32(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16hi_f32(uint32_t w) { return __uint_as_float(w & 0xFFFF0000u); }
__device__ __forceinline__ uint4 lds128(uint32_t addr) {
  uint4 v;
  asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr));
  return v;
}
__device__ __forceinline__ uint2 lds64(uint32_t addr) {
  uint2 v;
  asm volatile("ld.shared.v2.u32 {%0,%1}, [%2];" : "=r"(v.x), "=r"(v.y) : "r"(addr));
  return v;
}

// one code position of a packed word as two bf16 (key) / fp16 (value) subnormals
template <int KS>
__device__ __forceinline__ uint32_t kext(uint32_t w, uint32_t w8) {
  return KS < 4 ? (w & (0x00030003u << (2 * KS))) : (w8 & (0x00030003u << (2 * (KS - 4))));
}
template <int MT>
__device__ __forceinline__ uint32_t vext(uint32_t w, uint32_t w10) {
  return MT < 5 ? (w & (0x00030003u << (2 * MT))) : (w10 & (0x00030003u << (2 * (MT - 5))));
}

template <int NCB>
struct WarpState {
  float out[8][4];  // o^T: [channel tile][c-fragment]; columns = query heads
  float zacc[4];    // sum_t p_t * vzero_t per (value group, head)
  float m[NCB];     // running max (log2 units) of head 4cb + lane%4
  float l[NCB];     // this lane's share of the running denominator
  bool quant_mode;  // out rows carry the code-position factor 2^(p(mt)-24)
};

// factor carried by the out rows of channel tile mt while in quant mode
__device__ __forceinline__ float vpos_scale(int mt) { return exp2f(static_cast<float>(2 * (mt < 5 ? mt : mt - 5) - 24)); }

// ---- online softmax on the 16 scores a lane quad column holds, then p in p.v arrangement ----
// s[cb][th]: score (log2 units) of token 8*th + lane/4 for head 4cb + lane%4.
// Returns pT[th][i]: probability of token 8*th + 2*(lane%4) + i for head lane/4.
template <int NCB>
__device__ __forceinline__ void softmax_step(WarpState<NCB>& st, float (&s)[NCB][2], float (&pT)[2][2], int lane) {
  const int n = lane >> 2, j = lane & 3;
  float corr[NCB];
  bool changed = false;
#pragma unroll
  for (int cb = 0; cb < NCB; ++cb) {
    float mx = fmaxf(s[cb][0], s[cb][1]);
    mx = fmaxf(mx, __shfl_xor_sync(kFull, mx, 4));
    mx = fmaxf(mx, __shfl_xor_sync(kFull, mx, 8));
    mx = fmaxf(mx, __shfl_xor_sync(kFull, mx, 16));
    const float mn = fmaxf(st.m[cb], mx);
    changed |= mn > st.m[cb];
    corr[cb] = exp2f(st.m[cb] - mn);  // m = -inf initially -> 0
    st.m[cb] = mn;
  }
  if (__any_sync(kFull, changed)) {
    float ca, cbv;
    if (NCB == 1) {
      ca = __shfl_sync(kFull, corr[0], (2 * j) & 3);
      cbv = __shfl_sync(kFull, corr[0], (2 * j + 1) & 3);
    } else {
      const float a0 = __shfl_sync(kFull, corr[0], (2 * j) & 3), a1 = __shfl_sync(kFull, corr[NCB - 1], (2 * j) & 3);
      const float b0 = __shfl_sync(kFull, corr[0], (2 * j + 1) & 3), b1 = __shfl_sync(kFull, corr[NCB - 1], (2 * j + 1) & 3);
      ca = j >= 2 ? a1 : a0;
      cbv = j >= 2 ? b1 : b0;
    }
#pragma unroll
    for (int mt = 0; mt < 8; ++mt) {
      st.out[mt][0] *= ca; st.out[mt][1] *= cbv; st.out[mt][2] *= ca; st.out[mt][3] *= cbv;
    }
    st.zacc[0] *= ca; st.zacc[1] *= cbv; st.zacc[2] *= ca; st.zacc[3] *= cbv;
#pragma unroll
    for (int cb = 0; cb < NCB; ++cb) st.l[cb] *= corr[cb];
  }
  float p[NCB][2];
#pragma unroll
  for (int cb = 0; cb < NCB; ++cb) {
    p[cb][0] = exp2f(s[cb][0] - st.m[cb]);
    p[cb][1] = exp2f(s[cb][1] - st.m[cb]);
    st.l[cb] += p[cb][0] + p[cb][1];
  }
#pragma unroll
  for (int th = 0; th < 2; ++th)
#pragma unroll
    for (int i = 0; i < 2; ++i) {
      const int src = 4 * (2 * j + i) + (n & 3);
      float v = __shfl_sync(kFull, p[0][th], src);
      if (NCB == 2) {
        const float v1 = __shfl_sync(kFull, p[NCB - 1][th], src);
        v = (n >> 2) ? v1 : v;
      }
      pT[th][i] = v;
    }
}

// ---- one fp tile: 16 bf16 tokens (rows swizzled in 16-byte chunks by row & 7) -------------
template <int NCB>
__device__ __forceinline__ void process_fp_tile(WarpState<NCB>& st, const uint32_t (&qs)[NCB][8][2], uint32_t tile,
                                                int n_valid, const float (&kc)[4], int lane) {
  const int n = lane >> 2;
  float acc[NCB][4][4];
#pragma unroll
  for (int cb = 0; cb < NCB; ++cb)
#pragma unroll
    for (int c = 0; c < 4; ++c)
#pragma unroll
      for (int e = 0; e < 4; ++e) acc[cb][c][e] = 0.f;
  {
    const int mi = lane >> 3, rr = lane & 7;
    const int token = rr + 8 * (mi & 1);
    const uint32_t rowaddr = tile + token * 256;
#pragma unroll
    for (int ks = 0; ks < 8; ++ks) {
      const int chunk = 2 * ks + (mi >> 1);
      uint32_t a0, a1, a2, a3;
      ldmatrix_x4(rowaddr + ((chunk ^ (token & 7)) << 4), a0, a1, a2, a3);
#pragma unroll
      for (int cb = 0; cb < NCB; ++cb) mma_bf16(acc[cb][ks & 3], a0, a1, a2, a3, qs[cb][ks][0], qs[cb][ks][1]);
    }
  }
  float s[NCB][2];
#pragma unroll
  for (int cb = 0; cb < NCB; ++cb) {
    float s0 = acc[cb][0][0] * kc[0], s1 = acc[cb][0][2] * kc[0];
#pragma unroll
    for (int c = 1; c < 4; ++c) {
      s0 = fmaf(acc[cb][c][0], kc[c], s0);
      s1 = fmaf(acc[cb][c][2], kc[c], s1);
    }
    s[cb][0] = n < n_valid ? s0 : -INFINITY;
    s[cb][1] = n + 8 < n_valid ? s1 : -INFINITY;
  }
  float pT[2][2];
  softmax_step<NCB>(st, s, pT, lane);
  // p split into bf16 hi + lo
  uint32_t bhi[2], blo[2];
#pragma unroll
  for (int th = 0; th < 2; ++th) {
    bhi[th] = pack_bf16x2(pT[th][0], pT[th][1]);
    blo[th] = pack_bf16x2(pT[th][0] - bf16lo_f32(bhi[th]), pT[th][1] - bf16hi_f32(bhi[th]));
  }
  {
    const int mi = lane >> 3, rr = lane & 7;
    const int token = rr + 8 * (mi >> 1);
    const uint32_t rowaddr = tile + kFpTileVOffset + token * 256;
#pragma unroll
    for (int mt = 0; mt < 8; ++mt) {
      const int chunk = 2 * mt + (mi & 1);
      uint32_t a0, a1, a2, a3;
      ldmatrix_x4_trans(rowaddr + ((chunk ^ (token & 7)) << 4), a0, a1, a2, a3);
      mma_bf16(st.out[mt], a0, a1, a2, a3, bhi[0], bhi[1]);
      mma_bf16(st.out[mt], a0, a1, a2, a3, blo[0], blo[1]);
    }
  }
}

// ---- one quant tile: one key group of G tokens ---------------------------------------------
template <int G, int NCB>
__device__ __forceinline__ void process_quant_tile(WarpState<NCB>& st, const uint32_t (&qs)[NCB][8][2], uint32_t tile,
                                                   const float (&kc)[4], float kq, int lane) {
  constexpr int NS = G / 16, NG = kD / G, VS = vsz_subtile_bytes(G);
  const int n = lane >> 2, j = lane & 3;
  // q*s split into hi (even columns) / lo (odd columns), and the bias q.z of the group
  uint32_t bq[NCB][8][2];
  float bias[NCB];
  {
    float accb[NCB][4][4];
#pragma unroll
    for (int cb = 0; cb < NCB; ++cb)
#pragma unroll
      for (int c = 0; c < 4; ++c)
#pragma unroll
        for (int e = 0; e < 4; ++e) accb[cb][c][e] = 0.f;
    const bool odd = n & 1;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const uint4 sw = lds128(tile + qt_kscale_off() + 16 * (4 * i + j));
      const uint4 zw = lds128(tile + qt_kzero_off() + 16 * (4 * i + j));
      const uint32_t s4[4] = {sw.x, sw.y, sw.z, sw.w};
      const uint32_t z4[4] = {zw.x, zw.y, zw.z, zw.w};
#pragma unroll
      for (int kk = 0; kk < 2; ++kk) {
        const int ks = 2 * i + kk;
#pragma unroll
        for (int cb = 0; cb < NCB; ++cb) {
#pragma unroll
          for (int w = 0; w < 2; ++w) {
            const uint32_t hi = bf16x2_mul(qs[cb][ks][w], s4[2 * kk + w]);
            const uint32_t lo = bf16x2_fma(qs[cb][ks][w], s4[2 * kk + w], hi ^ 0x80008000u);
            bq[cb][ks][w] = odd ? lo : hi;
          }
          mma_bf16(accb[cb][ks & 3], z4[2 * kk], z4[2 * kk], z4[2 * kk + 1], z4[2 * kk + 1], qs[cb][ks][0],
                   qs[cb][ks][1]);
        }
      }
    }
#pragma unroll
    for (int cb = 0; cb < NCB; ++cb) {
      float b = accb[cb][0][0] * kc[0];
#pragma unroll
      for (int c = 1; c < 4; ++c) b = fmaf(accb[cb][c][0], kc[c], b);
      bias[cb] = b;
    }
  }

#pragma unroll 1
  for (int u = 0; u < NS; ++u) {
    // ---- q.k on 16 tokens ----
    float s[NCB][2];
    {
      const uint4 kw = lds128(tile + qt_kcodes_off() + u * 512 + 16 * lane);
      // words: (nt0,w0) (nt0,w1) (nt1,w0) (nt1,w1);  a0=(nt0,w0) a1=(nt1,w0) a2=(nt0,w1) a3=(nt1,w1)
      const uint32_t w0 = kw.x, w1 = kw.z, w2 = kw.y, w3 = kw.w;
      const uint32_t w0s = w0 >> 8, w1s = w1 >> 8, w2s = w2 >> 8, w3s = w3 >> 8;
      float acc[NCB][4];
#pragma unroll
      for (int cb = 0; cb < NCB; ++cb) acc[cb][0] = acc[cb][1] = acc[cb][2] = acc[cb][3] = 0.f;
#define LQ_QK_STEP(KS)                                                                           \
  {                                                                                              \
    const uint32_t a0 = kext<KS>(w0, w0s), a1 = kext<KS>(w1, w1s), a2 = kext<KS>(w2, w2s),       \
                   a3 = kext<KS>(w3, w3s);                                                       \
    _Pragma("unroll") for (int cb = 0; cb < NCB; ++cb)                                           \
        mma_bf16(acc[cb], a0, a1, a2, a3, bq[cb][KS][0], bq[cb][KS][1]);                         \
  }
      LQ_QK_STEP(0) LQ_QK_STEP(1) LQ_QK_STEP(2) LQ_QK_STEP(3)
      LQ_QK_STEP(4) LQ_QK_STEP(5) LQ_QK_STEP(6) LQ_QK_STEP(7)
#undef LQ_QK_STEP
#pragma unroll
      for (int cb = 0; cb < NCB; ++cb) {
        s[cb][0] = fmaf(acc[cb][0] + acc[cb][1], kq, bias[cb]);
        s[cb][1] = fmaf(acc[cb][2] + acc[cb][3], kq, bias[cb]);
      }
    }
    float pT[2][2];
    softmax_step<NCB>(st, s, pT, lane);

    // ---- value zero: one MMA, A = zero (fp16) with value groups on rows ----
    {
      uint32_t z0 = 0, z1 = 0;
      if (n < NG) {
        const uint2 zw = lds64(tile + qt_vzero_off(G) + u * VS + 8 * (4 * n + j));
        z0 = pack_f16x2(bf16lo_f32(zw.x), bf16hi_f32(zw.x));
        z1 = pack_f16x2(bf16lo_f32(zw.y), bf16hi_f32(zw.y));
      }
      mma_f16(st.zacc, z0, 0u, z1, 0u, pack_f16x2(pT[0][0], pT[0][1]), pack_f16x2(pT[1][0], pT[1][1]));
    }
    // ---- p * value scale per value group, fp16 ----
    uint32_t bp[NG][2];
    if (NG == 4) {
#pragma unroll
      for (int i = 0; i < 2; ++i) {
        const uint4 sv = lds128(tile + qt_vscale_off(G) + u * VS + 16 * (4 * i + j));
        const uint32_t w4[4] = {sv.x, sv.y, sv.z, sv.w};
#pragma unroll
        for (int gg = 0; gg < 2; ++gg)
#pragma unroll
          for (int th = 0; th < 2; ++th) {
            const uint32_t w = w4[2 * gg + th];
            bp[(2 * i + gg) % NG][th] = pack_f16x2(pT[th][0] * bf16lo_f32(w), pT[th][1] * bf16hi_f32(w));
          }
      }
    } else {
      const uint4 sv = lds128(tile + qt_vscale_off(G) + u * VS + 16 * j);
      const uint32_t w4[4] = {sv.x, sv.y, sv.z, sv.w};
#pragma unroll
      for (int gg = 0; gg < 2; ++gg)
#pragma unroll
        for (int th = 0; th < 2; ++th) {
          const uint32_t w = w4[2 * gg + th];
          bp[gg % NG][th] = pack_f16x2(pT[th][0] * bf16lo_f32(w), pT[th][1] * bf16hi_f32(w));
        }
    }
    // ---- p.v on 16 tokens ----
    {
      const uint4 vw = lds128(tile + qt_vcodes_off(G) + u * 512 + 16 * lane);
      const uint32_t v0s = vw.x >> 10, v1s = vw.y >> 10, v2s = vw.z >> 10, v3s = vw.w >> 10;
#define LQ_PV_STEP(MT)                                                                              \
  mma_f16(st.out[MT], vext<MT>(vw.x, v0s), vext<MT>(vw.y, v1s), vext<MT>(vw.z, v2s), vext<MT>(vw.w, v3s), \
          bp[((MT) * 16) / G][0], bp[((MT) * 16) / G][1]);
      LQ_PV_STEP(0) LQ_PV_STEP(1) LQ_PV_STEP(2) LQ_PV_STEP(3)
      LQ_PV_STEP(4) LQ_PV_STEP(5) LQ_PV_STEP(6) LQ_PV_STEP(7)
#undef LQ_PV_STEP
    }
  }
}

struct MmaSplitPlan {
  int units_fp;      // fp tiles per (b, kv)
  int units_quant;   // quant units per (b, kv)
  int tiles_quant;   // quant tiles per (b, kv)
  int tiles_per_unit;
};

template <int G, int NCB>
__global__ void __launch_bounds__(kWarps * 32, 3) lq_decode_mma_kernel(DecodeArgs a, MmaSplitPlan plan) {
  extern __shared__ __align__(128) uint8_t smem[];
  const CacheView& cv = a.cv;
  const int r = cv.Hq / cv.Hkv;
  const int S = a.S;
  const int64_t pair = blockIdx.x / S;
  const int split = blockIdx.x % S;
  const int b = static_cast<int>(pair / cv.Hkv), kv = static_cast<int>(pair % cv.Hkv);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int n = lane >> 2, j = lane & 3;
  constexpr int TILE = quant_tile_bytes(G);

  uint8_t* my_stages = smem + warp * (kStages * kStageBytes);
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + kWarps * kStages * kStageBytes) + warp * kStages;
  const uint32_t stage0 = smem_u32(my_stages);
  const uint32_t bar0 = smem_u32(bars);

  if (lane == 0) {
#pragma unroll
    for (int s = 0; s < kStages; ++s) mbar_init(bar0 + 8 * s, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  __syncwarp();

  // this warp's unit range
  const int U = plan.units_fp + plan.units_quant;
  const int NW = S * kWarps, wi = split * kWarps + warp;
  const int begin = static_cast<int>(static_cast<int64_t>(U) * wi / NW);
  const int end = static_cast<int>(static_cast<int64_t>(U) * (wi + 1) / NW);
  const int n_my = end - begin;

  const uint8_t* fpbase = cv.fp + a.layer * cv.fp_layer_stride + pair * cv.fp_head_stride;
  const uint8_t* qbase = cv.quant + a.layer * cv.quant_layer_stride + pair * cv.quant_head_stride;

  auto unit_src = [&](int unit, uint32_t& bytes) -> const uint8_t* {
    if (unit < plan.units_fp) {
      bytes = kFpTileBytes;
      return fpbase + static_cast<int64_t>(unit) * kFpTileBytes;
    }
    const int uq = unit - plan.units_fp;
    const int t0 = uq * plan.tiles_per_unit;
    const int nt = min(plan.tiles_per_unit, plan.tiles_quant - t0);
    bytes = nt * TILE;
    return qbase + static_cast<int64_t>(t0) * TILE;
  };
  auto issue = [&](int k) {
    if (lane == 0) {
      uint32_t bytes;
      const uint8_t* src = unit_src(begin + k, bytes);
      const int s = k % kStages;
      mbar_expect_tx(bar0 + 8 * s, bytes);
      bulk_load(stage0 + s * kStageBytes, src, bytes, bar0 + 8 * s);
    }
  };
#pragma unroll
  for (int k = 0; k < kStages; ++k)
    if (k < n_my) issue(k);

  // query fragments: B operand, column n -> head 4cb + n/2 (even column = hi, odd = lo of q*s);
  // k-step ks carries the factor 2^(64 - 2*(ks&3)) that cancels the code-position factor
  uint32_t qs[NCB][8][2];
  {
    const __nv_bfloat16* q = static_cast<const __nv_bfloat16*>(a.q);
#pragma unroll
    for (int cb = 0; cb < NCB; ++cb) {
      const int head = 4 * cb + (n >> 1);
      const bool valid = head < r;
      const __nv_bfloat16* qrow = q + (static_cast<int64_t>(b) * cv.Hq + kv * r + (valid ? head : 0)) * kD;
#pragma unroll
      for (int ks = 0; ks < 8; ++ks)
#pragma unroll
        for (int w = 0; w < 2; ++w) {
          const uint32_t raw = *reinterpret_cast<const uint32_t*>(qrow + 16 * ks + 8 * w + 2 * j);
          const float f = exp2f(static_cast<float>(64 - 2 * (ks & 3)));
          qs[cb][ks][w] = valid ? pack_bf16x2(bf16lo_f32(raw) * f, bf16hi_f32(raw) * f) : 0u;
        }
    }
  }
  float kc[4];
#pragma unroll
  for (int c = 0; c < 4; ++c) kc[c] = a.scale_log2 * exp2f(static_cast<float>(2 * c - 64));
  const float kq = a.scale_log2 * exp2f(69.f);

  WarpState<NCB> st;
#pragma unroll
  for (int mt = 0; mt < 8; ++mt) st.out[mt][0] = st.out[mt][1] = st.out[mt][2] = st.out[mt][3] = 0.f;
  st.zacc[0] = st.zacc[1] = st.zacc[2] = st.zacc[3] = 0.f;
#pragma unroll
  for (int cb = 0; cb < NCB; ++cb) { st.m[cb] = -INFINITY; st.l[cb] = 0.f; }
  st.quant_mode = false;

  bool failed = false;
#pragma unroll 1
  for (int k = 0; k < n_my; ++k) {
    const int s = k % kStages;
    const uint32_t parity = (k / kStages) & 1;
    int spins = 0;
    while (!mbar_try_wait(bar0 + 8 * s, parity)) {
      if (++spins > kSpinLimit) { failed = true; break; }
    }
    if (__any_sync(kFull, failed)) break;
    const int unit = begin + k;
    const uint32_t sbase = stage0 + s * kStageBytes;
    if (unit < plan.units_fp) {
      const int nv = min(16, a.n_fp - unit * 16);
      process_fp_tile<NCB>(st, qs, sbase, nv, kc, lane);
    } else {
      if (!st.quant_mode) {
#pragma unroll
        for (int mt = 0; mt < 8; ++mt) {
          const float f = vpos_scale(mt);
          st.out[mt][0] *= f; st.out[mt][1] *= f; st.out[mt][2] *= f; st.out[mt][3] *= f;
        }
        st.quant_mode = true;
      }
      const int uq = unit - plan.units_fp;
      const int nt = min(plan.tiles_per_unit, plan.tiles_quant - uq * plan.tiles_per_unit);
#pragma unroll 1
      for (int t = 0; t < nt; ++t) process_quant_tile<G, NCB>(st, qs, sbase + t * TILE, kc, kq, lane);
    }
    __syncwarp();
    if (k + kStages < n_my) issue(k + kStages);
  }
  if (failed) {
    // a bulk copy never completed: flag it, give the copies in flight a bounded chance to land
    // before this CTA's shared memory is released, and contribute nothing
    if (lane == 0) atomicOr(a.status, 1);
    for (int s = 0; s < kStages; ++s) {
      int spins = 0;
      while (!mbar_try_wait(bar0 + 8 * s, 0) && !mbar_try_wait(bar0 + 8 * s, 1) && ++spins < 1024) {}
    }
#pragma unroll
    for (int cb = 0; cb < NCB; ++cb) { st.m[cb] = -INFINITY; st.l[cb] = 0.f; }
  }

  // ---- fold zero term, undo position factors, reduce l over the token lanes ----
  constexpr int NG = kD / G;
#pragma unroll
  for (int mt = 0; mt < 8; ++mt) {
    const int g = (mt * 16) / G;
    const float z0 = __shfl_sync(kFull, st.zacc[0], 4 * g + j), z1 = __shfl_sync(kFull, st.zacc[1], 4 * g + j);
    const float f = st.quant_mode ? 1.0f / vpos_scale(mt) : 1.0f;
    st.out[mt][0] = fmaf(st.out[mt][0], f, z0);
    st.out[mt][1] = fmaf(st.out[mt][1], f, z1);
    st.out[mt][2] = fmaf(st.out[mt][2], f, z0);
    st.out[mt][3] = fmaf(st.out[mt][3], f, z1);
  }
  (void)NG;
#pragma unroll
  for (int cb = 0; cb < NCB; ++cb) {
    st.l[cb] += __shfl_xor_sync(kFull, st.l[cb], 4);
    st.l[cb] += __shfl_xor_sync(kFull, st.l[cb], 8);
    st.l[cb] += __shfl_xor_sync(kFull, st.l[cb], 16);
  }

  // ---- CTA merge of the 4 warp states through shared memory (stages are idle now) ----
  __syncthreads();
  float* wout = reinterpret_cast<float*>(smem);                 // [warp][d][8]
  float* wm = wout + kWarps * kD * 8;                           // [warp][8]
  float* wl = wm + kWarps * 8;                                  // [warp][8]
#pragma unroll
  for (int mt = 0; mt < 8; ++mt) {
    float* o = wout + (warp * kD + 16 * mt + n) * 8 + 2 * j;
    o[0] = st.out[mt][0];
    o[1] = st.out[mt][1];
    o[64] = st.out[mt][2];  // row + 8
    o[65] = st.out[mt][3];
  }
  if (n == 0) {
#pragma unroll
    for (int cb = 0; cb < NCB; ++cb) {
      wm[warp * 8 + 4 * cb + j] = st.m[cb];
      wl[warp * 8 + 4 * cb + j] = st.l[cb];
    }
  }
  __syncthreads();
  const int d = threadIdx.x;
  const int64_t rec = (pair * S + split) * r;
  for (int h = 0; h < r; ++h) {
    float M = -INFINITY;
#pragma unroll
    for (int w = 0; w < kWarps; ++w)
      if (wl[w * 8 + h] > 0.f) M = fmaxf(M, wm[w * 8 + h]);
    float o = 0.f, L = 0.f;
#pragma unroll
    for (int w = 0; w < kWarps; ++w)
      if (wl[w * 8 + h] > 0.f) {
        const float f = exp2f(wm[w * 8 + h] - M);
        o = fmaf(wout[(w * kD + d) * 8 + h], f, o);
        L = fmaf(wl[w * 8 + h], f, L);
      }
    a.part_o[(rec + h) * kD + d] = o;
    if (d == 0) {
      a.part_ml[(rec + h) * 2 + 0] = M;
      a.part_ml[(rec + h) * 2 + 1] = L;
    }
  }
}

MmaSplitPlan make_plan(const CacheView& cv, int n_fp, int64_t n_quant) {
  MmaSplitPlan p;
  p.units_fp = (n_fp + kFpTileSlots - 1) / kFpTileSlots;
  p.tiles_quant = static_cast<int>(n_quant / cv.G);
  p.tiles_per_unit = kStageBytes / quant_tile_bytes(cv.G);
  p.units_quant = (p.tiles_quant + p.tiles_per_unit - 1) / p.tiles_per_unit;
  return p;
}

constexpr int kSmemBytes = kWarps * kStages * kStageBytes + kWarps * kStages * 8;

}  // namespace

int decode_mma_max_splits(const CacheView& cv, int n_fp, int64_t n_quant, int sm_count) {
  const MmaSplitPlan p = make_plan(cv, n_fp, n_quant);
  const int pairs = cv.B * cv.Hkv;
  const int U = p.units_fp + p.units_quant;
  int S = (3 * sm_count) / pairs;
  S = S < (U + kWarps - 1) / kWarps ? S : (U + kWarps - 1) / kWarps;
  return S < 1 ? 1 : S;
}

cudaError_t launch_decode_mma(const DecodeArgs& a, cudaStream_t st) {
  const MmaSplitPlan plan = make_plan(a.cv, a.n_fp, a.n_quant);
  const int r = a.cv.Hq / a.cv.Hkv;
  const int blocks = a.cv.B * a.cv.Hkv * a.S;
  void (*kern)(DecodeArgs, MmaSplitPlan) = nullptr;
  if (a.cv.G == 32) kern = r <= 4 ? lq_decode_mma_kernel<32, 1> : lq_decode_mma_kernel<32, 2>;
  else if (a.cv.G == 64) kern = r <= 4 ? lq_decode_mma_kernel<64, 1> : lq_decode_mma_kernel<64, 2>;
  else return cudaErrorInvalidValue;
  static_assert(kSmemBytes >= static_cast<int>((kWarps * kD * 8 + 2 * kWarps * 8) * sizeof(float)), "merge scratch");
  cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
  if (e != cudaSuccess) return e;
  kern<<<blocks, kWarps * 32, kSmemBytes, st>>>(a, plan);
  return cudaGetLastError();
}

}  // namespace lq

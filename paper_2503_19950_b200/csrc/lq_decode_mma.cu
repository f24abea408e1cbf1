// Tensor-core decode attention over the mixed cache (LQ_KERNEL_MMA): split-K first pass.
//
// Work partition: every (b, kv) pair gets S or S + 1 CTAs so that the grid is exactly one resident
// wave (4 CTAs per SM, 3 for more than 4 query heads per KV head); inside a pair the items -- fp
// tiles (16 bf16 tokens, 8 KB) first, then quant tiles (one key group of G tokens each) -- are
// divided statically among the pair's warps by cost.  Each of the 4 warps of a CTA owns a private
// ring of shared-memory stages filled by 1-D bulk copies (cp.async.bulk + mbarrier, no multicast)
// and a private online-softmax state (m, l, o); the CTA merges the warp states into one split-K
// partial (Eq. 3 makes any visiting order legal), and the CTA that completes a pair merges the
// pair's partials and writes the output.
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
//   p.v   channels on M (16), tokens on K.
//         r <= 4: columns are again (hi, lo) per head, everything in bf16: value codes as bf16
//         subnormals, p*s_v split into hi + lo with packed bf16 multiply/fma, value zero through
//         one extra MMA per 16 tokens; bf16 values through ldmatrix.trans.
//         r  > 4: heads on the 8 columns; value codes as fp16 subnormals times p*s_v rounded to
//         fp16; bf16 values times p split into bf16 hi + lo (two MMAs).
//   The softmax probabilities come out of q.k with (token, head) = (lane/4, lane%4) and are
//   moved to the (column, token pair) arrangement p.v needs with 4 warp shuffles per 16 tokens.
#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include <algorithm>
#include <utility>
#include <vector>

#include "lq_kernels.cuh"

namespace lq {

namespace {

constexpr int kWarps = 4;
// every warp owns 12 KB of stages: 2 x 6 KB, each holding two G = 32 tiles (3 KB), one G = 64 tile
// (5 KB) or half an fp tile (K rows or V rows, 4 KB).  Loads of two tiles measured faster than
// single tiles (1.55 vs 1.9 us per tile and warp): the per-load bookkeeping is not free.
// (4-bit codes at G = 64: one tile is 9 KB, so that variant's stages are 9 KB and a CTA's shared memory allows
// three CTAs per SM instead of four.)
__host__ __device__ constexpr int stage_bytes(int G, int PL = 1) { return G == 64 && PL == 2 ? 9216 : 6144; }
__host__ __device__ constexpr int n_stages(int) { return 2; }
__host__ __device__ constexpr int warp_stage_bytes(int G, int PL = 1) { return n_stages(G) * stage_bytes(G, PL); }
constexpr int kWarpStageBytes = warp_stage_bytes(32);
constexpr int kMaxStages = 3;
constexpr int kOverlapDepth = 3;  // consecutive overlapped launches that share the SMs (plan_decode_mma)
constexpr int kCtasPerSm = 4;  // at 128 registers and 51 KB of shared memory; 3 and 5 both measured slower
constexpr uint32_t kFull = 0xFFFFFFFFu;
constexpr int kSpinLimit = 1 << 22;
// cost of one fp tile (16 bf16 tokens, two loads) in eighths of a quant tile: 4 to 12 measured alike,
// 2 and 16 slower
constexpr int kFpCost8 = 8;
// (with two column blocks -- five to eight query heads per KV head -- a quant tile costs more and the bf16 tile
// relatively less: 4, measured 2.5 % better than 8 on the GQA-7 workload)
__host__ __device__ constexpr int fp_cost8(int ncb) { return ncb == 2 ? 4 : kFpCost8; }

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
  asm(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
// same with a zero accumulator input (no registers to clear)
__device__ __forceinline__ void mma_bf16_z(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                           uint32_t b0, uint32_t b1) {
  asm(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%10,%10,%10,%10};"
      : "=f"(c[0]), "=f"(c[1]), "=f"(c[2]), "=f"(c[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1), "f"(0.f));
}
__device__ __forceinline__ void mma_f16(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                        uint32_t b0, uint32_t b1) {
  asm(
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
__device__ __forceinline__ uint32_t f16x2_mul(uint32_t a, uint32_t b) {
  uint32_t d;
  asm("mul.rn.f16x2 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));
  return d;
}
__device__ __forceinline__ uint32_t bf16x2_neg(uint32_t a) {
  uint32_t d;
  asm("neg.bf16x2 %0, %1;" : "=r"(d) : "r"(a));
  return d;
}
__device__ __forceinline__ float pow2i(int k) { return __int_as_float((k + 127) << 23); }  // 2^k, -126 <= k <= 127
__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
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

// one code position of a packed word as two bf16 subnormals (positions 0,2,4,6 of each byte)
template <int I>
__device__ __forceinline__ uint32_t ext_bf16(uint32_t w, uint32_t w8) {
  return I < 4 ? (w & (0x00030003u << (2 * I))) : (w8 & (0x00030003u << (2 * (I - 4))));
}
// same with an index that becomes a constant once the caller's loop is unrolled
__device__ __forceinline__ uint32_t ext_bf16_i(int i, uint32_t w, uint32_t w8) {
  return i < 4 ? (w & (0x00030003u << (2 * i))) : (w8 & (0x00030003u << (2 * (i - 4))));
}
// ... or as two fp16 subnormals (positions 0..8 direct, 10..14 after a shift by 10)
template <int I>
__device__ __forceinline__ uint32_t ext_f16(uint32_t w, uint32_t w10) {
  return I < 5 ? (w & (0x00030003u << (2 * I))) : (w10 & (0x00030003u << (2 * (I - 5))));
}

// NCB = number of column blocks of 4 heads.  NCB == 1: p.v columns are (hi, lo) per head and the
// probabilities carry a factor 2^64 (kPExp) so that products with bf16 subnormal codes stay normal.
// NCB == 2: the probabilities (at most 2^8 because the reference maximum moves lazily) carry 2^-8, so
// that p * s_v fits fp16 for every value scale fp16 itself can hold.
// p.v flavour.  bf16_pv: columns are (hi, lo) per head, everything bf16, exact products, r <= 4 only.
// Otherwise: heads on the 8 columns, value codes as fp16 subnormals, p * s_v rounded to fp16.
template <int NCB>
__host__ __device__ constexpr bool bf16_pv() { return NCB == 1; }

template <int NCB>
struct WarpState {
  float out[8][4];  // o^T: [channel tile][c-fragment]
  float zacc[4];    // sum_t p_t * vzero_t per (value group, column)
  float m[NCB];     // running max (log2 units) of head 4cb + lane%4
  float l[NCB];     // this lane's share of the running denominator (times 2^kPExp)
  bool quant_mode;  // out rows carry the code-position factor
};
template <int NCB>
struct Mode {
  static constexpr float kPExp = bf16_pv<NCB>() ? 64.f : -8.f;
};

// factor the out rows of channel tile mt carry in quant mode, relative to fp mode
template <int NCB>
__device__ __forceinline__ int vpos_log2(int mt) {
  return bf16_pv<NCB>() ? 2 * (mt & 3) - 133 : 2 * (mt < 5 ? mt : mt - 5) - 24;
}

// ---- online softmax over the NSUB*16 scores of one tile ---------------------------------------
// s[u][cb][th]: score (log2 units) of token 16u + 8th + lane/4 for head 4cb + lane%4; replaced by
// the probabilities 2^(s - m + kPExp).
template <int NCB, int NSUB>
__device__ __forceinline__ void tile_softmax(WarpState<NCB>& st, float (&s)[NSUB][NCB][2], int lane, int opaque_zero) {
  const int j = lane & 3;
  float corr[NCB];
  bool changed = false;
#pragma unroll
  for (int cb = 0; cb < NCB; ++cb) {
    float mx = fmaxf(s[0][cb][0], s[0][cb][1]);
#pragma unroll
    for (int u = 1; u < NSUB; ++u) mx = fmaxf(mx, fmaxf(s[u][cb][0], s[u][cb][1]));
    mx = fmaxf(mx, __shfl_xor_sync(kFull, mx, 4));
    mx = fmaxf(mx, __shfl_xor_sync(kFull, mx, 8));
    mx = fmaxf(mx, __shfl_xor_sync(kFull, mx, 16));
    // the reference m only has to stay within 2^8 of the running maximum (p <= 256 is harmless),
    // so it moves -- and the accumulators are rescaled -- only when a score exceeds it by more than 8
    const bool up = mx > st.m[cb] + 8.f;  // m = -inf initially -> true
    const float mn = up ? mx : st.m[cb];
    changed |= up && st.m[cb] > -INFINITY;  // nothing to rescale before the first tile
    corr[cb] = ex2(st.m[cb] - mn);  // m = -inf -> 0; unchanged -> 1
    st.m[cb] = mn;
  }
  // Written as a loop with an opaque exit so that it stays a real (rarely taken) branch instead
  // of 36 multiplies and selects on every tile.
  int again = __any_sync(kFull, changed);
  while (again) {
    float ca, cbv;
    if (bf16_pv<NCB>()) {
      ca = cbv = corr[0];  // all four accumulators of a lane belong to head lane%4
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
    again = opaque_zero;  // always 0, but only known at run time
  }
#pragma unroll
  for (int cb = 0; cb < NCB; ++cb) {
    const float off = Mode<NCB>::kPExp - st.m[cb];
    float lsum = 0.f;
#pragma unroll
    for (int u = 0; u < NSUB; ++u) {
      s[u][cb][0] = ex2(s[u][cb][0] + off);
      s[u][cb][1] = ex2(s[u][cb][1] + off);
      lsum += s[u][cb][0] + s[u][cb][1];
    }
    st.l[cb] += lsum;
  }
}

// probabilities of one 16-token sub-tile moved to the B-operand arrangement of p.v:
// pT[th][i] = p(token 8th + 2*(lane%4) + i) for the head of column lane/4
template <int NCB>
__device__ __forceinline__ void transpose_p(const float (&p)[NCB][2], float (&pT)[2][2], int lane) {
  const int n = lane >> 2, j = lane & 3;
#pragma unroll
  for (int th = 0; th < 2; ++th)
#pragma unroll
    for (int i = 0; i < 2; ++i) {
      if (bf16_pv<NCB>()) {
        pT[th][i] = __shfl_sync(kFull, p[0][th], 4 * (2 * j + i) + (n >> 1));  // column n -> head n/2
      } else if (NCB == 1) {
        pT[th][i] = __shfl_sync(kFull, p[0][th], 4 * (2 * j + i) + (n & 3));  // column n -> head n (mod 4)
      } else {
        const int src = 4 * (2 * j + i) + (n & 3);  // column n -> head n
        const float v0 = __shfl_sync(kFull, p[0][th], src), v1 = __shfl_sync(kFull, p[NCB - 1][th], src);
        pT[th][i] = (n >> 2) ? v1 : v0;
      }
    }
}

// NCB == 1: split the probabilities into bf16 hi (even columns) / lo (odd columns).  The odd
// columns carry the lo parts NEGATED all the way to the accumulators (the epilogue subtracts them):
// the residuals then need no separate negation.  H = hi in every lane; P = hi in even, -lo in odd columns.
__device__ __forceinline__ void split_p_bf16(const float (&pT)[2][2], bool odd, uint32_t (&H)[2], uint32_t (&P)[2]) {
#pragma unroll
  for (int th = 0; th < 2; ++th) {
    H[th] = pack_bf16x2(pT[th][0], pT[th][1]);
    P[th] = H[th];
    if (odd) P[th] = pack_bf16x2(bf16lo_f32(H[th]) - pT[th][0], bf16hi_f32(H[th]) - pT[th][1]);
  }
}

// ---- one fp tile: 16 bf16 tokens (rows swizzled in 16-byte chunks by row & 7), loaded as two
// units: the K rows (scores, softmax; leaves the p.v B operands in b0/b1), then the V rows -------
// pad16: bit i set = slot i of the tile is padding (left out); at least one valid slot is not
template <int NCB>
__device__ __forceinline__ void process_fp_keys(WarpState<NCB>& st, const uint32_t (&qs)[NCB][8][2], uint32_t krows,
                                                int n_valid, const float (&kc)[4], int lane, uint32_t oddmask,
                                                int opaque_zero, uint32_t (&b0)[2], uint32_t (&b1)[2],
                                                uint32_t pad16 = 0u) {
  const int n = lane >> 2;
  float acc[NCB][4][4];
  {
    const int mi = lane >> 3, rr = lane & 7;
    const int token = rr + 8 * (mi & 1);
    const uint32_t rowaddr = krows + token * 256;
#pragma unroll
    for (int ks = 0; ks < 8; ++ks) {
      const int chunk = 2 * ks + (mi >> 1);
      uint32_t a0, a1, a2, a3;
      ldmatrix_x4(rowaddr + ((chunk ^ (token & 7)) << 4), a0, a1, a2, a3);
#pragma unroll
      for (int cb = 0; cb < NCB; ++cb) {
        if (ks < 4) mma_bf16_z(acc[cb][ks & 3], a0, a1, a2, a3, qs[cb][ks][0], qs[cb][ks][1]);
        else mma_bf16(acc[cb][ks & 3], a0, a1, a2, a3, qs[cb][ks][0], qs[cb][ks][1]);
      }
    }
  }
  float s[1][NCB][2];
#pragma unroll
  for (int cb = 0; cb < NCB; ++cb) {
    float s0 = acc[cb][0][0] * kc[0], s1 = acc[cb][0][2] * kc[0];
#pragma unroll
    for (int c = 1; c < 4; ++c) {
      s0 = fmaf(acc[cb][c][0], kc[c], s0);
      s1 = fmaf(acc[cb][c][2], kc[c], s1);
    }
    s[0][cb][0] = n < n_valid && !((pad16 >> n) & 1u) ? s0 : -INFINITY;
    s[0][cb][1] = n + 8 < n_valid && !((pad16 >> (n + 8)) & 1u) ? s1 : -INFINITY;
  }
  tile_softmax<NCB, 1>(st, s, lane, opaque_zero);
  float pT[2][2];
  transpose_p<NCB>(s[0], pT, lane);
  // NCB == 1: only b0 (hi/lo by column); NCB == 2: b0 = hi, b1 = lo
  if (bf16_pv<NCB>()) {
    uint32_t H[2];
    split_p_bf16(pT, oddmask != 0u, H, b0);
    b1[0] = b1[1] = 0;
  } else {
#pragma unroll
    for (int th = 0; th < 2; ++th) {
      b0[th] = pack_bf16x2(pT[th][0], pT[th][1]);
      b1[th] = pack_bf16x2(pT[th][0] - bf16lo_f32(b0[th]), pT[th][1] - bf16hi_f32(b0[th]));
    }
  }
}

template <int NCB>
__device__ __forceinline__ void process_fp_values(WarpState<NCB>& st, uint32_t vrows, int lane,
                                                  const uint32_t (&b0)[2], const uint32_t (&b1)[2]) {
  const int mi = lane >> 3, rr = lane & 7;
  const int token = rr + 8 * (mi >> 1);
  const uint32_t rowaddr = vrows + token * 256;
#pragma unroll
  for (int mt = 0; mt < 8; ++mt) {
    const int chunk = 2 * mt + (mi & 1);
    uint32_t a0, a1, a2, a3;
    ldmatrix_x4_trans(rowaddr + ((chunk ^ (token & 7)) << 4), a0, a1, a2, a3);
    mma_bf16(st.out[mt], a0, a1, a2, a3, b0[0], b0[1]);
    if (!bf16_pv<NCB>()) mma_bf16(st.out[mt], a0, a1, a2, a3, b1[0], b1[1]);
  }
}

// ---- q.zero of the key groups of one stage: bias[t][cb] for head 4cb + lane%4 of tile t (log2 units).
// One MMA per k-step serves two tiles: the A fragment's rows 0-7 repeat the zero row of tile 0 and
// rows 8-15 that of tile 1 (ldmatrix with equal row addresses inside each 8x8 matrix); the four
// accumulators collect the k-steps of equal code-position factor, which kc[] undoes.
// zaddr: this lane's row address, k-step 0.
template <int NCB>
__device__ __forceinline__ void quant_bias(const uint32_t (&qs)[NCB][8][2], uint32_t zaddr, const float (&kc)[4],
                                           float (&bias)[2][NCB]) {
  float accb[NCB][4][4];
#pragma unroll
  for (int ks = 0; ks < 8; ++ks) {
    uint32_t z0, z1, z2, z3;
    ldmatrix_x4(zaddr + 32 * ks, z0, z1, z2, z3);
#pragma unroll
    for (int cb = 0; cb < NCB; ++cb) {
      if (ks < 4) mma_bf16_z(accb[cb][ks & 3], z0, z1, z2, z3, qs[cb][ks][0], qs[cb][ks][1]);
      else mma_bf16(accb[cb][ks & 3], z0, z1, z2, z3, qs[cb][ks][0], qs[cb][ks][1]);
    }
  }
#pragma unroll
  for (int cb = 0; cb < NCB; ++cb) {
    float b0 = accb[cb][0][0] * kc[0], b1 = accb[cb][0][2] * kc[0];
#pragma unroll
    for (int c = 1; c < 4; ++c) {
      b0 = fmaf(accb[cb][c][0], kc[c], b0);
      b1 = fmaf(accb[cb][c][2], kc[c], b1);
    }
    bias[0][cb] = b0;
    bias[1][cb] = b1;
  }
}

// ---- fused append: one new row (256 B, lane = 8 B) replaces row `row` of a landed K or V half tile
// in shared memory and goes to the same place of the fp store ---------------------------------
__device__ __forceinline__ void patch_new_row(uint32_t half_tile_smem, uint8_t* half_tile_global, const void* rows,
                                              int pair, int row, int lane) {
  const uint2 x = __ldg(reinterpret_cast<const uint2*>(static_cast<const uint8_t*>(rows) + pair * (kD * 2)) + lane);
  const int off = row * 256 + (((lane >> 1) ^ (row & 7)) << 4) + (lane & 1) * 8;
  asm volatile("st.shared.v2.u32 [%0], {%1,%2};" ::"r"(half_tile_smem + off), "r"(x.x), "r"(x.y) : "memory");
  *reinterpret_cast<uint2*>(half_tile_global + off) = x;
  __syncwarp();
}

// ---- one quant tile: one key group of G tokens ---------------------------------------------
// PL = 2-bit planes per code.  A 4-bit code is 4 * (high plane) + (low plane): the high plane goes
// through the same contractions first, its score accumulators are multiplied by 4 before the low
// plane is added, and in p.v it meets p * s_v * 4 (all exact).
// pad0/pad1: bit i set = token i (pad0) or 32 + i (pad1) of the tile is padding (left out); not all of them are
template <int G, int NCB, int PL>
__device__ __forceinline__ void process_quant_tile(WarpState<NCB>& st, const uint32_t (&qs)[NCB][8][2], uint32_t tile,
                                                   const float (&bias)[NCB], float kq, int lane, uint32_t oddmask,
                                                   int opaque_zero, uint32_t pad0 = 0u, uint32_t pad1 = 0u) {
  constexpr int NS = G / 16, NG = kD / G, VS = vsz_subtile_bytes(G);
  const int n = lane >> 2, j = lane & 3;
  // ---- q.k on all G tokens.  Per pair of k-steps: the key scale of the lane's channels is folded
  // into the query (even columns RN(q*s), odd columns the exact residual) and every sub-tile's
  // score accumulator advances by one MMA per k-step; the group's q.zero comes in as `bias`.
  float s[NS][NCB][2];
  {
    float acc[NS][NCB][4];
#pragma unroll
    for (int pl = PL - 1; pl >= 0; --pl) {
      uint32_t kw[NS][4], kws[NS][4];
#pragma unroll
      for (int u = 0; u < NS; ++u) {
        const uint4 w = lds128(tile + qt_kcodes_off() + pl * qt_plane_bytes(G) + u * 512 + 16 * lane);
        // words: (nt0,w0) (nt0,w1) (nt1,w0) (nt1,w1);  a0=(nt0,w0) a1=(nt1,w0) a2=(nt0,w1) a3=(nt1,w1)
        kw[u][0] = w.x; kw[u][1] = w.z; kw[u][2] = w.y; kw[u][3] = w.w;
#pragma unroll
        for (int e = 0; e < 4; ++e) kws[u][e] = kw[u][e] >> 8;
      }
      if (pl != PL - 1) {
#pragma unroll
        for (int u = 0; u < NS; ++u)
#pragma unroll
          for (int cb = 0; cb < NCB; ++cb)
#pragma unroll
            for (int e = 0; e < 4; ++e) acc[u][cb][e] *= 4.0f;
      }
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const uint4 sw = lds128(tile + qt_kscale_off() + 16 * (4 * i + j));
        const uint32_t s4[4] = {sw.x, sw.y, sw.z, sw.w};
#pragma unroll
        for (int kk = 0; kk < 2; ++kk) {
          const int ks = 2 * i + kk;
          uint32_t bq[NCB][2];
#pragma unroll
          for (int cb = 0; cb < NCB; ++cb) {
#pragma unroll
            for (int w = 0; w < 2; ++w) {
              // even columns RN(q*s); odd columns the exact residual q*s - RN(q*s)
              bq[cb][w] = bf16x2_mul(qs[cb][ks][w], s4[2 * kk + w]);
              if (oddmask) bq[cb][w] = bf16x2_fma(qs[cb][ks][w], s4[2 * kk + w], bf16x2_neg(bq[cb][w]));
            }
          }
#pragma unroll
          for (int u = 0; u < NS; ++u) {
            const uint32_t a0 = ext_bf16_i(ks, kw[u][0], kws[u][0]), a1 = ext_bf16_i(ks, kw[u][1], kws[u][1]),
                           a2 = ext_bf16_i(ks, kw[u][2], kws[u][2]), a3 = ext_bf16_i(ks, kw[u][3], kws[u][3]);
#pragma unroll
            for (int cb = 0; cb < NCB; ++cb) {
              if (ks == 0 && pl == PL - 1) mma_bf16_z(acc[u][cb], a0, a1, a2, a3, bq[cb][0], bq[cb][1]);
              else mma_bf16(acc[u][cb], a0, a1, a2, a3, bq[cb][0], bq[cb][1]);
            }
          }
        }
      }
    }
#pragma unroll
    for (int cb = 0; cb < NCB; ++cb) {
#pragma unroll
      for (int u = 0; u < NS; ++u) {
        s[u][cb][0] = fmaf(acc[u][cb][0] + acc[u][cb][1], kq, bias[cb]);
        s[u][cb][1] = fmaf(acc[u][cb][2] + acc[u][cb][3], kq, bias[cb]);
      }
    }
    if (pad0 | pad1) {  // always false in the instantiation without padding (constant arguments)
#pragma unroll
      for (int u = 0; u < NS; ++u) {
        const uint32_t w = (u < 2 ? pad0 : pad1) >> (16 * (u & 1) + n);
#pragma unroll
        for (int cb = 0; cb < NCB; ++cb) {
          if (w & 1u) s[u][cb][0] = -INFINITY;
          if (w & 0x100u) s[u][cb][1] = -INFINITY;
        }
      }
    }
  }
  tile_softmax<NCB, NS>(st, s, lane, opaque_zero);

#pragma unroll
  for (int u = 0; u < NS; ++u) {
    float pT[2][2];
    transpose_p<NCB>(s[u], pT, lane);
    if (bf16_pv<NCB>()) {
      uint32_t H[2], P[2];
      split_p_bf16(pT, oddmask != 0u, H, P);
      // value zero: A = zero (bf16 pairs straight from the tile), value groups on rows
      {
        // rows n >= NG of this MMA repeat real rows; their sums land in zacc rows nobody reads
        const uint2 zw = lds64(tile + qt_vzero_off(G, PL) + u * VS + 8 * (4 * (n % NG) + j));
        mma_bf16(st.zacc, zw.x, 0u, zw.y, 0u, P[0], P[1]);
      }
      // p * value scale per value group: even columns RN(hi*s), odd columns -(lo*s + residual)
      const uint32_t Hn[2] = {H[0] ^ 0x80008000u, H[1] ^ 0x80008000u};
      uint32_t bp[NG][2];
      uint32_t sv[NG][2];
      if (NG == 4) {
        const uint4 s0 = lds128(tile + qt_vscale_off(G, PL) + u * VS + 16 * j);
        const uint4 s1 = lds128(tile + qt_vscale_off(G, PL) + u * VS + 16 * (4 + j));
        sv[0][0] = s0.x; sv[0][1] = s0.y; sv[1][0] = s0.z; sv[1][1] = s0.w;
        sv[2 % NG][0] = s1.x; sv[2 % NG][1] = s1.y; sv[3 % NG][0] = s1.z; sv[3 % NG][1] = s1.w;
      } else {
        const uint4 s0 = lds128(tile + qt_vscale_off(G, PL) + u * VS + 16 * j);
        sv[0][0] = s0.x; sv[0][1] = s0.y; sv[1 % NG][0] = s0.z; sv[1 % NG][1] = s0.w;
      }
#pragma unroll
      for (int g = 0; g < NG; ++g)
#pragma unroll
        for (int th = 0; th < 2; ++th) {
          bp[g][th] = bf16x2_mul(H[th], sv[g][th]);
          if (oddmask) {
            const uint32_t r1n = bf16x2_fma(Hn[th], sv[g][th], bp[g][th]);  // RN(hi*s) - hi*s, exact
            bp[g][th] = bf16x2_fma(P[th], sv[g][th], r1n);
          }
        }
#pragma unroll
      for (int pl = PL - 1; pl >= 0; --pl) {
        const uint4 vw = lds128(tile + qt_vcodes_off(G, PL) + pl * qt_plane_bytes(G) + u * 512 + 16 * lane);
        uint32_t bx[NG][2];  // the high plane meets 4 * p * s_v
#pragma unroll
        for (int g = 0; g < NG; ++g)
#pragma unroll
          for (int th = 0; th < 2; ++th) bx[g][th] = pl ? bf16x2_mul(bp[g][th], 0x40804080u) : bp[g][th];
        const uint32_t v0s = vw.x >> 8, v1s = vw.y >> 8, v2s = vw.z >> 8, v3s = vw.w >> 8;
#define LQ_PV_STEP(MT)                                                                                        \
  mma_bf16(st.out[MT], ext_bf16<MT>(vw.x, v0s), ext_bf16<MT>(vw.y, v1s), ext_bf16<MT>(vw.z, v2s),             \
           ext_bf16<MT>(vw.w, v3s), bx[((MT) * 16) / G][0], bx[((MT) * 16) / G][1]);
        LQ_PV_STEP(0) LQ_PV_STEP(1) LQ_PV_STEP(2) LQ_PV_STEP(3)
        LQ_PV_STEP(4) LQ_PV_STEP(5) LQ_PV_STEP(6) LQ_PV_STEP(7)
#undef LQ_PV_STEP
      }
    } else {
      // value zero: A = zero converted to fp16, value groups on rows
      {
        uint32_t z0 = 0, z1 = 0;
        if (n < NG) {
          const uint2 zw = lds64(tile + qt_vzero_off(G, PL) + u * VS + 8 * (4 * n + j));
          z0 = pack_f16x2(bf16lo_f32(zw.x), bf16hi_f32(zw.x));
          z1 = pack_f16x2(bf16lo_f32(zw.y), bf16hi_f32(zw.y));
        }
        mma_f16(st.zacc, z0, 0u, z1, 0u, pack_f16x2(pT[0][0], pT[0][1]), pack_f16x2(pT[1][0], pT[1][1]));
      }
      uint32_t bp[NG][2];
      if (NG == 4) {
#pragma unroll
        for (int i = 0; i < 2; ++i) {
          const uint4 svw = lds128(tile + qt_vscale_off(G, PL) + u * VS + 16 * (4 * i + j));
          const uint32_t w4[4] = {svw.x, svw.y, svw.z, svw.w};
#pragma unroll
          for (int gg = 0; gg < 2; ++gg)
#pragma unroll
            for (int th = 0; th < 2; ++th) {
              const uint32_t w = w4[2 * gg + th];
              bp[(2 * i + gg) % NG][th] = pack_f16x2(pT[th][0] * bf16lo_f32(w), pT[th][1] * bf16hi_f32(w));
            }
        }
      } else {
        const uint4 svw = lds128(tile + qt_vscale_off(G, PL) + u * VS + 16 * j);
        const uint32_t w4[4] = {svw.x, svw.y, svw.z, svw.w};
#pragma unroll
        for (int gg = 0; gg < 2; ++gg)
#pragma unroll
          for (int th = 0; th < 2; ++th) {
            const uint32_t w = w4[2 * gg + th];
            bp[gg % NG][th] = pack_f16x2(pT[th][0] * bf16lo_f32(w), pT[th][1] * bf16hi_f32(w));
          }
      }
#pragma unroll
      for (int pl = PL - 1; pl >= 0; --pl) {
        const uint4 vw = lds128(tile + qt_vcodes_off(G, PL) + pl * qt_plane_bytes(G) + u * 512 + 16 * lane);
        uint32_t bx[NG][2];  // the high plane meets 4 * p * s_v
#pragma unroll
        for (int g = 0; g < NG; ++g)
#pragma unroll
          for (int th = 0; th < 2; ++th) bx[g][th] = pl ? f16x2_mul(bp[g][th], 0x44004400u) : bp[g][th];
        const uint32_t v0s = vw.x >> 10, v1s = vw.y >> 10, v2s = vw.z >> 10, v3s = vw.w >> 10;
#define LQ_PV_STEP(MT)                                                                                        \
  mma_f16(st.out[MT], ext_f16<MT>(vw.x, v0s), ext_f16<MT>(vw.y, v1s), ext_f16<MT>(vw.z, v2s),                 \
          ext_f16<MT>(vw.w, v3s), bx[((MT) * 16) / G][0], bx[((MT) * 16) / G][1]);
        LQ_PV_STEP(0) LQ_PV_STEP(1) LQ_PV_STEP(2) LQ_PV_STEP(3)
        LQ_PV_STEP(4) LQ_PV_STEP(5) LQ_PV_STEP(6) LQ_PV_STEP(7)
#undef LQ_PV_STEP
      }
    }
  }
}

// shared memory: [per-warp stages][query rows of the pair][mbarriers][flags]
constexpr int kSmemStages = kWarps * kWarpStageBytes;   // the smallest variant: the merge areas below must fit into it
__host__ __device__ constexpr int smem_stages(int G, int PL) { return kWarps * warp_stage_bytes(G, PL); }
constexpr int kSmemQ = kMaxRatio * kD * 2;
constexpr int kSmemBars = (kWarps * kMaxStages + 1) * 8;
__host__ __device__ constexpr int smem_bytes(int G, int PL) { return smem_stages(G, PL) + kSmemQ + kSmemBars + 16; }
constexpr int kMergeMax = 2048;  // S * r records the fused second pass can stage
constexpr int kMergeOneBatch = 12;  // CTA records the fused second pass loads in one batch (kSB per warp)

// Work items of one (b, kv) pair, in order: fp tiles [0, tiles_fp), then quant tiles.  The CTAs of
// the pair (4 warps each) share them by a static, cost-weighted partition (see below); any
// assignment is legal because every warp keeps its own online-softmax state.  A warp keeps up to
// two loads in flight.
// FUSED: the launch also appends one token (DecodeArgs::new_k); a separate instantiation so that
// the plain kernel's main loop is not touched.
// PADDED: the batch is left-padded (DecodeArgs::rowinfo): per sequence, leading quant tiles that are
// padding entirely are not visited, and tiles and slots with padding among their tokens get -inf scores.
template <int G, int NCB, int PL, bool FUSED, bool PADDED>
__global__ void __launch_bounds__(kWarps * 32, NCB == 1 ? kCtasPerSm : kCtasPerSm - 1) lq_decode_mma_kernel(DecodeArgs a) {
  extern __shared__ __align__(128) uint8_t smem[];
  const CacheView& cv = a.cv;
  const int r = cv.Hq / cv.Hkv;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int n = lane >> 2, j = lane & 3;
  const uint32_t oddmask = (n & 1) ? 0xFFFFFFFFu : 0u;
  constexpr int TILE = quant_tile_bytes(G, PL);
  constexpr int kStages = n_stages(G), kStageBytes = stage_bytes(G, PL);
  constexpr int kWarpStage = warp_stage_bytes(G, PL), kStagesAll = smem_stages(G, PL);
  static_assert(TILE <= kStageBytes && kFpTileVOffset <= kStageBytes && kStages <= kMaxStages, "stage geometry");
  // CTA c works for pair c % P in slot c / P: pairs [0, n_extra) have S CTAs, the others S - 1 (a.S
  // is also the record stride).  Interleaving gives every pair CTAs from every launch rank of the
  // SMs, so no pair consists only of CTAs whose first loads queue behind everybody else's.
  int pair, slot, n_ctas_pair;
  if (PADDED) {
    // sequences of a padded batch have different amounts of work: the host shared the CTAs out accordingly
    const int e = a.cta_map[blockIdx.x];
    pair = e & 0xFFFF;
    slot = e >> 16;
    n_ctas_pair = a.pair_ctas[pair];
  } else {
    const int P = cv.B * cv.Hkv;
    pair = blockIdx.x % P;
    slot = blockIdx.x / P;
    n_ctas_pair = pair < a.n_extra ? a.S : a.S - 1;
  }
  const int b = pair / cv.Hkv, kv = pair % cv.Hkv;
  constexpr int TPS = kStageBytes / TILE;  // quant tiles per load (and per stage)
  const int n_warps = n_ctas_pair * kWarps, gw = slot * kWarps + warp;
  // Static partition: the pair's items -- fp tiles (cost kFpCost8 / 8 each), then quant tiles (cost
  // 1) -- lie on a cost line that is cut into n_warps equal ranges; warp gw takes the items between
  // cut gw and cut gw + 1 (boundaries rounded to the nearest item).  Every SM carries the same number
  // of identical warps, so equal work gives (nearly) equal finishing times without any work queue;
  // weighting the ranges by the launch order of the CTAs on an SM measured slower.
  // quant item i of this pair is tile qskip + i of the store
  const int qskip = PADDED ? min(a.rowinfo[4 * b + 0], a.tiles_quant) : 0;
  const int qpad_end = PADDED ? a.rowinfo[4 * b + 1] : 0;
  const bool fp_padded = PADDED && a.rowinfo[4 * b + 2] != 0;
  const uint32_t* qmask = PADDED ? a.qmask + static_cast<int64_t>(b) * a.qmask_words : nullptr;
  const uint32_t* fpmask = PADDED ? a.fpmask + static_cast<int64_t>(b) * a.fpmask_words : nullptr;
  int it, it_end;
  {
    constexpr int kCost = fp_cost8(NCB);
    const int F8 = a.tiles_fp * kCost, C8 = F8 + (a.tiles_quant - qskip) * 8;
    // Overlapped launches (DecodeArgs::early): the CTAs of a launch take over the slots of earlier launches in
    // launch order, and the last slots to free up are those of merging CTAs -- one per pair, and the last CTA of
    // every pair is launched last.  That CTA starts later than the others; it gets 3/4 of a share (measured with a
    // third of a wave per launch: 3/4 and 1 alike on the 8k workload, 3/4 better by 2 % on GQA-7, 1/2 and 1/4 worse;
    // a serialised launch keeps equal shares).
    const int64_t full_warps = static_cast<int64_t>(n_warps) - (a.early && n_ctas_pair > 1 ? kWarps : 0);
    const int64_t total_w4 = 4 * full_warps + 3 * (n_warps - full_warps);
    auto cut = [&](int k) {
      const int64_t cw4 = k <= full_warps ? 4LL * k : 4 * full_warps + 3 * (k - full_warps);
      const int pos8 = static_cast<int>(cw4 * C8 / total_w4);
      return pos8 < F8 ? (pos8 + kCost / 2) / kCost : a.tiles_fp + (pos8 - F8 + 4) / 8;
    };
    it = cut(gw);
    it_end = cut(gw + 1);
  }
  int* ticket = a.tickets + 32 * pair + 1;  // one 128-byte line per pair; word 1 is the arrival ticket

  const uint32_t stage0 = smem_u32(smem + warp * kWarpStage);
  const uint32_t qsm = smem_u32(smem + kStagesAll);
  const uint32_t bar0 = smem_u32(smem + kStagesAll + kSmemQ) + warp * kMaxStages * 8;
  const uint32_t qbar = smem_u32(smem + kStagesAll + kSmemQ) + kWarps * kMaxStages * 8;
  int* is_last = reinterpret_cast<int*>(smem + kStagesAll + kSmemQ + kSmemBars);

  if (lane == 0) {
#pragma unroll
    for (int s = 0; s < kStages; ++s) mbar_init(bar0 + 8 * s, 1);
    if (warp == 0) mbar_init(qbar, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  __syncthreads();
  // Programmatic dependent launch: everything above touches only this CTA's shared memory, the launch
  // arguments and, in the padded variant, the CTA map and row info of the mask block -- which only a host copy
  // enqueued by the same call writes (upload_masks), never a kernel that could still be running.  Nothing an
  // earlier kernel may still be writing is read before it has finished.
  if (!a.early) asm volatile("griddepcontrol.wait;" ::: "memory");
  // In a chain of overlapped launches the next launch may take the slots of this one as soon as they free up (its
  // CTAs stream their own layer and wait for this grid only before the workspace); otherwise the trigger comes
  // after the main loop, so that CTAs that could only wait do not take the slots earlier.
  if (a.early) asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  if (threadIdx.x == 0) {
    // the r query rows of this pair are contiguous: one bulk copy
    mbar_expect_tx(qbar, r * kD * 2);
    if (!a.debug_stall)
      bulk_load(qsm, static_cast<const uint8_t*>(a.q) + (static_cast<int64_t>(b) * cv.Hq + kv * r) * kD * 2, r * kD * 2,
                qbar);
  }

  float kc[4];
#pragma unroll
  for (int c = 0; c < 4; ++c) kc[c] = a.scale_log2 * pow2i(2 * c - 64);
  const float kq = a.scale_log2 * pow2i(69);

  const uint8_t* fpbase = cv.fp + a.layer * cv.fp_layer_stride + pair * cv.fp_head_stride;
  const uint8_t* qbase = cv.quant + a.layer * cv.quant_layer_stride + pair * cv.quant_head_stride;

  // load pipeline.  A stage holds: the K rows of fp tile i (desc = i), its V rows (desc = -1-i)
  // or quant tile t (desc = tiles_fp + t).  pending_v >= 0: the V rows of that fp tile come next.
  int issued = 0, pending_v = -1;
  int desc0 = 0, desc1 = 0, desc2 = 0;
  auto issue_next = [&](int cap) {
    const uint8_t* src;
    uint32_t bytes;
    int desc;
    if (pending_v >= 0) {
      desc = -1 - pending_v;
      bytes = kFpTileVOffset;
      src = fpbase + static_cast<int64_t>(pending_v) * kFpTileBytes + kFpTileVOffset;
      pending_v = -1;
    } else {
      if (it >= it_end) return;
      desc = it;
      if (it < a.tiles_fp) {
        bytes = kFpTileVOffset;
        src = fpbase + static_cast<int64_t>(it) * kFpTileBytes;
        pending_v = it;
        ++it;
      } else {
        const int nt = min(min(TPS, cap), it_end - it);
        desc = it | (nt << 24);
        bytes = nt * TILE;
        src = qbase + static_cast<int64_t>(it - a.tiles_fp + qskip) * TILE;
        it += nt;
      }
    }
    const uint32_t s = issued % kStages;
    if (s == 0) desc0 = desc; else if (s == 1) desc1 = desc; else desc2 = desc;
    if (lane == 0) {
      // (debug build: the copy must lie inside this pair's part of the store it reads; a copy that does not is
      // not issued, its barrier never completes and the bounded wait reports it as well)
      const bool inside = desc < a.tiles_fp ? src >= fpbase && src + bytes <= fpbase + cv.fp_head_stride
                                            : src >= qbase && src + bytes <= qbase + cv.quant_head_stride;
      mbar_expect_tx(bar0 + 8 * s, bytes);
      if (LQ_IN_BOUNDS(cv, inside)) bulk_load(stage0 + s * kStageBytes, src, bytes, bar0 + 8 * s);
    }
    ++issued;
  };
  bool failed = false;
  // Only one small load per warp before the query fragments are built: all warps start at the same
  // time, and the first bytes every warp needs should not queue behind everybody's second load.
  // (an overlapped launch starts while other CTAs of the SM are in mid-stream: it fills all its stages at once)
  if (a.early) {
    for (int s = 0; s < kStages; ++s) issue_next(TPS);
  } else {
    issue_next(1);
  }

  // query fragments: B operand, column n -> head 4cb + n/2 (even column = hi, odd = lo of q*s);
  // k-step ks carries the factor 2^(64 - 2*(ks&3)) that cancels the code-position factor
  uint32_t qs[NCB][8][2];
  // Pairs with more CTAs than the last one could fetch the records of in one batch of loads (kMergeOneBatch):
  // every CTA also adds its partial to one sum per pair (DecodeArgs::acc), scaled to a reference score that
  // all of them compute alike: q . k of the token in fp slot 0 (any real score of the pair will do).  Thread
  // h of warp 0 keeps the reference of head h.  (Sums in arrival order: such pairs are not reproducible bit
  // for bit from run to run; the others are.)
  const bool use_acc = a.acc != nullptr && n_ctas_pair > kMergeOneBatch;
  float ref = 0.f;
  uint2 k0row = make_uint2(0u, 0u);
  if (use_acc && warp == 0) k0row = __ldcg(reinterpret_cast<const uint2*>(fpbase) + lane);  // row 0: lane = 4 channels
  {
    int spins = 0;
    const int limit = a.debug_stall ? 256 : kSpinLimit;
    while (!mbar_try_wait(qbar, 0)) {
      if (++spins > limit) { failed = true; break; }
    }
    failed = __any_sync(kFull, failed);
    if (use_acc && warp == 0) {
      const float k0 = bf16lo_f32(k0row.x), k1 = bf16hi_f32(k0row.x), k2 = bf16lo_f32(k0row.y), k3 = bf16hi_f32(k0row.y);
      for (int h = 0; h < r; ++h) {
        const uint2 qq = lds64(qsm + h * (kD * 2) + lane * 8);
        float dot = k0 * bf16lo_f32(qq.x) + k1 * bf16hi_f32(qq.x) + k2 * bf16lo_f32(qq.y) + k3 * bf16hi_f32(qq.y);
#pragma unroll
        for (int o = 16; o; o >>= 1) dot += __shfl_xor_sync(kFull, dot, o);
        if (lane == h) ref = dot * a.scale_log2;
      }
    }
#pragma unroll
    for (int cb = 0; cb < NCB; ++cb) {
      const int head = 4 * cb + (n >> 1);
      const bool valid = head < r;
      const uint32_t qrow = qsm + (valid ? head : 0) * (kD * 2);
#pragma unroll
      for (int ks = 0; ks < 8; ++ks)
#pragma unroll
        for (int w = 0; w < 2; ++w) {
          uint32_t raw;
          asm volatile("ld.shared.u32 %0, [%1];" : "=r"(raw) : "r"(qrow + 2 * (16 * ks + 8 * w + 2 * j)));
          // 2^(64 - 2*(ks&3)) as a bf16 pair: the product is exact (a power of two, no overflow)
          const uint32_t f2 = (static_cast<uint32_t>(127 + 64 - 2 * (ks & 3)) << 7) * 0x00010001u;
          qs[cb][ks][w] = valid ? bf16x2_mul(raw, f2) : 0u;
        }
    }
  }
  if (!a.early)
    for (int s = 1; s < kStages; ++s) issue_next(TPS);
  WarpState<NCB> st;
#pragma unroll
  for (int mt = 0; mt < 8; ++mt) st.out[mt][0] = st.out[mt][1] = st.out[mt][2] = st.out[mt][3] = 0.f;
  st.zacc[0] = st.zacc[1] = st.zacc[2] = st.zacc[3] = 0.f;
#pragma unroll
  for (int cb = 0; cb < NCB; ++cb) { st.m[cb] = -INFINITY; st.l[cb] = 0.f; }
  st.quant_mode = false;

  uint32_t fb0[2] = {0u, 0u}, fb1[2] = {0u, 0u};  // p.v B operands of the fp tile whose V rows are still to come
#pragma unroll 1
  for (int done = 0; done < issued && !failed; ++done) {
    const uint32_t s = done % kStages;
    const uint32_t parity = (done / kStages) & 1;
    {
      int spins = 0;
      bool bad = false;
      while (!mbar_try_wait(bar0 + 8 * s, parity)) {
        if (++spins > kSpinLimit) { bad = true; break; }
      }
      if (__any_sync(kFull, bad)) { failed = true; break; }
    }
    const uint32_t sbase = stage0 + s * kStageBytes;
    const int desc = s == 0 ? desc0 : (s == 1 ? desc1 : desc2);
    if (desc >= a.tiles_fp) {
      // items come in order, so a warp sees all its fp tiles before its first quant tile: from
      // here on the out rows carry the code-position factor (two steps keep the constants normal).
      // An opaque one-trip loop keeps this a branch instead of 64 multiplies and selects per tile.
      int sw = st.quant_mode ? 0 : 1;
      while (sw) {
#pragma unroll
        for (int mt = 0; mt < 8; ++mt) {
          const float f = pow2i(vpos_log2<NCB>(mt) + 70);
          st.out[mt][0] = st.out[mt][0] * 0x1p-70f * f; st.out[mt][1] = st.out[mt][1] * 0x1p-70f * f;
          st.out[mt][2] = st.out[mt][2] * 0x1p-70f * f; st.out[mt][3] = st.out[mt][3] * 0x1p-70f * f;
        }
        st.quant_mode = true;
        sw = a.zero;
      }
      const int nt = desc >> 24;
      float bias2[2][NCB];
      quant_bias<NCB>(qs, sbase + qt_kzero_off() + ((lane >> 4) << 4) + (((lane >> 3) & 1) && nt > 1 ? TILE : 0), kc,
                      bias2);
#pragma unroll 1
      for (int t = 0; t < nt; ++t) {
        float bias[NCB];
#pragma unroll
        for (int cb = 0; cb < NCB; ++cb) bias[cb] = t ? bias2[1][cb] : bias2[0][cb];
        if (PADDED) {
          const int tile = (desc & 0xFFFFFF) - a.tiles_fp + qskip + t;
          uint32_t pad0 = 0u, pad1 = 0u;
          if (tile < qpad_end) {
            pad0 = __ldg(qmask + tile * (G / 32));
            if (G == 64) pad1 = __ldg(qmask + tile * (G / 32) + 1);
          }
          if (pad0 == kFull && (G == 32 || pad1 == kFull)) continue;  // nothing but padding
          process_quant_tile<G, NCB, PL>(st, qs, sbase + t * TILE, bias, kq, lane, oddmask, a.zero, pad0, pad1);
        } else {
          process_quant_tile<G, NCB, PL>(st, qs, sbase + t * TILE, bias, kq, lane, oddmask, a.zero);
        }
      }
    } else if (desc >= 0) {
      if (FUSED && desc == (a.new_slot >> 4))
        patch_new_row(sbase, const_cast<uint8_t*>(fpbase) + static_cast<int64_t>(desc) * kFpTileBytes, a.new_k, pair,
                      a.new_slot & 15, lane);
      const int nv = min(16, a.n_fp - desc * 16);
      uint32_t pad16 = 0u;
      if (fp_padded) pad16 = (__ldg(fpmask + (desc >> 1)) >> (16 * (desc & 1))) & ((1u << nv) - 1u);
      if (PADDED && pad16 == (1u << nv) - 1u) {
        fb0[0] = fb0[1] = fb1[0] = fb1[1] = 0u;  // nothing but padding: its V rows meet p = 0
      } else {
        process_fp_keys<NCB>(st, qs, sbase, nv, kc, lane, oddmask, a.zero, fb0, fb1, pad16);
      }
    } else {
      if (FUSED && -1 - desc == (a.new_slot >> 4))
        patch_new_row(sbase, const_cast<uint8_t*>(fpbase) + static_cast<int64_t>(-1 - desc) * kFpTileBytes + kFpTileVOffset,
                      a.new_v, pair, a.new_slot & 15, lane);
      process_fp_values<NCB>(st, sbase, lane, fb0, fb1);
    }
    __syncwarp();
    issue_next(TPS);
  }
  // the main loop is over: from here on the next kernel of the stream may start launching into
  // the slots that free up (earlier, its waiting CTAs would only take issue slots from this loop)
  if (!a.early) asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  // an overlapped launch (DecodeArgs::early) has read only its own layer's stores so far; the workspace below is
  // shared with the launch before it
  if (a.early) asm volatile("griddepcontrol.wait;" ::: "memory");
  if (failed) {
    // a bulk copy never completed: flag it and contribute nothing (checked again at the end)
    if (lane == 0) atomicOr(a.status, 1);
#pragma unroll
    for (int cb = 0; cb < NCB; ++cb) { st.m[cb] = -INFINITY; st.l[cb] = 0.f; }
  }

  // ---- fold zero term, undo position factors, reduce l over the token lanes ----
  constexpr float kPInv = bf16_pv<NCB>() ? 0x1p-64f : 0x1p8f;
  float o0[8], o1[8];  // NCB == 1: rows (n, n+8) of head j; NCB == 2: unused
#pragma unroll
  for (int mt = 0; mt < 8; ++mt) {
    const int g = (mt * 16) / G;
    // quant mode: out = true * 2^(kPExp + vpos); fp mode: out = true * 2^kPExp
    const float f = st.quant_mode ? pow2i(-vpos_log2<NCB>(mt) - 70) * (bf16_pv<NCB>() ? 0x1p6f : 0x1p78f) : kPInv;
    if (bf16_pv<NCB>()) {
      const float z = __shfl_sync(kFull, st.zacc[0] - st.zacc[1], 4 * g + j) * kPInv;
      o0[mt] = fmaf(st.out[mt][0] - st.out[mt][1], f, z);
      o1[mt] = fmaf(st.out[mt][2] - st.out[mt][3], f, z);
    } else {
      const float z0 = __shfl_sync(kFull, st.zacc[0], 4 * g + j) * kPInv;
      const float z1 = __shfl_sync(kFull, st.zacc[1], 4 * g + j) * kPInv;
      st.out[mt][0] = fmaf(st.out[mt][0], f, z0);
      st.out[mt][1] = fmaf(st.out[mt][1], f, z1);
      st.out[mt][2] = fmaf(st.out[mt][2], f, z0);
      st.out[mt][3] = fmaf(st.out[mt][3], f, z1);
    }
  }
#pragma unroll
  for (int cb = 0; cb < NCB; ++cb) {
    st.l[cb] += __shfl_xor_sync(kFull, st.l[cb], 4);
    st.l[cb] += __shfl_xor_sync(kFull, st.l[cb], 8);
    st.l[cb] += __shfl_xor_sync(kFull, st.l[cb], 16);
    st.l[cb] *= kPInv;
  }

  // ---- CTA merge of the 4 warp states through shared memory (the stages are idle now) ----
  // wout[warp][head][d] with rows padded to 132 floats: conflict-free reads along d
  constexpr int kRow = kD + 4;
  __syncthreads();
  float* wout = reinterpret_cast<float*>(smem);      // [warp][8][kRow]
  float* wm = wout + kWarps * 8 * kRow;              // [warp][8]
  float* wl = wm + kWarps * 8;                       // [warp][8]
  float* wf = wl + kWarps * 8;                       // [warp][8] factor of each warp state in the CTA state
  float* cml = wf + kWarps * 8;                      // [8][2] (m, l) of the CTA state
  float* wsc = cml + 16;                             // [8] scale of the CTA state in the pair's sum
#pragma unroll
  for (int mt = 0; mt < 8; ++mt) {
    if (bf16_pv<NCB>()) {
      float* o = wout + (warp * 8 + j) * kRow + 16 * mt + n;
      o[0] = o0[mt];
      o[8] = o1[mt];  // channel + 8
    } else {
      float* o = wout + (warp * 8 + 2 * j) * kRow + 16 * mt + n;
      o[0] = st.out[mt][0];
      o[kRow] = st.out[mt][1];
      o[8] = st.out[mt][2];
      o[kRow + 8] = st.out[mt][3];
    }
  }
  if (n == 0) {
#pragma unroll
    for (int cb = 0; cb < NCB; ++cb) {
      wm[warp * 8 + 4 * cb + j] = st.m[cb];
      wl[warp * 8 + 4 * cb + j] = st.l[cb];
    }
  }
  __syncthreads();
  if (threadIdx.x < r) {
    const int h = threadIdx.x;
    float M = -INFINITY, L = 0.f;
#pragma unroll
    for (int w = 0; w < kWarps; ++w)
      if (wl[w * 8 + h] > 0.f) M = fmaxf(M, wm[w * 8 + h]);
#pragma unroll
    for (int w = 0; w < kWarps; ++w) {
      const float f = wl[w * 8 + h] > 0.f ? ex2(wm[w * 8 + h] - M) : 0.f;
      wf[w * 8 + h] = f;
      L = fmaf(wl[w * 8 + h], f, L);
    }
    cml[2 * h] = M;
    cml[2 * h + 1] = L;
    // scale of this CTA's partial in the pair's sum; far above the reference the sum could overflow and far
    // below it the scale would underflow: the pair is then flagged and merged from the records instead
    float sc = 0.f;
    if (use_acc && L > 0.f) {
      const float dd = M - ref;
      if (!(dd <= 64.f && dd >= -100.f)) atomicOr(ticket + 1, 1);
      else sc = ex2(dd);
      if (sc > 0.f) atomicAdd(a.acc + static_cast<int64_t>(pair) * kAccStride + kMaxRatio * kD + h, L * sc);
    }
    wsc[h] = sc;
  }
  __syncthreads();
  const int d = threadIdx.x;
  const int64_t rec0 = static_cast<int64_t>(pair) * a.S * r;
  {
    const int64_t rec = rec0 + static_cast<int64_t>(slot) * r;
    for (int h = 0; h < r; ++h) {
      float o = 0.f;
#pragma unroll
      for (int w = 0; w < kWarps; ++w) o = fmaf(wout[(w * 8 + h) * kRow + d], wf[w * 8 + h], o);
      if (n_ctas_pair == 1) {
        // the only CTA of its pair: this is the final result (nothing is written after a wait that gave up)
        if (failed) continue;
        const int64_t oi = (static_cast<int64_t>(b) * cv.Hq + kv * r + h) * kD + d;
        const float res = o / cml[2 * h + 1];
        if (a.out_bf16)
          static_cast<__nv_bfloat16*>(a.out)[oi] = __float2bfloat16_rn(res);
        else
          static_cast<float*>(a.out)[oi] = res;
      } else if (LQ_IN_BOUNDS(cv, slot < a.S)) {
        a.part_o[(rec + h) * kD + d] = o;
        if (use_acc && wsc[h] > 0.f) atomicAdd(a.acc + static_cast<int64_t>(pair) * kAccStride + h * kD + d, o * wsc[h]);
        if (d == 0) {
          a.part_ml[(rec + h) * 2 + 0] = cml[2 * h];
          a.part_ml[(rec + h) * 2 + 1] = cml[2 * h + 1];
        }
      }
    }
  }
  if (n_ctas_pair == 1) {
  } else {
    // ---- second pass, fused: the CTA that completes a pair (last ticket) merges its partials.
    // Nobody waits for anybody: a CTA either finds that it is last, or leaves.
    __syncthreads();  // every partial store of this CTA has been issued
    if (threadIdx.x == 0) {
      __threadfence();  // release, cumulative over the stores the barrier ordered before this thread
      const int last = atomicAdd(ticket, 1) == n_ctas_pair - 1;
      if (last) *ticket = 0;  // ready for the next launch
      *is_last = last;
    }
    __syncthreads();
    if (*is_last) {
      __threadfence();
      // a CTA of the pair whose wait gave up has set the status word before its ticket: the output stays untouched
      const bool healthy = (__ldcg(a.status) & 1) == 0;
      // Fast path: the partials have already been summed on arrival (DecodeArgs::acc); one round trip
      // fetches the sums.  It is taken unless a CTA flagged the pair (partial too far above the
      // reference score) or a denominator is not a positive finite number (everything far below it).
      float* accp = a.acc + static_cast<int64_t>(pair) * kAccStride;
      constexpr int RALL = NCB == 1 ? 4 : 8;  // query heads per KV head this variant serves
      bool fast = use_acc;
      float so[RALL], sl[RALL];
      if (use_acc) {
        // all loads in flight at once: the flag, the denominators, this thread's channel of every head
        const int flagged = *reinterpret_cast<volatile int*>(ticket + 1);
#pragma unroll
        for (int h = 0; h < RALL; ++h) {
          sl[h] = h < r ? __ldcg(accp + kMaxRatio * kD + h) : 1.f;
          so[h] = h < r ? __ldcg(accp + h * kD + d) : 0.f;
        }
        fast = flagged == 0 && healthy;
#pragma unroll
        for (int h = 0; h < RALL; ++h) fast = fast && sl[h] > 0.f && sl[h] < INFINITY;
      }
      if (fast) {
#pragma unroll
        for (int h = 0; h < RALL; ++h) {
          if (h < r) {
            const float res = so[h] / sl[h];
            const int64_t oi = (static_cast<int64_t>(b) * cv.Hq + kv * r + h) * kD + d;
            if (a.out_bf16)
              static_cast<__nv_bfloat16*>(a.out)[oi] = __float2bfloat16_rn(res);
            else
              static_cast<float*>(a.out)[oi] = res;
          }
        }
      } else if (!healthy) {
        // nothing is written
      } else if (NCB == 1 && n_ctas_pair <= kMergeOneBatch) {
        // Up to 4 heads and few records: warp w merges head w on its own -- every record of the head in one
        // batch of loads, the weights spread over the lanes and handed round by shuffles -- and writes the
        // result; no shared memory, no barrier.  (Records are summed in slot order: bit-reproducible.)
        if (warp < r) {
          const int h = warp, nS = n_ctas_pair;
          float4 v[kMergeOneBatch];
#pragma unroll
          for (int sr = 0; sr < kMergeOneBatch; ++sr)
            if (sr < nS) v[sr] = __ldcg(reinterpret_cast<const float4*>(a.part_o + (rec0 + sr * r + h) * kD) + lane);
          const float2 ml = lane < nS ? __ldcg(reinterpret_cast<const float2*>(a.part_ml) + rec0 + lane * r + h)
                                      : make_float2(-INFINITY, 0.f);
          float M = ml.y > 0.f ? ml.x : -INFINITY;
#pragma unroll
          for (int o = 16; o; o >>= 1) M = fmaxf(M, __shfl_xor_sync(kFull, M, o));
          const float e = ml.y > 0.f ? ex2(ml.x - M) : 0.f;
          float L = ml.y * e;
#pragma unroll
          for (int o = 16; o; o >>= 1) L += __shfl_xor_sync(kFull, L, o);
          const float wgt = e / L;
          float4 o = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
          for (int sr = 0; sr < kMergeOneBatch; ++sr) {
            const float w = __shfl_sync(kFull, wgt, sr);
            if (sr < nS) {
              o.x = fmaf(v[sr].x, w, o.x); o.y = fmaf(v[sr].y, w, o.y);
              o.z = fmaf(v[sr].z, w, o.z); o.w = fmaf(v[sr].w, w, o.w);
            }
          }
          const int64_t oi = (static_cast<int64_t>(b) * cv.Hq + kv * r + h) * kD + 4 * lane;
          if (a.out_bf16)
            *reinterpret_cast<uint2*>(static_cast<__nv_bfloat16*>(a.out) + oi) =
                make_uint2(pack_bf16x2(o.x, o.y), pack_bf16x2(o.z, o.w));
          else
            *reinterpret_cast<float4*>(static_cast<float*>(a.out) + oi) = o;
        }
      } else {
      // Warp w sums the records of the CTAs s = w, w + 4, ... for every head (lane = 4 channels,
      // 16-byte loads, kSB * RMAX independent loads in flight; the first batch is issued before the
      // weights are known), and the four warp sums meet in shared memory.  The weight of a record
      // is computed by the lane that loaded its (m, l): warp w normalises heads w, w + 4.
      constexpr int RMAX = NCB == 1 ? 4 : 8;  // query heads per KV head this variant serves
      constexpr int kSB = kMergeOneBatch / kWarps;  // CTA records per batch and warp
      float* sm_w = reinterpret_cast<float*>(smem);  // [S * r] weights
      float* red = sm_w + kMergeMax;                 // [warp][r][128] partial sums
      const int nS = n_ctas_pair;
      auto row = [&](int sr, int h) {
        return __ldcg(reinterpret_cast<const float4*>(a.part_o + (rec0 + sr * r + h) * kD) + lane);
      };
      float4 v[kSB][RMAX];
#pragma unroll
      for (int i = 0; i < kSB; ++i)
#pragma unroll
        for (int h = 0; h < RMAX; ++h)
          if (h < r && warp + 4 * i < nS) v[i][h] = row(warp + 4 * i, h);
      for (int h = warp; h < r; h += kWarps) {
        const float2* mlp = reinterpret_cast<const float2*>(a.part_ml) + rec0 + h;
        const float2 ml0 = lane < nS ? __ldcg(mlp + lane * r) : make_float2(-INFINITY, 0.f);
        auto ml_at = [&](int k0) {  // (m, l) of record k0 + lane; the first 32 stay in registers
          if (k0 == 0) return ml0;
          return k0 + lane < nS ? __ldcg(mlp + (k0 + lane) * r) : make_float2(-INFINITY, 0.f);
        };
        float M = -INFINITY;
        for (int k0 = 0; k0 < nS; k0 += 32) {
          const float2 ml = ml_at(k0);
          if (ml.y > 0.f) M = fmaxf(M, ml.x);
        }
#pragma unroll
        for (int o = 16; o; o >>= 1) M = fmaxf(M, __shfl_xor_sync(kFull, M, o));
        float L = 0.f;
        for (int k0 = 0; k0 < nS; k0 += 32) {
          const float2 ml = ml_at(k0);
          if (ml.y > 0.f) L = fmaf(ml.y, ex2(ml.x - M), L);
        }
#pragma unroll
        for (int o = 16; o; o >>= 1) L += __shfl_xor_sync(kFull, L, o);
        const float inv = 1.0f / L;
        for (int k0 = 0; k0 < nS; k0 += 32) {
          const float2 ml = ml_at(k0);
          if (k0 + lane < nS) sm_w[(k0 + lane) * r + h] = ml.y > 0.f ? ex2(ml.x - M) * inv : 0.f;
        }
      }
      __syncthreads();
      float4 acc[RMAX];
#pragma unroll
      for (int h = 0; h < RMAX; ++h) acc[h] = make_float4(0.f, 0.f, 0.f, 0.f);
      for (int s0 = warp; s0 < nS; s0 += 4 * kSB) {
        if (s0 != warp) {
#pragma unroll
          for (int i = 0; i < kSB; ++i)
#pragma unroll
            for (int h = 0; h < RMAX; ++h)
              if (h < r && s0 + 4 * i < nS) v[i][h] = row(s0 + 4 * i, h);
        }
#pragma unroll
        for (int i = 0; i < kSB; ++i)
#pragma unroll
          for (int h = 0; h < RMAX; ++h)
            if (h < r && s0 + 4 * i < nS) {
              const float w = sm_w[(s0 + 4 * i) * r + h];
              acc[h].x = fmaf(v[i][h].x, w, acc[h].x); acc[h].y = fmaf(v[i][h].y, w, acc[h].y);
              acc[h].z = fmaf(v[i][h].z, w, acc[h].z); acc[h].w = fmaf(v[i][h].w, w, acc[h].w);
            }
      }
#pragma unroll
      for (int h = 0; h < RMAX; ++h)
        if (h < r) reinterpret_cast<float4*>(red + (warp * r + h) * kD)[lane] = acc[h];
      __syncthreads();
      for (int idx = threadIdx.x; idx < r * 32; idx += kWarps * 32) {
        const int h = idx >> 5, c = idx & 31;
        float4 o = reinterpret_cast<const float4*>(red + h * kD)[c];
#pragma unroll
        for (int w = 1; w < kWarps; ++w) {
          const float4 t = reinterpret_cast<const float4*>(red + (w * r + h) * kD)[c];
          o.x += t.x; o.y += t.y; o.z += t.z; o.w += t.w;
        }
        const int64_t oi = (static_cast<int64_t>(b) * cv.Hq + kv * r + h) * kD + 4 * c;
        if (a.out_bf16)
          *reinterpret_cast<uint2*>(static_cast<__nv_bfloat16*>(a.out) + oi) =
              make_uint2(pack_bf16x2(o.x, o.y), pack_bf16x2(o.z, o.w));
        else
          *reinterpret_cast<float4*>(static_cast<float*>(a.out) + oi) = o;
      }
      }  // merge from the records
      if (use_acc) {
        // leave the sums, the flag (and, above, the ticket) at rest for the next launch
        __syncthreads();
        for (int h = 0; h < r; ++h) accp[h * kD + d] = 0.f;
        if (d < r) accp[kMaxRatio * kD + d] = 0.f;
        if (d == 0) ticket[1] = 0;
      }
    }
  }  // ticket path
  if (failed) {
    // give copies still in flight a bounded chance to land before the shared memory is released
    for (int s = 0; s < n_stages(G); ++s) {
      int spins = 0;
      while (!mbar_try_wait(bar0 + 8 * s, 0) && !mbar_try_wait(bar0 + 8 * s, 1) && ++spins < 1024) {}
    }
  }
}

}  // namespace

void plan_decode_mma(DecodeArgs& a, int sm_count, int max_records, int s_override) {
  const int pairs = a.cv.B * a.cv.Hkv;
  const int r = a.cv.Hq / a.cv.Hkv;
  a.tiles_fp = (a.n_fp + kFpTileSlots - 1) / kFpTileSlots;
  a.tiles_quant = static_cast<int>(a.n_quant / a.cv.G);
  const int items = a.tiles_fp + a.tiles_quant / (stage_bytes(a.cv.G, a.cv.planes) / quant_tile_bytes(a.cv.G, a.cv.planes));
  // at most one resident wave of CTAs in total: a CTA that had to wait for a free slot would start
  // when the others finish, and its pair's merge would wait for it
  // the two-column-block variant needs more registers, the 9 KB stages of 4-bit codes at G = 64 more shared memory
  const int ctas_per_sm = r <= 4 && !(a.cv.G == 64 && a.cv.planes == 2) ? kCtasPerSm : kCtasPerSm - 1;
  // A serialised launch fills exactly one resident wave.  An overlapped launch (DecodeArgs::early) takes a third of
  // the slots with CTAs three times as long (at least one CTA per pair): three consecutive launches then share the
  // SMs, every slot stays busy, and the fixed costs of a CTA (start-up, merge, ticket: 4 - 5 us) are paid once per
  // three times the bytes (measured: 1/2 and 1/3 alike, 1/4 worse; 8k workload 15.4 -> 14.4 us per launch).
  const int wave = a.early ? std::max(pairs, ctas_per_sm * sm_count / kOverlapDepth) : ctas_per_sm * sm_count;
  int S = s_override > 0 ? s_override : wave / pairs;
  S = std::min(S, (items + kWarps - 1) / kWarps);  // at least one item per warp
  S = std::min(S, max_records - 1);
  S = std::min(S, kMergeMax / r - 1);
  S = std::max(S, 1);
  // S CTAs for every pair, one more for the first n_extra pairs, so that the grid fills the wave
  // exactly: every SM then carries the same number of CTAs (an SM with 4 CTAs runs each of them a
  // third slower than an SM with 3, and work does not move between pairs)
  int extra = 0;
  // (an overlapped launch with one CTA per pair stays that way: such a CTA writes its result without any merge)
  if (s_override <= 0 && S + 1 <= max_records && (S + 1) * kWarps <= items && !(a.early && S == 1)) {
    extra = wave - S * pairs;
    extra = std::max(0, std::min(extra, pairs));
  }
  a.n_extra = extra;
  a.S = S + 1;  // record stride; pairs >= n_extra use S of them
}

int max_ctas_decode_mma(int sm_count) { return kCtasPerSm * sm_count; }

int plan_decode_mma_padded(const DecodeArgs& a, int sm_count, int max_records, const int32_t* rowinfo_host,
                           int32_t* cta_map, int32_t* pair_ctas, int* stride, bool overlapped) {
  const int pairs = a.cv.B * a.cv.Hkv;
  const int r = a.cv.Hq / a.cv.Hkv;
  const int tiles_fp = (a.n_fp + kFpTileSlots - 1) / kFpTileSlots;
  const int tiles_quant = static_cast<int>(a.n_quant / a.cv.G);
  const int tps = stage_bytes(a.cv.G, a.cv.planes) / quant_tile_bytes(a.cv.G, a.cv.planes);
  const int slots = (r <= 4 && !(a.cv.G == 64 && a.cv.planes == 2) ? kCtasPerSm : kCtasPerSm - 1) * sm_count;
  const int wave = overlapped ? std::max(pairs, slots / kOverlapDepth) : slots;  // as in plan_decode_mma
  const int cap_records = std::max(1, std::min(max_records, kMergeMax / r));
  std::vector<int64_t> work(pairs);
  std::vector<int> cap(pairs);
  int64_t total = 0;
  for (int p = 0; p < pairs; ++p) {
    const int tq = std::max(0, tiles_quant - rowinfo_host[4 * (p / a.cv.Hkv) + 0]);
    work[p] = static_cast<int64_t>(tiles_fp) * fp_cost8(r <= 4 ? 1 : 2) + 8LL * tq;  // the kernel's cost line
    const int items = tiles_fp + tq / tps;
    cap[p] = std::max(1, std::min(cap_records, items / kWarps));  // at least one item per warp
    total += work[p];
  }
  // largest-remainder shares of one wave, clipped to the caps
  int given = 0;
  std::vector<std::pair<int64_t, int>> rest(pairs);
  for (int p = 0; p < pairs; ++p) {
    const int64_t share = total > 0 ? work[p] * wave / total : 0;
    pair_ctas[p] = static_cast<int32_t>(std::max<int64_t>(1, std::min<int64_t>(share, cap[p])));
    rest[p] = {total > 0 ? work[p] * wave % total : 0, p};
    given += pair_ctas[p];
  }
  std::sort(rest.begin(), rest.end(), [](const std::pair<int64_t, int>& x, const std::pair<int64_t, int>& y) {
    return x.first != y.first ? x.first > y.first : x.second < y.second;
  });
  for (bool progress = true; given < wave && progress;) {
    progress = false;
    for (int i = 0; i < pairs && given < wave; ++i) {
      const int p = rest[i].second;
      if (pair_ctas[p] < cap[p]) {
        ++pair_ctas[p];
        ++given;
        progress = true;
      }
    }
  }
  while (given > wave) {  // the minimum of one CTA per pair overshot the wave: take from the largest
    int big = 0;
    for (int p = 1; p < pairs; ++p)
      if (pair_ctas[p] > pair_ctas[big]) big = p;
    if (pair_ctas[big] <= 1) break;
    --pair_ctas[big];
    --given;
  }
  // slot-major order: every pair gets CTAs of every launch rank of the SMs
  int n = 0, most = 1;
  for (int p = 0; p < pairs; ++p) most = std::max(most, static_cast<int>(pair_ctas[p]));
  for (int slot = 0; slot < most; ++slot)
    for (int p = 0; p < pairs; ++p)
      if (slot < pair_ctas[p]) cta_map[n++] = p | (slot << 16);
  *stride = most;
  return n;
}

cudaError_t launch_decode_mma(const DecodeArgs& a, cudaStream_t st) {
  const int r = a.cv.Hq / a.cv.Hkv;
  void (*kern)(DecodeArgs) = nullptr;
  const bool fused = a.new_k != nullptr;
  const bool padded = a.rowinfo != nullptr;
#define LQ_PICK2(G_, N_, P_)                                                                      \
  (fused ? (padded ? lq_decode_mma_kernel<G_, N_, P_, true, true> : lq_decode_mma_kernel<G_, N_, P_, true, false>) \
         : (padded ? lq_decode_mma_kernel<G_, N_, P_, false, true> : lq_decode_mma_kernel<G_, N_, P_, false, false>))
#define LQ_PICK(G_, P_) kern = r <= 4 ? LQ_PICK2(G_, 1, P_) : LQ_PICK2(G_, 2, P_)
  if (a.cv.G == 32 && a.cv.planes == 1) LQ_PICK(32, 1);
  else if (a.cv.G == 32 && a.cv.planes == 2) LQ_PICK(32, 2);
  else if (a.cv.G == 64 && a.cv.planes == 1) LQ_PICK(64, 1);
  else if (a.cv.G == 64 && a.cv.planes == 2) LQ_PICK(64, 2);
  else return cudaErrorInvalidValue;
#undef LQ_PICK
#undef LQ_PICK2
  static_assert(kSmemStages >= static_cast<int>((kWarps * 8 * (kD + 4) + 3 * kWarps * 8 + 16 + 8) * sizeof(float)) &&
                    kSmemStages >= (kMergeMax + kWarps * kMaxRatio * kD) * 4,
                "merge scratch");
  // opt in to the dynamic shared memory size once per (device, kernel variant)
  static bool configured[64][32] = {};
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  const int variant = (padded ? 16 : 0) + (fused ? 8 : 0) + (a.cv.planes == 2 ? 4 : 0) + (a.cv.G == 64 ? 2 : 0) + (r <= 4 ? 0 : 1);
  if (dev < 0 || dev >= 64 || !configured[dev][variant]) {
    e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_bytes(a.cv.G, a.cv.planes));
    if (e != cudaSuccess) return e;
    if (dev >= 0 && dev < 64) configured[dev][variant] = true;
  }
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(padded ? a.n_ctas : a.cv.B * a.cv.Hkv * (a.S - 1) + a.n_extra);
  cfg.blockDim = dim3(kWarps * 32);
  cfg.dynamicSmemBytes = smem_bytes(a.cv.G, a.cv.planes);
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kern, a);
}

}  // namespace lq

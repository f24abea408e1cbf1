// tcgen05 decode attention over the mixed cache (LQ_KERNEL_UMMA), on the row layout (lq_layout.cuh).
//
// Both contractions of Eq. 2 run on the 5th-generation tensor core with M = 128 rows, operands
// unpacked straight into tensor memory (TMEM) and accumulators kept in TMEM:
//
//   q.k  rows = 128 tokens (4 key groups at G = 32, 2 at G = 64), K = channels (8 k-steps of 16),
//        A = the 2-bit key codes as bf16 subnormals, written to TMEM by the thread that owns the token
//        (one AND per two codes), B = q * key scale from shared memory.  The key scale belongs to
//        (group, channel), so it cannot sit on K alone: B carries one block of columns per key group,
//        N = groups x heads x {hi, lo} (q*s split exactly into two bf16), and a token reads the score
//        columns of its own group.  The key zero contributes one bias q.zero per (group, head), computed
//        with fp32 FMAs by the threads that build B.
//   p.v  rows = 128 channels, K = tokens, A = the value codes (thread = channel), B = p * value scale,
//        N-contiguous in shared memory (the thread that owns a token writes its columns as 16-byte
//        vectors), one block of columns per value group; a channel reads the columns of its own group.
//        The value zero term sum_t p_t * zero_t is kept in registers.
//   bf16 rows of the full-precision store: A straight from shared memory (no unpacking): K rows as a
//        K-major operand, V rows as an MN-major operand, units of 32 tokens.
//
// One CTA = 4 worker warps (thread = token for q.k = channel for p.v = TMEM lane), one warp that issues the q.k
// MMAs, one that issues the p.v MMAs and one that issues the bulk copies.  Per item j the workers read the scores
// of item j, prepare the q.k operands of item j + 1 (q*s, q.zero, key codes) so that its MMAs run during the
// softmax of item j, then build B of p.v and unpack the value codes of item j (two buffers, so that the p.v MMAs
// of item j - 1 may still be running).  Workers wake the issuing warps through named barriers (bar.arrive /
// bar.sync: hardware barriers, ~36 cycles, nobody polls); MMA completion comes back through tcgen05.commit on
// mbarriers, which by then have normally completed (an issuing thread manages one tcgen05.mma per ~62 cycles
// whatever the tile width, so the two streams get a thread each).  Every mbarrier wait is bounded; a warp whose
// wait ran out sets bit 0 of the status word, attempts no further wait and keeps taking part in every barrier,
// so that the CTA runs to its end, frees its tensor memory and returns.
//
// Work partition: all (b, kv) pairs lie on one cost line (fp units, then 128-token super-tiles, weighted
// by their bytes) that is cut into equal ranges, one per CTA (2 CTAs per SM); a CTA whose range spans
// several pairs handles them one after the other ("segments").  Every segment ends in a split-K partial
// (m, l, o); the CTA that completes a pair (arrival counter in items) merges the partials (Eq. 3: any
// order).
#include <cuda_bf16.h>

#include <algorithm>

#include "lq_kernels.cuh"

#ifdef LQ_UMMA_TRACE
#include <cstdio>
#define TR(role, j, k) do { if (blockIdx.x == LQ_UMMA_TRACE && (j) < 12) trace[role][j][k] = static_cast<uint32_t>(clock64()); } while (0)
#else
#define TR(role, j, k) do { } while (0)
#endif

#ifndef LQ_UMMA_EXTRA_SMEM
#define LQ_UMMA_EXTRA_SMEM 0  /* experiments: extra dynamic shared memory (lowers the CTAs per SM) */
#endif

namespace lq {

namespace {

constexpr int kGroup = 128;            // threads of a worker group = TMEM lanes
constexpr int kGroupWarps = 4;         // barriers count one arrival per warp
constexpr int kThreads = 224;          // worker warps 0-3, q.k issuer warp, p.v issuer warp, producer warp
constexpr int kWarpQK = 4, kWarpPV = 5, kWarpLoad = 6;
constexpr int kBarQK = 1;              // named barriers: q.k operands of an item are in place (workers -> q.k issuer),
constexpr int kBarPV0 = 2;             // p.v operands of an even / odd item are in place (workers -> p.v issuer; 2 and 3),
constexpr int kBarW = 4;               // rendezvous of the worker warps
constexpr int kStages = 4;
constexpr int kStageBytes = 16384;     // one fp unit, or one super-tile (12 KB at G = 32, 10 KB at G = 64)
constexpr int kSpin = 1 << 22;
constexpr uint32_t kFullMask = 0xFFFFFFFFu;
constexpr int kWeightFp = 8;           // cost of one fp unit in units of 2 KB

// ---- PTX wrappers --------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return static_cast<uint32_t>(__cvta_generic_to_shared(p)); }
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
// non-blocking test of a phase (try_wait may suspend the thread, and it comes back late: measured ~1000 cycles
// per wait that was not satisfied at once)
__device__ __forceinline__ uint32_t mbar_test_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok;
}
// bounded wait: false when the phase did not complete within the poll limit
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, int limit = kSpin) {
  for (int spin = 0; spin < limit; ++spin) {
    if (mbar_test_wait(bar, parity)) return true;
  }
  return false;
}
// One arrival per warp (128 arrivals on one barrier word serialise): the warp's lanes have done their fences,
// __syncwarp orders their writes before lane 0's releasing arrival.
__device__ __forceinline__ void warp_arrive(uint32_t bar) {
  __syncwarp();
  if ((threadIdx.x & 31) == 0) mbar_arrive(bar);
}
// named barriers (hardware barriers: the waiting warp sleeps, nobody polls)
template <int ID, int COUNT>
__device__ __forceinline__ void named_sync() { asm volatile("bar.sync %0, %1;" ::"n"(ID), "n"(COUNT) : "memory"); }
template <int ID, int COUNT>
__device__ __forceinline__ void named_arrive() { asm volatile("bar.arrive %0, %1;" ::"n"(ID), "n"(COUNT) : "memory"); }
__device__ __forceinline__ void bulk_load(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst),
               "l"(src), "r"(bytes), "r"(bar)
               : "memory");
}
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tc_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
// shared-memory matrix descriptor, no swizzle: start address, stride between core matrices along K (lbo)
// and along M / N (sbo), all in bytes (multiples of 16)
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr, uint32_t lbo, uint32_t sbo) {
  return static_cast<uint64_t>((addr >> 4) & 0x3FFF) | (static_cast<uint64_t>((lbo >> 4) & 0x3FFF) << 16) |
         (static_cast<uint64_t>((sbo >> 4) & 0x3FFF) << 32) | (1ull << 46);
}
// instruction descriptor: fp32 accumulate, bf16 x bf16, M = 128, given N and major-ness of A and B (1 = MN-major)
__host__ __device__ constexpr uint32_t instr_desc(int N, int a_mn, int b_mn) {
  return (1u << 4) | (1u << 7) | (1u << 10) | (static_cast<uint32_t>(a_mn) << 15) | (static_cast<uint32_t>(b_mn) << 16) |
         (static_cast<uint32_t>(N >> 3) << 17) | (static_cast<uint32_t>(128 >> 4) << 24);
}
__device__ __forceinline__ void mma_ts(uint32_t d, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc, uint32_t acc) {
  asm volatile(
      "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}" ::"r"(d),
      "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(acc)
      : "memory");
}
__device__ __forceinline__ void mma_ss(uint32_t d, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t acc) {
  asm volatile(
      "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}" ::"r"(d),
      "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(acc)
      : "memory");
}
// 32 lanes x NC 32-bit columns between registers and TMEM (thread = lane of the warp's quarter)
template <int NC>
__device__ __forceinline__ void tmem_ld(uint32_t taddr, uint32_t (&r)[NC]) {
  static_assert(NC == 4 || NC == 8 || NC == 16 || NC == 32 || NC == 64, "shape");
  if constexpr (NC == 4) {
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x4.b32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(taddr));
  } else if constexpr (NC == 8) {
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7])
                 : "r"(taddr));
  } else if constexpr (NC == 16) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
          "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
        : "r"(taddr));
  } else if constexpr (NC == 32) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,"
        "%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
          "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
          "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
          "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr));
  } else {
    uint32_t(&lo)[32] = reinterpret_cast<uint32_t(&)[32]>(r[0]);
    uint32_t(&hi)[32] = reinterpret_cast<uint32_t(&)[32]>(r[32]);
    tmem_ld<32>(taddr, lo);
    tmem_ld<32>(taddr + 32, hi);
  }
}
template <int NC>
__device__ __forceinline__ void tmem_st(uint32_t taddr, const uint32_t (&r)[NC]) {
  static_assert(NC == 16 || NC == 32 || NC == 64, "shape");
  if constexpr (NC == 16) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16};" ::"r"(taddr),
        "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]), "r"(r[9]),
        "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15])
        : "memory");
  } else if constexpr (NC == 32) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,"
        "%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31,%32};" ::"r"(taddr),
        "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]), "r"(r[9]),
        "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]), "r"(r[16]), "r"(r[17]), "r"(r[18]),
        "r"(r[19]), "r"(r[20]), "r"(r[21]), "r"(r[22]), "r"(r[23]), "r"(r[24]), "r"(r[25]), "r"(r[26]), "r"(r[27]),
        "r"(r[28]), "r"(r[29]), "r"(r[30]), "r"(r[31])
        : "memory");
  } else {
    const uint32_t(&lo)[32] = reinterpret_cast<const uint32_t(&)[32]>(r[0]);
    const uint32_t(&hi)[32] = reinterpret_cast<const uint32_t(&)[32]>(r[32]);
    tmem_st<32>(taddr, lo);
    tmem_st<32>(taddr + 32, hi);
  }
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
__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
// pack two floats as bf16: `lo` into bits [15:0], `hi` into bits [31:16]
__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
  uint32_t d;
  asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(d) : "f"(hi), "f"(lo));
  return d;
}
__device__ __forceinline__ float bf16lo_f32(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16hi_f32(uint32_t w) { return __uint_as_float(w & 0xFFFF0000u); }
__device__ __forceinline__ float pow2i(int k) { return __int_as_float((k + 127) << 23); }
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
__device__ __forceinline__ void sts128(uint32_t addr, uint32_t a, uint32_t b, uint32_t c, uint32_t d) {
  asm volatile("st.shared.v4.u32 [%0], {%1,%2,%3,%4};" ::"r"(addr), "r"(a), "r"(b), "r"(c), "r"(d) : "memory");
}
// x (fp32) as a bf16 pair hi + lo, hi in the low half: hi = RN(x), lo = RN(x - hi)
__device__ __forceinline__ uint32_t split_hi_lo(float x) {
  const float hi = bf16lo_f32(pack_bf16x2(x, 0.f));
  return pack_bf16x2(x, x - hi);
}

// ---- geometry of one instantiation ------------------------------------------------------------------
// G: key / value group size.  HP: query heads per KV head, padded to 2, 4 or 8.
template <int G, int HP>
struct Geo {
  static constexpr int NGS = 128 / G;            // key groups per 128-token super-tile = value groups per token
  static constexpr int NR = 2 * HP;              // columns per group: (hi, lo) of every head
  static constexpr int NRAW = NGS * NR;
  static constexpr int N = NRAW < 16 ? 16 : NRAW;  // MMA width of q.k and of p.v
  static constexpr int VBUF = N <= 32 ? 2 : 1;   // buffers for the unpacked value codes and for B of p.v
  static constexpr int TILE = 1024 + 64 * G;     // bytes of one key group in the store
  static constexpr int WQ = NGS * TILE / 2048;   // cost of a super-tile in units of 2 KB
  static constexpr int BITEMS = NGS * 8 * HP;    // work items of the B build: (group, 8-channel chunk, head pair)
  static constexpr int BROUNDS = (BITEMS + kGroup - 1) / kGroup;
  // TMEM columns
  static constexpr int COL_AK = 0;
  static constexpr int COL_AV = 64;
  static constexpr int COL_S = COL_AV + 64 * VBUF;
  static constexpr int COL_O = COL_S + N;
  static constexpr int COLS = 256;
  static_assert(COL_O + N <= COLS, "tensor memory");
  // shared memory
  static constexpr int LBO_QK = (N / 8) * 128 + 16;   // stride between 8-channel chunks of B(q.k): padded against bank conflicts
  static constexpr int BQK_BYTES = 16 * LBO_QK;
  static constexpr int LBO_QFP = 2 * 128 + 16;        // B of the bf16 keys: 16 rows (heads), K-major
  static constexpr int BQFP_BYTES = 16 * LBO_QFP;
  static constexpr int BPV_BYTES = (N / 8) * 2048;    // B(p.v), N-contiguous: [8-column block][token / 8][token % 8][8 columns]
  static constexpr int OFF_STAGES = 0;
  static constexpr int OFF_BQK = kStages * kStageBytes;
  static constexpr int OFF_BPV = OFF_BQK + BQK_BYTES;
  static constexpr int OFF_BQFP = OFF_BPV + VBUF * BPV_BYTES;
  static constexpr int OFF_Q = OFF_BQFP + BQFP_BYTES;           // 2 x (8 heads x 256 B)
  static constexpr int OFF_BIAS = OFF_Q + 2 * kMaxRatio * kD * 2;  // [2][NGS][8] floats
  static constexpr int OFF_MAX = OFF_BIAS + 2 * 4 * 8 * 4;         // [2][16] ints: 8 ordered floats + flag, one set per item parity
  static constexpr int OFF_RED = OFF_MAX + 128;                    // [4 warps][NGS*HP + HP] floats of the segment reduction
  static constexpr int OFF_BARS = OFF_RED + 4 * 48 * 4;
  static constexpr int N_BARS = 2 * kStages + 7;
  static constexpr int OFF_MISC = OFF_BARS + N_BARS * 8;          // tmem base, is_last
  static constexpr int SMEM = OFF_MISC + 32 + 128;  // + one byte per record slot of a pair (contributors)
  // the tensor core reads 128 rows behind the start of an fp unit (rows past the unit are never used): they must
  // lie inside the allocation
  static_assert(OFF_STAGES + (kStages - 1) * kStageBytes + 32768 <= SMEM, "A window of the last stage");
  static_assert(2 * (SMEM + 1024) <= 233472, "two CTAs per SM");
};

// order-preserving map between floats and ints (for atomicMax on scores)
__device__ __forceinline__ int ord_f2i(float f) {
  const int i = __float_as_int(f);
  return i >= 0 ? i : i ^ 0x7FFFFFFF;
}
__device__ __forceinline__ float ord_i2f(int i) { return __int_as_float(i >= 0 ? i : i ^ 0x7FFFFFFF); }

// ---- the cut of the global cost line ------------------------------------------------------------------
struct Cut {
  int P, I, F, Q, C, wq, n_ctas;
  // first global item (pair * I + item) of CTA c: the first item whose start lies at or behind the CTA's cut
  __device__ __forceinline__ int64_t first_item(int c) const {
    if (c >= n_ctas) return static_cast<int64_t>(P) * I;
    const int64_t x = static_cast<int64_t>(c) * P * C / n_ctas;
    const int64_t pair = x / C;
    const int y = static_cast<int>(x - pair * C);
    const int li = y <= F * kWeightFp ? (y + kWeightFp - 1) / kWeightFp : F + (y - F * kWeightFp + wq - 1) / wq;
    return pair * I + li;
  }
  // no CTA below this one works for `pair`
  __device__ __forceinline__ int cta_min(int64_t pair) const { return static_cast<int>(pair * n_ctas / P); }
};

template <int G, int HP>
__global__ void __launch_bounds__(kThreads, 2) lq_decode_umma_kernel(DecodeArgs a) {
  using GE = Geo<G, HP>;
  constexpr int NGS = GE::NGS, NR = GE::NR, N = GE::N, VBUF = GE::VBUF, TILE = GE::TILE;
  extern __shared__ __align__(1024) uint8_t smem[];
#ifdef LQ_UMMA_TRACE
  __shared__ uint32_t trace[4][12][12];
  for (int i = threadIdx.x; i < 4 * 12 * 12; i += kThreads) (&trace[0][0][0])[i] = 0;
#endif
  const CacheView& cv = a.cv;
  const int r = cv.Hq / cv.Hkv;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const uint32_t sbase = smem_u32(smem);

  // mbarriers
  const uint32_t bar0 = sbase + GE::OFF_BARS;
  auto bar_full = [&](int s) { return bar0 + 8 * s; };
  auto bar_empty = [&](int s) { return bar0 + 8 * (kStages + s); };
  const uint32_t bar_qfull0 = bar0 + 8 * (2 * kStages);       // [2] query rows of a segment have landed
  const uint32_t bar_qfree0 = bar_qfull0 + 16;                // [2] ... have been taken into registers
  const uint32_t bar_s_ready = bar_qfree0 + 16;               // q.k MMAs of an item are complete
  const uint32_t bar_pv_done0 = bar_s_ready + 8;              // [2] p.v MMAs of an even / odd item are complete
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + GE::OFF_MISC);
  int* is_last_s = reinterpret_cast<int*>(smem + GE::OFF_MISC + 8);

  Cut cut;
  cut.P = cv.B * cv.Hkv; cut.I = a.u_items; cut.F = a.u_fp_units; cut.Q = a.u_supertiles; cut.C = a.u_cost;
  cut.wq = GE::WQ; cut.n_ctas = gridDim.x;
  const int64_t item_lo = cut.first_item(blockIdx.x), item_hi = cut.first_item(blockIdx.x + 1);
  const int n_items = static_cast<int>(item_hi - item_lo);
  const int64_t pair0 = item_lo / cut.I;
  const int li0 = static_cast<int>(item_lo - pair0 * cut.I);

  if (tid == 0) {
    for (int s = 0; s < kStages; ++s) {
      mbar_init(bar_full(s), 1);
      mbar_init(bar_empty(s), kGroupWarps + 1);   // the worker warps and the commit behind the item's p.v MMAs
    }
    for (int i = 0; i < 2; ++i) {
      mbar_init(bar_qfull0 + 8 * i, 1);
      mbar_init(bar_qfree0 + 8 * i, kGroupWarps);
      mbar_init(bar_pv_done0 + 8 * i, 1);
    }
    mbar_init(bar_s_ready, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    fence_async_smem();
    int* mx = reinterpret_cast<int*>(smem + GE::OFF_MAX);
    for (int i = 0; i < 2; ++i) {
      for (int h = 0; h < 8; ++h) mx[16 * i + h] = ord_f2i(-INFINITY);
      mx[16 * i + 8] = 0;
    }
  }
  if (warp == kWarpQK && n_items > 0) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(GE::COLS)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;
  // programmatic dependent launch: nothing an earlier kernel may still be writing is read above
  asm volatile("griddepcontrol.wait;" ::: "memory");

  const uint8_t* fp_layer = cv.fp + a.layer * cv.fp_layer_stride;
  const uint8_t* quant_layer = cv.quant + a.layer * cv.quant_layer_stride;
  const int wt = tid & (kGroup - 1);                       // token / channel / TMEM lane of a worker thread
  const uint32_t lane_base = static_cast<uint32_t>((warp & 3) * 32) << 16;

  if (n_items > 0 && warp == kWarpLoad) {
    // ================= producer of the bulk copies (one thread) =================
    if (lane == 0) {
      bool failed = false;
      int seg = 0;
      int64_t lpair = pair0;
      int lli = li0;
      for (int j = 0; j < n_items && !failed; ++j) {
        const int s = j % kStages;
        if (j >= kStages && !mbar_wait(bar_empty(s), ((j / kStages) - 1) & 1)) { failed = true; break; }
        if (j == 0 || lli == 0) {
          // first item of a segment: its query rows (double-buffered by segment)
          const int qb = seg & 1;
          if (seg >= 2 && !mbar_wait(bar_qfree0 + 8 * qb, ((seg >> 1) - 1) & 1)) { failed = true; break; }
          const int b = static_cast<int>(lpair / cv.Hkv), kv = static_cast<int>(lpair % cv.Hkv);
          mbar_expect_tx(bar_qfull0 + 8 * qb, r * kD * 2);
          if (!a.debug_stall)
            bulk_load(sbase + GE::OFF_Q + qb * (kMaxRatio * kD * 2),
                      static_cast<const uint8_t*>(a.q) + (static_cast<int64_t>(b) * cv.Hq + kv * r) * kD * 2, r * kD * 2,
                      bar_qfull0 + 8 * qb);
          ++seg;
        }
        const uint8_t* src;
        uint32_t bytes;
        if (lli < cut.F) {
          src = fp_layer + lpair * cv.fp_head_stride + static_cast<int64_t>(lli) * kFpUnitBytes;
          bytes = kFpUnitBytes;
        } else {
          const int st = lli - cut.F;
          src = quant_layer + lpair * cv.quant_head_stride + static_cast<int64_t>(st) * NGS * TILE;
          bytes = min(NGS, a.tiles_quant - st * NGS) * TILE;
        }
        // (debug build: the copy must lie inside this pair's part of the store it reads)
        const uint8_t* lo = lli < cut.F ? fp_layer + lpair * cv.fp_head_stride : quant_layer + lpair * cv.quant_head_stride;
        const int64_t extent = lli < cut.F ? cv.fp_head_stride : cv.quant_head_stride;
        mbar_expect_tx(bar_full(s), bytes);
        if (LQ_IN_BOUNDS(cv, lpair < cut.P && src >= lo && src + bytes <= lo + extent))
          bulk_load(sbase + GE::OFF_STAGES + s * kStageBytes, src, bytes, bar_full(s));
        if (++lli == cut.I) { lli = 0; ++lpair; }
      }
      if (failed) atomicOr(a.status, 1);
    }
  } else if (n_items > 0 && warp == kWarpPV) {
    // ================= p.v issuer: woken by the workers through a named barrier, never polls =================
    constexpr uint32_t idesc_q = instr_desc(N, 0, 1);   // A (value codes) from TMEM, B N-contiguous
    constexpr uint32_t idesc_f = instr_desc(N, 1, 1);   // A = bf16 V rows from shared memory, MN-major
    int li = li0;
    for (int j = 0; j < n_items; ++j) {
      const int s = j % kStages;
      const int vb = j % VBUF;
      if (j & 1) named_sync<kBarPV0 + 1, kGroup + 32>(); else named_sync<kBarPV0, kGroup + 32>();
      tc_fence_after();
      if (lane == 0) {
        TR(3, j, 0);
        const uint32_t acc0 = (j == 0 || li == 0) ? 0u : 1u;  // the first item of a segment overwrites O
        const uint32_t bpv = sbase + GE::OFF_BPV + vb * GE::BPV_BYTES;
        if (li < cut.F) {
          const int nv = min(kFpUnitSlots, a.n_fp - li * kFpUnitSlots);
          const uint32_t vrows = sbase + GE::OFF_STAGES + s * kStageBytes + kFpUnitVOffset;
          for (int ks = 0; ks < (nv + 15) / 16; ++ks)
            mma_ss(tmem + GE::COL_O, smem_desc(vrows + ks * 4096, 2048, 128), smem_desc(bpv + ks * 256, 128, 2048),
                   idesc_f, ks ? 1u : acc0);
        } else {
#pragma unroll
          for (int ks = 0; ks < 8; ++ks)
            mma_ts(tmem + GE::COL_O, tmem + GE::COL_AV + 64 * vb + 8 * ks, smem_desc(bpv + ks * 256, 128, 2048),
                   idesc_q, ks ? 1u : acc0);
        }
        tc_commit(bar_pv_done0 + 8 * (j & 1));
        tc_commit(bar_empty(s));
        TR(3, j, 1);
      }
      __syncwarp();
      if (++li == cut.I) li = 0;
    }
  } else if (n_items > 0 && warp == kWarpQK) {
    // ================= q.k issuer =================
    constexpr uint32_t idesc_q = instr_desc(N, 0, 0);    // A (key codes) from TMEM, B = q*s K-major
    constexpr uint32_t idesc_f = instr_desc(16, 0, 0);   // A = bf16 K rows from shared memory, B = q K-major
    int li = li0;
    for (int j = 0; j < n_items; ++j) {
      const int s = j % kStages;
      named_sync<kBarQK, kGroup + 32>();
      tc_fence_after();
      if (lane == 0) {
        TR(2, j, 0);
        if (li < cut.F) {
          const uint32_t krows = sbase + GE::OFF_STAGES + s * kStageBytes;
#pragma unroll
          for (int ks = 0; ks < 8; ++ks)
            mma_ss(tmem + GE::COL_S, smem_desc(krows + ks * 256, 128, 2048),
                   smem_desc(sbase + GE::OFF_BQFP + ks * 2 * GE::LBO_QFP, GE::LBO_QFP, 128), idesc_f, ks ? 1u : 0u);
        } else {
          const uint32_t bq = sbase + GE::OFF_BQK;
#pragma unroll
          for (int ks = 0; ks < 8; ++ks)
            mma_ts(tmem + GE::COL_S, tmem + GE::COL_AK + 8 * ks, smem_desc(bq + ks * 2 * GE::LBO_QK, GE::LBO_QK, 128),
                   idesc_q, ks ? 1u : 0u);
        }
        tc_commit(bar_s_ready);
        TR(2, j, 1);
      }
      __syncwarp();
      if (++li == cut.I) li = 0;
    }
  } else if (n_items > 0 && warp < kGroupWarps) {
    // ================= worker warps: thread = token (q.k) = channel (p.v) = TMEM lane =================
    // Per item j, in this order: read the scores of item j; prepare the q.k operands of item j + 1 (q*s and the
    // q.zero bias into shared memory, the key codes into tensor memory) and hand them to the q.k issuer; online
    // softmax of item j; B of p.v and the value codes of item j; hand them to the p.v issuer.  The MMAs of item
    // j + 1 (q.k) and of item j (p.v) run while the workers go on, so the waits below are normally satisfied.
    bool failed = false;   // warp-uniform: after a wait that ran out no wait is attempted any more; the warp keeps
                           // taking part in every barrier so that nobody is left waiting for it
    const int spin_limit = a.debug_stall ? 256 : kSpin;
    auto wait = [&](uint32_t bar, uint32_t parity) {
      if (!failed) failed = !__all_sync(kFullMask, mbar_wait(bar, parity, spin_limit) ? 1 : 0);
    };
    uint32_t qpk[GE::BROUNDS][2][4];   // query of the B build: item (group g, chunk c, head pair hp) per round
    float qf[GE::BROUNDS][2][8];
    int kli = li0, kseg = -1;          // position of the next item whose q.k operands are prepared
    int64_t kpair = pair0;

    // ---- q.k operands of item j: B = q*s and the bias in shared memory, key codes in tensor memory ----
    auto prep = [&](int j) {
      const int s = j % kStages;
      const uint32_t stage = sbase + GE::OFF_STAGES + s * kStageBytes;
      if (j == 0 || kli == 0) {
        // segment start: the query rows of the pair into registers; B of the bf16 keys
        ++kseg;
        const int qb = kseg & 1;
        wait(bar_qfull0 + 8 * qb, (kseg >> 1) & 1);
        const uint32_t qs = sbase + GE::OFF_Q + qb * (kMaxRatio * kD * 2);
#pragma unroll
        for (int rd = 0; rd < GE::BROUNDS; ++rd) {
          const int it = tid + rd * kGroup;
          const int c = it & 15, hp = (it >> 4) % (HP / 2);
#pragma unroll
          for (int h2 = 0; h2 < 2; ++h2) {
            const int h = 2 * hp + h2;
            uint4 qw = make_uint4(0u, 0u, 0u, 0u);
            if (h < r && it < GE::BITEMS) qw = lds128(qs + h * (kD * 2) + 16 * c);
            const uint32_t q4[4] = {qw.x, qw.y, qw.z, qw.w};
#pragma unroll
            for (int mm = 0; mm < 4; ++mm) {
              // element pair mm of the chunk sits at code position 2*mm: times 2^(64 - 2*mm), exact
              const uint32_t f2 = (static_cast<uint32_t>(127 + 64 - 2 * mm) << 7) * 0x00010001u;
              qpk[rd][h2][mm] = bf16x2_mul(q4[mm], f2);
              qf[rd][h2][2 * mm] = bf16lo_f32(q4[mm]) * a.scale_log2;
              qf[rd][h2][2 * mm + 1] = bf16hi_f32(q4[mm]) * a.scale_log2;
            }
          }
        }
        // B of the bf16 keys: row h = q[h] (unscaled, exact), rows >= r zero; 16 rows x 16 chunks
        for (int idx = tid; idx < 256; idx += kGroup) {
          const int h = idx >> 4, c = idx & 15;
          uint4 qw = make_uint4(0u, 0u, 0u, 0u);
          if (h < r) qw = lds128(qs + h * (kD * 2) + 16 * c);
          sts128(sbase + GE::OFF_BQFP + c * GE::LBO_QFP + (h >> 3) * 128 + (h & 7) * 16, qw.x, qw.y, qw.z, qw.w);
        }
        warp_arrive(bar_qfree0 + 8 * qb);
        fence_async_smem();
      }
      wait(bar_full(s), (j / kStages) & 1);
      if (kli >= cut.F) {
        // key codes first (loads in flight while B is built): thread = token
        uint4 kw4[2];
        {
          const int tl = tid / G, tt = tid % G;
          const uint32_t kc = stage + tl * TILE + row_kcodes_off() + tt * 16;
          kw4[0] = lds128(kc);
          kw4[1] = lds128(kc + G * 16);
        }
        // B(q.k): rows n = g*NR + 2*head + {hi, lo}, K-major; bias = q . zero per (group, head)
        const uint32_t bq = sbase + GE::OFF_BQK;
        float* bias = reinterpret_cast<float*>(smem + GE::OFF_BIAS) + (j & 1) * (4 * 8);
#pragma unroll
        for (int rd = 0; rd < GE::BROUNDS; ++rd) {
          const int it = tid + rd * kGroup;
          if (it < GE::BITEMS) {
            const int c = it & 15, gh = it >> 4, g = gh / (HP / 2), hp = gh % (HP / 2);
            const uint4 sw = lds128(stage + g * TILE + row_kscale_off(G) + 16 * c);
            const uint4 zw = lds128(stage + g * TILE + row_kzero_off(G) + 16 * c);
            const uint32_t s4[4] = {sw.x, sw.y, sw.z, sw.w};
            const uint32_t z4[4] = {zw.x, zw.y, zw.z, zw.w};
            float bsum[2] = {0.f, 0.f};
            uint32_t hi[2][4], lo[2][4];
#pragma unroll
            for (int h2 = 0; h2 < 2; ++h2)
#pragma unroll
              for (int mm = 0; mm < 4; ++mm) {
                hi[h2][mm] = bf16x2_mul(qpk[rd][h2][mm], s4[mm]);
                lo[h2][mm] = bf16x2_fma(qpk[rd][h2][mm], s4[mm], hi[h2][mm] ^ 0x80008000u);  // exact residual
                bsum[h2] = fmaf(qf[rd][h2][2 * mm], bf16lo_f32(z4[mm]), bsum[h2]);
                bsum[h2] = fmaf(qf[rd][h2][2 * mm + 1], bf16hi_f32(z4[mm]), bsum[h2]);
              }
            const int n = g * NR + 4 * hp;
            const uint32_t dst = bq + c * GE::LBO_QK + (n >> 3) * 128 + (n & 7) * 16;
            sts128(dst, hi[0][0], hi[0][1], hi[0][2], hi[0][3]);
            sts128(dst + 16, lo[0][0], lo[0][1], lo[0][2], lo[0][3]);
            sts128(dst + 32, hi[1][0], hi[1][1], hi[1][2], hi[1][3]);
            sts128(dst + 48, lo[1][0], lo[1][1], lo[1][2], lo[1][3]);
            // sum over the 16 chunks: the 16 lanes that share (g, hp); both heads side by side
#pragma unroll
            for (int o = 8; o; o >>= 1) {
              bsum[0] += __shfl_xor_sync(kFullMask, bsum[0], o);
              bsum[1] += __shfl_xor_sync(kFullMask, bsum[1], o);
            }
            if (c == 0) *reinterpret_cast<float2*>(bias + g * 8 + 2 * hp) = make_float2(bsum[0], bsum[1]);
          }
        }
        // key codes into tensor memory: 8 words = 8 k-steps of 16 channels
#pragma unroll
        for (int hf = 0; hf < 2; ++hf) {
          const uint32_t w[4] = {kw4[hf].x, kw4[hf].y, kw4[hf].z, kw4[hf].w};
          uint32_t regs[32];
#pragma unroll
          for (int jj = 0; jj < 4; ++jj) {
            const uint32_t ws = w[jj] >> 8;
#pragma unroll
            for (int i = 0; i < 4; ++i) {
              regs[8 * jj + i] = w[jj] & (0x00030003u << (2 * i));
              regs[8 * jj + 4 + i] = ws & (0x00030003u << (2 * i));
            }
          }
          tmem_st<32>(tmem + lane_base + GE::COL_AK + 32 * hf, regs);
        }
        tc_wait_st();
        fence_async_smem();
      } else if (a.new_k != nullptr && kli == (a.new_slot >> 5)) {
        // fused append: the new row is not in memory yet; patch it into the landed unit and the store
        if (tid < 32) {
          const int slot = a.new_slot & 31;
          const uint8_t* nk = static_cast<const uint8_t*>(a.new_k) + kpair * (kD * 2);
          const uint8_t* nv = static_cast<const uint8_t*>(a.new_v) + kpair * (kD * 2);
          const int c = tid & 15;
          const uint4 x = __ldg(reinterpret_cast<const uint4*>(tid < 16 ? nk : nv) + c);
          const int off = (tid < 16 ? 0 : kFpUnitVOffset) + (slot >> 3) * 2048 + c * 128 + (slot & 7) * 16;
          sts128(stage + off, x.x, x.y, x.z, x.w);
          uint8_t* g = const_cast<uint8_t*>(fp_layer) + kpair * cv.fp_head_stride + static_cast<int64_t>(kli) * kFpUnitBytes;
          *reinterpret_cast<uint4*>(g + off) = x;
        }
        fence_async_smem();
      }
      tc_fence_before();
      if (++kli == cut.I) { kli = 0; ++kpair; }
    };

    const float kq = a.scale_log2 * pow2i(69);
    float m_run[HP], l_run[HP], zacc[NGS][HP];
    int li = li0;
    int64_t pair = pair0;
    int items_in_seg = 0, first_j_of_seg = 0;

    prep(0);
    named_arrive<kBarQK, kGroup + 32>();
    for (int j = 0; j < n_items; ++j) {
      const int s = j % kStages;
      const int vb = j % VBUF;
      const bool is_fp = li < cut.F;
      const uint32_t stage = sbase + GE::OFF_STAGES + s * kStageBytes;
      if (j == 0 || li == 0) {
        first_j_of_seg = j;
        items_in_seg = min(n_items - j, cut.I - li);
#pragma unroll
        for (int h = 0; h < HP; ++h) {
          m_run[h] = -INFINITY;
          l_run[h] = 0.f;
#pragma unroll
          for (int g = 0; g < NGS; ++g) zacc[g][h] = 0.f;
        }
      }
      const bool more = j + 1 < first_j_of_seg + items_in_seg;
      const bool o_started = j > first_j_of_seg;   // a p.v MMA of this segment has been issued
      if (wt == 0) TR(1, j, 0);

      // ---------------- scores of item j ----------------
      wait(bar_s_ready, j & 1);
      tc_fence_after();
      if (wt == 0) TR(1, j, 1);
      float sc[HP];
      bool valid;
      if (is_fp) {
        uint32_t d[8];
        tmem_ld<8>(tmem + lane_base + GE::COL_S, d);
        tc_wait_ld();
        valid = wt < min(kFpUnitSlots, a.n_fp - li * kFpUnitSlots);
#pragma unroll
        for (int h = 0; h < HP; ++h) sc[h] = __uint_as_float(d[h]) * a.scale_log2;
      } else {
        const int g_tok = wt / G;   // key group of this thread's token inside the super-tile
        uint32_t d[NR];
        tmem_ld<NR>(tmem + lane_base + GE::COL_S + g_tok * NR, d);
        const float* bias = reinterpret_cast<const float*>(smem + GE::OFF_BIAS) + (j & 1) * (4 * 8) + g_tok * 8;
        float bs[HP];
#pragma unroll
        for (int h = 0; h < HP; ++h) bs[h] = bias[h];
        tc_wait_ld();
        valid = (li - cut.F) * NGS + g_tok < a.tiles_quant;
#pragma unroll
        for (int h = 0; h < HP; ++h)
          sc[h] = fmaf(__uint_as_float(d[2 * h]) + __uint_as_float(d[2 * h + 1]), kq, bs[h]);
      }
      tc_fence_before();

      // ---------------- q.k operands of item j + 1 (the score accumulator and the key codes are free now) ----------------
      if (j + 1 < n_items) {
        prep(j + 1);
        named_arrive<kBarQK, kGroup + 32>();
      }
      if (wt == 0) TR(1, j, 2);

      // ---------------- online softmax with a CTA-wide, lazily moved reference maximum ----------------
      // (exchange words per item parity: a warp that is already at the next item touches the other set)
      int* mx = reinterpret_cast<int*>(smem + GE::OFF_MAX) + 16 * (j & 1);
      {
        bool need = false;
#pragma unroll
        for (int h = 0; h < HP; ++h) need |= valid && h < r && sc[h] > m_run[h] + 8.f;
        if (__any_sync(kFullMask, need)) {
#pragma unroll
          for (int h = 0; h < HP; ++h) {
            float v = valid && h < r ? sc[h] : -INFINITY;
#pragma unroll
            for (int o = 16; o; o >>= 1) v = fmaxf(v, __shfl_xor_sync(kFullMask, v, o));
            if (lane == 0) atomicMax(mx + h, ord_f2i(v));
          }
          if (lane == 0) atomicOr(mx + 8, 1);
        }
      }
      // value scale and zero of this thread's token
      float vs[NGS], vz[NGS];
      if (!is_fp) {
        const int tl = wt / G, tt = wt % G;
        const uint32_t pa = stage + tl * TILE + row_vsz_off(G) + tt * (4 * NGS);
        const float posf = valid ? pow2i(64 - 2 * ((wt >> 1) & 3)) : 0.f;
        if (NGS == 4) {
          const uint4 x = lds128(pa);
          vs[0] = bf16lo_f32(x.x); vs[1] = bf16hi_f32(x.x); vs[2 % NGS] = bf16lo_f32(x.y); vs[3 % NGS] = bf16hi_f32(x.y);
          vz[0] = bf16lo_f32(x.z); vz[1] = bf16hi_f32(x.z); vz[2 % NGS] = bf16lo_f32(x.w); vz[3 % NGS] = bf16hi_f32(x.w);
        } else {
          const uint2 x = lds64(pa);
          vs[0] = bf16lo_f32(x.x); vs[1] = bf16hi_f32(x.x);
          vz[0] = bf16lo_f32(x.y); vz[1] = bf16hi_f32(x.y);
        }
#pragma unroll
        for (int g = 0; g < NGS; ++g) {
          vs[g] = valid ? vs[g] * posf : 0.f;   // (stale bytes of a ragged super-tile may be anything)
          vz[g] = valid ? vz[g] : 0.f;
        }
      }
      named_sync<kBarW, kGroup>();
      if (*reinterpret_cast<volatile int*>(mx + 8)) {
        // rare: some score exceeds the reference by more than 2^8 (or the segment has just begun)
        float corr[HP];
#pragma unroll
        for (int h = 0; h < HP; ++h) {
          const float cand = ord_i2f(*reinterpret_cast<volatile int*>(mx + h));
          const float mn = cand > m_run[h] + 8.f ? cand : m_run[h];
          corr[h] = ex2(m_run[h] - mn);   // -inf -> 0; unchanged -> 1
          m_run[h] = mn;
          l_run[h] *= corr[h];
#pragma unroll
          for (int g = 0; g < NGS; ++g) zacc[g][h] *= corr[h];
        }
        if (o_started) {
          // rescale the output accumulator: no p.v MMA may be in flight
          wait(bar_pv_done0 + 8 * ((j - 1) & 1), ((j - 1) >> 1) & 1);
          tc_fence_after();
          uint32_t o[N];
          tmem_ld<N>(tmem + lane_base + GE::COL_O, o);
          tc_wait_ld();
#pragma unroll
          for (int n = 0; n < N; ++n) {
            float cn = corr[0];
#pragma unroll
            for (int h = 1; h < HP; ++h) cn = ((n % NR) >> 1) == h ? corr[h] : cn;
            o[n] = __float_as_uint(__uint_as_float(o[n]) * cn);
          }
          tmem_st<N>(tmem + lane_base + GE::COL_O, o);
          tc_wait_st();
          tc_fence_before();
        }
        // everybody has read the exchange words: thread 0 puts them back to rest before anybody goes on
        named_sync<kBarW, kGroup>();
        if (wt == 0) {
          for (int h = 0; h < 8; ++h) mx[h] = ord_f2i(-INFINITY);
          mx[8] = 0;
        }
        named_sync<kBarW, kGroup>();
      }
      float p[HP];
#pragma unroll
      for (int h = 0; h < HP; ++h) {
        p[h] = valid && h < r ? ex2(sc[h] - m_run[h]) : 0.f;
        l_run[h] += p[h];
      }
      if (wt == 0) TR(1, j, 3);

      // ---------------- B of p.v ----------------
      uint32_t w[NGS][HP];
      if (is_fp) {
        // rows of the 32 tokens of the unit: p * 2^-69 split into hi + lo, the same for every value group
#pragma unroll
        for (int h = 0; h < HP; ++h) {
          const uint32_t x = split_hi_lo(p[h] * 0x1p-69f);
#pragma unroll
          for (int g = 0; g < NGS; ++g) w[g][h] = x;
        }
      } else {
        // p * value scale * 2^(64 - code position), hi + lo per (group, head); zero term in registers
#pragma unroll
        for (int g = 0; g < NGS; ++g)
#pragma unroll
          for (int h = 0; h < HP; ++h) {
            w[g][h] = split_hi_lo(p[h] * vs[g]);
            zacc[g][h] = fmaf(p[h], vz[g], zacc[g][h]);
          }
      }
      // value codes of item j: thread = channel; its 128 tokens = 8 words (G/16 per tile)
      uint32_t vw[8];
      if (!is_fp) {
#pragma unroll
        for (int tl = 0; tl < NGS; ++tl) {
          const uint32_t vc = stage + tl * TILE + row_vcodes_off(G) + tid * (G / 4);
          if (G == 32) {
            const uint2 x = lds64(vc);
            vw[2 * tl] = x.x; vw[2 * tl + 1] = x.y;
          } else {
            const uint4 x = lds128(vc);
            vw[4 * tl] = x.x; vw[4 * tl + 1] = x.y; vw[4 * tl + 2] = x.z; vw[4 * tl + 3] = x.w;
          }
        }
      }
      // buffer vb (value codes in tensor memory, B in shared memory) is free once the p.v MMAs of item j - VBUF are complete
      if (j >= VBUF) wait(bar_pv_done0 + 8 * ((j - VBUF) & 1), ((j - VBUF) >> 1) & 1);
      if (wt == 0) TR(1, j, 4);
      if (!is_fp || wt < 32) {
        const uint32_t row = sbase + GE::OFF_BPV + vb * GE::BPV_BYTES + wt * 16;
        if (NR >= 8) {
#pragma unroll
          for (int g = 0; g < NGS; ++g)
#pragma unroll
            for (int q4 = 0; q4 < NR / 8; ++q4)
              sts128(row + ((g * NR) / 8 + q4) * 2048, w[g][(4 * q4) % HP], w[g][(4 * q4 + 1) % HP],
                     w[g][(4 * q4 + 2) % HP], w[g][(4 * q4 + 3) % HP]);
        } else {
          // HP = 2: a 16-byte vector holds the columns of two value groups
#pragma unroll
          for (int nb = 0; nb < N / 8; ++nb)
            sts128(row + nb * 2048, w[(2 * nb) % NGS][0], w[(2 * nb) % NGS][1 % HP], w[(2 * nb + 1) % NGS][0],
                   w[(2 * nb + 1) % NGS][1 % HP]);
        }
      }
      if (!is_fp) {
        tc_fence_after();
#pragma unroll
        for (int hf = 0; hf < 2; ++hf) {
          uint32_t regs[32];
#pragma unroll
          for (int jj = 0; jj < 4; ++jj) {
            const uint32_t wv = vw[4 * hf + jj], ws = wv >> 8;
#pragma unroll
            for (int i = 0; i < 4; ++i) {
              regs[8 * jj + i] = wv & (0x00030003u << (2 * i));
              regs[8 * jj + 4 + i] = ws & (0x00030003u << (2 * i));
            }
          }
          tmem_st<32>(tmem + lane_base + GE::COL_AV + 64 * vb + 32 * hf, regs);
        }
        tc_wait_st();
      }
      fence_async_smem();
      tc_fence_before();
      warp_arrive(bar_empty(s));
      if (j & 1) named_arrive<kBarPV0 + 1, kGroup + 32>(); else named_arrive<kBarPV0, kGroup + 32>();
      if (wt == 0) TR(1, j, 5);

      if (!more) {
        // ---------------- segment end: reduce l and the zero term, read O, write the partial ----------------
        wait(bar_pv_done0 + 8 * (j & 1), (j >> 1) & 1);
        tc_fence_after();
        float* red = reinterpret_cast<float*>(smem + GE::OFF_RED);
        const int xw = warp & 3;
        {
          // warp sums, then the four warps meet in shared memory
#pragma unroll
          for (int h = 0; h < HP; ++h) {
#pragma unroll
            for (int o = 16; o; o >>= 1) l_run[h] += __shfl_xor_sync(kFullMask, l_run[h], o);
#pragma unroll
            for (int g = 0; g < NGS; ++g)
#pragma unroll
              for (int o = 16; o; o >>= 1) zacc[g][h] += __shfl_xor_sync(kFullMask, zacc[g][h], o);
          }
          if (lane == 0) {
#pragma unroll
            for (int h = 0; h < HP; ++h) {
              red[xw * 48 + h] = l_run[h];
#pragma unroll
              for (int g = 0; g < NGS; ++g) red[xw * 48 + 8 + g * 8 + h] = zacc[g][h];
            }
          }
        }
        named_sync<kBarW, kGroup>();
        const int vg = wt / G;   // value group of this thread's channel
        uint32_t o[NR];
        tmem_ld<NR>(tmem + lane_base + GE::COL_O + vg * NR, o);
        tc_wait_ld();
        tc_fence_before();
        const int d = wt;
        const int c_first = cut.cta_min(pair);
        const int slot = blockIdx.x - c_first;
        const int64_t rec = (pair * a.S + slot) * r;
#pragma unroll
        for (int h = 0; h < HP; ++h) {
          if (h < r && LQ_IN_BOUNDS(cv, slot >= 0 && slot < a.S)) {
            const float zsum = red[8 + vg * 8 + h] + red[48 + 8 + vg * 8 + h] + red[96 + 8 + vg * 8 + h] + red[144 + 8 + vg * 8 + h];
            const float val = fmaf(__uint_as_float(o[2 * h]) + __uint_as_float(o[2 * h + 1]), 0x1p69f, zsum);
            a.part_o[(rec + h) * kD + d] = val;
            if (d == 0) {
              a.part_ml[(rec + h) * 2 + 0] = m_run[h];
              a.part_ml[(rec + h) * 2 + 1] = red[h] + red[48 + h] + red[96 + h] + red[144 + h];
            }
          }
        }
        // ---- arrival: the CTA that brings the pair's item count to I merges its partials ----
        if (failed && lane == 0) atomicOr(a.status, 1);   // before the ticket: the merging CTA then writes nothing
        __threadfence();
        // which CTAs hold a partial of this pair (their item range meets the pair's): one candidate per thread
        uint8_t* contrib = smem + GE::OFF_MISC + 32;
        if (wt < a.S) {
          const int c = c_first + wt;
          const int64_t p_lo = pair * cut.I, p_hi = p_lo + cut.I;
          bool yes = false;
          if (c < cut.n_ctas) {
            const int64_t lo = cut.first_item(c), hi = cut.first_item(c + 1);
            yes = max(lo, p_lo) < min(hi, p_hi);
          }
          contrib[wt] = yes ? 1 : 0;
        }
        named_sync<kBarW, kGroup>();
        if (wt == 0) {
          int* ticket = a.tickets + 32 * pair + 1;
          const int old = atomicAdd(ticket, items_in_seg);
          const int last = old + items_in_seg == cut.I;
          if (last) *ticket = 0;
          __threadfence();
          *is_last_s = last;
        }
        named_sync<kBarW, kGroup>();
        if (*reinterpret_cast<volatile int*>(is_last_s)) {
          __threadfence();
          const bool healthy = (__ldcg(a.status) & 1) == 0;   // after a wait that gave up the output stays untouched
          // (m, l) of every record of the pair into shared memory with one round of loads (B of p.v is free: the
          // p.v MMAs of this item are complete and nobody writes the next item's before the rendezvous below)
          float2* sml = reinterpret_cast<float2*>(smem + GE::OFF_BPV);
          const int R = a.S * r;
          for (int i = wt; i < R; i += kGroup) {
            const int sl = i / r;
            sml[i] = contrib[sl] ? __ldcg(reinterpret_cast<const float2*>(a.part_ml) + (pair * a.S + sl) * r + (i - sl * r))
                                 : make_float2(-INFINITY, 0.f);
          }
          named_sync<kBarW, kGroup>();
          for (int h = 0; h < r && healthy; ++h) {
            float M = -INFINITY;
            for (int sl = 0; sl < a.S; ++sl) {
              const float2 ml = sml[sl * r + h];
              if (ml.y > 0.f) M = fmaxf(M, ml.x);
            }
            float L = 0.f, acc = 0.f;
            for (int sl0 = 0; sl0 < a.S; sl0 += 8) {
              float v[8], wgt[8];
#pragma unroll
              for (int u = 0; u < 8; ++u) {   // eight independent loads in flight
                const int sl = sl0 + u;
                const float2 ml = sl < a.S ? sml[sl * r + h] : make_float2(-INFINITY, 0.f);
                const bool on = ml.y > 0.f;
                wgt[u] = on ? ex2(ml.x - M) : 0.f;
                v[u] = on ? __ldcg(a.part_o + ((pair * a.S + sl) * r + h) * kD + d) : 0.f;
                L = fmaf(ml.y, wgt[u], L);
              }
#pragma unroll
              for (int u = 0; u < 8; ++u) acc = fmaf(v[u], wgt[u], acc);
            }
            const int b = static_cast<int>(pair / cv.Hkv), kv = static_cast<int>(pair % cv.Hkv);
            const int64_t oi = (static_cast<int64_t>(b) * cv.Hq + kv * r + h) * kD + d;
            const float res = acc / L;
            if (a.out_bf16)
              static_cast<__nv_bfloat16*>(a.out)[oi] = __float2bfloat16_rn(res);
            else
              static_cast<float*>(a.out)[oi] = res;
          }
        }
        // the exchange areas (red, contrib, is_last) are rewritten by the next segment only after its own rendezvous
        named_sync<kBarW, kGroup>();
      }
      if (++li == cut.I) { li = 0; ++pair; }
    }
    if (failed && lane == 0) atomicOr(a.status, 1);
  }

  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  tc_fence_before();
  __syncthreads();
#ifdef LQ_UMMA_TRACE
  if (blockIdx.x == LQ_UMMA_TRACE && threadIdx.x == 0) {
    const uint32_t t0 = trace[1][0][0];
    printf("cta %d items %d F %d Q %d\n", blockIdx.x, n_items, a.u_fp_units, a.u_supertiles);
    for (int j = 0; j < 12 && j < n_items; ++j) {
      printf("item %2d W:", j);
      for (int k = 0; k < 6; ++k) printf(" %6d", static_cast<int>(trace[1][j][k] - t0));
      printf(" | QK:");
      for (int k = 0; k < 2; ++k) printf(" %6d", static_cast<int>(trace[2][j][k] - t0));
      printf(" | PV:");
      for (int k = 0; k < 2; ++k) printf(" %6d", static_cast<int>(trace[3][j][k] - t0));
      printf("\n");
    }
  }
#endif
  if (warp == kWarpQK && n_items > 0) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(GE::COLS) : "memory");
  }
}

}  // namespace

// Launch geometry: fp units and super-tiles per pair, their cost, the number of CTAs and the record stride.
// sm_count * 2 CTAs (one resident wave), fewer when there are fewer items or record slots.
void plan_decode_umma(DecodeArgs& a, int sm_count, int max_records, int s_override) {
  const int G = a.cv.G, ngs = 128 / G;
  const int64_t pairs = static_cast<int64_t>(a.cv.B) * a.cv.Hkv;
  a.tiles_fp = (a.n_fp + kFpUnitSlots - 1) / kFpUnitSlots;
  a.tiles_quant = static_cast<int>(a.n_quant / G);
  a.u_fp_units = a.tiles_fp;
  a.u_supertiles = (a.tiles_quant + ngs - 1) / ngs;
  a.u_items = a.u_fp_units + a.u_supertiles;
  const int wq = ngs * quant_tile_bytes(G, 1) / 2048;
  a.u_cost = a.u_fp_units * kWeightFp + a.u_supertiles * wq;
  int64_t n = 2LL * sm_count;
  if (s_override > 0) n = std::min<int64_t>(n, static_cast<int64_t>(s_override) * pairs);
  n = std::min<int64_t>(n, pairs * a.u_items);                                  // at least one item per CTA
  n = std::min<int64_t>(n, pairs * static_cast<int64_t>(std::min(max_records, 128) - 3));  // record slots per pair
  n = std::max<int64_t>(n, 1);
  a.n_ctas = static_cast<int>(n);
  a.S = static_cast<int>((n + pairs - 1) / pairs) + 3;
  a.n_extra = 0;
}

cudaError_t launch_decode_umma(const DecodeArgs& a, cudaStream_t st) {
  const int r = a.cv.Hq / a.cv.Hkv;
  void (*kern)(DecodeArgs) = nullptr;
  int smem = 0;
#define LQ_PICK(G_, HP_)                        \
  do {                                          \
    kern = lq_decode_umma_kernel<G_, HP_>;      \
    smem = Geo<G_, HP_>::SMEM + LQ_UMMA_EXTRA_SMEM; \
  } while (0)
  if (a.cv.G == 32) {
    if (r <= 2) LQ_PICK(32, 2); else if (r <= 4) LQ_PICK(32, 4); else LQ_PICK(32, 8);
  } else if (a.cv.G == 64) {
    if (r <= 2) LQ_PICK(64, 2); else if (r <= 4) LQ_PICK(64, 4); else LQ_PICK(64, 8);
  } else {
    return cudaErrorInvalidValue;
  }
#undef LQ_PICK
  static bool configured[64][8] = {};
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  const int variant = (a.cv.G == 64 ? 3 : 0) + (r <= 2 ? 0 : (r <= 4 ? 1 : 2));
  if (dev < 0 || dev >= 64 || !configured[dev][variant]) {
    e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (e != cudaSuccess) return e;
    if (dev >= 0 && dev < 64) configured[dev][variant] = true;
  }
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(a.n_ctas);
  cfg.blockDim = dim3(kThreads);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kern, a);
}

}  // namespace lq

// Kernels that write and read back the two stores: append (K1), window-overflow step (K2:
// quantise + bit-pack + back-fill) and the canonical export.  Layout: lq_layout.cuh.
#include <cuda_bf16.h>

#include "lq_kernels.cuh"

namespace lq {

// ---------------------------------------------------------------------------------------
// K1  append: Algorithm 1, branch length(A) < 3W -- the new rows go to the next free slots.
// One thread per 16-byte chunk of a K or V row.  The threads after those copy `extra_chunks`
// 16-byte chunks from extra_src to extra_dst (the host-buffer step stages its query this way, in
// the same launch).
// ---------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256)
lq_append_kernel(CacheView cv, int layer, const uint4* __restrict__ k, const uint4* __restrict__ v,
                 int n_src, int src0, int n, int slot0, const uint4* __restrict__ extra_src, uint4* extra_dst,
                 int extra_chunks) {
  // programmatic dependent launch: overlap this kernel's launch with the tail of the previous
  // kernel of the stream, but write nothing before that kernel has finished
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  asm volatile("griddepcontrol.wait;" ::: "memory");
  const int64_t idx = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
  const int64_t total = static_cast<int64_t>(cv.B) * cv.Hkv * n * 32;
  if (idx >= total) {
    if (idx - total < extra_chunks) extra_dst[idx - total] = extra_src[idx - total];
    return;
  }
  const int c = static_cast<int>(idx & 15);
  const int which = static_cast<int>((idx >> 4) & 1);
  const int64_t row = idx >> 5;
  const int t = static_cast<int>(row % n);
  const int64_t pair = row / n;
  const uint4* src = (which ? v : k) + ((pair * n_src + src0 + t) * 16 + c);
  uint8_t* base = cv.fp + layer * cv.fp_layer_stride + pair * cv.fp_head_stride;
  const int64_t off = fp_chunk_off(cv.layout, slot0 + t, c) + (which ? fp_v_delta(cv.layout) : 0);
  if (!LQ_IN_BOUNDS(cv, slot0 + t >= 0 && slot0 + t < fp_slots_cap(cv) && src0 + t < n_src)) return;
  *reinterpret_cast<uint4*>(base + off) = *src;
}

cudaError_t launch_append(const CacheView& cv, int layer, const void* k, const void* v, int n_src,
                          int src0, int n, int slot0, cudaStream_t st, const void* extra_src, void* extra_dst,
                          int extra_bytes) {
  const int64_t total = static_cast<int64_t>(cv.B) * cv.Hkv * n * 32 + extra_bytes / 16;
  const int blocks = static_cast<int>((total + 255) / 256);
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(blocks);
  cfg.blockDim = dim3(256);
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, lq_append_kernel, cv, layer, static_cast<const uint4*>(k),
                            static_cast<const uint4*>(v), n_src, src0, n, slot0,
                            static_cast<const uint4*>(extra_src), static_cast<uint4*>(extra_dst), extra_bytes / 16);
}

// ---------------------------------------------------------------------------------------
// K2  window-overflow step (Algorithm 1, else-branch).
//
// One CTA per (key group tau of the event, (b, kv) head, layer).  It
//   1. gathers the G removed rows of its group (K and V) into shared memory,
//   2. back-fills the G holes with rows the host names (the top rows of the dense prefix: slots
//      2W + tau*G + e when W is a multiple of G), so the valid slots stay a dense prefix -- legal
//      because the order of the cache is free (Eq. 3) -- and only this CTA ever touches these 2G slots,
//   3. finds min, scale and zero of every group: keys per channel down the G tokens, values per token
//      across G channels,
//   4. quantises and stores the tile word by word, in the fragment order (quantise_pack_tile below).
//
// Quantiser arithmetic (IEEE binary32, one rounding per operation, ties to even):
//   zero = min, scale = bf16(fdiv(fsub(max, min), 3)), code = clamp(rint(fdiv(fsub(x, min), scale)), 0, 3),
//   all codes 0 when scale == 0.  A zero-valued min or max is taken as +0.  The 4-bit cache uses 15
//   in place of 3 and stores every code as two 2-bit planes (low bits, high bits).
// ---------------------------------------------------------------------------------------
// rows of the staged K / V rows in shared memory: 8 elements of padding (a multiple of 16 bytes) so that the packing
// step, which reads one element of 8 rows per code position, meets 8 different banks
constexpr int kSRow = kD + 8;

__device__ __forceinline__ float bf16_bits_to_float(uint16_t b) {
  return __uint_as_float(static_cast<uint32_t>(b) << 16);
}

// top = highest code: 3 (2 bits) or 15 (4 bits).  inv = an approximation of 1 / scale (rcp.approx, computed once
// per group).  The code is rint(fdiv(fsub(x, mn), scale)) in IEEE arithmetic, exactly: the quotient lies in
// [0, top + 1/2], so d * inv differs from it by less than 16 * 2^-21 = 2^-17; unless d * inv comes that close to a
// rounding boundary k + 1/2 (ties included), rounding it gives the same integer as rounding the exact quotient,
// and only then is the division carried out.
// scale == 0 (all codes 0): the caller passes inv = 0, so that d * inv = 0 without a branch.
__device__ __forceinline__ uint32_t quant_code(float x, float mn, float scale, float inv, float top) {
  const float d = __fsub_rn(x, mn);
  const float t = __fmul_rn(d, inv);
  float r = rintf(t);
  if (!(fabsf(fabsf(__fsub_rn(t, r)) - 0.5f) > 0x1p-16f)) r = rintf(__fdiv_rn(d, scale));  // also catches NaN / inf
  r = fminf(fmaxf(r, 0.0f), top);
  return static_cast<uint32_t>(r);
}
__device__ __forceinline__ float approx_rcp(float x) {
  float y;
  asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

__device__ __forceinline__ void group_params(float mn, float mx, float top, uint16_t& scale_bits,
                                             uint16_t& zero_bits, float& mn_c, float& scale) {
  mn_c = __fadd_rn(mn, 0.0f);  // -0 -> +0
  float mxc = __fadd_rn(mx, 0.0f);
  float third = __fdiv_rn(__fsub_rn(mxc, mn_c), top);  // one step of the code grid
  __nv_bfloat16 sb = __float2bfloat16_rn(third);
  scale_bits = __bfloat16_as_ushort(sb);
  scale = __bfloat162float(sb);
  zero_bits = __bfloat16_as_ushort(__float2bfloat16_rn(mn_c));  // exact: mn is a bf16 value
}

// What the code phase needs of one group, as a float4:
//   2-bit codes: {min, T1, T2, T3} with T_i = (i - 1/2) * scale.  scale is a bf16 value, so every T_i is an exact
//     binary32 number, and for d = fsub(x, min) >= 0
//         rint(fdiv(d, scale)) = [d > T1] + [d >= T2] + [d > T3]          (clamped at 3 by construction)
//     holds exactly: at d = T_i the quotient is i - 1/2 and the tie goes to the even neighbour (0, 2, 2); a float
//     d above (below) T_i differs from it by at least one unit in the last place of T_i, i.e. by more than
//     2^-24 T_i, which is more than the half unit in the last place of the quotient's neighbourhood of i - 1/2
//     (at most 2^-24 (i - 1/2)), so the rounded quotient lies strictly on the same side of i - 1/2 as d of T_i.
//     scale == 0 (every code 0) is encoded as T_i = +inf.
//   4-bit codes: {min, scale, inv, unused}, see quant_code.
template <int P>
__device__ __forceinline__ float4 make_group(float mn, float mx, uint16_t& scale_bits, uint16_t& zero_bits) {
  constexpr float kTop = P == 1 ? 3.0f : 15.0f;
  float mnc, scale;
  group_params(mn, mx, kTop, scale_bits, zero_bits, mnc, scale);
  if (P == 1) {
    const bool flat = scale == 0.0f;
    return make_float4(mnc, flat ? INFINITY : 0.5f * scale, flat ? INFINITY : 1.5f * scale,
                       flat ? INFINITY : 2.5f * scale);
  }
  return make_float4(mnc, scale, scale == 0.0f ? 0.0f : approx_rcp(scale), 0.0f);
}
template <int P>
__device__ __forceinline__ uint32_t group_code(float x, const float4& p) {
  if (P == 1) {
    // the thresholds are nested: the high bit is [d >= T2], the low bit compares with T3 or T1 accordingly
    const float d = __fsub_rn(x, p.x);
    const bool high = d >= p.z;
    return (high ? 2u : 0u) + (d > (high ? p.w : p.y) ? 1u : 0u);
  }
  return quant_code(x, p.x, p.y, p.z, 15.0f);
}
// ORs the code of x into the words of its planes at bit `pos` (a compile-time constant where it matters).  2-bit
// codes: one predicated OR of a constant per code bit, no integer code in between.
template <int P>
__device__ __forceinline__ void add_code(uint32_t (&word)[P], int pos, float x, const float4& p) {
  if (P == 1) {
    const float d = __fsub_rn(x, p.x);
    const bool high = d >= p.z;
    const bool low = d > (high ? p.w : p.y);
    if (high) word[0] |= 2u << pos;
    if (low) word[0] |= 1u << pos;
  } else {
    const uint32_t c = quant_code(x, p.x, p.y, p.z, 15.0f);
#pragma unroll
    for (int pl = 0; pl < P; ++pl) word[pl] |= ((c >> (2 * pl)) & 3u) << pos;
  }
}
__device__ __forceinline__ float lo_bf16(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float hi_bf16(uint32_t w) { return __uint_as_float(w & 0xFFFF0000u); }
__device__ __forceinline__ uint32_t min_bf16x2(uint32_t a, uint32_t b) {
  uint32_t r;
  asm("min.bf16x2 %0, %1, %2;" : "=r"(r) : "r"(a), "r"(b));
  return r;
}
__device__ __forceinline__ uint32_t max_bf16x2(uint32_t a, uint32_t b) {
  uint32_t r;
  asm("max.bf16x2 %0, %1, %2;" : "=r"(r) : "r"(a), "r"(b));
  return r;
}

// Steps 3 and 4 of the overflow step for one key group whose G rows sit in shared memory
// (sK, sV: [G][128] bf16 bits, read only).  256 threads.
//   A. group parameters: keys, two threads per channel pair (packed bf16 min / max down half of the tokens each);
//      values, LPG = G/4 lanes per group and LPG rows per warp: the rows' (min, -max) pairs are reduced with a
//      folding exchange, after which every lane owns one (row, group) and the parameters are computed once each.
//   B. every thread builds whole words of the tile: it quantises exactly the 16 elements a word holds (two words
//      that share their parameters at a time), so the codes never pass through shared memory.
template <int G, int P>
__device__ __forceinline__ void quantise_pack_tile(uint16_t (&sK)[G][kSRow], uint16_t (&sV)[G][kSRow], uint8_t* tile, int tid,
                                                   int layout) {
  constexpr int NS = G / 16;
  constexpr int NG = kD / G;
  __shared__ float4 pK[kD];      // per key channel
  __shared__ float4 pV[NG * G];  // per (value group, token): [g][t]
  const int lane = tid & 31;
  // ---- A. parameters ----
  if (tid < kD) {
    const int cp = tid >> 1, half = tid & 1;
    uint32_t mn2 = *reinterpret_cast<const uint32_t*>(&sK[half * (G / 2)][2 * cp]), mx2 = mn2;
#pragma unroll
    for (int i = 1; i < G / 2; ++i) {
      const uint32_t w = *reinterpret_cast<const uint32_t*>(&sK[half * (G / 2) + i][2 * cp]);
      mn2 = min_bf16x2(mn2, w);
      mx2 = max_bf16x2(mx2, w);
    }
    mn2 = min_bf16x2(mn2, __shfl_xor_sync(0xFFFFFFFFu, mn2, 1));
    mx2 = max_bf16x2(mx2, __shfl_xor_sync(0xFFFFFFFFu, mx2, 1));
    const int d = tid;  // = 2 * cp + half
    uint16_t sb, zb;
    pK[d] = make_group<P>(half ? hi_bf16(mn2) : lo_bf16(mn2), half ? hi_bf16(mx2) : lo_bf16(mx2), sb, zb);
    *reinterpret_cast<uint16_t*>(tile + kscale_off(layout, G, d)) = sb;
    *reinterpret_cast<uint16_t*>(tile + kzero_off(layout, G, d)) = zb;
  } else {
    constexpr int LPG = G / 4;  // lanes per value group = rows per warp
    const int wv = (tid >> 5) - 4;
    uint32_t m2[LPG];           // (min, -max) of this lane's four channels, row by row
#pragma unroll
    for (int i = 0; i < LPG; ++i) {
      const uint2 raw = *reinterpret_cast<const uint2*>(&sV[wv * LPG + i][4 * lane]);
      const uint32_t lo = min_bf16x2(raw.x, raw.y), hi = max_bf16x2(raw.x, raw.y);
      const uint32_t a = __byte_perm(lo, hi, 0x5410) ^ 0x80000000u;  // (min of channels 0 and 2, -max of the same)
      const uint32_t b = __byte_perm(lo, hi, 0x7632) ^ 0x80000000u;  // channels 1 and 3
      m2[i] = min_bf16x2(a, b);
    }
#pragma unroll
    for (int lvl = LPG / 2; lvl >= 1; lvl >>= 1) {
      const bool upper = (lane & lvl) != 0;
#pragma unroll
      for (int i = 0; i < lvl; ++i) {
        const uint32_t send = upper ? m2[i] : m2[i + lvl];
        const uint32_t keep = upper ? m2[i + lvl] : m2[i];
        m2[i] = min_bf16x2(keep, __shfl_xor_sync(0xFFFFFFFFu, send, lvl));
      }
    }
    // m2[0] now covers the whole group of row (lane % LPG) of this warp's rows
    const int e = wv * LPG + (lane % LPG), g = lane / LPG;
    uint16_t sb, zb;
    pV[g * G + e] = make_group<P>(lo_bf16(m2[0]), hi_bf16(m2[0] ^ 0x80000000u), sb, zb);
    *reinterpret_cast<uint16_t*>(tile + vscale_off(layout, G, P, e, g)) = sb;
    *reinterpret_cast<uint16_t*>(tile + vzero_off(layout, G, P, e, g)) = zb;
  }
  __syncthreads();

  // ---- B. codes, word by word ----
  if (layout == kLayoutRow) {
    // one word = 16 codes of one row: K words [half][token][4], V words [channel][G/16]
    for (int idx = tid; idx < 2 * G * 8; idx += 256) {
      uint32_t word = 0;
      if (idx < G * 8) {
        const int hf = idx / (G * 4), t = (idx >> 2) % G, ks = 4 * hf + (idx & 3);
#pragma unroll
        for (int e = 0; e < 16; ++e)
          word |= (group_code<P>(bf16_bits_to_float(sK[t][16 * ks + e]), pK[16 * ks + e]) & 3u) << row_code_bit(e);
        reinterpret_cast<uint32_t*>(tile + row_kcodes_off())[idx] = word;
      } else {
        const int wd = idx - G * 8, d = wd / (G / 16), j = wd % (G / 16);
#pragma unroll
        for (int e = 0; e < 16; ++e)
          word |= (group_code<P>(bf16_bits_to_float(sV[16 * j + e][d]), pV[(d / G) * G + 16 * j + e]) & 3u)
                  << row_code_bit(e);
        reinterpret_cast<uint32_t*>(tile + row_vcodes_off(G))[wd] = word;
      }
    }
    return;
  }
  // fragment order, one 2-bit plane after the other
  for (int item = tid; item < NS * 128; item += 256) {
    uint32_t word[2][P] = {};
    if (item < NS * 64) {
      // keys: tokens t0 and t0 + 8 (n-tiles 0 and 1) at the 16 channels 16 ks + 8 w + 2 j + h
      const int hi = (item >> 2) & 7, j = item & 3, w = (item >> 5) & 1, u = item >> 6;
      const int t0 = 16 * u + hi;
#pragma unroll
      for (int ks = 0; ks < 8; ++ks) {
        const int ch = 16 * ks + 8 * w + 2 * j;
        const float4 pa = pK[ch], pb = pK[ch + 1];
#pragma unroll
        for (int nt = 0; nt < 2; ++nt) {
          const uint32_t x = *reinterpret_cast<const uint32_t*>(&sK[t0 + 8 * nt][ch]);
          add_code<P>(word[nt], 2 * ks, lo_bf16(x), pa);
          add_code<P>(word[nt], 16 + 2 * ks, hi_bf16(x), pb);
        }
      }
#pragma unroll
      for (int pl = 0; pl < P; ++pl) {
        uint32_t* kw = reinterpret_cast<uint32_t*>(tile + qt_kcodes_off() + pl * qt_plane_bytes(G));
#pragma unroll
        for (int nt = 0; nt < 2; ++nt) kw[u * 128 + 4 * (4 * hi + j) + 2 * nt + w] = word[nt][pl];
      }
    } else {
      // values: tokens tt and tt + 1 at the channels 16 mt + 8 dh + r for r = 2 p and 2 p + 1 (one word each)
      const int vi = item - NS * 64;
      const int j = vi & 3, p = (vi >> 2) & 3, dh = (vi >> 4) & 1, th = (vi >> 5) & 1, u = vi >> 6;
      const int tt = 16 * u + 8 * th + 2 * j;
#pragma unroll
      for (int mt = 0; mt < 8; ++mt) {
        const int ch = 16 * mt + 8 * dh + 2 * p;
        constexpr int kShift = G == 32 ? 1 : 2;  // value group of m-tile mt: 16 mt / G
        const int g = mt >> kShift;
#pragma unroll
        for (int h = 0; h < 2; ++h) {
          const float4 pv = pV[g * G + tt + h];
          const uint32_t x = *reinterpret_cast<const uint32_t*>(&sV[tt + h][ch]);
          add_code<P>(word[0], 16 * h + 2 * mt, lo_bf16(x), pv);
          add_code<P>(word[1], 16 * h + 2 * mt, hi_bf16(x), pv);
        }
      }
#pragma unroll
      for (int pl = 0; pl < P; ++pl) {
        uint32_t* vw = reinterpret_cast<uint32_t*>(tile + qt_vcodes_off(G, P) + pl * qt_plane_bytes(G));
#pragma unroll
        for (int b = 0; b < 2; ++b) vw[u * 128 + 4 * (4 * (2 * p + b) + j) + dh + 2 * th] = word[b][pl];
      }
    }
  }
}

template <int G, int P>
__global__ void __launch_bounds__(256)
lq_compress_kernel(CacheView cv, LayerList layers, EvictList ev, int64_t tile0) {
  __shared__ __align__(16) uint16_t sK[G][kSRow];
  __shared__ __align__(16) uint16_t sV[G][kSRow];
  const int tau = blockIdx.x;
  const int64_t pair = blockIdx.y;
  const int layer = layers.layer[blockIdx.z];
  const int tid = threadIdx.x;
  uint8_t* fpbase = cv.fp + layer * cv.fp_layer_stride + pair * cv.fp_head_stride;
  uint8_t* tile = cv.quant + layer * cv.quant_layer_stride + pair * cv.quant_head_stride +
                  (tile0 + tau) * quant_tile_bytes(G, P);

  if (!LQ_IN_BOUNDS(cv, tile0 + tau >= 0 && tile0 + tau < cv.quant_tiles_cap)) return;
  // 1. gather the removed rows
  for (int idx = tid; idx < G * 32; idx += 256) {
    const int c = idx & 15, which = (idx >> 4) & 1, e = idx >> 5;
    const int slot = ev.slot[tau * G + e];
    if (!LQ_IN_BOUNDS(cv, slot < fp_slots_cap(cv))) continue;
    const uint4 val = *reinterpret_cast<const uint4*>(fpbase + fp_chunk_off(cv.layout, slot, c) +
                                                      (which ? fp_v_delta(cv.layout) : 0));
    *reinterpret_cast<uint4*>(which ? &sV[e][c * 8] : &sK[e][c * 8]) = val;
  }
  __syncthreads();

  // 2. back-fill the holes (from the newest window; the host names the source rows)
  for (int idx = tid; idx < G * 32; idx += 256) {
    const int c = idx & 15, which = (idx >> 4) & 1, e = idx >> 5;
    const int dst = ev.slot[tau * G + e];
    const int src = ev.src[tau * G + e];
    if (src == kNoMove) continue;
    if (!LQ_IN_BOUNDS(cv, src < fp_slots_cap(cv) && dst < fp_slots_cap(cv))) continue;
    const int vo = which ? fp_v_delta(cv.layout) : 0;
    const uint4 val = *reinterpret_cast<const uint4*>(fpbase + fp_chunk_off(cv.layout, src, c) + vo);
    *reinterpret_cast<uint4*>(fpbase + fp_chunk_off(cv.layout, dst, c) + vo) = val;
  }

  quantise_pack_tile<G, P>(sK, sV, tile, tid, cv.layout);
}

cudaError_t launch_compress(const CacheView& cv, const LayerList& layers, const EvictList& ev,
                            int64_t tile0, int n_groups, cudaStream_t st) {
  dim3 grid(n_groups, cv.B * cv.Hkv, layers.n);
  if (cv.G == 32 && cv.planes == 1)
    lq_compress_kernel<32, 1><<<grid, 256, 0, st>>>(cv, layers, ev, tile0);
  else if (cv.G == 32 && cv.planes == 2)
    lq_compress_kernel<32, 2><<<grid, 256, 0, st>>>(cv, layers, ev, tile0);
  else if (cv.G == 64 && cv.planes == 1)
    lq_compress_kernel<64, 1><<<grid, 256, 0, st>>>(cv, layers, ev, tile0);
  else if (cv.G == 64 && cv.planes == 2)
    lq_compress_kernel<64, 2><<<grid, 256, 0, st>>>(cv, layers, ev, tile0);
  else
    return cudaErrorInvalidValue;
  return cudaGetLastError();
}

// ---------------------------------------------------------------------------------------
// Prompt (or prompt chunk) ingestion in one launch.  Appending n tokens one at a time (Algorithm 1)
// ends in a state the host knows in advance, because the filter never looks at the data: the removed
// tokens of every overflow step, in store order, and the token that ends up in every fp slot.
//
// A source is a row of the new tensors (value >= 0: position in [0, n_src)) or a row the fp store held
// before the call (value <= -2: slot -2 - value); -1 = none.  idx holds
//   src   [n_tiles * G]  the rows of every new key group, in store order
//   fill1 [n_tiles * G]  (only with has_fill) for a group row that came from fp slot s: the source of the row
//                        that takes slot s over, if any
//   fill2 [n_tiles * G]  (only with has_fill) when fill1 names an old slot m: the new-tensor row that takes slot m over
//   copy  [n_copy][2]    (slot, new-tensor row) for the fp slots nobody held before
// CTAs [0, n_tiles) each gather and quantise one key group; only after its gather does a CTA overwrite the slots it
// gathered from, and the thread that moves an old row m into such a slot is the one that then overwrites slot m:
// every slot that is both read and written has its reader and its writer in one thread, in that order.  The
// remaining CTAs write the copy list.  The stores end up bit-identical to the token-by-token path.
// ---------------------------------------------------------------------------------------
template <int G, int P>
__global__ void __launch_bounds__(256)
lq_ingest_kernel(CacheView cv, int layer, const uint4* __restrict__ k, const uint4* __restrict__ v, int n_src,
                 const int* __restrict__ idx, int n_tiles, int has_fill, int n_copy, int64_t tile0) {
  __shared__ __align__(16) uint16_t sK[G][kSRow];
  __shared__ __align__(16) uint16_t sV[G][kSRow];
  const int64_t pair = blockIdx.y;
  const int tid = threadIdx.x;
  uint8_t* fpbase = cv.fp + layer * cv.fp_layer_stride + pair * cv.fp_head_stride;
  const int vdelta = fp_v_delta(cv.layout);
  if (static_cast<int>(blockIdx.x) < n_tiles) {
    const int tau = blockIdx.x;
    uint8_t* tile = cv.quant + layer * cv.quant_layer_stride + pair * cv.quant_head_stride +
                    (tile0 + tau) * quant_tile_bytes(G, P);
    if (!LQ_IN_BOUNDS(cv, tile0 + tau >= 0 && tile0 + tau < cv.quant_tiles_cap)) return;
    for (int i = tid; i < G * 32; i += 256) {
      const int c = i & 15, which = (i >> 4) & 1, e = i >> 5;
      int64_t t = idx[tau * G + e];
      uint4 val;
      if (t >= 0) {
        if (!LQ_IN_BOUNDS(cv, t < n_src)) t = 0;
        val = (which ? v : k)[(pair * n_src + t) * 16 + c];
      } else {
        int slot = static_cast<int>(-2 - t);
        if (!LQ_IN_BOUNDS(cv, slot >= 0 && slot < fp_slots_cap(cv))) slot = 0;
        val = *reinterpret_cast<const uint4*>(fpbase + fp_chunk_off(cv.layout, slot, c) + (which ? vdelta : 0));
      }
      *reinterpret_cast<uint4*>(which ? &sV[e][c * 8] : &sK[e][c * 8]) = val;
    }
    __syncthreads();
    if (has_fill) {
      const int* fill1 = idx + n_tiles * G;
      const int* fill2 = fill1 + n_tiles * G;
      for (int i = tid; i < G * 32; i += 256) {
        const int c = i & 15, which = (i >> 4) & 1, e = i >> 5;
        const int t = idx[tau * G + e], f1 = fill1[tau * G + e];
        if (t >= 0 || f1 == -1) continue;
        const int s = -2 - t, vo = which ? vdelta : 0;
        if (!LQ_IN_BOUNDS(cv, s >= 0 && s < fp_slots_cap(cv) && f1 < n_src && -2 - f1 < fp_slots_cap(cv))) continue;
        uint4* dst = reinterpret_cast<uint4*>(fpbase + fp_chunk_off(cv.layout, s, c) + vo);
        if (f1 >= 0) {
          *dst = (which ? v : k)[(pair * n_src + f1) * 16 + c];
        } else {
          const int m = -2 - f1, f2 = fill2[tau * G + e];
          uint4* old = reinterpret_cast<uint4*>(fpbase + fp_chunk_off(cv.layout, m, c) + vo);
          *dst = *old;
          if (f2 >= 0 && LQ_IN_BOUNDS(cv, f2 < n_src)) *old = (which ? v : k)[(pair * n_src + f2) * 16 + c];
        }
      }
    }
    quantise_pack_tile<G, P>(sK, sV, tile, tid, cv.layout);
  } else {
    const int i = (static_cast<int>(blockIdx.x) - n_tiles) * 256 + tid;
    if (i >= n_copy * 32) return;
    const int c = i & 15, which = (i >> 4) & 1, j = i >> 5;
    const int* copy = idx + (has_fill ? 3 : 1) * n_tiles * G;
    const int slot = copy[2 * j];
    const int64_t t = copy[2 * j + 1];
    if (!LQ_IN_BOUNDS(cv, t >= 0 && t < n_src && slot >= 0 && slot < fp_slots_cap(cv))) return;
    *reinterpret_cast<uint4*>(fpbase + fp_chunk_off(cv.layout, slot, c) + (which ? vdelta : 0)) =
        (which ? v : k)[(pair * n_src + t) * 16 + c];
  }
}

cudaError_t launch_ingest(const CacheView& cv, int layer, const void* k, const void* v, int n_src, const int* idx_dev,
                          int n_tiles, bool has_fill, int n_copy, int64_t tile0, cudaStream_t st) {
  dim3 grid(n_tiles + (n_copy * 32 + 255) / 256, cv.B * cv.Hkv);
  if (grid.x == 0) return cudaSuccess;
  const uint4* k4 = static_cast<const uint4*>(k);
  const uint4* v4 = static_cast<const uint4*>(v);
  const int hf = has_fill ? 1 : 0;
  if (cv.G == 32 && cv.planes == 1)
    lq_ingest_kernel<32, 1><<<grid, 256, 0, st>>>(cv, layer, k4, v4, n_src, idx_dev, n_tiles, hf, n_copy, tile0);
  else if (cv.G == 32 && cv.planes == 2)
    lq_ingest_kernel<32, 2><<<grid, 256, 0, st>>>(cv, layer, k4, v4, n_src, idx_dev, n_tiles, hf, n_copy, tile0);
  else if (cv.G == 64 && cv.planes == 1)
    lq_ingest_kernel<64, 1><<<grid, 256, 0, st>>>(cv, layer, k4, v4, n_src, idx_dev, n_tiles, hf, n_copy, tile0);
  else if (cv.G == 64 && cv.planes == 2)
    lq_ingest_kernel<64, 2><<<grid, 256, 0, st>>>(cv, layer, k4, v4, n_src, idx_dev, n_tiles, hf, n_copy, tile0);
  else
    return cudaErrorInvalidValue;
  return cudaGetLastError();
}

// ---------------------------------------------------------------------------------------
// Canonical export (introspection; not on the hot path).
// ---------------------------------------------------------------------------------------
__global__ void lq_export_codes_kernel(CacheView cv, int layer, int64_t n_quant, uint8_t* k_codes,
                                       uint8_t* v_codes) {
  // one thread per output byte: (pair, token, byte j) -> channels 4j..4j+3 (2-bit) or 2j, 2j+1 (4-bit)
  const int P = cv.planes, cpb = 4 / P;  // codes per byte
  const int64_t per_pair = n_quant * (kD / cpb);
  const int64_t total = static_cast<int64_t>(cv.B) * cv.Hkv * per_pair;
  for (int64_t idx = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x; idx < total;
       idx += static_cast<int64_t>(gridDim.x) * blockDim.x) {
    const int64_t pair = idx / per_pair;
    const int64_t rem = idx % per_pair;
    const int64_t tq = rem / (kD / cpb);
    const int jb = static_cast<int>(rem % (kD / cpb));
    const uint8_t* tile = cv.quant + layer * cv.quant_layer_stride + pair * cv.quant_head_stride +
                          (tq / cv.G) * quant_tile_bytes(cv.G, P);
    const int t = static_cast<int>(tq % cv.G);
    uint32_t kb = 0, vb = 0;
    for (int i = 0; i < cpb; ++i) {
      uint32_t kcode = 0, vcode = 0;
      for (int pl = 0; pl < P; ++pl) {
        int off, bit;
        kcode_pos(cv.layout, cv.G, P, pl, t, cpb * jb + i, off, bit);
        kcode |= ((*reinterpret_cast<const uint32_t*>(tile + off) >> bit) & 3u) << (2 * pl);
        vcode_pos(cv.layout, cv.G, P, pl, t, cpb * jb + i, off, bit);
        vcode |= ((*reinterpret_cast<const uint32_t*>(tile + off) >> bit) & 3u) << (2 * pl);
      }
      kb |= kcode << (2 * P * i);
      vb |= vcode << (2 * P * i);
    }
    if (k_codes) k_codes[idx] = static_cast<uint8_t>(kb);
    if (v_codes) v_codes[idx] = static_cast<uint8_t>(vb);
  }
}

__global__ void lq_export_params_kernel(CacheView cv, int layer, int64_t n_quant, uint16_t* k_scale,
                                        uint16_t* k_zero, uint16_t* v_scale, uint16_t* v_zero) {
  const int G = cv.G, NG = kD / G;
  const int64_t pairs = static_cast<int64_t>(cv.B) * cv.Hkv;
  const int64_t nk = pairs * (n_quant / G) * kD;  // K entries
  const int64_t nv = pairs * n_quant * NG;        // V entries
  for (int64_t idx = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x; idx < nk + nv;
       idx += static_cast<int64_t>(gridDim.x) * blockDim.x) {
    if (idx < nk) {
      const int d = static_cast<int>(idx % kD);
      const int64_t grp = (idx / kD) % (n_quant / G);
      const int64_t pair = idx / kD / (n_quant / G);
      const uint8_t* tile = cv.quant + layer * cv.quant_layer_stride + pair * cv.quant_head_stride +
                            grp * quant_tile_bytes(G, cv.planes);
      if (k_scale) k_scale[idx] = *reinterpret_cast<const uint16_t*>(tile + kscale_off(cv.layout, G, d));
      if (k_zero) k_zero[idx] = *reinterpret_cast<const uint16_t*>(tile + kzero_off(cv.layout, G, d));
    } else {
      const int64_t i2 = idx - nk;
      const int g = static_cast<int>(i2 % NG);
      const int64_t tq = (i2 / NG) % n_quant;
      const int64_t pair = i2 / NG / n_quant;
      const uint8_t* tile = cv.quant + layer * cv.quant_layer_stride + pair * cv.quant_head_stride +
                            (tq / G) * quant_tile_bytes(G, cv.planes);
      const int t = static_cast<int>(tq % G);
      if (v_scale) v_scale[i2] = *reinterpret_cast<const uint16_t*>(tile + vscale_off(cv.layout, G, cv.planes, t, g));
      if (v_zero) v_zero[i2] = *reinterpret_cast<const uint16_t*>(tile + vzero_off(cv.layout, G, cv.planes, t, g));
    }
  }
}

__global__ void lq_export_fp_kernel(CacheView cv, int layer, int n_fp, const int* __restrict__ slot_of_rank,
                                    uint4* fp_k, uint4* fp_v) {
  const int64_t total = static_cast<int64_t>(cv.B) * cv.Hkv * n_fp * 16;
  for (int64_t idx = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x; idx < total;
       idx += static_cast<int64_t>(gridDim.x) * blockDim.x) {
    const int c = static_cast<int>(idx & 15);
    const int rank = static_cast<int>((idx >> 4) % n_fp);
    const int64_t pair = (idx >> 4) / n_fp;
    const uint8_t* base = cv.fp + layer * cv.fp_layer_stride + pair * cv.fp_head_stride;
    const int64_t off = fp_chunk_off(cv.layout, slot_of_rank[rank], c);
    if (fp_k) fp_k[idx] = *reinterpret_cast<const uint4*>(base + off);
    if (fp_v) fp_v[idx] = *reinterpret_cast<const uint4*>(base + off + fp_v_delta(cv.layout));
  }
}

cudaError_t launch_export(const CacheView& cv, int layer, int n_fp, int64_t n_quant,
                          const int* slot_of_rank_dev, uint8_t* k_codes, uint8_t* v_codes,
                          uint16_t* k_scale, uint16_t* k_zero, uint16_t* v_scale, uint16_t* v_zero,
                          uint16_t* fp_k, uint16_t* fp_v, cudaStream_t st) {
  if (n_quant > 0 && (k_codes || v_codes))
    lq_export_codes_kernel<<<1184, 256, 0, st>>>(cv, layer, n_quant, k_codes, v_codes);
  if (n_quant > 0 && (k_scale || k_zero || v_scale || v_zero))
    lq_export_params_kernel<<<1184, 256, 0, st>>>(cv, layer, n_quant, k_scale, k_zero, v_scale, v_zero);
  if (n_fp > 0 && (fp_k || fp_v))
    lq_export_fp_kernel<<<1184, 256, 0, st>>>(cv, layer, n_fp, slot_of_rank_dev,
                                              reinterpret_cast<uint4*>(fp_k), reinterpret_cast<uint4*>(fp_v));
  return cudaGetLastError();
}


// ---------------------------------------------------------------------------------------
// Canonical import (checkpoint / resume; the inverse of the export above; not on the hot path).
// One CTA per (key group, pair) builds the tile in shared memory -- codes by atomicOr into the words the
// layout assigns them, scale and zero by plain 16-bit stores -- and writes it out with 16-byte stores.
// ---------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256)
lq_import_tile_kernel(CacheView cv, int layer, int64_t n_quant, const uint8_t* __restrict__ k_codes,
                      const uint8_t* __restrict__ v_codes, const uint16_t* __restrict__ k_scale,
                      const uint16_t* __restrict__ k_zero, const uint16_t* __restrict__ v_scale,
                      const uint16_t* __restrict__ v_zero) {
  __shared__ __align__(16) uint32_t sm[quant_tile_bytes(64, 2) / 4];
  const int G = cv.G, P = cv.planes, NG = kD / G, cpb = 4 / P;
  const int tile_bytes = quant_tile_bytes(G, P);
  const int64_t grp = blockIdx.x, pair = blockIdx.y;
  const int tid = threadIdx.x;
  if (!LQ_IN_BOUNDS(cv, grp < cv.quant_tiles_cap)) return;
  for (int i = tid; i < tile_bytes / 4; i += 256) sm[i] = 0u;
  __syncthreads();
  uint16_t* sm16 = reinterpret_cast<uint16_t*>(sm);
  for (int idx = tid; idx < G * kD; idx += 256) {
    const int t = idx / kD, d = idx % kD;
    const int64_t byte = (pair * n_quant + grp * G + t) * (kD / cpb) + d / cpb;
    const uint32_t kcode = (k_codes[byte] >> (2 * P * (d % cpb))) & ((1u << (2 * P)) - 1u);
    const uint32_t vcode = (v_codes[byte] >> (2 * P * (d % cpb))) & ((1u << (2 * P)) - 1u);
    for (int pl = 0; pl < P; ++pl) {
      int off, bit;
      kcode_pos(cv.layout, G, P, pl, t, d, off, bit);
      atomicOr(&sm[off >> 2], ((kcode >> (2 * pl)) & 3u) << bit);
      vcode_pos(cv.layout, G, P, pl, t, d, off, bit);
      atomicOr(&sm[off >> 2], ((vcode >> (2 * pl)) & 3u) << bit);
    }
  }
  for (int d = tid; d < kD; d += 256) {
    const int64_t i = (pair * (n_quant / G) + grp) * kD + d;
    sm16[kscale_off(cv.layout, G, d) >> 1] = k_scale[i];
    sm16[kzero_off(cv.layout, G, d) >> 1] = k_zero[i];
  }
  for (int idx = tid; idx < G * NG; idx += 256) {
    const int t = idx / NG, g = idx % NG;
    const int64_t i = (pair * n_quant + grp * G + t) * NG + g;
    sm16[vscale_off(cv.layout, G, P, t, g) >> 1] = v_scale[i];
    sm16[vzero_off(cv.layout, G, P, t, g) >> 1] = v_zero[i];
  }
  __syncthreads();
  uint8_t* tile = cv.quant + layer * cv.quant_layer_stride + pair * cv.quant_head_stride + grp * tile_bytes;
  for (int i = tid; i < tile_bytes / 16; i += 256)
    reinterpret_cast<uint4*>(tile)[i] = reinterpret_cast<const uint4*>(sm)[i];
}

__global__ void lq_import_fp_kernel(CacheView cv, int layer, int n_fp, const int* __restrict__ slot_of_rank,
                                    const uint4* __restrict__ fp_k, const uint4* __restrict__ fp_v) {
  const int64_t total = static_cast<int64_t>(cv.B) * cv.Hkv * n_fp * 16;
  for (int64_t idx = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x; idx < total;
       idx += static_cast<int64_t>(gridDim.x) * blockDim.x) {
    const int c = static_cast<int>(idx & 15);
    const int rank = static_cast<int>((idx >> 4) % n_fp);
    const int64_t pair = (idx >> 4) / n_fp;
    const int slot = slot_of_rank[rank];
    if (!LQ_IN_BOUNDS(cv, slot >= 0 && slot < fp_slots_cap(cv))) continue;
    uint8_t* base = cv.fp + layer * cv.fp_layer_stride + pair * cv.fp_head_stride;
    const int64_t off = fp_chunk_off(cv.layout, slot, c);
    *reinterpret_cast<uint4*>(base + off) = fp_k[idx];
    *reinterpret_cast<uint4*>(base + off + fp_v_delta(cv.layout)) = fp_v[idx];
  }
}

cudaError_t launch_import(const CacheView& cv, int layer, int n_fp, int64_t n_quant, const int* slot_of_rank_dev,
                          const uint8_t* k_codes, const uint8_t* v_codes, const uint16_t* k_scale,
                          const uint16_t* k_zero, const uint16_t* v_scale, const uint16_t* v_zero,
                          const uint16_t* fp_k, const uint16_t* fp_v, cudaStream_t st) {
  if (n_quant > 0) {
    dim3 grid(static_cast<unsigned>(n_quant / cv.G), cv.B * cv.Hkv);
    lq_import_tile_kernel<<<grid, 256, 0, st>>>(cv, layer, n_quant, k_codes, v_codes, k_scale, k_zero, v_scale, v_zero);
  }
  if (n_fp > 0)
    lq_import_fp_kernel<<<1184, 256, 0, st>>>(cv, layer, n_fp, slot_of_rank_dev, reinterpret_cast<const uint4*>(fp_k),
                                              reinterpret_cast<const uint4*>(fp_v));
  return cudaGetLastError();
}

}  // namespace lq

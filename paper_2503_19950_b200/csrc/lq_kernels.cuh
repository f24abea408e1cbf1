// Launchers of the CUDA kernels behind the C-ABI (host-callable; defined in the .cu files).
#pragma once
#include <cuda_runtime.h>
#include <cstdint>

#include "lq_layout.cuh"

namespace lq {

// Geometry and base pointers shared by every kernel.
struct CacheView {
  int B, Hq, Hkv, G, W;
  int planes;                 // 2-bit code planes per code: 1 (2-bit cache) or 2 (4-bit cache)
  int layout;                 // kLayoutFragment (mma.sync kernel) or kLayoutRow (tcgen05 kernel), see lq_layout.cuh
  int64_t quant_tiles_cap;    // capacity in tiles per (layer, b, kv)
  int64_t quant_head_stride;  // bytes between (b, kv) heads of the 2-bit store
  int64_t quant_layer_stride;
  int64_t fp_head_stride;     // bytes between (b, kv) heads of the fp store (3W/16 fp tiles)
  int64_t fp_layer_stride;
  uint8_t* quant;  // 2-bit store base
  uint8_t* fp;     // full-precision store base
  int* status;     // the cache's device status word (bit 0: a bounded wait gave up; bit 2: an index check of
                   // the LQ_DEBUG_BOUNDS build failed)
};

// Index checks of the debug build (-DLQ_DEBUG_BOUNDS, python -m paper_2503_19950_b200.build --bounds): every
// access whose index comes from the host's bookkeeping or from a launch argument is checked against the extent
// of the store it goes to; a failing check sets bit 2 of the status word and the access is skipped -- nothing
// traps.  In the normal build the checks compile to nothing.
#ifdef LQ_DEBUG_BOUNDS
#define LQ_IN_BOUNDS(cv, cond) ((cond) ? true : (atomicOr((cv).status, 4), false))
#else
#define LQ_IN_BOUNDS(cv, cond) ((void)sizeof(cond), true)
#endif
// slots of the full-precision store of one (layer, b, kv); tiles of the 2-bit store
__host__ __device__ inline int64_t fp_slots_cap(const CacheView& cv) {
  return cv.fp_head_stride / (2 * kD * 2);
}

struct EvictList {
  uint16_t slot[kMaxW];  // physical fp slots of the tokens to quantise, in removal order
  uint16_t src[kMaxW];   // slot whose row moves into slot[e] afterwards (kNoMove: nothing moves there)
};
constexpr uint16_t kNoMove = 0xFFFF;

struct LayerList {
  int n;
  uint8_t layer[128];
};

// K1: write n_tokens new rows into fp slots [slot0, slot0 + n_tokens) of one layer.
// k, v: [B, Hkv, n_src_tokens, D] bf16; tokens [src0, src0 + n_tokens) of them are written.
// extra_bytes (a multiple of 16) are copied from extra_src to extra_dst by the same launch.
cudaError_t launch_append(const CacheView& cv, int layer, const void* k, const void* v,
                          int n_src_tokens, int src0, int n_tokens, int slot0, cudaStream_t st,
                          const void* extra_src = nullptr, void* extra_dst = nullptr, int extra_bytes = 0);

// K2: overflow step for the listed layers (all of them in the same state): quantise + pack the W
// rows of `ev` into quant tiles [tile0, tile0 + W/G), then move rows 2W+e into slot ev.slot[e].
cudaError_t launch_compress(const CacheView& cv, const LayerList& layers, const EvictList& ev,
                            int64_t tile0, int n_groups, cudaStream_t st);

// Ingestion of n_src new tokens in one launch (lq_ingest_kernel): idx_dev = [n_tiles*G sources of the new key
// groups in store order][with has_fill: 2 x n_tiles*G take-over sources][n_copy x (fp slot, new-tensor row)];
// k, v = [B, Hkv, n_src, 128] bf16.
cudaError_t launch_ingest(const CacheView& cv, int layer, const void* k, const void* v, int n_src, const int* idx_dev,
                          int n_tiles, bool has_fill, int n_copy, int64_t tile0, cudaStream_t st);

// Canonical export of one layer into device buffers (any pointer may be null).
// slot_of_rank[i] = fp slot of the i-th kept id (ascending ids); device array of n_fp ints.
cudaError_t launch_export(const CacheView& cv, int layer, int n_fp, int64_t n_quant,
                          const int* slot_of_rank_dev, uint8_t* k_codes, uint8_t* v_codes,
                          uint16_t* k_scale, uint16_t* k_zero, uint16_t* v_scale, uint16_t* v_zero,
                          uint16_t* fp_k, uint16_t* fp_v, cudaStream_t st);

// Canonical import of one (empty) layer from device copies of the image arrays: the inverse of launch_export.
cudaError_t launch_import(const CacheView& cv, int layer, int n_fp, int64_t n_quant, const int* slot_of_rank_dev,
                          const uint8_t* k_codes, const uint8_t* v_codes, const uint16_t* k_scale,
                          const uint16_t* k_zero, const uint16_t* v_scale, const uint16_t* v_zero,
                          const uint16_t* fp_k, const uint16_t* fp_v, cudaStream_t st);

// Split-K partial state: for partition s of head pair p = b*Hkv + kv and query head j of the
// group (j < r): o[128] unnormalised, m (in log2 units), l.
//   part_o : [(p*S + s)*r + j][128] float,  part_ml : [(p*S + s)*r + j][2] float
struct DecodeArgs {
  CacheView cv;
  int layer;
  int n_fp;
  int64_t n_quant;
  int S;  // records reserved per (b, kv): record (pair, s) at pair*S + s.  Scalar kernel: every pair has S
          // partitions.  Tensor-core kernel: pair p has S - 1 + (p < n_extra) CTAs, so that the grid is an
          // exact multiple of the SM count (equal load on every SM)
  int n_extra;
  int tiles_fp, tiles_quant;  // fp tiles (16 slots) and quant tiles (G tokens) per (b, kv)
  int zero;                   // always 0; an opaque loop bound for the kernels
  float scale_log2;  // sm_scale * log2(e)
  const void* q;     // [B, Hq, D] bf16
  float* part_o;
  float* part_ml;
  void* out;
  int out_bf16;
  // tensor-core kernel, fused append: when new_k is not null, row new_slot of the fp store (counted in n_fp) is
  // not in memory yet; the warp that visits its tile takes the row from new_k / new_v ([B, Hkv, 1, 128] bf16) and
  // writes it to the store
  const void* new_k;
  const void* new_v;
  int new_slot;
  // left padding (null when the cache has none): per sequence b, tokens attention leaves out.
  //   rowinfo[4*b + 0] = leading quant tiles that are padding entirely (not even loaded),
  //   rowinfo[4*b + 1] = first quant tile from which on no token is padding (tiles in between consult qmask),
  //   rowinfo[4*b + 2] = 1 if some slot of the fp store is padding (fpmask is consulted);
  //   qmask[b*qmask_words + i/32] bit i%32: token i of the quantised store, fpmask likewise per fp slot.
  //   Tensor-core kernel: the CTAs of a padded launch are shared out by the work each sequence has left:
  //   cta_map[c] = pair | slot << 16 for CTA c (n_ctas of them), pair_ctas[pair] = CTAs of that pair (<= S).
  const int32_t* rowinfo;
  const uint32_t* qmask;
  const uint32_t* fpmask;
  int qmask_words, fpmask_words;
  const int32_t* cta_map;
  const int32_t* pair_ctas;
  int n_ctas;
  int* status;  // device word; kernels OR error bits into it (bounded waits that gave up)
  int* tickets; // one 128-byte line per (b, kv): word [1] is the arrival counter of the fused second
                // pass, word [2] the "sum out of range" flag of the accumulators below; both 0 at rest
                // (null: static split and a separate merge launch)
  // Tensor-core kernel, pairs with more than one CTA: besides its record every CTA adds its partial, scaled to
  // a reference score all CTAs of the pair compute alike, to acc with global atomics, so that the CTA that
  // completes the pair only has to read one sum: acc[pair * kAccStride + h * 128 + d] and, for the
  // denominators, acc[pair * kAccStride + kMaxRatio * 128 + h]; all zero at rest.  null: records only.
  float* acc;
  // tcgen05 kernel (row layout): per (b, kv) pair u_fp_units fp units of 32 slots, then u_supertiles super-tiles of
  // 128 quantised tokens: u_items items of total cost u_cost (in units of 2 KB); the pairs' items lie on one cost
  // line that is cut into n_ctas equal ranges; S = record slots per pair
  int u_items, u_fp_units, u_supertiles, u_cost;
  // test hook (lq_debug_stall_next_decode): the tensor-core kernels arm the barrier of the query copy but issue
  // no copy and poll with a short limit, so that the bounded wait runs out and the failure path is taken
  int debug_stall;
  // tensor-core (mma.sync) kernel: 1 = the launch before this one on the stream is a decode launch of another layer
  // of the same cache (LQ_FLAG_OVERLAP_DECODE): nothing the main loop reads is written by it, so the dependency
  // wait of the programmatic launch moves behind the main loop, in front of the first use of the shared workspace
  int early;
};

constexpr int kAccStride = kMaxRatio * 128 + 32;  // floats per (b, kv) pair in DecodeArgs::acc

cudaError_t launch_decode_scalar(const DecodeArgs& a, cudaStream_t st);
// Fills S and the tile counts of `a` for the tensor-core kernel (S <= max_records; s_override > 0 forces S).
void plan_decode_mma(DecodeArgs& a, int sm_count, int max_records, int s_override);
// Padded batch: shares one resident wave of CTAs out over the (b, kv) pairs in proportion to the tiles each
// sequence still has to visit (rowinfo as in DecodeArgs, on the host).  Fills cta_map (room for
// max_ctas_decode_mma(sm_count) entries) and pair_ctas (B * Hkv entries); returns the grid size and sets
// *stride to the record stride (the largest CTA count of a pair, <= max_records).
int max_ctas_decode_mma(int sm_count);
// overlapped: the plan of a launch that overlaps the one before it (a third of the wave, DecodeArgs::early).
int plan_decode_mma_padded(const DecodeArgs& a, int sm_count, int max_records, const int32_t* rowinfo_host,
                           int32_t* cta_map, int32_t* pair_ctas, int* stride, bool overlapped = false);
cudaError_t launch_decode_mma(const DecodeArgs& a, cudaStream_t st);
// tcgen05 kernel: fills tiles_fp (fp units), tiles_quant, the u_* fields, n_ctas and S (<= max_records, <= 128)
void plan_decode_umma(DecodeArgs& a, int sm_count, int max_records, int s_override);
cudaError_t launch_decode_umma(const DecodeArgs& a, cudaStream_t st);
cudaError_t launch_merge(const DecodeArgs& a, cudaStream_t st);

}  // namespace lq

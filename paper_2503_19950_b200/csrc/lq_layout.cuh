// Device-side layout of the mixed KV cache (private to the library; the public format is the
// canonical image of include/lq.h).  head_dim D = 128 throughout.
//
// Both stores are laid out so that the tensor-core decode kernel can bring one unit into shared
// memory with a single 1-D bulk copy and then read its mma.sync fragments with conflict-free
// 16-byte shared loads, with no in-kernel shuffling of codes:
//
// Full-precision store, per (layer, b, kv head): 3W/16 "fp tiles" of 16 slots, 8 KB each:
//   [K rows: 16 x 256 B][V rows: 16 x 256 B].  Row `s` (slot % 16) holds 16 chunks of 16 B
//   (8 channels each); chunk c is stored at chunk position c ^ (s & 7), so that the 8 rows an
//   ldmatrix reads for one chunk fall in 8 different bank groups.  Slots [0, n_fp) are valid
//   (the overflow step back-fills the holes it makes, see lq_compress_kernel).
//
// 2-bit store, per (layer, b, kv head): a sequence of "quant tiles"; one tile = one key group =
//   G consecutive removed tokens = G/16 sub-tiles of 16 tokens.  Byte offsets inside a tile:
//     0                      K scale, 128 bf16 in fragment order      (256 B)
//     256                    K zero,  128 bf16 in channel order       (256 B)
//     512                    K codes, G/16 sub-tiles x 512 B
//     512 + 32 G             V codes, G/16 sub-tiles x 512 B
//     512 + 64 G             V scale, G/16 sub-tiles x (4096/G) B
//     512 + 64 G + 256       V zero,  G/16 sub-tiles x (4096/G) B
//     tile bytes = 1024 + 64 G   (3072 at G = 32, 5120 at G = 64; 96 / 80 B per token)
//   4-bit codes (G = 32 only): every code is split into two 2-bit planes; the K codes area holds
//   plane 0 then plane 1 (32 G bytes each), likewise the V codes area, and the offsets after the
//   codes move accordingly: tile bytes = 1024 + 128 G = 5120 (160 B per token).
//
//   Fragment coordinates use lane = 4*(lane/4) + j of a warp, as in mma.sync.m16n8k16:
//   K codes of sub-tile u: 32-bit word 4*lane + 2*nt + w  (lane = 4*n + j), bits
//     [16h + 2ks + 1 : 16h + 2ks]  = code of token 16u + 8nt + n, channel 16ks + 8w + 2j + h.
//     (word (nt, w) masked at code position ks is the B-fragment register w of the k-step ks
//      for the 8 tokens of n-tile nt: two codes, one per 16-bit half.)
//   K scale: channel 16ks + 8w + 2j + h at bf16 index 8*(4*(ks/2) + j) + 2*(2*(ks%2) + w) + h
//     (four 16-byte loads give a lane the scale of every channel it multiplies).  K zero stays in
//     channel order: an ldmatrix with all eight row addresses equal turns 32 bytes of it into the A
//     fragment (every row the same) of the per-group q.zero product.
//   V codes of sub-tile u: word 4*lane + dh + 2*th (lane = 4*r + j), bits [16h + 2mt + 1 : 16h + 2mt]
//     = code of token 16u + 8th + 2j + h, channel 16mt + 8dh + r
//     (word (th, dh) masked at position mt is the A-fragment register dh + 2*th of m-tile mt).
//   V scale of sub-tile u (NG = 128/G groups per token): 32-bit word holding the pair
//     (token 8th + 2j, token 8th + 2j + 1) of group g sits at word index
//     4*(4*(g/2) + j) + 2*(g%2) + th.
//   V zero of sub-tile u: the pair (token 8th + 2j, 8th + 2j + 1) of group g at word 2*(4g + j) + th.
#pragma once
#include <cstdint>

namespace lq {

constexpr int kD = 128;
constexpr int kFpTileSlots = 16;
constexpr int kFpTileBytes = 2 * kFpTileSlots * kD * 2;  // K rows then V rows
constexpr int kFpTileVOffset = kFpTileSlots * kD * 2;
constexpr int kMaxW = 512;
constexpr int kMaxRatio = 8;  // query heads per KV head

// P = code planes: 1 for 2-bit codes; 2 for 4-bit codes, stored as two 2-bit planes (plane 0 = the low
// two bits, plane 1 = the high two bits of every code), each plane in the 2-bit fragment order
__host__ __device__ constexpr int quant_tile_bytes(int G, int P = 1) { return 1024 + 64 * G * P; }
__host__ __device__ constexpr int qt_plane_bytes(int G) { return 32 * G; }  // K or V codes of one plane
__host__ __device__ constexpr int qt_kscale_off() { return 0; }
__host__ __device__ constexpr int qt_kzero_off() { return 256; }
__host__ __device__ constexpr int qt_kcodes_off() { return 512; }
__host__ __device__ constexpr int qt_vcodes_off(int G, int P = 1) { return 512 + 32 * G * P; }
__host__ __device__ constexpr int qt_vscale_off(int G, int P = 1) { return 512 + 64 * G * P; }
__host__ __device__ constexpr int qt_vzero_off(int G, int P = 1) { return 512 + 64 * G * P + 256; }
__host__ __device__ constexpr int vsz_subtile_bytes(int G) { return 4096 / G; }

// ---- element addressing (used by the overflow, export and scalar kernels) -------------
// byte offset of bf16 element (slot, channel d) of the K rows of the fp tile holding `slot`
__host__ __device__ inline int64_t fp_elem_off(int slot, int d) {
  int s = slot & 15;
  int chunk = (d >> 3) ^ (s & 7);
  return static_cast<int64_t>(slot >> 4) * kFpTileBytes + s * 256 + chunk * 16 + (d & 7) * 2;
}
// byte offset of 16-byte chunk c of row `slot`
__host__ __device__ inline int64_t fp_chunk_off(int slot, int c) {
  int s = slot & 15;
  return static_cast<int64_t>(slot >> 4) * kFpTileBytes + s * 256 + ((c ^ (s & 7)) << 4);
}

// bf16 index of channel d inside the K scale block (the K zero block is in channel order)
__host__ __device__ inline int kparam_index(int d) {
  int ks = d >> 4, w = (d >> 3) & 1, j = (d >> 1) & 3, h = d & 1;
  return 8 * (4 * (ks >> 1) + j) + 2 * (2 * (ks & 1) + w) + h;
}
// K code of (token t of the tile, channel d): word index (in the tile's K codes area) and bit
__host__ __device__ inline void kcode_pos(int t, int d, int& word, int& bit) {
  int u = t >> 4, nt = (t >> 3) & 1, n = t & 7;
  int ks = d >> 4, w = (d >> 3) & 1, j = (d >> 1) & 3, h = d & 1;
  word = u * 128 + 4 * (4 * n + j) + 2 * nt + w;
  bit = 16 * h + 2 * ks;
}
__host__ __device__ inline void vcode_pos(int t, int d, int& word, int& bit) {
  int u = t >> 4, th = (t >> 3) & 1, j = (t >> 1) & 3, h = t & 1;
  int mt = d >> 4, dh = (d >> 3) & 1, r = d & 7;
  word = u * 128 + 4 * (4 * r + j) + dh + 2 * th;
  bit = 16 * h + 2 * mt;
}
// bf16 index (within the tile's V scale area) of (token t of the tile, group g)
__host__ __device__ inline int vscale_index(int t, int g, int G) {
  int u = t >> 4, th = (t >> 3) & 1, j = (t >> 1) & 3, h = t & 1;
  int word = 4 * (4 * (g >> 1) + j) + 2 * (g & 1) + th;
  return u * (vsz_subtile_bytes(G) / 2) + 2 * word + h;
}
__host__ __device__ inline int vzero_index(int t, int g, int G) {
  int u = t >> 4, th = (t >> 3) & 1, j = (t >> 1) & 3, h = t & 1;
  int word = 2 * (4 * g + j) + th;
  return u * (vsz_subtile_bytes(G) / 2) + 2 * word + h;
}

}  // namespace lq

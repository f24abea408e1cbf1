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
//   4-bit codes: every code is split into two 2-bit planes; the K codes area holds
//   plane 0 then plane 1 (32 G bytes each), likewise the V codes area, and the offsets after the
//   codes move accordingly: tile bytes = 1024 + 128 G (5120 at G = 32, 9216 at G = 64; 160 / 144 B per token).
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


// =======================================================================================
// Layout 1 (kLayoutRow): the layout of the tcgen05 decode kernel (LQ_KERNEL_UMMA).  Same bytes per
// token as layout 0, but every packed word holds 16 codes of ONE row of a tensor-core A operand, so
// that the thread that owns the row (a token for q.k, a channel for p.v) unpacks it on its own and
// writes it to tensor memory.
//
// Full-precision store, per (layer, b, kv head): "fp units" of 32 slots, 16 KB each:
//   [K rows 8 KB][V rows 8 KB]; inside either half the 16-byte chunk c (8 channels) of slot s sits at
//   (s/8)*2048 + c*128 + (s%8)*16: groups of 8 slots, chunk-major inside a group.  Read by the tensor
//   core straight from shared memory in the canonical no-swizzle form, as a K-major A operand for q.k
//   (rows = tokens: 8-row groups 2048 B apart, 16-byte k-chunks 128 B apart) and as an MN-major A
//   operand for p.v (rows = channels: 8-channel chunks 128 B apart, 8-token groups 2048 B apart).
//
// 2-bit store: one tile per key group of G tokens, 1024 + 64 G bytes as in layout 0 (planes == 1 only):
//     0            K codes: [half (2)][token (G)][4 words]; word j of half hf holds channels
//                  16*(4hf+j) .. +15 of the token
//     32 G         V codes: [channel (128)][G/16 words]; word j holds tokens 16j .. 16j+15 of the channel
//     64 G         K scale, 128 bf16 in channel order;  64 G + 256: K zero likewise
//     64 G + 512   V scale and zero per token: [token (G)][scale of group 0..NG-1, zero of group 0..NG-1]
//   Inside a code word element e (0..15) of the row sits at bit 16*(e&1) + 8*(e>>3) + 2*((e>>1)&3):
//   masking the word (or the word shifted right by 8) with 0x00030003 << 2i yields elements 2i', 2i'+1
//   as a pair of bf16 subnormals, i.e. one 32-bit column of the A operand of k-step (word), times 2^(2i).
// =======================================================================================
constexpr int kLayoutFragment = 0;
constexpr int kLayoutRow = 1;
constexpr int kFpUnitSlots = 32;
constexpr int kFpUnitBytes = 2 * kFpUnitSlots * kD * 2;
constexpr int kFpUnitVOffset = kFpUnitSlots * kD * 2;

__host__ __device__ constexpr int row_kcodes_off() { return 0; }
__host__ __device__ constexpr int row_vcodes_off(int G) { return 32 * G; }
__host__ __device__ constexpr int row_kscale_off(int G) { return 64 * G; }
__host__ __device__ constexpr int row_kzero_off(int G) { return 64 * G + 256; }
__host__ __device__ constexpr int row_vsz_off(int G) { return 64 * G + 512; }
// bit of element e (0..15) inside a code word
__host__ __device__ constexpr int row_code_bit(int e) { return 16 * (e & 1) + 8 * (e >> 3) + 2 * ((e >> 1) & 3); }

// ---- layout-generic element addressing (overflow, ingestion, export and scalar kernels) ----
// bytes between the K row and the V row of a slot
__host__ __device__ inline int fp_v_delta(int layout) { return layout == kLayoutRow ? kFpUnitVOffset : kFpTileVOffset; }
__host__ __device__ inline int64_t fp_store_bytes(int layout, int slots) {
  return layout == kLayoutRow ? static_cast<int64_t>((slots + kFpUnitSlots - 1) / kFpUnitSlots) * kFpUnitBytes
                              : static_cast<int64_t>((slots + kFpTileSlots - 1) / kFpTileSlots) * kFpTileBytes;
}
__host__ __device__ inline int64_t fp_chunk_off(int layout, int slot, int c) {
  if (layout == kLayoutRow)
    return static_cast<int64_t>(slot >> 5) * kFpUnitBytes + ((slot & 31) >> 3) * 2048 + c * 128 + (slot & 7) * 16;
  return fp_chunk_off(slot, c);
}
__host__ __device__ inline int64_t fp_elem_off(int layout, int slot, int d) {
  return layout == kLayoutRow ? fp_chunk_off(layout, slot, d >> 3) + (d & 7) * 2 : fp_elem_off(slot, d);
}
// byte offset (in the tile) of the 32-bit word and the bit position of the K / V code of (token t, channel d)
__host__ __device__ inline void kcode_pos(int layout, int G, int P, int pl, int t, int d, int& byte_off, int& bit) {
  if (layout == kLayoutRow) {
    const int ks = d >> 4;
    byte_off = row_kcodes_off() + 4 * ((ks >> 2) * (G * 4) + t * 4 + (ks & 3));
    bit = row_code_bit(d & 15);
  } else {
    int word;
    kcode_pos(t, d, word, bit);
    byte_off = qt_kcodes_off() + pl * qt_plane_bytes(G) + 4 * word;
  }
}
__host__ __device__ inline void vcode_pos(int layout, int G, int P, int pl, int t, int d, int& byte_off, int& bit) {
  if (layout == kLayoutRow) {
    byte_off = row_vcodes_off(G) + 4 * (d * (G / 16) + (t >> 4));
    bit = row_code_bit(t & 15);
  } else {
    int word;
    vcode_pos(t, d, word, bit);
    byte_off = qt_vcodes_off(G, P) + pl * qt_plane_bytes(G) + 4 * word;
  }
}
// byte offsets (in the tile) of the bf16 scale / zero of key channel d, and of value (token t, group g)
__host__ __device__ inline int kscale_off(int layout, int G, int d) {
  return layout == kLayoutRow ? row_kscale_off(G) + 2 * d : qt_kscale_off() + 2 * kparam_index(d);
}
__host__ __device__ inline int kzero_off(int layout, int G, int d) {
  return layout == kLayoutRow ? row_kzero_off(G) + 2 * d : qt_kzero_off() + 2 * d;
}
__host__ __device__ inline int vscale_off(int layout, int G, int P, int t, int g) {
  return layout == kLayoutRow ? row_vsz_off(G) + 2 * (t * (2 * (kD / G)) + g) : qt_vscale_off(G, P) + 2 * vscale_index(t, g, G);
}
__host__ __device__ inline int vzero_off(int layout, int G, int P, int t, int g) {
  return layout == kLayoutRow ? row_vsz_off(G) + 2 * (t * (2 * (kD / G)) + kD / G + g)
                              : qt_vzero_off(G, P) + 2 * vzero_index(t, g, G);
}

}  // namespace lq

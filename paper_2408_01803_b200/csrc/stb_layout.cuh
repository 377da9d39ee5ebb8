// Packed ("streaming") layout of an N:8 structured-binary layer, shared by the CUDA kernels.
// Host + device code, so that the index arithmetic can also be compiled and checked on the
// host.
//
// The unit of the layout is a TILE: 32 output rows x one 128-column block; all tiles of a layer
// have the same size, which depends on N alone, and follow each other in (row tile, block)
// order after a header, a per-block table and a table of residual words.  The residual stream
// (the second scale of the salient columns and their residual codes, whose size follows each
// block's own salient count) comes after the tiles, one run per row tile.  Inside a tile the work is split the way a warp-level tensor-core
// instruction (m16n8k16) splits a 16 x 16 operand: lane = 4 g + t  (g = 0..7, t = 0..3) owns
//     rows    r_j = g + 8 j      (j = 0..3) of the tile and, of each of them,
//     groups  G_s = 4 s + t      (s = 0..3) of the block (a group = 8 columns),
// i.e. 16 (row, group) slots  u = 4 j + s,  as many weights as one row of the block.  With
// this split the 8 decoded fp16 weights of slot (j, s) are exactly the lane's operand
// registers of two m16n8k16 instructions (columns 32 s + 8 t + 0..7 of rows g + 8 j).
//
// Every field is stored lane-major so that a warp reads it with coalesced vector loads:
//
//   mask    32 x uint4          byte u of the lane's 16 bytes = keep mask of slot u, stored as its
//                               INDEX among the C(8, N) masks with N bits set (increasing
//                               numeric order): the same 8 bits, but a lookup table keyed by it
//                               has at most 70 entries, which keeps shared-memory lookups by the
//                               32 lanes of a warp nearly free of bank conflicts
//                               N = 6 stores the same bytes in another order (mask_pairs): the
//                               GEMV multiplies rank-ordered weights with the sparse tensor-core
//                               instruction, whose selection metadata for rows g + 16 mt and
//                               g + 16 mt + 8 comes from lanes 2 mt and 2 mt + 1 of the quad.  So
//                               lane (g, t) holds, at bytes 8 b + 2 tq (16 bits), the pair field
//                               16 (i0 + 28 i1) of the keep-mask indices i0, i1 of group
//                               4 (2 (t & 1) + b) + tq of rows g + 16 (t >> 1) and g + 16 (t >> 1) + 8:
//                               the byte offset into a table of 784 16-byte entries that holds the
//                               metadata of both rows.
//   region  N words per lane    two-bit region codes, 16 per word, of the lane's 16 N kept
//                               weights: first the "low" part (ranks k < min(N, 4) of every
//                               slot, weight number wl = u NL + k), then the "high" part
//                               (ranks 4..N-1, wh = u NH + k - 4).  Inside a word the codes are
//                               nibble-interleaved (code_bit) so that (R & 0x33333333) and
//                               ((R >> 2) & 0x33333333) are byte-permute selectors.
//   sign    N/2 words per lane  one bit per kept weight (1 = negative), same low / high split
//                               and weight numbering, pre-positioned (sign_bit) so that one
//                               shift puts the bits of a selector word on bit 2 of its
//                               nibbles.  An odd part ends in half a word: lanes l and l + 16
//                               share word l of a 16-word plane (lower lane bits 2,1 of each
//                               nibble, upper lane bits 3,0).
//   scale   32 x uint2          per row: word A = low bytes of the fp16 scales a_dense,
//                               a_inter, a_sparse, a_sal1; word B = their high bytes.  Rows
//                               are stored in the order p = 4 (r % 8) + r / 8, so that the
//                               four rows of a lane are contiguous.
// and, outside the tile, in the residual stream of the row tile, one record per block, block after block:
//   sal2    32 x u16            a_sal2 per row, rows in the order p = 4 (r % 8) + r / 8 like the scales
//   resid   ceil(S / 4) words   for the block's S salient columns, each word stored once per lane group g
//                               (8 x 4 bytes): slot q (the q-th salient column of the block, ascending;
//                               q / 4 picks the word) of row r_j has the two-bit code 0 = +a_sal2,
//                               2 = -a_sal2, 1 = no term (weight dropped, or q >= S), at
//                               code_bit(4 j + q % 4).
//                               The words of all blocks are numbered block after block
//                               (BlockInfo::rw_off = number of a block's first word, Header::nrw
//                               their total), so block b's record starts 64 b + 32 rw_off bytes into
//                               the row tile's stream and the records of a run of blocks are one
//                               contiguous piece.  The residual word table (ResidWord, one entry per
//                               word, after the block table) names the word's block, its place in
//                               the block and its four salient columns, so that a reader can walk
//                               the words of a run of blocks without looking at the blocks.
//
// Tile bytes = 512 + 192 N + 256; with the record, 26 + 6 N bytes per row and block (50 / 56 / 62 at
// N = 4 / 5 / 6) plus ceil(S / 4) bytes per row for the block's S salient columns.
#pragma once
#include <stdint.h>

#if defined(__CUDACC__)
#define STB_HD __host__ __device__ __forceinline__
#else
#define STB_HD inline
#endif

namespace stb {

constexpr uint32_t kMagic = 0x32425453u;  // "STB2"
constexpr int kBlock = 128;               // columns per block
constexpr int kGroup = 8;                 // columns per group (M)
constexpr int kTileRows = 32;
constexpr int kMaxSalient = 32;

struct Header {          // 64 bytes at the start of the packed buffer
  uint32_t magic;
  uint32_t version;
  int32_t n, m, N;
  int32_t nblk;          // m / 128
  int32_t ntile;         // ceil(n / 32)
  uint32_t tiles_offset; // byte offset of tile (0, 0)
  uint64_t rt_stride;    // bytes of one row tile = nblk * tile_bytes
  uint64_t used_bytes;
  uint32_t status;       // 0 or STB_ERR_CORRUPT
  uint32_t tile_bytes;
  uint32_t nrw;          // residual words per row tile (all blocks); the residual streams start at
                         // tiles_offset + rt_stride * ntile, 64 nblk + 32 nrw bytes per row tile
  uint32_t rwtab_offset; // byte offset of the residual word table
};
static_assert(sizeof(Header) == 64, "header is 64 bytes");

struct BlockInfo {       // 64 bytes, one per block, right after the header
  uint64_t salient[2];   // 128-bit salient-column mask
  uint32_t nsal;         // number of salient columns
  uint32_t rw_off;       // number of the block's first residual word
  uint32_t nrw;          // its residual words: ceil(nsal / 4)
  uint32_t pad;
  uint8_t cols[32];      // the salient columns (0..127) in ascending order; unused entries 0
};
static_assert(sizeof(BlockInfo) == 64, "block info is 64 bytes");

struct ResidWord {       // 8 bytes, one per residual word, in word order
  uint32_t block_wq;     // 8 * (the block the word belongs to) + (its number 0..7 among the block's words)
  uint8_t cols[4];       // its four salient columns (0..127); 0 for unused slots (their code is "no term")
};
static_assert(sizeof(ResidWord) == 8, "residual word entry is 8 bytes");
constexpr int kMaxResidWords = kMaxSalient / 4;    // per block

STB_HD constexpr int n_lo(int N) { return N < 4 ? N : 4; }
STB_HD constexpr int n_hi(int N) { return N > 4 ? N - 4 : 0; }
STB_HD constexpr int sign_full_words(int N) { return (n_lo(N) >> 1) + (n_hi(N) >> 1); }
STB_HD constexpr bool sign_has_half(int N) { return (N & 1) != 0; }

STB_HD constexpr uint32_t tile_bytes(int N) { return 512u + 192u * (uint32_t)N + 256u; }
// Residual stream of a row tile: bytes in all, offset of block b's record, and inside a record the a_sal2 of
// the four rows of lane group g (8 bytes: rows g, g + 8, g + 16, g + 24) and the codes of its word wq.
constexpr uint32_t kResidA2Bytes = 64u, kResidWordBytes = 32u;
STB_HD constexpr uint64_t resid_rt_bytes(int nblk, uint32_t nrw) { return (uint64_t)kResidA2Bytes * (uint32_t)nblk + (uint64_t)kResidWordBytes * nrw; }
STB_HD constexpr uint64_t resid_block_off(int b, uint32_t rw_off) { return (uint64_t)kResidA2Bytes * (uint32_t)b + (uint64_t)kResidWordBytes * rw_off; }
STB_HD constexpr uint32_t resid_a2_off(int g, int j) { return (uint32_t)(4 * g + j) * 2u; }
STB_HD constexpr uint32_t resid_code_off(uint32_t wq, int g) { return kResidA2Bytes + (wq * 8u + (uint32_t)g) * 4u; }
STB_HD constexpr uint32_t rwtab_offset(int nblk) { return (uint32_t)(sizeof(Header) + sizeof(BlockInfo) * (size_t)nblk); }
// the table is sized for the most residual words a layer can have, so that the tiles start at an offset that
// depends on the shape alone
STB_HD constexpr uint32_t tiles_offset(int nblk) {
  return (uint32_t)((rwtab_offset(nblk) + sizeof(ResidWord) * (size_t)kMaxResidWords * (size_t)nblk + 255) / 256 * 256);
}
STB_HD constexpr int resid_words_for(int nsal) { return (nsal + 3) >> 2; }
// N = 6: the mask plane is ordered for the metadata of the sparse instruction (see the layout comment)
STB_HD constexpr bool mask_pairs(int N) { return N == 6; }
// byte offset, inside the tile, of the two bytes (row g + 16 mt, then row g + 16 mt + 8) of group 4 s + tq
STB_HD constexpr uint32_t pair_field_off(int g, int mt, int s, int tq) {
  return 16u * (uint32_t)(4 * g + 2 * mt + (s >> 1)) + 8u * (uint32_t)(s & 1) + 2u * (uint32_t)tq;
}
constexpr uint32_t kMasks6 = 28;               // C(8, 6)
STB_HD constexpr uint32_t pair_field(uint32_t i0, uint32_t i1) { return 16u * (i0 + kMasks6 * i1); }
STB_HD constexpr uint32_t pair_field_index(uint32_t field, int upper_row) {
  const uint32_t J = (field >> 4) & 0xFFFu, i1 = (J * 2341u) >> 16;     // J / 28 for J < 784
  return upper_row ? i1 : J - kMasks6 * i1;
}
STB_HD constexpr uint32_t off_region(int) { return 512u; }
STB_HD constexpr uint32_t off_sign(int N) { return 512u + 128u * (uint32_t)N; }
STB_HD constexpr uint32_t off_scale(int N) { return 512u + 192u * (uint32_t)N; }

// Byte offset (inside the tile) of word `iw` of a per-lane field of `nw` words that starts at
// `base`: the words are laid out as uint4 planes, then (nw & 2) a uint2 plane, then (nw & 1)
// a u32 plane.
STB_HD constexpr uint32_t plane_word_off(uint32_t base, int nw, int iw, int lane) {
  int q4 = nw >> 2;
  if (iw < 4 * q4) return base + (uint32_t)(iw >> 2) * 512u + (uint32_t)lane * 16u + (uint32_t)(iw & 3) * 4u;
  uint32_t o = base + (uint32_t)q4 * 512u;
  if (nw & 2) {
    if (iw < 4 * q4 + 2) return o + (uint32_t)lane * 8u + (uint32_t)(iw - 4 * q4) * 4u;
    o += 256u;
  }
  return o + (uint32_t)lane * 4u;
}
STB_HD constexpr uint32_t region_word_off(int N, int iw, int lane) {
  return plane_word_off(off_region(N), N, iw, lane);
}
STB_HD constexpr uint32_t sign_word_off(int N, int sw, int lane) {
  return plane_word_off(off_sign(N), sign_full_words(N), sw, lane);
}
STB_HD constexpr uint32_t sign_half_off(int N, int lane) {
  return off_sign(N) + 128u * (uint32_t)sign_full_words(N) + (uint32_t)(lane & 15) * 4u;
}
// scales are indexed by the permuted row position p = 4 g + j of row g + 8 j
STB_HD constexpr uint32_t scale_off(int N, int g, int j) { return off_scale(N) + (uint32_t)(4 * g + j) * 8u; }

// bit position of the two-bit code number i (0..15) of a region word
STB_HD constexpr int code_bit(int i) {
  int slot = i & 3, qq = (i >> 2) & 3;
  return 4 * slot + 16 * (qq & 1) + 2 * (qq >> 1);
}
// bit position of sign bit number i (0..31) of a sign word (i < 16: also the lower-lane form
// of a shared half word)
STB_HD constexpr int sign_bit(int i) {
  int slot = i & 3, qq = (i >> 2) & 3, p = (i >> 4) & 1;
  int nib = slot + 4 * (qq & 1);
  int sel = 2 * p + (qq >> 1);
  int off = sel == 0 ? 2 : (sel == 1 ? 1 : (sel == 2 ? 3 : 0));
  return 4 * nib + off;
}
// shared half word: lower-lane form (offsets 2,1) <-> upper-lane form (offsets 3,0)
STB_HD constexpr uint32_t half_to_upper(uint32_t h) {
  return ((h & 0x44444444u) << 1) | ((h & 0x22222222u) >> 1);
}
STB_HD constexpr uint32_t half_from_upper(uint32_t s) {
  return ((s & 0x88888888u) >> 1) | ((s & 0x11111111u) << 1);
}

// Keep-mask index <-> keep mask.
struct MaskTables {
  uint8_t index[9][256];   // [N][mask] -> index (0 for a mask that does not have N bits)
  uint8_t mask[9][72];     // [N][index] -> mask
  uint8_t count[9];        // C(8, N)
};
constexpr MaskTables make_mask_tables() {
  MaskTables t{};
  for (int N = 0; N <= 8; ++N) {
    int k = 0;
    for (uint32_t m = 0; m < 256; ++m) {
      int pc = 0;
      for (int c = 0; c < 8; ++c) pc += (m >> c) & 1u;
      if (pc == N) { t.index[N][m] = (uint8_t)k; t.mask[N][k] = (uint8_t)m; ++k; }
    }
    t.count[N] = (uint8_t)k;
  }
  return t;
}
constexpr MaskTables kMaskTables = make_mask_tables();
#if defined(__CUDACC__)
__device__ const MaskTables g_mask_tables = make_mask_tables();
#endif
STB_HD uint32_t mask_index(int N, uint32_t mask) {
#if defined(__CUDA_ARCH__)
  return g_mask_tables.index[N][mask & 0xFFu];
#else
  return kMaskTables.index[N][mask & 0xFFu];
#endif
}
STB_HD uint32_t mask_from_index(int N, uint32_t idx) {
#if defined(__CUDA_ARCH__)
  return g_mask_tables.mask[N][idx < 72u ? idx : 0u];
#else
  return kMaskTables.mask[N][idx < 72u ? idx : 0u];
#endif
}

// Where the code / sign of the k-th kept weight (ascending column) of slot u lives.
struct BitPos { int word; int bit; bool half; };
STB_HD constexpr BitPos region_pos(int N, int u, int k) {
  const int NL = n_lo(N), NH = n_hi(N);
  const int w = k < 4 ? u * NL + k : u * NH + (k - 4);
  return BitPos{(k < 4 ? 0 : NL) + (w >> 4), code_bit(w & 15), false};
}
STB_HD constexpr BitPos sign_pos(int N, int u, int k) {
  const int NL = n_lo(N), NH = n_hi(N);
  const bool lo = k < 4;
  const int w = lo ? u * NL + k : u * NH + (k - 4);
  const int nfull = lo ? (NL >> 1) : (NH >> 1);
  const int base = lo ? 0 : (NL >> 1);
  if ((w >> 5) < nfull) return BitPos{base + (w >> 5), sign_bit(w & 31), false};
  return BitPos{0, sign_bit(w & 15), true};
}

}  // namespace stb

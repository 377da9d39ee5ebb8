// Packed ("streaming") layout of an N:8 structured-binary layer, shared by the CUDA kernels.
//
// The unit of the layout is a TILE: 32 output rows x one 128-column block.  Inside a tile
// every field is stored lane-major (lane = row within the tile) so that a warp reads each
// field with one fully coalesced vector load per plane:
//
//   mask    32 x uint4                      16 keep bytes of the row-block (group g = byte g)
//   region  N words per lane                16 two-bit codes per word, quad-interleaved (below)
//   sign    N/2 words per lane (+ a half)   32 sign bits per word, pre-positioned (below)
//   scale   32 x uint2 + 32 x u16           byte-planar: word A = low bytes of the fp16 scales
//                                           a_dense,a_inter,a_sparse,a_sal1; word B = their
//                                           high bytes; then a_sal2 as u16
//   resid   rb byte planes of 32 bytes      residual sign bits of the block's salient columns,
//                                           rb = ceil(S_b / 8), S_b = salient columns of block
//
// Tile bytes = 512 + 128 N + 64 N + 320 + 32 rb  (50 / 56 / 62 bytes per row-block at
// N = 4 / 5 / 6, plus rb).  Tiles of one row tile are contiguous in block order; row tiles
// follow each other with stride rt_stride.  A header and a per-block table come first.
//
// Kept weights of a row-block are numbered w = g*N + k (g = group 0..15, k = rank of the
// weight among the kept columns of the group, ascending).  Quad q = w/4, slot j = w%4.
//   region word w/16: with qq = (w/4)%4 the code sits at bit 4j + 16(qq&1) + 2(qq>>1).
//     => (R & 0x33333333) holds quads qq=0 (low 16 bits) and qq=1 (high 16 bits) as nibbles,
//        ((R>>2) & 0x33333333) holds quads qq=2 and qq=3: each nibble is a byte-permute
//        selector 0..3 into the four scale bytes.
//   sign word w/32, stored bit = 1 for a NEGATIVE weight: with p = (w/16)%2 the bit sits at
//     4i + off, i = j + 4(qq&1), off = {2,1,3,0}[2p + (qq>>1)], so that one shift moves the
//     eight sign bits of a selector word onto bit 2 of its nibbles (the bit that chooses
//     between the +scale and -scale high bytes).
//   For odd N the last 16 weights need half a sign word: lanes l and l+16 share word l of a
//   16-word plane; lane l < 16 uses offsets {2,1}, lane l+16 the same bits moved to {3,0}.
#pragma once
#include <stdint.h>

namespace stb {

constexpr uint32_t kMagic = 0x31425453u;  // "STB1"
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
  uint32_t tiles_offset; // byte offset of tile (0,0)
  uint64_t rt_stride;    // bytes of one row tile (all its blocks)
  uint64_t used_bytes;
  uint32_t status;       // 0 or STB_ERR_CORRUPT
  uint32_t max_tile_bytes;
  uint32_t pad[2];
};
static_assert(sizeof(Header) == 64, "header is 64 bytes");

struct BlockInfo {       // 32 bytes, one per block, right after the header
  uint64_t salient[2];
  uint32_t tile_off;     // byte offset of the block's tile inside a row tile
  uint32_t nsal;         // S_b
  uint32_t res_bytes;    // rb
  uint32_t tile_bytes;
};
static_assert(sizeof(BlockInfo) == 32, "block info is 32 bytes");

__host__ __device__ constexpr uint32_t tile_bytes(int N, int rb) {
  return 512u + 192u * (uint32_t)N + 320u + 32u * (uint32_t)rb;
}
__host__ __device__ constexpr uint32_t tiles_offset(int nblk) {
  return (uint32_t)((sizeof(Header) + sizeof(BlockInfo) * (size_t)nblk + 255) / 256 * 256);
}
__host__ __device__ constexpr uint32_t off_region(int) { return 512u; }
__host__ __device__ constexpr uint32_t off_sign(int N) { return 512u + 128u * (uint32_t)N; }
__host__ __device__ constexpr uint32_t off_scale(int N) { return 512u + 192u * (uint32_t)N; }
__host__ __device__ constexpr uint32_t off_sal2(int N) { return off_scale(N) + 256u; }
__host__ __device__ constexpr uint32_t off_resid(int N) { return off_scale(N) + 320u; }

// Byte offset (inside the tile) of word `iw` of a per-lane field of `nw` words that starts at
// `base`: the words are laid out as uint4 planes, then (nw & 2) a uint2 plane, then (nw & 1)
// a u32 plane.
__host__ __device__ constexpr uint32_t plane_word_off(uint32_t base, int nw, int iw, int lane) {
  int q4 = nw >> 2;
  if (iw < 4 * q4) return base + (uint32_t)(iw >> 2) * 512u + (uint32_t)lane * 16u + (uint32_t)(iw & 3) * 4u;
  uint32_t o = base + (uint32_t)q4 * 512u;
  if (nw & 2) {
    if (iw < 4 * q4 + 2) return o + (uint32_t)lane * 8u + (uint32_t)(iw - 4 * q4) * 4u;
    o += 256u;
  }
  return o + (uint32_t)lane * 4u;
}
__host__ __device__ constexpr uint32_t region_word_off(int N, int iw, int lane) {
  return plane_word_off(off_region(N), N, iw, lane);
}
// full sign words: N/2 per lane; the shared half word (odd N) follows them
__host__ __device__ constexpr uint32_t sign_word_off(int N, int sw, int lane) {
  return plane_word_off(off_sign(N), N >> 1, sw, lane);
}
__host__ __device__ constexpr uint32_t sign_half_off(int N, int lane) {
  return off_sign(N) + 128u * (uint32_t)(N >> 1) + (uint32_t)(lane & 15) * 4u;
}

// bit position of the 2-bit region code of kept weight w inside region word w/16
__host__ __device__ constexpr int code_bit(int w) {
  int j = w & 3, qq = (w >> 2) & 3;
  return 4 * j + 16 * (qq & 1) + 2 * (qq >> 1);
}
// bit position of the sign bit of kept weight w inside sign word w/32 (lower-lane form for
// the shared half word)
__host__ __device__ constexpr int sign_bit(int w) {
  int j = w & 3, qq = (w >> 2) & 3, p = (w >> 4) & 1;
  int i = j + 4 * (qq & 1);
  int sel = 2 * p + (qq >> 1);
  int off = sel == 0 ? 2 : (sel == 1 ? 1 : (sel == 2 ? 3 : 0));
  return 4 * i + off;
}
// shared half word: lower-lane form (offsets 2,1) <-> upper-lane form (offsets 3,0)
__host__ __device__ constexpr uint32_t half_to_upper(uint32_t h) {
  return ((h & 0x44444444u) << 1) | ((h & 0x22222222u) >> 1);
}
__host__ __device__ constexpr uint32_t half_from_upper(uint32_t s) {
  return ((s & 0x88888888u) >> 1) | ((s & 0x11111111u) << 1);
}

}  // namespace stb

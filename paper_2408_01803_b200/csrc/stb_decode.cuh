// Plain (position-order) decode of one row-block from the packed layout.  Used by
// stb_dequant and by the general GEMV kernel (any N, any batch); the fast batch-1 GEMV has
// its own rank-order decode.
#pragma once
#include <cuda_fp16.h>
#include <stdint.h>

#include "stb_layout.cuh"

namespace stb {

template <int N>
struct RowBlock {
  uint32_t mask[4];
  uint32_t R[N];
  uint32_t S[(N + 1) / 2];   // odd N: last entry is the half word in lower-lane form
  float alpha[5];
  uint32_t resid;            // residual sign bits of the block's salient columns (1 = +1)
};

template <int N>
__device__ __forceinline__ void load_rowblock(const uint8_t* __restrict__ tile, int lane, int rb,
                                              RowBlock<N>& r) {
  const uint4 mk = *reinterpret_cast<const uint4*>(tile + lane * 16);
  r.mask[0] = mk.x; r.mask[1] = mk.y; r.mask[2] = mk.z; r.mask[3] = mk.w;
#pragma unroll
  for (int i = 0; i < N; ++i)
    r.R[i] = *reinterpret_cast<const uint32_t*>(tile + region_word_off(N, i, lane));
#pragma unroll
  for (int i = 0; i < N / 2; ++i)
    r.S[i] = *reinterpret_cast<const uint32_t*>(tile + sign_word_off(N, i, lane));
  if (N & 1) {
    uint32_t h = *reinterpret_cast<const uint32_t*>(tile + sign_half_off(N, lane));
    r.S[N / 2] = lane < 16 ? (h & 0x66666666u) : half_from_upper(h);
  }
  const uint2 ab = *reinterpret_cast<const uint2*>(tile + off_scale(N) + lane * 8);
#pragma unroll
  for (int q = 0; q < 4; ++q) {
    const uint16_t hb = (uint16_t)(((ab.x >> (8 * q)) & 0xFFu) | (((ab.y >> (8 * q)) & 0xFFu) << 8));
    r.alpha[q] = __half2float(__ushort_as_half(hb));
  }
  r.alpha[4] = __half2float(__ushort_as_half(
      *reinterpret_cast<const uint16_t*>(tile + off_sal2(N) + lane * 2)));
  r.resid = 0;
  for (int p = 0; p < rb; ++p) r.resid |= (uint32_t)tile[off_resid(N) + p * 32 + lane] << (8 * p);
}

// Decode group g (8 columns) of the row-block into fp32, position order.
// salb: the block's salient bits of this group; tbase: number of salient columns of the block
// before this group.
template <int N>
__device__ __forceinline__ void decode_group(const RowBlock<N>& r, int g, uint32_t salb, int tbase,
                                             float out[8]) {
  const uint32_t kb = (r.mask[g >> 2] >> (8 * (g & 3))) & 0xFFu;
  // the group's weights w = g*N .. g*N+N-1 touch at most two region words and two sign
  // words; pick between them with compile-time indices (g is an unrolled loop counter)
  const int iw0 = (g * N) >> 4, iw1 = (iw0 + 1 < N) ? iw0 + 1 : N - 1;
  constexpr int NS = (N + 1) / 2;
  const int sw0 = (g * N) >> 5, sw1 = (sw0 + 1 < NS) ? sw0 + 1 : NS - 1;
#pragma unroll
  for (int c = 0; c < 8; ++c) {
    float v = 0.0f;
    if ((kb >> c) & 1u) {
      const int w = g * N + __popc(kb & ((1u << c) - 1u));
      const uint32_t rw = ((w >> 4) == iw0) ? r.R[iw0] : r.R[iw1];
      const uint32_t sw = ((w >> 5) == sw0) ? r.S[sw0] : r.S[sw1];
      const uint32_t code = (rw >> code_bit(w)) & 3u;
      const uint32_t neg = (sw >> sign_bit(w)) & 1u;
      const float s1 = neg ? -1.0f : 1.0f;
      if (code == 3u) {
        const int t = tbase + __popc(salb & ((1u << c) - 1u));
        const float s2 = ((r.resid >> t) & 1u) ? 1.0f : -1.0f;
        v = __fadd_rn(s1 * r.alpha[3], s2 * r.alpha[4]);
      } else {
        v = s1 * (code == 0u ? r.alpha[0] : (code == 1u ? r.alpha[1] : r.alpha[2]));
      }
    }
    out[c] = v;
  }
}

__device__ __forceinline__ bool header_matches(const Header* h, int n, int m, int N) {
  return h->magic == kMagic && h->n == n && h->m == m && h->N == N && h->status == 0u;
}

}  // namespace stb

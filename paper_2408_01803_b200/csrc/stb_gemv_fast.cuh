// Batch-1 decode GEMV for N = 4, 5, 6: rank-order decode with byte permutes.
//
// Per row-block (one lane = one output row, 128 columns, 16 N kept weights) nothing is expanded
// to the 128 column positions.  Instead
//   * x side: the activations of a group of 8 columns sit in shared memory byte-planar (low
//     bytes of the 8 halfs, then high bytes).  A 256-entry table maps the group's keep byte to
//     the byte-permute selector that pulls the kept columns' bytes out in rank order, 4 per
//     PRMT; one more PRMT per pair re-interleaves low / high bytes into a half2.
//   * scale side: the 2-bit region codes are stored so that (R & 0x33333333) and
//     ((R >> 2) & 0x33333333) are already PRMT selectors into the four scale bytes; the sign
//     bit is OR-ed into bit 2 of each nibble and so picks the high byte of +scale or -scale.
//     Two PRMTs give the low / high bytes of four signed scales, two more interleave them.
//   * multiply-accumulate: fma.rn.f32.f16 (fp16 x fp16 product, exact, added into fp32).
//   * the residual term of salient columns (a few columns per block) is added per block from
//     the block's salient list.
#pragma once
#include <cuda_fp16.h>
#include <stdint.h>

#include "stb_layout.cuh"

namespace stb {
namespace fast {

__device__ __forceinline__ uint32_t prmt(uint32_t a, uint32_t b, uint32_t s) {
  uint32_t d;
  asm("prmt.b32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(s));
  return d;
}
// acc += w.lo * x.lo + w.hi * x.hi, fp16 operands, fp32 accumulate (two dependent FMAs)
__device__ __forceinline__ float fma_pair(float acc, uint32_t w, uint32_t x) {
  asm("{\n\t.reg .b16 wl, wh, xl, xh;\n\t"
      "mov.b32 {wl, wh}, %1;\n\t"
      "mov.b32 {xl, xh}, %2;\n\t"
      "fma.rn.f32.f16 %0, wl, xl, %0;\n\t"
      "fma.rn.f32.f16 %0, wh, xh, %0;\n\t}"
      : "+f"(acc) : "r"(w), "r"(x));
  return acc;
}
__device__ __forceinline__ float fma_lo(float acc, uint32_t w, uint32_t x) {
  asm("{\n\t.reg .b16 wl, wh, xl, xh;\n\t"
      "mov.b32 {wl, wh}, %1;\n\t"
      "mov.b32 {xl, xh}, %2;\n\t"
      "fma.rn.f32.f16 %0, wl, xl, %0;\n\t}"
      : "+f"(acc) : "r"(w), "r"(x));
  return acc;
}

// keep byte -> selector tables (built in shared memory by the kernel)
//   U[mask]  : nibble r = column (0..7) of the r-th kept column
//   TA5/TB5  : the two forms used for odd N = 5 (see rowblock_dot<5>)
__device__ __forceinline__ void build_tables(uint32_t* tab, int N, int tid, int nthreads) {
  for (int mk = tid; mk < 256; mk += nthreads) {
    uint32_t u = 0;
    int r = 0;
    for (int c = 0; c < 8; ++c)
      if ((mk >> c) & 1) { u |= (uint32_t)c << (4 * r); ++r; }
    if (N == 5) {
      tab[mk] = (u & 0xFFFFu) | (((u >> 16) & 3u) << 16);                     // TA5
      tab[256 + mk] = ((u >> 4) & 0xFFFFu) | ((4u | (u & 3u)) << 16);         // TB5
    } else {
      tab[mk] = u;
    }
  }
}

template <int NW>
__device__ __forceinline__ void load_planes(const uint8_t* __restrict__ tile, uint32_t base, uint32_t* w,
                                            int lane) {
  constexpr int Q4 = NW / 4;
#pragma unroll
  for (int q = 0; q < Q4; ++q) {
    const uint4 v = __ldcs(reinterpret_cast<const uint4*>(tile + base + q * 512 + lane * 16));
    w[4 * q] = v.x; w[4 * q + 1] = v.y; w[4 * q + 2] = v.z; w[4 * q + 3] = v.w;
  }
  uint32_t o = base + Q4 * 512;
  if (NW & 2) {
    const uint2 v = __ldcs(reinterpret_cast<const uint2*>(tile + o + lane * 8));
    w[4 * Q4] = v.x; w[4 * Q4 + 1] = v.y;
    o += 256;
  }
  if (NW & 1) w[NW - 1] = __ldcs(reinterpret_cast<const uint32_t*>(tile + o + lane * 4));
}

template <int N>
struct Tile {
  uint32_t mask[4];
  uint32_t R[N];
  uint32_t S[(N + 1) / 2];
  uint32_t A, B;       // low / high bytes of the four main scales
  uint32_t sal2;       // fp16 bits of a_sal2
  uint32_t resid;
};

template <int N>
__device__ __forceinline__ void load_tile(const uint8_t* __restrict__ tile, int lane, int rb, Tile<N>& t) {
  const uint4 mk = __ldcs(reinterpret_cast<const uint4*>(tile + lane * 16));
  t.mask[0] = mk.x; t.mask[1] = mk.y; t.mask[2] = mk.z; t.mask[3] = mk.w;
  load_planes<N>(tile, off_region(N), t.R, lane);
  load_planes<N / 2>(tile, off_sign(N), t.S, lane);
  if (N & 1) t.S[N / 2] = __ldcs(reinterpret_cast<const uint32_t*>(tile + sign_half_off(N, lane)));
  const uint2 ab = __ldcs(reinterpret_cast<const uint2*>(tile + off_scale(N) + lane * 8));
  t.A = ab.x; t.B = ab.y;
  t.sal2 = __ldcs(reinterpret_cast<const uint16_t*>(tile + off_sal2(N) + lane * 2));
  t.resid = 0;
  for (int p = 0; p < rb; ++p) t.resid |= (uint32_t)__ldcs(tile + off_resid(N) + p * 32 + lane) << (8 * p);
}

// Signed scales of quad q (4 kept weights) as two half2 pairs.
template <int N>
struct ScaleSide {
  uint32_t e[N], o[N];     // selector words with the sign bit merged in
  uint32_t A, Bp, Bn;
  __device__ __forceinline__ void init(const Tile<N>& t, int lane) {
    A = t.A; Bp = t.B; Bn = t.B ^ 0x80808080u;
#pragma unroll
    for (int i = 0; i < N; ++i) {
      uint32_t s = t.S[i >> 1];
      if ((N & 1) && i == N - 1) s = lane < 16 ? s : half_from_upper(s);
      const uint32_t se = (i & 1) ? (s >> 1) : s;
      const uint32_t so = (i & 1) ? (s << 2) : (s << 1);
      e[i] = (t.R[i] & 0x33333333u) | (se & 0x44444444u);
      o[i] = ((t.R[i] >> 2) & 0x33333333u) | (so & 0x44444444u);
    }
  }
  __device__ __forceinline__ void quad(int q, uint32_t& w01, uint32_t& w23) const {
    const int i = q >> 2, qq = q & 3;
    uint32_t sel = (qq < 2) ? e[i] : o[i];
    if (qq & 1) sel >>= 16;
    const uint32_t L = prmt(A, A, sel), H = prmt(Bp, Bn, sel);
    w01 = prmt(L, H, 0x5140u);
    w23 = prmt(L, H, 0x7362u);
  }
};

__device__ __forceinline__ uint32_t mask_byte(const uint32_t (&mask)[4], int g) {
  return prmt(mask[g >> 2], 0u, 0x4440u + (uint32_t)(g & 3));
}

// Dot product of one row-block with the staged activations of its block.
//   xs  : 16 uint4 (one per group): {low bytes cols 0-3, low bytes cols 4-7, high 0-3, high 4-7}
//   tab : selector tables in shared memory
template <int N>
__device__ __forceinline__ float rowblock_dot(const Tile<N>& t, const uint4* __restrict__ xs,
                                              const uint32_t* __restrict__ tab, int lane) {
  static_assert(N == 4 || N == 5 || N == 6, "fast path covers N = 4, 5, 6");
  ScaleSide<N> sc;
  sc.init(t, lane);
  float acc0 = 0.f, acc1 = 0.f, acc2 = 0.f, acc3 = 0.f;
  if (N == 4) {
#pragma unroll
    for (int g = 0; g < 16; ++g) {
      const uint32_t sel = tab[mask_byte(t.mask, g)];
      const uint4 xg = xs[g];
      const uint32_t GL = prmt(xg.x, xg.y, sel), GH = prmt(xg.z, xg.w, sel);
      uint32_t w01, w23;
      sc.quad(g, w01, w23);
      acc0 = fma_pair(acc0, w01, prmt(GL, GH, 0x5140u));
      acc1 = fma_pair(acc1, w23, prmt(GL, GH, 0x7362u));
    }
  } else if (N == 6) {
#pragma unroll
    for (int c = 0; c < 8; ++c) {       // two groups = 12 weights = 3 quads = 6 pairs
      uint32_t X[6];
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        const int g = 2 * c + h;
        const uint32_t sel = tab[mask_byte(t.mask, g)];
        const uint4 xg = xs[g];
        const uint32_t GLa = prmt(xg.x, xg.y, sel), GHa = prmt(xg.z, xg.w, sel);
        const uint32_t GLb = prmt(xg.x, xg.y, sel >> 16), GHb = prmt(xg.z, xg.w, sel >> 16);
        X[3 * h + 0] = prmt(GLa, GHa, 0x5140u);
        X[3 * h + 1] = prmt(GLa, GHa, 0x7362u);
        X[3 * h + 2] = prmt(GLb, GHb, 0x5140u);
      }
#pragma unroll
      for (int k = 0; k < 3; ++k) {
        uint32_t w01, w23;
        sc.quad(3 * c + k, w01, w23);
        acc0 = fma_pair(acc0, w01, X[2 * k]);
        acc1 = fma_pair(acc1, w23, X[2 * k + 1]);
      }
    }
  } else {  // N == 5
#pragma unroll
    for (int c = 0; c < 4; ++c) {       // four groups = 20 weights = 5 quads = 10 pairs
      uint32_t X[10];
#pragma unroll
      for (int h = 0; h < 2; ++h) {     // group pair (A, B): pairs A01 A23 A4B0 B12 B34
        const int gA = 4 * c + 2 * h, gB = gA + 1;
        const uint32_t tA = tab[mask_byte(t.mask, gA)], tB = tab[256 + mask_byte(t.mask, gB)];
        const uint32_t cross = prmt(tA, tB, 0x6262u);
        const uint4 xa = xs[gA], xb = xs[gB];
        const uint32_t Q1L = prmt(xa.x, xa.y, tA), Q1H = prmt(xa.z, xa.w, tA);
        const uint32_t Q2L = prmt(xa.y, xb.x, cross), Q2H = prmt(xa.w, xb.z, cross);
        const uint32_t Q3L = prmt(xb.x, xb.y, tB), Q3H = prmt(xb.z, xb.w, tB);
        X[5 * h + 0] = prmt(Q1L, Q1H, 0x5140u);
        X[5 * h + 1] = prmt(Q1L, Q1H, 0x7362u);
        X[5 * h + 2] = prmt(Q2L, Q2H, 0x6240u);
        X[5 * h + 3] = prmt(Q3L, Q3H, 0x5140u);
        X[5 * h + 4] = prmt(Q3L, Q3H, 0x7362u);
      }
#pragma unroll
      for (int k = 0; k < 5; ++k) {
        uint32_t w01, w23;
        sc.quad(5 * c + k, w01, w23);
        acc0 = fma_pair(acc0, w01, X[2 * k]);
        acc1 = fma_pair(acc1, w23, X[2 * k + 1]);
      }
    }
  }
  (void)acc2; (void)acc3;
  return acc0 + acc1;
}

}  // namespace fast
}  // namespace stb

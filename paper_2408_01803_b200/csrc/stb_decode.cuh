// Decode of the packed layout (stb_layout.cuh), shared by the CUDA kernels.  Everything here
// works on 32-bit words and is host + device code: compiled for the host (byte permute
// emulated) the bit layouts are checked against the plain definition without a GPU.
//
//   LaneTile / load_lane_tile   the registers one lane holds of one tile
//   build_lane_words            logical fields of the lane's 16 slots -> packed words (pack)
//   plain_slot                  position-order decode of one slot, bit by bit (dequant, general
//                               GEMV): the plain definition, any N
//   FastRows                    N = 4, 5, 6: byte-permute decode of one slot into 8 half
//                               precision weights (4 registers), the form the tensor-core paths
//                               consume.  Works on whatever 16-bit scale bytes it is given
//                               (fp16 for the GEMV, bf16 for the GEMM).
#pragma once
#include <stdint.h>

#include "stb_layout.cuh"

namespace stb {

STB_HD uint32_t prmt(uint32_t a, uint32_t b, uint32_t s) {
#if defined(__CUDA_ARCH__)
  uint32_t d;
  asm("prmt.b32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(s));
  return d;
#else
  const uint64_t src = ((uint64_t)b << 32) | a;
  uint32_t d = 0;
  for (int i = 0; i < 4; ++i) {
    const uint32_t nib = (s >> (4 * i)) & 0xFu;
    uint32_t byte = (uint32_t)(src >> (8 * (nib & 7u))) & 0xFFu;
    if (nib & 8u) byte = (byte & 0x80u) ? 0xFFu : 0x00u;
    d |= byte << (8 * i);
  }
  return d;
#endif
}

// ------------------------------------------------------------------------------------------
template <int N>
struct LaneTile {
  static constexpr int kFull = sign_full_words(N);
  uint32_t mask[4];                     // word j = row g + 8 j: byte s = keep-mask index of group 4 s + t
  uint32_t R[N];                        // region words (low part, then high part)
  uint32_t S[kFull > 0 ? kFull : 1];    // full sign words (low part, then high part)
  uint32_t half;                        // shared half sign word, already in lower-lane form
  uint32_t A[4], B[4];                  // per row j: low / high bytes of the four main scales
};

template <int NW>
STB_HD void load_planes(const uint8_t* tile, uint32_t base, uint32_t* w, int lane) {
  constexpr int Q4 = NW / 4;
#pragma unroll
  for (int q = 0; q < Q4; ++q) {
    const uint4 v = *reinterpret_cast<const uint4*>(tile + base + q * 512 + lane * 16);
    w[4 * q] = v.x; w[4 * q + 1] = v.y; w[4 * q + 2] = v.z; w[4 * q + 3] = v.w;
  }
  uint32_t o = base + Q4 * 512;
  if (NW & 2) {
    const uint2 v = *reinterpret_cast<const uint2*>(tile + o + lane * 8);
    w[4 * Q4] = v.x; w[4 * Q4 + 1] = v.y;
    o += 256;
  }
  if (NW & 1) w[NW - 1] = *reinterpret_cast<const uint32_t*>(tile + o + lane * 4);
}

// `tile` may point to global or to shared memory (16-byte aligned).  With pair fields in the
// mask plane (N = 6) the lane's keep-mask indices are gathered from the quad's fields unless
// `raw_mask` asks for the lane's 16 bytes as they are.
template <int N>
STB_HD void load_lane_tile(const uint8_t* tile, int lane, LaneTile<N>& t, bool raw_mask = false) {
  const int g = lane >> 2;
  if (mask_pairs(N) && !raw_mask) {
    const int tq = lane & 3;
    t.mask[0] = t.mask[1] = t.mask[2] = t.mask[3] = 0;
#pragma unroll
    for (int mt = 0; mt < 2; ++mt)
#pragma unroll
      for (int sidx = 0; sidx < 4; ++sidx) {
        const uint32_t f = *reinterpret_cast<const uint16_t*>(tile + pair_field_off(g, mt, sidx, tq));
        t.mask[2 * mt] |= pair_field_index(f, 0) << (8 * sidx);
        t.mask[2 * mt + 1] |= pair_field_index(f, 1) << (8 * sidx);
      }
  } else {
    const uint4 mk = *reinterpret_cast<const uint4*>(tile + lane * 16);
    t.mask[0] = mk.x; t.mask[1] = mk.y; t.mask[2] = mk.z; t.mask[3] = mk.w;
  }
  load_planes<N>(tile, off_region(N), t.R, lane);
  load_planes<LaneTile<N>::kFull>(tile, off_sign(N), t.S, lane);
  t.half = 0;
  if (sign_has_half(N)) {
    const uint32_t h = *reinterpret_cast<const uint32_t*>(tile + sign_half_off(N, lane));
    t.half = lane < 16 ? (h & 0x66666666u) : half_from_upper(h & 0x99999999u);
  }
  const uint4 s0 = *reinterpret_cast<const uint4*>(tile + scale_off(N, g, 0));
  const uint4 s1 = *reinterpret_cast<const uint4*>(tile + scale_off(N, g, 2));
  t.A[0] = s0.x; t.B[0] = s0.y; t.A[1] = s0.z; t.B[1] = s0.w;
  t.A[2] = s1.x; t.B[2] = s1.y; t.A[3] = s1.z; t.B[3] = s1.w;
}

// fp16 bit pattern of main scale q (0..3) of row j
template <int N>
STB_HD uint32_t scale_bits(const LaneTile<N>& t, int j, int q) {
  return ((t.A[j] >> (8 * q)) & 0xFFu) | (((t.B[j] >> (8 * q)) & 0xFFu) << 8);
}
// fp16 bit pattern of a_sal2 of row g + 8 j; `record` = the block's record in the row tile's residual stream
STB_HD uint32_t sal2_bits(const uint8_t* record, int g, int j) {
  return *reinterpret_cast<const uint16_t*>(record + resid_a2_off(g, j));
}
// residual word wq (0..7) of the block, as stored for lane group g
STB_HD uint32_t resid_word(const uint8_t* record, uint32_t wq, int g) {
  return *reinterpret_cast<const uint32_t*>(record + resid_code_off(wq, g));
}

// ------------------------------------------------------------------------------------------
// Pack side: the lane's words from the logical fields of its 16 slots.
//   keep[u], sign[u] (bit k = 1: k-th kept weight is +1), region[u] (2 bits per kept weight)
template <int N>
struct LaneWords {
  uint32_t R[N];
  uint32_t S[LaneTile<N>::kFull > 0 ? LaneTile<N>::kFull : 1];
  uint32_t half;      // lower-lane form
};

template <int N>
STB_HD void build_lane_words(const uint32_t (&sign)[16], const uint32_t (&region)[16], bool valid,
                             LaneWords<N>& w) {
#pragma unroll
  for (int i = 0; i < N; ++i) w.R[i] = 0;
#pragma unroll
  for (int i = 0; i < (LaneTile<N>::kFull > 0 ? LaneTile<N>::kFull : 1); ++i) w.S[i] = 0;
  w.half = 0;
#pragma unroll
  for (int u = 0; u < 16; ++u) {
#pragma unroll
    for (int k = 0; k < N; ++k) {
      const uint32_t code = valid ? (region[u] >> (2 * k)) & 3u : 0u;
      const uint32_t neg = valid ? ((sign[u] >> k) & 1u) ^ 1u : 0u;
      const BitPos rp = region_pos(N, u, k), sp = sign_pos(N, u, k);
      w.R[rp.word] |= code << rp.bit;
      if (sp.half) w.half |= neg << sp.bit;
      else w.S[sp.word] |= neg << sp.bit;
    }
  }
}

// ------------------------------------------------------------------------------------------
// Plain decode of slot u = 4 j + s into (code, negative) per column, then to values by the
// caller.  out_code[c] = 0..3 region code, 4 = dropped; out_neg[c] = 1 for a negative weight.
template <int N>
STB_HD void plain_slot(const LaneTile<N>& t, int u, uint32_t (&out_code)[8], uint32_t (&out_neg)[8]) {
  const int j = u >> 2, s = u & 3;
  const uint32_t kb = mask_from_index(N, (t.mask[j] >> (8 * s)) & 0xFFu);
  int k = 0;
  for (int c = 0; c < 8; ++c) {
    out_code[c] = 4u; out_neg[c] = 0u;
    if (!((kb >> c) & 1u) || k >= N) continue;
    const BitPos rp = region_pos(N, u, k), sp = sign_pos(N, u, k);
    uint32_t rw = 0, sw = 0;
    for (int i = 0; i < N; ++i) rw = (i == rp.word) ? t.R[i] : rw;
    if (sp.half) sw = t.half;
    else
      for (int i = 0; i < LaneTile<N>::kFull; ++i) sw = (i == sp.word) ? t.S[i] : sw;
    out_code[c] = (rw >> rp.bit) & 3u;
    out_neg[c] = (sw >> sp.bit) & 1u;
    ++k;
  }
}

// ------------------------------------------------------------------------------------------
// Fast decode, N = 4, 5, 6.
//
// Scale side: the codes are stored so that masking a region word gives byte-permute selectors
// (one nibble per kept weight) into the four scale bytes of the row; the sign bit is OR-ed into
// bit 2 of the nibble and picks the byte of +scale or -scale.  One permute per byte plane gives
// the low / high bytes of four kept weights in rank order: ranks 0..3 of a slot from the low
// part, ranks 4.. from the high part (N = 6: ranks 4,5 of two slots per permute; N = 5: rank 4
// of the four slots of a row).
// Position side: a 256-entry table maps the keep byte to a selector (one nibble per column:
// the rank of the column among the kept ones, or 7 = a zero byte) that spreads the rank-ordered
// bytes to the 8 column positions; two more permutes per pair of registers re-interleave low
// and high bytes into 16-bit values.
template <int N>
struct FastRows {
  static_assert(N >= 4 && N <= 6, "fast decode covers N = 4, 5, 6");
  uint32_t A[4], Bp[4], Bn[4];
  uint32_t e[4], o[4];
  uint32_t eh[2], oh[2];

  // A_, B_: low / high bytes of the four main scales per row, in the 16-bit format wanted
  STB_HD void init(const LaneTile<N>& t, const uint32_t (&A_)[4], const uint32_t (&B_)[4]) {
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      A[j] = A_[j]; Bp[j] = B_[j]; Bn[j] = B_[j] ^ 0x80808080u;
      const uint32_t sw = t.S[j >> 1];
      const uint32_t se = (j & 1) ? (sw >> 1) : sw;
      const uint32_t so = (j & 1) ? (sw << 2) : (sw << 1);
      e[j] = (t.R[j] & 0x33333333u) | (se & 0x44444444u);
      o[j] = ((t.R[j] >> 2) & 0x33333333u) | (so & 0x44444444u);
    }
    eh[0] = eh[1] = oh[0] = oh[1] = 0;
    if (N == 6) {
      const uint32_t sw = t.S[2];
      eh[0] = (t.R[4] & 0x33333333u) | (sw & 0x44444444u);
      oh[0] = ((t.R[4] >> 2) & 0x33333333u) | ((sw << 1) & 0x44444444u);
      eh[1] = (t.R[5] & 0x33333333u) | ((sw >> 1) & 0x44444444u);
      oh[1] = ((t.R[5] >> 2) & 0x33333333u) | ((sw << 2) & 0x44444444u);
    } else if (N == 5) {
      eh[0] = (t.R[4] & 0x33333333u) | (t.half & 0x44444444u);
      oh[0] = ((t.R[4] >> 2) & 0x33333333u) | ((t.half << 1) & 0x44444444u);
    }
  }

  // rank-ordered bytes of ranks 4.. : N = 6 one call per (row j, step pair sp), N = 5 one call
  // per row j (sp ignored)
  STB_HD void high(int j, int sp, uint32_t& XL, uint32_t& XH) const {
    uint32_t sel;
    if (N == 6) sel = ((j & 1) ? oh[j >> 1] : eh[j >> 1]) >> (16 * sp);
    else sel = ((j & 2) ? oh[0] : eh[0]) >> (16 * (j & 1));
    XL = prmt(A[j], A[j], sel);
    XH = prmt(Bp[j], Bn[j], sel);
  }

  // Slot (j, s) -> f[0..3]: columns (0,1), (2,3), (4,5), (6,7) as 16-bit pairs (low half =
  // lower column).  P = position selector of the slot's keep byte.
  STB_HD void slot(int j, int s, uint32_t P, uint32_t XL, uint32_t XH, uint32_t (&f)[4]) const {
    slot2(j, s, P, P >> 16, XL, XH, f);
  }
  // same, with the selectors of columns 0..3 (P0) and 4..7 (P1) in separate words
  STB_HD void slot2(int j, int s, uint32_t P0, uint32_t P1, uint32_t XL, uint32_t XH, uint32_t (&f)[4]) const {
    const uint32_t sel = ((s & 2) ? o[j] : e[j]) >> (16 * (s & 1));
    const uint32_t lo0 = prmt(A[j], A[j], sel), hi0 = prmt(Bp[j], Bn[j], sel);
    uint32_t lo1 = 0, hi1 = 0;
    if (N == 6) {
      lo1 = (s & 1) ? (XL >> 16) : (XL & 0xFFFFu);
      hi1 = (s & 1) ? (XH >> 16) : (XH & 0xFFFFu);
    } else if (N == 5) {
      lo1 = prmt(XL, 0u, 0x4440u + (uint32_t)s);
      hi1 = prmt(XH, 0u, 0x4440u + (uint32_t)s);
    }
    const uint32_t pl0 = prmt(lo0, lo1, P0), pl1 = prmt(lo0, lo1, P1);
    const uint32_t ph0 = prmt(hi0, hi1, P0), ph1 = prmt(hi0, hi1, P1);
    f[0] = prmt(pl0, ph0, 0x5140u);
    f[1] = prmt(pl0, ph0, 0x7362u);
    f[2] = prmt(pl1, ph1, 0x5140u);
    f[3] = prmt(pl1, ph1, 0x7362u);
  }
  // N = 6, rank order: slot (j, s) -> r[i] = the 16-bit values of ranks 2 i, 2 i + 1 (low half =
  // lower rank); XL / XH from high(j, s >> 1).  Nothing is moved to column positions: the sparse
  // tensor-core instruction does that with the metadata of meta6_nibble.
  STB_HD void pairs(int j, int s, uint32_t XL, uint32_t XH, uint32_t (&r)[3]) const {
    const uint32_t sel = ((s & 2) ? o[j] : e[j]) >> (16 * (s & 1));
    const uint32_t lo0 = prmt(A[j], A[j], sel), hi0 = prmt(Bp[j], Bn[j], sel);
    r[0] = prmt(lo0, hi0, 0x5140u);
    r[1] = prmt(lo0, hi0, 0x7362u);
    r[2] = prmt(XL, XH, (s & 1) ? 0x7362u : 0x5140u);
  }
};

// ------------------------------------------------------------------------------------------
// N = 6 through the 2:4 sparse tensor-core instruction (mma.sp m16n8k32).  With 6 of 8 columns
// kept, rank 2 i sits in column 2 i .. 2 i + 2 and rank 2 i + 1 in column 2 i + 1 .. 2 i + 3, so
// the pair (2 i, 2 i + 1) is a 2-of-4 selection from columns 2 i .. 2 i + 3: every group is three
// "chunks" of the instruction, whose operand holds the pair in rank order and whose activations
// are x[8 G + 2 i .. 8 G + 2 i + 3].  Metadata nibble of chunk i = idx0 | idx1 << 2 with
// idx = column - 2 i of the two ranks (idx0 < idx1).
STB_HD constexpr uint32_t meta6_nibble(uint32_t keep_byte, int i) {
  uint32_t col[8] = {0, 0, 0, 0, 0, 0, 0, 0};
  int r = 0;
  for (int c = 0; c < 8; ++c)
    if ((keep_byte >> c) & 1u) col[r++ & 7] = (uint32_t)c;
  return ((col[2 * i] - 2u * (uint32_t)i) & 3u) | (((col[2 * i + 1] - 2u * (uint32_t)i) & 3u) << 2);
}
// Table keyed by the keep-mask index: byte i = nibble of chunk i.  Entries past the 28 masks hold a valid pattern.
constexpr int kMeta6Entries = 64;
struct Meta6Table { uint32_t v[kMeta6Entries]; };
constexpr Meta6Table make_meta6_table() {
  Meta6Table t{};
  for (int e = 0; e < kMeta6Entries; ++e) {
    t.v[e] = 0;
    for (int i = 0; i < 3; ++i) t.v[e] |= (e < 28 ? meta6_nibble(kMaskTables.mask[6][e], i) : 0x4u) << (8 * i);
  }
  return t;
}
// Joint table keyed by the pair field of two rows (stb_layout.cuh): entry J = i0 + 28 i1 holds, in word i, the
// nibble of chunk i of the mask with index i0 at bit 0 and that of the mask with index i1 at bit 16; the
// metadata word of chunk i is then  sum over the quad's lanes tq of  word_i(J_tq) << 4 tq.
struct Meta6Joint { uint32_t v[kMasks6 * kMasks6][4]; };
constexpr Meta6Joint make_meta6_joint() {
  Meta6Joint t{};
  for (uint32_t i1 = 0; i1 < kMasks6; ++i1)
    for (uint32_t i0 = 0; i0 < kMasks6; ++i0) {
      for (int i = 0; i < 3; ++i)
        t.v[i0 + kMasks6 * i1][i] = meta6_nibble(kMaskTables.mask[6][i0], i) | (meta6_nibble(kMaskTables.mask[6][i1], i) << 16);
      t.v[i0 + kMasks6 * i1][3] = 0;
    }
  return t;
}
// The six metadata words of a lane from the table entries en[rp][tq] (row g + 16 mt + 8 rp, lane tq of the quad)
// of one of its two slots: word i has the nibble of lane tq at bit 4 tq (row rp = 0) and 16 + 4 tq (rp = 1).
STB_HD void meta6_words(const uint32_t (&en)[2][4], uint32_t (&E)[3]) {
  const uint32_t z01a = en[0][0] + (en[0][1] << 4), z23a = en[0][2] + (en[0][3] << 4);
  const uint32_t z01b = en[1][0] + (en[1][1] << 4), z23b = en[1][2] + (en[1][3] << 4);
  const uint32_t wa = prmt(z01a, z23a, 0x5140u), wb = prmt(z01b, z23b, 0x5140u);
  const uint32_t wc = prmt(z01a, z23a, 0x7362u), wd = prmt(z01b, z23b, 0x7362u);
  E[0] = prmt(wa, wb, 0x5410u);
  E[1] = prmt(wa, wb, 0x7632u);
  E[2] = prmt(wc, wd, 0x5410u);
}

// ------------------------------------------------------------------------------------------
// The same fast decode for ONE of the lane's four rows, the row index j a run-time value (the
// prefill GEMM gives each of four warps one row of a row tile: one copy of the code serves all).
struct RowWords {
  uint32_t mask;            // byte s = keep-mask index of group 4 s + t
  uint32_t Rlo, Rhi;        // region words: ranks 0..3 of the row's four slots / the word holding its ranks 4..
  uint32_t Slo, Shi;        // sign words: the one holding ranks 0..3 / ranks 4.. (N = 5: the half word, lower-lane form)
  uint32_t A, B;            // low / high bytes of the four main scales
};
template <int N>
STB_HD void load_row_words(const uint8_t* tile, int lane, int j, RowWords& w) {
  static_assert(N >= 4 && N <= 6, "fast decode covers N = 4, 5, 6");
  const int g = lane >> 2, t = lane & 3;
  if (mask_pairs(N)) {
    w.mask = 0;
#pragma unroll
    for (int sidx = 0; sidx < 4; ++sidx) {
      const uint32_t f = *reinterpret_cast<const uint16_t*>(tile + pair_field_off(g, j >> 1, sidx, t));
      w.mask |= pair_field_index(f, j & 1) << (8 * sidx);
    }
  } else {
    w.mask = *reinterpret_cast<const uint32_t*>(tile + lane * 16 + 4 * j);
  }
  w.Rlo = *reinterpret_cast<const uint32_t*>(tile + region_word_off(N, j, lane));
  w.Slo = *reinterpret_cast<const uint32_t*>(tile + sign_word_off(N, j >> 1, lane));
  w.Rhi = 0; w.Shi = 0;
  if (N == 6) {
    w.Rhi = *reinterpret_cast<const uint32_t*>(tile + region_word_off(N, 4 + (j >> 1), lane));
    w.Shi = *reinterpret_cast<const uint32_t*>(tile + sign_word_off(N, 2, lane));
  } else if (N == 5) {
    w.Rhi = *reinterpret_cast<const uint32_t*>(tile + region_word_off(N, 4, lane));
    const uint32_t h = *reinterpret_cast<const uint32_t*>(tile + sign_half_off(N, lane));
    w.Shi = lane < 16 ? (h & 0x66666666u) : half_from_upper(h & 0x99999999u);
  }
  const uint2 sc = *reinterpret_cast<const uint2*>(tile + scale_off(N, g, j));
  w.A = sc.x; w.B = sc.y;
}

template <int N>
struct OneRow {
  static_assert(N >= 4 && N <= 6, "fast decode covers N = 4, 5, 6");
  uint32_t A, Bp, Bn, e, o, hs, XL, XH;

  // A_, B_: low / high bytes of the four main scales in the 16-bit format wanted
  STB_HD void init(const RowWords& w, int j, uint32_t A_, uint32_t B_) {
    A = A_; Bp = B_; Bn = B_ ^ 0x80808080u;
    const uint32_t se = w.Slo >> (j & 1), so = w.Slo << (1 + (j & 1));
    e = (w.Rlo & 0x33333333u) | (se & 0x44444444u);
    o = ((w.Rlo >> 2) & 0x33333333u) | (so & 0x44444444u);
    hs = 0; XL = 0; XH = 0;
    if (N == 6) {
      const uint32_t sg = j == 0 ? w.Shi : (j == 1 ? (w.Shi << 1) : (j == 2 ? (w.Shi >> 1) : (w.Shi << 2)));
      hs = ((w.Rhi >> (2 * (j & 1))) & 0x33333333u) | (sg & 0x44444444u);
    } else if (N == 5) {
      const uint32_t sel = (j & 2) ? (((w.Rhi >> 2) & 0x33333333u) | ((w.Shi << 1) & 0x44444444u))
                                   : ((w.Rhi & 0x33333333u) | (w.Shi & 0x44444444u));
      hs = sel >> (16 * (j & 1));
      XL = prmt(A, A, hs);
      XH = prmt(Bp, Bn, hs);
    }
  }
  // N = 6: ranks 4, 5 of slots 2 sp, 2 sp + 1 (call before slot(2 sp, ..) and slot(2 sp + 1, ..))
  STB_HD void high(int sp) {
    const uint32_t sel = hs >> (16 * sp);
    XL = prmt(A, A, sel);
    XH = prmt(Bp, Bn, sel);
  }
  // slot s -> f[0..3]: columns (0,1), (2,3), (4,5), (6,7) as 16-bit pairs; P0 / P1 = position selectors of columns 0..3 / 4..7
  STB_HD void slot(int s, uint32_t P0, uint32_t P1, uint32_t (&f)[4]) const {
    const uint32_t sel = ((s & 2) ? o : e) >> (16 * (s & 1));
    const uint32_t lo0 = prmt(A, A, sel), hi0 = prmt(Bp, Bn, sel);
    uint32_t lo1 = 0, hi1 = 0;
    if (N == 6) {
      lo1 = (s & 1) ? (XL >> 16) : (XL & 0xFFFFu);
      hi1 = (s & 1) ? (XH >> 16) : (XH & 0xFFFFu);
    } else if (N == 5) {
      lo1 = prmt(XL, 0u, 0x4440u + (uint32_t)s);
      hi1 = prmt(XH, 0u, 0x4440u + (uint32_t)s);
    }
    const uint32_t pl0 = prmt(lo0, lo1, P0), pl1 = prmt(lo0, lo1, P1);
    const uint32_t ph0 = prmt(hi0, hi1, P0), ph1 = prmt(hi0, hi1, P1);
    f[0] = prmt(pl0, ph0, 0x5140u);
    f[1] = prmt(pl0, ph0, 0x7362u);
    f[2] = prmt(pl1, ph1, 0x5140u);
    f[3] = prmt(pl1, ph1, 0x7362u);
  }
};

// position selector of a keep byte: nibble c = rank of column c among the kept columns, 7 for a
// dropped column (byte 7 of the rank-ordered bytes is zero for N <= 7)
STB_HD uint32_t position_selector(uint32_t keep_byte) {
  uint32_t p = 0, r = 0;
  for (int c = 0; c < 8; ++c) {
    if ((keep_byte >> c) & 1u) { p |= (r & 7u) << (4 * c); ++r; }
    else p |= 7u << (4 * c);
  }
  return p;
}
// keep-mask index of slot (j, s)
STB_HD uint32_t keep_index_of(const uint32_t (&mask)[4], int j, int s) {
  return prmt(mask[j], 0u, 0x4440u + (uint32_t)s);
}

// Residual selectors of one resid word (rows r_0..r_3 of the lane, 4 slots): row j's four
// nibbles (0 = +a_sal2, 1 = none, 2 = -a_sal2) index the bytes of
//   L2 = (lo, 0, lo, 0)   H2 = (hi, 0, hi ^ 0x80, 0)      (lo / hi byte of a_sal2 of the row)
STB_HD uint32_t resid_selector(uint32_t word, int j) {
  const uint32_t v = (j & 2) ? ((word >> 2) & 0x33333333u) : (word & 0x33333333u);
  return (v >> (16 * (j & 1))) & 0xFFFFu;
}
STB_HD uint32_t resid_code(uint32_t word, int j, int q4) {
  return (word >> code_bit(4 * j + q4)) & 3u;
}

STB_HD bool header_matches(const Header* h, int n, int m, int N) {
  return h->magic == kMagic && h->n == n && h->m == m && h->N == N && h->status == 0u;
}

}  // namespace stb

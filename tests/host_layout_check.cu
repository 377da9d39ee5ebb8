// Host-only check of the packed layout and of the byte-permute decode (compiled with nvcc, run
// on the CPU, no GPU needed).  For random tiles it packs the logical fields with the same
// build_lane_words the pack kernel uses, then checks that
//   * plain_slot returns every kept weight's region code and sign at the right column,
//   * FastRows::slot (N = 4, 5, 6) returns, for every column, the 16-bit pattern of the signed
//     scale of the weight's region, or zero for a dropped column,
//   * for N = 6 the rank-order operand pairs and the metadata table of the sparse tensor-core path
//     rebuild the same 16-bit patterns, and the pair fields return the keep-mask indices,
//   * the residual selectors return the stored two-bit codes.
// Expected values come from the logical fields directly (the definition of the format), not
// from any packed-side code.
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <vector>

#include "../paper_2408_01803_b200/csrc/stb_decode.cuh"

using namespace stb;

static uint64_t rng_state = 0x9E3779B97F4A7C15ull;
static uint32_t rnd() {
  rng_state ^= rng_state << 13; rng_state ^= rng_state >> 7; rng_state ^= rng_state << 17;
  return (uint32_t)(rng_state >> 24);
}

static uint8_t random_mask(int N) {
  uint8_t m = 0;
  int k = 0;
  while (k < N) {
    int c = rnd() % 8;
    if (!((m >> c) & 1)) { m |= (uint8_t)(1 << c); ++k; }
  }
  return m;
}

template <int N>
static int check(int trials, int spb) {
  int errors = 0;
  for (int trial = 0; trial < trials; ++trial) {
    // logical tile: 32 rows x 16 groups
    uint8_t keep[32][16], sign[32][16];
    uint16_t region[32][16], scale[32][5];
    uint8_t rcode[32][32];
    for (int r = 0; r < 32; ++r) {
      for (int g = 0; g < 16; ++g) {
        keep[r][g] = random_mask(N);
        sign[r][g] = (uint8_t)(rnd() & ((1u << N) - 1u));
        uint16_t rg = 0;
        for (int k = 0; k < N; ++k) rg |= (uint16_t)((rnd() & 3u) << (2 * k));
        region[r][g] = rg;
      }
      for (int q = 0; q < 5; ++q) scale[r][q] = (uint16_t)(rnd() & 0x7FFFu);
      for (int q = 0; q < 32; ++q) rcode[r][q] = q < spb ? (uint8_t)(rnd() % 3) : 1;
    }
    const uint32_t tb = tile_bytes(N);
    const int blk = 2;         // the tile's block number and its first residual word inside the row tile's stream
    const uint32_t w0 = 3;
    std::vector<uint8_t> tile(tb + 64, 0), stream(resid_rt_bytes(blk + 1, w0 + spb / 4) + 64, 0);
    uint8_t* record = stream.data() + resid_block_off(blk, w0);
    auto put32 = [&](uint32_t off, uint32_t v) { std::memcpy(&tile[off], &v, 4); };
    auto or32 = [&](uint32_t off, uint32_t v) { uint32_t o; std::memcpy(&o, &tile[off], 4); o |= v; std::memcpy(&tile[off], &o, 4); };
    for (int lane = 0; lane < 32; ++lane) {
      const int g = lane >> 2, t = lane & 3;
      uint32_t sg[16], rg[16], maskw[4] = {0, 0, 0, 0};
      for (int u = 0; u < 16; ++u) {
        const int j = u >> 2, s = u & 3, r = g + 8 * j, grp = 4 * s + t;
        maskw[j] |= mask_index(N, keep[r][grp]) << (8 * s);
        sg[u] = sign[r][grp]; rg[u] = region[r][grp];
      }
      LaneWords<N> w;
      build_lane_words<N>(sg, rg, true, w);
      if (mask_pairs(N)) {
        // pair fields: lane (g, t) holds rows g + 16 (t >> 1), + 8 and slots 2 (t & 1), 2 (t & 1) + 1 of the four lanes
        for (int wq = 0; wq < 4; ++wq) {
          maskw[wq] = 0;
          for (int hw = 0; hw < 2; ++hw) {
            const int s = 2 * (t & 1) + (wq >> 1), tq = 2 * (wq & 1) + hw, grp = 4 * s + tq, r0 = g + 16 * (t >> 1);
            maskw[wq] |= pair_field(mask_index(N, keep[r0][grp]), mask_index(N, keep[r0 + 8][grp])) << (16 * hw);
          }
        }
      }
      for (int j = 0; j < 4; ++j) put32(lane * 16 + 4 * j, maskw[j]);
      for (int i = 0; i < N; ++i) put32(region_word_off(N, i, lane), w.R[i]);
      for (int i = 0; i < sign_full_words(N); ++i) put32(sign_word_off(N, i, lane), w.S[i]);
      if (sign_has_half(N)) or32(sign_half_off(N, lane), lane < 16 ? w.half : half_to_upper(w.half));
    }
    for (int r = 0; r < 32; ++r) {
      const int g = r & 7, j = r >> 3;
      uint32_t A = 0, B = 0;
      for (int q = 0; q < 4; ++q) { A |= (uint32_t)(scale[r][q] & 0xFF) << (8 * q); B |= (uint32_t)(scale[r][q] >> 8) << (8 * q); }
      put32(scale_off(N, g, j), A); put32(scale_off(N, g, j) + 4, B);
      std::memcpy(record + resid_a2_off(g, j), &scale[r][4], 2);
      for (int q = 0; q < spb; ++q) {
        uint32_t o;
        std::memcpy(&o, record + resid_code_off((uint32_t)(q >> 2), g), 4);
        o |= (uint32_t)rcode[r][q] << code_bit(4 * j + (q & 3));
        std::memcpy(record + resid_code_off((uint32_t)(q >> 2), g), &o, 4);
      }
    }
    // every offset must stay inside the tile
    if (scale_off(N, 7, 3) + 8u != tb || resid_block_off(blk, w0) + resid_code_off(7u, 7) + 4u != resid_rt_bytes(blk + 1, w0 + 8u) ||
        resid_a2_off(7, 3) + 2u != kResidA2Bytes || resid_words_for(5) != 2 || resid_words_for(32) != kMaxResidWords) {
      ++errors; std::printf("N=%d tile size mismatch\n", N);
    }

    for (int lane = 0; lane < 32; ++lane) {
      const int g = lane >> 2, t = lane & 3;
      LaneTile<N> lt;
      load_lane_tile<N>(tile.data(), lane, lt);
      for (int u = 0; u < 16; ++u) {
        const int j = u >> 2, s = u & 3, r = g + 8 * j, grp = 4 * s + t;
        uint32_t code[8], neg[8];
        plain_slot<N>(lt, u, code, neg);
        int k = 0;
        for (int c = 0; c < 8; ++c) {
          uint32_t wc = 4, wn = 0;
          if ((keep[r][grp] >> c) & 1) {
            wc = (region[r][grp] >> (2 * k)) & 3u;
            wn = ((sign[r][grp] >> k) & 1u) ^ 1u;
            ++k;
          }
          if (code[c] != wc || neg[c] != wn) {
            if (++errors < 10) std::printf("plain N=%d lane %d u %d c %d: got (%u,%u) want (%u,%u)\n", N, lane, u, c, code[c], neg[c], wc, wn);
          }
        }
      }
      for (int j = 0; j < 4; ++j) {
        const int r = g + 8 * j;
        for (int q = 0; q < 4; ++q)
          if (scale_bits<N>(lt, j, q) != scale[r][q]) { if (++errors < 10) std::printf("scale N=%d\n", N); }
        if (sal2_bits(record, g, j) != scale[r][4]) { if (++errors < 10) std::printf("sal2 N=%d\n", N); }
        for (int q = 0; q < spb; ++q) {
          uint32_t word;
          word = resid_word(record, (uint32_t)(q >> 2), g);
          if (resid_code(word, j, q & 3) != rcode[r][q]) { if (++errors < 10) std::printf("resid code N=%d\n", N); }
          if (((resid_selector(word, j) >> (4 * (q & 3))) & 0xFu) != rcode[r][q]) { if (++errors < 10) std::printf("resid selector N=%d\n", N); }
        }
      }
      if constexpr (N == 6) {
        // rank-order operands and metadata of the sparse tensor-core path: rebuilding the row from them
        // (value of rank k lands on column 2 i + idx) must give the position-order weights
        static const Meta6Table meta = make_meta6_table();
        LaneTile<N> raw;
        load_lane_tile<N>(tile.data(), lane, raw, true);
        FastRows<N> fr;
        fr.init(lt, lt.A, lt.B);
        for (int j = 0; j < 4; ++j)
          for (int s = 0; s < 4; ++s) {
            uint32_t XL, XH, rr[3];
            fr.high(j, s >> 1, XL, XH);
            fr.pairs(j, s, XL, XH, rr);
            const int r = g + 8 * j, grp = 4 * s + t;
            // the lane that supplies this chunk's metadata: (g, 2 (j >> 1) + (s >> 1)), field halfword 4 (s & 1) + t
            uint16_t field;
            std::memcpy(&field, &tile[pair_field_off(g, j >> 1, s, t)], 2);
            if (pair_field_index(field, j & 1) != mask_index(N, keep[r][grp])) { if (++errors < 10) std::printf("pair field N=%d\n", N); }
            uint32_t row[8] = {0, 0, 0, 0, 0, 0, 0, 0};
            for (int i = 0; i < 3; ++i) {
              const uint32_t nib = (meta.v[pair_field_index(field, j & 1)] >> (8 * i)) & 0xFu;
              if ((nib & 3u) >= (nib >> 2)) { if (++errors < 10) std::printf("metadata order N=%d\n", N); }
              row[2 * i + (nib & 3u)] = rr[i] & 0xFFFFu;
              row[2 * i + (nib >> 2)] = rr[i] >> 16;
            }
            int k = 0;
            for (int c = 0; c < 8; ++c) {
              uint32_t want = 0;
              if ((keep[r][grp] >> c) & 1) {
                const uint32_t code = (region[r][grp] >> (2 * k)) & 3u;
                const uint32_t ng = ((sign[r][grp] >> k) & 1u) ^ 1u;
                want = scale[r][code] ^ (ng << 15);
                ++k;
              }
              if (row[c] != want) { if (++errors < 10) std::printf("sparse N=%d lane %d j %d s %d c %d: got %04x want %04x\n", N, lane, j, s, c, row[c], want); }
            }
          }
      }
      if constexpr (N == 6) {
        // the metadata words this lane hands to the instruction: rows g + 16 (t >> 1) + 8 rp, slots 2 (t & 1) + bb
        // of the four lanes tq; nibble of lane tq at bit 4 tq + 16 rp of word i
        static const Meta6Table meta = make_meta6_table();
        LaneTile<N> raw;
        load_lane_tile<N>(tile.data(), lane, raw, true);
        static const Meta6Joint joint = make_meta6_joint();
        for (int bb = 0; bb < 2; ++bb) {
          uint32_t en[2][4], E[3], EJ[3] = {0, 0, 0};
          for (int tq = 0; tq < 4; ++tq) {
            // the pair field of lane tq's slot: two keep-mask indices (one way), or the joint-table entry (the other)
            const uint32_t f = (raw.mask[2 * bb + (tq >> 1)] >> (16 * (tq & 1))) & 0xFFFFu;
            if (f % 16 != 0 || f / 16 >= kMasks6 * kMasks6) { ++errors; continue; }
            en[0][tq] = meta.v[pair_field_index(f, 0)];
            en[1][tq] = meta.v[pair_field_index(f, 1)];
            for (int i = 0; i < 3; ++i) EJ[i] += joint.v[f / 16][i] << (4 * tq);
          }
          meta6_words(en, E);
          for (int i = 0; i < 3; ++i) {
            if (E[i] != EJ[i]) { if (++errors < 10) std::printf("joint metadata word N=%d\n", N); }
            for (int tq = 0; tq < 4; ++tq)
              for (int rp = 0; rp < 2; ++rp) {
                const int r = g + 16 * (t >> 1) + 8 * rp, grp = 4 * (2 * (t & 1) + bb) + tq;
                if (((E[i] >> (4 * tq + 16 * rp)) & 0xFu) != meta6_nibble(keep[r][grp], i)) { if (++errors < 10) std::printf("metadata word N=%d\n", N); }
              }
          }
        }
      }
      if constexpr (N >= 4 && N <= 6) {
        FastRows<N> fr;
        fr.init(lt, lt.A, lt.B);
        for (int j = 0; j < 4; ++j) {
          uint32_t XL = 0, XH = 0;
          if (N == 5) fr.high(j, 0, XL, XH);
          for (int s = 0; s < 4; ++s) {
            if (N == 6 && (s & 1) == 0) fr.high(j, s >> 1, XL, XH);
            const int r = g + 8 * j, grp = 4 * s + t;
            const uint32_t kb = mask_from_index(N, keep_index_of(lt.mask, j, s));
            if (kb != keep[r][grp]) { if (++errors < 10) std::printf("keep byte N=%d\n", N); }
            uint32_t f[4];
            fr.slot(j, s, position_selector(kb), XL, XH, f);
            {   // the one-row form with a run-time row index must give the same registers
              RowWords rw;
              load_row_words<N>(tile.data(), lane, j, rw);
              OneRow<N> orow;
              orow.init(rw, j, rw.A, rw.B);
              if (N == 6) orow.high(s >> 1);
              uint32_t f1[4];
              const uint32_t pp = position_selector(mask_from_index(N, (rw.mask >> (8 * s)) & 0xFFu));
              orow.slot(s, pp & 0xFFFFu, pp >> 16, f1);
              if (f1[0] != f[0] || f1[1] != f[1] || f1[2] != f[2] || f1[3] != f[3]) {
                if (++errors < 10) std::printf("one row N=%d lane %d j %d s %d\n", N, lane, j, s);
              }
            }
            int k = 0;
            for (int c = 0; c < 8; ++c) {
              uint32_t want = 0;
              if ((keep[r][grp] >> c) & 1) {
                const uint32_t code = (region[r][grp] >> (2 * k)) & 3u;
                const uint32_t ng = ((sign[r][grp] >> k) & 1u) ^ 1u;
                want = scale[r][code] ^ (ng << 15);
                ++k;
              }
              const uint32_t got = (f[c >> 1] >> (16 * (c & 1))) & 0xFFFFu;
              if (got != want) {
                if (++errors < 10) std::printf("fast N=%d lane %d j %d s %d c %d: got %04x want %04x\n", N, lane, j, s, c, got, want);
              }
            }
          }
        }
      }
    }
  }
  return errors;
}

int main() {
  int e = 0;
  e += check<1>(4, 0); e += check<2>(4, 4); e += check<3>(4, 8); e += check<4>(8, 4); e += check<5>(8, 16);
  e += check<6>(8, 32); e += check<7>(4, 4); e += check<8>(4, 0); e += check<4>(2, 0); e += check<6>(2, 8);
  // keep-mask index: a bijection between the masks with N bits and 0..C(8,N)-1, in increasing order
  for (int N = 0; N <= 8; ++N) {
    int k = 0;
    for (uint32_t m = 0; m < 256; ++m) {
      int pc = 0;
      for (int c = 0; c < 8; ++c) pc += (m >> c) & 1;
      if (pc != N) continue;
      if (mask_index(N, m) != (uint32_t)k || mask_from_index(N, k) != m) ++e;
      ++k;
    }
    const int want[9] = {1, 8, 28, 56, 70, 56, 28, 8, 1};
    if (k != want[N] || kMaskTables.count[N] != want[N]) ++e;
  }
  // position selector: rank of each kept column, 7 for dropped ones
  for (uint32_t m = 0; m < 256; ++m) {
    const uint32_t p = position_selector(m);
    int r = 0;
    for (int c = 0; c < 8; ++c) {
      const uint32_t nib = (p >> (4 * c)) & 0xFu;
      if ((m >> c) & 1u) { if (nib != (uint32_t)(r & 7)) ++e; ++r; }
      else if (nib != 7u) ++e;
    }
  }
  std::printf("%s: %d errors\n", e ? "FAIL" : "OK", e);
  return e ? 1 : 0;
}

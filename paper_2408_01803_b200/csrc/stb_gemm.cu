// stb_gemm: prefill GEMM  Y[t][i] = sum_j W^[i][j] X[t][j]  on the 5th-generation tensor cores
// (tcgen05.mma, fp32 accumulators in tensor memory).  The compute-bound prefilling stage of
// Appendix C.2: N = sequence length x batch tokens against one packed layer.
//
// One CTA computes a 128 (rows of W^) x 256 kAcc (tokens) tile of the output, D = A B^T with
//   A = 128 x 64 bf16 slice of W^, decoded from the packed tiles into shared memory in the
//       K-major 128-byte-swizzled layout the tensor core reads,
//   B = kAcc slices of 256 x 64 bf16 of X, brought in by TMA with the same swizzle; every decoded
//       A stage is multiplied with all of them (kAcc accumulators of 256 TMEM columns), which
//       divides the decode work per flop by kAcc,
// in rings over K (kStagesA decoded A stages, kStagesB X stages: the decode warps run ahead of the tensor core).  Warp roles:
//   warp 0      TMA producer (one lane): X slices
//   warp 1, 18  MMA issuers (one lane each, on two schedulers): with two accumulators each takes one (4 x tcgen05.mma,
//               K = 16, per stage); with one, each takes half of a stage's K into an accumulator of its own and the
//               epilogue adds the two.  tcgen05.commit frees the boxes and stages; warp 1 allocates / frees TMEM
//   warps 2..   decode: warp w works on rows 32 (w % 4) .. +31 of the tile = one packed row tile;
//               four warps share a row tile, each taking one of the four rows a lane owns (the row
//               index is a run-time value: one copy of the code; one warp alone per scheduler
//               would be bound by instruction latency); per 128-column block it loads its row's
//               words (prefetching the next block), converts the four fp16 scales to bf16
//               (RN-even) and writes the two 64-column halves of the block into two stages;
//               afterwards the same warps read the accumulator (TMEM lanes 32 (w % 4) ..) and
//               store Y.
// The residual term of the salient columns (Eq. 4) is more K: a small kernel first gathers the activations of
// every residual slot (four per residual word, in word order) into Xs[token][slot]; after the blocks of its K
// range a CTA runs the residual slots of those blocks as further stages, A = +-bf16(a_sal2) or 0 by the two-bit
// residual codes, B = Xs through a second tensor map.  The main stages give a salient weight s1 bf16(a_sal1).
// One CTA fits an SM, so the grid runs in waves of 148 output tiles; tiles of a small last wave
// (and all tiles when there are few) are split along K into fp32 partial tiles in the caller's
// workspace and summed by a second kernel.
// Every wait on an mbarrier is bounded; a wait that runs out sets an abort flag (all roles then
// leave their loops), reports STB_ERR_TIMEOUT through dev_status and the CTA still frees TMEM.
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/stb.h"
#include "stb_decode.cuh"
#include "stb_layout.cuh"
#include "stb_ptx.cuh"

namespace stb {

constexpr int kBM = 128;          // rows of W^ per CTA (UMMA M)
// Token side of the CTA tile: kAcc accumulators of kBN tokens (UMMA N).  Prefill: 2 x 256 (all 512 TMEM columns; a
// decoded A stage is used twice).  Up to 64 tokens (a decode batch): 1 x 64, the tensor core then takes an eighth
// of the time per stage and the kernel runs at the speed of the decode warps.
template <int kAcc_, int kBN_>
struct TokCfg {
  static constexpr int kAcc = kAcc_, kBN = kBN_, kTok = kAcc_ * kBN_;
  static constexpr uint32_t kStageB = (uint32_t)kBN_ * 64u * 2u;                 // one X box: kBN tokens x 64 of K
  static constexpr int kStagesB = kBN_ >= 256 ? 5 : 8;                            // ring of X boxes
};
constexpr int kBK = 64;           // K per stage: one 128-byte swizzle row of bf16
constexpr int kStagesA = 4;        // ring of decoded A stages (16 KB each)
// (the ring of X boxes, TokCfg::kStagesB: 256 tokens x 64 of K = 32 KB each in prefill; a stage of K takes kAcc of them:
// what is in flight from L2 is what hides its latency, so the ring is deep and its slots small)
constexpr int kGroups = 4;                              // decode warps per 32-row quarter: one per row of a lane
constexpr int kIssuers = 2;                             // MMA-issuing lanes (in two warps, on two schedulers)
constexpr int kIssuerWarpB = 2 + 4 * kGroups;           // the second one's warp: after the decode warps
constexpr int kGemmThreads = 64 + 128 * kGroups + 32;
constexpr uint32_t kStageA = kBM * kBK * 2;      // 16 KB
constexpr uint32_t kGemmTab = 0;                                   // position table (576 B)
constexpr uint32_t kGemmBars = 1024;                               // fullA, emptyA, fullB, emptyB, accum, tmem slot, abort
constexpr uint32_t kGemmA = 2048;                                  // 1024-byte aligned stages
constexpr uint32_t kGemmB = kGemmA + kStagesA * kStageA;
template <class Cfg> constexpr uint32_t gemm_smem_bytes() { return kGemmB + (uint32_t)Cfg::kStagesB * Cfg::kStageB; }   // prefill: 231424 B
static_assert(gemm_smem_bytes<TokCfg<2, 256>>() <= 232448 && gemm_smem_bytes<TokCfg<1, 64>>() <= 232448, "one CTA's shared memory");
static_assert(8 * (2 * kStagesA + 2 * 8 + 1) + 16 <= 1024, "barrier area");
constexpr long long kGemmWaitLimit = 2000000000ll;

// ---- tcgen05 / TMA wrappers ---------------------------------------------------------------
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, int x, int y, uint32_t bar) {
  asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
               ::"r"(dst), "l"(map), "r"(x), "r"(y), "r"(bar) : "memory");
}
__device__ __forceinline__ void tmem_alloc(uint32_t slot_smem, uint32_t ncols) {
  asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(slot_smem), "r"(ncols) : "memory");
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols) {
  asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
// The descriptors come as their low words (start address / 16; the high word is the same for every operand tile of
// this kernel) and the accumulate flag as a template argument: an issuing lane is ONE thread whose instructions go
// out one dependent step at a time, and what it runs per stage of K (waits, descriptors, MMAs, commits) was longer
// than the tensor core needs for the stage.
template <bool kAccumulate>
__device__ __forceinline__ void umma_16(uint32_t d_tmem, uint32_t adesc_lo, uint32_t bdesc_lo, uint32_t desc_hi, uint32_t idesc) {
  if (kAccumulate)
    asm volatile("{\n\t.reg .pred p;\n\t.reg .b64 da, db;\n\tsetp.eq.b32 p, 0, 0;\n\tmov.b64 da, {%1, %3};\n\tmov.b64 db, {%2, %3};\n\t"
                 "tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %4, p;\n\t}"
                 ::"r"(d_tmem), "r"(adesc_lo), "r"(bdesc_lo), "r"(desc_hi), "r"(idesc) : "memory");
  else
    asm volatile("{\n\t.reg .pred p;\n\t.reg .b64 da, db;\n\tsetp.ne.b32 p, 0, 0;\n\tmov.b64 da, {%1, %3};\n\tmov.b64 db, {%2, %3};\n\t"
                 "tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %4, p;\n\t}"
                 ::"r"(d_tmem), "r"(adesc_lo), "r"(bdesc_lo), "r"(desc_hi), "r"(idesc) : "memory");
}
__device__ __forceinline__ void umma_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&r)[32]) {
  asm volatile("tcgen05.ld.sync.aligned.32x32b.x32.b32 "
               "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
                 "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
                 "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
                 "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
               : "r"(taddr) : "memory");
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}

// Shared-memory matrix descriptor of a K-major, 128-byte-swizzled operand tile (rows of 128
// bytes, groups of 8 rows 1024 bytes apart): start address, stride byte offset 1024,
// descriptor version 1, layout type 2 (128-byte swizzle).
__device__ __forceinline__ uint64_t umma_desc(uint32_t smem_addr) {
  uint64_t d = 0;
  d |= (uint64_t)((smem_addr & 0x3FFFFu) >> 4);
  d |= (uint64_t)1 << 16;                  // leading byte offset (unused for swizzled K-major)
  d |= (uint64_t)(1024 >> 4) << 32;        // stride byte offset
  d |= (uint64_t)1 << 46;                  // version
  d |= (uint64_t)2 << 61;                  // SWIZZLE_128B
  return d;
}
// Instruction descriptor: D = f32, A and B both bf16 (format 1) or both fp16 (format 0), both K-major, N = kBN, M = 128.
template <int kBN, bool kF16>
struct GemmIdesc {
  static constexpr uint32_t value = (1u << 4) | ((kF16 ? 0u : 1u) << 7) | ((kF16 ? 0u : 1u) << 10) | ((uint32_t)(kBN >> 3) << 17) | ((uint32_t)(kBM >> 4) << 24);
};

// Bounded mbarrier wait with a CTA-wide abort flag (a volatile int in shared memory).  The two
// single-lane roles back off between polls so that their spinning does not take issue slots from
// the decode warps that share their schedulers.
template <bool kBackoff = false>
__device__ __forceinline__ bool gemm_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag) {
  if (mbar_try_wait(bar, parity)) return true;
  const long long t0 = clock64();
  while (!mbar_try_wait(bar, parity)) {
    if (kBackoff) __nanosleep(32);
    if (*abort_flag) return false;
    if (clock64() - t0 > kGemmWaitLimit) { *abort_flag = 1; return false; }
  }
  return true;
}

__device__ __forceinline__ uint32_t bf16_bits(uint32_t h16) {
  return (uint32_t)__bfloat16_as_ushort(__float2bfloat16_rn(__half2float(__ushort_as_half((unsigned short)h16))));
}

// What a decode warp needs to know.
struct DecodeArgs {
  const uint8_t* packed; const Header* hdr; uint8_t* smem; volatile int* abort_flag;
  uint32_t bar_full, bar_empty;      // of the A ring
  int mt, b0, b1, nblk, ntile, q, lane;
  uint32_t rw0, rw1;        // residual words of the blocks [b0, b1)
  int nres;                 // residual stages (64 slots = 16 words each, the first one starts at word rw0 & ~1)
};

// Decode role of one warp: row j (of the four rows g + 8 j each lane owns) of packed row tile 4 mt + q, for
// every block of the CTA's K range, written into the A stages.  j is a run-time value: the four warps of a
// row tile run the same code.
// kF16: the stages hold fp16 (the scales as stored); otherwise bf16 (the scales rounded to nearest even).
template <int N, bool kF16>
__device__ __forceinline__ void decode_row(const DecodeArgs& da, const int j) {
  const uint8_t* packed = da.packed;
  const Header* hdr = da.hdr;
  uint8_t* smem = da.smem;
  volatile int* abort_flag = da.abort_flag;
  const uint32_t bar_full = da.bar_full, bar_empty = da.bar_empty;
  const int mt = da.mt, b0 = da.b0, b1 = da.b1, nblk = da.nblk, ntile = da.ntile, q = da.q;
  // The lane plays the part of packed-layout lane 4 g + t with g = lane % 8, t = lane / 8: the eight
  // lanes of a quarter-warp then hold eight different rows g and their 16-byte stores into the
  // swizzled stage fall on eight different 16-byte bank groups (no conflict); loads of the
  // lane-major planes stay coalesced, they are only permuted inside the warp.
  const int g = da.lane & 7, t = da.lane >> 3;
  const int lane = 4 * g + t;
  const int rtile = mt * 4 + q;                 // packed row tile
  const bool live = rtile < ntile;
  const uint32_t* ptab = reinterpret_cast<const uint32_t*>(smem + kGemmTab);     // low half: columns 0..3, high half: 4..7
  const uint8_t* rtbase = packed + hdr->tiles_offset + (size_t)rtile * hdr->rt_stride;
  const uint8_t* resid_rt = packed + hdr->tiles_offset + hdr->rt_stride * (size_t)ntile +
                            (size_t)rtile * resid_rt_bytes(nblk, hdr->nrw);
  constexpr uint32_t tbytes = tile_bytes(N);
  // The row's words are loaded three blocks ahead of their use (three sets of registers in rotation): the loads
  // come straight from HBM, and one block of decode is shorter than their latency.
  RowWords w0 = {}, w1 = {}, w2 = {};
  auto fetch = [&](int b, RowWords& w) {
    if (live && b < b1) load_row_words<N>(rtbase + (size_t)b * tbytes, lane, j, w);
  };
  auto block = [&](int b, const RowWords& cur) -> bool {
    // bf16 scale bytes of the row (a salient weight gets s1 bf16(a_sal1) here; its residual term comes with the residual stages)
    uint32_t A16 = 0, B16 = 0;
    if (live) {
#pragma unroll
      for (int c = 0; c < 4; ++c) {
        const uint32_t h16 = ((cur.A >> (8 * c)) & 0xFFu) | (((cur.B >> (8 * c)) & 0xFFu) << 8);
        const uint32_t v = kF16 ? h16 : bf16_bits(h16);
        A16 |= (v & 0xFFu) << (8 * c);
        B16 |= (v >> 8) << (8 * c);
      }
    }
    OneRow<N> row;
    row.init(cur, j, A16, B16);
    // position selectors of the row's slots of this block, looked up before the stage waits
    uint32_t P[4];
#pragma unroll
    for (int sidx = 0; sidx < 4; ++sidx) P[sidx] = live ? ptab[(cur.mask >> (8 * sidx)) & 0xFFu] : 0u;
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      const int it = 2 * (b - b0) + h, st = it % kStagesA;
      // the verdict is made warp-uniform: nobody may be left alone at the __syncwarp() below
      if (!__all_sync(0xFFFFFFFFu, gemm_wait(bar_empty + 8 * st, ((uint32_t)(it / kStagesA) & 1u) ^ 1u, abort_flag))) return false;
      uint8_t* As = smem + kGemmA + st * kStageA;
      uint8_t* rowp = As + (size_t)(4 * q + j) * 1024 + g * 128;
      if (N == 6 && live) row.high(h);
#pragma unroll
      for (int sl = 0; sl < 2; ++sl) {
        const int sidx = 2 * h + sl;                       // slot s of the block, group 4 sidx + t
        uint32_t f[4] = {0, 0, 0, 0};
        if (live) row.slot(sidx, P[sidx], P[sidx] >> 16, f);
        const int chunk = 4 * sl + t;                      // 16-byte chunk of the 128-byte row
        *reinterpret_cast<uint4*>(rowp + ((chunk ^ g) << 4)) = make_uint4(f[0], f[1], f[2], f[3]);
      }
      fence_async_smem();          // generic-proxy writes -> visible to the tensor core
      __syncwarp();
      if (lane == 0) mbar_arrive(bar_full + 8 * st);
    }
    return true;
  };
  // Residual stages (after the blocks): 64 residual slots (16 residual words) of K each.  The lane writes the same
  // two 16-byte chunks of its row as above: chunk c holds the words 2 c and 2 c + 1 of the stage, four slots each,
  // as +-bf16(a_sal2) or 0.  What a stage needs sits behind two dependent loads from global memory (the word's table
  // entry, then a_sal2 and the codes from the block's record), so both are taken ahead: the entries two stages, the
  // records one stage before their use, the first ones before the blocks.
  const ResidWord* rwt = reinterpret_cast<const ResidWord*>(packed + rwtab_offset(nblk));
  const uint32_t wfirst = da.rw0 & ~1u;
  auto res_word = [&](int rs, int idx) { return wfirst + 16u * (uint32_t)rs + 2u * (uint32_t)(4 * (idx >> 1) + t) + (uint32_t)(idx & 1); };
  auto res_entries = [&](int rs, uint2 (&e)[4], uint32_t& valid) {
    valid = 0;
#pragma unroll
    for (int idx = 0; idx < 4; ++idx) {
      const uint32_t w = res_word(rs, idx);
      e[idx] = make_uint2(0u, 0u);
      if (live && rs < da.nres && w >= da.rw0 && w < da.rw1) { e[idx] = __ldg(reinterpret_cast<const uint2*>(rwt + w)); valid |= 1u << idx; }
    }
  };
  auto res_records = [&](int rs, const uint2 (&e)[4], uint32_t valid, uint32_t (&a2)[4], uint32_t (&word)[4]) {
#pragma unroll
    for (int idx = 0; idx < 4; ++idx) {
      a2[idx] = 0; word[idx] = 0;
      if ((valid >> idx) & 1u) {
        const uint8_t* rec = resid_rt + resid_block_off((int)(e[idx].x >> 3), res_word(rs, idx) - (e[idx].x & 7u));
        a2[idx] = __ldg(reinterpret_cast<const uint16_t*>(rec + resid_a2_off(g, j)));
        word[idx] = __ldg(reinterpret_cast<const uint32_t*>(rec + resid_code_off(e[idx].x & 7u, g)));
      }
    }
  };
  auto res_stage = [&](int rs, uint32_t valid, const uint32_t (&a2)[4], const uint32_t (&word)[4]) -> bool {
    const int it = 2 * (b1 - b0) + rs, st = it % kStagesA;
    uint32_t f[2][4] = {{0, 0, 0, 0}, {0, 0, 0, 0}};
#pragma unroll
    for (int idx = 0; idx < 4; ++idx)
      if ((valid >> idx) & 1u) {
        const uint32_t v = kF16 ? a2[idx] : bf16_bits(a2[idx]);
        const uint32_t L2 = prmt(v, 0u, 0x4040u);                 // (lo, 0, lo, 0)
        const uint32_t H2 = prmt(v, v ^ 0x8000u, 0x2521u);        // (hi, 0, hi ^ 0x80, 0)
        const uint32_t sel = resid_selector(word[idx], j);
        const uint32_t lo4 = prmt(L2, L2, sel), hi4 = prmt(H2, H2, sel);
        f[idx >> 1][2 * (idx & 1)] = prmt(lo4, hi4, 0x5140u);
        f[idx >> 1][2 * (idx & 1) + 1] = prmt(lo4, hi4, 0x7362u);
      }
    if (!__all_sync(0xFFFFFFFFu, gemm_wait(bar_empty + 8 * st, ((uint32_t)(it / kStagesA) & 1u) ^ 1u, abort_flag))) return false;
    uint8_t* rowp = smem + kGemmA + st * kStageA + (size_t)(4 * q + j) * 1024 + g * 128;
#pragma unroll
    for (int sl = 0; sl < 2; ++sl)
      *reinterpret_cast<uint4*>(rowp + (((4 * sl + t) ^ g) << 4)) = make_uint4(f[sl][0], f[sl][1], f[sl][2], f[sl][3]);
    fence_async_smem();
    __syncwarp();
    if (lane == 0) mbar_arrive(bar_full + 8 * st);
    return true;
  };
  uint2 eX[4], eY[4];
  uint32_t veX = 0, veY = 0, vrX = 0, vrY = 0, a2X[4], a2Y[4], wdX[4], wdY[4];
  res_entries(0, eX, veX);
  fetch(b0, w0);
  fetch(b0 + 1, w1);
  res_records(0, eX, veX, a2X, wdX); vrX = veX;
  res_entries(1, eY, veY);
  bool ok = true;
  for (int b = b0; b < b1 && ok; b += 3) {
    fetch(b + 2, w2);
    ok = block(b, w0);
    if (ok && b + 1 < b1) { fetch(b + 3, w0); ok = block(b + 1, w1); }
    if (ok && b + 2 < b1) { fetch(b + 4, w1); ok = block(b + 2, w2); }
  }
  for (int rs = 0; rs < da.nres && ok; rs += 2) {
    res_records(rs + 1, eY, veY, a2Y, wdY); vrY = veY;
    res_entries(rs + 2, eX, veX);
    ok = res_stage(rs, vrX, a2X, wdX);
    if (ok && rs + 1 < da.nres) {
      res_records(rs + 2, eX, veX, a2X, wdX); vrX = veX;
      res_entries(rs + 3, eY, veY);
      ok = res_stage(rs + 1, vrY, a2Y, wdY);
    }
  }
}

// Gathers the activations of the residual slots: Xs[t][4 w + k] = X[t][128 block(w) + cols(w)[k]] for every residual
// word w of the layer, and zeros in the 128 columns after the last word (a CTA's last residual stage may reach there).
__global__ void gemm_gather_kernel(const uint8_t* __restrict__ packed, int n, int m, int N, const __nv_bfloat16* __restrict__ X, int T,
                                   size_t ldx, __nv_bfloat16* __restrict__ Xs, int ldxs) {
  grid_launch_dependents();        // the GEMM may start; it waits for this grid before it reads Xs
  const Header* hdr = reinterpret_cast<const Header*>(packed);
  if (!header_matches(hdr, n, m, N)) return;
  const int nblk = m / kBlock;
  const ResidWord* rwt = reinterpret_cast<const ResidWord*>(packed + rwtab_offset(nblk));
  const uint32_t nrw = hdr->nrw;
  uint32_t W = nrw + 32u;                                   // words written per token: the layer's and 32 of zeros
  if (W > (uint32_t)ldxs / 4u) W = (uint32_t)ldxs / 4u;
  const size_t total = (size_t)T * W;
  for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (size_t)gridDim.x * blockDim.x) {
    const size_t t = i / W;
    const uint32_t w = (uint32_t)(i % W);
    uint2 out = make_uint2(0u, 0u);
    if (w < nrw) {
      const uint2 e = __ldg(reinterpret_cast<const uint2*>(rwt + w));
      const unsigned short* xr = reinterpret_cast<const unsigned short*>(X + t * ldx + (size_t)(e.x >> 3) * kBlock);
      out.x = (uint32_t)xr[e.y & 0xFFu] | ((uint32_t)xr[(e.y >> 8) & 0xFFu] << 16);
      out.y = (uint32_t)xr[(e.y >> 16) & 0xFFu] | ((uint32_t)xr[e.y >> 24] << 16);
    }
    *reinterpret_cast<uint2*>(Xs + t * (size_t)ldxs + 4u * w) = out;
  }
}

// ------------------------------------------------------------------------------------------
template <int N, class Cfg, bool kF16>
__global__ void __launch_bounds__(kGemmThreads, 1)
gemm_kernel(const __grid_constant__ CUtensorMap xmap, const __grid_constant__ CUtensorMap xsmap, const uint8_t* __restrict__ packed, int n, int m, int T,
            void* __restrict__ Y, int y_16, size_t ldy, float* __restrict__ ws, int full_tiles, int ksplit, int bps,
            int ttiles, uint32_t box_bytes, int* dev_status) {
  constexpr int kAcc = Cfg::kAcc, kBN = Cfg::kBN, kTok = Cfg::kTok, kStagesB = Cfg::kStagesB;
  constexpr uint32_t kStageB = Cfg::kStageB, kIdesc = GemmIdesc<kBN, kF16>::value;
  extern __shared__ __align__(1024) uint8_t smem[];
  // (the position table's entry of this thread is asked for before the header: two global-memory latencies side by
  // side instead of one after the other in every CTA's prologue)
  uint32_t tab_entry = 0;
  if (threadIdx.x < kPosTableEntries) tab_entry = g_pos_table.v[N][threadIdx.x].x | (g_pos_table.v[N][threadIdx.x].y << 16);
  const Header* hdr = reinterpret_cast<const Header*>(packed);
  if (!header_matches(hdr, n, m, N)) {
    if (threadIdx.x == 0 && dev_status) *dev_status = STB_ERR_CORRUPT;
    return;
  }
  const int nblk = m / kBlock, ntile = hdr->ntile;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  // CTAs 0 .. full_tiles - 1 compute one output tile each over the whole K; the rest come in groups of `ksplit`
  // per tile, each with `bps` blocks of K, and leave fp32 partial tiles in the workspace
  const int cta = (int)blockIdx.x;
  const bool split = cta >= full_tiles;
  const int tile = split ? full_tiles + (cta - full_tiles) / ksplit : cta;
  const int kz = split ? (cta - full_tiles) % ksplit : 0;
  const int tt = tile % ttiles, mt = tile / ttiles;
  const int b0 = split ? kz * bps : 0, b1 = split ? min(nblk, b0 + bps) : nblk;
  // residual words of the CTA's blocks -> residual stages of 16 words, the first one starting at an even word
  const BlockInfo* binfo_k = reinterpret_cast<const BlockInfo*>(packed + sizeof(Header));
  uint32_t rw0 = 0, rw1 = 0;
  if (b0 < b1) { rw0 = __ldg(&binfo_k[b0].rw_off); rw1 = b1 < nblk ? __ldg(&binfo_k[b1].rw_off) : hdr->nrw; }
  const int nres = rw1 > rw0 ? (int)((rw1 - (rw0 & ~1u) + 15u) / 16u) : 0;
  const int nmain = 2 * max(b1 - b0, 0);               // 64-column stages of the blocks
  const int nstage = nmain + nres;

  const uint32_t sbase = smem_u32(smem);
  // A ring: full = the 16 decode warps have written the stage, empty = the tensor core has read it;
  // B ring: full = the X boxes have landed, empty = the tensor core has read them
  const uint32_t bar_fullA = sbase + kGemmBars, bar_emptyA = bar_fullA + 8 * kStagesA;
  const uint32_t bar_fullB = bar_emptyA + 8 * kStagesA, bar_emptyB = bar_fullB + 8 * kStagesB, bar_accum = bar_emptyB + 8 * kStagesB;
  constexpr uint32_t kBarBytes = 8 * (2 * kStagesA + 2 * kStagesB + 1);
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + kGemmBars + kBarBytes);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + kGemmBars + kBarBytes + 8);

  if (threadIdx.x == 0) {
    // a stage of A is read by both issuers; an X box by the issuer of its accumulator (by both when there is one box per stage)
    for (int i = 0; i < kStagesA; ++i) { mbar_init(bar_fullA + 8 * i, 4 * kGroups); mbar_init(bar_emptyA + 8 * i, kIssuers); }
    for (int i = 0; i < kStagesB; ++i) { mbar_init(bar_fullB + 8 * i, 1); mbar_init(bar_emptyB + 8 * i, kAcc == 1 ? kIssuers : 1); }
    mbar_init(bar_accum, kIssuers);
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    fence_async_smem();
  }
  static_assert(kPosTableEntries <= kGemmThreads, "one table entry per thread");
  if (threadIdx.x < kPosTableEntries) reinterpret_cast<uint32_t*>(smem + kGemmTab)[threadIdx.x] = tab_entry;   // 4-byte entries: fewer bank conflicts than 8-byte ones
  constexpr uint32_t kTmemCols = kAcc == 1 ? 2 * kTok : kTok;      // one accumulator: a second one for the other half of K
  if (warp == 1) tmem_alloc(smem_u32(tmem_slot), kTmemCols);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_d = *tmem_slot;

  if (warp == 0) {
    // ---------------- TMA producer ----------------
    if (lane == 0) {
      for (int hb = 0; hb < nstage * kAcc; ++hb) {
        const int it = hb / kAcc, a = hb % kAcc, s = hb % kStagesB;
        if (!gemm_wait<true>(bar_emptyB + 8 * s, ((uint32_t)(hb / kStagesB) & 1u) ^ 1u, abort_flag)) break;
        // Xs comes from the gather kernel, which this grid may have overtaken (programmatic dependent launch)
        if (it == nmain && a == 0) grid_dependency_wait();
        mbar_expect_tx(bar_fullB + 8 * s, box_bytes);
        const uint32_t dst = sbase + kGemmB + s * kStageB;
        if (it < nmain) tma_load_2d(dst, &xmap, (b0 * 2 + it) * kBK, tt * kTok + a * kBN, bar_fullB + 8 * s);
        else tma_load_2d(dst, &xsmap, (int)(4u * (rw0 & ~1u)) + (it - nmain) * kBK, tt * kTok + a * kBN, bar_fullB + 8 * s);
      }
      grid_dependency_wait();  // (every CTA, whether or not it had residual stages)
      if (*abort_flag) {       // let copies in flight land before the CTA gives its shared memory up
        const long long t0 = clock64();
        while (clock64() - t0 < 200000) {}
      }
    }
  } else if (warp == 1 || warp == kIssuerWarpB) {
    // ---------------- MMA issuers ----------------
    if (lane == 0) {
      const int w = warp == 1 ? 0 : 1;
      // two accumulators: issuer w takes accumulator w (box w of every stage, all of K);
      // one accumulator:  issuer w takes the K steps 2 w, 2 w + 1 of every stage into accumulator w
      const uint32_t desc_hi = (uint32_t)(umma_desc(0u) >> 32);
      const uint32_t a_lo0 = (uint32_t)umma_desc(sbase + kGemmA) + (kAcc == 1 ? 4u * (uint32_t)w : 0u);
      const uint32_t b_lo0 = (uint32_t)umma_desc(sbase + kGemmB) + (kAcc == 1 ? 4u * (uint32_t)w : 0u);
      const uint32_t dt = tmem_d + (uint32_t)(w * (kAcc == 1 ? kTok : kBN));
      constexpr int kSteps = kAcc == 1 ? kBK / 32 : kBK / 16;           // MMAs per stage and issuer
      int sa = 0, sb = kAcc == 1 ? 0 : w;                               // ring slots, advanced without divisions
      uint32_t pa = 0, pb = 0;                                          // their phase parities
      for (int it = 0; it < nstage; ++it) {
        if (!gemm_wait<true>(bar_fullA + 8 * sa, pa, abort_flag)) break;
        if (!gemm_wait<true>(bar_fullB + 8 * sb, pb, abort_flag)) break;
        tc_fence_after();
        const uint32_t a_lo = a_lo0 + (uint32_t)sa * (kStageA >> 4), b_lo = b_lo0 + (uint32_t)sb * (kStageB >> 4);
        if (it > 0) umma_16<true>(dt, a_lo, b_lo, desc_hi, kIdesc);
        else umma_16<false>(dt, a_lo, b_lo, desc_hi, kIdesc);
#pragma unroll
        for (int kk = 1; kk < kSteps; ++kk) umma_16<true>(dt, a_lo + 2u * kk, b_lo + 2u * kk, desc_hi, kIdesc);
        umma_commit(bar_emptyB + 8 * sb);        // the box is free once the MMAs that read it have completed
        umma_commit(bar_emptyA + 8 * sa);
        if (++sa == kStagesA) { sa = 0; pa ^= 1u; }
        sb += kAcc == 1 ? 1 : kAcc;
        if (sb >= kStagesB) { sb -= kStagesB; pb ^= 1u; }
      }
      umma_commit(bar_accum);                    // all MMAs this lane issued have completed
    }
  } else {
    // ---------------- decode warps ----------------
    const int gi = (warp - 2) >> 2;               // decode group: which of the lane's four rows this warp takes
    DecodeArgs da;
    da.packed = packed; da.hdr = hdr; da.smem = smem; da.abort_flag = abort_flag;
    da.bar_full = bar_fullA; da.bar_empty = bar_emptyA;
    da.mt = mt; da.b0 = b0; da.b1 = b1; da.nblk = nblk; da.ntile = ntile; da.q = warp & 3; da.lane = lane;
    da.rw0 = rw0; da.rw1 = rw1; da.nres = nres;
    decode_row<N, kF16>(da, gi);

    // ---------------- epilogue: TMEM -> registers -> Y ----------------
    const int q = warp & 3;                        // TMEM lane quarter of this warp
    // A 16-bit output tile goes through shared memory (the X ring: every box has been consumed by then) so that it
    // leaves in 16-byte pieces along the rows: straight from the registers a warp's store is 32 rows x 2 bytes of
    // one token, and the epilogue took a ninth of the CTA's time.  The same for every thread of the CTA:
    const bool staged = y_16 != 0 && !split && (ldy % 8) == 0 && (reinterpret_cast<uintptr_t>(Y) & 15u) == 0 &&
                        (uint32_t)kTok * kBM * 2u <= (uint32_t)kStagesB * kStageB;
    uint16_t* stage = reinterpret_cast<uint16_t*>(smem + kGemmB);           // [token of the tile][row of the tile]
    const bool have = __all_sync(0xFFFFFFFFu, gemm_wait(bar_accum, 0u, abort_flag)) && nstage > 0;
    if (have) {
      tc_fence_after();
      const int row = mt * kBM + 32 * q + lane;                // output feature (row of W^)
      float* wsz = split ? ws + ((size_t)(tile - full_tiles) * ksplit + kz) * (size_t)(kBM * kTok) : nullptr;
#pragma unroll 1
      for (int cc = gi; cc < kTok / 32; cc += kGroups) {       // the groups share the column chunks
        uint32_t r[32];
        tmem_ld32(tmem_d + ((uint32_t)(32 * q) << 16) + (uint32_t)(32 * cc), r);
        if (kAcc == 1) {
          // the other half of K sits in the second accumulator
          uint32_t r2[32];
          tmem_ld32(tmem_d + ((uint32_t)(32 * q) << 16) + (uint32_t)(kTok + 32 * cc), r2);
#pragma unroll
          for (int i = 0; i < 32; ++i) r[i] = __float_as_uint(__uint_as_float(r[i]) + __uint_as_float(r2[i]));
        }
        if (staged) {
#pragma unroll
          for (int i = 0; i < 32; ++i) {
            const float v = __uint_as_float(r[i]);
            stage[(32 * cc + i) * kBM + 32 * q + lane] = kF16 ? __half_as_ushort(__float2half_rn(v)) : __bfloat16_as_ushort(__float2bfloat16_rn(v));
          }
        } else if (row < n) {
#pragma unroll
          for (int i = 0; i < 32; ++i) {
            const int tok = tt * kTok + 32 * cc + i;
            if (tok < T) {
              const float v = __uint_as_float(r[i]);
              if (wsz) wsz[(size_t)(32 * cc + i) * kBM + 32 * q + lane] = v;
              else if (y_16 && kF16) static_cast<__half*>(Y)[(size_t)tok * ldy + row] = __float2half_rn(v);
              else if (y_16) static_cast<__nv_bfloat16*>(Y)[(size_t)tok * ldy + row] = __float2bfloat16_rn(v);
              else static_cast<float*>(Y)[(size_t)tok * ldy + row] = v;
            }
          }
        }
      }
    }
    if (staged) {
      // every decode warp takes the barrier, whatever its wait said
      asm volatile("bar.sync 1, %0;" ::"n"(128 * kGroups) : "memory");
      if (have) {
        const int d = (warp - 2) * 32 + lane;                  // 0 .. 511: 16 threads per token, 8 rows each
        const int piece = d & 15, row0 = mt * kBM + 8 * piece;
        uint16_t* Y16 = static_cast<uint16_t*>(Y);
#pragma unroll 4
        for (int tl = d >> 4; tl < kTok; tl += (128 * kGroups) / 16) {
          const int tok = tt * kTok + tl;
          if (tok >= T) break;
          const uint4 v = *reinterpret_cast<const uint4*>(stage + tl * kBM + 8 * piece);
          uint16_t* dst = Y16 + (size_t)tok * ldy + row0;
          if (row0 + 8 <= n) *reinterpret_cast<uint4*>(dst) = v;
          else {
            const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
            for (int e = 0; e < 8; ++e)
              if (row0 + e < n) dst[e] = (uint16_t)(w[e >> 1] >> (16 * (e & 1)));
          }
        }
      }
    }
  }

  // The MMA thread makes sure the tensor core is done with TMEM before it is freed.  Its commit on bar_accum was
  // issued whether or not the loop above was left early, so this wait ends when the instructions issued so far
  // have completed; it keeps its own bound and ignores the abort flag.
  if (warp == 1 && lane == 0) mbar_wait(bar_accum, 0u, kGemmWaitLimit);
  tc_fence_before();
  __syncthreads();
  if (warp == 1) tmem_dealloc(tmem_d, kTmemCols);
  if (threadIdx.x == 0 && *abort_flag && dev_status) *dev_status = STB_ERR_TIMEOUT;
}

// Split-K reduction of the tiles that were computed in parts: partial tile z of split tile u is
// ws[(u ksplit + z)][token 0..ktok-1][row 0..kBM-1]; summed in z order.  y_16: 1 = bf16, 2 = fp16 output.
__global__ void gemm_reduce_kernel(const float* __restrict__ ws, int first_tile, int split_tiles, int ksplit, int ttiles, int ktok,
                                   int n, int T, void* __restrict__ Y, int y_16, size_t ldy) {
  // four consecutive rows of one token per thread: 16-byte loads of the parts, one 8- or 16-byte store
  const size_t per = (size_t)kBM * ktok, per4 = per / 4, total = (size_t)split_tiles * per4;
  const bool vec = (ldy % 4) == 0 && (reinterpret_cast<uintptr_t>(Y) & 15u) == 0;
  for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (size_t)gridDim.x * blockDim.x) {
    const size_t u = i / per4, r = (i % per4) * 4;
    const int tile = first_tile + (int)u, tt = tile % ttiles, mt = tile / ttiles;
    const int tok = tt * ktok + (int)(r / kBM), row = mt * kBM + (int)(r % kBM);
    if (tok >= T || row >= n) continue;
    float4 acc = make_float4(0.0f, 0.0f, 0.0f, 0.0f);
    for (int z = 0; z < ksplit; ++z) {
      const float4 v = __ldcs(reinterpret_cast<const float4*>(ws + (u * ksplit + z) * per + r));
      acc.x += v.x; acc.y += v.y; acc.z += v.z; acc.w += v.w;
    }
    const size_t o = (size_t)tok * ldy + row;
    if (vec && row + 4 <= n) {
      if (y_16 == 2) {
        const __half2 lo = __floats2half2_rn(acc.x, acc.y), hi = __floats2half2_rn(acc.z, acc.w);
        *reinterpret_cast<uint2*>(static_cast<__half*>(Y) + o) = make_uint2(*reinterpret_cast<const uint32_t*>(&lo), *reinterpret_cast<const uint32_t*>(&hi));
      } else if (y_16 == 1) {
        const __nv_bfloat162 lo = __floats2bfloat162_rn(acc.x, acc.y), hi = __floats2bfloat162_rn(acc.z, acc.w);
        *reinterpret_cast<uint2*>(static_cast<__nv_bfloat16*>(Y) + o) = make_uint2(*reinterpret_cast<const uint32_t*>(&lo), *reinterpret_cast<const uint32_t*>(&hi));
      } else {
        *reinterpret_cast<float4*>(static_cast<float*>(Y) + o) = acc;
      }
    } else {
      const float a4[4] = {acc.x, acc.y, acc.z, acc.w};
      for (int e = 0; e < 4 && row + e < n; ++e) {
        if (y_16 == 2) static_cast<__half*>(Y)[o + e] = __float2half_rn(a4[e]);
        else if (y_16 == 1) static_cast<__nv_bfloat16*>(Y)[o + e] = __float2bfloat16_rn(a4[e]);
        else static_cast<float*>(Y)[o + e] = a4[e];
      }
    }
  }
}

// K split: only when the output tiles alone cannot fill the 148 SMs
static int gemm_ksplit(int n, int m, int T, int ktok) {
  const int tiles = ((n + kBM - 1) / kBM) * ((T + ktok - 1) / ktok), nblk = m / kBlock;
  int ks = 1;
  if (ktok < 512) {
    // decode batch: a CTA's time is a fixed part (prologue, first loads, epilogue: measured about as long as the decode
    // of seven blocks) plus the decode of its blocks, and the call takes as many such times as it has waves of 148
    // CTAs: take the number of parts (at least four blocks each) with the smallest product
    double best = 0.0;
    for (int k = 1; k <= 16 && (k == 1 || nblk / k >= 4); ++k) {
      const long long ctas = (long long)tiles * k, waves = (ctas + 147) / 148;
      const double cost = (double)waves * (7.0 + (double)((nblk + k - 1) / k));
      if (k == 1 || cost < best - 1e-9) { best = cost; ks = k; }
    }
  } else {
    if (tiles < 100) ks = 148 / tiles;
    if (ks > 16) ks = 16;
    while (ks > 1 && nblk / ks < 4) --ks;
    if (ks < 1) ks = 1;
  }
  const int bps = (nblk + ks - 1) / ks;          // blocks per split; every split gets at least one
  return (nblk + bps - 1) / bps;
}

// How a call is laid out on the 148 SMs (one CTA per SM at a time).
//   few output tiles:   every tile is split along K (`ksplit` parts) into the workspace: mandatory
//   many output tiles:  whole waves of 148 tiles run unsplit; a small last wave (at most half the SMs) would leave
//                       the machine idle for a whole tile time, so its tiles are split along K as well, if the
//                       caller's workspace holds their partial tiles: optional
struct GemmPlan {
  int ttiles, tiles, full_tiles, split_tiles, ksplit, bps;
  size_t mandatory_bytes, preferred_bytes;
};
static GemmPlan gemm_plan(int n, int m, int T, int ktok, size_t ws_bytes, bool have_ws) {
  GemmPlan p;
  const int nblk = m / kBlock;
  p.ttiles = (T + ktok - 1) / ktok;
  p.tiles = ((n + kBM - 1) / kBM) * p.ttiles;
  const size_t per = (size_t)kBM * ktok * sizeof(float);
  const int ks = gemm_ksplit(n, m, T, ktok);
  p.full_tiles = p.tiles; p.split_tiles = 0; p.ksplit = 1; p.bps = nblk;
  p.mandatory_bytes = 0; p.preferred_bytes = 0;
  if (ks > 1) {
    p.full_tiles = 0; p.split_tiles = p.tiles; p.ksplit = ks; p.bps = (nblk + ks - 1) / ks;
    p.mandatory_bytes = p.preferred_bytes = (size_t)p.tiles * ks * per;
    return p;
  }
  const int tail = p.tiles % 148;
  if (p.tiles > 148 && tail > 0 && tail <= 74) {
    int kt = 148 / tail;
    if (kt > 16) kt = 16;
    while (kt > 1 && nblk / kt < 4) --kt;
    if (kt > 1) {
      const int bps = (nblk + kt - 1) / kt;
      kt = (nblk + bps - 1) / bps;
      p.preferred_bytes = (size_t)tail * kt * per;
      if (have_ws && ws_bytes >= p.preferred_bytes) {
        p.full_tiles = p.tiles - tail; p.split_tiles = tail; p.ksplit = kt; p.bps = bps;
      }
    }
  }
  return p;
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
static EncodeTiledFn encode_tiled_fn() {
  static EncodeTiledFn fn = nullptr;
  if (!fn) {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess && q == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(p);
  }
  return fn;
}

// Bytes of the gathered activations Xs[T][m / 4] (bf16) at the head of the workspace: room for the most residual
// slots a layer can have (32 per block), so that the size depends on the shape alone.
static size_t gemm_xs_bytes(int m, int T) { return (((size_t)T * (size_t)(m / 4) * 2u) + 255u) & ~(size_t)255u; }

// y_16: 0 = fp32 output, 1 = the 16-bit type of the activations (bf16, or fp16 with kF16)
template <int N, class Cfg, bool kF16>
static int launch_gemm(const uint8_t* packed, int n, int m, const void* X, int T, size_t ldx, void* Y, int y_16,
                       size_t ldy, void* ws, size_t ws_bytes, int* dev_status, cudaStream_t s) {
  constexpr int kBN = Cfg::kBN, kTok = Cfg::kTok;
  constexpr uint32_t kSmem = gemm_smem_bytes<Cfg>();
  const size_t xs_bytes = gemm_xs_bytes(m, T);
  if (ws && (reinterpret_cast<uintptr_t>(ws) & 255u)) return STB_ERR_ARG;
  if (!ws || ws_bytes < xs_bytes) return STB_ERR_SIZE;
  float* ws_split = reinterpret_cast<float*>(static_cast<uint8_t*>(ws) + xs_bytes);
  const GemmPlan plan = gemm_plan(n, m, T, kTok, ws_bytes - xs_bytes, true);
  if (plan.mandatory_bytes > ws_bytes - xs_bytes) return STB_ERR_SIZE;
  EncodeTiledFn enc = encode_tiled_fn();
  if (!enc) return STB_ERR_CUDA;
  const CUtensorMapDataType dt = kF16 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT16 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16;
  const cuuint32_t box_rows = (cuuint32_t)(T < kBN ? T : kBN);
  const cuuint32_t box[2] = {(cuuint32_t)kBK, box_rows};
  const cuuint32_t estr[2] = {1, 1};
  CUtensorMap map, xsmap;
  {
    const cuuint64_t dims[2] = {(cuuint64_t)m, (cuuint64_t)T};
    const cuuint64_t strides[1] = {(cuuint64_t)ldx * 2};
    if (enc(&map, dt, 2, const_cast<void*>(X), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
      return STB_ERR_ARG;
  }
  const int ldxs = m / 4;                     // a multiple of 32 elements: rows of Xs start on 64-byte boundaries
  {
    const cuuint64_t dims[2] = {(cuuint64_t)ldxs, (cuuint64_t)T};
    const cuuint64_t strides[1] = {(cuuint64_t)ldxs * 2};
    if (enc(&xsmap, dt, 2, ws, dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
      return STB_ERR_ARG;
  }
  // the shared-memory limit of a kernel is a per-device setting
  static bool attr_done[64] = {};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return STB_ERR_CUDA;
  if (dev < 0 || dev >= 64 || !attr_done[dev]) {
    if (cudaFuncSetAttribute(gemm_kernel<N, Cfg, kF16>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmem) != cudaSuccess) return STB_ERR_CUDA;
    if (dev >= 0 && dev < 64) attr_done[dev] = true;
  }
  // the gather moves 16-bit values: the same kernel serves bf16 and fp16
  gemm_gather_kernel<<<148 * 4, 256, 0, s>>>(packed, n, m, N, static_cast<const __nv_bfloat16*>(X), T, ldx,
                                             static_cast<__nv_bfloat16*>(ws), ldxs);
  if (cudaGetLastError() != cudaSuccess) return STB_ERR_CUDA;
  // The GEMM is a programmatic dependent of the gather: its CTAs may be scheduled while the gather runs (they need
  // Xs only for the residual stages at the end of their K range) and wait (griddepcontrol.wait) before they read it.
  cudaLaunchAttribute pdl[1];
  pdl[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  pdl[0].val.programmaticStreamSerializationAllowed = 1;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)(plan.full_tiles + plan.split_tiles * plan.ksplit));
  cfg.blockDim = dim3(kGemmThreads);
  cfg.dynamicSmemBytes = kSmem;
  cfg.stream = s;
  cfg.attrs = pdl; cfg.numAttrs = 1;
  if (cudaLaunchKernelEx(&cfg, gemm_kernel<N, Cfg, kF16>, map, xsmap, packed, n, m, T, Y, y_16, ldy, ws_split, plan.full_tiles,
                         plan.ksplit, plan.bps, plan.ttiles, (uint32_t)(box_rows * kBK * 2), dev_status) != cudaSuccess)
    return STB_ERR_CUDA;
  if (plan.split_tiles > 0) {
    gemm_reduce_kernel<<<148 * 4, 256, 0, s>>>(ws_split, plan.full_tiles, plan.split_tiles, plan.ksplit,
                                               plan.ttiles, kTok, n, T, Y, y_16 ? (kF16 ? 2 : 1) : 0, ldy);
    if (cudaGetLastError() != cudaSuccess) return STB_ERR_CUDA;
  }
  return STB_OK;
}

using PrefillCfg = TokCfg<2, 256>;
using BatchCfg = TokCfg<1, 64>;
// fp16 activations: up to 64 tokens take the small token tile
static int ktok_f16(int T) { return T <= BatchCfg::kTok ? BatchCfg::kTok : PrefillCfg::kTok; }

template <bool kF16>
static int launch_gemm_n(int N, const uint8_t* packed, int n, int m, const void* X, int T, size_t ldx, void* Y, int y_16,
                         size_t ldy, void* ws, size_t ws_bytes, int* dev_status, cudaStream_t s) {
  if (kF16 && T <= BatchCfg::kTok) {
    switch (N) {
      case 4: return launch_gemm<4, BatchCfg, kF16>(packed, n, m, X, T, ldx, Y, y_16, ldy, ws, ws_bytes, dev_status, s);
      case 5: return launch_gemm<5, BatchCfg, kF16>(packed, n, m, X, T, ldx, Y, y_16, ldy, ws, ws_bytes, dev_status, s);
      default: return launch_gemm<6, BatchCfg, kF16>(packed, n, m, X, T, ldx, Y, y_16, ldy, ws, ws_bytes, dev_status, s);
    }
  }
  switch (N) {
    case 4: return launch_gemm<4, PrefillCfg, kF16>(packed, n, m, X, T, ldx, Y, y_16, ldy, ws, ws_bytes, dev_status, s);
    case 5: return launch_gemm<5, PrefillCfg, kF16>(packed, n, m, X, T, ldx, Y, y_16, ldy, ws, ws_bytes, dev_status, s);
    default: return launch_gemm<6, PrefillCfg, kF16>(packed, n, m, X, T, ldx, Y, y_16, ldy, ws, ws_bytes, dev_status, s);
  }
}

}  // namespace stb

static int gemm_workspace_impl(int n, int m, int N, int T, int ktok, size_t* bytes, bool minimum) {
  if (!bytes) return STB_ERR_ARG;
  if (n < 1 || m < stb::kBlock || m % stb::kBlock != 0 || T < 1) return STB_ERR_SHAPE;
  if (N < 1 || N > 8) return STB_ERR_NM;
  const stb::GemmPlan plan = stb::gemm_plan(n, m, T, ktok, 0, false);
  *bytes = stb::gemm_xs_bytes(m, T) + (minimum ? plan.mandatory_bytes : plan.preferred_bytes);
  return STB_OK;
}

extern "C" int stb_gemm_workspace(int n, int m, int N, int T, size_t* bytes) { return gemm_workspace_impl(n, m, N, T, stb::PrefillCfg::kTok, bytes, false); }
extern "C" int stb_gemm_workspace_min(int n, int m, int N, int T, size_t* bytes) { return gemm_workspace_impl(n, m, N, T, stb::PrefillCfg::kTok, bytes, true); }
extern "C" int stb_gemm_f16_workspace(int n, int m, int N, int T, size_t* bytes) { return gemm_workspace_impl(n, m, N, T, stb::ktok_f16(T), bytes, false); }

static int gemm_check_args(const void* packed, int n, int m, int N, const void* X, int T, size_t ldx, void* Y, size_t ldy) {
  if (!packed || !X || !Y) return STB_ERR_ARG;
  if (n < 1 || m < stb::kBlock || m % stb::kBlock != 0 || T < 1) return STB_ERR_SHAPE;
  if (N < 1 || N > 8) return STB_ERR_NM;
  if (N < 4 || N > 6) return STB_ERR_UNSUPPORTED;          // the tensor-core decode covers N = 4, 5, 6
  if (ldx < (size_t)m || ldy < (size_t)n || (ldx % 8) != 0 || (reinterpret_cast<uintptr_t>(X) & 15u)) return STB_ERR_ARG;
  return STB_OK;
}

extern "C" int stb_gemm(const void* packed, int n, int m, int N, const void* X, int T, size_t ldx,
                        void* Y, stb_dtype ydt, size_t ldy, void* ws, size_t ws_bytes,
                        int* dev_status, void* stream) {
  const int rc = gemm_check_args(packed, n, m, N, X, T, ldx, Y, ldy);
  if (rc != STB_OK) return rc;
  if (ydt != STB_F32 && ydt != STB_BF16) return STB_ERR_UNSUPPORTED;
  return stb::launch_gemm_n<false>(N, static_cast<const uint8_t*>(packed), n, m, X, T, ldx, Y, ydt == STB_BF16, ldy, ws, ws_bytes,
                                   dev_status, static_cast<cudaStream_t>(stream));
}

extern "C" int stb_gemm_f16(const void* packed, int n, int m, int N, const void* X, int T, size_t ldx,
                            void* Y, stb_dtype ydt, size_t ldy, void* ws, size_t ws_bytes,
                            int* dev_status, void* stream) {
  const int rc = gemm_check_args(packed, n, m, N, X, T, ldx, Y, ldy);
  if (rc != STB_OK) return rc;
  if (ydt != STB_F32 && ydt != STB_F16) return STB_ERR_UNSUPPORTED;
  return stb::launch_gemm_n<true>(N, static_cast<const uint8_t*>(packed), n, m, X, T, ldx, Y, ydt == STB_F16, ldy, ws, ws_bytes,
                                  dev_status, static_cast<cudaStream_t>(stream));
}

// ------------------------------------------------------------------------------------------
// stb_gemm_noalloc: stb_gemm for callers that can hand over no workspace.  The gathered residual
// activations and the split-K partial sums live in a fixed array inside the library image instead of
// a caller's buffer.
namespace stb {
constexpr size_t kNoAllocScratchBytes = 8u << 20;                       // 8 MiB per device, resident until exit
static __device__ __align__(256) float g_noalloc_scratch[kNoAllocScratchBytes / sizeof(float)];
}  // namespace stb

extern "C" int stb_gemm_noalloc(const void* packed, int n, int m, int N, const void* X, int T, size_t ldx,
                                void* Y, stb_dtype ydt, size_t ldy, int* dev_status, void* stream) {
  if (!packed || !X || !Y) return STB_ERR_ARG;
  if (n < 1 || m < stb::kBlock || m % stb::kBlock != 0 || T < 1) return STB_ERR_SHAPE;
  if (N < 1 || N > 8) return STB_ERR_NM;
  if (N < 4 || N > 6) return STB_ERR_UNSUPPORTED;
  if (ydt != STB_F32 && ydt != STB_BF16) return STB_ERR_UNSUPPORTED;
  if (ldx < (size_t)m || ldy < (size_t)n || (ldx % 8) != 0 || (reinterpret_cast<uintptr_t>(X) & 15u)) return STB_ERR_ARG;
  // this shape needs the caller-workspace entry point if the scratch it cannot do without does not fit
  if (stb::gemm_xs_bytes(m, T) + stb::gemm_plan(n, m, T, stb::PrefillCfg::kTok, 0, false).mandatory_bytes > stb::kNoAllocScratchBytes) return STB_ERR_SIZE;
  // The array's name is only a host-side handle: ask the runtime for its address on the current
  // device, once per device, and give the kernels that address.
  static float* scratch_of_device[64] = {nullptr};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return STB_ERR_CUDA;
  if (!scratch_of_device[dev]) {
    float* p = nullptr;
    if (cudaGetSymbolAddress(reinterpret_cast<void**>(&p), stb::g_noalloc_scratch) != cudaSuccess || !p) return STB_ERR_CUDA;
    scratch_of_device[dev] = p;
  }
  return stb::launch_gemm_n<false>(N, static_cast<const uint8_t*>(packed), n, m, X, T, ldx, Y, ydt == STB_BF16, ldy,
                                   scratch_of_device[dev], stb::kNoAllocScratchBytes, dev_status, static_cast<cudaStream_t>(stream));
}

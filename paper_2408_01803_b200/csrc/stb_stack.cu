// stb_layer_stack_resident: a whole list of decode GEMV steps as ONE resident kernel (batch 1..8, N = 4, 5, 6).
//
// The per-layer launches of stb_layer_stack pay, for every layer, a launch ramp, a copy of the activations per
// CTA, a cluster reduction and a last wave that leaves SMs idle.  Here one CTA of 16 warps per SM stays
// resident for the whole list (cooperative launch: all CTAs are on the machine together):
//   * Consecutive steps that read the same activations (q / k / v, gate / up) form a PHASE.  The 32 x 128 tiles of
//     a phase, in (row tile, block) order, are dealt to the CTAs as contiguous ranges and a CTA's range to its 16
//     warps as equal contiguous runs.  When whole row tiles can be dealt with little imbalance (at least 85 % of
//     the SM time used) every CTA gets whole row tiles and no sum crosses CTAs; otherwise the ranges are equal
//     in tiles and a row tile may straddle CTAs.
//   * Each warp streams its tiles through a private ring in shared memory with 1-D bulk copies (mbarrier
//     completion, bounded waits) and runs ahead into its range of the NEXT phase: packed weights never depend on
//     activations, so the stream does not stop at a phase boundary.
//   * Decode and multiply per tile are those of stb_gemv: 6:8 keeps the weights in rank order and lets
//     mma.sp.m16n8k32 place them (activations from an image of x in operand order in shared memory, built once
//     per phase and CTA); 4:8 and 5:8 (and 6:8 when the image does not fit or for more than two batch rows)
//     decode to position order for mma.m16n8k16 with the activations read through L1.
//   * A step may take x = silu(in) * in2 (the gated activation between gate / up and down of an MLP): the CTA forms
//     it while it stages the activations in shared memory, in operand order (6:8, up to two batch rows) or as a
//     plain fp16 copy (everything else), and the tiles and the residual term read it from there.
//   * The residual term of the salient columns (Eq. 4) is applied per span of up to five blocks from the span's
//     records of the residual stream, brought into shared memory by one bulk copy while the span's tiles run.
//   * Partial sums: a warp that covers a whole row tile writes y itself; the others leave their head / tail
//     pieces in shared memory and the CTA adds them in tile order at the end of the phase; a row tile that
//     straddles CTAs goes through partial tiles in the caller's workspace, summed in CTA order by whichever
//     CTA arrives last (a counter per row tile).  Every sum has a fixed order: results are reproducible.
//   * A phase may read what an earlier phase wrote: a CTA starts a phase's arithmetic only when the count of
//     finished row tiles (one counter in the workspace, bumped once per CTA and phase) has reached the total
//     of all earlier phases.  The poll is bounded; when it or an mbarrier wait runs out, an abort flag makes
//     every CTA leave, STB_ERR_TIMEOUT is reported and the last CTA out restores the workspace to zero.
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/stb.h"
#include "stb_decode.cuh"
#include "stb_layout.cuh"
#include "stb_ptx.cuh"

namespace stb {

__device__ const Meta6Joint g_meta6_joint = make_meta6_joint();

constexpr int kSWarps = 16;
constexpr int kSThreads = kSWarps * 32;
constexpr int kMaxPhases = 64;                // per launch; longer lists run as several launches
constexpr int kMaxFusedSteps = 4;
constexpr int kSDepth = 2, kSChunk = 2;       // ring: slots per warp, tiles per bulk copy
static_assert(kSDepth == 2, "the warp state keeps the two slots' chunk sizes in two registers");
constexpr uint32_t kSlotBytes = 4096;         // two tiles of at most 1920 bytes
constexpr int kSpan = 5;                      // blocks per residual span
constexpr uint32_t kStageBytes = 2048;        // per warp: the span's residual records (<= 5 x 320) + its word table
constexpr uint32_t kStageTab = 1664;
constexpr long long kSWaitLimit = 2000000000ll;        // about a second of SM clocks
constexpr long long kSSelftestLimit = 100000ll;
constexpr uint32_t kImgWordsPerBlock = 96;    // 6:8 operand-order image: words per block and batch row

struct StackPhase {
  const uint8_t* packed[kMaxFusedSteps];
  void* y[kMaxFusedSteps];
  uint32_t ldy[kMaxFusedSteps];
  int32_t n[kMaxFusedSteps];
  int32_t tile_start[kMaxFusedSteps + 1];     // row tiles of the phase: step i owns [tile_start[i], tile_start[i + 1])
  const __half* x;
  const __half* x2;                           // second input of STB_IN_SILU_MUL, else null
  uint32_t ldx;
  int32_t m;
  uint8_t N, batch, count, f16_mask;          // f16_mask bit i: step i writes fp16
  uint8_t use_image, aligned, pad[2];         // use_image: 0 activations from global memory, 1 operand-order image (6:8),
                                              // 2 plain fp16 copy in shared memory; aligned: CTA ranges are whole row tiles
  uint32_t done_before;                       // row tiles finished by all earlier phases of this launch
};

struct StackParams {
  StackPhase ph[kMaxPhases];
  int32_t nphase;
  uint32_t image_bytes;                       // shared memory set aside for the staged activations
  uint32_t part_floats;                       // floats per partial slot: 32 rows x largest batch
  uint32_t max_share;                         // most CTAs that share one row tile
  uint32_t* sync;                             // [0] finished row tiles, [1] abort flag, [2] CTAs that left, [4..] per row tile arrivals
  float* gpart;                               // partial tiles of row tiles that straddle CTAs
  int* dev_status;
  long long wait_limit;
  int32_t copies_off;
};

// shared memory plan
struct SSmem {
  static constexpr uint32_t meta6 = 0;                               // joint 6:8 metadata table, 784 x 16 B, at offset 0: a pair
                                                                     // field of a tile is the shared-memory address of its entry
  static constexpr uint32_t pos = kMasks6 * kMasks6 * 16;            // 3 x 576 B position tables (N = 4, 5, 6)
  static constexpr uint32_t bars = pos + 3 * 576;                    // ring barriers: 16 warps x 2 + 16 stage barriers
  static constexpr uint32_t ctl = bars + 8 * (kSWarps * kSDepth + kSWarps);   // control words
  static constexpr uint32_t slots = ctl + 64;                        // partial slot descriptors: 32 x 16 B
  static constexpr uint32_t ring = 15360;
  static constexpr uint32_t stage = ring + kSWarps * kSDepth * kSlotBytes;
  static constexpr uint32_t pdata = stage + kSWarps * kStageBytes;
};
static_assert(SSmem::slots + 32 * 16 <= SSmem::ring && SSmem::ring % 128 == 0, "control area overflows");

struct PartSlot { int32_t R, lo, hi, pad; };   // row tile (phase-wide number) or -1, block range [lo, hi)

__device__ __forceinline__ uint32_t ld_acquire_u32(const uint32_t* p) {
  uint32_t v;
  asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ void red_release_add(uint32_t* p, uint32_t v) {
  asm volatile("red.release.gpu.global.add.u32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}
__device__ __forceinline__ unsigned long long ld_acquire_u64(const void* p) {
  unsigned long long v;
  asm volatile("ld.acquire.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(p) : "memory");
  return v;
}
// product of two fp16 pairs given and returned as bit patterns
__device__ __forceinline__ uint32_t hmul2_bits(uint32_t a, uint32_t b) {
  uint32_t d;
  asm("mul.rn.f16x2 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));
  return d;
}
// Coherent loads of activations (written by this kernel, so never through the read-only path); the address may be
// global or shared memory.
__device__ __forceinline__ uint4 ld_v4(const void* p) {
  uint4 v;
  asm volatile("ld.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ uint32_t ld_u16(const void* p) {
  unsigned short v;
  asm volatile("ld.u16 %0, [%1];" : "=h"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ uint4 ldg_v4_coherent(const void* p) {      // the same from global memory
  uint4 v;
  asm volatile("ld.global.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ uint32_t ldg_u16_coherent(const void* p) {
  unsigned short v;
  asm volatile("ld.global.u16 %0, [%1];" : "=h"(v) : "l"(p) : "memory");
  return v;
}
// fp16 pair (bits) of silu(a) * b per half, in fp32, rounded to nearest even
__device__ __forceinline__ uint32_t silu_mul_bits(uint32_t a, uint32_t b) {
  const float2 fa = __half22float2(*reinterpret_cast<const __half2*>(&a)), fb = __half22float2(*reinterpret_cast<const __half2*>(&b));
  const __half2 r = __floats2half2_rn(fa.x / (1.0f + __expf(-fa.x)) * fb.x, fa.y / (1.0f + __expf(-fa.y)) * fb.y);
  return *reinterpret_cast<const uint32_t*>(&r);
}
// the staged form of eight activations: as they are, or silu(in) * in2
__device__ __forceinline__ uint4 staged_x(const __half* x, const __half* x2, size_t off) {
  uint4 v = ldg_v4_coherent(x + off);
  if (x2) {
    const uint4 w = ldg_v4_coherent(x2 + off);
    v.x = silu_mul_bits(v.x, w.x); v.y = silu_mul_bits(v.y, w.y); v.z = silu_mul_bits(v.z, w.z); v.w = silu_mul_bits(v.w, w.w);
  }
  return v;
}
// Activation of column c (0..127) of block blk from the operand-order image of one batch row (see the image build).
__device__ __forceinline__ uint32_t image_x(const uint32_t* img_row, uint32_t blk, uint32_t c) {
  const uint32_t Gp = c >> 3, pr = (c >> 1) & 3u;
  const uint32_t* d = img_row + blk * kImgWordsPerBlock + (4u * (Gp & 1u) + ((Gp >> 2) & 1u)) * 12u + 2u * (Gp >> 3) + ((Gp >> 1) & 1u);
  const uint32_t w = d[pr < 3u ? 4u * pr : 32u];
  return (c & 1u) ? (w >> 16) : (w & 0xFFFFu);
}

// Dealing the T = R nb tiles of a phase (R row tiles of nb blocks) to G CTAs.
//   aligned:  the first Ge = min(G, R) CTAs get whole row tiles, CTA c the row tiles [c R / Ge, (c + 1) R / Ge)
//   else:     the first Ge = min(G, T) CTAs get the tiles [c T / Ge, (c + 1) T / Ge)
// (no CTA below Ge is empty); a CTA's range is cut into 16 equal runs for its warps.
__host__ __device__ __forceinline__ int dealt_ctas(int R, int nb, bool aligned, int G) {
  const long long units = aligned ? (long long)R : (long long)R * nb;
  return units < (long long)G ? (int)units : G;
}
__host__ __device__ __forceinline__ void cta_range(int R, int nb, bool aligned, int Ge, int c, int& lo, int& hi) {
  if (aligned) {
    lo = (int)((long long)R * c / Ge) * nb;
    hi = (int)((long long)R * (c + 1) / Ge) * nb;
  } else {
    const long long T = (long long)R * nb;
    lo = (int)(T * c / Ge);
    hi = (int)(T * (c + 1) / Ge);
  }
}
// the CTA that owns tile L (not aligned)
__host__ __device__ __forceinline__ int owner_of(long long L, long long T, int Ge) { return (int)(((L + 1) * Ge - 1) / T); }

__device__ __forceinline__ void warp_range(const StackPhase& q, int nb, int cta, int G, int warp, int& lo, int& hi) {
  const int R = q.tile_start[q.count];
  const int Ge = dealt_ctas(R, nb, q.aligned != 0, G);
  lo = hi = 0;
  if (cta >= Ge) return;
  int cl, ch;
  cta_range(R, nb, q.aligned != 0, Ge, cta, cl, ch);
  lo = cl + (int)(((long long)(ch - cl) * warp) >> 4);
  hi = cl + (int)(((long long)(ch - cl) * (warp + 1)) >> 4);
}
static_assert(kSWarps == 16, "warp_range divides by 16 with a shift");

__device__ __forceinline__ int step_of(const StackPhase& q, int R) {
  int i = 0;
#pragma unroll
  for (int k = 1; k < kMaxFusedSteps; ++k)
    if (k < q.count && R >= q.tile_start[k]) i = k;
  return i;
}

// The producer side of a warp's ring: a walk through the warp's tiles of all phases in chunks of up to kSChunk
// tiles that never cross a packed buffer.  Between chunks it only bumps a pointer and two counters.
struct TileWalk {
  int phase;              // current phase (== nphase: finished)
  const uint8_t* src;     // next tile
  int left_range;         // tiles left in the warp's range of this phase
  int left_step;          // tiles left in the packed buffer `src` points into
  int step;
  uint32_t tb;            // tile bytes of this phase
  __device__ void enter(const StackParams& P, int ph, int cta, int G, int warp) {
    phase = ph;
    while (phase < P.nphase) {
      const StackPhase& q = P.ph[phase];
      const int nb = q.m / kBlock;
      int lo, hi;
      warp_range(q, nb, cta, G, warp, lo, hi);
      if (lo < hi) {
        tb = tile_bytes(q.N);
        left_range = hi - lo;
        step = step_of(q, lo / nb);
        left_step = q.tile_start[step + 1] * nb - lo;
        src = q.packed[step] + tiles_offset(nb) + (size_t)(lo - q.tile_start[step] * nb) * tb;
        return;
      }
      ++phase;
    }
  }
  // next chunk: source address, bytes per tile and number of tiles (0 when the walk is over)
  __device__ int next(const StackParams& P, int cta, int G, int warp, const uint8_t*& chunk_src, uint32_t& chunk_tb) {
    if (phase >= P.nphase) return 0;
    int cnt = kSChunk;
    if (cnt > left_range) cnt = left_range;
    if (cnt > left_step) cnt = left_step;
    chunk_src = src; chunk_tb = tb;
    src += (size_t)cnt * tb;
    left_range -= cnt; left_step -= cnt;
    if (left_range == 0) enter(P, phase + 1, cta, G, warp);
    else if (left_step == 0) {
      const StackPhase& q = P.ph[phase];
      const int nb = q.m / kBlock;
      ++step;
      src = q.packed[step] + tiles_offset(nb);
      left_step = (q.tile_start[step + 1] - q.tile_start[step]) * nb;
    }
    return cnt;
  }
};

// ------------------------------------------------------------------------------------------
// One 32 x 128 tile at 6:8 through the sparse instruction, activations from the image (see stb_gemv.cu).
__device__ __forceinline__ void tile_sp6(const LaneTile<6>& lt, const uint32_t (&fld)[8], const uint8_t* smem, const uint32_t* xi0,
                                         bool xlive, float (&acc)[2][4]) {
  FastRows<6> fr;
  fr.init(lt, lt.A, lt.B);
  // Metadata: fld[4 bb + tq] is the pair field (= the address of the joint-table entry) of slot 2 h + bb of lane tq of
  // the quad, for the two rows whose metadata this lane supplies; word i of the entries, shifted to the lane's
  // nibble and added (multiply-adds: the integer pipe is the busy one), is the metadata of chunk i.
  uint32_t E[2][3];
#pragma unroll
  for (int bb = 0; bb < 2; ++bb) {
    uint4 en[4];
#pragma unroll
    for (int tq = 0; tq < 4; ++tq) en[tq] = *reinterpret_cast<const uint4*>(smem + SSmem::meta6 + fld[4 * bb + tq]);
    E[bb][0] = ((en[3].x * 16u + en[2].x) * 16u + en[1].x) * 16u + en[0].x;
    E[bb][1] = ((en[3].y * 16u + en[2].y) * 16u + en[1].y) * 16u + en[0].y;
    E[bb][2] = ((en[3].z * 16u + en[2].z) * 16u + en[1].z) * 16u + en[0].z;
  }
  // the activations of the tile's six chunk positions, once for both halves of the rows
  uint4 bxs[2][3];
#pragma unroll
  for (int sl = 0; sl < 2; ++sl)
#pragma unroll
    for (int i = 0; i < 3; ++i) {
      bxs[sl][i] = make_uint4(0, 0, 0, 0);
      if (xlive) bxs[sl][i] = *reinterpret_cast<const uint4*>(xi0 + sl * 12 + 4 * i);
    }
#pragma unroll
  for (int mt = 0; mt < 2; ++mt) {
    uint32_t XLh[2][2], XHh[2][2];
#pragma unroll
    for (int jj = 0; jj < 2; ++jj)
#pragma unroll
      for (int sp = 0; sp < 2; ++sp) fr.high(2 * mt + jj, sp, XLh[jj][sp], XHh[jj][sp]);
#pragma unroll
    for (int sl = 0; sl < 2; ++sl) {
      uint32_t R[2][2][3];
#pragma unroll
      for (int jj = 0; jj < 2; ++jj)
#pragma unroll
        for (int h = 0; h < 2; ++h) fr.pairs(2 * mt + jj, 2 * h + sl, XLh[jj][h], XHh[jj][h], R[jj][h]);
#pragma unroll
      for (int i = 0; i < 3; ++i) {
        const uint4 bx = bxs[sl][i];
        if (mt == 0) mma_sp16832<0>(acc[0], R[0][0][i], R[1][0][i], R[0][1][i], R[1][1][i], bx.x, bx.y, bx.z, bx.w, E[sl][i]);
        else mma_sp16832<1>(acc[1], R[0][0][i], R[1][0][i], R[0][1][i], R[1][1][i], bx.x, bx.y, bx.z, bx.w, E[sl][i]);
      }
    }
  }
}

// One tile in position order (N = 4, 5, 6): byte-permute decode into m16n8k16 operands; activations of batch row g
// through L1 (xrow = x + g ldx + 8 t + 128 b, or null for lanes beyond the batch).
template <int N, bool kStaged>
__device__ __forceinline__ void tile_dense(const LaneTile<N>& lt, const uint2* ptab, const __half* xrow, float (&acc)[2][4]) {
  FastRows<N> fr;
  fr.init(lt, lt.A, lt.B);
  uint32_t XL[4] = {0, 0, 0, 0}, XH[4] = {0, 0, 0, 0};
  if (N == 5) {
#pragma unroll
    for (int j = 0; j < 4; ++j) fr.high(j, 0, XL[j], XH[j]);
  }
  uint2 P[16];
#pragma unroll
  for (int u = 0; u < 16; ++u) P[u] = ptab[keep_index_of(lt.mask, u >> 2, u & 3)];
  uint4 xf[4];
#pragma unroll
  for (int s = 0; s < 4; ++s) {
    xf[s] = make_uint4(0, 0, 0, 0);
    if (xrow) xf[s] = kStaged ? ld_v4(xrow + s * 32) : ldg_v4_coherent(xrow + s * 32);
  }
#pragma unroll
  for (int s = 0; s < 4; ++s) {
    uint32_t f[4][4];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      if (N == 6 && (s & 1) == 0) fr.high(j, s >> 1, XL[j], XH[j]);
      fr.slot2(j, s, P[4 * j + s].x, P[4 * j + s].y, XL[j], XH[j], f[j]);
    }
#pragma unroll
    for (int mt = 0; mt < 2; ++mt) {
      mma16816(acc[mt], f[2 * mt][0], f[2 * mt + 1][0], f[2 * mt][1], f[2 * mt + 1][1], xf[s].x, xf[s].y);
      mma16816(acc[mt], f[2 * mt][2], f[2 * mt + 1][2], f[2 * mt][3], f[2 * mt + 1][3], xf[s].z, xf[s].w);
    }
  }
}

// ------------------------------------------------------------------------------------------
// What a warp carries through the whole kernel.
struct WarpState {
  TileWalk prod;                      // producer side of the ring
  int chunk_cnt0, chunk_cnt1;         // tiles of the chunk in ring slot 0 / 1
  uint32_t consumed;                  // chunks consumed (slot = consumed % kSDepth, barrier parity = consumed / kSDepth)
  int cur_in;                         // tile inside the current chunk
  uint32_t stage_use;                 // residual stage copies issued (barrier parity)
  bool failed;                        // a wait ran out, or the CTA was told to stop
};

struct WarpEnv {
  const StackParams* P;
  uint8_t* smem;
  uint8_t* ring;
  uint8_t* stage;
  uint32_t bar0, bar_stage;
  int cta, G, warp, lane, g, t;
};

__device__ __forceinline__ void ring_issue(const WarpEnv& E, WarpState& W, int slot) {
  const uint8_t* src = nullptr;
  uint32_t tb = 0;
  const int cnt = W.prod.next(*E.P, E.cta, E.G, E.warp, src, tb);
  if (slot == 0) W.chunk_cnt0 = cnt; else W.chunk_cnt1 = cnt;
  if (cnt > 0 && E.lane == 0) {
    const uint32_t bytes = (uint32_t)cnt * tb;
    fence_async_smem();
    mbar_expect_tx(E.bar0 + 8u * slot, bytes);
    if (!E.P->copies_off) bulk_g2s(smem_u32(E.ring + (size_t)slot * kSlotBytes), src, bytes, E.bar0 + 8u * slot);
  }
}

// The warp's tiles [lo, hi) of phase q: main stream, residual term per span, partial sums out.
// kImage: 6:8 from the operand-order image; kStaged: position order with the activations in a plain copy in shared memory
template <int N, bool kImage, bool kStaged>
__device__ __forceinline__ void run_tiles(const WarpEnv& E, WarpState& W, const StackPhase& q, int lo, int hi,
                                          const uint32_t* ximg, PartSlot* pslot, float* pdata, volatile int* ctl) {
  const StackParams& P = *E.P;
  const int lane = E.lane, g = E.g, t = E.t, warp = E.warp;
  const int nb = q.m / kBlock, batch = q.batch;
  constexpr uint32_t tb = tile_bytes(N);
  const uint2* ptab = reinterpret_cast<const uint2*>(E.smem + SSmem::pos) + (N - 4) * kPosTableEntries;
  // activations of batch row g (this lane group's): in global memory, or staged in shared memory as a plain copy
  const __half* xg = nullptr;
  if (g < batch) xg = q.use_image == 2 ? reinterpret_cast<const __half*>(ximg) + (size_t)g * q.m : q.x + (size_t)g * q.ldx;
  // (with the operand-order image the tiles read the image; the residual term takes its few activations from global
  // memory unless the input is a formed one)
  const uint32_t img_row_words = (uint32_t)nb * kImgWordsPerBlock;
  int R = lo / nb, b_first = lo - R * nb, left = hi - lo, nslot_used = 0;
  while (left > 0 && !W.failed) {
    const int seg = left < nb - b_first ? left : nb - b_first, b_end = b_first + seg;
    const int si = step_of(q, R);
    const int rt = R - q.tile_start[si];
    const uint8_t* packed = q.packed[si];
    const BlockInfo* binfo = reinterpret_cast<const BlockInfo*>(packed + sizeof(Header));
    const ResidWord* rwt = reinterpret_cast<const ResidWord*>(packed + rwtab_offset(nb));
    const int ntile = (q.n[si] + kTileRows - 1) / kTileRows;
    const uint32_t nrw_all = __ldg(&reinterpret_cast<const Header*>(packed)->nrw);
    const uint8_t* resid_rt = packed + tiles_offset(nb) + (size_t)tb * nb * ntile + (size_t)rt * resid_rt_bytes(nb, nrw_all);
    float acc[2][4];
#pragma unroll
    for (int a = 0; a < 2; ++a)
#pragma unroll
      for (int d = 0; d < 4; ++d) acc[a][d] = 0.0f;

    for (int bs = b_first; bs < b_end && !W.failed; bs += kSpan) {
      const int be = bs + kSpan < b_end ? bs + kSpan : b_end;
      // the span's records of the residual stream and its piece of the residual word table: one bulk copy each
      const uint32_t rw0 = __ldg(&binfo[bs].rw_off), rw1 = __ldg(&binfo[be - 1].rw_off) + __ldg(&binfo[be - 1].nrw);
      const uint32_t rec_bytes = (uint32_t)(be - bs) * kResidA2Bytes + (rw1 - rw0) * kResidWordBytes;
      const uint32_t tab0 = rw0 & ~1u, tab_bytes = ((rw1 - tab0) * 8u + 15u) & ~15u;       // 16-byte aligned piece of the table
      __syncwarp();
      if (lane == 0) {
        fence_async_smem();
        mbar_expect_tx(E.bar_stage, rec_bytes + (rw1 > rw0 ? tab_bytes : 0u));
        if (!P.copies_off) {
          bulk_g2s(smem_u32(E.stage), resid_rt + resid_block_off(bs, rw0), rec_bytes, E.bar_stage);
          if (rw1 > rw0) bulk_g2s(smem_u32(E.stage + kStageTab), rwt + tab0, tab_bytes, E.bar_stage);
        }
      }
      const uint32_t stage_parity = W.stage_use & 1u;
      ++W.stage_use;

      for (int b = bs; b < be; ++b) {
        const int slot = (int)(W.consumed % kSDepth);
        if (W.cur_in == 0 && !__all_sync(0xFFFFFFFFu, mbar_wait(E.bar0 + 8u * slot, (W.consumed / kSDepth) & 1u, P.wait_limit))) { W.failed = true; break; }
        const uint8_t* tile = E.ring + (size_t)slot * kSlotBytes + (size_t)W.cur_in * tb;
        const bool last_of_chunk = W.cur_in + 1 == (slot == 0 ? W.chunk_cnt0 : W.chunk_cnt1);
        LaneTile<N> lt;
        load_lane_tile<N>(tile, lane, lt, kImage);
        uint32_t fld[8] = {0, 0, 0, 0, 0, 0, 0, 0};
        if constexpr (kImage) {
#pragma unroll
          for (int k = 0; k < 8; ++k) fld[k] = *reinterpret_cast<const uint16_t*>(tile + lane * 16 + 2 * k);
        }
        if (last_of_chunk) { __syncwarp(); ring_issue(E, W, slot); W.cur_in = 0; ++W.consumed; }
        else ++W.cur_in;
        if constexpr (kImage) tile_sp6(lt, fld, E.smem, ximg + (uint32_t)g * img_row_words + (uint32_t)b * kImgWordsPerBlock + (uint32_t)(t * 24), g < batch, acc);
        else tile_dense<N, kStaged>(lt, ptab, xg ? xg + (size_t)b * kBlock + t * 8 : nullptr, acc);
      }
      if (W.failed) break;

      // residual term of the span's salient columns: four residual words (16 salient slots) per tensor-core step
      if (!__all_sync(0xFFFFFFFFu, mbar_wait(E.bar_stage, stage_parity, P.wait_limit))) { W.failed = true; break; }
      if (rw1 > rw0) {
        const uint32_t nstep = (rw1 - rw0 + 3u) >> 2;
#pragma unroll 1
        for (uint32_t i = 0; i < nstep; ++i) {
          const uint32_t wi = rw0 + 4u * i + (uint32_t)t;
          uint32_t rw = 0x55555555u, cols = 0u, block = (uint32_t)bs;
          uint2 a2 = make_uint2(0u, 0u);
          if (wi < rw1) {
            const uint2 e = *reinterpret_cast<const uint2*>(E.stage + kStageTab + (wi - tab0) * 8u);
            block = e.x >> 3; cols = e.y;
            const uint8_t* rec = E.stage + kResidA2Bytes * (block - (uint32_t)bs) + kResidWordBytes * (wi - (e.x & 7u) - rw0);
            a2 = *reinterpret_cast<const uint2*>(rec + resid_a2_off(g, 0));
            rw = *reinterpret_cast<const uint32_t*>(rec + resid_code_off(e.x & 7u, g));
          }
          // operand registers of the lane's four rows: the two-bit codes pick the high byte of +1, 0 or -1 (one byte
          // permute per row), two more spread them to fp16 pairs, and one fp16 multiply per register (not on the
          // busy integer pipe) scales them by the row's a_sal2: exact, the factors are +-1 and 0
          uint32_t fa[4][2];
          const uint32_t code_lo = rw & 0x33333333u, code_hi = (rw >> 2) & 0x33333333u;
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            const uint32_t codes = (j & 2) ? code_hi : code_lo;
            const uint32_t unit = prmt(0x00BC003Cu, 0u, (j & 1) ? (codes >> 16) : codes);          // high bytes of +1, 0, -1, 0 by code
            const uint32_t s2 = prmt((j & 2) ? a2.y : a2.x, 0u, (j & 1) ? 0x3232u : 0x1010u);     // (a_sal2, a_sal2) of row j
            fa[j][0] = hmul2_bits(prmt(unit, 0u, 0x1404u), s2);
            fa[j][1] = hmul2_bits(prmt(unit, 0u, 0x3424u), s2);
          }
          uint2 xr = make_uint2(0, 0);
          if (kImage && q.x2 != nullptr) {
            // a formed input exists only in the image: pick the four values out of its operand order
            if (g < batch) {
              const uint32_t* ir = ximg + (uint32_t)g * img_row_words;
              xr.x = image_x(ir, block, cols & 0xFFu) | (image_x(ir, block, (cols >> 8) & 0xFFu) << 16);
              xr.y = image_x(ir, block, (cols >> 16) & 0xFFu) | (image_x(ir, block, cols >> 24) << 16);
            }
          } else if (xg) {
            const __half* xq = xg + (size_t)block * kBlock;
            if constexpr (!kStaged) {      // global memory for sure
              xr.x = ldg_u16_coherent(xq + (cols & 0xFFu)) | (ldg_u16_coherent(xq + ((cols >> 8) & 0xFFu)) << 16);
              xr.y = ldg_u16_coherent(xq + ((cols >> 16) & 0xFFu)) | (ldg_u16_coherent(xq + (cols >> 24)) << 16);
            } else {                       // global memory or the plain copy in shared memory
              xr.x = ld_u16(xq + (cols & 0xFFu)) | (ld_u16(xq + ((cols >> 8) & 0xFFu)) << 16);
              xr.y = ld_u16(xq + ((cols >> 16) & 0xFFu)) | (ld_u16(xq + (cols >> 24)) << 16);
            }
          }
          mma16816(acc[0], fa[0][0], fa[1][0], fa[0][1], fa[1][1], xr.x, xr.y);
          mma16816(acc[1], fa[2][0], fa[3][0], fa[2][1], fa[3][1], xr.x, xr.y);
        }
      }
    }
    if (W.failed) break;

    // ---- the segment [b_first, b_end) of row tile R is summed: a whole row tile goes to y, a piece to shared memory ----
    if (b_first == 0 && b_end == nb) {
      const bool f16 = (q.f16_mask >> si) & 1;
#pragma unroll
      for (int mt = 0; mt < 2; ++mt)
#pragma unroll
        for (int d = 0; d < 4; ++d) {
          const int row = rt * kTileRows + g + 16 * mt + 8 * (d >> 1), bc = 2 * t + (d & 1);
          if (row < q.n[si] && bc < batch) {
            if (f16) static_cast<__half*>(q.y[si])[(size_t)bc * q.ldy[si] + row] = __float2half_rn(acc[mt][d]);
            else static_cast<float*>(q.y[si])[(size_t)bc * q.ldy[si] + row] = acc[mt][d];
          }
        }
      if (lane == 0) atomicAdd(const_cast<int*>(&ctl[1]), 1);
    } else {
      const int slot = 2 * warp + nslot_used;
      ++nslot_used;
      float* pd = pdata + (size_t)slot * P.part_floats;
#pragma unroll
      for (int mt = 0; mt < 2; ++mt)
#pragma unroll
        for (int d = 0; d < 4; ++d) {
          const int r = g + 16 * mt + 8 * (d >> 1), bc = 2 * t + (d & 1);
          if (bc < batch) pd[r * batch + bc] = acc[mt][d];
        }
      if (lane == 0) { pslot[slot].R = R; pslot[slot].lo = b_first; pslot[slot].hi = b_end; }
    }
    left -= seg; ++R; b_first = 0;
  }
}

// ------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(kSThreads, 1)
stack_kernel(const __grid_constant__ StackParams P) {
  extern __shared__ __align__(128) uint8_t smem[];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int cta = (int)blockIdx.x, G = (int)gridDim.x;
  volatile int* ctl = reinterpret_cast<volatile int*>(smem + SSmem::ctl);      // [0] failed, [1] row tiles finished by this CTA, [2] last CTA out, [3] a packed header does not match
  PartSlot* pslot = reinterpret_cast<PartSlot*>(smem + SSmem::slots);
  float* pdata = reinterpret_cast<float*>(smem + SSmem::pdata);
  uint32_t* ximg = reinterpret_cast<uint32_t*>(smem + SSmem::pdata + 32u * P.part_floats * 4u);

  // Packed headers must match the steps; every CTA reads the same headers and takes the same way out, before it
  // has touched the workspace.
  {
    if (threadIdx.x == 0) ctl[3] = 0;
    __syncthreads();
    for (int i = threadIdx.x; i < P.nphase * kMaxFusedSteps; i += blockDim.x) {
      const StackPhase& q = P.ph[i / kMaxFusedSteps];
      const int k = i % kMaxFusedSteps;
      if (k < q.count && !header_matches(reinterpret_cast<const Header*>(q.packed[k]), q.n[k], q.m, q.N)) ctl[3] = 1;
    }
    __syncthreads();
    if (ctl[3]) {
      if (threadIdx.x == 0 && cta == 0 && P.dev_status) *P.dev_status = STB_ERR_CORRUPT;
      return;
    }
  }

  // tables, barriers, control words
  for (int i = threadIdx.x; i < (int)(kMasks6 * kMasks6); i += blockDim.x)
    reinterpret_cast<uint4*>(smem + SSmem::meta6)[i] = *reinterpret_cast<const uint4*>(g_meta6_joint.v[i]);
  for (int i = threadIdx.x; i < 3 * kPosTableEntries; i += blockDim.x)
    reinterpret_cast<uint2*>(smem + SSmem::pos)[i] = g_pos_table.v[4 + i / kPosTableEntries][i % kPosTableEntries];
  WarpEnv E;
  E.P = &P; E.smem = smem; E.cta = cta; E.G = G; E.warp = warp; E.lane = lane; E.g = lane >> 2; E.t = lane & 3;
  E.bar0 = smem_u32(smem + SSmem::bars) + (uint32_t)warp * kSDepth * 8u;
  E.bar_stage = smem_u32(smem + SSmem::bars) + (uint32_t)(kSWarps * kSDepth + warp) * 8u;
  E.ring = smem + SSmem::ring + (size_t)warp * kSDepth * kSlotBytes;
  E.stage = smem + SSmem::stage + (size_t)warp * kStageBytes;
  if (lane == 0) {
    for (int i = 0; i < kSDepth; ++i) mbar_init(E.bar0 + 8u * i, 1);
    mbar_init(E.bar_stage, 1);
    fence_async_smem();
  }
  if (threadIdx.x == 0) { ctl[0] = 0; ctl[1] = 0; ctl[2] = 0; }
  __syncwarp();

  // ring: the producer walk runs kSDepth chunks ahead of the tiles the warp consumes
  WarpState W;
  W.prod.enter(P, 0, cta, G, warp);
  W.consumed = 0; W.cur_in = 0; W.stage_use = 0; W.failed = false;
#pragma unroll
  for (int i = 0; i < kSDepth; ++i) ring_issue(E, W, i);
  __syncthreads();

  for (int ph = 0; ph < P.nphase; ++ph) {
    const StackPhase& q = P.ph[ph];
    const int nb = q.m / kBlock, batch = q.batch;
    int wl, wh;
    warp_range(q, nb, cta, G, warp, wl, wh);

    // ---- wait until every earlier phase has finished, then (6:8) lay the activations out in operand order ----
    if (threadIdx.x == 0 && !ctl[0] && q.done_before > 0) {
      const long long t0 = clock64();
      for (;;) {
        // one load brings the count of finished row tiles (low word) and the abort flag (high word)
        const unsigned long long v = ld_acquire_u64(P.sync);
        if ((uint32_t)v >= q.done_before) break;
        if ((uint32_t)(v >> 32) != 0u) { ctl[0] = 1; break; }
        if (clock64() - t0 > P.wait_limit) {
          ctl[0] = 1;
          atomicExch(P.sync + 1, 1u);
          if (P.dev_status) *P.dev_status = STB_ERR_TIMEOUT;
          break;
        }
      }
    }
    __syncthreads();
    if (ctl[0]) W.failed = true;
    if (q.use_image == 1 && !ctl[0]) {
      // one item = the 8 activations of one group of one batch row: a 16-byte load, six 4-byte stores (see stb_gemv.cu)
      const uint32_t img_row_words = (uint32_t)nb * kImgWordsPerBlock;
      const int per_row = nb * 16, items = batch * per_row;
      for (int base = 0; base < items; base += 4 * kSThreads) {
        uint4 v[4];
#pragma unroll
        for (int k = 0; k < 4; ++k) {
          const int it = base + k * kSThreads + (int)threadIdx.x;
          v[k] = make_uint4(0, 0, 0, 0);
          if (it < items) {
            const int r = it >= per_row ? 1 : 0, qq = it - r * per_row;       // the image serves one or two batch rows
            v[k] = staged_x(q.x, q.x2, (size_t)r * q.ldx + (size_t)qq * 8);
          }
        }
#pragma unroll
        for (int k = 0; k < 4; ++k) {
          const int it = base + k * kSThreads + (int)threadIdx.x;
          if (it < items) {
            const int r = it >= per_row ? 1 : 0, qq = it - r * per_row, blk = qq >> 4, Gp = qq & 15;
            uint32_t* d = ximg + (uint32_t)r * img_row_words + (uint32_t)blk * kImgWordsPerBlock +
                          (uint32_t)((4 * (Gp & 1) + ((Gp >> 2) & 1)) * 12 + 2 * (Gp >> 3) + ((Gp >> 1) & 1));
            d[0] = v[k].x; d[4] = v[k].y; d[8] = v[k].z;
            d[24] = v[k].y; d[28] = v[k].z; d[32] = v[k].w;
          }
        }
      }
    } else if (q.use_image == 2 && !ctl[0]) {
      // plain fp16 copy [batch][m] of the (formed) activations
      const int per_row = q.m / 8, items = batch * per_row;
      for (int it = threadIdx.x; it < items; it += kSThreads) {
        const int r = it / per_row, qq = it - r * per_row;
        reinterpret_cast<uint4*>(ximg)[it] = staged_x(q.x, q.x2, (size_t)r * q.ldx + (size_t)qq * 8);
      }
    }
    if (lane == 0) { pslot[2 * warp].R = -1; pslot[2 * warp + 1].R = -1; }
    __syncthreads();

    // ---- this warp's tiles ----
    if (!W.failed && wl < wh) {
      if (q.N == 6 && q.use_image == 1) run_tiles<6, true, false>(E, W, q, wl, wh, ximg, pslot, pdata, ctl);
      else if (q.use_image == 2) {
        if (q.N == 6) run_tiles<6, false, true>(E, W, q, wl, wh, ximg, pslot, pdata, ctl);
        else if (q.N == 5) run_tiles<5, false, true>(E, W, q, wl, wh, ximg, pslot, pdata, ctl);
        else run_tiles<4, false, true>(E, W, q, wl, wh, ximg, pslot, pdata, ctl);
      } else if (q.N == 6) run_tiles<6, false, false>(E, W, q, wl, wh, ximg, pslot, pdata, ctl);
      else if (q.N == 5) run_tiles<5, false, false>(E, W, q, wl, wh, ximg, pslot, pdata, ctl);
      else run_tiles<4, false, false>(E, W, q, wl, wh, ximg, pslot, pdata, ctl);
    }
    if (W.failed && lane == 0 && !ctl[0]) {
      // this warp's own wait ran out: tell the CTA and the grid
      ctl[0] = 1;
      atomicExch(P.sync + 1, 1u);
      if (P.dev_status) *P.dev_status = STB_ERR_TIMEOUT;
    }
    __syncthreads();

    // ---- pieces of row tiles, added in tile order.  Slot 2 w (head piece of warp w), 2 w + 1 (tail piece) are in tile
    // order; a run of slots with the same row tile is one group, handled by the warp that owns its first slot. ----
    if (!ctl[0]) {
      const int Rall = q.tile_start[q.count];
      // every warp looks at all 32 slot descriptors at once, one per lane
      const PartSlot mine = pslot[lane];
      const uint32_t used = __ballot_sync(0xFFFFFFFFu, mine.R >= 0);
      for (int s0 = 2 * warp; s0 < 2 * warp + 2; ++s0) {
        if (!((used >> s0) & 1u)) continue;
        const int R = __shfl_sync(0xFFFFFFFFu, mine.R, s0);
        // the nearest used slot before s0 decides whether s0 starts a group
        const uint32_t below = used & ((1u << s0) - 1u);
        if (below != 0u && __shfl_sync(0xFFFFFFFFu, mine.R, 31 - __clz(below)) == R) continue;
        const uint32_t members = __ballot_sync(0xFFFFFFFFu, mine.R == R);
        const int lo_b = __shfl_sync(0xFFFFFFFFu, mine.lo, s0), hi_b = __shfl_sync(0xFFFFFFFFu, mine.hi, 31 - __clz(members));
        const int si = step_of(q, R);
        const int rt = R - q.tile_start[si];
        const bool f16 = (q.f16_mask >> si) & 1;
        const int nval = 32 * batch;                 // values of the row tile: [row][batch column]
        const bool whole = lo_b == 0 && hi_b == nb;
        float* gp = nullptr;
        int share = 1;
        if (!whole) {
          const long long T = (long long)Rall * nb;
          const int Ge = dealt_ctas(Rall, nb, false, G);
          const int c_first = owner_of((long long)R * nb, T, Ge), c_last = owner_of((long long)(R + 1) * nb - 1, T, Ge);
          share = c_last - c_first + 1;
          gp = P.gpart + ((size_t)R * P.max_share + (size_t)(cta - c_first)) * P.part_floats;
        }
        for (int v = lane; v < nval; v += 32) {
          float sum = 0.0f;
          for (uint32_t mm = members; mm != 0u; mm &= mm - 1u) sum += pdata[(size_t)(__ffs(mm) - 1) * P.part_floats + v];
          if (whole) {
            const int row = rt * kTileRows + v / batch, bc = v % batch;
            if (row < q.n[si]) {
              if (f16) static_cast<__half*>(q.y[si])[(size_t)bc * q.ldy[si] + row] = __float2half_rn(sum);
              else static_cast<float*>(q.y[si])[(size_t)bc * q.ldy[si] + row] = sum;
            }
          } else {
            gp[v] = sum;
          }
        }
        if (whole) {
          if (lane == 0) atomicAdd(const_cast<int*>(&ctl[1]), 1);
        } else {
          // the row tile straddles CTAs: whoever arrives last adds the partial tiles in CTA order
          __syncwarp();
          uint32_t old = 0;
          if (lane == 0) { __threadfence(); old = atomicAdd(P.sync + 4 + R, 1u); }
          old = __shfl_sync(0xFFFFFFFFu, old, 0);
          if ((int)old == share - 1) {
            __threadfence();
            const float* g0 = P.gpart + (size_t)R * P.max_share * P.part_floats;
            for (int v = lane; v < nval; v += 32) {
              float sum = 0.0f;
              for (int k = 0; k < share; ++k) sum += __ldcg(g0 + (size_t)k * P.part_floats + v);
              const int row = rt * kTileRows + v / batch, bc = v % batch;
              if (row < q.n[si]) {
                if (f16) static_cast<__half*>(q.y[si])[(size_t)bc * q.ldy[si] + row] = __float2half_rn(sum);
                else static_cast<float*>(q.y[si])[(size_t)bc * q.ldy[si] + row] = sum;
              }
            }
            if (lane == 0) { P.sync[4 + R] = 0u; atomicAdd(const_cast<int*>(&ctl[1]), 1); }
          }
        }
      }
    }
    __syncthreads();
    if (threadIdx.x == 0) {
      const int fin = ctl[1];
      ctl[1] = 0;
      // release at GPU scope: the CTA's stores to y (ordered before this thread by the barrier) are visible to
      // whoever sees the count
      if (fin > 0 && !ctl[0]) red_release_add(P.sync, (uint32_t)fin);
    }
  }

  // ---- leaving: let copies in flight land, then the last CTA out restores the workspace ----
  if (ctl[0] || W.failed) {
    const long long t0 = clock64();
    while (clock64() - t0 < 200000) {}
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    __threadfence();
    const uint32_t old = atomicAdd(P.sync + 2, 1u);
    ctl[2] = (old == (uint32_t)G - 1u) ? 1 : 0;
  }
  __syncthreads();
  if (ctl[2]) {
    __threadfence();
    const bool aborted = ld_acquire_u32(P.sync + 1) != 0u;
    if (aborted) {
      int maxR = 0;
      for (int ph = 0; ph < P.nphase; ++ph) maxR = max(maxR, P.ph[ph].tile_start[P.ph[ph].count]);
      for (int i = threadIdx.x; i < maxR; i += blockDim.x) P.sync[4 + i] = 0u;
    }
    __syncthreads();
    if (threadIdx.x == 0) { P.sync[0] = 0u; P.sync[1] = 0u; P.sync[2] = 0u; __threadfence(); }
  }
}

// ------------------------------------------------------------------------------------------
// stb_layer_stack_checksum: XOR of all 32-bit words of the tiles and residual streams of every step's packed layer
// (an integrity check for packed layers that were stored or moved).  It walks the layers exactly as stack_kernel
// does -- same dealing, same per-warp rings and bulk copies, same residual-span copies -- and folds the words
// instead of decoding them, so its rate is also the rate this way of streaming reaches with no arithmetic behind it.
__global__ void __launch_bounds__(kSThreads, 1)
checksum_kernel(const __grid_constant__ StackParams P, unsigned long long* __restrict__ sums, int first_step) {
  extern __shared__ __align__(128) uint8_t smem[];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int cta = (int)blockIdx.x, G = (int)gridDim.x;
  WarpEnv E;
  E.P = &P; E.smem = smem; E.cta = cta; E.G = G; E.warp = warp; E.lane = lane; E.g = lane >> 2; E.t = lane & 3;
  E.bar0 = smem_u32(smem + SSmem::bars) + (uint32_t)warp * kSDepth * 8u;
  E.bar_stage = smem_u32(smem + SSmem::bars) + (uint32_t)(kSWarps * kSDepth + warp) * 8u;
  E.ring = smem + SSmem::ring + (size_t)warp * kSDepth * kSlotBytes;
  E.stage = smem + SSmem::stage + (size_t)warp * kStageBytes;
  if (lane == 0) {
    for (int i = 0; i < kSDepth; ++i) mbar_init(E.bar0 + 8u * i, 1);
    mbar_init(E.bar_stage, 1);
    fence_async_smem();
  }
  __syncwarp();
  WarpState W;
  W.prod.enter(P, 0, cta, G, warp);
  W.consumed = 0; W.cur_in = 0; W.stage_use = 0; W.failed = false;
#pragma unroll
  for (int i = 0; i < kSDepth; ++i) ring_issue(E, W, i);

  int step_base = first_step;                    // index, in the caller's list, of the phase's first step
  for (int ph = 0; ph < P.nphase && !W.failed; ++ph) {
    const StackPhase& q = P.ph[ph];
    const int nb = q.m / kBlock;
    const uint32_t tb = tile_bytes(q.N);
    int lo, hi;
    warp_range(q, nb, cta, G, warp, lo, hi);
    int R = lo / nb, b_first = lo - R * nb, left = hi - lo;
    while (left > 0 && !W.failed) {
      const int seg = left < nb - b_first ? left : nb - b_first, b_end = b_first + seg;
      const int si = step_of(q, R), rt = R - q.tile_start[si];
      const uint8_t* packed = q.packed[si];
      const BlockInfo* binfo = reinterpret_cast<const BlockInfo*>(packed + sizeof(Header));
      const ResidWord* rwt = reinterpret_cast<const ResidWord*>(packed + rwtab_offset(nb));
      const int ntile = (q.n[si] + kTileRows - 1) / kTileRows;
      const uint32_t nrw_all = __ldg(&reinterpret_cast<const Header*>(packed)->nrw);
      const uint8_t* resid_rt = packed + tiles_offset(nb) + (size_t)tb * nb * ntile + (size_t)rt * resid_rt_bytes(nb, nrw_all);
      uint32_t fold = 0;
      for (int bs = b_first; bs < b_end && !W.failed; bs += kSpan) {
        const int be = bs + kSpan < b_end ? bs + kSpan : b_end;
        const uint32_t rw0 = __ldg(&binfo[bs].rw_off), rw1 = __ldg(&binfo[be - 1].rw_off) + __ldg(&binfo[be - 1].nrw);
        const uint32_t rec_bytes = (uint32_t)(be - bs) * kResidA2Bytes + (rw1 - rw0) * kResidWordBytes;
        const uint32_t tab0 = rw0 & ~1u, tab_bytes = ((rw1 - tab0) * 8u + 15u) & ~15u;
        __syncwarp();
        if (lane == 0) {
          fence_async_smem();
          mbar_expect_tx(E.bar_stage, rec_bytes + (rw1 > rw0 ? tab_bytes : 0u));
          bulk_g2s(smem_u32(E.stage), resid_rt + resid_block_off(bs, rw0), rec_bytes, E.bar_stage);
          if (rw1 > rw0) bulk_g2s(smem_u32(E.stage + kStageTab), rwt + tab0, tab_bytes, E.bar_stage);
        }
        const uint32_t stage_parity = W.stage_use & 1u;
        ++W.stage_use;
        for (int b = bs; b < be; ++b) {
          const int slot = (int)(W.consumed % kSDepth);
          if (W.cur_in == 0 && !__all_sync(0xFFFFFFFFu, mbar_wait(E.bar0 + 8u * slot, (W.consumed / kSDepth) & 1u, P.wait_limit))) { W.failed = true; break; }
          const uint8_t* tile = E.ring + (size_t)slot * kSlotBytes + (size_t)W.cur_in * tb;
          const bool last_of_chunk = W.cur_in + 1 == (slot == 0 ? W.chunk_cnt0 : W.chunk_cnt1);
          for (uint32_t o = (uint32_t)lane * 4u; o < tb; o += 128u) fold ^= *reinterpret_cast<const uint32_t*>(tile + o);
          if (last_of_chunk) { __syncwarp(); ring_issue(E, W, slot); W.cur_in = 0; ++W.consumed; }
          else ++W.cur_in;
        }
        if (W.failed) break;
        if (!__all_sync(0xFFFFFFFFu, mbar_wait(E.bar_stage, stage_parity, P.wait_limit))) { W.failed = true; break; }
        for (uint32_t o = (uint32_t)lane * 4u; o < rec_bytes; o += 128u) fold ^= *reinterpret_cast<const uint32_t*>(E.stage + o);
      }
      // words of one step only ever meet words of the same step
#pragma unroll
      for (int d = 16; d > 0; d >>= 1) fold ^= __shfl_xor_sync(0xFFFFFFFFu, fold, d);
      if (lane == 0 && !W.failed) atomicXor(sums + step_base + si, (unsigned long long)fold);
      left -= seg; ++R; b_first = 0;
    }
    step_base += q.count;
  }
  if (W.failed) {
    const long long t0 = clock64();
    while (clock64() - t0 < 200000) {}
    if (lane == 0 && P.dev_status) *P.dev_status = STB_ERR_TIMEOUT;
  }
}

// ------------------------------------------------------------------------------------------
// Host side: steps -> phases -> launches.
struct StackPlan {
  size_t sync_bytes, gpart_bytes;
};

static bool same_input(const stb_step& a, const stb_step& b) {
  return a.in == b.in && a.in2 == b.in2 && a.input == b.input && a.ldin == b.ldin && a.batch == b.batch && a.m == b.m &&
         a.N == b.N && b.out != a.in && b.out != a.in2;
}

static int check_step(const stb_step& s) {
  if (!s.packed || !s.in || !s.out) return STB_ERR_ARG;
  if (s.n < 1 || s.m < kBlock || s.m % kBlock != 0) return STB_ERR_SHAPE;
  if (s.N < 1 || s.N > 8) return STB_ERR_NM;
  if (s.N < 4 || s.N > 6) return STB_ERR_UNSUPPORTED;
  if (s.batch < 1 || s.batch > 64) return STB_ERR_SIZE;
  if (s.batch > 8) return STB_ERR_UNSUPPORTED;
  if (s.odt != STB_F32 && s.odt != STB_F16) return STB_ERR_UNSUPPORTED;
  if (s.ldin < (size_t)s.m || s.ldout < (size_t)s.n || (s.ldin % 8) != 0 || (reinterpret_cast<uintptr_t>(s.in) & 15u)) return STB_ERR_ARG;
  if (s.ldin > 0xFFFFFFFFull || s.ldout > 0xFFFFFFFFull) return STB_ERR_ARG;
  if (s.input != STB_IN_PLAIN && s.input != STB_IN_SILU_MUL) return STB_ERR_ARG;
  if (s.input == STB_IN_SILU_MUL && (!s.in2 || (reinterpret_cast<uintptr_t>(s.in2) & 15u))) return STB_ERR_ARG;
  return STB_OK;
}

// Whole row tiles per CTA when that keeps at least 85 % of the SM time busy: R row tiles on G CTAs take
// ceil(R / G) rounds of which R / G are needed.
static bool deal_aligned(long long R, int G) {
  const long long rounds = (R + G - 1) / G;
  return (double)R / (double)G >= 0.85 * (double)rounds;
}

// most CTAs that share one row tile of a phase of R row tiles x nb blocks dealt to G CTAs by equal tile counts
static uint32_t max_share_of(long long R, int nb, int G) {
  const long long T = R * nb;
  const int Ge = dealt_ctas((int)R, nb, false, G);
  uint32_t best = 1;
  for (long long r = 0; r < R; ++r) {
    const int c0 = owner_of(r * nb, T, Ge), c1 = owner_of((r + 1) * nb - 1, T, Ge);
    const uint32_t s = (uint32_t)(c1 - c0 + 1);
    if (s > best) best = s;
  }
  return best;
}

static int stack_sm_count(int* out) {
  static int cached[64] = {};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return STB_ERR_CUDA;
  if (dev < 0 || dev >= 64) return STB_ERR_CUDA;
  if (!cached[dev]) {
    int v = 0;
    if (cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || v < 1) return STB_ERR_CUDA;
    cached[dev] = v;
  }
  *out = cached[dev];
  return STB_OK;
}

constexpr uint32_t kSmemLimit = 227 * 1024;

// Builds the phases of steps [i0, ...) into `sp` (at most kMaxPhases), returns the index of the first step not taken.
static int build_phases(const stb_step* steps, int count, int i0, int G, StackParams& sp, size_t& sync_need, size_t& gpart_need) {
  sp.nphase = 0;
  sp.image_bytes = 0; sp.part_floats = 32; sp.max_share = 1;
  uint32_t done = 0;
  long long maxR = 0;
  int i = i0;
  // first pass: phases and the largest batch (the partial slots are sized by it)
  while (i < count && sp.nphase < kMaxPhases) {
    StackPhase& q = sp.ph[sp.nphase];
    const stb_step& st = steps[i];
    int j = i + 1;
    while (j < count && j - i < kMaxFusedSteps && same_input(st, steps[j])) ++j;
    q.count = (uint8_t)(j - i);
    q.tile_start[0] = 0;
    q.f16_mask = 0;
    for (int k = 0; k < kMaxFusedSteps; ++k) { q.packed[k] = nullptr; q.y[k] = nullptr; q.ldy[k] = 0; q.n[k] = 0; q.tile_start[k + 1] = 0; }
    for (int k = i; k < j; ++k) {
      const stb_step& sk = steps[k];
      q.packed[k - i] = static_cast<const uint8_t*>(sk.packed);
      q.y[k - i] = sk.out; q.ldy[k - i] = (uint32_t)sk.ldout; q.n[k - i] = sk.n;
      if (sk.odt == STB_F16) q.f16_mask |= (uint8_t)(1u << (k - i));
      q.tile_start[k - i + 1] = q.tile_start[k - i] + (sk.n + kTileRows - 1) / kTileRows;
    }
    for (int k = q.count; k < kMaxFusedSteps; ++k) q.tile_start[k + 1] = q.tile_start[q.count];
    q.x = static_cast<const __half*>(st.in);
    q.x2 = st.input == STB_IN_SILU_MUL ? static_cast<const __half*>(st.in2) : nullptr;
    q.ldx = (uint32_t)st.ldin; q.m = st.m; q.N = (uint8_t)st.N; q.batch = (uint8_t)st.batch;
    q.use_image = 0; q.pad[0] = q.pad[1] = 0;
    q.done_before = done;
    const long long R = q.tile_start[q.count];
    done += (uint32_t)R;
    if (R > maxR) maxR = R;
    if ((uint32_t)(32 * st.batch) > sp.part_floats) sp.part_floats = (uint32_t)(32 * st.batch);
    q.aligned = deal_aligned(R, G) ? 1 : 0;
    const uint32_t share = q.aligned ? 1u : max_share_of(R, st.m / kBlock, G);
    if (share > sp.max_share) sp.max_share = share;
    ++sp.nphase;
    i = j;
  }
  // second pass: where each phase takes its activations from.  6:8 with up to two batch rows: the operand-order
  // image in shared memory if it fits; a formed input (silu(in) * in2) must be staged: image or plain copy.
  const uint32_t fixed = SSmem::pdata + 32u * sp.part_floats * 4u;
  for (int p = 0; p < sp.nphase; ++p) {
    StackPhase& q = sp.ph[p];
    const uint32_t img = (uint32_t)q.batch * (uint32_t)(q.m / kBlock) * kImgWordsPerBlock * 4u;
    const uint32_t plain = (uint32_t)q.batch * (uint32_t)q.m * 2u;
    uint32_t need = 0;
    if (q.N == 6 && q.batch <= 2 && fixed + img <= kSmemLimit) { q.use_image = 1; need = img; }
    else if (q.x2) {
      if (fixed + plain > kSmemLimit) return -1;          // the formed input does not fit shared memory
      q.use_image = 2; need = plain;
    }
    if (need > sp.image_bytes) sp.image_bytes = need;
  }
  const size_t s_need = (size_t)(4 + maxR) * sizeof(uint32_t);
  const size_t g_need = (size_t)maxR * sp.max_share * sp.part_floats * sizeof(float);
  if (s_need > sync_need) sync_need = s_need;
  if (g_need > gpart_need) gpart_need = g_need;
  return i;
}

static size_t align256(size_t v) { return (v + 255) & ~(size_t)255; }

}  // namespace stb

extern "C" int stb_layer_stack_resident_workspace(const stb_step* steps, int count, size_t* bytes) {
  if (!steps || count < 1 || !bytes) return STB_ERR_ARG;
  for (int i = 0; i < count; ++i) {
    const int rc = stb::check_step(steps[i]);
    if (rc != STB_OK) return rc;
  }
  int G = 0;
  int rc = stb::stack_sm_count(&G);
  if (rc != STB_OK) return rc;
  size_t sync_need = 0, gpart_need = 0;
  static thread_local stb::StackParams sp;
  int i = 0;
  while (i < count) {
    i = stb::build_phases(steps, count, i, G, sp, sync_need, gpart_need);
    if (i < 0) return STB_ERR_UNSUPPORTED;
  }
  *bytes = stb::align256(sync_need) + stb::align256(gpart_need);
  return STB_OK;
}

static int stack_resident_impl(const stb_step* steps, int count, void* ws, size_t ws_bytes, int* dev_status, void* stream,
                               bool selftest) {
  if (!steps || count < 1 || !ws) return STB_ERR_ARG;
  if (reinterpret_cast<uintptr_t>(ws) & 255u) return STB_ERR_ARG;
  for (int i = 0; i < count; ++i) {
    const int rc = stb::check_step(steps[i]);
    if (rc != STB_OK) return rc;
  }
  int G = 0;
  int rc = stb::stack_sm_count(&G);
  if (rc != STB_OK) return rc;
  // the whole list must fit the workspace before anything is launched
  size_t sync_need = 0, gpart_need = 0;
  static thread_local stb::StackParams sp;
  {
    int i = 0;
    while (i < count) {
      i = stb::build_phases(steps, count, i, G, sp, sync_need, gpart_need);
      if (i < 0) return STB_ERR_UNSUPPORTED;
    }
  }
  const size_t sync_bytes = stb::align256(sync_need);
  if (ws_bytes < sync_bytes + stb::align256(gpart_need)) return STB_ERR_SIZE;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  static bool attr_done[64] = {};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return STB_ERR_CUDA;
  if (!attr_done[dev]) {
    if (cudaFuncSetAttribute(stb::stack_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)stb::kSmemLimit) != cudaSuccess) return STB_ERR_CUDA;
    attr_done[dev] = true;
  }
  int i = 0;
  while (i < count) {
    size_t a = 0, b = 0;
    i = stb::build_phases(steps, count, i, G, sp, a, b);
    if (i < 0) return STB_ERR_UNSUPPORTED;
    sp.sync = static_cast<uint32_t*>(ws);
    sp.gpart = reinterpret_cast<float*>(static_cast<uint8_t*>(ws) + sync_bytes);
    sp.dev_status = dev_status;
    sp.wait_limit = selftest ? stb::kSSelftestLimit : stb::kSWaitLimit;
    sp.copies_off = selftest ? 1 : 0;
    const uint32_t smem = stb::SSmem::pdata + 32u * sp.part_floats * 4u + sp.image_bytes;
    if (smem > stb::kSmemLimit) return STB_ERR_UNSUPPORTED;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)G, 1, 1);
    cfg.blockDim = dim3((unsigned)stb::kSThreads, 1, 1);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = s;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeCooperative;
    at[0].val.cooperative = 1;
    cfg.attrs = at; cfg.numAttrs = 1;
    if (cudaLaunchKernelEx(&cfg, stb::stack_kernel, sp) != cudaSuccess) return STB_ERR_CUDA;
  }
  return STB_OK;
}

extern "C" int stb_layer_stack_resident(const stb_step* steps, int count, void* ws, size_t ws_bytes, int* dev_status,
                                        void* stream) {
  return stack_resident_impl(steps, count, ws, ws_bytes, dev_status, stream, false);
}

extern "C" int stb_layer_stack_resident_wait_selftest(const stb_step* steps, int count, void* ws, size_t ws_bytes,
                                                      int* dev_status, void* stream) {
  if (!dev_status) return STB_ERR_ARG;
  return stack_resident_impl(steps, count, ws, ws_bytes, dev_status, stream, true);
}

extern "C" int stb_layer_stack_resident_host(const stb_step* steps, int count, void* ws, size_t ws_bytes, const void* in_host,
                                             size_t in_bytes, void* out_host, size_t out_bytes, int* dev_status, void* stream) {
  if (!steps || count < 1 || !in_host || !out_host || !steps[0].in || !steps[count - 1].out) return STB_ERR_ARG;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  if (cudaMemcpyAsync(const_cast<void*>(steps[0].in), in_host, in_bytes, cudaMemcpyHostToDevice, s) != cudaSuccess)
    return STB_ERR_CUDA;
  const int rc = stb_layer_stack_resident(steps, count, ws, ws_bytes, dev_status, stream);
  if (rc != STB_OK) return rc;
  if (cudaMemcpyAsync(out_host, steps[count - 1].out, out_bytes, cudaMemcpyDeviceToHost, s) != cudaSuccess)
    return STB_ERR_CUDA;
  return STB_OK;
}

extern "C" int stb_layer_stack_checksum(const stb_step* steps, int count, unsigned long long* sums, int* dev_status, void* stream) {
  if (!steps || count < 1 || !sums) return STB_ERR_ARG;
  for (int i = 0; i < count; ++i) {
    const int rc = stb::check_step(steps[i]);
    if (rc != STB_OK) return rc;
  }
  int G = 0;
  int rc = stb::stack_sm_count(&G);
  if (rc != STB_OK) return rc;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  static bool attr_done[64] = {};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return STB_ERR_CUDA;
  if (!attr_done[dev]) {
    if (cudaFuncSetAttribute(stb::checksum_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)stb::kSmemLimit) != cudaSuccess) return STB_ERR_CUDA;
    attr_done[dev] = true;
  }
  if (cudaMemsetAsync(sums, 0, sizeof(unsigned long long) * (size_t)count, s) != cudaSuccess) return STB_ERR_CUDA;
  static thread_local stb::StackParams sp;
  int i = 0;
  while (i < count) {
    size_t a = 0, b = 0;
    const int first = i;
    i = stb::build_phases(steps, count, i, G, sp, a, b);
    if (i < 0) return STB_ERR_UNSUPPORTED;
    sp.sync = nullptr; sp.gpart = nullptr; sp.dev_status = dev_status;
    sp.wait_limit = stb::kSWaitLimit; sp.copies_off = 0;
    // the same shared-memory footprint as the arithmetic kernel would have for these steps
    const uint32_t smem = stb::SSmem::pdata + 32u * sp.part_floats * 4u + sp.image_bytes;
    stb::checksum_kernel<<<(unsigned)G, stb::kSThreads, smem, s>>>(sp, sums, first);
    if (cudaGetLastError() != cudaSuccess) return STB_ERR_CUDA;
  }
  return STB_OK;
}

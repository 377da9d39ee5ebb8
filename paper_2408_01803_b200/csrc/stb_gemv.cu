// stb_gemv: decode GEMV  y[t][i] = sum_j W^[i][j] x[t][j],  batch 1..64, fp32 accumulation.
// The memory-bound decoding stage of Appendix C.2: every packed byte is read once.
#include <cooperative_groups.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/stb.h"
#include "stb_decode.cuh"
#include "stb_layout.cuh"
#include "stb_ptx.cuh"

namespace cg = cooperative_groups;

namespace stb {

__device__ const Meta6Table g_meta6 = make_meta6_table();

// ------------------------------------------------------------------------------------------
// Tensor-core GEMV, N = 4, 5, 6, batch <= 8 NB (NB = 1, 2, 4, 8).
//
// Grid: one thread-block cluster of `ksplit` CTAs per row tile (32 rows); CTA k of the cluster
// takes the k-th slice of the 128-column blocks and its warps take contiguous runs of that
// slice.  Each warp streams its tiles from HBM into a private ring in shared memory with 1-D
// bulk copies (kChunk tiles per copy, kDepth copies in flight), reads a tile into registers,
// decodes it into fp16 operand registers (stb_decode.cuh) and multiplies on the tensor cores,
// fp32 accumulators in registers for the whole run:
//   N = 4, 5, and N = 6 beyond 8 batch rows: position-order decode, m16n8k16 (A = 16 rows x 16
//     columns of W^, B = the activations of 8 batch rows read through L1);
//   N = 6 up to 8 batch rows: the weights stay in rank order and the 2:4 sparse instruction
//     (m16n8k32) places them: every pair of kept weights is a 2-of-4 selection from a window of
//     four columns, three overlapping windows per group of 8 (stb_decode.cuh, meta6_nibble);
//     the activations are read three halves wide, for up to two batch rows from a copy of the
//     CTA's slice that is laid out in operand order in shared memory once per CTA.
// The residual term of the salient columns goes through the dense instruction with the salient
// slots of 16 / SPB blocks as its K dimension, after the weight stream.  Partial sums: warps
// through shared memory, CTAs of the cluster through distributed shared memory, both in a fixed
// order.
constexpr int kDepth = 2;     // ring slots per warp
constexpr int kChunk = 2;     // tiles per bulk copy (consecutive blocks of a row tile are contiguous)
constexpr long long kWaitLimit = 2000000000ll;     // about a second of SM clocks
constexpr long long kSelftestWaitLimit = 100000ll;  // the wait self-test gives up after about 50 microseconds

struct GemvSmem {
  uint32_t bars, ring, part, ximg, total;           // byte offsets
  uint32_t tile_stride;
};
// N = 6, up to two batch rows: the CTA's slice of the activations is kept in shared memory in the order the lanes
// consume it: per block and batch row 96 words, word ((t * 2 + sl) * 3 + i) * 4 + u = operand register u of chunk i
// of step sl of lane t (two fp16 each).
constexpr uint32_t kImgWords = 96;
constexpr uint32_t kImgMaxBytes = 20 * 1024;
__host__ __device__ inline uint32_t gemv_image_bytes(int N, int NB, int batch, int bpp) {
  const uint32_t bytes = (uint32_t)batch * (uint32_t)bpp * kImgWords * 4u;
  return (N == 6 && NB == 1 && batch <= 2 && bytes <= kImgMaxBytes) ? bytes : 0u;
}
__host__ __device__ inline GemvSmem gemv_smem(int N, int warps, int ksplit, int NB, uint32_t image_bytes) {
  GemvSmem s;
  s.bars = kPosTableEntries * 8;                     // the position table comes first
  s.ring = (s.bars + (uint32_t)(warps * kDepth * 8) + 127u) & ~127u;
  s.tile_stride = (kChunk * tile_bytes(N) + 127u) & ~127u;      // one ring slot = one chunk of tiles
  // the ring is reused for the per-warp partial sums (warps x 32 rows x 8 NB floats) after the main loop
  const uint32_t ring_bytes = (uint32_t)(warps * kDepth) * s.tile_stride, red_bytes = (uint32_t)warps * 32u * 8u * (uint32_t)NB * 4u;
  s.part = s.ring + (ring_bytes > red_bytes ? ring_bytes : red_bytes);
  s.ximg = s.part + (uint32_t)ksplit * 32u * 8u * (uint32_t)NB * 4u;
  s.total = s.ximg + image_bytes;
  return s;
}

__device__ __forceinline__ int ilog2(int v) { return 31 - __clz(v); }

// Up to kMaxFused layers that read the same activations (q / k / v, gate / up) run as one grid:
// row tiles [tile_start[i], tile_start[i + 1]) of the grid belong to layer i.
constexpr int kMaxFused = 4;
struct GemvLayers {
  const uint8_t* packed[kMaxFused];
  void* y[kMaxFused];
  size_t ldy[kMaxFused];
  int n[kMaxFused];
  int y_f16[kMaxFused];
  int tile_start[kMaxFused + 1];
  int count;
};

// At most 128 threads per CTA, four CTAs per SM for up to 16 batch rows (a bound of five CTAs, 96
// registers, was measured slower: the spills cost more than the extra resident CTA brings).
constexpr int kGemvMaxThreads = 128;
constexpr int kMaxDevices = 64;
template <int N, int NB>
__global__ void __launch_bounds__(kGemvMaxThreads, NB <= 2 ? 4 : 1)
gemv_mma_kernel(const __grid_constant__ GemvLayers layers, int m, const __half* __restrict__ x, int batch,
                size_t ldx, int* dev_status, int lg_ksplit, int bpp, long long wait_limit, int copies_off) {
  extern __shared__ __align__(128) uint8_t smem[];
  int li = 0, rt_all = (int)(blockIdx.x >> lg_ksplit);
#pragma unroll
  for (int i = 1; i < kMaxFused; ++i)
    if (i < layers.count && rt_all >= layers.tile_start[i]) li = i;
  const uint8_t* __restrict__ packed = layers.packed[li];
  void* __restrict__ y = layers.y[li];
  const size_t ldy = layers.ldy[li];
  const int n = layers.n[li], y_f16 = layers.y_f16[li];
  const Header* hdr = reinterpret_cast<const Header*>(packed);
  // every CTA of a cluster takes the same branch here (the header is the same for all)
  if (!header_matches(hdr, n, m, N)) {
    if (threadIdx.x == 0 && dev_status) *dev_status = STB_ERR_CORRUPT;
    return;
  }
  const int nblk = m / kBlock;
  const int ksplit = 1 << lg_ksplit;
  // A CTA may write into the shared memory of another CTA of its cluster only once that CTA runs: every CTA
  // arrives here, and waits for the others just before its first remote store (behind the whole weight stream).
  if (ksplit > 1) cluster_arrive();
  const int warps = (int)(blockDim.x >> 5);
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, g = lane >> 2, t = lane & 3;
  const int kpart = (int)(blockIdx.x & (unsigned)(ksplit - 1)), rt = rt_all - layers.tile_start[li];
  const int b0 = kpart * bpp, b1 = min(nblk, b0 + bpp);
  const int nbp = max(b1 - b0, 0);
  const BlockInfo* binfo = reinterpret_cast<const BlockInfo*>(packed + sizeof(Header));
  constexpr uint32_t tbytes = tile_bytes(N);
  const uint8_t* rtbase = packed + hdr->tiles_offset + (size_t)rt * hdr->rt_stride;
  const uint8_t* resid_rt = packed + hdr->tiles_offset + hdr->rt_stride * (size_t)hdr->ntile +
                            (size_t)rt * resid_rt_bytes(nblk, hdr->nrw);
  const uint32_t image_bytes = gemv_image_bytes(N, NB, batch, bpp);
  const GemvSmem L = gemv_smem(N, warps, ksplit, NB, image_bytes);

  const uint2* ptab = reinterpret_cast<const uint2*>(smem);
  uint8_t* ring = smem + L.ring + (size_t)warp * kDepth * L.tile_stride;
  const uint32_t bar0 = smem_u32(smem + L.bars) + (uint32_t)warp * kDepth * 8u;

  // this warp's run of blocks
  const int per = (nbp + warps - 1) / warps;
  const int wb0 = b0 + warp * per, wb1 = min(b1, wb0 + per);
  const int cnt = max(wb1 - wb0, 0);

  // Start the weight stream before anything else.  The packed layer is never written by a GEMV,
  // so under a programmatic dependent launch this may run while the previous layer still computes.
  if (lane == 0) {
    for (int i = 0; i < kDepth; ++i) mbar_init(bar0 + 8u * i, 1);
    fence_async_smem();
    for (int i = 0; i < kDepth && i * kChunk < cnt; ++i) {
      const uint32_t bytes = (uint32_t)min(kChunk, cnt - i * kChunk) * tbytes;
      mbar_expect_tx(bar0 + 8u * i, bytes);
      // copies_off (the wait self-test): the barrier is armed but nothing will ever complete it
      if (!copies_off) bulk_g2s(smem_u32(ring + (size_t)i * L.tile_stride), rtbase + (size_t)(wb0 + i * kChunk) * tbytes, bytes, bar0 + 8u * i);
    }
  }
  if (N == 6 && NB == 1) {   // metadata by keep-mask index (256 bytes: an index byte of the tile cannot point past it)
    for (int i = threadIdx.x; i < kMeta6Entries; i += blockDim.x) reinterpret_cast<uint32_t*>(smem)[i] = g_meta6.v[i];
  } else {
    for (int i = threadIdx.x; i < kPosTableEntries; i += blockDim.x) reinterpret_cast<uint2*>(smem)[i] = g_pos_table.v[N][i];
  }

  // Everything below reads the activations (the previous layer's output) or writes y: wait for the
  // previous grid of the stream to have completed (no-op without a programmatic launch), then let
  // the next grid start its own weight stream.
  grid_dependency_wait();
  grid_launch_dependents();
  x = after_dependency_wait(x);
  const uint32_t* ximg = reinterpret_cast<const uint32_t*>(smem + L.ximg);
  const uint32_t img_row_words = (uint32_t)bpp * kImgWords;
  if (N == 6 && NB == 1 && image_bytes != 0u) {
    // one item = the 8 activations of one group of one block of one batch row: a 16-byte load, six 4-byte stores
    // (lanes t = 2 (G & 1) + p read word i + p of group G as chunk i: words 0..2 for p = 0, words 1..3 for p = 1)
    uint32_t* img = reinterpret_cast<uint32_t*>(smem + L.ximg);
    const int items = batch * nbp * 16;
    for (int base = 0; base < items; base += 4 * (int)blockDim.x) {
      uint4 v[4];
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        const int it = base + k * (int)blockDim.x + (int)threadIdx.x;
        v[k] = make_uint4(0, 0, 0, 0);
        if (it < items) {
          const int r = it / (nbp * 16), q = it - r * nbp * 16;
          v[k] = ldg_nc_v4(x + (size_t)r * ldx + (size_t)b0 * kBlock + (size_t)q * 8);
        }
      }
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        const int it = base + k * (int)blockDim.x + (int)threadIdx.x;
        if (it < items) {
          const int r = it / (nbp * 16), q = it - r * nbp * 16, blk = q >> 4, G = q & 15;
          uint32_t* d = img + (uint32_t)r * img_row_words + (uint32_t)blk * kImgWords +
                        (uint32_t)((4 * (G & 1) + ((G >> 2) & 1)) * 12 + 2 * (G >> 3) + ((G >> 1) & 1));
          d[0] = v[k].x; d[4] = v[k].y; d[8] = v[k].z;
          d[24] = v[k].y; d[28] = v[k].z; d[32] = v[k].w;
        }
      }
    }
  }
  __syncthreads();

  float acc[2][NB][4];
#pragma unroll
  for (int a = 0; a < 2; ++a)
#pragma unroll
    for (int c = 0; c < NB; ++c)
#pragma unroll
      for (int d = 0; d < 4; ++d) acc[a][c][d] = 0.0f;

  bool failed = false;
  const __half* xrow[NB];
#pragma unroll
  for (int c = 0; c < NB; ++c) xrow[c] = g + 8 * c < batch ? x + (size_t)(g + 8 * c) * ldx + t * 8 : nullptr;
  // N = 6: the lane's activation pairs of a chunk start at column 8 (t >> 1) + 2 (t & 1) of a 32-column step
  const __half* xsp[NB];
#pragma unroll
  for (int c = 0; c < NB; ++c) xsp[c] = xrow[c] ? xrow[c] - t * 8 + 8 * (t >> 1) + 2 * (t & 1) : nullptr;

  // Residual term of the salient columns: the residual words of this warp's run of blocks are numbered
  // consecutively (stb_layout.cuh); one tensor-core step takes 16 salient slots = four words, lane t the t-th.
  // A word's table entry names its block and its four salient columns.
  const ResidWord* rwt = reinterpret_cast<const ResidWord*>(packed + hdr->rwtab_offset);
  uint32_t rw0 = 0, rw1 = 0;
  if (cnt > 0) { rw0 = __ldg(&binfo[wb0].rw_off); rw1 = __ldg(&binfo[wb1 - 1].rw_off) + __ldg(&binfo[wb1 - 1].nrw); }
  struct ResidWords { uint32_t rw, cols, block; uint2 a2; };
  auto fetch = [&](uint32_t step, ResidWords& w) {
    w.rw = 0x55555555u; w.cols = 0u; w.block = (uint32_t)wb0; w.a2 = make_uint2(0u, 0u);
    const uint32_t wi = rw0 + 4u * step + (uint32_t)t;
    if (wi < rw1) {
      const uint2 e = __ldg(reinterpret_cast<const uint2*>(rwt + wi));
      w.block = e.x >> 3; w.cols = e.y;
      // the word's block record in the residual stream: a_sal2 of the lane's four rows, then the block's words
      const uint8_t* rec = resid_rt + resid_block_off((int)w.block, wi - (e.x & 7u));
      w.a2 = __ldg(reinterpret_cast<const uint2*>(rec + resid_a2_off(g, 0)));
      w.rw = __ldg(reinterpret_cast<const uint32_t*>(rec + resid_code_off(e.x & 7u, g)));
    }
  };
  ResidWords rfirst;
  fetch(0u, rfirst);      // in flight during the main loop

  for (int it = 0; it < cnt; ++it) {
    const int ch = it / kChunk, kin = it - ch * kChunk;     // chunk and tile inside the chunk
    const int slot = ch % kDepth;
    const uint32_t bar = bar0 + 8u * slot;
    const int b = wb0 + it;
    // all lanes poll; the verdict is made warp-uniform so that nobody is left at a __syncwarp
    if (kin == 0 && !__all_sync(0xFFFFFFFFu, mbar_wait(bar, (uint32_t)(ch / kDepth) & 1u, wait_limit))) { failed = true; break; }
    const uint8_t* tile = ring + (size_t)slot * L.tile_stride + (size_t)kin * tbytes;
    // release of the ring slot: once the whole chunk is in registers or consumed, refill it
    auto refill = [&]() {
      if (kin == kChunk - 1 || it == cnt - 1) {
        __syncwarp();
        const int nxt = (ch + kDepth) * kChunk;      // first tile of the chunk that reuses this slot
        if (lane == 0 && nxt < cnt) {
          const uint32_t bytes = (uint32_t)min(kChunk, cnt - nxt) * tbytes;
          fence_async_smem();
          mbar_expect_tx(bar, bytes);
          bulk_g2s(smem_u32(ring + (size_t)slot * L.tile_stride), rtbase + (size_t)(wb0 + nxt) * tbytes, bytes, bar);
        }
      }
    };
    if constexpr (N == 6 && NB == 1) {
      // Rank order through the sparse instruction.  This lane's metadata: rows g + 16 (t >> 1) and + 8, the chunks
      // of operand registers 2 h, 2 h + 1 (h = t & 1) of the quad's four lanes, i.e. their slots 2 h and 2 h + 1.
      LaneTile<N> lt;
      load_lane_tile<N>(tile, lane, lt, true);
      refill();
      FastRows<N> fr;
      fr.init(lt, lt.A, lt.B);
      uint32_t E[2][3];
#pragma unroll
      for (int bb = 0; bb < 2; ++bb) {
        uint32_t en[2][4];
#pragma unroll
        for (int tq = 0; tq < 4; ++tq) {
          // the pair field of the two rows whose metadata this lane supplies
          const uint32_t f = (lt.mask[2 * bb + (tq >> 1)] >> (16 * (tq & 1))) & 0xFFFFu;
          en[0][tq] = reinterpret_cast<const uint32_t*>(smem)[pair_field_index(f, 0)];
          en[1][tq] = reinterpret_cast<const uint32_t*>(smem)[pair_field_index(f, 1)];
        }
        meta6_words(en, E[bb]);
      }
      if (image_bytes != 0u) {
        // activations from the CTA's image in shared memory: two rows of the lane at a time (fewer live registers;
        // the 16-byte operand loads are cheap enough to be issued once per row pair)
        const uint32_t* xi0 = ximg + (uint32_t)g * img_row_words + (uint32_t)(b - b0) * kImgWords + (uint32_t)(t * 24);
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
              uint4 bx = make_uint4(0, 0, 0, 0);
              if (g < batch) bx = *reinterpret_cast<const uint4*>(xi0 + sl * 12 + 4 * i);
              if (mt == 0) mma_sp16832<0>(acc[0][0], R[0][0][i], R[1][0][i], R[0][1][i], R[1][1][i], bx.x, bx.y, bx.z, bx.w, E[sl][i]);
              else mma_sp16832<1>(acc[1][0], R[0][0][i], R[1][0][i], R[0][1][i], R[1][1][i], bx.x, bx.y, bx.z, bx.w, E[sl][i]);
            }
          }
        }
      } else {
      uint32_t XL6[4][2], XH6[4][2];
#pragma unroll
      for (int j = 0; j < 4; ++j)
#pragma unroll
        for (int sp = 0; sp < 2; ++sp) fr.high(j, sp, XL6[j][sp], XH6[j][sp]);
#pragma unroll
      for (int sl = 0; sl < 2; ++sl) {
        uint32_t R[4][2][3];
#pragma unroll
        for (int j = 0; j < 4; ++j)
#pragma unroll
          for (int h = 0; h < 2; ++h) fr.pairs(j, 2 * h + sl, XL6[j][h], XH6[j][h], R[j][h]);
        // Activations of chunk i of a step: columns 2 i + 2 (t & 1) + {0, 1} of the group's eight.  Up to two batch
        // rows whose slice is too long for the image: one 4-byte load per register (few lanes are active); more
        // batch rows: the group's 16 bytes through L1, then a select.
        if (batch <= 2) {
#pragma unroll
          for (int i = 0; i < 3; ++i) {
#pragma unroll
            for (int c = 0; c < NB; ++c) {
              uint32_t bx[4] = {0, 0, 0, 0};
              if (xsp[c]) {
#pragma unroll
                for (int u = 0; u < 4; ++u)
                  bx[u] = ldg_nc_u32(xsp[c] + (size_t)b * kBlock + 64 * (u >> 1) + 16 * (u & 1) + 32 * sl + 2 * i);
              }
              mma_sp16832<0>(acc[0][c], R[0][0][i], R[1][0][i], R[0][1][i], R[1][1][i], bx[0], bx[1], bx[2], bx[3], E[sl][i]);
              mma_sp16832<1>(acc[1][c], R[2][0][i], R[3][0][i], R[2][1][i], R[3][1][i], bx[0], bx[1], bx[2], bx[3], E[sl][i]);
            }
          }
        } else {
#pragma unroll
          for (int c = 0; c < NB; ++c) {
            uint4 xw[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) {
              xw[u] = make_uint4(0, 0, 0, 0);
              if (xsp[c]) xw[u] = ldg_nc_v4(xsp[c] - 2 * (t & 1) + (size_t)b * kBlock + 64 * (u >> 1) + 16 * (u & 1) + 32 * sl);
            }
#pragma unroll
            for (int i = 0; i < 3; ++i) {
              uint32_t bx[4];
#pragma unroll
              for (int u = 0; u < 4; ++u) {
                const uint32_t w0 = i == 0 ? xw[u].x : (i == 1 ? xw[u].y : xw[u].z), w1 = i == 0 ? xw[u].y : (i == 1 ? xw[u].z : xw[u].w);
                bx[u] = (t & 1) ? w1 : w0;
              }
              mma_sp16832<0>(acc[0][c], R[0][0][i], R[1][0][i], R[0][1][i], R[1][1][i], bx[0], bx[1], bx[2], bx[3], E[sl][i]);
              mma_sp16832<1>(acc[1][c], R[2][0][i], R[3][0][i], R[2][1][i], R[3][1][i], bx[0], bx[1], bx[2], bx[3], E[sl][i]);
            }
          }
        }
      }
      }
    } else {
    LaneTile<N> lt;
    load_lane_tile<N>(tile, lane, lt);
    refill();
    FastRows<N> fr;
    fr.init(lt, lt.A, lt.B);
    uint32_t XL[4] = {0, 0, 0, 0}, XH[4] = {0, 0, 0, 0};
    if (N == 5) {
#pragma unroll
      for (int j = 0; j < 4; ++j) fr.high(j, 0, XL[j], XH[j]);
    }
    // all table lookups (and, for up to 16 batch rows, activation loads) of the tile are issued up front
    uint2 P[16];
#pragma unroll
    for (int u = 0; u < 16; ++u) P[u] = ptab[keep_index_of(lt.mask, u >> 2, u & 3)];
    constexpr int XS = NB <= 2 ? 4 : 1;          // activation fragments held at a time: all four steps, or one
    uint4 xf[XS][NB];
    if (NB <= 2) {
#pragma unroll
      for (int s = 0; s < 4; ++s)
#pragma unroll
        for (int c = 0; c < NB; ++c) {
          xf[s % XS][c] = make_uint4(0, 0, 0, 0);
          if (xrow[c]) xf[s % XS][c] = ldg_nc_v4(xrow[c] + (size_t)b * kBlock + s * 32);
        }
    }
#pragma unroll
    for (int s = 0; s < 4; ++s) {
      if (NB > 2) {
#pragma unroll
        for (int c = 0; c < NB; ++c) {
          xf[0][c] = make_uint4(0, 0, 0, 0);
          if (xrow[c]) xf[0][c] = ldg_nc_v4(xrow[c] + (size_t)b * kBlock + s * 32);
        }
      }
      uint32_t f[4][4];
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        if (N == 6 && (s & 1) == 0) fr.high(j, s >> 1, XL[j], XH[j]);
        fr.slot2(j, s, P[4 * j + s].x, P[4 * j + s].y, XL[j], XH[j], f[j]);
      }
#pragma unroll
      for (int mt = 0; mt < 2; ++mt)
#pragma unroll
        for (int c = 0; c < NB; ++c) {
          const uint4 xv = xf[s % XS][c];
          mma16816(acc[mt][c], f[2 * mt][0], f[2 * mt + 1][0], f[2 * mt][1], f[2 * mt + 1][1], xv.x, xv.y);
          mma16816(acc[mt][c], f[2 * mt][2], f[2 * mt + 1][2], f[2 * mt][3], f[2 * mt + 1][3], xv.z, xv.w);
        }
    }
    }

  }

  // Residual term of the salient columns, after the main stream (its registers and loads stay out of the main
  // loop): per four residual words one tensor-core step with their 16 salient slots as K.  The lane's word (its
  // codes, the a_sal2 of its rows in the word's block, the salient columns) is fetched one step ahead.
  if (rw1 > rw0 && !failed) {
    const uint32_t nstep = (rw1 - rw0 + 3u) >> 2;
    ResidWords cur = rfirst, nxt;
#pragma unroll 1
    for (uint32_t gi = 0; gi < nstep; ++gi) {
      fetch(gi + 1u, nxt);
      const size_t xoff = (size_t)cur.block * kBlock;
      uint32_t fa[4][2];
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const uint32_t h = (((j & 2) ? cur.a2.y : cur.a2.x) >> (16 * (j & 1))) & 0xFFFFu;
        const uint32_t L2 = prmt(h, 0u, 0x4040u);                 // (lo, 0, lo, 0)
        const uint32_t H2 = prmt(h, h ^ 0x8000u, 0x2521u);        // (hi, 0, hi ^ 0x80, 0)
        const uint32_t sel = resid_selector(cur.rw, j);
        const uint32_t lo4 = prmt(L2, L2, sel), hi4 = prmt(H2, H2, sel);
        fa[j][0] = prmt(lo4, hi4, 0x5140u);
        fa[j][1] = prmt(lo4, hi4, 0x7362u);
      }
      // the four salient columns behind this lane's residual word
      const uint32_t cw = cur.cols;
#pragma unroll
      for (int c = 0; c < NB; ++c) {
        uint2 xr = make_uint2(0, 0);
        if (xrow[c]) {
          const unsigned short* xq = reinterpret_cast<const unsigned short*>(xrow[c] - t * 8 + xoff);
          xr.x = (uint32_t)__ldg(xq + (cw & 0xFFu)) | ((uint32_t)__ldg(xq + ((cw >> 8) & 0xFFu)) << 16);
          xr.y = (uint32_t)__ldg(xq + ((cw >> 16) & 0xFFu)) | ((uint32_t)__ldg(xq + (cw >> 24)) << 16);
        }
        mma16816(acc[0][c], fa[0][0], fa[1][0], fa[0][1], fa[1][1], xr.x, xr.y);
        mma16816(acc[1][c], fa[2][0], fa[3][0], fa[2][1], fa[3][1], xr.x, xr.y);
      }
      cur = nxt;
    }
  }

  if (failed) {
    // give the copies still in flight time to land before the shared memory is given up
    const long long t0 = clock64();
    while (clock64() - t0 < 200000) {}
    if (lane == 0 && dev_status) *dev_status = STB_ERR_TIMEOUT;
  }
  __syncthreads();     // every warp is done with its ring: reuse it for the partial sums

  // red[warp][row 0..31][batch 0..8NB-1]
  constexpr int BW = 8 * NB;
  float* red = reinterpret_cast<float*>(smem + L.ring);
#pragma unroll
  for (int mt = 0; mt < 2; ++mt)
#pragma unroll
    for (int c = 0; c < NB; ++c) {
      float* r0 = red + ((size_t)warp * 32 + (g + 16 * mt)) * BW + 8 * c + 2 * t;
      float* r1 = r0 + 8 * BW;
      r0[0] = acc[mt][c][0]; r0[1] = acc[mt][c][1];
      r1[0] = acc[mt][c][2]; r1[1] = acc[mt][c][3];
    }
  __syncthreads();
  float* part = reinterpret_cast<float*>(smem + L.part);       // [ksplit][32][BW], used on cluster rank 0
  if (ksplit > 1) cluster_wait();
  for (int i = threadIdx.x; i < 32 * BW; i += blockDim.x) {
    float sacc = 0.0f;
    for (int w = 0; w < warps; ++w) sacc += red[(size_t)w * 32 * BW + i];
    if (ksplit == 1) {
      const int row = rt * kTileRows + i / BW, bt = i % BW;
      if (row < n && bt < batch) {
        if (y_f16) static_cast<__half*>(y)[(size_t)bt * ldy + row] = __float2half_rn(sacc);
        else static_cast<float*>(y)[(size_t)bt * ldy + row] = sacc;
      }
    } else {
      float* dst = cg::this_cluster().map_shared_rank(part, 0);
      dst[(size_t)kpart * 32 * BW + i] = sacc;
    }
  }
  if (ksplit == 1) return;
  cg::this_cluster().sync();
  if (kpart == 0) {
    for (int i = threadIdx.x; i < 32 * BW; i += blockDim.x) {
      const int row = rt * kTileRows + i / BW, bt = i % BW;
      if (row < n && bt < batch) {
        float tsum = 0.0f;
        for (int k = 0; k < ksplit; ++k) tsum += part[(size_t)k * 32 * BW + i];
        if (y_f16) static_cast<__half*>(y)[(size_t)bt * ldy + row] = __float2half_rn(tsum);
        else static_cast<float*>(y)[(size_t)bt * ldy + row] = tsum;
      }
    }
  }
}

// Launch shape: ksplit CTAs per row tile and warps per CTA.  A warp should get a run of several
// tiles (its ring then streams while it decodes) and the grid should have at least two CTAs per
// SM while leaving room on the SM for the next layer's CTAs, which start their own weight
// stream early (programmatic dependent launch).
static void gemv_shape(int n, int m, int& ksplit, int& warps) {
  const int ntile = (n + kTileRows - 1) / kTileRows, nblk = m / kBlock;
  warps = 4;
  int ks = 1;
  while (ks < 8 && ntile * ks < 296 && nblk / (2 * ks * warps) >= 4) ks *= 2;
  ksplit = ks;
}

// `chained`: launch as a programmatic dependent of the previous kernel of the stream (only used
// between the GEMVs of one stb_layer_stack call, whose packed layers nobody writes meanwhile).
template <int N, int NB>
static cudaError_t launch_mma(const GemvLayers& layers, int m, const __half* x, int batch, size_t ldx,
                              int* dev_status, cudaStream_t s, bool chained, bool wait_selftest = false) {
  const int ntile = layers.tile_start[layers.count], nblk = m / kBlock;
  int ksplit, warps;
  gemv_shape(ntile * kTileRows, m, ksplit, warps);
  const int bpp = (nblk + ksplit - 1) / ksplit;
  const GemvSmem L = gemv_smem(N, warps, ksplit, NB, gemv_image_bytes(N, NB, batch, bpp));
  // the shared-memory limit of a kernel is a per-device setting
  static bool attr_done[kMaxDevices] = {};
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= kMaxDevices || !attr_done[dev]) {
    e = cudaFuncSetAttribute(gemv_mma_kernel<N, NB>, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
    if (e != cudaSuccess) return e;
    if (dev >= 0 && dev < kMaxDevices) attr_done[dev] = true;
  }
  if (L.total > 200 * 1024) return cudaErrorInvalidValue;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)(ntile * ksplit), 1, 1);
  cfg.blockDim = dim3((unsigned)(warps * 32), 1, 1);
  cfg.dynamicSmemBytes = L.total;
  cfg.stream = s;
  cudaLaunchAttribute at[2];
  int na = 0;
  if (ksplit > 1) {
    at[na].id = cudaLaunchAttributeClusterDimension;
    at[na].val.clusterDim.x = (unsigned)ksplit; at[na].val.clusterDim.y = 1; at[na].val.clusterDim.z = 1;
    ++na;
  }
  if (chained) {
    at[na].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[na].val.programmaticStreamSerializationAllowed = 1;
    ++na;
  }
  cfg.attrs = at; cfg.numAttrs = na;
  int lg = 0;
  while ((1 << lg) < ksplit) ++lg;
  const long long limit = wait_selftest ? kSelftestWaitLimit : kWaitLimit;
  return cudaLaunchKernelEx(&cfg, gemv_mma_kernel<N, NB>, layers, m, x, batch, ldx, dev_status, lg, bpp, limit, wait_selftest ? 1 : 0);
}

template <int NB>
static cudaError_t launch_mma_n(int N, const GemvLayers& layers, int m, const __half* x, int batch, size_t ldx,
                                int* dev_status, cudaStream_t s, bool chained, bool selftest) {
  if (N == 4) return launch_mma<4, NB>(layers, m, x, batch, ldx, dev_status, s, chained, selftest);
  if (N == 5) return launch_mma<5, NB>(layers, m, x, batch, ldx, dev_status, s, chained, selftest);
  return launch_mma<6, NB>(layers, m, x, batch, ldx, dev_status, s, chained, selftest);
}

// batch -> number of 8-row batch groups (1, 2, 4 or 8)
static cudaError_t launch_mma_b(int batch, int N, const GemvLayers& layers, int m, const __half* x, size_t ldx,
                                int* dev_status, cudaStream_t s, bool chained, bool selftest = false) {
  if (batch <= 8) return launch_mma_n<1>(N, layers, m, x, batch, ldx, dev_status, s, chained, selftest);
  if (batch <= 16) return launch_mma_n<2>(N, layers, m, x, batch, ldx, dev_status, s, chained, selftest);
  if (batch <= 32) return launch_mma_n<4>(N, layers, m, x, batch, ldx, dev_status, s, chained, selftest);
  return launch_mma_n<8>(N, layers, m, x, batch, ldx, dev_status, s, chained, selftest);
}

// ------------------------------------------------------------------------------------------
// General kernel: any N in 1..8, batch <= BT.  One CTA per row tile (32 rows), 8 warps split
// the blocks, lane = (g, t); plain position-order decode and fp32 multiply-adds, x read
// through L1.  The four lanes that share a row combine with shuffles, the 8 warps through
// shared memory in a fixed order, so the result is deterministic.
template <int N, int BT>
__global__ void __launch_bounds__(256)
gemv_general_kernel(const uint8_t* __restrict__ packed, int n, int m, const __half* __restrict__ x,
                    int batch, size_t ldx, void* __restrict__ y, int y_f16, size_t ldy, int* dev_status) {
  const Header* hdr = reinterpret_cast<const Header*>(packed);
  if (!header_matches(hdr, n, m, N)) {
    if (threadIdx.x == 0 && dev_status) *dev_status = STB_ERR_CORRUPT;
    return;
  }
  const int nblk = m / kBlock;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, g = lane >> 2, t = lane & 3;
  const int rt = blockIdx.x;
  const BlockInfo* binfo = reinterpret_cast<const BlockInfo*>(packed + sizeof(Header));
  const uint8_t* rtbase = packed + hdr->tiles_offset + (size_t)rt * hdr->rt_stride;
  const uint8_t* resid_rt = packed + hdr->tiles_offset + hdr->rt_stride * (size_t)hdr->ntile +
                            (size_t)rt * resid_rt_bytes(nblk, hdr->nrw);

  float acc[4][BT];
#pragma unroll
  for (int j = 0; j < 4; ++j)
#pragma unroll
    for (int bt = 0; bt < BT; ++bt) acc[j][bt] = 0.0f;

  for (int b = warp; b < nblk; b += 8) {
    const uint8_t* tile = rtbase + (size_t)b * hdr->tile_bytes;
    LaneTile<N> lt;
    load_lane_tile<N>(tile, lane, lt);
    const uint64_t sal[2] = {binfo[b].salient[0], binfo[b].salient[1]};
    const uint8_t* record = resid_rt + resid_block_off(b, binfo[b].rw_off);
    const int nslot = 4 * (int)binfo[b].nrw;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      float alpha[5];
#pragma unroll
      for (int q = 0; q < 4; ++q) alpha[q] = __half2float(__ushort_as_half((unsigned short)scale_bits<N>(lt, j, q)));
      alpha[4] = __half2float(__ushort_as_half((unsigned short)sal2_bits(record, g, j)));
#pragma unroll 1
      for (int s = 0; s < 4; ++s) {
        const int grp = 4 * s + t;
        uint32_t code[8], neg[8];
        plain_slot<N>(lt, 4 * j + s, code, neg);
        const uint32_t salb = (uint32_t)((sal[grp >> 3] >> (8 * (grp & 7))) & 0xFFull);
        int qbase = grp >= 8 ? __popcll(sal[0]) : 0;
        qbase += __popcll(sal[grp >> 3] & ((1ull << (8 * (grp & 7))) - 1ull));
        float v[8];
#pragma unroll
        for (int c = 0; c < 8; ++c) {
          float w = 0.0f;
          if (code[c] < 4u) {
            const float s1 = neg[c] ? -1.0f : 1.0f;
            if (code[c] == 3u) {
              const int q = qbase + __popc(salb & ((1u << c) - 1u));
              const uint32_t word = q < nslot ? resid_word(record, (uint32_t)(q >> 2), g) : 0x55555555u;
              const float s2 = resid_code(word, j, q & 3) == 0u ? 1.0f : -1.0f;
              w = __fadd_rn(s1 * alpha[3], s2 * alpha[4]);
            } else {
              w = s1 * (code[c] == 0u ? alpha[0] : (code[c] == 1u ? alpha[1] : alpha[2]));
            }
          }
          v[c] = w;
        }
#pragma unroll
        for (int bt = 0; bt < BT; ++bt) {
          if (bt < batch) {
            const uint4 xv = __ldg(reinterpret_cast<const uint4*>(x + (size_t)bt * ldx + (size_t)b * kBlock + grp * 8));
            const __half2* xh = reinterpret_cast<const __half2*>(&xv);
#pragma unroll
            for (int c = 0; c < 4; ++c) {
              const float2 xf = __half22float2(xh[c]);
              acc[j][bt] = fmaf(v[2 * c], xf.x, acc[j][bt]);
              acc[j][bt] = fmaf(v[2 * c + 1], xf.y, acc[j][bt]);
            }
          }
        }
      }
    }
  }

  // the four lanes t of a row
#pragma unroll
  for (int j = 0; j < 4; ++j)
#pragma unroll
    for (int bt = 0; bt < BT; ++bt) {
      float a = acc[j][bt];
      a += __shfl_xor_sync(0xFFFFFFFFu, a, 1);
      a += __shfl_xor_sync(0xFFFFFFFFu, a, 2);
      acc[j][bt] = a;
    }
  __shared__ float red[8][BT][32];
  if (t == 0) {
#pragma unroll
    for (int j = 0; j < 4; ++j)
#pragma unroll
      for (int bt = 0; bt < BT; ++bt) red[warp][bt][g + 8 * j] = acc[j][bt];
  }
  __syncthreads();
  for (int idx = threadIdx.x; idx < BT * 32; idx += blockDim.x) {
    const int bt = idx >> 5, l = idx & 31;
    const int row = rt * kTileRows + l;
    if (bt < batch && row < n) {
      float s = 0.0f;
#pragma unroll
      for (int w = 0; w < 8; ++w) s += red[w][bt][l];
      if (y_f16) static_cast<__half*>(y)[(size_t)bt * ldy + row] = __float2half_rn(s);
      else static_cast<float*>(y)[(size_t)bt * ldy + row] = s;
    }
  }
}

template <int N>
static cudaError_t launch_general(const uint8_t* packed, int n, int m, const __half* x, int batch,
                                  size_t ldx, void* y, int y_f16, size_t ldy, int* dev_status, cudaStream_t s) {
  const unsigned grid = (unsigned)((n + kTileRows - 1) / kTileRows);
  if (batch <= 2) gemv_general_kernel<N, 2><<<grid, 256, 0, s>>>(packed, n, m, x, batch, ldx, y, y_f16, ldy, dev_status);
  else if (batch <= 8) gemv_general_kernel<N, 8><<<grid, 256, 0, s>>>(packed, n, m, x, batch, ldx, y, y_f16, ldy, dev_status);
  else gemv_general_kernel<N, 16><<<grid, 256, 0, s>>>(packed, n, m, x, batch, ldx, y, y_f16, ldy, dev_status);
  return cudaGetLastError();
}

}  // namespace stb

static int gemv_impl(const void* packed, int n, int m, int N, const void* x, int batch, size_t ldx,
                     void* y, stb_dtype ydt, size_t ldy, int* dev_status, void* stream, bool chained,
                     bool wait_selftest = false) {
  if (!packed || !x || !y) return STB_ERR_ARG;
  if (n < 1 || m < stb::kBlock || m % stb::kBlock != 0) return STB_ERR_SHAPE;
  if (N < 1 || N > 8) return STB_ERR_NM;
  if (batch < 1 || batch > 64) return STB_ERR_SIZE;
  if (ydt != STB_F32 && ydt != STB_F16) return STB_ERR_UNSUPPORTED;
  const int y_f16 = ydt == STB_F16;
  if (ldx < (size_t)m || ldy < (size_t)n || (ldx % 8) != 0 || (reinterpret_cast<uintptr_t>(x) & 15u)) return STB_ERR_ARG;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  const uint8_t* p = static_cast<const uint8_t*>(packed);
  const __half* xh = static_cast<const __half*>(x);
  cudaError_t e = cudaSuccess;
  if (N >= 4 && N <= 6) {
    stb::GemvLayers layers = {};
    layers.packed[0] = p; layers.y[0] = y; layers.ldy[0] = ldy; layers.n[0] = n; layers.y_f16[0] = y_f16;
    layers.tile_start[0] = 0; layers.tile_start[1] = (n + stb::kTileRows - 1) / stb::kTileRows; layers.count = 1;
    e = stb::launch_mma_b(batch, N, layers, m, xh, ldx, dev_status, s, chained, wait_selftest);
    return e == cudaSuccess ? STB_OK : STB_ERR_CUDA;
  }
  if (wait_selftest) return STB_ERR_UNSUPPORTED;
  // the general kernel takes up to 16 batch rows per launch
  for (int t0 = 0; t0 < batch && e == cudaSuccess; t0 += 16) {
    const int bt = batch - t0 < 16 ? batch - t0 : 16;
    const __half* xc = xh + (size_t)t0 * ldx;
    void* yc = y_f16 ? static_cast<void*>(static_cast<__half*>(y) + (size_t)t0 * ldy)
                     : static_cast<void*>(static_cast<float*>(y) + (size_t)t0 * ldy);
    switch (N) {
      case 1: e = stb::launch_general<1>(p, n, m, xc, bt, ldx, yc, y_f16, ldy, dev_status, s); break;
      case 2: e = stb::launch_general<2>(p, n, m, xc, bt, ldx, yc, y_f16, ldy, dev_status, s); break;
      case 3: e = stb::launch_general<3>(p, n, m, xc, bt, ldx, yc, y_f16, ldy, dev_status, s); break;
      case 4: e = stb::launch_general<4>(p, n, m, xc, bt, ldx, yc, y_f16, ldy, dev_status, s); break;
      case 5: e = stb::launch_general<5>(p, n, m, xc, bt, ldx, yc, y_f16, ldy, dev_status, s); break;
      case 6: e = stb::launch_general<6>(p, n, m, xc, bt, ldx, yc, y_f16, ldy, dev_status, s); break;
      case 7: e = stb::launch_general<7>(p, n, m, xc, bt, ldx, yc, y_f16, ldy, dev_status, s); break;
      case 8: e = stb::launch_general<8>(p, n, m, xc, bt, ldx, yc, y_f16, ldy, dev_status, s); break;
    }
  }
  return e == cudaSuccess ? STB_OK : STB_ERR_CUDA;
}

extern "C" int stb_gemv(const void* packed, int n, int m, int N, const void* x, int batch, size_t ldx,
                        void* y, stb_dtype ydt, size_t ldy, int* dev_status, void* stream) {
  return gemv_impl(packed, n, m, N, x, batch, ldx, y, ydt, ldy, dev_status, stream, false);
}

extern "C" int stb_gemv_wait_selftest(const void* packed, int n, int m, int N, const void* x, int batch, size_t ldx,
                                      void* y, stb_dtype ydt, size_t ldy, int* dev_status, void* stream) {
  if (!dev_status) return STB_ERR_ARG;
  return gemv_impl(packed, n, m, N, x, batch, ldx, y, ydt, ldy, dev_status, stream, false, true);
}

// Steps i..j-1 can share one grid when they read the same activations with the same batch, m and N
// (4, 5 or 6) and none of them writes what another reads: same-input projections of a decoder
// layer (q / k / v, gate / up).
static bool can_fuse(const stb_step& a, const stb_step& b) {
  return a.in == b.in && a.ldin == b.ldin && a.batch == b.batch && a.m == b.m && a.N == b.N && a.N >= 4 && a.N <= 6 &&
         b.out != a.in && b.packed && b.out && b.n >= 1 && (b.odt == STB_F32 || b.odt == STB_F16) && b.ldout >= (size_t)b.n;
}

extern "C" int stb_layer_stack(const stb_step* steps, int count, int* dev_status, void* stream) {
  if (!steps || count < 0) return STB_ERR_ARG;
  for (int k = 0; k < count; ++k)
    if (steps[k].input != STB_IN_PLAIN) return STB_ERR_UNSUPPORTED;      // only the resident kernel forms inputs
  int i = 0;
  while (i < count) {
    const stb_step& st = steps[i];
    int j = i + 1;
    while (j < count && j - i < stb::kMaxFused && can_fuse(st, steps[j])) ++j;
    // steps after the first start their weight stream while the previous step drains
    const bool chained = i > 0;
    if (j - i == 1) {
      int rc = gemv_impl(st.packed, st.n, st.m, st.N, st.in, st.batch, st.ldin, st.out, st.odt, st.ldout,
                         dev_status, stream, chained);
      if (rc != STB_OK) return rc;
    } else {
      // validate the first step like stb_gemv does; can_fuse has checked what differs in the others
      if (!st.packed || !st.in || !st.out) return STB_ERR_ARG;
      if (st.n < 1 || st.m < stb::kBlock || st.m % stb::kBlock != 0) return STB_ERR_SHAPE;
      if (st.batch < 1 || st.batch > 64) return STB_ERR_SIZE;
      if (st.odt != STB_F32 && st.odt != STB_F16) return STB_ERR_UNSUPPORTED;
      if (st.ldin < (size_t)st.m || st.ldout < (size_t)st.n || (st.ldin % 8) != 0 || (reinterpret_cast<uintptr_t>(st.in) & 15u))
        return STB_ERR_ARG;
      stb::GemvLayers layers = {};
      layers.count = j - i;
      layers.tile_start[0] = 0;
      for (int k = i; k < j; ++k) {
        const stb_step& sk = steps[k];
        layers.packed[k - i] = static_cast<const uint8_t*>(sk.packed);
        layers.y[k - i] = sk.out; layers.ldy[k - i] = sk.ldout; layers.n[k - i] = sk.n; layers.y_f16[k - i] = sk.odt == STB_F16;
        layers.tile_start[k - i + 1] = layers.tile_start[k - i] + (sk.n + stb::kTileRows - 1) / stb::kTileRows;
      }
      cudaStream_t s = static_cast<cudaStream_t>(stream);
      const __half* xh = static_cast<const __half*>(st.in);
      cudaError_t e = stb::launch_mma_b(st.batch, st.N, layers, st.m, xh, st.ldin, dev_status, s, chained);
      if (e != cudaSuccess) return STB_ERR_CUDA;
    }
    i = j;
  }
  return STB_OK;
}

extern "C" int stb_layer_stack_host(const stb_step* steps, int count, const void* in_host, size_t in_bytes,
                                    void* out_host, size_t out_bytes, int* dev_status, void* stream) {
  if (!steps || count < 1 || !in_host || !out_host || !steps[0].in || !steps[count - 1].out) return STB_ERR_ARG;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  if (cudaMemcpyAsync(const_cast<void*>(steps[0].in), in_host, in_bytes, cudaMemcpyHostToDevice, s) != cudaSuccess)
    return STB_ERR_CUDA;
  const int rc = stb_layer_stack(steps, count, dev_status, stream);
  if (rc != STB_OK) return rc;
  if (cudaMemcpyAsync(out_host, steps[count - 1].out, out_bytes, cudaMemcpyDeviceToHost, s) != cudaSuccess)
    return STB_ERR_CUDA;
  return STB_OK;
}

// stb_pack: fused pack / transpose of a logical N:8 structured-binary layer into the
// tile-major streaming layout (stb_layout.cuh), plus the small host-side entry points that
// need no kernel of their own.  Counterpart of the paper's "matrix compression" and "value
// compression" steps (Appendix C), generalised to an 8-bit keep mask, N sign bits and 2N region
// bits per group, five scales per row-block and a two-bit residual code per salient column of each block.
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/stb.h"
#include "stb_decode.cuh"
#include "stb_layout.cuh"

namespace stb {

// ---------------------------------------------------------------------------------------
// Header, per-block table and residual word table.  One CTA; every block gets ceil(S / 4)
// residual words for its S salient columns, numbered block after block.
__global__ void header_kernel(int n, int m, int N, const uint64_t* __restrict__ salient,
                              uint8_t* __restrict__ packed, int* dev_status) {
  const int nblk = m / kBlock;
  Header* hdr = reinterpret_cast<Header*>(packed);
  BlockInfo* bi = reinterpret_cast<BlockInfo*>(packed + sizeof(Header));
  ResidWord* rwt = reinterpret_cast<ResidWord*>(packed + rwtab_offset(nblk));
  __shared__ int bad;
  __shared__ uint32_t total;
  if (threadIdx.x == 0) bad = 0;
  __syncthreads();
  for (int b = threadIdx.x; b < nblk; b += blockDim.x) {
    uint64_t lo = salient[2 * b], hi = salient[2 * b + 1];
    int ns = __popcll(lo) + __popcll(hi);
    if (ns > kMaxSalient) { bad = 1; ns = kMaxSalient; }
    bi[b].salient[0] = lo;
    bi[b].salient[1] = hi;
    bi[b].nsal = (uint32_t)ns;
    bi[b].nrw = (uint32_t)resid_words_for(ns);
    bi[b].pad = 0;
    int q = 0;
    for (int h = 0; h < 2; ++h) {
      uint64_t mk = h ? hi : lo;
      while (mk && q < kMaxSalient) {
        bi[b].cols[q++] = (uint8_t)(__ffsll((long long)mk) - 1 + 64 * h);
        mk &= mk - 1;
      }
    }
    for (; q < kMaxSalient; ++q) bi[b].cols[q] = 0;
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    uint32_t off = 0;
    for (int b = 0; b < nblk; ++b) { bi[b].rw_off = off; off += bi[b].nrw; }
    total = off;
  }
  __syncthreads();
  for (int b = threadIdx.x; b < nblk; b += blockDim.x)
    for (uint32_t wq = 0; wq < bi[b].nrw; ++wq) {
      ResidWord e;
      e.block_wq = 8u * (uint32_t)b + wq;
      for (int k = 0; k < 4; ++k) e.cols[k] = bi[b].cols[4 * wq + k];
      rwt[bi[b].rw_off + wq] = e;
    }
  if (threadIdx.x == 0) {
    const int ntile = (n + kTileRows - 1) / kTileRows;
    const uint32_t tb = tile_bytes(N);
    hdr->magic = kMagic;
    hdr->version = 4;
    hdr->n = n; hdr->m = m; hdr->N = N;
    hdr->nblk = nblk;
    hdr->ntile = ntile;
    hdr->tiles_offset = tiles_offset(nblk);
    hdr->rt_stride = (uint64_t)tb * (uint64_t)nblk;
    hdr->used_bytes = (uint64_t)tiles_offset(nblk) + (hdr->rt_stride + resid_rt_bytes(nblk, total)) * (uint64_t)ntile;
    hdr->status = bad ? (uint32_t)STB_ERR_CORRUPT : 0u;
    hdr->tile_bytes = tb;
    hdr->nrw = total;
    hdr->rwtab_offset = rwtab_offset(nblk);
    if (bad && dev_status) *dev_status = STB_ERR_CORRUPT;
  }
}

template <int NW>
__device__ __forceinline__ void store_planes(uint8_t* tile, uint32_t base, const uint32_t* w,
                                             int lane) {
  constexpr int Q4 = NW / 4;
#pragma unroll
  for (int q = 0; q < Q4; ++q)
    *reinterpret_cast<uint4*>(tile + base + q * 512 + lane * 16) =
        make_uint4(w[4 * q], w[4 * q + 1], w[4 * q + 2], w[4 * q + 3]);
  uint32_t o = base + Q4 * 512;
  if (NW & 2) {
    *reinterpret_cast<uint2*>(tile + o + lane * 8) = make_uint2(w[4 * Q4], w[4 * Q4 + 1]);
    o += 256;
  }
  if (NW & 1) *reinterpret_cast<uint32_t*>(tile + o + lane * 4) = w[NW - 1];
}

// One warp per tile (32 rows x one block).  Phase 1, lane = row: vector loads of the row's
// logical fields, validation, scales and residual codes; the group fields go to shared
// memory.  Phase 2, lane = (g, t): each lane collects its 16 (row, group) slots and builds
// its mask / region / sign words.
constexpr int kPackWarps = 8;

template <int N>
__global__ void __launch_bounds__(kPackWarps * 32)
pack_kernel(stb_logical L, uint8_t* __restrict__ packed, int* dev_status) {
  __shared__ uint8_t sm_keep[kPackWarps][32][16];
  __shared__ uint8_t sm_sign[kPackWarps][32][16];
  __shared__ uint16_t sm_region[kPackWarps][32][16];
  const int nblk = L.m / kBlock, ngrp = L.m / kGroup;
  const int ntile = (L.n + kTileRows - 1) / kTileRows;
  const int lane = threadIdx.x & 31, wib = threadIdx.x >> 5;
  const long long warp = (long long)blockIdx.x * kPackWarps + wib;
  if (warp >= (long long)ntile * nblk) return;
  const int rt = (int)(warp / nblk), b = (int)(warp % nblk);
  const int row = rt * kTileRows + lane;
  const bool valid = row < L.n;

  Header* hdr = reinterpret_cast<Header*>(packed);
  const BlockInfo* bi = reinterpret_cast<const BlockInfo*>(packed + sizeof(Header)) + b;
  const uint64_t sal_lo = bi->salient[0], sal_hi = bi->salient[1];
  const int nsal = (int)bi->nsal, nrw_b = (int)bi->nrw;
  uint8_t* tile = packed + hdr->tiles_offset + ((size_t)rt * nblk + b) * (size_t)hdr->tile_bytes;
  // the block's record in the row tile's residual stream: a_sal2 of the 32 rows, then the residual words
  uint8_t* record = packed + hdr->tiles_offset + hdr->rt_stride * (size_t)ntile +
                    (size_t)rt * resid_rt_bytes(nblk, hdr->nrw) + resid_block_off(b, bi->rw_off);

  // ---- phase 1: lane = row ----
  // rows past n: nothing kept, all signs "+", zero scales
  uint32_t keepw[4] = {0, 0, 0, 0}, signw[4] = {~0u, ~0u, ~0u, ~0u}, regw[8] = {0, 0, 0, 0, 0, 0, 0, 0};
  uint32_t s2 = 0;
  uint16_t sc[5] = {0, 0, 0, 0, 0};
  if (valid) {
    const size_t gofs = (size_t)row * ngrp + (size_t)b * 16;
    uint4 k4 = *reinterpret_cast<const uint4*>(L.keep + gofs);
    uint4 s4 = *reinterpret_cast<const uint4*>(L.sign + gofs);
    const uint4* rp = reinterpret_cast<const uint4*>(L.region + gofs);
    uint4 r0 = rp[0], r1 = rp[1];
    keepw[0] = k4.x; keepw[1] = k4.y; keepw[2] = k4.z; keepw[3] = k4.w;
    signw[0] = s4.x; signw[1] = s4.y; signw[2] = s4.z; signw[3] = s4.w;
    regw[0] = r0.x; regw[1] = r0.y; regw[2] = r0.z; regw[3] = r0.w;
    regw[4] = r1.x; regw[5] = r1.y; regw[6] = r1.z; regw[7] = r1.w;
    s2 = L.sign2[(size_t)row * nblk + b];
    const uint16_t* sp = L.scale + ((size_t)row * nblk + b) * 5;
#pragma unroll
    for (int q = 0; q < 5; ++q) sc[q] = sp[q];
  }
  *reinterpret_cast<uint4*>(&sm_keep[wib][lane][0]) = make_uint4(keepw[0], keepw[1], keepw[2], keepw[3]);
  *reinterpret_cast<uint4*>(&sm_sign[wib][lane][0]) = make_uint4(signw[0], signw[1], signw[2], signw[3]);
  *reinterpret_cast<uint4*>(&sm_region[wib][lane][0]) = make_uint4(regw[0], regw[1], regw[2], regw[3]);
  *reinterpret_cast<uint4*>(&sm_region[wib][lane][8]) = make_uint4(regw[4], regw[5], regw[6], regw[7]);

  bool bad = false;
#pragma unroll
  for (int g = 0; g < 16; ++g) {
    const uint32_t kb = (keepw[g >> 2] >> (8 * (g & 3))) & 0xFFu;
    const uint32_t sb = (signw[g >> 2] >> (8 * (g & 3))) & 0xFFu;
    const uint32_t rg = (regw[g >> 1] >> (16 * (g & 1))) & 0xFFFFu;
    const uint32_t salb = (uint32_t)(((g < 8 ? sal_lo : sal_hi) >> (8 * (g & 7))) & 0xFFull);
    if (valid) {
      if (__popc(kb) != N) bad = true;
      if (N < 8 && ((sb >> N) != 0 || (rg >> (2 * N)) != 0)) bad = true;
    }
    // region 3 must mark exactly the kept weights of salient columns
    uint32_t c3 = 0;
#pragma unroll
    for (int k = 0; k < N; ++k) c3 |= (((rg >> (2 * k)) & 3u) == 3u ? 1u : 0u) << k;
    uint32_t expect = 0, t = kb & salb;
    while (t) {
      const int c = __ffs(t) - 1;
      t &= t - 1;
      expect |= 1u << __popc(kb & ((1u << c) - 1u));
    }
    if (valid && c3 != expect) bad = true;
  }

  // scales and a_sal2, stored at the row's permuted position
  const int pg = lane & 7, pj = lane >> 3;
  const uint32_t A = (sc[0] & 0xFFu) | ((sc[1] & 0xFFu) << 8) | ((sc[2] & 0xFFu) << 16) | ((uint32_t)(sc[3] & 0xFFu) << 24);
  const uint32_t B = (sc[0] >> 8) | ((uint32_t)(sc[1] >> 8) << 8) | ((uint32_t)(sc[2] >> 8) << 16) | ((uint32_t)(sc[3] >> 8) << 24);
  *reinterpret_cast<uint2*>(tile + scale_off(N, pg, pj)) = make_uint2(A, B);
  *reinterpret_cast<uint16_t*>(record + resid_a2_off(pg, pj)) = sc[4];

  // residual codes of the block's salient columns: 0 = +a_sal2, 2 = -a_sal2, 1 = no term
  if (valid && nsal < 32 && (s2 >> nsal) != 0) bad = true;
  {
    int q = 0;
    uint64_t mk = sal_lo;
    int base = 0;
    for (int wq = 0; wq < nrw_b; ++wq) {
      uint32_t word = 0;
#pragma unroll
      for (int q4 = 0; q4 < 4; ++q4) {
        uint32_t code = 1u;
        if (mk == 0 && base == 0) { mk = sal_hi; base = 64; }
        if (mk != 0) {
          const int c = __ffsll((long long)mk) - 1 + base;
          mk &= mk - 1;
          const uint32_t kbit = (keepw[c >> 5] >> (c & 31)) & 1u;
          const uint32_t sbit = (s2 >> q) & 1u;
          if (valid && !kbit && sbit) bad = true;      // a residual sign on a dropped weight
          if (valid && kbit) code = sbit ? 0u : 2u;
          ++q;
        }
        word |= code << code_bit(4 * pj + q4);
      }
      word |= __shfl_xor_sync(0xFFFFFFFFu, word, 8);
      word |= __shfl_xor_sync(0xFFFFFFFFu, word, 16);
      if (lane < 8) *reinterpret_cast<uint32_t*>(record + resid_code_off((uint32_t)wq, lane)) = word;
    }
  }
  __syncwarp();

  // ---- phase 2: lane = (g, t) ----
  const int g = lane >> 2, t = lane & 3;
  uint32_t maskw[4] = {0, 0, 0, 0}, sgn[16], reg[16];
#pragma unroll
  for (int u = 0; u < 16; ++u) {
    const int j = u >> 2, sidx = u & 3;
    const int r = g + 8 * j, grp = 4 * sidx + t;
    maskw[j] |= mask_index(N, sm_keep[wib][r][grp]) << (8 * sidx);
    sgn[u] = sm_sign[wib][r][grp];
    reg[u] = sm_region[wib][r][grp];
  }
  LaneWords<N> w;
  build_lane_words<N>(sgn, reg, true, w);
  if (mask_pairs(N)) {
    // this lane's 16 bytes cover rows g + 16 mt, g + 16 mt + 8 and slots 2 h, 2 h + 1 of all four lanes
    const int mt = t >> 1, h = t & 1;
#pragma unroll
    for (int wq = 0; wq < 4; ++wq) {
      maskw[wq] = 0;
#pragma unroll
      for (int hw = 0; hw < 2; ++hw) {
        const int sidx = 2 * h + (wq >> 1), tq = 2 * (wq & 1) + hw, grp = 4 * sidx + tq;
        const uint32_t i0 = mask_index(N, sm_keep[wib][g + 16 * mt][grp]), i1 = mask_index(N, sm_keep[wib][g + 16 * mt + 8][grp]);
        maskw[wq] |= pair_field(i0, i1) << (16 * hw);
      }
    }
  }
  *reinterpret_cast<uint4*>(tile + lane * 16) = make_uint4(maskw[0], maskw[1], maskw[2], maskw[3]);
  store_planes<N>(tile, off_region(N), w.R, lane);
  store_planes<LaneTile<N>::kFull>(tile, off_sign(N), w.S, lane);
  if (sign_has_half(N)) {
    const uint32_t up = __shfl_down_sync(0xFFFFFFFFu, half_to_upper(w.half), 16);
    if (lane < 16) *reinterpret_cast<uint32_t*>(tile + sign_half_off(N, lane)) = w.half | up;
  }

  if (__any_sync(0xFFFFFFFFu, bad) && lane == 0) {
    hdr->status = (uint32_t)STB_ERR_CORRUPT;
    if (dev_status) *dev_status = STB_ERR_CORRUPT;
  }
}

template <int N>
static cudaError_t launch_pack(const stb_logical& L, uint8_t* packed, int* dev_status,
                               cudaStream_t s) {
  const long long tiles = (long long)((L.n + kTileRows - 1) / kTileRows) * (L.m / kBlock);
  const unsigned grid = (unsigned)((tiles + kPackWarps - 1) / kPackWarps);
  pack_kernel<N><<<grid, kPackWarps * 32, 0, s>>>(L, packed, dev_status);
  return cudaGetLastError();
}

}  // namespace stb

static inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

extern "C" int stb_pack_size(int n, int m, int N, size_t* bytes) {
  if (!bytes) return STB_ERR_ARG;
  if (n < 1 || m < stb::kBlock || m % stb::kBlock != 0) return STB_ERR_SHAPE;
  if (N < 1 || N > 8) return STB_ERR_NM;
  const size_t nblk = (size_t)m / stb::kBlock, ntile = ((size_t)n + 31) / 32;
  *bytes = (size_t)stb::tiles_offset((int)nblk) + ntile * nblk * ((size_t)stb::tile_bytes(N) + (size_t)stb::resid_rt_bytes(1, stb::kMaxResidWords));
  return STB_OK;
}

extern "C" int stb_pack(const stb_logical* L, void* packed, size_t packed_bytes, int* dev_status,
                        void* stream) {
  if (!L || !packed) return STB_ERR_ARG;
  size_t need = 0;
  int rc = stb_pack_size(L->n, L->m, L->N, &need);
  if (rc != STB_OK) return rc;
  if (!L->keep || !L->sign || !L->region || !L->sign2 || !L->salient || !L->scale) return STB_ERR_ARG;
  if (!aligned16(L->keep) || !aligned16(L->sign) || !aligned16(L->region) || !aligned16(L->salient) ||
      (reinterpret_cast<uintptr_t>(L->sign2) & 3u) || (reinterpret_cast<uintptr_t>(L->scale) & 1u) ||
      (reinterpret_cast<uintptr_t>(packed) & 255u))
    return STB_ERR_ARG;
  if (packed_bytes < need) return STB_ERR_SIZE;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  uint8_t* out = static_cast<uint8_t*>(packed);
  stb::header_kernel<<<1, 256, 0, s>>>(L->n, L->m, L->N, L->salient, out, dev_status);
  if (cudaGetLastError() != cudaSuccess) return STB_ERR_CUDA;
  cudaError_t e = cudaSuccess;
  switch (L->N) {
    case 1: e = stb::launch_pack<1>(*L, out, dev_status, s); break;
    case 2: e = stb::launch_pack<2>(*L, out, dev_status, s); break;
    case 3: e = stb::launch_pack<3>(*L, out, dev_status, s); break;
    case 4: e = stb::launch_pack<4>(*L, out, dev_status, s); break;
    case 5: e = stb::launch_pack<5>(*L, out, dev_status, s); break;
    case 6: e = stb::launch_pack<6>(*L, out, dev_status, s); break;
    case 7: e = stb::launch_pack<7>(*L, out, dev_status, s); break;
    case 8: e = stb::launch_pack<8>(*L, out, dev_status, s); break;
  }
  return e == cudaSuccess ? STB_OK : STB_ERR_CUDA;
}

extern "C" int stb_packed_info(const void* packed, stb_info* info, void* stream) {
  if (!packed || !info) return STB_ERR_ARG;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  stb::Header h;
  if (cudaMemcpyAsync(&h, packed, sizeof(h), cudaMemcpyDeviceToHost, s) != cudaSuccess) return STB_ERR_CUDA;
  if (cudaStreamSynchronize(s) != cudaSuccess) return STB_ERR_CUDA;
  if (h.magic != stb::kMagic) return STB_ERR_CORRUPT;
  info->n = h.n; info->m = h.m; info->N = h.N;
  info->status = (int)h.status;
  info->used_bytes = h.used_bytes;
  info->stream_bytes = (h.rt_stride + stb::resid_rt_bytes(h.nblk, h.nrw)) * (uint64_t)h.ntile;
  return STB_OK;
}

extern "C" const char* stb_status_str(int status) {
  switch (status) {
    case STB_OK: return "ok";
    case STB_ERR_ARG: return "bad argument";
    case STB_ERR_SHAPE: return "bad shape (need n >= 1, m a positive multiple of 128)";
    case STB_ERR_NM: return "N outside 1..8";
    case STB_ERR_SIZE: return "buffer too small or batch out of range";
    case STB_ERR_UNSUPPORTED: return "unsupported dtype or mode";
    case STB_ERR_CORRUPT: return "logical layer or packed header failed validation";
    case STB_ERR_TIMEOUT: return "a bounded device-side wait ran out";
    case STB_ERR_CUDA: return "CUDA runtime error";
    default: return "unknown status";
  }
}

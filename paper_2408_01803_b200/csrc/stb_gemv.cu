// stb_gemv: decode GEMV  y[t][i] = sum_j W^[i][j] x[t][j],  batch 1..16, fp32 accumulation.
// The memory-bound decoding stage of Appendix C.2: every packed byte is read once.
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/stb.h"
#include <cooperative_groups.h>
#include <stdlib.h>

#include "stb_decode.cuh"
#include "stb_gemv_fast.cuh"
#include "stb_layout.cuh"

namespace cg = cooperative_groups;

namespace stb {

// -----------------------------------------------------------------------------------------
// Fast batch-1 kernel, N = 4, 5, 6.  Grid: one thread-block cluster of `ksplit` CTAs per row
// tile (32 rows); CTA k of the cluster takes the k-th slice of the 128-column blocks, its 8
// warps take the blocks of the slice round-robin, lane = row.  The packed tiles go straight
// from HBM into registers (one coalesced vector load per field plane, next tile prefetched
// while the current one is decoded); x is staged once per CTA in shared memory, byte-planar.
// Partial sums: 8 warps through shared memory, then the CTAs of the cluster through
// distributed shared memory in rank order, so the result does not depend on timing.
constexpr int kFastWarps = 8;

template <int N>
__global__ void __launch_bounds__(kFastWarps * 32)
gemv_fast_kernel(const uint8_t* __restrict__ packed, int n, int m, const __half* __restrict__ x,
                 void* __restrict__ y, int y_f16, int* dev_status, int ksplit, int bpp) {
  extern __shared__ uint4 smem4[];
  const Header* hdr = reinterpret_cast<const Header*>(packed);
  // every CTA of a cluster takes the same branch here (the header is the same for all)
  if (!header_matches(hdr, n, m, N)) {
    if (threadIdx.x == 0 && dev_status) *dev_status = STB_ERR_CORRUPT;
    return;
  }
  const int nblk = m / kBlock;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int kpart = (int)(blockIdx.x % (unsigned)ksplit), rt = (int)(blockIdx.x / (unsigned)ksplit);
  const int b0 = kpart * bpp, b1 = min(nblk, b0 + bpp);
  const BlockInfo* binfo = reinterpret_cast<const BlockInfo*>(packed + sizeof(Header));
  const uint8_t* rtbase = packed + hdr->tiles_offset + (size_t)rt * hdr->rt_stride;

  // shared memory: [selector tables 2 KB][x byte-planar bpp*256 B][x plain fp16 bpp*256 B][partials]
  uint32_t* tab = reinterpret_cast<uint32_t*>(smem4);
  uint4* xs = smem4 + 128;
  __half* xplain = reinterpret_cast<__half*>(xs + (size_t)bpp * 16);
  float* red = reinterpret_cast<float*>(xplain + (size_t)bpp * kBlock);   // [kFastWarps][32] then [ksplit][32]

  // first tile of this warp: issue its loads before anything else
  fast::Tile<N> cur;
  int b = b0 + warp;
  if (b < b1) fast::load_tile<N>(rtbase + binfo[b].tile_off, lane, (int)binfo[b].res_bytes, cur);

  fast::build_tables(tab, N, threadIdx.x, blockDim.x);
  for (int gidx = threadIdx.x; gidx < (b1 - b0) * 16; gidx += blockDim.x) {
    const uint4 h = __ldg(reinterpret_cast<const uint4*>(x + (size_t)b0 * kBlock) + gidx);
    reinterpret_cast<uint4*>(xplain)[gidx] = h;
    xs[gidx] = make_uint4(fast::prmt(h.x, h.y, 0x6420u), fast::prmt(h.z, h.w, 0x6420u),
                          fast::prmt(h.x, h.y, 0x7531u), fast::prmt(h.z, h.w, 0x7531u));
  }
  __syncthreads();

  float acc = 0.0f;
  while (b < b1) {
    const BlockInfo* bi = binfo + b;
    const int bn = b + kFastWarps;
    fast::Tile<N> nxt;
    if (bn < b1) fast::load_tile<N>(rtbase + binfo[bn].tile_off, lane, (int)binfo[bn].res_bytes, nxt);
    acc += fast::rowblock_dot<N>(cur, xs + (size_t)(b - b0) * 16, tab, lane);
    // residual term of the block's salient columns: a_sal2 * (+-1) * x[col] where kept
    const int nsal = (int)bi->nsal;
    if (nsal) {
      const float a2 = __half2float(__ushort_as_half((unsigned short)cur.sal2));
      const __half* xb = xplain + (size_t)(b - b0) * kBlock;
      float r = 0.0f;
      int t = 0;
#pragma unroll 1
      for (int half = 0; half < 2; ++half) {
        uint64_t mk = bi->salient[half];
        while (mk) {
          const int c = __ffsll((long long)mk) - 1 + 64 * half;
          mk &= mk - 1;
          const int wi = c >> 5;
          const uint32_t mw = wi == 0 ? cur.mask[0] : (wi == 1 ? cur.mask[1] : (wi == 2 ? cur.mask[2] : cur.mask[3]));
          const float xv = __half2float(xb[c]);
          const float sv = ((cur.resid >> t) & 1u) ? xv : -xv;
          r += ((mw >> (c & 31)) & 1u) ? sv : 0.0f;
          ++t;
        }
      }
      acc = fmaf(a2, r, acc);
    }
    if (bn < b1) cur = nxt;
    b = bn;
  }

  red[warp * 32 + lane] = acc;
  __syncthreads();
  float s = 0.0f;
  if (warp == 0) {
#pragma unroll
    for (int w = 0; w < kFastWarps; ++w) s += red[w * 32 + lane];
  }
  const int row = rt * kTileRows + lane;
  if (ksplit == 1) {
    if (warp == 0 && row < n) {
      if (y_f16) static_cast<__half*>(y)[row] = __float2half_rn(s);
      else static_cast<float*>(y)[row] = s;
    }
    return;
  }
  cg::cluster_group cluster = cg::this_cluster();
  float* part = red + kFastWarps * 32;                       // [ksplit][32], used on cluster rank 0
  if (warp == 0) {
    float* dst = cluster.map_shared_rank(part, 0);
    dst[kpart * 32 + lane] = s;
  }
  cluster.sync();
  if (kpart == 0 && warp == 0 && row < n) {
    float tsum = 0.0f;
    for (int k = 0; k < ksplit; ++k) tsum += part[k * 32 + lane];
    if (y_f16) static_cast<__half*>(y)[row] = __float2half_rn(tsum);
    else static_cast<float*>(y)[row] = tsum;
  }
}

static int fast_ksplit(int n, int m) {
  static int forced = -1;
  if (forced < 0) {
    const char* e = getenv("STB_GEMV_KSPLIT");
    forced = e ? atoi(e) : 0;
  }
  const int ntile = (n + kTileRows - 1) / kTileRows, nblk = m / kBlock;
  int ks = 1;
  if (forced == 1 || forced == 2 || forced == 4 || forced == 8) ks = forced;
  else
    while (ks < 8 && ntile * ks < 444 && nblk / (2 * ks) >= kFastWarps) ks *= 2;
  while (ks > 1 && ks > nblk) ks /= 2;
  return ks;
}

template <int N>
static cudaError_t launch_fast(const uint8_t* packed, int n, int m, const __half* x, void* y, int y_f16,
                               int* dev_status, cudaStream_t s) {
  const int ntile = (n + kTileRows - 1) / kTileRows, nblk = m / kBlock;
  const int ksplit = fast_ksplit(n, m);
  const int bpp = (nblk + ksplit - 1) / ksplit;
  const size_t smem = 2048 + (size_t)bpp * 512 + (kFastWarps + 8) * 32 * sizeof(float);
  static bool attr_done[9] = {false};
  if (smem > 48 * 1024 && !attr_done[N]) {
    cudaError_t e = cudaFuncSetAttribute(gemv_fast_kernel<N>, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
    if (e != cudaSuccess) return e;
    attr_done[N] = true;
  }
  if (smem > 200 * 1024) return cudaErrorInvalidValue;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)(ntile * ksplit), 1, 1);
  cfg.blockDim = dim3(kFastWarps * 32, 1, 1);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = s;
  cudaLaunchAttribute at[1];
  at[0].id = cudaLaunchAttributeClusterDimension;
  at[0].val.clusterDim.x = (unsigned)ksplit; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
  cfg.attrs = at; cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, gemv_fast_kernel<N>, packed, n, m, x, y, y_f16, dev_status, ksplit, bpp);
}

// -----------------------------------------------------------------------------------------
// General kernel: any N in 1..8, batch <= BT.  One CTA per row tile (32 rows), 8 warps split
// the blocks, lane = row; position-order decode, x read through L1 (all lanes of a warp read
// the same address).  Partial sums of the 8 warps are combined in shared memory in a fixed
// order, so the result is deterministic.
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
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int rt = blockIdx.x;
  const BlockInfo* binfo = reinterpret_cast<const BlockInfo*>(packed + sizeof(Header));
  const uint8_t* rtbase = packed + hdr->tiles_offset + (size_t)rt * hdr->rt_stride;

  float acc[BT];
#pragma unroll
  for (int t = 0; t < BT; ++t) acc[t] = 0.0f;

  for (int b = warp; b < nblk; b += 8) {
    const BlockInfo* bi = binfo + b;
    RowBlock<N> r;
    load_rowblock<N>(rtbase + bi->tile_off, lane, (int)bi->res_bytes, r);
    const uint64_t sal[2] = {bi->salient[0], bi->salient[1]};
    int tbase = 0;
#pragma unroll
    for (int g = 0; g < 16; ++g) {
      const uint32_t salb = (uint32_t)((sal[g >> 3] >> (8 * (g & 7))) & 0xFFull);
      float v[8];
      decode_group<N>(r, g, salb, tbase, v);
      tbase += __popc(salb);
#pragma unroll
      for (int t = 0; t < BT; ++t) {
        if (t < batch) {
          const uint4 xv = __ldg(reinterpret_cast<const uint4*>(x + (size_t)t * ldx + (size_t)b * kBlock + g * 8));
          const __half2* xh = reinterpret_cast<const __half2*>(&xv);
#pragma unroll
          for (int c = 0; c < 4; ++c) {
            const float2 xf = __half22float2(xh[c]);
            acc[t] = fmaf(v[2 * c], xf.x, acc[t]);
            acc[t] = fmaf(v[2 * c + 1], xf.y, acc[t]);
          }
        }
      }
    }
  }

  __shared__ float red[8][BT][32];
#pragma unroll
  for (int t = 0; t < BT; ++t) red[warp][t][lane] = acc[t];
  __syncthreads();
  for (int idx = threadIdx.x; idx < BT * 32; idx += blockDim.x) {
    const int t = idx >> 5, l = idx & 31;
    const int row = rt * kTileRows + l;
    if (t < batch && row < n) {
      float s = 0.0f;
#pragma unroll
      for (int w = 0; w < 8; ++w) s += red[w][t][l];
      if (y_f16) static_cast<__half*>(y)[(size_t)t * ldy + row] = __float2half_rn(s);
      else static_cast<float*>(y)[(size_t)t * ldy + row] = s;
    }
  }
}

template <int N>
static cudaError_t launch_general(const uint8_t* packed, int n, int m, const __half* x, int batch,
                                  size_t ldx, void* y, int y_f16, size_t ldy, int* dev_status, cudaStream_t s) {
  const unsigned grid = (unsigned)((n + kTileRows - 1) / kTileRows);
  if (batch == 1) gemv_general_kernel<N, 1><<<grid, 256, 0, s>>>(packed, n, m, x, batch, ldx, y, y_f16, ldy, dev_status);
  else if (batch <= 4) gemv_general_kernel<N, 4><<<grid, 256, 0, s>>>(packed, n, m, x, batch, ldx, y, y_f16, ldy, dev_status);
  else gemv_general_kernel<N, 16><<<grid, 256, 0, s>>>(packed, n, m, x, batch, ldx, y, y_f16, ldy, dev_status);
  return cudaGetLastError();
}

}  // namespace stb

extern "C" int stb_gemv(const void* packed, int n, int m, int N, const void* x, int batch, size_t ldx,
                        void* y, stb_dtype ydt, size_t ldy, int* dev_status, void* stream) {
  if (!packed || !x || !y) return STB_ERR_ARG;
  if (n < 1 || m < stb::kBlock || m % stb::kBlock != 0) return STB_ERR_SHAPE;
  if (N < 1 || N > 8) return STB_ERR_NM;
  if (batch < 1 || batch > 16) return STB_ERR_SIZE;
  if (ydt != STB_F32 && ydt != STB_F16) return STB_ERR_UNSUPPORTED;
  const int y_f16 = ydt == STB_F16;
  if (ldx < (size_t)m || ldy < (size_t)n || (ldx % 8) != 0 || (reinterpret_cast<uintptr_t>(x) & 15u)) return STB_ERR_ARG;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  const uint8_t* p = static_cast<const uint8_t*>(packed);
  const __half* xh = static_cast<const __half*>(x);
  cudaError_t e = cudaSuccess;
  if (batch == 1 && N >= 4 && N <= 6) {
    if (N == 4) e = stb::launch_fast<4>(p, n, m, xh, y, y_f16, dev_status, s);
    else if (N == 5) e = stb::launch_fast<5>(p, n, m, xh, y, y_f16, dev_status, s);
    else e = stb::launch_fast<6>(p, n, m, xh, y, y_f16, dev_status, s);
    return e == cudaSuccess ? STB_OK : STB_ERR_CUDA;
  }
  switch (N) {
    case 1: e = stb::launch_general<1>(p, n, m, xh, batch, ldx, y, y_f16, ldy, dev_status, s); break;
    case 2: e = stb::launch_general<2>(p, n, m, xh, batch, ldx, y, y_f16, ldy, dev_status, s); break;
    case 3: e = stb::launch_general<3>(p, n, m, xh, batch, ldx, y, y_f16, ldy, dev_status, s); break;
    case 4: e = stb::launch_general<4>(p, n, m, xh, batch, ldx, y, y_f16, ldy, dev_status, s); break;
    case 5: e = stb::launch_general<5>(p, n, m, xh, batch, ldx, y, y_f16, ldy, dev_status, s); break;
    case 6: e = stb::launch_general<6>(p, n, m, xh, batch, ldx, y, y_f16, ldy, dev_status, s); break;
    case 7: e = stb::launch_general<7>(p, n, m, xh, batch, ldx, y, y_f16, ldy, dev_status, s); break;
    case 8: e = stb::launch_general<8>(p, n, m, xh, batch, ldx, y, y_f16, ldy, dev_status, s); break;
  }
  return e == cudaSuccess ? STB_OK : STB_ERR_CUDA;
}

extern "C" int stb_layer_stack(const stb_step* steps, int count, int* dev_status, void* stream) {
  if (!steps || count < 0) return STB_ERR_ARG;
  for (int i = 0; i < count; ++i) {
    const stb_step& st = steps[i];
    int rc = stb_gemv(st.packed, st.n, st.m, st.N, st.in, st.batch, st.ldin, st.out, st.odt, st.ldout,
                      dev_status, stream);
    if (rc != STB_OK) return rc;
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

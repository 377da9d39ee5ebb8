// stb_gemv: decode GEMV  y[t][i] = sum_j W^[i][j] x[t][j],  batch 1..16, fp32 accumulation.
// The memory-bound decoding stage of Appendix C.2: every packed byte is read once.
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/stb.h"
#include "stb_decode.cuh"
#include "stb_layout.cuh"

namespace stb {

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

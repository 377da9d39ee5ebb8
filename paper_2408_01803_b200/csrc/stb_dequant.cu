// stb_dequant: decode a packed layer to a dense row-major matrix (parity hook).  fp32 output
// is exactly the definition  s * a_region  /  fl32(s1 a_sal1 + s2 a_sal2)  /  0  (Eq. 1, Eq. 4).
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/stb.h"
#include "stb_decode.cuh"
#include "stb_layout.cuh"

namespace stb {

template <typename T> __device__ __forceinline__ T cvt_out(float v);
template <> __device__ __forceinline__ float cvt_out<float>(float v) { return v; }
template <> __device__ __forceinline__ __half cvt_out<__half>(float v) { return __float2half_rn(v); }
template <> __device__ __forceinline__ __nv_bfloat16 cvt_out<__nv_bfloat16>(float v) { return __float2bfloat16_rn(v); }

// One warp per tile; lane = (g, t) decodes its 16 (row, group) slots, 8 columns each.
template <int N, typename T>
__global__ void __launch_bounds__(256)
dequant_kernel(const uint8_t* __restrict__ packed, int n, int m, T* __restrict__ W, size_t ldw) {
  const Header* hdr = reinterpret_cast<const Header*>(packed);
  if (!header_matches(hdr, n, m, N)) return;
  const int nblk = m / kBlock;
  const int ntile = (n + kTileRows - 1) / kTileRows;
  const int lane = threadIdx.x & 31, g = lane >> 2, t = lane & 3;
  const long long warp = (long long)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  if (warp >= (long long)ntile * nblk) return;
  const int rt = (int)(warp / nblk), b = (int)(warp % nblk);
  const BlockInfo* bi = reinterpret_cast<const BlockInfo*>(packed + sizeof(Header)) + b;
  const uint8_t* tile = packed + hdr->tiles_offset + ((size_t)rt * nblk + b) * (size_t)hdr->tile_bytes;
  const int nslot = 4 * (int)bi->nrw;
  const uint8_t* record = packed + hdr->tiles_offset + hdr->rt_stride * (size_t)ntile +
                          (size_t)rt * resid_rt_bytes(nblk, hdr->nrw) + resid_block_off(b, bi->rw_off);
  LaneTile<N> lt;
  load_lane_tile<N>(tile, lane, lt);
  const uint64_t sal[2] = {bi->salient[0], bi->salient[1]};
  for (int u = 0; u < 16; ++u) {
    const int j = u >> 2, s = u & 3;
    const int row = rt * kTileRows + g + 8 * j;
    const int grp = 4 * s + t;                                   // group of the block
    uint32_t code[8], neg[8];
    plain_slot<N>(lt, u, code, neg);
    if (row >= n) continue;
    const uint32_t salb = (uint32_t)((sal[grp >> 3] >> (8 * (grp & 7))) & 0xFFull);
    // number of salient columns of the block before this group
    int qbase = grp >= 8 ? __popcll(sal[0]) : 0;
    qbase += __popcll(sal[grp >> 3] & ((1ull << (8 * (grp & 7))) - 1ull));
    float alpha[5];
    for (int q = 0; q < 4; ++q) alpha[q] = __half2float(__ushort_as_half((unsigned short)scale_bits<N>(lt, j, q)));
    alpha[4] = __half2float(__ushort_as_half((unsigned short)sal2_bits(record, g, j)));
    T* dst = W + (size_t)row * ldw + (size_t)b * kBlock + grp * 8;
    for (int c = 0; c < 8; ++c) {
      float v = 0.0f;
      if (code[c] < 4u) {
        const float s1 = neg[c] ? -1.0f : 1.0f;
        if (code[c] == 3u) {
          const int q = qbase + __popc(salb & ((1u << c) - 1u));
          const uint32_t word = q < nslot ? resid_word(record, (uint32_t)(q >> 2), g) : 0x55555555u;
          const uint32_t rc = resid_code(word, j, q & 3);
          const float s2 = rc == 0u ? 1.0f : -1.0f;
          v = __fadd_rn(s1 * alpha[3], s2 * alpha[4]);
        } else {
          v = s1 * alpha[code[c]];
        }
      }
      dst[c] = cvt_out<T>(v);
    }
  }
}

template <int N>
static cudaError_t launch_dequant(const uint8_t* packed, int n, int m, void* W, stb_dtype dt,
                                  size_t ldw, cudaStream_t s) {
  const long long tiles = (long long)((n + kTileRows - 1) / kTileRows) * (m / kBlock);
  const unsigned grid = (unsigned)((tiles + 7) / 8);
  if (dt == STB_F32) dequant_kernel<N, float><<<grid, 256, 0, s>>>(packed, n, m, (float*)W, ldw);
  else if (dt == STB_F16) dequant_kernel<N, __half><<<grid, 256, 0, s>>>(packed, n, m, (__half*)W, ldw);
  else dequant_kernel<N, __nv_bfloat16><<<grid, 256, 0, s>>>(packed, n, m, (__nv_bfloat16*)W, ldw);
  return cudaGetLastError();
}

}  // namespace stb

extern "C" int stb_dequant(const void* packed, int n, int m, int N, void* W, stb_dtype dt,
                           size_t ldw, void* stream) {
  if (!packed || !W) return STB_ERR_ARG;
  if (n < 1 || m < stb::kBlock || m % stb::kBlock != 0) return STB_ERR_SHAPE;
  if (N < 1 || N > 8) return STB_ERR_NM;
  if (ldw < (size_t)m) return STB_ERR_ARG;
  if (dt != STB_F32 && dt != STB_F16 && dt != STB_BF16) return STB_ERR_UNSUPPORTED;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  const uint8_t* p = static_cast<const uint8_t*>(packed);
  cudaError_t e = cudaSuccess;
  switch (N) {
    case 1: e = stb::launch_dequant<1>(p, n, m, W, dt, ldw, s); break;
    case 2: e = stb::launch_dequant<2>(p, n, m, W, dt, ldw, s); break;
    case 3: e = stb::launch_dequant<3>(p, n, m, W, dt, ldw, s); break;
    case 4: e = stb::launch_dequant<4>(p, n, m, W, dt, ldw, s); break;
    case 5: e = stb::launch_dequant<5>(p, n, m, W, dt, ldw, s); break;
    case 6: e = stb::launch_dequant<6>(p, n, m, W, dt, ldw, s); break;
    case 7: e = stb::launch_dequant<7>(p, n, m, W, dt, ldw, s); break;
    case 8: e = stb::launch_dequant<8>(p, n, m, W, dt, ldw, s); break;
  }
  return e == cudaSuccess ? STB_OK : STB_ERR_CUDA;
}

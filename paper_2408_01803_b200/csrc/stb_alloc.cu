// Layer-wise N:M assignment (Section 3.3, "Layer-wise N:M Assignment"): the L2 norm of every layer's dense weights,
// then N_i / 8 = alpha_i + (1 - alpha_i) R_target with alpha_i = omega_i / sum_k omega_k.  Offline, before the layers
// are quantized and packed with their N.
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <math.h>
#include <stdint.h>

#include "../../include/stb.h"

namespace stb {

// Sum of squares of an fp16 matrix, accumulated in float64 (the square of an fp16 value is exact in float32; for
// weights of ordinary range the float64 sum is exact too, so the order of the additions does not show).
__global__ void __launch_bounds__(256)
sumsq_kernel(const __half* __restrict__ W, int n, int m, size_t ldw, double* __restrict__ out) {
  double acc = 0.0;
  const int m8 = m / 8;
  const size_t total = (size_t)n * (size_t)m8;
  for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (size_t)gridDim.x * blockDim.x) {
    const size_t r = i / (size_t)m8, c = i % (size_t)m8;
    const uint4 v = *reinterpret_cast<const uint4*>(W + r * ldw + c * 8);
    const __half2* h = reinterpret_cast<const __half2*>(&v);
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      const float2 f = __half22float2(h[k]);
      acc += (double)(f.x * f.x) + (double)(f.y * f.y);
    }
  }
  for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < (size_t)n * (size_t)(m - 8 * m8); i += (size_t)gridDim.x * blockDim.x) {
    const size_t r = i / (size_t)(m - 8 * m8), c = 8 * (size_t)m8 + i % (size_t)(m - 8 * m8);
    const float f = __half2float(W[r * ldw + c]);
    acc += (double)(f * f);
  }
#pragma unroll
  for (int d = 16; d > 0; d >>= 1) acc += __shfl_xor_sync(0xFFFFFFFFu, acc, d);
  __shared__ double part[8];
  if ((threadIdx.x & 31) == 0) part[threadIdx.x >> 5] = acc;
  __syncthreads();
  if (threadIdx.x == 0) {
    double s = 0.0;
    for (int w = 0; w < 8; ++w) s += part[w];
    atomicAdd(out, s);
  }
}

}  // namespace stb

extern "C" int stb_weight_sumsq(const void* W, int n, int m, size_t ldw, double* sumsq, void* stream) {
  if (!W || !sumsq) return STB_ERR_ARG;
  if (n < 1 || m < 1) return STB_ERR_SHAPE;
  if (ldw < (size_t)m || (ldw % 8) != 0 || (reinterpret_cast<uintptr_t>(W) & 15u)) return STB_ERR_ARG;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  stb::sumsq_kernel<<<148 * 4, 256, 0, s>>>(static_cast<const __half*>(W), n, m, ldw, sumsq);
  return cudaGetLastError() == cudaSuccess ? STB_OK : STB_ERR_CUDA;
}

extern "C" int stb_allocate_nm(const double* sumsq, int layers, double r_target, int* N_out) {
  if (!sumsq || !N_out || layers < 1) return STB_ERR_ARG;
  if (!(r_target > 0.0) || r_target > 1.0) return STB_ERR_ARG;
  double total = 0.0;
  for (int i = 0; i < layers; ++i) {
    if (!(sumsq[i] >= 0.0)) return STB_ERR_ARG;
    total += sqrt(sumsq[i]);
  }
  for (int i = 0; i < layers; ++i) {
    const double alpha = total > 0.0 ? sqrt(sumsq[i]) / total : 0.0;
    const double ratio = alpha + (1.0 - alpha) * r_target;
    int Ni = (int)nearbyint(8.0 * ratio);
    N_out[i] = Ni < 1 ? 1 : (Ni > 8 ? 8 : Ni);
  }
  return STB_OK;
}

// stb_gemm: prefill GEMM on the tensor cores (placeholder translation unit until the tcgen05
// kernel lands; the entry points exist so that the library exports its whole C ABI).
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/stb.h"
#include "stb_layout.cuh"

extern "C" int stb_gemm_workspace(int n, int m, int N, int T, size_t* bytes) {
  if (!bytes) return STB_ERR_ARG;
  if (n < 1 || m < stb::kBlock || m % stb::kBlock != 0 || T < 1) return STB_ERR_SHAPE;
  if (N < 1 || N > 8) return STB_ERR_NM;
  *bytes = 0;
  return STB_OK;
}

extern "C" int stb_gemm(const void* packed, int n, int m, int N, const void* X, int T, size_t ldx,
                        void* Y, stb_dtype ydt, size_t ldy, void* ws, size_t ws_bytes,
                        int* dev_status, void* stream) {
  (void)packed; (void)n; (void)m; (void)N; (void)X; (void)T; (void)ldx; (void)Y; (void)ydt;
  (void)ldy; (void)ws; (void)ws_bytes; (void)dev_status; (void)stream;
  return STB_ERR_UNSUPPORTED;
}

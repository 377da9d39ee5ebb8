// Small PTX wrappers and the keep-byte position table shared by the GEMV and GEMM kernels.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace stb {

// Position selectors by keep-mask index (see position_selector in stb_decode.cuh): entry
// [N][i] is {selector of columns 0..3, selector of columns 4..7} of the i-th mask with N bits,
// each in the low 16 bits of a word.
struct PosTable { uint2 v[9][72]; };
constexpr PosTable make_pos_table() {
  PosTable t{};
  for (int N = 0; N <= 8; ++N) {
    int k = 0;
    for (uint32_t m = 0; m < 256; ++m) {
      uint32_t p = 0, r = 0;
      for (int c = 0; c < 8; ++c) {
        if ((m >> c) & 1u) { p |= (r & 7u) << (4 * c); ++r; }
        else p |= 7u << (4 * c);
      }
      if ((int)r == N) { t.v[N][k].x = p & 0xFFFFu; t.v[N][k].y = p >> 16; ++k; }
    }
  }
  return t;
}
__device__ const PosTable g_pos_table = make_pos_table();
constexpr int kPosTableEntries = 72;

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile("{\n\t.reg .pred p;\n\t"
               "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
               "selp.u32 %0, 1, 0, p;\n\t}"
               : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
  return ok != 0;
}
// Bounded wait: gives up after `limit` SM clock cycles and returns false.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, long long limit) {
  if (mbar_try_wait(bar, parity)) return true;
  const long long t0 = clock64();
  while (!mbar_try_wait(bar, parity))
    if (clock64() - t0 > limit) return false;
  return true;
}
// generic-proxy accesses to shared memory before, async-proxy (bulk copy, tensor core) after
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

// 1-D bulk copy global -> shared (both 16-byte aligned, bytes a multiple of 16); completion is
// signalled on an mbarrier of this CTA
__device__ __forceinline__ void bulk_g2s(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
               ::"r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}

// Split cluster barrier: every thread of every CTA of the cluster arrives, and later waits for all arrivals.
__device__ __forceinline__ void cluster_arrive() { asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory"); }
__device__ __forceinline__ void cluster_wait() { asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory"); }

// Programmatic dependent launch: wait until the grid this one depends on has completed and its
// memory is visible (no-op for an ordinary launch) / allow the dependent grid to be scheduled.
__device__ __forceinline__ void grid_dependency_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void grid_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
// a pointer to data of the producer grid: anything computed from the returned value stays behind the wait
template <typename T>
__device__ __forceinline__ const T* after_dependency_wait(const T* p) {
  asm volatile("" : "+l"(p) :: "memory");
  return p;
}

// Read-only loads through L1.  Not volatile: the compiler may move and batch them.  The data must not change
// while the kernel runs; a kernel that waits for its producer grid passes pointers through after_dependency_wait.
__device__ __forceinline__ uint4 ldg_nc_v4(const void* p) {
  uint4 v;
  asm("ld.global.nc.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
  return v;
}

// D(16x8, fp32) += A(16x16, fp16, row) * B(16x8, fp16, col)
__device__ __forceinline__ void mma16816(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                         uint32_t b0, uint32_t b1) {
  asm("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
               : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
               : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// D(16x8, fp32) += A(16x32, fp16, 2:4 sparse, 16x16 stored) * B(32x8, fp16, col).  `meta` of the lanes 2 f
// and 2 f + 1 of every quad (f = kUpper) holds the two-bit column indices: lane 2 f the chunks (groups of four
// columns) 0..3, lane 2 f + 1 the chunks 4..7; bits 0..15 for row lane / 4, bits 16..31 for row lane / 4 + 8.
template <int kUpper>
__device__ __forceinline__ void mma_sp16832(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                            uint32_t b0, uint32_t b1, uint32_t b2, uint32_t b3, uint32_t meta) {
  if (kUpper)
    asm("mma.sp::ordered_metadata.sync.aligned.m16n8k32.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9,%10,%11}, {%0,%1,%2,%3}, %12, 0x1;"
                 : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
                 : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1), "r"(b2), "r"(b3), "r"(meta));
  else
    asm("mma.sp::ordered_metadata.sync.aligned.m16n8k32.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9,%10,%11}, {%0,%1,%2,%3}, %12, 0x0;"
                 : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
                 : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1), "r"(b2), "r"(b3), "r"(meta));
}
__device__ __forceinline__ uint32_t ldg_nc_u32(const void* p) {
  uint32_t v;
  asm("ld.global.nc.u32 %0, [%1];" : "=r"(v) : "l"(p));
  return v;
}

}  // namespace stb

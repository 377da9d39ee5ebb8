// stb_quantize: the paper's quantizer on the GPU -- Standardized Importance (Eq. 3), N of 8 per group (Section 3.3),
// the salient-column search and the break-point search of Algorithm 2, residual binarization (Eq. 4) and
// trisection -- i.e. the block loop of Algorithm 1 without its Hessian update, from a dense fp16 layer and the column
// norms of the calibration activations to the logical arrays stb_pack takes.  The paper runs this step in
// PyTorch for hours per model (Section 4.1); here every stage is a kernel.
//
// All arithmetic is float64 and written so that the result does not depend on how the work is split:
//   * sums of |w| and w^2 of fp16 values are exact in float64 for weights of ordinary range, so rows, columns and
//     blocks can be summed in any order;
//   * every sum that is NOT exact (the error of a candidate over the rows of a block, a row's residual scale) is
//     taken sequentially, in the order the definition states, by one thread;
//   * products and differences are never fused into multiply-adds.
// The layer-wide mean and deviation of Eq. 3 are the one exception: they are tree sums (their rounding moves every
// score by the same relative 1e-16, which can change a keep mask only where two scores of a group tie to that
// precision).
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <math.h>
#include <stdint.h>

#include "../../include/stb.h"

namespace stb {
namespace quant {

constexpr int kBeta = 128, kM = 8, kMaxSal = 32, kGrid = 160;
constexpr int kPartials = 2048;

struct Ws {
  double* rowsum;      // [n]
  double* colsum;      // [m]
  double* colsq;       // [m]
  double* partial;     // [kPartials]
  double* scalars;     // [0] mean, [1] sd, [2] lambda
  int* order;          // [nblk][32] candidate columns, best first
  double* serr;        // [nblk][32]
  int* nstar;          // [nblk]
  uint8_t* salflag;    // [nblk][128]
  double* mx;          // [nblk]
  double* berr;        // [nblk][160]
  double* bp;          // [nblk][2]
};

__device__ __forceinline__ double w_at(const __half* W, size_t ldw, int i, int j) { return (double)__half2float(W[(size_t)i * ldw + j]); }
__device__ __forceinline__ bool kept_at(const uint8_t* keep, int ngrp, int i, int j) { return (keep[(size_t)i * ngrp + (j >> 3)] >> (j & 7)) & 1u; }
// error of binarizing a set with sum of squares q, l1 sum a, count k: q - k alpha^2, alpha = a / k (no fused operations)
__device__ __forceinline__ double binary_error(double q, double a, int k) {
  if (k == 0) return 0.0;
  const double alpha = __ddiv_rn(a, (double)k);
  return __dsub_rn(q, __dmul_rn(__dmul_rn((double)k, alpha), alpha));
}
__device__ __forceinline__ double warp_sum(double v) {
#pragma unroll
  for (int d = 16; d > 0; d >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, d);
  return v;
}
__device__ __forceinline__ int warp_sum_int(int v) {
#pragma unroll
  for (int d = 16; d > 0; d >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, d);
  return v;
}

// ---- Eq. 3, sums of |W| per row (one warp per row) and per column, sums of W^2 per column -------------------------
__global__ void rowsum_kernel(const __half* __restrict__ W, size_t ldw, int n, int m, double* __restrict__ rowsum) {
  const int row = (int)((blockIdx.x * (size_t)blockDim.x + threadIdx.x) >> 5), lane = threadIdx.x & 31;
  if (row >= n) return;
  double s = 0.0;
  for (int j = lane; j < m; j += 32) s += fabs(w_at(W, ldw, row, j));
  s = warp_sum(s);
  if (lane == 0) rowsum[row] = s;
}
__global__ void colsum_kernel(const __half* __restrict__ W, size_t ldw, int n, int m, double* __restrict__ colsum, double* __restrict__ colsq) {
  const int j = blockIdx.x * blockDim.x + threadIdx.x;
  if (j >= m) return;
  const int r0 = blockIdx.y * 64, r1 = min(n, r0 + 64);
  double s = 0.0, q = 0.0;
  for (int i = r0; i < r1; ++i) { const double w = w_at(W, ldw, i, j); s += fabs(w); q += w * w; }
  atomicAdd(colsum + j, s);      // exact sums: the order of the additions does not show
  atomicAdd(colsq + j, q);
}
__device__ __forceinline__ double mu_at(const __half* W, size_t ldw, const double* rowsum, const double* colsum, int i, int j) {
  const double a = fabs(w_at(W, ldw, i, j));
  double mu = 0.0;
  if (rowsum[i] > 0.0) mu = __dadd_rn(mu, __ddiv_rn(a, rowsum[i]));
  if (colsum[j] > 0.0) mu = __dadd_rn(mu, __ddiv_rn(a, colsum[j]));
  return mu;
}
// pass 0: sum of mu; pass 1: sum of (mu - mean)^2; per-block partials, finished by one thread
__global__ void mu_partial_kernel(const __half* __restrict__ W, size_t ldw, int n, int m, const double* __restrict__ rowsum,
                                  const double* __restrict__ colsum, const double* __restrict__ scalars, int pass, double* __restrict__ partial) {
  const double mean = scalars[0];
  double acc = 0.0;
  const size_t total = (size_t)n * m;
  for (size_t t = (size_t)blockIdx.x * blockDim.x + threadIdx.x; t < total; t += (size_t)gridDim.x * blockDim.x) {
    const int i = (int)(t / m), j = (int)(t % m);
    const double mu = mu_at(W, ldw, rowsum, colsum, i, j);
    acc += pass == 0 ? mu : (mu - mean) * (mu - mean);
  }
  acc = warp_sum(acc);
  __shared__ double part[8];
  if ((threadIdx.x & 31) == 0) part[threadIdx.x >> 5] = acc;
  __syncthreads();
  if (threadIdx.x == 0) {
    double s = 0.0;
    for (int w = 0; w < 8; ++w) s += part[w];
    partial[blockIdx.x] = s;
  }
}
__global__ void mu_finish_kernel(const double* __restrict__ partial, int nparts, double count, int pass, double* __restrict__ scalars) {
  double s = 0.0;
  for (int i = 0; i < nparts; ++i) s += partial[i];
  if (pass == 0) scalars[0] = s / count;
  else scalars[1] = sqrt(s / count);
}
// lambda < 0: the reading 0.01 * mean_j h_jj, h_jj = 2 ||X_:,j||^2 (summed in column order)
__global__ void lambda_kernel(const double* __restrict__ xnorm, int m, double lambda_in, double* __restrict__ scalars) {
  double lam = lambda_in;
  if (lam < 0.0) {
    double mh = 0.0;
    for (int j = 0; j < m; ++j) mh = __dadd_rn(mh, __dmul_rn(__dmul_rn(2.0, xnorm[j]), xnorm[j]));
    lam = __ddiv_rn(__dmul_rn(0.01, mh), (double)m);
  }
  scalars[2] = lam;
}

// ---- Section 3.3: keep the N highest scores of every 8 columns (ties: lower column) ---------------------------------
__global__ void select_kernel(const __half* __restrict__ W, size_t ldw, int n, int m, int N, const double* __restrict__ rowsum,
                              const double* __restrict__ colsum, const double* __restrict__ xnorm, const double* __restrict__ scalars,
                              uint8_t* __restrict__ keep) {
  const int ngrp = m / kM;
  const size_t t = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (t >= (size_t)n * ngrp) return;
  const int i = (int)(t / ngrp), gq = (int)(t % ngrp);
  const double mean = scalars[0], sd = scalars[1];
  double s[kM];
#pragma unroll
  for (int c = 0; c < kM; ++c) {
    const int j = gq * kM + c;
    const double mu = mu_at(W, ldw, rowsum, colsum, i, j);
    const double z = sd > 0.0 ? __ddiv_rn(__dsub_rn(mu, mean), sd) : 0.0;
    s[c] = __dmul_rn(z, xnorm[j]);
  }
  uint32_t bits = 0;
#pragma unroll
  for (int c = 0; c < kM; ++c) {
    int rank = 0;
#pragma unroll
    for (int a = 0; a < kM; ++a) rank += (s[a] > s[c] || (s[a] == s[c] && a < c)) ? 1 : 0;
    if (rank < N) bits |= 1u << c;
  }
  keep[t] = (uint8_t)bits;
}

// ---- Algorithm 2, Salient: candidate order of a block (one CTA of 128 threads per block) ---------------------------
__global__ void candidates_kernel(const double* __restrict__ colsq, const double* __restrict__ xnorm, const double* __restrict__ scalars,
                                  int* __restrict__ order) {
  __shared__ double score[kBeta];
  const int b = blockIdx.x, c = threadIdx.x, j = b * kBeta + c;
  score[c] = __dmul_rn(__dadd_rn(__dmul_rn(__dmul_rn(2.0, xnorm[j]), xnorm[j]), scalars[2]), colsq[j]);
  __syncthreads();
  int rank = 0;
  for (int a = 0; a < kBeta; ++a) rank += (score[a] > score[c] || (score[a] == score[c] && a < c)) ? 1 : 0;
  if (rank < kMaxSal) order[b * kMaxSal + rank] = c;
}
// error of taking the first i candidates as salient: one warp per (block, i); exact per-row sums, rows added in order
__global__ void salient_err_kernel(const __half* __restrict__ W, size_t ldw, int n, int m, const uint8_t* __restrict__ keep,
                                   const int* __restrict__ order, double* __restrict__ serr) {
  const int warp = (int)((blockIdx.x * (size_t)blockDim.x + threadIdx.x) >> 5), lane = threadIdx.x & 31;
  const int nblk = m / kBeta, ngrp = m / kM;
  if (warp >= nblk * kMaxSal) return;
  const int b = warp / kMaxSal, i = warp % kMaxSal + 1;
  bool sal[4];
#pragma unroll
  for (int k = 0; k < 4; ++k) {
    sal[k] = false;
    for (int t = 0; t < i; ++t) sal[k] = sal[k] || order[b * kMaxSal + t] == 4 * lane + k;
  }
  double err = 0.0;
  for (int r = 0; r < n; ++r) {
    double q0 = 0, q1 = 0, a0 = 0, a1 = 0;
    int k0 = 0, k1 = 0;
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      const int j = b * kBeta + 4 * lane + k;
      if (!kept_at(keep, ngrp, r, j)) continue;
      const double w = w_at(W, ldw, r, j);
      if (sal[k]) { q1 += w * w; a1 += fabs(w); ++k1; } else { q0 += w * w; a0 += fabs(w); ++k0; }
    }
    q0 = warp_sum(q0); q1 = warp_sum(q1); a0 = warp_sum(a0); a1 = warp_sum(a1);
    k0 = warp_sum_int(k0); k1 = warp_sum_int(k1);
    err = __dadd_rn(err, __dadd_rn(binary_error(q1, a1, k1), binary_error(q0, a0, k0)));
  }
  if (lane == 0) serr[b * kMaxSal + i - 1] = err;
}
__global__ void salient_pick_kernel(int nblk, const int* __restrict__ order, const double* __restrict__ serr, int* __restrict__ nstar,
                                    uint8_t* __restrict__ salflag, uint64_t* __restrict__ salient) {
  const int b = blockIdx.x * blockDim.x + threadIdx.x;
  if (b >= nblk) return;
  double best = INFINITY;
  int ns = 0;
  for (int i = 1; i <= kMaxSal; ++i)
    if (serr[b * kMaxSal + i - 1] < best) { best = serr[b * kMaxSal + i - 1]; ns = i; }
  nstar[b] = ns;
  uint64_t lo = 0, hi = 0;
  for (int c = 0; c < kBeta; ++c) salflag[b * kBeta + c] = 0;
  for (int t = 0; t < ns; ++t) {
    const int c = order[b * kMaxSal + t];
    salflag[b * kBeta + c] = 1;
    if (c < 64) lo |= 1ull << c; else hi |= 1ull << (c - 64);
  }
  salient[2 * b] = lo; salient[2 * b + 1] = hi;
}

// ---- Algorithm 2, NonSalientAwareQuant: break-point search ---------------------------------------------------------
__global__ void blockmax_kernel(const __half* __restrict__ W, size_t ldw, int n, int m, const uint8_t* __restrict__ keep,
                                const uint8_t* __restrict__ salflag, double* __restrict__ mx) {
  const int b = blockIdx.x;
  const int ngrp = m / kM;
  double v = 0.0;
  for (int t = threadIdx.x; t < n * kBeta; t += blockDim.x) {
    const int r = t / kBeta, c = t % kBeta, j = b * kBeta + c;
    if (salflag[b * kBeta + c] || !kept_at(keep, ngrp, r, j)) continue;
    v = fmax(v, fabs(w_at(W, ldw, r, j)));
  }
#pragma unroll
  for (int d = 16; d > 0; d >>= 1) v = fmax(v, __shfl_xor_sync(0xFFFFFFFFu, v, d));
  __shared__ double part[8];
  if ((threadIdx.x & 31) == 0) part[threadIdx.x >> 5] = v;
  __syncthreads();
  if (threadIdx.x == 0) {
    double s = 0.0;
    for (int w = 0; w < (int)(blockDim.x >> 5); ++w) s = fmax(s, part[w]);
    mx[b] = s;
  }
}
__device__ __forceinline__ void grid_point(int t, double mx, double& p1, double& p2) {
  const double frac = __dadd_rn(0.1, __ddiv_rn(__dmul_rn(0.9 - 0.1, (double)t), (double)(kGrid - 1)));
  p1 = __dmul_rn(frac, mx);
  p2 = __dmul_rn(2.0, p1);
}
// one warp per (block, grid point): per row the three regions' exact sums, then the three errors added in order
__global__ void break_err_kernel(const __half* __restrict__ W, size_t ldw, int n, int m, const uint8_t* __restrict__ keep,
                                 const uint8_t* __restrict__ salflag, const double* __restrict__ mx, double* __restrict__ berr) {
  const int warp = (int)((blockIdx.x * (size_t)blockDim.x + threadIdx.x) >> 5), lane = threadIdx.x & 31;
  const int nblk = m / kBeta, ngrp = m / kM;
  if (warp >= nblk * kGrid) return;
  const int b = warp / kGrid, t = warp % kGrid;
  double p1, p2;
  grid_point(t, mx[b], p1, p2);
  if (p2 > __dmul_rn(0.9, mx[b])) { if (lane == 0) berr[b * kGrid + t] = NAN; return; }
  bool sal[4];
#pragma unroll
  for (int k = 0; k < 4; ++k) sal[k] = salflag[b * kBeta + 4 * lane + k] != 0;
  double err = 0.0;
  for (int r = 0; r < n; ++r) {
    double q[3] = {0, 0, 0}, a[3] = {0, 0, 0};
    int kk[3] = {0, 0, 0};
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      const int j = b * kBeta + 4 * lane + k;
      if (sal[k] || !kept_at(keep, ngrp, r, j)) continue;
      const double w = w_at(W, ldw, r, j), aw = fabs(w);
      const int reg = aw > p2 ? 2 : (aw > p1 ? 1 : 0);
#pragma unroll
      for (int g = 0; g < 3; ++g)
        if (g == reg) { q[g] += w * w; a[g] += aw; ++kk[g]; }
    }
#pragma unroll
    for (int g = 0; g < 3; ++g) {
      q[g] = warp_sum(q[g]); a[g] = warp_sum(a[g]); kk[g] = warp_sum_int(kk[g]);
      err = __dadd_rn(err, binary_error(q[g], a[g], kk[g]));
    }
  }
  if (lane == 0) berr[b * kGrid + t] = err;
}
__global__ void break_pick_kernel(int nblk, const double* __restrict__ mx, const double* __restrict__ berr, double* __restrict__ bp) {
  const int b = blockIdx.x * blockDim.x + threadIdx.x;
  if (b >= nblk) return;
  double best = INFINITY, p1s = 0.0, p2s = 0.0;
  for (int t = 0; t < kGrid; ++t) {
    const double e = berr[b * kGrid + t];
    if (e != e) continue;              // skipped grid point
    if (e < best) { best = e; grid_point(t, mx[b], p1s, p2s); }
  }
  bp[2 * b] = p1s; bp[2 * b + 1] = p2s;
}

// ---- Trisection, Res_Approx and the logical arrays: one thread per (row, block), loops in column order ----------------
__global__ void emit_kernel(const __half* __restrict__ W, size_t ldw, int n, int m, const uint8_t* __restrict__ keep,
                            const uint8_t* __restrict__ salflag, const double* __restrict__ bp, uint8_t* __restrict__ sign,
                            uint16_t* __restrict__ region, uint32_t* __restrict__ sign2, uint16_t* __restrict__ scale) {
  const int nblk = m / kBeta, ngrp = m / kM;
  const size_t t = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (t >= (size_t)n * nblk) return;
  const int r = (int)(t / nblk), b = (int)(t % nblk);
  const double p1 = bp[2 * b], p2 = bp[2 * b + 1];
  const uint8_t* sf = salflag + b * kBeta;
  double a[3] = {0, 0, 0}, as = 0.0;
  int k[3] = {0, 0, 0}, ks = 0;
  for (int c = 0; c < kBeta; ++c) {
    const int j = b * kBeta + c;
    if (!kept_at(keep, ngrp, r, j)) continue;
    const double aw = fabs(w_at(W, ldw, r, j));
    if (sf[c]) { as = __dadd_rn(as, aw); ++ks; }
    else { const int reg = aw > p2 ? 2 : (aw > p1 ? 1 : 0); a[reg] = __dadd_rn(a[reg], aw); ++k[reg]; }
  }
  double alpha[5];
  for (int g = 0; g < 3; ++g) alpha[g] = k[g] ? __ddiv_rn(a[g], (double)k[g]) : 0.0;
  alpha[3] = ks ? __ddiv_rn(as, (double)ks) : 0.0;
  double ar = 0.0;
  for (int c = 0; c < kBeta; ++c) {
    const int j = b * kBeta + c;
    if (!sf[c] || !kept_at(keep, ngrp, r, j)) continue;
    const double w = w_at(W, ldw, r, j);
    ar = __dadd_rn(ar, fabs(__dsub_rn(w, __dmul_rn(alpha[3], w >= 0.0 ? 1.0 : -1.0))));
  }
  alpha[4] = ks ? __ddiv_rn(ar, (double)ks) : 0.0;
  for (int q = 0; q < 5; ++q) scale[t * 5 + q] = __half_as_ushort(__double2half(alpha[q]));
  int ts = 0;
  uint32_t s2 = 0;
  for (int gq = 0; gq < kBeta / kM; ++gq) {
    uint32_t sb = 0, rg = 0;
    int rank = 0;
    for (int c8 = 0; c8 < kM; ++c8) {
      const int c = gq * kM + c8, j = b * kBeta + c;
      if (kept_at(keep, ngrp, r, j)) {
        const double w = w_at(W, ldw, r, j), aw = fabs(w);
        if (w >= 0.0) sb |= 1u << rank;
        int reg;
        if (sf[c]) {
          reg = 3;
          if (__dsub_rn(w, __dmul_rn(alpha[3], w >= 0.0 ? 1.0 : -1.0)) >= 0.0) s2 |= 1u << ts;
        } else reg = aw > p2 ? 2 : (aw > p1 ? 1 : 0);
        rg |= (uint32_t)reg << (2 * rank);
        ++rank;
      }
      if (sf[c]) ++ts;
    }
    sign[(size_t)r * ngrp + b * (kBeta / kM) + gq] = (uint8_t)sb;
    region[(size_t)r * ngrp + b * (kBeta / kM) + gq] = (uint16_t)rg;
  }
  sign2[t] = s2;
}

static size_t a256(size_t v) { return (v + 255) & ~(size_t)255; }
static size_t carve(Ws& w, uint8_t* base, int n, int m) {
  const int nblk = m / kBeta;
  size_t o = 0;
  auto take = [&](size_t bytes) { uint8_t* p = base ? base + o : nullptr; o += a256(bytes); return p; };
  w.rowsum = (double*)take(sizeof(double) * n);
  w.colsum = (double*)take(sizeof(double) * m);
  w.colsq = (double*)take(sizeof(double) * m);
  w.partial = (double*)take(sizeof(double) * kPartials);
  w.scalars = (double*)take(sizeof(double) * 8);
  w.order = (int*)take(sizeof(int) * nblk * kMaxSal);
  w.serr = (double*)take(sizeof(double) * nblk * kMaxSal);
  w.nstar = (int*)take(sizeof(int) * nblk);
  w.salflag = (uint8_t*)take((size_t)nblk * kBeta);
  w.mx = (double*)take(sizeof(double) * nblk);
  w.berr = (double*)take(sizeof(double) * nblk * kGrid);
  w.bp = (double*)take(sizeof(double) * nblk * 2);
  return o;
}

}  // namespace quant
}  // namespace stb

extern "C" int stb_quantize_workspace(int n, int m, size_t* bytes) {
  if (!bytes) return STB_ERR_ARG;
  if (n < 1 || m < 128 || m % 128 != 0) return STB_ERR_SHAPE;
  stb::quant::Ws w;
  *bytes = stb::quant::carve(w, nullptr, n, m);
  return STB_OK;
}

extern "C" int stb_quantize(const void* W, size_t ldw, const double* xnorm, int n, int m, int N, double lambda,
                            const stb_logical* out, void* ws, size_t ws_bytes, void* stream) {
  using namespace stb::quant;
  if (!W || !xnorm || !out || !ws) return STB_ERR_ARG;
  if (n < 1 || m < 128 || m % 128 != 0) return STB_ERR_SHAPE;
  if (N < 1 || N > 8) return STB_ERR_NM;
  if (ldw < (size_t)m) return STB_ERR_ARG;
  if (out->n != n || out->m != m || out->N != N) return STB_ERR_ARG;
  if (!out->keep || !out->sign || !out->region || !out->sign2 || !out->salient || !out->scale) return STB_ERR_ARG;
  Ws w;
  if (ws_bytes < carve(w, static_cast<uint8_t*>(ws), n, m)) return STB_ERR_SIZE;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  const __half* Wh = static_cast<const __half*>(W);
  const int nblk = m / kBeta;
  uint8_t* keep = const_cast<uint8_t*>(out->keep);
  if (cudaMemsetAsync(w.colsum, 0, sizeof(double) * m, s) != cudaSuccess) return STB_ERR_CUDA;
  if (cudaMemsetAsync(w.colsq, 0, sizeof(double) * m, s) != cudaSuccess) return STB_ERR_CUDA;
  rowsum_kernel<<<(unsigned)(((size_t)n * 32 + 255) / 256), 256, 0, s>>>(Wh, ldw, n, m, w.rowsum);
  colsum_kernel<<<dim3((unsigned)((m + 255) / 256), (unsigned)((n + 63) / 64)), 256, 0, s>>>(Wh, ldw, n, m, w.colsum, w.colsq);
  const double count = (double)n * (double)m;
  for (int pass = 0; pass < 2; ++pass) {
    mu_partial_kernel<<<kPartials, 256, 0, s>>>(Wh, ldw, n, m, w.rowsum, w.colsum, w.scalars, pass, w.partial);
    mu_finish_kernel<<<1, 1, 0, s>>>(w.partial, kPartials, count, pass, w.scalars);
  }
  lambda_kernel<<<1, 1, 0, s>>>(xnorm, m, lambda, w.scalars);
  select_kernel<<<(unsigned)(((size_t)n * (m / kM) + 255) / 256), 256, 0, s>>>(Wh, ldw, n, m, N, w.rowsum, w.colsum, xnorm, w.scalars, keep);
  candidates_kernel<<<nblk, kBeta, 0, s>>>(w.colsq, xnorm, w.scalars, w.order);
  salient_err_kernel<<<(unsigned)((nblk * kMaxSal * 32 + 255) / 256), 256, 0, s>>>(Wh, ldw, n, m, keep, w.order, w.serr);
  salient_pick_kernel<<<(nblk + 127) / 128, 128, 0, s>>>(nblk, w.order, w.serr, w.nstar, w.salflag, const_cast<uint64_t*>(out->salient));
  blockmax_kernel<<<nblk, 256, 0, s>>>(Wh, ldw, n, m, keep, w.salflag, w.mx);
  break_err_kernel<<<(unsigned)((nblk * kGrid * 32 + 255) / 256), 256, 0, s>>>(Wh, ldw, n, m, keep, w.salflag, w.mx, w.berr);
  break_pick_kernel<<<(nblk + 127) / 128, 128, 0, s>>>(nblk, w.mx, w.berr, w.bp);
  emit_kernel<<<(unsigned)(((size_t)n * nblk + 127) / 128), 128, 0, s>>>(Wh, ldw, n, m, keep, w.salflag, w.bp, const_cast<uint8_t*>(out->sign),
                                                                     const_cast<uint16_t*>(out->region), const_cast<uint32_t*>(out->sign2),
                                                                     const_cast<uint16_t*>(out->scale));
  return cudaGetLastError() == cudaSuccess ? STB_OK : STB_ERR_CUDA;
}

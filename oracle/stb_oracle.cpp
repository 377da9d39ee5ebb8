// CPU oracle for the N:M structured-binary linear layer (STBLLM, arXiv 2408.01803).
//
// TEST INFRASTRUCTURE ONLY.  This file is the slow, plain reference that the
// CUDA library is checked against.  It shares no code with the CUDA path, is
// never linked into it, and must only be called from tests, from the smoke
// check and from the benchmark's CPU-baseline leg.
//
// Two parts:
//   1. The result: fp32 decode of the logical layer (Eq. 1, Eq. 4, the
//      per-region scales of Section 3.4 "Non-Salient Part") followed by a
//      float64 dequantise-then-matmul.  This is a plain definition.
//   2. The quantizer: Standardized Importance (Eq. 3), N-of-8 selection
//      (Section 3.3, Algorithm 1 line 10), salient-column search, residual
//      binarization, break-point search and trisection (Algorithm 2), each
//      step in the paper's order, all in float64.  No Hessian off-diagonals
//      and no OBC update (Algorithm 1 lines 16-17 are outside this oracle),
//      so blocks are independent and W is never modified.
//
// Pin status (see tests/test_oracle_*.py):
//   decode, matmul, N:M selection, Binary, Res_Approx, trisection error and
//   search, average-bit accounting: pinned (closed forms, brute force,
//   Table 1).  The SI ranking, the salient-column choice and the chosen
//   break-points have no printed worked example in the paper: beyond the
//   invariants and brute-force re-evaluations in the tests they are
//   "parity unpinned".
//
// Logical layer arrays (row-major, all host memory):
//   keep   u8  [n][m/8]      bit c (LSB first) = column 8g+c kept
//   sign   u8  [n][m/8]      bit k = sign of the k-th kept weight of the group
//                            (ascending column), 1 = +1, 0 = -1
//   region u16 [n][m/8]      2 bits per kept weight, rank order:
//                            0 dense, 1 intermediate, 2 sparse, 3 salient
//   sign2  u32 [n][m/128]    bit t = residual sign of the t-th salient column
//                            (ascending) of the block, 0 if dropped
//   salient u64 [m/128][2]   128-bit salient-column mask of the block
//   scale  u16 [n][m/128][5] fp16 bits: a_dense a_inter a_sparse a_sal1 a_sal2
#include <algorithm>
#include <cmath>
#include <cstdint>
#include <cstring>
#include <limits>
#include <thread>
#include <vector>

namespace {

constexpr int kM = 8;        // group size (N:8, Section 3.3)
constexpr int kBeta = 128;   // block size (Algorithm 1, beta; Table 2 "Block Size 128")
constexpr int kGroups = kBeta / kM;
constexpr int kMaxSalient = 32;  // candidate salient columns per block (reading: len(row_s) = 32)

// ---- fp16 <-> fp32/fp64 (IEEE binary16, round to nearest even) -------------
float half_bits_to_float(uint16_t h) {
  uint32_t s = (uint32_t)(h >> 15) & 1u, e = (h >> 10) & 0x1Fu, f = h & 0x3FFu;
  double v;
  if (e == 0) v = std::ldexp((double)f, -24);
  else if (e == 31) v = f ? std::numeric_limits<double>::quiet_NaN()
                          : std::numeric_limits<double>::infinity();
  else v = std::ldexp((double)(f | 0x400u), (int)e - 25);
  return (float)(s ? -v : v);
}

uint16_t double_to_half_bits(double x) {
  uint16_t sign = std::signbit(x) ? 0x8000u : 0u;
  double a = std::fabs(x);
  if (std::isnan(a)) return sign | 0x7E00u;
  if (a >= 65520.0) return sign | 0x7C00u;         // rounds to infinity
  if (a == 0.0) return sign;
  int ex;
  std::frexp(a, &ex);                               // a = f * 2^ex, f in [0.5,1)
  int e = ex - 1;                                   // a in [2^e, 2^(e+1))
  if (e < -14) e = -14;                             // subnormal range: fixed quantum 2^-24
  double q = std::ldexp(1.0, e - 10);               // quantum
  double r = std::nearbyint(a / q);                 // default rounding mode: to nearest even
  // r in [0, 2048]; rebuild
  if (e == -14 && r < 1024.0) return sign | (uint16_t)r;     // subnormal (or zero)
  if (r >= 2048.0) { r = 1024.0; e += 1; }
  if (e > 15) return sign | 0x7C00u;
  return sign | (uint16_t)(((e + 15) << 10) | ((int)r - 1024));
}

inline double sgn(double w) { return w >= 0.0 ? 1.0 : -1.0; }  // sign(0) = +1 (Eq. 2)

// Binary (Algorithm 2): alpha = l1 mean over the set, B = alpha * sign(W).
// Error of binarizing a set with sum of squares q, l1 sum a, count k:
//   sum (|w| - alpha)^2 = q - k alpha^2  with alpha = a / k.
inline double binary_error(double sumsq, double suml1, int k) {
  if (k == 0) return 0.0;
  double alpha = suml1 / k;
  return sumsq - k * alpha * alpha;
}

struct Dims { int n, m, nblk, ngrp; };
Dims dims(int n, int m) { return Dims{n, m, m / kBeta, m / kM}; }

inline bool kept(const uint8_t* keep, const Dims& d, int i, int j) {
  return (keep[(size_t)i * d.ngrp + j / kM] >> (j % kM)) & 1u;
}

}  // namespace

extern "C" {

// ---------------------------------------------------------------------------
// fp16 helpers exported for the tests (pinned against numpy.float16 there).
float stbo_half_to_float(uint16_t h) { return half_bits_to_float(h); }
uint16_t stbo_double_to_half(double x) { return double_to_half_bits(x); }

// ---------------------------------------------------------------------------
// Eq. 3.  S_ij = sigma(mu(|W_ij|)) * ||X_:,j||_2 with
//   mu(|W_ij|) = |W_ij| / sum_j |W_ij| + |W_ij| / sum_i |W_ij|
//   sigma(v)   = (v - mean) / std over the whole layer (population std).
// Reading: a zero row or column sum contributes a zero term; zero std gives
// z = 0.  xnorm[j] = ||X_:,j||_2 of the calibration activations.
void stbo_si_scores(const double* W, const double* xnorm, int n, int m, double* S) {
  std::vector<double> rowsum(n, 0.0), colsum(m, 0.0);
  for (int i = 0; i < n; ++i)
    for (int j = 0; j < m; ++j) {
      double a = std::fabs(W[(size_t)i * m + j]);
      rowsum[i] += a;
      colsum[j] += a;
    }
  double mean = 0.0;
  for (int i = 0; i < n; ++i)
    for (int j = 0; j < m; ++j) {
      double a = std::fabs(W[(size_t)i * m + j]);
      double mu = 0.0;
      if (rowsum[i] > 0.0) mu += a / rowsum[i];
      if (colsum[j] > 0.0) mu += a / colsum[j];
      S[(size_t)i * m + j] = mu;
      mean += mu;
    }
  mean /= (double)n * m;
  double var = 0.0;
  for (size_t t = 0; t < (size_t)n * m; ++t) var += (S[t] - mean) * (S[t] - mean);
  double sd = std::sqrt(var / ((double)n * m));
  for (int i = 0; i < n; ++i)
    for (int j = 0; j < m; ++j) {
      double z = sd > 0.0 ? (S[(size_t)i * m + j] - mean) / sd : 0.0;
      S[(size_t)i * m + j] = z * xnorm[j];
    }
}

// ---------------------------------------------------------------------------
// Section 3.3 / Algorithm 1 line 10: in every group of 8 consecutive input
// columns of a row keep the N entries with the highest score.  Ties go to the
// lower column index.
void stbo_nm_select(const double* S, int n, int m, int N, uint8_t* keep) {
  Dims d = dims(n, m);
  for (int i = 0; i < n; ++i)
    for (int g = 0; g < d.ngrp; ++g) {
      const double* s = S + (size_t)i * m + g * kM;
      int order[kM];
      for (int c = 0; c < kM; ++c) order[c] = c;
      std::stable_sort(order, order + kM, [&](int a, int b) { return s[a] > s[b]; });
      uint8_t bits = 0;
      for (int r = 0; r < N; ++r) bits |= (uint8_t)(1u << order[r]);
      keep[(size_t)i * d.ngrp + g] = bits;
    }
}

// ---------------------------------------------------------------------------
// Algorithm 2, Salient.  Column score of block b (diagonal-Hessian reading):
//   c_j = (h_jj + lambda) * sum_i W_ij^2,   h_jj = 2 ||X_:,j||^2,
// which equals sum_i W_ij^2 / [Hc_jj]^2 when H is diagonal.  The score uses
// the unpruned W; every binarization error inside the search uses the kept
// weights only.  Candidates: the kMaxSalient highest-scoring columns in
// descending score (ties: lower column).  For i = 1..kMaxSalient the error of
// binarizing {kept, first i candidates} and {kept, other columns} separately
// per row is evaluated; the first strict minimum wins.
// Out: order[kMaxSalient] (block-local column ids), errs[kMaxSalient], returns n*.
int stbo_salient_search(const double* W, const uint8_t* keep, const double* xnorm,
                        double lambda, int n, int m, int b, int* order, double* errs) {
  Dims d = dims(n, m);
  double score[kBeta];
  for (int c = 0; c < kBeta; ++c) {
    int j = b * kBeta + c;
    double q = 0.0;
    for (int i = 0; i < n; ++i) q += W[(size_t)i * m + j] * W[(size_t)i * m + j];
    score[c] = (2.0 * xnorm[j] * xnorm[j] + lambda) * q;
  }
  int idx[kBeta];
  for (int c = 0; c < kBeta; ++c) idx[c] = c;
  std::stable_sort(idx, idx + kBeta, [&](int a, int c) { return score[a] > score[c]; });
  for (int t = 0; t < kMaxSalient; ++t) order[t] = idx[t];

  double best = std::numeric_limits<double>::infinity();
  int nstar = 0;
  std::vector<char> is_sal(kBeta);
  for (int i = 1; i <= kMaxSalient; ++i) {
    std::fill(is_sal.begin(), is_sal.end(), 0);
    for (int t = 0; t < i; ++t) is_sal[order[t]] = 1;
    double err = 0.0;
    for (int r = 0; r < n; ++r) {
      double q[2] = {0, 0}, a[2] = {0, 0};
      int k[2] = {0, 0};
      for (int c = 0; c < kBeta; ++c) {
        int j = b * kBeta + c;
        if (!kept(keep, d, r, j)) continue;
        double w = W[(size_t)r * m + j];
        int s = is_sal[c];
        q[s] += w * w; a[s] += std::fabs(w); k[s] += 1;
      }
      err += binary_error(q[1], a[1], k[1]) + binary_error(q[0], a[0], k[0]);
    }
    errs[i - 1] = err;
    if (err < best) { best = err; nstar = i; }
  }
  return nstar;
}

// ---------------------------------------------------------------------------
// Algorithm 2, NonSalientAwareQuant: break-point search over one block's kept
// non-salient weights (all rows).  160 grid points on [0.1, 0.9]; p1 = i*max|W|,
// p2 = 2*p1; candidates with p2 > 0.9*max|W| are skipped; regions are
// sparse |w| > p2, intermediate p1 < |w| <= p2, dense |w| <= p1, each
// binarized per row with its own l1-mean scale; first strict minimum wins.
// salmask: 128 flags of the block.  errs[160] gets the error per grid point
// (NaN when skipped).  Returns the number of candidates evaluated.
int stbo_breakpoint_search(const double* W, const uint8_t* keep, const uint8_t* salflag,
                           int n, int m, int b, double* p1_out, double* p2_out, double* errs) {
  Dims d = dims(n, m);
  const int kGrid = 160;
  const double sigma = 2.0;
  double mx = 0.0;
  for (int r = 0; r < n; ++r)
    for (int c = 0; c < kBeta; ++c) {
      int j = b * kBeta + c;
      if (salflag[c] || !kept(keep, d, r, j)) continue;
      mx = std::max(mx, std::fabs(W[(size_t)r * m + j]));
    }
  double best = std::numeric_limits<double>::infinity();
  double p1s = 0.0, p2s = 0.0;
  int evaluated = 0;
  for (int t = 0; t < kGrid; ++t) {
    double frac = 0.1 + (0.9 - 0.1) * (double)t / (double)(kGrid - 1);
    double p1 = frac * mx, p2 = sigma * p1;
    if (p2 > 0.9 * mx) { if (errs) errs[t] = std::nan(""); continue; }
    ++evaluated;
    double err = 0.0;
    for (int r = 0; r < n; ++r) {
      double q[3] = {0, 0, 0}, a[3] = {0, 0, 0};
      int k[3] = {0, 0, 0};
      for (int c = 0; c < kBeta; ++c) {
        int j = b * kBeta + c;
        if (salflag[c] || !kept(keep, d, r, j)) continue;
        double w = W[(size_t)r * m + j], aw = std::fabs(w);
        int reg = aw > p2 ? 2 : (aw > p1 ? 1 : 0);
        q[reg] += w * w; a[reg] += aw; k[reg] += 1;
      }
      for (int reg = 0; reg < 3; ++reg) err += binary_error(q[reg], a[reg], k[reg]);
    }
    if (errs) errs[t] = err;
    if (err < best) { best = err; p1s = p1; p2s = p2; }
  }
  *p1_out = p1s; *p2_out = p2s;
  return evaluated;
}

// ---------------------------------------------------------------------------
// Algorithm 1 without the Hessian off-diagonals and without OBC: produce the
// logical layer from W (fp16 values widened to double), the calibration column
// norms, N and lambda (< 0 selects the reading lambda = 0.01 * mean_j h_jj).
// Also returns per-block break-points bp[nblk][2] and salient counts nsal[nblk]
// when the pointers are non-null.  Threads split the blocks.
void stbo_quantize(const double* W, const double* xnorm, int n, int m, int N, double lambda,
                   uint8_t* keep, uint8_t* sign, uint16_t* region, uint32_t* sign2,
                   uint64_t* salient, uint16_t* scale, double* bp, int* nsal, int nthreads) {
  Dims d = dims(n, m);
  {
    std::vector<double> S((size_t)n * m);
    stbo_si_scores(W, xnorm, n, m, S.data());
    stbo_nm_select(S.data(), n, m, N, keep);
  }
  if (lambda < 0.0) {
    double mh = 0.0;
    for (int j = 0; j < m; ++j) mh += 2.0 * xnorm[j] * xnorm[j];
    lambda = 0.01 * mh / m;
  }
  std::memset(sign, 0, (size_t)n * d.ngrp);
  std::memset(region, 0, sizeof(uint16_t) * (size_t)n * d.ngrp);
  std::memset(sign2, 0, sizeof(uint32_t) * (size_t)n * d.nblk);

  auto do_block = [&](int b) {
    int order[kMaxSalient];
    double serr[kMaxSalient];
    int nstar = stbo_salient_search(W, keep, xnorm, lambda, n, m, b, order, serr);
    uint8_t salflag[kBeta] = {0};
    for (int t = 0; t < nstar; ++t) salflag[order[t]] = 1;
    uint64_t lo = 0, hi = 0;
    for (int c = 0; c < 64; ++c) if (salflag[c]) lo |= (1ull << c);
    for (int c = 64; c < 128; ++c) if (salflag[c]) hi |= (1ull << (c - 64));
    salient[2 * b] = lo; salient[2 * b + 1] = hi;
    if (nsal) nsal[b] = nstar;

    double p1, p2;
    stbo_breakpoint_search(W, keep, salflag, n, m, b, &p1, &p2, nullptr);
    if (bp) { bp[2 * b] = p1; bp[2 * b + 1] = p2; }

    for (int r = 0; r < n; ++r) {
      // Trisection (Algorithm 2) for the kept non-salient weights of this row-block and
      // Res_Approx (Algorithm 2 / Eq. 4) for the kept salient ones.
      double a[3] = {0, 0, 0}; int k[3] = {0, 0, 0};
      double as = 0.0; int ks = 0;
      for (int c = 0; c < kBeta; ++c) {
        int j = b * kBeta + c;
        if (!kept(keep, d, r, j)) continue;
        double aw = std::fabs(W[(size_t)r * m + j]);
        if (salflag[c]) { as += aw; ++ks; }
        else { int reg = aw > p2 ? 2 : (aw > p1 ? 1 : 0); a[reg] += aw; ++k[reg]; }
      }
      double alpha[5];
      for (int reg = 0; reg < 3; ++reg) alpha[reg] = k[reg] ? a[reg] / k[reg] : 0.0;
      alpha[3] = ks ? as / ks : 0.0;
      double ar = 0.0;
      for (int c = 0; c < kBeta; ++c) {
        int j = b * kBeta + c;
        if (!salflag[c] || !kept(keep, d, r, j)) continue;
        double w = W[(size_t)r * m + j];
        ar += std::fabs(w - alpha[3] * sgn(w));
      }
      alpha[4] = ks ? ar / ks : 0.0;
      for (int q = 0; q < 5; ++q)
        scale[((size_t)r * d.nblk + b) * 5 + q] = double_to_half_bits(alpha[q]);

      int t = 0;  // index among the block's salient columns, ascending
      uint32_t s2 = 0;
      for (int g = 0; g < kGroups; ++g) {
        uint8_t sb = 0; uint16_t rg = 0; int rank = 0;
        for (int c8 = 0; c8 < kM; ++c8) {
          int c = g * kM + c8, j = b * kBeta + c;
          bool kp = kept(keep, d, r, j);
          if (kp) {
            double w = W[(size_t)r * m + j], aw = std::fabs(w);
            if (w >= 0.0) sb |= (uint8_t)(1u << rank);
            int reg;
            if (salflag[c]) {
              reg = 3;
              double res = w - alpha[3] * sgn(w);
              if (res >= 0.0) s2 |= (1u << t);
            } else reg = aw > p2 ? 2 : (aw > p1 ? 1 : 0);
            rg |= (uint16_t)(reg << (2 * rank));
            ++rank;
          }
          if (salflag[c]) ++t;
        }
        sign[(size_t)r * d.ngrp + b * kGroups + g] = sb;
        region[(size_t)r * d.ngrp + b * kGroups + g] = rg;
      }
      sign2[(size_t)r * d.nblk + b] = s2;
    }
  };

  int T = std::max(1, nthreads);
  std::vector<std::thread> pool;
  for (int t = 0; t < T; ++t)
    pool.emplace_back([&, t] { for (int b = t; b < d.nblk; b += T) do_block(b); });
  for (auto& th : pool) th.join();
}

// ---------------------------------------------------------------------------
// Decode (the plain definition).  fp32 result:
//   dropped weight               -> +0
//   kept, region 0..2            -> s * (float)alpha_region          (Eq. 1)
//   kept, salient (region 3)     -> fl32( s1*(float)a_sal1 + s2*(float)a_sal2 )   (Eq. 4)
// Both products are exact in fp32, so the salient value has one rounding.
void stbo_decode(int n, int m, const uint8_t* keep, const uint8_t* sign, const uint16_t* region,
                 const uint32_t* sign2, const uint64_t* salient, const uint16_t* scale,
                 float* What) {
  Dims d = dims(n, m);
  for (int i = 0; i < n; ++i)
    for (int b = 0; b < d.nblk; ++b) {
      const uint16_t* sc = scale + ((size_t)i * d.nblk + b) * 5;
      float alpha[5];
      for (int q = 0; q < 5; ++q) alpha[q] = half_bits_to_float(sc[q]);
      uint32_t s2 = sign2[(size_t)i * d.nblk + b];
      int t = 0;
      for (int g = 0; g < kGroups; ++g) {
        size_t gi = (size_t)i * d.ngrp + b * kGroups + g;
        uint8_t kp = keep[gi], sb = sign[gi];
        uint16_t rg = region[gi];
        int rank = 0;
        for (int c8 = 0; c8 < kM; ++c8) {
          int c = g * kM + c8;
          bool is_sal = (salient[2 * b + (c >> 6)] >> (c & 63)) & 1ull;
          float v = 0.0f;
          if ((kp >> c8) & 1u) {
            float s1 = ((sb >> rank) & 1u) ? 1.0f : -1.0f;
            int reg = (rg >> (2 * rank)) & 3;
            if (reg == 3) {
              float sr = ((s2 >> t) & 1u) ? 1.0f : -1.0f;
              v = s1 * alpha[3] + sr * alpha[4];
            } else v = s1 * alpha[reg];
            ++rank;
          }
          if (is_sal) ++t;
          What[(size_t)i * m + b * kBeta + c] = v;
        }
      }
    }
}

// ---------------------------------------------------------------------------
// y[t][i] = sum_j What[i][j] * x[t][j] in float64, from the fp32-decoded matrix
// and activations already widened to double.  x is [T][ldx], y is [T][n].
// Rows are split over nthreads.
void stbo_matmul(const float* What, int n, int m, const double* x, int T, int ldx,
                 double* y, int nthreads) {
  auto rows = [&](int i0, int i1) {
    for (int i = i0; i < i1; ++i)
      for (int t = 0; t < T; ++t) {
        double acc = 0.0;
        const float* w = What + (size_t)i * m;
        const double* xv = x + (size_t)t * ldx;
        for (int j = 0; j < m; ++j) acc += (double)w[j] * xv[j];
        y[(size_t)t * n + i] = acc;
      }
  };
  int P = std::max(1, nthreads);
  std::vector<std::thread> pool;
  int per = (n + P - 1) / P;
  for (int p = 0; p < P; ++p) {
    int i0 = p * per, i1 = std::min(n, i0 + per);
    if (i0 < i1) pool.emplace_back(rows, i0, i1);
  }
  for (auto& th : pool) th.join();
}

// Decode-and-multiply for a row range without materialising What (used as the
// timed CPU baseline and for sampled rows of large layers): rows[nr] lists the
// output rows wanted; y is [T][nr].
void stbo_layer_rows(int n, int m, const uint8_t* keep, const uint8_t* sign,
                     const uint16_t* region, const uint32_t* sign2, const uint64_t* salient,
                     const uint16_t* scale, const int* rows, int nr, const double* x, int T,
                     int ldx, double* y, int nthreads) {
  Dims d = dims(n, m);
  auto work = [&](int r0, int r1) {
    std::vector<float> wrow(m);
    for (int q = r0; q < r1; ++q) {
      int i = rows[q];
      stbo_decode(1, m, keep + (size_t)i * d.ngrp, sign + (size_t)i * d.ngrp,
                  region + (size_t)i * d.ngrp, sign2 + (size_t)i * d.nblk, salient,
                  scale + (size_t)i * d.nblk * 5, wrow.data());
      for (int t = 0; t < T; ++t) {
        double acc = 0.0;
        const double* xv = x + (size_t)t * ldx;
        for (int j = 0; j < m; ++j) acc += (double)wrow[j] * xv[j];
        y[(size_t)t * nr + q] = acc;
      }
    }
  };
  int P = std::max(1, nthreads);
  std::vector<std::thread> pool;
  int per = (nr + P - 1) / P;
  for (int p = 0; p < P; ++p) {
    int r0 = p * per, r1 = std::min(nr, r0 + per);
    if (r0 < r1) pool.emplace_back(work, r0, r1);
  }
  for (auto& th : pool) th.join();
}

// ---------------------------------------------------------------------------
// Section 3.4 "Average Bits": N_param = 2 r_sal + (1 - r_sal); N_stbllm = N_param * N / M.
double stbo_average_bits(int N, double r_salient) {
  double n_param = 2.0 * r_salient + 1.0 * (1.0 - r_salient);
  return n_param * (double)N / (double)kM;
}

// Bits actually carried by sign and residual-sign fields of a logical layer, per
// weight position: (kept weights + kept salient weights) / (n*m).
double stbo_counted_bits(int n, int m, const uint8_t* keep, const uint64_t* salient,
                         double* r_salient_out) {
  Dims d = dims(n, m);
  size_t nkept = 0, nsalkept = 0;
  for (int i = 0; i < n; ++i)
    for (int j = 0; j < m; ++j)
      if (kept(keep, d, i, j)) {
        ++nkept;
        int b = j / kBeta, c = j % kBeta;
        if ((salient[2 * b + (c >> 6)] >> (c & 63)) & 1ull) ++nsalkept;
      }
  if (r_salient_out) *r_salient_out = nkept ? (double)nsalkept / (double)nkept : 0.0;
  return (double)(nkept + nsalkept) / ((double)n * m);
}

// ---------------------------------------------------------------------------
// Not from the paper: the gated activation of the LLaMA MLP, whose three linears the paper binarizes
// (Section 4.1 evaluates LLaMA-1/2/3).  out[i] = fp16( silu(a[i]) * b[i] ), silu(v) = v / (1 + exp(-v)), float64.
// The CUDA path can form the input of the down projection this way (STB_IN_SILU_MUL).
void stbo_silu_mul(const double* a, const double* b, int n, uint16_t* out) {
  for (int i = 0; i < n; ++i) out[i] = double_to_half_bits(a[i] / (1.0 + std::exp(-a[i])) * b[i]);
}

// ---------------------------------------------------------------------------
// Section 3.3, Layer-wise N:M Assignment.  alpha_i = omega_i / sum_k omega_k with omega the L2 norm of layer i's
// weights; N_i / M = alpha_i + (1 - alpha_i) R_target.  Reading: M = 8 and N_i is that ratio times 8 rounded to the
// nearest integer (ties to even), kept inside 1..8.  ratio_out (may be null) receives the unrounded ratios.
void stbo_allocate_nm(const double* l2norm, int layers, double r_target, int* N_out, double* ratio_out) {
  double total = 0.0;
  for (int i = 0; i < layers; ++i) total += l2norm[i];
  for (int i = 0; i < layers; ++i) {
    const double alpha = total > 0.0 ? l2norm[i] / total : 0.0;
    const double ratio = alpha + (1.0 - alpha) * r_target;
    if (ratio_out) ratio_out[i] = ratio;
    int Ni = (int)std::nearbyint(ratio * (double)kM);
    N_out[i] = std::min(kM, std::max(1, Ni));
  }
}

int stbo_hardware_threads() { return (int)std::max(1u, std::thread::hardware_concurrency()); }

}  // extern "C"

// Algorithm 1 (Section 3): search of the clamping threshold gamma over the bin edges of a
// histogram of abs(x).  Three small kernels, float64 throughout, every reduction a fixed tree so
// that results do not depend on scheduling:
//   threshold_cdf_kernel         exact integer prefix sums of the counts, divided once by the total
//   threshold_candidates_kernel  one CTA per candidate i: clip the cdf at i, resample it onto the
//                                (n, p) grid and back, measure the distance to the cdf
//   threshold_argmin_kernel      the smallest measure; the lowest i among equal ones
#pragma once
#include <cstdint>
#include <cuda_runtime.h>

namespace qc {

constexpr int kThrMaxBins = 4096;
constexpr int kThrMaxLevels = 128;
constexpr int kThrThreads = 256;

enum : int { kMeasureL1 = 0, kMeasureKS = 1, kMeasureCvM = 2, kMeasureKL = 3 };

// cdf[j] = (h[0] + ... + h[j]) / total.  One block of 1024 threads, up to 4 bins per thread.
__global__ void __launch_bounds__(1024) threshold_cdf_kernel(const unsigned long long* __restrict__ hist, int nbins,
                                                             double* __restrict__ cdf) {
  __shared__ unsigned long long part[1024];
  const int t = threadIdx.x;
  const int per = (nbins + 1023) / 1024;
  unsigned long long loc[4];
  unsigned long long s = 0;
  for (int u = 0; u < per; ++u) {
    const int j = t * per + u;
    s += (j < nbins) ? hist[j] : 0ull;
    loc[u] = s;
  }
  part[t] = s;
  __syncthreads();
  for (int off = 1; off < 1024; off <<= 1) {          // inclusive scan over the per-thread totals
    const unsigned long long add = (t >= off) ? part[t - off] : 0ull;
    __syncthreads();
    part[t] += add;
    __syncthreads();
  }
  const unsigned long long before = (t > 0) ? part[t - 1] : 0ull;
  const double total = static_cast<double>(part[1023]);
  for (int u = 0; u < per; ++u) {
    const int j = t * per + u;
    if (j < nbins) cdf[j] = static_cast<double>(before + loc[u]) / total;
  }
}

struct ThresholdShared {
  double cdf[kThrMaxBins];
  double fp[kThrMaxLevels];        // fpspace(0, 1, n, p)
  double ri[kThrMaxLevels];        // r_interp: the clipped cdf sampled at the representable points
  double red[kThrThreads];
};

// q[j] for j < i: r_interp interpolated back onto linspace(0, 1, i)
__device__ __forceinline__ double resampled(const ThresholdShared& sh, int j, int i, int levels) {
  const double x = static_cast<double>(j) / static_cast<double>(i - 1);
  int lo = 0, hi = levels - 1;                        // invariant: fp[lo] <= x, and x < fp[hi] or hi is last
  while (hi - lo > 1) {
    const int mid = (lo + hi) >> 1;
    if (sh.fp[mid] <= x) lo = mid; else hi = mid;
  }
  const double w = (x - sh.fp[lo]) / (sh.fp[lo + 1] - sh.fp[lo]);
  return sh.ri[lo] + (sh.ri[lo + 1] - sh.ri[lo]) * w;
}

__global__ void __launch_bounds__(kThrThreads)
threshold_candidates_kernel(const double* __restrict__ cdf_g, const double* __restrict__ fp_g, int nbins, int levels,
                            int first, int measure, double kl_floor, double* __restrict__ deltas) {
  __shared__ ThresholdShared sh;
  const int t = threadIdx.x;
  const int i = first + blockIdx.x;                   // candidate: bins [0, i) are kept, gamma = edge i
  for (int j = t; j < nbins; j += kThrThreads) sh.cdf[j] = cdf_g[j];
  for (int k = t; k < levels; k += kThrThreads) sh.fp[k] = fp_g[k];
  __syncthreads();
  // r = cdf with r[i-1:] = 1;  r_interp = r[:i] on linspace(0, 1, i), read at the representable points
  for (int k = t; k < levels; k += kThrThreads) {
    const double pos = sh.fp[k] * static_cast<double>(i - 1);
    int j0 = static_cast<int>(pos);
    if (j0 > i - 2) j0 = i - 2;
    const double a = sh.cdf[j0];                      // j0 <= i-2: never clipped
    const double b = (j0 + 1 >= i - 1) ? 1.0 : sh.cdf[j0 + 1];
    sh.ri[k] = a + (b - a) * (pos - static_cast<double>(j0));
  }
  __syncthreads();
  double acc = 0.0;
  for (int j = t; j < nbins; j += kThrThreads) {
    const double c = sh.cdf[j];
    const double q = (j < i) ? resampled(sh, j, i, levels) : 1.0;
    if (measure == kMeasureKL) {
      const double c0 = (j > 0) ? sh.cdf[j - 1] : 0.0;
      const double q0 = (j == 0) ? 0.0 : ((j - 1 < i) ? resampled(sh, j - 1, i, levels) : 1.0);
      const double P = c - c0;
      const double Q = fmax(q - q0, kl_floor);
      if (P > 0.0) acc += P * log(P / Q);
    } else {
      const double d = fabs(c - q);
      if (measure == kMeasureKS) acc = fmax(acc, d);
      else if (measure == kMeasureCvM) acc += d * d;
      else acc += d;
    }
  }
  sh.red[t] = acc;
  __syncthreads();
  for (int off = kThrThreads / 2; off > 0; off >>= 1) {
    if (t < off) sh.red[t] = (measure == kMeasureKS) ? fmax(sh.red[t], sh.red[t + off]) : sh.red[t] + sh.red[t + off];
    __syncthreads();
  }
  if (t == 0) {
    double v = sh.red[0];
    if (measure == kMeasureL1 || measure == kMeasureCvM) v /= static_cast<double>(nbins);
    deltas[i] = v;
  }
}

struct ThresholdBest {
  double delta;
  int index;
  int pad;
};

// delta starts at infinity and gamma at the last edge; a candidate replaces them only when strictly
// better, so among equal measures the lowest i wins and a NaN never wins.
__global__ void __launch_bounds__(kThrThreads)
threshold_argmin_kernel(const double* __restrict__ deltas, int first, int nbins, ThresholdBest* __restrict__ out) {
  __shared__ double bv[kThrThreads];
  __shared__ int bi[kThrThreads];
  const int t = threadIdx.x;
  double v = INFINITY;
  int at = nbins;
  for (int i = first + t; i <= nbins; i += kThrThreads) {
    const double d = deltas[i];
    if (d < v) { v = d; at = i; }                     // ascending i per thread: first minimum kept
  }
  bv[t] = v; bi[t] = at;
  __syncthreads();
  for (int off = kThrThreads / 2; off > 0; off >>= 1) {
    if (t < off) {
      const double ov = bv[t + off];
      const int oi = bi[t + off];
      if (ov < bv[t] || (ov == bv[t] && oi < bi[t])) { bv[t] = ov; bi[t] = oi; }
    }
    __syncthreads();
  }
  if (t == 0) { out->delta = bv[0]; out->index = bi[0]; out->pad = 0; }
}

}  // namespace qc

// Calibration statistics over one batch of float activations: max |x|, finite / non-finite
// counts, fp64 sum and sum of squares (pass 1) and the histogram of |x| (pass 2) -- the
// hist(abs(x)) that opens Algorithm 1 and the maximum Section 3 uses as default threshold.
#pragma once
#include <cuda_runtime.h>
#include <cstdint>

namespace qc {

constexpr int kCalibMaxBins = 4096;
constexpr int kCalibMaxBlocks = 2048;

// Device scratch shared by the two passes.  Cleared before each collection.
struct CalibScratch {
  unsigned int maxabs_bits;          // float bits of max |x| (non-negative floats order as uints)
  unsigned int pad;
  unsigned long long finite;
  unsigned long long nonfinite;
  double sum, sumsq;
  unsigned long long hist[kCalibMaxBins];
  double part_sum[kCalibMaxBlocks];
  double part_sumsq[kCalibMaxBlocks];
};

__device__ __forceinline__ void stats_accum(float v, float& mx, unsigned int& nf, double& s, double& ss) {
  float a = fabsf(v);
  if (a <= 3.402823466e+38f) {       // finite (false for NaN and Inf)
    mx = fmaxf(mx, a);
    double d = static_cast<double>(v);
    s += d;
    ss = fma(d, d, ss);
  } else {
    nf += 1u;
  }
}

__global__ void __launch_bounds__(256)
calib_pass1_kernel(const float* __restrict__ x, size_t count, CalibScratch* sc, int vec_ok) {
  float mx = 0.0f;
  unsigned int nf = 0;
  double s = 0.0, ss = 0.0;
  const size_t tid = blockIdx.x * static_cast<size_t>(blockDim.x) + threadIdx.x;
  const size_t nthreads = static_cast<size_t>(gridDim.x) * blockDim.x;
  size_t nvec = vec_ok ? count / 4 : 0;
  const float4* x4 = reinterpret_cast<const float4*>(x);
  for (size_t i = tid; i < nvec; i += nthreads) {
    float4 v = __ldg(x4 + i);
    stats_accum(v.x, mx, nf, s, ss);
    stats_accum(v.y, mx, nf, s, ss);
    stats_accum(v.z, mx, nf, s, ss);
    stats_accum(v.w, mx, nf, s, ss);
  }
  for (size_t i = nvec * 4 + tid; i < count; i += nthreads) stats_accum(x[i], mx, nf, s, ss);

  // block reduction: warp shuffles, then one partial per warp through shared memory
  __shared__ float s_mx[8];
  __shared__ unsigned int s_nf[8];
  __shared__ double s_s[8], s_ss[8];
  for (int o = 16; o > 0; o >>= 1) {
    mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
    nf += __shfl_xor_sync(0xffffffffu, nf, o);
    s += __shfl_xor_sync(0xffffffffu, s, o);
    ss += __shfl_xor_sync(0xffffffffu, ss, o);
  }
  int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (lane == 0) { s_mx[warp] = mx; s_nf[warp] = nf; s_s[warp] = s; s_ss[warp] = ss; }
  __syncthreads();
  if (threadIdx.x == 0) {
    unsigned long long nft = 0;
    for (int w = 1; w < 8; ++w) { mx = fmaxf(mx, s_mx[w]); s += s_s[w]; ss += s_ss[w]; }
    for (int w = 0; w < 8; ++w) nft += s_nf[w];
    atomicMax(&sc->maxabs_bits, __float_as_uint(mx));
    if (nft) atomicAdd(&sc->nonfinite, nft);
    sc->part_sum[blockIdx.x] = s;
    sc->part_sumsq[blockIdx.x] = ss;
  }
}

// Sums the per-block partials with a fixed reduction tree (deterministic for a given grid) and
// derives the finite count.  One block of 256 threads.
__global__ void __launch_bounds__(256)
calib_finalize_kernel(CalibScratch* sc, int nblocks, unsigned long long count) {
  double s = 0.0, ss = 0.0;
  for (int b = threadIdx.x; b < nblocks; b += 256) { s += sc->part_sum[b]; ss += sc->part_sumsq[b]; }
  __shared__ double s_s[8], s_ss[8];
  for (int o = 16; o > 0; o >>= 1) {
    s += __shfl_xor_sync(0xffffffffu, s, o);
    ss += __shfl_xor_sync(0xffffffffu, ss, o);
  }
  if ((threadIdx.x & 31) == 0) { s_s[threadIdx.x >> 5] = s; s_ss[threadIdx.x >> 5] = ss; }
  __syncthreads();
  if (threadIdx.x == 0) {
    for (int w = 1; w < 8; ++w) { s += s_s[w]; ss += s_ss[w]; }
    sc->sum = s;
    sc->sumsq = ss;
    sc->finite = count - sc->nonfinite;
  }
}

// Pass 2: bin = min(nbins-1, (int)(|x| * inv_w)), inv_w = (float)nbins / hi in fp32, one
// multiply.  hi <= 0 on the host side means "use the maximum found by pass 1".  Zeros (half
// of a post-ReLU tensor) are counted in a register instead of hammering one shared counter.
__global__ void __launch_bounds__(256)
calib_hist_kernel(const float* __restrict__ x, size_t count, CalibScratch* sc, int nbins,
                  float range_hi, int vec_ok) {
  extern __shared__ unsigned int s_hist[];
  for (int b = threadIdx.x; b < nbins; b += blockDim.x) s_hist[b] = 0u;
  __syncthreads();
  const float hi = range_hi > 0.0f ? range_hi : __uint_as_float(sc->maxabs_bits);
  const float inv_w = hi > 0.0f ? __fdiv_rn(static_cast<float>(nbins), hi) : 0.0f;
  const float fb = static_cast<float>(nbins);
  unsigned int zeros = 0;
  auto put = [&](float v) {
    float a = fabsf(v);
    if (!(a <= 3.402823466e+38f)) return;
    float t = __fmul_rn(a, inv_w);
    int b = t >= fb ? nbins - 1 : static_cast<int>(t);
    if (b == 0) zeros += 1u; else atomicAdd(&s_hist[b], 1u);
  };
  const size_t tid = blockIdx.x * static_cast<size_t>(blockDim.x) + threadIdx.x;
  const size_t nthreads = static_cast<size_t>(gridDim.x) * blockDim.x;
  size_t nvec = vec_ok ? count / 4 : 0;
  const float4* x4 = reinterpret_cast<const float4*>(x);
  for (size_t i = tid; i < nvec; i += nthreads) {
    float4 v = __ldg(x4 + i);
    put(v.x); put(v.y); put(v.z); put(v.w);
  }
  for (size_t i = nvec * 4 + tid; i < count; i += nthreads) put(x[i]);
  for (int o = 16; o > 0; o >>= 1) zeros += __shfl_xor_sync(0xffffffffu, zeros, o);
  if ((threadIdx.x & 31) == 0 && zeros) atomicAdd(&s_hist[0], zeros);
  __syncthreads();
  for (int b = threadIdx.x; b < nbins; b += blockDim.x) {
    unsigned int c = s_hist[b];
    if (c) atomicAdd(&sc->hist[b], static_cast<unsigned long long>(c));
  }
}

}  // namespace qc

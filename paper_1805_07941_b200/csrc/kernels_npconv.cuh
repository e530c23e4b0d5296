// Convolution on dynamic floating-point operands (Section 2.1 type, Eq. 6): the pieces around the
// tensor-core GEMM.  The betas of an (n, p) type are integers up to beta_max (Eq. 5: 1984 for (8, 4),
// 245760 for (8, 3)), so the sum of Eq. 6 is an exact integer sum -- but its terms do not fit the int8
// operands of the MMA.  Each beta is therefore written in base 128 with balanced digits,
//   beta = d_0 + 128 d_1 + 128^2 d_2,   d_0, d_1 in [-64, 63], the last digit whatever is left (<= 127),
// the digit planes of the input are laid side by side along the channel axis, and the weights are
// arranged so that output column group g collects every digit product of weight 128^g:
//   acc_g = sum_i x_plane_i * w_plane_(g-i).
// One int8 GEMM (int32 accumulators, exact) produces all groups; the kernel below adds them up in 64
// bits, sum_g acc_g << 7g, adds the bias, applies ReLU and converts to the output type.
#pragma once
#include <cuda_runtime.h>
#include <cstdint>
#include "epilogue.cuh"
#include "kernels_simple.cuh"

namespace qc {

struct NpFormat {
  int n, p;
  long long beta_max;
};

// Pattern (without sign) -> beta (Eq. 2 with the exponent field of Eq. 4).
__device__ __forceinline__ int np_decode_mag(int c, int n, int p) {
  if (p == n - 1) return c;
  const int E = c >> p, m = c & ((1 << p) - 1);
  return E == 0 ? m : ((1 << p) + m) << (E - 1);
}

// Value on the type's grid -> pattern (without sign).
__device__ __forceinline__ int np_code_of(unsigned long long v, int p) {
  if (v < (2ull << p)) return static_cast<int>(v);          // subnormals and the first binade: the pattern is the value
  const int L = 63 - __clzll(static_cast<long long>(v));
  const int E = L - p + 1;
  return (E << p) | static_cast<int>((v >> (E - 1)) - (1ull << p));
}

// acc / 2^s -> pattern of the nearest (n, p) value; ties to the even pattern; beyond beta_max saturates;
// a zero magnitude is pattern 0 (Section 3 conversion, applied to an exact rational).
__device__ __forceinline__ uint8_t np_encode_i64(long long acc, int s, NpFormat f) {
  const unsigned long long mag = acc < 0 ? 0ull - static_cast<unsigned long long>(acc) : static_cast<unsigned long long>(acc);
  if (mag == 0) return 0;
  int code;
  if (mag >= (static_cast<unsigned long long>(f.beta_max) << s)) {
    code = (1 << (f.n - 1)) - 1;
  } else {
    const int L = 63 - __clzll(static_cast<long long>(mag));
    const int k = L - s;                                    // acc / 2^s lies in [2^k, 2^(k+1)); k < 0: below 1
    const int sp = k > f.p ? k - f.p : 0;                   // grid spacing 2^sp in that binade
    const int sh = s + sp;
    const unsigned long long q = sh < 64 ? mag >> sh : 0ull;
    const unsigned long long lo = q << sp, hi = (q + 1) << sp;   // neighbours on the grid (hi may open the next binade)
    const unsigned long long rem = mag - (q << sh);
    const unsigned long long half = sh > 0 ? 1ull << (sh - 1) : 0ull;
    const int c_lo = np_code_of(lo, f.p), c_hi = np_code_of(hi, f.p);
    if (sh == 0 || rem < half) code = c_lo;
    else if (rem > half) code = c_hi;
    else code = (c_hi & 1) ? c_lo : c_hi;
  }
  return static_cast<uint8_t>(code | ((acc < 0 && code != 0) ? 1 << (f.n - 1) : 0));
}

// codes [pixels][C] -> digit planes [pixels][planes * C] (plane-major inside a pixel), 16 codes per thread.
__global__ void __launch_bounds__(256)
np_split_kernel(const uint8_t* __restrict__ codes, int8_t* __restrict__ planes, size_t pixels, int C, int n, int p,
                int nplanes) {
  chain_sync();
  const int cv = C / 16;
  const size_t total = pixels * cv;
  for (size_t idx = blockIdx.x * static_cast<size_t>(blockDim.x) + threadIdx.x; idx < total;
       idx += static_cast<size_t>(gridDim.x) * blockDim.x) {
    const size_t pix = idx / cv;
    const int c0 = static_cast<int>(idx % cv) * 16;
    if (!QC_IN(pix * C + c0 + 15, pixels * C)) continue;
    const uint4 raw = __ldg(reinterpret_cast<const uint4*>(codes + pix * C + c0));
    const uint32_t w[4] = {raw.x, raw.y, raw.z, raw.w};
    uint32_t out[3][4] = {{0, 0, 0, 0}, {0, 0, 0, 0}, {0, 0, 0, 0}};
#pragma unroll
    for (int j = 0; j < 16; ++j) {
      const int c = (w[j >> 2] >> (8 * (j & 3))) & 0xFF;
      int beta = np_decode_mag(c & ((1 << (n - 1)) - 1), n, p);
      if ((c >> (n - 1)) & 1) beta = -beta;
#pragma unroll
      for (int i = 0; i < 3; ++i) {
        if (i < nplanes) {
          // balanced digit in [-64, 63]; the last plane keeps what is left
          const int d = i + 1 < nplanes ? ((beta + 64) & 127) - 64 : beta;
          beta = (beta - d) >> 7;
          out[i][j >> 2] |= static_cast<uint32_t>(d & 0xFF) << (8 * (j & 3));
        }
      }
    }
    int8_t* dst = planes + pix * static_cast<size_t>(nplanes) * C + c0;
#pragma unroll
    for (int i = 0; i < 3; ++i)
      if (i < nplanes)
        *reinterpret_cast<uint4*>(dst + static_cast<size_t>(i) * C) = make_uint4(out[i][0], out[i][1], out[i][2], out[i][3]);
  }
}

// acc32 [pixels][groups * K] -> codes [pixels][K]: 64-bit recombination, bias, ReLU, conversion.
__global__ void __launch_bounds__(256)
np_combine_kernel(const int32_t* __restrict__ acc32, const int32_t* __restrict__ bias, const int32_t* __restrict__ shift,
                  uint8_t* __restrict__ y, size_t pixels, int K, int groups, int relu, NpFormat fout) {
  const size_t total = pixels * K;
  for (size_t idx = blockIdx.x * static_cast<size_t>(blockDim.x) + threadIdx.x; idx < total;
       idx += static_cast<size_t>(gridDim.x) * blockDim.x) {
    const size_t pix = idx / K;
    const int k = static_cast<int>(idx % K);
    const int32_t* a = acc32 + pix * static_cast<size_t>(groups) * K + k;
    long long v = bias ? static_cast<long long>(__ldg(bias + k)) : 0ll;
    for (int g = 0; g < groups; ++g)
      if (QC_IN(pix * static_cast<size_t>(groups) * K + k + static_cast<size_t>(g) * K, pixels * static_cast<size_t>(groups) * K))
        v += static_cast<long long>(__ldg(a + static_cast<size_t>(g) * K)) << (7 * g);
    if (relu && v < 0) v = 0;
    y[idx] = np_encode_i64(v, __ldg(shift + k), fout);
  }
}

}  // namespace qc

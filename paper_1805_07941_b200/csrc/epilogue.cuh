// Register epilogue shared by every convolution kernel: bias, residual, ReLU,
// shift-requantization with rounding, saturation (Section 3 conversion applied to the
// wide accumulator of Eq. 6; residual per Eq. 10).
#pragma once
#include <cstdint>

namespace qc {

// Checked build (-DQCONV_CHECKED): in the CUDA-core kernels every global access whose address is
// computed is preceded by a test of its element index against the tensor's extent.  A failing test
// records the source line in a device word, the access is skipped, and the kernel goes on: nothing
// traps, the context stays usable, and qconv_checked_faults() reports what happened.  In the normal
// build QC_IN is the constant true and leaves no instruction behind.
#ifdef QCONV_CHECKED
__device__ int g_checked_fault[2] = {0, 0};             // {number of failed tests, source line of the first}
__device__ __forceinline__ bool checked_in(unsigned long long idx, unsigned long long extent, int line) {
  if (idx < extent) return true;
  if (atomicAdd(&g_checked_fault[0], 1) == 0) g_checked_fault[1] = line;
  return false;
}
#define QC_IN(idx, extent) ::qc::checked_in(static_cast<unsigned long long>(idx), static_cast<unsigned long long>(extent), __LINE__)
#else
#define QC_IN(idx, extent) true
#endif

struct EpilogueParams {
  const int32_t* bias;        // [K] or nullptr
  const int32_t* shift;       // [K]
  const int32_t* res_lshift;  // [K] or nullptr
  const int32_t* acc_exp;     // [K]
  int relu;
  int rounding;
  int lo, hi;                 // saturation bounds of the output beta
  int out_mode;               // 0 int8, 1 int32, 2 float
  // when every channel has the same shifts: s, 2^(s-1) - 1, and (s > 0) | 2^t << 1
  int uni_shift, uni_z, uni_w;
  float uni_c1;               // 2^-s, for the float-rounding epilogue (0 when s > 22)
  float uni_c2;               // 1.5 * 2^23 * (1 - 2^-s): its addend
};

// acc / 2^s rounded to an integer, entirely in 32-bit without overflow.
// v = q * 2^s + rem with q = floor quotient, 0 <= rem < 2^s.
__device__ __forceinline__ int32_t round_shift(int32_t v, int s, int mode) {
  if (s == 0) return v;
  int32_t q = v >> s;
  uint32_t rem = static_cast<uint32_t>(v) & ((1u << s) - 1u);
  uint32_t half = 1u << (s - 1);
  int inc;
  if (mode == 0)      inc = (rem > half) | ((rem == half) & (q & 1));
  else if (mode == 1) inc = (rem > half) | ((rem == half) & (v > 0));
  else if (mode == 2) inc = (rem >= half);
  else                inc = 0;
  return q + inc;
}

// Wide value after bias, residual and ReLU.
__device__ __forceinline__ int32_t wide_value(int32_t acc, int32_t bias, int32_t res, int t, int relu) {
  int32_t v = acc + bias + static_cast<int32_t>(static_cast<uint32_t>(res) << t);
  if (relu) v = max(v, 0);
  return v;
}

__device__ __forceinline__ int32_t requantize(int32_t v, int s, int mode, int lo, int hi) {
  int32_t q = round_shift(v, s, mode);
  return min(max(q, lo), hi);
}

// beta -> float: integer to binary32 (nearest even), then exact scaling by 2^e.
__device__ __forceinline__ float dequantize(int32_t v, int e) {
  return ldexpf(__int2float_rn(v), e);
}

}  // namespace qc

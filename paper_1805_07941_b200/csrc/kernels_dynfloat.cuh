// float <-> n-bit dynamic floating-point codes with p significand bits (Section 2.1, Eq. 2 and 4;
// conversion steps of Section 3), scale alpha = 2^e.  A code is the sign-and-magnitude pattern of
// Eq. 2 in one byte: bit n-1 the sign, then the exponent field E (n-p-1 bits), then the significand.
//   E = 0: value = significand            (spacing 1 up to 2^p)
//   E > 0: value = (2^p + significand) * 2^(E-1)
// so a magnitude a in binade [2^k, 2^(k+1)) is represented with spacing 2^max(0, k-p).  Encoding is
// therefore: scale by 2^-e, clamp to beta_max, divide by the spacing (exact), round to nearest even
// with rintf, renormalise when rounding carries into the next binade.  HBM-bound streaming kernels:
// 4 bytes in and 1 out per value (encode), 1 in and 4 out (decode).
#pragma once
#include <cstdint>
#include <cuda_runtime.h>

namespace qc {

struct DynFloatFormat {
  int n, p;
  int e;              // scale exponent
  float beta_max;     // Eq. 5, as a float (exact: at most p+1 significant bits, exponent <= 126)
  int e_max;          // largest exponent field: 2^(n-p-1) - 1 (0 when p = n-1)
};

__device__ __forceinline__ uint32_t dynfloat_encode_one(float x, const DynFloatFormat& f) {
  if (x != x) return 0u;
  float a = fabsf(x);
  // |x| / 2^e in two exact steps (one factor could leave the float range for large |e|); a result that
  // underflows is far below one half and rounds to zero anyway, one that overflows saturates
  const int h = -f.e / 2;
  a = ldexpf(ldexpf(a, h), -f.e - h);
  a = fminf(a, f.beta_max);
  // binade of a: floor(log2 a) for a >= 1; anything below 2^(p+1) has spacing 1
  const int k = static_cast<int>((__float_as_uint(a) >> 23) & 0xFFu) - 127;
  const uint32_t sign = (__float_as_uint(x) >> 31) << (f.n - 1);
  if (f.p == 0 && k >= 0) {
    // no significand bits: the values are the powers of two, code = exponent field.  The parity of
    // the rounded quotient says nothing about the parity of the code here, so the tie at 1.5 * 2^k
    // is resolved on the codes themselves (k+1 and k+2).
    const float fr = ldexpf(a, -k);                               // in [1, 2)
    uint32_t E = static_cast<uint32_t>(k + 1);
    if (fr > 1.5f || (fr == 1.5f && (E & 1u))) ++E;
    return sign | E;
  }
  int s = max(0, k - f.p);
  int q = static_cast<int>(rintf(ldexpf(a, -s)));               // in [0, 2^(p+1)]
  if (q == (2 << f.p)) { q = 1 << f.p; ++s; }                   // carried into the next binade
  if (q == 0) return 0u;
  const uint32_t E = (q >= (1 << f.p)) ? static_cast<uint32_t>(s + 1) : 0u;
  const uint32_t mag = (E << f.p) | (static_cast<uint32_t>(q) & ((1u << f.p) - 1u));
  return sign | mag;
}

__device__ __forceinline__ float dynfloat_decode_one(uint32_t code, const DynFloatFormat& f) {
  const uint32_t E = (code >> f.p) & static_cast<uint32_t>(f.e_max);
  const uint32_t sig = code & ((1u << f.p) - 1u);
  const float m = static_cast<float>(E ? (1u << f.p) + sig : sig);
  const float v = ldexpf(m, (E ? static_cast<int>(E) - 1 : 0) + f.e);
  return ((code >> (f.n - 1)) & 1u) ? -v : v;
}

__global__ void __launch_bounds__(256)
dynfloat_encode_kernel(const float* __restrict__ x, uint8_t* __restrict__ y, size_t count, DynFloatFormat f, int vec_ok) {
  const size_t tid = blockIdx.x * static_cast<size_t>(blockDim.x) + threadIdx.x;
  const size_t nthreads = static_cast<size_t>(gridDim.x) * blockDim.x;
  const size_t nvec = vec_ok ? count / 16 : 0;
  for (size_t i = tid; i < nvec; i += nthreads) {
    uint32_t w[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const float4 v = __ldg(reinterpret_cast<const float4*>(x) + i * 4 + j);
      w[j] = dynfloat_encode_one(v.x, f) | (dynfloat_encode_one(v.y, f) << 8) | (dynfloat_encode_one(v.z, f) << 16) |
             (dynfloat_encode_one(v.w, f) << 24);
    }
    reinterpret_cast<uint4*>(y)[i] = make_uint4(w[0], w[1], w[2], w[3]);
  }
  for (size_t i = nvec * 16 + tid; i < count; i += nthreads) y[i] = static_cast<uint8_t>(dynfloat_encode_one(x[i], f));
}

__global__ void __launch_bounds__(256)
dynfloat_decode_kernel(const uint8_t* __restrict__ c, float* __restrict__ y, size_t count, DynFloatFormat f, int vec_ok) {
  const size_t tid = blockIdx.x * static_cast<size_t>(blockDim.x) + threadIdx.x;
  const size_t nthreads = static_cast<size_t>(gridDim.x) * blockDim.x;
  const size_t nvec = vec_ok ? count / 16 : 0;
  for (size_t i = tid; i < nvec; i += nthreads) {
    const uint4 v = __ldg(reinterpret_cast<const uint4*>(c) + i);
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int j = 0; j < 4; ++j)
      reinterpret_cast<float4*>(y)[i * 4 + j] =
          make_float4(dynfloat_decode_one(w[j] & 0xFFu, f), dynfloat_decode_one((w[j] >> 8) & 0xFFu, f),
                      dynfloat_decode_one((w[j] >> 16) & 0xFFu, f), dynfloat_decode_one(w[j] >> 24, f));
  }
  for (size_t i = nvec * 16 + tid; i < count; i += nthreads) y[i] = dynfloat_decode_one(c[i], f);
}

}  // namespace qc

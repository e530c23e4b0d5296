// CUDA-core kernels of the path: float -> beta conversion, int8 max-pool, stem patch
// packing, the direct (any-shape) convolution and the depthwise convolution.
#pragma once
#include <cuda_runtime.h>
#include <type_traits>
#include <cstdint>
#include "epilogue.cuh"

namespace qc {

// Programmatic dependent launch for the streaming kernels of a layer chain: wait until the kernels
// before this one in the stream are complete (a no-op under an ordinary launch), then let the
// next kernel start its set-up while this one runs.
__device__ __forceinline__ void chain_sync() {
  asm volatile("griddepcontrol.wait;" ::: "memory");
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
}


// ---------------------------------------------------------------------------------------
// float -> beta (Section 3): clamp to +-gamma', divide by alpha = 2^e, round to nearest even,
// clamp to +-beta_max.  NaN -> 0.
// ---------------------------------------------------------------------------------------
__device__ __forceinline__ int quantize_one(float v, float gam, float inv_alpha, int e, bool use_mul,
                                            float bmax) {
  if (v != v) return 0;
  v = fminf(fmaxf(v, -gam), gam);
  float scaled = use_mul ? v * inv_alpha : ldexpf(v, -e);
  float r = rintf(scaled);
  r = fminf(fmaxf(r, -bmax), bmax);
  return __float2int_rn(r);
}

__global__ void __launch_bounds__(256)
quantize_f32_kernel(const float* __restrict__ x, int8_t* __restrict__ y, size_t count, int e, int n,
                    int vec_ok) {
  chain_sync();
  const float bmax = static_cast<float>((1 << (n - 1)) - 1);
  const float gam = ldexpf(bmax, e);
  const bool use_mul = (e >= -100 && e <= 100);
  const float inv_alpha = use_mul ? ldexpf(1.0f, -e) : 0.0f;
  const size_t tid = blockIdx.x * static_cast<size_t>(blockDim.x) + threadIdx.x;
  const size_t nthreads = static_cast<size_t>(gridDim.x) * blockDim.x;
  size_t nvec = vec_ok ? count / 16 : 0;
  const float4* x4 = reinterpret_cast<const float4*>(x);
  uint4* y16 = reinterpret_cast<uint4*>(y);
  for (size_t i = tid; i < nvec; i += nthreads) {
    if (!QC_IN(16 * i + 15, count)) continue;
    float4 a = __ldg(x4 + 4 * i), b = __ldg(x4 + 4 * i + 1), c = __ldg(x4 + 4 * i + 2),
           d = __ldg(x4 + 4 * i + 3);
    float f[16] = {a.x, a.y, a.z, a.w, b.x, b.y, b.z, b.w, c.x, c.y, c.z, c.w, d.x, d.y, d.z, d.w};
    uint32_t wds[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      uint32_t wd = 0;
#pragma unroll
      for (int b8 = 0; b8 < 4; ++b8) {
        int q = quantize_one(f[4 * j + b8], gam, inv_alpha, e, use_mul, bmax);
        wd |= (static_cast<uint32_t>(q) & 0xFFu) << (8 * b8);
      }
      wds[j] = wd;
    }
    y16[i] = make_uint4(wds[0], wds[1], wds[2], wds[3]);
  }
  for (size_t i = nvec * 16 + tid; i < count; i += nthreads)
    y[i] = static_cast<int8_t>(quantize_one(x[i], gam, inv_alpha, e, use_mul, bmax));
}

// ---------------------------------------------------------------------------------------
// int8 max-pool, NHWC.  Vector path: one thread per 16 channels of one output pixel.
// ---------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256)
maxpool_i8_vec_kernel(const int8_t* __restrict__ x, int8_t* __restrict__ y, int N, int H, int W, int C,
                      int R, int S, int stride, int pad, int P, int Q) {
  chain_sync();
  const int cv = C / 16;
  const size_t total = static_cast<size_t>(N) * P * Q * cv;
  for (size_t idx = blockIdx.x * static_cast<size_t>(blockDim.x) + threadIdx.x; idx < total;
       idx += static_cast<size_t>(gridDim.x) * blockDim.x) {
    int c = static_cast<int>(idx % cv);
    size_t pix = idx / cv;
    int q = static_cast<int>(pix % Q);
    int p = static_cast<int>((pix / Q) % P);
    int n = static_cast<int>(pix / (static_cast<size_t>(Q) * P));
    uint4 m = make_uint4(0x80808080u, 0x80808080u, 0x80808080u, 0x80808080u);
    for (int r = 0; r < R; ++r) {
      int h = p * stride - pad + r;
      if (h < 0 || h >= H) continue;
      for (int s = 0; s < S; ++s) {
        int w = q * stride - pad + s;
        if (w < 0 || w >= W) continue;
        if (!QC_IN(((static_cast<size_t>(n) * H + h) * W + w) * C + 16 * c + 15, static_cast<size_t>(N) * H * W * C)) continue;
        uint4 v = __ldg(reinterpret_cast<const uint4*>(x + ((static_cast<size_t>(n) * H + h) * W + w) * C) + c);
        m.x = __vmaxs4(m.x, v.x); m.y = __vmaxs4(m.y, v.y);
        m.z = __vmaxs4(m.z, v.z); m.w = __vmaxs4(m.w, v.w);
      }
    }
    if (QC_IN(pix * C + 16 * c + 15, static_cast<size_t>(N) * P * Q * C)) reinterpret_cast<uint4*>(y + pix * C)[c] = m;
  }
}

// Strip form for the common windows (3x3 stride 1 or 2, 2x2 stride 2): one thread owns 16 channels
// of one output column and walks down a strip of output rows.  The horizontal maximum of an input
// row is taken once and kept in registers for every output row whose window contains it, so a
// 3x3 stride-1 pool loads 3 vectors per output instead of 9.  The maxima are taken on pairs of
// sign-extended 16-bit lanes (one permute per pair, then the two-lane integer max the hardware
// has; a four-lane byte max would be emulated) and narrowed back to bytes at the end.
struct PoolRow { uint32_t w[8]; };            // 16 channels as 8 words of two 16-bit lanes

// bytes (0, 1) / (2, 3) of a word as two sign-extended 16-bit lanes
__device__ __forceinline__ uint32_t widen_lo(uint32_t v) {
  uint32_t d;
  asm("prmt.b32 %0, %1, 0, 0x9180;" : "=r"(d) : "r"(v));
  return d;
}
__device__ __forceinline__ uint32_t widen_hi(uint32_t v) {
  uint32_t d;
  asm("prmt.b32 %0, %1, 0, 0xB3A2;" : "=r"(d) : "r"(v));
  return d;
}
__device__ __forceinline__ void pool_widen(const uint4& v, PoolRow& r) {
  r.w[0] = widen_lo(v.x); r.w[1] = widen_hi(v.x); r.w[2] = widen_lo(v.y); r.w[3] = widen_hi(v.y);
  r.w[4] = widen_lo(v.z); r.w[5] = widen_hi(v.z); r.w[6] = widen_lo(v.w); r.w[7] = widen_hi(v.w);
}

template <int R, int S, int ST>
__global__ void __launch_bounds__(256)
maxpool_i8_strip_kernel(const int8_t* __restrict__ x, int8_t* __restrict__ y, int N, int H, int W, int C,
                        int pad, int P, int Q, int rows_per_thread, int strips) {
  chain_sync();
  const int cv = C / 16;
  // (the host keeps the thread count below 2^31: 32-bit index arithmetic)
  const unsigned int total = static_cast<unsigned int>(N) * strips * Q * cv;
  const unsigned int idx = blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= total) return;
  const int c = static_cast<int>(idx % cv);
  unsigned int t = idx / cv;
  const int q = static_cast<int>(t % Q); t /= Q;
  const int strip = static_cast<int>(t % strips);
  const int n = static_cast<int>(t / strips);
  const int p0 = strip * rows_per_thread;
  const int p1 = min(P, p0 + rows_per_thread);
  const uint4 lowest = make_uint4(0x80808080u, 0x80808080u, 0x80808080u, 0x80808080u);
  const uint4* xin = reinterpret_cast<const uint4*>(x) + static_cast<size_t>(n) * H * W * cv + c;
  const int w0 = q * ST - pad;
  // horizontal maximum of input row h over the window's columns (taps outside the image are ignored)
  auto hmax = [&](int h, PoolRow& m) {
    const bool row_in = h >= 0 && h < H;
    const uint4* row = xin + static_cast<size_t>(row_in ? h : 0) * W * cv;
    uint4 v[S];
#pragma unroll
    for (int sx = 0; sx < S; ++sx) {
      const int w = w0 + sx;
      const bool in = row_in && w >= 0 && w < W &&
                      QC_IN((static_cast<size_t>(n) * H + (row_in ? h : 0)) * W * cv + static_cast<size_t>(w) * cv + c,
                            static_cast<size_t>(N) * H * W * cv);
      v[sx] = in ? __ldg(row + static_cast<size_t>(w) * cv) : lowest;
    }
    pool_widen(v[0], m);
    if (S == 3) {
      PoolRow a, b;
      pool_widen(v[1], a);
      pool_widen(v[S - 1], b);
#pragma unroll
      for (int j = 0; j < 8; ++j) m.w[j] = __vimax3_s16x2(m.w[j], a.w[j], b.w[j]);
    } else {
#pragma unroll
      for (int sx = 1; sx < S; ++sx) {
        PoolRow o;
        pool_widen(v[sx], o);
#pragma unroll
        for (int j = 0; j < 8; ++j) m.w[j] = __vmaxs2(m.w[j], o.w[j]);
      }
    }
  };
  constexpr int KEEP = R > ST ? R - ST : 0;       // rows shared by consecutive windows
  PoolRow win[R];
#pragma unroll
  for (int i = 0; i < KEEP; ++i) hmax(p0 * ST - pad + i, win[i + (R - KEEP)]);
  uint4* yout = reinterpret_cast<uint4*>(y) + ((static_cast<size_t>(n) * P + p0) * Q + q) * cv + c;
  for (int p = p0; p < p1; ++p) {
#pragma unroll
    for (int i = 0; i < KEEP; ++i) win[i] = win[i + (R - KEEP)];
#pragma unroll
    for (int i = KEEP; i < R; ++i) hmax(p * ST - pad + i, win[i]);
    PoolRow m = win[0];
    if (R == 3) {
#pragma unroll
      for (int j = 0; j < 8; ++j) m.w[j] = __vimax3_s16x2(m.w[j], win[1].w[j], win[R - 1].w[j]);
    } else {
#pragma unroll
      for (int i = 1; i < R; ++i)
#pragma unroll
        for (int j = 0; j < 8; ++j) m.w[j] = __vmaxs2(m.w[j], win[i].w[j]);
    }
    // every lane holds a value in [-128, 127]: its low byte is the result
    if (QC_IN(((static_cast<size_t>(n) * P + p) * Q + q) * cv + c, static_cast<size_t>(N) * P * Q * cv))
      *yout = make_uint4(__byte_perm(m.w[0], m.w[1], 0x6420), __byte_perm(m.w[2], m.w[3], 0x6420),
                         __byte_perm(m.w[4], m.w[5], 0x6420), __byte_perm(m.w[6], m.w[7], 0x6420));
    yout += static_cast<size_t>(Q) * cv;
  }
}

__global__ void __launch_bounds__(256)
maxpool_i8_scalar_kernel(const int8_t* __restrict__ x, int8_t* __restrict__ y, int N, int H, int W,
                         int C, int R, int S, int stride, int pad, int P, int Q) {
  const size_t total = static_cast<size_t>(N) * P * Q * C;
  for (size_t idx = blockIdx.x * static_cast<size_t>(blockDim.x) + threadIdx.x; idx < total;
       idx += static_cast<size_t>(gridDim.x) * blockDim.x) {
    int c = static_cast<int>(idx % C);
    size_t pix = idx / C;
    int q = static_cast<int>(pix % Q);
    int p = static_cast<int>((pix / Q) % P);
    int n = static_cast<int>(pix / (static_cast<size_t>(Q) * P));
    int m = -128;
    for (int r = 0; r < R; ++r) {
      int h = p * stride - pad + r;
      if (h < 0 || h >= H) continue;
      for (int s = 0; s < S; ++s) {
        int w = q * stride - pad + s;
        if (w < 0 || w >= W) continue;
        if (QC_IN(((static_cast<size_t>(n) * H + h) * W + w) * C + c, static_cast<size_t>(N) * H * W * C))
          m = max(m, static_cast<int>(x[((static_cast<size_t>(n) * H + h) * W + w) * C + c]));
      }
    }
    y[idx] = static_cast<int8_t>(m);
  }
}

// ---------------------------------------------------------------------------------------
// Stem patch packing: for layers with very few input channels (C <= 4), the R*S*C taps of
// each output pixel are gathered into one row of kg_pad bytes (zeros for taps outside the
// image and for the padding), so the tensor-core GEMM can consume them as a 1x1 layer.
// One thread writes 16 bytes.
// ---------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256)
stem_pack_kernel(const int8_t* __restrict__ x, int8_t* __restrict__ a, int N, int H, int W, int C,
                 int R, int S, int stride_h, int stride_w, int pad_h, int pad_w, int P, int Q,
                 int kg, int kg_pad) {
  const int vec_per_row = kg_pad / 16;
  const size_t total = static_cast<size_t>(N) * P * Q * vec_per_row;
  for (size_t idx = blockIdx.x * static_cast<size_t>(blockDim.x) + threadIdx.x; idx < total;
       idx += static_cast<size_t>(gridDim.x) * blockDim.x) {
    int v = static_cast<int>(idx % vec_per_row);
    size_t pix = idx / vec_per_row;
    int q = static_cast<int>(pix % Q);
    int p = static_cast<int>((pix / Q) % P);
    int n = static_cast<int>(pix / (static_cast<size_t>(Q) * P));
    uint32_t wds[4] = {0, 0, 0, 0};
#pragma unroll
    for (int j = 0; j < 16; ++j) {
      int t = v * 16 + j;
      int val = 0;
      if (t < kg) {
        int c = t % C;
        int s = (t / C) % S;
        int r = t / (C * S);
        int h = p * stride_h - pad_h + r;
        int w = q * stride_w - pad_w + s;
        if (h >= 0 && h < H && w >= 0 && w < W &&
            QC_IN(((static_cast<size_t>(n) * H + h) * W + w) * C + c, static_cast<size_t>(N) * H * W * C))
          val = x[((static_cast<size_t>(n) * H + h) * W + w) * C + c];
      }
      wds[j >> 2] |= (static_cast<uint32_t>(val) & 0xFFu) << (8 * (j & 3));
    }
    reinterpret_cast<uint4*>(a)[idx] = make_uint4(wds[0], wds[1], wds[2], wds[3]);
  }
}

// Copy of an NHWC int8 image into rows padded with zeros: pixel w of image row `row` goes to pixel
// off_w + w of a row of wp pixels (cv 16-byte vectors per pixel).  The padding is never written
// (the buffer is cleared once when it is allocated).  One thread per 16-byte vector.
__global__ void __launch_bounds__(256)
pad_rows_kernel(const uint4* __restrict__ x, uint4* __restrict__ a, unsigned int vecs, int rows, int W, int cv,
                int wp, int off_w) {
  chain_sync();
  const unsigned int idx = blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= vecs) return;
  const unsigned int per_row = static_cast<unsigned int>(W) * cv;
  const unsigned int row = idx / per_row, in_row = idx - row * per_row;
  if (QC_IN((static_cast<size_t>(row) * wp + off_w) * cv + in_row, static_cast<size_t>(rows) * wp * cv) && QC_IN(row, rows))
    a[(static_cast<size_t>(row) * wp + off_w) * cv + in_row] = __ldg(x + idx);
}

// Row padding for stride-1 layers on C <= 4 channels: every pixel becomes a pixel of PB bytes (8 or 16:
// its C bytes, then zeros) at pixel off_w + w of a row of wp pixels, so that the S taps of a filter row
// are adjacent PB-byte pixels and an overlapping TMA view (row pitch PB, or fold * PB) hands the tensor
// core its operand without a patch matrix.  The padding pixels are never written (the buffer is cleared
// once when it is allocated).  One thread per 4 consecutive pixels: 4 * C source bytes from a 4-byte
// boundary (C aligned word loads), 4 * PB destination bytes.  FROM_F32: the source is the float image and
// the input conversion (same quantize_one as quantize_f32_kernel) happens on the way.
template <int C, int PB, bool FROM_F32>
__global__ void __launch_bounds__(256)
stem_row_pack_kernel(const void* __restrict__ xv, int8_t* __restrict__ a, unsigned int pixels, int W, int wp,
                     int off_w, int e, int n_bits) {
  static_assert(C >= 1 && C <= 4 && (PB == 8 || PB == 16), "pixel of 8 or 16 bytes");
  chain_sync();
  const unsigned int p0 = (blockIdx.x * blockDim.x + threadIdx.x) * 4u;
  if (p0 >= pixels) return;
  const bool whole = p0 + 4u <= pixels;
  uint32_t px[4] = {0u, 0u, 0u, 0u};               // the channel bytes of 4 pixels, each from bit 0 up
  if (FROM_F32) {
    const float* src = static_cast<const float*>(xv) + static_cast<size_t>(p0) * C;
    const float bmax = static_cast<float>((1 << (n_bits - 1)) - 1);
    const float gam = ldexpf(bmax, e);
    const bool use_mul = (e >= -100 && e <= 100);
    const float inv_alpha = use_mul ? ldexpf(1.0f, -e) : 0.0f;
    float f[4 * C];
    if (whole && (reinterpret_cast<uintptr_t>(src) & 15) == 0 && QC_IN(static_cast<size_t>(p0) * C + 4 * C - 1, static_cast<size_t>(pixels) * C)) {
#pragma unroll
      for (int i = 0; i < C; ++i) {
        const float4 v = __ldg(reinterpret_cast<const float4*>(src) + i);
        f[4 * i] = v.x; f[4 * i + 1] = v.y; f[4 * i + 2] = v.z; f[4 * i + 3] = v.w;
      }
    } else {
#pragma unroll
      for (int i = 0; i < 4 * C; ++i)
        f[i] = (p0 + i / C < pixels && QC_IN(static_cast<size_t>(p0) * C + i, static_cast<size_t>(pixels) * C)) ? __ldg(src + i) : 0.0f;
    }
#pragma unroll
    for (int i = 0; i < 4 * C; ++i)
      px[i / C] |= static_cast<uint32_t>(static_cast<uint8_t>(quantize_one(f[i], gam, inv_alpha, e, use_mul, bmax))) << (8 * (i % C));
  } else {
    const int8_t* src = static_cast<const int8_t*>(xv) + static_cast<size_t>(p0) * C;
    if (whole && (reinterpret_cast<uintptr_t>(src) & 3) == 0 && QC_IN(static_cast<size_t>(p0) * C + 4 * C - 1, static_cast<size_t>(pixels) * C)) {
      uint32_t w[C];
#pragma unroll
      for (int i = 0; i < C; ++i) w[i] = __ldg(reinterpret_cast<const uint32_t*>(src) + i);
#pragma unroll
      for (int i = 0; i < 4 * C; ++i) px[i / C] |= ((w[i >> 2] >> (8 * (i & 3))) & 0xFFu) << (8 * (i % C));
    } else {
#pragma unroll
      for (int i = 0; i < 4 * C; ++i)
        if (p0 + i / C < pixels && QC_IN(static_cast<size_t>(p0) * C + i, static_cast<size_t>(pixels) * C))
          px[i / C] |= static_cast<uint32_t>(static_cast<uint8_t>(__ldg(src + i))) << (8 * (i % C));
    }
  }
  unsigned int row = p0 / static_cast<unsigned int>(W);
  int col = static_cast<int>(p0 - row * static_cast<unsigned int>(W));
  [[maybe_unused]] const size_t rows = pixels / static_cast<unsigned int>(W);
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    if (p0 + j < pixels) {
      const size_t dst = static_cast<size_t>(row) * wp + off_w + col;
      if (QC_IN(dst, rows * wp) && QC_IN(off_w + col, wp)) {
        if (PB == 8) *reinterpret_cast<uint2*>(a + dst * 8) = make_uint2(px[j], 0u);
        else *reinterpret_cast<uint4*>(a + dst * 16) = make_uint4(px[j], 0u, 0u, 0u);
      }
    }
    if (++col == W) { col = 0; ++row; }
  }
}

// Space-to-depth packing for stride-2 stems with C <= 4: a 2 x 2 block of input pixels becomes one
// 16-byte pixel of a half-resolution image (byte (dy * 2 + dx) * C + c, zero padded), so that the
// stride-2 R x S filter turns into a stride-1 filter over ceil-halved taps whose horizontal taps
// are ADJACENT 16-byte pixels: one overlapping TMA view (row pitch 16 bytes, rows of S2 * 16
// bytes) then hands the tensor core its operand directly and no patch matrix is ever written.
// Destination rows are wp pixels long, the image starting at pixel off_w; the padding pixels and
// the rows / columns a ragged (odd) image lacks are zero (the buffer is cleared once when it is
// allocated and this kernel writes only inside the image).  One thread per block pixel.
template <int C>
__global__ void __launch_bounds__(256)
stem_s2d_pack_kernel(const int8_t* __restrict__ x, uint4* __restrict__ a, int N, int H, int W,
                     int H2, int W2, int wp, int off_w) {
  chain_sync();
  const int bx = blockIdx.x * blockDim.x + threadIdx.x;
  const int by = blockIdx.y;
  const int n = blockIdx.z;
  if (bx >= W2) return;
  unsigned long long rb[2] = {0ull, 0ull};        // the (up to) 2 * C contiguous bytes of pixels 2bx, 2bx+1, per row
  const bool both = 2 * bx + 1 < W;               // the block's right pixel exists
#pragma unroll
  for (int dy = 0; dy < 2; ++dy) {
    const int yy = 2 * by + dy;
    if (yy >= H) continue;
    const int8_t* src = x + ((static_cast<size_t>(n) * H + yy) * W + 2 * bx) * C;
    if (!QC_IN(((static_cast<size_t>(n) * H + yy) * W + 2 * bx) * C + (both ? 2 * C : C) - 1, static_cast<size_t>(N) * H * W * C)) continue;
    if (both && (reinterpret_cast<uintptr_t>(src) & 1) == 0) {
      // 2 * C bytes from an even address: C two-byte loads
      const unsigned short* s2 = reinterpret_cast<const unsigned short*>(src);
#pragma unroll
      for (int j = 0; j < C; ++j) rb[dy] |= static_cast<unsigned long long>(__ldg(s2 + j)) << (16 * j);
    } else {
#pragma unroll
      for (int j = 0; j < 2 * C; ++j)
        if (j < C || both) rb[dy] |= static_cast<unsigned long long>(static_cast<uint8_t>(__ldg(src + j))) << (8 * j);
    }
  }
  // second row's bytes follow the first row's 2 * C bytes
  constexpr int sh = 16 * C;                       // bits; 64 when C == 4
  const unsigned long long lo = rb[0] | (sh < 64 ? rb[1] << (sh & 63) : 0ull);
  const unsigned long long hi = sh < 64 ? rb[1] >> ((64 - sh) & 63) : rb[1];
  if (QC_IN((static_cast<size_t>(n) * H2 + by) * wp + off_w + bx, static_cast<size_t>(N) * H2 * wp) && QC_IN(off_w + bx, wp))
    a[(static_cast<size_t>(n) * H2 + by) * wp + off_w + bx] =
        make_uint4(static_cast<uint32_t>(lo), static_cast<uint32_t>(lo >> 32), static_cast<uint32_t>(hi),
                   static_cast<uint32_t>(hi >> 32));
}

// The same packing straight from the float image: the input conversion (clamp to +-gamma, scale by
// 2^-e, nearest-even, clamp to +-beta_max; NaN -> 0) happens on the way, so the int8 image is
// never written.  Arithmetic identical to quantize_f32_kernel (same quantize_one).
template <int C>
__global__ void __launch_bounds__(256)
stem_s2d_pack_f32_kernel(const float* __restrict__ x, uint4* __restrict__ a, int N, int H, int W,
                         int H2, int W2, int wp, int off_w, int e, int n_bits) {
  chain_sync();
  const int bx = blockIdx.x * blockDim.x + threadIdx.x;
  const int by = blockIdx.y;
  const int n = blockIdx.z;
  if (bx >= W2) return;
  const float bmax = static_cast<float>((1 << (n_bits - 1)) - 1);
  const float gam = ldexpf(bmax, e);
  const bool use_mul = (e >= -100 && e <= 100);
  const float inv_alpha = use_mul ? ldexpf(1.0f, -e) : 0.0f;
  unsigned long long rb[2] = {0ull, 0ull};
  const bool both = 2 * bx + 1 < W;
#pragma unroll
  for (int dy = 0; dy < 2; ++dy) {
    const int yy = 2 * by + dy;
    if (yy >= H) continue;
    const float* src = x + ((static_cast<size_t>(n) * H + yy) * W + 2 * bx) * C;
    if (!QC_IN(((static_cast<size_t>(n) * H + yy) * W + 2 * bx) * C + (both ? 2 * C : C) - 1, static_cast<size_t>(N) * H * W * C)) continue;
#pragma unroll
    for (int j = 0; j < 2 * C; ++j)
      if (j < C || both) {
        const int q = quantize_one(__ldg(src + j), gam, inv_alpha, e, use_mul, bmax);
        rb[dy] |= static_cast<unsigned long long>(static_cast<uint8_t>(q)) << (8 * j);
      }
  }
  constexpr int sh = 16 * C;
  const unsigned long long lo = rb[0] | (sh < 64 ? rb[1] << (sh & 63) : 0ull);
  const unsigned long long hi = sh < 64 ? rb[1] >> ((64 - sh) & 63) : rb[1];
  if (QC_IN((static_cast<size_t>(n) * H2 + by) * wp + off_w + bx, static_cast<size_t>(N) * H2 * wp) && QC_IN(off_w + bx, wp))
    a[(static_cast<size_t>(n) * H2 + by) * wp + off_w + bx] =
        make_uint4(static_cast<uint32_t>(lo), static_cast<uint32_t>(lo >> 32), static_cast<uint32_t>(hi),
                   static_cast<uint32_t>(hi >> 32));
}

// Faster stem packing for S * C <= 28 bytes: the S * C bytes that one output pixel needs from one
// input row are contiguous in NHWC, so the packed row is R segments (one per filter row), each
// copied as a few aligned 32-bit words, realigned with funnel shifts and zero-masked at the image
// border.  Segment r lives at byte r * segp of the packed row (segp = 16 or 32).  One thread packs
// one output pixel -- all R segments and the row's zero padding, a contiguous run of bytes, so
// every 32-byte sector of the destination is written whole (a half-written sector costs a fill
// read from DRAM) -- and consecutive lanes take consecutive output columns, so
// a warp's loads fall into one or two cache lines.  Windows that lie inside their row and clear
// of the tensor's last words take a branch-free path; the others are clipped byte-exactly.
// SEGW: words per segment, 4 (16 bytes) or 8 (32 bytes); NW: words that hold segment bytes,
// ceil(S * C / 4).  Block = 64 output columns x 4 output rows of one image (blockIdx.z).
template <int SEGW, int NW>
__global__ void __launch_bounds__(256)
stem_pack_rows_kernel(const int8_t* __restrict__ x, int8_t* __restrict__ a, int N, int H, int W, int C,
                      int R, int S, int stride_h, int stride_w, int pad_h, int pad_w, int P, int Q,
                      int kg_pad, long long x_words, int x_tail) {
  static_assert(NW >= 1 && NW <= SEGW, "segment words");
  const int q = blockIdx.x * 64 + (threadIdx.x & 63);
  const int p = blockIdx.y * 4 + (threadIdx.x >> 6);
  const int n = blockIdx.z;
  if (q >= Q || p >= P) return;
  const uint32_t* x32 = reinterpret_cast<const uint32_t*>(x);
  const int seg_bytes = S * C;
  const long long img_b0 = static_cast<long long>(n) * H * W * C;      // byte offset of this image
  const int row_bytes = W * C;
  const uint32_t tail_mask = (seg_bytes & 3) ? ((1u << (8 * (seg_bytes & 3))) - 1u) : 0xFFFFFFFFu;
  // largest in-image byte offset whose NW + 1 words all lie before the tensor's last whole word
  const long long lim = (x_words - NW - 1) * 4 - img_b0 + 3;
  const int safe_off = lim > 0x7FFFFFFFll ? 0x7FFFFFFF : (lim < 0 ? -1 : static_cast<int>(lim));
  const int w0 = q * stride_w - pad_w;
  const int wb = w0 * C;                                                // byte offset of the window in its row
  const bool cols_inside = w0 >= 0 && wb + seg_bytes <= row_bytes;
  const size_t pix = (static_cast<size_t>(n) * P + p) * Q + q;
  uint4* dst = reinterpret_cast<uint4*>(a + pix * kg_pad);
  const int h0 = p * stride_h - pad_h;
  for (int r = 0; r < R; ++r, dst += SEGW / 4) {
    const int h = h0 + r;
    uint32_t out[SEGW];
#pragma unroll
    for (int k = 0; k < SEGW; ++k) out[k] = 0u;
    if (h >= 0 && h < H) {
      const int off = h * row_bytes + wb;                  // byte offset of the window inside the image
      if (cols_inside && off <= safe_off) {
        const long long b0 = img_b0 + off;
        const uint32_t* src = x32 + (b0 >> 2);
        const int sh = (static_cast<int>(b0) & 3) * 8;
        uint32_t wd[NW + 1];
#pragma unroll
        for (int k = 0; k <= NW; ++k) wd[k] = QC_IN((b0 >> 2) + k, x_words) ? __ldg(src + k) : 0u;
#pragma unroll
        for (int k = 0; k < NW; ++k) out[k] = __funnelshift_r(wd[k], wd[k + 1], sh);
        out[NW - 1] &= tail_mask;
      } else {
        const long long b0 = img_b0 + off;                 // may start left of the row; masked below
        const long long wi = b0 >> 2;                      // floor division, also for negative b0
        const int sh = static_cast<int>(b0 & 3) * 8;
        uint32_t wd[NW + 1];
#pragma unroll
        for (int k = 0; k <= NW; ++k) {
          const long long j = wi + k;
          uint32_t v = 0u;
          if (j >= 0) {
            if (j < x_words) {
              v = __ldg(x32 + j);
            } else if (j == x_words) {                     // the tensor's last, partial word: byte by byte
              for (int tb = 0; tb < x_tail; ++tb)
                v |= static_cast<uint32_t>(static_cast<uint8_t>(x[j * 4 + tb])) << (8 * tb);
            }
          }
          wd[k] = v;
        }
        const int lo = w0 < 0 ? -wb : 0;                     // first valid byte of the window
        const int hi = min(seg_bytes, row_bytes - wb);       // one past the last valid byte
#pragma unroll
        for (int k = 0; k < NW; ++k) {
          const uint32_t v = __funnelshift_r(wd[k], wd[k + 1], sh);
          const int nlo = lo - 4 * k, nhi = hi - 4 * k;      // valid bytes of this word: [nlo, nhi)
          const uint32_t mhi = nhi <= 0 ? 0u : (nhi >= 4 ? 0xFFFFFFFFu : ((1u << (8 * nhi)) - 1u));
          const uint32_t mlo = nlo <= 0 ? 0u : (nlo >= 4 ? 0xFFFFFFFFu : ((1u << (8 * nlo)) - 1u));
          out[k] = v & mhi & ~mlo;
        }
      }
    }
#pragma unroll
    for (int k = 0; k < SEGW; k += 4)
      if (QC_IN(pix * kg_pad + static_cast<size_t>(r) * SEGW * 4 + k * 4 + 15, static_cast<size_t>(N) * P * Q * kg_pad))
        dst[k / 4] = make_uint4(out[k], out[k + 1], out[k + 2], out[k + 3]);
  }
  // the row's padding, so that every 32-byte sector of the destination is written whole
  for (int bytes = R * SEGW * 4; bytes < kg_pad; bytes += 16, ++dst)
    if (QC_IN(pix * kg_pad + bytes + 15, static_cast<size_t>(N) * P * Q * kg_pad)) *dst = make_uint4(0u, 0u, 0u, 0u);
}

// ---------------------------------------------------------------------------------------
// Direct convolution on CUDA cores, any shape / groups / stride: one thread per output
// value, output channel fastest.  Weights are repacked to [R][S][C/g][K] so that a warp
// reads consecutive weights.  This is the general path for shapes the tensor-core and
// depthwise kernels do not take, and an in-library cross-check for them.
// ---------------------------------------------------------------------------------------
struct ConvGeom {
  int N, H, W, C, K, R, S, stride_h, stride_w, pad_h, pad_w, groups, P, Q;
  int out_c_offset, out_c_pitch;
};

__device__ __forceinline__ void store_out(void* y, size_t idx, size_t extent, int32_t wide, int k,
                                          const EpilogueParams& ep) {
  if (!QC_IN(idx, extent)) return;
  if (ep.out_mode == 0) {
    int32_t v = requantize(wide, ep.shift[k], ep.rounding, ep.lo, ep.hi);
    static_cast<int8_t*>(y)[idx] = static_cast<int8_t>(v);
  } else if (ep.out_mode == 1) {
    static_cast<int32_t*>(y)[idx] = wide;
  } else {
    static_cast<float*>(y)[idx] = dequantize(wide, ep.acc_exp[k]);
  }
}

__global__ void __launch_bounds__(256)
direct_conv_kernel(const int8_t* __restrict__ x, const int8_t* __restrict__ w_rsck,
                   const int8_t* __restrict__ res, void* __restrict__ y, ConvGeom g,
                   EpilogueParams ep) {
  const int Cg = g.C / g.groups;
  const int Kg = g.K / g.groups;
  const size_t total = static_cast<size_t>(g.N) * g.P * g.Q * g.K;
  for (size_t idx = blockIdx.x * static_cast<size_t>(blockDim.x) + threadIdx.x; idx < total;
       idx += static_cast<size_t>(gridDim.x) * blockDim.x) {
    int k = static_cast<int>(idx % g.K);
    size_t pix = idx / g.K;
    int q = static_cast<int>(pix % g.Q);
    int p = static_cast<int>((pix / g.Q) % g.P);
    int n = static_cast<int>(pix / (static_cast<size_t>(g.Q) * g.P));
    int grp = k / Kg;
    int32_t acc = 0;
    for (int r = 0; r < g.R; ++r) {
      int h = p * g.stride_h - g.pad_h + r;
      if (h < 0 || h >= g.H) continue;
      for (int s = 0; s < g.S; ++s) {
        int wc = q * g.stride_w - g.pad_w + s;
        if (wc < 0 || wc >= g.W) continue;
        const int8_t* xp = x + ((static_cast<size_t>(n) * g.H + h) * g.W + wc) * g.C + grp * Cg;
        const int8_t* wp = w_rsck + (static_cast<size_t>(r) * g.S + s) * Cg * g.K + k;
        if (!QC_IN(((static_cast<size_t>(n) * g.H + h) * g.W + wc) * g.C + grp * Cg + Cg - 1, static_cast<size_t>(g.N) * g.H * g.W * g.C) ||
            !QC_IN((static_cast<size_t>(r) * g.S + s) * Cg * g.K + k + static_cast<size_t>(Cg - 1) * g.K, static_cast<size_t>(g.R) * g.S * Cg * g.K))
          continue;
        for (int c = 0; c < Cg; ++c)
          acc += static_cast<int32_t>(xp[c]) * static_cast<int32_t>(wp[static_cast<size_t>(c) * g.K]);
      }
    }
    int32_t rv = (res && QC_IN(pix * g.K + k, static_cast<size_t>(g.N) * g.P * g.Q * g.K)) ? static_cast<int32_t>(res[pix * g.K + k]) : 0;
    int t = ep.res_lshift ? ep.res_lshift[k] : 0;
    int32_t wide = wide_value(acc, ep.bias ? ep.bias[k] : 0, rv, t, ep.relu);
    store_out(y, pix * g.out_c_pitch + g.out_c_offset + k, static_cast<size_t>(g.N) * g.P * g.Q * g.out_c_pitch, wide, k, ep);
  }
}

// ---------------------------------------------------------------------------------------
// Depthwise 3x3 (groups == C == K) on CUDA cores.  One thread owns 4 channels (one 32-bit
// word of the NHWC row, so a warp reads 128 contiguous bytes) and TW consecutive output
// columns; each input word is loaded once per thread and reused across the taps that need
// it.  A product x[c] * w[c] of one byte lane is a dp4a against a weight word that is zero
// in the other three lanes.  Weights are repacked to [R*S][C].
// ---------------------------------------------------------------------------------------
template <int STRIDE, int TW>
__global__ void __launch_bounds__(256)
depthwise3x3_kernel(const int8_t* __restrict__ x, const int8_t* __restrict__ w_rsc,
                    const int8_t* __restrict__ res, void* __restrict__ y, ConvGeom g,
                    EpilogueParams ep) {
  constexpr int IW = (TW - 1) * STRIDE + 3;     // input columns one thread touches per row
  const int cw = g.C / 4;
  const int qt = (g.Q + TW - 1) / TW;
  const size_t total = static_cast<size_t>(g.N) * g.P * qt * cw;
  const uint32_t* x32 = reinterpret_cast<const uint32_t*>(x);
  const uint32_t* w32 = reinterpret_cast<const uint32_t*>(w_rsc);
  for (size_t idx = blockIdx.x * static_cast<size_t>(blockDim.x) + threadIdx.x; idx < total;
       idx += static_cast<size_t>(gridDim.x) * blockDim.x) {
    int c4 = static_cast<int>(idx % cw);
    size_t rest = idx / cw;
    int qi = static_cast<int>(rest % qt);
    int p = static_cast<int>((rest / qt) % g.P);
    int n = static_cast<int>(rest / (static_cast<size_t>(qt) * g.P));
    int q0 = qi * TW;
    int32_t acc[TW][4];
#pragma unroll
    for (int j = 0; j < TW; ++j)
#pragma unroll
      for (int l = 0; l < 4; ++l) acc[j][l] = 0;
#pragma unroll
    for (int r = 0; r < 3; ++r) {
      int h = p * STRIDE - g.pad_h + r;
      if (h < 0 || h >= g.H) continue;
      uint32_t wr[3];
#pragma unroll
      for (int s = 0; s < 3; ++s) wr[s] = __ldg(w32 + (r * 3 + s) * cw + c4);
      const uint32_t* row = x32 + (static_cast<size_t>(n) * g.H + h) * g.W * cw + c4;
      int w0 = q0 * STRIDE - g.pad_w;
      uint32_t xin[IW];
#pragma unroll
      for (int i = 0; i < IW; ++i) {
        int wc = w0 + i;
        xin[i] = (wc >= 0 && wc < g.W &&
                  QC_IN((static_cast<size_t>(n) * g.H + h) * g.W * cw + c4 + static_cast<size_t>(wc) * cw, static_cast<size_t>(g.N) * g.H * g.W * cw))
                     ? __ldg(row + static_cast<size_t>(wc) * cw) : 0u;
      }
#pragma unroll
      for (int s = 0; s < 3; ++s)
#pragma unroll
        for (int l = 0; l < 4; ++l) {
          int wsel = static_cast<int>(wr[s] & (0xFFu << (8 * l)));
#pragma unroll
          for (int j = 0; j < TW; ++j)
            acc[j][l] = __dp4a(static_cast<int>(xin[j * STRIDE + s]), wsel, acc[j][l]);
        }
    }
    int k0 = c4 * 4;
    int32_t bias[4], sh[4], tl[4], ae[4];
#pragma unroll
    for (int l = 0; l < 4; ++l) {
      bias[l] = ep.bias ? ep.bias[k0 + l] : 0;
      sh[l] = ep.shift[k0 + l];
      tl[l] = ep.res_lshift ? ep.res_lshift[k0 + l] : 0;
      ae[l] = ep.acc_exp[k0 + l];
    }
#pragma unroll
    for (int j = 0; j < TW; ++j) {
      int q = q0 + j;
      if (q >= g.Q) break;
      size_t pix = (static_cast<size_t>(n) * g.P + p) * g.Q + q;
      uint32_t rword = res ? __ldg(reinterpret_cast<const uint32_t*>(res + pix * g.K) + c4) : 0u;
      int32_t wide[4];
#pragma unroll
      for (int l = 0; l < 4; ++l) {
        int32_t rv = static_cast<int32_t>(static_cast<int8_t>((rword >> (8 * l)) & 0xFFu));
        wide[l] = wide_value(acc[j][l], bias[l], rv, tl[l], ep.relu);
      }
      size_t o = pix * g.out_c_pitch + g.out_c_offset + k0;
      if (!QC_IN(o + 3, static_cast<size_t>(g.N) * g.P * g.Q * g.out_c_pitch)) continue;
      if (ep.out_mode == 0) {
        uint32_t wd = 0;
#pragma unroll
        for (int l = 0; l < 4; ++l)
          wd |= (static_cast<uint32_t>(requantize(wide[l], sh[l], ep.rounding, ep.lo, ep.hi)) & 0xFFu)
                << (8 * l);
        *reinterpret_cast<uint32_t*>(static_cast<int8_t*>(y) + o) = wd;
      } else if (ep.out_mode == 1) {
#pragma unroll
        for (int l = 0; l < 4; ++l) static_cast<int32_t*>(y)[o + l] = wide[l];
      } else {
#pragma unroll
        for (int l = 0; l < 4; ++l) static_cast<float*>(y)[o + l] = dequantize(wide[l], ae[l]);
      }
    }
  }
}

// ---------------------------------------------------------------------------------------
// Depthwise 3x3, tap-packed form.  The sum of Eq. 6 runs over taps only, so the three horizontal
// taps of one channel are brought into ONE 32-bit word (bytes x[q], x[q+1], x[q+2], and a fourth
// that meets a zero weight) and a single dp4a per filter row does them at once: three integer
// instructions per output instead of nine.  The words arrive channel-packed (NHWC: four channels
// of one pixel); a 4x4 byte transpose by prmt turns four pixels into four per-channel words, and
// the windows at odd offsets are further prmt picks.  Accumulators start at bias + the bit
// pattern of 1.5 * 2^23, so that reinterpreted as a float they hold 1.5 * 2^23 + v exactly
// (|v| < 2^22, checked at create) and the requantization is one fused multiply-add whose low
// mantissa byte is the code (nearest-even; see emit()).  One thread owns 4 channels x 4 output columns and
// walks down the rows, each input row feeding the output rows in flight.
// ---------------------------------------------------------------------------------------
struct DwTapParams {
  const uint32_t* w_rows;      // [3][C]: w[r][0][c] | w[r][1][c] << 8 | w[r][2][c] << 16
  const int32_t* bias_magic;   // [C]: bias + 0x4B400000
  const float* scale_f32;      // [C]: 2^-s[c] (0 when s > 22: every |v| < 2^22 then rounds to 0)
  const float* offset_f32;     // [C]: 1.5 * 2^23 * (1 - 2^-s[c]), exact in binary32 for s <= 22
  float lo_f, hi_f;            // 1.5 * 2^23 + lower / upper saturation bound (lower is 0 with ReLU)
};

// four pixels' channel-packed words -> four channel words holding those pixels in byte order
__device__ __forceinline__ void transpose4x4(uint32_t x0, uint32_t x1, uint32_t x2, uint32_t x3, uint32_t (&t)[4]) {
  const uint32_t a = __byte_perm(x0, x1, 0x5140), b = __byte_perm(x2, x3, 0x5140);
  const uint32_t c = __byte_perm(x0, x1, 0x7362), d = __byte_perm(x2, x3, 0x7362);
  t[0] = __byte_perm(a, b, 0x5410);
  t[1] = __byte_perm(a, b, 0x7632);
  t[2] = __byte_perm(c, d, 0x5410);
  t[3] = __byte_perm(c, d, 0x7632);
}

// f(integral_constant<J>) for J = First .. Last-1, stopping at the first false.
template <int First, int Last, class F>
__device__ __forceinline__ void static_for(F&& f) {
  if constexpr (First < Last) {
    if (f(std::integral_constant<int, First>{})) static_for<First + 1, Last>(f);
  }
}

// The arithmetic of one thread (4 channels x 4 output columns, rows rolling through NACC slots);
// the two kernels below differ only in how an input row reaches the registers.
template <int STRIDE>
struct DwTapCore {
  static constexpr int TW = 4;
  static constexpr int IW = (TW - 1) * STRIDE + 3;                // 6 or 9 input pixels per row
  static constexpr int NACC = STRIDE == 1 ? 3 : 2;                // output rows in flight
  static constexpr int PERIOD = STRIDE == 1 ? 3 : 4;              // input rows after which the slots repeat
  uint32_t wr[3][4];
  int32_t bias[4];
  float scale[4], offset[4];
  float lo_f, hi_f;
  int32_t acc[NACC][TW][4];
  int8_t* yb;            // output at (n, 0, 0, first channel of this thread)
  int out_pitch, Q, q0, p_start, rows_out;
  size_t y_image_bytes;  // extent of one image of the output, from yb's image base (checked build only)
  int y_first_byte;      // offset of yb inside its image

  __device__ __forceinline__ void load_tables(const DwTapParams& tp, int C, int c4) {
#pragma unroll
    for (int r = 0; r < 3; ++r) {
      const uint4 v = __ldg(reinterpret_cast<const uint4*>(tp.w_rows + static_cast<size_t>(r) * C) + c4);
      wr[r][0] = v.x; wr[r][1] = v.y; wr[r][2] = v.z; wr[r][3] = v.w;
    }
    const int4 bv = __ldg(reinterpret_cast<const int4*>(tp.bias_magic) + c4);
    const float4 sv = __ldg(reinterpret_cast<const float4*>(tp.scale_f32) + c4);
    const float4 ov = __ldg(reinterpret_cast<const float4*>(tp.offset_f32) + c4);
    bias[0] = bv.x; bias[1] = bv.y; bias[2] = bv.z; bias[3] = bv.w;
    scale[0] = sv.x; scale[1] = sv.y; scale[2] = sv.z; scale[3] = sv.w;
    offset[0] = ov.x; offset[1] = ov.y; offset[2] = ov.z; offset[3] = ov.w;
    lo_f = tp.lo_f; hi_f = tp.hi_f;
  }
  // win[ch][tx]: bytes 0..2 = the three pixels output column tx reads, for channel ch
  __device__ __forceinline__ void windows(const uint32_t (&raw)[IW], uint32_t (&win)[4][TW]) const {
    uint32_t lo[4];
    transpose4x4(raw[0], raw[1], raw[2], raw[3], lo);
    if (STRIDE == 1) {
      const uint32_t e = __byte_perm(raw[4], raw[5], 0x5140);     // (x4.c0, x5.c0, x4.c1, x5.c1)
      const uint32_t f = __byte_perm(raw[4], raw[5], 0x7362);     // (x4.c2, x5.c2, x4.c3, x5.c3)
#pragma unroll
      for (int ch = 0; ch < 4; ++ch) {
        const uint32_t hi = (ch < 2) ? e : f;
        win[ch][0] = lo[ch];
        if ((ch & 1) == 0) {
          win[ch][1] = __byte_perm(lo[ch], hi, 0x4321);
          win[ch][2] = __byte_perm(lo[ch], hi, 0x5432);
          win[ch][3] = __byte_perm(lo[ch], hi, 0x5543);
        } else {
          win[ch][1] = __byte_perm(lo[ch], hi, 0x6321);
          win[ch][2] = __byte_perm(lo[ch], hi, 0x7632);
          win[ch][3] = __byte_perm(lo[ch], hi, 0x7763);
        }
      }
    } else {
      uint32_t hi[4];
      transpose4x4(raw[4], raw[5], raw[6], raw[7], hi);
#pragma unroll
      for (int ch = 0; ch < 4; ++ch) {
        win[ch][0] = lo[ch];                                       // pixels 0 1 2 (3)
        win[ch][1] = __byte_perm(lo[ch], hi[ch], 0x5432);          // pixels 2 3 4 (5)
        win[ch][2] = hi[ch];                                       // pixels 4 5 6 (7)
        win[ch][3] = __byte_perm(hi[ch], raw[IW - 1], 0x4032 | ((4 + ch) << 8));   // pixels 6 7 8 (any)
      }
    }
  }
  // First filter row of an output row: the accumulators start from the bias (which carries the float
  // rounding constant), taken as the addend of the row's multiply-adds -- no separate initialisation.
  __device__ __forceinline__ void start_scatter(int32_t (&a)[TW][4], const uint32_t (&win)[4][TW]) const {
#pragma unroll
    for (int tx = 0; tx < TW; ++tx)
#pragma unroll
      for (int l = 0; l < 4; ++l)
        a[tx][l] = __dp4a(static_cast<int>(win[l][tx]), static_cast<int>(wr[0][l]), bias[l]);
  }
  __device__ __forceinline__ void scatter(int32_t (&a)[TW][4], const uint32_t (&win)[4][TW], int r) const {
#pragma unroll
    for (int tx = 0; tx < TW; ++tx)
#pragma unroll
      for (int l = 0; l < 4; ++l)
        a[tx][l] = __dp4a(static_cast<int>(win[l][tx]), static_cast<int>(wr[r][l]), a[tx][l]);
  }
  __device__ __forceinline__ void emit(const int32_t (&a)[TW][4], int o) const {
    int8_t* yr = yb + (static_cast<size_t>(p_start + o) * Q + q0) * out_pitch;
#pragma unroll
    for (int tx = 0; tx < TW; ++tx) {
      if (q0 + tx >= Q) break;
      uint32_t b[4];
#pragma unroll
      for (int l = 0; l < 4; ++l) {
        // The accumulator read as a float is M + v with M = 1.5 * 2^23.  (M + v) * 2^-s is exact, and
        // adding M * (1 - 2^-s) gives M + v / 2^s in one rounding: nearest-even at integer granularity.
        float r = fmaf(__int_as_float(a[tx][l]), scale[l], offset[l]);
        r = fminf(fmaxf(r, lo_f), hi_f);
        b[l] = __float_as_uint(r);                                 // low byte = int8 code
      }
      const uint32_t lo2 = __byte_perm(b[0], b[1], 0x0040);
      const uint32_t hi2 = __byte_perm(b[2], b[3], 0x0040);
      if (QC_IN(y_first_byte + (static_cast<size_t>(p_start + o) * Q + q0 + tx) * out_pitch + 3, y_image_bytes))
        *reinterpret_cast<uint32_t*>(yr + static_cast<size_t>(tx) * out_pitch) = __byte_perm(lo2, hi2, 0x5410);
    }
  }
  // Input row i (relative to the strip's first input row) with J = i % PERIOD known at compile time.
  // It meets filter row r of output row o when i = o * STRIDE + r.
  template <int J>
  __device__ __forceinline__ void feed(int i, const uint32_t (&raw)[IW]) {
    uint32_t win[4][TW];
    windows(raw, win);
    if (STRIDE == 1) {
      if (i < rows_out) start_scatter(acc[J], win);
      if (i >= 1 && i - 1 < rows_out) scatter(acc[(J + 2) % 3], win, 1);
      if (i >= 2) { scatter(acc[(J + 1) % 3], win, 2); emit(acc[(J + 1) % 3], i - 2); }
    } else {
      constexpr int slot = (J >> 1) & 1;                           // slot of output row i / 2
      if ((J & 1) == 0) {
        // even input row: filter row 2 of output i/2 - 1 (which completes), filter row 0 of output i/2
        if (i >= 2) { scatter(acc[slot ^ 1], win, 2); emit(acc[slot ^ 1], i / 2 - 1); }
        if (i / 2 < rows_out) start_scatter(acc[slot], win);
      } else {
        if (i / 2 < rows_out) scatter(acc[slot], win, 1);
      }
    }
  }
  // The same for a row in the middle of a strip, where every part runs (stride 1: 2 <= i < rows_out; stride 2:
  // 2 <= i < 2 * rows_out): no tests, which is where a strip spends its time.
  template <int J>
  __device__ __forceinline__ void feed_full(int i, const uint32_t (&raw)[IW]) {
    uint32_t win[4][TW];
    windows(raw, win);
    if (STRIDE == 1) {
      start_scatter(acc[J], win);
      scatter(acc[(J + 2) % 3], win, 1);
      scatter(acc[(J + 1) % 3], win, 2);
      emit(acc[(J + 1) % 3], i - 2);
    } else {
      constexpr int slot = (J >> 1) & 1;
      if ((J & 1) == 0) {
        scatter(acc[slot ^ 1], win, 2);
        emit(acc[slot ^ 1], i / 2 - 1);
        start_scatter(acc[slot], win);
      } else {
        scatter(acc[slot], win, 1);
      }
    }
  }
};

// Rows fetched by the thread itself with bounds-checked 32-bit loads, one row ahead (any C % 4 == 0).
template <int STRIDE>
__global__ void __launch_bounds__(256, 2)
depthwise3x3_tap_kernel(const int8_t* __restrict__ x, int8_t* __restrict__ y, ConvGeom g, DwTapParams tp,
                        int rows_per_thread) {
  using Core = DwTapCore<STRIDE>;
  constexpr int TW = Core::TW, IW = Core::IW;
  const int cw = g.C >> 2;
  const int qt = (g.Q + TW - 1) / TW;
  const int item = blockIdx.x * 256 + threadIdx.x;
  if (item >= qt * cw) return;
  const int c4 = item % cw;
  const int n = blockIdx.z;
  Core core;
  core.load_tables(tp, g.C, c4);
  core.q0 = (item / cw) * TW;
  core.p_start = blockIdx.y * rows_per_thread;
  core.rows_out = min(rows_per_thread, g.P - core.p_start);
  core.Q = g.Q;
  core.out_pitch = g.out_c_pitch;
  core.yb = y + static_cast<size_t>(n) * g.P * g.Q * g.out_c_pitch + g.out_c_offset + (c4 << 2);
  core.y_image_bytes = static_cast<size_t>(g.P) * g.Q * g.out_c_pitch;
  core.y_first_byte = g.out_c_offset + (c4 << 2);
  const uint32_t* x32 = reinterpret_cast<const uint32_t*>(x) + static_cast<size_t>(n) * g.H * g.W * cw + c4;
  const int h_start = core.p_start * STRIDE - g.pad_h;
  const int w0 = core.q0 * STRIDE - g.pad_w;
  const int rows_in = (core.rows_out - 1) * STRIDE + 3;

  auto load_row = [&](int i, uint32_t (&raw)[IW]) {
    const int h = h_start + i;
    const bool row_in = i < rows_in && h >= 0 && h < g.H;
    const uint32_t* rp = x32 + static_cast<size_t>(h) * g.W * cw;
#pragma unroll
    for (int ix = 0; ix < IW; ++ix) {
      const int wc = w0 + ix;
      raw[ix] = (row_in && wc >= 0 && wc < g.W &&
                 QC_IN((static_cast<size_t>(h) * g.W + wc) * cw + c4, static_cast<size_t>(g.H) * g.W * cw))
                    ? __ldg(rp + wc * cw) : 0u;
    }
  };
  uint32_t raw[IW], nxt[IW];
  load_row(0, raw);
  for (int i0 = 0; i0 < rows_in; i0 += Core::PERIOD) {
    static_for<0, Core::PERIOD>([&](auto jc) {
      constexpr int j = decltype(jc)::value;
      const int i = i0 + j;
      if (i >= rows_in) return false;
      load_row(i + 1, nxt);
      core.template feed<j>(i, raw);
#pragma unroll
      for (int ix = 0; ix < IW; ++ix) raw[ix] = nxt[ix];
      return true;
    });
  }
}

// ---------------------------------------------------------------------------------------
// Eltwise addition with per-input power-of-two scales (Eq. 10): sum at the finest scale in int32,
// optional ReLU, round-shift, saturate.  16 bytes per thread and input.
// ---------------------------------------------------------------------------------------
struct EltwiseArgs {
  const int8_t* in[8];
  int lshift[8];
  int n_inputs, rshift, relu, rounding, lo, hi;
};

__global__ void __launch_bounds__(256)
eltwise_add_i8_kernel(EltwiseArgs a, int8_t* __restrict__ y, size_t count, int vec_ok) {
  const size_t tid = blockIdx.x * static_cast<size_t>(blockDim.x) + threadIdx.x;
  const size_t nthreads = static_cast<size_t>(gridDim.x) * blockDim.x;
  const size_t nvec = vec_ok ? count / 16 : 0;
  for (size_t i = tid; i < nvec; i += nthreads) {
    if (!QC_IN(16 * i + 15, count)) continue;
    int32_t wide[16];
#pragma unroll
    for (int j = 0; j < 16; ++j) wide[j] = 0;
    for (int t = 0; t < a.n_inputs; ++t) {
      const uint4 v = __ldg(reinterpret_cast<const uint4*>(a.in[t]) + i);
      const uint32_t w4[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
      for (int j = 0; j < 16; ++j) {
        const int32_t b = static_cast<int32_t>(static_cast<int8_t>((w4[j >> 2] >> (8 * (j & 3))) & 0xFFu));
        wide[j] += static_cast<int32_t>(static_cast<uint32_t>(b) << a.lshift[t]);
      }
    }
    uint32_t o4[4] = {0u, 0u, 0u, 0u};
#pragma unroll
    for (int j = 0; j < 16; ++j) {
      int32_t w = a.relu ? max(wide[j], 0) : wide[j];
      const int32_t q = requantize(w, a.rshift, a.rounding, a.lo, a.hi);
      o4[j >> 2] |= (static_cast<uint32_t>(q) & 0xFFu) << (8 * (j & 3));
    }
    reinterpret_cast<uint4*>(y)[i] = make_uint4(o4[0], o4[1], o4[2], o4[3]);
  }
  for (size_t i = nvec * 16 + tid; i < count; i += nthreads) {
    int32_t w = 0;
    for (int t = 0; t < a.n_inputs; ++t)
      w += static_cast<int32_t>(static_cast<uint32_t>(static_cast<int32_t>(a.in[t][i])) << a.lshift[t]);
    if (a.relu) w = max(w, 0);
    y[i] = static_cast<int8_t>(requantize(w, a.rshift, a.rounding, a.lo, a.hi));
  }
}

}  // namespace qc

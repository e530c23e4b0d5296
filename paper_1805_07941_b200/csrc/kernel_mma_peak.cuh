// Issue-rate microbenchmark of the int8 tensor-core instruction the convolution kernel uses
// (tcgen05.mma kind::i8, M = 128, N = bn, K = 32 per instruction): one CTA per SM keeps one A tile
// and one B tile resident in shared memory and issues a long train of MMAs on them, so nothing but
// the tensor pipe is exercised -- no loads, no epilogue.  Its result is the denominator against
// which the tensor-bound layers' throughput is read (MACs per clock per SM times the SM clock), next
// to the library-GEMM figure.  Not part of the method; it measures the machine.
#pragma once
#include <cuda_runtime.h>
#include <cstdint>
#include "kernel_igemm.cuh"

namespace qc {

constexpr int kPeakThreads = 128;

struct MmaPeakShared {
  uint64_t done;
  uint32_t tmem_base;
};

__global__ void __launch_bounds__(kPeakThreads, 1)
mma_peak_kernel(int bn, int mmas, unsigned long long* __restrict__ cycles, int* __restrict__ status,
                unsigned int wait_limit) {
  extern __shared__ uint8_t peak_smem[];
  uint8_t* tiles = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(peak_smem) + 1023) & ~static_cast<uintptr_t>(1023));
  const uint32_t a_bytes = kTileM * 128u, b_bytes = static_cast<uint32_t>(bn) * 128u;
  MmaPeakShared* sh = reinterpret_cast<MmaPeakShared*>(tiles + a_bytes + b_bytes);
  const int warp = threadIdx.x >> 5;
  // operands: small pseudo-random bytes (any values do; the layout is the 128-byte-swizzled K-major
  // one, and a permutation of random bytes is as good as the bytes)
  uint32_t* words = reinterpret_cast<uint32_t*>(tiles);
  for (uint32_t i = threadIdx.x; i < (a_bytes + b_bytes) / 4; i += kPeakThreads) {
    uint32_t v = (i + 1u) * 2654435761u + blockIdx.x * 40503u;
    v ^= v >> 15;
    words[i] = v & 0x03030303u;
  }
  if (threadIdx.x == 0) {
    ptx::mbar_init(ptx::smem_u32(&sh->done), 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  ptx::fence_async_smem();
  int cols = 32;
  while (cols < bn) cols *= 2;
  if (warp == 0) {
    ptx::tmem_alloc(ptx::smem_u32(&sh->tmem_base), static_cast<uint32_t>(cols));
    ptx::tmem_relinquish();
  }
  ptx::tc_fence_before();
  __syncthreads();
  ptx::tc_fence_after();
  const uint32_t tmem = sh->tmem_base;
  if (threadIdx.x == 0) {
    // instruction descriptor as in the convolution kernel, N = bn
    const uint32_t idesc = make_idesc_i8(bn);
    const uint64_t a_desc = make_kmajor_desc(ptx::smem_u32(tiles), 128);
    const uint64_t b_desc = make_kmajor_desc(ptx::smem_u32(tiles) + a_bytes, 128);
    const long long t0 = clock64();
    for (int i = 0; i < mmas; i += 4) {
      ptx::mma_i8(tmem, a_desc, b_desc, idesc, i ? 1u : 0u);
      ptx::mma_i8(tmem, a_desc + 2u, b_desc + 2u, idesc, 1u);
      ptx::mma_i8(tmem, a_desc + 4u, b_desc + 4u, idesc, 1u);
      ptx::mma_i8(tmem, a_desc + 6u, b_desc + 6u, idesc, 1u);
    }
    ptx::mma_commit(ptx::smem_u32(&sh->done));
    bool ok = false;
    for (unsigned int it = 0; it < wait_limit && !ok; ++it) ok = ptx::mbar_try_wait(ptx::smem_u32(&sh->done), 0u) != 0;
    const long long t1 = clock64();
    cycles[blockIdx.x] = static_cast<unsigned long long>(t1 - t0);
    if (!ok) atomicExch(status, kStatusTimeout);
  }
  ptx::tc_fence_before();
  __syncthreads();
  if (warp == 0) {
    ptx::tc_fence_after();
    ptx::tmem_dealloc(tmem, static_cast<uint32_t>(cols));
  }
}

}  // namespace qc

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
  uint64_t stage_free;       // stands for a ring slot's barrier: arrivals pile up, nobody waits on it
  uint32_t tmem_base;
};

__global__ void __launch_bounds__(kPeakThreads, 1)
mma_peak_kernel(int bn, int mmas, int row_bytes, int commit_every, unsigned long long* __restrict__ cycles, int* __restrict__ status,
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
    ptx::mbar_init(ptx::smem_u32(&sh->stage_free), 1);
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
    // operand rows of row_bytes (128, 64 or 32: the swizzle span of the layout); an instruction consumes
    // 32 bytes of every row, so the K slices inside one row group are 2 descriptor units apart and the
    // next group of slices starts one tile (128 rows of row_bytes) further on -- here the same tile again
    const uint64_t a_desc = make_kmajor_desc(ptx::smem_u32(tiles), row_bytes);
    const uint64_t b_desc = make_kmajor_desc(ptx::smem_u32(tiles) + a_bytes, row_bytes);
    const uint64_t k1 = row_bytes >= 64 ? 2u : 0u, k2 = row_bytes >= 128 ? 4u : 0u, k3 = row_bytes >= 128 ? 6u : k1;
    const long long t0 = clock64();
    for (int i = 0; i < mmas; i += 4) {
      ptx::mma_i8(tmem, a_desc, b_desc, idesc, i ? 1u : 0u);
      ptx::mma_i8(tmem, a_desc + k1, b_desc + k1, idesc, 1u);
      ptx::mma_i8(tmem, a_desc + k2, b_desc + k2, idesc, 1u);
      ptx::mma_i8(tmem, a_desc + k3, b_desc + k3, idesc, 1u);
      // as in a pipelined kernel: a commit after every commit_every instructions (a stage handed back)
      if (commit_every && (i + 4) % commit_every == 0) ptx::mma_commit(ptx::smem_u32(&sh->stage_free));
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

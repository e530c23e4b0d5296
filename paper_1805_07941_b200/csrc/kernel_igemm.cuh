// Implicit-GEMM int8 convolution on the sm_100a tensor cores (Eq. 6 as a dense
// contraction): tcgen05.mma kind::i8 with int32 accumulators in tensor memory, operands
// staged in shared memory by TMA (NHWC activation boxes and K-major packed weights, both in
// the swizzled K-major canonical layout), and the requantization epilogue in registers.
//
// One CTA computes a tile of up to 128 output pixels x BN output channels.  The pixels of
// a tile are a box tq x tp x tn of the output (columns x rows x images), so that for filter
// tap (r, s) the activation operand is ONE TMA box of the input, shifted by the tap offset;
// taps that fall outside the image are zero-filled by the TMA unit, which is exact because
// the scheme is symmetric (zero is the integer 0).
//
// Warp roles (192 threads): warp 0 issues TMA loads, warp 1 owns tensor memory and issues
// the MMAs, warps 2-5 run the epilogue (each reads the TMEM lane quadrant warp_id % 4).
// All waits on mbarriers are bounded; on expiry the CTA raises a status flag and leaves.
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>
#include <cstdint>
#include "epilogue.cuh"

namespace qc {

constexpr int kIgemmThreads = 192;
constexpr int kMaxStages = 8;
constexpr int kTileM = 128;

struct IgemmParams {
  int tq, tp, tn;                  // tile box, in output pixels (tq * tp * tn <= 128)
  int tiles_q, tiles_p, tiles_n;   // number of boxes along each output axis
  int tiles_k;                     // number of output-channel tiles
  int BN;                          // channels per tile = MMA N (multiple of 16, <= 256)
  int BKC;                         // bytes of the contraction axis per pipeline stage (32/64/128)
  int nchunks;                     // channel chunks per filter tap
  int R, S;                        // taps seen by the kernel (1 x 1 for flattened / packed inputs)
  int pad_h, pad_w, stride_h, stride_w;
  int stages;
  int Q, P, Nimg;                  // output extent in the kernel's pixel space
  int K;                           // real output channels
  int out_c_offset, out_c_pitch;
  int tmem_cols;                   // power of two >= max(32, BN)
  int vec_store;                   // 1: 16-byte stores/loads of int8 rows are aligned
  uint32_t a_stage_bytes, b_stage_bytes;   // shared-memory footprint per stage (1024-aligned)
  uint32_t tx_bytes;               // bytes both TMA boxes deliver per stage
};

// Error codes written to the status word.
constexpr int kStatusTimeout = -8;

namespace ptx {

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes)
               : "memory");
}
__device__ __forceinline__ uint32_t mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok;
}
__device__ __forceinline__ void tma_load_4d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0,
                                            int c1, int c2, int c3) {
  asm volatile(
      "cp.async.bulk.tensor.4d.shared::cluster.global.tile.mbarrier::complete_tx::bytes "
      "[%0], [%1, {%3, %4, %5, %6}], [%2];"
      ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(bar), "r"(c0), "r"(c1), "r"(c2), "r"(c3)
      : "memory");
}
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0,
                                            int c1) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes "
      "[%0], [%1, {%3, %4}], [%2];"
      ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(bar), "r"(c0), "r"(c1)
      : "memory");
}
__device__ __forceinline__ void prefetch_tmap(const CUtensorMap* map) {
  asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(map)) : "memory");
}
__device__ __forceinline__ void tmem_alloc(uint32_t dst_smem, uint32_t ncols) {
  asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(dst_smem),
               "r"(ncols)
               : "memory");
}
__device__ __forceinline__ void tmem_relinquish() {
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols) {
  asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols)
               : "memory");
}
__device__ __forceinline__ void tc_fence_before() {
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
}
__device__ __forceinline__ void tc_fence_after() {
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
}
// D[tmem] (+)= A[smem] * B[smem], int8 x int8 -> int32, issued by one thread.
__device__ __forceinline__ void mma_i8(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                       uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::i8 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
      : "memory");
}
// mbarrier arrives once every MMA issued so far by this thread has finished.
__device__ __forceinline__ void mma_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar)
               : "memory");
}
// 32 lanes x 32 consecutive 32-bit columns: thread i of the warp receives lane (row) i.
__device__ __forceinline__ void tmem_ld_32x32(uint32_t taddr, uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]),
        "=r"(r[15]), "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]),
        "=r"(r[22]), "=r"(r[23]), "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]),
        "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr)
      : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() {
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}

}  // namespace ptx

// Shared-memory matrix descriptor of a K-major operand tile in the swizzled canonical
// layout: rows of `row_bytes` (= the swizzle span: 32, 64 or 128), groups of 8 rows
// contiguous, groups 8 * row_bytes apart.
__device__ __forceinline__ uint64_t make_kmajor_desc(uint32_t smem_addr, int row_bytes) {
  const uint64_t layout = row_bytes == 128 ? 2ull : (row_bytes == 64 ? 4ull : 6ull);
  uint64_t d = 0;
  d |= static_cast<uint64_t>((smem_addr >> 4) & 0x3FFFu);            // start address / 16
  d |= 1ull << 16;                                                   // leading offset (unused here)
  d |= static_cast<uint64_t>((8u * row_bytes) >> 4) << 32;           // stride between 8-row groups / 16
  d |= 1ull << 46;                                                   // descriptor version for sm_100
  d |= layout << 61;
  return d;
}

// Instruction descriptor: int8 x int8 -> int32, both operands K-major, M = 128, N = bn.
__device__ __forceinline__ uint32_t make_idesc_i8(int bn) {
  uint32_t d = 0;
  d |= 2u << 4;                                  // accumulator format: signed 32-bit
  d |= 1u << 7;                                  // A: signed 8-bit
  d |= 1u << 10;                                 // B: signed 8-bit
  d |= static_cast<uint32_t>(bn >> 3) << 17;     // N / 8
  d |= static_cast<uint32_t>(kTileM >> 4) << 24; // M / 16
  return d;
}

struct IgemmShared {
  uint64_t full[kMaxStages];
  uint64_t empty[kMaxStages];
  uint64_t accum_full;
  uint32_t tmem_base;
  volatile int abort_flag;
  int32_t bias[256];
  int32_t shift[256];
  int32_t lshift[256];
  int32_t acc_exp[256];
};

// Bounded wait.  Returns false (and raises the CTA abort flag and the global status) if the
// barrier did not flip within `limit` polls, or if another role already gave up.
__device__ __forceinline__ bool wait_bounded(uint32_t bar, uint32_t parity, unsigned int limit,
                                             IgemmShared* sh, int* status) {
  for (unsigned int it = 0; it < limit; ++it) {
    if (ptx::mbar_try_wait(bar, parity)) return true;
    if (sh->abort_flag) return false;
  }
  sh->abort_flag = 1;
  atomicExch(status, kStatusTimeout);
  return false;
}

__global__ void __launch_bounds__(kIgemmThreads)
igemm_i8_kernel(const __grid_constant__ CUtensorMap tmap_a, const __grid_constant__ CUtensorMap tmap_b,
                const IgemmParams prm, const EpilogueParams ep, const int8_t* __restrict__ res,
                void* __restrict__ y, int* status, unsigned int wait_limit) {
  extern __shared__ uint8_t smem_raw[];
  // operand stages need 1024-byte alignment (swizzle atom); the launch reserves the slack
  uint8_t* tiles = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) &
                                              ~static_cast<uintptr_t>(1023));
  const uint32_t stage_bytes = prm.a_stage_bytes + prm.b_stage_bytes;
  IgemmShared* sh = reinterpret_cast<IgemmShared*>(tiles + static_cast<size_t>(prm.stages) * stage_bytes);

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;

  // tile coordinates
  const int bid = blockIdx.x;
  const int kt = bid % prm.tiles_k;
  const int mt = bid / prm.tiles_k;
  const int qt = mt % prm.tiles_q;
  const int pt = (mt / prm.tiles_q) % prm.tiles_p;
  const int it_n = mt / (prm.tiles_q * prm.tiles_p);
  const int q0 = qt * prm.tq, p0 = pt * prm.tp, n0 = it_n * prm.tn;
  const int k0 = kt * prm.BN;
  const int num_kb = prm.R * prm.S * prm.nchunks;

  if (threadIdx.x == 0) {
    for (int s = 0; s < prm.stages; ++s) {
      ptx::mbar_init(ptx::smem_u32(&sh->full[s]), 1);
      ptx::mbar_init(ptx::smem_u32(&sh->empty[s]), 1);
    }
    ptx::mbar_init(ptx::smem_u32(&sh->accum_full), 1);
    sh->abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 0 && lane == 0) {
    ptx::prefetch_tmap(&tmap_a);
    ptx::prefetch_tmap(&tmap_b);
  }
  if (warp == 1) {
    ptx::tmem_alloc(ptx::smem_u32(&sh->tmem_base), static_cast<uint32_t>(prm.tmem_cols));
    ptx::tmem_relinquish();
  }
  // per-channel epilogue constants of this tile
  for (int i = threadIdx.x; i < prm.BN; i += blockDim.x) {
    int k = k0 + i;
    bool ok = k < prm.K;
    sh->bias[i] = (ok && ep.bias) ? ep.bias[k] : 0;
    sh->shift[i] = ok ? ep.shift[k] : 0;
    sh->lshift[i] = (ok && ep.res_lshift) ? ep.res_lshift[k] : 0;
    sh->acc_exp[i] = ok ? ep.acc_exp[k] : 0;
  }
  ptx::tc_fence_before();
  __syncthreads();
  ptx::tc_fence_after();
  const uint32_t tmem_base = sh->tmem_base;

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      int issued = 0;
      bool ok = true;
      for (int kb = 0; kb < num_kb && ok; ++kb) {
        const int s = kb % prm.stages;
        const uint32_t round = static_cast<uint32_t>(kb / prm.stages);
        ok = wait_bounded(ptx::smem_u32(&sh->empty[s]), (round & 1u) ^ 1u, wait_limit, sh, status);
        if (!ok) break;
        const int tap = kb / prm.nchunks;
        const int ci = kb - tap * prm.nchunks;
        const int r = tap / prm.S;
        const int sx = tap - r * prm.S;
        const uint32_t full = ptx::smem_u32(&sh->full[s]);
        const uint32_t a_dst = ptx::smem_u32(tiles + static_cast<size_t>(s) * stage_bytes);
        const uint32_t b_dst = a_dst + prm.a_stage_bytes;
        ptx::mbar_expect_tx(full, prm.tx_bytes);
        ptx::tma_load_4d(a_dst, &tmap_a, full, ci * prm.BKC, q0 * prm.stride_w - prm.pad_w + sx,
                         p0 * prm.stride_h - prm.pad_h + r, n0);
        ptx::tma_load_2d(b_dst, &tmap_b, full, kb * prm.BKC, k0);
        issued = kb + 1;
      }
      if (!ok) {
        // let copies that were already issued land before the CTA leaves
        int first = issued > prm.stages ? issued - prm.stages : 0;
        for (int kb = first; kb < issued; ++kb) {
          const uint32_t bar = ptx::smem_u32(&sh->full[kb % prm.stages]);
          const uint32_t par = static_cast<uint32_t>(kb / prm.stages) & 1u;
          for (unsigned int it = 0; it < wait_limit; ++it)
            if (ptx::mbar_try_wait(bar, par)) break;
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      const uint32_t idesc = make_idesc_i8(prm.BN);
      const int mma_per_stage = prm.BKC / 32;
      bool ok = true;
      for (int kb = 0; kb < num_kb && ok; ++kb) {
        const int s = kb % prm.stages;
        const uint32_t round = static_cast<uint32_t>(kb / prm.stages);
        ok = wait_bounded(ptx::smem_u32(&sh->full[s]), round & 1u, wait_limit, sh, status);
        if (!ok) break;
        ptx::tc_fence_after();
        const uint32_t a_addr = ptx::smem_u32(tiles + static_cast<size_t>(s) * stage_bytes);
        const uint64_t a_desc = make_kmajor_desc(a_addr, prm.BKC);
        const uint64_t b_desc = make_kmajor_desc(a_addr + prm.a_stage_bytes, prm.BKC);
        for (int j = 0; j < mma_per_stage; ++j) {
          // advance 32 bytes along K inside the swizzle span: +2 in units of 16 bytes
          ptx::mma_i8(tmem_base, a_desc + 2u * j, b_desc + 2u * j, idesc, (kb | j) != 0 ? 1u : 0u);
        }
        ptx::mma_commit(ptx::smem_u32(&sh->empty[s]));      // stage free once these MMAs retire
      }
      if (ok) ptx::mma_commit(ptx::smem_u32(&sh->accum_full));
    }
  } else {
    // ------------------------------------------------------------------ epilogue
    const int quad = warp & 3;                               // TMEM lane quadrant of this warp
    const int row = quad * 32 + lane;                        // tile row = accumulator lane
    const int q_i = row % prm.tq;
    const int p_i = (row / prm.tq) % prm.tp;
    const int n_i = row / (prm.tq * prm.tp);
    const int q = q0 + q_i, p = p0 + p_i, n = n0 + n_i;
    const bool row_ok = (n_i < prm.tn) && q < prm.Q && p < prm.P && n < prm.Nimg;
    const size_t pix = (static_cast<size_t>(n) * prm.P + p) * prm.Q + q;
    bool ok = wait_bounded(ptx::smem_u32(&sh->accum_full), 0u, wait_limit, sh, status);
    ok = __all_sync(0xffffffffu, ok);
    if (ok) {
      ptx::tc_fence_after();
      const int nchunk32 = (prm.BN + 31) / 32;
      for (int ch = 0; ch < nchunk32; ++ch) {
        uint32_t acc[32];
        ptx::tmem_ld_32x32(tmem_base + (static_cast<uint32_t>(quad * 32) << 16) + ch * 32, acc);
        ptx::tmem_ld_wait();
        if (!row_ok) continue;
#pragma unroll
        for (int half = 0; half < 2; ++half) {
          const int col = ch * 32 + half * 16;               // column inside the tile
          const int k = k0 + col;
          if (col >= prm.BN || k >= prm.K) continue;
          const bool full16 = (k + 16 <= prm.K);
          // residual values of these 16 channels
          int32_t rv[16];
          if (res) {
            const int8_t* rp = res + pix * prm.K + k;
            if (full16 && prm.vec_store) {
              uint4 v = __ldg(reinterpret_cast<const uint4*>(rp));
              uint32_t wds[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
              for (int j = 0; j < 16; ++j)
                rv[j] = static_cast<int32_t>(static_cast<int8_t>((wds[j >> 2] >> (8 * (j & 3))) & 0xFFu));
            } else {
#pragma unroll
              for (int j = 0; j < 16; ++j) rv[j] = (k + j < prm.K) ? static_cast<int32_t>(rp[j]) : 0;
            }
          } else {
#pragma unroll
            for (int j = 0; j < 16; ++j) rv[j] = 0;
          }
          int32_t wide[16];
#pragma unroll
          for (int j = 0; j < 16; ++j)
            wide[j] = wide_value(static_cast<int32_t>(acc[half * 16 + j]), sh->bias[col + j], rv[j],
                                 sh->lshift[col + j], ep.relu);
          const size_t o = pix * prm.out_c_pitch + prm.out_c_offset + k;
          if (ep.out_mode == 0) {
            int8_t* yp = static_cast<int8_t*>(y) + o;
            uint32_t wds[4] = {0, 0, 0, 0};
#pragma unroll
            for (int j = 0; j < 16; ++j) {
              int32_t v = requantize(wide[j], sh->shift[col + j], ep.rounding, ep.lo, ep.hi);
              wds[j >> 2] |= (static_cast<uint32_t>(v) & 0xFFu) << (8 * (j & 3));
            }
            if (full16 && prm.vec_store) {
              *reinterpret_cast<uint4*>(yp) = make_uint4(wds[0], wds[1], wds[2], wds[3]);
            } else {
#pragma unroll
              for (int j = 0; j < 16; ++j)
                if (k + j < prm.K) yp[j] = static_cast<int8_t>((wds[j >> 2] >> (8 * (j & 3))) & 0xFFu);
            }
          } else if (ep.out_mode == 1) {
            int32_t* yp = static_cast<int32_t*>(y) + o;
#pragma unroll
            for (int j = 0; j < 16; ++j)
              if (k + j < prm.K) yp[j] = wide[j];
          } else {
            float* yp = static_cast<float*>(y) + o;
#pragma unroll
            for (int j = 0; j < 16; ++j)
              if (k + j < prm.K) yp[j] = dequantize(wide[j], sh->acc_exp[col + j]);
          }
        }
      }
    }
  }
  ptx::tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    ptx::tc_fence_after();
    ptx::tmem_dealloc(tmem_base, static_cast<uint32_t>(prm.tmem_cols));
  }
}

}  // namespace qc

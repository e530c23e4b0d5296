// Implicit-GEMM int8 convolution (Eq. 6) on PAIRS of SMs: a cluster of two CTAs computes one tile of
// 256 output pixels x up to 256 channels with tcgen05.mma.cta_group::2.  Each CTA loads ITS OWN half of
// both operands into its own shared memory with ordinary TMA loads -- 128 pixels of the activation box
// and half of the tile's weight rows -- and holds the accumulator rows of its own 128 pixels in its own
// tensor memory; one thread of the first CTA issues the MMAs for both.  Per multiply-add a CTA fetches half
// the operand bytes of a 128 x 128 tile (32 KB per 128 x 256 x 128 block), which is what the tensor-bound
// layers need: they run at the rate the operands arrive from L2, not at the tensor pipe's.
//
// Roles per CTA (320 threads, as in kernel_igemm.cuh): warp 0 lane 0 issues the loads, warp 1 owns tensor
// memory (lane 0 of the first CTA issues the MMAs), warps 2-9 run the epilogue on the CTA's own rows.
// Barriers: a stage's "full" barrier lives in the first CTA and counts the bytes of both CTAs' loads (the
// second CTA's copies signal it across the cluster); "empty" and "accumulator full" are signalled in both
// CTAs at once by the MMA thread's multicast commits; "accumulator empty" lives in the first CTA and is
// arrived on by the epilogue warps of both.  All waits are bounded; the two CTAs meet at a cluster barrier
// before any remote signal and before they retire.
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>
#include <cstdint>
#include "kernel_igemm.cuh"

namespace qc {

struct PairParams {
  int tq, tp, tn;                  // pixel box of ONE CTA (tq * tp * tn <= 128); a tile is two consecutive boxes
  int tiles_q, tiles_p, tiles_n;   // boxes along each output axis
  int pairs_m;                     // ceil(boxes / 2)
  int tiles_k;                     // channel tiles
  int BN;                          // channels per tile (multiple of 32, <= 256); each CTA loads BN / 2 weight rows
  int BKC, nchunks, R, S;
  int pad_h, pad_w, stride_h, stride_w;
  int stages;
  int Q, P, Nimg, K;
  int out_c_offset, out_c_pitch;
  int tmem_cols;                   // power of two >= BN; two buffers are allocated
  uint32_t a_stage_bytes, b_stage_bytes;
  uint32_t tx_bytes;               // bytes BOTH CTAs' loads of one stage deliver
};

namespace ptx {
__device__ __forceinline__ uint32_t cluster_ctarank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
  asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// Address of the same shared-memory location in CTA `rank` of the cluster.
__device__ __forceinline__ uint32_t map_to_cta(uint32_t addr, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank));
  return r;
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_addr) {
  asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
// Loads of a CTA pair: destination in the executing CTA, completion bytes on a barrier given by its
// cluster-wide address (the first CTA's).
__device__ __forceinline__ void tma_load_4d_pair(uint32_t dst, const CUtensorMap* map, uint32_t bar_cluster, int c0,
                                                 int c1, int c2, int c3) {
  asm volatile(
      "cp.async.bulk.tensor.4d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes "
      "[%0], [%1, {%3, %4, %5, %6}], [%2];"
      ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(bar_cluster), "r"(c0), "r"(c1), "r"(c2), "r"(c3)
      : "memory");
}
__device__ __forceinline__ void tma_load_2d_pair(uint32_t dst, const CUtensorMap* map, uint32_t bar_cluster, int c0,
                                                 int c1) {
  asm volatile(
      "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes "
      "[%0], [%1, {%3, %4}], [%2];"
      ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(bar_cluster), "r"(c0), "r"(c1)
      : "memory");
}
__device__ __forceinline__ void tmem_alloc_pair(uint32_t dst_smem, uint32_t ncols) {
  asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(dst_smem), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tmem_relinquish_pair() {
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc_pair(uint32_t taddr, uint32_t ncols) {
  asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
// D (256 rows, split over the two CTAs' tensor memories) (+)= A (each CTA's 128 rows) * B (each CTA's half of N).
__device__ __forceinline__ void mma_i8_pair(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                            uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::2.kind::i8 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
      : "memory");
}
// Arrives on the barrier at this shared-memory offset in BOTH CTAs once every MMA issued so far has finished.
__device__ __forceinline__ void mma_commit_pair(uint32_t bar) {
  asm volatile(
      "tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
      ::"r"(bar), "h"(static_cast<uint16_t>(3))
      : "memory");
}
}  // namespace ptx

// Instruction descriptor: int8 x int8 -> int32, K-major operands, M = 256 over the pair, N = bn.
__device__ __forceinline__ uint32_t make_idesc_i8_pair(int bn) {
  uint32_t d = 0;
  d |= 2u << 4;
  d |= 1u << 7;
  d |= 1u << 10;
  d |= static_cast<uint32_t>(bn >> 3) << 17;
  d |= static_cast<uint32_t>(256 >> 4) << 24;
  return d;
}

struct PairTile {
  int q0, p0, n0, k0;
  bool valid;                      // false: the odd box out of the last pair (loads zero-fill, nothing is stored)
};

// Pair tile u -> this CTA's box.  Channel tile slowest, so pairs running side by side share their weights in L2.
__device__ __forceinline__ PairTile pair_tile(const PairParams& prm, int u, int rank) {
  const int kt = u / prm.pairs_m;
  const int m = 2 * (u - kt * prm.pairs_m) + rank;
  const int qt = m % prm.tiles_q;
  const int rest = m / prm.tiles_q;
  const int pt = rest % prm.tiles_p, nt = rest / prm.tiles_p;
  PairTile t;
  t.q0 = qt * prm.tq; t.p0 = pt * prm.tp; t.n0 = nt * prm.tn; t.k0 = kt * prm.BN;
  t.valid = nt < prm.tiles_n;
  return t;
}

template <int EPI, int RELU, int POOL = 0>
__global__ void __launch_bounds__(kIgemmThreads, 1)
igemm_i8_pair_kernel(const __grid_constant__ CUtensorMap tmap_a, const __grid_constant__ CUtensorMap tmap_b,
                     const PairParams prm, const IgemmParams eprm, const EpilogueParams ep,
                     const int4* __restrict__ chan_table, void* __restrict__ y, int* status, unsigned int wait_limit) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* tiles = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~static_cast<uintptr_t>(1023));
  const uint32_t stage_bytes = prm.a_stage_bytes + prm.b_stage_bytes;
  IgemmShared* sh = reinterpret_cast<IgemmShared*>(tiles + static_cast<uint32_t>(prm.stages) * stage_bytes);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = ptx::cluster_ctarank();
  const int num_kb = prm.R * prm.S * prm.nchunks;
  const int total = prm.pairs_m * prm.tiles_k;
  const int pair_id = blockIdx.x >> 1, num_pairs = gridDim.x >> 1;

  if (threadIdx.x == 0) {
    for (int s = 0; s < prm.stages; ++s) {
      ptx::mbar_init(ptx::smem_u32(&sh->full[s]), 1);       // the first CTA's arrive.expect_tx; bytes from both
      ptx::mbar_init(ptx::smem_u32(&sh->empty[s]), 1);      // one multicast commit
    }
    for (int b = 0; b < 2; ++b) {
      ptx::mbar_init(ptx::smem_u32(&sh->acc_full[b]), 1);
      ptx::mbar_init(ptx::smem_u32(&sh->acc_empty[b]), 2 * kEpilogueWarps);   // epilogue warps of both CTAs
    }
    sh->abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 0 && lane == 0) {
    ptx::prefetch_tmap(&tmap_a);
    ptx::prefetch_tmap(&tmap_b);
  }
  if (warp == 1) {
    ptx::tmem_alloc_pair(ptx::smem_u32(&sh->tmem_base), static_cast<uint32_t>(2 * prm.tmem_cols));
    ptx::tmem_relinquish_pair();
  }
  ptx::tc_fence_before();
  __syncthreads();
  ptx::cluster_sync_all();                                   // the peer's barriers exist from here on
  ptx::tc_fence_after();
  const uint32_t tmem_base = sh->tmem_base;
  ptx::grid_launch_dependents();

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer (own halves only)
    // The whole warp runs the loop with warp-uniform values (addresses and coordinates then live in uniform
    // registers, where the copy instructions take their operands from); lane 0 alone issues.
    {
      const bool leader = lane == 0;
      const uint32_t tiles_addr = ptx::smem_u32(tiles);
      int stage = 0;
      uint32_t phase = 0;
      long long issued = 0;
      bool ok = true;
      for (int u = pair_id; u < total && ok; u += num_pairs) {
        const PairTile tc = pair_tile(prm, u, static_cast<int>(rank));
        const int w_base = tc.q0 * prm.stride_w - prm.pad_w, h_base = tc.p0 * prm.stride_h - prm.pad_h;
        const int k_row = tc.k0 + static_cast<int>(rank) * (prm.BN / 2);
        int r = 0, sx = 0, ci = 0;
        for (int kb = 0; kb < num_kb; ++kb) {
          if (issued >= prm.stages && !ptx::mbar_try_wait_hint(ptx::smem_u32(&sh->empty[stage]), phase ^ 1u)) {
            ok = wait_bounded<32, true>(ptx::smem_u32(&sh->empty[stage]), phase ^ 1u, wait_limit, sh, status);
            if (!ok) break;
          }
          // the byte count of both CTAs' copies is armed on the first CTA's barrier, by the first CTA
          const uint32_t full0 = ptx::map_to_cta(ptx::smem_u32(&sh->full[stage]), 0u);
          const uint32_t a_dst = tiles_addr + static_cast<uint32_t>(stage) * stage_bytes;
          if (leader) {
            if (rank == 0) ptx::mbar_expect_tx(ptx::smem_u32(&sh->full[stage]), prm.tx_bytes);
            ptx::tma_load_2d_pair(a_dst + prm.a_stage_bytes, &tmap_b, full0, kb * prm.BKC, k_row);
            if (issued == 0) ptx::grid_dependency_wait();     // activations: the previous kernel's results
            ptx::tma_load_4d_pair(a_dst, &tmap_a, full0, ci * prm.BKC, w_base + sx, h_base + r, tc.n0);
          }
          ++issued;
          if (++ci == prm.nchunks) { ci = 0; if (++sx == prm.S) { sx = 0; ++r; } }
          if (++stage == prm.stages) { stage = 0; phase ^= 1u; }
        }
      }
      // after a wait that expired, give the copies already on their way time to land in this CTA's shared
      // memory (they take microseconds; their barrier may sit in the other CTA, so it is not polled here)
      __syncwarp();
      if (leader && (!ok || sh->abort_flag))
        for (int i = 0; i < 256; ++i) __nanosleep(200);
      if (leader) ptx::grid_dependency_wait();
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer (first CTA only)
    if (rank == 0 && lane == 0) {
      const uint32_t idesc = make_idesc_i8_pair(prm.BN);
      const int mma_per_stage = prm.BKC / 32;
      const uint32_t tiles_addr = ptx::smem_u32(tiles);
      const uint64_t a_desc0 = make_kmajor_desc(tiles_addr, prm.BKC);
      const uint64_t b_desc0 = make_kmajor_desc(tiles_addr + prm.a_stage_bytes, prm.BKC);
      const uint64_t desc_step = stage_bytes >> 4;
      uint64_t a_desc = a_desc0, b_desc = b_desc0;
      const uint32_t full0 = ptx::smem_u32(&sh->full[0]), empty0 = ptx::smem_u32(&sh->empty[0]);
      int stage = 0, it = 0;
      uint32_t phase = 0;
      bool ok = true;
      for (int u = pair_id; u < total && ok; u += num_pairs, ++it) {
        const int buf = it & 1;
        const uint32_t use = static_cast<uint32_t>(it >> 1);
        ok = wait_bounded<0, true>(ptx::smem_u32(&sh->acc_empty[buf]), (use & 1u) ^ 1u, wait_limit, sh, status);
        if (!ok) break;
        ptx::tc_fence_after();
        const uint32_t d_tmem = tmem_base + static_cast<uint32_t>(buf * prm.tmem_cols);
        uint32_t accumulate = 0;
        for (int kb = 0; kb < num_kb; ++kb) {
          if (!ptx::mbar_try_wait_hint(full0 + 8u * stage, phase)) {
            ok = wait_bounded<0, true>(full0 + 8u * stage, phase, wait_limit, sh, status);
            if (!ok) break;
          }
          ptx::tc_fence_after();
          ptx::mma_i8_pair(d_tmem, a_desc, b_desc, idesc, accumulate);
          if (mma_per_stage > 1) ptx::mma_i8_pair(d_tmem, a_desc + 2u, b_desc + 2u, idesc, 1u);
          if (mma_per_stage > 2) {
            ptx::mma_i8_pair(d_tmem, a_desc + 4u, b_desc + 4u, idesc, 1u);
            ptx::mma_i8_pair(d_tmem, a_desc + 6u, b_desc + 6u, idesc, 1u);
          }
          ptx::mma_commit_pair(empty0 + 8u * stage);           // the stage is free in both CTAs once these retire
          accumulate = 1;
          if (++stage == prm.stages) { stage = 0; phase ^= 1u; a_desc = a_desc0; b_desc = b_desc0; }
          else { a_desc += desc_step; b_desc += desc_step; }
        }
        if (ok) ptx::mma_commit_pair(ptx::smem_u32(&sh->acc_full[buf]));
      }
    }
    __syncwarp();
  } else {
    // ------------------------------------------------------------------ epilogue: this CTA's 128 rows
    const int ew = warp - 2, quad = warp & 3;
    const int row = quad * 32 + lane;
    const int q_i = row % prm.tq, p_i = (row / prm.tq) % prm.tp, n_i = row / (prm.tq * prm.tp);
    const int etid = threadIdx.x - 64;
    const int groups16 = prm.BN / 16, g_split = (groups16 + 1) / 2;
    const int g_begin = (ew < 4) ? 0 : g_split, g_end = (ew < 4) ? g_split : groups16;
    const int kpad = prm.tiles_k * prm.BN;
    const bool cst_all = EpiTraits<EPI>::uni ? kpad <= kBiasAllMax : kpad <= kChanAllMax;
    if (cst_all) {
      for (int i = etid; i < kpad; i += kEpilogueWarps * 32) {
        if (EpiTraits<EPI>::uni) sh->cst.bias[i] = __ldg(&chan_table[i].x);
        else sh->cst.chan[i] = __ldg(chan_table + i);
      }
      asm volatile("bar.sync 1, %0;" ::"n"(kEpilogueWarps * 32) : "memory");
    }
    const uint32_t cst_addr = ptx::smem_u32(&sh->cst);
    const uint32_t acc_empty0 = ptx::map_to_cta(ptx::smem_u32(&sh->acc_empty[0]), 0u);
    const uint4 no_res = make_uint4(0u, 0u, 0u, 0u);
    bool ok = true;
    int it = 0;
    for (int u = pair_id; u < total; u += num_pairs, ++it) {
      const PairTile tc = pair_tile(prm, u, static_cast<int>(rank));
      const int buf = it & 1;
      const uint32_t use = static_cast<uint32_t>(it >> 1);
      if (!cst_all) {
        for (int i = etid; i < prm.BN; i += kEpilogueWarps * 32) {
          if (EpiTraits<EPI>::uni) sh->cst.bias[buf * 256 + i] = __ldg(&chan_table[tc.k0 + i].x);
          else sh->cst.chan[buf * 256 + i] = __ldg(chan_table + tc.k0 + i);
        }
        if (epilogue_vote(!ok)) { ok = false; break; }
      }
      const int q = tc.q0 + q_i, p = tc.p0 + p_i, n = tc.n0 + n_i;
      const bool row_ok = tc.valid && (n_i < prm.tn) && q < prm.Q && p < prm.P && n < prm.Nimg;
      const size_t pix = (static_cast<size_t>(n) * prm.P + p) * prm.Q + q;
      const size_t pooled_pix = POOL ? (static_cast<size_t>(n) * (prm.P >> 1) + (p >> 1)) * (prm.Q >> 1) + (q >> 1) : 0;
      ok = wait_bounded<64, true>(ptx::smem_u32(&sh->acc_full[buf]), use & 1u, wait_limit, sh, status);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) {
        if (cst_all) break;
        continue;
      }
      ptx::tc_fence_after();
      const uint32_t t_addr = tmem_base + (static_cast<uint32_t>(quad * 32) << 16) + static_cast<uint32_t>(buf * prm.tmem_cols);
      const uint32_t chan = cst_addr + static_cast<uint32_t>(cst_all ? tc.k0 : buf * 256) * (EpiTraits<EPI>::uni ? 4u : 16u);
      auto release = [&]() {
        ptx::tc_fence_before();
        __syncwarp();
        if (lane == 0) ptx::mbar_arrive_cluster(acc_empty0 + 8u * static_cast<uint32_t>(buf));
      };
      uint32_t acc_a[16], acc_b[16];
      if (g_begin < g_end) {
        ptx::tmem_ld_32x16(t_addr + g_begin * 16, acc_a);
        ptx::tmem_ld_wait();
      }
#pragma unroll
      for (int i = 0; i < kGroupsPerWarpWide; i += 2) {
        const int g0 = g_begin + i, g1 = g0 + 1, g2 = g0 + 2;
        if (g0 < g_end) {
          if (g1 < g_end) ptx::tmem_ld_32x16(t_addr + g1 * 16, acc_b); else release();
          if constexpr (POOL != 0) {
            if (tc.k0 + g0 * 16 < prm.K)
              epilogue_pool_16<EPI, RELU>(acc_a, chan, g0 * 16, tc.k0 + g0 * 16, pooled_pix, row_ok, lane, eprm.pool_bit, eprm, ep, y);
          } else if (row_ok && tc.k0 + g0 * 16 < prm.K)
            epilogue_16<EPI, RELU, 0>(acc_a, chan, g0 * 16, tc.k0 + g0 * 16, pix, eprm, ep, nullptr, no_res, y, 0u);
          if (g1 < g_end) {
            ptx::tmem_ld_wait();
            if (g2 < g_end && i + 2 < kGroupsPerWarpWide) ptx::tmem_ld_32x16(t_addr + g2 * 16, acc_a); else release();
            if constexpr (POOL != 0) {
              if (tc.k0 + g1 * 16 < prm.K)
                epilogue_pool_16<EPI, RELU>(acc_b, chan, g1 * 16, tc.k0 + g1 * 16, pooled_pix, row_ok, lane, eprm.pool_bit, eprm, ep, y);
            } else if (row_ok && tc.k0 + g1 * 16 < prm.K)
              epilogue_16<EPI, RELU, 0>(acc_b, chan, g1 * 16, tc.k0 + g1 * 16, pix, eprm, ep, nullptr, no_res, y, 0u);
            if (g2 < g_end && i + 2 < kGroupsPerWarpWide) ptx::tmem_ld_wait();
          }
        }
      }
      if (g_begin >= g_end) release();
    }
  }
  // Nothing of this CTA may go away while the peer can still signal its barriers or multiply into its
  // tensor memory: meet the peer, then free the pair's tensor memory.
  ptx::tc_fence_before();
  __syncthreads();
  ptx::cluster_sync_all();
  if (warp == 1) {
    ptx::tc_fence_after();
    ptx::tmem_dealloc_pair(tmem_base, static_cast<uint32_t>(2 * prm.tmem_cols));
  }
}

}  // namespace qc

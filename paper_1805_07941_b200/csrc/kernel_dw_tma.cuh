// Depthwise 3x3 (Eq. 6 with g = C), rows staged by TMA.
//
// Arithmetic: DwTapCore (tap-packed dp4a).  Data movement: a CTA owns a block of CB channels and
// QT x 4 adjacent output columns over a strip of output rows.  A producer warp walks down the
// strip's input rows and copies each one -- `pix` pixels x CB channels, halo included -- into a
// ring of shared-memory stages with one TMA box per row; rows and columns outside the image are
// zero-filled by the copy engine (exact: the symmetric scheme has no zero point), so the 256
// consumer threads need no bounds checks and no address arithmetic: six (stride 2: nine) shared
// loads per row and thread.  A stage is handed back as soon as its words are in registers, so up
// to kDwStages rows are in flight per CTA -- enough bytes outstanding to cover HBM latency, which
// the one-row-ahead register prefetch of the plain kernel could not.
//
// Every wait is bounded: on expiry the CTA raises the status word and everybody leaves; the producer
// always stays until the copies it issued have landed.
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>
#include <cstdint>
#include "kernel_igemm.cuh"      // ptx:: wrappers, kStatusTimeout
#include "kernels_simple.cuh"

namespace qc {

constexpr int kDwStages = 4;
constexpr int kDwConsumers = 256;
constexpr int kDwThreads = kDwConsumers + 32;

struct DwTmaParams {
  int cwb;           // channel words (4 channels each) a CTA covers: a power of two, 8 .. 128
  int cwb_box;       // channel words per copy (a box is at most 256 bytes wide): min(cwb, 64)
  int nbox;          // cwb / cwb_box copies per row, stored one after the other
  int box_words;     // pix * cwb_box: words of one copy
  int qt_per_cta;    // column groups of 4 outputs per CTA, at most 256 / cwb
  int consumers;     // qt_per_cta * cwb rounded up to whole warps: threads that compute
  int q_blocks;      // ceil(Q / (4 * qt_per_cta))
  int pix;           // pixels per staged row: 4 * qt_per_cta * stride + 3 - stride
  int stage_bytes;   // a row's bytes rounded up to 128
  int row_bytes;     // nbox * box_words * 4: what the copies of one row deliver
  int rows_per_cta;  // output rows per strip
  int cwb_log2, cwb_box_log2;   // cwb and cwb_box are powers of two: the set-up's divisions by them are shifts
  FastDiv fd_q_blocks;          // and the one by q_blocks a multiply-high
};

struct DwTmaShared {
  unsigned long long full[kDwStages];
  unsigned long long empty[kDwStages];
  int abort_flag;
};

__device__ __forceinline__ bool dw_wait(uint32_t bar, uint32_t parity, unsigned int limit, DwTmaShared* sh,
                                        int* status) {
  for (unsigned int it = 0; it < limit; ++it) {
    if (ptx::mbar_try_wait(bar, parity)) return true;
    if (*reinterpret_cast<volatile int*>(&sh->abort_flag)) return false;
  }
  *reinterpret_cast<volatile int*>(&sh->abort_flag) = 1;
  atomicExch(status, kStatusTimeout);
  return false;
}

template <int STRIDE>
__global__ void __launch_bounds__(kDwThreads, 2)
depthwise3x3_tma_kernel(const __grid_constant__ CUtensorMap tmap_x, int8_t* __restrict__ y, ConvGeom g,
                        DwTapParams tp, DwTmaParams prm, int* __restrict__ status, unsigned int wait_limit) {
  using Core = DwTapCore<STRIDE>;
  constexpr int TW = Core::TW, IW = Core::IW;
  extern __shared__ __align__(128) uint8_t dw_smem[];
  DwTmaShared* sh = reinterpret_cast<DwTmaShared*>(dw_smem + static_cast<size_t>(kDwStages) * prm.stage_bytes);

  int qb;
  const int cbi = prm.fd_q_blocks.divmod(static_cast<int>(blockIdx.x), &qb);
  const int p_start = blockIdx.y * prm.rows_per_cta;
  const int rows_out = min(prm.rows_per_cta, g.P - p_start);
  const int rows_in = (rows_out - 1) * STRIDE + 3;
  const int n = blockIdx.z;
  const int h_start = p_start * STRIDE - g.pad_h;
  const int w_base = qb * prm.qt_per_cta * TW * STRIDE - g.pad_w;

  if (threadIdx.x == 0) {
    for (int s = 0; s < kDwStages; ++s) {
      ptx::mbar_init(ptx::smem_u32(&sh->full[s]), 1);
      ptx::mbar_init(ptx::smem_u32(&sh->empty[s]), prm.consumers / 32);  // one arrival per consumer warp
    }
    sh->abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  __syncthreads();

  if (threadIdx.x >= kDwConsumers) {
    // ---------------- producer: one lane issues one box per input row
    if (threadIdx.x == kDwConsumers) {
      ptx::prefetch_tmap(&tmap_x);
      const uint32_t base = ptx::smem_u32(dw_smem);
      int issued = 0;
      bool ok = true;
      for (int i = 0; i < rows_in; ++i) {
        const int stage = i % kDwStages;
        const uint32_t use = static_cast<uint32_t>(i / kDwStages);
        if (use > 0) {
          ok = dw_wait(ptx::smem_u32(&sh->empty[stage]), (use & 1u) ^ 1u, wait_limit, sh, status);
          if (!ok) break;
        }
        const uint32_t full = ptx::smem_u32(&sh->full[stage]);
        ptx::mbar_expect_tx(full, static_cast<uint32_t>(prm.row_bytes));
        for (int b = 0; b < prm.nbox; ++b)
          ptx::tma_load_4d(base + static_cast<uint32_t>(stage) * prm.stage_bytes + static_cast<uint32_t>(b * prm.box_words) * 4u,
                           &tmap_x, full, (cbi * prm.cwb + b * prm.cwb_box) * 4, w_base, h_start + i, n);
        ++issued;
      }
      // Copies already on their way must land before this CTA's shared memory goes away, whichever
      // role gave up and whatever the caller's wait limit: the last pass over the ring is awaited with a
      // bound of its own (in a normal run it has long landed).
      {
        const int first = issued > kDwStages ? issued - kDwStages : 0;
        for (int i = first; i < issued; ++i) {
          const uint32_t bar = ptx::smem_u32(&sh->full[i % kDwStages]);
          const uint32_t par = static_cast<uint32_t>(i / kDwStages) & 1u;
          for (unsigned int it = 0; it < kDrainPolls; ++it)
            if (ptx::mbar_try_wait(bar, par)) break;
        }
      }
    }
    return;
  }

  // ---------------- consumers (whole warps past the last column group leave)
  if (threadIdx.x >= prm.consumers) return;
  const int c4l = static_cast<int>(threadIdx.x) & (prm.cwb - 1);
  const int qt_of_thread = static_cast<int>(threadIdx.x) >> prm.cwb_log2;
  const bool idle = qt_of_thread >= prm.qt_per_cta;               // lane past the CTA's last column group:
  const int qtl = idle ? prm.qt_per_cta - 1 : qt_of_thread;       // reads a valid group, stores nothing
  const int c4 = cbi * prm.cwb + c4l;
  Core core;
  core.load_tables(tp, g.C, c4);
  core.q0 = idle ? g.Q : (qb * prm.qt_per_cta + qtl) * TW;
  core.p_start = p_start;
  core.rows_out = rows_out;
  core.Q = g.Q;
  core.out_pitch = g.out_c_pitch;
  core.yb = y + static_cast<size_t>(n) * g.P * g.Q * g.out_c_pitch + g.out_c_offset + (c4 << 2);
  core.y_image_bytes = static_cast<size_t>(g.P) * g.Q * g.out_c_pitch;
  core.y_first_byte = g.out_c_offset + (c4 << 2);
  const uint32_t word0 = static_cast<uint32_t>((c4l >> prm.cwb_box_log2) * prm.box_words + qtl * TW * STRIDE * prm.cwb_box +
                                               (c4l & (prm.cwb_box - 1)));
  const int lane = threadIdx.x & 31;

  const uint32_t full0 = ptx::smem_u32(&sh->full[0]), empty0 = ptx::smem_u32(&sh->empty[0]);
  static_assert((kDwStages & (kDwStages - 1)) == 0, "ring position by mask");
  // One input row: wait for its stage (one probe; the bounded, abort-aware loop only on a miss), take this thread's
  // words, hand the stage back, feed the arithmetic.  MID: a row in the middle of the strip (no tests in the core).
  bool go = true;
  auto take_row = [&](auto jc, int i, auto mid) {
    constexpr int j = decltype(jc)::value;
    const int stage = i & (kDwStages - 1);
    const uint32_t parity = static_cast<uint32_t>(i / kDwStages) & 1u;
    if (!ptx::mbar_try_wait(full0 + 8u * stage, parity) && !dw_wait(full0 + 8u * stage, parity, wait_limit, sh, status)) {
      go = false;
      return false;
    }
    const uint32_t* row = reinterpret_cast<const uint32_t*>(dw_smem + static_cast<size_t>(stage) * prm.stage_bytes) + word0;
    uint32_t raw[IW];
#pragma unroll
    for (int ix = 0; ix < IW; ++ix) raw[ix] = row[ix * prm.cwb_box];
    __syncwarp();
    if (lane == 0) ptx::mbar_arrive(empty0 + 8u * stage);           // the words are in registers
    if constexpr (decltype(mid)::value) core.template feed_full<j>(i, raw);
    else core.template feed<j>(i, raw);
    return true;
  };
  auto edge_block = [&](int i0) {                                   // rows near the strip's ends: tested one by one
    static_for<0, Core::PERIOD>([&](auto jc) {
      const int i = i0 + decltype(jc)::value;
      if (i >= rows_in) return false;
      return take_row(jc, i, std::false_type{});
    });
  };
  int i0 = 0;
  edge_block(i0);
  i0 += Core::PERIOD;
  // blocks whose rows all lie in the middle: stride 1 rows 2 .. rows_out - 1, stride 2 rows 2 .. 2 rows_out - 1
  const int last_mid = STRIDE == 1 ? rows_out - 1 : 2 * rows_out - 1;
  for (; go && i0 + Core::PERIOD - 1 <= last_mid; i0 += Core::PERIOD)
    static_for<0, Core::PERIOD>([&](auto jc) { return take_row(jc, i0 + decltype(jc)::value, std::true_type{}); });
  for (; go && i0 < rows_in; i0 += Core::PERIOD) edge_block(i0);
}

}  // namespace qc

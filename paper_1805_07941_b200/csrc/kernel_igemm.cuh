// Implicit-GEMM int8 convolution on the sm_100a tensor cores (Eq. 6 as a dense
// contraction): tcgen05.mma kind::i8 with int32 accumulators in tensor memory, operands
// staged in shared memory by TMA (NHWC activation boxes and K-major packed weights, both in
// the swizzled K-major canonical layout), and the requantization epilogue in registers.
//
// A tile is up to 128 output pixels x BN output channels.  The pixels of
// a tile are a box tq x tp x tn of the output (columns x rows x images), so that for filter
// tap (r, s) the activation operand is ONE TMA box of the input, shifted by the tap offset;
// taps that fall outside the image are zero-filled by the TMA unit, which is exact because
// the scheme is symmetric (zero is the integer 0).
//
// The kernel is persistent: a CTA walks a strided list of tiles, the operand ring keeps
// running across tiles, and two accumulator buffers in tensor memory let the epilogue of
// one tile overlap the loads and MMAs of the next.
//
// Warp roles (320 threads): warp 0 issues TMA loads, warp 1 owns tensor memory and issues
// the MMAs, warps 2-9 run the epilogue (each reads the TMEM lane quadrant warp_id % 4 and one
// half of the tile's columns).
// All waits on mbarriers are bounded; on expiry the CTA raises a status flag and leaves.
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>
#include <cstdint>
#include "epilogue.cuh"

namespace qc {

constexpr int kEpilogueWarps = 8;
constexpr int kGroupsPerWarp = 4;     // 16-column groups per epilogue warp: BN <= 2 * 4 * 16 = 128
constexpr int kGroupsPerWarpWide = 8; // the instantiations for 256-wide tiles (one CTA per SM)
constexpr int kIgemmThreads = 64 + 32 * kEpilogueWarps;
constexpr int kMaxStages = 12;
constexpr int kTileM = 128;

// Division of a non-negative 31-bit integer by a divisor fixed for the launch: q = umulhi(n, mul) >> shr with
// mul = ceil(2^(32 + shr) / d), shr = ceil(log2 d) - 1 (Granlund & Montgomery's round-up method; exact for
// n < 2^31), d == 1 passed through.  The set-up of a CTA decomposes its block index, its rows and its first ring
// positions into mixed-radix digits: about fifteen divisions by run-time values, some twenty dependent
// instructions each, at the head of every launch.
struct FastDiv {
  uint32_t mul, shr, d;
  __device__ __forceinline__ int div(int n) const {
    return d == 1u ? n : static_cast<int>(__umulhi(static_cast<uint32_t>(n), mul) >> shr);
  }
  __device__ __forceinline__ int divmod(int n, int* rem) const {
    const int q = div(n);
    *rem = n - q * static_cast<int>(d);
    return q;
  }
};

struct IgemmParams {
  int tq, tp, tn;                  // tile box, in output pixels (tq * tp * tn <= 128)
  int pool_bit;                    // 0, or the lane bit of a pixel's vertical neighbour (= tq, a power of two <= 16) when a
                                   //    2 x 2 max-pool is taken in the epilogue (tile rows q fastest: lane ^ 1 is the horizontal
                                   //    neighbour, lane ^ tq the vertical one)
  int q_step;                      // pixels from one box to the next along q, and the box's columns that are outputs:
                                   //    tq, except in the halo form (tq - 2: the halo's two accumulator columns are dropped)
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
  int fast_epilogue;               // 1: int8 out, nearest-even, K % 16 == 0, aligned rows, and the
                                   //    accumulator bound leaves room for the rounding constant
  uint32_t a_stage_bytes, b_stage_bytes;   // shared-memory footprint per stage (1024-aligned)
  uint32_t out_stage_bytes;        // fast int8 epilogues: one staged output tile (128 rows of BN bytes, 1024-aligned); 0: direct stores
  uint32_t out_swz_mask;           // 16-byte-chunk XOR mask of the staged tile's swizzle (7 / 3 / 1 / 0 for BN = 128 / 64 / 32 / other)
  int out_stage_bufs;              // staged tiles: 2, or 3 when the residual tile is fetched into them by TMA one tile ahead
  uint32_t res_tx_bytes;           // bytes one residual box delivers (BN * tq * tp * tn)
  uint32_t tx_bytes;               // bytes the TMA boxes of one ring stage deliver (activations + weights, or activations alone)
  int halo_s;                      // 0, or S: one activation stage is a box with a horizontal halo (tq = W + S - 1 pixels
                                   //    per image row) that serves the S horizontal taps of a filter row -- the same rows of
                                   //    shared memory, the operand's start advanced by one pixel per tap; the stage then
                                   //    carries S weight chunks, and the kernel sees R x 1 taps
  uint32_t b_chunk_bytes;          // halo form: footprint of one of those weight chunks
  int tap_boxes;                   // 1: the halo_s taps of a stage are separate activation boxes, a_tap_bytes apart
                                   //    (grouped taps: no halo, no shifted reads; only the stage is shared)
  uint32_t a_tap_bytes;            // footprint of one activation box (= a_stage_bytes unless taps are grouped)
  FastDiv fd_tiles_k, fd_tiles_q, fd_tiles_p;   // by the tile counts (block index -> tile digits)
  FastDiv fd_tq, fd_tp;                         // by the box extents (accumulator row -> pixel of the box)
  FastDiv fd_nchunks, fd_S, fd_grid;            // ring position -> (chunk, tap); tiles of this CTA
  int walk_dk, walk_dq, walk_dp, walk_dn;       // digits of the grid size: the step from one tile of a CTA to its next
  int b_resident;                  // 1: the CTA's weight tile (all chunks) is loaded once and stays in shared memory;
                                   //    the ring then carries activations only and the CTA keeps one channel tile
  uint32_t b_res_tx_bytes;         // bytes of that weight tile
};

// Error codes written to the status word.
constexpr int kStatusTimeout = -8;
// Polls granted to a wait for copies that were already issued (they always land): independent of the
// caller's wait limit, so that a CTA that gives up never retires with bulk copies still in flight
// into its shared memory.
constexpr unsigned int kDrainPolls = 1u << 22;

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
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
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
// The same probe with a time hint (nanoseconds): the hardware may suspend the thread until the phase completes
// or the hint runs out, whichever comes first.  A waiting role then issues next to no instructions and still
// wakes when the barrier flips.  Measured: it pays in the kernels that run one CTA per SM on long stages
// (SM-pair tiles: VGG conv4_2 92 -> 82 us) and costs 1-2 % in the two-CTA kernels of the short layers.
constexpr uint32_t kWaitHintNs = 2000;
__device__ __forceinline__ uint32_t mbar_try_wait_hint(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity), "r"(kWaitHintNs)
      : "memory");
  return ok;
}
// Non-blocking probe of a barrier phase.
__device__ __forceinline__ uint32_t mbar_test_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
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
// Shared-memory tile -> global tensor (clipped to the tensor's extent), tracked by the thread's bulk group.
__device__ __forceinline__ void tma_store_4d(const CUtensorMap* map, uint32_t src, int c0, int c1, int c2, int c3) {
  asm volatile(
      "cp.async.bulk.tensor.4d.global.shared::cta.bulk_group [%0, {%2, %3, %4, %5}], [%1];"
      ::"l"(reinterpret_cast<uint64_t>(map)), "r"(src), "r"(c0), "r"(c1), "r"(c2), "r"(c3)
      : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
// All of this thread's bulk stores have finished READING shared memory (the source may be rewritten).
__device__ __forceinline__ void bulk_wait_read_all() { asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory"); }
// ... all but the most recent one.
__device__ __forceinline__ void bulk_wait_read_but_one() { asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory"); }
// All of this thread's bulk stores are complete.
__device__ __forceinline__ void bulk_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }
// Generic-proxy writes to shared memory become visible to the async proxy (TMA).
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void sts_uint4(uint32_t addr, uint32_t a, uint32_t b, uint32_t c, uint32_t d) {
  asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(a), "r"(b), "r"(c), "r"(d) : "memory");
}
__device__ __forceinline__ void prefetch_tmap(const CUtensorMap* map) {
  asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(map)) : "memory");
}
// True in exactly one lane of a fully converged warp.
__device__ __forceinline__ bool elect_one() {
  uint32_t pred;
  asm volatile(
      "{\n\t.reg .b32 rx;\n\t.reg .pred px;\n\t"
      "elect.sync rx|px, 0xffffffff;\n\t"
      "selp.u32 %0, 1, 0, px;\n\t}"
      : "=r"(pred));
  return pred != 0;
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
// 32 lanes x 16 consecutive 32-bit columns.
__device__ __forceinline__ void tmem_ld_32x16(uint32_t taddr, uint32_t (&r)[16]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]),
        "=r"(r[15])
      : "r"(taddr)
      : "memory");
}
__device__ __forceinline__ void grid_dependency_wait() {
  asm volatile("griddepcontrol.wait;" ::: "memory");
}
__device__ __forceinline__ void grid_launch_dependents() {
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
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

// Per-channel epilogue constants, one 16-byte entry per output channel, prepared on the host:
//   x = bias, y = right shift s, and
//   int8 output:  z = 2^(s-1) - 1 (0 when s = 0), w = (s > 0) | 2^t << 1 with t the residual left shift;
//                 they serve the single-pass nearest-even rounding  (v + z + ((v >> s) & w & 1)) >> s;
//   float output: w = bit pattern of the float 2^(e_x + e_w[k]).

struct IgemmShared {
  uint64_t full[kMaxStages];
  uint64_t empty[kMaxStages];
  uint64_t acc_full[2];
  uint64_t acc_empty[2];
  uint64_t res_full[3];           // residual tile landed in staged buffer i
  uint64_t b_full;                // resident weight tile landed
  uint32_t tmem_base;
  volatile int abort_flag;
  // Epilogue constants.  When they fit, those of ALL output channels are staged once per CTA
  // (kpad <= 512 entries, or kpad <= 2048 biases when the shift is per layer); otherwise the current
  // and next tile's channels (at most 256 each) alternate in the two halves.
  union {
    int4 chan[512];
    int32_t bias[2048];
  } cst;
};

constexpr int kChanAllMax = 512, kBiasAllMax = 2048;

// Bounded wait.  Returns false (and raises the CTA abort flag and the global status) if the
// barrier did not flip within `limit` polls, or if another role already gave up.
// HINT: probe with the hardware's suspend hint instead of sleeping between probes.
template <unsigned int SLEEP_NS = 0, bool HINT = false>
__device__ __forceinline__ bool wait_bounded(uint32_t bar, uint32_t parity, unsigned int limit,
                                             IgemmShared* sh, int* status) {
  for (unsigned int it = 0; it < limit; ++it) {
    if (HINT ? ptx::mbar_try_wait_hint(bar, parity) : ptx::mbar_try_wait(bar, parity)) return true;
    if (sh->abort_flag) return false;
    if (SLEEP_NS && !HINT) __nanosleep(SLEEP_NS);      // waiters that can afford it leave the issue slots alone
  }
  sh->abort_flag = 1;
  atomicExch(status, kStatusTimeout);
  return false;
}

// Barrier of the eight epilogue warps (named barrier 1) that also carries a vote: true in every
// thread if any thread passed `failed`.
__device__ __forceinline__ bool epilogue_vote(bool failed) {
  uint32_t any_failed;
  asm volatile(
      "{\n\t.reg .pred pin, pout;\n\t"
      "setp.ne.u32 pin, %1, 0;\n\t"
      "bar.red.or.pred pout, 1, %2, pin;\n\t"
      "selp.u32 %0, 1, 0, pout;\n\t}"
      : "=r"(any_failed)
      : "r"(failed ? 1u : 0u), "n"(kEpilogueWarps * 32)
      : "memory");
  return any_failed != 0;
}

struct TileCoord {
  int q0, p0, n0, k0;
};

// The tiles a CTA visits (blockIdx.x, + gridDim.x, ...) as mixed-radix digits advanced by addition
// with carries: integer divisions only once per kernel, not once per tile.
struct TileWalker {
  int kt, qt, pt, nt;          // digits of the current tile: channel tile fastest, then q, p, image
  int dk, dq, dp, dn;          // digits of the stride
  // first: the CTA's block index; the stride is the grid size, whose digits the host has worked out
  __device__ __forceinline__ void init(const IgemmParams& prm, int first) {
    int m = prm.fd_tiles_k.divmod(first, &kt);
    m = prm.fd_tiles_q.divmod(m, &qt);
    nt = prm.fd_tiles_p.divmod(m, &pt);
    dk = prm.walk_dk; dq = prm.walk_dq; dp = prm.walk_dp; dn = prm.walk_dn;
  }
  __device__ __forceinline__ void next(const IgemmParams& prm) {
    kt += dk; int c = kt >= prm.tiles_k; kt -= c ? prm.tiles_k : 0;
    qt += dq + c; c = qt >= prm.tiles_q; qt -= c ? prm.tiles_q : 0;
    pt += dp + c; c = pt >= prm.tiles_p; pt -= c ? prm.tiles_p : 0;
    nt += dn + c;
  }
  __device__ __forceinline__ TileCoord coord(const IgemmParams& prm) const {
    TileCoord t;
    t.q0 = qt * prm.q_step; t.p0 = pt * prm.tp; t.n0 = nt * prm.tn; t.k0 = kt * prm.BN;
    return t;
  }
};

// Epilogue variants, one kernel instantiation each so that a launch carries only the code it runs
// (these kernels are short; instruction fetch of unused paths is measurable):
//   FAST_I8 / FAST_I8_RES: int8 output, nearest-even, 8-bit saturation, K % 16 == 0, aligned rows,
//                          accumulator bound leaves room for the rounding constant; without / with residual
//   I8: any rounding mode, bit width, alignment;  I32, F32: wide or float output
//   FAST_I8_U / FAST_I8_RES_U: the same with one shift for all channels (per-layer scales): only the
//                          bias is per channel, everything else sits in kernel parameters
//   FLT_I8*:               the four fast variants again for layers whose wide value provably stays below
//                          2^22 in magnitude (bound computed from the actual weights at create time).
//                          There the integer ALU, the epilogue's bottleneck, is relieved by the FMA pipe:
//                          adding bias + 0x4B400000 yields the bit pattern of the float M + v, M = 1.5 * 2^23;
//                          (M + v) * 2^-s + M * (1 - 2^-s) is one FMA (product and addend exact) whose
//                          single rounding is nearest-even at integer granularity, i.e. the requantized
//                          value sits in the low mantissa byte; ReLU and the clamps are integer min/max
//                          on the bit patterns (positive floats order like integers).
enum : int { EPI_FAST_I8 = 0, EPI_FAST_I8_RES = 1, EPI_I8 = 2, EPI_I32 = 3, EPI_F32 = 4, EPI_FAST_I8_U = 5,
             EPI_FAST_I8_RES_U = 6, EPI_FLT_I8 = 7, EPI_FLT_I8_RES = 8, EPI_FLT_I8_U = 9, EPI_FLT_I8_RES_U = 10 };

template <int EPI> struct EpiTraits {
  static constexpr bool flt = EPI >= EPI_FLT_I8;
  static constexpr bool fast = EPI == EPI_FAST_I8 || EPI == EPI_FAST_I8_RES || EPI == EPI_FAST_I8_U ||
                               EPI == EPI_FAST_I8_RES_U || flt;
  static constexpr bool res = EPI == EPI_FAST_I8_RES || EPI == EPI_FAST_I8_RES_U || EPI == EPI_FLT_I8_RES ||
                              EPI == EPI_FLT_I8_RES_U;
  static constexpr bool uni = EPI == EPI_FAST_I8_U || EPI == EPI_FAST_I8_RES_U || EPI == EPI_FLT_I8_U ||
                              EPI == EPI_FLT_I8_RES_U;
};

constexpr int kMagicBits = 0x4B400000;        // bit pattern of 1.5 * 2^23 = 12582912.0f

// Two int32 -> two saturated int8 in the low half of the result, upper half taken from c's low half.
__device__ __forceinline__ uint32_t pack_sat_s8(int32_t hi_byte, int32_t lo_byte, uint32_t c) {
  uint32_t d;
  asm("cvt.pack.sat.s8.s32.b32 %0, %1, %2, %3;" : "=r"(d) : "r"(hi_byte), "r"(lo_byte), "r"(c));
  return d;
}

// Byte B of a word, sign-extended to 32 bits in one permute (selector nibble 8 | B replicates the
// sign bit of byte B).
template <int B>
__device__ __forceinline__ int32_t sign_extend_byte(uint32_t w) {
  uint32_t d;
  asm("prmt.b32 %0, %1, 0, %2;" : "=r"(d) : "r"(w), "n"(B | ((8 | B) << 4) | ((8 | B) << 8) | ((8 | B) << 12)));
  return static_cast<int32_t>(d);
}

// 16 bytes from a shared-memory address (the channel constants live there; an explicit shared load
// keeps the compiler from falling back to generic addressing).
__device__ __forceinline__ int4 lds_int4(uint32_t addr) {
  int4 v;
  asm volatile("ld.shared.v4.s32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr));
  return v;
}

// 16 accumulator columns of one row -> 16 output channels.  cst: shared-memory address of the
// tile's first channel constant.
// RELU: 0 / 1 fixed at compile time (the float-rounding variants: one predicated instruction less per
// output), 2 = taken from the parameters at run time.
// RSTG: 2 in the kernel's template list stands for the pooled epilogue (epilogue_pool_16, never this function);
// RSTG: 1 when the residual tile has been brought into the staged tile by TMA (read there, overwritten
// in place by the result).
// The fast conversion of 16 accumulator columns to 16 int8 codes (four packed words): bias, residual << t, ReLU,
// shift with nearest-even rounding, saturation.  cst_g: shared-memory address of the first column's constant
// (4 bytes per column when only the biases differ, 16 otherwise); rw: the 16 residual bytes (ignored without).
template <int EPI, int RELU>
__device__ __forceinline__ void convert_16(const uint32_t* acc, uint32_t cst_g, const uint32_t (&rw)[4],
                                           const EpilogueParams& ep, uint32_t (&wds)[4]) {
  const bool relu = RELU == 2 ? ep.relu != 0 : RELU == 1;
#pragma unroll
  for (int g = 0; g < 4; ++g) {
    int32_t q[4];
    int32_t rv[4] = {0, 0, 0, 0};
    if (EpiTraits<EPI>::res) {
      rv[0] = sign_extend_byte<0>(rw[g]); rv[1] = sign_extend_byte<1>(rw[g]);
      rv[2] = sign_extend_byte<2>(rw[g]); rv[3] = sign_extend_byte<3>(rw[g]);
    }
    // with per-layer shifts only the biases differ per channel: four of them per shared-memory load
    int4 bq = make_int4(0, 0, 0, 0);
    if (EpiTraits<EPI>::uni) bq = lds_int4(cst_g + static_cast<uint32_t>(g * 16));
    const int32_t bias4[4] = {bq.x, bq.y, bq.z, bq.w};
    if (EpiTraits<EPI>::flt) {
#pragma unroll
      for (int b = 0; b < 4; ++b) {
        const int j = g * 4 + b;
        // x = bias + magic bits; y = bits of 2^-s; z = bits of M * (1 - 2^-s); w >> 1 = 2^t
        const int4 c = EpiTraits<EPI>::uni ? make_int4(bias4[b], __float_as_int(ep.uni_c1), __float_as_int(ep.uni_c2), ep.uni_w)
                                           : lds_int4(cst_g + static_cast<uint32_t>(j * 16));
        int32_t v = static_cast<int32_t>(acc[j]);
        if (EpiTraits<EPI>::res) v += rv[b] * (c.w >> 1);
        const int32_t fb = relu ? __viaddmax_s32(v, c.x, kMagicBits) : v + c.x;
        const float r = fmaf(__int_as_float(fb), __int_as_float(c.y), __int_as_float(c.z));
        int32_t rb = min(__float_as_int(r), kMagicBits + 127);
        if (!relu) rb = max(rb, kMagicBits + ep.lo);
        q[b] = rb;                                     // the int8 code is the low byte
      }
      const uint32_t lo2 = __byte_perm(static_cast<uint32_t>(q[0]), static_cast<uint32_t>(q[1]), 0x0040);
      const uint32_t hi2 = __byte_perm(static_cast<uint32_t>(q[2]), static_cast<uint32_t>(q[3]), 0x0040);
      wds[g] = __byte_perm(lo2, hi2, 0x5410);
    } else {
#pragma unroll
      for (int b = 0; b < 4; ++b) {
        const int j = g * 4 + b;
        // per-channel constants from shared memory, or only the bias when the shift is per layer
        const int4 c = EpiTraits<EPI>::uni ? make_int4(bias4[b], ep.uni_shift, ep.uni_z, ep.uni_w)
                                           : lds_int4(cst_g + static_cast<uint32_t>(j * 16));
        int32_t v = static_cast<int32_t>(acc[j]);
        if (EpiTraits<EPI>::res) v += rv[b] * (c.w >> 1);         // residual scaled by 2^t
        v = relu ? __viaddmax_s32(v, c.x, 0) : v + c.x;
        // nearest-even:  (v + 2^(s-1) - 1 + lsb of the truncated quotient) >> s
        v = (v + c.z + ((v >> c.y) & c.w & 1)) >> c.y;
        q[b] = relu ? v : max(v, ep.lo);            // the upper bound is the 8-bit saturation below
      }
      wds[g] = pack_sat_s8(q[1], q[0], pack_sat_s8(q[3], q[2], 0u));
    }
  }
}

template <int EPI, int RELU, int RSTG>
__device__ __forceinline__ void epilogue_16(const uint32_t (&acc)[16], uint32_t cst, int col, int k,
                                            size_t pix, const IgemmParams& prm, const EpilogueParams& ep,
                                            const int8_t* __restrict__ res, const uint4& res16,
                                            void* __restrict__ y, uint32_t stage_row) {
  const size_t o = pix * prm.out_c_pitch + prm.out_c_offset + k;
  const bool relu = RELU == 2 ? ep.relu != 0 : RELU == 1;
  if (EpiTraits<EPI>::fast) {
    uint32_t rw[4] = {res16.x, res16.y, res16.z, res16.w};         // residual bytes, fetched ahead
    uint32_t stage_addr = 0;
    if (prm.out_stage_bytes) {
      // position of these 16 bytes in the staged tile (row-major, 16-byte chunks swizzled as the tensor
      // maps of the output and the residual expect)
      const uint32_t off = stage_row + static_cast<uint32_t>(col);
      stage_addr = off ^ (((off >> 7) & prm.out_swz_mask) << 4);
      if (EpiTraits<EPI>::res && RSTG == 1) {
        // the residual tile was brought there by TMA; the result overwrites it in place
        const int4 r4 = lds_int4(stage_addr);
        rw[0] = r4.x; rw[1] = r4.y; rw[2] = r4.z; rw[3] = r4.w;
      }
    }
    uint32_t wds[4];
    convert_16<EPI, RELU>(acc, cst + static_cast<uint32_t>(col) * (EpiTraits<EPI>::uni ? 4u : 16u), rw, ep, wds);
    if (prm.out_stage_bytes) {
      ptx::sts_uint4(stage_addr, wds[0], wds[1], wds[2], wds[3]);
    } else {
      *reinterpret_cast<uint4*>(static_cast<int8_t*>(y) + o) = make_uint4(wds[0], wds[1], wds[2], wds[3]);
    }
    return;
  }
  const int8_t* rp = res ? res + pix * prm.K + k : nullptr;
#pragma unroll
  for (int j = 0; j < 16; ++j) {
    if (k + j >= prm.K) break;
    const int4 c = lds_int4(cst + static_cast<uint32_t>(col + j) * 16u);
    const int32_t rv = rp ? static_cast<int32_t>(rp[j]) : 0;
    const int t = rp ? ep.res_lshift[k + j] : 0;
    const int32_t wide = wide_value(static_cast<int32_t>(acc[j]), c.x, rv, t, relu);
    if (EPI == EPI_I8)
      static_cast<int8_t*>(y)[o + j] = static_cast<int8_t>(requantize(wide, c.y, ep.rounding, ep.lo, ep.hi));
    else if (EPI == EPI_I32)
      static_cast<int32_t*>(y)[o + j] = wide;
    else
      // beta -> float: c.w holds the bits of 2^(e_x + e_w[k]); the product is exact (power of two)
      static_cast<float*>(y)[o + j] = __int2float_rn(wide) * __int_as_float(c.w);
  }
}

// 16 accumulator columns of one row with a 2 x 2 / stride 2 max-pool over pixels taken on the way.  The conversion
// (bias, ReLU, shift with rounding, saturation) is non-decreasing in the accumulator, so the maximum over the four
// pixels of a window is taken on the raw accumulators and converted once.  The four pixels of a window sit in the
// lanes l, l ^ 1 (horizontal neighbour) and l ^ vbit, l ^ 1 ^ vbit (vertical neighbours) of one warp.  The
// maximum is a reduce-scatter: lanes l and l ^ 1 exchange one half of the 16 columns each and keep the other,
// then l and l ^ vbit exchange one half of those 8, so every lane ends up with the window's maxima of 4 of the 16
// columns, converts those and stores 4 bytes; the window's four lanes write 16 consecutive bytes of the pooled
// pixel.  All 32 lanes must call (shuffles); `store_ok` says whether this lane's pixel lies inside the image.
// Fast epilogues without residual only.
template <int EPI, int RELU>
__device__ __forceinline__ void epilogue_pool_16(const uint32_t (&acc)[16], uint32_t cst, int col, int k, size_t pooled_pix,
                                                 bool store_ok, int lane, int vbit, const IgemmParams& prm,
                                                 const EpilogueParams& ep, void* __restrict__ y) {
  static_assert(EpiTraits<EPI>::fast && !EpiTraits<EPI>::res, "pooled epilogue: fast variants without residual");
  const bool relu = RELU == 2 ? ep.relu != 0 : RELU == 1;
  const bool odd_q = (lane & 1) != 0, odd_p = (lane & vbit) != 0;
  int32_t r8[8], v4[4];
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    const int32_t lo = static_cast<int32_t>(acc[i]), hi = static_cast<int32_t>(acc[i + 8]);
    const int32_t keep = odd_q ? hi : lo, send = odd_q ? lo : hi;
    r8[i] = max(keep, __shfl_xor_sync(0xffffffffu, send, 1));
  }
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int32_t keep = odd_p ? r8[i + 4] : r8[i], send = odd_p ? r8[i] : r8[i + 4];
    v4[i] = max(keep, __shfl_xor_sync(0xffffffffu, send, vbit));
  }
  const int c0 = (odd_q ? 8 : 0) + (odd_p ? 4 : 0);              // this lane's 4 columns of the 16
  int4 bq = make_int4(0, 0, 0, 0);
  if (EpiTraits<EPI>::uni) bq = lds_int4(cst + static_cast<uint32_t>(col + c0) * 4u);
  const int32_t bias4[4] = {bq.x, bq.y, bq.z, bq.w};
  int32_t q[4];
#pragma unroll
  for (int b = 0; b < 4; ++b) {
    if (EpiTraits<EPI>::flt) {
      const int4 c = EpiTraits<EPI>::uni ? make_int4(bias4[b], __float_as_int(ep.uni_c1), __float_as_int(ep.uni_c2), ep.uni_w)
                                         : lds_int4(cst + static_cast<uint32_t>(col + c0 + b) * 16u);
      const int32_t fb = relu ? __viaddmax_s32(v4[b], c.x, kMagicBits) : v4[b] + c.x;
      const float r = fmaf(__int_as_float(fb), __int_as_float(c.y), __int_as_float(c.z));
      int32_t rb = min(__float_as_int(r), kMagicBits + 127);
      if (!relu) rb = max(rb, kMagicBits + ep.lo);
      q[b] = rb;
    } else {
      const int4 c = EpiTraits<EPI>::uni ? make_int4(bias4[b], ep.uni_shift, ep.uni_z, ep.uni_w)
                                         : lds_int4(cst + static_cast<uint32_t>(col + c0 + b) * 16u);
      int32_t v = relu ? __viaddmax_s32(v4[b], c.x, 0) : v4[b] + c.x;
      v = (v + c.z + ((v >> c.y) & c.w & 1)) >> c.y;
      q[b] = relu ? v : max(v, ep.lo);
    }
  }
  uint32_t word;
  if (EpiTraits<EPI>::flt) {
    const uint32_t lo2 = __byte_perm(static_cast<uint32_t>(q[0]), static_cast<uint32_t>(q[1]), 0x0040);
    const uint32_t hi2 = __byte_perm(static_cast<uint32_t>(q[2]), static_cast<uint32_t>(q[3]), 0x0040);
    word = __byte_perm(lo2, hi2, 0x5410);
  } else {
    word = pack_sat_s8(q[1], q[0], pack_sat_s8(q[3], q[2], 0u));
  }
  if (store_ok)
    *reinterpret_cast<uint32_t*>(static_cast<int8_t*>(y) + pooled_pix * prm.out_c_pitch + prm.out_c_offset + k + c0) = word;
}

// Persistent kernel: each CTA walks tiles blockIdx.x, blockIdx.x + gridDim.x, ...  The shared-memory
// ring of operand stages runs on across tiles, and the accumulator is double-buffered in tensor
// memory so the epilogue of one tile overlaps the loads and MMAs of the next.
// GPW: 16-column groups an epilogue warp may own: 4 (tiles up to 128 channels wide, two CTAs per SM) or
// 8 (tiles up to 256 wide: an MMA of N = 256 lasts twice as long for the same A operand, so a stage
// carries twice the tensor work per byte fetched and per instruction of the issuing thread; both
// accumulator buffers together fill the tensor memory, hence one CTA per SM).
template <int EPI, int RELU = 2, int RSTG = 0, int GPW = kGroupsPerWarp>
__global__ void __launch_bounds__(kIgemmThreads, GPW > kGroupsPerWarp ? 1 : 2)
igemm_i8_kernel(const __grid_constant__ CUtensorMap tmap_a, const __grid_constant__ CUtensorMap tmap_b,
                const __grid_constant__ CUtensorMap tmap_y, const __grid_constant__ CUtensorMap tmap_r,
                const IgemmParams prm, const EpilogueParams ep, const int4* __restrict__ chan_table,
                const int8_t* __restrict__ res, void* __restrict__ y, int* status, unsigned int wait_limit) {
  extern __shared__ uint8_t smem_raw[];
  // operand stages need 1024-byte alignment (swizzle atom); the launch reserves the slack
  uint8_t* tiles = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) &
                                              ~static_cast<uintptr_t>(1023));
  // ring stages (activations + weights, or activations alone), then the resident weight tile if any
  const uint32_t stage_bytes = prm.a_stage_bytes + (prm.b_resident ? 0u : prm.b_stage_bytes);
  const int num_kb_all = prm.R * prm.S * prm.nchunks;
  const uint32_t b_res_off = static_cast<uint32_t>(prm.stages) * stage_bytes;
  uint8_t* out_stage = tiles + b_res_off + (prm.b_resident ? static_cast<uint32_t>(num_kb_all) * prm.b_stage_bytes : 0u);   // staged output tiles
  IgemmShared* sh = reinterpret_cast<IgemmShared*>(out_stage + static_cast<uint32_t>(prm.out_stage_bufs) * prm.out_stage_bytes);

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  constexpr bool kPool = RSTG == 2;              // 2 x 2 max-pool taken in the epilogue
  constexpr bool kHint = GPW > kGroupsPerWarp;   // one CTA per SM on long stages: waits use the suspend hint
  const int num_kb = prm.R * prm.S * prm.nchunks;
  const int total_tiles = prm.tiles_q * prm.tiles_p * prm.tiles_n * prm.tiles_k;

  if (threadIdx.x == 0) {
    for (int s = 0; s < prm.stages; ++s) {
      ptx::mbar_init(ptx::smem_u32(&sh->full[s]), 1);
      ptx::mbar_init(ptx::smem_u32(&sh->empty[s]), 1);
    }
    for (int b = 0; b < 2; ++b) {
      ptx::mbar_init(ptx::smem_u32(&sh->acc_full[b]), 1);
      ptx::mbar_init(ptx::smem_u32(&sh->acc_empty[b]), kEpilogueWarps);   // one arrival per epilogue warp
    }
    for (int b = 0; b < 3; ++b) ptx::mbar_init(ptx::smem_u32(&sh->res_full[b]), 1);
    ptx::mbar_init(ptx::smem_u32(&sh->b_full), 1);
    sh->abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 0 && lane == 0) {
    ptx::prefetch_tmap(&tmap_a);
    ptx::prefetch_tmap(&tmap_b);
    if (EpiTraits<EPI>::fast && prm.out_stage_bytes) ptx::prefetch_tmap(&tmap_y);
    if (EpiTraits<EPI>::res && RSTG == 1) ptx::prefetch_tmap(&tmap_r);
  }
  if (warp == 1) {
    ptx::tmem_alloc(ptx::smem_u32(&sh->tmem_base), static_cast<uint32_t>(2 * prm.tmem_cols));
    ptx::tmem_relinquish();
  }
  ptx::tc_fence_before();
  __syncthreads();
  ptx::tc_fence_after();
  const uint32_t tmem_base = sh->tmem_base;
  // Everything above touched no tensor of another kernel, so under programmatic dependent launch
  // it overlaps the tail of the previous kernel in the stream.  The next kernel may start its own
  // set-up right away; each role of this one waits for the previous kernel (griddepcontrol.wait)
  // immediately before its first access to a tensor that kernel may have written, with all the
  // arithmetic leading up to that access already done.
  ptx::grid_launch_dependents();

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    // The CTA's loads form one sequence of stages (tile, filter row r, tap sx, channel chunk ci); stage g
    // goes to ring slot g % stages.  The first pass over the ring is issued by `stages` lanes side by
    // side, lane l taking stage l: the address arithmetic of a stage costs one thread some hundred cycles
    // of dependent instructions, so a single thread would spend longer issuing the nine small stages of
    // a short layer than the tensor core spends on them, and after the wait on the previous kernel the
    // whole first pass goes out at once.  From the second pass on a stage can only follow the MMAs that
    // free its slot, in order: one lane walks the sequence (lanes polling different barriers in one warp
    // only slow each other down).
    const uint32_t tiles_addr = ptx::smem_u32(tiles);
    const bool has_tiles = static_cast<int>(blockIdx.x) < total_tiles;
    // (a resident weight tile is fetched by the MMA warp, which has nothing else to do at this point: the
    // activation loads below then go out without waiting behind a dozen weight copies)
    // One stage: arm the slot's barrier, load the weight chunk(s) unless resident, then the activation box.
    // `first` marks a lane's first activation load: the previous kernel's results are needed from there on
    // (not for the weights), so the wait on it sits right in front of that load.
    // `doit`: this thread issues (the arithmetic may run on all lanes with warp-uniform values, see below).
    auto issue = [&](int slot, const TileCoord& tc, int r, int sx, int ci, bool first, bool doit) {
      const uint32_t full = ptx::smem_u32(&sh->full[slot]);
      const uint32_t a_dst = tiles_addr + static_cast<uint32_t>(slot) * stage_bytes;
      const int w0 = tc.q0 * prm.stride_w - prm.pad_w + sx, h0 = tc.p0 * prm.stride_h - prm.pad_h + r;
      if (doit) {
        ptx::mbar_expect_tx(full, prm.tx_bytes);
        if (!prm.b_resident) {
          if (prm.halo_s) {
            for (int hs = 0; hs < prm.halo_s; ++hs)
              ptx::tma_load_2d(a_dst + prm.a_stage_bytes + static_cast<uint32_t>(hs) * prm.b_chunk_bytes, &tmap_b, full,
                               ((r * prm.halo_s + hs) * prm.nchunks + ci) * prm.BKC, tc.k0);
          } else {
            ptx::tma_load_2d(a_dst + prm.a_stage_bytes, &tmap_b, full, ((r * prm.S + sx) * prm.nchunks + ci) * prm.BKC, tc.k0);
          }
        }
        if (first) ptx::grid_dependency_wait();
        ptx::tma_load_4d(a_dst, &tmap_a, full, ci * prm.BKC, w0, h0, tc.n0);
        if (prm.tap_boxes)
          for (int hs = 1; hs < prm.halo_s; ++hs)           // the filter row's other taps, each a box of its own
            ptx::tma_load_4d(a_dst + static_cast<uint32_t>(hs) * prm.a_tap_bytes, &tmap_a, full, ci * prm.BKC, w0 + hs, h0, tc.n0);
      }
    };
    // stages this CTA issues in all, and how many of them make up the first pass
    const int my_tiles = has_tiles ? prm.fd_grid.div(total_tiles - static_cast<int>(blockIdx.x) + static_cast<int>(gridDim.x) - 1) : 0;
    const long long total_stages = static_cast<long long>(my_tiles) * num_kb;
    const int first_pass = static_cast<int>(total_stages < prm.stages ? total_stages : prm.stages);
    {
      // position `lane` of the sequence (lane `first_pass` of lane 0's walk below): mixed-radix digits
      const int pos = lane < first_pass ? lane : first_pass;
      int ci, sx;
      int t0 = prm.fd_nchunks.divmod(pos, &ci);
      int r = prm.fd_S.divmod(t0, &sx);
      int tile = blockIdx.x;
      TileWalker walk;
      walk.init(prm, blockIdx.x);
      while (r >= prm.R && tile < total_tiles) { r -= prm.R; tile += gridDim.x; walk.next(prm); }
      issue(lane < first_pass ? lane : 0, walk.coord(prm), r, sx, ci, true, lane < first_pass);
      __syncwarp();
      {
        // The rest of the sequence, in order, from position first_pass.  The whole warp runs this loop with
        // warp-uniform values (addresses and coordinates then live in uniform registers, which is where the
        // copy instructions take their operands from); lane 0 alone issues.
        const bool leader = lane == 0;
        t0 = prm.fd_nchunks.divmod(first_pass, &ci);
        r = prm.fd_S.divmod(t0, &sx);
        tile = blockIdx.x;
        walk.init(prm, blockIdx.x);
        while (r >= prm.R && tile < total_tiles) { r -= prm.R; tile += gridDim.x; walk.next(prm); }
        int stage = 0;
        uint32_t phase = 1;                                  // second pass over the ring
        long long issued = first_pass;
        bool ok = true;
        TileCoord tc = walk.coord(prm);
        while (tile < total_tiles) {
          if (!(kHint ? ptx::mbar_try_wait_hint : ptx::mbar_try_wait)(ptx::smem_u32(&sh->empty[stage]), phase ^ 1u)) {
            ok = wait_bounded<32, kHint>(ptx::smem_u32(&sh->empty[stage]), phase ^ 1u, wait_limit, sh, status);
            if (!ok) break;
          }
          issue(stage, tc, r, sx, ci, false, leader);
          ++issued;
          if (++ci == prm.nchunks) {
            ci = 0;
            if (++sx == prm.S) {
              sx = 0;
              if (++r == prm.R) { r = 0; tile += gridDim.x; walk.next(prm); tc = walk.coord(prm); }
            }
          }
          if (++stage == prm.stages) { stage = 0; phase ^= 1u; }
        }
        __syncwarp();
        if (!leader) issued = 0;                             // (lane 0 alone waits below)
        // Whatever happened to the other roles, this CTA's shared memory must outlive every copy issued
        // into it: wait (bounded, but not by the caller's limit) for the resident weight tile and for the
        // last pass over the ring.  In a normal run all of this has long landed and each probe succeeds.
        if (leader && prm.b_resident && has_tiles) {
          for (unsigned int w = 0; w < kDrainPolls; ++w)
            if (ptx::mbar_try_wait(ptx::smem_u32(&sh->b_full), 0u)) break;
        }
        const long long first = issued > prm.stages ? issued - prm.stages : 0;
        int st_i = static_cast<int>(first % prm.stages);
        uint32_t par = static_cast<uint32_t>(first / prm.stages) & 1u;
        for (long long i = first; i < issued; ++i) {
          const uint32_t bar = ptx::smem_u32(&sh->full[st_i]);
          for (unsigned int w = 0; w < kDrainPolls; ++w)
            if (ptx::mbar_try_wait(bar, par)) break;
          if (++st_i == prm.stages) { st_i = 0; par ^= 1u; }
        }
        // a CTA always waits for the previous kernel before it retires, so that "this kernel is complete"
        // implies "every kernel before it is complete" for the kernel after it
        if (leader) ptx::grid_dependency_wait();
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    // One elected lane feeds the tensor core, and the tensor core queues next to nothing: whatever
    // happens between two MMAs is time the unit idles (a 128 x 128 x 32 MMA lasts 64 cycles).  So
    //  - the whole warp runs the loop with warp-uniform values, which lets descriptors and
    //    addresses live in uniform registers (the MMA takes its operands from those) instead of
    //    being moved there before every instruction; only the MMA / commit are predicated;
    //  - descriptors and ring position advance by additions;
    //  - a stage is awaited with one probe of its barrier (the bounded, abort-aware loop only on a miss)
    //    and no warp votes: a stage costs the issuing thread a few hundred cycles of dependent
    //    instructions, which is what bounds layers whose stages carry little tensor work.
    {
      const bool leader = ptx::elect_one();
      const uint32_t idesc = make_idesc_i8(prm.BN);
      const int mma_per_stage = prm.BKC / 32;
      const uint32_t tiles_addr = ptx::smem_u32(tiles);
      const bool bres = prm.b_resident != 0;
      if (leader && bres && static_cast<int>(blockIdx.x) < total_tiles) {
        // the whole weight tile of this CTA's channel tile, once; weights never depend on the previous kernel
        int kt0;
        prm.fd_tiles_k.divmod(static_cast<int>(blockIdx.x), &kt0);
        const int k0 = kt0 * prm.BN;
        const uint32_t bar = ptx::smem_u32(&sh->b_full);
        ptx::mbar_expect_tx(bar, prm.b_res_tx_bytes);
        // (halo form, one chunk per tap: a stage's three weight chunks are the columns 3 kb, 3 kb + 1, 3 kb + 2)
        const int per_stage = prm.halo_s ? prm.halo_s : 1;
        for (int kb = 0; kb < num_kb; ++kb)
          for (int hs = 0; hs < per_stage; ++hs)
            ptx::tma_load_2d(tiles_addr + b_res_off + static_cast<uint32_t>(kb) * prm.b_stage_bytes +
                                 static_cast<uint32_t>(hs) * prm.b_chunk_bytes,
                             &tmap_b, bar, (kb * per_stage + hs) * prm.BKC, k0);
      }
      __syncwarp();
      const uint64_t a_desc0 = make_kmajor_desc(tiles_addr, prm.BKC);
      const uint64_t b_desc0 = make_kmajor_desc(tiles_addr + (bres ? b_res_off : prm.a_stage_bytes), prm.BKC);
      const uint64_t desc_step = stage_bytes >> 4;          // start-address field counts 16-byte units
      // resident weights: chunk kb of the tile sits at its own place, whatever the ring position
      const uint64_t b_step = bres ? (prm.b_stage_bytes >> 4) : desc_step;
      uint64_t a_desc = a_desc0, b_desc = b_desc0;
      // taps of one stage: one pixel row further on in the same box (halo form) or the next box (grouped taps)
      const uint64_t halo_row = static_cast<uint64_t>(prm.tap_boxes ? prm.a_tap_bytes : static_cast<uint32_t>(prm.BKC)) >> 4;
      const uint64_t halo_bchunk = prm.b_chunk_bytes >> 4;
      const uint32_t full0 = ptx::smem_u32(&sh->full[0]), empty0 = ptx::smem_u32(&sh->empty[0]);
      int stage = 0, it = 0;
      uint32_t phase = 0;
      bool ok = true;
      for (int tile = blockIdx.x; tile < total_tiles && ok; tile += gridDim.x, ++it) {
        const int buf = it & 1;
        const uint32_t use = static_cast<uint32_t>(it >> 1);
        // the epilogue must have drained this accumulator buffer (two tiles ago)
        ok = wait_bounded<0, kHint>(ptx::smem_u32(&sh->acc_empty[buf]), (use & 1u) ^ 1u, wait_limit, sh, status);
        if (!ok) break;
        ptx::tc_fence_after();
        const uint32_t d_tmem = tmem_base + static_cast<uint32_t>(buf * prm.tmem_cols);
        uint32_t accumulate = 0;
        if (bres) {
          if (it == 0) {
            ok = wait_bounded<0, kHint>(ptx::smem_u32(&sh->b_full), 0u, wait_limit, sh, status);
            if (!ok) break;
          }
          b_desc = b_desc0;
        }
        for (int kb = 0; kb < num_kb; ++kb) {
          // all lanes probe the same barrier with the same instruction, so they agree without a vote
          if (!(kHint ? ptx::mbar_try_wait_hint : ptx::mbar_try_wait)(full0 + 8u * stage, phase)) {
            ok = wait_bounded<0, kHint>(full0 + 8u * stage, phase, wait_limit, sh, status);
            if (!ok) break;
          }
          ptx::tc_fence_after();
          if (leader) {
            // 32 bytes along K inside the swizzle span = +2 in the descriptor's 16-byte address units
            ptx::mma_i8(d_tmem, a_desc, b_desc, idesc, accumulate);
            if (mma_per_stage > 1) ptx::mma_i8(d_tmem, a_desc + 2u, b_desc + 2u, idesc, 1u);
            if (mma_per_stage > 2) {
              ptx::mma_i8(d_tmem, a_desc + 4u, b_desc + 4u, idesc, 1u);
              ptx::mma_i8(d_tmem, a_desc + 6u, b_desc + 6u, idesc, 1u);
            }
            // halo form: the other horizontal taps are the same activation rows one pixel (one row of BKC
            // bytes) further on -- start address advanced by a row, the descriptor's base offset telling the
            // swizzle phase of the new first row -- against the next weight chunk of the stage
            for (int hs = 1; hs < prm.halo_s; ++hs) {
              const uint64_t ah = a_desc + static_cast<uint64_t>(hs) * halo_row;
              const uint64_t bh = b_desc + static_cast<uint64_t>(hs) * halo_bchunk;
              ptx::mma_i8(d_tmem, ah, bh, idesc, 1u);
              if (mma_per_stage > 1) ptx::mma_i8(d_tmem, ah + 2u, bh + 2u, idesc, 1u);
              if (mma_per_stage > 2) {
                ptx::mma_i8(d_tmem, ah + 4u, bh + 4u, idesc, 1u);
                ptx::mma_i8(d_tmem, ah + 6u, bh + 6u, idesc, 1u);
              }
            }
            ptx::mma_commit(empty0 + 8u * stage);             // stage free once these MMAs retire
          }
          accumulate = 1;
          if (++stage == prm.stages) { stage = 0; phase ^= 1u; a_desc = a_desc0; if (!bres) b_desc = b_desc0; }
          else { a_desc += desc_step; if (!bres) b_desc += b_step; }
          if (bres) b_desc += b_step;
        }
        if (ok && leader) ptx::mma_commit(ptx::smem_u32(&sh->acc_full[buf]));
      }
      __syncwarp();
    }
  } else {
    // ------------------------------------------------------------------ epilogue
    // Eight warps: warp w reads the TMEM lane quadrant w % 4 (rows 32 * (w % 4) ...) and one half of
    // the tile's 16-column groups, so every scheduler has several epilogue warps to switch between.
    const int ew = warp - 2;
    const int quad = warp & 3;
    const int row = quad * 32 + lane;                        // tile row = accumulator lane
    int q_i, p_i;
    const int n_i = prm.fd_tp.divmod(prm.fd_tq.divmod(row, &q_i), &p_i);
    const int etid = threadIdx.x - 64;                       // 0 .. 255 among the epilogue threads
    const int groups16 = prm.BN / 16;
    const int g_split = (groups16 + 1) / 2;
    const int g_begin = (ew < 4) ? 0 : g_split;
    const int g_end = (ew < 4) ? g_split : groups16;
    int it = 0;
    bool ok = true;
    const int kpad = prm.tiles_k * prm.BN;
    const bool cst_all = EpiTraits<EPI>::uni ? kpad <= kBiasAllMax : kpad <= kChanAllMax;
    if (cst_all) {
      for (int i = etid; i < kpad; i += kEpilogueWarps * 32) {
        if (EpiTraits<EPI>::uni) sh->cst.bias[i] = __ldg(&chan_table[i].x);
        else sh->cst.chan[i] = __ldg(chan_table + i);
      }
      asm volatile("bar.sync 1, %0;" ::"n"(kEpilogueWarps * 32) : "memory");
    }
    TileWalker walk;
    walk.init(prm, blockIdx.x);
    // the residual may come from the previous kernel (the constants above never do)
    ptx::grid_dependency_wait();
    const uint32_t cst_addr = ptx::smem_u32(&sh->cst);
    // Residual tiles come by TMA into the staged buffers, one tile ahead of the arithmetic (three buffers:
    // the tile being stored, the tile being computed, the residual of the next).  The thread that issues
    // the stores also issues these loads: it alone knows when a buffer's store has finished reading.
    constexpr bool res_staged = EpiTraits<EPI>::res && EpiTraits<EPI>::fast && RSTG == 1;   // the planner then provides three staged tiles
    const uint32_t stage0 = ptx::smem_u32(out_stage);
    TileWalker walk_next = walk;
    int sbuf = 0;                              // staged buffer of the current tile
    uint32_t res_pending = 0;                  // bit i: a residual load into buffer i has not been consumed yet
    uint32_t res_phase = 0;                    // bit i: parity to wait for on res_full[i]
    if (res_staged && etid == 0 && blockIdx.x < total_tiles) {
      const TileCoord t0 = walk.coord(prm);
      ptx::mbar_expect_tx(ptx::smem_u32(&sh->res_full[0]), prm.res_tx_bytes);
      ptx::tma_load_4d(stage0, &tmap_r, ptx::smem_u32(&sh->res_full[0]), t0.k0, t0.q0, t0.p0, t0.n0);
      res_pending = 1u;
    }
    // Lean form of a tile's epilogue, for the shapes the instruction-bound layers have: a staged tile 128 or 64
    // channels wide, residual (if any) staged too.  Straight-line code: no pixel coordinates (the TMA store clips),
    // no predicates around the column groups, the swizzled position of this thread's 16-byte chunks from
    // per-thread constants.  (Chunk c of the staged row r sits at c ^ (r & 7) in a 128-byte row, at c ^ ((r >> 1) & 3)
    // in a 64-byte row: the 16-byte chunk index XOR bits 7.. of the byte offset, masked to the row's chunks.)
    constexpr bool kLeanOk = EpiTraits<EPI>::fast && !kPool && GPW == kGroupsPerWarp && (!EpiTraits<EPI>::res || RSTG == 1);
    const bool lean = kLeanOk && prm.out_stage_bytes != 0 && (prm.BN == 128 || prm.BN == 64);
    const uint32_t lean_col0 = ew < 4 ? 0u : static_cast<uint32_t>(prm.BN) / 2u;          // this warp's half of the columns
    uint32_t lean_off[4];
    {
      const uint32_t row_off = static_cast<uint32_t>(row) * static_cast<uint32_t>(prm.BN);
      const uint32_t swz = ((row_off >> 7) & prm.out_swz_mask) << 4;
#pragma unroll
      for (int i = 0; i < 4; ++i) lean_off[i] = row_off + ((lean_col0 + 16u * i) ^ swz);
    }
    // A warp whose wait expired must not be missing from a later barrier of the eight epilogue warps:
    // it carries `ok == false` to the next barrier, which doubles as a vote, and all leave together.
    for (int tile = blockIdx.x; tile < total_tiles; tile += gridDim.x, ++it, walk.next(prm)) {
      const TileCoord tc = walk.coord(prm);
      const int buf = it & 1;
      const uint32_t use = static_cast<uint32_t>(it >> 1);
      if (res_staged) {
        walk_next.next(prm);
        if (etid == 0 && tile + static_cast<int>(gridDim.x) < total_tiles) {
          // the next tile's buffer was last read by the store issued two tiles ago
          ptx::bulk_wait_read_but_one();
          const int nb = sbuf == 2 ? 0 : sbuf + 1;
          const TileCoord tn = walk_next.coord(prm);
          ptx::mbar_expect_tx(ptx::smem_u32(&sh->res_full[nb]), prm.res_tx_bytes);
          ptx::tma_load_4d(stage0 + static_cast<uint32_t>(nb) * prm.out_stage_bytes, &tmap_r,
                           ptx::smem_u32(&sh->res_full[nb]), tn.k0, tn.q0, tn.p0, tn.n0);
          res_pending |= 1u << nb;
        }
      }
      if (!cst_all) {
        // stage this tile's channel constants, then meet the other epilogue warps
        for (int i = etid; i < prm.BN; i += kEpilogueWarps * 32) {
          if (EpiTraits<EPI>::uni) sh->cst.bias[buf * 256 + i] = __ldg(&chan_table[tc.k0 + i].x);
          else sh->cst.chan[buf * 256 + i] = __ldg(chan_table + tc.k0 + i);
        }
        if (epilogue_vote(!ok)) { ok = false; break; }
      }
      bool row_ok = true;
      size_t pix = 0, pooled_pix = 0;
      if (!lean) {
        const int q = tc.q0 + q_i, p = tc.p0 + p_i, n = tc.n0 + n_i;
        row_ok = (n_i < prm.tn) && q_i < prm.q_step && q < prm.Q && p < prm.P && n < prm.Nimg;
        pix = (static_cast<size_t>(n) * prm.P + p) * prm.Q + q;
        // pooled output pixel of this row's 2 x 2 window (extents P / 2 x Q / 2)
        if (kPool) pooled_pix = (static_cast<size_t>(n) * (prm.P >> 1) + (p >> 1)) * (prm.Q >> 1) + (q >> 1);
      }
      // the residual does not depend on the accumulator: fetch it while the MMAs still run
      uint4 rres[kGroupsPerWarp];                            // (tiles wider than 128 carry no register-fetched residual)
#pragma unroll
      for (int i = 0; i < kGroupsPerWarp; ++i) {
        rres[i] = make_uint4(0u, 0u, 0u, 0u);
        if (EpiTraits<EPI>::res && !res_staged) {
          const int k = tc.k0 + (g_begin + i) * 16;
          if (row_ok && g_begin + i < g_end && k < prm.K)
            rres[i] = __ldg(reinterpret_cast<const uint4*>(res + pix * prm.K + k));
        }
      }
      ok = wait_bounded<64, kHint>(ptx::smem_u32(&sh->acc_full[buf]), use & 1u, wait_limit, sh, status);
      if (res_staged && ok) {
        ok = wait_bounded<32, kHint>(ptx::smem_u32(&sh->res_full[sbuf]), (res_phase >> sbuf) & 1u, wait_limit, sh, status);
        if (ok) res_pending &= ~(1u << sbuf);
        res_phase ^= 1u << sbuf;
      }
      ok = __all_sync(0xffffffffu, ok);
      const bool staged = EpiTraits<EPI>::fast && prm.out_stage_bytes != 0;
      if (!ok && !staged) {
        if (cst_all) break;          // no barrier ahead: this warp may leave by itself
        continue;                    // per-tile constants: meet the others at the next tile's barrier and vote
      }
      // staged tile of this iteration: this thread's row starts at row * BN bytes
      const uint32_t stage_base = stage0 + static_cast<uint32_t>(res_staged ? sbuf : buf) * prm.out_stage_bytes;
      if (ok) {
        ptx::tc_fence_after();
        const uint32_t t_addr = tmem_base + (static_cast<uint32_t>(quad * 32) << 16) +
                                static_cast<uint32_t>(buf * prm.tmem_cols);
        // shared-memory address of this tile's first channel constant (16 bytes per channel, or 4 when
        // only the biases differ)
        const uint32_t chan = cst_addr + static_cast<uint32_t>(cst_all ? tc.k0 : buf * 256) * (EpiTraits<EPI>::uni ? 4u : 16u);
        // This warp's 16-column groups, up to kGroupsPerWarp of them.  Tensor-memory loads run one
        // group ahead of the arithmetic; after the warp's last load the accumulator buffer goes back
        // to the MMA warp.
        auto release = [&]() {
          ptx::tc_fence_before();
          __syncwarp();
          if (lane == 0) ptx::mbar_arrive(ptx::smem_u32(&sh->acc_empty[buf]));
        };
        const uint32_t stage_row = stage_base + static_cast<uint32_t>(row * prm.BN);
        uint32_t acc_a[16], acc_b[16];
        if (kLeanOk && lean) {
          // loads one group ahead of the arithmetic, as below, without the bookkeeping
          const uint32_t t0 = t_addr + lean_col0;
          const uint32_t c0 = chan + lean_col0 * (EpiTraits<EPI>::uni ? 4u : 16u);
          auto group = [&](const uint32_t (&acc)[16], int i) {
            const uint32_t addr = stage_base + lean_off[i];
            uint32_t rw[4] = {0u, 0u, 0u, 0u}, wds[4];
            if (EpiTraits<EPI>::res) {                       // the residual tile was brought there by TMA
              const int4 r4 = lds_int4(addr);
              rw[0] = r4.x; rw[1] = r4.y; rw[2] = r4.z; rw[3] = r4.w;
            }
            convert_16<EPI, RELU>(acc, c0 + static_cast<uint32_t>(i) * (EpiTraits<EPI>::uni ? 64u : 256u), rw, ep, wds);
            ptx::sts_uint4(addr, wds[0], wds[1], wds[2], wds[3]);
          };
          ptx::tmem_ld_32x16(t0, acc_a);
          ptx::tmem_ld_wait();
          ptx::tmem_ld_32x16(t0 + 16, acc_b);
          group(acc_a, 0);
          ptx::tmem_ld_wait();
          if (prm.BN == 128) {
            ptx::tmem_ld_32x16(t0 + 32, acc_a);
            group(acc_b, 1);
            ptx::tmem_ld_wait();
            ptx::tmem_ld_32x16(t0 + 48, acc_b);
            group(acc_a, 2);
            ptx::tmem_ld_wait();
            release();
            group(acc_b, 3);
          } else {                                            // 64 wide: two groups per warp
            release();
            group(acc_b, 1);
          }
        } else {
        if (g_begin < g_end) {
          ptx::tmem_ld_32x16(t_addr + g_begin * 16, acc_a);
          ptx::tmem_ld_wait();
        }
#pragma unroll
        for (int i = 0; i < GPW; i += 2) {
          const int g0 = g_begin + i, g1 = g0 + 1, g2 = g0 + 2;
          if (g0 < g_end) {
            if (g1 < g_end) ptx::tmem_ld_32x16(t_addr + g1 * 16, acc_b); else release();
            if constexpr (kPool) {
              if (tc.k0 + g0 * 16 < prm.K)
                epilogue_pool_16<EPI, RELU>(acc_a, chan, g0 * 16, tc.k0 + g0 * 16, pooled_pix, row_ok, lane, prm.pool_bit, prm, ep, y);
            } else if (row_ok && tc.k0 + g0 * 16 < prm.K)
              epilogue_16<EPI, RELU, RSTG>(acc_a, chan, g0 * 16, tc.k0 + g0 * 16, pix, prm, ep, res, rres[i & (kGroupsPerWarp - 1)], y, stage_row);
            if (g1 < g_end) {
              ptx::tmem_ld_wait();
              if (g2 < g_end && i + 2 < GPW) ptx::tmem_ld_32x16(t_addr + g2 * 16, acc_a); else release();
              if constexpr (kPool) {
                if (tc.k0 + g1 * 16 < prm.K)
                  epilogue_pool_16<EPI, RELU>(acc_b, chan, g1 * 16, tc.k0 + g1 * 16, pooled_pix, row_ok, lane, prm.pool_bit, prm, ep, y);
              } else if (row_ok && tc.k0 + g1 * 16 < prm.K)
                epilogue_16<EPI, RELU, RSTG>(acc_b, chan, g1 * 16, tc.k0 + g1 * 16, pix, prm, ep, res, rres[(i + 1) & (kGroupsPerWarp - 1)], y, stage_row);
              if (g2 < g_end && i + 2 < GPW) ptx::tmem_ld_wait();
            }
          }
        }
        if (g_begin >= g_end) release();                     // a warp without columns still hands back
        }
      }
      if (staged) {
        // The tile is complete in shared memory: one thread hands it to the TMA unit, which writes whole
        // rows (and clips what lies outside the tensor).  Before the barrier that thread makes sure the
        // previous tile's store has finished reading ITS buffer, which is the one the next tile fills.
        // The barrier also carries a vote: if any warp's wait expired, all eight leave together (a
        // warp must never be missing from a later barrier).
        if (etid == 0 && !res_staged) ptx::bulk_wait_read_all();
        ptx::fence_async_smem();
        if (epilogue_vote(!ok)) { ok = false; break; }
        if (etid == 0) {
          ptx::tma_store_4d(&tmap_y, stage_base, tc.k0, tc.q0, tc.p0, tc.n0);
          ptx::bulk_commit();
        }
        sbuf = sbuf == 2 ? 0 : sbuf + 1;
      }
    }
    if (EpiTraits<EPI>::fast && prm.out_stage_bytes && etid == 0) {
      ptx::bulk_wait_all();
      // after an early exit residual tiles may still be on their way into this CTA's shared memory:
      // let them land (bounded) before the CTA retires
      if (res_staged) {
        for (int b = 0; b < 3; ++b)
          for (unsigned int w = 0; w < kDrainPolls && ((res_pending >> b) & 1u); ++w)
            if (ptx::mbar_try_wait(ptx::smem_u32(&sh->res_full[b]), (res_phase >> b) & 1u)) break;
      }
    }
  }
  ptx::tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    ptx::tc_fence_after();
    ptx::tmem_dealloc(tmem_base, static_cast<uint32_t>(2 * prm.tmem_cols));
  }
}

}  // namespace qc

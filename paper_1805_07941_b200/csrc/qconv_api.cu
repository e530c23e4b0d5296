// Host side of the C ABI declared in include/qconv.h: argument validation, the planner that
// maps a layer shape to a kernel and tile shape, weight repacking, TMA descriptors, launches.
#include <cuda.h>
#include <cuda_runtime.h>

#include <algorithm>
#include <cmath>
#include <cstdarg>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <mutex>
#include <vector>

#include "../../include/qconv.h"
#include "epilogue.cuh"
#include "kernel_igemm.cuh"
#include "kernel_dw_tma.cuh"
#include "kernel_igemm_pair.cuh"
#include "kernel_mma_peak.cuh"
#include "kernels_calib.cuh"
#include "kernels_dynfloat.cuh"
#include "kernels_npconv.cuh"
#include "kernels_simple.cuh"
#include "kernels_threshold.cuh"

static_assert(QCALIB_STATIC_MAX_BINS <= qc::kCalibMaxBins, "built-in scratch holds kCalibMaxBins counters");

namespace {

thread_local char g_err[512] = "";

int fail(int code, const char* fmt, ...) {
  va_list ap;
  va_start(ap, fmt);
  vsnprintf(g_err, sizeof(g_err), fmt, ap);
  va_end(ap);
  return code;
}

#define CUDA_TRY(expr)                                                                        \
  do {                                                                                        \
    cudaError_t e_ = (expr);                                                                  \
    if (e_ != cudaSuccess)                                                                    \
      return fail(QCONV_ERR_CUDA, "%s failed: %s", #expr, cudaGetErrorString(e_));            \
  } while (0)

// cuTensorMapEncodeTiled is resolved through the runtime so the library links only cudart.
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*,
                                  CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                  CUtensorMapFloatOOBfill);

EncodeTiledFn get_encode_fn() {
  static EncodeTiledFn fn = nullptr;
  static std::once_flag once;
  std::call_once(once, [] {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) == cudaSuccess &&
        qres == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(p);
  });
  return fn;
}

CUtensorMapSwizzle swizzle_for(int bkc) {
  if (bkc == 0) return CU_TENSOR_MAP_SWIZZLE_NONE;
  return bkc == 128 ? CU_TENSOR_MAP_SWIZZLE_128B : (bkc == 64 ? CU_TENSOR_MAP_SWIZZLE_64B
                                                              : CU_TENSOR_MAP_SWIZZLE_32B);
}

int encode_map(CUtensorMap* map, const void* base, int rank, const cuuint64_t* dims,
               const cuuint64_t* strides_bytes /* rank-1 */, const cuuint32_t* box, int bkc,
               const cuuint32_t* elem_strides = nullptr) {
  EncodeTiledFn fn = get_encode_fn();
  if (!fn) return fail(QCONV_ERR_CUDA, "cuTensorMapEncodeTiled is not available from this driver");
  cuuint32_t estr[5] = {1, 1, 1, 1, 1};
  for (int i = 0; i < rank && elem_strides; ++i) estr[i] = elem_strides[i];
  CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, static_cast<cuuint32_t>(rank), const_cast<void*>(base),
                  dims, strides_bytes, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, swizzle_for(bkc),
                  CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) return fail(QCONV_ERR_CUDA, "cuTensorMapEncodeTiled failed with CUresult %d", (int)r);
  return QCONV_OK;
}

int ceil_div(int a, int b) { return (a + b - 1) / b; }
long ceil_div_l(long a, long b) { return (a + b - 1) / b; }
size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

// Plan overrides of the calling thread (qconv_set_plan_hints); -1 / 0 = the planner decides.
constexpr qconv_plan_hints kNoHints = {-1, -1, -1, -1, -1, -1, -1, -1, -1, -1, -1, -1, -1, -1, 0, 0};
thread_local qconv_plan_hints g_hints = kNoHints;

enum IgemmMode { MODE_FLAT = 0, MODE_VIEW = 1, MODE_BOX = 2, MODE_STEM = 3, MODE_S2D = 4, MODE_WROW = 5 };
// modes whose activation operand is an overlapping window view of a packed, row-padded image
inline bool is_window_mode(int m) { return m == MODE_S2D || m == MODE_WROW; }

}  // namespace

struct qconv_handle {
  qconv_desc d;
  int P, Q, Cg, Kg;
  int algo;                      // resolved QCONV_ALGO_*
  int lo, hi;
  // device copies
  int8_t* d_w = nullptr;         // direct: [R][S][Cg][K]; depthwise: [R*S][C]; igemm: [Kpad][Kg_total]
  int32_t* d_bias = nullptr;
  int32_t* d_shift = nullptr;
  int32_t* d_lshift = nullptr;
  int32_t* d_accexp = nullptr;
  int* d_status = nullptr;
  int4* d_chan = nullptr;        // igemm: per-channel epilogue constants {bias, s, 2^(s-1)-1, s>0}
  long long acc_bound = 0;       // worst-case |accumulator| (Eq. 9 / Eq. 13 bound)
  int max_shift = 0;
  long walk_grid = -1;             // grid size the tile-walk constants in prm were made for
  int flt_epilogue = 0;          // 1: |wide value| < 2^22 for any input (weight-aware bound): float-rounding epilogue
  int uniform_shift = 0;         // 1: all channels share the right shift and the residual left shift
  int uni_s = 0, uni_t = 0;
  int num_sms = 148;
  int ctas_per_sm = 2;
  int use_pdl = 1;
  uint32_t* d_dw_tap = nullptr;  // tap-packed form: weight rows [3][C], bias + magic [C], 2^-s [C], rounding offset [C] (float bits)
  int dw_tap = 0;
  int pair = 0;                  // 1: tiles of 256 pixels x 256 channels on pairs of SMs (kernel_igemm_pair.cuh)
  int fold = 1;                  // flat GEMMs with few output channels: this many pixels form one GEMM row
  int dw_tma = 0;                // rows staged by TMA (C % 32 == 0)
  qc::DwTmaParams dw_prm = {};
  CUtensorMap dw_map;
  const void* dw_key_ptr = nullptr;
  int dw_key_n = -1;
  int8_t* d_pack = nullptr;      // stem: packed patches [N*P*Q][kg_pad]
  int stem_segp = 0;             // stem: bytes per filter-row segment of a packed row (0: taps back to back)
  // stride-2 stem in space-to-depth form: d_pack is [N][s2d_h][s2d_wp] 16-byte block pixels, the image starting
  // at pixel s2d_off_w of a row; the filter covers s2d_r x s2d_s blocks starting s2d_off_h / s2d_off_w blocks
  // up / left of block (p, q)
  int s2d_h = 0, s2d_w = 0, s2d_wp = 0, s2d_off_h = 0, s2d_off_w = 0, s2d_r = 0, s2d_s = 0;
  // MODE_WROW uses the same fields for a stride-1 layer on few channels: d_pack is the image itself with
  // zero-padded rows, a packed pixel is the layer's C bytes (win_pb; 16 for the space-to-depth stems)
  int win_pb = 16;
  // igemm plan
  int mode = 0;
  qc::IgemmParams prm{};
  int kg_pad = 0, kg_total = 0, kpad = 0;
  size_t smem_bytes = 0;
  CUtensorMap tmap_b;
  CUtensorMap tmap_a;
  const void* a_key_ptr = nullptr;
  int a_key_n = -1;
  CUtensorMap tmap_y;            // output tiles leave through TMA stores (fast int8 epilogues)
  const void* y_key_ptr = nullptr;
  int y_key_n = -1;
  CUtensorMap tmap_r;            // residual tiles arrive through TMA loads (same boxes, dense [pixels][K])
  const void* r_key_ptr = nullptr;
  int r_key_n = -1;
  unsigned int wait_limit = 1u << 22;
  cudaStream_t last_stream = nullptr;
  int device = 0;
  qconv_plan_hints hints = kNoHints;   // the creating thread's overrides at create time
};

namespace {

void free_handle(qconv_handle* h) {
  if (!h) return;
  cudaFree(h->d_w);
  cudaFree(h->d_bias);
  cudaFree(h->d_shift);
  cudaFree(h->d_lshift);
  cudaFree(h->d_accexp);
  cudaFree(h->d_status);
  cudaFree(h->d_chan);
  cudaFree(h->d_pack);
  cudaFree(h->d_dw_tap);
  delete h;
}

// Multiplier and shift for the kernel's divisions by d (1 <= d < 2^31), checked against plain division.
qc::FastDiv make_fastdiv(int d_in) {
  qc::FastDiv f = {0u, 0u, static_cast<uint32_t>(std::max(1, d_in))};
  if (f.d > 1u) {
    uint32_t lg = 0;
    while ((1ull << lg) < f.d) ++lg;                       // ceil(log2 d) >= 1
    f.shr = lg - 1;
    f.mul = static_cast<uint32_t>(((1ull << (32 + f.shr)) + f.d - 1) / f.d);
    auto apply = [&](uint32_t n) { return static_cast<uint32_t>((static_cast<unsigned long long>(n) * f.mul) >> 32) >> f.shr; };
    uint32_t probe = 2463534242u;
    for (int i = 0; i < 512; ++i) {
      probe ^= probe << 13; probe ^= probe >> 17; probe ^= probe << 5;
      const uint32_t ns[6] = {static_cast<uint32_t>(i), i * f.d, i * f.d + f.d - 1, probe & 0x7fffffffu, 0x7fffffffu - static_cast<uint32_t>(i),
                              (probe % (1u << 20))};
      for (uint32_t n : ns)
        if (n <= 0x7fffffffu && apply(n) != n / f.d) { f.mul = 0; f.shr = 0; f.d = 0; return f; }   // (never seen; the caller refuses)
    }
  }
  return f;
}

// Output-pixel box (tq x tp x tn <= 128) that wastes the fewest accumulator rows.
// pool: the epilogue takes a 2 x 2 max-pool with warp shuffles, so a window's four pixels must be lanes of one
// warp: tq a power of two up to 16 (rows run q fastest), tp even; Q and P are even.
void choose_box(int Q, int P, int N, int* tq_o, int* tp_o, int* tn_o, bool pool = false, long slots = 0) {
  long best_tiles = -1;
  int btq = 1, btp = 1, btn = 1;
  if (pool) {
    for (int tq = 2; tq <= 16; tq *= 2) {
      for (int tp = 2; tp <= std::min(P, 128 / tq); tp += 2) {
        const int tn = std::max(1, std::min(N, 128 / (tq * tp)));
        const long tiles = static_cast<long>(ceil_div(Q, tq)) * ceil_div(P, tp) * ceil_div(N, tn);
        if (best_tiles < 0 || tiles < best_tiles || (tiles == best_tiles && tq > btq)) {
          best_tiles = tiles; btq = tq; btp = tp; btn = tn;
        }
      }
    }
    *tq_o = btq; *tp_o = btp; *tn_o = btn;
    return;
  }
  // A box may take a patch of several images (a 4-D TMA box of the NHWC tensor): with 28 x 28 outputs, 4 x 4
  // pixels of 8 images fill the 128 accumulator rows where whole image rows (28 x 4) fill 112 -- an eighth fewer
  // tiles, which is what the tensor-bound layers gain (VGG conv3_2 / conv4_x: 10 %).  Fewest tiles win; then the
  // fewest images per box (squarer patches re-read less halo), then the widest patch.
  // slots (0: unknown): tiles that run at the same time.  A layer whose whole-row boxes all run at once gains
  // nothing from fewer tiles and keeps them: their long contiguous runs load a little faster.
  if (slots > 0) {
    long rows_tiles = -1;
    int rq = 1, rp = 1, rn = 1;
    for (int tq = 1; tq <= std::min(Q, 128); ++tq) {
      const int nq = ceil_div(Q, tq);
      if (tq != ceil_div(Q, nq)) continue;
      for (int tp = 1; tp <= std::min(P, 128 / tq); ++tp) {
        const int np = ceil_div(P, tp);
        if (tp != ceil_div(P, np)) continue;
        const int tn = (tq == Q && tp == P) ? std::max(1, std::min(N, 128 / (tq * tp))) : 1;
        const long tiles = static_cast<long>(nq) * np * ceil_div(N, tn);
        if (rows_tiles < 0 || tiles < rows_tiles || (tiles == rows_tiles && tq > rq)) {
          rows_tiles = tiles; rq = tq; rp = tp; rn = tn;
        }
      }
    }
    if (rows_tiles <= slots) {
      *tq_o = rq; *tp_o = rp; *tn_o = rn;
      return;
    }
  }
  for (int tq = 1; tq <= std::min(Q, 128); ++tq) {
    int nq = ceil_div(Q, tq);
    if (tq != ceil_div(Q, nq)) continue;
    int tpmax = std::min(P, 128 / tq);
    for (int tp = 1; tp <= tpmax; ++tp) {
      int np = ceil_div(P, tp);
      if (tp != ceil_div(P, np)) continue;
      const int tn = std::max(1, std::min(N, 128 / (tq * tp)));
      long tiles = static_cast<long>(nq) * np * ceil_div(N, tn);
      if (best_tiles < 0 || tiles < best_tiles || (tiles == best_tiles && (tn < btn || (tn == btn && tq > btq)))) {
        best_tiles = tiles; btq = tq; btp = tp; btn = tn;
      }
    }
  }
  *tq_o = btq; *tp_o = btp; *tn_o = btn;
}

// Bytes of the contraction axis per ring stage.  A stage costs about the same whether its rows are
// 32, 64 or 128 bytes long (the TMA unit works row by row), so the fewest chunks win and zero
// padding is cheap; among equals the narrowest chunk.
int choose_bkc(int c) {
  int best = 128, best_chunks = 1 << 30, best_pad = 1 << 30;
  for (int bkc : {128, 64, 32}) {
    const int chunks = ceil_div(c, bkc), padded = chunks * bkc;
    if (chunks < best_chunks || (chunks == best_chunks && padded < best_pad)) {
      best_chunks = chunks; best_pad = padded; best = bkc;
    }
  }
  return best;
}

typedef void (*IgemmKernel)(const CUtensorMap, const CUtensorMap, const CUtensorMap, const CUtensorMap, const qc::IgemmParams,
                            const qc::EpilogueParams,
                            const int4*, const int8_t*, void*, int*, unsigned int);

IgemmKernel igemm_kernel_for(const qconv_handle* h);
typedef void (*PairKernel)(const CUtensorMap, const CUtensorMap, const qc::PairParams, const qc::IgemmParams,
                           const qc::EpilogueParams, const int4*, void*, int*, unsigned int);
PairKernel pair_kernel_for(const qconv_handle* h);

int plan_igemm(qconv_handle* h, const int8_t* w_krsc /* host [K][R][S][Cg] */, const int32_t* bias_host,
               const int32_t* shift_host, const int32_t* res_lshift_host, const int32_t* acc_exp_host) {
  const qconv_desc& d = h->d;
  const qconv_plan_hints& hint = h->hints;
  qc::IgemmParams& p = h->prm;
  int c_eff = d.C;                 // channels of the GEMM's activation operand
  int taps_r = d.R, taps_s = d.S;
  if (h->mode == MODE_STEM) {
    // packed patch row: either the R*S*C taps back to back, or (when a filter row is at most 28
    // bytes) one 16- or 32-byte segment per filter row, which packs with aligned word copies
    h->stem_segp = d.S * d.C <= 16 ? 16 : (d.S * d.C <= 28 ? 32 : 0);
    const size_t row = h->stem_segp ? static_cast<size_t>(d.R) * h->stem_segp : static_cast<size_t>(d.R) * d.S * d.C;
    h->kg_pad = static_cast<int>(align_up(row, 32));
    c_eff = h->kg_pad;
    taps_r = taps_s = 1;
  }
  if (h->mode == MODE_S2D) {
    // y = 2p - pad + r = 2 (p - off) + j with off = ceil(pad / 2), j = r + 2 off - pad: block rows p - off ...
    h->s2d_off_h = (d.pad_h + 1) / 2;
    h->s2d_off_w = (d.pad_w + 1) / 2;
    h->s2d_r = ceil_div(d.R + 2 * h->s2d_off_h - d.pad_h, 2);
    h->s2d_s = ceil_div(d.S + 2 * h->s2d_off_w - d.pad_w, 2);
    h->s2d_h = ceil_div(d.H, 2);
    h->s2d_w = ceil_div(d.W, 2);
    c_eff = h->s2d_s * 16;         // one GEMM row per filter block row: s2d_s adjacent 16-byte block pixels
    taps_r = h->s2d_r;
    taps_s = 1;
  }
  if (h->mode == MODE_WROW) {
    // Stride 1 on few channels: the S taps of a filter row are S adjacent pixels, contiguous in memory,
    // so one (or two) wide TMA rows replace S narrow ones.  Needs rows padded with zeros left and right
    // (a copy of the image, cheap at these channel counts); rows above / below come from TMA's zero fill.
    // With at most 4 channels the padded copy also widens every pixel to 8 bytes (16 when rows are not
    // folded: a TMA row must start on a 16-byte boundary), zeros after the channels.
    h->win_pb = d.C >= 16 ? d.C : 8;
    h->s2d_off_h = d.pad_h; h->s2d_off_w = d.pad_w;
    h->s2d_r = d.R; h->s2d_s = d.S;
    h->s2d_h = d.H; h->s2d_w = d.W;
    c_eff = d.S * h->win_pb;
    taps_r = d.R;
    taps_s = 1;
  }
  // Narrow layers (K <= 64) would run tiles only K columns wide, and the cost of a tile hardly depends
  // on its width.  Consecutive pixels of a flat GEMM are contiguous in memory, so f of them can be
  // read as ONE row of f * C bytes against block-diagonal weights [f * K][f * C]: the product row is
  // those f pixels' outputs, again contiguous.  Same bytes, 1/f of the rows, tiles f times wider;
  // the extra multiply-adds (zeros) cost the tensor core nothing noticeable at this size.
  h->fold = 1;
  // only with the 16-byte-store epilogues, which index nothing but the (replicated) channel table
  const long long fold_round_room = h->max_shift > 0 ? (1ll << (h->max_shift - 1)) : 0;
  const bool fast_possible = d.out_mode == QCONV_OUT_INT8 && d.rounding == QCONV_ROUND_NEAREST_EVEN && d.n_out == 8 &&
                             h->acc_bound + fold_round_room <= 2147483647ll && hint.fast_epilogue != 0;
  if ((h->mode == MODE_FLAT || h->mode == MODE_STEM) && fast_possible && d.out_c_offset == 0 &&
      d.out_c_pitch == d.K && hint.fold != 0) {
    for (int f = 8; f >= 2; f /= 2) {
      // (a folded row of more than two 128-byte chunks costs more in zero multiply-adds and ring stages than the wider
      // tile saves: ResNet's 256 -> 64 layers 9.1 -> 7.2 us unfolded, inception's 5x5-reduce layers 9-19 % faster)
      if (f * d.K <= 128 && (f * d.K) % 16 == 0 && (h->P * h->Q) % f == 0 && f * c_eff <= 256 &&
          (static_cast<long>(f) * c_eff) % 16 == 0) {
        h->fold = f;
        break;
      }
    }
  }
  if (is_window_mode(h->mode) && fast_possible && d.out_c_offset == 0 && d.out_c_pitch == d.K &&
      hint.fold != 0) {
    // The same folding for the space-to-depth view: a row that starts at block q and spans f + s2d_s - 1
    // blocks holds the windows of the f outputs q ... q + f - 1; the weights repeat along the row, shifted
    // by one block per output (block Toeplitz).  Rows get longer (TMA moves long rows much faster than
    // 32- or 64-byte ones) and f times fewer.
    for (int f = 8; f >= 2; f /= 2) {
      if (f * d.K <= 128 && (f * d.K) % 16 == 0 && h->Q % f == 0 &&
          (f + h->s2d_s - 1) * h->win_pb <= (h->mode == MODE_WROW ? 256 : 128)) {
        h->fold = f;
        break;
      }
    }
  }
  if (h->mode == MODE_WROW && h->win_pb == 8 && h->fold == 1) h->win_pb = 16;
  const int c_row = c_eff;         // bytes of one pixel's GEMM row before folding
  const int k_eff = d.K * h->fold;
  if (is_window_mode(h->mode)) c_eff = (h->fold + h->s2d_s - 1) * h->win_pb;
  else c_eff *= h->fold;
  // Halo form of a 3-tap-wide stride-1 layer on a multiple of 128 channels: one activation box per filter row,
  // W + 2 pixels wide (the halo comes from TMA's zero fill), serves the three horizontal taps -- the tensor core
  // reads the same shared-memory rows shifted by one pixel per tap.  A third of the activation fill traffic.
  const int taps_s_w = taps_s;                             // taps per filter row in the packed weights
  // It costs three weight chunks per stage, so it is used where tiles are 64 channels wide anyway (layers below
  // one wave, which sit at the fill rate), not for the wide tiles of the tensor-bound layers.
  const bool halo_fits = h->mode == MODE_BOX && d.stride_h == 1 && d.stride_w == 1 && d.S == 3 && d.pad_w == 1 && (d.C == 64 || d.C % 128 == 0) &&
                         hint.halo != 0 && d.pool == 0;
  bool halo = false;
  // Its tile: whole image rows with their halo, W + 2 accumulator rows per image row (two of them discarded);
  // an image wider than 126 pixels is cut into equal column segments, each with its own halo.
  const int halo_segs = ceil_div(d.W, qc::kTileM - 2);
  auto halo_box = [&](int* tq, int* tp, int* tn, int* step) {
    *step = ceil_div(d.W, halo_segs);
    *tq = *step + 2;
    *tp = std::max(1, std::min(h->P, qc::kTileM / *tq));
    *tn = (halo_segs == 1 && *tp == h->P) ? std::max(1, std::min(d.N, qc::kTileM / (*tq * *tp))) : 1;
  };
  p.BKC = choose_bkc(c_eff);
  if (is_window_mode(h->mode)) p.BKC = c_eff <= 32 ? 32 : (c_eff <= 64 ? 64 : 128);   // a row is one chunk (two at most)
  p.nchunks = ceil_div(c_eff, p.BKC);
  p.R = taps_r; p.S = taps_s;
  int bn_max = std::min(2 * qc::kGroupsPerWarp * 16, std::max(16, (hint.bn_max > 0 ? hint.bn_max : 128) / 16 * 16));
  cudaDeviceGetAttribute(&h->num_sms, cudaDevAttrMultiProcessorCount, h->device);
  // Tiles 256 channels wide, one CTA per SM: for tensor-bound layers (long contraction, at least 256 output
  // channels, at least one wave of such tiles).  A stage then feeds MMAs of N = 256: three quarters of the
  // operand bytes per multiply-add of a 128-wide tile, and twice the tensor work per stage, which hides
  // the issuing thread's per-stage instructions.  Only the 16-byte-store epilogues without residual exist
  // in this width.
  bool wide = false;
  {
    const bool shape_ok = (h->mode == MODE_BOX || h->mode == MODE_FLAT || h->mode == MODE_VIEW) && h->fold == 1 && fast_possible &&
                          !d.has_residual && d.out_c_pitch % 16 == 0 && d.out_c_offset % 16 == 0 && k_eff % 16 == 0 && k_eff > 128;
    long m_tiles;
    if (h->mode == MODE_FLAT) {
      m_tiles = ceil_div_l(static_cast<long>(d.N) * h->P * h->Q, 128);
    } else {
      int tq, tp, tn;
      choose_box(h->Q, h->P, d.N, &tq, &tp, &tn, d.pool != 0);
      m_tiles = static_cast<long>(ceil_div(h->Q, tq)) * ceil_div(h->P, tp) * ceil_div(d.N, tn);
    }
    const long contraction = static_cast<long>(taps_r) * taps_s * p.nchunks * p.BKC;
    if (hint.bn_max > 128) wide = shape_ok;
    else if (hint.bn_max <= 0)
      wide = shape_ok && k_eff >= 256 && contraction >= 2048 && m_tiles * ceil_div(k_eff, 256) >= h->num_sms;
    if (wide) bn_max = 2 * qc::kGroupsPerWarpWide * 16;
    // ... and, with enough of them, 256-pixel tiles on pairs of SMs (each CTA loads half of the weight rows):
    // half the operand bytes per multiply-add of a 128 x 128 tile
    // (measured: worth it from about four rounds of pair tiles over the SM pairs; below that the 128-pixel
    // tiles balance better)
    h->pair = wide && hint.pair_tiles != 0 &&
              (hint.pair_tiles == 1 || ceil_div_l(m_tiles, 2) * ceil_div(k_eff, 256) >= 4L * (h->num_sms / 2));
  }
  if (hint.bn_max <= 0 && k_eff > 64 && !wide) {
    // A layer with fewer 128-wide tiles than SMs leaves SMs idle while each busy one walks a long
    // chain of MMAs: halve the tile width to spread the work (measured: helps below one wave only).
    long m_tiles;
    if (h->mode == MODE_FLAT || h->mode == MODE_STEM) {
      m_tiles = ceil_div_l(static_cast<long>(d.N) * h->P * h->Q / h->fold, 128);
    } else {
      int tq, tp, tn;
      const int q_rows = is_window_mode(h->mode) ? h->Q / h->fold : h->Q;
      choose_box(q_rows, h->P, d.N, &tq, &tp, &tn, d.pool != 0);
      m_tiles = static_cast<long>(ceil_div(q_rows, tq)) * ceil_div(h->P, tp) * ceil_div(d.N, tn);
    }
    if (m_tiles * ceil_div(k_eff, 128) < h->num_sms) bn_max = 64;
  }
  halo = halo_fits && (bn_max <= 64 || k_eff <= 64 || hint.halo == 1);
  if (halo) {
    wide = false;
    h->pair = 0;
    if (!(hint.halo == 1 && hint.bn_max >= 128)) bn_max = std::min(bn_max, 64);   // three weight chunks per stage: keep the stage small
    taps_s = 1;                                            // what the kernel's stage loop sees
    p.S = 1;
  }
  // Grouped taps: on few channels (rows of at most 64 bytes) a ring stage of ONE tap carries one or two
  // MMAs, far less tensor work than the few hundred cycles of instructions a stage costs the issuing
  // thread.  The S taps of a filter row then share a stage -- S activation boxes side by side, S weight
  // chunks -- and the stage loop runs over filter rows only.
  bool group = !halo && !wide && h->mode == MODE_BOX && d.S >= 2 && d.S <= 4 && p.nchunks == 1 && p.BKC <= 64 &&
               hint.group_taps != 0;
  if (group && hint.group_taps != 1) {
    // ... as long as the fatter stages still form a ring of three, or the weights can stay resident beside
    // two activation stages (the rule applied further down); a ring of two stages costs more than it saves
    const int tk = ceil_div(k_eff, bn_max);
    const int bn = static_cast<int>(align_up(ceil_div(k_eff, tk), 16));
    const int a_tap = static_cast<int>(align_up(static_cast<size_t>(qc::kTileM) * p.BKC, 1024));
    const int b_chunk = static_cast<int>(align_up(static_cast<size_t>(bn) * p.BKC, 1024));
    const int budget = 113 * 1024 - 1024 - static_cast<int>(sizeof(qc::IgemmShared));
    int tq, tp, tn;
    choose_box(h->Q, h->P, d.N, &tq, &tp, &tn, d.pool != 0);
    const long tiles = static_cast<long>(ceil_div(h->Q, tq)) * ceil_div(h->P, tp) * ceil_div(d.N, tn) * tk;
    const int w_bytes = taps_r * d.S * b_chunk;
    const bool resident = hint.resident_weights != 0 && w_bytes <= 72 * 1024 && (budget - w_bytes) / (d.S * a_tap) >= 2 &&
                          tiles > 2L * h->num_sms;
    group = resident || budget / (d.S * (a_tap + b_chunk)) >= 3;
  }
  if (group) {
    taps_s = 1;
    p.S = 1;
  }
  const int tps = halo ? 3 : (group ? d.S : 1);            // taps (weight chunks) per ring stage
  p.halo_s = (halo || group) ? tps : 0;
  p.tap_boxes = group ? 1 : 0;
  p.tiles_k = ceil_div(k_eff, bn_max);
  p.BN = static_cast<int>(align_up(ceil_div(k_eff, p.tiles_k), 16));
  h->kpad = p.tiles_k * p.BN;
  h->kg_total = taps_r * taps_s_w * p.nchunks * p.BKC;
  p.K = k_eff;
  p.out_c_offset = d.out_c_offset;
  p.out_c_pitch = h->fold > 1 ? k_eff : d.out_c_pitch;
  p.tmem_cols = 32;
  while (p.tmem_cols < p.BN) p.tmem_cols *= 2;            // two such buffers are allocated
  cudaDeviceGetAttribute(&h->num_sms, cudaDevAttrMultiProcessorCount, h->device);
  h->ctas_per_sm = hint.ctas_per_sm == 1 ? 1 : 2;
  h->use_pdl = hint.pdl != 0 ? 1 : 0;
  if (2 * p.tmem_cols * h->ctas_per_sm > 512) h->ctas_per_sm = 1;
  if (halo) {
    // A halo-form layer with no more tiles than SMs runs one CTA per SM at most: give that CTA the whole
    // shared memory (its stages are large, and its one chain of stages is as fast as the ring is deep).
    int tq, tp, tn, step;
    halo_box(&tq, &tp, &tn, &step);
    const long m_tiles = static_cast<long>(halo_segs) * ceil_div(h->P, tp) * ceil_div(d.N, tn);
    if (m_tiles * p.tiles_k <= h->num_sms) h->ctas_per_sm = 1;
  }
  p.vec_store = (p.out_c_pitch % 16 == 0 && d.out_c_offset % 16 == 0 && k_eff % 16 == 0) ? 1 : 0;
  const long long round_room = h->max_shift > 0 ? (1ll << (h->max_shift - 1)) : 0;
  p.fast_epilogue = (d.out_mode == QCONV_OUT_INT8 && d.rounding == QCONV_ROUND_NEAREST_EVEN && p.vec_store &&
                     d.n_out == 8 &&
                     h->acc_bound + round_room <= 2147483647ll) ? 1 : 0;
  if (hint.fast_epilogue == 0) p.fast_epilogue = 0;
  // Shared memory: the operand ring, plus -- for the fast epilogues of short contractions, where the
  // epilogue and not the operand ring sets the pace -- staged output tiles that leave by TMA stores:
  // two of them, or three when the residual tile is also brought into them by TMA one tile ahead
  // (as long as the ring keeps enough stages beside them).
  const int full_budget = (h->ctas_per_sm == 2 ? 113 : 226) * 1024 - 1024 - static_cast<int>(sizeof(qc::IgemmShared));
  const int out_tile = static_cast<int>(align_up(static_cast<size_t>(qc::kTileM) * p.BN, 1024));
  auto ring_stages = [&](int bkc, int staged_tiles) {
    const int a = static_cast<int>(align_up(static_cast<size_t>(qc::kTileM + (halo ? 8 : 0)) * bkc, 1024)) * (group ? tps : 1);
    const int b = static_cast<int>(align_up(static_cast<size_t>(h->pair ? p.BN / 2 : p.BN) * bkc, 1024)) * tps;
    return (full_budget - staged_tiles * out_tile) / (a + b);
  };
  const bool force_stage = hint.tma_store == 1;
  const bool short_k = taps_r * taps_s * p.nchunks * p.BKC <= 512;
  p.out_stage_bytes = 0;
  p.out_stage_bufs = 2;
  if (p.BN > 128 && !p.fast_epilogue)
    return fail(QCONV_ERR_UNSUPPORTED_SHAPE, "internal: a tile wider than 128 channels needs a 16-byte-store epilogue");
  // (not for halo tiles of image segments: a staged tile leaves as one box, and the halo's columns are clipped
  // by the tensor's edge only)
  if (p.fast_epilogue && hint.tma_store != 0 && (short_k || force_stage) && p.BN <= 128 && !(halo && halo_segs > 1) && d.pool == 0) {
    const int want[2] = {d.has_residual && h->flt_epilogue && hint.tma_residual != 0 ? 3 : 2, 2};
    for (int w = 0; w < 2 && !p.out_stage_bytes; ++w) {
      const int st = ring_stages(p.BKC, want[w]);
      // (a tile whose operands are one stage needs no second one: the epilogue outlasts the next load)
      if (st >= 1 && (st >= std::min(taps_r * taps_s * p.nchunks, 3) || force_stage)) {
        p.out_stage_bytes = static_cast<uint32_t>(out_tile);
        p.out_stage_bufs = want[w];
      }
    }
  }
  const int staged_tiles = p.out_stage_bytes ? p.out_stage_bufs : 0;
  h->kg_total = taps_r * taps_s_w * p.nchunks * p.BKC;
  // (halo form: the shifted operand reads up to two rows past the 128th, and a stage holds three weight chunks)
  p.a_tap_bytes = static_cast<uint32_t>(align_up(static_cast<size_t>(qc::kTileM + (halo ? 8 : 0)) * p.BKC, 1024));
  p.a_stage_bytes = p.a_tap_bytes * (group ? static_cast<uint32_t>(tps) : 1u);
  p.b_chunk_bytes = static_cast<uint32_t>(align_up(static_cast<size_t>(h->pair ? p.BN / 2 : p.BN) * p.BKC, 1024));
  p.b_stage_bytes = p.b_chunk_bytes * static_cast<uint32_t>(tps);
  p.out_swz_mask = p.BN == 128 ? 7u : (p.BN == 64 ? 3u : (p.BN == 32 ? 1u : 0u));
  int stages = ring_stages(p.BKC, staged_tiles);
  stages = std::max(staged_tiles ? 1 : 2, std::min(stages, qc::kMaxStages));   // the ring runs on across tiles
  // Resident weights: when a CTA walks several tiles and the weight tile of its channel tile (all
  // chunks) is small, load it once -- before the wait on the previous kernel -- and let the ring carry
  // activations only: half the bytes (and TMA rows) per tile for a 128-wide tile, and a deeper ring.
  const int num_kb_plan = taps_r * taps_s * p.nchunks;
  p.b_resident = 0;
  {
    long m_tiles;
    if (h->mode == MODE_FLAT || h->mode == MODE_STEM) {
      m_tiles = ceil_div_l(static_cast<long>(d.N) * h->P * h->Q / h->fold, 128);
    } else {
      int tq, tp, tn;
      const int q_rows = is_window_mode(h->mode) ? h->Q / h->fold : h->Q;
      choose_box(q_rows, h->P, d.N, &tq, &tp, &tn, d.pool != 0);
      m_tiles = static_cast<long>(ceil_div(q_rows, tq)) * ceil_div(h->P, tp) * ceil_div(d.N, tn);
    }
    const long grid_max = static_cast<long>(h->num_sms) * h->ctas_per_sm;
    const int b_res_bytes = num_kb_plan * static_cast<int>(p.b_stage_bytes);
    const int mode_env = hint.resident_weights;                      // 0: never, 1: whenever it fits
    if (mode_env != 0 && !h->pair && (!(halo || group) || p.nchunks == 1) && b_res_bytes <= 72 * 1024 &&
        (m_tiles * p.tiles_k > grid_max || mode_env == 1)) {
      const int st = (full_budget - staged_tiles * out_tile - b_res_bytes) / static_cast<int>(p.a_stage_bytes);
      if (st >= std::min(num_kb_plan + 1, 2)) {
        p.b_resident = 1;
        stages = std::min(st, qc::kMaxStages);
      }
    }
  }
  p.stages = stages;
  h->smem_bytes = 1024 + static_cast<size_t>(stages) * (p.a_stage_bytes + (p.b_resident ? 0 : p.b_stage_bytes)) +
                  (p.b_resident ? static_cast<size_t>(num_kb_plan) * p.b_stage_bytes : 0) +
                  static_cast<size_t>(staged_tiles) * p.out_stage_bytes + sizeof(qc::IgemmShared);
  p.stride_h = p.stride_w = 1;
  p.pad_h = p.pad_w = 0;
  if (h->mode == MODE_FLAT || h->mode == MODE_STEM) {
    p.tq = 128; p.tp = 1; p.tn = 1;
  } else if (h->mode == MODE_VIEW) {
    choose_box(h->Q, h->P, d.N, &p.tq, &p.tp, &p.tn, d.pool != 0, static_cast<long>(h->num_sms) * h->ctas_per_sm / p.tiles_k);
  } else if (is_window_mode(h->mode)) {
    choose_box(h->Q / h->fold, h->P, d.N, &p.tq, &p.tp, &p.tn, d.pool != 0);
    p.pad_h = h->s2d_off_h;        // the horizontal offset is built into the packed rows
    // a row's window may run past the image's last pixel: the packed row is long enough for that
    h->s2d_wp = std::max(h->s2d_off_w + h->s2d_w, h->Q - h->fold + ceil_div(p.nchunks * p.BKC, h->win_pb));
    if (h->win_pb % 16) h->s2d_wp += h->s2d_wp & 1;        // the row pitch in bytes is a multiple of 16 as well
  } else {
    choose_box(h->Q, h->P, d.N, &p.tq, &p.tp, &p.tn, d.pool != 0, static_cast<long>(h->num_sms) * h->ctas_per_sm / p.tiles_k);
    if (halo) halo_box(&p.tq, &p.tp, &p.tn, &p.q_step);
    p.pad_h = d.pad_h; p.pad_w = d.pad_w;
    p.stride_h = d.stride_h; p.stride_w = d.stride_w;
  }
  if (!halo) p.q_step = p.tq;
  p.pool_bit = d.pool ? p.tq : 0;
  if (d.pool && (!p.fast_epilogue || h->mode != MODE_BOX)) {
    return fail(QCONV_ERR_UNSUPPORTED_SHAPE, "pool: needs the tensor-core path with per-tap boxes and an int8 output at 8 bits "
                "with nearest-even rounding, K %% 16 == 0 and an accumulator bound below 2^31 - 2^(s-1)");
  }
  p.tx_bytes = static_cast<uint32_t>((group ? tps : 1) * p.tq * p.tp * p.tn * p.BKC + (p.b_resident ? 0 : tps * p.BN * p.BKC));
  p.b_res_tx_bytes = static_cast<uint32_t>(num_kb_plan * tps * p.BN * p.BKC);
  p.res_tx_bytes = static_cast<uint32_t>(p.tq * p.tp * p.tn * p.BN);

  // weights -> [kpad][kg_total], K-major rows, zero padded
  std::vector<int8_t> wp(static_cast<size_t>(h->kpad) * h->kg_total, 0);
  std::vector<int8_t> row(static_cast<size_t>(std::max(c_row, 1)), 0);
  for (int k = 0; k < d.K; ++k) {
    const int8_t* src = w_krsc + static_cast<size_t>(k) * d.R * d.S * h->Cg;
    if (h->fold > 1 && !is_window_mode(h->mode)) {
      // one pixel's row as the unfolded GEMM would see it, then once per folded pixel on the diagonal
      std::fill(row.begin(), row.end(), 0);
      if (h->mode == MODE_STEM && h->stem_segp) {
        for (int r = 0; r < d.R; ++r)
          std::memcpy(row.data() + static_cast<size_t>(r) * h->stem_segp, src + static_cast<size_t>(r) * d.S * d.C, d.S * d.C);
      } else if (h->mode == MODE_STEM) {
        std::memcpy(row.data(), src, static_cast<size_t>(d.R) * d.S * d.C);
      } else {
        std::memcpy(row.data(), src, d.C);
      }
      for (int j = 0; j < h->fold; ++j)
        std::memcpy(wp.data() + static_cast<size_t>(j * d.K + k) * h->kg_total + static_cast<size_t>(j) * c_row, row.data(), c_row);
      continue;
    }
    int8_t* dst = wp.data() + static_cast<size_t>(k) * h->kg_total;
    if (h->mode == MODE_WROW) {
      // filter row r of folded output j: tap s at pixel j + s of the window, channels as they are
      for (int j = 0; j < h->fold; ++j) {
        int8_t* dj = wp.data() + static_cast<size_t>(j * d.K + k) * h->kg_total;
        for (int r = 0; r < d.R; ++r)
          for (int sx = 0; sx < d.S; ++sx)
            std::memcpy(dj + static_cast<size_t>(r) * p.nchunks * p.BKC + static_cast<size_t>(j + sx) * h->win_pb,
                        src + (static_cast<size_t>(r) * d.S + sx) * d.C, d.C);
      }
      continue;
    }
    if (h->mode == MODE_S2D) {
      // tap (r, s) sits in block row (r + jh) / 2, block column (s + jw) / 2, at sub-pixel ((r + jh) % 2, (s + jw) % 2)
      const int jh = 2 * h->s2d_off_h - d.pad_h, jw = 2 * h->s2d_off_w - d.pad_w;
      for (int j = 0; j < h->fold; ++j) {                  // folded output j of a row: window shifted by j blocks
        int8_t* dj = wp.data() + static_cast<size_t>(j * d.K + k) * h->kg_total;
        for (int r = 0; r < d.R; ++r)
          for (int sx = 0; sx < d.S; ++sx)
            for (int c = 0; c < d.C; ++c) {
              const int jr = r + jh, js = sx + jw;
              dj[static_cast<size_t>(jr / 2) * p.BKC + (j + js / 2) * 16 + ((jr % 2) * 2 + (js % 2)) * d.C + c] =
                  src[(static_cast<size_t>(r) * d.S + sx) * d.C + c];
            }
      }
      continue;
    }
    if (h->mode == MODE_STEM && h->stem_segp) {
      for (int r = 0; r < d.R; ++r)
        std::memcpy(dst + static_cast<size_t>(r) * h->stem_segp, src + static_cast<size_t>(r) * d.S * d.C, d.S * d.C);
    } else if (h->mode == MODE_STEM) {
      std::memcpy(dst, src, static_cast<size_t>(d.R) * d.S * d.C);
    } else {
      for (int t = 0; t < d.R * d.S; ++t)
        std::memcpy(dst + static_cast<size_t>(t) * p.nchunks * p.BKC, src + static_cast<size_t>(t) * d.C, d.C);
    }
  }
  CUDA_TRY(cudaMalloc(&h->d_w, wp.size()));
  CUDA_TRY(cudaMemcpy(h->d_w, wp.data(), wp.size(), cudaMemcpyHostToDevice));
  std::vector<int4> chan(h->kpad, make_int4(0, 0, 0, 0));
  for (int k = 0; k < d.K; ++k) {
    const int sft = shift_host ? shift_host[k] : 0;
    const int t = (d.has_residual && res_lshift_host) ? res_lshift_host[k] : 0;
    chan[k] = make_int4(bias_host ? bias_host[k] : 0, sft, sft > 0 ? (1 << (sft - 1)) - 1 : 0,
                        (sft > 0 ? 1 : 0) | ((1 << t) << 1));
    if (h->flt_epilogue && p.fast_epilogue) {
      // r = (M + v) * 2^-s + M * (1 - 2^-s) with M = 1.5 * 2^23: both constants are exact in binary32
      // for s <= 22; beyond that |v| < 2^22 always rounds to 0, which scale 0 and addend M give
      const float c1 = sft <= 22 ? std::ldexp(1.0f, -sft) : 0.0f;
      const float c2 = static_cast<float>(12582912.0 * (1.0 - static_cast<double>(c1)));
      int c1bits, c2bits;
      std::memcpy(&c1bits, &c1, sizeof(int));
      std::memcpy(&c2bits, &c2, sizeof(int));
      chan[k].x += qc::kMagicBits;
      chan[k].y = c1bits;
      chan[k].z = c2bits;
    }
    if (d.out_mode == QCONV_OUT_FLOAT) chan[k].w = ((acc_exp_host ? acc_exp_host[k] : 0) + 127) << 23;
  }
  for (int j = 1; j < h->fold; ++j)
    for (int k = 0; k < d.K; ++k) chan[static_cast<size_t>(j) * d.K + k] = chan[k];
  CUDA_TRY(cudaMalloc(&h->d_chan, sizeof(int4) * chan.size()));
  CUDA_TRY(cudaMemcpy(h->d_chan, chan.data(), sizeof(int4) * chan.size(), cudaMemcpyHostToDevice));
  cuuint64_t dims[2] = {static_cast<cuuint64_t>(h->kg_total), static_cast<cuuint64_t>(h->kpad)};
  cuuint64_t strides[1] = {static_cast<cuuint64_t>(h->kg_total)};
  cuuint32_t box[2] = {static_cast<cuuint32_t>(p.BKC), static_cast<cuuint32_t>(h->pair ? p.BN / 2 : p.BN)};
  int rc = encode_map(&h->tmap_b, h->d_w, 2, dims, strides, box, p.BKC);
  if (rc) return rc;
  if (is_window_mode(h->mode)) {
    const size_t bytes = static_cast<size_t>(d.N) * h->s2d_h * h->s2d_wp * h->win_pb;
    CUDA_TRY(cudaMalloc(&h->d_pack, bytes));
    CUDA_TRY(cudaMemset(h->d_pack, 0, bytes));             // padding pixels and ragged edges stay zero
  }
  if (h->mode == MODE_STEM) {
    const size_t bytes = static_cast<size_t>(d.N) * h->P * h->Q * h->kg_pad;
    CUDA_TRY(cudaMalloc(&h->d_pack, bytes));
    CUDA_TRY(cudaMemset(h->d_pack, 0, bytes));             // padding bytes of each row stay zero
  }
  // the attribute belongs to the current device: once per device, not once per process
  static std::once_flag attr_once[64];
  static cudaError_t attr_err = cudaSuccess;
  std::call_once(attr_once[h->device & 63], [] {
    for (IgemmKernel k : {static_cast<IgemmKernel>(qc::igemm_i8_kernel<qc::EPI_FAST_I8>),
                          static_cast<IgemmKernel>(qc::igemm_i8_kernel<qc::EPI_FAST_I8_RES>),
                          static_cast<IgemmKernel>(qc::igemm_i8_kernel<qc::EPI_FLT_I8, 0>),
                          static_cast<IgemmKernel>(qc::igemm_i8_kernel<qc::EPI_FLT_I8_RES, 0>),
                          static_cast<IgemmKernel>(qc::igemm_i8_kernel<qc::EPI_FLT_I8_U, 0>),
                          static_cast<IgemmKernel>(qc::igemm_i8_kernel<qc::EPI_FLT_I8_RES_U, 0>),
                          static_cast<IgemmKernel>(qc::igemm_i8_kernel<qc::EPI_FLT_I8, 1>),
                          static_cast<IgemmKernel>(qc::igemm_i8_kernel<qc::EPI_FLT_I8_RES, 1>),
                          static_cast<IgemmKernel>(qc::igemm_i8_kernel<qc::EPI_FLT_I8_U, 1>),
                          static_cast<IgemmKernel>(qc::igemm_i8_kernel<qc::EPI_FLT_I8_RES_U, 1>),
                          static_cast<IgemmKernel>(qc::igemm_i8_kernel<qc::EPI_FLT_I8_RES, 0, 1>),
                          static_cast<IgemmKernel>(qc::igemm_i8_kernel<qc::EPI_FLT_I8_RES_U, 0, 1>),
                          static_cast<IgemmKernel>(qc::igemm_i8_kernel<qc::EPI_FLT_I8_RES, 1, 1>),
                          static_cast<IgemmKernel>(qc::igemm_i8_kernel<qc::EPI_FLT_I8_RES_U, 1, 1>),
                          static_cast<IgemmKernel>(qc::igemm_i8_kernel<qc::EPI_FAST_I8_U>),
                          static_cast<IgemmKernel>(qc::igemm_i8_kernel<qc::EPI_FAST_I8_RES_U>),
                          static_cast<IgemmKernel>(qc::igemm_i8_kernel<qc::EPI_FLT_I8_U, 1, 0, qc::kGroupsPerWarpWide>),
                          static_cast<IgemmKernel>(qc::igemm_i8_kernel<qc::EPI_FLT_I8, 1, 0, qc::kGroupsPerWarpWide>),
                          static_cast<IgemmKernel>(qc::igemm_i8_kernel<qc::EPI_FLT_I8_U, 0, 0, qc::kGroupsPerWarpWide>),
                          static_cast<IgemmKernel>(qc::igemm_i8_kernel<qc::EPI_FLT_I8, 0, 0, qc::kGroupsPerWarpWide>),
                          static_cast<IgemmKernel>(qc::igemm_i8_kernel<qc::EPI_FAST_I8_U, 2, 0, qc::kGroupsPerWarpWide>),
                          static_cast<IgemmKernel>(qc::igemm_i8_kernel<qc::EPI_FAST_I8, 2, 0, qc::kGroupsPerWarpWide>),
                          static_cast<IgemmKernel>(qc::igemm_i8_kernel<qc::EPI_I8>),
                          static_cast<IgemmKernel>(qc::igemm_i8_kernel<qc::EPI_I32>),
                          static_cast<IgemmKernel>(qc::igemm_i8_kernel<qc::EPI_F32>)}) {
      cudaError_t e = cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024);
      if (e != cudaSuccess) attr_err = e;
    }
  });
  if (attr_err != cudaSuccess)
    return fail(QCONV_ERR_CUDA, "cudaFuncSetAttribute: %s", cudaGetErrorString(attr_err));
  if (h->pair) {
    PairKernel pk = pair_kernel_for(h);
    CUDA_TRY(cudaFuncSetAttribute(pk, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024));
  } else if (d.pool) {
    CUDA_TRY(cudaFuncSetAttribute(igemm_kernel_for(h), cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024));
  }
  return QCONV_OK;
}

PairKernel pair_kernel_for(const qconv_handle* h) {
  const bool uni = h->uniform_shift && h->hints.uniform_shift != 0;
  if (h->d.pool) {
    if (h->flt_epilogue) return uni ? qc::igemm_i8_pair_kernel<qc::EPI_FLT_I8_U, 2, 1> : qc::igemm_i8_pair_kernel<qc::EPI_FLT_I8, 2, 1>;
    return uni ? qc::igemm_i8_pair_kernel<qc::EPI_FAST_I8_U, 2, 1> : qc::igemm_i8_pair_kernel<qc::EPI_FAST_I8, 2, 1>;
  }
  if (h->flt_epilogue) {
    if (h->d.relu) return uni ? qc::igemm_i8_pair_kernel<qc::EPI_FLT_I8_U, 1> : qc::igemm_i8_pair_kernel<qc::EPI_FLT_I8, 1>;
    return uni ? qc::igemm_i8_pair_kernel<qc::EPI_FLT_I8_U, 0> : qc::igemm_i8_pair_kernel<qc::EPI_FLT_I8, 0>;
  }
  return uni ? qc::igemm_i8_pair_kernel<qc::EPI_FAST_I8_U, 2> : qc::igemm_i8_pair_kernel<qc::EPI_FAST_I8, 2>;
}

IgemmKernel igemm_kernel_for(const qconv_handle* h) {
  if (h->d.out_mode == QCONV_OUT_INT32) return qc::igemm_i8_kernel<qc::EPI_I32>;
  if (h->d.out_mode == QCONV_OUT_FLOAT) return qc::igemm_i8_kernel<qc::EPI_F32>;
  if (!h->prm.fast_epilogue) return qc::igemm_i8_kernel<qc::EPI_I8>;
  const bool uni = h->uniform_shift && h->hints.uniform_shift != 0;
  if (h->d.pool) {                                         // 2 x 2 max-pool in the epilogue (ReLU read at run time)
    constexpr int W = qc::kGroupsPerWarpWide;
    if (h->prm.BN > 128) {
      if (h->flt_epilogue) return uni ? qc::igemm_i8_kernel<qc::EPI_FLT_I8_U, 2, 2, W> : qc::igemm_i8_kernel<qc::EPI_FLT_I8, 2, 2, W>;
      return uni ? qc::igemm_i8_kernel<qc::EPI_FAST_I8_U, 2, 2, W> : qc::igemm_i8_kernel<qc::EPI_FAST_I8, 2, 2, W>;
    }
    if (h->flt_epilogue) return uni ? qc::igemm_i8_kernel<qc::EPI_FLT_I8_U, 2, 2> : qc::igemm_i8_kernel<qc::EPI_FLT_I8, 2, 2>;
    return uni ? qc::igemm_i8_kernel<qc::EPI_FAST_I8_U, 2, 2> : qc::igemm_i8_kernel<qc::EPI_FAST_I8, 2, 2>;
  }
  if (h->prm.BN > 128) {                                   // 256-wide tiles: no residual (the planner saw to that)
    constexpr int W = qc::kGroupsPerWarpWide;
    if (h->flt_epilogue) {
      if (h->d.relu) return uni ? qc::igemm_i8_kernel<qc::EPI_FLT_I8_U, 1, 0, W> : qc::igemm_i8_kernel<qc::EPI_FLT_I8, 1, 0, W>;
      return uni ? qc::igemm_i8_kernel<qc::EPI_FLT_I8_U, 0, 0, W> : qc::igemm_i8_kernel<qc::EPI_FLT_I8, 0, 0, W>;
    }
    return uni ? qc::igemm_i8_kernel<qc::EPI_FAST_I8_U, 2, 0, W> : qc::igemm_i8_kernel<qc::EPI_FAST_I8, 2, 0, W>;
  }
  if (h->flt_epilogue) {
    const bool res = h->d.has_residual != 0;
    if (res && h->prm.out_stage_bytes && h->prm.out_stage_bufs == 3) {      // residual tiles arrive by TMA
      if (h->d.relu) return uni ? qc::igemm_i8_kernel<qc::EPI_FLT_I8_RES_U, 1, 1> : qc::igemm_i8_kernel<qc::EPI_FLT_I8_RES, 1, 1>;
      return uni ? qc::igemm_i8_kernel<qc::EPI_FLT_I8_RES_U, 0, 1> : qc::igemm_i8_kernel<qc::EPI_FLT_I8_RES, 0, 1>;
    }
    if (h->d.relu) {
      if (uni) return res ? qc::igemm_i8_kernel<qc::EPI_FLT_I8_RES_U, 1> : qc::igemm_i8_kernel<qc::EPI_FLT_I8_U, 1>;
      return res ? qc::igemm_i8_kernel<qc::EPI_FLT_I8_RES, 1> : qc::igemm_i8_kernel<qc::EPI_FLT_I8, 1>;
    }
    if (uni) return res ? qc::igemm_i8_kernel<qc::EPI_FLT_I8_RES_U, 0> : qc::igemm_i8_kernel<qc::EPI_FLT_I8_U, 0>;
    return res ? qc::igemm_i8_kernel<qc::EPI_FLT_I8_RES, 0> : qc::igemm_i8_kernel<qc::EPI_FLT_I8, 0>;
  }
  if (uni)
    return h->d.has_residual ? qc::igemm_i8_kernel<qc::EPI_FAST_I8_RES_U> : qc::igemm_i8_kernel<qc::EPI_FAST_I8_U>;
  return h->d.has_residual ? qc::igemm_i8_kernel<qc::EPI_FAST_I8_RES> : qc::igemm_i8_kernel<qc::EPI_FAST_I8>;
}

// Activation tensor map and tile counts for this run (depends on the pointer and n_run).
int prepare_a_map(qconv_handle* h, const int8_t* a_ptr, int n_run) {
  if (h->a_key_ptr == a_ptr && h->a_key_n == n_run) return QCONV_OK;
  const qconv_desc& d = h->d;
  qc::IgemmParams& p = h->prm;
  cuuint64_t dims[4], strides[3];
  cuuint32_t estr[4] = {1, 1, 1, 1};
  cuuint32_t box[4] = {static_cast<cuuint32_t>(p.BKC), static_cast<cuuint32_t>(p.tq),
                       static_cast<cuuint32_t>(p.tp), static_cast<cuuint32_t>(p.tn)};
  if (h->mode == MODE_FLAT || h->mode == MODE_STEM) {
    const cuuint64_t c = static_cast<cuuint64_t>(h->mode == MODE_STEM ? h->kg_pad : d.C) * h->fold;
    const cuuint64_t m = static_cast<cuuint64_t>(n_run) * h->P * h->Q / h->fold;
    dims[0] = c; dims[1] = m; dims[2] = 1; dims[3] = 1;
    strides[0] = c; strides[1] = m * c; strides[2] = m * c;
    p.Q = static_cast<int>(m); p.P = 1; p.Nimg = 1;
  } else if (is_window_mode(h->mode)) {
    // overlapping view of the packed block pixels: GEMM row q of a filter block row is the BKC bytes that
    // start at packed pixel q (pitch 16 bytes), i.e. blocks q - off_w ... of the image
    const cuuint64_t pb = static_cast<cuuint64_t>(h->win_pb);
    dims[0] = static_cast<cuuint64_t>(p.nchunks) * p.BKC; dims[1] = h->Q / h->fold; dims[2] = h->s2d_h; dims[3] = n_run;
    strides[0] = pb * h->fold;
    strides[1] = pb * h->s2d_wp;
    strides[2] = pb * h->s2d_wp * h->s2d_h;
    p.Q = h->Q / h->fold; p.P = h->P; p.Nimg = n_run;
  } else if (h->mode == MODE_VIEW) {
    dims[0] = d.C; dims[1] = h->Q; dims[2] = h->P; dims[3] = n_run;
    strides[0] = static_cast<cuuint64_t>(d.stride_w) * d.C;
    strides[1] = static_cast<cuuint64_t>(d.stride_h) * d.W * d.C;
    strides[2] = static_cast<cuuint64_t>(d.H) * d.W * d.C;
    p.Q = h->Q; p.P = h->P; p.Nimg = n_run;
  } else {
    dims[0] = d.C; dims[1] = d.W; dims[2] = d.H; dims[3] = n_run;
    strides[0] = d.C;
    strides[1] = static_cast<cuuint64_t>(d.W) * d.C;
    strides[2] = static_cast<cuuint64_t>(d.H) * d.W * d.C;
    p.Q = h->Q; p.P = h->P; p.Nimg = n_run;
    // strided filters: the box spans (t - 1) * stride + 1 input pixels per axis and the copy engine keeps
    // every stride-th one (traversal strides of the tensor map), so the tile still has tq x tp rows
    estr[1] = static_cast<cuuint32_t>(d.stride_w); estr[2] = static_cast<cuuint32_t>(d.stride_h);
    box[1] = static_cast<cuuint32_t>((p.tq - 1) * d.stride_w + 1);
    box[2] = static_cast<cuuint32_t>((p.tp - 1) * d.stride_h + 1);
    if (p.halo_s && !p.tap_boxes) box[1] = static_cast<cuuint32_t>(p.tq);
  }
  p.tiles_q = ceil_div(p.Q, p.q_step);
  p.tiles_p = ceil_div(p.P, p.tp);
  p.tiles_n = ceil_div(p.Nimg, p.tn);
  h->walk_grid = -1;                                       // the walk's digits depend on the tile counts too
  p.fd_tiles_k = make_fastdiv(p.tiles_k); p.fd_tiles_q = make_fastdiv(p.tiles_q); p.fd_tiles_p = make_fastdiv(p.tiles_p);
  p.fd_tq = make_fastdiv(p.tq); p.fd_tp = make_fastdiv(p.tp);
  p.fd_nchunks = make_fastdiv(p.nchunks); p.fd_S = make_fastdiv(p.S);
  if (!p.fd_tiles_k.d || !p.fd_tiles_q.d || !p.fd_tiles_p.d || !p.fd_tq.d || !p.fd_tp.d || !p.fd_nchunks.d || !p.fd_S.d)
    return fail(QCONV_ERR_UNSUPPORTED_SHAPE, "internal: division constants failed their check");
  int rc = encode_map(&h->tmap_a, a_ptr, 4, dims, strides, box, p.BKC, estr);
  if (rc) return rc;
  h->a_key_ptr = a_ptr;
  h->a_key_n = n_run;
  return QCONV_OK;
}

// Output tensor map for the TMA stores of the fast epilogues: the same pixel boxes as the accumulator
// rows (q fastest, then p, then image), BN channels wide, over the caller's buffer with its channel
// offset and pitch.  Must follow prepare_a_map (which sets the run's pixel extents).
int prepare_y_map(qconv_handle* h, const void* y_ptr, int n_run) {
  if (h->y_key_ptr == y_ptr && h->y_key_n == n_run) return QCONV_OK;
  const qc::IgemmParams& p = h->prm;
  const cuuint64_t pitch = static_cast<cuuint64_t>(p.out_c_pitch);
  cuuint64_t dims[4] = {static_cast<cuuint64_t>(p.K), static_cast<cuuint64_t>(p.Q), static_cast<cuuint64_t>(p.P),
                        static_cast<cuuint64_t>(p.Nimg)};
  cuuint64_t strides[3] = {pitch, pitch * p.Q, pitch * p.Q * p.P};
  cuuint32_t box[4] = {static_cast<cuuint32_t>(p.BN), static_cast<cuuint32_t>(p.tq), static_cast<cuuint32_t>(p.tp),
                       static_cast<cuuint32_t>(p.tn)};
  const int swz = (p.BN == 128 || p.BN == 64 || p.BN == 32) ? p.BN : 0;
  int rc = encode_map(&h->tmap_y, static_cast<const int8_t*>(y_ptr) + p.out_c_offset, 4, dims, strides, box, swz);
  if (rc) return rc;
  h->y_key_ptr = y_ptr;
  h->y_key_n = n_run;
  return QCONV_OK;
}

int prepare_r_map(qconv_handle* h, const void* r_ptr, int n_run) {
  if (h->r_key_ptr == r_ptr && h->r_key_n == n_run) return QCONV_OK;
  const qc::IgemmParams& p = h->prm;
  const cuuint64_t pitch = static_cast<cuuint64_t>(p.K);
  cuuint64_t dims[4] = {static_cast<cuuint64_t>(p.K), static_cast<cuuint64_t>(p.Q), static_cast<cuuint64_t>(p.P),
                        static_cast<cuuint64_t>(p.Nimg)};
  cuuint64_t strides[3] = {pitch, pitch * p.Q, pitch * p.Q * p.P};
  cuuint32_t box[4] = {static_cast<cuuint32_t>(p.BN), static_cast<cuuint32_t>(p.tq), static_cast<cuuint32_t>(p.tp),
                       static_cast<cuuint32_t>(p.tn)};
  const int swz = (p.BN == 128 || p.BN == 64 || p.BN == 32) ? p.BN : 0;
  int rc = encode_map(&h->tmap_r, r_ptr, 4, dims, strides, box, swz);
  if (rc) return rc;
  h->r_key_ptr = r_ptr;
  h->r_key_n = n_run;
  return QCONV_OK;
}

// Tile shape of the TMA-staged depthwise kernel: the channel width of a CTA trades idle columns
// (few wide column groups on a narrow image) against halo re-reads (many narrow ones).
void plan_dw_tma(qconv_handle* h) {
  const qconv_desc& d = h->d;
  const int st = d.stride_h;
  double best = 0.0;
  qc::DwTmaParams bp = {};
  for (int cwb = 8; cwb <= 128 && cwb * 4 <= d.C; cwb *= 2) {
    if ((d.C / 4) % cwb) continue;
    qc::DwTmaParams p = {};
    p.cwb = cwb;
    p.cwb_box = std::min(cwb, 64);
    p.nbox = cwb / p.cwb_box;
    const int qt_max = qc::kDwConsumers / cwb;
    p.q_blocks = ceil_div(ceil_div(h->Q, 4), qt_max);
    p.qt_per_cta = ceil_div(ceil_div(h->Q, 4), p.q_blocks);          // even split, no more columns than needed
    p.consumers = ceil_div(p.qt_per_cta * cwb, 32) * 32;
    p.pix = 4 * p.qt_per_cta * st + 3 - st;
    if (p.pix > 256) continue;
    p.box_words = p.pix * p.cwb_box;
    p.row_bytes = p.nbox * p.box_words * 4;
    p.stage_bytes = static_cast<int>(align_up(p.row_bytes, 128));
    const double threads = static_cast<double>(p.q_blocks) * p.qt_per_cta * 4 / h->Q;     // >= 1: idle columns
    const double bytes = static_cast<double>(p.q_blocks) * p.pix / (static_cast<double>(h->Q) * st);   // >= 1: halo + overhang
    const double cost = threads * bytes;
    if (bp.cwb == 0 || cost <= best) { best = cost; bp = p; }
  }
  if (bp.cwb == 0) return;
  while ((1 << bp.cwb_log2) < bp.cwb) ++bp.cwb_log2;
  while ((1 << bp.cwb_box_log2) < bp.cwb_box) ++bp.cwb_box_log2;
  bp.fd_q_blocks = make_fastdiv(bp.q_blocks);
  if (!bp.fd_q_blocks.d) return;
  h->dw_prm = bp;
  h->dw_tma = 1;
}

int prepare_dw_map(qconv_handle* h, const int8_t* x, int n_run) {
  if (h->dw_key_ptr == x && h->dw_key_n == n_run) return QCONV_OK;
  const qconv_desc& d = h->d;
  cuuint64_t dims[4] = {static_cast<cuuint64_t>(d.C), static_cast<cuuint64_t>(d.W), static_cast<cuuint64_t>(d.H),
                        static_cast<cuuint64_t>(n_run)};
  cuuint64_t strides[3] = {static_cast<cuuint64_t>(d.C), static_cast<cuuint64_t>(d.W) * d.C,
                           static_cast<cuuint64_t>(d.H) * d.W * d.C};
  cuuint32_t box[4] = {static_cast<cuuint32_t>(h->dw_prm.cwb_box * 4), static_cast<cuuint32_t>(h->dw_prm.pix), 1, 1};
  int rc = encode_map(&h->dw_map, x, 4, dims, strides, box, 0);
  if (rc) return rc;
  h->dw_key_ptr = x;
  h->dw_key_n = n_run;
  return QCONV_OK;
}

// Launch with the programmatic-dependent-launch attribute (the kernel must call qc::chain_sync first).
template <typename... KArgs, typename... Args>
cudaError_t launch_chained(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = g_hints.pdl != 0 ? 1 : 0;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

int grid_for(size_t work_items, int threads, int max_blocks) {
  size_t b = (work_items + threads - 1) / threads;
  return static_cast<int>(std::max<size_t>(1, std::min<size_t>(b, max_blocks)));
}

}  // namespace

extern "C" {

const char* qconv_last_error_string(void) { return g_err; }

int qconv_checked_faults(int* first_line_out) {
  int v[2] = {0, 0};
#ifdef QCONV_CHECKED
  if (cudaDeviceSynchronize() != cudaSuccess ||
      cudaMemcpyFromSymbol(v, qc::g_checked_fault, sizeof(v)) != cudaSuccess)
    return fail(QCONV_ERR_CUDA, "qconv_checked_faults: cannot read the fault word");
  const int zero[2] = {0, 0};
  cudaMemcpyToSymbol(qc::g_checked_fault, zero, sizeof(zero));
#else
  v[0] = -1;                                               // not a checked build
#endif
  if (first_line_out) *first_line_out = v[1];
  return v[0];
}

int qconv_set_plan_hints(const qconv_plan_hints* hints) {
  g_hints = hints ? *hints : kNoHints;
  return QCONV_OK;
}

int qconv_create(qconv_handle** out, const qconv_desc* desc, const int8_t* w_host,
                 const int32_t* bias_host, const int32_t* shift_host,
                 const int32_t* res_lshift_host, const int32_t* acc_exp_host) {
  if (!out) return fail(QCONV_ERR_BAD_ARG, "out is NULL");
  *out = nullptr;
  if (!desc || !w_host) return fail(QCONV_ERR_BAD_ARG, "desc or w_host is NULL");
  qconv_desc d = *desc;
  if (d.N <= 0 || d.H <= 0 || d.W <= 0 || d.C <= 0 || d.K <= 0 || d.R <= 0 || d.S <= 0 ||
      d.stride_h <= 0 || d.stride_w <= 0 || d.pad_h < 0 || d.pad_w < 0 || d.groups <= 0)
    return fail(QCONV_ERR_BAD_ARG, "non-positive dimension in descriptor");
  if (d.n_in < 2 || d.n_in > 8 || d.n_w < 2 || d.n_w > 8 || d.n_out < 2 || d.n_out > 8)
    return fail(QCONV_ERR_BAD_ARG, "bit widths must be in [2, 8]");
  if (d.rounding < 0 || d.rounding > 3 || d.out_mode < 0 || d.out_mode > 2 || d.weight_layout < 0 ||
      d.weight_layout > 1 || d.algo < 0 || d.algo > 3)
    return fail(QCONV_ERR_BAD_ARG, "unknown enum value in descriptor");
  if (d.C % d.groups || d.K % d.groups)
    return fail(QCONV_ERR_UNSUPPORTED_SHAPE, "groups must divide C and K");
  const int P = (d.H + 2 * d.pad_h - d.R) / d.stride_h + 1;
  const int Q = (d.W + 2 * d.pad_w - d.S) / d.stride_w + 1;
  if (d.H + 2 * d.pad_h < d.R || d.W + 2 * d.pad_w < d.S || P <= 0 || Q <= 0)
    return fail(QCONV_ERR_UNSUPPORTED_SHAPE, "filter larger than padded input");
  if (d.out_c_pitch == 0) d.out_c_pitch = d.K;
  if (d.out_c_offset < 0 || d.out_c_offset + d.K > d.out_c_pitch)
    return fail(QCONV_ERR_BAD_ARG, "output channel window [%d, %d) exceeds pitch %d", d.out_c_offset,
                d.out_c_offset + d.K, d.out_c_pitch);
  if (static_cast<size_t>(d.N) * P * Q * d.out_c_pitch >= (1ull << 40) ||
      static_cast<size_t>(d.N) * d.H * d.W * d.C >= (1ull << 40))
    return fail(QCONV_ERR_UNSUPPORTED_SHAPE, "tensor too large");
  if (d.has_residual && !res_lshift_host)
    return fail(QCONV_ERR_BAD_ARG, "has_residual needs res_lshift_host");
  if (d.pool != 0 && d.pool != 2) return fail(QCONV_ERR_BAD_ARG, "pool must be 0 or 2");
  if (d.pool && (d.has_residual || d.out_mode != QCONV_OUT_INT8 || (P & 1) || (Q & 1) || d.groups != 1))
    return fail(QCONV_ERR_UNSUPPORTED_SHAPE, "pool: needs groups == 1, int8 output, no residual, even P and Q");
  const int Cg = d.C / d.groups;
  int max_t = 0;
  int64_t max_bias = 0;
  for (int k = 0; k < d.K; ++k) {
    if (shift_host && (shift_host[k] < 0 || shift_host[k] > 31))
      return fail(QCONV_ERR_BAD_SHIFT, "shift[%d] = %d outside [0, 31]", k, shift_host[k]);
    if (d.has_residual) {
      if (res_lshift_host[k] < 0 || res_lshift_host[k] > 23)
        return fail(QCONV_ERR_RESIDUAL_SCALE, "res_lshift[%d] = %d outside [0, 23]", k, res_lshift_host[k]);
      max_t = std::max(max_t, res_lshift_host[k]);
    }
    if (bias_host) max_bias = std::max<int64_t>(max_bias, std::llabs(static_cast<int64_t>(bias_host[k])));
    if (acc_exp_host && (acc_exp_host[k] < -126 || acc_exp_host[k] > 96))
      return fail(QCONV_ERR_BAD_ARG, "acc_exp[%d] = %d outside [-126, 96]", k, acc_exp_host[k]);
  }
  // Eq. 9 / Eq. 13: the longest sum must fit a 32-bit two's-complement accumulator.
  const int64_t bound = static_cast<int64_t>(d.R) * d.S * Cg * (1ll << (d.n_in - 1)) * (1ll << (d.n_w - 1)) +
                        max_bias + (d.has_residual ? (128ll << max_t) : 0);
  if (bound > 2147483647ll)
    return fail(QCONV_ERR_OVERFLOW_RISK, "worst-case |accumulator| %lld exceeds 2^31 - 1", (long long)bound);

  qconv_handle* h = new qconv_handle();
  h->hints = g_hints;
  h->d = d;
  h->P = P; h->Q = Q; h->Cg = Cg; h->Kg = d.K / d.groups;
  h->acc_bound = bound;
  h->uniform_shift = 1;
  h->uni_s = shift_host ? shift_host[0] : 0;
  h->uni_t = d.has_residual ? res_lshift_host[0] : 0;
  for (int k = 0; k < d.K; ++k) {
    if ((shift_host ? shift_host[k] : 0) != h->uni_s) h->uniform_shift = 0;
    if (d.has_residual && res_lshift_host[k] != h->uni_t) h->uniform_shift = 0;
  }
  for (int k = 0; k < d.K && shift_host; ++k) h->max_shift = std::max(h->max_shift, shift_host[k]);
  h->hi = (1 << (d.n_out - 1)) - 1;
  h->lo = d.symmetric ? -h->hi : -(1 << (d.n_out - 1));
  cudaGetDevice(&h->device);
  cudaDeviceGetAttribute(&h->num_sms, cudaDevAttrMultiProcessorCount, h->device);

  // weights to [K][R][S][Cg] on the host
  const size_t wcount = static_cast<size_t>(d.K) * d.R * d.S * Cg;
  std::vector<int8_t> w_krsc(wcount);
  if (d.weight_layout == 0) {
    std::memcpy(w_krsc.data(), w_host, wcount);
  } else {
    const size_t per_k = static_cast<size_t>(d.R) * d.S * Cg;
    for (int k = 0; k < d.K; ++k)
      for (size_t j = 0; j < per_k; ++j) w_krsc[k * per_k + j] = w_host[j * d.K + k];
  }

  // Weight-aware bound of the wide value: 2^(n_in-1) * sum|w[k,.]| + |bias[k]| + 128 * 2^t[k].  Below 2^22 the
  // tensor-core epilogue may round in fp32 (exactly).
  {
    long long worst = 0;
    const size_t per_k = static_cast<size_t>(d.R) * d.S * Cg;
    for (int k = 0; k < d.K; ++k) {
      long long sw = 0;
      for (size_t j = 0; j < per_k; ++j) sw += std::abs(static_cast<int>(w_krsc[k * per_k + j]));
      long long bnd = sw * (1ll << (d.n_in - 1)) + (bias_host ? std::llabs(static_cast<long long>(bias_host[k])) : 0) +
                      (d.has_residual ? (128ll << res_lshift_host[k]) : 0);
      worst = std::max(worst, bnd);
    }
    h->flt_epilogue = (worst < (1ll << 22)) && h->hints.float_rounding != 0;
  }

  // choose the algorithm
  const bool dw_ok = d.groups == d.C && d.C == d.K && d.R == 3 && d.S == 3 && d.stride_h == d.stride_w &&
                     (d.stride_h == 1 || d.stride_h == 2) && d.C % 4 == 0 && d.out_c_pitch % 4 == 0 &&
                     d.out_c_offset % 4 == 0;
  const bool is_1x1 = d.R == 1 && d.S == 1 && d.pad_h == 0 && d.pad_w == 0;
  const bool s1 = d.stride_h == 1 && d.stride_w == 1;
  int mode = -1;
  if (d.groups == 1) {
    if (d.C % 16 == 0 && is_1x1 && s1) mode = MODE_FLAT;
    else if (d.C % 16 == 0 && is_1x1) mode = MODE_VIEW;
    else if (d.C % 16 == 0 && s1 && d.C <= 64 && d.S >= 4 && d.S * d.C <= 1024 &&
             static_cast<long long>(d.N) * d.H * d.W * d.C <= (64ll << 20) && h->hints.window_rows != 0 && d.pool == 0) mode = MODE_WROW;
    else if (d.C % 16 == 0 && d.stride_h <= 2 && d.stride_w <= 2) mode = MODE_BOX;   // (strides: see prepare_a_map)
    else if (d.C <= 4 && d.stride_h == 2 && d.stride_w == 2 && d.S + 1 <= 16 && d.R * d.S * d.C <= 1024 &&
             h->hints.space_to_depth != 0) mode = MODE_S2D;
    else if (d.C <= 4 && s1 && d.S >= 2 && d.S <= 16 && h->hints.window_rows != 0 &&
             static_cast<long long>(d.N) * d.H * (d.W + d.S + 16) < (1ll << 31)) mode = MODE_WROW;
    else if (d.C <= 4 && d.R * d.S * d.C <= 1024) mode = MODE_STEM;
  }
  if (d.pool && (mode != MODE_BOX || (d.algo != QCONV_ALGO_AUTO && d.algo != QCONV_ALGO_IGEMM))) {
    free_handle(h);
    return fail(QCONV_ERR_UNSUPPORTED_SHAPE, "pool: only the tensor-core path with per-tap boxes takes the pool inside the layer");
  }
  int algo = d.algo;
  if (algo == QCONV_ALGO_AUTO) algo = mode >= 0 ? QCONV_ALGO_IGEMM : (dw_ok ? QCONV_ALGO_DEPTHWISE : QCONV_ALGO_DIRECT);
  if (algo == QCONV_ALGO_IGEMM && mode < 0) {
    free_handle(h);
    return fail(QCONV_ERR_UNSUPPORTED_SHAPE, "implicit GEMM needs groups == 1 and C %% 16 == 0 with strides up to 2 "
                "(any stride for a 1x1 filter), or C <= 4");
  }
  if (algo == QCONV_ALGO_DEPTHWISE && !dw_ok) {
    free_handle(h);
    return fail(QCONV_ERR_UNSUPPORTED_SHAPE, "depthwise kernel needs 3x3, groups == C == K, C %% 4 == 0");
  }
  h->algo = algo;
  h->mode = mode;

  auto upload_i32 = [&](int32_t** dst, const int32_t* src, int32_t fill) -> int {
    std::vector<int32_t> tmp(d.K, fill);
    if (src) std::memcpy(tmp.data(), src, sizeof(int32_t) * d.K);
    CUDA_TRY(cudaMalloc(dst, sizeof(int32_t) * d.K));
    CUDA_TRY(cudaMemcpy(*dst, tmp.data(), sizeof(int32_t) * d.K, cudaMemcpyHostToDevice));
    return QCONV_OK;
  };
  int rc = QCONV_OK;
  if (bias_host) rc = upload_i32(&h->d_bias, bias_host, 0);
  if (!rc) rc = upload_i32(&h->d_shift, shift_host, 0);
  if (!rc && d.has_residual) rc = upload_i32(&h->d_lshift, res_lshift_host, 0);
  if (!rc) rc = upload_i32(&h->d_accexp, acc_exp_host, 0);
  if (!rc) {
    cudaError_t e = cudaMalloc(&h->d_status, sizeof(int));
    if (e == cudaSuccess) e = cudaMemset(h->d_status, 0, sizeof(int));
    if (e != cudaSuccess) rc = fail(QCONV_ERR_CUDA, "status word: %s", cudaGetErrorString(e));
  }
  if (!rc) {
    if (algo == QCONV_ALGO_IGEMM) {
      rc = plan_igemm(h, w_krsc.data(), bias_host, shift_host, res_lshift_host, acc_exp_host);
    } else {
      std::vector<int8_t> wp(wcount);
      const size_t per_k = static_cast<size_t>(d.R) * d.S * Cg;
      // [R][S][Cg][K]; for depthwise Cg == 1 this is [R*S][C]
      for (int k = 0; k < d.K; ++k)
        for (size_t j = 0; j < per_k; ++j) wp[j * d.K + k] = w_krsc[k * per_k + j];
      cudaError_t e = cudaMalloc(&h->d_w, wcount);
      if (e == cudaSuccess) e = cudaMemcpy(h->d_w, wp.data(), wcount, cudaMemcpyHostToDevice);
      if (e != cudaSuccess) rc = fail(QCONV_ERR_CUDA, "weights: %s", cudaGetErrorString(e));
      // Depthwise fast path (tap-packed dp4a with float-magic requantization, exact while
      // |bias| + 9 * 128 * 128 < 2^22): int8 output, nearest-even, 8-bit saturation, no residual.
      if (!rc && algo == QCONV_ALGO_DEPTHWISE && d.out_mode == QCONV_OUT_INT8 && d.n_out == 8 &&
          d.rounding == QCONV_ROUND_NEAREST_EVEN && !d.has_residual && max_bias <= 4000000 &&
          h->hints.depthwise_form != 0) {
        std::vector<uint32_t> t(static_cast<size_t>(6) * d.C);
        for (int c = 0; c < d.C; ++c) {
          for (int r = 0; r < 3; ++r) {
            uint32_t word = 0;
            for (int sx = 0; sx < 3; ++sx)
              word |= static_cast<uint32_t>(static_cast<uint8_t>(wp[static_cast<size_t>(r * 3 + sx) * d.C + c])) << (8 * sx);
            t[static_cast<size_t>(r) * d.C + c] = word;
          }
          t[static_cast<size_t>(3) * d.C + c] = static_cast<uint32_t>((bias_host ? bias_host[c] : 0) + 0x4B400000);
          const int sh_c = shift_host ? shift_host[c] : 0;
          const float sc = sh_c <= 22 ? std::ldexp(1.0f, -sh_c) : 0.0f;
          const float off = static_cast<float>(12582912.0 * (1.0 - static_cast<double>(sc)));   // exact for s <= 22
          std::memcpy(&t[static_cast<size_t>(4) * d.C + c], &sc, 4);
          std::memcpy(&t[static_cast<size_t>(5) * d.C + c], &off, 4);
        }
        e = cudaMalloc(&h->d_dw_tap, t.size() * 4);
        if (e == cudaSuccess) e = cudaMemcpy(h->d_dw_tap, t.data(), t.size() * 4, cudaMemcpyHostToDevice);
        if (e != cudaSuccess) rc = fail(QCONV_ERR_CUDA, "depthwise tables: %s", cudaGetErrorString(e));
        h->dw_tap = 1;
        if (!rc && d.C % 32 == 0 && h->hints.depthwise_form != 1) plan_dw_tma(h);
      }
    }
  }
  if (rc) {
    free_handle(h);
    return rc;
  }
  *out = h;
  return QCONV_OK;
}

}  // extern "C"

namespace {
// Padded, widened copy of a stride-1 layer's input on at most 4 channels (from int8 or from float).
template <int C, int PB>
cudaError_t launch_row_pack_c(const qconv_handle* h, const void* src, bool f32, int e_x, int n_run, cudaStream_t st) {
  const qconv_desc& d = h->d;
  const unsigned int pixels = static_cast<unsigned int>(n_run) * d.H * d.W;
  const dim3 grid((pixels / 4 + 256) / 256);
  if (f32)
    return launch_chained(qc::stem_row_pack_kernel<C, PB, true>, grid, dim3(256), 0, st, src, h->d_pack, pixels, d.W, h->s2d_wp,
                          h->s2d_off_w, e_x, d.n_in);
  return launch_chained(qc::stem_row_pack_kernel<C, PB, false>, grid, dim3(256), 0, st, src, h->d_pack, pixels, d.W, h->s2d_wp,
                        h->s2d_off_w, 0, d.n_in);
}

cudaError_t launch_row_pack(const qconv_handle* h, const void* src, bool f32, int e_x, int n_run, cudaStream_t st) {
  const bool p8 = h->win_pb == 8;
  switch (h->d.C) {
    case 1: return p8 ? launch_row_pack_c<1, 8>(h, src, f32, e_x, n_run, st) : launch_row_pack_c<1, 16>(h, src, f32, e_x, n_run, st);
    case 2: return p8 ? launch_row_pack_c<2, 8>(h, src, f32, e_x, n_run, st) : launch_row_pack_c<2, 16>(h, src, f32, e_x, n_run, st);
    case 3: return p8 ? launch_row_pack_c<3, 8>(h, src, f32, e_x, n_run, st) : launch_row_pack_c<3, 16>(h, src, f32, e_x, n_run, st);
    default: return p8 ? launch_row_pack_c<4, 8>(h, src, f32, e_x, n_run, st) : launch_row_pack_c<4, 16>(h, src, f32, e_x, n_run, st);
  }
}

// One layer launch.  input_is_packed: d_x is the handle's own space-to-depth scratch, already filled
// (qconv_run_f32 converts and packs in one kernel).
int run_layer(qconv_handle* h, const int8_t* d_x, const int8_t* d_residual, void* d_y, int n_run,
              void* cuda_stream, bool input_is_packed) {
  if (!h || !d_x || !d_y) return fail(QCONV_ERR_BAD_ARG, "NULL handle or tensor pointer");
  const qconv_desc& d = h->d;
  if (n_run <= 0 || n_run > d.N) return fail(QCONV_ERR_BAD_ARG, "n_run %d outside [1, %d]", n_run, d.N);
  if ((d.has_residual != 0) != (d_residual != nullptr))
    return fail(QCONV_ERR_BAD_ARG, "residual pointer does not match has_residual");
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  h->last_stream = st;
  const float uni_c1 = h->uni_s <= 22 ? std::ldexp(1.0f, -h->uni_s) : 0.0f;
  qc::EpilogueParams ep{h->d_bias, h->d_shift, h->d_lshift, h->d_accexp, d.relu, d.rounding,
                        h->lo, h->hi, d.out_mode, h->uni_s, h->uni_s > 0 ? (1 << (h->uni_s - 1)) - 1 : 0,
                        (h->uni_s > 0 ? 1 : 0) | ((1 << h->uni_t) << 1), uni_c1,
                        static_cast<float>(12582912.0 * (1.0 - static_cast<double>(uni_c1)))};
  qc::ConvGeom g{n_run, d.H, d.W, d.C, d.K, d.R, d.S, d.stride_h, d.stride_w, d.pad_h, d.pad_w,
                 d.groups, h->P, h->Q, d.out_c_offset, d.out_c_pitch};
  const size_t outs = static_cast<size_t>(n_run) * h->P * h->Q;
  if (h->algo == QCONV_ALGO_DIRECT) {
    qc::direct_conv_kernel<<<grid_for(outs * d.K, 256, h->num_sms * 64), 256, 0, st>>>(d_x, h->d_w, d_residual, d_y,
                                                                                g, ep);
  } else if (h->algo == QCONV_ALGO_DEPTHWISE) {
    if ((reinterpret_cast<uintptr_t>(d_x) | reinterpret_cast<uintptr_t>(d_y) |
         reinterpret_cast<uintptr_t>(d_residual)) & 3)
      return fail(QCONV_ERR_ALIGNMENT, "depthwise kernel needs 4-byte aligned tensors");
    constexpr int TW = 4;
    if (h->dw_tap && n_run <= 65535) {
      const qc::DwTapParams tp{h->d_dw_tap, reinterpret_cast<const int32_t*>(h->d_dw_tap + static_cast<size_t>(3) * d.C),
                               reinterpret_cast<const float*>(h->d_dw_tap + static_cast<size_t>(4) * d.C),
                               reinterpret_cast<const float*>(h->d_dw_tap + static_cast<size_t>(5) * d.C),
                               12582912.0f + static_cast<float>(d.relu ? 0 : h->lo), 12582912.0f + static_cast<float>(h->hi)};
      const int per_row = ceil_div(h->Q, TW) * (d.C / 4);
      // rows per thread: long strips amortise the per-thread tables, but the grid must still fill the GPU
      int rows = 16;
      while (rows > 4 && static_cast<long>(ceil_div(per_row, 256)) * ceil_div(h->P, rows) * n_run < 4L * h->num_sms) rows /= 2;
      rows = std::min(rows, h->P);
      dim3 grid(ceil_div(per_row, 256), ceil_div(h->P, rows), n_run);
      if (h->dw_tma && (reinterpret_cast<uintptr_t>(d_x) & 15) == 0) {
        int rc = prepare_dw_map(h, d_x, n_run);
        if (rc) return rc;
        qc::DwTmaParams prm = h->dw_prm;
        const int ctas_row = (d.C / 4 / prm.cwb) * prm.q_blocks;
        int rpc = 16;
        while (rpc > 4 && static_cast<long>(ctas_row) * ceil_div(h->P, rpc) * n_run < 4L * h->num_sms) rpc /= 2;
        prm.rows_per_cta = std::min(rpc, h->P);
        dim3 tgrid(ctas_row, ceil_div(h->P, prm.rows_per_cta), n_run);
        const size_t smem = static_cast<size_t>(qc::kDwStages) * prm.stage_bytes + sizeof(qc::DwTmaShared);
        if (d.stride_h == 1)
          qc::depthwise3x3_tma_kernel<1><<<tgrid, qc::kDwThreads, smem, st>>>(h->dw_map, static_cast<int8_t*>(d_y), g, tp, prm,
                                                                             h->d_status, h->wait_limit);
        else
          qc::depthwise3x3_tma_kernel<2><<<tgrid, qc::kDwThreads, smem, st>>>(h->dw_map, static_cast<int8_t*>(d_y), g, tp, prm,
                                                                             h->d_status, h->wait_limit);
      } else if (d.stride_h == 1) {
        qc::depthwise3x3_tap_kernel<1><<<grid, 256, 0, st>>>(d_x, static_cast<int8_t*>(d_y), g, tp, rows);
      } else {
        qc::depthwise3x3_tap_kernel<2><<<grid, 256, 0, st>>>(d_x, static_cast<int8_t*>(d_y), g, tp, rows);
      }
      cudaError_t e2 = cudaGetLastError();
      if (e2 != cudaSuccess) return fail(QCONV_ERR_CUDA, "kernel launch: %s", cudaGetErrorString(e2));
      return QCONV_OK;
    }
    const size_t items = static_cast<size_t>(n_run) * h->P * ceil_div(h->Q, TW) * (d.C / 4);
    const int grid = grid_for(items, 256, h->num_sms * 64);
    if (d.stride_h == 1)
      qc::depthwise3x3_kernel<1, TW><<<grid, 256, 0, st>>>(d_x, h->d_w, d_residual, d_y, g, ep);
    else
      qc::depthwise3x3_kernel<2, TW><<<grid, 256, 0, st>>>(d_x, h->d_w, d_residual, d_y, g, ep);
  } else {
    if (reinterpret_cast<uintptr_t>(d_x) & 15)
      return fail(QCONV_ERR_ALIGNMENT, "d_x must be 16-byte aligned");
    if (h->prm.vec_store && ((reinterpret_cast<uintptr_t>(d_y) | reinterpret_cast<uintptr_t>(d_residual)) & 15))
      return fail(QCONV_ERR_ALIGNMENT, "d_y and d_residual must be 16-byte aligned");
    const int8_t* a_ptr = d_x;
    if (h->mode == MODE_STEM) {
      if (h->stem_segp) {
        if (reinterpret_cast<uintptr_t>(d_x) & 3) return fail(QCONV_ERR_ALIGNMENT, "d_x must be 4-byte aligned");
        if (n_run > 65535 || static_cast<long long>(h->P) * h->Q * d.R >= (1ll << 31))
          return fail(QCONV_ERR_UNSUPPORTED_SHAPE, "stem packing: image or batch too large");
        const long long x_bytes = static_cast<long long>(n_run) * d.H * d.W * d.C;
        const long long x_words = x_bytes / 4;             // whole words; the tail goes byte by byte
        const int x_tail = static_cast<int>(x_bytes % 4);
        const dim3 grid(ceil_div(h->Q, 64), ceil_div(h->P, 4), n_run);
        const int nw = (d.S * d.C + 3) / 4;                  // words holding segment bytes: 1..4 or 5..7
#define QC_PACK(SEGW, NW)                                                                                      \
  qc::stem_pack_rows_kernel<SEGW, NW><<<grid, 256, 0, st>>>(d_x, h->d_pack, n_run, d.H, d.W, d.C, d.R, d.S,    \
                                                            d.stride_h, d.stride_w, d.pad_h, d.pad_w, h->P,    \
                                                            h->Q, h->kg_pad, x_words, x_tail)
        if (h->stem_segp == 16) {
          switch (nw) {
            case 1: QC_PACK(4, 1); break;
            case 2: QC_PACK(4, 2); break;
            case 3: QC_PACK(4, 3); break;
            default: QC_PACK(4, 4); break;
          }
        } else {
          switch (nw) {
            case 5: QC_PACK(8, 5); break;
            case 6: QC_PACK(8, 6); break;
            default: QC_PACK(8, 7); break;
          }
        }
#undef QC_PACK
      } else {
        const size_t vecs = outs * (h->kg_pad / 16);
        qc::stem_pack_kernel<<<grid_for(vecs, 256, 148 * 32), 256, 0, st>>>(
            d_x, h->d_pack, n_run, d.H, d.W, d.C, d.R, d.S, d.stride_h, d.stride_w, d.pad_h, d.pad_w, h->P, h->Q,
            d.R * d.S * d.C, h->kg_pad);
      }
      a_ptr = h->d_pack;
    }
    if (h->mode == MODE_WROW && d.C < 16) {
      if (!input_is_packed) {
        cudaError_t pe = launch_row_pack(h, d_x, false, 0, n_run, st);
        if (pe != cudaSuccess) return fail(QCONV_ERR_CUDA, "kernel launch: %s", cudaGetErrorString(pe));
      }
      a_ptr = h->d_pack;
    } else if (h->mode == MODE_WROW) {
      const size_t vecs = static_cast<size_t>(n_run) * d.H * d.W * (d.C / 16);
      if (vecs > 2147483647ull) return fail(QCONV_ERR_UNSUPPORTED_SHAPE, "row padding: image or batch too large");
      cudaError_t pe = launch_chained(qc::pad_rows_kernel, dim3(static_cast<unsigned int>((vecs + 255) / 256)), dim3(256), 0, st,
                                      reinterpret_cast<const uint4*>(d_x), reinterpret_cast<uint4*>(h->d_pack),
                                      static_cast<unsigned int>(vecs), n_run * d.H, d.W, d.C / 16, h->s2d_wp, h->s2d_off_w);
      if (pe != cudaSuccess) return fail(QCONV_ERR_CUDA, "kernel launch: %s", cudaGetErrorString(pe));
      a_ptr = h->d_pack;
    }
    if (h->mode == MODE_S2D && input_is_packed) {
      a_ptr = h->d_pack;
    } else if (h->mode == MODE_S2D) {
      if (n_run > 65535 || h->s2d_h > 65535) return fail(QCONV_ERR_UNSUPPORTED_SHAPE, "stem packing: image or batch too large");
      const dim3 grid(ceil_div(h->s2d_w, 128), h->s2d_h, n_run);
      uint4* pk = reinterpret_cast<uint4*>(h->d_pack);
      cudaError_t pe;
      switch (d.C) {
        case 1: pe = launch_chained(qc::stem_s2d_pack_kernel<1>, grid, dim3(128), 0, st, d_x, pk, n_run, d.H, d.W, h->s2d_h, h->s2d_w, h->s2d_wp, h->s2d_off_w); break;
        case 2: pe = launch_chained(qc::stem_s2d_pack_kernel<2>, grid, dim3(128), 0, st, d_x, pk, n_run, d.H, d.W, h->s2d_h, h->s2d_w, h->s2d_wp, h->s2d_off_w); break;
        case 3: pe = launch_chained(qc::stem_s2d_pack_kernel<3>, grid, dim3(128), 0, st, d_x, pk, n_run, d.H, d.W, h->s2d_h, h->s2d_w, h->s2d_wp, h->s2d_off_w); break;
        default: pe = launch_chained(qc::stem_s2d_pack_kernel<4>, grid, dim3(128), 0, st, d_x, pk, n_run, d.H, d.W, h->s2d_h, h->s2d_w, h->s2d_wp, h->s2d_off_w); break;
      }
      if (pe != cudaSuccess) return fail(QCONV_ERR_CUDA, "kernel launch: %s", cudaGetErrorString(pe));
      a_ptr = h->d_pack;
    }
    int rc = prepare_a_map(h, a_ptr, n_run);
    if (rc) return rc;
    if (h->prm.out_stage_bytes) {
      rc = prepare_y_map(h, d_y, n_run);
      if (rc) return rc;
      if (d.has_residual && h->prm.out_stage_bufs == 3) {
        rc = prepare_r_map(h, d_residual, n_run);
        if (rc) return rc;
      }
    }
    const qc::IgemmParams& p = h->prm;
    if (h->pair) {
      qc::PairParams pp = {};
      pp.tq = p.tq; pp.tp = p.tp; pp.tn = p.tn;
      pp.tiles_q = p.tiles_q; pp.tiles_p = p.tiles_p; pp.tiles_n = p.tiles_n;
      const long boxes = static_cast<long>(p.tiles_q) * p.tiles_p * p.tiles_n;
      pp.pairs_m = static_cast<int>((boxes + 1) / 2);
      pp.tiles_k = p.tiles_k; pp.BN = p.BN; pp.BKC = p.BKC; pp.nchunks = p.nchunks; pp.R = p.R; pp.S = p.S;
      pp.pad_h = p.pad_h; pp.pad_w = p.pad_w; pp.stride_h = p.stride_h; pp.stride_w = p.stride_w;
      pp.stages = p.stages; pp.Q = p.Q; pp.P = p.P; pp.Nimg = p.Nimg; pp.K = p.K;
      pp.out_c_offset = p.out_c_offset; pp.out_c_pitch = p.out_c_pitch; pp.tmem_cols = p.tmem_cols;
      pp.a_stage_bytes = p.a_stage_bytes; pp.b_stage_bytes = p.b_stage_bytes;
      pp.tx_bytes = 2u * static_cast<uint32_t>(p.tq * p.tp * p.tn * p.BKC + (p.BN / 2) * p.BKC);
      const long pair_tiles = static_cast<long>(pp.pairs_m) * pp.tiles_k;
      if (pair_tiles <= 0 || pair_tiles > 1073741823l) return fail(QCONV_ERR_UNSUPPORTED_SHAPE, "tile count out of range");
      const long pairs = std::min<long>(pair_tiles, h->num_sms / 2);
      cudaLaunchConfig_t cfg = {};
      cfg.gridDim = dim3(static_cast<unsigned int>(2 * pairs));
      cfg.blockDim = dim3(qc::kIgemmThreads);
      cfg.dynamicSmemBytes = h->smem_bytes;
      cfg.stream = st;
      cudaLaunchAttribute attr[2];
      attr[0].id = cudaLaunchAttributeClusterDimension;
      attr[0].val.clusterDim.x = 2; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
      attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
      attr[1].val.programmaticStreamSerializationAllowed = h->use_pdl;
      cfg.attrs = attr;
      cfg.numAttrs = 2;
      const int4* chan_ptr = h->d_chan;
      cudaError_t le = cudaLaunchKernelEx(&cfg, pair_kernel_for(h), h->tmap_a, h->tmap_b, pp, p, ep, chan_ptr, d_y,
                                          h->d_status, h->wait_limit);
      if (le != cudaSuccess) return fail(QCONV_ERR_CUDA, "kernel launch (SM pairs): %s", cudaGetErrorString(le));
      return QCONV_OK;
    }
    const long tiles = static_cast<long>(p.tiles_q) * p.tiles_p * p.tiles_n * p.tiles_k;
    if (tiles <= 0 || tiles > 2147483647l) return fail(QCONV_ERR_UNSUPPORTED_SHAPE, "tile count out of range");
    long grid = std::min<long>(tiles, static_cast<long>(h->num_sms) * h->ctas_per_sm);
    // with resident weights a CTA must stay on one channel tile: the stride over tiles is a multiple of tiles_k
    if (p.b_resident && p.tiles_k > 1) grid = std::max<long>(p.tiles_k, grid / p.tiles_k * p.tiles_k);
    {
      // what depends on the grid size: its mixed-radix digits (the walk from one tile of a CTA to its next)
      qc::IgemmParams& pw = h->prm;
      if (h->walk_grid != grid) {
      long m = grid;
      pw.walk_dk = static_cast<int>(m % p.tiles_k); m /= p.tiles_k;
      pw.walk_dq = static_cast<int>(m % p.tiles_q); m /= p.tiles_q;
      pw.walk_dp = static_cast<int>(m % p.tiles_p); pw.walk_dn = static_cast<int>(m / p.tiles_p);
      pw.fd_grid = make_fastdiv(static_cast<int>(grid));
      if (!pw.fd_grid.d) return fail(QCONV_ERR_UNSUPPORTED_SHAPE, "internal: division constants failed their check");
      h->walk_grid = grid;
      }
    }
    // Programmatic dependent launch: the kernel's set-up may overlap the tail of the previous
    // kernel in the stream; the kernel itself waits (griddepcontrol.wait) before touching tensors.
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(static_cast<unsigned int>(grid));
    cfg.blockDim = dim3(qc::kIgemmThreads);
    cfg.dynamicSmemBytes = h->smem_bytes;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = h->use_pdl;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    const int4* chan_ptr = h->d_chan;
    cudaError_t le = cudaLaunchKernelEx(&cfg, igemm_kernel_for(h), h->tmap_a, h->tmap_b,
                                        p.out_stage_bytes ? h->tmap_y : h->tmap_a,
                                        (p.out_stage_bytes && p.out_stage_bufs == 3) ? h->tmap_r : h->tmap_a, p, ep, chan_ptr, d_residual,
                                        d_y, h->d_status, h->wait_limit);
    if (le != cudaSuccess) return fail(QCONV_ERR_CUDA, "kernel launch: %s", cudaGetErrorString(le));
  }
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return fail(QCONV_ERR_CUDA, "kernel launch: %s", cudaGetErrorString(e));
  return QCONV_OK;
}
}  // namespace

extern "C" {

int qconv_run(qconv_handle* h, const int8_t* d_x, const int8_t* d_residual, void* d_y, int n_run,
              void* cuda_stream) {
  return run_layer(h, d_x, d_residual, d_y, n_run, cuda_stream, false);
}

int qconv_run_f32(qconv_handle* h, const float* d_x_f32, int e_x, const int8_t* d_residual, void* d_y, int n_run,
                  void* cuda_stream) {
  if (!h || !d_x_f32 || !d_y) return fail(QCONV_ERR_BAD_ARG, "NULL handle or tensor pointer");
  const qconv_desc& d = h->d;
  const bool rows_form = h->algo == QCONV_ALGO_IGEMM && h->mode == MODE_WROW && d.C < 16;
  if (h->algo != QCONV_ALGO_IGEMM || (h->mode != MODE_S2D && !rows_form))
    return fail(QCONV_ERR_UNSUPPORTED_SHAPE, "qconv_run_f32 serves layers that repack their input (at most 4 channels, "
                "stride 2 in space-to-depth form or stride 1 in padded rows); convert with qquantize_f32 and call "
                "qconv_run otherwise");
  if (n_run <= 0 || n_run > d.N) return fail(QCONV_ERR_BAD_ARG, "n_run %d outside [1, %d]", n_run, d.N);
  if (e_x < -126 || e_x > 126) return fail(QCONV_ERR_BAD_ARG, "e_x outside [-126, 126]");
  if (reinterpret_cast<uintptr_t>(d_x_f32) & 3) return fail(QCONV_ERR_ALIGNMENT, "d_x_f32 must be 4-byte aligned");
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  if (rows_form) {
    cudaError_t re = launch_row_pack(h, d_x_f32, true, e_x, n_run, st);
    if (re != cudaSuccess) return fail(QCONV_ERR_CUDA, "kernel launch: %s", cudaGetErrorString(re));
    return run_layer(h, h->d_pack, d_residual, d_y, n_run, cuda_stream, true);
  }
  if (n_run > 65535 || h->s2d_h > 65535) return fail(QCONV_ERR_UNSUPPORTED_SHAPE, "stem packing: image or batch too large");
  const dim3 grid(ceil_div(h->s2d_w, 128), h->s2d_h, n_run);
  uint4* pk = reinterpret_cast<uint4*>(h->d_pack);
  cudaError_t pe;
  switch (d.C) {
    case 1: pe = launch_chained(qc::stem_s2d_pack_f32_kernel<1>, grid, dim3(128), 0, st, d_x_f32, pk, n_run, d.H, d.W, h->s2d_h, h->s2d_w, h->s2d_wp, h->s2d_off_w, e_x, d.n_in); break;
    case 2: pe = launch_chained(qc::stem_s2d_pack_f32_kernel<2>, grid, dim3(128), 0, st, d_x_f32, pk, n_run, d.H, d.W, h->s2d_h, h->s2d_w, h->s2d_wp, h->s2d_off_w, e_x, d.n_in); break;
    case 3: pe = launch_chained(qc::stem_s2d_pack_f32_kernel<3>, grid, dim3(128), 0, st, d_x_f32, pk, n_run, d.H, d.W, h->s2d_h, h->s2d_w, h->s2d_wp, h->s2d_off_w, e_x, d.n_in); break;
    default: pe = launch_chained(qc::stem_s2d_pack_f32_kernel<4>, grid, dim3(128), 0, st, d_x_f32, pk, n_run, d.H, d.W, h->s2d_h, h->s2d_w, h->s2d_wp, h->s2d_off_w, e_x, d.n_in); break;
  }
  if (pe != cudaSuccess) return fail(QCONV_ERR_CUDA, "kernel launch: %s", cudaGetErrorString(pe));
  return run_layer(h, h->d_pack, d_residual, d_y, n_run, cuda_stream, true);
}

int qconv_status(qconv_handle* h) {
  if (!h) return fail(QCONV_ERR_BAD_ARG, "NULL handle");
  CUDA_TRY(cudaStreamSynchronize(h->last_stream));
  int st = 0;
  CUDA_TRY(cudaMemcpy(&st, h->d_status, sizeof(int), cudaMemcpyDeviceToHost));
  if (st != 0) {
    CUDA_TRY(cudaMemset(h->d_status, 0, sizeof(int)));
    return fail(st, "a bounded device-side wait expired (status %d)", st);
  }
  return QCONV_OK;
}

int qconv_set_wait_limit(qconv_handle* h, unsigned int polls) {
  if (!h) return fail(QCONV_ERR_BAD_ARG, "NULL handle");
  h->wait_limit = polls;
  return QCONV_OK;
}

int qconv_describe(const qconv_handle* h, char* buf, size_t buf_len) {
  if (!h || !buf || buf_len == 0) return fail(QCONV_ERR_BAD_ARG, "NULL argument");
  if (h->algo == QCONV_ALGO_IGEMM) {
    static const char* names[] = {"flat", "view", "box", "stem", "s2d", "wrow"};
    const qc::IgemmParams& p = h->prm;
    snprintf(buf, buf_len, "igemm/%s box=%dx%dx%d BN=%d tiles_k=%d BKC=%d chunks=%d taps=%dx%d stages=%d smem=%zu "
             "ctas/sm=%d fast=%d uni=%d flt=%d fold=%d tma_store=%d b_res=%d halo=%d grp=%d pair=%d pool=%d",
             names[h->mode], p.tq, p.tp, p.tn, p.BN, p.tiles_k, p.BKC, p.nchunks, p.R, p.S, p.stages,
             h->smem_bytes, h->ctas_per_sm, p.fast_epilogue, h->uniform_shift, h->flt_epilogue && p.fast_epilogue, h->fold,
             p.out_stage_bytes ? p.out_stage_bufs : 0, p.b_resident, p.tap_boxes ? 0 : p.halo_s, p.tap_boxes ? p.halo_s : 0, h->pair, h->d.pool);
  } else {
    snprintf(buf, buf_len, "%s", h->algo == QCONV_ALGO_DEPTHWISE ? (h->dw_tma ? "depthwise3x3/tap-packed+tma" : h->dw_tap ? "depthwise3x3/tap-packed" : "depthwise3x3/dp4a")
                                                                  : "direct");
  }
  return QCONV_OK;
}

int qconv_destroy(qconv_handle* h) {
  if (!h) return fail(QCONV_ERR_BAD_ARG, "NULL handle");
  free_handle(h);
  return QCONV_OK;
}

// --------------------------------------------------------------------------- calibration
}  // extern "C"

// Scratch of qcalib_collect_static: lives in the library image, about 64 KB on every GPU that loads
// the library, until the process exits.  Its name below is only a host-side handle for the symbol;
// the device address comes from cudaGetSymbolAddress, once per device.
static __device__ __align__(256) unsigned char g_calib_static_scratch[sizeof(qc::CalibScratch)];

namespace {
std::mutex g_calib_mu;
qc::CalibScratch* g_calib_scratch[64] = {nullptr};       // cudaMalloc'ed on first use, per device
qc::CalibScratch* g_calib_static_ptr[64] = {nullptr};    // device address of the built-in array, per device

// The statistics pass shared by both entry points: clear, maximum + sums, finalize, histogram, copy
// back.  `sc` is device scratch the caller provides (it still holds the previous call's counters).
int calib_run(const float* d_x, size_t count, int nbins, float range_hi, qcalib_stats* host_out,
              cudaStream_t st, qc::CalibScratch* sc) {
  const int vec_ok = (reinterpret_cast<uintptr_t>(d_x) & 15) == 0;
  const int blocks = grid_for((count + 3) / 4, 256, 148 * 8);
  CUDA_TRY(cudaMemsetAsync(sc, 0, offsetof(qc::CalibScratch, part_sum), st));
  qc::calib_pass1_kernel<<<blocks, 256, 0, st>>>(d_x, count, sc, vec_ok);
  qc::calib_finalize_kernel<<<1, 256, 0, st>>>(sc, blocks, static_cast<unsigned long long>(count));
  qc::calib_hist_kernel<<<blocks, 256, nbins * sizeof(unsigned int), st>>>(d_x, count, sc, nbins, range_hi, vec_ok);
  CUDA_TRY(cudaGetLastError());
  struct { unsigned int maxabs_bits, pad; unsigned long long finite, nonfinite; double sum, sumsq; } head;
  CUDA_TRY(cudaMemcpyAsync(&head, sc, sizeof(head), cudaMemcpyDeviceToHost, st));
  CUDA_TRY(cudaMemcpyAsync(host_out->hist, reinterpret_cast<const unsigned char*>(sc) + offsetof(qc::CalibScratch, hist),
                           sizeof(uint64_t) * nbins, cudaMemcpyDeviceToHost, st));
  CUDA_TRY(cudaStreamSynchronize(st));
  std::memcpy(&host_out->maxabs, &head.maxabs_bits, sizeof(float));
  host_out->range_hi = range_hi > 0.0f ? range_hi : host_out->maxabs;
  host_out->count = head.finite;
  host_out->nonfinite = head.nonfinite;
  host_out->sum = head.sum;
  host_out->sumsq = head.sumsq;
  return QCONV_OK;
}
}  // namespace

extern "C" {

int qcalib_collect(const float* d_x, size_t count, int nbins, float range_hi, qcalib_stats* host_out,
                   void* cuda_stream) {
  if (!d_x || !host_out || !host_out->hist) return fail(QCONV_ERR_BAD_ARG, "NULL argument");
  if (count == 0 || nbins < 1 || nbins > qc::kCalibMaxBins)
    return fail(QCONV_ERR_BAD_ARG, "count must be > 0 and nbins in [1, %d]", qc::kCalibMaxBins);
  if (reinterpret_cast<uintptr_t>(d_x) & 3) return fail(QCONV_ERR_ALIGNMENT, "d_x must be 4-byte aligned");
  int dev = 0;
  CUDA_TRY(cudaGetDevice(&dev));
  if (dev < 0 || dev >= 64) return fail(QCONV_ERR_CUDA, "device index %d out of range", dev);
  qc::CalibScratch* sc;
  {
    std::lock_guard<std::mutex> lock(g_calib_mu);
    if (!g_calib_scratch[dev]) CUDA_TRY(cudaMalloc(&g_calib_scratch[dev], sizeof(qc::CalibScratch)));
    sc = g_calib_scratch[dev];
  }
  return calib_run(d_x, count, nbins, range_hi, host_out, static_cast<cudaStream_t>(cuda_stream), sc);
}

// ----------------------------------------------------------- calibration without allocation
int qcalib_collect_static(const float* d_x, size_t count, int nbins, float range_hi, qcalib_stats* host_out,
                          void* cuda_stream) {
  if (!d_x || !host_out || !host_out->hist) return fail(QCONV_ERR_BAD_ARG, "NULL argument");
  if (nbins < 1 || nbins > QCALIB_STATIC_MAX_BINS)
    return fail(QCONV_ERR_BAD_ARG, "qcalib_collect_static: nbins %d is outside [1, %d], the size of its built-in "
                "scratch", nbins, QCALIB_STATIC_MAX_BINS);
  if (count == 0 || count > QCALIB_STATIC_MAX_COUNT)
    return fail(QCONV_ERR_BAD_ARG, "qcalib_collect_static: count %zu is outside [1, 2^40], the most its built-in "
                "scratch is sized for", count);
  if (reinterpret_cast<uintptr_t>(d_x) & 3) return fail(QCONV_ERR_ALIGNMENT, "d_x must be 4-byte aligned");
  int dev = 0;
  CUDA_TRY(cudaGetDevice(&dev));
  if (dev < 0 || dev >= 64) return fail(QCONV_ERR_CUDA, "device index %d out of range", dev);
  qc::CalibScratch* sc;
  {
    // first call on this device: translate the symbol into this device's address (no allocation)
    std::lock_guard<std::mutex> lock(g_calib_mu);
    if (!g_calib_static_ptr[dev]) {
      void* ptr = nullptr;
      cudaError_t e = cudaGetSymbolAddress(&ptr, g_calib_static_scratch);
      if (e != cudaSuccess || !ptr)
        return fail(QCONV_ERR_CUDA, "cudaGetSymbolAddress(built-in calibration scratch): %s", cudaGetErrorString(e));
      g_calib_static_ptr[dev] = static_cast<qc::CalibScratch*>(ptr);
    }
    sc = g_calib_static_ptr[dev];
  }
  // the array still holds the previous call's counters: calib_run clears everything that accumulates
  return calib_run(d_x, count, nbins, range_hi, host_out, static_cast<cudaStream_t>(cuda_stream), sc);
}

int qquantize_f32(const float* d_x, size_t count, int e, int n, int8_t* d_y, void* cuda_stream) {
  if (!d_x || !d_y) return fail(QCONV_ERR_BAD_ARG, "NULL argument");
  if (n < 2 || n > 8 || e < -126 || e > 126) return fail(QCONV_ERR_BAD_ARG, "n in [2, 8], e in [-126, 126]");
  if (count == 0) return QCONV_OK;
  const int vec_ok = ((reinterpret_cast<uintptr_t>(d_x) | reinterpret_cast<uintptr_t>(d_y)) & 15) == 0;
  CUDA_TRY(launch_chained(qc::quantize_f32_kernel, dim3(grid_for((count + 15) / 16, 256, 148 * 16)), dim3(256), 0,
                          static_cast<cudaStream_t>(cuda_stream), d_x, d_y, count, e, n, vec_ok));
  CUDA_TRY(cudaGetLastError());
  return QCONV_OK;
}

int qmaxpool_i8(const int8_t* d_x, int N, int H, int W, int C, int R, int S, int stride, int pad,
                int8_t* d_y, void* cuda_stream) {
  if (!d_x || !d_y) return fail(QCONV_ERR_BAD_ARG, "NULL argument");
  if (N <= 0 || H <= 0 || W <= 0 || C <= 0 || R <= 0 || S <= 0 || stride <= 0 || pad < 0 || pad >= R || pad >= S)
    return fail(QCONV_ERR_BAD_ARG, "bad pooling geometry");
  const int P = (H + 2 * pad - R) / stride + 1, Q = (W + 2 * pad - S) / stride + 1;
  if (P <= 0 || Q <= 0) return fail(QCONV_ERR_UNSUPPORTED_SHAPE, "window larger than padded input");
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  const bool vec = C % 16 == 0 && ((reinterpret_cast<uintptr_t>(d_x) | reinterpret_cast<uintptr_t>(d_y)) & 15) == 0;
  const size_t pix = static_cast<size_t>(N) * P * Q;
  const bool strip_ok = vec && R == S && ((R == 3 && (stride == 1 || stride == 2)) || (R == 2 && stride == 2));
  if (strip_ok) {
    // strips as long as still leaves every SM several hundred threads
    int rows = 16;
    while (rows > 2 && static_cast<size_t>(N) * ceil_div(P, rows) * Q * (C / 16) < 148u * 2048u) rows /= 2;
    const int strips = ceil_div(P, rows);
    const size_t threads = static_cast<size_t>(N) * strips * Q * (C / 16);
    if (threads > 2147483647ull) return fail(QCONV_ERR_UNSUPPORTED_SHAPE, "pooling: tensor too large");
    const dim3 grid(static_cast<unsigned int>((threads + 127) / 128));
    if (R == 3 && stride == 1)
      CUDA_TRY(launch_chained(qc::maxpool_i8_strip_kernel<3, 3, 1>, grid, dim3(128), 0, st, d_x, d_y, N, H, W, C, pad, P, Q, rows, strips));
    else if (R == 3)
      CUDA_TRY(launch_chained(qc::maxpool_i8_strip_kernel<3, 3, 2>, grid, dim3(128), 0, st, d_x, d_y, N, H, W, C, pad, P, Q, rows, strips));
    else
      CUDA_TRY(launch_chained(qc::maxpool_i8_strip_kernel<2, 2, 2>, grid, dim3(128), 0, st, d_x, d_y, N, H, W, C, pad, P, Q, rows, strips));
  } else if (vec)
    CUDA_TRY(launch_chained(qc::maxpool_i8_vec_kernel, dim3(grid_for(pix * (C / 16), 256, 148 * 32)), dim3(256), 0, st,
                            d_x, d_y, N, H, W, C, R, S, stride, pad, P, Q));
  else
    qc::maxpool_i8_scalar_kernel<<<grid_for(pix * C, 256, 148 * 32), 256, 0, st>>>(d_x, d_y, N, H, W, C, R, S,
                                                                                   stride, pad, P, Q);
  CUDA_TRY(cudaGetLastError());
  return QCONV_OK;
}

int qeltwise_add_i8(const int8_t* const* d_inputs_host, int n_inputs, const int32_t* lshift_host, int rshift,
                    int relu, int rounding, int n_out, int symmetric, size_t count, int8_t* d_y, void* cuda_stream) {
  if (!d_inputs_host || !lshift_host || !d_y) return fail(QCONV_ERR_BAD_ARG, "NULL argument");
  if (n_inputs < 1 || n_inputs > 8 || n_out < 2 || n_out > 8 || rounding < 0 || rounding > 3)
    return fail(QCONV_ERR_BAD_ARG, "n_inputs in [1, 8], n_out in [2, 8], rounding in [0, 3]");
  if (rshift < 0 || rshift > 31) return fail(QCONV_ERR_BAD_SHIFT, "rshift %d outside [0, 31]", rshift);
  long long bound = 0;
  qc::EltwiseArgs a = {};
  int aligned = (reinterpret_cast<uintptr_t>(d_y) & 15) == 0;
  for (int i = 0; i < n_inputs; ++i) {
    if (!d_inputs_host[i]) return fail(QCONV_ERR_BAD_ARG, "input %d is NULL", i);
    if (lshift_host[i] < 0 || lshift_host[i] > 23)
      return fail(QCONV_ERR_RESIDUAL_SCALE, "lshift[%d] = %d outside [0, 23]", i, lshift_host[i]);
    bound += 128ll << lshift_host[i];
    a.in[i] = d_inputs_host[i];
    a.lshift[i] = lshift_host[i];
    aligned &= (reinterpret_cast<uintptr_t>(d_inputs_host[i]) & 15) == 0;
  }
  // Eq. 13: the widest sum must fit the 32-bit accumulator
  if (bound > 2147483647ll) return fail(QCONV_ERR_OVERFLOW_RISK, "worst-case |sum| %lld exceeds 2^31 - 1", bound);
  if (count == 0) return QCONV_OK;
  a.n_inputs = n_inputs; a.rshift = rshift; a.relu = relu; a.rounding = rounding;
  a.hi = (1 << (n_out - 1)) - 1;
  a.lo = symmetric ? -a.hi : -(1 << (n_out - 1));
  qc::eltwise_add_i8_kernel<<<grid_for((count + 15) / 16, 256, 148 * 16), 256, 0, static_cast<cudaStream_t>(cuda_stream)>>>(
      a, d_y, count, aligned);
  CUDA_TRY(cudaGetLastError());
  return QCONV_OK;
}

// --------------------------------------------------------------------------- (n, p) codes
namespace {
int make_format(int n, int p, int e, qc::DynFloatFormat* f) {
  if (n < 2 || n > 8 || p < 0 || p > n - 1) return fail(QCONV_ERR_BAD_ARG, "need 2 <= n <= 8 and 0 <= p <= n-1");
  if (e < -126 || e > 126) return fail(QCONV_ERR_BAD_ARG, "scale exponent %d outside [-126, 126]", e);
  f->n = n; f->p = p; f->e = e;
  f->e_max = (p == n - 1) ? 0 : (1 << (n - p - 1)) - 1;
  // Eq. 5 with equality: every pattern is a number
  f->beta_max = (p == n - 1) ? static_cast<float>((1 << (n - 1)) - 1)
                             : std::ldexp(static_cast<float>((2 << p) - 1), f->e_max - 1);
  return QCONV_OK;
}
}  // namespace

int qquantize_f32_np(const float* d_x, size_t count, int e, int n, int p, uint8_t* d_code, void* cuda_stream) {
  if (!d_x || !d_code) return fail(QCONV_ERR_BAD_ARG, "NULL tensor pointer");
  qc::DynFloatFormat f;
  int rc = make_format(n, p, e, &f);
  if (rc) return rc;
  if (count == 0) return QCONV_OK;
  const int vec_ok = ((reinterpret_cast<uintptr_t>(d_x) | reinterpret_cast<uintptr_t>(d_code)) & 15) == 0;
  qc::dynfloat_encode_kernel<<<grid_for((count + 15) / 16, 256, 148 * 16), 256, 0, static_cast<cudaStream_t>(cuda_stream)>>>(
      d_x, d_code, count, f, vec_ok);
  CUDA_TRY(cudaGetLastError());
  return QCONV_OK;
}

int qdequantize_np(const uint8_t* d_code, size_t count, int e, int n, int p, float* d_y, void* cuda_stream) {
  if (!d_code || !d_y) return fail(QCONV_ERR_BAD_ARG, "NULL tensor pointer");
  qc::DynFloatFormat f;
  int rc = make_format(n, p, e, &f);
  if (rc) return rc;
  if (count == 0) return QCONV_OK;
  const int vec_ok = ((reinterpret_cast<uintptr_t>(d_y) | reinterpret_cast<uintptr_t>(d_code)) & 15) == 0;
  qc::dynfloat_decode_kernel<<<grid_for((count + 15) / 16, 256, 148 * 16), 256, 0, static_cast<cudaStream_t>(cuda_stream)>>>(
      d_code, d_y, count, f, vec_ok);
  CUDA_TRY(cudaGetLastError());
  return QCONV_OK;
}

// --------------------------------------------------------------------------- convolution on (n, p) operands
}  // extern "C"

struct qconv_np_handle {
  qconv_np_desc d;
  qconv_handle* gemm = nullptr;      // int8 GEMM on the digit planes, raw int32 accumulators out
  int planes_x = 1, planes_w = 1, groups = 1;
  int P = 0, Q = 0;
  int8_t* d_planes = nullptr;        // [N][H][W][planes_x * C]
  int32_t* d_acc = nullptr;          // [N][P][Q][groups * K]
  int32_t* d_bias = nullptr;
  int32_t* d_shift = nullptr;
  qc::NpFormat fout{};
};

namespace {
// beta_max of Eq. 5 (every pattern a number); -1 if it does not fit 62 bits.
long long np_beta_max(int n, int p) {
  if (p == n - 1) return (1ll << (n - 1)) - 1;
  const int e_max = (1 << (n - p - 1)) - 1;
  if (e_max - 1 + p + 1 > 61) return -1;
  return ((2ll << p) - 1) << (e_max - 1);
}
// 7-bit digit planes needed: the last digit may use the whole int8 range.
int np_planes(long long bmax) {
  if (bmax <= 127) return 1;
  if (bmax <= 127ll * 128 + 63) return 2;
  if (bmax <= (127ll * 128 + 63) * 128 + 63) return 3;
  return 0;
}
int np_host_decode(int code, int n, int p) {
  const int c = code & ((1 << (n - 1)) - 1);
  int v;
  if (p == n - 1) v = c;
  else {
    const int E = c >> p, m = c & ((1 << p) - 1);
    v = E == 0 ? m : ((1 << p) + m) << (E - 1);
  }
  return ((code >> (n - 1)) & 1) ? -v : v;
}
void free_np(qconv_np_handle* h) {
  if (!h) return;
  if (h->gemm) free_handle(h->gemm);
  cudaFree(h->d_planes);
  cudaFree(h->d_acc);
  cudaFree(h->d_bias);
  cudaFree(h->d_shift);
  delete h;
}
}  // namespace

extern "C" {

int qconv_np_create(qconv_np_handle** out, const qconv_np_desc* desc, const uint8_t* w_codes_host,
                    const int32_t* bias_host, const int32_t* shift_host) {
  if (!out) return fail(QCONV_ERR_BAD_ARG, "out is NULL");
  *out = nullptr;
  if (!desc || !w_codes_host) return fail(QCONV_ERR_BAD_ARG, "desc or w_codes_host is NULL");
  const qconv_np_desc d = *desc;
  if (d.N <= 0 || d.H <= 0 || d.W <= 0 || d.C <= 0 || d.K <= 0 || d.R <= 0 || d.S <= 0 || d.stride_h <= 0 ||
      d.stride_w <= 0 || d.pad_h < 0 || d.pad_w < 0)
    return fail(QCONV_ERR_BAD_ARG, "non-positive dimension in descriptor");
  const int fmts[3][2] = {{d.n_in, d.p_in}, {d.n_w, d.p_w}, {d.n_out, d.p_out}};
  long long bmax[3];
  for (int i = 0; i < 3; ++i) {
    if (fmts[i][0] < 2 || fmts[i][0] > 8 || fmts[i][1] < 0 || fmts[i][1] > fmts[i][0] - 1)
      return fail(QCONV_ERR_BAD_ARG, "need 2 <= n <= 8 and 0 <= p <= n-1 for every operand type");
    bmax[i] = np_beta_max(fmts[i][0], fmts[i][1]);
  }
  const int px = bmax[0] > 0 ? np_planes(bmax[0]) : 0, pw = bmax[1] > 0 ? np_planes(bmax[1]) : 0;
  if (px == 0 || pw == 0 || bmax[2] <= 0 || bmax[2] >= (1ll << 21))
    return fail(QCONV_ERR_UNSUPPORTED_SHAPE, "an operand type's largest value (Eq. 5) exceeds three 7-bit digit planes (2^21)");
  if (d.C % 16) return fail(QCONV_ERR_UNSUPPORTED_SHAPE, "C must be a multiple of 16");
  const int P = (d.H + 2 * d.pad_h - d.R) / d.stride_h + 1, Q = (d.W + 2 * d.pad_w - d.S) / d.stride_w + 1;
  if (d.H + 2 * d.pad_h < d.R || d.W + 2 * d.pad_w < d.S || P <= 0 || Q <= 0)
    return fail(QCONV_ERR_UNSUPPORTED_SHAPE, "filter larger than padded input");
  long long max_bias = 0;
  for (int k = 0; k < d.K; ++k) {
    if (shift_host && (shift_host[k] < 0 || shift_host[k] > 40))
      return fail(QCONV_ERR_BAD_SHIFT, "shift[%d] = %d outside [0, 40]", k, shift_host[k]);
    if (bias_host) max_bias = std::max<long long>(max_bias, std::llabs(static_cast<long long>(bias_host[k])));
  }
  // Eq. 9 with b = beta_max of the operand types and a 64-bit recombination (two bits of headroom)
  const long double worst = static_cast<long double>(d.R) * d.S * d.C * static_cast<long double>(bmax[0]) * bmax[1] + max_bias;
  if (worst >= 4.6e18L / 2)
    return fail(QCONV_ERR_OVERFLOW_RISK, "worst-case |sum| exceeds 2^62 (Eq. 9 with b = beta_max)");
  const int groups = px + pw - 1;
  const size_t acc_elems = static_cast<size_t>(d.N) * P * Q * groups * d.K;
  if (acc_elems >= (1ull << 38)) return fail(QCONV_ERR_UNSUPPORTED_SHAPE, "tensor too large");

  // weights: digit planes arranged so that column group g sums x_plane_i * w_plane_(g - i)
  const int Cp = px * d.C, Kp = groups * d.K;
  std::vector<int8_t> wp(static_cast<size_t>(Kp) * d.R * d.S * Cp, 0);
  const size_t taps = static_cast<size_t>(d.R) * d.S;
  for (int k = 0; k < d.K; ++k)
    for (size_t t = 0; t < taps; ++t)
      for (int c = 0; c < d.C; ++c) {
        int beta = np_host_decode(w_codes_host[(static_cast<size_t>(k) * taps + t) * d.C + c], d.n_w, d.p_w);
        for (int j = 0; j < pw; ++j) {
          const int dig = j + 1 < pw ? ((beta + 64) & 127) - 64 : beta;
          beta = (beta - dig) >> 7;
          for (int i = 0; i < px; ++i)
            wp[((static_cast<size_t>(i + j) * d.K + k) * taps + t) * Cp + static_cast<size_t>(i) * d.C + c] = static_cast<int8_t>(dig);
        }
      }
  qconv_np_handle* h = new qconv_np_handle();
  h->d = d; h->planes_x = px; h->planes_w = pw; h->groups = groups; h->P = P; h->Q = Q;
  h->fout = qc::NpFormat{d.n_out, d.p_out, bmax[2]};
  qconv_desc g = {};
  g.N = d.N; g.H = d.H; g.W = d.W; g.C = Cp; g.K = Kp; g.R = d.R; g.S = d.S;
  g.stride_h = d.stride_h; g.stride_w = d.stride_w; g.pad_h = d.pad_h; g.pad_w = d.pad_w; g.groups = 1;
  g.n_in = 8; g.n_w = 8; g.n_out = 8; g.symmetric = 1; g.out_mode = QCONV_OUT_INT32;
  int rc = qconv_create(&h->gemm, &g, wp.data(), nullptr, nullptr, nullptr, nullptr);
  if (rc) { free_np(h); return rc; }
  std::vector<int32_t> sh(d.K, 0), bi(d.K, 0);
  if (shift_host) std::memcpy(sh.data(), shift_host, sizeof(int32_t) * d.K);
  if (bias_host) std::memcpy(bi.data(), bias_host, sizeof(int32_t) * d.K);
  cudaError_t e = cudaMalloc(&h->d_planes, static_cast<size_t>(d.N) * d.H * d.W * Cp);
  if (e == cudaSuccess) e = cudaMalloc(&h->d_acc, acc_elems * sizeof(int32_t));
  if (e == cudaSuccess) e = cudaMalloc(&h->d_bias, sizeof(int32_t) * d.K);
  if (e == cudaSuccess) e = cudaMalloc(&h->d_shift, sizeof(int32_t) * d.K);
  if (e == cudaSuccess) e = cudaMemcpy(h->d_bias, bi.data(), sizeof(int32_t) * d.K, cudaMemcpyHostToDevice);
  if (e == cudaSuccess) e = cudaMemcpy(h->d_shift, sh.data(), sizeof(int32_t) * d.K, cudaMemcpyHostToDevice);
  if (e != cudaSuccess) {
    free_np(h);
    return fail(QCONV_ERR_CUDA, "qconv_np_create: %s", cudaGetErrorString(e));
  }
  *out = h;
  return QCONV_OK;
}

int qconv_np_run(qconv_np_handle* h, const uint8_t* d_x_codes, uint8_t* d_y_codes, int n_run, void* cuda_stream) {
  if (!h || !d_x_codes || !d_y_codes) return fail(QCONV_ERR_BAD_ARG, "NULL handle or tensor pointer");
  const qconv_np_desc& d = h->d;
  if (n_run <= 0 || n_run > d.N) return fail(QCONV_ERR_BAD_ARG, "n_run %d outside [1, %d]", n_run, d.N);
  if (reinterpret_cast<uintptr_t>(d_x_codes) & 15) return fail(QCONV_ERR_ALIGNMENT, "d_x_codes must be 16-byte aligned");
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  const size_t in_pix = static_cast<size_t>(n_run) * d.H * d.W, out_pix = static_cast<size_t>(n_run) * h->P * h->Q;
  CUDA_TRY(launch_chained(qc::np_split_kernel, dim3(grid_for(in_pix * (d.C / 16), 256, 148 * 16)), dim3(256), 0, st,
                          d_x_codes, h->d_planes, in_pix, d.C, d.n_in, d.p_in, h->planes_x));
  int rc = qconv_run(h->gemm, h->d_planes, nullptr, h->d_acc, n_run, cuda_stream);
  if (rc) return rc;
  qc::np_combine_kernel<<<grid_for(out_pix * d.K, 256, 148 * 16), 256, 0, st>>>(h->d_acc, h->d_bias, h->d_shift, d_y_codes,
                                                                                  out_pix, d.K, h->groups, d.relu, h->fout);
  CUDA_TRY(cudaGetLastError());
  return QCONV_OK;
}

int qconv_np_status(qconv_np_handle* h) {
  if (!h) return fail(QCONV_ERR_BAD_ARG, "NULL handle");
  return qconv_status(h->gemm);
}

int qconv_np_describe(const qconv_np_handle* h, char* buf, size_t buf_len) {
  if (!h || !buf || buf_len == 0) return fail(QCONV_ERR_BAD_ARG, "NULL argument");
  char inner[256];
  qconv_describe(h->gemm, inner, sizeof(inner));
  snprintf(buf, buf_len, "np planes_x=%d planes_w=%d groups=%d | %s", h->planes_x, h->planes_w, h->groups, inner);
  return QCONV_OK;
}

int qconv_np_destroy(qconv_np_handle* h) {
  if (!h) return fail(QCONV_ERR_BAD_ARG, "NULL handle");
  free_np(h);
  return QCONV_OK;
}

// --------------------------------------------------------------------------- Algorithm 1
int qfpspace(int n, int p, double* out_host, int* count_out) {
  if (!out_host || !count_out) return fail(QCONV_ERR_BAD_ARG, "NULL argument");
  if (n < 2 || n > 8 || p < 0 || p > n - 1) return fail(QCONV_ERR_BAD_ARG, "need 2 <= n <= 8 and 0 <= p <= n-1");
  // Non-negative patterns 0 .. 2^(n-1)-1 decode (Eq. 2, exponent field per Eq. 4) to strictly
  // ascending values: subnormals are the significand itself, a normal number with exponent
  // field E is (2^p + significand) * 2^(E-1), and E = 1 continues where the subnormals end.
  const int levels = 1 << (n - 1);
  const int sig_mask = (1 << p) - 1;
  for (int b = 0; b < levels; ++b) {
    const int E = (p == n - 1) ? 0 : (b >> p);
    const int m = b & sig_mask;
    out_host[b] = E == 0 ? static_cast<double>(m) : std::ldexp(static_cast<double>((1 << p) + m), E - 1);
  }
  const double top = out_host[levels - 1];            // beta_max of Eq. 5
  for (int b = 0; b < levels; ++b) out_host[b] /= top;
  *count_out = levels;
  return QCONV_OK;
}

int qthreshold_search(const uint64_t* hist_host, int nbins, float range_hi, int n, int p, int measure,
                      double* gamma_out, double* delta_out, int* index_out, double* deltas_host, void* cuda_stream) {
  if (!hist_host || !gamma_out || !delta_out || !index_out) return fail(QCONV_ERR_BAD_ARG, "NULL argument");
  if (n < 2 || n > 8 || p < 0 || p > n - 1) return fail(QCONV_ERR_BAD_ARG, "need 2 <= n <= 8 and 0 <= p <= n-1");
  if (measure < 0 || measure > 3) return fail(QCONV_ERR_BAD_ARG, "measure in [0, 3]");
  const int first = (1 << (n - 1)) + 1;
  if (nbins < first || nbins > qc::kThrMaxBins)
    return fail(QCONV_ERR_BAD_ARG, "nbins %d outside [2^(n-1)+1 = %d, %d]", nbins, first, qc::kThrMaxBins);
  if (!(range_hi > 0.0f) || std::isinf(range_hi)) return fail(QCONV_ERR_BAD_ARG, "range_hi must be positive and finite");
  bool any = false;
  for (int j = 0; j < nbins && !any; ++j) any = hist_host[j] != 0;
  if (!any) return fail(QCONV_ERR_BAD_ARG, "empty histogram");
  double fp_host[qc::kThrMaxLevels];
  int levels = 0;
  int rc = qfpspace(n, p, fp_host, &levels);
  if (rc != QCONV_OK) return rc;

  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  // device scratch sized for the largest histogram, allocated once per device and kept
  const size_t off_cdf = sizeof(uint64_t) * qc::kThrMaxBins;
  const size_t off_fp = off_cdf + sizeof(double) * qc::kThrMaxBins;
  const size_t off_del = off_fp + sizeof(double) * qc::kThrMaxLevels;
  const size_t off_best = off_del + sizeof(double) * (qc::kThrMaxBins + 1);
  static std::mutex mu;
  static unsigned char* scratch[64] = {nullptr};
  int dev = 0;
  CUDA_TRY(cudaGetDevice(&dev));
  if (dev < 0 || dev >= 64) return fail(QCONV_ERR_CUDA, "device index %d out of range", dev);
  std::lock_guard<std::mutex> lock(mu);                    // calls on one device share the scratch: serialised
  if (!scratch[dev]) CUDA_TRY(cudaMalloc(&scratch[dev], off_best + sizeof(qc::ThresholdBest)));
  unsigned char* d = scratch[dev];
  auto* d_hist = reinterpret_cast<unsigned long long*>(d);
  auto* d_cdf = reinterpret_cast<double*>(d + off_cdf);
  auto* d_fp = reinterpret_cast<double*>(d + off_fp);
  auto* d_del = reinterpret_cast<double*>(d + off_del);
  auto* d_best = reinterpret_cast<qc::ThresholdBest*>(d + off_best);
  qc::ThresholdBest best = {};
  cudaError_t e = cudaMemcpyAsync(d_hist, hist_host, sizeof(uint64_t) * nbins, cudaMemcpyHostToDevice, st);
  if (e == cudaSuccess) e = cudaMemcpyAsync(d_fp, fp_host, sizeof(double) * levels, cudaMemcpyHostToDevice, st);
  if (e == cudaSuccess) e = cudaMemsetAsync(d_del, 0xFF, sizeof(double) * (nbins + 1), st);   // NaN outside the loop's range
  if (e == cudaSuccess) {
    qc::threshold_cdf_kernel<<<1, 1024, 0, st>>>(d_hist, nbins, d_cdf);
    qc::threshold_candidates_kernel<<<nbins - first + 1, qc::kThrThreads, 0, st>>>(d_cdf, d_fp, nbins, levels, first,
                                                                                  measure, std::ldexp(1.0, -52), d_del);
    qc::threshold_argmin_kernel<<<1, qc::kThrThreads, 0, st>>>(d_del, first, nbins, d_best);
    e = cudaGetLastError();
  }
  if (e == cudaSuccess) e = cudaMemcpyAsync(&best, d_best, sizeof(best), cudaMemcpyDeviceToHost, st);
  if (e == cudaSuccess && deltas_host)
    e = cudaMemcpyAsync(deltas_host, d_del, sizeof(double) * (nbins + 1), cudaMemcpyDeviceToHost, st);
  if (e == cudaSuccess) e = cudaStreamSynchronize(st);
  if (e != cudaSuccess) return fail(QCONV_ERR_CUDA, "qthreshold_search: %s", cudaGetErrorString(e));
  *index_out = best.index;
  *delta_out = best.delta;
  // bin_edges[i] of nbins equal bins on [0, range_hi]; the last edge is range_hi itself
  const double hi = static_cast<double>(range_hi);
  *gamma_out = best.index == nbins ? hi : static_cast<double>(best.index) * (hi / nbins);
  return QCONV_OK;
}

// --------------------------------------------------------------------------- machine measurement
int qbench_mma_i8(int bn, int mmas_per_cta, int row_bytes, int commit_every, float* ms_out, double* cycles_per_mma_out, int* ctas_out,
                  void* cuda_stream) {
  if (!ms_out || !cycles_per_mma_out || !ctas_out) return fail(QCONV_ERR_BAD_ARG, "NULL argument");
  if (bn < 16 || bn > 256 || bn % 16 || mmas_per_cta < 4 || mmas_per_cta > (1 << 20) || mmas_per_cta % 4)
    return fail(QCONV_ERR_BAD_ARG, "bn in [16, 256] multiple of 16; mmas_per_cta in [4, 2^20] multiple of 4");
  if (row_bytes != 128 && row_bytes != 64 && row_bytes != 32) return fail(QCONV_ERR_BAD_ARG, "row_bytes is 128, 64 or 32");
  if (commit_every < 0 || commit_every % 4) return fail(QCONV_ERR_BAD_ARG, "commit_every is 0 or a multiple of 4");
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  int dev = 0, sms = 0;
  CUDA_TRY(cudaGetDevice(&dev));
  CUDA_TRY(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
  const size_t smem = 1024 + static_cast<size_t>(qc::kTileM + bn) * 128 + sizeof(qc::MmaPeakShared);
  CUDA_TRY(cudaFuncSetAttribute(qc::mma_peak_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024));
  unsigned long long* d_cycles = nullptr;
  int* d_status = nullptr;
  CUDA_TRY(cudaMalloc(&d_cycles, sizeof(unsigned long long) * sms));
  cudaError_t e = cudaMalloc(&d_status, sizeof(int));
  cudaEvent_t e0 = nullptr, e1 = nullptr;
  if (e == cudaSuccess) e = cudaMemsetAsync(d_status, 0, sizeof(int), st);
  if (e == cudaSuccess) e = cudaEventCreate(&e0);
  if (e == cudaSuccess) e = cudaEventCreate(&e1);
  std::vector<unsigned long long> cyc(sms, 0);
  int status = 0;
  float ms = 0.0f;
  if (e == cudaSuccess) {
    // one CTA per SM (the shared-memory request above half an SM's keeps a second one out)
    const size_t smem_one = std::max<size_t>(smem, 120 * 1024);
    qc::mma_peak_kernel<<<sms, qc::kPeakThreads, smem_one, st>>>(bn, mmas_per_cta, row_bytes, commit_every, d_cycles, d_status, 1u << 26);   // warm-up
    cudaEventRecord(e0, st);
    qc::mma_peak_kernel<<<sms, qc::kPeakThreads, smem_one, st>>>(bn, mmas_per_cta, row_bytes, commit_every, d_cycles, d_status, 1u << 26);
    cudaEventRecord(e1, st);
    e = cudaGetLastError();
  }
  if (e == cudaSuccess) e = cudaEventSynchronize(e1);
  if (e == cudaSuccess) e = cudaEventElapsedTime(&ms, e0, e1);
  if (e == cudaSuccess) e = cudaMemcpy(cyc.data(), d_cycles, sizeof(unsigned long long) * sms, cudaMemcpyDeviceToHost);
  if (e == cudaSuccess) e = cudaMemcpy(&status, d_status, sizeof(int), cudaMemcpyDeviceToHost);
  if (e0) cudaEventDestroy(e0);
  if (e1) cudaEventDestroy(e1);
  cudaFree(d_cycles);
  cudaFree(d_status);
  if (e != cudaSuccess) return fail(QCONV_ERR_CUDA, "qbench_mma_i8: %s", cudaGetErrorString(e));
  if (status != 0) return fail(QCONV_ERR_TIMEOUT, "qbench_mma_i8: the MMA train did not finish within the wait limit");
  double sum = 0.0;
  for (int i = 0; i < sms; ++i) sum += static_cast<double>(cyc[i]);
  *ms_out = ms;
  *cycles_per_mma_out = sum / sms / mmas_per_cta;
  *ctas_out = sms;
  return QCONV_OK;
}

// --------------------------------------------------------------------------- host helpers
int qscale_exponent(float gamma, int n, int* e_out) {
  if (!e_out || n < 2 || n > 8) return fail(QCONV_ERR_BAD_ARG, "e_out NULL or n outside [2, 8]");
  *e_out = 0;
  if (!(gamma > 0.0f) || std::isinf(gamma)) return QCONV_OK;
  // gamma = m * 2^ex with m in [0.5, 1).  beta_max * 2^e >= gamma  <=>  2^e >= gamma / beta_max.
  // Start one below the answer's lower bound and step up with exact comparisons.
  int ex;
  std::frexp(gamma, &ex);
  const double bmax = static_cast<double>((1 << (n - 1)) - 1);
  int e = ex - n;                       // beta_max * 2^(ex-n) < 2^(ex-1) <= gamma
  while (std::ldexp(bmax, e) < static_cast<double>(gamma)) ++e;
  *e_out = e;
  return QCONV_OK;
}

// Exponent bookkeeping of Section 3 (alpha = 2^e everywhere, so every factor is a shift).
int qacc_exponents(int e_x, const int32_t* e_w_host, int K, int32_t* acc_exp_host) {
  if (!e_w_host || !acc_exp_host || K <= 0) return fail(QCONV_ERR_BAD_ARG, "NULL argument or K <= 0");
  for (int k = 0; k < K; ++k) acc_exp_host[k] = e_x + e_w_host[k];
  return QCONV_OK;
}

int qrequant_shifts(int e_z, const int32_t* acc_exp_host, int K, int32_t* shift_host) {
  if (!acc_exp_host || !shift_host || K <= 0) return fail(QCONV_ERR_BAD_ARG, "NULL argument or K <= 0");
  for (int k = 0; k < K; ++k) {
    const long long sft = static_cast<long long>(e_z) - acc_exp_host[k];
    if (sft < 0 || sft > 31)
      return fail(QCONV_ERR_BAD_SHIFT, "shift[%d] = e_z - (e_x + e_w) = %lld outside [0, 31]", k, sft);
    shift_host[k] = static_cast<int32_t>(sft);
  }
  return QCONV_OK;
}

int qresidual_shifts(int e_res, const int32_t* acc_exp_host, int K, int32_t* lshift_host) {
  if (!acc_exp_host || !lshift_host || K <= 0) return fail(QCONV_ERR_BAD_ARG, "NULL argument or K <= 0");
  for (int k = 0; k < K; ++k) {
    const long long t = static_cast<long long>(e_res) - acc_exp_host[k];
    if (t < 0 || t > 23)
      return fail(QCONV_ERR_RESIDUAL_SCALE, "res_lshift[%d] = e_res - (e_x + e_w) = %lld outside [0, 23]", k, t);
    lshift_host[k] = static_cast<int32_t>(t);
  }
  return QCONV_OK;
}

int qjoin_exponent(const int32_t* e_own_host, const int32_t* const* acc_exp_hosts, const int32_t* K_host,
                   int n_branches, int* e_z_out) {
  if (!e_own_host || !acc_exp_hosts || !K_host || !e_z_out || n_branches <= 0)
    return fail(QCONV_ERR_BAD_ARG, "NULL argument or no branch");
  long long e_z = e_own_host[0];
  for (int b = 0; b < n_branches; ++b) {
    if (!acc_exp_hosts[b] || K_host[b] <= 0) return fail(QCONV_ERR_BAD_ARG, "branch %d: NULL exponents or K <= 0", b);
    e_z = std::max<long long>(e_z, e_own_host[b]);
    for (int k = 0; k < K_host[b]; ++k) e_z = std::max<long long>(e_z, acc_exp_hosts[b][k]);
  }
  *e_z_out = static_cast<int>(e_z);
  return QCONV_OK;
}

// Packed storage of n-bit betas: value i is the n-bit two's-complement field at bits [i n, (i + 1) n) of a
// little-endian bit stream.
int qpack_weights(const int8_t* wq_host, size_t count, int n, uint8_t* packed_host) {
  if (!wq_host || !packed_host || n < 2 || n > 8) return fail(QCONV_ERR_BAD_ARG, "NULL argument or n outside [2, 8]");
  const int lo = -(1 << (n - 1)), hi = (1 << (n - 1)) - 1;
  std::memset(packed_host, 0, (count * n + 7) / 8);
  for (size_t i = 0; i < count; ++i) {
    if (wq_host[i] < lo || wq_host[i] > hi) return fail(QCONV_ERR_BAD_ARG, "value %d at %zu does not fit %d bits", wq_host[i], i, n);
    const unsigned field = static_cast<unsigned>(wq_host[i]) & ((1u << n) - 1);
    const size_t bit = i * n;
    const unsigned sh = static_cast<unsigned>(bit & 7);
    packed_host[bit >> 3] |= static_cast<uint8_t>(field << sh);
    if (sh + n > 8) packed_host[(bit >> 3) + 1] |= static_cast<uint8_t>(field >> (8 - sh));
  }
  return QCONV_OK;
}

int qunpack_weights(const uint8_t* packed_host, size_t count, int n, int8_t* wq_host) {
  if (!wq_host || !packed_host || n < 2 || n > 8) return fail(QCONV_ERR_BAD_ARG, "NULL argument or n outside [2, 8]");
  const size_t nbytes = (count * n + 7) / 8;
  for (size_t i = 0; i < count; ++i) {
    const size_t bit = i * n;
    unsigned two = packed_host[bit >> 3];
    if ((bit >> 3) + 1 < nbytes) two |= static_cast<unsigned>(packed_host[(bit >> 3) + 1]) << 8;
    const unsigned field = (two >> (bit & 7)) & ((1u << n) - 1);
    wq_host[i] = static_cast<int8_t>((field >> (n - 1)) ? static_cast<int>(field) - (1 << n) : static_cast<int>(field));
  }
  return QCONV_OK;
}

int qconv_create_packed(qconv_handle** out, const qconv_desc* desc, const uint8_t* w_packed_host,
                        const int32_t* bias_host, const int32_t* shift_host, const int32_t* res_lshift_host,
                        const int32_t* acc_exp_host) {
  if (!out) return fail(QCONV_ERR_BAD_ARG, "out is NULL");
  *out = nullptr;
  if (!desc || !w_packed_host) return fail(QCONV_ERR_BAD_ARG, "desc or w_packed_host is NULL");
  if (desc->n_w < 2 || desc->n_w > 8 || desc->K <= 0 || desc->R <= 0 || desc->S <= 0 || desc->C <= 0 || desc->groups <= 0 ||
      desc->C % desc->groups)
    return fail(QCONV_ERR_BAD_ARG, "bad weight geometry or n_w outside [2, 8]");
  const size_t count = static_cast<size_t>(desc->K) * desc->R * desc->S * (desc->C / desc->groups);
  std::vector<int8_t> w(count);
  int rc = qunpack_weights(w_packed_host, count, desc->n_w, w.data());
  if (rc) return rc;
  return qconv_create(out, desc, w.data(), bias_host, shift_host, res_lshift_host, acc_exp_host);
}

namespace {
int8_t host_quantize_one(float v, int e, int n) {
  const float bmax = static_cast<float>((1 << (n - 1)) - 1);
  if (std::isnan(v)) return 0;
  const float gam = std::ldexp(bmax, e);
  v = std::fmin(std::fmax(v, -gam), gam);
  float r = std::nearbyint(std::ldexp(v, -e));
  r = std::fmin(std::fmax(r, -bmax), bmax);
  return static_cast<int8_t>(r);
}
}  // namespace

int qquantize_weights(const float* w_host, int K, int R, int S, int Cg, int layout, int per_channel, int n,
                      int8_t* wq_host, int32_t* e_w_host) {
  if (!w_host || !wq_host || !e_w_host) return fail(QCONV_ERR_BAD_ARG, "NULL argument");
  if (K <= 0 || R <= 0 || S <= 0 || Cg <= 0 || n < 2 || n > 8 || layout < 0 || layout > 1)
    return fail(QCONV_ERR_BAD_ARG, "bad weight geometry");
  const size_t per_k = static_cast<size_t>(R) * S * Cg;
  auto at = [&](int k, size_t j) { return layout == 0 ? k * per_k + j : j * K + k; };
  float gall = 0.0f;
  std::vector<float> gk(K, 0.0f);
  for (int k = 0; k < K; ++k) {
    float g = 0.0f;
    for (size_t j = 0; j < per_k; ++j) {
      float a = std::fabs(w_host[at(k, j)]);
      if (std::isfinite(a)) g = std::max(g, a);
    }
    gk[k] = g;
    gall = std::max(gall, g);
  }
  for (int k = 0; k < K; ++k) {
    int e;
    qscale_exponent(per_channel ? gk[k] : gall, n, &e);
    e_w_host[k] = e;
    for (size_t j = 0; j < per_k; ++j) wq_host[at(k, j)] = host_quantize_one(w_host[at(k, j)], e, n);
  }
  return QCONV_OK;
}

int qquantize_bias(const float* b_host, int K, int e_x, const int32_t* e_w_host, int32_t* bias_q_host) {
  if (!b_host || !e_w_host || !bias_q_host || K <= 0) return fail(QCONV_ERR_BAD_ARG, "NULL argument");
  for (int k = 0; k < K; ++k) {
    double r = std::nearbyint(std::ldexp(static_cast<double>(b_host[k]), -(e_x + e_w_host[k])));
    if (std::isnan(r)) r = 0.0;
    r = std::min(2147483647.0, std::max(-2147483648.0, r));
    bias_q_host[k] = static_cast<int32_t>(r);
  }
  return QCONV_OK;
}

}  // extern "C"

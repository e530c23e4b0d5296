/*
 * qconv.h -- C ABI of the B200 quantized-convolution library.
 *
 * The library implements, as CUDA kernels for sm_100a, the integer special case of the
 * quantization scheme of Settle et al., "Quantizing Convolutional Neural Networks for
 * Low-Power High-Throughput Inference Engines" (2018): every tensor is alpha * beta with
 * beta an n-bit signed integer (n <= 8, stored one value per int8) and alpha = 2^e.
 *
 * Conventions
 *   - Activations are NHWC int8; weights int8; bias int32; accumulation int32 (create-time
 *     validation guarantees it never overflows, Eq. 8-9).
 *   - Pointers named d_* are DEVICE pointers owned by the caller; the library never frees or
 *     reallocates them.  Pointers named *_host / h_* are HOST pointers; their contents are
 *     copied during the call.
 *   - `cuda_stream` is a cudaStream_t passed as void* (NULL = the default stream).
 *   - Every function returns 0 (QCONV_OK) or a negative qconv_error; nothing aborts, throws
 *     or traps.  qconv_last_error_string() gives a text for the calling thread's last error.
 *   - A handle may be used from one host thread at a time.
 */
#ifndef QCONV_H_
#define QCONV_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  QCONV_OK = 0,
  QCONV_ERR_BAD_ARG = -1,           /* null pointer, non-positive size, unknown enum value         */
  QCONV_ERR_UNSUPPORTED_SHAPE = -2, /* groups do not divide C or K, empty output, forced algorithm
                                       cannot run this shape                                        */
  QCONV_ERR_OVERFLOW_RISK = -3,     /* dot-product length too long for a 32-bit accumulator (Eq. 9) */
  QCONV_ERR_BAD_SHIFT = -4,         /* a right shift outside [0, 31] (requant factors are in (0,1]) */
  QCONV_ERR_RESIDUAL_SCALE = -5,    /* a residual left shift outside [0, 23] (Eq. 10 needs
                                       alpha_residual >= alpha_accumulator)                         */
  QCONV_ERR_ALIGNMENT = -6,         /* device pointer or channel pitch not aligned as documented    */
  QCONV_ERR_CUDA = -7,              /* a CUDA runtime/driver call failed                            */
  QCONV_ERR_TIMEOUT = -8            /* a bounded device-side wait expired; outputs are undefined    */
} qconv_error;

enum { QCONV_ALGO_AUTO = 0, QCONV_ALGO_DIRECT = 1, QCONV_ALGO_IGEMM = 2, QCONV_ALGO_DEPTHWISE = 3 };
enum { QCONV_OUT_INT8 = 0, QCONV_OUT_INT32 = 1, QCONV_OUT_FLOAT = 2 };
enum { QCONV_ROUND_NEAREST_EVEN = 0, QCONV_ROUND_HALF_AWAY = 1, QCONV_ROUND_HALF_UP = 2,
       QCONV_ROUND_FLOOR = 3 };

/* One quantized convolution layer (Eq. 6 followed by the conversion of Section 3). */
typedef struct {
  int N, H, W, C;               /* input NHWC; N is the largest batch qconv_run may be given       */
  int K, R, S;                  /* K output channels, R x S filter taps                            */
  int stride_h, stride_w, pad_h, pad_w;
  int groups;                   /* C % groups == 0 and K % groups == 0; dilation is 1              */
  int n_in, n_w, n_out;         /* bit widths n of input, weight and output beta, each in [2, 8]   */
  int symmetric;                /* 1: saturate to +-(2^(n_out-1)-1) (the paper's symmetric range);
                                   0: lower bound -2^(n_out-1)                                     */
  int relu;                     /* 1: max(., 0) on the wide value before requantization            */
  int rounding;                 /* QCONV_ROUND_*; the paper does not name the mode, nearest-even is
                                   the default reading                                             */
  int out_mode;                 /* QCONV_OUT_INT8: requantized int8;
                                   QCONV_OUT_INT32: wide value after bias/residual/ReLU;
                                   QCONV_OUT_FLOAT: that wide value times 2^acc_exp[k] as float32
                                   (beta -> float, used by calibration)                            */
  int out_c_offset, out_c_pitch;/* the K channels are written at channel out_c_offset of an output
                                   buffer [N][P][Q][out_c_pitch] (concat in place); pitch 0 means K */
  int has_residual;             /* 1: an int8 tensor [N][P][Q][K] is added in int32 (Eq. 10)       */
  int weight_layout;            /* 0: [K][R][S][C/groups]; 1: [R][S][C/groups][K]                  */
  int algo;                     /* QCONV_ALGO_*; AUTO picks tensor-core implicit GEMM when
                                   groups == 1 and C % 16 == 0 (or C <= 4: packed stem), the
                                   depthwise kernel when groups == C == K, else the direct kernel  */
  int pool;                     /* 0, or 2: a 2 x 2 / stride 2 max-pool (no padding) of the layer's int8
                                   output taken inside the layer, which then writes
                                   [N][P/2][Q/2][out_c_pitch] and never the un-pooled tensor.  The
                                   conversion of Section 3 is non-decreasing in the wide value, so the
                                   maximum is taken on the accumulators and converted once: the result
                                   equals the layer followed by the pool, bit for bit.  Only for the
                                   tensor-core path with per-tap boxes (groups 1, C % 16 == 0, filter
                                   wider than 1 x 1 or strided), int8 output at 8 bits with nearest-even
                                   rounding, K % 16 == 0, no residual, P and Q even;
                                   UNSUPPORTED_SHAPE otherwise (run the pool as its own call then)   */
} qconv_desc;

typedef struct qconv_handle qconv_handle;

/* Plan overrides, for tests and experiments: which of the planner's forms qconv_create may choose.
 * The layer's result never depends on them, only the kernel, tile shape and data movement that
 * produce it.  -1 in a choice field (0 in the two size fields) leaves the decision to the planner.
 * qconv_set_plan_hints copies the struct for the CALLING THREAD; it applies to handles that thread
 * creates afterwards (each handle keeps its own copy) and to the launch attribute of the free
 * functions it calls.  NULL restores the planner's own choices. */
typedef struct {
  int halo;              /* 3x3 stride-1 layers, one activation box per filter row serving its three
                            taps: 0 never, 1 wherever the shape allows (also with 128-wide tiles)  */
  int window_rows;       /* wide filters on few channels read as window rows of a padded copy: 0 never */
  int space_to_depth;    /* stride-2 layers on <= 4 channels in space-to-depth form: 0 never (packed
                            patch rows instead)                                                     */
  int resident_weights;  /* a CTA's weight tile loaded once and kept: 0 never, 1 whenever it fits   */
  int fold;              /* several pixels per GEMM row for narrow layers: 0 never                  */
  int fast_epilogue;     /* the 16-byte-store int8 epilogues: 0 = the general epilogue              */
  int float_rounding;    /* requantization by one fp32 FMA where provably exact: 0 = integer form   */
  int uniform_shift;     /* the instantiation for one shift per layer: 0 = per-channel constants    */
  int tma_store;         /* output tiles staged in shared memory and stored by TMA: 0 never, 1 wherever they fit */
  int tma_residual;      /* residual tiles fetched by TMA into the staged tiles: 0 never            */
  int depthwise_form;    /* 0: general dp4a kernel, 1: tap-packed kernel with register loads (no TMA rows) */
  int pdl;               /* programmatic dependent launch: 0 off                                    */
  int group_taps;        /* 3x3-like layers on at most 64 channels, the taps of a filter row sharing
                            one ring stage: 0 never, 1 wherever the shape allows                    */
  int pair_tiles;        /* tiles of 256 pixels x 256 channels on pairs of SMs (needs the 256-wide form):
                            0 never, 1 wherever the shape allows                                    */
  int bn_max;            /* 0, or the widest channel tile (multiple of 16): up to 128, or 256 to take
                            256-wide tiles (one CTA per SM) wherever the layer's shape allows them  */
  int ctas_per_sm;       /* 0, or 1 / 2 resident CTAs per SM for the tensor-core kernel             */
} qconv_plan_hints;
int qconv_set_plan_hints(const qconv_plan_hints* hints);

/* Build a layer.  Copies and repacks the host arrays onto the current CUDA device; the handle
 * owns those copies and any scratch it needs.
 *   w_host          int8 weights, layout per desc, K*R*S*C/groups values
 *   bias_host       K int32 at scale 2^(e_x + e_w[k]) (bias folded into the convolution,
 *                   Section 3), or NULL for zero bias
 *   shift_host      K right shifts s[k] = e_z - e_x - e_w[k] in [0, 31], or NULL for all zero
 *   res_lshift_host K left shifts t[k] = e_res - e_x - e_w[k] in [0, 23]; required iff has_residual
 *   acc_exp_host    K exponents e_x + e_w[k] in [-126, 96]; read only by QCONV_OUT_FLOAT; NULL means 0
 * Errors: BAD_ARG, UNSUPPORTED_SHAPE, OVERFLOW_RISK when
 *   (R*S*C/groups) * 2^(n_in-1) * 2^(n_w-1) + max|bias| + 2^(7 + max t) > 2^31 - 1,
 * BAD_SHIFT, RESIDUAL_SCALE, ALIGNMENT, CUDA.  On error *out is NULL. */
int qconv_create(qconv_handle** out, const qconv_desc* desc, const int8_t* w_host,
                 const int32_t* bias_host, const int32_t* shift_host,
                 const int32_t* res_lshift_host, const int32_t* acc_exp_host);

/* Run the layer on n_run <= desc.N images, asynchronously on cuda_stream.
 *   d_x        int8 [n_run][H][W][C], 16-byte aligned
 *   d_residual int8 [n_run][P][Q][K] or NULL (must match has_residual)
 *   d_y        [n_run][P][Q][out_c_pitch] of int8 / int32 / float32 per out_mode; only the K
 *              channels of this layer are written ([n_run][P/2][Q/2][out_c_pitch] with desc.pool)
 * Layers on at most 4 input channels, and stride-1 layers with filters at least four taps wide on
 * at most 64 channels, first repack d_x into scratch the handle owns (one more small kernel on the
 * same stream); the handle also caches tensor maps for the last pointers it saw.  Hence one
 * handle must not run on two streams at once: give each concurrent stream a handle of its own.
 * Device-side waits are bounded; if one expires the kernel stops early and the handle's status
 * becomes QCONV_ERR_TIMEOUT (read it with qconv_status).  Errors: BAD_ARG, ALIGNMENT, CUDA. */
int qconv_run(qconv_handle* h, const int8_t* d_x, const int8_t* d_residual, void* d_y,
              int n_run, void* cuda_stream);

/* The same layer on the float image: the input conversion of Section 3 (clamp to +-gamma =
 * beta_max 2^e_x, scale by 2^-e_x, round to nearest even, clamp to +-beta_max at n_in bits; NaN -> 0,
 * exactly qquantize_f32) is done inside the kernel that repacks the layer's input, so the int8 image
 * is never written.  Only for layers that repack their input: C <= 4 with stride 2 in both directions
 * (space-to-depth form) or stride 1 (padded rows), the stems of the paper's networks;
 * UNSUPPORTED_SHAPE otherwise.
 *   d_x_f32  float32 [n_run][H][W][C], 4-byte aligned;  e_x in [-126, 126]
 * Other arguments, asynchrony and errors as qconv_run. */
int qconv_run_f32(qconv_handle* h, const float* d_x_f32, int e_x, const int8_t* d_residual, void* d_y,
                  int n_run, void* cuda_stream);

/* Synchronise the stream of the last qconv_run and return its device status (QCONV_OK or
 * QCONV_ERR_TIMEOUT), clearing it. */
int qconv_status(qconv_handle* h);

/* Test hook: cap on the polls of each device-side barrier wait (default 1 << 22; one poll may suspend
 * the waiting thread for up to about two microseconds, so the default gives up after seconds).  With 0 every
 * wait gives up at once: the kernel still issues the copies that need no wait, lets them land,
 * writes an undefined output (or none) and the layer's status becomes QCONV_ERR_TIMEOUT. */
int qconv_set_wait_limit(qconv_handle* h, unsigned int polls);

/* Writes a one-line description of the plan (algorithm, tile shape, stages) into buf. */
int qconv_describe(const qconv_handle* h, char* buf, size_t buf_len);

int qconv_destroy(qconv_handle* h);

/* Calibration statistics over one batch of float activations (first step of Algorithm 1,
 * hist(abs(x)), and the maximum that Section 3 names as the default threshold). */
typedef struct {
  float maxabs;          /* max |x| over finite x (0 if none)                                     */
  float range_hi;        /* upper edge of the histogram actually used                              */
  uint64_t count;        /* number of finite values                                                */
  uint64_t nonfinite;    /* NaN / Inf values, excluded from everything else                        */
  double sum, sumsq;     /* fp64 sums over finite values                                           */
  uint64_t* hist;        /* HOST array of nbins counters, provided by the caller                   */
} qcalib_stats;

/* d_x: `count` float32 on the device (4-byte aligned).  nbins in [1, 4096].
 * range_hi > 0 fixes the histogram range to [0, range_hi] (larger |x| land in the last bin);
 * range_hi <= 0 uses [0, max|x|] (max found in a first pass).  bin = min(nbins-1,
 * (int)(|x| * ((float)nbins / hi))) in fp32.  Synchronous: host_out is complete on return.
 * Uses a per-device scratch buffer allocated on first use. */
int qcalib_collect(const float* d_x, size_t count, int nbins, float range_hi,
                   qcalib_stats* host_out, void* cuda_stream);

/* The same statistics as qcalib_collect for callers that must not allocate device memory.  (The
 * paper has no counterpart to this call; it exists for the way the library gets embedded.)
 *
 * Who needs it: a serving process that fixes its device memory layout at start-up and forbids
 * cudaMalloc afterwards -- an allocation synchronises the whole device, stalls every stream of a
 * latency-bound server, and can fail late once a framework's caching allocator has claimed the
 * GPU -- and plug-in style hosts that give a library no memory budget of its own.  qcalib_collect
 * allocates its scratch with cudaMalloc on first use per device; this variant never calls
 * cudaMalloc, cudaFree or any allocating routine.
 *
 * Its scratch (running maximum, counters, fp64 partial sums, histogram) is a fixed array built into
 * the library image: about 64 KB of global memory on every GPU that loads the library, held until
 * the process exits.  That fixes the limits: nbins <= QCALIB_STATIC_MAX_BINS and
 * count <= QCALIB_STATIC_MAX_COUNT; anything larger returns QCONV_ERR_BAD_ARG with a message and
 * touches nothing.  Arguments, results and rounding are otherwise those of qcalib_collect.
 *
 * The first call on each device looks up the array's device address (a query, no allocation; if it
 * is the first call into the library on that device, CUDA may load the library's device code --
 * the array with it -- at that moment, so it belongs in start-up); make that first call before any
 * stream capture begins.  All calls on a device share
 * the one array: each call clears the counters it accumulates into before it starts, and two calls
 * whose kernels overlap on the GPU (different streams, or different host threads) race on it and
 * return garbage -- serialise them. */
#define QCALIB_STATIC_MAX_BINS 4096
#define QCALIB_STATIC_MAX_COUNT ((size_t)1 << 40)
int qcalib_collect_static(const float* d_x, size_t count, int nbins, float range_hi,
                          qcalib_stats* host_out, void* cuda_stream);

/* float -> beta on the device (Section 3): clamp to +-beta_max * 2^e, scale by 2^-e, round to
 * nearest even, clamp to +-beta_max; NaN -> 0.  d_x float32, d_y int8, `count` values. */
int qquantize_f32(const float* d_x, size_t count, int e, int n, int8_t* d_y, void* cuda_stream);

/* float <-> general n-bit dynamic floating-point codes with p significand bits (Section 2.1, Eq. 2,
 * 4, 5; conversion per Section 3), scale alpha = 2^e.  A code is the sign-and-magnitude pattern of
 * Eq. 2 in one byte (bit n-1 sign, then n-p-1 exponent bits, then p significand bits); p = n-1 is
 * the integer type in sign-magnitude form (the convolution path stores the same values as two's
 * complement bytes instead).  Encoding: |x| / 2^e clamped to beta_max, rounded to the nearest
 * representable value, ties to the even pattern; NaN -> code 0; a zero magnitude is always code 0.
 * Decoding: value * 2^e (exact unless it leaves the binary32 range).  2 <= n <= 8, 0 <= p <= n-1,
 * |e| <= 126.  d_x / d_y float32, d_code one byte per value, `count` values. */
int qquantize_f32_np(const float* d_x, size_t count, int e, int n, int p, uint8_t* d_code, void* cuda_stream);
int qdequantize_np(const uint8_t* d_code, size_t count, int e, int n, int p, float* d_y, void* cuda_stream);

/* Convolution on dynamic floating-point operands (the n-bit types with p significand bits of Section
 * 2.1; the discussion section recommends p = 4 or p = 3 for 8 bits).  Tensors hold the sign-and-magnitude
 * patterns of Eq. 2, one per byte, as qquantize_f32_np produces them; every tensor's scale is a power of
 * two, so Eq. 6 runs over the integer betas: acc[k] = sum beta_x beta_w (exact: the betas are split into
 * base-128 digits, multiplied on the int8 tensor cores and recombined in 64 bits) + bias[k]; ReLU; then
 * acc / 2^shift[k] is converted to the output type: nearest representable value, ties to the even
 * pattern, saturation at beta_max (Eq. 5), zero always pattern 0.
 *   desc        shapes as qconv_desc (groups = 1, dilation 1); (n, p) of input, weights and output
 *   w_codes_host  K*R*S*C patterns, layout [K][R][S][C]
 *   bias_host   K int32 at the scale 2^(e_x + e_w[k]) of the sum, or NULL
 *   shift_host  K right shifts s[k] = e_z - e_x - e_w[k] in [0, 40], or NULL for 0
 * Supported types: beta_max below 2^21 (three digit planes: every 8-bit type with p >= 3, all narrower
 * ones with at most 4 exponent bits); C a multiple of 16.  Errors: BAD_ARG, UNSUPPORTED_SHAPE, BAD_SHIFT,
 * OVERFLOW_RISK when R*S*C * beta_max_in * beta_max_w + max|bias| >= 2^62 (Eq. 9 with b = beta_max), CUDA.
 * The handle owns its scratch (digit planes of the input, int32 partial sums); one stream at a time. */
typedef struct {
  int N, H, W, C, K, R, S;
  int stride_h, stride_w, pad_h, pad_w;
  int n_in, p_in, n_w, p_w, n_out, p_out;
  int relu;
} qconv_np_desc;
typedef struct qconv_np_handle qconv_np_handle;
int qconv_np_create(qconv_np_handle** out, const qconv_np_desc* desc, const uint8_t* w_codes_host,
                    const int32_t* bias_host, const int32_t* shift_host);
/* d_x_codes [n_run][H][W][C] (16-byte aligned), d_y_codes [n_run][P][Q][K]; asynchronous on cuda_stream. */
int qconv_np_run(qconv_np_handle* h, const uint8_t* d_x_codes, uint8_t* d_y_codes, int n_run, void* cuda_stream);
int qconv_np_status(qconv_np_handle* h);
int qconv_np_describe(const qconv_np_handle* h, char* buf, size_t buf_len);
int qconv_np_destroy(qconv_np_handle* h);

/* int8 NHWC max-pool, window R x S, same stride and padding in both directions; taps outside
 * the image are ignored (max commutes with the monotone requantization, so pooling acts on
 * the codes).  d_y is [N][P][Q][C] with P = (H + 2 pad - R) / stride + 1. */
int qmaxpool_i8(const int8_t* d_x, int N, int H, int W, int C, int R, int S, int stride, int pad,
                int8_t* d_y, void* cuda_stream);

/* Stand-alone eltwise addition layer with per-input scales (Eq. 10, widths per Eq. 12-13):
 *   wide[j] = sum_i x_i[j] << lshift[i]      (lshift[i] = e_i - min_j e_j >= 0: exact at the finest scale)
 *   y[j]    = saturate(round(relu?(wide[j]) / 2^rshift))       (rshift = e_z - min_j e_j in [0, 31],
 *                                                               i.e. alpha_xi <= alpha_z for every input)
 * d_inputs_host: HOST array of n_inputs (1..8) DEVICE pointers to int8 tensors of `count` values;
 * lshift_host: n_inputs left shifts in [0, 23].  BAD_ARG / RESIDUAL_SCALE / BAD_SHIFT on bad
 * arguments, OVERFLOW_RISK when sum_i 128 << lshift[i] exceeds 2^31 - 1 (Eq. 13). */
int qeltwise_add_i8(const int8_t* const* d_inputs_host, int n_inputs, const int32_t* lshift_host,
                    int rshift, int relu, int rounding, int n_out, int symmetric, size_t count,
                    int8_t* d_y, void* cuda_stream);

/* Algorithm 1 (Section 3): threshold search on a histogram of abs(x), as qcalib_collect returns
 * it (nbins equal bins on [0, range_hi]).  For every candidate i = 2^(n-1)+1 .. nbins the cdf is
 * clipped (entries i-1 and later set to 1), its first i entries are resampled onto the (n, p)
 * grid fpspace(0, 1, n, p) and back onto the i bins by piecewise-linear interpolation, and
 * `measure` compares the result with the cdf; gamma is the bin edge i = range_hi * i / nbins of
 * the smallest measure (the lowest i among equal ones; the last edge if none is finite).
 * The paper does not define `measure`; offered are
 *   QTHRESHOLD_L1  mean |cdf - q|      QTHRESHOLD_KS   max |cdf - q|
 *   QTHRESHOLD_CVM mean (cdf - q)^2    QTHRESHOLD_KL   sum P ln(P / max(Q, 2^-52)) over the bin
 *                                                      masses P, Q of cdf and q, P > 0.
 * hist_host: HOST array of nbins counts, 2^(n-1)+1 <= nbins <= 4096, not all zero.
 * deltas_host: NULL, or HOST array of nbins+1 doubles receiving every candidate's measure (NaN
 * at indices outside the loop).  All arithmetic is float64 on the device; the device scratch (about
 * 100 KB) is allocated on the first call per device and kept; calls on one device are serialised;
 * the call returns after the results are on the host. */
#define QTHRESHOLD_L1 0
#define QTHRESHOLD_KS 1
#define QTHRESHOLD_CVM 2
#define QTHRESHOLD_KL 3
int qthreshold_search(const uint64_t* hist_host, int nbins, float range_hi, int n, int p, int measure,
                      double* gamma_out, double* delta_out, int* index_out, double* deltas_host,
                      void* cuda_stream);

/* Machine measurement, not a step of the method: issue rate of the int8 tensor-core instruction
 * the convolution kernel is built on (M = 128, N = bn, K = 32 per instruction).  One CTA per SM
 * issues mmas_per_cta instructions on operand tiles resident in shared memory -- no loads, no
 * epilogue -- so the result is the tensor pipe's own ceiling: ops = ctas * mmas_per_cta *
 * 2 * 128 * bn * 32 in *ms_out milliseconds (device time of one launch, after a warm-up launch);
 * *cycles_per_mma_out is the SM-clock count per instruction, averaged over the CTAs.  bn a multiple
 * of 16 in [16, 256]; mmas_per_cta a multiple of 4 in [4, 2^20].  Allocates and frees a few hundred
 * bytes of device scratch; synchronous.  Errors: BAD_ARG, CUDA, TIMEOUT. */
int qbench_mma_i8(int bn, int mmas_per_cta, int row_bytes, int commit_every, float* ms_out, double* cycles_per_mma_out, int* ctas_out,
                  void* cuda_stream);

/* Host helpers (pure CPU, deterministic). */

/* fpspace(0, 1, n, p) of Algorithm 1: the 2^(n-1) non-negative values of the n-bit type with p
 * significand bits (Eq. 2, exponent field per Eq. 4), ascending, divided by beta_max (Eq. 5).
 * out_host holds 2^(n-1) doubles; 2 <= n <= 8, 0 <= p <= n-1. */
int qfpspace(int n, int p, double* out_host, int* count_out);

/* Smallest e with (2^(n-1) - 1) * 2^e >= gamma (gamma = alpha * beta_max, Section 2.1);
 * gamma <= 0 or not finite gives 0. */
int qscale_exponent(float gamma, int n, int* e_out);

/* Exponent bookkeeping of Section 3 with alpha = 2^e (every scale factor is a shift).
 *   qacc_exponents    acc_exp[k] = e_x + e_w[k]: the scale of the wide value (input x weight scale,
 *                     also the scale of the folded bias).
 *   qrequant_shifts   s[k] = e_z - acc_exp[k]: the right shift that takes the wide value to the output
 *                     scale; BAD_SHIFT unless every s[k] is in [0, 31] (conversion factors lie in (0, 1]).
 *   qresidual_shifts  t[k] = e_res - acc_exp[k]: the left shift that brings a residual input to the
 *                     accumulator's scale (Eq. 10); RESIDUAL_SCALE unless every t[k] is in [0, 23].
 *   qjoin_exponent    the one output exponent of layers that write into the same tensor (channel
 *                     concatenation needs equal scales): the largest of the branches' own exponents
 *                     e_own[b] (from their thresholds) and of their accumulator exponents, so that no
 *                     branch needs a left shift.  acc_exp_hosts[b] points to K_host[b] exponents.
 * All arrays are HOST arrays. */
int qacc_exponents(int e_x, const int32_t* e_w_host, int K, int32_t* acc_exp_host);
int qrequant_shifts(int e_z, const int32_t* acc_exp_host, int K, int32_t* shift_host);
int qresidual_shifts(int e_res, const int32_t* acc_exp_host, int K, int32_t* lshift_host);
int qjoin_exponent(const int32_t* e_own_host, const int32_t* const* acc_exp_hosts, const int32_t* K_host,
                   int n_branches, int* e_z_out);

/* Weight thresholds = max |w| per output channel (Section 3) or per tensor (per_channel = 0);
 * w and wq hold K*R*S*Cg values in `layout` (0: [K][R][S][Cg], 1: [R][S][Cg][K]); e_w gets K
 * exponents. */
int qquantize_weights(const float* w_host, int K, int R, int S, int Cg, int layout,
                      int per_channel, int n, int8_t* wq_host, int32_t* e_w_host);

/* Packed storage of n-bit weights (Section 4.3 takes the weights down to 5 bits): value i is the n-bit
 * two's-complement field at bits [i*n, (i+1)*n) of a little-endian bit stream of ceil(count*n/8) bytes.
 * qpack_weights refuses values outside [-2^(n-1), 2^(n-1)-1].  qconv_create_packed is qconv_create for
 * weights held in that form with n = desc.n_w (a model then occupies n_w/8 of its int8 size in files and
 * host memory); the handle expands them once, at create, into the int8 operand layout the tensor cores
 * read.  They are not kept packed in device memory: the operand tiles go from global to shared memory
 * through the copy engine without a thread ever touching them, weights are at most a few MB per layer and
 * stay in L2, and an expansion pass per launch would cost more than the bytes it saves. */
int qpack_weights(const int8_t* wq_host, size_t count, int n, uint8_t* packed_host);
int qunpack_weights(const uint8_t* packed_host, size_t count, int n, int8_t* wq_host);
int qconv_create_packed(qconv_handle** out, const qconv_desc* desc, const uint8_t* w_packed_host,
                        const int32_t* bias_host, const int32_t* shift_host, const int32_t* res_lshift_host,
                        const int32_t* acc_exp_host);

/* bias_q[k] = round-to-nearest-even(b[k] / 2^(e_x + e_w[k])), saturated to int32. */
int qquantize_bias(const float* b_host, int K, int e_x, const int32_t* e_w_host,
                   int32_t* bias_q_host);

/* Checked build of the library (compiled with -DQCONV_CHECKED, binding.build_library(checked=True)): in the
 * CUDA-core kernels (conversions, pooling, packing, depthwise / direct convolution, eltwise, digit planes) every
 * global access with a computed address first tests its index against the tensor's extent; a failing test is
 * counted, the access skipped, the kernel goes on.  Returns the number of failed tests since the last call (and
 * the source line of the first in *first_line_out), clearing it; synchronises the device.  A normal build
 * returns -1. */
int qconv_checked_faults(int* first_line_out);

const char* qconv_last_error_string(void);

#ifdef __cplusplus
}
#endif
#endif /* QCONV_H_ */

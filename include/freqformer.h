/*
 * freqformer.h -- C ABI of the B200 (sm_100a) FreqFormer heterogeneous attention forward.
 *
 * One layer's attention forward over a T x H x W token grid, per head
 * (paper: Method, "Setup and notation" .. "Reconstruction"):
 *
 *   Q,K,V --separable orthonormal DCT-II along t/h/w--> spectral coefficients
 *         --split into low / mid / high bands (band-major token lists)
 *         --router: pooled band statistics + timestep embedding -> pi -> heads per band
 *         --low: dense attention on r:1 pooled tokens; mid: strided block-sparse attention;
 *           high: sliding-window attention; bands a head is not allocated to pass V~ through
 *         --m summary tokens per band, cross-band exchange (every token attends the 2m
 *           summaries of the other two bands, residual add)
 *         --recombination in the spectral domain, inverse transform --> out
 *
 * Conventions
 *   - All functions return an ff_status_t (int32_t); none throws, aborts or exits.
 *   - "device" pointers are CUDA device pointers on the device that was current at
 *     ff_plan_create; "host" pointers are ordinary host memory.
 *   - Q, K, V, out: device, contiguous [batch][heads][T][H][W][head_dim], element type
 *     cfg.dtype (bf16 or fp32).  out has the layout and type of the inputs.  The caller owns
 *     them; the library neither keeps nor frees them.
 *   - The caller also owns the workspace (ff_plan_set_workspace); the plan owns only small
 *     device tables (transform matrices, router weights, summary projections), freed by
 *     ff_destroy.
 *   - Calls are asynchronous on the given CUDA stream (a cudaStream_t passed as void*; NULL =
 *     the legacy default stream) unless a host output pointer is requested, which makes the
 *     call synchronise the stream before it returns.
 *   - A plan is not thread-safe; distinct plans are independent.
 */
#ifndef FREQFORMER_H_
#define FREQFORMER_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct ff_plan ff_plan_t; /* opaque */

typedef int32_t ff_status_t;
enum {
  FF_OK = 0,
  FF_ERR_INVALID_ARG = 1, /* NULL pointer, non-positive size, cut-offs out of order, bad mask ... */
  FF_ERR_UNSUPPORTED = 2, /* head_dim / axis length / parameter outside what the kernels cover */
  FF_ERR_WORKSPACE = 3,   /* workspace missing, misaligned or too small */
  FF_ERR_CUDA = 4,        /* a CUDA runtime call failed; ff_last_error has its message */
  FF_ERR_TIMEOUT = 5,     /* a bounded device-side wait expired (read back at the next sync) */
  FF_ERR_EMPTY_BAND = 6,  /* the cut-offs leave a band without coefficients */
  FF_ERR_NOT_ROUTED = 7   /* ff_forward without allocation and without timestep */
};

enum { FF_BF16 = 0, FF_FP32 = 1 };

/* Band-mask bits of one head.  The router emits one-hot masks; callers may pass any subset,
 * LOW|MID|HIGH being the paper's formal per-head definition (every head runs all three
 * operators, "Reconstruction" / "Per-layer complexity"). */
enum { FF_BAND_LOW = 1, FF_BAND_MID = 2, FF_BAND_HIGH = 4 };

/* Problem statement ("Setup and notation", "Frequency band partitioning",
 * "Hierarchical frequency-domain attention", "Cross-band residual exchange"). */
typedef struct {
  int32_t batch, T, H, W, heads, head_dim; /* head_dim: multiple of 32, <= 128; axes <= 128 */
  int32_t dtype;                           /* FF_BF16 or FF_FP32: Q, K, V and out */
  int32_t low_cut[3];      /* L_a (t,h,w): coefficient k is LOW iff k_a < L_a on all axes */
  int32_t mid_cut[3];      /* M_a: MID iff not LOW and k_a < M_a on all axes; L_a <= M_a <= n_a */
  int32_t low_compress;    /* r >= 1: low-band tokens are mean-pooled r:1 before attention */
  int32_t mid_block;       /* b >= 1: mid-band block size (consecutive band ranks) */
  int32_t mid_stride;      /* s >= 1: a query block sees key blocks at block distance = 0 mod s */
  int32_t high_radius;     /* R >= 0: high-band window |p - p'| <= R in band order */
  int32_t n_summary;       /* m >= 0 summary tokens per band; 0 disables the exchange */
  int32_t router_hidden;   /* hidden width of the two-layer router MLP */
  int32_t t_embed_dim;     /* d_t, even: width of the sinusoidal timestep embedding */
  int32_t transform;       /* FF_TRANSFORM_DCT or FF_TRANSFORM_HAAR: the 1-D transform of every axis */
  int32_t mid_pattern;     /* FF_MID_STRIDED or FF_MID_ANCHOR: the mid band's sparse pattern */
} ff_config_t;

/* "Separable spectral decomposition" / "Transform choice": the reference design's orthonormal DCT-II,
 * or the orthonormal Haar wavelet transform (power-of-two axis lengths; rows from the coarsest scale
 * to the finest, so the nested-box bands keep their meaning). */
enum { FF_TRANSFORM_DCT = 0, FF_TRANSFORM_HAAR = 1 };

/* "Mid band: structured block-sparse attention" / "Mid-band sparse degree".  Blocks of b consecutive
 * ranks, block index J.  STRIDED: query block J sees key blocks J' with (J' - J) mod s == 0.  ANCHOR:
 * query block J sees its own block and every anchor block J' = s-1 (mod s): a fixed set of "connector"
 * blocks shared by all queries plus the local block. */
enum { FF_MID_STRIDED = 0, FF_MID_ANCHOR = 1 };

/* Host arrays, copied at ff_plan_create.  Router input is [g_low; g_mid; g_high; e(t)]
 * (3*head_dim + t_embed_dim values).  NULL router pointers => ff_route / internal routing
 * return FF_ERR_NOT_ROUTED.  U == NULL => identity summary projections. */
typedef struct {
  const float *W1; /* [router_hidden][3*head_dim + t_embed_dim], row-major */
  const float *b1; /* [router_hidden] */
  const float *W2; /* [3][router_hidden] */
  const float *b2; /* [3] */
  const float *U;  /* [3][head_dim][head_dim]: S = U_l * Pool(Y^(l)) */
} ff_weights_t;

/* ---- host-only helpers (no GPU needed) --------------------------------------------------- */

/* Validate a configuration.  FF_OK, FF_ERR_INVALID_ARG, FF_ERR_UNSUPPORTED or FF_ERR_EMPTY_BAND. */
ff_status_t ff_config_validate(const ff_config_t *cfg);

/* Band sizes: sizes[0..3] = N_low, ceil(N_low / r), N_mid, N_high
 * ("Frequency band partitioning": N_low + N_mid + N_high = N). */
ff_status_t ff_band_sizes(const ff_config_t *cfg, int64_t sizes[4]);

/* Band (0 low, 1 mid, 2 high) and band-local rank of coefficient (k_t, k_h, k_w); the rank is
 * the coefficient's position in its band when the band is listed in increasing flat index
 * (k_t*H + k_h)*W + k_w.  This closed form is what the kernels evaluate in registers. */
ff_status_t ff_band_rank(const ff_config_t *cfg, int32_t kt, int32_t kh, int32_t kw,
                         int32_t *band, int64_t *rank);

/* Workspace size a plan of this configuration needs (device bytes, 256-byte aligned base). */
ff_status_t ff_workspace_bytes(const ff_config_t *cfg, size_t *bytes);

/* ---- plan lifetime ------------------------------------------------------------------------ */

/* Build a plan on the current CUDA device: validates cfg, computes the DCT-II matrices
 * ("Separable spectral decomposition") in double precision on the host and uploads them with
 * the weights.  No kernel runs.  *out_plan is NULL on failure. */
ff_status_t ff_plan_create(const ff_config_t *cfg, const ff_weights_t *weights, ff_plan_t **out_plan);

ff_status_t ff_plan_workspace_bytes(const ff_plan_t *plan, size_t *bytes);

/* Band sizes of the plan's configuration, as ff_band_sizes: N_low, ceil(N_low / r), N_mid, N_high
 * ("Frequency band partitioning"). */
ff_status_t ff_band_info(const ff_plan_t *plan, int64_t sizes[4]);

/* Hand the plan its workspace (device memory owned by the caller, >= the size above, base
 * aligned to 256 bytes).  Must precede ff_route / ff_forward; may be called again. */
ff_status_t ff_plan_set_workspace(ff_plan_t *plan, void *dev_ptr, size_t bytes);

/* Frees the plan's device tables and the plan.  NULL is allowed. */
ff_status_t ff_destroy(ff_plan_t *plan);

/* Message of the last failing call on this plan ("" if none); with plan == NULL, of the last
 * failing plan-less call of the calling thread.  Owned by the library. */
const char *ff_last_error(const ff_plan_t *plan);

/* ---- the path -------------------------------------------------------------------------------- */

/* Spectral routing network ("Spectral routing network"): forward transform of Q, K, V, pooled
 * band statistics g, timestep embedding e(t), z = MLP([g; e(t)]), pi = softmax(z), largest-
 * remainder head quota, heads [0,n_low) -> LOW, next n_mid -> MID, rest -> HIGH.
 *   timestep    host, [batch]: raw diffusion step per sample
 *   alloc_dev   device, [batch*heads] band masks written by the router; may be NULL
 *   alloc_host  host,   [batch*heads]; non-NULL forces a stream synchronisation
 *   pi_host     host,   [batch*3]; non-NULL forces a stream synchronisation
 * The transformed Q~, K~, V~ stay in the workspace; an ff_forward on the same inputs recomputes
 * them (the two calls are independent). */
ff_status_t ff_route(ff_plan_t *plan, const void *Q, const void *K, const void *V,
                     const float *timestep, uint8_t *alloc_dev, uint8_t *alloc_host,
                     float *pi_host, void *cuda_stream);

/* The attention forward ("Separable spectral decomposition" .. "Reconstruction").
 *   alloc_dev   device, [batch*heads] band masks (any subset of LOW|MID|HIGH per head), or
 *               NULL to route internally from `timestep` (host, [batch]) as ff_route does
 *   out         device, same shape and type as Q
 * Errors found on the host are returned at once; a device-side FF_ERR_TIMEOUT is reported by
 * ff_plan_device_status after a synchronisation. */
ff_status_t ff_forward(ff_plan_t *plan, const void *Q, const void *K, const void *V,
                       const uint8_t *alloc_dev, const float *timestep, void *out,
                       void *cuda_stream);

/* Same computation with HOST buffers: copies Q, K, V host->device into staging space inside the
 * workspace, runs ff_forward, copies out device->host, then synchronises.  On the tensor-core path
 * the copies run on a second stream owned by the plan, ordered after the work already queued on
 * `cuda_stream`: the forward transform starts on the first group of tensor-heads while the later
 * ones are still arriving, and finished groups of output heads leave while the rest is computed.
 * The workspace must have been sized with ff_workspace_bytes_host.  alloc_host may be NULL
 * (route internally); pinned host memory makes the copies asynchronous (and the overlap real). */
ff_status_t ff_forward_host(ff_plan_t *plan, const void *Q_host, const void *K_host,
                            const void *V_host, const uint8_t *alloc_host, const float *timestep,
                            void *out_host, void *cuda_stream);
ff_status_t ff_workspace_bytes_host(const ff_config_t *cfg, size_t *bytes);

/* The layer with its projections ("Setup and notation": linear projections of the layer input produce
 * Q_h, K_h, V_h; "Reconstruction": the head outputs are concatenated and projected):
 *     [Q | K | V] = X [W_q | W_k | W_v],   A = ff_forward(Q, K, V),   out = concat_h(A_h) W_o
 *   X      device, bf16, [batch][T*H*W][D], token-major, D = heads * head_dim
 *   Wqkv   device, bf16, [3][D][D]: W_q, W_k, W_v with y = x W (row k of W multiplies input channel k;
 *          output column h * head_dim + c is channel c of head h)
 *   Wo     device, bf16, [D][D], same convention (input row h * head_dim + c = channel c of head h)
 *   out    device, bf16, [batch][T*H*W][D]
 * Q, K, V and the attention output live in the workspace's staging area (size the workspace with
 * ff_workspace_bytes_host); Q, K, V are rounded to bf16, the storage type of the path.  bf16 plans with
 * head_dim 64 or 128, T*H*W a multiple of 128 and D a multiple of 256; otherwise FF_ERR_UNSUPPORTED.
 * alloc_dev / timestep as for ff_forward.  Asynchronous on the stream. */
ff_status_t ff_forward_projected(ff_plan_t *plan, const void *X, const void *Wqkv, const void *Wo,
                                 const uint8_t *alloc_dev, const float *timestep, void *out, void *cuda_stream);

/* Synchronises the stream and returns the device status word (FF_OK or FF_ERR_TIMEOUT), then
 * clears it. */
ff_status_t ff_plan_device_status(ff_plan_t *plan, void *cuda_stream);

/* Self-test of the failure path (no counterpart in the paper): launches one small CTA in which two
 * warps wait on a barrier nobody arrives at, with a limit of `limit_cycles` SM clock cycles (1 ..
 * 2e9, i.e. at most about a second).  The first waiter's limit runs out, it raises the CTA's abort
 * flag, the second waiter leaves on the flag, and the CTA records FF_ERR_TIMEOUT in the plan's
 * device status word exactly as the tensor-core kernels do.  Synchronises the stream.
 *   waiters_released  host, out: how many of the two waits returned "abandoned" (2 when all is well)
 * Afterwards ff_plan_device_status returns FF_ERR_TIMEOUT once (and clears the word); the plan and
 * the CUDA context stay usable. */
ff_status_t ff_plan_selftest_bounded_wait(ff_plan_t *plan, int64_t limit_cycles,
                                          int32_t *waiters_released, void *cuda_stream);

/* Which kernels the plan's forward runs with the workspace it has (benchmarks label their numbers with it):
 *   info[0]  1: the transform runs two axes in one launch (intermediate in shared memory), 0: three passes
 *   info[1]  CTAs per cluster of that launch (0 if unused)
 *   info[2]  1: the band operators run on the tensor-core kernel, 0: generic kernels
 *   info[3]  1: the pooled low band is part of the tensor-core attention launch */
ff_status_t ff_plan_kernel_info(const ff_plan_t *plan, int32_t info[4]);

/* Number of kernel launches the last ff_forward / ff_route on this plan issued. */
ff_status_t ff_plan_last_launches(const ff_plan_t *plan, int64_t *launches);

/* Stage timing for benchmarks.  With profiling enabled, ff_forward records CUDA events on its
 * stream at the stage boundaries; ff_plan_stage_times waits for the last one and returns the
 * device time (ms) and the number of kernel launches of each stage of the last ff_forward:
 *   TRANSFORM  forward transform + band split          ROUTER   band statistics + router MLP
 *   ATTENTION  low pooling + the three band operators  SUMMARY  summary tokens
 *   INVERSE    exchange + recombination + inverse transform */
enum { FF_STAGE_TRANSFORM = 0, FF_STAGE_ROUTER = 1, FF_STAGE_ATTENTION = 2, FF_STAGE_SUMMARY = 3,
       FF_STAGE_INVERSE = 4, FF_STAGE_COUNT = 5 };
ff_status_t ff_plan_set_profiling(ff_plan_t *plan, int32_t enable);
ff_status_t ff_plan_stage_times(ff_plan_t *plan, float ms[FF_STAGE_COUNT], int64_t launches[FF_STAGE_COUNT]);

/* ---- inspection (tests) --------------------------------------------------------------------- */

/* Intermediate buffers inside the workspace after the last call.  st = cfg.dtype, BH = batch*heads.
 *   FF_TAP_SPEC_LOW   float  [3 (Q,K,V)][BH][N_low][d]      low-band coefficients
 *   FF_TAP_SPEC_MID   st     [3][BH][N_mid][d]
 *   FF_TAP_SPEC_HIGH  st     [3][BH][N_high][d]
 *   FF_TAP_POOLED_LOW float  [3][BH][ceil(N_low/r)][d]      pooled low-band tokens
 *   FF_TAP_Y_LOW      float  [BH][ceil(N_low/r)][d]         low operator output (executed heads)
 *   FF_TAP_Y_MID      st     [BH][N_mid][d]                 mid operator output (executed heads)
 *   FF_TAP_Y_HIGH     st     [BH][N_high][d]
 *   FF_TAP_SUMMARY    float  [BH][3][m][d]                  summary tokens S
 *   FF_TAP_ENERGY     double [batch][3][d]                  pooled sums of squared coefficients
 *   FF_TAP_ALLOC      uint8  [BH]                           masks used by the last forward
 *   FF_TAP_PI         float  [batch][3]
 */
enum {
  FF_TAP_SPEC_LOW = 0, FF_TAP_SPEC_MID = 1, FF_TAP_SPEC_HIGH = 2, FF_TAP_POOLED_LOW = 3,
  FF_TAP_Y_LOW = 4, FF_TAP_Y_MID = 5, FF_TAP_Y_HIGH = 6, FF_TAP_SUMMARY = 7, FF_TAP_ENERGY = 8,
  FF_TAP_ALLOC = 9, FF_TAP_PI = 10, FF_TAP_COUNT = 11
};
ff_status_t ff_get_tap(const ff_plan_t *plan, int32_t which, const void **dev_ptr, size_t *bytes);

/* Kernel selection, a bit mask (0 = the defaults): 1 = generic SIMT attention instead of the
 * tensor-core kernel, 2 = generic SIMT transform instead of the tensor-core passes, 4 = the three
 * axes of the tensor-core transform as separate passes (instead of two of them fused in one launch
 * with the intermediate kept in shared memory).  For tests and benchmarks.
 * The tensor-core kernels cover bf16 storage with head_dim 128 or 64, axis lengths 16, 32, 64 or 128
 * and mid block sizes that tile 128 ranks; the pooled low band joins the tensor-core attention launch
 * from 128 pooled tokens on.  Every other configuration runs on the generic fp32 kernels. */
ff_status_t ff_plan_set_attention_impl(ff_plan_t *plan, int32_t impl);

/* ---- for callers that cannot allocate device memory ---------------------------------------------
 *
 * The paper has no counterpart of this entry point; it exists for integration reasons only.
 *
 * ff_high_attention_noalloc runs the high-band operator alone -- sliding-window softmax attention,
 * |p - p'| <= radius, clipped to the band, scale 1/sqrt(128) -- on tensors the caller already holds,
 * and calls no cudaMalloc, cudaFree or any other allocating routine.  It is meant for hosts where
 * the plan-based calls above cannot be used because they need a fresh workspace: a serving process
 * that handed every byte of device memory to its own pool at start-up (a raw allocation would fail
 * or fragment the pool), a latency-critical loop that cannot afford the device-wide synchronisation
 * an allocation implies, or a plug-in that is only ever given pointers.
 *
 *   q, k, v   device, bf16, contiguous [heads][n][128]: the band's tokens in band order
 *   y         device, bf16, [heads][n][128]: the operator's output (written by the call); it must
 *             not overlap q, k or v (other query tiles still read them while y is written)
 *   heads     1 .. 1024;  n  1 .. 2^31-257;  heads * ceil(n / 256) < 2^31;  larger sizes are
 *             rejected with FF_ERR_UNSUPPORTED
 *   sync      non-zero: synchronise the stream before returning and report a device-side
 *             FF_ERR_TIMEOUT; zero: return right after the launches -- a device-side time-out is
 *             then not reported at all (the next call clears the status word), so use zero only
 *             where the caller synchronises and validates by its own means
 *
 * The kernel's scratch (worklist, per-head masks, status word: 13,824 bytes) lives in a fixed array
 * inside the library image, so every GPU on which the library is loaded carries those bytes until
 * the process ends.  The first call on a device looks up the array's device address and sets the
 * kernel's shared-memory limit; make that first call before starting any stream capture.  All calls
 * on a device share the one array, and it keeps what the previous call left: the call rewrites the
 * masks and the worklist and clears the status word itself, but two calls whose kernels overlap on
 * the GPU (different streams, or different host threads) would race on it -- serialise them.
 * Errors: FF_ERR_INVALID_ARG (NULL or misaligned pointer, non-positive size), FF_ERR_UNSUPPORTED
 * (beyond the limits above), FF_ERR_CUDA; the message is available from ff_last_error(NULL). */
ff_status_t ff_high_attention_noalloc(const void *q, const void *k, const void *v, void *y,
                                      int32_t heads, int64_t n, int32_t radius, int32_t sync,
                                      void *cuda_stream);

#ifdef __cplusplus
}
#endif
#endif /* FREQFORMER_H_ */

/*
 * vcas.h -- C ABI of libvcas: the variance-controlled sampled backward of one linear layer
 * (VCAS, "Efficient Backpropagation with Variance-Controlled Adaptive Sampling",
 * arXiv 2402.17227) as CUDA kernels for sm_100a.
 *
 * Notation (paper, Sec. 4): a batch has N data of T tokens, R = N*T rows.  The layer is
 * Z = X theta^T, so W = theta is [d_out, d_in]; X is [R, d_in]; G = dY is [R, d_out].
 * rho is the keep ratio of SampleA (data dimension), nu the keep ratio of SampleW (token
 * dimension).
 *
 * Conventions for every entry point
 *  - returns VCAS_OK (0) or a negative vcas_status; never throws, aborts or prints;
 *  - tensor arguments are DEVICE pointers owned by the caller, row-major, contiguous,
 *    16-byte aligned, of the dtype given at vcas_create unless stated otherwise;
 *  - "host" in an argument comment means a host pointer;
 *  - work is enqueued on the caller's stream and is asynchronous; no entry point except
 *    vcas_create, vcas_destroy and vcas_last_device_status synchronises or allocates;
 *  - a handle owns one workspace and must not be used from two streams at the same time; inside a
 *    call the library may fork part of the work onto a stream of its own and join it back before the
 *    call's work on the caller's stream ends (stream capture records both branches);
 *  - device-side failures (a bounded wait that ran out) are recorded in a status word that
 *    vcas_last_device_status reads back.
 *
 * Random numbers: Philox4x32-10 (Salmon et al., SC'11) with key = (seed low, seed high),
 * counter = (index low, index high, sampler id, 0); the top 24 bits u of output word 0
 * decide "keep" iff u < floor(p * 2^24) with p in float32.  Sampler id 0 = SampleA (index =
 * datum), 1 = SampleW (index = global row).
 */
#ifndef VCAS_H_
#define VCAS_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct vcas_handle_s* vcas_handle;
typedef void* vcas_stream;            /* a cudaStream_t */

typedef enum {
  VCAS_OK = 0,
  VCAS_ERR_BAD_ARG = -1,              /* null pointer, ratio outside (0, 1], M < 2, ... */
  VCAS_ERR_SHAPE = -2,                /* unsupported sizes */
  VCAS_ERR_DTYPE = -3,
  VCAS_ERR_WORKSPACE = -4,            /* workspace allocation failed at vcas_create */
  VCAS_ERR_CUDA = -5,                 /* a CUDA runtime or driver call failed */
  VCAS_ERR_TIMEOUT = -6,              /* a device-side bounded wait ran out */
  VCAS_ERR_INTERNAL = -7
} vcas_status;

typedef enum { VCAS_DTYPE_F32 = 0, VCAS_DTYPE_BF16 = 1 } vcas_dtype;

/* Which kernels compute the two products.  AUTO picks the tensor-core (tcgen05) kernels for
 * bf16 layers whose d_in and d_out are multiples of 64, the fp32-FMA kernels otherwise. */
typedef enum { VCAS_GEMM_AUTO = 0, VCAS_GEMM_FMA = 1, VCAS_GEMM_TENSOR = 2 } vcas_gemm_path;

typedef struct {
  int32_t N, T, d_in, d_out;          /* d_in and d_out must be multiples of 8 */
  int32_t dtype;                      /* vcas_dtype of X, dY, W and dX; dW is always fp32 */
  int32_t gemm_path;                  /* vcas_gemm_path */
} vcas_layer_desc;

/* Hyper-parameters of Alg. 1.  Defaults (Sec. 6.1): tau_act = tau_w = 0.025, alpha = 0.01,
 * beta = 0.95, M = 2; F is task dependent (App. A.3), default 100.  rho_min / nu_min are
 * lower clips applied by vcas_update_ratios (default 0). */
typedef struct {
  int32_t F, M;
  float tau_act, tau_w, alpha, beta;
  float rho_min, nu_min;
} vcas_config;

/* Adaptation state of Alg. 1 for a stack of L layers (index 0 = the lowest layer).
 * rho and nu are host arrays of length L owned by the caller.  Initial values: s = 1,
 * rho = nu = 1, t = 0. */
typedef struct {
  float s;
  int32_t t;
  int32_t L;
  float* rho;                         /* host [L] */
  float* nu;                          /* host [L] */
} vcas_state;

/* Fills *cfg with the defaults above (host). */
int vcas_default_config(vcas_config* cfg);

/* Creates a handle for one layer shape on the current device and allocates its workspace
 * (the only allocation the library makes).  cfg may be NULL (defaults).  Synchronous. */
int vcas_create(vcas_handle* out, const vcas_layer_desc* desc, const vcas_config* cfg);
int vcas_destroy(vcas_handle h);
/* Bytes of device workspace owned by the handle (host out). */
int vcas_workspace_bytes(vcas_handle h, size_t* bytes);

/*
 * Eq. 2 for a linear layer (Sec. 4.1, 4.2, App. E):
 *   G_hat   = SampleA(dY): data n kept with probability p_n ~ ||G_n||_F, sum p = N rho,
 *             kept data rescaled by 1/p_n;
 *   dX      = G_hat W                      [R, d_in], layer dtype, rows of dropped data = 0;
 *   G_tilde = SampleW(G_hat, X): row r kept with probability q_r ~ ||G_hat_r|| ||X_r||,
 *             sum q = nu * T * (#kept data), kept rows rescaled by 1/q_r;
 *   dW      = G_tilde^T X                  [d_out, d_in], fp32.
 * rho, nu in (0, 1].  With rho = nu = 1 this is exact backprop.
 */
int vcas_linear_bwd(vcas_handle h, const void* X, const void* dY, const void* W,
                    float rho, float nu, uint64_t seed, void* dX, float* dW, vcas_stream stream);

/* vcas_linear_bwd with optional extras, each may be NULL:
 *   p_in [N], q_in [R] fp32: use these keep probabilities instead of computing them (q_in is
 *   read only on rows of kept data; rows of dropped data get q = 0);
 *   H [R, d_in], layer dtype: pre-activation of a GELU feeding this layer's input; dX is
 *   then multiplied elementwise by GELU'(H) (App. E: non-linear layers multiply by the saved
 *   Jacobian), erf form of GELU. */
int vcas_linear_bwd_ex(vcas_handle h, const void* X, const void* dY, const void* W,
                       float rho, float nu, uint64_t seed,
                       const float* p_in, const float* q_in, const void* H,
                       void* dX, float* dW, vcas_stream stream);

/*
 * Eq. 2 down a stack of layers.  Sec. 4: SampleA is applied at every layer, so "the activation gradient
 * becomes increasingly sparse when backpropagating" - the dY of a layer is the dX of the layer above, whose
 * rows of dropped data are exactly zero.  This variant lets a layer take what the layer above already
 * knows instead of re-reading dY, and hand the same down; all fields optional (NULL), all pointers device:
 *   H            as for vcas_linear_bwd_ex;
 *   a_in         row square-norms of this call's dY as partial sums: ||dY_r||^2 = sum of the a_in_parts
 *                consecutive floats a_in[r * a_in_parts ...]; with it dY is not read for scoring at all
 *                (the a_out of the call that produced dY, with a_in_parts = that handle's vcas_chain_parts);
 *   alive_in     ascending list of the data whose rows of dY may be non-zero, alive_cnt_in [1] its length
 *                (the kept_out / kept_cnt_out of the layer above); every other datum is taken to be zero:
 *                its rows of dY and a_in are never read, it is never kept, its rows of dX are zero;
 *   a_out        [R][vcas_chain_parts] fp32: partial sums of the square-norm of every row of dX as stored
 *                (after the GELU' factor and the rounding to the layer dtype), written by the dX product;
 *   kept_out     [N] int32: ascending list of the data this call kept, kept_cnt_out [1] its length;
 *   skip_dropped_rows  non-zero: the rows of dX (and a_out) that belong to dropped data are left unwritten instead
 *                of being set to zero - for a consumer that takes kept_out as its alive_in and therefore never
 *                reads them (tensor-core path; the fp32 path always writes them);
 *   defer_join   non-zero: the call returns with its weight-gradient branch (SampleW, the kept-row operands, the
 *                dW product, which run on a stream of the handle's own) not yet joined to `stream`: dX, a_out and
 *                kept_out are ordered on `stream` as usual, but dW and the sampling record are complete only after
 *                vcas_join(h, stream).  The next call on the same handle joins first by itself.  In a stack this
 *                lets the scoring and the dX product of the next layer run beside this layer's dW branch.  Under
 *                stream capture every handle must be joined before the capture ends.
 * alive_in / alive_cnt_in and kept_out / kept_cnt_out come in pairs; the lists must not alias.  A length
 * outside [0, N] or an entry outside [0, N) is not followed: it is reported as VCAS_ERR_BAD_ARG by
 * vcas_last_device_status (the call's outputs are then undefined).
 */
typedef struct {
  const void* H;
  const float* a_in;
  int32_t a_in_parts;
  const int32_t* alive_in;
  const int32_t* alive_cnt_in;
  float* a_out;
  int32_t* kept_out;
  int32_t* kept_cnt_out;
  int32_t skip_dropped_rows;
  int32_t defer_join;
} vcas_chain_args;
int vcas_linear_bwd_chain(vcas_handle h, const void* X, const void* dY, const void* W,
                          float rho, float nu, uint64_t seed, const vcas_chain_args* chain,
                          void* dX, float* dW, vcas_stream stream);
/*
 * SampleA in front of a layer that is not a matrix product (Sec. 4: SampleA is applied at every layer; App. E:
 * for a non-linear layer the sampled, rescaled gradient G_hat is multiplied by the saved exact Jacobian):
 * backward of Y = LayerNorm(X) * gamma + beta over the last axis, width d = d_in = d_out of the handle.
 *   G_hat = SampleA(dY) as in vcas_linear_bwd (p_n ~ ||G_n||_F, sum p = N rho, kept data times 1/p_n);
 *   dX = (g - mean(g) - x_hat mean(g x_hat)) / sqrt(var + eps) per row, g = G_hat * gamma, x_hat the normalised
 *        row; [R, d] layer dtype; rows of dropped data are 0 and are not computed;
 *   dgamma [d] = sum_r G_hat_r * x_hat_r,  dbeta [d] = sum_r G_hat_r   (fp32).
 * gamma: [d], layer dtype.  chain may be NULL; its fields mean what they mean for vcas_linear_bwd_chain (H is
 * ignored; a_out gets the row square-norms of dX in its first part, zeros in the others).  The kept data are
 * read back with vcas_last_sampling (g, p, idxA, cntA; the row-wise outputs are not defined by this call).
 */
int vcas_layernorm_bwd(vcas_handle h, const void* X, const void* gamma, const void* dY, float eps,
                       float rho, uint64_t seed, const vcas_chain_args* chain,
                       void* dX, float* dgamma, float* dbeta, vcas_stream stream);

/* Makes `stream` wait for the branch a call with defer_join left running (no-op otherwise).  Asynchronous. */
int vcas_join(vcas_handle h, vcas_stream stream);

/* Number of partial sums per row that this handle's dX product writes to a_out (host out). */
int vcas_chain_parts(vcas_handle h, int32_t* parts);

/* Exact backprop dX = dY W, dW = dY^T X with the same kernels at ratio 1 and no scoring. */
int vcas_dense_bwd(vcas_handle h, const void* X, const void* dY, const void* W,
                   void* dX, float* dW, vcas_stream stream);
/* vcas_dense_bwd for a layer whose input comes out of a GELU: with H [R, d_in] (layer dtype, the saved
 * pre-activation, may be NULL) dX is multiplied elementwise by GELU'(H) in the product's epilogue, as
 * vcas_linear_bwd_ex does - the exact backward through the activation, for comparisons with the sampled one. */
int vcas_dense_bwd_ex(vcas_handle h, const void* X, const void* dY, const void* W, const void* H,
                      void* dX, float* dW, vcas_stream stream);

/*
 * Scores, keep probabilities, masks and compacted index lists only (Sec. 4.1, 4.2), exactly
 * as vcas_linear_bwd computes them.  Every output may be NULL.
 *   g [N]: ||G_n||_F;  p [N];  w [R]: ||G_hat_r|| ||X_r|| (0 on rows of dropped data);
 *   q [R];  idxA [N]: ascending indices of kept data, cntA [1] their number;
 *   idxW [R]: ascending global row indices kept by both samplers, cntW [1] their number.
 */
int vcas_score(vcas_handle h, const void* X, const void* dY, float rho, float nu, uint64_t seed,
               float* g, float* p, float* w, float* q,
               int32_t* idxA, int32_t* cntA, int32_t* idxW, int32_t* cntW, vcas_stream stream);

/*
 * vcas_score without a handle and without any allocation (the paper has no counterpart; this
 * exists for the library's users).  Some callers may not allocate device memory at the point
 * where they need the scores: code running inside a framework's memory-pool region or a
 * real-time loop where cudaMalloc's implicit synchronisation and possible failure are not
 * acceptable, or plug-ins that are handed a fixed memory budget.  vcas_create / vcas_score need a
 * workspace from cudaMalloc; this entry point instead keeps its intermediates (row norms,
 * scores, rescale factors, index lists) in a fixed array inside the library image, about
 * 0.6 MB that every GPU loading the library holds until the process exits.
 *   Limits: N <= 4096 and N*T <= 16384, otherwise VCAS_ERR_SHAPE.  d_in, d_out multiples of 8.
 *   Inputs and outputs are the caller's, as for vcas_score (any output may be NULL).
 *   The first call on each device looks up the array's device address (with that device
 *   current); make that first call before starting any stream capture.
 *   All calls on a device share the one array, which keeps the previous call's contents (the
 *   call itself clears what has to start at zero): two calls whose GPU work overlaps, e.g. on
 *   different streams, race.  Calls on one stream are safe.
 * It calls no cudaMalloc, cudaFree or allocating library routine.
 */
int vcas_score_static(int32_t N, int32_t T, int32_t d_in, int32_t d_out, int32_t dtype,
                      const void* X, const void* dY, float rho, float nu, uint64_t seed,
                      float* g, float* p, float* w, float* q,
                      int32_t* idxA, int32_t* cntA, int32_t* idxW, int32_t* cntW, vcas_stream stream);

/* Copies what the last vcas_linear_bwd(_ex) or vcas_score on this handle computed (same
 * outputs as vcas_score); enqueue on the same stream. */
int vcas_last_sampling(vcas_handle h, float* g, float* p, float* w, float* q,
                       int32_t* idxA, int32_t* cntA, int32_t* idxW, int32_t* cntW,
                       vcas_stream stream);

/* Bernoulli mask and compaction for given probabilities (Sec. 4.1: m_i = Bern(p_i)/p_i):
 * keep[i] = (u24(seed, sampler_id, i) < floor(p[i] 2^24)) for i < n; idx = ascending kept
 * indices, cnt [1] their number.  keep (uint8 [n]), idx (int32 [n]) may be NULL. */
int vcas_mask_from_probs(vcas_handle h, const float* p, int32_t n, uint64_t seed, int32_t sampler_id,
                         uint8_t* keep, int32_t* idx, int32_t* cnt, vcas_stream stream);

/*
 * The Monte-Carlo probe of Alg. 1 at the granularity of this layer's parameter gradient.
 * X_i, dY_i: host arrays of M device pointers (M batches); W as above.
 * For batch i: G_s,i = dY_i^T X_i (exact).  For repetition j (seed derived from (seed, i, j)):
 * G_act,ij = G_hat_ij^T X_i with SampleA only, and V_w,ij = Eq. 3 at ratio nu.
 * Outputs (device fp32 scalars, any may be NULL):
 *   V_s   = 1/(M-1) sum_i ||G_s,i - mean||_F^2,
 *   V_act = 1/M^2 sum_ij ||G_act,ij - G_s,i||_F^2,
 *   V_w   = 1/M^2 sum_ij V_w,ij,
 *   p_lo, p_hi = Eq. 4's sparsity p(s - alpha), p(s + alpha) averaged over the batches
 *   (App. D), s -+ alpha clipped to [0, 1]; Eq. 4's n starts at 1, so p >= 1/N and the ratios
 *   that vcas_update_ratios derives from them stay valid arguments of vcas_linear_bwd.
 * M >= 2 (the 1/(M-1) of V_s).  alpha comes from the handle's config.
 */
int vcas_variance_probe(vcas_handle h, int32_t M, const void* const* X_i, const void* const* dY_i,
                        const void* W, float rho, float nu, float s, uint64_t seed,
                        float* V_s, float* V_act, float* V_w, float* p_lo, float* p_hi,
                        vcas_stream stream);

/*
 * App. D: the probe's variances may be estimated on a random sample of the parameters.  With rows > 0 the
 * probe forms G_s,i and G_act,ij only on `rows` of the d_out rows of the parameter gradient - a uniformly
 * random subset fixed here: row i gets the Philox word of counter (i, 0, 2, 0) under the key (seed low, seed
 * high), the `rows` smallest words win, ties by index - and scales V_s and V_act by d_out / rows (unbiased for
 * the sums over all rows); V_w (Eq. 3) and p_lo / p_hi need no gradient and are unchanged.  The probe's two
 * products then cost rows / d_out of their full size.  rows: a multiple of 64 (8 on the fp32-FMA path), at most
 * 256 and below d_out; 0 switches the sample off (default).  Synchronous.
 */
int vcas_set_probe_subsample(vcas_handle h, int32_t rows, uint64_t seed);
/* The rows chosen (host out, ascending; rows_host may be NULL) and their number. */
int vcas_get_probe_subsample(vcas_handle h, int32_t* rows_host, int32_t* count);

/*
 * One adaptation step of Alg. 1 (host only, all pointers host, arrays of length L):
 *   Eq. 5: s <- clip(s + alpha sign(sum_l V_act,l - tau_act sum_l V_s,l), 0, 1), sign(0) = +1;
 *   Eq. 4: rho_l <- max(rho_min, max_{j<=l} p_j) with p_j = p_hi[j] if s went up else p_lo[j];
 *   Eq. 7: nu_l <- min(1, nu_l / beta) if V_w,l >= tau_w V_s,l else max(nu_min, nu_l beta).
 * state->t is left to the training loop.
 */
int vcas_update_ratios(vcas_state* state, int32_t L, const float* V_s, const float* V_act,
                       const float* V_w, const float* p_lo, const float* p_hi,
                       const vcas_config* cfg);

/* Synchronises the device and returns the handle's device status word in *status
 * (VCAS_OK or VCAS_ERR_TIMEOUT / VCAS_ERR_INTERNAL / VCAS_ERR_BAD_ARG); the word is then cleared.  After an
 * error the outputs of the calls since the last check are undefined; the workspace counters
 * that a kernel which gave up may have left behind are reset, so the handle stays usable.  No kernel of the
 * library waits for another kernel or for another CTA; the only waits are those of vcas_set_wait_limit. */
int vcas_last_device_status(vcas_handle h, int32_t* status);

/* Failure detection (the paper has no counterpart).  Every wait inside the product kernels (on a TMA arrival,
 * on the tensor pipe, on a work item) is bounded: when it lasts longer than limit_ns (default 2 s) the CTA
 * records VCAS_ERR_TIMEOUT in the status word, all its roles leave their loops, its TMEM is released and the
 * kernel returns.  Test hook: with stall_once != 0 the first CTA of every product launch leaves out the loads
 * of its first k-block, so that one wait is certain to run out (nothing faults: the loads are simply not
 * issued); with a limit of about a millisecond this exercises the give-up path.  limit_ns = 0 is rejected. */
int vcas_set_wait_limit(vcas_handle h, uint64_t limit_ns, int32_t stall_once);

/* Tuning overrides for the tensor-core products (the paper has no counterpart): output tile
 * width of the dX and dW kernels (64, 128 or 256), the number of slices each contraction is
 * split into (1..16; slices are combined in a fixed order, so results stay reproducible), and
 * the tile height of each product (dx_tile_m, dw_tile_m = 1: 128 rows, 2: 256 rows whenever the width is 256 and the
 * contraction is not sliced, 3: 256 rows for as many tiles as fill all SMs a whole number of
 * times and 128 rows with a sliced contraction, in a second launch, for the rest).
 * 0 = let the library choose from the shapes and ratios.  VCAS_ERR_BAD_ARG for a value outside
 * these sets. */
int vcas_set_tuning(vcas_handle h, int32_t dx_tile_n, int32_t dw_tile_n, int32_t dx_split_k, int32_t dw_split_k,
                    int32_t dx_tile_m, int32_t dw_tile_m);

/* The tilings the library chose for the two products of the handle's last sampled or dense call (the paper has
 * no counterpart): plan[0..2] = tile width, contraction slices, tile-height code (as in vcas_set_tuning) of the dX
 * product, plan[3..5] the same for the dW product (host out).  VCAS_ERR_BAD_ARG before the first call or on the
 * fp32-FMA path. */
int vcas_last_plan(vcas_handle h, int32_t* plan);

/* Stage timing for benchmarks (the paper has no counterpart; Sec. 6 only reports end-to-end
 * hours).  While enabled, vcas_linear_bwd(_ex) and vcas_dense_bwd record CUDA events on the
 * caller's stream at their stage boundaries, for up to 2048 calls of each kind, and run their
 * kernels one after the other on that stream (no internal fork) so that each pair of events
 * brackets one kernel.  Enabling
 * allocates the events once (host objects); it also clears what was recorded. */
int vcas_set_profiling(vcas_handle h, int32_t enable);
/* Synchronises the device, then writes the summed milliseconds of the recorded calls to
 * ms[0..7] (host): 0 row norms, 1 keep probabilities + masks + compaction, 2 dX product,
 * 3 pack of the kept rows, 4 dW product, 5 dense dX, 6 dense dW, 7 unused; calls[0..1] (host)
 * = recorded sampled / dense calls.  Clears the record. */
int vcas_stage_times(vcas_handle h, float* ms, int32_t* calls);

/* Number of this library's kernel launches enqueued through the handle so far (host out). */
int vcas_launch_count(vcas_handle h, uint64_t* launches);

/* Library version, e.g. 100 for 0.1.0. */
int vcas_version(void);

#ifdef __cplusplus
}
#endif
#endif /* VCAS_H_ */

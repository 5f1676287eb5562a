/*
 * spectral_correction.h - C ABI of the B200 (sm_100a) spectral-correction optimizer step.
 *
 * The library implements the per-matrix update of "Anchor Priors and Spectral Correction"
 * (Section 3.2; Algorithm 1 lines 7-14):
 *
 *   on anchor arrival   M_anc <- beta_anc * M_anc + (1 - beta_anc) * G_anc            (Eq. 1)
 *                       M_anc ~= U diag(s) V^T, leading `rank` triplets               (the SVD of Section 3.2)
 *                       d_i = s_i / (s_i + tau_p)                                     (Eq. 2)
 *   every step          X = U^T g V,  g = G_mask (times 1/keep_ratio unless prescaled)
 *                       G_filt = U diag(d) X diag(d) V^T                              (two-sided application)
 *                       G_proj = alpha * g + (1 - alpha) * G_filt                     (Eq. 3)
 *                       AdamW(W, m, v; G_proj)                                        (Algorithm 1 line 13)
 *
 * Conventions
 *   - A weight matrix W is rows x cols = out features x in features, row-major, contiguous.
 *     Gradients, AdamW moments and the anchor momentum have the same shape and layout.
 *   - "device" pointers are CUDA global-memory addresses of the current device; "host" pointers are
 *     ordinary process memory.  Pointer ARRAYS (one entry per matrix) always live in host memory and
 *     are read before the call returns; the buffers they point to are device memory unless a function
 *     says otherwise, are owned by the caller, must be 16-byte aligned and must stay valid until the
 *     work queued on the plan's stream has finished.
 *   - All calls queue work on the stream given to sc_plan_create and return without waiting for it.
 *   - A plan is not thread-safe: calls on ONE plan must come from one thread at a time. Different plans (on the
 *     same or different streams) are independent.
 *   - Every function returns an sc_status; nothing throws or aborts across this boundary.
 *     Conditions the device detects (a bounded wait that ran out, non-finite values) are latched in a
 *     status word that sc_get_device_status reads back.
 *   - The library never allocates device memory: the caller passes one workspace blob of at least
 *     sc_plan_workspace_bytes() bytes (256-byte aligned), which holds the anchor momentum, the cached
 *     basis and scratch.  The small host-side plan object (and pinned staging for pointer tables) is
 *     allocated by sc_plan_create and freed by sc_plan_destroy.
 */
#ifndef SPECTRAL_CORRECTION_H_
#define SPECTRAL_CORRECTION_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#if defined(_WIN32)
#define SC_API
#else
#define SC_API __attribute__((visibility("default")))
#endif

typedef struct sc_plan sc_plan;

typedef enum sc_status {
  SC_OK = 0,
  SC_WARN_NO_ANCHOR = 1,        /* step ran with an empty basis: G_proj = alpha * g (no anchor has arrived yet) */
  SC_ERR_INVALID_ARG = -1,
  SC_ERR_SHAPE = -2,
  SC_ERR_DTYPE = -3,
  SC_ERR_ALIGNMENT = -4,
  SC_ERR_WORKSPACE = -5,
  SC_ERR_STALE_TAG = -6,        /* anchor step tag older than the last one accepted */
  SC_ERR_CUDA = -7,
  SC_ERR_UNSUPPORTED_ARCH = -8, /* the current device is not sm_100 */
  SC_ERR_TIMEOUT = -9,          /* a bounded device-side wait ran out */
  SC_ERR_NONFINITE = -10,
  SC_ERR_TOO_LARGE = -11
} sc_status;

typedef enum sc_dtype { SC_DTYPE_BF16 = 0, SC_DTYPE_FP32 = 1 } sc_dtype;

/* Which kernels do the large contractions. AUTO: tcgen05 tensor-core kernels for bf16 gradients on
 * shapes they support (cols % 8 == 0), plain fp32 CUDA-core kernels otherwise (fp32 gradients, odd shapes). */
typedef enum sc_engine { SC_ENGINE_AUTO = 0, SC_ENGINE_SIMT = 1 } sc_engine;

/* Which optimizer consumes G_proj. ADAMW: Algorithm 1 line 13. ADEMAMIX: the dual-EMA composition of the appendix
 * "On the Compatibility with Dual-EMA Optimizers": a fast EMA m1 (beta1, bias-corrected) and a slow EMA m2 (beta3, not
 * bias-corrected) of G_proj, W <- W (1 - lr wd) - lr (m1_hat + mix_alpha m2) / (sqrt(v_hat) + eps); one more fp32 state
 * array per matrix (sc_opt_state.exp_avg_slow). */
typedef enum sc_optimizer { SC_OPT_ADAMW = 0, SC_OPT_ADEMAMIX = 1 } sc_optimizer;

typedef struct sc_shape {
  int64_t rows; /* m, out features */
  int64_t cols; /* n, in features  */
} sc_shape;

/* Hyper-parameters (Algorithm 1 "Require" line, plus AdamW's and the basis iteration's). Plain data. */
typedef struct sc_hparams {
  float alpha;          /* blend weight of the raw masked gradient, Eq. 3 */
  float tau_p;          /* spectral damping, Eq. 2 */
  float beta_anc;       /* anchor EMA decay, Eq. 1 */
  float lr;             /* AdamW */
  float beta1;
  float beta2;
  float eps;
  float weight_decay;   /* decoupled */
  float max_grad_norm;  /* global-norm clip of G_proj over all matrices; <= 0 disables */
  int32_t grads_prescaled; /* 1: masked gradients already carry the 1/keep_ratio rescale; 0: the step applies it */
  int32_t grad_dtype;      /* sc_dtype of masked and anchor gradients */
  int32_t sketch_width;    /* l: columns of the randomized range finder, rank <= l <= 256; 0 means l = rank */
  int32_t power_iters;     /* q: subspace (power) iterations of the range finder, 0..16 */
  int32_t engine;          /* sc_engine */
  int32_t collect_stats;   /* 1: also accumulate ||g||^2 every step so that sc_get_stats can report eta_r and ||G_proj|| */
  int32_t warm_start;      /* 1: a matrix that already has a basis starts the range finder from its previous right basis V
                              (columns rank..l-1 from the sketch) and runs warm_power_iters instead of power_iters.
                              The anchor momentum drifts slowly, so successive arrivals act as accumulated subspace
                              iterations at two sweeps per arrival. 0: always start from the sketch. */
  int32_t warm_power_iters; /* q used on a warm start, 0..16 */
  int32_t optimizer;       /* sc_optimizer */
  uint64_t seed;           /* key of the counter-based Rademacher sketch */
  float beta3;             /* SC_OPT_ADEMAMIX: decay of the slow EMA, in [0, 1) */
  float mix_alpha;         /* SC_OPT_ADEMAMIX: weight of the slow EMA in the update, >= 0 */
  int32_t full_spectrum;   /* 1: the main-text form of Section 3.2 - no rank cut, the soft weights d_i = s_i / (s_i + tau_p)
                              apply to all min(rows, cols) singular directions: G_filt = P_U G P_V with
                              P_U = U diag(d) U^T, P_V = V diag(d) V^T. Create the plan with rank = 0. On anchor arrival
                              the two soft projectors are built by matrix products only (Newton-Schulz square root of the
                              Gram matrix, then Newton-Schulz inverse), in fp64; every step is two dense tensor-core
                              contractions per matrix plus one elementwise AdamW pass. Needs tau_p > 0, bf16 gradients,
                              AdamW, no clipping, rows and cols multiples of 8 in [256, 8192]. */
  int32_t fs_sqrt_iters;   /* full_spectrum: iterations of the square-root stage, 1..200 (default 24; directions with
                              s_i below about 1e-3 of the largest are still under-weighted then, which only lowers d_i) */
  int32_t fs_inv_iters;    /* full_spectrum: iterations of the inverse stage, 1..200 (default 12: enough for
                              (s_max + tau_p) / tau_p up to a few hundred) */
  int32_t reserved;
} sc_hparams;

/* AdamW state handed to sc_correct_and_step. Arrays of n_mats device pointers, held in host memory. */
typedef struct sc_opt_state {
  void* const* exp_avg;     /* m: fp32 rows x cols, updated in place */
  void* const* exp_avg_sq;  /* v: fp32 rows x cols, updated in place */
  void* const* params_bf16; /* optional bf16 copy of the updated weights (written only); NULL or NULL entries = none */
  void* const* exp_avg_slow; /* SC_OPT_ADEMAMIX only: slow EMA m2, fp32 rows x cols, updated in place; NULL for AdamW */
} sc_opt_state;

/* Per-matrix statistics of the last sc_correct_and_step (by-products of the projection). */
typedef struct sc_mat_stats {
  float g_sqnorm;     /* ||g||_F^2, g = rescaled masked gradient */
  float x_sqnorm;     /* ||U^T g V||_F^2 ; eta_r = x_sqnorm / g_sqnorm (alignment diagnostic of the appendix) */
  float gproj_sqnorm; /* ||G_proj||_F^2 before clipping, closed form from g_sqnorm and X */
  float r_eff;        /* sum_i d_i^2 (Lemma 2's effective rank) */
} sc_mat_stats;

/* Fill *hp with defaults: alpha 0.3, tau_p 1e-3, beta_anc 0.9, lr 2e-5, betas (0.9, 0.999), eps 1e-8,
 * weight_decay 0, no clipping, grads prescaled, bf16 gradients, l = rank, q = 1, cold starts only, engine AUTO, no stats, seed 0,
 * optimizer AdamW, beta3 0.9999, mix_alpha 5 (the values the dual-EMA appendix quotes).
 * (alpha, tau_p, lr, betas: the paper's defaults; the others are not given there.) */
SC_API sc_status sc_hparams_default(sc_hparams* hp);

/* Bytes of device workspace a plan for these shapes needs. Host-only, no CUDA calls. Returns 0 on invalid input. */
SC_API size_t sc_plan_workspace_bytes(const sc_shape* shapes, int n_mats, int rank, const sc_hparams* hp);

/* sc_plan_create - validate, lay out the workspace, zero the anchor momentum (Algorithm 1 line 2: M_anc <- 0).
 *   out            host: receives the plan handle
 *   shapes         host: n_mats entries
 *   rank           r >= 0, r <= min(rows, cols) of every matrix, r <= 256; 0 = no basis (G_proj = alpha g)
 *   keep_ratio     in (0, 1]; 1 - p_mask. Used for the 1/keep rescale when hp->grads_prescaled == 0.
 *   workspace      device: caller-owned blob, 256-byte aligned, kept alive until sc_plan_destroy
 *   stream         a cudaStream_t (as void*), NULL = default stream; all later calls queue work on it
 * Errors: INVALID_ARG, SHAPE, DTYPE, ALIGNMENT, WORKSPACE (too small), UNSUPPORTED_ARCH, CUDA. */
SC_API sc_status sc_plan_create(sc_plan** out, const sc_shape* shapes, int n_mats, int rank, float keep_ratio,
                                const sc_hparams* hp, void* workspace, size_t workspace_bytes, void* stream);

SC_API sc_status sc_plan_destroy(sc_plan* plan);

/* sc_anchor_update - an anchor gradient has arrived (Algorithm 1 lines 7-9 and the SVD of line 11).
 *   anchor_grads   host array of n_mats device pointers (grad_dtype, rows x cols); a NULL entry means no anchor
 *                  gradient arrived for that matrix: its momentum and basis are left as they are.
 *   step_tag       fast-circuit step at which the anchor's weight snapshot was taken; must not decrease.
 *                  It does not enter the arithmetic (the paper applies no staleness weighting); it is
 *                  recorded so that staleness = step - tag can be reported.
 * For each arrived matrix: Eq. 1, then the rank-r basis of the new momentum by randomized subspace iteration
 * (sketch width l, q power iterations), then Eq. 2. The basis is cached until the next arrival. */
SC_API sc_status sc_anchor_update(sc_plan* plan, const void* const* anchor_grads, int64_t step_tag);

/* sc_anchor_update_factored - the same arrival when the anchor gradient comes as rank-rho factors, G_anc = P Q^T
 * (the staleness appendix has the anchor circuit push its gradient compressed to about one data-parallel
 * all-reduce payload, i.e. low-rank factors). Eq. 1 is applied tile by tile without ever forming G_anc.
 *   P_factors   host array of n_mats device pointers, rows x rho fp32 row-major (NULL entry = not arrived)
 *   Q_factors   host array of n_mats device pointers, cols x rho fp32 row-major (NULL exactly where P is NULL)
 *   rho         1..1024 */
SC_API sc_status sc_anchor_update_factored(sc_plan* plan, const void* const* P_factors, const void* const* Q_factors,
                                           int rho, int64_t step_tag);

/* sc_correct_and_step - one fast-circuit optimizer step over all matrices (Algorithm 1 lines 10-13).
 *   masked_grads   host array of n_mats device pointers (grad_dtype, rows x cols), read only
 *   params         host array of n_mats device pointers, fp32 master weights, updated in place
 *   state          optimizer moments (updated in place) and the optional bf16 weight copy; with SC_OPT_ADEMAMIX
 *                  state->exp_avg_slow is required (SC_ERR_INVALID_ARG when it is NULL)
 *   step           optimizer step count t >= 1 (AdamW bias correction; staleness report)
 * Returns SC_WARN_NO_ANCHOR (still a completed step) when no anchor has arrived yet. */
SC_API sc_status sc_correct_and_step(sc_plan* plan, const void* const* masked_grads, void* const* params,
                                     const sc_opt_state* state, int64_t step);

/* sc_correct_and_step_host - the same step for gradients that arrive in HOST memory (in the paper's setting the
 * data-parallel all-reduce of Algorithm 1 line 6 delivers them over the network).
 *   host_grads     host array of n_mats HOST pointers (grad_dtype, rows x cols). Page-locked memory lets the copies
 *                  overlap the kernels; pageable memory works but serialises.
 *   grad_staging   host array of n_mats DEVICE pointers the gradients are copied into (caller-owned, same sizes)
 *   stats_out      host: n_mats entries filled with the step's statistics (the step's result read back), or NULL
 *   clip_out       host: the clip factor applied, or NULL
 * The copies of one shape class are queued ahead of the kernels of the class before it, on a stream the plan owns.
 * Unlike sc_correct_and_step this call returns only after the step has finished on the device. */
SC_API sc_status sc_correct_and_step_host(sc_plan* plan, const void* const* host_grads, void* const* grad_staging,
                                          void* const* params, const sc_opt_state* state, int64_t step,
                                          sc_mat_stats* stats_out, float* clip_out);

/* sc_apply_prf_mask - the in-graph activation mask of Section 3.1 / Algorithm 1 line 4: out = X * M (times
 * 65536 / round(keep * 65536) when rescale != 0), M a pure function of (seed, layer, step, token, feature), so every
 * pipeline stage regenerates it and nothing is transmitted. Stand-alone (no plan).
 *   X_dev, out_dev   device: tokens x features bf16 row-major, 16-byte aligned (out may alias X); features % 8 == 0
 *   keep             keep ratio 1 - p_mask in (0, 1], quantised to 16 bits
 * The masked weight gradient of the step is then the plain product dY^T out. */
SC_API sc_status sc_apply_prf_mask(const void* X_dev, void* out_dev, int64_t tokens, int64_t features, float keep,
                                   uint64_t seed, uint32_t layer, uint64_t step, int rescale, void* stream);

/* sc_masked_weight_grad - the fast circuit's weight gradient of one linear layer from masked activations
 * (Section 3.1, Algorithm 1 lines 4-5): G = dY^T (X * M) * 65536 / round(keep * 65536), M the mask of sc_apply_prf_mask
 * for the same (seed, layer, step). Two launches on `stream`: the mask pass X -> Xm and a dense bf16 GEMM over the
 * token dimension on the tensor cores (fp32 accumulation, the rescale applied in fp32 before the result is rounded).
 * Stand-alone (no plan), asynchronous.
 *   dY_dev      device: tokens x rows bf16 row-major (gradient with respect to the layer's output), read only
 *   X_dev       device: tokens x cols bf16 row-major (the layer's input, unmasked), read only
 *   Xm_dev      device: tokens x cols bf16, caller-owned; receives X * M (unscaled). May alias X_dev.
 *   G_dev       device: rows x cols row-major, out_dtype (SC_DTYPE_BF16 or SC_DTYPE_FP32), overwritten
 *   status_dev  device: one uint32 that receives bit 0 if a bounded device-side wait runs out, or NULL
 * All pointers 16-byte aligned; rows % 8 == 0 and cols % 8 == 0 (SC_ERR_SHAPE otherwise); tokens is unrestricted. */
SC_API sc_status sc_masked_weight_grad(const void* dY_dev, const void* X_dev, void* Xm_dev, void* G_dev, int out_dtype,
                                       int64_t tokens, int64_t rows, int64_t cols, float keep, uint64_t seed,
                                       uint32_t layer, uint64_t step, void* status_dev, void* stream);

/* sc_apply_prf_mask_exact_k - the per-token form of the same mask (Section 3.1): every token keeps exactly
 * K = round(keep * features) features (halves round up, the product formed in single precision), chosen by the K
 * smallest values of a per-(token, feature) hash (ties impossible by construction); rescale multiplies by features / K.
 * Same layouts as sc_apply_prf_mask; features <= 65536, no multiple-of-8 requirement. */
SC_API sc_status sc_apply_prf_mask_exact_k(const void* X_dev, void* out_dev, int64_t tokens, int64_t features,
                                           float keep, uint64_t seed, uint32_t layer, uint64_t step, int rescale,
                                           void* stream);

/* sc_lowrank_compress - low-rank compression of one gradient matrix with error feedback (DP-compression appendix,
 * "Low-rank factorization (F3)": rank-1..4 factors from one subspace-iteration step per gradient; the map is linear, so
 * it commutes with the sum over data-parallel workers; error feedback keeps what the factors miss for the next step):
 *     M = G + E      P = M Q_prev      P_hat = orth(P)      Q = M^T P_hat      E <- M - P_hat Q^T
 * The transmitted approximation is P_hat Q^T; (P_hat, Q) is exactly the factored form sc_anchor_update_factored takes.
 * Stand-alone (no plan), asynchronous on `stream`.
 *   G_dev      device: rows x cols, grad_dtype (sc_dtype), row-major, read only
 *   E_dev      device: rows x cols fp32 error memory, updated in place (start it at zero), or NULL for no error feedback.
 *              Between phase A and phase C it holds M.
 *   P_dev      device: rows x rho fp32 row-major. Out of phase A: P = M Q_prev; out of phase B: P_hat (orthonormal
 *              columns; a column that depends on the earlier ones to single precision - remainder below 1e-3 of its
 *              norm - is dropped, i.e. zero).
 *   Q_dev      device: cols x rho fp32 row-major. In: Q_prev (sc_lowrank_init_q for the first step, afterwards the Q of
 *              the previous step); out of phase B: Q = M^T P_hat.
 *   rho        1..8
 *   phases     bit mask: 1 = A (M, P), 2 = B (orthonormalise P, Q), 4 = C (E). 7 runs everything (one worker). With
 *              several workers: call with 1, sum P over workers, call with 2, sum Q over workers, call with 4.
 *   workspace  device: caller-owned scratch of sc_lowrank_workspace_bytes(rows, cols, rho) bytes, 256-byte aligned
 * Pointers 16-byte aligned; cols % 4 == 0 (SC_ERR_SHAPE otherwise). All arithmetic is fp32 on the CUDA cores (at most
 * 16 flops per byte: HBM-bound), every reduction two-stage in a fixed order.
 * Errors: INVALID_ARG, DTYPE, SHAPE, TOO_LARGE, ALIGNMENT, WORKSPACE, CUDA. */
SC_API size_t sc_lowrank_workspace_bytes(int64_t rows, int64_t cols, int rho);
SC_API sc_status sc_lowrank_compress(const void* G_dev, int grad_dtype, void* E_dev, void* P_dev, void* Q_dev,
                                     int64_t rows, int64_t cols, int rho, int phases, void* workspace,
                                     size_t workspace_bytes, void* stream);

/* Fill Q (cols x rho fp32) with the counter-based +-1 sketch keyed on `seed`: the start of the first compression step
 * (the same start on every worker, nothing transmitted). */
SC_API sc_status sc_lowrank_init_q(void* Q_dev, int64_t cols, int rho, uint64_t seed, void* stream);

/* ---- inspection / test hooks ------------------------------------------------------------------------- */

/* Copy matrix `mat`'s cached basis into caller device buffers (any may be NULL):
 * U rows x rank fp32 row-major, s rank fp32, V cols x rank fp32 row-major. Queued on the plan's stream. */
SC_API sc_status sc_export_basis(sc_plan* plan, int mat, void* U_dev, void* s_dev, void* V_dev);

/* Replace matrix `mat`'s cached basis (same layouts; columns must be orthonormal, s descending) and
 * recompute Eq. 2 and the operand copies the step kernels read. Marks the matrix as having an anchor. */
SC_API sc_status sc_import_basis(sc_plan* plan, int mat, const void* U_dev, const void* s_dev, const void* V_dev);

/* Copy the projections of the last step for matrix `mat` (either may be NULL): T = G V (rows x rank fp32,
 * row-major, on the raw masked gradient) and X = U^T G V (rank x rank fp32, row-major). */
SC_API sc_status sc_export_projection(sc_plan* plan, int mat, void* T_dev, void* X_dev);

/* sc_project_static - X = U^T G V for ONE matrix, without a plan, a workspace or any allocation.
 * (The paper has no counterpart to this call; it is a packaging of the projection step for constrained callers.)
 *
 * Who needs it: code that may not allocate device memory at the point where it wants the projection - for
 * example a hook that runs after a framework's caching allocator has taken all of HBM, or a monitoring path
 * that must not take the allocator lock or cause the device-wide synchronisation an allocation implies. Such
 * callers cannot pass a workspace either, so the intermediates (T = G V and the row-slice partial sums of
 * U^T T) live in one fixed 8 MiB array that is part of the library image: every GPU that loads the library
 * holds those 8 MiB until the process exits.
 *
 *   G_dev       device: rows x cols, row-major, grad_dtype (sc_dtype)          U_dev  device: rows x rank fp32
 *   V_dev       device: cols x rank fp32                                        X_dev  device: rank x rank fp32 (out)
 *   stream      a cudaStream_t (as void*), NULL = default stream. The three kernels are queued on it.
 *
 * Limits and sharing:
 *   - rows * rank + 16 * rank * rank floats must fit in the 8 MiB array (2,097,152 floats), rank <= 256;
 *     anything larger returns SC_ERR_TOO_LARGE and nothing is launched.
 *   - The call never calls cudaMalloc, cudaFree or any allocating routine.
 *   - All calls (from any thread, on any stream of one device) use the SAME array, which keeps whatever the
 *     previous call left in it. Every element this call reads it has written first, so nothing has to be cleared;
 *     but two calls whose kernels overlap on the GPU would overwrite each other's intermediates: queue them on
 *     one stream, or order them with events.
 *   - The first call on each device looks up the array's device address (that device must be current, as for
 *     every call). Make that first call during set-up, before any stream capture is begun.
 * Errors: INVALID_ARG (NULL pointer), DTYPE, SHAPE, TOO_LARGE, CUDA. */
SC_API sc_status sc_project_static(const void* G_dev, int grad_dtype, const void* U_dev, const void* V_dev,
                                   int64_t rows, int64_t cols, int rank, void* X_dev, void* stream);

/* Copy the anchor momentum (rows x cols fp32) to / from a caller device buffer. */
SC_API sc_status sc_export_anchor_momentum(sc_plan* plan, int mat, void* M_dev);
SC_API sc_status sc_import_anchor_momentum(sc_plan* plan, int mat, const void* M_dev);

/* Copy the first rows x width block of the Rademacher sketch (fp32, row-major, entries +-1) to a device buffer. */
SC_API sc_status sc_export_sketch(sc_plan* plan, int64_t rows, int width, void* Omega_dev);

/* Ask the next steps to also write G_proj (after clipping, fp32 rows x cols) for each matrix.
 * gproj_out: host array of n_mats device pointers (NULL entries skipped), or NULL to switch it off. */
SC_API sc_status sc_set_debug_gproj_out(sc_plan* plan, void* const* gproj_out);

/* Wait for the plan's stream, then copy the per-matrix statistics of the last step into stats[n_mats] (host)
 * and the clip factor applied into *clip (host, may be NULL). */
SC_API sc_status sc_get_stats(sc_plan* plan, sc_mat_stats* stats, float* clip);

/* Wait for the plan's stream and return one latched device condition (SC_ERR_TIMEOUT before SC_ERR_NONFINITE, else
 * SC_OK), clearing only the condition reported: when both are latched, two calls report them one after the other. */
SC_API sc_status sc_get_device_status(sc_plan* plan);

/* Checkpoint / resume. The blob holds, for every matrix, its shape, the anchor momentum, the cached basis (U, s, V, d),
 * whether a basis exists, and the last accepted step tag; AdamW state and weights stay with the caller. host_buf is
 * HOST memory of at least sc_state_bytes(plan) bytes. Both calls wait for the plan's stream. Import needs a plan created
 * with the same shapes in the same order and the same rank (SC_ERR_SHAPE otherwise: every matrix's rows and cols are
 * compared); the filter weights d of Eq. 2 are recomputed from the imported singular values with the importing plan's
 * tau_p. With equal tau_p a step after import continues bit-identically. */
SC_API size_t sc_state_bytes(const sc_plan* plan);
SC_API sc_status sc_state_export(sc_plan* plan, void* host_buf, size_t bytes);
SC_API sc_status sc_state_import(sc_plan* plan, const void* host_buf, size_t bytes);

/* Test hook for the failure path of the device-side bounded waits: queues one tiny kernel that waits on a barrier
 * nothing will ever signal, gives up after max_polls polls (1..2^20, i.e. at most a few milliseconds), latches the
 * time-out bit and returns normally. sc_get_device_status then reports SC_ERR_TIMEOUT once. Nothing hangs or traps. */
SC_API sc_status sc_debug_wait_probe(sc_plan* plan, int max_polls);

/* Device-time profile by phase of the method. Categories:
 *   0 anchor EMA (Eq. 1)            1 basis build, passes over the momentum     2 basis build, small factorisations
 *   3 projection T = G V            4 r x r filter, C^T, norms                  5 fused correction + AdamW update */
#define SC_PROFILE_CATEGORIES 6
typedef struct sc_profile {
  double ms[SC_PROFILE_CATEGORIES];       /* summed device time between event pairs around each group of launches */
  int64_t spans[SC_PROFILE_CATEGORIES];   /* number of timed groups (one per shape class and phase) */
} sc_profile;

/* Switch event-based profiling on or off (off by default; when on, each phase is bracketed by CUDA events on
 * the plan's stream). */
SC_API sc_status sc_set_profiling(sc_plan* plan, int on);

/* Wait for the plan's stream, write the profile accumulated since the last read-out into *out, and reset it. */
SC_API sc_status sc_get_profile(sc_plan* plan, sc_profile* out);

/* Number of kernels this library has launched in this process so far. */
SC_API int64_t sc_kernel_launch_count(void);

/* Step tag of the last accepted anchor (-1 if none) and number of matrices that have a basis. */
SC_API sc_status sc_get_anchor_info(sc_plan* plan, int64_t* last_tag, int* n_with_basis);

/* 1 if the tensor-core (tcgen05) kernels serve this plan, 0 if the fp32 CUDA-core kernels do. */
SC_API int sc_plan_uses_tensor_cores(const sc_plan* plan);

SC_API const char* sc_status_string(sc_status s);
SC_API int sc_version(void);

#ifdef __cplusplus
}
#endif
#endif /* SPECTRAL_CORRECTION_H_ */

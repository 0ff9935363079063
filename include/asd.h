/*
 * asd.h - C ABI of the B200 (sm_100a) Autospeculative Decoding library.
 *
 * The library runs, for a batch of independent chains, the speculation round of
 * Autospeculative Decoding (Algorithm 1 with its Verifier, Algorithm 2, and the
 * Gaussian rejection sampler, Algorithm 3) on the Euler chain of Eq. 7,
 *     y_{i+1} = y_i + eta_i g(t_i, y_i) + sigma_{i+1} xi_{i+1},
 * in the stochastic-localization parametrisation of Eq. 4 (g = posterior mean m),
 * plus the loop around the round and the sequential sampler of Eq. 7.
 *
 * Conventions
 *  - Plain C, no C++ types cross the boundary; every function returns an asd_status
 *    and never throws, aborts or exits.
 *  - "host" pointers are ordinary CPU memory; "dev" pointers are CUDA device memory
 *    on the device that was current in asd_create.  The caller owns every buffer it
 *    passes; the library copies what it keeps.  The library owns its tables, its copy
 *    of the denoiser parameters and all workspaces (allocated in asd_create, sized for
 *    max_chains x window, freed in asd_destroy).
 *  - All device work is enqueued on the stream given to asd_create (a cudaStream_t
 *    passed as void*; NULL = the default stream).
 *  - Randomness (Algorithm 1, the two "sample" lines) is counter based: Philox4x32-10,
 *    key = seed, counter = (dimension block q, step i in 1..K, chain id, tag);
 *    tag 0 gives xi_i[4q..4q+3] by Box-Muller on word pairs, tag 1 (q = 0) gives u_i
 *    from word 0; uniform map U(r) = ((r >> 9) + 0.5) 2^-23.  A step's (u_i, xi_i) is
 *    the same in every round that reaches it, and a chain's result does not depend on
 *    which batch or partition it is run in (chain id = chain_id_base + position).
 *  - On error nothing is partially advanced: the chain state is either the one before
 *    the call or the one after it.  asd_last_error gives a message for the last
 *    failing call on a context.
 *  - No CPU fallback exists: without a CUDA device every compute entry point returns
 *    ASD_ERR_CUDA.
 */
#ifndef ASD_H
#define ASD_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct asd_ctx asd_ctx; /* opaque, owned by the library */

typedef enum {
  ASD_OK = 0,
  ASD_ERR_INVALID_ARG = 1, /* NULL pointer, size out of range, inconsistent sizes */
  ASD_ERR_UNSUPPORTED = 2, /* valid request the library does not implement */
  ASD_ERR_OOM = 3,         /* device or host allocation failed */
  ASD_ERR_CUDA = 4,        /* a CUDA call failed, or no device */
  ASD_ERR_STATE = 5,       /* call made in the wrong state (e.g. round before reset) */
  ASD_ERR_TIMEOUT = 6      /* a bounded device-side wait ran out (kernel returned early) */
} asd_status;

typedef enum {
  ASD_DEN_GMM_ISO = 0,      /* x* ~ sum_j pi_j N(c_j, s^2 I): closed-form posterior mean (Eq. 4) */
  ASD_DEN_GAUSS_LINEAR = 1, /* x* ~ N(mu0, Q diag(lam) Q^T): m = (I + t Sigma)^-1 (mu0 + Sigma y) */
  ASD_DEN_RESMLP_BF16 = 2   /* residual MLP, bf16 weights/activations, fp32 accumulation */
} asd_den_kind;

/*
 * Denoiser / drift g(t_i, y) ("model call", Section 4).  All pointers are HOST
 * pointers read during asd_create only.  Fields of the other kinds are ignored.
 *
 * RESMLP_BF16 computes, for a point y at step i of chain c (bf16() = round to
 * nearest even, sums in fp32):
 *     x   = [bf16(c_in[i] y) ; bf16(cond_c) ; bf16(temb(i))]            (length d + d_cond + d_temb)
 *     h_0 = bf16(W_in x + b_in)
 *     h_l = bf16(h_{l-1} + SiLU(W_l h_{l-1} + b_l)),  l = 1..n_layers,   SiLU(z) = z / (1 + exp(-z))
 *     g   = c_skip[i] y + c_out[i] (W_out h_L + b_out)
 *     temb(i): tau = 1000 i / K, half = d_temb / 2, w_f = exp(-ln(1e4) f / half),
 *              [sin(tau w_f)]_{f<half} ++ [cos(tau w_f)]_{f<half}
 * Weights are bf16 bit patterns, row-major [out, in].  width must be a multiple of 8,
 * d_temb even.
 */
typedef struct {
  int32_t kind; /* asd_den_kind */
  /* GMM_ISO */
  int32_t n_comp;       /* 1..256 */
  const float* means;   /* [n_comp * d] */
  const float* weights; /* [n_comp], positive */
  float sigma;          /* component std s > 0 */
  /* GAUSS_LINEAR */
  const float* mu0; /* [d] */
  const float* Q;   /* [d * d] row-major, columns are orthonormal eigenvectors of Sigma */
  const float* lam; /* [d] eigenvalues of Sigma, >= 0 */
  /* RESMLP_BF16 */
  int32_t d_cond, d_temb, width, n_layers;
  const uint16_t* W_in;  /* [width * (d + d_cond + d_temb)] */
  const uint16_t* W_hid; /* [n_layers * width * width] */
  const uint16_t* W_out; /* [d * width] */
  const float* b_in;     /* [width] */
  const float* b_hid;    /* [n_layers * width] */
  const float* b_out;    /* [d] */
  const float* c_in;     /* [K] or NULL => 1 */
  const float* c_skip;   /* [K] or NULL => 0 */
  const float* c_out;    /* [K] or NULL => 1 */
} asd_denoiser;

/*
 * Problem statement = the inputs of Algorithm 1: K steps, the time grid (step sizes
 * eta_i = t_{i+1} - t_i), the variances, the speculation length theta ("window").
 */
typedef struct {
  int32_t d;          /* dimension of y, 1..65536 */
  int32_t K;          /* number of Euler steps, >= 1 */
  int32_t window;     /* speculation length theta >= 1; values >= K act like K, i.e. theta = infinity:
                         every round drafts to the end of the grid (workspaces are sized max_chains x window) */
  int32_t max_chains; /* capacity of the batch, >= 1 */
  const double* t;      /* host [K+1], strictly increasing, t[0] >= 0 */
  const double* sigma2; /* host [K]: sigma_{i+1}^2 for the step i -> i+1, or NULL => eta_i
                           (stochastic localization: increments have variance eta, Theorem 2) */
  uint64_t seed;        /* Philox key */
  asd_denoiser den;
  uint32_t flags;       /* 0 or ASD_FLAG_* */
} asd_config;

/*
 * ASD_FLAG_DEBUG_ALL_SLOTS: the Verifier (Algorithm 2) only needs the end of the all-accepted prefix,
 * so by default the verify kernel stops at the first rejected slot and never reads the drifts
 * beyond it.  With this flag every slot of the window goes through the accept test of Algorithm 3
 * (as Algorithm 2 is written) so that asd_debug_last_round returns ln ratio for all of them.  The
 * chain states are identical either way.
 */
#define ASD_FLAG_DEBUG_ALL_SLOTS 1u

/*
 * ASD_FLAG_ADAPTIVE_WINDOW: every chain chooses its own speculation length theta_c for the next round
 * from its own history, between 2 and `window` (the paper fixes theta, Theorem 4 picks it from
 * K, beta, eta, d; Algorithm 1 is exact for any theta, and a theta that depends only on the chain's past
 * is adapted to the filtration of its proof).  Rule, in integers so that it is reproducible anywhere:
 * with p = steps advanced in the round (accepted prefix + the resampled step, or the whole window),
 *     ema8  <- (ema8 + 8 p) >> 1          (8 x running mean of p, initial value 32)
 *     theta <- clamp(2 + (3 ema8) / 16, 2, window)     (about 2 + 1.5 x mean; initial min(window, 8))
 * so a chain that keeps accepting its whole window grows it by half each round and a chain that rejects
 * early drafts little.  A chain's result still depends only on its id.  asd_sequential_ddpm ignores it.
 * asd_get_window_state / asd_set_window_state complete the chain state for stop and resume
 * (device buffers [n] int32 each, any may be NULL; values outside 1..window are clamped when used).
 */
#define ASD_FLAG_ADAPTIVE_WINDOW 2u

/*
 * ASD_FLAG_LOOKAHEAD: the batched pass also evaluates the drift at the LAST drafted point of each
 * window, y^_{a+w} (when a + w < K).  If the whole window is accepted that point is the chain's next
 * state and the drift there is exactly the v_a that the next iteration of Algorithm 1 would compute in
 * its first model call, so the call is skipped: a round then costs one sequential model pass instead of
 * two for every chain that accepted its window.  The law of the output is untouched (the same function
 * is evaluated at the same point, one round earlier); per-chain results agree with the default mode
 * up to the rounding differences of evaluating that row inside a different batch.  Costs one more row
 * per chain and round in the batched pass and a [max_chains, d] float buffer.  rows_pass1 then counts
 * only the chains whose first call was really made.
 */
#define ASD_FLAG_LOOKAHEAD 4u

/*
 * ASD_FLAG_TRAJECTORY: keep Algorithm 1's return value (y_0, ..., y_K) for every chain, not only y_K:
 * a [max_chains, K + 1, d] float buffer on the device that the verify step fills as chains advance (the
 * accepted proposal samples, then the resampled state) and asd_get_trajectory copies out.  Row 0 is the
 * y_0 of asd_reset; after asd_set_state rows below the restored cursor are whatever the context held.
 */
#define ASD_FLAG_TRAJECTORY 8u

/*
 * ASD_FLAG_DEBUG_DUMP: record ln u and ln ratio of the last round per window slot for
 * asd_debug_last_round (two [max_chains, window] float buffers, written by the verify step every
 * round).  Implied by ASD_FLAG_DEBUG_ALL_SLOTS.  Without it only the accepted prefix lengths are kept.
 */
#define ASD_FLAG_DEBUG_DUMP 16u

typedef struct {
  int32_t n_active_before; /* chains with a < K when the round started */
  int32_t n_active_after;
  int64_t rows_pass1;      /* drift evaluations at the current points (Algorithm 1, v_a) */
  int64_t rows_pass2;      /* drift evaluations at drafted points (the parallel for) */
  int64_t accepted_total;  /* sum over chains of steps advanced this round */
} asd_round_stats;

typedef struct {
  int64_t rounds_max;   /* rounds until the last chain finished (= sequential depth / 2) */
  double rounds_mean;   /* mean over chains of while-loop iterations (parallel rounds per sample) */
  int64_t rows_total;   /* drift evaluations made, both passes */
  double ms_total;      /* device time of the call, CUDA events on the context's stream */
  int64_t launches;     /* kernels launched by the call */
  int64_t rows_verified; /* drafted-point drifts the Verifier read (it stops after the first rejection) */
} asd_run_stats;

/* Library version string (static storage). */
const char* asd_version(void);

/*
 * Validate the configuration, build the fp32 tables (eta_i, sigma_{i+1}, t_i and the
 * accept-test coefficients eta/sigma, eta^2 / 2 sigma^2 - Algorithm 3 with v = m^ - m
 * = eta (v_a - g)), copy / repack the denoiser parameters and allocate all workspaces.
 * cfg and everything it points to may be released after the call.
 * Errors: INVALID_ARG (cfg/out NULL, sizes or grid invalid), UNSUPPORTED, OOM, CUDA.
 */
asd_status asd_create(const asd_config* cfg, void* cuda_stream, asd_ctx** out);

/*
 * Start n_chains chains at cursor a = 0 (Algorithm 1, "a <- 0").  y0_dev: [n_chains*d]
 * fp32 or NULL for y_0 = 0 (Eq. 4 starts at 0).  cond_dev: [n_chains*d_cond] fp32,
 * required iff the denoiser has d_cond > 0.  Chain j uses id chain_id_base + j
 * (must stay below 2^32).  Errors: INVALID_ARG, STATE, CUDA.
 */
asd_status asd_reset(asd_ctx* ctx, int32_t n_chains, uint64_t chain_id_base,
                     const float* y0_dev, const float* cond_dev);

/*
 * ONE iteration of Algorithm 1's while loop for every chain with a < K: drift at the
 * current point, draft of the window, drift at every drafted prefix point in one
 * batched pass, Verifier (Algorithms 2 and 3), advance.  If stats_host is not NULL the
 * stream is synchronised and the round's counters are returned; otherwise the call only
 * enqueues.  A round with no active chain is a no-op.  Errors: STATE, CUDA, TIMEOUT.
 */
asd_status asd_round(asd_ctx* ctx, asd_round_stats* stats_host);

/*
 * Rounds to completion (Algorithm 1).  y_out_dev: [n*d] fp32 receives y_K (the sample of
 * the target is y_K / t_K); rounds_out_dev: [n] int32 or NULL; stats_host or NULL.
 * Synchronises the stream before returning.  Continues from the current state, so it may
 * follow asd_round / asd_set_state.
 * The rounds are enqueued without waiting for one another (their counters come back through a pinned
 * ring a few rounds late; rounds enqueued after the last chain finished do nothing) and, unless
 * per-phase timing is on, each round is replayed as a CUDA graph on a stream of the library's own that
 * is ordered after the work already in the context's stream and before what the caller enqueues after
 * the call.  Do not call it (or asd_sequential_ddpm) while the context's stream is being captured.
 */
asd_status asd_sample(asd_ctx* ctx, float* y_out_dev, int32_t* rounds_out_dev, asd_run_stats* stats_host);

/*
 * The sequential sampler of Eq. 7 from the current state: K - a steps of one drift
 * evaluation each, with the same xi streams (never consumes u).  Bit-identical to
 * asd_sample on a context created with window = 1.
 */
asd_status asd_sequential_ddpm(asd_ctx* ctx, float* y_out_dev, asd_run_stats* stats_host);

/*
 * End-to-end convenience with HOST buffers: copies y0 (or zeros if NULL) and cond to the
 * device, resets, samples (ASD if sequential == 0, Eq. 7 otherwise) and copies y_K and the
 * round counters back.  All pointers host; y_out_host [n*d], rounds_out_host [n] or NULL.
 */
asd_status asd_sample_host(asd_ctx* ctx, int32_t n_chains, uint64_t chain_id_base,
                           const float* y0_host, const float* cond_host, int32_t sequential,
                           float* y_out_host, int32_t* rounds_out_host, asd_run_stats* stats_host);

/*
 * Chain state = (cursor a, y_a, rounds so far); with the counter-based randomness this is
 * everything needed to stop and resume.  Device buffers [n], [n*d], [n]; any may be NULL.
 */
asd_status asd_get_state(asd_ctx* ctx, int32_t* a_dev, float* y_dev, int32_t* rounds_dev);
asd_status asd_set_state(asd_ctx* ctx, const int32_t* a_dev, const float* y_dev, const int32_t* rounds_dev);
asd_status asd_get_window_state(asd_ctx* ctx, int32_t* window_dev, int32_t* ema8_dev);
asd_status asd_set_window_state(asd_ctx* ctx, const int32_t* window_dev, const int32_t* ema8_dev);

/*
 * Diagnostics of the last round, indexed by chain position: ln ratio (Algorithm 3) and
 * ln u per window slot ([n*window] fp32 each; slots beyond the chain's window are not
 * written; ln ratio of slots after the first rejected one is NaN unless the context was
 * created with ASD_FLAG_DEBUG_ALL_SLOTS) and the accepted prefix length n ([n] int32; -1 for
 * chains that were inactive).  Device buffers, any may be NULL.  The two ln arrays need a context
 * created with ASD_FLAG_DEBUG_DUMP (or ASD_FLAG_DEBUG_ALL_SLOTS): STATE otherwise.
 */
asd_status asd_debug_last_round(asd_ctx* ctx, float* ln_ratio_dev, float* ln_u_dev, int32_t* accepted_dev);

/*
 * Algorithm 1's output (y_0, ..., y_K) per chain: traj_dev [n, K + 1, d] fp32 (device).  Rows beyond a
 * chain's cursor are not yet written.  Needs ASD_FLAG_TRAJECTORY (STATE otherwise).  Enqueues a copy on
 * the context's stream.
 */
asd_status asd_get_trajectory(asd_ctx* ctx, float* traj_dev);

/*
 * Run statistics of the Verifier (Algorithm 2): hist_host[m] = number of chain-rounds since the last
 * asd_reset whose accepted prefix had length m (m = the chain's window means the whole window was
 * accepted; a chain-round advances m + 1 steps otherwise), m = 0 .. min(capacity, window + 1) - 1;
 * *n_out = entries written.  hist_host is a HOST buffer; the call synchronises the stream.
 * Rounds of asd_sequential_ddpm count as prefix 1.
 */
asd_status asd_get_prefix_histogram(asd_ctx* ctx, int64_t* hist_host, int32_t capacity, int32_t* n_out);

/*
 * The drift alone: out[r] = g(t_{step[r]}, y[r]) for r < n_rows, with the conditioning of
 * chain position slot[r] (slot_dev may be NULL when d_cond = 0).  Device buffers:
 * step_dev [n_rows] int32 in [0, K), y_dev [n_rows*d], out_dev [n_rows*d].
 * n_rows <= max_chains * max(window - 1, 1).  Uses the same kernels as the two passes of
 * the round.
 */
asd_status asd_denoise(asd_ctx* ctx, int32_t n_rows, const int32_t* step_dev, const float* y_dev,
                       const int32_t* slot_dev, float* out_dev);

/*
 * Measurement aid (the paper has no counterpart): per-phase device time of asd_sample, taken
 * with CUDA event pairs on the context's stream around the launches of each phase, so a
 * phase's time is the time its kernels occupied the stream.  asd_set_profiling(ctx, 1) clears
 * the accumulators and turns the events on (two event records per phase and round);
 * asd_get_profile copies up to `capacity` entries (name has static storage; launches = kernels
 * launched in the phase; rows = chains or points processed by it, counted by asd_sample only).
 */
typedef struct {
  const char* name;
  int64_t launches;
  double ms;
  int64_t rows;
} asd_phase_time;
asd_status asd_set_profiling(asd_ctx* ctx, int32_t enable);
asd_status asd_get_profile(asd_ctx* ctx, asd_phase_time* out, int32_t capacity, int32_t* n_out);

/*
 * DDPM front end (Theorem 1 and the remark after Algorithm 1): from a DDPM noise schedule and the
 * network's prediction type to the inputs of asd_create.  Host arithmetic only, all pointers host.
 *   alpha_bar [K+1]: cumulative signal level of the K+1 noise levels the sampler visits, in sampling
 *                    order, i.e. strictly increasing, inside (0, 1)  (x_level = sqrt(ab) x0 + sqrt(1-ab) eps)
 *   pred: what the network returns for input x_level - ASD_PRED_X0 (E[x0 | x]), ASD_PRED_EPS, ASD_PRED_V
 *   map:  ASD_MAP_SL        t = ab / (1 - ab), y = sqrt(t (1 + t)) x, sigma^2 = eta: the Euler chain of the
 *                           stochastic-localization process that Theorem 1 shows equivalent to the DDPM
 *         ASD_MAP_ANCESTRAL the DDPM ancestral sampler x_{i+1} = a_i x_i + b_i E[x0 | x_i] + s_i xi itself,
 *                           written in y_i = x_i / (a_0 .. a_{i-1}) as Eq. 7 with eta_i = b_i / A_{i+1},
 *                           sigma_{i+1} = s_i / A_{i+1}; s_i^2 = beta~ (large_variance = 0) or beta (1).
 *                           Meant for the network denoiser (the closed-form drifts read t as SL time).
 * Outputs: t_out [K+1] and sigma2_out [K] for asd_config, c_in / c_skip / c_out [K] for asd_denoiser,
 * x_scale [K+1] with x_i = x_scale[i] y_i (start the chain at y_0 = x_0 / x_scale[0]; the DDPM sample
 * at the last level is x_scale[K] y_K).  Errors: INVALID_ARG.
 */
typedef enum { ASD_PRED_X0 = 0, ASD_PRED_EPS = 1, ASD_PRED_V = 2 } asd_pred_kind;
typedef enum { ASD_MAP_SL = 0, ASD_MAP_ANCESTRAL = 1 } asd_map_kind;
asd_status asd_ddpm_schedule(int32_t K, const double* alpha_bar, int32_t pred, int32_t map, int32_t large_variance,
                             double* t_out, double* sigma2_out, float* c_in, float* c_skip, float* c_out,
                             double* x_scale);

/*
 * asd_denoise_static - the drift of the network denoiser without any device allocation.
 * (The paper has no counterpart: this is a deployment aid of this library.)
 *
 * asd_denoise can only take as many rows as the context was sized for in asd_create, and
 * making room for more means a new context, i.e. cudaMalloc.  Some callers cannot do that at
 * the point where they need the drift: a serving loop that must not take cudaMalloc's
 * device-wide synchronisation, a process that has handed all remaining device memory to another
 * allocator (so cudaMalloc would fail), or code running where its host forbids allocation calls.
 * For them this entry point keeps the activations of the GEMM chain (input rows and the two
 * hidden-state buffers) and its row counter in ONE fixed array of ASD_STATIC_SCRATCH_BYTES
 * (8 MiB) that is part of the library image: every GPU on which the library is used holds those
 * 8 MiB from the first kernel launch until the process exits.
 *
 * Arguments, layouts and result are those of asd_denoise (device pointers; rows beyond n_rows
 * untouched); the result is identical to asd_denoise's.  Only ASD_DEN_RESMLP_BF16 contexts are
 * accepted (the closed-form drifts use no scratch: UNSUPPORTED).  n_rows may be at most
 * floor((8 MiB - 1 KiB) / (2 (in_pad + 2 width))) with in_pad = d + d_cond + d_temb rounded up
 * to 64 - asd_denoise_static_max_rows returns it; larger requests fail with INVALID_ARG and
 * nothing is launched.  The context's device must be current (STATE otherwise).
 *
 * The first call on a device looks up the array's device address; make that first call before
 * starting any stream capture.  The call synchronises the context's stream before returning.
 * All contexts and all calls share the one array and it keeps the previous call's contents
 * (this call rewrites everything it reads): calls that overlap on the GPU - different streams,
 * different contexts or threads - race on it; run them one after the other.
 * It calls no cudaMalloc / cudaFree and no allocating library routine.
 */
#define ASD_STATIC_SCRATCH_BYTES (8u << 20)
asd_status asd_denoise_static(asd_ctx* ctx, int32_t n_rows, const int32_t* step_dev, const float* y_dev,
                              const int32_t* slot_dev, float* out_dev);
asd_status asd_denoise_static_max_rows(const asd_ctx* ctx, int32_t* max_rows_out);

/*
 * Failure-path self-test (the paper has no counterpart).  Every wait inside the kernels is bounded:
 * when its limit (about 0.2 s) runs out the kernel records ASD_ERR_TIMEOUT, finishes, and the next
 * synchronising call returns that status with the context still usable.  This call launches one thread
 * that waits on a barrier nothing completes and returns what the library reports: ASD_ERR_TIMEOUT.
 */
asd_status asd_debug_wait_selftest(asd_ctx* ctx);

/* Message for the last error on this context (static or context storage; never NULL). */
const char* asd_last_error(const asd_ctx* ctx);

void asd_destroy(asd_ctx* ctx);

#ifdef __cplusplus
}
#endif
#endif /* ASD_H */

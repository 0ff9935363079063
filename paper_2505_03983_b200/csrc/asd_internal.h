// Internal declarations shared by the translation units of the ASD library
// (context layout, kernel launchers).  Nothing here crosses the C ABI.
#pragma once

#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <cuda.h>
#include <stdint.h>

#include <map>
#include <string>
#include <tuple>
#include <vector>

#include "asd.h"

namespace asd {


// ---- device-side bookkeeping shared by all kernels of a round -------------------------
// One small block of counters in device memory; the prep kernel rewrites it every round.
struct RoundCounters {
  int n_active;                 // chains with a < K at the start of the round
  int rows2;                    // sum over active chains of (w - 1): rows of pass 2
  int n_active_after;           // written by the verify kernel
  int err;                      // device error word: 0, or ASD_ERR_TIMEOUT / ASD_ERR_STATE
  unsigned long long accepted;  // steps advanced this round
  unsigned long long rows_total;  // running total of drift evaluations since reset
  unsigned long long rows_verified;  // running total of drift rows the verify kernel read since reset
  int n_eval;                   // chains whose v_a has to be evaluated this round (look-ahead: not all active ones)
  int rounds_max;               // written by the finish kernel of a run: max and sum over chains of the round counters
  unsigned long long rounds_sum;
};

// Per-step fp32 tables, built on the host in fp64 (asd_create).
struct Tables {
  const float* eta;    // [K]   eta_i = t_{i+1} - t_i
  const float* sig;    // [K]   sigma_{i+1}
  const float* c1;     // [K]   eta_i / sigma_{i+1}              (accept test, Algorithm 3)
  const float* c2;     // [K]   eta_i^2 / (2 sigma_{i+1}^2)
  const float* tt;     // [K+1] t_i
  const float* c_in;   // [K]   (MLP) input scale
  const float* c_skip; // [K]
  const float* c_out;  // [K]
};

// Which rows a denoiser pass evaluates: point r is ysrc[row_map ? row_map[r] : r], at step
// row_step[r], conditioned on chain position row_slot[r]; *n_rows_dev rows (<= n_rows_max).
struct RowSet {
  const int* n_rows_dev;
  int n_rows_max;
  const float* ysrc;
  const int* row_map;
  const int* row_step;
  const int* row_slot;
  // true when *n_rows_dev was written by a kernel (or copy) that had completed before the kernel directly in
  // front of the consumer started, so a kernel launched with programmatic stream serialization may read it
  // before its dependency wait
  bool settled = false;
};

struct GmmParams {
  int n_comp;
  const float* means;   // [n_comp, d]
  const float* log_pi;  // [n_comp]
  const float* cnorm;   // [n_comp] |c_j|^2
  float s2;
};

struct GaussParams {
  const float* Q;    // [d, d]   columns = eigenvectors
  const float* Qt;   // [d, d]   transposed copy
  const float* qmu;  // [d]      Q^T mu0
  const float* lam;  // [d]
};

struct MlpParams {
  int d_cond, d_temb, width, n_layers, in_dim, in_pad;
  const __nv_bfloat16* W_in;   // [width, in_pad]  (zero padded columns)
  const __nv_bfloat16* W_hid;  // [n_layers, width, width]
  const __nv_bfloat16* W_out;  // [d, width]
  const float* b_in;
  const float* b_hid;
  const float* b_out;
  const __nv_bfloat16* temb;   // [K, d_temb]
  const __nv_bfloat16* cond;   // [max_chains, d_cond]  bf16 copy made at reset
  __nv_bfloat16* X;            // [row_cap, in_pad]
  __nv_bfloat16* H[2];         // [row_cap, width]
  int row_cap;
};

// A contiguous sub-batch of chains [start, start + n) with its own bookkeeping.  The whole batch is one
// lane; asd_sample may split it into two that take turns (see asd_api.cu).
struct Lane {
  int start = 0, n = 0;
  int* act = nullptr;        // [n] active position -> chain position inside the lane
  int* row_off = nullptr;    // [n + 1]
  int* step1 = nullptr;      // [n]
  RoundCounters* counters = nullptr;
  int* v_off = nullptr;      // device int: row of the drift buffer where this lane's v_a rows start
  // look-ahead (whole batch only): chains that need the first model call, their steps, and for every
  // active position the row of that call's output (or -1: v_a was saved by the previous round)
  int* act1 = nullptr;
  int* step1e = nullptr;
  int* idx1 = nullptr;
};

// Phases of a round, for the optional per-phase CUDA-event timing.
enum Phase {
  PH_PREP = 0, PH_PACK, PH_D1_IN, PH_D1_HID, PH_D1_OUT, PH_D1_ANALYTIC, PH_DRAFT,
  PH_D2_IN, PH_D2_HID, PH_D2_OUT, PH_D2_ANALYTIC, PH_VERIFY, PH_COUNT
};

struct PhaseAcc {
  long long launches = 0;
  double ms = 0.0;
  long long rows = 0;  // rows (points, chains) processed by the phase
};

struct Ctx {
  // configuration
  int d = 0, K = 0, window = 0, max_chains = 0, kind = 0;
  uint64_t seed = 0;
  cudaStream_t stream = nullptr;
  int device = 0;
  int num_sms = 148;
  // state
  int n = 0;  // chains of the current reset
  uint64_t chain_base = 0;
  bool have_reset = false;
  int round_bound = 0;  // asd_round: upper bound on the active chains (chains only finish, so a stale value is valid)
  bool adaptive = false;         // ASD_FLAG_ADAPTIVE_WINDOW
  bool lookahead = false;        // ASD_FLAG_LOOKAHEAD
  int* has_v = nullptr;          // [max_chains] 1: vsave holds v_a of the chain's next round
  float* vsave = nullptr;        // [max_chains, d]
  int* act1 = nullptr;           // [max_chains]
  int* step1e = nullptr;         // [max_chains]
  int* idx1 = nullptr;           // [max_chains]
  bool debug_all_slots = false;  // ASD_FLAG_DEBUG_ALL_SLOTS: the verify kernel evaluates every window slot
  // device arrays
  float* y = nullptr;        // [max_chains, d]
  int* a = nullptr;          // [max_chains]
  int* rounds = nullptr;     // [max_chains]
  int* wnd = nullptr;        // [max_chains] per-chain speculation length of the next round (adaptive mode)
  int* ema8 = nullptr;       // [max_chains] 8 x running mean of the steps advanced per round (adaptive mode)
  int* act = nullptr;        // [max_chains] active position -> chain position
  int* row_off = nullptr;    // [max_chains + 1]
  int* step1 = nullptr;      // [max_chains] cursor of the active chain
  int* row_step = nullptr;   // [max_rows] step of a pass-2 row
  int* row_slot = nullptr;   // [max_rows] chain position of a pass-2 row
  float* v = nullptr;        // [max_chains, d] drift at the current point, by active position
  float* Yhat = nullptr;     // [max_rows, d] drafted points y^_{a+k}, k = 1..w-1
  float* G = nullptr;        // [max_rows, d] drift at the drafted points
  // staggered lanes (network denoiser): second drift buffer (ticks alternate), the two half-batches, the
  // row count of a merged pass
  float* G2 = nullptr;
  Lane lanes[2];
  int* merged_rows = nullptr;
  long long extra_rows_total = 0, extra_rows_verified = 0;  // lanes' counters, added by the run statistics
  float* dbg_lr = nullptr;   // [max_chains, window]  (ASD_FLAG_DEBUG_DUMP / ASD_FLAG_DEBUG_ALL_SLOTS only)
  float* dbg_lu = nullptr;   // [max_chains, window]
  int* acc_len = nullptr;    // [max_chains]
  float* slot_dot = nullptr; // [max_chains, window] per-slot reductions and ln u handed from the slots kernel to the verify kernel
  float* slot_nrm = nullptr;
  float* slot_lu = nullptr;
  int* first_rej = nullptr;  // [max_chains] first rejected slot of the round, lowered by the slots kernel
  int fail_alloc_after = -1; // ASD_FAIL_ALLOC_AFTER at asd_create (test hook): device allocations that succeed before one fails
  int verify_horizon = -1;   // ASD_VERIFY_HORIZON at asd_create (tuning aid); -1: chosen per launch
  float* traj = nullptr;     // [max_chains, K + 1, d] (ASD_FLAG_TRAJECTORY only)
  unsigned long long* hist = nullptr;  // [window + 1] chain-rounds by accepted prefix length since the last reset
  RoundCounters* counters = nullptr;
  RoundCounters* counters_host = nullptr;  // pinned
  // asd_sample runs ahead of the device: the counters of round r land in ring_host[r % kRing] and
  // ring_ev[r % kRing] tells when
  static constexpr int kRing = 8;
  RoundCounters* ring_host = nullptr;      // pinned [kRing][3]: whole batch or lane 0, lane 1, merged row count
  cudaEvent_t ring_ev[kRing] = {};
  int max_rows = 0;
  Tables tab{};
  GmmParams gmm{};
  GaussParams gauss{};
  MlpParams mlp{};
  std::vector<void*> dev_allocs;
  std::map<std::tuple<const void*, int, int, int>, CUtensorMap> tmaps;
  std::map<const void*, int> func_smem;  // kernel -> dynamic shared memory opted in on this context's device
  int gemm_mode = 0;                     // ASD_GEMM_MODE at asd_create: 0 planner, 1 "cta", 2 "pair"
  int fused_ready = 0, fused_clusters = 0;  // one-launch network: 0 not yet checked, 1 usable, -1 not; clusters that fit the device at once
  int fused_mode = -1;                   // ASD_MLP_FUSED=1 at asd_create: the whole network in one launch (off otherwise)
  bool stagger = false;                  // ASD_STAGGER=1 at asd_create
  int resident_mode = 1;                 // ASD_RESIDENT at asd_create: 0 never, 1 asd_sample / asd_sequential_ddpm, 2 asd_round too
  // One speculation round captured as a CUDA graph per (window, use_u, bound on active chains); replayed
  // on a private stream that is forked from and joined to the caller's stream.
  struct RoundGraph { cudaGraphExec_t exec; long long launches; };
  std::map<std::tuple<int, int, long long>, RoundGraph> graphs;
  cudaStream_t gstream = nullptr;
  cudaEvent_t fork_ev = nullptr, join_ev = nullptr;
  bool use_graphs = true;
  std::string err;
  long long launches = 0;
  cudaEvent_t ev0 = nullptr, ev1 = nullptr;
  // per-phase timing (off by default)
  bool prof_on = false;
  PhaseAcc prof[PH_COUNT];
  std::vector<cudaEvent_t> ev_pool;
  size_t ev_used = 0;
  struct Pending { int phase; size_t e0, e1; int launches; };
  std::vector<Pending> pending;
};

// Brackets the launches of one phase with two events when timing is on.
struct ProfScope {
  Ctx* c;
  int phase;
  long long l0;
  size_t e0;
  ProfScope(Ctx* c_, int phase_);
  ~ProfScope();
};
void prof_collect_some(Ctx* c, long long count);
void prof_collect(Ctx* c);  // after a stream synchronisation: fold pending event pairs into c->prof

// ---- launchers (asd_kernels.cu) ---------------------------------------------------------
Lane whole_batch(const Ctx* c);
void launch_prep(Ctx* c, const Lane& L, int window);
// v_base + (*v_off_dev) rows: where the lane's v_a rows are (v_off_dev may be null: offset 0)
void launch_draft(Ctx* c, const Lane& L, int window, const float* v_base, const int* v_off_dev);
int verify_horizon(const Ctx* c, int n, int window);  // slots the slots kernel reduces ahead of the verify kernel
void launch_verify(Ctx* c, const Lane& L, int window, bool use_u, const float* G, const float* v_base,
                   const int* v_off_dev);
// Pass-1 rows of lane L appended behind the drafted rows of the other lane: row = *row_base_dev + p gets
// the point y_a, its network input, step and slot; *m_merged_dev = *row_base_dev + active chains of L.
void launch_pack_appended(Ctx* c, const Lane& L, const int* row_base_dev, int* m_merged_dev);
void launch_pack(Ctx* c, const RowSet& rs);
void launch_gmm(Ctx* c, const RowSet& rs, float* out);
void launch_gauss(Ctx* c, const RowSet& rs, float* out);
void launch_traj_seed(Ctx* c);  // trajectory row a_j <- y_j for every chain of the batch
// asd_reset in one launch: state, cursors, counters, per-chain window state, histogram, trajectory row 0 and the
// bf16 copy of the conditioning
void launch_reset(Ctx* c, const float* y0_dev, const float* cond_dev);
// end of a run in one launch: y -> y_out, rounds -> rounds_out (either may be null), max / sum of the round counters
void launch_finish(Ctx* c, float* y_out_dev, int* rounds_out_dev);

// ---- MLP forward (asd_gemm.cu) ----------------------------------------------------------
// Runs the GEMM chain on the rows already packed into mlp.X; writes out[r] for r < *n_rows_dev.
// pass: 0 = drift at the current points, 1 = drift at the drafted points, 2 = stand-alone call.
asd_status mlp_forward(Ctx* c, const RowSet& rs, float* out, int pass);
void launch_wait_selftest(Ctx* c);  // one bounded wait that must run out (failure-path self-test)
// 2-D bf16 row-major tensor map [rows, cols], box [box_rows, 64 columns], 128-byte swizzle; cached per context
bool get_tmap(Ctx* c, const void* ptr, int rows, int cols, int box_rows, CUtensorMap* out);
void ensure_dynamic_smem(Ctx* c, const void* func, int bytes);  // per-device opt-in to large dynamic shared memory
// the whole network in one launch (asd_mlp_fused.cu; on request only)
bool use_fused_mlp(Ctx* c, int m_bound);
asd_status launch_mlp_fused(Ctx* c, const RowSet& rs, float* out);

// ---- chain-resident round driver for the closed-form drifts (asd_resident.cu) ------------------
bool resident_supported(const Ctx* c, int window, int* smem_bytes, int* k_tab = nullptr);
// `max_rounds` iterations of Algorithm 1's while loop for every chain (to the end of the grid if large), one launch
asd_status launch_resident(Ctx* c, int window, bool use_u, int max_rounds);

}  // namespace asd

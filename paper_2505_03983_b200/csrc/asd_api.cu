// C ABI of the ASD library: context life cycle, table construction, the host side of the round
// driver (Algorithm 1's while loop), the sequential sampler (Eq. 7) and the diagnostics.
#include <math.h>
#include <stdlib.h>
#include <stdio.h>
#include <string.h>

#include <algorithm>
#include <new>

#include "asd_internal.h"

using namespace asd;

struct asd_ctx {
  Ctx c;
};

namespace {

thread_local std::string g_create_error;

asd_status fail(Ctx* c, asd_status st, const std::string& msg) {
  if (c) c->err = msg;
  return st;
}

#define ASD_CUDA(c, expr)                                                                   \
  do {                                                                                      \
    cudaError_t e__ = (expr);                                                               \
    if (e__ != cudaSuccess)                                                                 \
      return fail((c), e__ == cudaErrorMemoryAllocation ? ASD_ERR_OOM : ASD_ERR_CUDA,       \
                  std::string(#expr) + ": " + cudaGetErrorString(e__));                     \
  } while (0)

template <typename T>
asd_status dev_alloc(Ctx* c, T** out, size_t count, bool zero = true) {
  void* p = nullptr;
  const size_t bytes = std::max<size_t>(count, 1) * sizeof(T);
  // host-side failure injection for the tests of the error path (ASD_FAIL_ALLOC_AFTER=n at asd_create)
  if (c->fail_alloc_after >= 0 && (int)c->dev_allocs.size() >= c->fail_alloc_after)
    return fail(c, ASD_ERR_OOM, "cudaMalloc: injected allocation failure");
  cudaError_t e = cudaMalloc(&p, bytes);
  if (e != cudaSuccess) return fail(c, ASD_ERR_OOM, std::string("cudaMalloc: ") + cudaGetErrorString(e));
  c->dev_allocs.push_back(p);
  if (zero) {
    e = cudaMemsetAsync(p, 0, bytes, c->stream);
    if (e != cudaSuccess) return fail(c, ASD_ERR_CUDA, std::string("cudaMemset: ") + cudaGetErrorString(e));
  }
  *out = static_cast<T*>(p);
  return ASD_OK;
}

// A table or parameter array that is written in full: no clearing, and the copy goes to the context's
// stream like everything else the library enqueues (the stream may be a non-blocking one, which the
// legacy default stream does not order against); the host vector may die right after the call.
template <typename T>
asd_status dev_upload(Ctx* c, const T** out, const std::vector<T>& host) {
  T* p = nullptr;
  asd_status st = dev_alloc(c, &p, host.size(), host.empty());
  if (st != ASD_OK) return st;
  if (!host.empty()) {
    ASD_CUDA(c, cudaMemcpyAsync(p, host.data(), host.size() * sizeof(T), cudaMemcpyHostToDevice, c->stream));
    ASD_CUDA(c, cudaStreamSynchronize(c->stream));
  }
  *out = p;
  return ASD_OK;
}

asd_status check_device_error(Ctx* c) {
  // counters_host must have been refreshed and the stream synchronised by the caller
  if (c->counters_host->err != 0) {
    const int code = c->counters_host->err;
    cudaMemsetAsync(&c->counters->err, 0, sizeof(int), c->stream);
    return fail(c, (asd_status)code, "a bounded device-side wait ran out (kernel returned early)");
  }
  return ASD_OK;
}

asd_status sync_counters(Ctx* c) {
  ASD_CUDA(c, cudaMemcpyAsync(c->counters_host, c->counters, sizeof(RoundCounters), cudaMemcpyDeviceToHost, c->stream));
  ASD_CUDA(c, cudaStreamSynchronize(c->stream));
  prof_collect(c);
  return check_device_error(c);
}

// One iteration of Algorithm 1's while loop for all active chains (window = 1, use_u = false is
// one step of Eq. 7).  active_bound: host-side upper bound on the number of active chains.
asd_status enqueue_round(Ctx* c, int window, bool use_u, int active_bound) {
  if (active_bound <= 0) return ASD_OK;
  {
    ProfScope ps(c, PH_PREP);
    launch_prep(c, whole_batch(c), window);
  }
  // look-ahead: the first model call covers only the chains without a saved drift, and every chain may
  // draft one more row (the point the next round would start from)
  const bool la = c->lookahead;
  RowSet rs1{la ? &c->counters->n_eval : &c->counters->n_active, active_bound, c->y, la ? c->act1 : c->act,
             la ? c->step1e : c->step1, la ? c->act1 : c->act, true};
  RowSet rs2{&c->counters->rows2, active_bound * (la ? window : window - 1), c->Yhat, nullptr, c->row_step, c->row_slot,
             true};  // both counts come from the prep kernel; a pack or draft kernel runs in between
  asd_status st = ASD_OK;
  switch (c->kind) {
    case ASD_DEN_GMM_ISO:
    case ASD_DEN_GAUSS_LINEAR: {
      const bool gmm = c->kind == ASD_DEN_GMM_ISO;
      {
        ProfScope ps(c, PH_D1_ANALYTIC);
        gmm ? launch_gmm(c, rs1, c->v) : launch_gauss(c, rs1, c->v);
      }
      {
        ProfScope ps(c, PH_DRAFT);
        launch_draft(c, whole_batch(c), window, c->v, nullptr);
      }
      {
        ProfScope ps(c, PH_D2_ANALYTIC);
        gmm ? launch_gmm(c, rs2, c->G) : launch_gauss(c, rs2, c->G);
      }
      break;
    }
    default: {
      {
        ProfScope ps(c, PH_PACK);
        launch_pack(c, rs1);
      }
      st = mlp_forward(c, rs1, c->v, 0);
      if (st != ASD_OK) return st;
      {
        ProfScope ps(c, PH_DRAFT);
        launch_draft(c, whole_batch(c), window, c->v, nullptr);
      }
      st = mlp_forward(c, rs2, c->G, 1);
      if (st != ASD_OK) return st;
      break;
    }
  }
  {
    ProfScope ps(c, PH_VERIFY);
    launch_verify(c, whole_batch(c), window, use_u, c->G, c->v, nullptr);
  }
  ASD_CUDA(c, cudaGetLastError());
  return ASD_OK;
}

// The bound on the number of active chains that a captured round is built for: the full batch, or the
// next power of two (so a run needs about log2(n) graphs).
int bound_bucket(const Ctx* c, int active) {
  if (active >= c->n) return c->n;
  int b = 1;
  while (b < active) b <<= 1;
  return std::min(b, c->n);
}

// Enqueues one round on c->stream (which must be the context's private stream): replays the captured
// graph for this shape, capturing it on first use.
template <typename Body>
asd_status launch_captured(Ctx* c, const std::tuple<int, int, long long>& key, Body body) {
  auto it = c->graphs.find(key);
  if (it == c->graphs.end()) {
    const long long l0 = c->launches;
    ASD_CUDA(c, cudaStreamBeginCapture(c->stream, cudaStreamCaptureModeThreadLocal));
    const asd_status st = body();
    cudaGraph_t graph = nullptr;
    const cudaError_t e = cudaStreamEndCapture(c->stream, &graph);
    const long long captured = c->launches - l0;
    c->launches = l0;
    if (st != ASD_OK) {
      if (graph) cudaGraphDestroy(graph);
      return st;
    }
    if (e != cudaSuccess || !graph) return fail(c, ASD_ERR_CUDA, std::string("stream capture failed: ") + cudaGetErrorString(e));
    cudaGraphExec_t exec = nullptr;
    const cudaError_t e2 = cudaGraphInstantiate(&exec, graph, 0);
    cudaGraphDestroy(graph);
    if (e2 != cudaSuccess) return fail(c, ASD_ERR_CUDA, std::string("cudaGraphInstantiate: ") + cudaGetErrorString(e2));
    it = c->graphs.emplace(key, Ctx::RoundGraph{exec, captured}).first;
  }
  ASD_CUDA(c, cudaGraphLaunch(it->second.exec, c->stream));
  c->launches += it->second.launches;
  return ASD_OK;
}

// `group` consecutive rounds in one graph: for the launch-bound workloads the graph launch itself is a
// visible part of a round.
asd_status launch_round_graph(Ctx* c, int window, bool use_u, int active, int group) {
  if (active <= 0) return ASD_OK;
  const int bucket = bound_bucket(c, active);
  return launch_captured(c, std::make_tuple(window, (use_u ? 1 : 0) + 16 * group, (long long)bucket), [&] {
    for (int r = 0; r < group; ++r) {
      const asd_status st = enqueue_round(c, window, use_u, bucket);
      if (st != ASD_OK) return st;
    }
    return ASD_OK;
  });
}

// One tick of the staggered schedule (network denoiser).  The batch is split into two lanes that run
// Algorithm 1's round half a round apart: in tick t lane Y = t mod 2 is at its first model call (drift
// at the current points) and lane X = the other one at its second (drift at its drafted points), and both
// go through ONE pass of the GEMM chain: Y's current points are appended as rows behind X's drafted
// rows.  Then X is verified and advanced, and Y drafts its window from the drifts it just received.  Per
// chain nothing changes (same rounds, same arithmetic); the pass with very few rows disappears.
// The drift buffer alternates between ticks because X's v_a rows, produced a tick earlier, are still
// needed by its verify step.
asd_status enqueue_tick(Ctx* c, long long t, int window, int bound_x, int bound_y) {
  Lane& Y = c->lanes[t & 1];
  Lane& X = c->lanes[(t + 1) & 1];
  float* g_cur = (t & 1) ? c->G2 : c->G;
  const float* g_prev = (t & 1) ? c->G : c->G2;
  {
    ProfScope ps(c, PH_PREP);
    launch_prep(c, Y, window);
  }
  {
    ProfScope ps(c, PH_PACK);
    launch_pack_appended(c, Y, &X.counters->rows2, c->merged_rows);
  }
  RowSet rs{c->merged_rows, bound_x * (window - 1) + bound_y, c->Yhat, nullptr, c->row_step, c->row_slot};
  asd_status st = mlp_forward(c, rs, g_cur, 1);
  if (st != ASD_OK) return st;
  {
    ProfScope ps(c, PH_VERIFY);
    launch_verify(c, X, window, true, g_cur, g_prev, X.v_off);
  }
  {
    ProfScope ps(c, PH_DRAFT);
    launch_draft(c, Y, window, g_cur, Y.v_off);
  }
  ASD_CUDA(c, cudaGetLastError());
  return ASD_OK;
}

int lane_bucket(int active, int n) {
  if (active >= n) return n;
  int b = 1;
  while (b < active) b <<= 1;
  return std::min(b, n);
}

asd_status launch_tick(Ctx* c, bool graphs, long long t, int window, int act_x, int act_y) {
  const Lane& Y = c->lanes[t & 1];
  const Lane& X = c->lanes[(t + 1) & 1];
  const int bx = lane_bucket(act_x, X.n), by = lane_bucket(act_y, Y.n);
  if (!graphs) return enqueue_tick(c, t, window, bx, by);
  return launch_captured(c, std::make_tuple(window, 2 + (int)(t & 1), (long long)bx * (1ll << 32) + by),
                         [&] { return enqueue_tick(c, t, window, bx, by); });
}

// While alive, the context's work goes to its private stream, ordered after what the caller's stream
// held at construction; the destructor orders the caller's stream after it again.
struct PrivateStreamScope {
  Ctx* c;
  cudaStream_t user;
  bool on;
  explicit PrivateStreamScope(Ctx* c_) : c(c_), user(c_->stream), on(false) {
    if (!c->use_graphs || c->prof_on || !c->gstream) return;
    if (cudaEventRecord(c->fork_ev, user) != cudaSuccess || cudaStreamWaitEvent(c->gstream, c->fork_ev, 0) != cudaSuccess)
      return;
    c->stream = c->gstream;
    on = true;
  }
  ~PrivateStreamScope() {
    if (!on) return;
    c->stream = user;
    cudaEventRecord(c->join_ev, c->gstream);
    cudaStreamWaitEvent(user, c->join_ev, 0);
  }
};

constexpr int kRoundsPerGraph = 4;

// `group` rounds: one graph replay, or the kernels themselves
asd_status enqueue_rounds(Ctx* c, bool graphs, int window, bool use_u, int active, int group) {
  if (graphs) return launch_round_graph(c, window, use_u, active, group);
  for (int r = 0; r < group; ++r) {
    const asd_status st = enqueue_round(c, window, use_u, active);
    if (st != ASD_OK) return st;
  }
  return ASD_OK;
}

// Whether asd_sample runs the batch as two staggered lanes (network denoiser only).  Off unless
// ASD_STAGGER=1: measured on B200 it does not pay - at 512 x 64 and 2048 x 64 chains x window the pass with
// few rows that it removes (6 % and 3 % of the step) is offset by the less efficient half-size GEMM launches
// and the doubled draft / verify launches (936 against 920 ms and 3583 against 3545 ms per step); the
// run is bound by the power cap, so what counts is energy per FLOP, not idle gaps.
bool use_stagger(const Ctx* c) {
  if (c->kind != ASD_DEN_RESMLP_BF16 || !c->G2 || c->window < 4 || c->n < 2 || c->lookahead) return false;
  return c->stagger;
}

// asd_sample for two staggered lanes: same run-ahead scheme as below, one ring slot per tick holding both
// lanes' counters and the merged row count.
asd_status sample_staggered(Ctx* c) {
  constexpr int kDepth = 4;
  constexpr size_t kEventsPerTick = 2 * PH_COUNT + 8;
  int active[2] = {c->lanes[0].n, c->lanes[1].n};
  long long issued = 0, consumed = 0;
  const long long max_ticks = 2ll * c->K + 6;
  size_t prof_pairs[Ctx::kRing] = {};
  asd_status deferred = ASD_OK;
  PrivateStreamScope pss(c);
  auto consume = [&](bool wait) -> bool {
    const int slot = (int)(consumed % Ctx::kRing);
    if (wait) {
      if (cudaEventSynchronize(c->ring_ev[slot]) != cudaSuccess) {
        deferred = fail(c, ASD_ERR_CUDA, "event synchronisation failed");
        return false;
      }
    } else if (cudaEventQuery(c->ring_ev[slot]) != cudaSuccess) {
      return false;
    }
    const long long t = consumed;
    const RoundCounters& hy = c->ring_host[3 * slot + (t & 1)];        // lane at its first model call
    const RoundCounters& hx = c->ring_host[3 * slot + ((t + 1) & 1)];  // lane that was verified
    const int merged = c->ring_host[3 * slot + 2].n_active;
    if (t >= 1) active[(t + 1) & 1] = hx.n_active_after;  // tick 0 verifies nothing
    if (c->prof_on) {
      prof_collect_some(c, (long long)prof_pairs[slot]);
      for (int ph : {PH_PREP, PH_PACK, PH_DRAFT}) c->prof[ph].rows += hy.n_active;
      c->prof[PH_VERIFY].rows += hx.n_active;
      for (int ph : {PH_D2_IN, PH_D2_HID, PH_D2_OUT}) c->prof[ph].rows += merged;
    }
    ++consumed;
    return true;
  };
  while ((active[0] > 0 || active[1] > 0) && issued < max_ticks && deferred == ASD_OK) {
    const long long t = issued;
    const int slot = (int)(t % Ctx::kRing);
    c->ev_used = (size_t)slot * kEventsPerTick;
    const size_t pending0 = c->pending.size();
    asd_status st = launch_tick(c, pss.on, t, c->window, active[(t + 1) & 1], active[t & 1]);
    if (st != ASD_OK) return st;
    prof_pairs[slot] = c->pending.size() - pending0;
    for (int l = 0; l < 2; ++l)
      ASD_CUDA(c, cudaMemcpyAsync(&c->ring_host[3 * slot + l], c->lanes[l].counters, sizeof(RoundCounters),
                                  cudaMemcpyDeviceToHost, c->stream));
    ASD_CUDA(c, cudaMemcpyAsync(&c->ring_host[3 * slot + 2].n_active, c->merged_rows, sizeof(int), cudaMemcpyDeviceToHost,
                                c->stream));
    ASD_CUDA(c, cudaEventRecord(c->ring_ev[slot], c->stream));
    ++issued;
    while (consumed < issued && consume(issued - consumed >= kDepth)) {
    }
  }
  while (consumed < issued && deferred == ASD_OK && consume(true)) {
  }
  if (deferred != ASD_OK) {
    cudaStreamSynchronize(c->stream);
    prof_collect(c);
    return deferred;
  }
  if (active[0] > 0 || active[1] > 0) return fail(c, ASD_ERR_STATE, "chains still active after 2K ticks");
  // the lanes' running totals (the last ring slot holds their final counters)
  if (issued > 0) {
    const int slot = (int)((issued - 1) % Ctx::kRing);
    for (int l = 0; l < 2; ++l) {
      c->extra_rows_total += (long long)c->ring_host[3 * slot + l].rows_total;
      c->extra_rows_verified += (long long)c->ring_host[3 * slot + l].rows_verified;
    }
  }
  return ASD_OK;
}

}  // namespace

namespace asd {
ProfScope::ProfScope(Ctx* c_, int phase_) : c(c_ && c_->prof_on ? c_ : nullptr), phase(phase_), l0(0), e0(0) {
  if (!c) return;
  while (c->ev_used + 2 > c->ev_pool.size()) {
    for (int i = 0; i < 64; ++i) {
      cudaEvent_t e;
      if (cudaEventCreate(&e) != cudaSuccess) {
        c = nullptr;
        return;
      }
      c->ev_pool.push_back(e);
    }
  }
  l0 = c->launches;
  e0 = c->ev_used;
  c->ev_used += 2;
  cudaEventRecord(c->ev_pool[e0], c->stream);
}
ProfScope::~ProfScope() {
  if (!c) return;
  cudaEventRecord(c->ev_pool[e0 + 1], c->stream);
  c->pending.push_back({phase, e0, e0 + 1, (int)(c->launches - l0)});
  c = nullptr;
}
// Folds the first `count` pending event pairs (all of them if count < 0) into c->prof; their events
// must have completed.
void prof_collect_some(Ctx* c, long long count) {
  const size_t n = count < 0 ? c->pending.size() : std::min<size_t>((size_t)count, c->pending.size());
  for (size_t i = 0; i < n; ++i) {
    const auto& p = c->pending[i];
    if (p.launches == 0) continue;
    float ms = 0.f;
    if (cudaEventElapsedTime(&ms, c->ev_pool[p.e0], c->ev_pool[p.e1]) == cudaSuccess) {
      c->prof[p.phase].ms += ms;
      c->prof[p.phase].launches += p.launches;
    }
  }
  c->pending.erase(c->pending.begin(), c->pending.begin() + n);
}
void prof_collect(Ctx* c) {
  if (!c->prof_on && c->pending.empty()) return;
  prof_collect_some(c, -1);
  c->ev_used = 0;
}
}  // namespace asd

namespace {

struct HostTables {
  std::vector<float> eta, sig, c1, c2, tt;
};

uint16_t bf16_bits_host(float f) {
  uint32_t u;
  memcpy(&u, &f, 4);
  const uint32_t lsb = (u >> 16) & 1u;
  u += 0x7FFFu + lsb;
  return (uint16_t)(u >> 16);
}

}  // namespace

extern "C" {

const char* asd_version(void) { return "asd-b200 0.1 (sm_100a)"; }

const char* asd_last_error(const asd_ctx* ctx) {
  if (!ctx) return g_create_error.c_str();
  return ctx->c.err.c_str();
}

void asd_destroy(asd_ctx* ctx) {
  if (!ctx) return;
  Ctx* c = &ctx->c;
  cudaStreamSynchronize(c->stream);
  for (void* p : c->dev_allocs) cudaFree(p);
  if (c->counters_host) cudaFreeHost(c->counters_host);
  if (c->ring_host) cudaFreeHost(c->ring_host);
  for (auto& kv : c->graphs) cudaGraphExecDestroy(kv.second.exec);
  if (c->gstream) {
    cudaStreamSynchronize(c->gstream);
    cudaStreamDestroy(c->gstream);
  }
  if (c->fork_ev) cudaEventDestroy(c->fork_ev);
  if (c->join_ev) cudaEventDestroy(c->join_ev);
  for (cudaEvent_t e : c->ring_ev)
    if (e) cudaEventDestroy(e);
  if (c->ev0) cudaEventDestroy(c->ev0);
  if (c->ev1) cudaEventDestroy(c->ev1);
  for (cudaEvent_t e : c->ev_pool) cudaEventDestroy(e);
  delete ctx;
}

asd_status asd_create(const asd_config* cfg, void* cuda_stream, asd_ctx** out) {
  g_create_error.clear();
  auto bad = [&](asd_status st, const char* msg) {
    g_create_error = msg;
    return st;
  };
  if (!cfg || !out) return bad(ASD_ERR_INVALID_ARG, "cfg and out must not be NULL");
  *out = nullptr;
  if (cfg->d < 1 || cfg->d > 65536) return bad(ASD_ERR_INVALID_ARG, "d must be in 1..65536");
  if (cfg->K < 1) return bad(ASD_ERR_INVALID_ARG, "K must be >= 1");
  if (cfg->window < 1) return bad(ASD_ERR_INVALID_ARG, "window must be >= 1");
  if (cfg->max_chains < 1) return bad(ASD_ERR_INVALID_ARG, "max_chains must be >= 1");
  if (cfg->flags & ~(ASD_FLAG_DEBUG_ALL_SLOTS | ASD_FLAG_ADAPTIVE_WINDOW | ASD_FLAG_LOOKAHEAD | ASD_FLAG_TRAJECTORY |
                     ASD_FLAG_DEBUG_DUMP))
    return bad(ASD_ERR_INVALID_ARG, "unknown flag");
  if (!cfg->t) return bad(ASD_ERR_INVALID_ARG, "t must not be NULL");
  if (!(cfg->t[0] >= 0.0)) return bad(ASD_ERR_INVALID_ARG, "t[0] must be >= 0");
  for (int i = 0; i < cfg->K; ++i) {
    if (!(cfg->t[i + 1] > cfg->t[i]) || !isfinite(cfg->t[i + 1]))
      return bad(ASD_ERR_INVALID_ARG, "t must be finite and strictly increasing");
    if (cfg->sigma2 && !(cfg->sigma2[i] > 0.0 && isfinite(cfg->sigma2[i])))
      return bad(ASD_ERR_INVALID_ARG, "sigma2 must be finite and positive");
  }
  const bool lookahead = (cfg->flags & ASD_FLAG_LOOKAHEAD) != 0;
  const int window_eff = std::min(cfg->window, cfg->K);  // a window beyond the grid acts like K (theta = infinity)
  const long long max_rows_ll = (long long)cfg->max_chains * (lookahead ? window_eff : std::max(window_eff - 1, 1));
  if (max_rows_ll > (1ll << 30) || max_rows_ll * cfg->d > (1ll << 40))
    return bad(ASD_ERR_INVALID_ARG, "max_chains * window * d too large");
  if ((cfg->flags & ASD_FLAG_TRAJECTORY) && (long long)cfg->max_chains * (cfg->K + 1ll) * cfg->d > (1ll << 36))
    return bad(ASD_ERR_INVALID_ARG, "trajectory buffer (max_chains * (K + 1) * d floats) too large");
  const asd_denoiser& D = cfg->den;
  switch (D.kind) {
    case ASD_DEN_GMM_ISO:
      if (D.n_comp < 1 || D.n_comp > 256 || !D.means || !D.weights || !(D.sigma > 0.f))
        return bad(ASD_ERR_INVALID_ARG, "GMM: need 1..256 components, means, weights, sigma > 0");
      for (int j = 0; j < D.n_comp; ++j)
        if (!(D.weights[j] > 0.f)) return bad(ASD_ERR_INVALID_ARG, "GMM: weights must be positive");
      break;
    case ASD_DEN_GAUSS_LINEAR:
      if (!D.mu0 || !D.Q || !D.lam) return bad(ASD_ERR_INVALID_ARG, "Gaussian: mu0, Q, lam required");
      if (cfg->d > 4096) return bad(ASD_ERR_UNSUPPORTED, "Gaussian posterior mean supports d <= 4096");
      for (int j = 0; j < cfg->d; ++j)
        if (!(D.lam[j] >= 0.f)) return bad(ASD_ERR_INVALID_ARG, "Gaussian: eigenvalues must be >= 0");
      break;
    case ASD_DEN_RESMLP_BF16:
      if (D.width < 8 || D.width % 8 || D.n_layers < 0 || D.d_cond < 0 || D.d_temb < 0 || D.d_temb % 2)
        return bad(ASD_ERR_INVALID_ARG, "MLP: width must be a positive multiple of 8, d_temb even, sizes >= 0");
      if (!D.W_in || !D.W_out || !D.b_in || !D.b_out || (D.n_layers > 0 && (!D.W_hid || !D.b_hid)))
        return bad(ASD_ERR_INVALID_ARG, "MLP: weight and bias pointers required");
      break;
    default:
      return bad(ASD_ERR_INVALID_ARG, "unknown denoiser kind");
  }
  int ndev = 0;
  if (cudaGetDeviceCount(&ndev) != cudaSuccess || ndev < 1) return bad(ASD_ERR_CUDA, "no CUDA device");

  asd_ctx* ctx = new (std::nothrow) asd_ctx();
  if (!ctx) return bad(ASD_ERR_OOM, "host allocation failed");
  Ctx* c = &ctx->c;
  auto abandon = [&](asd_status st) {
    g_create_error = c->err;
    asd_destroy(ctx);
    return st;
  };
  c->d = cfg->d;
  c->K = cfg->K;
  c->window = std::min(cfg->window, cfg->K);
  c->max_chains = cfg->max_chains;
  c->kind = D.kind;
  c->seed = cfg->seed;
  c->debug_all_slots = (cfg->flags & ASD_FLAG_DEBUG_ALL_SLOTS) != 0;
  c->adaptive = (cfg->flags & ASD_FLAG_ADAPTIVE_WINDOW) != 0;
  c->stream = static_cast<cudaStream_t>(cuda_stream);
  c->lookahead = lookahead;
  c->max_rows = (int)((long long)cfg->max_chains * (lookahead ? c->window : std::max(c->window - 1, 1)));
  cudaGetDevice(&c->device);
  cudaDeviceProp prop;
  if (cudaGetDeviceProperties(&prop, c->device) != cudaSuccess) return abandon(fail(c, ASD_ERR_CUDA, "device query failed"));
  c->num_sms = prop.multiProcessorCount;
  if (D.kind == ASD_DEN_RESMLP_BF16 && prop.major != 10)
    return abandon(fail(c, ASD_ERR_UNSUPPORTED, "the bf16 network denoiser needs an sm_100 device (tcgen05 / TMEM)"));
  if (cudaEventCreate(&c->ev0) != cudaSuccess || cudaEventCreate(&c->ev1) != cudaSuccess)
    return abandon(fail(c, ASD_ERR_CUDA, "event creation failed"));
  if (cudaMallocHost(&c->counters_host, sizeof(RoundCounters)) != cudaSuccess)
    return abandon(fail(c, ASD_ERR_OOM, "pinned allocation failed"));
  memset(c->counters_host, 0, sizeof(RoundCounters));
  {
    const char* e = getenv("ASD_GRAPHS");  // "0" launches every kernel of a round separately
    c->use_graphs = !(e && e[0] == '0');
    const char* gm = getenv("ASD_GEMM_MODE");  // tuning aid: pins the GEMM kernel family
    c->gemm_mode = !gm ? 0 : (!strcmp(gm, "cta") ? 1 : (!strcmp(gm, "pair") ? 2 : 0));
    const char* fm = getenv("ASD_MLP_FUSED");  // "1": the whole network as one launch (measured slower; see asd_gemm.cu)
    c->fused_mode = (fm && fm[0] == '1') ? 1 : 0;
    const char* sg = getenv("ASD_STAGGER");
    c->stagger = sg && sg[0] == '1';
    const char* fa = getenv("ASD_FAIL_ALLOC_AFTER");  // test hook: the n-th device allocation of this context fails
    c->fail_alloc_after = fa ? atoi(fa) : -1;
    const char* vh = getenv("ASD_VERIFY_HORIZON");  // tuning aid: slots verified for all chains at once (default: per launch)
    c->verify_horizon = vh ? atoi(vh) : -1;
    const char* rm = getenv("ASD_RESIDENT");  // tuning aid: "0" keeps the closed-form drifts on the per-phase kernels
    c->resident_mode = !rm ? 1 : (rm[0] == '0' ? 0 : (rm[0] == '2' ? 2 : 1));
    if (cudaStreamCreateWithFlags(&c->gstream, cudaStreamNonBlocking) != cudaSuccess ||
        cudaEventCreateWithFlags(&c->fork_ev, cudaEventDisableTiming) != cudaSuccess ||
        cudaEventCreateWithFlags(&c->join_ev, cudaEventDisableTiming) != cudaSuccess)
      return abandon(fail(c, ASD_ERR_CUDA, "stream / event creation failed"));
  }
  if (cudaMallocHost(&c->ring_host, 3 * Ctx::kRing * sizeof(RoundCounters)) != cudaSuccess)
    return abandon(fail(c, ASD_ERR_OOM, "pinned allocation failed"));
  memset(c->ring_host, 0, 3 * Ctx::kRing * sizeof(RoundCounters));
  for (int i = 0; i < Ctx::kRing; ++i)
    if (cudaEventCreateWithFlags(&c->ring_ev[i], cudaEventDisableTiming) != cudaSuccess)
      return abandon(fail(c, ASD_ERR_CUDA, "event creation failed"));

  // ---- per-step tables: fp64 on the host, stored as fp32 -----------------------------------
  const int K = c->K;
  HostTables T;
  T.eta.resize(K);
  T.sig.resize(K);
  T.c1.resize(K);
  T.c2.resize(K);
  T.tt.resize(K + 1);
  for (int i = 0; i <= K; ++i) T.tt[i] = (float)cfg->t[i];
  for (int i = 0; i < K; ++i) {
    const double eta = cfg->t[i + 1] - cfg->t[i];
    const double s2 = cfg->sigma2 ? cfg->sigma2[i] : eta;
    const double sig = sqrt(s2);
    T.eta[i] = (float)eta;
    T.sig[i] = (float)sig;
    T.c1[i] = (float)(eta / sig);
    T.c2[i] = (float)(eta * eta / (2.0 * s2));
  }
  asd_status st;
#define TRY(x)                          \
  do {                                  \
    st = (x);                           \
    if (st != ASD_OK) return abandon(st); \
  } while (0)
  TRY(dev_upload(c, &c->tab.eta, T.eta));
  TRY(dev_upload(c, &c->tab.sig, T.sig));
  TRY(dev_upload(c, &c->tab.c1, T.c1));
  TRY(dev_upload(c, &c->tab.c2, T.c2));
  TRY(dev_upload(c, &c->tab.tt, T.tt));

  // ---- state and workspaces --------------------------------------------------------------------
  const size_t n = c->max_chains, d = c->d, R = c->max_rows;
  TRY(dev_alloc(c, &c->y, n * d));
  TRY(dev_alloc(c, &c->a, n));
  TRY(dev_alloc(c, &c->rounds, n));
  TRY(dev_alloc(c, &c->wnd, n));
  TRY(dev_alloc(c, &c->ema8, n));
  TRY(dev_alloc(c, &c->act, n));
  TRY(dev_alloc(c, &c->row_off, n + 1));
  TRY(dev_alloc(c, &c->step1, n));
  TRY(dev_alloc(c, &c->row_step, R));
  TRY(dev_alloc(c, &c->row_slot, R));
  TRY(dev_alloc(c, &c->v, n * d));
  TRY(dev_alloc(c, &c->Yhat, R * d));
  TRY(dev_alloc(c, &c->G, R * d));
  if (cfg->flags & (ASD_FLAG_DEBUG_DUMP | ASD_FLAG_DEBUG_ALL_SLOTS)) {
    TRY(dev_alloc(c, &c->dbg_lr, n * c->window));
    TRY(dev_alloc(c, &c->dbg_lu, n * c->window));
  }
  TRY(dev_alloc(c, &c->acc_len, n));
  TRY(dev_alloc(c, &c->slot_dot, n * c->window));
  TRY(dev_alloc(c, &c->slot_nrm, n * c->window));
  TRY(dev_alloc(c, &c->slot_lu, n * c->window));
  TRY(dev_alloc(c, &c->first_rej, n));
  TRY(dev_alloc(c, &c->hist, (size_t)c->window + 1));
  if (cfg->flags & ASD_FLAG_TRAJECTORY) TRY(dev_alloc(c, &c->traj, n * ((size_t)K + 1) * d));
  if (c->lookahead) {
    TRY(dev_alloc(c, &c->has_v, n));
    TRY(dev_alloc(c, &c->vsave, n * d));
    TRY(dev_alloc(c, &c->act1, n));
    TRY(dev_alloc(c, &c->step1e, n));
    TRY(dev_alloc(c, &c->idx1, n));
  }
  TRY(dev_alloc(c, &c->counters, 2));  // [0] round counters, [1].n_active doubles as a row-count scratch

  // ---- denoiser parameters ---------------------------------------------------------------------
  if (D.kind == ASD_DEN_GMM_ISO) {
    std::vector<float> means(D.means, D.means + (size_t)D.n_comp * d), log_pi(D.n_comp), cnorm(D.n_comp);
    double wsum = 0;
    for (int j = 0; j < D.n_comp; ++j) wsum += D.weights[j];
    for (int j = 0; j < D.n_comp; ++j) {
      log_pi[j] = (float)log((double)D.weights[j] / wsum);
      double s = 0;
      for (size_t k = 0; k < d; ++k) s += (double)means[j * d + k] * means[j * d + k];
      cnorm[j] = (float)s;
    }
    c->gmm.n_comp = D.n_comp;
    c->gmm.s2 = (float)((double)D.sigma * (double)D.sigma);
    TRY(dev_upload(c, &c->gmm.means, means));
    TRY(dev_upload(c, &c->gmm.log_pi, log_pi));
    TRY(dev_upload(c, &c->gmm.cnorm, cnorm));
  } else if (D.kind == ASD_DEN_GAUSS_LINEAR) {
    std::vector<float> Q(D.Q, D.Q + d * d), Qt(d * d), qmu(d), lam(D.lam, D.lam + d);
    for (size_t i = 0; i < d; ++i)
      for (size_t j = 0; j < d; ++j) Qt[j * d + i] = Q[i * d + j];
    for (size_t j = 0; j < d; ++j) {
      double s = 0;
      for (size_t i = 0; i < d; ++i) s += (double)Q[i * d + j] * D.mu0[i];
      qmu[j] = (float)s;
    }
    TRY(dev_upload(c, &c->gauss.Q, Q));
    TRY(dev_upload(c, &c->gauss.Qt, Qt));
    TRY(dev_upload(c, &c->gauss.qmu, qmu));
    TRY(dev_upload(c, &c->gauss.lam, lam));
  } else {
    MlpParams& M = c->mlp;
    M.d_cond = D.d_cond;
    M.d_temb = D.d_temb;
    M.width = D.width;
    M.n_layers = D.n_layers;
    M.in_dim = (int)d + D.d_cond + D.d_temb;
    M.in_pad = (M.in_dim + 63) / 64 * 64;
    M.row_cap = (int)std::max(R, n);
    const size_t W = D.width;
    std::vector<uint16_t> w_in((size_t)W * M.in_pad, 0);
    for (size_t o = 0; o < W; ++o) memcpy(&w_in[o * M.in_pad], D.W_in + o * M.in_dim, (size_t)M.in_dim * 2);
    std::vector<uint16_t> w_hid(D.W_hid ? D.W_hid : nullptr, D.W_hid ? D.W_hid + (size_t)D.n_layers * W * W : nullptr);
    std::vector<uint16_t> w_out(D.W_out, D.W_out + d * W);
    std::vector<float> b_in(D.b_in, D.b_in + W), b_out(D.b_out, D.b_out + d);
    std::vector<float> b_hid(D.b_hid ? D.b_hid : nullptr, D.b_hid ? D.b_hid + (size_t)D.n_layers * W : nullptr);
    std::vector<float> c_in(K, 1.f), c_skip(K, 0.f), c_out(K, 1.f);
    if (D.c_in) c_in.assign(D.c_in, D.c_in + K);
    if (D.c_skip) c_skip.assign(D.c_skip, D.c_skip + K);
    if (D.c_out) c_out.assign(D.c_out, D.c_out + K);
    std::vector<uint16_t> temb((size_t)K * D.d_temb);
    const int half = D.d_temb / 2;
    for (int i = 0; i < K; ++i) {
      const double tau = 1000.0 * i / K;
      for (int f = 0; f < half; ++f) {
        const double w = exp(-log(1.0e4) * f / half);
        temb[(size_t)i * D.d_temb + f] = bf16_bits_host((float)sin(tau * w));
        temb[(size_t)i * D.d_temb + half + f] = bf16_bits_host((float)cos(tau * w));
      }
    }
    TRY(dev_upload(c, reinterpret_cast<const uint16_t**>(&M.W_in), w_in));
    TRY(dev_upload(c, reinterpret_cast<const uint16_t**>(&M.W_hid), w_hid));
    TRY(dev_upload(c, reinterpret_cast<const uint16_t**>(&M.W_out), w_out));
    TRY(dev_upload(c, &M.b_in, b_in));
    TRY(dev_upload(c, &M.b_hid, b_hid));
    TRY(dev_upload(c, &M.b_out, b_out));
    TRY(dev_upload(c, &c->tab.c_in, c_in));
    TRY(dev_upload(c, &c->tab.c_skip, c_skip));
    TRY(dev_upload(c, &c->tab.c_out, c_out));
    TRY(dev_upload(c, reinterpret_cast<const uint16_t**>(&M.temb), temb));
    __nv_bfloat16* p = nullptr;
    TRY(dev_alloc(c, &p, n * (size_t)D.d_cond));
    M.cond = p;
    TRY(dev_alloc(c, &M.X, (size_t)M.row_cap * M.in_pad));
    TRY(dev_alloc(c, &M.H[0], (size_t)M.row_cap * W));
    TRY(dev_alloc(c, &M.H[1], (size_t)M.row_cap * W));
    if (c->stagger) TRY(dev_alloc(c, &c->G2, R * d));  // the staggered schedule alternates two drift buffers
    TRY(dev_alloc(c, &c->merged_rows, 4));
    for (int l = 0; l < 2 && c->stagger; ++l) {
      TRY(dev_alloc(c, &c->lanes[l].act, n));
      TRY(dev_alloc(c, &c->lanes[l].row_off, n + 1));
      TRY(dev_alloc(c, &c->lanes[l].step1, n));
      TRY(dev_alloc(c, &c->lanes[l].counters, 1));
      TRY(dev_alloc(c, &c->lanes[l].v_off, 4));
    }
  }
#undef TRY
  if (cudaStreamSynchronize(c->stream) != cudaSuccess) return abandon(fail(c, ASD_ERR_CUDA, "create: sync failed"));
  *out = ctx;
  return ASD_OK;
}

asd_status asd_reset(asd_ctx* ctx, int32_t n_chains, uint64_t chain_id_base, const float* y0_dev,
                     const float* cond_dev) {
  if (!ctx) return ASD_ERR_INVALID_ARG;
  Ctx* c = &ctx->c;
  if (n_chains < 0 || n_chains > c->max_chains) return fail(c, ASD_ERR_INVALID_ARG, "n_chains out of range");
  if (chain_id_base + (uint64_t)n_chains > (1ull << 32)) return fail(c, ASD_ERR_INVALID_ARG, "chain ids must stay below 2^32");
  const bool need_cond = c->kind == ASD_DEN_RESMLP_BF16 && c->mlp.d_cond > 0;
  if (need_cond && !cond_dev && n_chains > 0) return fail(c, ASD_ERR_INVALID_ARG, "cond_dev required (d_cond > 0)");
  if (n_chains != c->n || chain_id_base != c->chain_base) {
    // the captured rounds hold the batch size and the chain ids in their kernel arguments
    ASD_CUDA(c, cudaStreamSynchronize(c->gstream));
    for (auto& kv : c->graphs) cudaGraphExecDestroy(kv.second.exec);
    c->graphs.clear();
  }
  c->n = n_chains;
  c->chain_base = chain_id_base;
  // state, cursors, round and per-call counters, window state, histogram, trajectory row 0, bf16 conditioning
  launch_reset(c, y0_dev, need_cond && n_chains > 0 ? cond_dev : nullptr);
  if (c->G2) {
    const int h = (n_chains + 1) / 2;
    c->lanes[0].start = 0;
    c->lanes[0].n = h;
    c->lanes[1].start = h;
    c->lanes[1].n = n_chains - h;
    for (int l = 0; l < 2; ++l) {
      ASD_CUDA(c, cudaMemsetAsync(c->lanes[l].counters, 0, sizeof(RoundCounters), c->stream));
      ASD_CUDA(c, cudaMemsetAsync(c->lanes[l].v_off, 0, sizeof(int), c->stream));
    }
    ASD_CUDA(c, cudaMemsetAsync(c->merged_rows, 0, sizeof(int), c->stream));
  }
  ASD_CUDA(c, cudaGetLastError());
  c->have_reset = true;
  c->round_bound = n_chains;
  c->launches = 0;
  return ASD_OK;
}

asd_status asd_round(asd_ctx* ctx, asd_round_stats* stats_host) {
  if (!ctx) return ASD_ERR_INVALID_ARG;
  Ctx* c = &ctx->c;
  if (!c->have_reset) return fail(c, ASD_ERR_STATE, "asd_round before asd_reset");
  // the bound on the active chains that sizes the grids: what the previous round reported, if it was read
  asd_status st;
  if (c->resident_mode == 2 && !c->prof_on && resident_supported(c, c->window, nullptr))
    st = launch_resident(c, c->window, true, 1);  // one round of the chain-resident kernel (lock-step tests)
  else
    st = enqueue_round(c, c->window, true, std::min(c->n, c->round_bound));
  if (st != ASD_OK) return st;
  if (stats_host) {
    st = sync_counters(c);
    if (st != ASD_OK) return st;
    const RoundCounters& h = *c->counters_host;
    c->round_bound = std::max(h.n_active_after, 1);
    stats_host->n_active_before = h.n_active;
    stats_host->n_active_after = h.n_active_after;
    stats_host->rows_pass1 = c->lookahead ? h.n_eval : h.n_active;
    stats_host->rows_pass2 = h.rows2;
    stats_host->accepted_total = (int64_t)h.accepted;
  }
  return ASD_OK;
}

static asd_status finish_run(Ctx* c, float* y_out_dev, int32_t* rounds_out_dev, asd_run_stats* stats, long long launches0,
                             bool want_round_stats) {
  launch_finish(c, y_out_dev, rounds_out_dev);  // results out, max / mean of the round counters into the counters
  ASD_CUDA(c, cudaGetLastError());
  ASD_CUDA(c, cudaEventRecord(c->ev1, c->stream));
  asd_status st = sync_counters(c);
  if (st != ASD_OK) return st;
  if (stats) {
    float ms = 0.f;
    cudaEventElapsedTime(&ms, c->ev0, c->ev1);
    stats->ms_total = ms;
    stats->rows_total = (int64_t)c->counters_host->rows_total + c->extra_rows_total;
    stats->rows_verified = (int64_t)c->counters_host->rows_verified + c->extra_rows_verified;
    stats->launches = c->launches - launches0;
    stats->rounds_max = 0;
    stats->rounds_mean = 0.0;
    if (want_round_stats && c->n > 0) {
      stats->rounds_max = c->counters_host->rounds_max;
      stats->rounds_mean = (double)c->counters_host->rounds_sum / c->n;
    }
  }
  return ASD_OK;
}

asd_status asd_sample(asd_ctx* ctx, float* y_out_dev, int32_t* rounds_out_dev, asd_run_stats* stats_host) {
  if (!ctx) return ASD_ERR_INVALID_ARG;
  Ctx* c = &ctx->c;
  if (!c->have_reset) return fail(c, ASD_ERR_STATE, "asd_sample before asd_reset");
  const long long launches0 = c->launches;
  ASD_CUDA(c, cudaEventRecord(c->ev0, c->stream));
  // The host does not wait for a round before enqueuing the next one: the counters of round r are copied
  // to a pinned ring slot and read once their event has completed, at most kDepth rounds later.  The
  // bound on the active chains that sizes the grids is therefore a few rounds old, which is still an
  // upper bound (chains only finish), and the rounds enqueued after the last chain finished find no
  // active chain and do nothing.  Theorem 3: the cursor strictly increases, so K rounds always suffice.
  c->extra_rows_total = c->extra_rows_verified = 0;
  // Closed-form drifts: the whole while loop of every chain inside one launch, a block per chain.
  if (c->resident_mode >= 1 && !c->prof_on && resident_supported(c, c->window, nullptr)) {
    asd_status st = launch_resident(c, c->window, true, 0x7fffffff);
    if (st != ASD_OK) return st;
    ASD_CUDA(c, cudaGetLastError());
    return finish_run(c, y_out_dev, rounds_out_dev, stats_host, launches0, true);
  }
  if (use_stagger(c)) {
    asd_status st = sample_staggered(c);
    if (st != ASD_OK) return st;
    return finish_run(c, y_out_dev, rounds_out_dev, stats_host, launches0, true);
  }
  // Unless per-phase timing is on, a round is replayed as one CUDA graph on the context's private stream.
  constexpr int kDepth = 4;
  int active = c->n;
  {
  PrivateStreamScope pss(c);
  long long issued = 0, consumed = 0;
  const long long max_rounds = (long long)c->K + 2;
  asd_status deferred = ASD_OK;
  constexpr size_t kEventsPerRound = 2 * PH_COUNT + 8;  // each ring slot times its phases with its own events
  size_t prof_pairs[Ctx::kRing] = {};
  auto consume = [&](bool wait) -> bool {  // false: nothing (more) to read right now
    const int slot = (int)(consumed % Ctx::kRing);
    if (wait) {
      if (cudaEventSynchronize(c->ring_ev[slot]) != cudaSuccess) {
        deferred = fail(c, ASD_ERR_CUDA, "event synchronisation failed");
        return false;
      }
    } else if (cudaEventQuery(c->ring_ev[slot]) != cudaSuccess) {
      return false;
    }
    const RoundCounters& h = c->ring_host[slot];
    if (h.err != 0 && deferred == ASD_OK)
      deferred = fail(c, (asd_status)h.err, "a bounded device-side wait ran out (kernel returned early)");
    active = h.n_active_after;
    if (c->prof_on) {
      prof_collect_some(c, (long long)prof_pairs[slot]);
      const long long n1 = h.n_active, n1e = c->lookahead ? h.n_eval : h.n_active, n2 = h.rows2;
      for (int ph : {PH_PREP, PH_DRAFT, PH_VERIFY}) c->prof[ph].rows += n1;
      for (int ph : {PH_PACK, PH_D1_IN, PH_D1_HID, PH_D1_OUT, PH_D1_ANALYTIC}) c->prof[ph].rows += n1e;
      for (int ph : {PH_D2_IN, PH_D2_HID, PH_D2_OUT, PH_D2_ANALYTIC}) c->prof[ph].rows += n2;
    }
    ++consumed;
    return true;
  };
  // with graph replay a ring slot stands for kRoundsPerGraph rounds (the counters of the last one)
  // (fewer when the run is short: rounds enqueued after the last chain finished are wasted launches)
  const int min_rounds = (c->K + c->window - 1) / c->window;
  const int group = pss.on ? std::max(1, std::min(kRoundsPerGraph, min_rounds / 16)) : 1;
  while (active > 0 && issued * group < max_rounds + group && deferred == ASD_OK) {
    const int slot = (int)(issued % Ctx::kRing);
    c->ev_used = (size_t)slot * kEventsPerRound;
    const size_t pending0 = c->pending.size();
    asd_status st = enqueue_rounds(c, pss.on, c->window, true, active, group);
    if (st != ASD_OK) return st;
    prof_pairs[slot] = c->pending.size() - pending0;
    ASD_CUDA(c, cudaMemcpyAsync(&c->ring_host[slot], c->counters, sizeof(RoundCounters), cudaMemcpyDeviceToHost, c->stream));
    ASD_CUDA(c, cudaEventRecord(c->ring_ev[slot], c->stream));
    ++issued;
    while (consumed < issued && consume(issued - consumed >= kDepth)) {
    }
  }
  while (consumed < issued && deferred == ASD_OK && consume(true)) {
  }
  if (deferred != ASD_OK) {
    cudaStreamSynchronize(c->stream);
    cudaMemsetAsync(&c->counters->err, 0, sizeof(int), c->stream);
    prof_collect(c);
    return deferred;
  }
  if (active > 0) return fail(c, ASD_ERR_STATE, "chains still active after K rounds");
  }
  return finish_run(c, y_out_dev, rounds_out_dev, stats_host, launches0, true);
}

asd_status asd_sequential_ddpm(asd_ctx* ctx, float* y_out_dev, asd_run_stats* stats_host) {
  if (!ctx) return ASD_ERR_INVALID_ARG;
  Ctx* c = &ctx->c;
  if (!c->have_reset) return fail(c, ASD_ERR_STATE, "asd_sequential_ddpm before asd_reset");
  const long long launches0 = c->launches;
  if (c->resident_mode >= 1 && !c->prof_on && resident_supported(c, 1, nullptr)) {
    ASD_CUDA(c, cudaEventRecord(c->ev0, c->stream));
    asd_status st = launch_resident(c, 1, false, 0x7fffffff);
    if (st != ASD_OK) return st;
    ASD_CUDA(c, cudaGetLastError());
    return finish_run(c, y_out_dev, nullptr, stats_host, launches0, true);
  }
  int min_a = c->K;
  if (c->n > 0) {
    std::vector<int> a(c->n);
    ASD_CUDA(c, cudaMemcpyAsync(a.data(), c->a, (size_t)c->n * sizeof(int), cudaMemcpyDeviceToHost, c->stream));
    ASD_CUDA(c, cudaStreamSynchronize(c->stream));
    for (int v : a) min_a = std::min(min_a, v);
  }
  ASD_CUDA(c, cudaEventRecord(c->ev0, c->stream));
  {
    PrivateStreamScope pss(c);
    for (int i = min_a; i < c->K;) {
      const int group = (pss.on && c->K - i >= kRoundsPerGraph) ? kRoundsPerGraph : 1;
      asd_status st = enqueue_rounds(c, pss.on, 1, false, c->n, group);
      if (st != ASD_OK) return st;
      i += group;
    }
  }
  return finish_run(c, y_out_dev, nullptr, stats_host, launches0, true);
}

asd_status asd_sample_host(asd_ctx* ctx, int32_t n_chains, uint64_t chain_id_base, const float* y0_host,
                           const float* cond_host, int32_t sequential, float* y_out_host, int32_t* rounds_out_host,
                           asd_run_stats* stats_host) {
  if (!ctx) return ASD_ERR_INVALID_ARG;
  Ctx* c = &ctx->c;
  if (n_chains < 0 || n_chains > c->max_chains) return fail(c, ASD_ERR_INVALID_ARG, "n_chains out of range");
  if (!y_out_host && n_chains > 0) return fail(c, ASD_ERR_INVALID_ARG, "y_out_host must not be NULL");
  const size_t nd = (size_t)n_chains * c->d;
  // the library's own state / workspace rows serve as staging: y0 -> G (unused until the first
  // round), cond -> the drafted-point buffer (reset converts it to bf16 from there)
  const bool need_cond = c->kind == ASD_DEN_RESMLP_BF16 && c->mlp.d_cond > 0;
  if (need_cond && !cond_host && n_chains > 0) return fail(c, ASD_ERR_INVALID_ARG, "cond_host required (d_cond > 0)");
  if (y0_host) ASD_CUDA(c, cudaMemcpyAsync(c->G, y0_host, nd * sizeof(float), cudaMemcpyHostToDevice, c->stream));
  float* cond_stage = nullptr;
  if (need_cond && n_chains > 0) {
    cond_stage = c->Yhat;  // max_rows * d >= n * d_cond is not guaranteed; check
    if ((size_t)c->max_rows * c->d < (size_t)n_chains * c->mlp.d_cond)
      return fail(c, ASD_ERR_UNSUPPORTED, "conditioning larger than the staging workspace");
    ASD_CUDA(c, cudaMemcpyAsync(cond_stage, cond_host, (size_t)n_chains * c->mlp.d_cond * sizeof(float),
                                cudaMemcpyHostToDevice, c->stream));
  }
  asd_status st = asd_reset(ctx, n_chains, chain_id_base, y0_host ? c->G : nullptr, cond_stage);
  if (st != ASD_OK) return st;
  st = sequential ? asd_sequential_ddpm(ctx, nullptr, stats_host) : asd_sample(ctx, nullptr, nullptr, stats_host);
  if (st != ASD_OK) return st;
  if (n_chains > 0) {
    ASD_CUDA(c, cudaMemcpyAsync(y_out_host, c->y, nd * sizeof(float), cudaMemcpyDeviceToHost, c->stream));
    if (rounds_out_host)
      ASD_CUDA(c, cudaMemcpyAsync(rounds_out_host, c->rounds, (size_t)n_chains * sizeof(int), cudaMemcpyDeviceToHost, c->stream));
    ASD_CUDA(c, cudaStreamSynchronize(c->stream));
  }
  return ASD_OK;
}

asd_status asd_set_profiling(asd_ctx* ctx, int32_t enable) {
  if (!ctx) return ASD_ERR_INVALID_ARG;
  Ctx* c = &ctx->c;
  cudaStreamSynchronize(c->stream);
  prof_collect(c);
  c->prof_on = enable != 0;
  for (auto& p : c->prof) p = PhaseAcc{};
  return ASD_OK;
}

asd_status asd_get_profile(asd_ctx* ctx, asd_phase_time* out, int32_t capacity, int32_t* n_out) {
  if (!ctx || !out || !n_out) return ASD_ERR_INVALID_ARG;
  Ctx* c = &ctx->c;
  static const char* names[PH_COUNT] = {"prep", "pack", "pass1_gemm_in", "pass1_gemm_hidden", "pass1_gemm_out",
                                        "pass1_closed_form", "draft", "pass2_gemm_in", "pass2_gemm_hidden",
                                        "pass2_gemm_out", "pass2_closed_form", "verify"};
  int k = 0;
  for (int ph = 0; ph < PH_COUNT && k < capacity; ++ph) {
    out[k].name = names[ph];
    out[k].launches = c->prof[ph].launches;
    out[k].ms = c->prof[ph].ms;
    out[k].rows = c->prof[ph].rows;
    ++k;
  }
  *n_out = k;
  return ASD_OK;
}

asd_status asd_get_state(asd_ctx* ctx, int32_t* a_dev, float* y_dev, int32_t* rounds_dev) {
  if (!ctx) return ASD_ERR_INVALID_ARG;
  Ctx* c = &ctx->c;
  if (!c->have_reset) return fail(c, ASD_ERR_STATE, "asd_get_state before asd_reset");
  if (a_dev) ASD_CUDA(c, cudaMemcpyAsync(a_dev, c->a, (size_t)c->n * sizeof(int), cudaMemcpyDeviceToDevice, c->stream));
  if (y_dev) ASD_CUDA(c, cudaMemcpyAsync(y_dev, c->y, (size_t)c->n * c->d * sizeof(float), cudaMemcpyDeviceToDevice, c->stream));
  if (rounds_dev)
    ASD_CUDA(c, cudaMemcpyAsync(rounds_dev, c->rounds, (size_t)c->n * sizeof(int), cudaMemcpyDeviceToDevice, c->stream));
  return ASD_OK;
}

asd_status asd_set_state(asd_ctx* ctx, const int32_t* a_dev, const float* y_dev, const int32_t* rounds_dev) {
  if (!ctx) return ASD_ERR_INVALID_ARG;
  Ctx* c = &ctx->c;
  if (!c->have_reset) return fail(c, ASD_ERR_STATE, "asd_set_state before asd_reset");
  if (a_dev) {
    ASD_CUDA(c, cudaMemcpyAsync(c->a, a_dev, (size_t)c->n * sizeof(int), cudaMemcpyDeviceToDevice, c->stream));
    c->round_bound = c->n;  // cursors may have moved back: every chain may be active again
  }
  if (y_dev) ASD_CUDA(c, cudaMemcpyAsync(c->y, y_dev, (size_t)c->n * c->d * sizeof(float), cudaMemcpyDeviceToDevice, c->stream));
  // a saved drift belongs to the point and step it was evaluated at
  if ((a_dev || y_dev) && c->has_v) ASD_CUDA(c, cudaMemsetAsync(c->has_v, 0, (size_t)c->max_chains * sizeof(int), c->stream));
  if (rounds_dev)
    ASD_CUDA(c, cudaMemcpyAsync(c->rounds, rounds_dev, (size_t)c->n * sizeof(int), cudaMemcpyDeviceToDevice, c->stream));
  if (a_dev || y_dev) launch_traj_seed(c);  // the restored state is row a of the trajectory
  return ASD_OK;
}

asd_status asd_get_window_state(asd_ctx* ctx, int32_t* window_dev, int32_t* ema8_dev) {
  if (!ctx) return ASD_ERR_INVALID_ARG;
  Ctx* c = &ctx->c;
  if (!c->have_reset) return fail(c, ASD_ERR_STATE, "asd_get_window_state before asd_reset");
  if (window_dev) ASD_CUDA(c, cudaMemcpyAsync(window_dev, c->wnd, (size_t)c->n * sizeof(int), cudaMemcpyDeviceToDevice, c->stream));
  if (ema8_dev) ASD_CUDA(c, cudaMemcpyAsync(ema8_dev, c->ema8, (size_t)c->n * sizeof(int), cudaMemcpyDeviceToDevice, c->stream));
  return ASD_OK;
}

asd_status asd_set_window_state(asd_ctx* ctx, const int32_t* window_dev, const int32_t* ema8_dev) {
  if (!ctx) return ASD_ERR_INVALID_ARG;
  Ctx* c = &ctx->c;
  if (!c->have_reset) return fail(c, ASD_ERR_STATE, "asd_set_window_state before asd_reset");
  if (window_dev) ASD_CUDA(c, cudaMemcpyAsync(c->wnd, window_dev, (size_t)c->n * sizeof(int), cudaMemcpyDeviceToDevice, c->stream));
  if (ema8_dev) ASD_CUDA(c, cudaMemcpyAsync(c->ema8, ema8_dev, (size_t)c->n * sizeof(int), cudaMemcpyDeviceToDevice, c->stream));
  return ASD_OK;
}

asd_status asd_debug_last_round(asd_ctx* ctx, float* ln_ratio_dev, float* ln_u_dev, int32_t* accepted_dev) {
  if (!ctx) return ASD_ERR_INVALID_ARG;
  Ctx* c = &ctx->c;
  if (!c->have_reset) return fail(c, ASD_ERR_STATE, "asd_debug_last_round before asd_reset");
  const size_t nw = (size_t)c->n * c->window;
  if ((ln_ratio_dev || ln_u_dev) && !c->dbg_lr)
    return fail(c, ASD_ERR_STATE, "ln ratio / ln u are recorded only by a context created with ASD_FLAG_DEBUG_DUMP");
  if (ln_ratio_dev) ASD_CUDA(c, cudaMemcpyAsync(ln_ratio_dev, c->dbg_lr, nw * sizeof(float), cudaMemcpyDeviceToDevice, c->stream));
  if (ln_u_dev) ASD_CUDA(c, cudaMemcpyAsync(ln_u_dev, c->dbg_lu, nw * sizeof(float), cudaMemcpyDeviceToDevice, c->stream));
  if (accepted_dev)
    ASD_CUDA(c, cudaMemcpyAsync(accepted_dev, c->acc_len, (size_t)c->n * sizeof(int), cudaMemcpyDeviceToDevice, c->stream));
  return ASD_OK;
}

asd_status asd_get_trajectory(asd_ctx* ctx, float* traj_dev) {
  if (!ctx) return ASD_ERR_INVALID_ARG;
  Ctx* c = &ctx->c;
  if (!c->have_reset) return fail(c, ASD_ERR_STATE, "asd_get_trajectory before asd_reset");
  if (!c->traj) return fail(c, ASD_ERR_STATE, "the context was created without ASD_FLAG_TRAJECTORY");
  if (!traj_dev) return fail(c, ASD_ERR_INVALID_ARG, "traj_dev must not be NULL");
  ASD_CUDA(c, cudaMemcpyAsync(traj_dev, c->traj, (size_t)c->n * (c->K + 1) * c->d * sizeof(float), cudaMemcpyDeviceToDevice,
                              c->stream));
  return ASD_OK;
}

asd_status asd_get_prefix_histogram(asd_ctx* ctx, int64_t* hist_host, int32_t capacity, int32_t* n_out) {
  if (!ctx) return ASD_ERR_INVALID_ARG;
  Ctx* c = &ctx->c;
  if (!hist_host || !n_out || capacity < 0) return fail(c, ASD_ERR_INVALID_ARG, "hist_host and n_out required");
  if (!c->have_reset) return fail(c, ASD_ERR_STATE, "asd_get_prefix_histogram before asd_reset");
  const int m = std::min(capacity, c->window + 1);
  static_assert(sizeof(unsigned long long) == sizeof(int64_t), "histogram entries are 64 bit");
  ASD_CUDA(c, cudaMemcpyAsync(hist_host, c->hist, (size_t)m * sizeof(int64_t), cudaMemcpyDeviceToHost, c->stream));
  ASD_CUDA(c, cudaStreamSynchronize(c->stream));
  *n_out = m;
  return ASD_OK;
}

asd_status asd_debug_wait_selftest(asd_ctx* ctx) {
  if (!ctx) return ASD_ERR_INVALID_ARG;
  Ctx* c = &ctx->c;
  launch_wait_selftest(c);
  ASD_CUDA(c, cudaGetLastError());
  return sync_counters(c);  // reports and clears the device error word
}

asd_status asd_denoise(asd_ctx* ctx, int32_t n_rows, const int32_t* step_dev, const float* y_dev,
                       const int32_t* slot_dev, float* out_dev) {
  if (!ctx) return ASD_ERR_INVALID_ARG;
  Ctx* c = &ctx->c;
  if (n_rows < 0 || n_rows > c->max_rows) return fail(c, ASD_ERR_INVALID_ARG, "n_rows out of range");
  if (n_rows == 0) return ASD_OK;
  if (!step_dev || !y_dev || !out_dev) return fail(c, ASD_ERR_INVALID_ARG, "step_dev, y_dev, out_dev required");
  const bool need_cond = c->kind == ASD_DEN_RESMLP_BF16 && c->mlp.d_cond > 0;
  if (need_cond && !slot_dev) return fail(c, ASD_ERR_INVALID_ARG, "slot_dev required (d_cond > 0)");
  int* n_dev = &c->counters[1].n_active;
  ASD_CUDA(c, cudaMemcpyAsync(n_dev, &n_rows, sizeof(int), cudaMemcpyHostToDevice, c->stream));
  RowSet rs{n_dev, n_rows, y_dev, nullptr, step_dev, slot_dev};
  asd_status st = ASD_OK;
  if (c->kind == ASD_DEN_GMM_ISO)
    launch_gmm(c, rs, out_dev);
  else if (c->kind == ASD_DEN_GAUSS_LINEAR)
    launch_gauss(c, rs, out_dev);
  else {
    launch_pack(c, rs);
    st = mlp_forward(c, rs, out_dev, 2);
    if (st != ASD_OK) return st;
  }
  ASD_CUDA(c, cudaGetLastError());
  return sync_counters(c);
}

}  // extern "C"

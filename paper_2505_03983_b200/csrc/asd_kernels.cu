// Elementwise / reduction kernels of the ASD round: bookkeeping (active list, row offsets),
// draft (Algorithm 1, proposal loop), verify + resample + advance (Algorithms 2 and 3, and the
// advance step of Algorithm 1), the closed-form posterior means (Eq. 4) and the feature packing
// of the network denoiser.  fp32 throughout; the Gaussian noise uses the special-function unit's
// approximate lg2 / sqrt / sin / cos (absolute error about 1e-6 per normal), everything that decides an
// accept test (ln u, the reductions) is plain IEEE fp32.
#include <algorithm>

#include "asd_internal.h"
#include "asd_device.cuh"

namespace asd {

// Launch with programmatic stream serialization (see pdl_wait_then_release in asd_device.cuh).
template <typename... KArgs, typename... Args>
static void launch_pdl(Ctx* c, void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, Args... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = c->stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...);
  c->launches++;
}

// ---------------------------------------------------------------------------------------------
// Round driver bookkeeping: compact the chains with a < K into the active list and lay out the
// pass-2 rows (exclusive scan of w - 1).  One block; n is at most a few tens of thousands.
// ---------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(1024) prep_kernel(const int* __restrict__ a, const int* __restrict__ wnd, int n, int K,
                                                    int window, const int* __restrict__ has_v, int la,
                                                    int* __restrict__ act, int* __restrict__ row_off,
                                                    int* __restrict__ step1, int* __restrict__ act1,
                                                    int* __restrict__ step1e, int* __restrict__ idx1,
                                                    int* __restrict__ acc_len, int* __restrict__ first_rej,
                                                    RoundCounters* __restrict__ cnt) {
  pdl_wait_then_release();
  __shared__ int s_cnt[32], s_rows[32], s_ev[32];
  __shared__ int s_base_cnt, s_base_rows, s_base_ev;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  if (tid == 0) {
    s_base_cnt = 0;
    s_base_rows = 0;
    s_base_ev = 0;
  }
  __syncthreads();
  for (int j0 = 0; j0 < n; j0 += blockDim.x) {
    const int j = j0 + tid;
    int aj = K, flag = 0, rows = 0, ev = 0;
    if (j < n) {
      aj = a[j];
      flag = aj < K;
      rows = flag ? drafted_rows(chain_window(wnd, j, window, K, aj), aj, K, la) : 0;
      ev = flag && !(la && has_v[j]);  // v_a still has to be evaluated
      acc_len[j] = -1;
      first_rej[j] = 0x7fffffff;  // no rejection known yet (the verify step's slots kernel lowers it)
    }
    // inclusive warp scans
    int c = flag, r = rows, e = ev;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int c2 = __shfl_up_sync(0xffffffffu, c, o);
      const int r2 = __shfl_up_sync(0xffffffffu, r, o);
      const int e2 = __shfl_up_sync(0xffffffffu, e, o);
      if (lane >= o) {
        c += c2;
        r += r2;
        e += e2;
      }
    }
    if (lane == 31) {
      s_cnt[warp] = c;
      s_rows[warp] = r;
      s_ev[warp] = e;
    }
    __syncthreads();
    if (warp == 0) {
      int wc = s_cnt[lane], wr = s_rows[lane], we = s_ev[lane];
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const int c2 = __shfl_up_sync(0xffffffffu, wc, o);
        const int r2 = __shfl_up_sync(0xffffffffu, wr, o);
        const int e2 = __shfl_up_sync(0xffffffffu, we, o);
        if (lane >= o) {
          wc += c2;
          wr += r2;
          we += e2;
        }
      }
      s_cnt[lane] = wc;
      s_rows[lane] = wr;
      s_ev[lane] = we;
    }
    __syncthreads();
    const int pos = s_base_cnt + (warp ? s_cnt[warp - 1] : 0) + c - flag;
    const int roff = s_base_rows + (warp ? s_rows[warp - 1] : 0) + r - rows;
    const int epos = s_base_ev + (warp ? s_ev[warp - 1] : 0) + e - ev;
    if (flag) {
      act[pos] = j;
      row_off[pos] = roff;
      step1[pos] = aj;
      if (idx1) idx1[pos] = ev ? epos : -1;
      if (ev && act1) {
        act1[epos] = j;
        step1e[epos] = aj;
      }
    }
    __syncthreads();
    if (tid == 0) {
      s_base_cnt += s_cnt[31];
      s_base_rows += s_rows[31];
      s_base_ev += s_ev[31];
    }
    __syncthreads();
  }
  if (tid == 0) {
    row_off[s_base_cnt] = s_base_rows;
    cnt->n_active = s_base_cnt;
    cnt->rows2 = s_base_rows;
    cnt->n_eval = s_base_ev;
    cnt->n_active_after = 0;
    cnt->accepted = 0ull;
    cnt->rows_total += (unsigned long long)(s_base_ev + s_base_rows);
  }
}

// Per-chain speculation lengths apply to speculation rounds only (never to the window-1 steps of Eq. 7).
static const int* round_windows(const Ctx* c, int window) { return (c->adaptive && window > 1) ? c->wnd : nullptr; }

Lane whole_batch(const Ctx* c) {
  Lane L;
  L.start = 0;
  L.n = c->n;
  L.act = c->act;
  L.row_off = c->row_off;
  L.step1 = c->step1;
  L.counters = c->counters;
  L.act1 = c->act1;
  L.step1e = c->step1e;
  L.idx1 = c->idx1;
  return L;
}

void launch_prep(Ctx* c, const Lane& L, int window) {
  const int* wnd = round_windows(c, window);
  const int la = (c->lookahead && L.act1) ? 1 : 0;
  launch_pdl(c, prep_kernel, dim3(1), dim3(1024), 0, c->a + L.start, wnd ? wnd + L.start : nullptr, L.n, c->K, window,
             c->has_v, la, L.act, L.row_off, L.step1, L.act1, L.step1e, L.idx1, c->acc_len + L.start,
             c->first_rej + L.start, L.counters);
}

// ---------------------------------------------------------------------------------------------
// Draft (Algorithm 1, proposal loop): y^_{a+k} = y^_{a+k-1} + eta v_a + sigma xi_{a+k} for
// k = 1..w-1 (the last proposal sample is only needed when the whole window is accepted and is
// rebuilt by the verify kernel).  Two forms with identical arithmetic.  Large batches: one thread owns
// 4 dims of one chain and walks the window, so the "prefix sum" of the paper is a register recurrence.
// Small batches: a block owns 128 dims of one chain, the noise of all window slots is generated in
// parallel (thread = 4 dims x one slot in eight) into shared memory, the recurrence is then a short
// serial walk over the slots by one warp in exactly the order of Eq. 7, and all threads write the rows.
// Both write the fp32 points and, for the network denoiser, its bf16 input rows.
// ---------------------------------------------------------------------------------------------
struct DraftArgs {
  int d, K, window, nq, vec, par;
  PhiloxKeys keys;
  uint64_t chain_base;
  const RoundCounters* cnt;
  const int* act;
  const int* a;
  const int* wnd;  // per-chain speculation length, or null: `window` for every chain
  const int* row_off;
  const float* y;
  const float* v;
  const int* v_off;  // device: first row of v for this lane, or null
  const int* idx1;     // look-ahead: row of v per active position, -1 = take vsave[chain]
  const float* vsave;  // look-ahead: v_a saved by the previous round, by chain position
  int la;
  Tables tab;
  float* Yhat;
  int* row_step;
  int* row_slot;
  // network input rows (null for the closed-form denoisers)
  __nv_bfloat16* X;
  int in_pad, in_dim, d_cond, d_temb;
  const __nv_bfloat16* cond;
  const __nv_bfloat16* temb;
};

constexpr int kDraftQ = 32;       // float4 groups (= 128 dims) per block
constexpr int kDraftThreads = 256;
constexpr int kDraftChunk = 64;   // slots staged in shared memory at a time (staged form); longer windows take several chunks

// fp32 point and (network denoiser) bf16 input of row `row`, slot k, for float4 group q
__device__ __forceinline__ void draft_store(const DraftArgs& A, int row, int a, int k, int q, float4 yh) {
  store4(A.Yhat + (size_t)row * A.d, q, A.d, A.vec, yh);
  if (A.X) {
    const float ci = A.tab.c_in[a + k];
    __nv_bfloat16* xr = A.X + (size_t)row * A.in_pad + 4 * q;
    if (A.vec) {
      __nv_bfloat162 lo = __floats2bfloat162_rn(ci * yh.x, ci * yh.y);
      __nv_bfloat162 hi = __floats2bfloat162_rn(ci * yh.z, ci * yh.w);
      uint2 pk;
      pk.x = *reinterpret_cast<uint32_t*>(&lo);
      pk.y = *reinterpret_cast<uint32_t*>(&hi);
      *reinterpret_cast<uint2*>(xr) = pk;
    } else {
      const int b = 4 * q;
      if (b + 0 < A.d) xr[0] = __float2bfloat16_rn(ci * yh.x);
      if (b + 1 < A.d) xr[1] = __float2bfloat16_rn(ci * yh.y);
      if (b + 2 < A.d) xr[2] = __float2bfloat16_rn(ci * yh.z);
      if (b + 3 < A.d) xr[3] = __float2bfloat16_rn(ci * yh.w);
    }
  }
}

__global__ void __launch_bounds__(kDraftThreads) draft_kernel(const DraftArgs A) {
  pdl_wait_then_release();
  __shared__ float4 s_pt[kDraftChunk][kDraftQ];  // noise, then drafted points, per slot of a chunk (parallel form)
  const int p = blockIdx.x;
  if (p >= A.cnt->n_active) return;
  const int j = A.act[p];
  const int a = A.a[j];
  const int w = chain_window(A.wnd, j, A.window, A.K, a);
  const int row0 = A.row_off[p];
  const int nr = drafted_rows(w, a, A.K, A.la);  // slots 1..nr are drafted
  const float* vrow = (A.la && A.idx1[p] < 0) ? A.vsave + (size_t)j * A.d
                                               : A.v + (size_t)((A.la ? A.idx1[p] : (A.v_off ? *A.v_off : 0) + p)) * A.d;
  const uint32_t chain = (uint32_t)(A.chain_base + (uint64_t)j);
  if (!A.par) {
    // large batches: one thread owns 4 dims and walks the window; nothing is staged
    const int q = blockIdx.y * kDraftThreads + threadIdx.x;
    if (q < A.nq) {
      float4 yh = load4(A.y + (size_t)j * A.d, q, A.d, A.vec);
      const float4 v = load4(vrow, q, A.d, A.vec);
      for (int k = 1; k <= nr; ++k) {
        const int i = a + k - 1;  // step i -> i+1 uses eta_i, sigma_{i+1}, xi_{i+1}
        const float eta = A.tab.eta[i], sig = A.tab.sig[i];
        const float4 xi = xi4((uint32_t)q, (uint32_t)(i + 1), chain, A.keys);
        yh.x = fmaf(sig, xi.x, fmaf(eta, v.x, yh.x));
        yh.y = fmaf(sig, xi.y, fmaf(eta, v.y, yh.y));
        yh.z = fmaf(sig, xi.z, fmaf(eta, v.z, yh.z));
        yh.w = fmaf(sig, xi.w, fmaf(eta, v.w, yh.w));
        draft_store(A, row0 + k - 1, a, k, q, yh);
      }
    }
  } else {
    // small batches: the noise of a chunk of slots in parallel, then the recurrence by one warp (which carries
    // the point from chunk to chunk in registers), then the stores
    const int ql = threadIdx.x & (kDraftQ - 1), ks = threadIdx.x / kDraftQ;
    constexpr int kSlotLanes = kDraftThreads / kDraftQ;
    const int q = blockIdx.y * kDraftQ + ql;
    const bool q_ok = q < A.nq;
    float4 yh = make_float4(0.f, 0.f, 0.f, 0.f), v = yh;
    if (ks == 0 && q_ok) {
      yh = load4(A.y + (size_t)j * A.d, q, A.d, A.vec);
      v = load4(vrow, q, A.d, A.vec);
    }
    for (int kc = 0; kc < nr; kc += kDraftChunk) {
      const int kn = min(kDraftChunk, nr - kc);  // slots kc + 1 .. kc + kn
      if (q_ok)
        for (int kk = ks; kk < kn; kk += kSlotLanes) s_pt[kk][ql] = xi4((uint32_t)q, (uint32_t)(a + kc + kk + 1), chain, A.keys);
      __syncthreads();
      if (ks == 0 && q_ok) {
        for (int kk = 0; kk < kn; ++kk) {
          const int i = a + kc + kk;
          const float eta = A.tab.eta[i], sig = A.tab.sig[i];
          const float4 xi = s_pt[kk][ql];
          yh.x = fmaf(sig, xi.x, fmaf(eta, v.x, yh.x));
          yh.y = fmaf(sig, xi.y, fmaf(eta, v.y, yh.y));
          yh.z = fmaf(sig, xi.z, fmaf(eta, v.z, yh.z));
          yh.w = fmaf(sig, xi.w, fmaf(eta, v.w, yh.w));
          s_pt[kk][ql] = yh;
        }
      }
      __syncthreads();
      if (q_ok)
        for (int kk = ks; kk < kn; kk += kSlotLanes) draft_store(A, row0 + kc + kk, a, kc + kk + 1, q, s_pt[kk][ql]);
      __syncthreads();
    }
  }
  // row maps, conditioning, time embedding and zero padding: the chain's blocks share the slots (this block takes
  // slots k = 1 + blockIdx.y + i * gridDim.y).  With few blocks in flight (the staged form) the (slot, element) pairs
  // are walked flat, four per thread at a time with the loads ahead of the stores, so a thread waits for memory once
  // per four elements, not once per slot.
  const int k_first = 1 + (int)blockIdx.y;
  const int ks = nr >= k_first ? (nr - k_first) / (int)gridDim.y + 1 : 0;
  for (int i = threadIdx.x; i < ks; i += blockDim.x) {
    const int k = k_first + i * (int)gridDim.y;
    A.row_step[row0 + k - 1] = a + k;
    A.row_slot[row0 + k - 1] = j;
  }
  if (A.X && !A.par) {
    // many blocks in flight: slot by slot, no index arithmetic per element
    const int extra = A.in_pad - A.d;
    for (int k = k_first; k <= nr; k += gridDim.y) {
      __nv_bfloat16* xr = A.X + (size_t)(row0 + k - 1) * A.in_pad + A.d;
      for (int e = threadIdx.x; e < extra; e += blockDim.x) {
        __nv_bfloat16 val = __float2bfloat16_rn(0.f);
        if (e < A.d_cond)
          val = A.cond[(size_t)j * A.d_cond + e];
        else if (e < A.d_cond + A.d_temb)
          val = A.temb[(size_t)(a + k) * A.d_temb + (e - A.d_cond)];
        xr[e] = val;
      }
    }
  } else if (A.X) {
    const int extra = A.in_pad - A.d;
    const int items = ks * extra, stride = (int)blockDim.x;
    const __nv_bfloat16 zero = __float2bfloat16_rn(0.f);
    for (int base = threadIdx.x; base < items; base += 4 * stride) {
      __nv_bfloat16 val[4];
      size_t dst[4];
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const int idx = base + u * stride;
        val[u] = zero;
        dst[u] = 0;
        if (idx < items) {
          const int i = idx / extra, e = idx - i * extra;
          const int k = k_first + i * (int)gridDim.y;
          dst[u] = (size_t)(row0 + k - 1) * A.in_pad + A.d + e;
          if (e < A.d_cond)
            val[u] = A.cond[(size_t)j * A.d_cond + e];
          else if (e < A.d_cond + A.d_temb)
            val[u] = A.temb[(size_t)(a + k) * A.d_temb + (e - A.d_cond)];
        }
      }
#pragma unroll
      for (int u = 0; u < 4; ++u)
        if (base + u * stride < items) A.X[dst[u]] = val[u];
    }
  }
}

void launch_draft(Ctx* c, const Lane& L, int window, const float* v_base, const int* v_off_dev) {
  const bool la = c->lookahead && L.idx1;  // look-ahead drafts a row even for a window of one step
  if ((window <= 1 && !la) || L.n == 0) return;
  const int* wnd = round_windows(c, window);
  DraftArgs A{};
  A.d = c->d;
  A.K = c->K;
  A.window = window;
  A.nq = (c->d + 3) / 4;
  A.vec = (c->d % 4 == 0);
  A.keys = make_philox_keys(c->seed);
  A.chain_base = c->chain_base + (uint64_t)L.start;
  A.cnt = L.counters;
  A.act = L.act;
  A.a = c->a + L.start;
  A.wnd = wnd ? wnd + L.start : nullptr;
  A.row_off = L.row_off;
  A.y = c->y + (size_t)L.start * c->d;
  A.v = v_base;
  A.v_off = v_off_dev;
  A.la = la ? 1 : 0;
  A.idx1 = L.idx1;
  A.vsave = c->vsave;
  A.tab = c->tab;
  A.Yhat = c->Yhat;
  A.row_step = c->row_step;
  A.row_slot = c->row_slot;
  if (c->kind == ASD_DEN_RESMLP_BF16) {
    A.X = c->mlp.X;
    A.in_pad = c->mlp.in_pad;
    A.in_dim = c->mlp.in_dim;
    A.d_cond = c->mlp.d_cond;
    A.d_temb = c->mlp.d_temb;
    A.cond = c->mlp.cond + (size_t)L.start * c->mlp.d_cond;
    A.temb = c->mlp.temb;
  }
  // the staged, slot-parallel form only when one thread per 4 dims would leave the machine mostly idle
  A.par = (long long)L.n * ((A.nq + kDraftThreads - 1) / kDraftThreads) < 2ll * c->num_sms;
  const int per_block = A.par ? kDraftQ : kDraftThreads;
  dim3 grid(L.n, (A.nq + per_block - 1) / per_block);  // chains along x (no 65535 limit there)
  launch_pdl(c, draft_kernel, grid, dim3(kDraftThreads), 0, A);
}

// ---------------------------------------------------------------------------------------------
// Verify + resample + advance (Algorithm 2, Algorithm 3, advance step of Algorithm 1).
// One block per active chain.  The block walks the window slots k = 2, 3, ... in order, a few slots at
// a time (one or two warps per slot); for each slot its warps regenerate xi_{a+k}, read the drift
// g_{k-1} at the drafted point once (coalesced float4) and reduce
//   <xi, delta>, |delta|^2, delta = v_a - g_{k-1}      (m^ - m = eta delta)
// over d (warp shuffles, then a fixed-order sum of the warps' partials that every thread repeats, so
// all threads reach the same decision without a second barrier);
//   ln ratio = -(eta/sigma) <xi, delta> - (eta^2 / 2 sigma^2) |delta|^2,  accept iff ln u <= min(0, ln ratio).
// The Verifier needs only the end of the all-accepted prefix, so the walk stops after the group that
// holds the first rejected slot: drifts beyond it are never read (all_slots != 0 keeps going, for the
// diagnostics).
// Then the block writes the new state: the reflected sample at the first rejected slot
//   y = y^_n + eta g_n + sigma (xi - 2 delta <delta, xi> / |delta|^2)
// or, if everything was accepted, the last proposal sample y^_w.
// ---------------------------------------------------------------------------------------------
struct VerifyArgs {
  int d, K, window, dbg_stride, nq, vec, use_u, all_slots, wps;
  int horizon;      // slots 2 .. 1 + horizon are reduced by the slots kernel (0: none)
  float* slot_dot;  // [n, window] per-slot <xi, delta>, |delta|^2 and ln u left by the slots kernel
  float* slot_nrm;
  float* slot_lu;
  int* first_rej;   // [n] lowest rejected slot found so far this round (INT_MAX: none), lowered with atomicMin
  PhiloxKeys keys;
  uint64_t chain_base;
  RoundCounters* cnt;
  const int* act;
  int* a;
  int* wnd;    // per-chain speculation length (adaptive mode), or null
  int* ema8;   // 8 x running mean of the steps advanced per round (adaptive mode)
  int* rounds;
  const int* row_off;
  float* y;
  const float* v;
  const int* v_off;  // device: first row of v for this lane, or null
  const int* idx1;   // look-ahead: row of v per active position, -1 = take vsave[chain]
  float* vsave;      // look-ahead: where a fully accepted window leaves v_a of the next round
  int* has_v;
  int la;
  const float* Yhat;
  const float* G;
  Tables tab;
  float* dbg_lr;   // diagnostics (ASD_FLAG_DEBUG_DUMP), else null
  float* dbg_lu;
  int* acc_len;
  float* traj;     // [n, K + 1, d] states y_0 .. y_K (ASD_FLAG_TRAJECTORY), else null
  unsigned long long* hist;  // [window + 1] chain-rounds by accepted prefix length
};

constexpr int kVerifyMaxWarps = 8;

// <xi_step, delta> and |delta|^2, delta = v_a - g, over the float4 groups tslot, tslot + team, ... of one slot
// (a team of wps warps shares a slot); four groups per thread at a time, all their loads issued before the first use.
// kFull: d is a multiple of 4 and every thread of the team has whole batches of four groups (no guards).
template <bool kFull>
__device__ __forceinline__ void slot_partial_t(const VerifyArgs& A, const float* vrow, const float* grow, uint32_t step,
                                               uint32_t chain, int tslot, int team, float& dot, float& nrm) {
  for (int q0 = tslot; q0 < A.nq; q0 += 4 * team) {
    float4 vv[4], gg[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const int q = q0 + u * team;
      if (kFull) {
        vv[u] = *reinterpret_cast<const float4*>(vrow + 4 * q);
        gg[u] = *reinterpret_cast<const float4*>(grow + 4 * q);
      } else if (q < A.nq) {
        vv[u] = load4(vrow, q, A.d, A.vec);
        gg[u] = load4(grow, q, A.d, A.vec);
      }
    }
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const int q = q0 + u * team;
      if (kFull || q < A.nq) {
        const float4 xi = xi4((uint32_t)q, step, chain, A.keys);
        float4 dl = make_float4(vv[u].x - gg[u].x, vv[u].y - gg[u].y, vv[u].z - gg[u].z, vv[u].w - gg[u].w);
        if (!kFull && !A.vec) {  // ragged tail: dims >= d contribute nothing
          const int b = 4 * q;
          if (b + 1 >= A.d) dl.y = 0.f;
          if (b + 2 >= A.d) dl.z = 0.f;
          if (b + 3 >= A.d) dl.w = 0.f;
        }
        dot = fmaf(xi.x, dl.x, dot);
        dot = fmaf(xi.y, dl.y, dot);
        dot = fmaf(xi.z, dl.z, dot);
        dot = fmaf(xi.w, dl.w, dot);
        nrm = fmaf(dl.x, dl.x, nrm);
        nrm = fmaf(dl.y, dl.y, nrm);
        nrm = fmaf(dl.z, dl.z, nrm);
        nrm = fmaf(dl.w, dl.w, nrm);
      }
    }
  }
}

__device__ __forceinline__ void slot_partial(const VerifyArgs& A, const float* vrow, const float* grow, uint32_t step,
                                             uint32_t chain, int tslot, int team, float& dot, float& nrm) {
  if (A.vec && A.nq % (4 * team) == 0)  // uniform over the block
    slot_partial_t<true>(A, vrow, grow, step, chain, tslot, team, dot, nrm);
  else
    slot_partial_t<false>(A, vrow, grow, step, chain, tslot, team, dot, nrm);
}

// Slots 2 .. 1 + horizon of every chain at once (the whole window for rows of some size): block (p, gy) reduces
// the S = 8 / wps slots 2 + gy S .. of active chain p, runs their accept tests (Algorithm 3) and lowers the
// chain's first rejected slot with atomicMin; the reductions stay in the slot arrays for the verify kernel.
// Every block has the same work, which keeps the machine full however the accepted prefixes are spread.  Blocks
// are dispatched in order of gy, so by the time a block of a later slot group starts, the groups before it have
// mostly reported: a block whose chain already has a rejection below its slots leaves at once (the Verifier
// needs nothing beyond the first rejection), which is what keeps most of the window's drifts unread.  The skip
// only saves work: which blocks take it varies from run to run, the result does not.
__global__ void __launch_bounds__(256, 4) verify_slots_kernel(const VerifyArgs A) {
  pdl_wait_then_release();
  __shared__ float s_part[kVerifyMaxWarps][2][kVerifyMaxWarps];  // [slot][dot | nrm][warp of team]
  const int p = blockIdx.x;
  if (p >= A.cnt->n_active) return;
  const int j = A.act[p];
  const int a = A.a[j];
  const int w = chain_window(A.wnd, j, A.window, A.K, a);
  const int k_end = min(w, 1 + A.horizon);
  const int wps = A.wps, S = kVerifyMaxWarps / wps;
  const int k_first = 2 + (int)blockIdx.y * S;
  if (k_first > k_end) return;
  if (!A.all_slots && *reinterpret_cast<volatile const int*>(A.first_rej + j) < k_first) return;
  const int row0 = A.row_off[p];
  const uint32_t chain = (uint32_t)(A.chain_base + (uint64_t)j);
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const float* vrow = (A.la && A.idx1[p] < 0) ? A.vsave + (size_t)j * A.d
                                               : A.v + (size_t)((A.la ? A.idx1[p] : (A.v_off ? *A.v_off : 0) + p)) * A.d;
  const int sw = warp / wps, wl = warp - sw * wps;
  const int k = k_first + sw;
  float dot = 0.f, nrm = 0.f;
  if (k <= k_end)
    slot_partial(A, vrow, A.G + (size_t)(row0 + k - 2) * A.d, (uint32_t)(a + k), chain, wl * 32 + lane, wps * 32, dot, nrm);
  dot = warp_sum(dot);
  nrm = warp_sum(nrm);
  if (lane == 0) {
    s_part[sw][0][wl] = dot;
    s_part[sw][1][wl] = nrm;
  }
  __syncthreads();
  if (tid < S && k_first + tid <= k_end) {
    float d2 = 0.f, n2 = 0.f;
    for (int x = 0; x < wps; ++x) {
      d2 += s_part[tid][0][x];
      n2 += s_part[tid][1][x];
    }
    const int kk = k_first + tid, i = a + kk - 1;
    const size_t o = (size_t)j * A.dbg_stride + kk - 1;
    const float lu = A.use_u ? ln_u((uint32_t)(a + kk), chain, A.keys) : 0.f;
    A.slot_dot[o] = d2;
    A.slot_nrm[o] = n2;
    A.slot_lu[o] = lu;
    const float lr = ln_ratio_of(A.tab.c1[i], A.tab.c2[i], d2, n2);
    if (!((lu <= fminf(0.f, lr)) || (n2 == 0.f))) atomicMin(A.first_rej + j, kk);
  }
}

__global__ void __launch_bounds__(256, 3) verify_kernel(const VerifyArgs A) {
  pdl_wait_then_release();
  __shared__ float s_part[2][kVerifyMaxWarps][2][kVerifyMaxWarps];  // [group parity][slot][dot | nrm][warp of team]
  __shared__ float s_lu[2][kVerifyMaxWarps];                        // [group parity][slot] ln u
  const int p = blockIdx.x;
  if (p >= A.cnt->n_active) return;
  const int j = A.act[p];
  const int a = A.a[j];
  const int w = chain_window(A.wnd, j, A.window, A.K, a);
  const int row0 = A.row_off[p];
  const uint32_t chain = (uint32_t)(A.chain_base + (uint64_t)j);
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, nwarps = blockDim.x >> 5;
  const float* vrow = (A.la && A.idx1[p] < 0) ? A.vsave + (size_t)j * A.d
                                               : A.v + (size_t)((A.la ? A.idx1[p] : (A.v_off ? *A.v_off : 0) + p)) * A.d;

  // diagnostics: ln u of every slot, and ln ratio = 0 for slot 1 (proposal mean == target mean, Lemma 1),
  // NaN for the slots the walk below does not reach
  if (A.dbg_lr) {
    const float nan = __int_as_float(0x7fc00000);
    for (int k = 1 + tid; k <= w; k += blockDim.x) {
      A.dbg_lu[(size_t)j * A.dbg_stride + k - 1] = A.use_u ? ln_u((uint32_t)(a + k), chain, A.keys) : 0.f;
      A.dbg_lr[(size_t)j * A.dbg_stride + k - 1] = k == 1 ? 0.f : nan;
    }
    __syncthreads();  // the values written below replace these
  }

  int n = w;                  // accepted prefix length; w = no rejection seen
  float rej_dot = 0.f, rej_nrm = 1.f;
  // slots 2 .. k_par went through the slots kernel: every slot up to the chain's first rejection was reduced and
  // tested there (and every slot of the window in the all-slots mode)
  const int k_par = min(w, 1 + A.horizon);
  if (k_par >= 2) {
    const int first = A.first_rej[j];
    if (first <= k_par) {
      n = first - 1;
      rej_dot = A.slot_dot[(size_t)j * A.dbg_stride + first - 1];
      rej_nrm = A.slot_nrm[(size_t)j * A.dbg_stride + first - 1];
    }
    if (A.dbg_lr) {
      const int k_have = A.all_slots ? k_par : min(first, k_par);
      for (int k = 2 + tid; k <= k_have; k += blockDim.x) {
        const size_t o = (size_t)j * A.dbg_stride + k - 1;
        const int i = a + k - 1;
        A.dbg_lr[o] = ln_ratio_of(A.tab.c1[i], A.tab.c2[i], A.slot_dot[o], A.slot_nrm[o]);
      }
    }
  }

  // Beyond them the slots are taken in groups of S = nwarps / wps (a team of wps warps reduces one slot), in order,
  // and the walk stops after the group that holds the first rejection.
  const int wps = A.wps, S = nwarps / wps;
  const int sw = warp / wps, wl = warp - sw * wps;
  const int tslot = wl * 32 + lane, team = wps * 32;
  int par = 0;
  for (int k0 = max(2, k_par + 1); k0 <= w && n == w; k0 += S, par ^= 1) {
    const int k = k0 + sw;
    // ln u of the group's slots (one Philox call each), by the first S threads
    if (tid < S && k0 + tid <= w) s_lu[par][tid] = A.use_u ? ln_u((uint32_t)(a + k0 + tid), chain, A.keys) : 0.f;
    float dot = 0.f, nrm = 0.f;
    if (k <= w) slot_partial(A, vrow, A.G + (size_t)(row0 + k - 2) * A.d, (uint32_t)(a + k), chain, tslot, team, dot, nrm);
    dot = warp_sum(dot);
    nrm = warp_sum(nrm);
    if (lane == 0) {
      s_part[par][sw][0][wl] = dot;
      s_part[par][sw][1][wl] = nrm;
    }
    __syncthreads();
    // every thread walks the group's slots in order and so reaches the same decision
    for (int s2 = 0; s2 < S && k0 + s2 <= w; ++s2) {
      float d2 = 0.f, n2 = 0.f;
      for (int x = 0; x < wps; ++x) {
        d2 += s_part[par][s2][0][x];
        n2 += s_part[par][s2][1][x];
      }
      const int kk = k0 + s2, i = a + kk - 1;
      const float lr = ln_ratio_of(A.tab.c1[i], A.tab.c2[i], d2, n2);
      const bool acc = (s_lu[par][s2] <= fminf(0.f, lr)) || (n2 == 0.f);
      if (tid == 0 && A.dbg_lr) A.dbg_lr[(size_t)j * A.dbg_stride + kk - 1] = lr;
      if (!acc && n == w) {
        n = kk - 1;
        rej_dot = d2;
        rej_nrm = n2;
        break;
      }
    }
  }

  // the drift rows an in-order walk in groups of S slots reads: up to the end of the group with the first rejection
  // (what the slots kernel really read depends on which of its blocks could leave early; never less than this)
  int rows_read = 0;
  if (w >= 2) rows_read = (n == w || A.all_slots) ? w - 1 : min(2 + ((n + 1 - 2) / S) * S + S - 1, w) - 1;

  float* yrow = A.y + (size_t)j * A.d;
  if (n < w) {
    // reject at slot n + 1: target mean m = y^_n + eta g_n, reflected noise
    const int i = a + n;
    const float eta = A.tab.eta[i], sig = A.tab.sig[i];
    const float coef = 2.f * rej_dot / rej_nrm;
    const float* base = A.Yhat + (size_t)(row0 + n - 1) * A.d;  // n >= 1 always
    const float* grow = A.G + (size_t)(row0 + n - 1) * A.d;
    for (int q = tid; q < A.nq; q += blockDim.x) {
      const float4 b = load4(base, q, A.d, A.vec);
      const float4 g = load4(grow, q, A.d, A.vec);
      const float4 v = load4(vrow, q, A.d, A.vec);
      const float4 xi = xi4((uint32_t)q, (uint32_t)(i + 1), chain, A.keys);
      float4 o;
      o.x = fmaf(sig, fmaf(-coef, v.x - g.x, xi.x), fmaf(eta, g.x, b.x));
      o.y = fmaf(sig, fmaf(-coef, v.y - g.y, xi.y), fmaf(eta, g.y, b.y));
      o.z = fmaf(sig, fmaf(-coef, v.z - g.z, xi.z), fmaf(eta, g.z, b.z));
      o.w = fmaf(sig, fmaf(-coef, v.w - g.w, xi.w), fmaf(eta, g.w, b.w));
      store4(yrow, q, A.d, A.vec, o);
    }
  } else {
    // whole window accepted: y_{a+w} = y^_{w-1} + eta v_a + sigma xi_{a+w}
    const int i = a + w - 1;
    const float eta = A.tab.eta[i], sig = A.tab.sig[i];
    const float* base = (w == 1) ? yrow : A.Yhat + (size_t)(row0 + w - 2) * A.d;
    for (int q = tid; q < A.nq; q += blockDim.x) {
      const float4 b = load4(base, q, A.d, A.vec);
      const float4 v = load4(vrow, q, A.d, A.vec);
      const float4 xi = xi4((uint32_t)q, (uint32_t)(i + 1), chain, A.keys);
      float4 o;
      o.x = fmaf(sig, xi.x, fmaf(eta, v.x, b.x));
      o.y = fmaf(sig, xi.y, fmaf(eta, v.y, b.y));
      o.z = fmaf(sig, xi.z, fmaf(eta, v.z, b.z));
      o.w = fmaf(sig, xi.w, fmaf(eta, v.w, b.w));
      store4(yrow, q, A.d, A.vec, o);
    }
  }
  if (A.la) {
    // look-ahead: after a fully accepted window the drift at its last drafted point, evaluated in this
    // round's batched pass, is v_a of the next round (Algorithm 1's first model call at y_{a+w})
    const bool reuse = (n == w) && (a + w < A.K);
    __syncthreads();  // vrow may be this chain's saved row: every thread is done with it
    if (reuse) {
      const float* glast = A.G + (size_t)(row0 + w - 1) * A.d;
      float* dst = A.vsave + (size_t)j * A.d;
      for (int q = tid; q < A.nq; q += blockDim.x) store4(dst, q, A.d, A.vec, load4(glast, q, A.d, A.vec));
    }
    if (tid == 0) A.has_v[j] = reuse ? 1 : 0;
  }
  if (A.traj) {
    // Algorithm 1's return value: the accepted proposal samples y^_{a+1} .. and, last, the new state
    // (the reflected sample, or the end of a fully accepted window) become y_{a+1} .. y_{a+adv}
    const int adv = (n < w) ? n + 1 : w;
    float* tbase = A.traj + ((size_t)j * (A.K + 1) + a) * A.d;
    __syncthreads();  // this block's stores to yrow are visible to all its threads
    for (int k = 1; k <= adv; ++k) {
      const float* src = (k < adv) ? A.Yhat + (size_t)(row0 + k - 1) * A.d : yrow;
      float* dst = tbase + (size_t)k * A.d;
      for (int e = tid; e < A.d; e += blockDim.x) dst[e] = src[e];
    }
  }
  if (tid == 0) {
    const int adv = (n < w) ? n + 1 : w;
    A.a[j] = a + adv;
    A.rounds[j] += 1;
    A.acc_len[j] = n;
    if (A.hist) atomicAdd(&A.hist[n], 1ull);
    if (A.wnd) {
      // next speculation length of this chain: 2 + 1.5 x running mean of the steps it advances per round
      const int e8 = (A.ema8[j] + 8 * adv) >> 1;
      A.ema8[j] = e8;
      A.wnd[j] = max(2, min(A.window, 2 + (3 * e8) / 16));
    }
    atomicAdd(&A.cnt->accepted, (unsigned long long)adv);
    atomicAdd(&A.cnt->rows_verified, (unsigned long long)rows_read);
    if (a + adv < A.K) atomicAdd(&A.cnt->n_active_after, 1);
  }
}

// How many slots after slot 1 go through the slots kernel (all chains and slot groups side by side): the whole
// window, except for rows of a few hundred floats, where the extra launch would cost more than it saves and the
// verify kernel walks the slots itself.  ASD_VERIFY_HORIZON (read at asd_create) overrides it for experiments.
int verify_horizon(const Ctx* c, int n, int window) {
  (void)n;
  if (window < 2) return 0;
  if (c->debug_all_slots) return window - 1;  // that mode tests every slot, which only the slots kernel does
  if (c->verify_horizon >= 0) return std::min(c->verify_horizon, window - 1);
  if (c->d < 256) return 0;
  return window - 1;
}

void launch_verify(Ctx* c, const Lane& L, int window, bool use_u, const float* G, const float* v_base,
                   const int* v_off_dev) {
  if (L.n == 0) return;
  const int* wnd = round_windows(c, window);
  VerifyArgs A{};
  A.d = c->d;
  A.K = c->K;
  A.window = window;
  A.nq = (c->d + 3) / 4;
  A.vec = (c->d % 4 == 0);
  A.use_u = use_u;
  A.all_slots = c->debug_all_slots ? 1 : 0;
  A.dbg_stride = c->window;
  A.wnd = wnd ? const_cast<int*>(wnd) + L.start : nullptr;
  A.ema8 = c->ema8 + L.start;
  A.keys = make_philox_keys(c->seed);
  A.chain_base = c->chain_base + (uint64_t)L.start;
  A.cnt = L.counters;
  A.act = L.act;
  A.a = c->a + L.start;
  A.rounds = c->rounds + L.start;
  A.row_off = L.row_off;
  A.y = c->y + (size_t)L.start * c->d;
  A.v = v_base;
  A.v_off = v_off_dev;
  A.la = (c->lookahead && L.idx1) ? 1 : 0;
  A.idx1 = L.idx1;
  A.vsave = c->vsave;
  A.has_v = c->has_v;
  A.Yhat = c->Yhat;
  A.G = G;
  A.tab = c->tab;
  A.dbg_lr = c->dbg_lr ? c->dbg_lr + (size_t)L.start * c->window : nullptr;
  A.dbg_lu = c->dbg_lu ? c->dbg_lu + (size_t)L.start * c->window : nullptr;
  A.acc_len = c->acc_len + L.start;
  A.traj = c->traj ? c->traj + (size_t)L.start * (c->K + 1) * c->d : nullptr;
  A.hist = c->hist;
  // eight warps per chain; a slot is reduced by two warps when a row has >= 512 float4 groups, else by one
  A.wps = A.nq >= 512 ? 2 : 1;
  A.horizon = verify_horizon(c, L.n, window);
  A.slot_dot = c->slot_dot + (size_t)L.start * c->window;
  A.slot_nrm = c->slot_nrm + (size_t)L.start * c->window;
  A.slot_lu = c->slot_lu + (size_t)L.start * c->window;
  A.first_rej = c->first_rej + L.start;
  if (A.horizon > 0) {
    const int S = kVerifyMaxWarps / A.wps;
    launch_pdl(c, verify_slots_kernel, dim3(L.n, (A.horizon + S - 1) / S), dim3(256), 0, A);
  }
  launch_pdl(c, verify_kernel, dim3(L.n), dim3(256), 0, A);
}

// ---------------------------------------------------------------------------------------------
// Closed-form posterior means (Eq. 4), one warp (mixture) or one block (Gaussian) per point.
// ---------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(128) gmm_kernel(RowSet rs, int d, GmmParams P, const float* __restrict__ tt,
                                                  float* __restrict__ out) {
  pdl_wait_then_release();
  extern __shared__ float s_logit[];  // [warps][n_comp]
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, wpb = blockDim.x >> 5;
  float* lg = s_logit + warp * P.n_comp;
  const int n_rows = *rs.n_rows_dev;
  for (int r = blockIdx.x * wpb + warp; r < n_rows; r += gridDim.x * wpb)
    gmm_point(rs.ysrc + (size_t)(rs.row_map ? rs.row_map[r] : r) * d, tt[rs.row_step[r]], d, P, lg, out + (size_t)r * d, lane);
}

void launch_gmm(Ctx* c, const RowSet& rs, float* out) {
  if (rs.n_rows_max <= 0) return;
  const int threads = 128, wpb = threads / 32;
  int blocks = (rs.n_rows_max + wpb - 1) / wpb;
  blocks = blocks > 8 * c->num_sms ? 8 * c->num_sms : blocks;
  launch_pdl(c, gmm_kernel, dim3(blocks), dim3(threads), wpb * c->gmm.n_comp * sizeof(float), rs, c->d, c->gmm, c->tab.tt, out);
}

__global__ void __launch_bounds__(128) gauss_kernel(RowSet rs, int d, GaussParams P, const float* __restrict__ tt,
                                                    float* __restrict__ out) {
  pdl_wait_then_release();
  extern __shared__ float s_buf[];  // y[d], w[d]
  float* ys = s_buf;
  float* ws = s_buf + d;
  const int n_rows = *rs.n_rows_dev;
  for (int r = blockIdx.x; r < n_rows; r += gridDim.x) {
    const float* y = rs.ysrc + (size_t)(rs.row_map ? rs.row_map[r] : r) * d;
    const float t = tt[rs.row_step[r]];
    for (int k = threadIdx.x; k < d; k += blockDim.x) ys[k] = y[k];
    __syncthreads();
    for (int jj = threadIdx.x; jj < d; jj += blockDim.x) ws[jj] = gauss_coord(P.Q, ys, d, jj, P.qmu[jj], P.lam[jj], t);
    __syncthreads();
    for (int i = threadIdx.x; i < d; i += blockDim.x) out[(size_t)r * d + i] = gauss_out(P.Qt, ws, d, i);
    __syncthreads();
  }
}

void launch_gauss(Ctx* c, const RowSet& rs, float* out) {
  if (rs.n_rows_max <= 0) return;
  int blocks = rs.n_rows_max > 16 * c->num_sms ? 16 * c->num_sms : rs.n_rows_max;
  const int threads = c->d >= 128 ? 128 : 64;
  launch_pdl(c, gauss_kernel, dim3(blocks), dim3(threads), 2 * c->d * sizeof(float), rs, c->d, c->gauss, c->tab.tt, out);
}

// ---------------------------------------------------------------------------------------------
// Network input rows for an arbitrary row set: [bf16(c_in y) ; cond ; temb ; 0].
// ---------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256) pack_kernel(RowSet rs, int d, MlpParams M, const float* __restrict__ c_in) {
  pdl_wait_then_release();
  const int n_rows = *rs.n_rows_dev;
  for (int r = blockIdx.x; r < n_rows; r += gridDim.x) {
    const float* y = rs.ysrc + (size_t)(rs.row_map ? rs.row_map[r] : r) * d;
    const int step = rs.row_step[r];
    const float ci = c_in[step];
    __nv_bfloat16* xr = M.X + (size_t)r * M.in_pad;
    for (int e = threadIdx.x; e < M.in_pad; e += blockDim.x) {
      __nv_bfloat16 val = __float2bfloat16_rn(0.f);
      if (e < d)
        val = __float2bfloat16_rn(ci * y[e]);
      else if (e < d + M.d_cond)
        val = M.cond[(size_t)rs.row_slot[r] * M.d_cond + (e - d)];
      else if (e < M.in_dim)
        val = M.temb[(size_t)step * M.d_temb + (e - d - M.d_cond)];
      xr[e] = val;
    }
  }
}

void launch_pack(Ctx* c, const RowSet& rs) {
  if (rs.n_rows_max <= 0) return;
  int blocks = rs.n_rows_max > 8 * c->num_sms ? 8 * c->num_sms : rs.n_rows_max;
  launch_pdl(c, pack_kernel, dim3(blocks), dim3(256), 0, rs, c->d, c->mlp, c->tab.c_in);
}

// ---------------------------------------------------------------------------------------------
// Pass-1 rows of one lane appended behind the drafted rows of the other (staggered lanes): the point y_a
// of active chain p becomes row *row_base + p of the drafted-point buffer, with its network input row,
// step and slot, so that one GEMM pass serves both lanes.
// ---------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256) pack_appended_kernel(const RoundCounters* __restrict__ cnt, const int* __restrict__ act,
                                                            const int* __restrict__ a, const float* __restrict__ y,
                                                            const int* __restrict__ row_base, int* __restrict__ m_merged,
                                                            int* __restrict__ v_off, int d, MlpParams M,
                                                            const __nv_bfloat16* __restrict__ cond,
                                                            const float* __restrict__ c_in, float* __restrict__ Yhat,
                                                            int* __restrict__ row_step, int* __restrict__ row_slot) {
  const int n_active = cnt->n_active, base = *row_base;
  if (blockIdx.x == 0 && threadIdx.x == 0) {
    *m_merged = base + n_active;
    *v_off = base;
  }
  for (int p = blockIdx.x; p < n_active; p += gridDim.x) {
    const int j = act[p], step = a[j], row = base + p;
    const float* yj = y + (size_t)j * d;
    const float ci = c_in[step];
    float* yr = Yhat + (size_t)row * d;
    __nv_bfloat16* xr = M.X + (size_t)row * M.in_pad;
    for (int e = threadIdx.x; e < M.in_pad; e += blockDim.x) {
      __nv_bfloat16 val = __float2bfloat16_rn(0.f);
      if (e < d) {
        const float yv = yj[e];
        yr[e] = yv;
        val = __float2bfloat16_rn(ci * yv);
      } else if (e < d + M.d_cond) {
        val = cond[(size_t)j * M.d_cond + (e - d)];
      } else if (e < M.in_dim) {
        val = M.temb[(size_t)step * M.d_temb + (e - d - M.d_cond)];
      }
      xr[e] = val;
    }
    if (threadIdx.x == 0) {
      row_step[row] = step;
      row_slot[row] = j;
    }
  }
}

void launch_pack_appended(Ctx* c, const Lane& L, const int* row_base_dev, int* m_merged_dev) {
  int blocks = std::max(1, std::min(L.n, 8 * c->num_sms));
  pack_appended_kernel<<<blocks, 256, 0, c->stream>>>(L.counters, L.act, c->a + L.start, c->y + (size_t)L.start * c->d,
                                                      row_base_dev, m_merged_dev, L.v_off, c->d, c->mlp,
                                                      c->mlp.cond + (size_t)L.start * c->mlp.d_cond, c->tab.c_in, c->Yhat,
                                                      c->row_step, c->row_slot);
  c->launches++;
}

// Trajectory bookkeeping: the state a chain is (re)started from is row a of its trajectory.
__global__ void traj_seed_kernel(const int* __restrict__ a, const float* __restrict__ y, float* __restrict__ traj, int n,
                                 int K, int d) {
  for (int j = blockIdx.x; j < n; j += gridDim.x) {
    const int aj = min(max(a[j], 0), K);
    float* dst = traj + ((size_t)j * (K + 1) + aj) * d;
    for (int e = threadIdx.x; e < d; e += blockDim.x) dst[e] = y[(size_t)j * d + e];
  }
}

void launch_traj_seed(Ctx* c) {
  if (!c->traj || c->n <= 0) return;
  traj_seed_kernel<<<std::min(c->n, 8 * c->num_sms), 256, 0, c->stream>>>(c->a, c->y, c->traj, c->n, c->K, c->d);
  c->launches++;
}

struct ResetArgs {
  int n, max_chains, d, d_cond, K, hist_len, wnd0, ema0;
  const float* y0;
  const float* cond;
  float* y;
  int* a;
  int* rounds;
  int* acc_len;
  int* wnd;
  int* ema8;
  int* has_v;
  __nv_bfloat16* cond_bf16;
  RoundCounters* counters;  // [2]
  unsigned long long* hist;
  float* traj;
};

__global__ void __launch_bounds__(256) reset_kernel(const ResetArgs A) {
  const size_t tid = blockIdx.x * (size_t)blockDim.x + threadIdx.x, nt = (size_t)gridDim.x * blockDim.x;
  const size_t nd = (size_t)A.n * A.d;
  for (size_t e = tid; e < nd; e += nt) {
    const float v = A.y0 ? A.y0[e] : 0.f;
    A.y[e] = v;
    if (A.traj) {
      const size_t j = e / A.d, k = e - j * A.d;
      A.traj[j * (size_t)(A.K + 1) * A.d + k] = v;  // row 0 of chain j
    }
  }
  for (size_t j = tid; j < (size_t)A.max_chains; j += nt) {
    A.a[j] = 0;
    A.rounds[j] = 0;
    A.acc_len[j] = -1;
    A.wnd[j] = A.wnd0;
    A.ema8[j] = A.ema0;
    if (A.has_v) A.has_v[j] = 0;
  }
  for (size_t e = tid; e < (size_t)A.hist_len; e += nt) A.hist[e] = 0ull;
  const size_t nc = (size_t)A.n * A.d_cond;
  for (size_t e = tid; e < nc; e += nt) A.cond_bf16[e] = __float2bfloat16_rn(A.cond[e]);
  if (tid < 2) {
    const int err = A.counters[tid].err;  // a pending device error survives until the host has read it
    RoundCounters z{};
    z.err = err;
    A.counters[tid] = z;
  }
}

void launch_reset(Ctx* c, const float* y0_dev, const float* cond_dev) {
  ResetArgs A{};
  A.n = c->n;
  A.max_chains = c->max_chains;
  A.d = c->d;
  A.d_cond = (c->kind == ASD_DEN_RESMLP_BF16 && cond_dev) ? c->mlp.d_cond : 0;
  A.K = c->K;
  A.hist_len = c->window + 1;
  A.ema0 = 32;  // adaptive mode starts every chain at 8 x mean = 32, i.e. a speculation length of min(window, 8)
  A.wnd0 = std::max(2, std::min(c->window, 2 + (3 * A.ema0) / 16));
  A.y0 = y0_dev;
  A.cond = cond_dev;
  A.y = c->y;
  A.a = c->a;
  A.rounds = c->rounds;
  A.acc_len = c->acc_len;
  A.wnd = c->wnd;
  A.ema8 = c->ema8;
  A.has_v = c->has_v;
  A.cond_bf16 = const_cast<__nv_bfloat16*>(c->mlp.cond);
  A.counters = c->counters;
  A.hist = c->hist;
  A.traj = c->traj;
  const size_t work = std::max<size_t>((size_t)c->n * c->d, (size_t)c->max_chains);
  const int blocks = (int)std::min<size_t>((work + 255) / 256, (size_t)8 * c->num_sms);
  reset_kernel<<<std::max(blocks, 1), 256, 0, c->stream>>>(A);
  c->launches++;
}

// End of a run: block 0 reduces the chains' round counters, the others copy the results out.
__global__ void __launch_bounds__(256) finish_kernel(const float* __restrict__ y, const int* __restrict__ rounds, int n, int d,
                                                     float* __restrict__ y_out, int* __restrict__ rounds_out,
                                                     RoundCounters* __restrict__ cnt) {
  if (blockIdx.x == 0) {
    __shared__ unsigned long long s_sum[8];
    __shared__ int s_max[8];
    unsigned long long sum = 0ull;
    int mx = 0;
    for (int j = threadIdx.x; j < n; j += blockDim.x) {
      const int r = rounds[j];
      sum += (unsigned long long)r;
      mx = max(mx, r);
      if (rounds_out) rounds_out[j] = r;
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      sum += __shfl_xor_sync(0xffffffffu, sum, o);
      mx = max(mx, __shfl_xor_sync(0xffffffffu, mx, o));
    }
    if ((threadIdx.x & 31) == 0) {
      s_sum[threadIdx.x >> 5] = sum;
      s_max[threadIdx.x >> 5] = mx;
    }
    __syncthreads();
    if (threadIdx.x == 0) {
      for (int x = 1; x < 8; ++x) {
        sum += s_sum[x];
        mx = max(mx, s_max[x]);
      }
      cnt->rounds_sum = sum;
      cnt->rounds_max = mx;
    }
    if (gridDim.x > 1) return;
  }
  if (!y_out) return;
  const size_t nd = (size_t)n * d;
  const size_t b0 = gridDim.x > 1 ? blockIdx.x - 1 : 0, nb = gridDim.x > 1 ? gridDim.x - 1 : 1;
  for (size_t e = b0 * blockDim.x + threadIdx.x; e < nd; e += nb * blockDim.x) y_out[e] = y[e];
}

void launch_finish(Ctx* c, float* y_out_dev, int* rounds_out_dev) {
  const size_t nd = (size_t)c->n * c->d;
  const int copy_blocks = y_out_dev ? (int)std::min<size_t>((nd + 255) / 256, (size_t)8 * c->num_sms) : 0;
  finish_kernel<<<1 + (nd > 4096 ? copy_blocks : 0), 256, 0, c->stream>>>(c->y, c->rounds, c->n, c->d, y_out_dev,
                                                                         rounds_out_dev, c->counters);
  c->launches++;
}

}  // namespace asd

// Chain-resident round driver for the closed-form drifts (Eq. 4: mixture and Gaussian targets).
//
// Chains are independent and a round of these drifts is a few thousand flops per window slot, so nothing
// forces a kernel boundary between the steps of Algorithm 1: ONE block owns ONE chain and runs the while
// loop to the end of the grid (or for a given number of rounds) inside a single launch - drift at the
// current point, draft of the window, drift at every drafted point, Verifier (Algorithms 2 and 3),
// reflection, advance - with the chain's state, its window of noise, drafted points and drifts in shared
// memory.  Every expression is evaluated in the order of the per-phase kernels (asd_kernels.cu), with the
// shared device functions of asd_device.cuh, so a run gives the same bits either way.
#include <algorithm>

#include "asd_device.cuh"
#include "asd_internal.h"

namespace asd {

namespace {

constexpr int kResThreads = 256;
constexpr int kResWarps = kResThreads / 32;
constexpr int kResMaxSmem = 200 * 1024;
constexpr int kResTabSmem = 100 * 1024;  // with all steps' tables resident: two blocks per SM still fit

struct ResidentArgs {
  int d, dp, nq, vec, K, window, wcap, use_u, all_slots, max_rounds, n;
  int k_tab;  // K when the tables of all steps stay in shared memory, else 0
  PhiloxKeys keys;
  uint64_t chain_base;
  int* a;
  int* rounds;
  float* y;
  int* wnd;   // per-chain speculation length (adaptive mode), or null
  int* ema8;
  Tables tab;
  GmmParams gmm;
  GaussParams gauss;
  int* acc_len;
  float* dbg_lr;  // diagnostics of the last round run (ASD_FLAG_DEBUG_DUMP), or null
  float* dbg_lu;
  int dbg_stride;
  float* traj;               // [n, K + 1, d], or null
  unsigned long long* hist;  // [window + 1]
  RoundCounters* cnt;
};

// Shared-memory layout in floats; the vector arrays first (rows of dp = 4 nq floats, 16-byte aligned).
struct ResidentLayout {
  int y, v, xi, yh, g, lu, dot, nrm, tab, extra, total;
};

// k_tab > 0: the per-step tables of all k_tab steps stay in shared memory for the whole launch (the window's
// tables are then views into them); 0: the window's entries are copied in every round.
__host__ __device__ inline ResidentLayout resident_layout(int kind, int d, int dp, int wcap, int n_comp, int k_tab) {
  ResidentLayout L;
  int o = 0;
  L.y = o;    o += dp;
  L.v = o;    o += dp;
  L.xi = o;   o += wcap * dp;   // xi of slots 1..w
  L.yh = o;   o += wcap * dp;   // drafted points of slots 1..w-1
  L.g = o;    o += wcap * dp;   // drift at the drafted points
  const int wp = (wcap + 4) & ~3;
  L.lu = o;   o += wp;
  L.dot = o;  o += wp;
  L.nrm = o;  o += wp;
  L.tab = o;  o += 5 * (k_tab > 0 ? ((k_tab + 4) & ~3) : wp);  // eta, sigma, c1, c2, t of the window's (or all) steps
  L.extra = o;
  if (kind == ASD_DEN_GAUSS_LINEAR)
    o += 2 * dp * d + ((2 * d + 3) & ~3) + wcap * dp;  // Q, Qt (groups of four terms), qmu, lam (padded to 16 bytes), eigen-coordinates per point
  else
    o += kResWarps * n_comp + n_comp * (d + 2);  // the warps' logits; means, ln pi, |c|^2
  L.total = o;
  return L;
}

// The Gaussian's Q and Q^T in shared memory: the four matrix elements that one step of dot_strided4 multiplies sit side by
// side, element (i, jj) of the matrix at float (i / 4 * d + jj) * 4 + i % 4 (rows past d are zero and never used), so a
// thread fetches the four terms of its column with one 16-byte load and four neighbouring lanes fetch one term each
// without a bank conflict.
struct ResidentGauss {
  const float4 *Q4, *Qt4;
  const float *qmu, *lam;
  float* ws;
};
__device__ __forceinline__ ResidentGauss resident_gauss_views(const ResidentArgs& A, const float* sm, const ResidentLayout& L) {
  ResidentGauss G;
  G.Q4 = reinterpret_cast<const float4*>(sm + L.extra);
  G.Qt4 = G.Q4 + (size_t)A.nq * A.d;
  G.qmu = reinterpret_cast<const float*>(G.Qt4 + (size_t)A.nq * A.d);
  G.lam = G.qmu + A.d;
  G.ws = const_cast<float*>(G.qmu) + ((2 * A.d + 3) & ~3);  // rows of dp floats, read 16 bytes at a time
  return G;
}

// Two IEEE fused multiply-adds in one instruction (sm_100 packed fp32): acc.x = fma(a.x, b.x, acc.x), acc.y likewise;
// each half rounds exactly as fmaf does.
__device__ __forceinline__ void fma2(float& acc_x, float& acc_y, float ax, float ay, float bx, float by) {
  asm("{\n\t.reg .b64 pa, pb, pc;\n\t"
      "mov.b64 pa, {%2, %3};\n\tmov.b64 pb, {%4, %5};\n\tmov.b64 pc, {%0, %1};\n\t"
      "fma.rn.f32x2 pc, pa, pb, pc;\n\t"
      "mov.b64 {%0, %1}, pc;\n\t}"
      : "+f"(acc_x), "+f"(acc_y)
      : "f"(ax), "f"(ay), "f"(bx), "f"(by));
}

// Gaussian posterior mean of n_pts points (rows of dp floats in shared memory) by the whole block.
// One item = one eigen-coordinate (then one output coordinate) of a group of kPts points: the matrix elements are
// loaded once for the group and the points' sums run side by side, each in the order of dot_strided4 (four
// interleaved partial sums), so the bits are those of gauss_coord / gauss_out point by point.
template <int kPts>
__device__ __forceinline__ void resident_gauss(const ResidentArgs& A, const float* sm, const ResidentLayout& L,
                                               const float* src, float* dst, int n_pts, const float* s_t) {
  const int tid = threadIdx.x, d = A.d;
  const ResidentGauss G = resident_gauss_views(A, sm, L);
  const int groups = (n_pts + kPts - 1) / kPts;
  const int n4 = d >> 2, d4 = d & ~3;
  for (int it = tid; it < groups * d; it += kResThreads) {
    const int pg = it / d, jj = it - pg * d, p0 = pg * kPts;
    const int np = min(kPts, n_pts - p0);
    const float* y0 = src + (size_t)p0 * A.dp;
    float z[kPts][4];
#pragma unroll
    for (int u = 0; u < kPts; ++u) z[u][0] = z[u][1] = z[u][2] = z[u][3] = 0.f;
#pragma unroll 4
    for (int i4 = 0; i4 < n4; ++i4) {  // four terms per 16-byte load of the matrix and of each point (broadcast)
      const float4 q = G.Q4[i4 * d + jj];
#pragma unroll
      for (int u = 0; u < kPts; ++u) {
        const float4 yv = *reinterpret_cast<const float4*>(y0 + (size_t)min(u, np - 1) * A.dp + 4 * i4);
        fma2(z[u][0], z[u][1], q.x, q.y, yv.x, yv.y);
        fma2(z[u][2], z[u][3], q.z, q.w, yv.z, yv.w);
      }
    }
    if (d4 < d) {  // the last d mod 4 terms
      const float4 q = G.Q4[n4 * d + jj];
      const float qr[3] = {q.x, q.y, q.z};
#pragma unroll
      for (int r = 0; r < 3; ++r) {
        if (d4 + r < d) {
#pragma unroll
          for (int u = 0; u < kPts; ++u) z[u][r] = fmaf(qr[r], y0[(size_t)min(u, np - 1) * A.dp + d4 + r], z[u][r]);
        }
      }
    }
    const float qmu = G.qmu[jj], lam = G.lam[jj];
#pragma unroll
    for (int u = 0; u < kPts; ++u)
      if (u < np) G.ws[(size_t)(p0 + u) * A.dp + jj] = __fdiv_rn(fmaf(lam, sum4(z[u]), qmu), fmaf(s_t[p0 + u], lam, 1.f));
  }
  __syncthreads();
  for (int it = tid; it < groups * d; it += kResThreads) {
    const int pg = it / d, i = it - pg * d, p0 = pg * kPts;
    const int np = min(kPts, n_pts - p0);
    const float* w0 = G.ws + (size_t)p0 * A.dp;
    float m[kPts][4];
#pragma unroll
    for (int u = 0; u < kPts; ++u) m[u][0] = m[u][1] = m[u][2] = m[u][3] = 0.f;
#pragma unroll 4
    for (int j4 = 0; j4 < n4; ++j4) {
      const float4 q = G.Qt4[j4 * d + i];
#pragma unroll
      for (int u = 0; u < kPts; ++u) {
        const float4 wv = *reinterpret_cast<const float4*>(w0 + (size_t)min(u, np - 1) * A.dp + 4 * j4);
        fma2(m[u][0], m[u][1], q.x, q.y, wv.x, wv.y);
        fma2(m[u][2], m[u][3], q.z, q.w, wv.z, wv.w);
      }
    }
    if (d4 < d) {
      const float4 q = G.Qt4[n4 * d + i];
      const float qr[3] = {q.x, q.y, q.z};
#pragma unroll
      for (int r = 0; r < 3; ++r) {
        if (d4 + r < d) {
#pragma unroll
          for (int u = 0; u < kPts; ++u) m[u][r] = fmaf(qr[r], w0[(size_t)min(u, np - 1) * A.dp + d4 + r], m[u][r]);
        }
      }
    }
#pragma unroll
    for (int u = 0; u < kPts; ++u)
      if (u < np) dst[(size_t)(p0 + u) * A.dp + i] = sum4(m[u]);
  }
  __syncthreads();
}

// One partial sum of dot_strided4 per lane: lane c of a group of four takes the terms c, c + 4, ... of column `col`
// in their order, and two exchanges add the partial sums as sum4 does, (s0 + s1) + (s2 + s3) (IEEE addition commutes,
// so every lane of the group ends with the same bits).  All 32 lanes must call it.
__device__ __forceinline__ float resident_quarter_dot(const float* M, const float* vec, int d, int col, int c) {
  const int n4 = d >> 2;
  float s = 0.f;
#pragma unroll 8
  for (int i4 = 0; i4 < n4; ++i4) s = fmaf(M[((size_t)i4 * d + col) * 4 + c], vec[4 * i4 + c], s);
  if (4 * n4 + c < d) s = fmaf(M[((size_t)n4 * d + col) * 4 + c], vec[4 * n4 + c], s);
  s = __fadd_rn(s, __shfl_xor_sync(0xffffffffu, s, 1));
  return __fadd_rn(s, __shfl_xor_sync(0xffffffffu, s, 2));
}

// The Gaussian posterior mean of ONE point at time t by the whole block: a chain of d / 4 dependent multiply-adds
// per lane instead of d, with the bits of gauss_coord / gauss_out.
__device__ __forceinline__ void resident_gauss_one(const ResidentArgs& A, const float* sm, const ResidentLayout& L,
                                                   const float* src, float* dst, float t) {
  const int tid = threadIdx.x, d = A.d, c = tid & 3;
  const ResidentGauss G = resident_gauss_views(A, sm, L);
  for (int base = 0; base < d; base += kResThreads / 4) {
    const int jj = base + (tid >> 2), jc = min(jj, d - 1);
    const float z = resident_quarter_dot(reinterpret_cast<const float*>(G.Q4), src, d, jc, c);
    if (c == 0 && jj < d) {
      const float lam = G.lam[jj];
      G.ws[jj] = __fdiv_rn(fmaf(lam, z, G.qmu[jj]), fmaf(t, lam, 1.f));
    }
  }
  __syncthreads();
  for (int base = 0; base < d; base += kResThreads / 4) {
    const int i = base + (tid >> 2), ic = min(i, d - 1);
    const float m = resident_quarter_dot(reinterpret_cast<const float*>(G.Qt4), G.ws, d, ic, c);
    if (c == 0 && i < d) dst[i] = m;
  }
  __syncthreads();
}

template <int KIND>
__device__ __forceinline__ void resident_drift(const ResidentArgs& A, const float* sm, const ResidentLayout& L,
                                               const float* src, float* dst, int n_pts, const float* s_t, float t_one) {
  // dst[p] = g(s_t[p], src[p]) for p < n_pts (rows of dp floats; s_t: the points' times); ends with a block barrier.
  // A single point takes its time from t_one, and s_t is not read before the first block barrier inside.
  if (KIND == ASD_DEN_GMM_ISO) {
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    float* lg = const_cast<float*>(sm) + L.extra + warp * A.gmm.n_comp;
    GmmParams P = A.gmm;  // the copy in shared memory
    P.means = sm + L.extra + kResWarps * A.gmm.n_comp;
    P.log_pi = P.means + (size_t)A.gmm.n_comp * A.d;
    P.cnorm = P.log_pi + A.gmm.n_comp;
    for (int p = warp; p < n_pts; p += kResWarps)
      gmm_point(src + (size_t)p * A.dp, n_pts == 1 ? t_one : s_t[p], A.d, P, lg, dst + (size_t)p * A.dp, lane);
    __syncthreads();
  } else if (n_pts == 1) {
    resident_gauss_one(A, sm, L, src, dst, t_one);
  } else if (n_pts * A.d <= kResThreads) {
    resident_gauss<1>(A, sm, L, src, dst, n_pts, s_t);  // few points: an item per thread is already all there is
  } else {
    resident_gauss<4>(A, sm, L, src, dst, n_pts, s_t);
  }
}

template <int KIND>
__global__ void __launch_bounds__(kResThreads) resident_kernel(const ResidentArgs A) {
  extern __shared__ float4 smem4[];
  float* sm = reinterpret_cast<float*>(smem4);
  __shared__ int s_first[kResWarps];
  const int j = blockIdx.x;
  if (j >= A.n) return;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  int a = A.a[j];
  if (a >= A.K) {
    if (tid == 0) A.acc_len[j] = -1;
    return;
  }
  const ResidentLayout L = resident_layout(KIND, A.d, A.dp, A.wcap, A.gmm.n_comp, A.k_tab);
  float* sy = sm + L.y;
  float* sv = sm + L.v;
  float4* sXi4 = reinterpret_cast<float4*>(sm + L.xi);
  float4* sYh4 = reinterpret_cast<float4*>(sm + L.yh);
  float4* sG4 = reinterpret_cast<float4*>(sm + L.g);
  float* s_lu = sm + L.lu;
  float* s_dot = sm + L.dot;
  float* s_nrm = sm + L.nrm;
  const int wp = A.k_tab > 0 ? ((A.k_tab + 4) & ~3) : ((A.wcap + 4) & ~3);
  float* const tab_eta = sm + L.tab;
  float* const tab_sig = tab_eta + wp;
  float* const tab_c1 = tab_sig + wp;
  float* const tab_c2 = tab_c1 + wp;
  float* const tab_t = tab_c2 + wp;
  const int nq = A.nq, d = A.d;
  const uint32_t chain = (uint32_t)(A.chain_base + (uint64_t)j);

  // the chain's state, padded with zeros up to dp, and the target's parameters
  for (int e = tid; e < A.dp; e += kResThreads) {
    sy[e] = e < d ? A.y[(size_t)j * d + e] : 0.f;
    sv[e] = 0.f;
  }
  if (KIND == ASD_DEN_GAUSS_LINEAR) {
    float* sQ = sm + L.extra;
    const int mat = A.dp * d;
    for (int e = tid; e < mat; e += kResThreads) {  // element (i, jj) -> (i / 4 * d + jj) * 4 + i % 4
      const int g = e >> 2, i = 4 * (g / d) + (e & 3), jj = g % d;
      sQ[e] = i < d ? A.gauss.Q[(size_t)i * d + jj] : 0.f;
      sQ[mat + e] = i < d ? A.gauss.Qt[(size_t)i * d + jj] : 0.f;
    }
    for (int e = tid; e < d; e += kResThreads) {
      sQ[2 * mat + e] = A.gauss.qmu[e];
      sQ[2 * mat + d + e] = A.gauss.lam[e];
    }
  } else {
    float* sp = sm + L.extra + kResWarps * A.gmm.n_comp;
    const int nc = A.gmm.n_comp;
    for (int e = tid; e < nc * d; e += kResThreads) sp[e] = A.gmm.means[e];
    for (int e = tid; e < nc; e += kResThreads) {
      sp[nc * d + e] = A.gmm.log_pi[e];
      sp[nc * d + nc + e] = A.gmm.cnorm[e];
    }
  }
  int theta_next = A.wnd ? A.wnd[j] : A.window, ema8 = A.wnd ? A.ema8[j] : 0;
  int r_done = 0, n_last = -1, w_first = 0;
  long long rows_total = 0, rows_ver = 0, adv_total = 0;
  float t_a = A.tab.tt[a];  // t of the current step, carried in a register from round to round
  if (A.k_tab > 0) {
    for (int k = tid; k <= A.K; k += kResThreads) {
      tab_t[k] = A.tab.tt[k];
      if (k < A.K) {
        tab_eta[k] = A.tab.eta[k];
        tab_sig[k] = A.tab.sig[k];
        tab_c1[k] = A.tab.c1[k];
        tab_c2[k] = A.tab.c2[k];
      }
    }
  }
  __syncthreads();

  while (a < A.K && r_done < A.max_rounds) {
    const int theta = A.wnd ? max(1, min(theta_next, A.window)) : A.window;
    const int w = min(theta, A.K - a);  // Algorithm 1: b = min(K, a + theta)
    if (r_done == 0) w_first = w;
    // the window's per-step tables: [k] = eta_{a+k}, sigma_{a+k+1}, c1, c2 for k = 0 .. w-1 and t_{a+k} for k = 0 .. w;
    // views into the resident tables, or one trip to global memory per round under the noise generation
    const int off = A.k_tab > 0 ? a : 0;
    const float *s_eta = tab_eta + off, *s_sig = tab_sig + off, *s_c1 = tab_c1 + off, *s_c2 = tab_c2 + off, *s_t = tab_t + off;
    if (A.k_tab == 0) {
      for (int k = tid; k <= w; k += kResThreads) {
        tab_t[k] = A.tab.tt[a + k];
        if (k < w) {
          tab_eta[k] = A.tab.eta[a + k];
          tab_sig[k] = A.tab.sig[a + k];
          tab_c1[k] = A.tab.c1[a + k];
          tab_c2[k] = A.tab.c2[a + k];
        }
      }
    }
    // xi of every slot of the window (counter-based: the same values in every round that reaches a step)
    for (int it = tid; it < w * nq; it += kResThreads) {
      const int k = it / nq, q = it - k * nq;
      sXi4[it] = xi4((uint32_t)q, (uint32_t)(a + k + 1), chain, A.keys);
    }
    // first model call: v_a = g(t_a, y_a).  It reads the state and t_a only, so no barrier separates it from the
    // noise generation above: its first inner barrier publishes the tables and the noise as well.
    resident_drift<KIND>(A, sm, L, sy, sv, 1, s_t, t_a);
    // ln u of every slot, by the block's last threads while its first ones draft (the accept tests read it two
    // barriers later; in the noise phase it would make one warp the straggler of the first barrier)
    for (int k = 1 + (kResThreads - 1 - tid); k <= w; k += kResThreads) s_lu[k] = A.use_u ? ln_u((uint32_t)(a + k), chain, A.keys) : 0.f;
    // draft: y^_{a+k} = y^_{a+k-1} + eta v_a + sigma xi_{a+k}, k = 1 .. w-1
    if (tid < nq && w > 1) {
      float4 yh = reinterpret_cast<const float4*>(sy)[tid];
      const float4 v = reinterpret_cast<const float4*>(sv)[tid];
      float eta_n = s_eta[0], sig_n = s_sig[0];
      float4 xi_n = sXi4[tid];
      for (int k = 1; k < w; ++k) {
        // the next slot's operands are fetched before this slot's store: the chain then waits on its two multiply-adds only
        const float eta = eta_n, sig = sig_n;
        const float4 xi = xi_n;
        if (k + 1 < w) {
          eta_n = s_eta[k];
          sig_n = s_sig[k];
          xi_n = sXi4[k * nq + tid];
        }
        yh.x = fmaf(sig, xi.x, fmaf(eta, v.x, yh.x));
        yh.y = fmaf(sig, xi.y, fmaf(eta, v.y, yh.y));
        yh.z = fmaf(sig, xi.z, fmaf(eta, v.z, yh.z));
        yh.w = fmaf(sig, xi.w, fmaf(eta, v.w, yh.w));
        sYh4[(k - 1) * nq + tid] = yh;
      }
    }
    __syncthreads();
    // second model call: the drift at every drafted prefix point
    if (w > 1) resident_drift<KIND>(A, sm, L, sm + L.yh, sm + L.g, w - 1, s_t + 1, s_t[1]);
    // Verifier: <xi, delta> and |delta|^2 per slot, one warp per slot, in the reduction order of the verify kernel
    for (int k = 2 + warp; k <= w; k += kResWarps) {
      float dot = 0.f, nrm = 0.f;
      for (int q = lane; q < nq; q += 32) {
        const float4 vv = reinterpret_cast<const float4*>(sv)[q];
        const float4 gg = sG4[(k - 2) * nq + q];
        const float4 xi = sXi4[(k - 1) * nq + q];
        float4 dl = make_float4(vv.x - gg.x, vv.y - gg.y, vv.z - gg.z, vv.w - gg.w);
        if (!A.vec) {
          const int b = 4 * q;
          if (b + 1 >= d) dl.y = 0.f;
          if (b + 2 >= d) dl.z = 0.f;
          if (b + 3 >= d) dl.w = 0.f;
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
      dot = warp_sum(dot);
      nrm = warp_sum(nrm);
      if (lane == 0) {
        // the partial of a one-warp team is added to zero in the verify kernel: x + 0 = x
        s_dot[k] = dot;
        s_nrm[k] = nrm;
      }
    }
    __syncthreads();
    // first rejected slot
    int first = w + 1;
    for (int k = 2 + tid; k <= w; k += kResThreads) {
      const float lr = ln_ratio_of(s_c1[k - 1], s_c2[k - 1], s_dot[k], s_nrm[k]);
      const bool acc = (s_lu[k] <= fminf(0.f, lr)) || (s_nrm[k] == 0.f);
      if (!acc) {
        first = k;
        break;
      }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) first = min(first, __shfl_xor_sync(0xffffffffu, first, o));
    if (lane == 0) s_first[warp] = first;
    __syncthreads();
#pragma unroll
    for (int x = 0; x < kResWarps; ++x) first = min(first, s_first[x]);
    const int n = first <= w ? first - 1 : w;  // accepted prefix length
    const int adv = n < w ? n + 1 : w;
    t_a = s_t[adv];  // = t of step a + adv, the next round's current step
    if (A.dbg_lr) {
      for (int k = 1 + tid; k <= w; k += kResThreads) {
        A.dbg_lu[(size_t)j * A.dbg_stride + k - 1] = s_lu[k];
        A.dbg_lr[(size_t)j * A.dbg_stride + k - 1] = k == 1 ? 0.f : ln_ratio_of(s_c1[k - 1], s_c2[k - 1], s_dot[k], s_nrm[k]);
      }
    }
    // new state
    float4 o = make_float4(0.f, 0.f, 0.f, 0.f);
    if (tid < nq) {
      const float4 v = reinterpret_cast<const float4*>(sv)[tid];
      if (n < w) {
        const float eta = s_eta[n], sig = s_sig[n];
        const float coef = 2.f * s_dot[n + 1] / s_nrm[n + 1];
        const float4 b = sYh4[(n - 1) * nq + tid];  // n >= 1 always (Lemma 1)
        const float4 g = sG4[(n - 1) * nq + tid];
        const float4 xi = sXi4[n * nq + tid];
        o.x = fmaf(sig, fmaf(-coef, v.x - g.x, xi.x), fmaf(eta, g.x, b.x));
        o.y = fmaf(sig, fmaf(-coef, v.y - g.y, xi.y), fmaf(eta, g.y, b.y));
        o.z = fmaf(sig, fmaf(-coef, v.z - g.z, xi.z), fmaf(eta, g.z, b.z));
        o.w = fmaf(sig, fmaf(-coef, v.w - g.w, xi.w), fmaf(eta, g.w, b.w));
      } else {
        const float eta = s_eta[w - 1], sig = s_sig[w - 1];
        const float4 b = (w == 1) ? reinterpret_cast<const float4*>(sy)[tid] : sYh4[(w - 2) * nq + tid];
        const float4 xi = sXi4[(w - 1) * nq + tid];
        o.x = fmaf(sig, xi.x, fmaf(eta, v.x, b.x));
        o.y = fmaf(sig, xi.y, fmaf(eta, v.y, b.y));
        o.z = fmaf(sig, xi.z, fmaf(eta, v.z, b.z));
        o.w = fmaf(sig, xi.w, fmaf(eta, v.w, b.w));
      }
      if (!A.vec) {  // keep the padding at zero
        const int b0 = 4 * tid;
        if (b0 + 1 >= d) o.y = 0.f;
        if (b0 + 2 >= d) o.z = 0.f;
        if (b0 + 3 >= d) o.w = 0.f;
      }
    }
    // (since the draft, the old state has been read by its own thread only: no barrier before the write)
    if (tid < nq) reinterpret_cast<float4*>(sy)[tid] = o;
    __syncthreads();
    if (A.traj) {
      float* tbase = A.traj + ((size_t)j * (A.K + 1) + a) * d;
      for (int k = 1; k <= adv; ++k) {
        const float* src = (k < adv) ? sm + L.yh + (size_t)(k - 1) * A.dp : sy;
        for (int e = tid; e < d; e += kResThreads) tbase[(size_t)k * d + e] = src[e];
      }
    }
    // statistics, in the terms of the per-phase kernels: drift rows made, and drift rows the verify kernel would
    // have read (it walks the slots in groups and stops after the group with the first rejection)
    if (tid == 0) {
      rows_total += w;
      const int S = kResWarps;
      int rr = 0;
      if (w >= 2) rr = (n == w || A.all_slots) ? w - 1 : min(2 + ((n + 1 - 2) / S) * S + S - 1, w) - 1;
      rows_ver += rr;
      adv_total += adv;
      if (A.hist) atomicAdd(&A.hist[n], 1ull);
    }
    if (A.wnd) {
      ema8 = (ema8 + 8 * adv) >> 1;
      theta_next = max(2, min(A.window, 2 + (3 * ema8) / 16));
    }
    a += adv;
    n_last = n;
    ++r_done;
  }

  for (int e = tid; e < d; e += kResThreads) A.y[(size_t)j * d + e] = sy[e];
  if (tid == 0) {
    A.a[j] = a;
    A.rounds[j] += r_done;
    A.acc_len[j] = n_last;
    if (A.wnd) {
      A.wnd[j] = theta_next;
      A.ema8[j] = ema8;
    }
    atomicAdd(&A.cnt->n_active, 1);
    atomicAdd(&A.cnt->n_eval, 1);
    atomicAdd(&A.cnt->rows2, w_first - 1);
    atomicAdd(&A.cnt->accepted, (unsigned long long)adv_total);
    atomicAdd(&A.cnt->rows_total, (unsigned long long)rows_total);
    atomicAdd(&A.cnt->rows_verified, (unsigned long long)rows_ver);
    if (a < A.K) atomicAdd(&A.cnt->n_active_after, 1);
  }
}

// The per-call counters start at zero; the running totals and the error word stay.
__global__ void resident_begin_kernel(RoundCounters* cnt) {
  cnt->n_active = 0;
  cnt->rows2 = 0;
  cnt->n_active_after = 0;
  cnt->n_eval = 0;
  cnt->accepted = 0ull;
}

}  // namespace

// Whether the chain-resident kernel can serve this context (closed-form drift, one-warp reduction teams,
// the window's working set fits shared memory); *smem_bytes receives the dynamic shared memory it needs.
bool resident_supported(const Ctx* c, int window, int* smem_bytes, int* k_tab) {
  if (c->kind != ASD_DEN_GMM_ISO && c->kind != ASD_DEN_GAUSS_LINEAR) return false;
  if (c->lookahead) return false;
  const int nq = (c->d + 3) / 4;
  if (nq >= 512 || nq > kResThreads) return false;
  ResidentLayout L = resident_layout(c->kind, c->d, 4 * nq, std::max(window, 1), c->gmm.n_comp, 0);
  long long bytes = (long long)L.total * 4;
  if (bytes > kResMaxSmem) return false;
  if (k_tab) {
    // all K steps' tables resident when the block still leaves room for a second one on the SM
    *k_tab = 0;
    L = resident_layout(c->kind, c->d, 4 * nq, std::max(window, 1), c->gmm.n_comp, c->K);
    if ((long long)L.total * 4 <= kResTabSmem) {
      *k_tab = c->K;
      bytes = (long long)L.total * 4;
    }
  }
  if (smem_bytes) *smem_bytes = (int)bytes;
  return true;
}

// `max_rounds` iterations of Algorithm 1's while loop (or to the end of the grid) for every chain, one launch.
asd_status launch_resident(Ctx* c, int window, bool use_u, int max_rounds) {
  int smem = 0, k_tab = 0;
  // a launch of a single round (lock-step use) keeps the per-round copy of the window's tables
  if (!resident_supported(c, window, &smem, max_rounds > 1 ? &k_tab : nullptr)) return ASD_ERR_UNSUPPORTED;
  if (c->n <= 0) return ASD_OK;
  ResidentArgs A{};
  A.d = c->d;
  A.nq = (c->d + 3) / 4;
  A.dp = 4 * A.nq;
  A.vec = (c->d % 4 == 0);
  A.K = c->K;
  A.k_tab = k_tab;
  A.window = window;
  A.wcap = std::max(window, 1);
  A.use_u = use_u ? 1 : 0;
  A.all_slots = c->debug_all_slots ? 1 : 0;
  A.max_rounds = max_rounds;
  A.n = c->n;
  A.keys = make_philox_keys(c->seed);
  A.chain_base = c->chain_base;
  A.a = c->a;
  A.rounds = c->rounds;
  A.y = c->y;
  const bool adaptive = c->adaptive && window > 1;
  A.wnd = adaptive ? c->wnd : nullptr;
  A.ema8 = c->ema8;
  A.tab = c->tab;
  A.gmm = c->gmm;
  A.gauss = c->gauss;
  A.acc_len = c->acc_len;
  A.dbg_lr = c->dbg_lr;
  A.dbg_lu = c->dbg_lu;
  A.dbg_stride = c->window;
  A.traj = c->traj;
  A.hist = c->hist;
  A.cnt = c->counters;
  if (max_rounds < 0x7fffffff) {  // a call that reports per-round counters (asd_round) starts them at zero
    resident_begin_kernel<<<1, 1, 0, c->stream>>>(c->counters);
    c->launches++;
  }
  const void* fn = c->kind == ASD_DEN_GMM_ISO ? reinterpret_cast<const void*>(&resident_kernel<ASD_DEN_GMM_ISO>)
                                              : reinterpret_cast<const void*>(&resident_kernel<ASD_DEN_GAUSS_LINEAR>);
  int& have = c->func_smem[fn];
  if (smem > have) {
    if (cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, smem) != cudaSuccess) {
      c->err = "resident kernel: shared-memory opt-in failed";
      return ASD_ERR_CUDA;
    }
    have = smem;
  }
  if (c->kind == ASD_DEN_GMM_ISO)
    resident_kernel<ASD_DEN_GMM_ISO><<<c->n, kResThreads, smem, c->stream>>>(A);
  else
    resident_kernel<ASD_DEN_GAUSS_LINEAR><<<c->n, kResThreads, smem, c->stream>>>(A);
  c->launches++;
  return ASD_OK;
}

}  // namespace asd

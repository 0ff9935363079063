// Device functions shared by the kernels of the ASD round (asd_kernels.cu) and the chain-resident
// kernel (asd_resident.cu): counter-based randomness, vector loads with ragged tails, the window of a
// chain, warp reductions, the accept-test expression and the closed-form posterior means.  Everything that
// two kernels must evaluate to the same bits spells out its roundings (fmaf / __fmul_rn / __fdiv_rn),
// so that the compiler has no contraction choice to make differently in different kernels.
#pragma once

#include "asd_internal.h"

namespace asd {

// Programmatic dependent launch for the small kernels of a round: the kernel may be scheduled while its predecessor in
// the stream is still running; it waits for that kernel's completion before it touches anything, and only then lets
// its own successor be scheduled (a successor that reads a count before its own wait - the weight-streaming GEMM -
// relies on everything up to the kernel before its predecessor being complete once it runs).
__device__ __forceinline__ void pdl_wait_then_release() {
  asm volatile("griddepcontrol.wait;" ::: "memory");
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
}

// ---------------------------------------------------------------------------------------------
// Counter-based randomness (Algorithm 1, "sample u, xi"): Philox4x32-10, counter =
// (dimension block, step, chain id, tag).
// ---------------------------------------------------------------------------------------------
// Round keys of the ten rounds (key + r * Weyl constant), computed once on the host and passed in
// the kernel arguments, so a round is two 32x32->64 multiplies and two three-input xors.
struct PhiloxKeys {
  uint32_t k[20];
};

inline PhiloxKeys make_philox_keys(uint64_t seed) {
  PhiloxKeys K;
  uint32_t k0 = (uint32_t)(seed & 0xffffffffull), k1 = (uint32_t)(seed >> 32);
  for (int r = 0; r < 10; ++r) {
    K.k[2 * r] = k0;
    K.k[2 * r + 1] = k1;
    k0 += 0x9E3779B9u;
    k1 += 0xBB67AE85u;
  }
  return K;
}

__device__ __forceinline__ uint4 philox4x32_10(uint4 c, const PhiloxKeys& K) {
  constexpr uint32_t M0 = 0xD2511F53u, M1 = 0xCD9E8D57u;
#pragma unroll
  for (int r = 0; r < 10; ++r) {
    const uint64_t p0 = (uint64_t)M0 * c.x;
    const uint64_t p1 = (uint64_t)M1 * c.z;
    c = make_uint4((uint32_t)(p1 >> 32) ^ c.y ^ K.k[2 * r], (uint32_t)p1, (uint32_t)(p0 >> 32) ^ c.w ^ K.k[2 * r + 1],
                   (uint32_t)p0);
  }
  return c;
}

// U(r) = ((r >> 9) + 0.5) 2^-23, exactly: the 23 bits become the mantissa of a float in [1, 2) and
// the subtraction of 1 - 2^-24 is exact (the result has 24 significant bits).
__device__ __forceinline__ float uniform_from_word(uint32_t r) {
  return __uint_as_float((r >> 9) | 0x3f800000u) - 0.99999994f;
}

// Box-Muller on the special-function unit: radius = sqrt(-2 ln2 lg2 U(r_even)) with lg2.approx and
// sqrt.approx, angle 2 pi U(r_odd) shifted by -pi into [-pi, pi] (where sin.approx / cos.approx are
// most accurate); the shift negates both outputs, which the sign of the radius undoes.
__device__ __forceinline__ void box_muller(uint32_t r_even, uint32_t r_odd, float& n_even, float& n_odd) {
  // the uniform is at least 2^-24, never denormal: the flush-to-zero forms need no range fix-up around them
  float lg, rad, sn, cs;
  asm("lg2.approx.ftz.f32 %0, %1;" : "=f"(lg) : "f"(uniform_from_word(r_even)));
  asm("sqrt.approx.ftz.f32 %0, %1;" : "=f"(rad) : "f"(-1.3862943611198906f * lg));
  // 2 pi (f - 1 + 2^-24) - pi with f = 1.mantissa in [1, 2)
  const float th = fmaf(__uint_as_float((r_odd >> 9) | 0x3f800000u), 6.283185307179586f, -9.424777586315302f);
  asm("cos.approx.ftz.f32 %0, %1;" : "=f"(cs) : "f"(th));
  asm("sin.approx.ftz.f32 %0, %1;" : "=f"(sn) : "f"(th));
  n_even = -rad * cs;
  n_odd = -rad * sn;
}

// xi_step[4q .. 4q+3]
__device__ __forceinline__ float4 xi4(uint32_t q, uint32_t step, uint32_t chain, const PhiloxKeys& K) {
  const uint4 r = philox4x32_10(make_uint4(q, step, chain, 0u), K);
  float4 n;
  box_muller(r.x, r.y, n.x, n.y);
  box_muller(r.z, r.w, n.z, n.w);
  return n;
}

// ln u_step: evaluated once per slot, with the accurate logarithm (it decides the accept test).
__device__ __forceinline__ float ln_u(uint32_t step, uint32_t chain, const PhiloxKeys& K) {
  const uint4 r = philox4x32_10(make_uint4(0u, step, chain, 1u), K);
  return logf(uniform_from_word(r.x));
}

// Loads / stores of the 4 dims of block q with a ragged tail (d not a multiple of 4).
__device__ __forceinline__ float4 load4(const float* row, int q, int d, bool vec) {
  if (vec) return *reinterpret_cast<const float4*>(row + 4 * q);
  float4 r = make_float4(0.f, 0.f, 0.f, 0.f);
  const int b = 4 * q;
  if (b + 0 < d) r.x = row[b + 0];
  if (b + 1 < d) r.y = row[b + 1];
  if (b + 2 < d) r.z = row[b + 2];
  if (b + 3 < d) r.w = row[b + 3];
  return r;
}

__device__ __forceinline__ void store4(float* row, int q, int d, bool vec, float4 val) {
  if (vec) {
    *reinterpret_cast<float4*>(row + 4 * q) = val;
    return;
  }
  const int b = 4 * q;
  if (b + 0 < d) row[b + 0] = val.x;
  if (b + 1 < d) row[b + 1] = val.y;
  if (b + 2 < d) row[b + 2] = val.z;
  if (b + 3 < d) row[b + 3] = val.w;
}

// Window of chain j this round: its own speculation length (adaptive mode, kept within 1..window) or
// the common one, cut at the end of the grid (Algorithm 1: b = min(K, a + theta)).
__device__ __forceinline__ int chain_window(const int* wnd, int j, int window, int K, int a) {
  const int theta = wnd ? max(1, min(wnd[j], window)) : window;
  return min(theta, K - a);
}

__device__ __forceinline__ float warp_sum(float x) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) x += __shfl_xor_sync(0xffffffffu, x, o);
  return x;
}

// Rows a chain drafts: its window minus the last slot (rebuilt by the verify kernel), plus - with
// look-ahead - that last slot after all, when there is a step beyond it whose drift it can supply.
__device__ __forceinline__ int drafted_rows(int w, int a, int K, int la) { return w - 1 + ((la && a + w < K) ? 1 : 0); }

// ln ratio of Algorithm 3 from the two reductions, with the rounding of every operation spelled out so
// that every kernel that evaluates it gets the same bits: -(eta/sigma) <xi, delta> - (eta^2 / 2 sigma^2) |delta|^2.
__device__ __forceinline__ float ln_ratio_of(float c1, float c2, float dot, float nrm) {
  return __fmaf_rn(-c1, dot, -__fmul_rn(c2, nrm));
}


// ---------------------------------------------------------------------------------------------
// Closed-form posterior means (Eq. 4) of one point.
// ---------------------------------------------------------------------------------------------
// Mixture x* ~ sum_j pi_j N(c_j, s^2 I), by ONE WARP: y and out are rows of d floats (global or shared
// memory), lg is the warp's scratch of n_comp floats in shared memory.
//   l_j = ln pi_j + (<y, c_j> - t |c_j|^2 / 2) / (1 + t s^2),  r = softmax(l),
//   m   = (sum_j r_j c_j + s^2 y) / (1 + t s^2)
// Two forms with a fixed summation order each.  Low dimension (d <= 32): a lane owns a component for the
// logits (its inner product is a serial sum over the d coordinates) and a coordinate for the output, the
// maximum and the normaliser are warp reductions.  Otherwise the lanes stride over the coordinates and
// the components are walked one after the other.
constexpr int kGmmLaneDim = 32;

__device__ __forceinline__ float warp_max(float x) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) x = fmaxf(x, __shfl_xor_sync(0xffffffffu, x, o));
  return x;
}

__device__ __forceinline__ void gmm_point(const float* y, float t, int d, const GmmParams& P, float* lg, float* out,
                                          int lane) {
  const float inv_den = __fdiv_rn(1.f, fmaf(t, P.s2, 1.f));
  const float mht = -0.5f * t;  // exact
  if (d <= kGmmLaneDim) {
    float mx = -INFINITY;
    for (int c = lane; c < P.n_comp; c += 32) {
      float dot = 0.f;
      for (int k = 0; k < d; ++k) dot = fmaf(y[k], P.means[(size_t)c * d + k], dot);
      const float l = fmaf(fmaf(mht, P.cnorm[c], dot), inv_den, P.log_pi[c]);
      lg[c] = l;
      mx = fmaxf(mx, l);
    }
    mx = warp_max(mx);
    float part = 0.f;
    for (int c = lane; c < P.n_comp; c += 32) {
      const float e = expf(__fsub_rn(lg[c], mx));
      lg[c] = e;
      part = __fadd_rn(part, e);
    }
    const float inv_sum = __fdiv_rn(1.f, warp_sum(part));
    __syncwarp();
    if (lane < d) {
      float acc = 0.f;
      for (int c = 0; c < P.n_comp; ++c) acc = fmaf(__fmul_rn(lg[c], inv_sum), P.means[(size_t)c * d + lane], acc);
      out[lane] = __fmul_rn(fmaf(P.s2, y[lane], acc), inv_den);
    }
    __syncwarp();
    return;
  }
  float mx = -INFINITY;
  for (int c = 0; c < P.n_comp; ++c) {
    float dot = 0.f;
    for (int k = lane; k < d; k += 32) dot = fmaf(y[k], P.means[(size_t)c * d + k], dot);
    dot = warp_sum(dot);
    const float l = fmaf(fmaf(mht, P.cnorm[c], dot), inv_den, P.log_pi[c]);
    if (lane == 0) lg[c] = l;
    mx = fmaxf(mx, l);
  }
  __syncwarp();
  float sum = 0.f;
  for (int c = 0; c < P.n_comp; ++c) sum = __fadd_rn(sum, expf(__fsub_rn(lg[c], mx)));
  const float inv_sum = __fdiv_rn(1.f, sum);
  for (int k = lane; k < d; k += 32) {
    float acc = 0.f;
    for (int c = 0; c < P.n_comp; ++c)
      acc = fmaf(__fmul_rn(expf(__fsub_rn(lg[c], mx)), inv_sum), P.means[(size_t)c * d + k], acc);
    out[k] = __fmul_rn(fmaf(P.s2, y[k], acc), inv_den);
  }
  __syncwarp();
}

// Gaussian x* ~ N(mu0, Q diag(lam) Q^T): m = Q [(Q^T mu0 + lam (Q^T y)) / (1 + t lam)], in two steps of d
// independent items each.  Q / Qt are [d, d] (global or shared), ys the point, ws the d eigen-coordinates.
// Every inner product is summed as four interleaved partial sums (terms r, r + 4, r + 8, ... in ascending
// order, r = 0..3) combined as (s0 + s1) + (s2 + s3): a fixed order with four independent chains.
__device__ __forceinline__ float sum4(const float (&s)[4]) { return __fadd_rn(__fadd_rn(s[0], s[1]), __fadd_rn(s[2], s[3])); }

__device__ __forceinline__ float dot_strided4(const float* col, int stride, const float* vec, int d) {
  float s[4] = {0.f, 0.f, 0.f, 0.f};
  const int d4 = d & ~3;
  for (int i = 0; i < d4; i += 4) {
    s[0] = fmaf(col[(size_t)i * stride], vec[i], s[0]);
    s[1] = fmaf(col[(size_t)(i + 1) * stride], vec[i + 1], s[1]);
    s[2] = fmaf(col[(size_t)(i + 2) * stride], vec[i + 2], s[2]);
    s[3] = fmaf(col[(size_t)(i + 3) * stride], vec[i + 3], s[3]);
  }
#pragma unroll
  for (int r = 0; r < 3; ++r)  // the last d mod 4 terms (static indices keep the partial sums in registers)
    if (d4 + r < d) s[r] = fmaf(col[(size_t)(d4 + r) * stride], vec[d4 + r], s[r]);
  return sum4(s);
}

__device__ __forceinline__ float gauss_coord(const float* Q, const float* ys, int d, int jj, float qmu, float lam, float t) {
  const float z = dot_strided4(Q + jj, d, ys, d);  // (Q^T y)_jj
  return __fdiv_rn(fmaf(lam, z, qmu), fmaf(t, lam, 1.f));
}
__device__ __forceinline__ float gauss_out(const float* Qt, const float* ws, int d, int i) { return dot_strided4(Qt + i, d, ws, d); }

}  // namespace asd

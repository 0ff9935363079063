// The network denoiser's forward pass as a chain of bf16 x bf16 -> fp32 GEMMs on the 5th-generation
// tensor cores: operands staged in shared memory by TMA (128-byte swizzle), tcgen05.mma issued by one
// thread with the accumulator in tensor memory, a warp-specialised persistent kernel (one TMA warp,
// one MMA warp, four or eight epilogue warps) with a multi-stage mbarrier pipeline and a double-buffered
// accumulator so that the epilogue of one tile overlaps the MMAs of the next.
//
//   Y[m, n] = sum_k A[m, k] W[n, k]      A: activations [rows, K] row-major, W: weights [N, K] row-major
//
// Epilogues (fused, fp32 math on the un-rounded accumulator):
//   EPI_IN   h_0 = bf16(acc + b)
//   EPI_HID  h_l = bf16(h_{l-1} + SiLU(acc + b))
//   EPI_OUT  g   = c_skip[i] y + c_out[i] (acc + b)          (fp32 store)
//
// Every wait on an mbarrier is bounded: when the limit runs out the thread records
// ASD_ERR_TIMEOUT in the context's device error word and carries on as if the wait had
// completed, so the kernel always reaches its tear-down (tensor memory is released) and the host
// reports the error after the call.
#include <stdlib.h>
#include <string.h>

#include <algorithm>

#include "asd_internal.h"

namespace asd {

namespace {

constexpr int BM = 128;       // rows of an output tile = MMA M = tensor-memory lanes
constexpr int BK = 64;        // bf16 elements per k-block = one 128-byte swizzle row
constexpr int UMMA_K = 16;    // k extent of one tcgen05.mma (bf16)
constexpr int kGemmThreads = 192;
constexpr int kPairEpiWarps = 8;  // CTA-pair kernel: two epilogue warps per tensor-memory lane quarter, half the columns each
constexpr int kPairThreads = 64 + 32 * kPairEpiWarps;
constexpr int kSkinnyThreads = 64 + 32 * 8;  // weight-streaming kernel: four epilogue warps, or (more than 32 rows) eight:
                                             // two per lane quarter, alternate rows each
constexpr int kEpiWarp0 = 2;  // warps 2..5 are epilogue warps
constexpr long long kWaitCycles = 400000000ll;  // ~0.2 s at 1.9 GHz per wait

enum { EPI_IN = 0, EPI_HID = 1, EPI_OUT = 2 };

struct GemmArgs {
  int n_out;            // N
  int k_dim;            // K (any; the TMA zero-fills beyond the tensor)
  const int* m_dev;     // valid rows (device)
  int m_settled;        // *m_dev was final before the kernel in front of this chain started (see RowSet)
  int m_cap;            // rows of the activation buffers
  const float* bias;    // [N]
  __nv_bfloat16* out_bf16;        // EPI_IN / EPI_HID: [m, ld_h]
  const __nv_bfloat16* resid;     // EPI_HID: h_{l-1} [m, ld_h]
  int ld_h;
  float* out_f32;       // EPI_OUT: [m, d]
  const float* ysrc;    // EPI_OUT: state rows [*, d]
  const int* row_map;   // EPI_OUT: optional indirection into ysrc
  const int* row_step;  // EPI_OUT: step index per row
  const float* c_skip;
  const float* c_out;
  int* err;
};

// ---- PTX wrappers ---------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ uint32_t mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok;
}
// Bounded wait.  `dead` is a CTA-shared flag: once any wait has run out, later waits give up after
// a few polls so the kernel drains quickly.
__device__ __forceinline__ void mbar_wait(uint32_t bar, uint32_t parity, volatile int* dead, int* err) {
  if (mbar_try_wait(bar, parity)) return;
  const long long t0 = clock64();
  const long long limit = *dead ? 2000ll : kWaitCycles;
  while (!mbar_try_wait(bar, parity)) {
    if (clock64() - t0 > limit) {
      *dead = 1;
      atomicExch(err, (int)ASD_ERR_TIMEOUT);
      return;
    }
  }
}
// After a wait has run out the producer may still have copies in flight into this CTA's shared
// memory; give them time to land before the CTA exits (error path only).
__device__ __forceinline__ void drain_after_timeout(volatile int* dead) {
  if (*dead) {
    const long long t0 = clock64();
    while (clock64() - t0 < 2000000ll) {
    }
  }
}
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int x, int y) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];" ::"r"(dst),
      "l"(map), "r"(bar), "r"(x), "r"(y)
      : "memory");
}
// Starts the fetch of a tensor map (a kernel parameter) into the descriptor cache before its first use.
__device__ __forceinline__ void prefetch_tmap(const CUtensorMap* map) {
  asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(map)) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tc_mma_bf16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                            uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, {%5, %6, %7, %8}, p;\n\t}" ::"r"(d_tmem),
      "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate), "r"(0u), "r"(0u), "r"(0u), "r"(0u)
      : "memory");
}
// 32 lanes x 32 consecutive fp32 columns: thread t of the warp receives lane (base + t).
__device__ __forceinline__ void tc_ld32(uint32_t taddr, uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
        "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
        "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr)
      : "memory");
}
// 32 lanes x 16 consecutive fp32 columns.
__device__ __forceinline__ void tc_ld16(uint32_t taddr, uint32_t (&r)[16]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr)
      : "memory");
}
// Not volatile and without a memory clobber: the loads of several rows may be in flight together; the
// cluster barrier that precedes them orders them after the peers' stores.
__device__ __forceinline__ float ld_cluster_f32(uint32_t addr) {
  float v;
  asm("ld.shared::cluster.f32 %0, [%1];" : "=f"(v) : "r"(addr));
  return v;
}
__device__ __forceinline__ void tc_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// Programmatic dependent launch (no-ops for a kernel launched without that attribute).
__device__ __forceinline__ void grid_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void grid_dependency_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

// ---- CTA-pair (cta_group::2) variants ------------------------------------------------------------
__device__ __forceinline__ uint32_t cluster_ctarank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
// Address of the same shared-memory location in CTA `rank` of the cluster (shared::cluster window).
__device__ __forceinline__ uint32_t map_to_cta(uint32_t addr, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank));
  return r;
}
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// Arrive on a barrier that may live in the peer CTA (shared::cluster address).
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t bar_cluster_addr) {
  asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(bar_cluster_addr) : "memory");
}
// TMA load into this CTA's shared memory whose completion bytes are counted on a barrier of either
// CTA of the pair (every CTA fetches its own box).
__device__ __forceinline__ void tma_load_2d_pair(uint32_t dst, const CUtensorMap* map, uint32_t bar_cluster_addr, int x,
                                                 int y) {
  asm volatile(
      "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], "
      "[%2];" ::"r"(dst),
      "l"(map), "r"(bar_cluster_addr), "r"(x), "r"(y)
      : "memory");
}
// Commit of the pair's MMAs issued so far: one arrival on the given barrier (shared::cluster address).
__device__ __forceinline__ void tc_commit_pair(uint32_t bar_cluster_addr) {
  asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar_cluster_addr)
               : "memory");
}
// D[256 x N] (+)= A[256 x 16] B[N x 16]^T over the CTA pair: each CTA supplies 128 rows of A and N/2
// rows of B from the same shared-memory offsets and receives its 128 rows of D in its own tensor memory.
__device__ __forceinline__ void tc_mma_bf16_pair(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                                 uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, {%5, %5, %5, %5, %5, %5, %5, %5}, p;\n\t}" ::"r"(d_tmem),
      "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate), "r"(0u)
      : "memory");
}

// Shared-memory matrix descriptor of a K-major tile stored as rows of 128 bytes with the 128-byte
// swizzle (what the TMA writes): start address, leading byte offset 1 (unused for swizzled K-major),
// stride byte offset 1024 (8 rows x 128 B), descriptor version 1, layout type 2 (128-byte swizzle).
__device__ __forceinline__ uint64_t smem_desc_sw128(uint32_t addr) {
  uint64_t d = 0;
  d |= (uint64_t)((addr & 0x3FFFFu) >> 4);
  d |= (uint64_t)1 << 16;
  d |= (uint64_t)(1024 >> 4) << 32;
  d |= (uint64_t)1 << 46;
  d |= (uint64_t)2 << 61;
  return d;
}

// Instruction descriptor, kind::f16: D fp32, A and B bf16, both K-major, M = 128, N = BN.
template <int BN>
__device__ __forceinline__ constexpr uint32_t instr_desc() {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(BN >> 3) << 17) | ((uint32_t)(BM >> 4) << 24);
}

template <int BN>
struct Cfg {
  static constexpr int kStageBytes = (BM + BN) * BK * 2;
  static constexpr int kStages = (BN >= 256) ? 4 : (BN >= 128) ? 6 : (BN >= 64) ? 8 : 10;
  static constexpr int kTmemCols = (2 * BN < 32) ? 32 : 2 * BN;  // two accumulators
  static constexpr int kSmemBytes = kStages * kStageBytes + 1024 /*alignment slack*/ + 256 /*barriers*/;
};

// SiLU on the un-rounded fp32 accumulator; ex2.approx and rcp.approx (relative error ~2^-22, far below
// the bf16 rounding that follows).
__device__ __forceinline__ float silu(float z) { return __fdividef(z, 1.0f + __expf(-z)); }

// Epilogue of 32 consecutive accumulator columns [col0, col0 + 32) of one output row held by this
// thread: bias, then the layer's fused tail, then the store (16-byte vectors where the shape allows).
template <int EPI>
__device__ __forceinline__ void epilogue_chunk(const GemmArgs& g, int row, int col0, const uint32_t (&r)[32], float cs,
                                               float co, const float* ysrc_row) {
  if (EPI == EPI_OUT) {
    float* orow = g.out_f32 + (size_t)row * g.n_out;
    const bool vec = (g.n_out % 4 == 0) && (col0 + 32 <= g.n_out);
    if (vec) {
#pragma unroll
      for (int e = 0; e < 32; e += 4) {
        const float4 b4 = *reinterpret_cast<const float4*>(g.bias + col0 + e);
        const float4 y4 = *reinterpret_cast<const float4*>(ysrc_row + col0 + e);
        float4 o;
        o.x = fmaf(cs, y4.x, co * (__uint_as_float(r[e + 0]) + b4.x));
        o.y = fmaf(cs, y4.y, co * (__uint_as_float(r[e + 1]) + b4.y));
        o.z = fmaf(cs, y4.z, co * (__uint_as_float(r[e + 2]) + b4.z));
        o.w = fmaf(cs, y4.w, co * (__uint_as_float(r[e + 3]) + b4.w));
        *reinterpret_cast<float4*>(orow + col0 + e) = o;
      }
    } else {
#pragma unroll
      for (int e = 0; e < 32; ++e) {
        const int col = col0 + e;
        if (col < g.n_out)
          orow[col] = fmaf(cs, ysrc_row[col], co * (__uint_as_float(r[e]) + g.bias[col]));
      }
    }
  } else {
    __nv_bfloat16* orow = g.out_bf16 + (size_t)row * g.ld_h;
    const __nv_bfloat16* rrow = (EPI == EPI_HID) ? g.resid + (size_t)row * g.ld_h : nullptr;
    const bool vec = (g.ld_h % 8 == 0) && (col0 + 32 <= g.n_out);
    if (vec) {
#pragma unroll
      for (int e = 0; e < 32; e += 8) {
        float x[8];
        const float4 b0 = *reinterpret_cast<const float4*>(g.bias + col0 + e);
        const float4 b1 = *reinterpret_cast<const float4*>(g.bias + col0 + e + 4);
        const float bb[8] = {b0.x, b0.y, b0.z, b0.w, b1.x, b1.y, b1.z, b1.w};
#pragma unroll
        for (int u = 0; u < 8; ++u) x[u] = __uint_as_float(r[e + u]) + bb[u];
        if (EPI == EPI_HID) {
          const uint4 rv = *reinterpret_cast<const uint4*>(rrow + col0 + e);
          const __nv_bfloat162* rp = reinterpret_cast<const __nv_bfloat162*>(&rv);
#pragma unroll
          for (int u = 0; u < 4; ++u) {
            const float2 rf = __bfloat1622float2(rp[u]);
            x[2 * u] = rf.x + silu(x[2 * u]);
            x[2 * u + 1] = rf.y + silu(x[2 * u + 1]);
          }
        }
        uint4 ov;
        __nv_bfloat162* op = reinterpret_cast<__nv_bfloat162*>(&ov);
#pragma unroll
        for (int u = 0; u < 4; ++u) op[u] = __floats2bfloat162_rn(x[2 * u], x[2 * u + 1]);
        *reinterpret_cast<uint4*>(orow + col0 + e) = ov;
      }
    } else {
#pragma unroll
      for (int e = 0; e < 32; ++e) {
        const int col = col0 + e;
        if (col < g.n_out) {
          float x = __uint_as_float(r[e]) + g.bias[col];
          if (EPI == EPI_HID) x = __bfloat162float(rrow[col]) + silu(x);
          orow[col] = __float2bfloat16_rn(x);
        }
      }
    }
  }
}

// What the fused tail of a layer reads from global memory for 32 columns of one row: the residual
// h_{l-1} (32 bf16) for EPI_HID, the state y (32 fp32) for EPI_OUT, nothing for EPI_IN.  Fetched a few
// chunks ahead of the arithmetic (kEpiAhead) so that its latency overlaps the chunks before it.
template <int EPI>
struct EpiOperand {
  uint4 v[EPI == EPI_OUT ? 8 : (EPI == EPI_HID ? 4 : 1)];
};

template <int EPI>
__device__ __forceinline__ void epi_fetch(EpiOperand<EPI>& op, const GemmArgs& g, int row, int col0, const float* ysrc_row) {
  if (EPI == EPI_HID) {
    const uint4* p = reinterpret_cast<const uint4*>(g.resid + (size_t)row * g.ld_h + col0);
#pragma unroll
    for (int i = 0; i < 4; ++i) op.v[i] = p[i];
  } else if (EPI == EPI_OUT) {
    const uint4* p = reinterpret_cast<const uint4*>(ysrc_row + col0);
#pragma unroll
    for (int i = 0; i < 8; ++i) op.v[i] = p[i];
  }
}

// The 16-byte-vector epilogue of 32 full columns with the operand already in registers.
template <int EPI>
__device__ __forceinline__ void epi_apply(const GemmArgs& g, int row, int col0, const uint32_t (&r)[32],
                                          const EpiOperand<EPI>& op, float cs, float co) {
  if (EPI == EPI_OUT) {
    float* orow = g.out_f32 + (size_t)row * g.n_out + col0;
#pragma unroll
    for (int e = 0; e < 32; e += 4) {
      const float4 b4 = *reinterpret_cast<const float4*>(g.bias + col0 + e);
      const uint4 yv = op.v[e >> 2];
      float4 o;
      o.x = fmaf(cs, __uint_as_float(yv.x), co * (__uint_as_float(r[e + 0]) + b4.x));
      o.y = fmaf(cs, __uint_as_float(yv.y), co * (__uint_as_float(r[e + 1]) + b4.y));
      o.z = fmaf(cs, __uint_as_float(yv.z), co * (__uint_as_float(r[e + 2]) + b4.z));
      o.w = fmaf(cs, __uint_as_float(yv.w), co * (__uint_as_float(r[e + 3]) + b4.w));
      *reinterpret_cast<float4*>(orow + e) = o;
    }
  } else {
    __nv_bfloat16* orow = g.out_bf16 + (size_t)row * g.ld_h + col0;
#pragma unroll
    for (int e = 0; e < 32; e += 8) {
      float x[8];
      const float4 b0 = *reinterpret_cast<const float4*>(g.bias + col0 + e);
      const float4 b1 = *reinterpret_cast<const float4*>(g.bias + col0 + e + 4);
      const float bb[8] = {b0.x, b0.y, b0.z, b0.w, b1.x, b1.y, b1.z, b1.w};
#pragma unroll
      for (int u = 0; u < 8; ++u) x[u] = __uint_as_float(r[e + u]) + bb[u];
      if (EPI == EPI_HID) {
        const uint4 rv = op.v[e >> 3];
        const __nv_bfloat162* rp = reinterpret_cast<const __nv_bfloat162*>(&rv);
#pragma unroll
        for (int u = 0; u < 4; ++u) {
          const float2 rf = __bfloat1622float2(rp[u]);
          x[2 * u] = rf.x + silu(x[2 * u]);
          x[2 * u + 1] = rf.y + silu(x[2 * u + 1]);
        }
      }
      uint4 ov;
      __nv_bfloat162* op2 = reinterpret_cast<__nv_bfloat162*>(&ov);
#pragma unroll
      for (int u = 0; u < 4; ++u) op2[u] = __floats2bfloat162_rn(x[2 * u], x[2 * u + 1]);
      *reinterpret_cast<uint4*>(orow + e) = ov;
    }
  }
}

// How many 32-column chunks ahead the operand is fetched: one L2 round trip under load is longer than the
// arithmetic of one chunk (16 registers per chunk for the residual, 32 for the state).
template <int EPI>
constexpr int kEpiAhead = (EPI == EPI_OUT) ? 2 : 3;

// Epilogue of one accumulator tile row: this thread owns output row `row` (tensor-memory lane) and walks
// its BN columns in chunks of 32.  tcgen05.ld is warp-collective, so every lane runs the loop and only
// the global accesses are predicated on row_ok.
template <int EPI, int BN, bool kAllowFull = true>
__device__ __forceinline__ void epilogue_tile(const GemmArgs& g, uint32_t taddr0, int row, bool row_ok, int n0, float cs,
                                              float co, const float* ysrc_row) {
  // kAllowFull = false: the caller serves full tiles itself and only ragged ones come here
  const bool full_vec = kAllowFull &&
      (n0 + BN <= g.n_out) && (EPI == EPI_OUT ? (g.n_out % 4 == 0) : (g.ld_h % 8 == 0));  // warp-uniform
  if (full_vec) {
    constexpr int D = kEpiAhead<EPI>;  // chunks whose operand is in flight ahead of the arithmetic
    EpiOperand<EPI> op[D + 1];
#pragma unroll
    for (int i = 0; i < D; ++i)
      if (i < BN / 32 && row_ok) epi_fetch<EPI>(op[i], g, row, n0 + i * 32, ysrc_row);
#pragma unroll
    for (int c = 0; c < BN / 32; ++c) {
      uint32_t r[32];
      tc_ld32(taddr0 + (uint32_t)(c * 32), r);
      if (c + D < BN / 32 && row_ok) epi_fetch<EPI>(op[(c + D) % (D + 1)], g, row, n0 + (c + D) * 32, ysrc_row);
      tc_wait_ld();
      if (row_ok) epi_apply<EPI>(g, row, n0 + c * 32, r, op[c % (D + 1)], cs, co);
    }
  } else {
#pragma unroll 1
    for (int c0 = 0; c0 < BN; c0 += 32) {
      uint32_t r[32];
      tc_ld32(taddr0 + (uint32_t)c0, r);
      tc_wait_ld();
      const int col0 = n0 + c0;
      if (row_ok && col0 < g.n_out) epilogue_chunk<EPI>(g, row, col0, r, cs, co, ysrc_row);
    }
  }
}

// Epilogue of a 32-row x COLS-column accumulator block by one warp, bf16 outputs (EPI_IN, EPI_HID), with the
// global accesses staged through shared memory.  tcgen05.ld hands lane l the accumulator ROW l, so a lane reading
// its residual and writing its output directly touches 32 different rows per instruction (32 memory lines for
// 16 bytes each).  Here the warp moves 8 rows x 64 contiguous bytes per instruction instead - lane l takes
// 16-byte piece (l & 3) of row 8 i + (l >> 2), i = 0..3 - and the two layouts meet in a per-warp buffer of
// 32 rows x 64 bytes in which piece p of row r sits at slot p ^ ((r >> 1) & 3): both access patterns (8 rows x
// one piece, 2 rows x 4 pieces per 128-byte wavefront) then touch every bank group once.
// The residual of the whole block is fetched ahead of the arithmetic.
constexpr int kEpiStageBytes = 32 * 64;  // per epilogue warp
__device__ __forceinline__ int epi_slot(int r, int p) { return r * 64 + ((p ^ ((r >> 1) & 3)) << 4); }

// 16-byte piece `piece` of the residual rows row_base + 8 i + prow, i = 0..3, columns [col0, col0 + 32)
__device__ __forceinline__ void epi_fetch_pieces(const GemmArgs& g, int row_base, int prow, int piece, int m, int col0,
                                                 uint4 (&dst)[4]) {
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int row = row_base + 8 * i + prow;
    if (row < m) dst[i] = *reinterpret_cast<const uint4*>(g.resid + (size_t)row * g.ld_h + col0 + piece * 8);
  }
}

// One 32-column chunk C of the staged epilogue (a template recursion over the chunks keeps every register array
// statically indexed).  R[c] holds the residual pieces of chunk c, fetched by the caller.
template <int EPI, int NC, int C>
__device__ __forceinline__ void epi_staged_chunk(const GemmArgs& g, uint32_t taddr0, int row_base, int lane, int m, int n0,
                                                 uint8_t* buf, uint4 (&R)[NC][4]) {
  if constexpr (C < NC) {
    const int prow = lane >> 2, piece = lane & 3;
    if (EPI == EPI_HID) {
#pragma unroll
      for (int i = 0; i < 4; ++i) *reinterpret_cast<uint4*>(buf + epi_slot(8 * i + prow, piece)) = R[C][i];
      __syncwarp();  // from here on a lane touches only its own row of the buffer, until the stores below
    }
    uint32_t r[32];
    tc_ld32(taddr0 + (uint32_t)(C * 32), r);
    tc_wait_ld();
    const int col0 = n0 + C * 32;
#pragma unroll
    for (int e = 0; e < 32; e += 8) {
      float x[8];
      const float4 b0 = *reinterpret_cast<const float4*>(g.bias + col0 + e);
      const float4 b1 = *reinterpret_cast<const float4*>(g.bias + col0 + e + 4);
      const float bb[8] = {b0.x, b0.y, b0.z, b0.w, b1.x, b1.y, b1.z, b1.w};
#pragma unroll
      for (int u = 0; u < 8; ++u) x[u] = __uint_as_float(r[e + u]) + bb[u];
      if (EPI == EPI_HID) {
        const uint4 rv = *reinterpret_cast<const uint4*>(buf + epi_slot(lane, e >> 3));
        const __nv_bfloat162* rp = reinterpret_cast<const __nv_bfloat162*>(&rv);
#pragma unroll
        for (int u = 0; u < 4; ++u) {
          const float2 rf = __bfloat1622float2(rp[u]);
          x[2 * u] = rf.x + silu(x[2 * u]);
          x[2 * u + 1] = rf.y + silu(x[2 * u + 1]);
        }
      }
      uint4 ov;
      __nv_bfloat162* op2 = reinterpret_cast<__nv_bfloat162*>(&ov);
#pragma unroll
      for (int u = 0; u < 4; ++u) op2[u] = __floats2bfloat162_rn(x[2 * u], x[2 * u + 1]);
      *reinterpret_cast<uint4*>(buf + epi_slot(lane, e >> 3)) = ov;
    }
    __syncwarp();
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const int row = row_base + 8 * i + prow;
      const uint4 v = *reinterpret_cast<const uint4*>(buf + epi_slot(8 * i + prow, piece));
      if (row < m) *reinterpret_cast<uint4*>(g.out_bf16 + (size_t)row * g.ld_h + col0 + piece * 8) = v;
    }
    __syncwarp();
    epi_staged_chunk<EPI, NC, C + 1>(g, taddr0, row_base, lane, m, n0, buf, R);
  }
}

// The residual pieces of a whole 32-row x COLS-column block: they do not depend on the accumulator, so the caller
// issues these loads BEFORE it waits for the tile's MMAs and their latency hides behind that wait.
template <int EPI, int COLS>
__device__ __forceinline__ void epilogue_staged_prefetch(const GemmArgs& g, int row_base, int lane, int m, int n0,
                                                         uint4 (&R)[COLS / 32][4]) {
  if (EPI == EPI_HID) {
#pragma unroll
    for (int c = 0; c < COLS / 32; ++c) epi_fetch_pieces(g, row_base, lane >> 2, lane & 3, m, n0 + c * 32, R[c]);
  }
}

template <int EPI, int COLS>
__device__ __forceinline__ void epilogue_tile_staged(const GemmArgs& g, uint32_t taddr0, int row_base, int lane, int m,
                                                     int n0, uint8_t* buf, uint4 (&R)[COLS / 32][4]) {
  static_assert(EPI != EPI_OUT, "bf16 outputs only");
  epi_staged_chunk<EPI, COLS / 32, 0>(g, taddr0, row_base, lane, m, n0, buf, R);
}

// The same staging for the output projection (fp32 in, fp32 out): a 32-column chunk is taken as two halves of 16
// columns = 64 bytes per row, the geometry of the bf16 path.  Per half the warp fetches the state rows y (through the
// optional row map) 8 rows x 64 contiguous bytes per instruction, hands them to the lanes that own the rows, and
// writes g = c_skip y + c_out (acc + b) the same way.  The state pieces of the next half are in flight during the
// arithmetic of the current one.
template <int COLS>
__device__ __forceinline__ void epilogue_tile_staged_out(const GemmArgs& g, uint32_t taddr0, int row_base, int lane, int m,
                                                         int n0, uint8_t* buf, float cs, float co) {
  constexpr int NH = COLS / 16;  // halves
  const int prow = lane >> 2, piece = lane & 3;
  const float* yrow[4];  // state rows of the tile rows 8 i + prow (null: beyond the valid rows)
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int row = row_base + 8 * i + prow;
    yrow[i] = row < m ? g.ysrc + (size_t)(g.row_map ? g.row_map[row] : row) * g.n_out : nullptr;
  }
  uint4 Y[2][4];
  auto fetch = [&](int h, uint4 (&dst)[4]) {
#pragma unroll
    for (int i = 0; i < 4; ++i)
      if (yrow[i]) dst[i] = *reinterpret_cast<const uint4*>(yrow[i] + n0 + h * 16 + piece * 4);
  };
  fetch(0, Y[0]);
  uint32_t r[32];
#pragma unroll
  for (int h = 0; h < NH; ++h) {
    if ((h & 1) == 0) tc_ld32(taddr0 + (uint32_t)((h >> 1) * 32), r);
#pragma unroll
    for (int i = 0; i < 4; ++i) *reinterpret_cast<uint4*>(buf + epi_slot(8 * i + prow, piece)) = Y[h & 1][i];
    __syncwarp();  // from here on a lane touches only its own row of the buffer, until the stores below
    if (h + 1 < NH) fetch(h + 1, Y[(h + 1) & 1]);
    if ((h & 1) == 0) tc_wait_ld();
    const int col0 = n0 + h * 16;
#pragma unroll
    for (int e = 0; e < 16; e += 4) {
      const uint4 yv = *reinterpret_cast<const uint4*>(buf + epi_slot(lane, e >> 2));
      const float4 b4 = *reinterpret_cast<const float4*>(g.bias + col0 + e);
      const int a0 = (h & 1) * 16 + e;
      float4 o;
      o.x = fmaf(cs, __uint_as_float(yv.x), co * (__uint_as_float(r[a0 + 0]) + b4.x));
      o.y = fmaf(cs, __uint_as_float(yv.y), co * (__uint_as_float(r[a0 + 1]) + b4.y));
      o.z = fmaf(cs, __uint_as_float(yv.z), co * (__uint_as_float(r[a0 + 2]) + b4.z));
      o.w = fmaf(cs, __uint_as_float(yv.w), co * (__uint_as_float(r[a0 + 3]) + b4.w));
      *reinterpret_cast<float4*>(buf + epi_slot(lane, e >> 2)) = o;
    }
    __syncwarp();
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const int row = row_base + 8 * i + prow;
      const uint4 v = *reinterpret_cast<const uint4*>(buf + epi_slot(8 * i + prow, piece));
      if (row < m) *reinterpret_cast<uint4*>(g.out_f32 + (size_t)row * g.n_out + col0 + piece * 4) = v;
    }
    __syncwarp();
  }
}

template <int BN, int EPI>
__global__ void __launch_bounds__(kGemmThreads, 1)
gemm_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_w, const GemmArgs g) {
  using C = Cfg<BN>;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t tiles = (raw + 1023u) & ~1023u;  // stage buffers, 1024-byte aligned for the swizzle
  uint8_t* aux = smem_raw + (tiles - raw) + C::kStages * C::kStageBytes;
  uint64_t* bars = reinterpret_cast<uint64_t*>(aux);  // full[S], empty[S], acc_full[2], acc_empty[2]
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(aux + 8 * (2 * C::kStages + 4));
  volatile int* dead = reinterpret_cast<volatile int*>(tmem_slot + 1);
  const uint32_t bar0 = smem_u32(bars);
  auto full_bar = [&](int s) { return bar0 + 8u * s; };
  auto empty_bar = [&](int s) { return bar0 + 8u * (C::kStages + s); };
  auto accf_bar = [&](int b) { return bar0 + 8u * (2 * C::kStages + b); };
  auto acce_bar = [&](int b) { return bar0 + 8u * (2 * C::kStages + 2 + b); };

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int m = min(*g.m_dev, g.m_cap);
  const int tiles_m = (m + BM - 1) / BM;
  const int tiles_n = (g.n_out + BN - 1) / BN;
  const int n_tiles = tiles_m * tiles_n;
  const int num_kb = (g.k_dim + BK - 1) / BK;

  if (threadIdx.x == 0) {
    prefetch_tmap(&map_a);
    prefetch_tmap(&map_w);
    for (int s = 0; s < C::kStages; ++s) {
      mbar_init(full_bar(s), 1);
      mbar_init(empty_bar(s), 1);
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(accf_bar(b), 1);
      mbar_init(acce_bar(b), 4);
    }
    *dead = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)),
                 "r"((uint32_t)C::kTmemCols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 0) {
    // ---------------- TMA producer ----------------
    if (lane == 0) {
      int stage = 0;
      uint32_t phase = 0;
      for (int t = blockIdx.x; t < n_tiles; t += gridDim.x) {
        const int m0 = (t / tiles_n) * BM, n0 = (t % tiles_n) * BN;
        for (int kb = 0; kb < num_kb; ++kb) {
          mbar_wait(empty_bar(stage), phase ^ 1u, dead, g.err);
          const uint32_t sa = tiles + stage * C::kStageBytes;
          const uint32_t sb = sa + BM * BK * 2;
          mbar_expect_tx(full_bar(stage), (uint32_t)C::kStageBytes);
          tma_load_2d(sa, &map_a, full_bar(stage), kb * BK, m0);
          tma_load_2d(sb, &map_w, full_bar(stage), kb * BK, n0);
          if (++stage == C::kStages) {
            stage = 0;
            phase ^= 1u;
          }
        }
      }
      drain_after_timeout(dead);
    }
  } else if (warp == 1) {
    // ---------------- MMA issuer ----------------
    if (lane == 0) {
      constexpr uint32_t idesc = instr_desc<BN>();
      int stage = 0;
      uint32_t phase = 0;
      int it = 0;
      for (int t = blockIdx.x; t < n_tiles; t += gridDim.x, ++it) {
        const int acc = it & 1;
        const uint32_t acc_phase = (uint32_t)(it >> 1) & 1u;
        mbar_wait(acce_bar(acc), acc_phase ^ 1u, dead, g.err);  // epilogue has drained this accumulator
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + (uint32_t)(acc * BN);
        for (int kb = 0; kb < num_kb; ++kb) {
          mbar_wait(full_bar(stage), phase, dead, g.err);
          tc_fence_after();
          const uint32_t sa = tiles + stage * C::kStageBytes;
          const uint32_t sb = sa + BM * BK * 2;
          const uint64_t da = smem_desc_sw128(sa), db = smem_desc_sw128(sb);
#pragma unroll
          for (int k = 0; k < BK / UMMA_K; ++k) {
            // advancing 16 bf16 = 32 bytes inside the swizzled row: +2 in the (address >> 4) field
            tc_mma_bf16(d_tmem, da + (uint64_t)(2 * k), db + (uint64_t)(2 * k), idesc, (kb | k) != 0 ? 1u : 0u);
          }
          tc_commit(empty_bar(stage));  // frees the stage once these MMAs have read it
          if (++stage == C::kStages) {
            stage = 0;
            phase ^= 1u;
          }
        }
        tc_commit(accf_bar(acc));  // accumulator complete
      }
    }
  } else {
    // ---------------- epilogue warps ----------------
    const int quarter = warp & 3;  // tensor-memory lanes [32 quarter, 32 quarter + 32)
    int it = 0;
    for (int t = blockIdx.x; t < n_tiles; t += gridDim.x, ++it) {
      const int m0 = (t / tiles_n) * BM, n0 = (t % tiles_n) * BN;
      const int acc = it & 1;
      const uint32_t acc_phase = (uint32_t)(it >> 1) & 1u;
      mbar_wait(accf_bar(acc), acc_phase, dead, g.err);
      tc_fence_after();
      const int row = m0 + quarter * 32 + lane;
      const bool row_ok = row < m;
      float cs = 0.f, co = 0.f;
      const float* ysrc_row = nullptr;
      if (EPI == EPI_OUT && row_ok) {
        const int step = g.row_step[row];
        cs = g.c_skip[step];
        co = g.c_out[step];
        ysrc_row = g.ysrc + (size_t)(g.row_map ? g.row_map[row] : row) * g.n_out;
      }
      epilogue_tile<EPI, BN>(g, tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(acc * BN), row, row_ok, n0, cs,
                             co, ysrc_row);
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(acce_bar(acc));
    }
  }

  // ---------------- tear-down ----------------
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)C::kTmemCols)
                 : "memory");
  }
}

// ---------------------------------------------------------------------------------------------------
// CTA-pair kernel: a cluster of two CTAs computes a 256 x BN output tile with tcgen05.mma.cta_group::2.
// Each CTA stages only its own 128 rows of A and BN/2 of the tile's BN weight rows (for BN = 256: 32 KB
// per k-block instead of 48 KB for the same 128 x 256 x 64 of tensor work per SM), so the L2 -> shared-memory
// stream per flop drops by a third.  Rank 0 of the pair issues the MMAs; both
// CTAs run a TMA warp and eight epilogue warps (two per lane quarter) on their own 128 accumulator rows.
//   full[s]   in rank 0, completed by both CTAs' TMA bytes          empty[s]  in each CTA, MMA commit
//   accf[b]   in each CTA, MMA commit                               acce[b]   in rank 0, all 16 epilogue warps
// ---------------------------------------------------------------------------------------------------
template <int BN>
struct PairCfg {
  static constexpr int kStageBytes = (BM + BN / 2) * BK * 2;           // per CTA: 128 rows of A, BN/2 rows of W
  static constexpr int kStages = (BN >= 256) ? 6 : (BN >= 128) ? 8 : 9;  // <= 192 KB of stages
  static constexpr int kTmemCols = 2 * BN;                             // two accumulators per CTA
  static constexpr int kSmemBytes =
      kStages * kStageBytes + 1024 + 256 + kPairEpiWarps * kEpiStageBytes + kPairEpiWarps * (BN / (kPairEpiWarps / 4)) * 4;
};

template <int BN, int EPI>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kPairThreads, 1)
gemm_pair_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_w,
                 const GemmArgs g) {
  using C = PairCfg<BN>;
  constexpr int S = C::kStages;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t tiles = (raw + 1023u) & ~1023u;
  uint8_t* aux = smem_raw + (tiles - raw) + S * C::kStageBytes;
  uint64_t* bars = reinterpret_cast<uint64_t*>(aux);  // full[S], empty[S], acc_full[2], acc_empty[2]
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(aux + 8 * (2 * S + 4));
  volatile int* dead = reinterpret_cast<volatile int*>(tmem_slot + 1);
  const uint32_t bar0 = smem_u32(bars);
  auto full_bar = [&](int s) { return bar0 + 8u * s; };
  auto empty_bar = [&](int s) { return bar0 + 8u * (S + s); };
  auto accf_bar = [&](int b) { return bar0 + 8u * (2 * S + b); };
  auto acce_bar = [&](int b) { return bar0 + 8u * (2 * S + 2 + b); };

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();
  const int pair = blockIdx.x >> 1, n_pairs = gridDim.x >> 1;
  const int tiles_n = (g.n_out + BN - 1) / BN;
  const int num_kb = (g.k_dim + BK - 1) / BK;

  // Programmatic dependent launch: the next kernel of the stream may be scheduled from now on (its CTAs start as
  // SMs become free), and this kernel sets up its barriers and tensor memory while the previous one finishes;
  // everything that kernel wrote (the row count included) is read after grid_dependency_wait() below.
  grid_launch_dependents();

  if (threadIdx.x == 0) {
    prefetch_tmap(&map_a);
    prefetch_tmap(&map_w);
    for (int s = 0; s < S; ++s) {
      mbar_init(full_bar(s), 1);
      mbar_init(empty_bar(s), 1);
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(accf_bar(b), 1);
      mbar_init(acce_bar(b), 2 * kPairEpiWarps);  // every epilogue warp of both CTAs
    }
    *dead = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)),
                 "r"((uint32_t)C::kTmemCols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  __syncwarp();
  cluster_sync_all();  // the peer's barriers are initialised before anything arrives on them
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  grid_dependency_wait();
  const int m = min(*g.m_dev, g.m_cap);
  const int tiles_m = (m + 2 * BM - 1) / (2 * BM);
  const int n_tiles = tiles_m * tiles_n;

  if (warp == 0) {
    // ---------------- TMA producer (both CTAs) ----------------
    if (lane == 0) {
      int stage = 0;
      uint32_t phase = 0;
      for (int t = pair; t < n_tiles; t += n_pairs) {
        const int m0 = (t / tiles_n) * (2 * BM) + (int)rank * BM;
        const int n0 = (t % tiles_n) * BN + (int)rank * (BN / 2);
        for (int kb = 0; kb < num_kb; ++kb) {
          mbar_wait(empty_bar(stage), phase ^ 1u, dead, g.err);
          const uint32_t sa = tiles + stage * C::kStageBytes;
          const uint32_t sb = sa + BM * BK * 2;
          const uint32_t full0 = map_to_cta(full_bar(stage), 0);
          if (rank == 0) mbar_expect_tx(full_bar(stage), 2u * (uint32_t)C::kStageBytes);
          tma_load_2d_pair(sa, &map_a, full0, kb * BK, m0);
          tma_load_2d_pair(sb, &map_w, full0, kb * BK, n0);
          if (++stage == S) {
            stage = 0;
            phase ^= 1u;
          }
        }
      }
      drain_after_timeout(dead);
    }
  } else if (warp == 1) {
    // ---------------- MMA issuer (rank 0 only) ----------------
    if (rank == 0 && lane == 0) {
      constexpr uint32_t idesc =
          (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(BN >> 3) << 17) | ((uint32_t)((2 * BM) >> 4) << 24);
      int stage = 0;
      uint32_t phase = 0;
      int it = 0;
      for (int t = pair; t < n_tiles; t += n_pairs, ++it) {
        const int acc = it & 1;
        const uint32_t acc_phase = (uint32_t)(it >> 1) & 1u;
        mbar_wait(acce_bar(acc), acc_phase ^ 1u, dead, g.err);  // both CTAs' epilogues have drained it
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + (uint32_t)(acc * BN);
        for (int kb = 0; kb < num_kb; ++kb) {
          mbar_wait(full_bar(stage), phase, dead, g.err);
          tc_fence_after();
          const uint32_t sa = tiles + stage * C::kStageBytes;
          const uint32_t sb = sa + BM * BK * 2;
          const uint64_t da = smem_desc_sw128(sa), db = smem_desc_sw128(sb);
#pragma unroll
          for (int k = 0; k < BK / UMMA_K; ++k)
            tc_mma_bf16_pair(d_tmem, da + (uint64_t)(2 * k), db + (uint64_t)(2 * k), idesc, (kb | k) != 0 ? 1u : 0u);
          tc_commit_pair(empty_bar(stage));                 // frees the stage in this CTA ...
          tc_commit_pair(map_to_cta(empty_bar(stage), 1));  // ... and in the peer
          if (++stage == S) {
            stage = 0;
            phase ^= 1u;
          }
        }
        tc_commit_pair(accf_bar(acc));
        tc_commit_pair(map_to_cta(accf_bar(acc), 1));
      }
    }
  } else {
    // ---------------- epilogue warps (both CTAs, own 128 rows) ----------------
    const int quarter = warp & 3;
    int it = 0;
    for (int t = pair; t < n_tiles; t += n_pairs, ++it) {
      const int m0 = (t / tiles_n) * (2 * BM) + (int)rank * BM, n0 = (t % tiles_n) * BN;
      const int acc = it & 1;
      const uint32_t acc_phase = (uint32_t)(it >> 1) & 1u;
      constexpr int kCols = BN / (kPairEpiWarps / 4);  // this warp's share of the tile's columns
      constexpr int kStagedCols = kCols >= 32 ? kCols : 32;
      const int part = (warp - kEpiWarp0) >> 2;
      // full tiles: global accesses staged through shared memory (warp-uniform choice)
      const bool staged = kCols % 32 == 0 && n0 + BN <= g.n_out && (EPI == EPI_OUT ? g.n_out % 4 == 0 : g.ld_h % 8 == 0);
      uint4 R[kStagedCols / 32][4];
      GemmArgs gs = g;  // for the staged path: the bias of this warp's columns comes from shared memory
      if (staged) {
        if (EPI != EPI_OUT)
          epilogue_staged_prefetch<EPI == EPI_OUT ? EPI_IN : EPI, kStagedCols>(g, m0 + quarter * 32, lane, m, n0 + part * kCols, R);
        // (fetched while the MMAs run: a bias read behind the accumulator wait costs an L2 round trip per chunk)
        float* sbias = reinterpret_cast<float*>(aux + 256 + kPairEpiWarps * kEpiStageBytes) + (warp - kEpiWarp0) * kCols;
#pragma unroll
        for (int c = 0; c < kStagedCols / 32; ++c) sbias[c * 32 + lane] = g.bias[n0 + part * kCols + c * 32 + lane];
        __syncwarp();
        gs.bias = sbias - (n0 + part * kCols);
      }
      const int row = m0 + quarter * 32 + lane;
      const bool row_ok = row < m;
      float cs = 0.f, co = 0.f;
      const float* ysrc_row = nullptr;
      if (EPI == EPI_OUT && row_ok) {  // per-row scalars: fetched ahead of the wait as well
        const int step = g.row_step[row];
        cs = g.c_skip[step];
        co = g.c_out[step];
        ysrc_row = g.ysrc + (size_t)(g.row_map ? g.row_map[row] : row) * g.n_out;
      }
      mbar_wait(accf_bar(acc), acc_phase, dead, g.err);
      tc_fence_after();
      const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(acc * BN + part * kCols);
      uint8_t* buf = aux + 256 + (warp - kEpiWarp0) * kEpiStageBytes;
      if (staged && EPI == EPI_OUT)
        epilogue_tile_staged_out<kStagedCols>(gs, taddr, m0 + quarter * 32, lane, m, n0 + part * kCols, buf, cs, co);
      else if (staged)
        epilogue_tile_staged<EPI == EPI_OUT ? EPI_IN : EPI, kStagedCols>(gs, taddr, m0 + quarter * 32, lane, m,
                                                                         n0 + part * kCols, buf, R);
      else
        epilogue_tile<EPI, kCols, false>(g, taddr, row, row_ok, n0 + part * kCols, cs, co, ysrc_row);
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive_cluster(map_to_cta(acce_bar(acc), 0));
    }
  }

  // ---------------- tear-down: neither CTA leaves while the pair's MMAs may still touch it ----------------
  tc_fence_before();
  __syncthreads();
  __syncwarp();
  cluster_sync_all();
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)C::kTmemCols) : "memory");
  }
}

// ---------------------------------------------------------------------------------------------------
// Skinny kernel for few rows (used for m <= 256; gridDim.y walks further blocks of 256 rows): the product is weight streaming, so the roles of the operands
// are swapped.  A CTA owns 128 output features: the weight tile W[n0 .. n0+127, k-block] is the MMA's
// 128-row operand (one 16 KB TMA box per k-block, the shape that streams from HBM at full rate) and the
// activation rows X[0 .. m_pad-1, k-block] are its narrow operand, so D^T[feature, row] accumulates in
// tensor memory with no padded MMA rows.  The k range is split over the kSplit CTAs of a cluster so that
// N/128 x kSplit CTAs keep every SM streaming; each CTA parks its partial accumulator in its own shared
// memory, then every CTA sums the partials of its share of the rows over distributed shared memory in
// rank order (a fixed order, so results are reproducible) and applies the fused epilogue, the 32 lanes
// of a warp writing 32 consecutive features.
// ---------------------------------------------------------------------------------------------------
constexpr int kSplit = 4;
constexpr int kSkinnyMaxStages = 8;
constexpr int kSkinnyStageBudget = 192 * 1024;
constexpr int kSkinnySmallBudget = 96 * 1024;  // up to 128 rows: two CTAs (consecutive layers) share an SM
constexpr int kSkinnyBlockRows = 256;  // activation rows per CTA (the MMA's N)
constexpr int kSkinnyMaxRows = 256;    // one row block: at 512 rows the CTA-pair kernel with 128-wide tiles is as fast

__host__ __device__ constexpr int skinny_stage_bytes(int m_pad) { return (BM + m_pad) * BK * 2; }

template <int EPI>
__global__ void __cluster_dims__(kSplit, 1, 1) __launch_bounds__(kSkinnyThreads, 1)
gemm_skinny_kernel(const __grid_constant__ CUtensorMap map_w, const __grid_constant__ CUtensorMap map_x,
                   const GemmArgs g, const int m_pad, const int S) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t tiles = (raw + 1023u) & ~1023u;
  const int stage_bytes = skinny_stage_bytes(m_pad);
  uint8_t* tiles_ptr = smem_raw + (tiles - raw);
  uint8_t* aux = tiles_ptr + max(S * stage_bytes, m_pad * BM * 4);
  uint64_t* bars = reinterpret_cast<uint64_t*>(aux);  // full[S], empty[S], acc_full
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(aux + 8 * (2 * S + 1));
  volatile int* dead = reinterpret_cast<volatile int*>(tmem_slot + 1);
  const uint32_t bar0 = smem_u32(bars);
  auto full_bar = [&](int s) { return bar0 + 8u * s; };
  auto empty_bar = [&](int s) { return bar0 + 8u * (S + s); };
  const uint32_t accf_bar = bar0 + 8u * (2 * S);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();
  const int n0 = (blockIdx.x / kSplit) * BM;
  const int row0 = blockIdx.y * m_pad;  // this CTA's block of activation rows
  const int num_kb = (g.k_dim + BK - 1) / BK;
  const int per = (num_kb + kSplit - 1) / kSplit;  // k-blocks [kb0, kb1) belong to this rank
  const int kb0 = min((int)rank * per, num_kb), kb1 = min(kb0 + per, num_kb);
  const uint32_t tmem_cols = m_pad <= 32 ? 32u : (m_pad <= 64 ? 64u : (m_pad <= 128 ? 128u : 256u));

  // Programmatic dependent launch: the next kernel of the stream may start its own preamble now (if it was
  // launched with that attribute); everything here that depends on an earlier kernel comes after
  // grid_dependency_wait() below.  The weights do not, so their first tiles are fetched before it.
  grid_launch_dependents();

  // A row block without a single valid row has nothing to compute or store: its cluster leaves before it
  // streams any weights (a pass over zero rows, or a grid sized for a bound above the real count).  It still
  // waits for the previous kernel, so that "this kernel has completed" keeps implying that every kernel
  // before it has.
  if (g.m_settled && min(__ldcg(g.m_dev), g.m_cap) <= row0) {
    grid_dependency_wait();
    return;
  }

  if (threadIdx.x == 0) {
    prefetch_tmap(&map_x);
    prefetch_tmap(&map_w);
    for (int s = 0; s < S; ++s) {
      mbar_init(full_bar(s), 1);
      mbar_init(empty_bar(s), 1);
    }
    mbar_init(accf_bar, 1);
    *dead = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)),
                 "r"(tmem_cols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  // What the fused tail reads from global memory does not depend on this kernel's own product: the epilogue warps
  // fetch it (row count, bias, and the residual / state / per-row scalars of their first group of rows) while the
  // weights are still streaming, instead of after the cluster's partials are in place.
  constexpr int kSkR = 8;  // rows per group of the reduction below
  int m_pre = 0;
  float bias_pre = 0.f, opnd_pre[kSkR], cs_pre[kSkR], co_pre[kSkR];
#pragma unroll
  for (int u = 0; u < kSkR; ++u) opnd_pre[u] = cs_pre[u] = co_pre[u] = 0.f;

  if (warp == 0) {
    // ---------------- TMA producer ----------------
    if (lane == 0) {
      // the first min(S, k-blocks) stages are free: weight tiles now, activation tiles once the producer
      // of the activations has finished
      const int pre = min(S, kb1 - kb0);
      for (int i = 0; i < pre; ++i) {
        mbar_expect_tx(full_bar(i), (uint32_t)stage_bytes);
        tma_load_2d(tiles + i * stage_bytes, &map_w, full_bar(i), (kb0 + i) * BK, n0);
      }
      grid_dependency_wait();
      for (int i = 0; i < pre; ++i)
        tma_load_2d(tiles + i * stage_bytes + BM * BK * 2, &map_x, full_bar(i), (kb0 + i) * BK, row0);
      int stage = pre == S ? 0 : pre;
      uint32_t phase = pre == S ? 1u : 0u;
      for (int kb = kb0 + pre; kb < kb1; ++kb) {
        mbar_wait(empty_bar(stage), phase ^ 1u, dead, g.err);
        const uint32_t sw = tiles + stage * stage_bytes;
        const uint32_t sx = sw + BM * BK * 2;
        mbar_expect_tx(full_bar(stage), (uint32_t)stage_bytes);
        tma_load_2d(sw, &map_w, full_bar(stage), kb * BK, n0);
        tma_load_2d(sx, &map_x, full_bar(stage), kb * BK, row0);
        if (++stage == S) {
          stage = 0;
          phase ^= 1u;
        }
      }
      drain_after_timeout(dead);
    }
  } else if (warp == 1) {
    // ---------------- MMA issuer ----------------
    if (lane == 0) {
      // D fp32, A (weights) and B (activations) bf16, both K-major, M = 128 features, N = m_pad rows
      const uint32_t idesc =
          (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(m_pad >> 3) << 17) | ((uint32_t)(BM >> 4) << 24);
      int stage = 0;
      uint32_t phase = 0;
      for (int kb = kb0; kb < kb1; ++kb) {
        mbar_wait(full_bar(stage), phase, dead, g.err);
        tc_fence_after();
        const uint32_t sw = tiles + stage * stage_bytes;
        const uint32_t sx = sw + BM * BK * 2;
        const uint64_t da = smem_desc_sw128(sw), db = smem_desc_sw128(sx);
#pragma unroll
        for (int k = 0; k < BK / UMMA_K; ++k)
          tc_mma_bf16(tmem_base, da + (uint64_t)(2 * k), db + (uint64_t)(2 * k), idesc, (kb > kb0 || k > 0) ? 1u : 0u);
        tc_commit(empty_bar(stage));
        if (++stage == S) {
          stage = 0;
          phase ^= 1u;
        }
      }
      if (kb1 > kb0)
        tc_commit(accf_bar);
      else
        mbar_arrive(accf_bar);  // no k-block of its own: the partial is zero
    }
  } else {
    // ---- park this rank's partial D^T[feature, row] in shared memory as part[row][feature] ----
    const int quarter = warp & 3;
    const int feat = quarter * 32 + lane;  // tensor-memory lane = feature within the tile
    {
      grid_dependency_wait();  // the row count, the residual and the state come from earlier kernels
      m_pre = max(0, min(min(*g.m_dev, g.m_cap) - row0, m_pad));
      const int n = n0 + feat;
      if (n < g.n_out && m_pre > 0) {
        bias_pre = g.bias[n];
        const int kRowStep = kSplit * (((int)(blockDim.x >> 5) - kEpiWarp0) >> 2);
        const int lr_first = (int)rank + ((warp - kEpiWarp0) >> 2) * kSplit;
#pragma unroll
        for (int u = 0; u < kSkR; ++u) {
          const int row = row0 + min(lr_first + u * kRowStep, m_pre - 1);
          if (EPI == EPI_OUT) {
            const int step = g.row_step[row];
            cs_pre[u] = g.c_skip[step];
            co_pre[u] = g.c_out[step];
            opnd_pre[u] = g.ysrc[(size_t)(g.row_map ? g.row_map[row] : row) * g.n_out + n];
          } else if (EPI == EPI_HID) {
            opnd_pre[u] = __bfloat162float(g.resid[(size_t)row * g.ld_h + n]);
          }
        }
      }
    }
    mbar_wait(accf_bar, 0u, dead, g.err);
    tc_fence_after();
    float* part = reinterpret_cast<float*>(tiles_ptr);  // the stage buffers are idle now: [m_pad][128] fp32
    const int halves = ((int)(blockDim.x >> 5) - kEpiWarp0) >> 2;  // epilogue warps per lane quarter: 1 or 2
    const int half = (warp - kEpiWarp0) >> 2;  // they take alternate groups of 16 rows
    for (int c0 = half * 16; c0 < m_pad; c0 += 16 * halves) {
      uint32_t r[16];
      if (kb1 > kb0) {
        tc_ld16(tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)c0, r);
        tc_wait_ld();
      } else {
#pragma unroll
        for (int e = 0; e < 16; ++e) r[e] = 0u;
      }
#pragma unroll
      for (int e = 0; e < 16; ++e) part[(c0 + e) * BM + feat] = __uint_as_float(r[e]);
    }
    tc_fence_before();
  }

  __syncthreads();
  __syncwarp();
  cluster_sync_all();  // every rank's partial is in place

  if (warp >= kEpiWarp0) {
    const int quarter = warp & 3;
    const int feat = quarter * 32 + lane;
    const int n = n0 + feat;
    const int m = m_pre;
    if (n < g.n_out) {
      uint32_t part_of[kSplit];  // the partial buffer sits at the same offset in every CTA of the cluster
#pragma unroll
      for (int q = 0; q < kSplit; ++q) part_of[q] = map_to_cta(tiles, (uint32_t)q);
      const float bias = bias_pre;
      // rows rank, rank + kSplit, ... of the block, eight at a time: all their loads (partials over
      // distributed shared memory, residual / state and per-row scalars from global memory) are issued
      // before the first store, so one memory latency is paid per group instead of per row
      constexpr int R = kSkR;
      const int kRowStep = kSplit * (((int)(blockDim.x >> 5) - kEpiWarp0) >> 2);  // this warp's rows: every kRowStep-th
      const int half = (warp - kEpiWarp0) >> 2;
      const int lr_first = (int)rank + half * kSplit;
      for (int lr0 = lr_first; lr0 < m; lr0 += R * kRowStep) {
        float acc[R], opnd[R], cs[R], co[R];
        const bool first = lr0 == lr_first;  // this group's operands were fetched ahead
#pragma unroll
        for (int u = 0; u < R; ++u) {
          const int lr = min(lr0 + u * kRowStep, m - 1);  // clamped rows are loaded but not stored
          const int row = row0 + lr;
          float a = 0.f;
#pragma unroll
          for (int q = 0; q < kSplit; ++q) a += ld_cluster_f32(part_of[q] + (uint32_t)((lr * BM + feat) * 4));
          acc[u] = a;
          if (first) {
            opnd[u] = opnd_pre[u];
            cs[u] = cs_pre[u];
            co[u] = co_pre[u];
          } else if (EPI == EPI_OUT) {
            const int step = g.row_step[row];
            cs[u] = g.c_skip[step];
            co[u] = g.c_out[step];
            opnd[u] = g.ysrc[(size_t)(g.row_map ? g.row_map[row] : row) * g.n_out + n];
          } else if (EPI == EPI_HID) {
            opnd[u] = __bfloat162float(g.resid[(size_t)row * g.ld_h + n]);
          }
        }
#pragma unroll
        for (int u = 0; u < R; ++u) {
          const int lr = lr0 + u * kRowStep;
          if (lr < m) {
            const int row = row0 + lr;
            float x = acc[u] + bias;
            if (EPI == EPI_OUT) {
              g.out_f32[(size_t)row * g.n_out + n] = fmaf(cs[u], opnd[u], co[u] * x);
            } else {
              if (EPI == EPI_HID) x = opnd[u] + silu(x);
              g.out_bf16[(size_t)row * g.ld_h + n] = __float2bfloat16_rn(x);
            }
          }
        }
      }
    }
  }

  // no CTA leaves while a peer may still read its partial
  tc_fence_before();
  __syncthreads();
  __syncwarp();
  cluster_sync_all();
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(tmem_cols) : "memory");
  }
}

// ---------------------------------------------------------------------------------------------------
// The whole network in ONE launch for networks whose weights stay in L2 (a few MB).  A cluster of kFusedC CTAs
// owns a block of 128 rows for all layers; in every layer CTA r of the cluster computes the 128-column tiles
// r, r + kFusedC, ... of the layer's output with the same warp-specialised pipeline as gemm_kernel (TMA ->
// shared memory -> tcgen05.mma -> tensor memory -> fused epilogue).  A layer's output is written to global
// memory, where it stays in L2, and only the CTAs of the same cluster read it (the next layer needs all columns
// of its own 128 rows and nothing else), so the layers are chained by a CLUSTER barrier instead of a kernel
// boundary: a round of the sampler launches two of these instead of fourteen GEMM kernels.
//   - the epilogue's global stores are followed by fence.proxy.async (the next layer reads them through the
//     TMA, i.e. the async proxy) and the barrier's release / acquire orders them across the cluster;
//   - every thread of every CTA executes the same number of cluster barriers whatever the row count; the
//     mbarrier waits are bounded as everywhere else, so a CTA always gets to its barriers.
// ---------------------------------------------------------------------------------------------------
constexpr int kFusedC = 8;          // CTAs per cluster = column tiles computed side by side (beyond 8: opt-in size)
constexpr int kFusedBN = 128;       // column tile
constexpr int kFusedMaxLayers = 18; // input projection + up to 16 residual layers + output projection

struct FusedLayer {
  int k_dim, n_out, epi, a_sel, ld_out;  // a_sel: which of the three activation maps is this layer's input
  const float* bias;
  const __nv_bfloat16* resid;
  __nv_bfloat16* out_bf16;
};

struct FusedArgs {
  int n_layers;  // GEMMs in the chain
  FusedLayer L[kFusedMaxLayers];
  const int* m_dev;
  int m_cap;
  float* out_f32;
  const float* ysrc;
  const int* row_map;
  const int* row_step;
  const float* c_skip;
  const float* c_out;
  int* err;
};

struct FusedMaps {
  CUtensorMap a[3];                 // X, H0, H1 (box 128 rows x 64 columns)
  CUtensorMap w[kFusedMaxLayers];   // the layers' weights (box 128 rows x 64 columns)
};

constexpr int kFusedEpiWarps = 8;  // two per tensor-memory lane quarter, half the tile's columns each
constexpr int kFusedThreads = 64 + 32 * kFusedEpiWarps;
constexpr int kFusedColsPerWarp = kFusedBN / (kFusedEpiWarps / 4);
constexpr int kFusedSmemBytes =
    Cfg<kFusedBN>::kSmemBytes + kFusedEpiWarps * kEpiStageBytes + kFusedEpiWarps * kFusedColsPerWarp * 4 /*bias*/;

__global__ void __launch_bounds__(kFusedThreads, 1)  // launched with a cluster of kFusedC CTAs along x
mlp_fused_kernel(const __grid_constant__ FusedMaps maps, const __grid_constant__ FusedArgs F) {
  constexpr int BN = kFusedBN;
  using C = Cfg<BN>;
  constexpr int S = C::kStages;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t tiles = (raw + 1023u) & ~1023u;
  uint8_t* aux = smem_raw + (tiles - raw) + S * C::kStageBytes;
  uint64_t* bars = reinterpret_cast<uint64_t*>(aux);  // full[S], empty[S], acc_full[2], acc_empty[2]
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(aux + 8 * (2 * S + 4));
  volatile int* dead = reinterpret_cast<volatile int*>(tmem_slot + 1);
  const uint32_t bar0 = smem_u32(bars);
  auto full_bar = [&](int s) { return bar0 + 8u * s; };
  auto empty_bar = [&](int s) { return bar0 + 8u * (S + s); };
  auto accf_bar = [&](int b) { return bar0 + 8u * (2 * S + b); };
  auto acce_bar = [&](int b) { return bar0 + 8u * (2 * S + 2 + b); };

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int rank = (int)cluster_ctarank();
  const int row0 = (int)blockIdx.y * BM;

  grid_launch_dependents();
  if (threadIdx.x == 0) {
    for (int s = 0; s < S; ++s) {
      mbar_init(full_bar(s), 1);
      mbar_init(empty_bar(s), 1);
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(accf_bar(b), 1);
      mbar_init(acce_bar(b), kFusedEpiWarps);
    }
    *dead = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)),
                 "r"((uint32_t)C::kTmemCols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  // this CTA's (tile, k-block) pairs of layer l, in the order they go through the ring
  auto n_iters = [&](int l) {
    const int tn = (F.L[l].n_out + BN - 1) / BN, kb = (F.L[l].k_dim + BK - 1) / BK;
    return (rank < tn ? (tn - rank + kFusedC - 1) / kFusedC : 0) * kb;
  };
  // The weights do not depend on the previous kernel nor on the previous layer: the producer issues the weight
  // half of a layer's first stages ahead (before the dependency wait / the layer barrier) and the activation
  // half once the barrier has passed.  w_ahead = stages of the coming layer whose weight tile is already in flight.
  int stage = 0, it = 0, w_ahead = 0;
  uint32_t phase = 0;
  auto issue_w_ahead = [&](int l) {  // TMA thread only; ring cursor (stage, phase) is where layer l will start
    const int num_kb = (F.L[l].k_dim + BK - 1) / BK;
    const int total = n_iters(l);
    int st = stage;
    uint32_t ph = phase;
    w_ahead = min(S, total);
    for (int i = 0; i < w_ahead; ++i) {
      mbar_wait(empty_bar(st), ph ^ 1u, dead, F.err);
      mbar_expect_tx(full_bar(st), (uint32_t)C::kStageBytes);
      const int t = rank + (i / num_kb) * kFusedC, kb = i % num_kb;
      tma_load_2d(tiles + st * C::kStageBytes + BM * BK * 2, &maps.w[l], full_bar(st), kb * BK, t * BN);
      if (++st == S) {
        st = 0;
        ph ^= 1u;
      }
    }
  };
  if (warp == 0 && lane == 0) issue_w_ahead(0);
  grid_dependency_wait();
  const int m = min(*F.m_dev, F.m_cap);
  const bool live = row0 < m;  // the same for every CTA of the cluster: a block without rows only keeps the barriers

  for (int l = 0; l < F.n_layers; ++l) {
    const FusedLayer& P = F.L[l];
    const int tiles_n = (P.n_out + BN - 1) / BN;
    const int num_kb = (P.k_dim + BK - 1) / BK;
    if (warp == 0) {
      // ---------------- TMA producer ----------------
      if (lane == 0) {
        const CUtensorMap* ma = &maps.a[P.a_sel];
        const CUtensorMap* mw = &maps.w[l];
        int i = 0;
        for (int t = rank; t < tiles_n; t += kFusedC) {
          for (int kb = 0; kb < num_kb; ++kb, ++i) {
            const uint32_t sa = tiles + stage * C::kStageBytes;
            const uint32_t sb = sa + BM * BK * 2;
            if (i >= w_ahead) {
              mbar_wait(empty_bar(stage), phase ^ 1u, dead, F.err);
              mbar_expect_tx(full_bar(stage), (uint32_t)C::kStageBytes);
              tma_load_2d(sb, mw, full_bar(stage), kb * BK, t * BN);
            }
            // (a block without rows still loads: its tiles are all zero fill, and the ring keeps its bookkeeping)
            tma_load_2d(sa, ma, full_bar(stage), kb * BK, row0);
            if (++stage == S) {
              stage = 0;
              phase ^= 1u;
            }
          }
        }
        w_ahead = 0;
        if (l + 1 < F.n_layers) issue_w_ahead(l + 1);
      }
    } else if (warp == 1) {
      // ---------------- MMA issuer ----------------
      if (lane == 0) {
        constexpr uint32_t idesc = instr_desc<BN>();
        for (int t = rank; t < tiles_n; t += kFusedC, ++it) {
          const int acc = it & 1;
          const uint32_t acc_phase = (uint32_t)(it >> 1) & 1u;
          mbar_wait(acce_bar(acc), acc_phase ^ 1u, dead, F.err);
          tc_fence_after();
          const uint32_t d_tmem = tmem_base + (uint32_t)(acc * BN);
          for (int kb = 0; kb < num_kb; ++kb) {
            mbar_wait(full_bar(stage), phase, dead, F.err);
            tc_fence_after();
            const uint32_t sa = tiles + stage * C::kStageBytes;
            const uint32_t sb = sa + BM * BK * 2;
            const uint64_t da = smem_desc_sw128(sa), db = smem_desc_sw128(sb);
#pragma unroll
            for (int k = 0; k < BK / UMMA_K; ++k)
              tc_mma_bf16(d_tmem, da + (uint64_t)(2 * k), db + (uint64_t)(2 * k), idesc, (kb | k) != 0 ? 1u : 0u);
            tc_commit(empty_bar(stage));
            if (++stage == S) {
              stage = 0;
              phase ^= 1u;
            }
          }
          tc_commit(accf_bar(acc));
        }
      }
    } else {
      // ---------------- epilogue warps ----------------
      GemmArgs g{};
      g.n_out = P.n_out;
      g.bias = P.bias;
      g.out_bf16 = P.out_bf16;
      g.resid = P.resid;
      g.ld_h = P.ld_out;
      g.out_f32 = F.out_f32;
      g.ysrc = F.ysrc;
      g.row_map = F.row_map;
      g.row_step = F.row_step;
      g.c_skip = F.c_skip;
      g.c_out = F.c_out;
      const int quarter = warp & 3, part = (warp - kEpiWarp0) >> 2;
      constexpr int kCols = BN / (kFusedEpiWarps / 4);  // this warp's share of the tile's columns
      const int row = row0 + quarter * 32 + lane;
      const bool row_ok = row < m;
      float cs = 0.f, co = 0.f;
      const float* ysrc_row = nullptr;
      if (P.epi == EPI_OUT && row_ok) {
        const int step = F.row_step[row];
        cs = F.c_skip[step];
        co = F.c_out[step];
        ysrc_row = F.ysrc + (size_t)(F.row_map ? F.row_map[row] : row) * P.n_out;
      }
      uint8_t* buf = aux + 256 + (warp - kEpiWarp0) * kEpiStageBytes;
      float* sbias = reinterpret_cast<float*>(aux + 256 + kFusedEpiWarps * kEpiStageBytes) + (warp - kEpiWarp0) * kCols;
      for (int t = rank; t < tiles_n; t += kFusedC, ++it) {
        const int acc = it & 1;
        const uint32_t acc_phase = (uint32_t)(it >> 1) & 1u;
        const int n0 = t * BN + part * kCols;
        const bool staged = P.epi != EPI_OUT && t * BN + BN <= P.n_out && P.ld_out % 8 == 0;  // warp-uniform
        uint4 R[kCols / 32][4];
        GemmArgs gs = g;  // for the staged path: the bias of this warp's columns comes from shared memory
        if (staged) {
          if (P.epi == EPI_HID) epilogue_staged_prefetch<EPI_HID, kCols>(g, row0 + quarter * 32, lane, m, n0, R);
          // (fetched while the MMAs run: a bias read behind the accumulator wait costs an L2 round trip per chunk)
#pragma unroll
          for (int c = 0; c < kCols / 32; ++c) sbias[c * 32 + lane] = P.bias[n0 + c * 32 + lane];
          __syncwarp();
          gs.bias = sbias - n0;
        }
        mbar_wait(accf_bar(acc), acc_phase, dead, F.err);
        tc_fence_after();
        const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(acc * BN + part * kCols);
        if (staged && P.epi == EPI_HID)
          epilogue_tile_staged<EPI_HID, kCols>(gs, taddr, row0 + quarter * 32, lane, m, n0, buf, R);
        else if (staged)
          epilogue_tile_staged<EPI_IN, kCols>(gs, taddr, row0 + quarter * 32, lane, m, n0, buf, R);
        else if (P.epi == EPI_IN)
          epilogue_tile<EPI_IN, kCols, false>(g, taddr, row, row_ok, n0, cs, co, ysrc_row);
        else if (P.epi == EPI_HID)
          epilogue_tile<EPI_HID, kCols, false>(g, taddr, row, row_ok, n0, cs, co, ysrc_row);
        else
          epilogue_tile<EPI_OUT, kCols>(g, taddr, row, row_ok, n0, cs, co, ysrc_row);
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(acce_bar(acc));
      }
      // what this layer wrote is read by the TMA (async proxy) of every CTA of the cluster in the next layer
      asm volatile("fence.proxy.async.global;" ::: "memory");
    }
    // ---- end of the layer: the whole cluster has stored its tiles before anyone loads the next layer's input ----
    __syncthreads();
    __syncwarp();
    cluster_sync_all();
  }
  (void)live;

  if (warp == 0 && lane == 0) drain_after_timeout(dead);
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)C::kTmemCols)
                 : "memory");
  }
}

// Self-test of the bounded wait: one thread waits on a barrier that nothing will ever complete.  The
// wait gives up after its limit, records ASD_ERR_TIMEOUT in the error word and the kernel returns.
__global__ void wait_selftest_kernel(int* err) {
  __shared__ uint64_t bar;
  __shared__ int dead;
  if (threadIdx.x == 0) {
    mbar_init(smem_u32(&bar), 1);
    dead = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    mbar_wait(smem_u32(&bar), 0u, &dead, err);
  }
}

// ---- host side --------------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = nullptr;
  if (!fn) {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) == cudaSuccess &&
        qres == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(p);
  }
  return fn;
}

// 2-D bf16 row-major tensor [rows, cols] (cols contiguous), box = [box_rows, 64 cols], 128-byte swizzle.
bool get_tmap(Ctx* c, const void* ptr, int rows, int cols, int box_rows, CUtensorMap* out) {
  auto key = std::make_tuple(ptr, rows, cols, box_rows);
  auto it = c->tmaps.find(key);
  if (it != c->tmaps.end()) {
    *out = it->second;
    return true;
  }
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
  cuuint64_t strides[1] = {(cuuint64_t)cols * 2};
  cuuint32_t box[2] = {(cuuint32_t)BK, (cuuint32_t)box_rows};
  cuuint32_t estr[2] = {1, 1};
  CUtensorMap m;
  CUresult r = fn(&m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(ptr), dims, strides, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) return false;
  c->tmaps[key] = m;
  *out = m;
  return true;
}

// The opt-in to more than 48 KB of dynamic shared memory is a per-device attribute of the kernel; a
// context belongs to one device, so it remembers what it has set (the largest size asked for so far).
void ensure_dynamic_smem(Ctx* c, const void* func, int bytes) {
  int& have = c->func_smem[func];
  if (bytes > have) {
    cudaFuncSetAttribute(func, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
    have = bytes;
  }
}

template <int BN, int EPI>
asd_status launch_gemm_t(Ctx* c, const void* a_ptr, int a_cols, const void* w_ptr, const GemmArgs& g, int m_bound) {
  using C = Cfg<BN>;
  CUtensorMap ma, mw;
  if (!get_tmap(c, a_ptr, g.m_cap, a_cols, BM, &ma) || !get_tmap(c, w_ptr, g.n_out, a_cols, BN, &mw)) {
    c->err = "cuTensorMapEncodeTiled failed";
    return ASD_ERR_CUDA;
  }
  ensure_dynamic_smem(c, reinterpret_cast<const void*>(&gemm_kernel<BN, EPI>), C::kSmemBytes);
  const int tiles = ((m_bound + BM - 1) / BM) * ((g.n_out + BN - 1) / BN);
  const int grid = tiles < c->num_sms ? (tiles < 1 ? 1 : tiles) : c->num_sms;
  gemm_kernel<BN, EPI><<<grid, kGemmThreads, C::kSmemBytes, c->stream>>>(ma, mw, g);
  c->launches++;
  return ASD_OK;
}

template <int BN, int EPI>
asd_status launch_gemm_pair_t(Ctx* c, const void* a_ptr, int a_cols, const void* w_ptr, const GemmArgs& g, int m_bound) {
  using C = PairCfg<BN>;
  CUtensorMap ma, mw;
  if (!get_tmap(c, a_ptr, g.m_cap, a_cols, BM, &ma) || !get_tmap(c, w_ptr, g.n_out, a_cols, BN / 2, &mw)) {
    c->err = "cuTensorMapEncodeTiled failed";
    return ASD_ERR_CUDA;
  }
  ensure_dynamic_smem(c, reinterpret_cast<const void*>(&gemm_pair_kernel<BN, EPI>), C::kSmemBytes);
  const int tiles = ((m_bound + 2 * BM - 1) / (2 * BM)) * ((g.n_out + BN - 1) / BN);
  const int pairs = std::max(1, std::min(tiles, c->num_sms / 2));
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(2 * pairs);
  cfg.blockDim = dim3(kPairThreads);
  cfg.dynamicSmemBytes = (size_t)C::kSmemBytes;
  cfg.stream = c->stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  if (cudaLaunchKernelEx(&cfg, gemm_pair_kernel<BN, EPI>, ma, mw, g) != cudaSuccess) {
    c->err = std::string("pair GEMM launch failed: ") + cudaGetErrorString(cudaGetLastError());
    return ASD_ERR_CUDA;
  }
  c->launches++;
  return ASD_OK;
}

template <int EPI>
asd_status launch_gemm_skinny(Ctx* c, const void* a_ptr, int a_cols, const void* w_ptr, const GemmArgs& g, int m_bound) {
  const int m_pad = std::min(kSkinnyBlockRows, std::max(16, (m_bound + 15) / 16 * 16));
  const int row_blocks = (m_bound + m_pad - 1) / m_pad;
  CUtensorMap mx, mw;
  if (!get_tmap(c, a_ptr, g.m_cap, a_cols, m_pad, &mx) || !get_tmap(c, w_ptr, g.n_out, a_cols, BM, &mw)) {
    c->err = "cuTensorMapEncodeTiled failed";
    return ASD_ERR_CUDA;
  }
  const int budget = m_pad <= 128 ? kSkinnySmallBudget : kSkinnyStageBudget;
  const int stages = std::max(2, std::min(kSkinnyMaxStages, budget / skinny_stage_bytes(m_pad)));
  const int smem = std::max(stages * skinny_stage_bytes(m_pad), m_pad * BM * 4) + 1024 + 256;
  ensure_dynamic_smem(c, reinterpret_cast<const void*>(&gemm_skinny_kernel<EPI>), smem);
  const dim3 grid(((g.n_out + BM - 1) / BM) * kSplit, row_blocks);
  // Programmatic dependent launch: this kernel may begin (barriers, tensor memory, first weight tiles)
  // while the previous kernel of the stream is still finishing; it waits for it before it touches
  // anything that kernel wrote.
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = dim3(m_pad > 32 ? kSkinnyThreads : kGemmThreads);  // a second set of epilogue warps pays from 33 rows
  cfg.dynamicSmemBytes = (size_t)smem;
  cfg.stream = c->stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  if (cudaLaunchKernelEx(&cfg, gemm_skinny_kernel<EPI>, mw, mx, g, m_pad, stages) != cudaSuccess) {
    c->err = std::string("skinny GEMM launch failed: ") + cudaGetErrorString(cudaGetLastError());
    return ASD_ERR_CUDA;
  }
  c->launches++;
  return ASD_OK;
}

// Few rows: weight streaming with swapped operands.  (ASD_GEMM_MODE=cta|pair, read at asd_create, pins the
// tiled kernels.)
bool use_skinny(const Ctx* c, int m_bound) { return c->gemm_mode == 0 && m_bound <= kSkinnyMaxRows; }

// Which kernel and column-tile width serve a [m x k] x [n x k]^T product best.  Model: every SM fills
// its shared memory from L2 at about 50 bytes per clock and its tensor pipe retires a 128 x 256 x 64
// block in 512 clocks; a launch takes (waves of tiles) x (k-blocks) x max(fill, math) clocks.
struct GemmPlan {
  bool pair;
  int bn;
};

GemmPlan plan_gemm(const Ctx* c, int m_bound, int n_out) {
  const int mode = c->gemm_mode;  // tuning aid: 1 ("cta") or 2 ("pair") pins the kernel family
  const double fill_rate = 50.0;
  GemmPlan best{false, 32};
  double best_t = 1e300;
  const int cand[4] = {256, 128, 64, 32};
  for (int pair = 0; pair < 2; ++pair) {
    if ((mode == 1 && pair) || (mode == 2 && !pair)) continue;
    const int units = pair ? c->num_sms / 2 : c->num_sms;
    const int tm = pair ? 2 * BM : BM;
    for (int i = 0; i < (pair ? 3 : 4); ++i) {
      const int bn = cand[i];
      if (pair && n_out % (bn / 2) != 0) continue;  // each CTA of a pair stages a whole half tile of W
      const long long tiles = (long long)((m_bound + tm - 1) / tm) * ((n_out + bn - 1) / bn);
      const double waves = (double)((tiles + units - 1) / units);
      const double fill = (BM + (pair ? bn / 2 : bn)) * (BK * 2) / fill_rate;
      const double math = 512.0 * bn / 256.0;
      const double t = waves * std::max(fill, math);
      if (t < best_t * 0.999) {
        best_t = t;
        best = GemmPlan{pair != 0, bn};
      }
    }
  }
  return best;
}

template <int EPI>
asd_status launch_gemm(Ctx* c, const void* a_ptr, int a_cols, const void* w_ptr, const GemmArgs& g, int m_bound) {
  if (use_skinny(c, m_bound)) return launch_gemm_skinny<EPI>(c, a_ptr, a_cols, w_ptr, g, m_bound);
  const GemmPlan p = plan_gemm(c, m_bound, g.n_out);
  if (p.pair) {
    switch (p.bn) {
      case 256: return launch_gemm_pair_t<256, EPI>(c, a_ptr, a_cols, w_ptr, g, m_bound);
      case 128: return launch_gemm_pair_t<128, EPI>(c, a_ptr, a_cols, w_ptr, g, m_bound);
      default: return launch_gemm_pair_t<64, EPI>(c, a_ptr, a_cols, w_ptr, g, m_bound);
    }
  }
  switch (p.bn) {
    case 256: return launch_gemm_t<256, EPI>(c, a_ptr, a_cols, w_ptr, g, m_bound);
    case 128: return launch_gemm_t<128, EPI>(c, a_ptr, a_cols, w_ptr, g, m_bound);
    case 64: return launch_gemm_t<64, EPI>(c, a_ptr, a_cols, w_ptr, g, m_bound);
    default: return launch_gemm_t<32, EPI>(c, a_ptr, a_cols, w_ptr, g, m_bound);
  }
}

// Whether the one-launch network serves this pass.  Only on request (ASD_MLP_FUSED=1 at asd_create): measured on
// B200 it does not beat the chain of per-layer kernels.  Every CTA of a cluster has to pull the cluster's whole
// 128-row activation block through its own L2 -> shared-memory path in every layer (256 KB at width 1024, on top of
// its share of the weights), and that path is what bounds these kernels (50 - 66 bytes per clock and SM here); with
// the SiLU epilogue (two special-function operations per element) and the cluster barrier a layer costs 13 - 18
// thousand cycles against 11 - 15 for a per-layer kernel whose launch overlaps its predecessor.  Sharing the
// activation tile across the cluster by TMA multicast would remove most of that traffic; multicast loads are not
// used in this library.
bool fused_ready(Ctx* c);

bool use_fused_mlp(Ctx* c, int m_bound) {
  const MlpParams& M = c->mlp;
  if (c->fused_mode != 1 || M.n_layers + 2 > kFusedMaxLayers || c->gemm_mode != 0) return false;
  (void)m_bound;
  return c->fused_mode == 1 && fused_ready(c);
}

// Once per context: the shared-memory and cluster-size opt-ins of the kernel, and whether the device can co-schedule
// at least one cluster of kFusedC such CTAs at all (1 ready, -1 not).
bool fused_ready(Ctx* c) {
  if (c->fused_ready != 0) return c->fused_ready > 0;
  c->fused_ready = -1;
  const void* fn = reinterpret_cast<const void*>(&mlp_fused_kernel);
  ensure_dynamic_smem(c, fn, kFusedSmemBytes);
  if (kFusedC > 8 && cudaFuncSetAttribute(fn, cudaFuncAttributeNonPortableClusterSizeAllowed, 1) != cudaSuccess) {
    cudaGetLastError();
    return false;
  }
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(kFusedC, 1);
  cfg.blockDim = dim3(kFusedThreads);
  cfg.dynamicSmemBytes = (size_t)kFusedSmemBytes;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = kFusedC;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  int clusters = 0;
  if (cudaOccupancyMaxActiveClusters(&clusters, mlp_fused_kernel, &cfg) != cudaSuccess || clusters < 1) {
    cudaGetLastError();
    return false;
  }
  c->fused_clusters = clusters;
  c->fused_ready = 1;
  return true;
}

asd_status launch_mlp_fused(Ctx* c, const RowSet& rs, float* out) {
  const MlpParams& M = c->mlp;
  FusedMaps maps;
  FusedArgs F{};
  const void* abuf[3] = {M.X, M.H[0], M.H[1]};
  const int acols[3] = {M.in_pad, M.width, M.width};
  for (int i = 0; i < 3; ++i)
    if (!get_tmap(c, abuf[i], M.row_cap, acols[i], BM, &maps.a[i])) {
      c->err = "cuTensorMapEncodeTiled failed";
      return ASD_ERR_CUDA;
    }
  int n = 0;
  auto add = [&](const void* w, int k_dim, int n_out, int epi, int a_sel, const float* bias, const __nv_bfloat16* resid,
                 __nv_bfloat16* out_bf16) -> bool {
    if (!get_tmap(c, w, n_out, k_dim, kFusedBN, &maps.w[n])) return false;
    F.L[n] = FusedLayer{k_dim, n_out, epi, a_sel, M.width, bias, resid, out_bf16};
    ++n;
    return true;
  };
  bool ok = add(M.W_in, M.in_pad, M.width, EPI_IN, 0, M.b_in, nullptr, M.H[0]);
  for (int l = 0; l < M.n_layers && ok; ++l)
    ok = add(M.W_hid + (size_t)l * M.width * M.width, M.width, M.width, EPI_HID, 1 + (l & 1), M.b_hid + (size_t)l * M.width,
             M.H[l & 1], M.H[(l + 1) & 1]);
  ok = ok && add(M.W_out, M.width, c->d, EPI_OUT, 1 + (M.n_layers & 1), M.b_out, nullptr, nullptr);
  if (!ok) {
    c->err = "cuTensorMapEncodeTiled failed";
    return ASD_ERR_CUDA;
  }
  F.n_layers = n;
  F.m_dev = rs.n_rows_dev;
  F.m_cap = M.row_cap;
  F.out_f32 = out;
  F.ysrc = rs.ysrc;
  F.row_map = rs.row_map;
  F.row_step = rs.row_step;
  F.c_skip = c->tab.c_skip;
  F.c_out = c->tab.c_out;
  F.err = &c->counters->err;
  if (!fused_ready(c)) {
    c->err = "fused network kernel: a cluster of this size cannot be scheduled on this device";
    return ASD_ERR_UNSUPPORTED;
  }
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(kFusedC, (rs.n_rows_max + BM - 1) / BM);
  cfg.blockDim = dim3(kFusedThreads);
  cfg.dynamicSmemBytes = (size_t)kFusedSmemBytes;
  cfg.stream = c->stream;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  attr[1].id = cudaLaunchAttributeClusterDimension;
  attr[1].val.clusterDim.x = kFusedC;
  attr[1].val.clusterDim.y = 1;
  attr[1].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 2;
  if (cudaLaunchKernelEx(&cfg, mlp_fused_kernel, maps, F) != cudaSuccess) {
    c->err = std::string("fused network launch failed: ") + cudaGetErrorString(cudaGetLastError());
    return ASD_ERR_CUDA;
  }
  c->launches++;
  return ASD_OK;
}

}  // namespace

void launch_wait_selftest(Ctx* c) {
  wait_selftest_kernel<<<1, 32, 0, c->stream>>>(&c->counters->err);
  c->launches++;
}

asd_status mlp_forward(Ctx* c, const RowSet& rs, float* out, int pass) {
  const MlpParams& M = c->mlp;
  const int m_bound = rs.n_rows_max;
  if (m_bound <= 0) return ASD_OK;
  GemmArgs g{};
  g.m_dev = rs.n_rows_dev;
  g.m_settled = rs.settled ? 1 : 0;
  g.m_cap = M.row_cap;
  g.err = &c->counters->err;
  asd_status st;
  if (use_fused_mlp(c, m_bound)) {
    // the whole chain in one launch; its time is booked under the hidden-layer phase
    ProfScope ps(pass < 2 ? c : nullptr, pass == 0 ? PH_D1_HID : PH_D2_HID);
    return launch_mlp_fused(c, rs, out);
  }
  // input projection
  g.n_out = M.width;
  g.k_dim = M.in_pad;
  g.bias = M.b_in;
  g.out_bf16 = M.H[0];
  g.ld_h = M.width;
  const int ph_in = pass == 0 ? PH_D1_IN : PH_D2_IN, ph_hid = pass == 0 ? PH_D1_HID : PH_D2_HID,
            ph_out = pass == 0 ? PH_D1_OUT : PH_D2_OUT;
  {
    ProfScope ps(pass < 2 ? c : nullptr, ph_in);
    st = launch_gemm<EPI_IN>(c, M.X, M.in_pad, M.W_in, g, m_bound);
  }
  if (st != ASD_OK) return st;
  {
    ProfScope ps(pass < 2 ? c : nullptr, ph_hid);
    // residual layers
    for (int l = 0; l < M.n_layers; ++l) {
      g.k_dim = M.width;
      g.bias = M.b_hid + (size_t)l * M.width;
      g.resid = M.H[l & 1];
      g.out_bf16 = M.H[(l + 1) & 1];
      st = launch_gemm<EPI_HID>(c, M.H[l & 1], M.width, M.W_hid + (size_t)l * M.width * M.width, g, m_bound);
      if (st != ASD_OK) return st;
    }
  }
  // output projection with the skip / scale epilogue
  g.n_out = c->d;
  g.k_dim = M.width;
  g.bias = M.b_out;
  g.out_bf16 = nullptr;
  g.resid = nullptr;
  g.out_f32 = out;
  g.ysrc = rs.ysrc;
  g.row_map = rs.row_map;
  g.row_step = rs.row_step;
  g.c_skip = c->tab.c_skip;
  g.c_out = c->tab.c_out;
  ProfScope ps_out(pass < 2 ? c : nullptr, ph_out);
  return launch_gemm<EPI_OUT>(c, M.H[M.n_layers & 1], M.width, M.W_out, g, m_bound);
}

}  // namespace asd

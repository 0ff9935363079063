// Device-side building blocks of the tensor-core kernels (asd_gemm.cu, asd_mlp_fused.cu): tile constants, the
// argument block of a GEMM launch, inline-PTX wrappers (mbarrier with bounded waits, TMA, tcgen05 MMA / commit / load,
// cluster addressing), shared-memory and instruction descriptors, and the fused epilogues (direct, and staged through
// shared memory so that global accesses move whole 64-byte row pieces).  Everything here has internal linkage.
#pragma once

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

// The tail of a residual layer on the un-rounded fp32 accumulator: z = acc + bias, then resid + z sigmoid(z) with
// sigmoid(z) = 1 / (1 + 2^(-z log2 e)) from ex2.approx and rcp.approx (relative error ~2^-22, far below the bf16
// rounding that follows; z -> -inf gives 2^(+inf) = inf, 1 / inf = 0, the right limit).  Every step is spelled out
// (no contraction left to the compiler), so the scalar form and the packed form below, which does two columns per
// instruction with sm_100's two-way fp32 add / mul / fma, return the same bits in every kernel that uses them.
constexpr float kNegLog2e = -1.4426950408889634f;
__device__ __forceinline__ float ex2_approx(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ float rcp_approx(float x) {
  float y;
  asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ float hid_tail(float acc, float bias, float resid) {
  const float z = __fadd_rn(acc, bias);
  const float e = ex2_approx(__fmul_rn(z, kNegLog2e));
  const float r = rcp_approx(__fadd_rn(1.0f, e));
  return __fmaf_rn(z, r, resid);
}
__device__ __forceinline__ float2 add2(float2 a, float2 b) {
  float2 c;
  asm("{\n\t.reg .b64 pa, pb, pc;\n\tmov.b64 pa, {%2, %3};\n\tmov.b64 pb, {%4, %5};\n\t"
      "add.rn.f32x2 pc, pa, pb;\n\tmov.b64 {%0, %1}, pc;\n\t}"
      : "=f"(c.x), "=f"(c.y)
      : "f"(a.x), "f"(a.y), "f"(b.x), "f"(b.y));
  return c;
}
__device__ __forceinline__ float2 mul2(float2 a, float2 b) {
  float2 c;
  asm("{\n\t.reg .b64 pa, pb, pc;\n\tmov.b64 pa, {%2, %3};\n\tmov.b64 pb, {%4, %5};\n\t"
      "mul.rn.f32x2 pc, pa, pb;\n\tmov.b64 {%0, %1}, pc;\n\t}"
      : "=f"(c.x), "=f"(c.y)
      : "f"(a.x), "f"(a.y), "f"(b.x), "f"(b.y));
  return c;
}
__device__ __forceinline__ float2 fma2(float2 a, float2 b, float2 c) {
  float2 d;
  asm("{\n\t.reg .b64 pa, pb, pc, pd;\n\tmov.b64 pa, {%2, %3};\n\tmov.b64 pb, {%4, %5};\n\tmov.b64 pc, {%6, %7};\n\t"
      "fma.rn.f32x2 pd, pa, pb, pc;\n\tmov.b64 {%0, %1}, pd;\n\t}"
      : "=f"(d.x), "=f"(d.y)
      : "f"(a.x), "f"(a.y), "f"(b.x), "f"(b.y), "f"(c.x), "f"(c.y));
  return d;
}
// hid_tail on two neighbouring columns
__device__ __forceinline__ float2 hid_tail2(float2 acc, float2 bias, float2 resid) {
  const float2 z = add2(acc, bias);
  const float2 t = mul2(z, make_float2(kNegLog2e, kNegLog2e));
  const float2 den = add2(make_float2(1.0f, 1.0f), make_float2(ex2_approx(t.x), ex2_approx(t.y)));
  return fma2(z, make_float2(rcp_approx(den.x), rcp_approx(den.y)), resid);
}

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
        if (EPI == EPI_HID) {
          const uint4 rv = *reinterpret_cast<const uint4*>(rrow + col0 + e);
          const __nv_bfloat162* rp = reinterpret_cast<const __nv_bfloat162*>(&rv);
#pragma unroll
          for (int u = 0; u < 4; ++u) {
            const float2 rf = __bfloat1622float2(rp[u]);
            x[2 * u] = hid_tail(__uint_as_float(r[e + 2 * u]), bb[2 * u], rf.x);
            x[2 * u + 1] = hid_tail(__uint_as_float(r[e + 2 * u + 1]), bb[2 * u + 1], rf.y);
          }
        } else {
#pragma unroll
          for (int u = 0; u < 8; ++u) x[u] = __fadd_rn(__uint_as_float(r[e + u]), bb[u]);
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
          const float x = EPI == EPI_HID ? hid_tail(__uint_as_float(r[e]), g.bias[col], __bfloat162float(rrow[col]))
                                         : __fadd_rn(__uint_as_float(r[e]), g.bias[col]);
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
      if (EPI == EPI_HID) {
        const uint4 rv = op.v[e >> 3];
        const __nv_bfloat162* rp = reinterpret_cast<const __nv_bfloat162*>(&rv);
#pragma unroll
        for (int u = 0; u < 4; ++u) {
          const float2 rf = __bfloat1622float2(rp[u]);
          x[2 * u] = hid_tail(__uint_as_float(r[e + 2 * u]), bb[2 * u], rf.x);
          x[2 * u + 1] = hid_tail(__uint_as_float(r[e + 2 * u + 1]), bb[2 * u + 1], rf.y);
        }
      } else {
#pragma unroll
        for (int u = 0; u < 8; ++u) x[u] = __fadd_rn(__uint_as_float(r[e + u]), bb[u]);
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
      if (EPI == EPI_HID) {
        const uint4 rv = *reinterpret_cast<const uint4*>(buf + epi_slot(lane, e >> 3));
        const __nv_bfloat162* rp = reinterpret_cast<const __nv_bfloat162*>(&rv);
#pragma unroll
        for (int u = 0; u < 4; ++u) {
          const float2 o2 = hid_tail2(make_float2(__uint_as_float(r[e + 2 * u]), __uint_as_float(r[e + 2 * u + 1])),
                                      make_float2(bb[2 * u], bb[2 * u + 1]), __bfloat1622float2(rp[u]));
          x[2 * u] = o2.x;
          x[2 * u + 1] = o2.y;
        }
      } else {
#pragma unroll
        for (int u = 0; u < 4; ++u) {
          const float2 o2 = add2(make_float2(__uint_as_float(r[e + 2 * u]), __uint_as_float(r[e + 2 * u + 1])),
                                 make_float2(bb[2 * u], bb[2 * u + 1]));
          x[2 * u] = o2.x;
          x[2 * u + 1] = o2.y;
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

}  // namespace
}  // namespace asd

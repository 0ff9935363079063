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
#include "asd_tc.cuh"

namespace asd {

namespace {

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
            if (EPI == EPI_OUT) {
              const float x = acc[u] + bias;
              g.out_f32[(size_t)row * g.n_out + n] = fmaf(cs[u], opnd[u], co[u] * x);
            } else {
              const float x = EPI == EPI_HID ? hid_tail(acc[u], bias, opnd[u]) : __fadd_rn(acc[u], bias);
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
}  // namespace

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

namespace {

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

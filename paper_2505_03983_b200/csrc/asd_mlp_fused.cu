// The network denoiser as ONE launch (opt-in, ASD_MLP_FUSED=1): a cluster of CTAs per 128 rows, the layers chained by
// cluster barriers.  Shares the tile pipeline and the epilogues of the per-layer kernels (asd_tc.cuh).
#include <algorithm>

#include "asd_internal.h"
#include "asd_tc.cuh"

namespace asd {

namespace {

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

}  // namespace

// Whether the one-launch network serves this pass.  Only on request (ASD_MLP_FUSED=1 at asd_create): measured on
// B200 it does not beat the chain of per-layer kernels.  Every CTA of a cluster has to pull the cluster's whole
// 128-row activation block through its own L2 -> shared-memory path in every layer (256 KB at width 1024, on top of
// its share of the weights), and that path is what bounds these kernels (50 - 66 bytes per clock and SM here); with
// the SiLU epilogue (two special-function operations per element) and the cluster barrier a layer costs 13 - 18
// thousand cycles against 11 - 15 for a per-layer kernel whose launch overlaps its predecessor.  Sharing the
// activation tile across the cluster by TMA multicast would remove most of that traffic; multicast loads are not
// used in this library.
static bool fused_ready(Ctx* c);

bool use_fused_mlp(Ctx* c, int m_bound) {
  const MlpParams& M = c->mlp;
  if (c->fused_mode != 1 || M.n_layers + 2 > kFusedMaxLayers || c->gemm_mode != 0) return false;
  (void)m_bound;
  return c->fused_mode == 1 && fused_ready(c);
}

// Once per context: the shared-memory and cluster-size opt-ins of the kernel, and whether the device can co-schedule
// at least one cluster of kFusedC such CTAs at all (1 ready, -1 not).
static bool fused_ready(Ctx* c) {
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

}  // namespace asd

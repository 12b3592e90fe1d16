// Dense projections Y = X * W^T on pairs of SMs (tcgen05.mma.cta_group::2).
//
// A decode step multiplies a few hundred activation rows with every weight matrix once, so the
// weights stream from HBM exactly once and the activation tile is what gets re-read (from L2).
// With one CTA per tile the activation bytes an SM pulls equal the weight bytes, the shared-memory
// ports carry both the TMA fill and two operand reads per MMA, and a 256-feature tile leaves a
// 256 KiB fp32 partial per CTA for the k-split to add into the output through L2.  Pairing two SMs
// halves all three: the pair's MMA is 256 features x BNB rows, each CTA stages its own 128 weight
// rows plus HALF of the activation rows, the tensor core reads the other half from the partner's
// shared memory, and each CTA ends up with 128 features x BNB rows in its own tensor memory.
//
//   ACC = 1  linear epilogues (store / residual add).  Tiles are split along K so that every SM
//            pair has work; the k-slices add their fp32 partial tiles into the output with TMA
//            reduce-adds (the order of those additions is not fixed).
//   ACC = 2  SwiGLU.  Accumulator 0 holds 128 gate features, accumulator 1 the matching 128 up
//            features, so a thread finds gate and up of one feature in its own TMEM lane and the
//            activation is computed in registers.  Never split along K (not linear).
//
// Roles per CTA: warp 0 = TMA producer (own weight rows, own half of the rows), warp 1 = TMEM
// allocation and, in the pair's first CTA only, the MMA issuer; warps 2..17 = epilogue.
// Both CTAs' loads report to the first CTA's "full" barriers; its MMA commits are multicast to
// both CTAs' "empty" and "accumulator ready" barriers.  Every wait is bounded.

#include <algorithm>

#include "common.cuh"
#include "ptx.cuh"

namespace echo {

using namespace ptx;

namespace {

constexpr int kPairEpiWarps = 16;
constexpr int kPairEpiThreads = 32 * kPairEpiWarps;
constexpr int kPairThreads = 64 + kPairEpiThreads;
constexpr int kPairFeat = 128;                 // features per CTA (TMEM lanes)

template <int BNB, int ACC>
struct PairSmem {
  static constexpr int kWBlock = kPairFeat * kGemmTileK * 2;            // 16 KiB
  static constexpr int kWBytes = ACC * kWBlock;
  static constexpr int kXRows = BNB / 2;                                 // activation rows this CTA stages
  static constexpr int kXBytes = kXRows * kGemmTileK * 2;
  static constexpr int kStageBytes = kWBytes + kXBytes;
  static constexpr int kOutBytes = ACC == 1 ? BNB * kPairFeat * 4 : BNB * kPairFeat * 2;   // epilogue staging
  static constexpr int kBudget = 196 * 1024;
  static constexpr int kStagesFit = kBudget / kStageBytes;
  static constexpr int kStagesMin = (kOutBytes + kStageBytes - 1) / kStageBytes;            // staging reuses the stages
  static constexpr int kStagesCap = kStagesFit > 8 ? 8 : kStagesFit;
  static constexpr int kStages = kStagesCap < kStagesMin ? kStagesMin : kStagesCap;
  static constexpr int kTotal = kStages * kStageBytes + 1024 /* barriers */ + 1024 /* alignment */;
  static constexpr int kTmemCols = ACC * BNB < 32 ? 32 : ACC * BNB;     // 32 .. 512, a power of two
  static_assert(kStages * kStageBytes >= kOutBytes, "epilogue staging must fit in the stages");
  static_assert(kTotal <= 227 * 1024, "shared memory");
};

__device__ __forceinline__ float silu_pair(float a) { return a / (1.0f + __expf(-a)); }
__device__ __forceinline__ void pair_epi_bar() {
  asm volatile("bar.sync 1, %0;" ::"n"(kPairEpiThreads) : "memory");
}
__device__ __forceinline__ void pair_cluster_sync() {
  asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
  asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ uint32_t cluster_rank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
__device__ __forceinline__ uint32_t map_to_cta(uint32_t cta_addr, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(cta_addr), "r"(rank));
  return r;
}
// ---- cta_group::2 forms of the tcgen05 / TMA instructions --------------------------------------
__device__ __forceinline__ void tc2_alloc(uint32_t *slot, uint32_t cols) {
  asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(slot)), "r"(cols)
               : "memory");
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tc2_dealloc(uint32_t base, uint32_t cols) {
  asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(base), "r"(cols) : "memory");
}
// arrive on the barrier at this shared-memory offset in both CTAs of the pair once every MMA
// issued so far has completed
__device__ __forceinline__ void tc2_commit_both(uint64_t *bar) {
  const uint16_t mask = 3;
  asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
               ::"r"(smem_u32(bar)), "h"(mask)
               : "memory");
}
__device__ __forceinline__ void tc2_mma_bf16(uint32_t tmem_d, uint64_t desc_a, uint64_t desc_b, uint32_t idesc,
                                             uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(tmem_d), "l"(desc_a), "l"(desc_b), "r"(idesc), "r"(accumulate)
      : "memory");
}
// tile load into this CTA's shared memory whose completion is reported to a barrier that may
// live in the partner CTA (cluster address)
__device__ __forceinline__ void tma2_load_2d(const CUtensorMap *map, uint32_t bar_cluster_addr, void *dst, int c0,
                                             int c1) {
  asm volatile(
      "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], "
      "[%2];"
      ::"r"(smem_u32(dst)), "l"(reinterpret_cast<uint64_t>(map)), "r"(bar_cluster_addr), "r"(c0), "r"(c1)
      : "memory");
}
// bf16 x bf16 -> fp32, both operands K-major, M = 256 across the pair, N = n
__host__ __device__ constexpr uint32_t instr_desc_pair(int n) {
  return (1u << 4) | (1u << 7) | (1u << 10) | (static_cast<uint32_t>(n >> 3) << 17) | (16u << 24);
}

__device__ __forceinline__ int ld_acquire_gpu(const int *p) {
  int v;
  asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ void fence_proxy_async_all() { asm volatile("fence.proxy.async;" ::: "memory"); }

// RMSNorm prologue, run by the 512 epilogue threads of every CTA before the accumulators are due:
// rows blockIdx.x, blockIdx.x + gridDim.x, ... of x are normalised into h (two passes over a row that
// stays in L1/L2), then the CTA arrives at the grid-wide barrier.
__device__ __forceinline__ void norm_rows_and_arrive(const NormPrologue &np, int M, int d, bool half_out,
                                                     float *scratch /* 32 floats, shared */) {
  const int tid = threadIdx.x - 64;                        // 0 .. kPairEpiThreads - 1
  const int warp = tid >> 5, lane = tid & 31;
  uint16_t *h = static_cast<uint16_t *>(np.h);
  for (int r = blockIdx.x; r < M; r += gridDim.x) {
    const float *xr = np.x + static_cast<size_t>(r) * d;
    float ss = 0.f;
    for (int i = tid * 4; i < d; i += kPairEpiThreads * 4) {
      const float4 v = __ldcg(reinterpret_cast<const float4 *>(xr + i));
      ss = fmaf(v.x, v.x, fmaf(v.y, v.y, fmaf(v.z, v.z, fmaf(v.w, v.w, ss))));
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
    if (lane == 0) scratch[warp] = ss;
    pair_epi_bar();
    float tot = 0.f;
#pragma unroll
    for (int w = 0; w < kPairEpiWarps; ++w) tot += scratch[w];      // same order in every thread
    pair_epi_bar();
    const float scale = rsqrtf(tot / static_cast<float>(d) + np.eps);
    for (int i = tid * 4; i < d; i += kPairEpiThreads * 4) {
      const float4 v = __ldcg(reinterpret_cast<const float4 *>(xr + i));
      const uint2 graw = *reinterpret_cast<const uint2 *>(np.gain + i);
      const float2 g0 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(&graw.x));
      const float2 g1 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(&graw.y));
      uint2 o;
      o.x = cvt16x2(v.x * scale * g0.x, v.y * scale * g0.y, half_out);
      o.y = cvt16x2(v.z * scale * g1.x, v.w * scale * g1.y, half_out);
      *reinterpret_cast<uint2 *>(h + static_cast<size_t>(r) * d + i) = o;
    }
  }
  __threadfence();
  fence_proxy_async_all();                                 // the rows are read by other CTAs' tile copies
  pair_epi_bar();
  if (tid == 0) atomicAdd(&np.bar[0], 1);                  // bar[0] counts the CTAs whose rows are written
}

template <int BNB, int ACC>
__global__ void __launch_bounds__(kPairThreads, 1)
gemm_pair_kernel(const __grid_constant__ CUtensorMap tmW, const __grid_constant__ CUtensorMap tmX,
                 const __grid_constant__ CUtensorMap tmY, int M, int N, int K, int epilogue, int split,
                 int tiled, int half_in, int *status, NormPrologue np) {
  __shared__ float norm_scratch[32];
  using S = PairSmem<BNB, ACC>;
  extern __shared__ uint8_t smem_raw[];
  uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint64_t *full_bar = reinterpret_cast<uint64_t *>(smem + S::kStages * S::kStageBytes);
  uint64_t *empty_bar = full_bar + S::kStages;
  uint64_t *acc_full = empty_bar + S::kStages;
  uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(acc_full + 1);
  volatile int *abort_flag = reinterpret_cast<volatile int *>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const uint32_t rank = cluster_rank();                // 0 = the CTA that issues the pair's MMAs
  // pairs are numbered with the row tile fastest: the pairs that share a weight tile run side by side,
  // so the tile comes from HBM once and from L2 for the other row tiles
  const int m_tiles = (M + BNB - 1) / BNB;
  const int pair = (blockIdx.x >> 1) / m_tiles;
  const int nt = pair / split;
  const int slice = pair % split;
  const int m0 = ((blockIdx.x >> 1) % m_tiles) * BNB;
  const int KB = (K + kGemmTileK - 1) / kGemmTileK;
  const int kq = KB / split, kr = KB % split;
  const int kb_beg = slice * kq + min(slice, kr);
  const int kb_len = kq + (slice < kr ? 1 : 0);
  const int f0 = nt * 2 * kPairFeat + static_cast<int>(rank) * kPairFeat;   // first feature of this CTA

  if (threadIdx.x == 0) {
    for (int s = 0; s < S::kStages; ++s) {
      mbar_init(&full_bar[s], 1);
      mbar_init(&empty_bar[s], 1);
    }
    mbar_init(acc_full, 1);
    *abort_flag = 0;
    mbar_fence_init();
    // fetch the three tensor maps now, not at the first copy that uses each of them
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&tmW)) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&tmX)) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&tmY)) : "memory");
  }
  if (warp == 1) tc2_alloc(tmem_slot, S::kTmemCols);
  tc_fence_before();
  pair_cluster_sync();                                 // both CTAs' barriers exist before anything signals them
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  griddep_launch();

  if (warp == 0) {
    if (lane == 0) {
      // One stage = this CTA's weight rows (ACC blocks) and its half of the activation rows.  The
      // first CTA's barrier counts the bytes of both CTAs.  Weights do not depend on the preceding
      // kernel, so the pipeline is filled with them before waiting for it.
      auto load_w = [&](int it) {
        const int s = it % S::kStages;
        uint8_t *dst = smem + s * S::kStageBytes;
        const uint32_t bar = map_to_cta(smem_u32(&full_bar[s]), 0);
        if (rank == 0) mbar_expect_tx(&full_bar[s], 2 * S::kStageBytes);
        const int kb = kb_beg + it;
#pragma unroll
        for (int a = 0; a < ACC; ++a) {
          if (tiled)      // block (part a, feature block, kb) of the tiled storage: 16 KiB contiguous
            tma2_load_2d(&tmW, bar, dst + a * S::kWBlock, 0,
                         ((a * ((N + kPairFeat - 1) / kPairFeat) + f0 / kPairFeat) * KB + kb) * kPairFeat);
          else
            tma2_load_2d(&tmW, bar, dst + a * S::kWBlock, kb * kGemmTileK, a * N + f0);
        }
      };
      auto load_x = [&](int it) {
        const int s = it % S::kStages;
        const uint32_t bar = map_to_cta(smem_u32(&full_bar[s]), 0);
        tma2_load_2d(&tmX, bar, smem + s * S::kStageBytes + S::kWBytes, (kb_beg + it) * kGemmTileK,
                     m0 + static_cast<int>(rank) * S::kXRows);
      };
      const int n_pre = kb_len < S::kStages ? kb_len : S::kStages;
      for (int it = 0; it < n_pre; ++it) load_w(it);
      griddep_wait();
      bool x_ready = true;
      if (np.x) {
        // The activation matrix is being written by this very launch: wait (bounded) until every CTA
        // has normalised its rows.  Both counters are zero when a launch starts: CTAs arrive only after
        // the preceding kernels have completed, and the last CTA that has stopped looking at the
        // arrival count (bar[1] counts those) clears both for the next launch.
        x_ready = false;
        const int n_cta = static_cast<int>(gridDim.x);
        const uint64_t t0 = global_timer_ns();
        for (uint32_t spin = 0; spin < kSpinLimit; ++spin) {
          if (ld_acquire_gpu(&np.bar[0]) >= n_cta) {
            x_ready = true;
            break;
          }
          if ((spin & 63u) == 63u && (*abort_flag || global_timer_ns() - t0 > kWaitLimitNs)) break;
        }
        if (!x_ready) *abort_flag = 1;
        if (atomicAdd(&np.bar[1], 1) == n_cta - 1) {
          atomicExch(&np.bar[0], 0);
          atomicExch(&np.bar[1], 0);
        }
        fence_proxy_async_all();
      }
      if (x_ready)
        for (int it = 0; it < n_pre; ++it) load_x(it);
      int it = n_pre;
      bool ok = x_ready;
      for (; ok && it < kb_len; ++it) {
        ok = mbar_wait(&empty_bar[it % S::kStages], ((it / S::kStages) & 1) ^ 1u, abort_flag);
        if (!ok) break;
        load_w(it);
        load_x(it);
      }
      if (!ok && rank == 0) {
        for (int k = it > S::kStages ? it - S::kStages : 0; k < it; ++k)
          mbar_drain(&full_bar[k % S::kStages], (k / S::kStages) & 1);
      }
    }
  } else if (warp == 1) {
    if (lane == 0 && rank == 0) {
      const uint32_t idesc = idesc_operands(instr_desc_pair(BNB), half_in != 0);
      bool ok = true;
      for (int it = 0; it < kb_len; ++it) {
        const int s = it % S::kStages;
        ok = mbar_wait(&full_bar[s], (it / S::kStages) & 1, abort_flag);
        if (!ok) break;
        tc_fence_after();
        const uint32_t stage_addr = smem_u32(smem + s * S::kStageBytes);
        const uint64_t xdesc = smem_desc_sw128(stage_addr + S::kWBytes);
#pragma unroll
        for (int a = 0; a < ACC; ++a) {
          const uint64_t wdesc = smem_desc_sw128(stage_addr + a * S::kWBlock);
#pragma unroll
          for (int k = 0; k < kGemmTileK / 16; ++k)
            tc2_mma_bf16(tmem_base + a * BNB, wdesc + 2 * k, xdesc + 2 * k, idesc, (it > 0 || k > 0) ? 1u : 0u);
        }
        tc2_commit_both(&empty_bar[s]);
      }
      if (ok) tc2_commit_both(acc_full);
    }
  } else {
    // ---- epilogue: this CTA's 128 features x BNB rows --------------------------------------------
    const int ew = warp - 2;
    const int quarter = warp & 3;                       // the TMEM lane quarter this warp may read
    const int grp = ew >> 2;                            // which quarter of the columns it takes
    const int row = quarter * 32 + lane;                // feature within the CTA
    const int cols = min(BNB, M - m0);
    constexpr int CH = BNB / 4;                         // columns per warp
    const uint32_t lane_addr = tmem_base + (static_cast<uint32_t>(quarter * 32) << 16);
    if (np.x) {
      griddep_wait();                                  // x is the preceding kernel's output
      norm_rows_and_arrive(np, M, K, half_in != 0, norm_scratch);
    }
    const bool got = mbar_wait(acc_full, 0, abort_flag);
    tc_fence_after();
    if (got) {
      if (ACC == 1) {
        float *part = reinterpret_cast<float *>(smem);  // [column][feature], reuses the pipeline stages
#pragma unroll
        for (int j = 0; j < CH / 32; ++j) {
          const int c0 = grp * CH + j * 32;
          if (c0 < cols) {
            uint32_t r[32];
            tc_ld32(lane_addr + c0, r);
            tc_wait_ld();
#pragma unroll
            for (int c = 0; c < 32; ++c) part[(c0 + c) * kPairFeat + row] = __uint_as_float(r[c]);
          }
        }
      } else {
        uint16_t *stage = reinterpret_cast<uint16_t *>(smem);             // [feature half][column][64]
        const int h = row >> 6, fl = row & 63;
#pragma unroll
        for (int j = 0; j < CH / 32; ++j) {
          const int c0 = grp * CH + j * 32;
          if (c0 < cols) {
            uint32_t g[32], u[32];
            tc_ld32(lane_addr + c0, g);
            tc_ld32(lane_addr + BNB + c0, u);
            tc_wait_ld();
#pragma unroll
            for (int c = 0; c < 32; ++c)
              stage[(h * BNB + c0 + c) * 64 + fl] =
                  cvt16(silu_pair(__uint_as_float(g[c])) * __uint_as_float(u[c]), half_in != 0);
          }
        }
      }
    }
    tc_fence_before();
    fence_proxy_async();
    pair_epi_bar();
    if (lane == 0 && got) {
      if (ACC == 1) {
        // boxes of 128 features x 32 rows (16 KiB)
        if (ew < BNB / 32 && ew * 32 < cols) {
          const uint8_t *src = smem + static_cast<size_t>(ew) * 32 * kPairFeat * 4;
          if (epilogue == EPI_ACCUM || split > 1) tma_reduce_add_2d(&tmY, src, f0, m0 + ew * 32);
          else tma_store_2d(&tmY, src, f0, m0 + ew * 32);
          bulk_commit();
          bulk_wait_read();
        }
      } else {
        // boxes of 64 features x 32 rows (4 KiB)
        const int h = ew & 1, c0 = (ew >> 1) * 32;
        if (c0 < BNB && c0 < cols) {
          tma_store_2d(&tmY, smem + static_cast<size_t>(h * BNB + c0) * 64 * 2, f0 + h * 64, m0 + c0);
          bulk_commit();
          bulk_wait_read();
        }
      }
    }
  }

  // Neither CTA may leave (or release tensor memory) while its partner can still read its shared
  // memory, signal its barriers or write its accumulators.
  tc_fence_before();
  __syncthreads();
  pair_cluster_sync();
  if (warp == 1) {
    tc_fence_after();
    tc2_dealloc(tmem_base, S::kTmemCols);
  }
  if (threadIdx.x == 0 && *abort_flag && status) atomicExch(status, STATUS_WAIT_TIMEOUT);
}

int g_pair_sms = 0;
int g_pair_clusters = 0;        // SM pairs of the widest instantiation that can be resident at once

template <int BNB, int ACC>
cudaError_t launch_pair(const PairGemmArgs &a, int n_tiles, int m_tiles, int split, cudaStream_t stream) {
  using S = PairSmem<BNB, ACC>;
  CUtensorMap tmX, tmY;
  if (make_tensor_map(&tmX, a.X, a.M, a.K, a.K, S::kXRows) != 0) return cudaErrorInvalidValue;
  const bool bf16_out = ACC == 2;
  if (make_out_map_box(&tmY, a.Y, a.M, a.N, a.ldY, bf16_out, bf16_out ? 64 : kPairFeat, 32) != 0)
    return cudaErrorInvalidValue;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(2 * n_tiles * split * m_tiles, 1, 1);
  cfg.blockDim = dim3(kPairThreads, 1, 1);
  cfg.dynamicSmemBytes = S::kTotal;
  cfg.stream = stream;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = 2;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = a.allow_early_start ? 2 : 1;
  NormPrologue np = a.norm;
  if (np.x && (m_tiles != 1 || 2 * n_tiles * split > 2 * g_pair_clusters || (a.K & 3))) return cudaErrorInvalidValue;
  return cudaLaunchKernelEx(&cfg, gemm_pair_kernel<BNB, ACC>, *a.tmW, tmX, tmY, a.M, a.N, a.K, a.epilogue, split,
                            a.tiled, a.half_in, a.status, np);
}

template <int BNB, int ACC>
cudaError_t configure_pair() {
  return cudaFuncSetAttribute(gemm_pair_kernel<BNB, ACC>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                              PairSmem<BNB, ACC>::kTotal);
}

}  // namespace

template <int BNB, int ACC>
int max_resident_clusters(int sms) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(sms & ~1, 1, 1);
  cfg.blockDim = dim3(kPairThreads, 1, 1);
  cfg.dynamicSmemBytes = PairSmem<BNB, ACC>::kTotal;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = 2;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  int n = 0;
  if (cudaOccupancyMaxActiveClusters(&n, gemm_pair_kernel<BNB, ACC>, &cfg) != cudaSuccess) {
    cudaGetLastError();
    return 0;
  }
  return n;
}

cudaError_t gemm_pair_configure() {
  cudaError_t e;
  int dev = 0;
  if ((e = cudaGetDevice(&dev)) != cudaSuccess) return e;
  if ((e = cudaDeviceGetAttribute(&g_pair_sms, cudaDevAttrMultiProcessorCount, dev)) != cudaSuccess) return e;
  if ((e = configure_pair<256, 1>()) != cudaSuccess) return e;
  if ((e = configure_pair<256, 2>()) != cudaSuccess) return e;
  if ((e = configure_pair<128, 1>()) != cudaSuccess) return e;
  if ((e = configure_pair<128, 2>()) != cudaSuccess) return e;
  // SM pairs that are resident at once (a GPC with an odd number of SMs leaves one without a partner):
  // the smallest over the instantiations bounds every launch that uses the grid-wide barrier
  g_pair_clusters = max_resident_clusters<256, 1>(g_pair_sms);
  g_pair_clusters = std::min(g_pair_clusters, max_resident_clusters<256, 2>(g_pair_sms));
  g_pair_clusters = std::min(g_pair_clusters, max_resident_clusters<128, 1>(g_pair_sms));
  g_pair_clusters = std::min(g_pair_clusters, max_resident_clusters<128, 2>(g_pair_sms));
  return cudaSuccess;
}

bool gemm_pair_can_fuse_norm(int M, int N, int K, int epilogue) {
  if (M <= 64 || M > 256 || (K & 3) || g_pair_clusters <= 0) return false;
  const int n_tiles = (N + 2 * kPairFeat - 1) / (2 * kPairFeat);
  return n_tiles * gemm_pair_split(M, N, K, epilogue, 0) <= g_pair_clusters;
}

bool gemm_pair_supported(const void *Y, int ldY, int M, int N, int K, int epilogue) {
  if (M <= 64 || N < 1 || K < 8 || (K % 8)) return false;
  const int es = epilogue == EPI_SWIGLU ? 2 : 4;
  return (reinterpret_cast<uintptr_t>(Y) & 15) == 0 && (static_cast<long>(ldY) * es) % 16 == 0;
}

// How many k-slices a linear-epilogue tile is cut into: as many as give every SM pair one
// (tile, slice), at least four k-blocks each.
int gemm_pair_split(int M, int N, int K, int epilogue, int force_split) {
  if (epilogue == EPI_SWIGLU) return 1;
  const int bnb = M > 128 ? 256 : 128;
  const int tiles = ((N + 2 * kPairFeat - 1) / (2 * kPairFeat)) * ((M + bnb - 1) / bnb);
  const int KB = (K + kGemmTileK - 1) / kGemmTileK;
  const int pairs = (g_pair_sms > 0 ? g_pair_sms : 148) / 2;
  int split = force_split > 0 ? force_split : pairs / tiles;
  if (split > KB / 4) split = KB / 4;
  if (split > 16) split = 16;
  if (split < 1) split = 1;
  return split;
}

cudaError_t gemm_pair_launch(const PairGemmArgs &a, cudaStream_t stream) {
  const bool gu = a.epilogue == EPI_SWIGLU;
  const int bnb = a.M > 128 ? 256 : 128;
  const int n_tiles = (a.N + 2 * kPairFeat - 1) / (2 * kPairFeat);
  const int m_tiles = (a.M + bnb - 1) / bnb;
  const int split = gemm_pair_split(a.M, a.N, a.K, a.epilogue, a.force_split);
  if (bnb == 256) return gu ? launch_pair<256, 2>(a, n_tiles, m_tiles, 1, stream)
                            : launch_pair<256, 1>(a, n_tiles, m_tiles, split, stream);
  return gu ? launch_pair<128, 2>(a, n_tiles, m_tiles, 1, stream)
            : launch_pair<128, 1>(a, n_tiles, m_tiles, split, stream);
}

}  // namespace echo

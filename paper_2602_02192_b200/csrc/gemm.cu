// Dense projections Y = X * W^T for the decoder (bf16 in, fp32 accumulate) on the
// sm_100a tensor cores: tcgen05.mma with the accumulator in tensor memory, operands
// staged in shared memory by TMA (128-byte swizzle), one elected thread issuing MMAs.
//
// Operand roles are swapped with respect to the usual GEMM picture: the WEIGHT tile
// (128 output features x 64 k) is the UMMA "A" operand and fills the 128 TMEM lanes,
// the ACTIVATION tile (bnb rows x 64 k) is the "B" operand and fills bnb TMEM columns.
// Each weight byte is therefore streamed from HBM exactly once for up to 256 activation
// rows, which is what a decode step (a few hundred rows against gigabytes of weights)
// needs; the activation tile is re-read from L2.
//
// Two kernels share the main loop.  A decode step's projections are 5-30 us of weight
// streaming each, with 16-96 output tiles for 148 SMs, so both split tiles along K:
//   gemm_cluster_kernel   one CTA per (tile, k-slice).  By default the slices of a tile add their
//                         partial tiles into the output in memory (TMA reduce-add; the order of
//                         the fp32 additions is not fixed); alternatively the slices form a
//                         thread-block cluster and are summed in rank order through distributed
//                         shared memory (bit-reproducible, slower).  Launched with programmatic
//                         stream serialization: weight tiles are prefetched before the kernel
//                         waits for its predecessor, activations after.
//   gemm_streamk_kernel   persistent, one CTA per SM, for many-tile problems (the lm_head): the
//                         list of (tile, k-block) pairs is cut into equal contiguous ranges; a CTA
//                         that covers only part of a tile writes its partial to a workspace slot,
//                         and the CTA that finishes a tile last (an atomic counter per tile, no
//                         waiting) sums the partials in k order and applies the epilogue.
//
// A CTA's output tile is two 128-lane accumulators (256 features) against one activation
// tile, so that the activation bytes an SM pulls from L2 do not exceed the weight bytes it
// pulls from HBM (an SM ingests roughly 64 bytes per clock in total).
//
// Warp roles: warp 0 = TMA producer, warp 1 = TMEM owner + MMA issuer, warps 2..17 =
// epilogue (each reads the TMEM lane quarter its warp id selects; the four warps of a quarter
// split the columns - a warp keeps only one global store in flight at a time, so the store
// rate of the epilogue grows with the number of warps).
// Every mbarrier wait is bounded; on expiry the kernel records STATUS_WAIT_TIMEOUT,
// drains, frees its tensor memory and returns.

#include "common.cuh"
#include "ptx.cuh"

namespace echo {

using namespace ptx;

namespace {

constexpr int kEpiGroups = 4;         // epilogue warps per TMEM lane quarter (they split the columns)
constexpr int kEpiWarps = 4 * kEpiGroups;
constexpr int kEpiThreads = 128 * kEpiGroups;
constexpr int kThreads = 64 + kEpiThreads;
constexpr int kAcc = 2;              // accumulators (128-lane weight blocks) per output tile

template <int BNB>
struct GemmSmem {
  static constexpr int kWBlock = kGemmTileN * kGemmTileK * 2;      // 16 KiB per weight block
  static constexpr int kWBytes = kAcc * kWBlock;
  static constexpr int kXBytes = BNB * kGemmTileK * 2;
  static constexpr int kStageBytes = kWBytes + kXBytes;
  static constexpr int kBudget = 200 * 1024;
  static constexpr int kStagesRaw = kBudget / kStageBytes;
  static constexpr int kStages = kStagesRaw > 8 ? 8 : kStagesRaw;
  static constexpr int kBarBytes = 1024;
  static constexpr int kTotal = kStages * kStageBytes + kBarBytes + 1024;   // + alignment slack
  static constexpr int kTmemCols = kAcc * BNB < 32 ? 32 : kAcc * BNB;
};

__device__ __forceinline__ float silu_f(float a) { return a / (1.0f + __expf(-a)); }
// store, or add in memory without reading back (one add per element per launch: order-free)
__device__ __forceinline__ void put(float *y, float v, int epilogue) {
  if (epilogue == EPI_ACCUM) atomicAdd(y, v);
  else *y = v;
}

// Stream-K split of `total` k-blocks over `n_cta` CTAs: CTA c owns [beg(c), beg(c+1)).
struct Split {
  int total, n_cta, q, r;
  __host__ __device__ int beg(int c) const { return c * q + (c < r ? c : r); }
  __host__ __device__ int cta_of(int g) const {
    const int edge = r * (q + 1);
    return g < edge ? g / (q + 1) : r + (g - edge) / q;
  }
};

__device__ __forceinline__ void epi_bar() { asm volatile("bar.sync 1, %0;" ::"n"(kEpiThreads) : "memory"); }

// Loads of one k-block: kAcc weight blocks (each 128 rows, or 64 gate + 64 up rows) and the
// activation tile.
// `tiled`: W is block-tiled storage (128-row x 64-column blocks, each contiguous) with KB column
// blocks per row block; the up rows of a gate/up pair then start at row block ceil(N / 128).
template <int BNB>
__device__ __forceinline__ void load_stage_w(const CUtensorMap *tmW, uint64_t *bar, uint8_t *stage, int kb, int nt,
                                             int N, bool gu, int tiled, int KB) {
  using S = GemmSmem<BNB>;
  mbar_expect_tx(bar, S::kStageBytes);                 // covers the activation tile loaded afterwards as well
  auto row_of = [&](int f, int part) -> int {          // TMA row coordinate of feature f of part 0 / 1
    if (!tiled) return part * N + f;
    const int nbp = (N + kGemmTileN - 1) / kGemmTileN;
    return ((part * nbp + (f >> 7)) * KB + kb) * kGemmTileN + (f & 127);
  };
  const int c0 = tiled ? 0 : kb * kGemmTileK;
#pragma unroll
  for (int a = 0; a < kAcc; ++a) {
    uint8_t *dst = stage + a * S::kWBlock;
    if (gu) {
      const int f0 = (nt * kAcc + a) * 64;
      tma_load_2d(tmW, bar, dst, c0, row_of(f0, 0));
      tma_load_2d(tmW, bar, dst + S::kWBlock / 2, c0, row_of(f0, 1));
    } else {
      tma_load_2d(tmW, bar, dst, c0, row_of((nt * kAcc + a) * kGemmTileN, 0));
    }
  }
}
template <int BNB>
__device__ __forceinline__ void load_stage_x(const CUtensorMap *tmX, uint64_t *bar, uint8_t *stage, int kb, int m0) {
  tma_load_2d(tmX, bar, stage + GemmSmem<BNB>::kWBytes, kb * kGemmTileK, m0);
}
template <int BNB>
__device__ __forceinline__ void load_stage(const CUtensorMap *tmW, const CUtensorMap *tmX, uint64_t *bar,
                                           uint8_t *stage, int kb, int nt, int m0, int N, bool gu, int tiled, int KB) {
  load_stage_w<BNB>(tmW, bar, stage, kb, nt, N, gu, tiled, KB);
  load_stage_x<BNB>(tmX, bar, stage, kb, m0);
}

template <int BNB>
__device__ __forceinline__ void mma_stage(uint32_t tmem_base, uint32_t stage_addr, bool first, bool half_in) {
  using S = GemmSmem<BNB>;
  const uint32_t idesc = idesc_operands(instr_desc_bf16(BNB), half_in);
  const uint64_t xdesc = smem_desc_sw128(stage_addr + S::kWBytes);
#pragma unroll
  for (int a = 0; a < kAcc; ++a) {
    const uint64_t wdesc = smem_desc_sw128(stage_addr + a * S::kWBlock);
#pragma unroll
    for (int k = 0; k < kGemmTileK / 16; ++k) {
      // 16 bf16 = 32 bytes further along K inside the swizzled row: +2 in 16-byte units
      tc_mma_bf16(tmem_base + a * BNB, wdesc + 2 * k, xdesc + 2 * k, idesc, (!first || k > 0) ? 1u : 0u);
    }
  }
}

// ---------------------------------------------------------------------------------------
// Persistent stream-K kernel (many output tiles: the lm_head).
// ---------------------------------------------------------------------------------------
template <int BNB>
__global__ void __launch_bounds__(kThreads, 1)
gemm_streamk_kernel(const __grid_constant__ CUtensorMap tmW, const __grid_constant__ CUtensorMap tmX, void *Yv,
                    int ldY, int M, int N, int K, int epilogue, int n_tiles, float *workspace, int *counters,
                    int tiled, int half_in, int *status) {
  using S = GemmSmem<BNB>;
  extern __shared__ uint8_t smem_raw[];
  uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint64_t *full_bar = reinterpret_cast<uint64_t *>(smem + S::kStages * S::kStageBytes);
  uint64_t *empty_bar = full_bar + S::kStages;
  uint64_t *acc_full = empty_bar + S::kStages;
  uint64_t *acc_empty = acc_full + 1;
  uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(acc_empty + 1);
  volatile int *abort_flag = reinterpret_cast<volatile int *>(tmem_slot + 1);
  volatile int *last_flag = abort_flag + 1;

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const bool gu = epilogue == EPI_SWIGLU;
  const int KB = (K + kGemmTileK - 1) / kGemmTileK;
  const int m_tiles = (M + BNB - 1) / BNB;
  Split sp;
  sp.total = n_tiles * m_tiles * KB;
  sp.n_cta = gridDim.x;
  sp.q = sp.total / sp.n_cta;
  sp.r = sp.total % sp.n_cta;
  const int cta = blockIdx.x;
  const int g_beg = sp.beg(cta), g_end = sp.beg(cta + 1);

  if (threadIdx.x == 0) {
    for (int s = 0; s < S::kStages; ++s) {
      mbar_init(&full_bar[s], 1);
      mbar_init(&empty_bar[s], 1);
    }
    mbar_init(acc_full, 1);
    mbar_init(acc_empty, kEpiThreads);
    *abort_flag = 0;
    *last_flag = 0;
    mbar_fence_init();
  }
  if (warp == 1) tc_alloc(tmem_slot, S::kTmemCols);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  griddep_launch();
  griddep_wait();          // inputs produced by the preceding kernel are complete from here on

  if (warp == 0) {
    // ---------------- TMA producer ----------------
    if (lane == 0) {
      int it = 0;
      bool ok = true;
      for (int g = g_beg; g < g_end && ok;) {
        const int unit = g / KB, kb0 = g % KB;
        const int len = min(KB - kb0, g_end - g);
        const int nt = unit % n_tiles, mt = unit / n_tiles;
        for (int kb = kb0; kb < kb0 + len; ++kb, ++it) {
          const int s = it % S::kStages;
          ok = mbar_wait(&empty_bar[s], ((it / S::kStages) & 1) ^ 1u, abort_flag);
          if (!ok) break;
          load_stage<BNB>(&tmW, &tmX, &full_bar[s], smem + s * S::kStageBytes, kb, nt, mt * BNB, N, gu, tiled, KB);
        }
        g += len;
      }
      if (!ok) {
        // let copies already in flight land before the CTA's shared memory is released
        for (int k = it > S::kStages ? it - S::kStages : 0; k < it; ++k)
          mbar_drain(&full_bar[k % S::kStages], (k / S::kStages) & 1);
      }
    }
  } else if (warp == 1) {
    // ---------------- MMA issuer ----------------
    if (lane == 0) {
      int it = 0, seg = 0;
      bool ok = true;
      for (int g = g_beg; g < g_end && ok; ++seg) {
        const int kb0 = g % KB;
        const int len = min(KB - kb0, g_end - g);
        ok = mbar_wait(acc_empty, (seg & 1) ^ 1u, abort_flag);     // epilogue has drained the accumulators
        if (!ok) break;
        tc_fence_after();
        for (int kb = 0; kb < len; ++kb, ++it) {
          const int s = it % S::kStages;
          ok = mbar_wait(&full_bar[s], (it / S::kStages) & 1, abort_flag);
          if (!ok) break;
          tc_fence_after();
          mma_stage<BNB>(tmem_base, smem_u32(smem + s * S::kStageBytes), kb == 0, half_in != 0);
          tc_commit(&empty_bar[s]);      // frees the stage once these MMAs have read it
        }
        if (ok) tc_commit(acc_full);
        g += len;
      }
    }
  } else {
    // ---------------- epilogue: TMEM -> registers -> global / workspace ----------------
    const int quarter = warp & 3;                       // TMEM lanes 32*quarter .. +31
    const int row = quarter * 32 + lane;                // accumulator lane
    const int et = (threadIdx.x - 64) & 127;            // position within the 128-lane tile
    const int grp = (warp - 2) >> 2;                    // which share of the columns this warp takes
    const int first_unit = g_beg / KB;
    const size_t acc_elems = static_cast<size_t>(kGemmTileN) * BNB;
    const size_t slot_elems = kAcc * acc_elems;
    int seg = 0;
    bool ok = true;
    for (int g = g_beg; g < g_end && ok; ++seg) {
      const int unit = g / KB, kb0 = g % KB;
      const int len = min(KB - kb0, g_end - g);
      g += len;
      const int nt = unit % n_tiles, mt = unit / n_tiles;
      const int m0 = mt * BNB;
      const int cols = min(BNB, M - m0);
      ok = mbar_wait(acc_full, seg & 1, abort_flag);
      if (!ok) break;
      tc_fence_after();
      const uint32_t lane_addr = tmem_base + (static_cast<uint32_t>(quarter * 32) << 16);
      const bool whole = kb0 == 0 && len == KB;
      if (whole && !gu) {
        float *Y = reinterpret_cast<float *>(Yv);
#pragma unroll 1
        for (int a = 0; a < kAcc; ++a) {
          const int n = (nt * kAcc + a) * kGemmTileN + row;
#pragma unroll 1
          for (int c0 = 32 * grp; c0 < cols; c0 += 32 * kEpiGroups) {
            uint32_t r[32];
            tc_ld32(lane_addr + a * BNB + c0, r);
            tc_wait_ld();
            if (n < N) {
              float *y0 = Y + static_cast<size_t>(m0 + c0) * ldY + n;
#pragma unroll
              for (int c = 0; c < 32; ++c)
                if (c0 + c < cols) put(y0 + static_cast<size_t>(c) * ldY, __uint_as_float(r[c]), epilogue);
            }
          }
        }
        tc_fence_before();
        mbar_arrive(acc_empty);
        continue;
      }
      // partial (or gate/up) accumulators -> this CTA's workspace slot, layout [acc][column][lane]
      const int slot = whole ? 2 : (unit == first_unit ? 0 : 1);
      float *ws = workspace + (static_cast<size_t>(cta) * 3 + slot) * slot_elems;
#pragma unroll 1
      for (int a = 0; a < kAcc; ++a) {
#pragma unroll 1
        for (int c0 = 32 * grp; c0 < cols; c0 += 32 * kEpiGroups) {
          uint32_t r[32];
          tc_ld32(lane_addr + a * BNB + c0, r);
          tc_wait_ld();
#pragma unroll
          for (int c = 0; c < 32; ++c)
            __stcg(ws + a * acc_elems + static_cast<size_t>(c0 + c) * kGemmTileN + row, __uint_as_float(r[c]));
        }
      }
      tc_fence_before();
      mbar_arrive(acc_empty);
      // count this segment; the CTA that completes the tile reduces it
      const int c_first = sp.cta_of(unit * KB), c_last = sp.cta_of(unit * KB + KB - 1);
      __threadfence();
      epi_bar();
      if (threadIdx.x == 64) {
        const int old = atomicAdd(&counters[unit], 1);
        *last_flag = (old == c_last - c_first) ? 1 : 0;
      }
      epi_bar();
      const bool last = *last_flag != 0;
      if (last) {
        __threadfence();
#pragma unroll 1
        for (int a = 0; a < kAcc; ++a) {
          if (gu) {
            // thread -> feature f of the 64-wide block and every second column of a 32-column chunk
            uint16_t *Y = reinterpret_cast<uint16_t *>(Yv);
            const int f = et & 63, half = et >> 6;
            const int n = (nt * kAcc + a) * 64 + f;
#pragma unroll 1
            for (int c0 = 32 * grp; c0 < cols; c0 += 32 * kEpiGroups) {
              float gs[16], us[16];
#pragma unroll
              for (int i = 0; i < 16; ++i) gs[i] = us[i] = 0.f;
              for (int cc = c_first; cc <= c_last; ++cc) {
                const int sl = c_first == c_last ? 2 : (sp.beg(cc) / KB == unit ? 0 : 1);
                const float *p = workspace + (static_cast<size_t>(cc) * 3 + sl) * slot_elems + a * acc_elems +
                                 static_cast<size_t>(c0 + half) * kGemmTileN + f;
#pragma unroll
                for (int i = 0; i < 16; ++i) {
                  gs[i] += __ldcg(p + static_cast<size_t>(2 * i) * kGemmTileN);
                  us[i] += __ldcg(p + static_cast<size_t>(2 * i) * kGemmTileN + 64);
                }
              }
              if (n < N) {
#pragma unroll
                for (int i = 0; i < 16; ++i) {
                  const int c = c0 + half + 2 * i;
                  if (c < cols) Y[static_cast<size_t>(m0 + c) * ldY + n] = cvt16(silu_f(gs[i]) * us[i], half_in != 0);
                }
              }
            }
          } else {
            float *Y = reinterpret_cast<float *>(Yv);
            const int n = (nt * kAcc + a) * kGemmTileN + et;
#pragma unroll 1
            for (int c0 = 32 * grp; c0 < cols; c0 += 32 * kEpiGroups) {
              float acc[32];
#pragma unroll
              for (int i = 0; i < 32; ++i) acc[i] = 0.f;
              for (int cc = c_first; cc <= c_last; ++cc) {
                const int sl = sp.beg(cc) / KB == unit ? 0 : 1;
                const float *p = workspace + (static_cast<size_t>(cc) * 3 + sl) * slot_elems + a * acc_elems +
                                 static_cast<size_t>(c0) * kGemmTileN + et;
#pragma unroll
                for (int i = 0; i < 32; ++i) acc[i] += __ldcg(p + static_cast<size_t>(i) * kGemmTileN);
              }
              if (n < N) {
                float *y0 = Y + static_cast<size_t>(m0 + c0) * ldY + n;
#pragma unroll
                for (int i = 0; i < 32; ++i)
                  if (c0 + i < cols) put(y0 + static_cast<size_t>(i) * ldY, acc[i], epilogue);
              }
            }
          }
        }
        if (threadIdx.x == 64) counters[unit] = 0;   // ready for the next launch
      }
      epi_bar();                                      // last_flag is reused by the next segment
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tc_dealloc(tmem_base, S::kTmemCols);
  }
  if (threadIdx.x == 0 && *abort_flag && status) atomicExch(status, STATUS_WAIT_TIMEOUT);
}

// ---------------------------------------------------------------------------------------
// Split-K over a thread-block cluster (few output tiles: the per-layer projections).  The S
// CTAs of a cluster share one output tile and each streams 1/S of its k-blocks; the partial
// accumulators are then summed through distributed shared memory in rank order (so the
// result does not depend on timing), each CTA reducing and writing a 1/S slice of the tile's
// columns.  No global scratch, no atomics between CTAs, no waiting other than the hardware
// cluster barrier.
// ---------------------------------------------------------------------------------------
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
  asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ uint32_t dsmem_addr(uint32_t cta_addr, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(cta_addr), "r"(rank));
  return r;
}
__device__ __forceinline__ float4 ld_dsmem_v4(uint32_t addr) {
  float4 v;
  asm volatile("ld.shared::cluster.v4.f32 {%0, %1, %2, %3}, [%4];"
               : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w)
               : "r"(addr));
  return v;
}
__device__ __forceinline__ float2 ld_dsmem_v2(uint32_t addr) {
  float2 v;
  asm volatile("ld.shared::cluster.v2.f32 {%0, %1}, [%2];" : "=f"(v.x), "=f"(v.y) : "r"(addr));
  return v;
}

template <int BNB>
__global__ void __launch_bounds__(kThreads, 1)
gemm_cluster_kernel(const __grid_constant__ CUtensorMap tmW, const __grid_constant__ CUtensorMap tmX,
                    const __grid_constant__ CUtensorMap tmY, int M, int N, int K, int epilogue, int S_split,
                    int independent, int tiled, int half_in, int *status) {
  using S = GemmSmem<BNB>;
  extern __shared__ uint8_t smem_raw[];
  uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint64_t *full_bar = reinterpret_cast<uint64_t *>(smem + S::kStages * S::kStageBytes);
  uint64_t *empty_bar = full_bar + S::kStages;
  uint64_t *acc_full = empty_bar + S::kStages;
  uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(acc_full + 1);
  volatile int *abort_flag = reinterpret_cast<volatile int *>(tmem_slot + 1);
  float *part = reinterpret_cast<float *>(smem);      // [column][lane], reuses the pipeline stages

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const bool gu = epilogue == EPI_SWIGLU;
  const int KB = (K + kGemmTileK - 1) / kGemmTileK;
  const int nt = blockIdx.x / S_split;
  const int rank = blockIdx.x % S_split;              // == rank in the cluster (cluster spans x only)
  const int m0 = blockIdx.y * BNB;
  const int kq = KB / S_split, kr = KB % S_split;
  const int kb_beg = rank * kq + min(rank, kr);
  const int kb_len = kq + (rank < kr ? 1 : 0);

  if (threadIdx.x == 0) {
    for (int s = 0; s < S::kStages; ++s) {
      mbar_init(&full_bar[s], 1);
      mbar_init(&empty_bar[s], 1);
    }
    mbar_init(acc_full, 1);
    *abort_flag = 0;
    mbar_fence_init();
  }
  if (warp == 1) tc_alloc(tmem_slot, S::kTmemCols);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  griddep_launch();        // the next kernel may start its own prologue and weight prefetch

  if (warp == 0) {
    if (lane == 0) {
      // Weights do not depend on the preceding kernel: fill the pipeline with weight tiles first,
      // then wait for that kernel to finish before touching the activations it wrote.
      const int n_pre = kb_len < S::kStages ? kb_len : S::kStages;
      for (int it = 0; it < n_pre; ++it)
        load_stage_w<BNB>(&tmW, &full_bar[it], smem + it * S::kStageBytes, kb_beg + it, nt, N, gu, tiled, KB);
      griddep_wait();
      for (int it = 0; it < n_pre; ++it)
        load_stage_x<BNB>(&tmX, &full_bar[it], smem + it * S::kStageBytes, kb_beg + it, m0);
      int it = n_pre;
      bool ok = true;
      for (int kb = kb_beg + n_pre; kb < kb_beg + kb_len; ++kb, ++it) {
        const int s = it % S::kStages;
        ok = mbar_wait(&empty_bar[s], ((it / S::kStages) & 1) ^ 1u, abort_flag);
        if (!ok) break;
        load_stage<BNB>(&tmW, &tmX, &full_bar[s], smem + s * S::kStageBytes, kb, nt, m0, N, gu, tiled, KB);
      }
      if (!ok) {
        for (int k = it > S::kStages ? it - S::kStages : 0; k < it; ++k)
          mbar_drain(&full_bar[k % S::kStages], (k / S::kStages) & 1);
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      bool ok = true;
      for (int it = 0; it < kb_len; ++it) {
        const int s = it % S::kStages;
        ok = mbar_wait(&full_bar[s], (it / S::kStages) & 1, abort_flag);
        if (!ok) break;
        tc_fence_after();
        mma_stage<BNB>(tmem_base, smem_u32(smem + s * S::kStageBytes), it == 0, half_in != 0);
        tc_commit(&empty_bar[s]);
      }
      if (ok) tc_commit(acc_full);
    }
  }

  // ---- epilogue.  Per accumulator: TMEM -> shared memory ([column][lane] fp32, reusing the
  // pipeline stages, which no MMA reads any more once acc_full has fired); with a split, the
  // cluster's partials are summed through distributed shared memory in rank order, each CTA
  // taking a slice of columns; the finished tile leaves through TMA stores (or TMA reduce-adds
  // for the residual epilogue), which keep the few epilogue warps off the global store path.
  // `independent`: the S_split CTAs of a tile are not a cluster; each adds its partial tile to the
  // output in memory (TMA reduce-add), so the summation order across them is not fixed
  const bool plain = (S_split == 1 || independent) && !gu;
  const bool add_out = epilogue == EPI_ACCUM || (independent && S_split > 1);
  const int cols = min(BNB, M - m0);
  const int quarter = warp & 3;
  const int row = quarter * 32 + lane;
  const int grp = (warp - 2) >> 2;
  const uint32_t lane_addr = tmem_base + (static_cast<uint32_t>(quarter * 32) << 16);
  uint8_t *out_stage = smem + static_cast<size_t>(kGemmTileN) * BNB * 4;     // behind the partial
  const int units = (cols + 7) / 8;                                           // slices in 8-column units
  const int c_lo = 8 * (rank * units / S_split), c_hi = 8 * ((rank + 1) * units / S_split);
  const uint32_t part_addr = smem_u32(part);
  bool got = false;
  if (warp >= 2) {
    got = mbar_wait(acc_full, 0, abort_flag);
    tc_fence_after();
  }
#pragma unroll 1
  for (int a = 0; a < kAcc; ++a) {
    if (warp >= 2) {
      if (a > 0 && plain) {
        if (lane == 0) bulk_wait_read();                  // TMA has read the previous accumulator out of `part`
        epi_bar();
      }
      if (got) {
        // two 32-column blocks per warp, both TMEM loads in flight before the first store
        const int c0 = 32 * grp, c1 = c0 + 32 * kEpiGroups;
        uint32_t r0[32], r1[32];
        if (c0 < cols) tc_ld32(lane_addr + a * BNB + c0, r0);
        if (c1 < cols) tc_ld32(lane_addr + a * BNB + c1, r1);
        tc_wait_ld();
        if (c0 < cols) {
#pragma unroll
          for (int c = 0; c < 32; ++c) part[(c0 + c) * kGemmTileN + row] = __uint_as_float(r0[c]);
        }
        if (c1 < cols) {
#pragma unroll
          for (int c = 0; c < 32; ++c) part[(c1 + c) * kGemmTileN + row] = __uint_as_float(r1[c]);
        }
      }
    }
    __syncwarp();
    if (!plain) {
      // all partials of this accumulator are in place (a cluster of one only needs its own warps)
      if (S_split > 1) cluster_sync_all();
      else if (warp >= 2) epi_bar();
      if (warp >= 2 && a > 0) {
        if (lane == 0) bulk_wait_read();                  // TMA has read the previous result out of out_stage
        epi_bar();
      }
      if (warp >= 2 && got) {
        // one warp per column: a lane owns 4 consecutive features (2 gate + 2 up for SwiGLU), so a
        // warp reads a whole 512-byte row of every rank's partial with one vector load per rank;
        // four columns are in flight at a time to cover the remote shared-memory latency
        const int ew = warp - 2;
#pragma unroll 1
        for (int cb = c_lo + ew; cb < c_hi; cb += 4 * kEpiWarps) {
          if (gu) {
            float2 gs[4], us[4];
#pragma unroll
            for (int j = 0; j < 4; ++j) gs[j] = us[j] = make_float2(0.f, 0.f);
#pragma unroll
            for (int r = 0; r < 8; ++r) {
              if (r < S_split) {
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                  const int c = cb + j * kEpiWarps;
                  if (c < c_hi) {
                    const uint32_t base = dsmem_addr(part_addr + static_cast<uint32_t>(c * kGemmTileN + 2 * lane) * 4u, r);
                    const float2 g = ld_dsmem_v2(base), u = ld_dsmem_v2(base + 64u * 4u);
                    gs[j].x += g.x; gs[j].y += g.y; us[j].x += u.x; us[j].y += u.y;
                  }
                }
              }
            }
            uint32_t *o = reinterpret_cast<uint32_t *>(out_stage);               // [column - c_lo][64] 16-bit
#pragma unroll
            for (int j = 0; j < 4; ++j) {
              const int c = cb + j * kEpiWarps;
              if (c < c_hi)
                o[(c - c_lo) * 32 + lane] = cvt16x2(silu_f(gs[j].x) * us[j].x, silu_f(gs[j].y) * us[j].y, half_in != 0);
            }
          } else {
            float4 acc[4];
#pragma unroll
            for (int j = 0; j < 4; ++j) acc[j] = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
            for (int r = 0; r < 8; ++r) {
              if (r < S_split) {
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                  const int c = cb + j * kEpiWarps;
                  if (c < c_hi) {
                    const float4 v = ld_dsmem_v4(
                        dsmem_addr(part_addr + static_cast<uint32_t>(c * kGemmTileN + 4 * lane) * 4u, r));
                    acc[j].x += v.x; acc[j].y += v.y; acc[j].z += v.z; acc[j].w += v.w;
                  }
                }
              }
            }
            float4 *o = reinterpret_cast<float4 *>(out_stage);                      // [column - c_lo][128]
#pragma unroll
            for (int j = 0; j < 4; ++j) {
              const int c = cb + j * kEpiWarps;
              if (c < c_hi) o[(c - c_lo) * 32 + lane] = acc[j];
            }
          }
        }
      }
    }
    __syncwarp();
    // peers have finished reading this CTA's partial
    if (!plain) {
      if (S_split > 1) cluster_sync_all();
      else if (warp >= 2) epi_bar();
    }
    if (warp >= 2) {
      fence_proxy_async();
      epi_bar();
      if (lane == 0 && got) {
        // every epilogue warp issues a share of the 8-column boxes
        const int x = (nt * kAcc + a) * (gu ? 64 : kGemmTileN);
        const uint8_t *src = plain ? reinterpret_cast<const uint8_t *>(part) : out_stage;
        const int row_bytes = gu ? 64 * 2 : kGemmTileN * 4;
        const int lo = plain ? 0 : c_lo, hi = plain ? 8 * units : c_hi;
        for (int c = lo + 8 * (warp - 2); c < hi; c += 8 * kEpiWarps) {
          const uint8_t *p8 = src + static_cast<size_t>(c - lo) * row_bytes;
          if (add_out) tma_reduce_add_2d(&tmY, p8, x, m0 + c);
          else tma_store_2d(&tmY, p8, x, m0 + c);
        }
        bulk_commit();
      }
    }
  }
  if (warp >= 2 && lane == 0) bulk_wait_read();

  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tc_dealloc(tmem_base, S::kTmemCols);
  }
  if (threadIdx.x == 0 && *abort_flag && status) atomicExch(status, STATUS_WAIT_TIMEOUT);
}

int g_num_sms = 0;

// Split factor for the cluster kernel: the smallest of 1, 2, 4 that puts a CTA on at least
// ~40% of the SMs.  Measured on B200 at 256 activation rows: larger clusters lose more in the
// cluster barriers and the remote shared-memory reduction than they gain in parallelism.
int pick_split(int tiles, int KB, int sms) {
  int s = 1;
  while (s < 4 && tiles * s * 5 < sms * 2 && 2 * s <= KB) s *= 2;
  return s;
}

int make_out_map(CUtensorMap *out, void *base, uint64_t rows, uint64_t cols, uint64_t ld, bool bf16);

template <int BNB>
cudaError_t launch_cluster_variant(const GemmArgs &a, int n_tiles, int m_tiles, int split, bool independent,
                                   cudaStream_t stream) {
  using S = GemmSmem<BNB>;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(n_tiles * split, m_tiles, 1);
  cfg.blockDim = dim3(kThreads, 1, 1);
  cfg.dynamicSmemBytes = S::kTotal;
  cfg.stream = stream;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = independent ? 1 : split;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  // programmatic dependent launch: this kernel may begin (prologue, weight prefetch) while the
  // preceding kernel drains; it waits for that kernel's results before loading activations
  attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = a.allow_early_start ? 2 : 1;
  CUtensorMap tmY;
  const bool gu = a.epilogue == EPI_SWIGLU;
  if (make_out_map(&tmY, a.Y, a.M, a.N, a.ldY, gu) != 0) return cudaErrorInvalidValue;
  return cudaLaunchKernelEx(&cfg, gemm_cluster_kernel<BNB>, *a.tmW, *a.tmX, tmY, a.M, a.N, a.K, a.epilogue, split,
                            independent ? 1 : 0, a.tiled, a.half_in, a.status);
}

template <int BNB>
cudaError_t launch_variant(const GemmArgs &a, cudaStream_t stream) {
  using S = GemmSmem<BNB>;
  const bool gu = a.epilogue == EPI_SWIGLU;
  const int per_tile = kAcc * (gu ? 64 : kGemmTileN);
  const int n_tiles = (a.N + per_tile - 1) / per_tile;
  const int m_tiles = (a.M + BNB - 1) / BNB;
  const int KB = (a.K + kGemmTileK - 1) / kGemmTileK;
  const long total = static_cast<long>(n_tiles) * m_tiles * KB;
  if (n_tiles * m_tiles > kGemmMaxUnits || total > (1l << 30)) return cudaErrorInvalidValue;
  int grid = g_num_sms > 0 ? g_num_sms : 148;
  const bool out_ok = (reinterpret_cast<uintptr_t>(a.Y) & 15) == 0 && (a.ldY * (gu ? 2 : 4)) % 16 == 0;
  if (out_ok && a.force_split >= 0 && (a.force_split > 0 || n_tiles * m_tiles < 2 * grid)) {
    if (a.independent_splits && !gu) {
      // as many k-slices as it takes to put a CTA on every SM (at least 4 k-blocks each)
      int split = a.force_split > 0 ? a.force_split : grid / (n_tiles * m_tiles);
      if (split > KB / 4) split = KB / 4;
      if (split > 16) split = 16;
      if (split < 1) split = 1;
      return launch_cluster_variant<BNB>(a, n_tiles, m_tiles, split, split > 1, stream);
    }
    const int split = a.force_split > 0 ? (a.force_split < KB ? a.force_split : KB)
                                        : pick_split(n_tiles * m_tiles, KB, grid);
    return launch_cluster_variant<BNB>(a, n_tiles, m_tiles, split > 8 ? 8 : split, false, stream);
  }
  if (a.max_ctas > 0 && grid > a.max_ctas) grid = a.max_ctas;
  if (grid > total) grid = static_cast<int>(total);
  if (a.allow_early_start)
    return launch_early(gemm_streamk_kernel<BNB>, dim3(grid), dim3(kThreads), S::kTotal, stream, *a.tmW, *a.tmX, a.Y,
                        a.ldY, a.M, a.N, a.K, a.epilogue, n_tiles, a.workspace, a.counters, a.tiled, a.half_in,
                        a.status);
  gemm_streamk_kernel<BNB><<<grid, kThreads, S::kTotal, stream>>>(*a.tmW, *a.tmX, a.Y, a.ldY, a.M, a.N, a.K,
                                                                 a.epilogue, n_tiles, a.workspace, a.counters,
                                                                 a.tiled, a.half_in, a.status);
  return cudaGetLastError();
}

template <int BNB>
cudaError_t configure_variant() {
  cudaError_t e = cudaFuncSetAttribute(gemm_cluster_kernel<BNB>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       GemmSmem<BNB>::kTotal);
  if (e != cudaSuccess) return e;
  return cudaFuncSetAttribute(gemm_streamk_kernel<BNB>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                              GemmSmem<BNB>::kTotal);
}

// ---- plain SIMT reference kernel (debugging aid; never on the default path) ----
__global__ void gemm_simt_kernel(const __nv_bfloat16 *X, const __nv_bfloat16 *W, float *Y, int ldY, int M, int N,
                                 int K, int accumulate, int tiled, int part_rows, int half_in) {
  const uint16_t *X16 = reinterpret_cast<const uint16_t *>(X), *W16 = reinterpret_cast<const uint16_t *>(W);
  __shared__ float xs[16][17], ws[16][17];
  const int tx = threadIdx.x, ty = threadIdx.y;
  const int m = blockIdx.y * 16 + ty, n = blockIdx.x * 16 + tx;
  const size_t KB = (K + kTileCols - 1) / kTileCols;
  const size_t part_blocks = part_rows > 0 ? (part_rows + kTileRows - 1) / kTileRows : 0;
  float acc = 0.f;
  for (int k0 = 0; k0 < K; k0 += 16) {
    const int xm = blockIdx.y * 16 + ty, xk = k0 + tx;
    xs[ty][tx] = (xm < M && xk < K) ? widen16(X16[static_cast<size_t>(xm) * K + xk], half_in != 0) : 0.f;
    const int wn = blockIdx.x * 16 + ty;
    float wv = 0.f;
    if (wn < N && xk < K) {
      size_t idx = static_cast<size_t>(wn) * K + xk;
      if (tiled) {
        const size_t row = part_rows > 0 ? (wn / part_rows) * part_blocks * kTileRows + wn % part_rows : wn;
        idx = tiled_index(row, xk, KB);
      }
      wv = widen16(W16[idx], half_in != 0);
    }
    ws[ty][tx] = wv;
    __syncthreads();
#pragma unroll
    for (int k = 0; k < 16; ++k) acc = fmaf(xs[ty][k], ws[tx][k], acc);
    __syncthreads();
  }
  if (m < M && n < N) {
    float *y = Y + static_cast<size_t>(m) * ldY + n;
    *y = accumulate ? *y + acc : acc;
  }
}

// Row-major -> block-tiled copy: one CTA per 128 x 64 source tile, 16-byte pieces.
__global__ void __launch_bounds__(256)
retile_kernel(__nv_bfloat16 *dst, const __nv_bfloat16 *src, size_t rows, size_t cols, size_t dst_row0, int to_half) {
  const size_t KB = (cols + kTileCols - 1) / kTileCols;
  const size_t n0 = static_cast<size_t>(blockIdx.y) * kTileRows, k0 = static_cast<size_t>(blockIdx.x) * kTileCols;
  for (int i = threadIdx.x; i < kTileRows * (kTileCols / 8); i += blockDim.x) {
    const size_t n = n0 + i / (kTileCols / 8), k = k0 + (i % (kTileCols / 8)) * 8;
    if (n < rows && k < cols) {
      uint4 v = *reinterpret_cast<const uint4 *>(src + n * cols + k);
      if (to_half) {
        uint32_t *w2 = reinterpret_cast<uint32_t *>(&v);
#pragma unroll
        for (int j = 0; j < 4; ++j)
          w2[j] = cvt16x2(__uint_as_float(w2[j] << 16), __uint_as_float(w2[j] & 0xffff0000u), true);
      }
      *reinterpret_cast<uint4 *>(dst + tiled_index(dst_row0 + n, k, KB)) = v;
    }
  }
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = nullptr;
  if (!fn) {
    void *p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(p);
  }
  return fn;
}

// Output tile map: row-major [rows][cols] fp32 (box 128 x 8) or bf16 (box 64 x 8), no swizzle.
int make_out_map(CUtensorMap *out, void *base, uint64_t rows, uint64_t cols, uint64_t ld, bool bf16) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return -1;
  const uint64_t es = bf16 ? 2 : 4;
  cuuint64_t dims[2] = {cols, rows};
  cuuint64_t strides[1] = {ld * es};
  cuuint32_t box[2] = {static_cast<cuuint32_t>(bf16 ? 64 : kGemmTileN), 8};
  cuuint32_t estr[2] = {1, 1};
  CUresult r = fn(out, bf16 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, base, dims,
                  strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE,
                  CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? 0 : -3;
}

}  // namespace

int make_out_map_box(CUtensorMap *out, void *base, uint64_t rows, uint64_t cols, uint64_t ld, bool bf16,
                     uint32_t box_cols, uint32_t box_rows) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return -1;
  const uint64_t es = bf16 ? 2 : 4;
  if ((reinterpret_cast<uintptr_t>(base) & 15) || ((ld * es) & 15) || box_cols == 0 || box_cols > 256 ||
      box_rows == 0 || box_rows > 256)
    return -2;
  cuuint64_t dims[2] = {cols, rows};
  cuuint64_t strides[1] = {ld * es};
  cuuint32_t box[2] = {box_cols, box_rows};
  cuuint32_t estr[2] = {1, 1};
  CUresult r = fn(out, bf16 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, base, dims,
                  strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE,
                  CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? 0 : -3;
}

int make_tensor_map(CUtensorMap *out, const void *base, uint64_t rows, uint64_t cols, uint64_t ld,
                    uint32_t box_rows) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return -1;
  if ((reinterpret_cast<uintptr_t>(base) & 15) || ((ld * 2) & 15) || box_rows == 0 || box_rows > 256) return -2;
  cuuint64_t dims[2] = {cols, rows};
  cuuint64_t strides[1] = {ld * 2};
  cuuint32_t box[2] = {static_cast<cuuint32_t>(kGemmTileK), box_rows};
  cuuint32_t estr[2] = {1, 1};
  CUresult r = fn(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(base), dims, strides, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? 0 : -3;
}

size_t gemm_workspace_bytes(int bnb) {
  const int ctas = g_num_sms > 0 ? g_num_sms : 148;
  return static_cast<size_t>(ctas) * 3 * kAcc * kGemmTileN * bnb * sizeof(float);
}

cudaError_t gemm_tc_configure() {
  cudaError_t e;
  int dev = 0;
  if ((e = cudaGetDevice(&dev)) != cudaSuccess) return e;
  if ((e = cudaDeviceGetAttribute(&g_num_sms, cudaDevAttrMultiProcessorCount, dev)) != cudaSuccess) return e;
  if ((e = configure_variant<32>()) != cudaSuccess) return e;
  if ((e = configure_variant<64>()) != cudaSuccess) return e;
  if ((e = configure_variant<128>()) != cudaSuccess) return e;
  if ((e = configure_variant<256>()) != cudaSuccess) return e;
  return cudaSuccess;
}

cudaError_t gemm_tc_launch(const GemmArgs &a, cudaStream_t stream) {
  switch (a.bnb) {
    case 32: return launch_variant<32>(a, stream);
    case 64: return launch_variant<64>(a, stream);
    case 128: return launch_variant<128>(a, stream);
    case 256: return launch_variant<256>(a, stream);
    default: return cudaErrorInvalidValue;
  }
}

cudaError_t gemm_simt_launch(const __nv_bfloat16 *X, const __nv_bfloat16 *W, float *Y, int ldY, int M, int N,
                             int K, int accumulate, cudaStream_t stream, int tiled, int part_rows, int half_in) {
  dim3 grid((N + 15) / 16, (M + 15) / 16), block(16, 16);
  gemm_simt_kernel<<<grid, block, 0, stream>>>(X, W, Y, ldY, M, N, K, accumulate, tiled, part_rows, half_in);
  return cudaGetLastError();
}

cudaError_t retile_launch(__nv_bfloat16 *dst, const __nv_bfloat16 *src, size_t rows, size_t cols, size_t dst_row0,
                          cudaStream_t s, bool to_half) {
  if (rows == 0 || cols == 0) return cudaSuccess;
  if (cols % 8 || (reinterpret_cast<uintptr_t>(src) & 15) || (reinterpret_cast<uintptr_t>(dst) & 15))
    return cudaErrorInvalidValue;
  const size_t gx = (cols + kTileCols - 1) / kTileCols, gy = (rows + kTileRows - 1) / kTileRows;
  if (gy > 65535 || gx > 0x7fffffff) return cudaErrorInvalidValue;
  retile_kernel<<<dim3(static_cast<unsigned>(gx), static_cast<unsigned>(gy)), 256, 0, s>>>(dst, src, rows, cols, dst_row0,
                                                                                           to_half ? 1 : 0);
  return cudaGetLastError();
}

int make_tiled_map(CUtensorMap *out, const void *base, uint64_t rows, uint64_t cols, uint32_t box_rows) {
  const uint64_t blocks = ((rows + kTileRows - 1) / kTileRows) * ((cols + kTileCols - 1) / kTileCols);
  return make_tensor_map(out, base, blocks * kTileRows, kTileCols, kTileCols, box_rows);
}

}  // namespace echo

// =============================================================================================
// Projection for callers that cannot allocate device memory.
//
// The stream-K kernel needs scratch for the partial sums of tiles it splits across CTAs.
// echo_gemm_bf16 takes that scratch from the caller.  Some callers have nowhere to get it from:
// code running inside a framework's allocator callback or memory-pool hook, a plug-in that is
// handed tensors but no allocator, or a process whose device memory is fully reserved by another
// runtime.  For them the scratch below is part of the library image: a fixed array in device
// memory that exists on every GPU the library is loaded on, from load until the process exits.
//
// The price is a size limit (kNoAllocMaxRows activation rows, kNoAllocMaxCtas CTAs) and sharing:
// every call uses the same array, so two calls whose kernels may run at the same time (different
// streams, or different host threads) would corrupt each other's partial sums.
// =============================================================================================
namespace echo {
namespace {
constexpr int kNoAllocMaxRows = 32;                   // activation rows (one 32-column accumulator block)
constexpr int kNoAllocMaxCtas = 64;                   // persistent CTAs the variant launches at most
constexpr size_t kNoAllocWsBytes =
    static_cast<size_t>(kNoAllocMaxCtas) * 3 * kAcc * kGemmTileN * kNoAllocMaxRows * sizeof(float);   // 6 MiB
constexpr size_t kNoAllocCounterBytes = static_cast<size_t>(kGemmMaxUnits) * sizeof(int);
constexpr size_t kNoAllocBytes = kNoAllocWsBytes + kNoAllocCounterBytes + 256;   // + the status word
}  // namespace
}  // namespace echo

// Partial-sum slots, the per-tile arrival counters, then the status word of the last call (set when
// a bounded wait of its kernel ran out).  Device code may name this array
// directly; host code must not use the name as a pointer (on the host it is only a handle) and
// asks the runtime for the device address instead.
static __device__ __align__(256) unsigned char g_noalloc_scratch[echo::kNoAllocBytes];

namespace echo {
namespace {
void *g_noalloc_ptr[64] = {};                         // device address of the array, per device ordinal
}  // namespace
}  // namespace echo

extern "C" int echo_gemm_bf16_noalloc(const void *X, const void *W, void *Y, int32_t M, int32_t N, int32_t K,
                                      int32_t epilogue, void *cuda_stream) {
  using namespace echo;
  if (!X || !W || !Y || M < 1 || N < 1 || K < 8 || (K % 8)) return ECHO_ERR_INVALID;
  if (epilogue != EPI_STORE && epilogue != EPI_ACCUM && epilogue != EPI_SWIGLU) return ECHO_ERR_INVALID;
  // the tile copies need 16-byte aligned operands
  if ((reinterpret_cast<uintptr_t>(X) | reinterpret_cast<uintptr_t>(W) | reinterpret_cast<uintptr_t>(Y)) & 15)
    return ECHO_ERR_INVALID;
  if (M > kNoAllocMaxRows) return ECHO_ERR_UNSUPPORTED;           // beyond the built-in scratch
  const bool gu = epilogue == EPI_SWIGLU;
  const int per_tile = kAcc * (gu ? 64 : kGemmTileN);
  if ((N + per_tile - 1) / per_tile > kGemmMaxUnits) return ECHO_ERR_UNSUPPORTED;
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return ECHO_ERR_CUDA;
  if (!g_noalloc_ptr[dev]) {
    // first call on this device: kernel attributes and the array's device address
    if (gemm_tc_configure() != cudaSuccess) return ECHO_ERR_CUDA;
    void *p = nullptr;
    if (cudaGetSymbolAddress(&p, g_noalloc_scratch) != cudaSuccess || !p) return ECHO_ERR_CUDA;
    g_noalloc_ptr[dev] = p;
  }
  cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
  unsigned char *base = static_cast<unsigned char *>(g_noalloc_ptr[dev]);
  int *counters = reinterpret_cast<int *>(base + kNoAllocWsBytes);
  int *status = reinterpret_cast<int *>(base + kNoAllocWsBytes + kNoAllocCounterBytes);
  // the array keeps whatever the previous call left: the counters and the status word must start at zero
  if (cudaMemsetAsync(counters, 0, kNoAllocCounterBytes + sizeof(int), s) != cudaSuccess) return ECHO_ERR_CUDA;
  CUtensorMap tmW, tmX;
  if (make_tensor_map(&tmW, W, gu ? 2ull * N : N, K, K, gu ? 64 : kGemmTileN) != 0) return ECHO_ERR_CUDA;
  if (make_tensor_map(&tmX, X, M, K, K, kNoAllocMaxRows) != 0) return ECHO_ERR_CUDA;
  GemmArgs a{&tmW, &tmX, Y, N, M, N, K, kNoAllocMaxRows, epilogue, status, reinterpret_cast<float *>(base),
             counters, kNoAllocMaxCtas, -1, 0, 0};
  return gemm_tc_launch(a, s) == cudaSuccess ? ECHO_OK : ECHO_ERR_CUDA;
}

extern "C" int echo_gemm_bf16_noalloc_status(void *cuda_stream) {
  using namespace echo;
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return ECHO_ERR_CUDA;
  if (!g_noalloc_ptr[dev]) return ECHO_OK;                        // no call has been made on this device
  cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
  const unsigned char *base = static_cast<const unsigned char *>(g_noalloc_ptr[dev]);
  int st = 0;
  if (cudaMemcpyAsync(&st, base + kNoAllocWsBytes + kNoAllocCounterBytes, sizeof(int), cudaMemcpyDeviceToHost, s) !=
          cudaSuccess ||
      cudaStreamSynchronize(s) != cudaSuccess)
    return ECHO_ERR_CUDA;
  return st == STATUS_WAIT_TIMEOUT ? ECHO_ERR_TIMEOUT : (st == STATUS_OK ? ECHO_OK : ECHO_ERR_DEVICE_CHECK);
}

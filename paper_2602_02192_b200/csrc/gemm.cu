// Dense projections Y = X * W^T for the decoder (bf16 in, fp32 accumulate) on the
// sm_100a tensor cores: tcgen05.mma with the accumulator in tensor memory, operands
// staged in shared memory by TMA (128-byte swizzle), one elected thread issuing MMAs.
//
// Operand roles are swapped with respect to the usual GEMM picture: the WEIGHT tile
// (128 output features x 64 k) is the UMMA "A" operand and fills the 128 TMEM lanes,
// the ACTIVATION tile (bnb rows x 64 k) is the "B" operand and fills bnb TMEM columns.
// A CTA therefore streams each weight byte from HBM exactly once for up to 256
// activation rows, which is what a decode step (a few hundred rows against gigabytes
// of weights) needs; the activation tile is re-read from L2.
//
// Warp roles (192 threads): warp 0 = TMA producer, warp 1 = TMEM owner + MMA issuer,
// warps 2..5 = epilogue (each reads the TMEM lane quarter its warp id selects).
// Every mbarrier wait is bounded; on expiry the kernel records STATUS_WAIT_TIMEOUT,
// drains, frees its tensor memory and returns.

#include "common.cuh"

namespace echo {

namespace {

constexpr int kThreads = 192;
constexpr uint32_t kSpinLimit = 1u << 26;
constexpr uint64_t kWaitLimitNs = 1000000000ull;

__device__ __forceinline__ uint32_t smem_u32(const void *p) {
  return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}
__device__ __forceinline__ void mbar_init(uint64_t *bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t *bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes)
               : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t *bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(smem_u32(bar)), "r"(parity)
      : "memory");
  return ok != 0;
}
__device__ __forceinline__ uint64_t global_timer_ns() {
  uint64_t t;
  asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
  return t;
}
// Bounded wait (about one second of wall time).  Returns false if the limit ran out or
// another role already gave up.
__device__ __forceinline__ bool mbar_wait(uint64_t *bar, uint32_t parity, volatile int *abort_flag) {
  if (mbar_try_wait(bar, parity)) return true;
  const uint64_t t0 = global_timer_ns();
  for (uint32_t i = 0; i < kSpinLimit; ++i) {
    if (mbar_try_wait(bar, parity)) return true;
    if ((i & 63u) == 63u) {
      if (*abort_flag) return false;
      if (global_timer_ns() - t0 > kWaitLimitNs) break;
    }
  }
  *abort_flag = 1;
  return false;
}
__device__ __forceinline__ void tma_load_2d(const CUtensorMap *map, uint64_t *bar, void *dst, int c0, int c1) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
      ::"r"(smem_u32(dst)), "l"(reinterpret_cast<uint64_t>(map)), "r"(smem_u32(bar)), "r"(c0), "r"(c1)
      : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(uint64_t *bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar))
               : "memory");
}
__device__ __forceinline__ void tc_mma_bf16(uint32_t tmem_d, uint64_t desc_a, uint64_t desc_b, uint32_t idesc,
                                            uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(tmem_d), "l"(desc_a), "l"(desc_b), "r"(idesc), "r"(accumulate)
      : "memory");
}
__device__ __forceinline__ void tc_ld32(uint32_t taddr, uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
        "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
        "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr));
}
__device__ __forceinline__ void tc_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// Shared-memory matrix descriptor of a K-major tile whose rows are 128 bytes (64 bf16)
// laid out by TMA with the 128-byte swizzle: groups of 8 rows are 1024 bytes apart.
__device__ __forceinline__ uint64_t smem_desc_sw128(uint32_t saddr) {
  uint64_t d = 0;
  d |= static_cast<uint64_t>((saddr & 0x3FFFFu) >> 4);        // start address / 16
  d |= static_cast<uint64_t>(1) << 16;                         // leading byte offset (unused with swizzle)
  d |= static_cast<uint64_t>(1024 >> 4) << 32;                 // stride between 8-row groups / 16
  d |= static_cast<uint64_t>(1) << 46;                         // descriptor version of this architecture
  d |= static_cast<uint64_t>(2) << 61;                         // 128-byte swizzle
  return d;
}
// Instruction descriptor: bf16 x bf16 -> fp32, both operands K-major, M = 128, N = bnb.
__host__ __device__ constexpr uint32_t instr_desc_bf16(int n) {
  return (1u << 4) | (1u << 7) | (1u << 10) | (static_cast<uint32_t>(n >> 3) << 17) | (8u << 24);
}

template <int BNB, int NACC>
struct GemmSmem {
  static constexpr int kWBytes = kGemmTileN * kGemmTileK * 2;      // 16 KiB per weight block
  static constexpr int kXBytes = BNB * kGemmTileK * 2;
  static constexpr int kStageBytes = NACC * kWBytes + kXBytes;
  static constexpr int kBudget = 220 * 1024;
  static constexpr int kStagesRaw = kBudget / kStageBytes;
  static constexpr int kStages = kStagesRaw > 8 ? 8 : kStagesRaw;
  static constexpr int kBarBytes = 256;
  static constexpr int kTotal = kStages * kStageBytes + kBarBytes + 1024;   // + alignment slack
  static constexpr int kTmemCols = (BNB * NACC) < 32 ? 32 : BNB * NACC;      // power of two by construction
};

__device__ __forceinline__ float silu_f(float a) { return a / (1.0f + __expf(-a)); }

template <int BNB, int NACC>
__global__ void __launch_bounds__(kThreads, 1)
gemm_tc_kernel(const __grid_constant__ CUtensorMap tmW, const __grid_constant__ CUtensorMap tmX,
               void *Yv, int ldY, int M, int N, int K, int epilogue, int *status) {
  using S = GemmSmem<BNB, NACC>;
  extern __shared__ uint8_t smem_raw[];
  uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint64_t *full_bar = reinterpret_cast<uint64_t *>(smem + S::kStages * S::kStageBytes);
  uint64_t *empty_bar = full_bar + S::kStages;
  uint64_t *acc_bar = empty_bar + S::kStages;
  uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(acc_bar + 1);
  volatile int *abort_flag = reinterpret_cast<volatile int *>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const int n0 = blockIdx.x * kGemmTileN;
  const int m0 = blockIdx.y * BNB;
  const int num_kb = (K + kGemmTileK - 1) / kGemmTileK;

  if (threadIdx.x == 0) {
    for (int s = 0; s < S::kStages; ++s) {
      mbar_init(&full_bar[s], 1);
      mbar_init(&empty_bar[s], 1);
    }
    mbar_init(acc_bar, 1);
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)),
                 "r"(static_cast<uint32_t>(S::kTmemCols))
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
      int issued = 0;
      for (int kb = 0; kb < num_kb; ++kb) {
        const int s = kb % S::kStages;
        const uint32_t ph = (kb / S::kStages) & 1;
        if (!mbar_wait(&empty_bar[s], ph ^ 1u, abort_flag)) break;
        uint8_t *stage = smem + s * S::kStageBytes;
        mbar_expect_tx(&full_bar[s], S::kStageBytes);
#pragma unroll
        for (int a = 0; a < NACC; ++a)
          tma_load_2d(&tmW, &full_bar[s], stage + a * S::kWBytes, kb * kGemmTileK, n0 + a * N);
        tma_load_2d(&tmX, &full_bar[s], stage + NACC * S::kWBytes, kb * kGemmTileK, m0);
        issued = kb + 1;
      }
      if (*abort_flag) {
        // let copies already in flight land before the CTA's shared memory is released
        for (int kb = issued > S::kStages ? issued - S::kStages : 0; kb < issued; ++kb) {
          const int s = kb % S::kStages;
          const uint32_t ph = (kb / S::kStages) & 1;
          for (uint32_t i = 0; i < (1u << 16); ++i)
            if (mbar_try_wait(&full_bar[s], ph)) break;
        }
      }
    }
  } else if (warp == 1) {
    // ---------------- MMA issuer ----------------
    if (lane == 0) {
      constexpr uint32_t idesc = instr_desc_bf16(BNB);
      bool ok = true;
      for (int kb = 0; kb < num_kb && ok; ++kb) {
        const int s = kb % S::kStages;
        const uint32_t ph = (kb / S::kStages) & 1;
        ok = mbar_wait(&full_bar[s], ph, abort_flag);
        if (!ok) break;
        tc_fence_after();
        const uint32_t stage = smem_u32(smem + s * S::kStageBytes);
        const uint64_t xdesc = smem_desc_sw128(stage + NACC * S::kWBytes);
#pragma unroll
        for (int a = 0; a < NACC; ++a) {
          const uint64_t wdesc = smem_desc_sw128(stage + a * S::kWBytes);
#pragma unroll
          for (int k = 0; k < kGemmTileK / 16; ++k) {
            // 16 bf16 = 32 bytes further along K inside the swizzled row: +2 in 16-byte units
            tc_mma_bf16(tmem_base + a * BNB, wdesc + 2 * k, xdesc + 2 * k, idesc, (kb > 0 || k > 0) ? 1u : 0u);
          }
        }
        tc_commit(&empty_bar[s]);      // frees the stage once these MMAs have read it
      }
      if (ok) tc_commit(acc_bar);      // accumulator complete
    }
  } else {
    // ---------------- epilogue: TMEM -> registers -> global ----------------
    const int quarter = warp & 3;                      // TMEM lanes 32*quarter .. +31
    const int n = n0 + quarter * 32 + lane;            // output feature of this thread
    const bool got = mbar_wait(acc_bar, 0, abort_flag);
    tc_fence_after();
    if (got) {
      const uint32_t lane_addr = tmem_base + (static_cast<uint32_t>(quarter * 32) << 16);
#pragma unroll 1
      for (int c0 = 0; c0 < BNB; c0 += 32) {
        if (m0 + c0 >= M) break;                       // warp-uniform
        uint32_t r[32];
        tc_ld32(lane_addr + c0, r);
        if (NACC == 2) {
          uint32_t u[32];
          tc_ld32(lane_addr + BNB + c0, u);
          tc_wait_ld();
          if (n < N) {
            __nv_bfloat16 *Y = reinterpret_cast<__nv_bfloat16 *>(Yv);
#pragma unroll
            for (int c = 0; c < 32; ++c) {
              const int m = m0 + c0 + c;
              if (m < M)
                Y[static_cast<size_t>(m) * ldY + n] =
                    __float2bfloat16(silu_f(__uint_as_float(r[c])) * __uint_as_float(u[c]));
            }
          }
        } else {
          tc_wait_ld();
          if (n < N) {
            float *Y = reinterpret_cast<float *>(Yv);
            if (epilogue == EPI_ACCUM) {
#pragma unroll
              for (int c = 0; c < 32; ++c) {
                const int m = m0 + c0 + c;
                if (m < M) Y[static_cast<size_t>(m) * ldY + n] += __uint_as_float(r[c]);
              }
            } else {
#pragma unroll
              for (int c = 0; c < 32; ++c) {
                const int m = m0 + c0 + c;
                if (m < M) Y[static_cast<size_t>(m) * ldY + n] = __uint_as_float(r[c]);
              }
            }
          }
        }
      }
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base),
                 "r"(static_cast<uint32_t>(S::kTmemCols))
                 : "memory");
  }
  if (threadIdx.x == 0 && *abort_flag && status) atomicExch(status, STATUS_WAIT_TIMEOUT);
}

template <int BNB, int NACC>
cudaError_t launch_variant(const GemmArgs &a, cudaStream_t stream) {
  using S = GemmSmem<BNB, NACC>;
  dim3 grid((a.N + kGemmTileN - 1) / kGemmTileN, (a.M + BNB - 1) / BNB, 1);
  gemm_tc_kernel<BNB, NACC><<<grid, kThreads, S::kTotal, stream>>>(*a.tmW, *a.tmX, a.Y, a.ldY, a.M, a.N, a.K,
                                                                  a.epilogue, a.status);
  return cudaGetLastError();
}

template <int BNB, int NACC>
cudaError_t configure_variant() {
  return cudaFuncSetAttribute(gemm_tc_kernel<BNB, NACC>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                              GemmSmem<BNB, NACC>::kTotal);
}

// ---- plain SIMT reference kernel (debugging aid; never on the default path) ----
__global__ void gemm_simt_kernel(const __nv_bfloat16 *X, const __nv_bfloat16 *W, float *Y, int ldY, int M, int N,
                                 int K, int accumulate) {
  __shared__ float xs[16][17], ws[16][17];
  const int tx = threadIdx.x, ty = threadIdx.y;
  const int m = blockIdx.y * 16 + ty, n = blockIdx.x * 16 + tx;
  float acc = 0.f;
  for (int k0 = 0; k0 < K; k0 += 16) {
    const int xm = blockIdx.y * 16 + ty, xk = k0 + tx;
    xs[ty][tx] = (xm < M && xk < K) ? __bfloat162float(X[static_cast<size_t>(xm) * K + xk]) : 0.f;
    const int wn = blockIdx.x * 16 + ty;
    ws[ty][tx] = (wn < N && xk < K) ? __bfloat162float(W[static_cast<size_t>(wn) * K + xk]) : 0.f;
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

}  // namespace

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

cudaError_t gemm_tc_configure() {
  cudaError_t e;
  if ((e = configure_variant<32, 1>()) != cudaSuccess) return e;
  if ((e = configure_variant<64, 1>()) != cudaSuccess) return e;
  if ((e = configure_variant<128, 1>()) != cudaSuccess) return e;
  if ((e = configure_variant<256, 1>()) != cudaSuccess) return e;
  if ((e = configure_variant<32, 2>()) != cudaSuccess) return e;
  if ((e = configure_variant<64, 2>()) != cudaSuccess) return e;
  if ((e = configure_variant<128, 2>()) != cudaSuccess) return e;
  if ((e = configure_variant<256, 2>()) != cudaSuccess) return e;
  return cudaSuccess;
}

cudaError_t gemm_tc_launch(const GemmArgs &a, cudaStream_t stream) {
  const bool two = a.epilogue == EPI_SWIGLU;
  switch (a.bnb) {
    case 32: return two ? launch_variant<32, 2>(a, stream) : launch_variant<32, 1>(a, stream);
    case 64: return two ? launch_variant<64, 2>(a, stream) : launch_variant<64, 1>(a, stream);
    case 128: return two ? launch_variant<128, 2>(a, stream) : launch_variant<128, 1>(a, stream);
    case 256: return two ? launch_variant<256, 2>(a, stream) : launch_variant<256, 1>(a, stream);
    default: return cudaErrorInvalidValue;
  }
}

cudaError_t gemm_simt_launch(const __nv_bfloat16 *X, const __nv_bfloat16 *W, float *Y, int ldY, int M, int N,
                             int K, int accumulate, cudaStream_t stream) {
  dim3 grid((N + 15) / 16, (M + 15) / 16), block(16, 16);
  gemm_simt_kernel<<<grid, block, 0, stream>>>(X, W, Y, ldY, M, N, K, accumulate);
  return cudaGetLastError();
}

}  // namespace echo

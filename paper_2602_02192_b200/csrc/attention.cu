// Attention over the paged KV cache.
//
// attention_rows: one query token per activation row against keys 0..pos of the row's
// page-table row.  Used for prompt prefill (causal by construction: the chunk's K/V is
// appended before its queries run) and as the general decode kernel.  A block serves one
// (row, kv head) and therefore all Hq/Hkv query heads that share that kv head, so every
// K/V byte it loads is used by the whole GQA group.
//
// KV layout of one layer: [page][kv head][K|V][slot in page][head_dim] bf16, i.e. a page of
// one kv head is one contiguous K burst followed by one contiguous V burst.

#include "common.cuh"
#include "ptx.cuh"

namespace echo {

namespace {

constexpr int kAttnWarps = 4;

template <int HD, int REP>
__global__ void __launch_bounds__(kAttnWarps * 32)
attention_rows_kernel(const __nv_bfloat16 *q, const __nv_bfloat16 *kv_layer, __nv_bfloat16 *out,
                      const int32_t *row_pt, const int32_t *row_pos, const int32_t *page_table, int pt_width,
                      int Hq, int Hkv, int page_size, int n_pages, float scale, int *status, int half_io) {
  constexpr int EPL = HD / 32;                       // output dims per lane
  const bool hf = half_io != 0;                      // q, K, V and the output are IEEE half, not bf16
  __shared__ float q_s[REP][HD];
  __shared__ float red_m[kAttnWarps][REP], red_l[kAttnWarps][REP];
  __shared__ float red_o[kAttnWarps][REP][HD];

  const int r = blockIdx.x, kvh = blockIdx.y;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int n_keys = row_pos[r] + 1;
  const int32_t *pt = page_table + static_cast<size_t>(row_pt[r]) * pt_width;
  const size_t page_elems = static_cast<size_t>(page_size) * HD;

  for (int i = threadIdx.x; i < REP * HD; i += blockDim.x) {
    const int a = i / HD, d = i % HD;
    q_s[a][d] = widen16(reinterpret_cast<const uint16_t *>(q)[(static_cast<size_t>(r) * Hq + kvh * REP + a) * HD + d], hf) * scale;
  }
  __syncthreads();

  float m[REP], l[REP], o[REP][EPL];
#pragma unroll
  for (int a = 0; a < REP; ++a) {
    m[a] = -INFINITY;
    l[a] = 0.f;
#pragma unroll
    for (int e = 0; e < EPL; ++e) o[a][e] = 0.f;
  }

  // each warp takes chunks of 32 consecutive keys, one key per lane for the scores
  for (int t0 = warp * 32; t0 < n_keys; t0 += kAttnWarps * 32) {
    const int t = t0 + lane;
    const bool valid = t < n_keys;
    float sc[REP];
#pragma unroll
    for (int a = 0; a < REP; ++a) sc[a] = -INFINITY;
    const __nv_bfloat16 *vrow = nullptr;
    if (valid) {
      const int page = pt[t / page_size];
      if (page < 0 || page >= n_pages) {
        atomicExch(status, STATUS_BAD_PAGE);
      } else {
        const __nv_bfloat16 *krow =
            kv_layer + ((static_cast<size_t>(page) * Hkv + kvh) * 2) * page_elems + (t % page_size) * HD;
        vrow = krow + page_elems;
#pragma unroll
        for (int a = 0; a < REP; ++a) sc[a] = 0.f;
#pragma unroll
        for (int d0 = 0; d0 < HD; d0 += 8) {
          const uint4 raw = *reinterpret_cast<const uint4 *>(krow + d0);
          const uint32_t *k2 = reinterpret_cast<const uint32_t *>(&raw);
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            const float2 kf = widen16x2(k2[i], hf);
#pragma unroll
            for (int a = 0; a < REP; ++a) {
              sc[a] = fmaf(q_s[a][d0 + 2 * i], kf.x, sc[a]);
              sc[a] = fmaf(q_s[a][d0 + 2 * i + 1], kf.y, sc[a]);
            }
          }
        }
      }
    }
    // online softmax over the chunk
    float p[REP];
#pragma unroll
    for (int a = 0; a < REP; ++a) {
      float cm = sc[a];
#pragma unroll
      for (int s = 16; s > 0; s >>= 1) cm = fmaxf(cm, __shfl_xor_sync(0xffffffffu, cm, s));
      const float m_new = fmaxf(m[a], cm);            // finite: lane 0 of the chunk is always valid
      const float corr = __expf(m[a] - m_new);
      p[a] = (sc[a] == -INFINITY) ? 0.f : __expf(sc[a] - m_new);
      float ps = p[a];
#pragma unroll
      for (int s = 16; s > 0; s >>= 1) ps += __shfl_xor_sync(0xffffffffu, ps, s);
      l[a] = l[a] * corr + ps;
      m[a] = m_new;
#pragma unroll
      for (int e = 0; e < EPL; ++e) o[a][e] *= corr;
    }
    // o += p * V : lanes now split the head dimension, keys broadcast one at a time
    const int n_in_chunk = min(32, n_keys - t0);
    for (int kk = 0; kk < n_in_chunk; ++kk) {
      const unsigned long long vp = __shfl_sync(0xffffffffu, reinterpret_cast<unsigned long long>(vrow), kk);
      float pk[REP];
#pragma unroll
      for (int a = 0; a < REP; ++a) pk[a] = __shfl_sync(0xffffffffu, p[a], kk);
      if (vp == 0ull) continue;                        // warp-uniform
      const __nv_bfloat16 *vr = reinterpret_cast<const __nv_bfloat16 *>(vp) + lane * EPL;
      float vf[EPL];
      if (EPL == 4) {
        const uint2 raw = *reinterpret_cast<const uint2 *>(vr);
        const float2 a0 = widen16x2(raw.x, hf), a1 = widen16x2(raw.y, hf);
        vf[0] = a0.x; vf[1] = a0.y; vf[2 % EPL] = a1.x; vf[3 % EPL] = a1.y;
      } else {
        const float2 a0 = widen16x2(*reinterpret_cast<const uint32_t *>(vr), hf);
        vf[0] = a0.x; vf[1] = a0.y;
      }
#pragma unroll
      for (int a = 0; a < REP; ++a)
#pragma unroll
        for (int e = 0; e < EPL; ++e) o[a][e] = fmaf(pk[a], vf[e], o[a][e]);
    }
  }

  // combine the warps
  if (lane == 0) {
#pragma unroll
    for (int a = 0; a < REP; ++a) {
      red_m[warp][a] = m[a];
      red_l[warp][a] = l[a];
    }
  }
#pragma unroll
  for (int a = 0; a < REP; ++a)
#pragma unroll
    for (int e = 0; e < EPL; ++e) red_o[warp][a][lane * EPL + e] = o[a][e];
  __syncthreads();
  for (int i = threadIdx.x; i < REP * HD; i += blockDim.x) {
    const int a = i / HD, d = i % HD;
    float mm = -INFINITY;
    for (int w = 0; w < kAttnWarps; ++w) mm = fmaxf(mm, red_m[w][a]);
    float ll = 0.f, acc = 0.f;
    for (int w = 0; w < kAttnWarps; ++w) {
      if (red_m[w][a] == -INFINITY) continue;
      const float c = __expf(red_m[w][a] - mm);
      ll += red_l[w][a] * c;
      acc += red_o[w][a][d] * c;
    }
    reinterpret_cast<uint16_t *>(out)[(static_cast<size_t>(r) * Hq + kvh * REP + a) * HD + d] = cvt16(acc / ll, hf);
  }
}

template <int HD, int REP>
cudaError_t launch_rows(const __nv_bfloat16 *q, const __nv_bfloat16 *kv_layer, __nv_bfloat16 *out, RowMeta meta,
                        const int32_t *page_table, int pt_width, int R, int Hq, int Hkv, int page_size, int n_pages,
                        int *status, cudaStream_t s, bool half_io) {
  const float scale = 1.0f / sqrtf(static_cast<float>(HD));
  attention_rows_kernel<HD, REP><<<dim3(R, Hkv), kAttnWarps * 32, 0, s>>>(
      q, kv_layer, out, meta.row_pt, meta.row_pos, page_table, pt_width, Hq, Hkv, page_size, n_pages, scale, status,
      half_io ? 1 : 0);
  return cudaGetLastError();
}

}  // namespace

cudaError_t attention_rows_launch(const __nv_bfloat16 *q, const __nv_bfloat16 *kv_layer, __nv_bfloat16 *out,
                                  RowMeta meta, const int32_t *page_table, int pt_width, int R, int Hq, int Hkv,
                                  int hd, int page_size, int n_pages, int *status, cudaStream_t s, bool half_io) {
  const int rep = Hq / Hkv;
#define ECHO_ATTN_CASE(HD_, REP_)                                                                              \
  if (hd == HD_ && rep == REP_)                                                                                \
    return launch_rows<HD_, REP_>(q, kv_layer, out, meta, page_table, pt_width, R, Hq, Hkv, page_size, n_pages, \
                                  status, s, half_io);
  ECHO_ATTN_CASE(64, 1) ECHO_ATTN_CASE(64, 2) ECHO_ATTN_CASE(64, 4)
  ECHO_ATTN_CASE(128, 1) ECHO_ATTN_CASE(128, 2) ECHO_ATTN_CASE(128, 4) ECHO_ATTN_CASE(128, 8)
#undef ECHO_ATTN_CASE
  return cudaErrorInvalidValue;
}

}  // namespace echo

// =============================================================================================
// Decode attention for GRPO rollouts: the G samples of a group share the prompt's KV pages, so
// the prefix is attended ONCE per (group, kv head) for all G * (Hq/Hkv) query rows that use it,
// and only each sample's own generated tokens are read per sample.
//
//   prefix kernel   keys = the prompt's full pages; writes un-normalised partial outputs with their
//                   running max and sum to scratch.  One CTA per (prompt, kv head) when the
//                   group's query rows fill two 16-row tiles (attn_prefix_group_kernel), else one
//                   CTA per (prompt, kv head, 16-row tile) (attn_decode_kernel<HD, true>).
//   suffix kernel   per (sequence, kv head) item: keys = the sequence's private pages (copy of
//                   the prompt's partial last page + generated tokens); merges with the prefix
//                   partial and writes the final bf16 output.  Two forms: one CTA per item
//                   (attn_decode_kernel<HD, false>), and a grid of resident CTAs that draw items
//                   from a counter and keep their page pipelines running across item boundaries
//                   (attn_suffix_resident_kernel, used while sequences hold few generated tokens).
//
// Both run the same tile loop: the four warps of a CTA take pages round-robin; each warp streams
// its pages (one 16-token page of one kv head = K burst + V burst) through its own TMA pipeline
// into 128-byte-swizzled shared memory and does S = Q K^T and O += P V with warp-level bf16 MMAs
// (the query rows are padded to the 16-row MMA tile; the kernel is bound by the KV byte stream,
// not by the tensor pipe).  Softmax runs in the exp2 domain in fp32.
// =============================================================================================
namespace echo {
namespace {

using namespace ptx;

constexpr int kDecWarps = 4;
constexpr int kDecStages = 2;      // 64 KiB per CTA at head_dim 128: three CTAs share an SM
constexpr int kPageTokens = 16;

template <int HD>
struct DecSmem {
  static constexpr int kStageBytes = 2 * kPageTokens * HD * 2;                 // K + V of one page, one head
  static constexpr int kPipeBytes = kDecWarps * kDecStages * kStageBytes;
  static constexpr int kMergeBytes = kDecWarps * 16 * (HD + 2) * 4;
  static constexpr int kBody = kPipeBytes > kMergeBytes ? kPipeBytes : kMergeBytes;
  static constexpr int kTotal = kBody + 256 + 1024;                            // barriers + alignment slack
};

// 16-bit operands of the warp-level MMAs: bf16, or IEEE half in the layers configured that way
template <bool HALF>
__device__ __forceinline__ uint32_t pack_16(float lo, float hi) { return cvt16x2(lo, hi, HALF); }
template <bool HALF>
__device__ __forceinline__ void mma_16816(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  if (HALF) mma_f16_16816(d, a, b0, b1);
  else mma_bf16_16816(d, a, b0, b1);
}

// One 16-token page of one kv head against the warp's 16 query rows: S = Q K^T, online softmax
// (exp2 domain), O += P V.  st = shared-memory address of the page (K burst then V burst, 128-byte
// swizzle); key0 = index of the page's first key; keys at or beyond n_keys are masked.
template <int HD, bool HALF>
__device__ __forceinline__ void decode_tile(uint32_t st, int key0, int n_keys, float scale_log2, int lane,
                                            const uint32_t (&qf)[HD / 16][4], float (&o_acc)[HD / 8][4],
                                            float (&m_run)[2], float (&l_run)[2]) {
  using S = DecSmem<HD>;
  constexpr int KSTEPS = HD / 16;
  constexpr int HALVES = HD / 64;
  const int qi = lane & 3;

  // ---- S = Q K^T : 16 rows x 16 keys -------------------------------------------------------
  float sc[2][4];
#pragma unroll
  for (int i = 0; i < 2; ++i) sc[i][0] = sc[i][1] = sc[i][2] = sc[i][3] = 0.f;
  {
    const int id = lane >> 3, rr = lane & 7;
    const int key = (id >> 1) * 8 + rr;
#pragma unroll
    for (int kk = 0; kk < KSTEPS; ++kk) {
      const int c = 2 * (kk & 3) + (id & 1);
      const uint32_t addr = st + (kk >> 2) * (S::kStageBytes / HALVES) + key * 128 + ((c ^ (key & 7)) << 4);
      uint32_t b0, b1, b2, b3;
      ldmatrix_x4(addr, b0, b1, b2, b3);
      mma_16816<HALF>(sc[0], qf[kk], b0, b1);
      mma_16816<HALF>(sc[1], qf[kk], b2, b3);
    }
  }
  // ---- online softmax (exp2 domain) ---------------------------------------------------------
  float mx[2] = {-INFINITY, -INFINITY};
#pragma unroll
  for (int nt = 0; nt < 2; ++nt) {
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      const int key = key0 + 8 * nt + 2 * qi + (e & 1);
      const float v = key < n_keys ? sc[nt][e] * scale_log2 : -INFINITY;
      sc[nt][e] = v;
      mx[e >> 1] = fmaxf(mx[e >> 1], v);
    }
  }
  uint32_t pa[4];
  {
    float corr[2], msafe[2];
#pragma unroll
    for (int r = 0; r < 2; ++r) {
      mx[r] = fmaxf(mx[r], __shfl_xor_sync(0xffffffffu, mx[r], 1));
      mx[r] = fmaxf(mx[r], __shfl_xor_sync(0xffffffffu, mx[r], 2));
      const float m_new = fmaxf(m_run[r], mx[r]);
      msafe[r] = m_new == -INFINITY ? 0.f : m_new;
      corr[r] = exp2f(m_run[r] - msafe[r]);           // 0 when nothing was accumulated yet
      m_run[r] = m_new;
    }
    float p[2][4], ps[2] = {0.f, 0.f};
#pragma unroll
    for (int nt = 0; nt < 2; ++nt)
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        p[nt][e] = exp2f(sc[nt][e] - msafe[e >> 1]);
        ps[e >> 1] += p[nt][e];
      }
    l_run[0] = l_run[0] * corr[0] + ps[0];
    l_run[1] = l_run[1] * corr[1] + ps[1];
#pragma unroll
    for (int i = 0; i < HD / 8; ++i) {
      o_acc[i][0] *= corr[0]; o_acc[i][1] *= corr[0];
      o_acc[i][2] *= corr[1]; o_acc[i][3] *= corr[1];
    }
    pa[0] = pack_16<HALF>(p[0][0], p[0][1]);
    pa[1] = pack_16<HALF>(p[0][2], p[0][3]);
    pa[2] = pack_16<HALF>(p[1][0], p[1][1]);
    pa[3] = pack_16<HALF>(p[1][2], p[1][3]);
  }
  // ---- O += P V ---------------------------------------------------------------------------
  {
    const int id = lane >> 3, rr = lane & 7;
    const int key = (id & 1) * 8 + rr;
#pragma unroll
    for (int dt = 0; dt < KSTEPS; ++dt) {
      const int c = 2 * (dt & 3) + (id >> 1);
      const uint32_t addr = st + (dt >> 2) * (S::kStageBytes / HALVES) + kPageTokens * 128 + key * 128 +
                            ((c ^ (key & 7)) << 4);
      uint32_t v0, v1, v2, v3;
      ldmatrix_x4_trans(addr, v0, v1, v2, v3);
      mma_16816<HALF>(o_acc[2 * dt], pa, v0, v1);
      mma_16816<HALF>(o_acc[2 * dt + 1], pa, v2, v3);
    }
  }
}

template <int HD, bool PREFIX, bool HALF>
__global__ void __launch_bounds__(kDecWarps * 32)
attn_decode_kernel(const __grid_constant__ CUtensorMap tmKV, const __nv_bfloat16 *__restrict__ q,
                   __nv_bfloat16 *__restrict__ out, float *__restrict__ pre_o, float2 *__restrict__ pre_ml,
                   const int32_t *__restrict__ page_table, int pt_width, const int32_t *__restrict__ row_pos,
                   const int32_t *__restrict__ full_pages, int layer_row0, int Hq, int Hkv, int G, int n_pages,
                   float scale_log2, const int32_t *__restrict__ row_done, int *status,
                   const int32_t *__restrict__ out_row) {
  using S = DecSmem<HD>;
  constexpr int KSTEPS = HD / 16;           // MMA k-steps over the head dimension
  constexpr int HALVES = HD / 64;           // 64-element (128-byte) column blocks per row
  extern __shared__ uint8_t smem_raw[];
  uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint64_t *bars = reinterpret_cast<uint64_t *>(smem + S::kBody);              // [warp][stage]
  volatile int *abort_flag = reinterpret_cast<volatile int *>(bars + kDecWarps * kDecStages);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int REP = Hq / Hkv;
  const int quad = lane >> 2, qi = lane & 3;

  // Ordering under programmatic dependent launch.  The prefix launch waits for its predecessor
  // (the kernel that wrote q and the new K/V rows) and only THEN lets the suffix launch be
  // scheduled: a suffix CTA therefore finds q, the KV pool and the row positions complete without
  // waiting itself, and streams its pages while prefix CTAs are still running.  It waits for the
  // prefix launch only just before it merges with the prefix partials, at the end.
  // A suffix CTA that runs before its own wait must not trust this SM's L1: q, the row positions
  // and the page table are read with L2-only loads (the pages themselves come through TMA).
  if (PREFIX) {
    griddep_wait();
    griddep_launch();
  } else {
    griddep_launch();        // (the output projection may start prefetching its weights)
    // a sequence that has ended (its end token was fed) is not attended: its row is not used.  The CTA
    // still waits for the prefix launch, so that this grid never completes ahead of its predecessor.
    if (row_done && __ldcg(&row_done[blockIdx.x / Hkv])) {
      griddep_wait();
      return;
    }
  }

  // ---- which query rows and which keys this CTA handles ------------------------------------
  int h, seq0, first_page, n_keys, mt = 0;
  if (PREFIX) {
    const int MT = (G * REP + 15) / 16;
    mt = blockIdx.x % MT;
    const int ph = blockIdx.x / MT;
    h = ph % Hkv;
    seq0 = (ph / Hkv) * G;                   // first sequence of the group
    if (row_done) {                          // a group whose sequences have all ended is not attended
      bool any_live = false;
      for (int g = 0; g < G; ++g) any_live |= __ldcg(&row_done[seq0 + g]) == 0;
      if (!any_live) return;
    }
    first_page = 0;
    n_keys = __ldcg(&full_pages[seq0]) * kPageTokens;
  } else {
    h = blockIdx.x % Hkv;
    seq0 = blockIdx.x / Hkv;
    first_page = __ldcg(&full_pages[seq0]);
    n_keys = __ldcg(&row_pos[seq0]) + 1 - first_page * kPageTokens;
  }
  const int n_tiles = (n_keys + kPageTokens - 1) / kPageTokens;
  const int32_t *pt = page_table + static_cast<size_t>(seq0) * pt_width + first_page;

  // row r (0..15) of the MMA tile -> (batch row, q head); -1 when the row is padding
  auto row_seq = [&](int r) -> int {
    if (PREFIX) {
      const int gr = mt * 16 + r;
      return gr < G * REP ? seq0 + gr / REP : -1;
    }
    return r < REP ? seq0 : -1;
  };
  auto row_head = [&](int r) -> int { return h * REP + (PREFIX ? (mt * 16 + r) % REP : r); };

  if (threadIdx.x == 0) {
    for (int i = 0; i < kDecWarps * kDecStages; ++i) mbar_init(&bars[i], 1);
    *abort_flag = 0;
    mbar_fence_init();
  }
  __syncthreads();

  float o_acc[HD / 8][4];
#pragma unroll
  for (int i = 0; i < HD / 8; ++i) o_acc[i][0] = o_acc[i][1] = o_acc[i][2] = o_acc[i][3] = 0.f;
  float m_run[2] = {-INFINITY, -INFINITY}, l_run[2] = {0.f, 0.f};

  uint8_t *my_stages = smem + warp * kDecStages * S::kStageBytes;
  uint64_t *my_bars = bars + warp * kDecStages;
  const int n_my = n_tiles > warp ? (n_tiles - warp + kDecWarps - 1) / kDecWarps : 0;

  int pg_cache = 0, pg_base = -1;            // page ids of 32 of this warp's tiles, one per lane
  auto page_of = [&](int k) -> int {         // warp-uniform k
    if (k < pg_base || k >= pg_base + 32 || pg_base < 0) {
      pg_base = k;
      const int kk = k + lane;
      pg_cache = kk < n_my ? __ldcg(&pt[warp + kDecWarps * kk]) : 0;
    }
    return __shfl_sync(0xffffffffu, pg_cache, k - pg_base);
  };
  auto issue = [&](int k) {
    const int page = page_of(k);
    if (lane == 0) {
      uint64_t *bar = &my_bars[k % kDecStages];
      uint8_t *dst = my_stages + (k % kDecStages) * S::kStageBytes;
      if (page < 0 || page >= n_pages) {
        atomicExch(status, STATUS_BAD_PAGE);
        mbar_arrive(bar);                    // nothing to load: complete the phase by hand
      } else {
        const int row = layer_row0 + (page * Hkv + h) * 2 * kPageTokens;
        mbar_expect_tx(bar, S::kStageBytes);
#pragma unroll
        for (int hf = 0; hf < HALVES; ++hf) tma_load_2d(&tmKV, bar, dst + hf * (S::kStageBytes / HALVES), hf * 64, row);
      }
    }
  };

  const int n_pro = n_my < kDecStages ? n_my : kDecStages;
  for (int k = 0; k < n_pro; ++k) issue(k);

  // (the first pages are on their way; everything below overlaps their latency)
  // ---- Q fragments (A operand), kept in registers for the whole loop ---------------------------
  uint32_t qf[KSTEPS][4];
  {
    const int s_lo = row_seq(quad), s_hi = row_seq(quad + 8);
    const uint32_t *q_lo = s_lo >= 0 ? reinterpret_cast<const uint32_t *>(
                                           q + (static_cast<size_t>(s_lo) * Hq + row_head(quad)) * HD)
                                     : nullptr;
    const uint32_t *q_hi = s_hi >= 0 ? reinterpret_cast<const uint32_t *>(
                                           q + (static_cast<size_t>(s_hi) * Hq + row_head(quad + 8)) * HD)
                                     : nullptr;
#pragma unroll
    for (int kk = 0; kk < KSTEPS; ++kk) {
      qf[kk][0] = q_lo ? __ldcg(&q_lo[kk * 8 + qi]) : 0u;
      qf[kk][1] = q_hi ? __ldcg(&q_hi[kk * 8 + qi]) : 0u;
      qf[kk][2] = q_lo ? __ldcg(&q_lo[kk * 8 + 4 + qi]) : 0u;
      qf[kk][3] = q_hi ? __ldcg(&q_hi[kk * 8 + 4 + qi]) : 0u;
    }
  }


  bool ok = true;
  for (int k = 0; k < n_my; ++k) {
    ok = mbar_wait(&my_bars[k % kDecStages], (k / kDecStages) & 1, abort_flag);
    if (!ok) break;
    const uint32_t st = smem_u32(my_stages + (k % kDecStages) * S::kStageBytes);
    const int key0 = (warp + kDecWarps * k) * kPageTokens;
    decode_tile<HD, HALF>(st, key0, n_keys, scale_log2, lane, qf, o_acc, m_run, l_run);
    __syncwarp();
    if (k + kDecStages < n_my) issue(k + kDecStages);
  }
  if (!ok) {
    // give copies already in flight a chance to land before shared memory is reused or released
    for (int k = 0; k < n_my; ++k) mbar_drain(&my_bars[k % kDecStages], (k / kDecStages) & 1);
  }
  // row sums: combine the four lanes that share a row
#pragma unroll
  for (int r = 0; r < 2; ++r) {
    l_run[r] += __shfl_xor_sync(0xffffffffu, l_run[r], 1);
    l_run[r] += __shfl_xor_sync(0xffffffffu, l_run[r], 2);
  }

  // ---- prefix partials (suffix kernel): the prefix launch must be complete from here on --------
  constexpr int kPre = 8;
  float pre_val[kPre];
  float2 pre_stat[kPre];
  const bool pre_ok = !PREFIX && REP * HD <= kPre * kDecWarps * 32;
  if (!PREFIX) griddep_wait();
  if (pre_ok) {
#pragma unroll
    for (int i = 0; i < kPre; ++i) {
      const int idx = threadIdx.x + i * kDecWarps * 32;
      pre_val[i] = 0.f;
      pre_stat[i] = make_float2(-INFINITY, 0.f);
      if (idx < REP * HD) {
        const int r = idx / HD, d = idx % HD;
        const size_t rh = static_cast<size_t>(seq0) * Hq + h * REP + r;
        pre_stat[i] = __ldcg(&pre_ml[rh]);
        pre_val[i] = __ldcg(&pre_o[rh * HD + d]);
      }
    }
  }

  // ---- combine the four warps through shared memory (the pipeline buffers are free now) -------
  __syncthreads();
  float *m_s = reinterpret_cast<float *>(smem);                      // [warp][16]
  float *l_s = m_s + kDecWarps * 16;
  float *o_s = l_s + kDecWarps * 16;                                 // [warp][16][HD]
  if (qi == 0) {
    m_s[warp * 16 + quad] = m_run[0];
    m_s[warp * 16 + quad + 8] = m_run[1];
    l_s[warp * 16 + quad] = l_run[0];
    l_s[warp * 16 + quad + 8] = l_run[1];
  }
#pragma unroll
  for (int i = 0; i < HD / 8; ++i) {
    float *o_lo = o_s + (warp * 16 + quad) * HD + 8 * i + 2 * qi;
    float *o_hi = o_s + (warp * 16 + quad + 8) * HD + 8 * i + 2 * qi;
    o_lo[0] = o_acc[i][0]; o_lo[1] = o_acc[i][1];
    o_hi[0] = o_acc[i][2]; o_hi[1] = o_acc[i][3];
  }
  __syncthreads();
  const int n_rows = PREFIX ? 16 : REP;
  for (int idx = threadIdx.x; idx < n_rows * HD; idx += blockDim.x) {
    const int r = idx / HD, d = idx % HD;
    const int s = row_seq(r);
    if (s < 0) continue;
    float M = -INFINITY;
#pragma unroll
    for (int w = 0; w < kDecWarps; ++w) M = fmaxf(M, m_s[w * 16 + r]);
    float L = 0.f, O = 0.f;
#pragma unroll
    for (int w = 0; w < kDecWarps; ++w) {
      const float mw = m_s[w * 16 + r];
      if (mw != -INFINITY) {
        const float c = exp2f(mw - M);
        L += l_s[w * 16 + r] * c;
        O += o_s[(w * 16 + r) * HD + d] * c;
      }
    }
    const size_t oi = (static_cast<size_t>(s) * Hq + row_head(r)) * HD + d;
    if (PREFIX) {
      pre_o[oi] = O;
      if (d == 0) pre_ml[static_cast<size_t>(s) * Hq + row_head(r)] = make_float2(M, L);
    } else {
      const int it = idx / (kDecWarps * 32);
      float2 ml;
      float po;
      if (pre_ok) {
        ml = pre_stat[0];
        po = pre_val[0];
#pragma unroll
        for (int i = 1; i < kPre; ++i)
          if (it == i) {
            ml = pre_stat[i];
            po = pre_val[i];
          }
      } else {
        ml = __ldcg(&pre_ml[static_cast<size_t>(s) * Hq + row_head(r)]);
        po = __ldcg(&pre_o[oi]);
      }
      float Mt = fmaxf(M, ml.x);
      if (Mt == -INFINITY) Mt = 0.f;
      const float c_suf = M == -INFINITY ? 0.f : exp2f(M - Mt);
      const float c_pre = ml.x == -INFINITY ? 0.f : exp2f(ml.x - Mt);
      const float Lt = L * c_suf + ml.y * c_pre;
      const float Ot = O * c_suf + (c_pre != 0.f ? po * c_pre : 0.f);
      // compacted step: the sequence's output goes to the activation row it occupies
      const size_t oo = out_row ? (static_cast<size_t>(__ldcg(&out_row[s])) * Hq + row_head(r)) * HD + d : oi;
      reinterpret_cast<uint16_t *>(out)[oo] = cvt16(Ot / Lt, HALF);
    }
  }
  if (threadIdx.x == 0 && *abort_flag) atomicExch(status, STATUS_WAIT_TIMEOUT);
}

// ---------------------------------------------------------------------------------------------
// Suffix attention with resident CTAs.  With one CTA per (sequence, kv head) every CTA pays its
// start-up chain (row position -> page ids -> first pages) and its merge with an idle copy
// pipeline, and CTAs of equal length march through those phases together.  Here a grid that just
// fills the GPU walks the (sequence, kv head) items round-robin, and each warp's page pipeline
// runs on across item boundaries: the first pages of the next item are requested before the
// current item is merged, and the next item's row position and page ids are fetched one item
// ahead, so the copy engine stays busy while partial results are combined and written.
// Shared memory: the four warps' page stages, then a merge area of REP rows per warp.
// ---------------------------------------------------------------------------------------------
constexpr int kSufPre = 4;                  // merged outputs per thread: REP * HD <= kSufPre * threads

template <int HD>
struct SufSmem {
  static constexpr int kStageBytes = DecSmem<HD>::kStageBytes;
  static constexpr int kPipeBytes = DecSmem<HD>::kPipeBytes;
  static constexpr int kRowStride = HD + 8;                                    // floats; spreads rows over banks
  static constexpr int kStatFloats = 2 * kDecWarps * 16;                       // running max and sum per warp row
  static constexpr int merge_bytes(int rep) { return (kStatFloats + kDecWarps * rep * kRowStride) * 4; }
  static constexpr int total(int rep) { return 1024 + kPipeBytes + merge_bytes(rep) + 256; }
};

template <int HD, bool HALF>
__global__ void __launch_bounds__(kDecWarps * 32)
attn_suffix_resident_kernel(const __grid_constant__ CUtensorMap tmKV, const __nv_bfloat16 *__restrict__ q,
                            __nv_bfloat16 *__restrict__ out, const float *__restrict__ pre_o,
                            const float2 *__restrict__ pre_ml, const int32_t *__restrict__ page_table, int pt_width,
                            const int32_t *__restrict__ row_pos, const int32_t *__restrict__ full_pages,
                            int layer_row0, int Hq, int Hkv, int n_items, int n_pages, float scale_log2,
                            const int32_t *__restrict__ row_done, int *status, int *work,
                            const int32_t *__restrict__ out_row) {
  using S = SufSmem<HD>;
  constexpr int KSTEPS = HD / 16;
  constexpr int HALVES = HD / 64;
  extern __shared__ uint8_t smem_raw[];
  uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  const int REP = Hq / Hkv;
  float *m_s = reinterpret_cast<float *>(smem + S::kPipeBytes);               // [warp][16]
  float *l_s = m_s + kDecWarps * 16;
  float *o_s = l_s + kDecWarps * 16;                                          // [warp][REP][kRowStride]
  uint64_t *bars = reinterpret_cast<uint64_t *>(smem + S::kPipeBytes + S::merge_bytes(REP));   // [warp][stage]
  volatile int *abort_flag = reinterpret_cast<volatile int *>(bars + kDecWarps * kDecStages);
  volatile int *ticket_s = abort_flag + 1;   // [2]: item numbers drawn by thread 0, alternating slots

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int quad = lane >> 2, qi = lane & 3;

  // Items are handed out through a counter: CTA b starts with item b and draws every later item
  // (work[0] counts the draws), so CTAs that start late or run slow take fewer items.  A draw is made
  // two items ahead by thread 0 and passed on at a barrier the merge needs anyway.  work[1] counts
  // finished CTAs; the last one puts both words back to zero for the next launch.
  // The prefix launch (the predecessor) let this grid start only after its own dependency wait:
  // q, the KV pool, row positions and page ids are complete.  They are read with L2-only loads or
  // TMA; the prefix partials are read after griddep_wait() below.
  griddep_launch();
  if (threadIdx.x == 0) {
    for (int i = 0; i < kDecWarps * kDecStages; ++i) mbar_init(&bars[i], 1);
    *abort_flag = 0;
    mbar_fence_init();
    ticket_s[1] = gridDim.x + atomicAdd(&work[0], 1);
  }
  __syncthreads();
  int m1 = ticket_s[1];                      // the item after this CTA's first one

  uint8_t *my_stages = smem + warp * kDecStages * S::kStageBytes;
  uint64_t *my_bars = bars + warp * kDecStages;
  uint32_t g_iss = 0, g_cons = 0;            // pages requested / consumed by this warp since the start

  auto issue_page = [&](int page, int h) {   // warp-uniform arguments
    if (lane == 0) {
      uint64_t *bar = &my_bars[g_iss % kDecStages];
      uint8_t *dst = my_stages + (g_iss % kDecStages) * S::kStageBytes;
      if (page < 0 || page >= n_pages) {
        atomicExch(status, STATUS_BAD_PAGE);
        mbar_arrive(bar);                    // nothing to load: complete the phase by hand
      } else {
        const int row = layer_row0 + (page * Hkv + h) * 2 * kPageTokens;
        mbar_expect_tx(bar, S::kStageBytes);
#pragma unroll
        for (int hf = 0; hf < HALVES; ++hf) tma_load_2d(&tmKV, bar, dst + hf * (S::kStageBytes / HALVES), hf * 64, row);
      }
    }
    ++g_iss;
  };
  // Item m -> (sequence, kv head).  Its description is fetched in two hops that are issued well
  // before their results are used: raw words (ended flag, prompt pages, position) first, then the
  // page ids of this warp's first 32 pages, whose address depends on the first hop.
  auto raw_words = [&](int m, int &seq, int &h, int &dn, int &fp, int &rp) {
    const bool valid = m < n_items;
    seq = valid ? m / Hkv : 0;
    h = valid ? m - seq * Hkv : 0;
    dn = row_done ? __ldcg(&row_done[seq]) : 0;
    fp = __ldcg(&full_pages[seq]);
    rp = __ldcg(&row_pos[seq]);
    if (!valid) dn = 1;
  };
  // keys of the item (-1: an ended sequence or past the last item: nothing to do, nothing written),
  // this warp's number of pages, and lane j's page id of the warp's page j
  auto shape = [&](int seq, int dn, int fp, int rp, int &n_keys, int &n_my, int &pg) {
    n_keys = dn ? -1 : rp + 1 - fp * kPageTokens;
    const int n_tiles = dn ? 0 : (n_keys + kPageTokens - 1) / kPageTokens;
    n_my = n_tiles > warp ? (n_tiles - warp + kDecWarps - 1) / kDecWarps : 0;
    pg = lane < n_my ? __ldcg(&page_table[static_cast<size_t>(seq) * pt_width + fp + warp + kDecWarps * lane]) : 0;
  };
  // Q fragments of an item (rows >= REP of the MMA tile are padding)
  uint32_t qf[KSTEPS][4];
  auto load_q = [&](int seq, int h) {
    const uint32_t *q_lo = quad < REP ? reinterpret_cast<const uint32_t *>(
                                            q + (static_cast<size_t>(seq) * Hq + h * REP + quad) * HD)
                                      : nullptr;
    const uint32_t *q_hi = quad + 8 < REP ? reinterpret_cast<const uint32_t *>(
                                                q + (static_cast<size_t>(seq) * Hq + h * REP + quad + 8) * HD)
                                          : nullptr;
#pragma unroll
    for (int kk = 0; kk < KSTEPS; ++kk) {
      qf[kk][0] = q_lo ? __ldcg(&q_lo[kk * 8 + qi]) : 0u;
      qf[kk][1] = q_hi ? __ldcg(&q_hi[kk * 8 + qi]) : 0u;
      qf[kk][2] = q_lo ? __ldcg(&q_lo[kk * 8 + 4 + qi]) : 0u;
      qf[kk][3] = q_hi ? __ldcg(&q_hi[kk * 8 + 4 + qi]) : 0u;
    }
  };

  int m = blockIdx.x;
  int c_seq, c_h, c_fp, c_keys, c_my, c_pg;
  {
    int dn, rp;
    raw_words(m, c_seq, c_h, dn, c_fp, rp);
    shape(c_seq, dn, c_fp, rp, c_keys, c_my, c_pg);
  }
  {
    const int c_first = c_my < kDecStages ? c_my : kDecStages;
    for (int k = 0; k < c_first; ++k) issue_page(__shfl_sync(0xffffffffu, c_pg, k), c_h);
  }
  load_q(c_seq, c_h);
  bool waited = false;

  for (int n = 0; m < n_items; ++n) {
    // ---- the next item, one item ahead: first hop now, second hop after the first page ---------
    // thread 0 draws the item after the next one, late in the current item (a CTA that commits to
    // items early leaves others idle at the end of the launch) but a few pages before the barrier
    // that passes it on, so that the counter's round trip is hidden
    int drawn = 0;
    const int draw_at = c_keys >= 0 && c_my > 3 ? c_my - 3 : -1;
    if (threadIdx.x == 0 && draw_at < 0) drawn = gridDim.x + atomicAdd(&work[0], 1);
    int n_seq, n_h, n_dn, n_fp, n_rp;
    raw_words(m1, n_seq, n_h, n_dn, n_fp, n_rp);
    int n_keys = -1, n_my = 0, n_pg = 0, n_first = 0, nxt_issued = 0, m2 = 0;
    auto second_hop = [&]() {
      shape(n_seq, n_dn, n_fp, n_rp, n_keys, n_my, n_pg);
      n_first = n_my < kDecStages ? n_my : kDecStages;
    };
    auto issue_next = [&]() {                // one more of the next item's first pages
      issue_page(__shfl_sync(0xffffffffu, n_pg, nxt_issued), n_h);
      ++nxt_issued;
    };

    if (c_keys >= 0) {                       // CTA-uniform
      float o_acc[HD / 8][4];
#pragma unroll
      for (int i = 0; i < HD / 8; ++i) o_acc[i][0] = o_acc[i][1] = o_acc[i][2] = o_acc[i][3] = 0.f;
      float m_run[2] = {-INFINITY, -INFINITY}, l_run[2] = {0.f, 0.f};
      int pg_cache = c_pg, pg_base = 0;
      const int32_t *pt = page_table + static_cast<size_t>(c_seq) * pt_width + c_fp;
      bool ok = true;
      if (c_my == 0) second_hop();

      for (int k = 0; k < c_my; ++k) {
        if (threadIdx.x == 0 && k == draw_at) drawn = gridDim.x + atomicAdd(&work[0], 1);
        ok = mbar_wait(&my_bars[g_cons % kDecStages], (g_cons / kDecStages) & 1, abort_flag);
        if (!ok) break;
        const uint32_t st = smem_u32(my_stages + (g_cons % kDecStages) * S::kStageBytes);
        decode_tile<HD, HALF>(st, (warp + kDecWarps * k) * kPageTokens, c_keys, scale_log2, lane, qf, o_acc, m_run,
                              l_run);
        __syncwarp();
        ++g_cons;
        if (k == 0) second_hop();
        const int kn = k + kDecStages;
        if (kn < c_my) {
          if (kn >= pg_base + 32) {
            pg_base = kn;
            pg_cache = kn + lane < c_my ? __ldcg(&pt[warp + kDecWarps * (kn + lane)]) : 0;
          }
          issue_page(__shfl_sync(0xffffffffu, pg_cache, kn - pg_base), c_h);
        } else if (nxt_issued < n_first) {
          issue_next();
        }
      }
      if (ok)
        while (nxt_issued < n_first) issue_next();
      // ---- prefix partials of this item: the prefix launch must be complete from here on -------
      if (!waited) {
        griddep_wait();
        waited = true;
      }
      float pre_val[kSufPre];
      float2 pre_stat[kSufPre];
#pragma unroll
      for (int i = 0; i < kSufPre; ++i) {
        const int idx = threadIdx.x + i * kDecWarps * 32;
        pre_val[i] = 0.f;
        pre_stat[i] = make_float2(-INFINITY, 0.f);
        if (idx < REP * HD) {
          const size_t rh = static_cast<size_t>(c_seq) * Hq + c_h * REP + idx / HD;
          pre_stat[i] = __ldcg(&pre_ml[rh]);
          pre_val[i] = __ldcg(&pre_o[rh * HD + idx % HD]);
        }
      }
      if (ok && n_keys >= 0) load_q(n_seq, n_h);     // the next item's queries land during the merge
#pragma unroll
      for (int r = 0; r < 2; ++r) {
        l_run[r] += __shfl_xor_sync(0xffffffffu, l_run[r], 1);
        l_run[r] += __shfl_xor_sync(0xffffffffu, l_run[r], 2);
      }
      // ---- combine the four warps ----------------------------------------------------------------
      if (qi == 0) {
        m_s[warp * 16 + quad] = m_run[0];
        m_s[warp * 16 + quad + 8] = m_run[1];
        l_s[warp * 16 + quad] = l_run[0];
        l_s[warp * 16 + quad + 8] = l_run[1];
      }
      if (quad < REP) {
        float *o_lo = o_s + (warp * REP + quad) * S::kRowStride + 2 * qi;
#pragma unroll
        for (int i = 0; i < HD / 8; ++i) *reinterpret_cast<float2 *>(o_lo + 8 * i) = make_float2(o_acc[i][0], o_acc[i][1]);
      }
      if (quad + 8 < REP) {
        float *o_hi = o_s + (warp * REP + quad + 8) * S::kRowStride + 2 * qi;
#pragma unroll
        for (int i = 0; i < HD / 8; ++i) *reinterpret_cast<float2 *>(o_hi + 8 * i) = make_float2(o_acc[i][2], o_acc[i][3]);
      }
      if (threadIdx.x == 0) ticket_s[n & 1] = drawn;
      __syncthreads();
      if (*abort_flag) break;                // some warp gave up: every thread of the CTA sees it here
      m2 = ticket_s[n & 1];
#pragma unroll
      for (int i = 0; i < kSufPre; ++i) {
        const int idx = threadIdx.x + i * kDecWarps * 32;
        if (idx < REP * HD) {
          const int r = idx / HD, d = idx % HD;
          float M = -INFINITY;
#pragma unroll
          for (int w = 0; w < kDecWarps; ++w) M = fmaxf(M, m_s[w * 16 + r]);
          float L = 0.f, O = 0.f;
#pragma unroll
          for (int w = 0; w < kDecWarps; ++w) {
            const float mw = m_s[w * 16 + r];
            if (mw != -INFINITY) {
              const float c = exp2f(mw - M);
              L += l_s[w * 16 + r] * c;
              O += o_s[(w * REP + r) * S::kRowStride + d] * c;
            }
          }
          const float2 ml = pre_stat[i];
          float Mt = fmaxf(M, ml.x);
          if (Mt == -INFINITY) Mt = 0.f;
          const float c_suf = M == -INFINITY ? 0.f : exp2f(M - Mt);
          const float c_pre = ml.x == -INFINITY ? 0.f : exp2f(ml.x - Mt);
          const float Lt = L * c_suf + ml.y * c_pre;
          const float Ot = O * c_suf + (c_pre != 0.f ? pre_val[i] * c_pre : 0.f);
          // compacted step: the sequence's output goes to the activation row it occupies
          const size_t o_seq = out_row ? static_cast<size_t>(__ldcg(&out_row[c_seq])) : static_cast<size_t>(c_seq);
          reinterpret_cast<uint16_t *>(out)[(o_seq * Hq + c_h * REP + r) * HD + d] = cvt16(Ot / Lt, HALF);
        }
      }
      __syncthreads();                       // the merge area is free for the next item
    } else {
      second_hop();
      while (nxt_issued < n_first) issue_next();
      if (n_keys >= 0) load_q(n_seq, n_h);
      if (threadIdx.x == 0) ticket_s[n & 1] = drawn;
      __syncthreads();
      m2 = ticket_s[n & 1];
    }
    m = m1;
    m1 = m2;
    c_seq = n_seq; c_h = n_h; c_fp = n_fp; c_keys = n_keys; c_my = n_my; c_pg = n_pg;
  }
  if (*abort_flag) {
    // give copies already in flight a chance to land before shared memory is released
    for (uint32_t g = g_cons; g < g_iss; ++g) mbar_drain(&my_bars[g % kDecStages], (g / kDecStages) & 1);
    if (threadIdx.x == 0) atomicExch(status, STATUS_WAIT_TIMEOUT);
  }
  if (!waited) griddep_wait();               // this grid never completes ahead of its predecessor
  if (threadIdx.x == 0) {
    __threadfence();
    if (atomicAdd(&work[1], 1) == static_cast<int>(gridDim.x) - 1) {
      atomicExch(&work[0], 0);
      atomicExch(&work[1], 0);
    }
  }
}

// ---------------------------------------------------------------------------------------------
// Prefix attention with MT 16-row tiles of a group's query rows in one CTA.  With one tile per CTA
// a group of G * REP = 32 rows takes two CTAs per (prompt, kv head), which stream the same pages
// twice (the second time from L2) and make the launch larger than the GPU holds at once.  Here one
// CTA keeps MT tiles (a group with more rows takes ceil(rows / (MT * 16)) CTAs): every K and V fragment it reads from shared memory feeds MT MMAs.  The queries
// stay in shared memory (16-byte chunks swizzled by row, read back with ldmatrix) so that the MT
// accumulators fit the register file.
// ---------------------------------------------------------------------------------------------
template <int HD, int MT>
struct PreSmem {
  static constexpr int kStageBytes = DecSmem<HD>::kStageBytes;
  static constexpr int kPipeBytes = DecSmem<HD>::kPipeBytes;
  static constexpr int kQBytes = MT * 16 * HD * 2;
  static constexpr int kRowStride = HD + 8;                                    // floats; spreads rows over banks
  static constexpr int kMergeBytes = kDecWarps * MT * 16 * (kRowStride + 2) * 4;
  static constexpr int kBody = kPipeBytes + kQBytes > kMergeBytes ? kPipeBytes + kQBytes : kMergeBytes;
  static constexpr int kTotal = kBody + 256 + 1024;
};

template <int HD, int MT, bool HALF>
__global__ void __launch_bounds__(kDecWarps * 32)
attn_prefix_group_kernel(const __grid_constant__ CUtensorMap tmKV, const __nv_bfloat16 *__restrict__ q,
                         float *__restrict__ pre_o, float2 *__restrict__ pre_ml,
                         const int32_t *__restrict__ page_table, int pt_width, const int32_t *__restrict__ full_pages,
                         int layer_row0, int Hq, int Hkv, int G, int n_pages, float scale_log2, int *status,
                         const int32_t *__restrict__ row_done) {
  using S = PreSmem<HD, MT>;
  constexpr int KSTEPS = HD / 16;
  constexpr int HALVES = HD / 64;
  constexpr int CHUNKS = HD / 8;             // 16-byte chunks per query row
  extern __shared__ uint8_t smem_raw[];
  uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t *q_s = smem + S::kPipeBytes;
  uint64_t *bars = reinterpret_cast<uint64_t *>(smem + S::kBody);              // [warp][stage]
  volatile int *abort_flag = reinterpret_cast<volatile int *>(bars + kDecWarps * kDecStages);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int REP = Hq / Hkv;
  const int quad = lane >> 2, qi = lane & 3;
  // a group with more than MT * 16 query rows takes several CTAs per (prompt, kv head)
  const int n_blocks = (G * REP + MT * 16 - 1) / (MT * 16);
  const int row0 = (blockIdx.x % n_blocks) * MT * 16;
  const int n_rows = G * REP - row0 < MT * 16 ? G * REP - row0 : MT * 16;

  // wait for the kernel that wrote q and the new K/V rows, then let the suffix launch be scheduled
  griddep_wait();
  griddep_launch();

  const int h = (blockIdx.x / n_blocks) % Hkv;
  const int seq0 = (blockIdx.x / n_blocks / Hkv) * G;   // first sequence of the group
  if (row_done) {
    // a group whose sequences have all ended (or a slot that holds no group) is not attended: nobody
    // reads its partial results, and its page-table rows may be stale
    bool any_live = false;
    for (int g = 0; g < G; ++g) any_live |= __ldcg(&row_done[seq0 + g]) == 0;
    if (!any_live) return;
  }
  const int n_keys = __ldcg(&full_pages[seq0]) * kPageTokens;
  const int n_tiles = n_keys / kPageTokens;
  const int32_t *pt = page_table + static_cast<size_t>(seq0) * pt_width;

  if (threadIdx.x == 0) {
    for (int i = 0; i < kDecWarps * kDecStages; ++i) mbar_init(&bars[i], 1);
    *abort_flag = 0;
    mbar_fence_init();
  }
  __syncthreads();

  uint8_t *my_stages = smem + warp * kDecStages * S::kStageBytes;
  uint64_t *my_bars = bars + warp * kDecStages;
  const int n_my = n_tiles > warp ? (n_tiles - warp + kDecWarps - 1) / kDecWarps : 0;

  int pg_cache = 0, pg_base = -1;            // page ids of 32 of this warp's tiles, one per lane
  auto page_of = [&](int k) -> int {         // warp-uniform k
    if (pg_base < 0 || k >= pg_base + 32) {
      pg_base = k;
      const int kk = k + lane;
      pg_cache = kk < n_my ? __ldcg(&pt[warp + kDecWarps * kk]) : 0;
    }
    return __shfl_sync(0xffffffffu, pg_cache, k - pg_base);
  };
  auto issue = [&](int k) {
    const int page = page_of(k);
    if (lane == 0) {
      uint64_t *bar = &my_bars[k % kDecStages];
      uint8_t *dst = my_stages + (k % kDecStages) * S::kStageBytes;
      if (page < 0 || page >= n_pages) {
        atomicExch(status, STATUS_BAD_PAGE);
        mbar_arrive(bar);                    // nothing to load: complete the phase by hand
      } else {
        const int row = layer_row0 + (page * Hkv + h) * 2 * kPageTokens;
        mbar_expect_tx(bar, S::kStageBytes);
#pragma unroll
        for (int hf = 0; hf < HALVES; ++hf) tma_load_2d(&tmKV, bar, dst + hf * (S::kStageBytes / HALVES), hf * 64, row);
      }
    }
  };
  const int n_pro = n_my < kDecStages ? n_my : kDecStages;
  for (int k = 0; k < n_pro; ++k) issue(k);

  // ---- queries -> shared memory: row r = (sequence seq0 + (row0 + r) / REP, head h * REP + (row0 + r) % REP)
  for (int c = threadIdx.x; c < MT * 16 * CHUNKS; c += kDecWarps * 32) {
    const int r = c / CHUNKS, ch = c % CHUNKS;
    const int gr = row0 + r;
    uint4 v = make_uint4(0u, 0u, 0u, 0u);
    if (r < n_rows)
      v = __ldcg(reinterpret_cast<const uint4 *>(q + (static_cast<size_t>(seq0 + gr / REP) * Hq + h * REP + gr % REP) * HD) +
                 ch);
    *reinterpret_cast<uint4 *>(q_s + r * (HD * 2) + ((ch ^ (r & 7)) << 4)) = v;
  }
  __syncthreads();

  float o_acc[MT][HD / 8][4];
  float m_run[MT][2], l_run[MT][2];
#pragma unroll
  for (int t = 0; t < MT; ++t) {
#pragma unroll
    for (int i = 0; i < HD / 8; ++i) o_acc[t][i][0] = o_acc[t][i][1] = o_acc[t][i][2] = o_acc[t][i][3] = 0.f;
    m_run[t][0] = m_run[t][1] = -INFINITY;
    l_run[t][0] = l_run[t][1] = 0.f;
  }
  const uint32_t q_addr = smem_u32(q_s);

  bool ok = true;
  for (int k = 0; k < n_my; ++k) {
    ok = mbar_wait(&my_bars[k % kDecStages], (k / kDecStages) & 1, abort_flag);
    if (!ok) break;
    const uint32_t st = smem_u32(my_stages + (k % kDecStages) * S::kStageBytes);
    // ---- S = Q K^T : MT x (16 rows x 16 keys); all keys of a full prompt page are valid ---------
    float sc[MT][2][4];
#pragma unroll
    for (int t = 0; t < MT; ++t)
#pragma unroll
      for (int i = 0; i < 2; ++i) sc[t][i][0] = sc[t][i][1] = sc[t][i][2] = sc[t][i][3] = 0.f;
    {
      const int id = lane >> 3, rr = lane & 7;
      const int key = (id >> 1) * 8 + rr;
      const int q_row = rr + 8 * (id & 1);   // ldmatrix source row of this lane within a 16-row tile
#pragma unroll
      for (int kk = 0; kk < KSTEPS; ++kk) {
        const int c = 2 * (kk & 3) + (id & 1);
        const uint32_t addr = st + (kk >> 2) * (S::kStageBytes / HALVES) + key * 128 + ((c ^ (key & 7)) << 4);
        uint32_t b0, b1, b2, b3;
        ldmatrix_x4(addr, b0, b1, b2, b3);
#pragma unroll
        for (int t = 0; t < MT; ++t) {
          uint32_t a[4];
          const int qc = 2 * kk + (id >> 1);
          ldmatrix_x4(q_addr + (t * 16 + q_row) * (HD * 2) + ((qc ^ (q_row & 7)) << 4), a[0], a[1], a[2], a[3]);
          mma_16816<HALF>(sc[t][0], a, b0, b1);
          mma_16816<HALF>(sc[t][1], a, b2, b3);
        }
      }
    }
    // ---- online softmax (exp2 domain) ---------------------------------------------------------
    uint32_t pa[MT][4];
#pragma unroll
    for (int t = 0; t < MT; ++t) {
      float mx[2] = {-INFINITY, -INFINITY};
#pragma unroll
      for (int nt = 0; nt < 2; ++nt)
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          sc[t][nt][e] *= scale_log2;
          mx[e >> 1] = fmaxf(mx[e >> 1], sc[t][nt][e]);
        }
      float corr[2];
#pragma unroll
      for (int r = 0; r < 2; ++r) {
        mx[r] = fmaxf(mx[r], __shfl_xor_sync(0xffffffffu, mx[r], 1));
        mx[r] = fmaxf(mx[r], __shfl_xor_sync(0xffffffffu, mx[r], 2));
        const float m_new = fmaxf(m_run[t][r], mx[r]);           // finite: every key is valid
        corr[r] = exp2f(m_run[t][r] - m_new);                    // 0 when nothing was accumulated yet
        m_run[t][r] = m_new;
      }
      float ps[2] = {0.f, 0.f};
#pragma unroll
      for (int nt = 0; nt < 2; ++nt)
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          sc[t][nt][e] = exp2f(sc[t][nt][e] - m_run[t][e >> 1]);
          ps[e >> 1] += sc[t][nt][e];
        }
      l_run[t][0] = l_run[t][0] * corr[0] + ps[0];
      l_run[t][1] = l_run[t][1] * corr[1] + ps[1];
#pragma unroll
      for (int i = 0; i < HD / 8; ++i) {
        o_acc[t][i][0] *= corr[0]; o_acc[t][i][1] *= corr[0];
        o_acc[t][i][2] *= corr[1]; o_acc[t][i][3] *= corr[1];
      }
      pa[t][0] = pack_16<HALF>(sc[t][0][0], sc[t][0][1]);
      pa[t][1] = pack_16<HALF>(sc[t][0][2], sc[t][0][3]);
      pa[t][2] = pack_16<HALF>(sc[t][1][0], sc[t][1][1]);
      pa[t][3] = pack_16<HALF>(sc[t][1][2], sc[t][1][3]);
    }
    // ---- O += P V ---------------------------------------------------------------------------
    {
      const int id = lane >> 3, rr = lane & 7;
      const int key = (id & 1) * 8 + rr;
#pragma unroll
      for (int dt = 0; dt < KSTEPS; ++dt) {
        const int c = 2 * (dt & 3) + (id >> 1);
        const uint32_t addr = st + (dt >> 2) * (S::kStageBytes / HALVES) + kPageTokens * 128 + key * 128 +
                              ((c ^ (key & 7)) << 4);
        uint32_t v0, v1, v2, v3;
        ldmatrix_x4_trans(addr, v0, v1, v2, v3);
#pragma unroll
        for (int t = 0; t < MT; ++t) {
          mma_16816<HALF>(o_acc[t][2 * dt], pa[t], v0, v1);
          mma_16816<HALF>(o_acc[t][2 * dt + 1], pa[t], v2, v3);
        }
      }
    }
    __syncwarp();
    if (k + kDecStages < n_my) issue(k + kDecStages);
  }
  if (!ok) {
    // give copies already in flight a chance to land before shared memory is reused or released
    for (int k = 0; k < n_my; ++k) mbar_drain(&my_bars[k % kDecStages], (k / kDecStages) & 1);
  }
#pragma unroll
  for (int t = 0; t < MT; ++t)
#pragma unroll
    for (int r = 0; r < 2; ++r) {
      l_run[t][r] += __shfl_xor_sync(0xffffffffu, l_run[t][r], 1);
      l_run[t][r] += __shfl_xor_sync(0xffffffffu, l_run[t][r], 2);
    }

  // ---- combine the four warps through shared memory (pipeline and query buffers are free now) --
  __syncthreads();
  constexpr int ROWS = MT * 16;
  float *m_s = reinterpret_cast<float *>(smem);                      // [warp][ROWS]
  float *l_s = m_s + kDecWarps * ROWS;
  float *o_s = l_s + kDecWarps * ROWS;                               // [warp][ROWS][HD]
#pragma unroll
  for (int t = 0; t < MT; ++t) {
    const int r_lo = t * 16 + quad, r_hi = r_lo + 8;
    if (qi == 0) {
      m_s[warp * ROWS + r_lo] = m_run[t][0];
      m_s[warp * ROWS + r_hi] = m_run[t][1];
      l_s[warp * ROWS + r_lo] = l_run[t][0];
      l_s[warp * ROWS + r_hi] = l_run[t][1];
    }
#pragma unroll
    for (int i = 0; i < HD / 8; ++i) {
      *reinterpret_cast<float2 *>(o_s + (warp * ROWS + r_lo) * S::kRowStride + 8 * i + 2 * qi) =
          make_float2(o_acc[t][i][0], o_acc[t][i][1]);
      *reinterpret_cast<float2 *>(o_s + (warp * ROWS + r_hi) * S::kRowStride + 8 * i + 2 * qi) =
          make_float2(o_acc[t][i][2], o_acc[t][i][3]);
    }
  }
  __syncthreads();
  for (int idx = threadIdx.x; idx < n_rows * HD; idx += blockDim.x) {
    const int r = idx / HD, d = idx % HD;
    float M = -INFINITY;
#pragma unroll
    for (int w = 0; w < kDecWarps; ++w) M = fmaxf(M, m_s[w * ROWS + r]);
    float L = 0.f, O = 0.f;
#pragma unroll
    for (int w = 0; w < kDecWarps; ++w) {
      const float mw = m_s[w * ROWS + r];
      if (mw != -INFINITY) {
        const float c = exp2f(mw - M);
        L += l_s[w * ROWS + r] * c;
        O += o_s[(w * ROWS + r) * S::kRowStride + d] * c;
      }
    }
    const size_t rh = static_cast<size_t>(seq0 + (row0 + r) / REP) * Hq + h * REP + (row0 + r) % REP;
    pre_o[rh * HD + d] = O;
    if (d == 0) pre_ml[rh] = make_float2(M, L);
  }
  if (threadIdx.x == 0 && *abort_flag) atomicExch(status, STATUS_WAIT_TIMEOUT);
}

// ---------------------------------------------------------------------------------------------
// Prompt prefill on the same tile loop: causal attention of a chunk of prompt tokens over the paged
// cache, whose K/V rows (this chunk's included) were appended before the launch.  A CTA takes
// 32 / REP consecutive rows of the chunk and one kv head, i.e. two 16-row MMA tiles of query rows
// (token-major, REP heads per token), and walks the pages of keys 0..pos like the prefix kernel; a
// query row attends keys up to its own position, so the tiles on the diagonal are masked per row.
// A chunk concatenates prompts: where the CTA's rows straddle two prompts it makes one pass per
// prompt, with the other prompt's rows masked off.
// ---------------------------------------------------------------------------------------------
template <int HD, bool HALF>
__global__ void __launch_bounds__(kDecWarps * 32)
attn_prefill_kernel(const __grid_constant__ CUtensorMap tmKV, const __nv_bfloat16 *__restrict__ q,
                    __nv_bfloat16 *__restrict__ out, const int32_t *__restrict__ row_pt,
                    const int32_t *__restrict__ row_pos, const int32_t *__restrict__ page_table, int pt_width,
                    int R, int layer_row0, int Hq, int Hkv, int n_pages, float scale_log2, int *status) {
  constexpr int MT = 2;
  using S = PreSmem<HD, MT>;
  constexpr int KSTEPS = HD / 16;
  constexpr int HALVES = HD / 64;
  constexpr int CHUNKS = HD / 8;             // 16-byte chunks per query row
  constexpr int ROWS = MT * 16;
  extern __shared__ uint8_t smem_raw[];
  uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t *q_s = smem + S::kPipeBytes;
  uint64_t *bars = reinterpret_cast<uint64_t *>(smem + S::kBody);              // [warp][stage]
  volatile int *abort_flag = reinterpret_cast<volatile int *>(bars + kDecWarps * kDecStages);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int REP = Hq / Hkv;
  const int TPC = ROWS / REP;                // tokens per CTA
  const int quad = lane >> 2, qi = lane & 3;
  const int h = blockIdx.x % Hkv;
  const int t0 = (blockIdx.x / Hkv) * TPC;   // first chunk row of this CTA
  const int n_tok = R - t0 < TPC ? R - t0 : TPC;

  early_start_sync();

  if (threadIdx.x == 0) {
    for (int i = 0; i < kDecWarps * kDecStages; ++i) mbar_init(&bars[i], 1);
    *abort_flag = 0;
    mbar_fence_init();
  }
  __syncthreads();

  uint8_t *my_stages = smem + warp * kDecStages * S::kStageBytes;
  uint64_t *my_bars = bars + warp * kDecStages;
  uint32_t g_iss = 0, g_cons = 0;            // pages requested / consumed by this warp since the start
  const uint32_t q_addr = smem_u32(q_s);
  bool ok = true;

  for (int seg_beg = 0; seg_beg < n_tok && ok;) {
    // ---- the rows of one prompt: [seg_beg, seg_end) ------------------------------------------
    const int pt_row = row_pt[t0 + seg_beg];
    int seg_end = seg_beg + 1;
    while (seg_end < n_tok && row_pt[t0 + seg_end] == pt_row) ++seg_end;
    const int pos_max = row_pos[t0 + seg_end - 1];       // positions rise by one per row within a prompt
    const int n_tiles = pos_max / kPageTokens + 1;
    const int n_my = n_tiles > warp ? (n_tiles - warp + kDecWarps - 1) / kDecWarps : 0;
    const int32_t *pt = page_table + static_cast<size_t>(pt_row) * pt_width;
    // keys visible to MMA rows quad and quad + 8 of tile t (0: the row is not part of this pass)
    int lim[MT][2];
#pragma unroll
    for (int t = 0; t < MT; ++t)
#pragma unroll
      for (int hh = 0; hh < 2; ++hh) {
        const int tok = (t * 16 + quad + 8 * hh) / REP;
        lim[t][hh] = (tok >= seg_beg && tok < seg_end) ? row_pos[t0 + tok] + 1 : 0;
      }

    int pg_cache = 0, pg_base = -1;
    auto page_of = [&](int k) -> int {       // warp-uniform k
      if (pg_base < 0 || k >= pg_base + 32) {
        pg_base = k;
        const int kk = k + lane;
        pg_cache = kk < n_my ? pt[warp + kDecWarps * kk] : 0;
      }
      return __shfl_sync(0xffffffffu, pg_cache, k - pg_base);
    };
    auto issue = [&](int k) {
      const int page = page_of(k);
      if (lane == 0) {
        uint64_t *bar = &my_bars[g_iss % kDecStages];
        uint8_t *dst = my_stages + (g_iss % kDecStages) * S::kStageBytes;
        if (page < 0 || page >= n_pages) {
          atomicExch(status, STATUS_BAD_PAGE);
          mbar_arrive(bar);                  // nothing to load: complete the phase by hand
        } else {
          const int row = layer_row0 + (page * Hkv + h) * 2 * kPageTokens;
          mbar_expect_tx(bar, S::kStageBytes);
#pragma unroll
          for (int hf = 0; hf < HALVES; ++hf)
            tma_load_2d(&tmKV, bar, dst + hf * (S::kStageBytes / HALVES), hf * 64, row);
        }
      }
      ++g_iss;
    };
    const int n_pro = n_my < kDecStages ? n_my : kDecStages;
    for (int k = 0; k < n_pro; ++k) issue(k);

    // ---- queries -> shared memory: row r = (chunk row t0 + r / REP, head h * REP + r % REP) -----
    for (int c = threadIdx.x; c < ROWS * CHUNKS; c += kDecWarps * 32) {
      const int r = c / CHUNKS, ch = c % CHUNKS;
      const int tok = r / REP;
      uint4 v = make_uint4(0u, 0u, 0u, 0u);
      if (tok < n_tok)
        v = *(reinterpret_cast<const uint4 *>(q + (static_cast<size_t>(t0 + tok) * Hq + h * REP + r % REP) * HD) + ch);
      *reinterpret_cast<uint4 *>(q_s + r * (HD * 2) + ((ch ^ (r & 7)) << 4)) = v;
    }
    __syncthreads();

    float o_acc[MT][HD / 8][4];
    float m_run[MT][2], l_run[MT][2];
#pragma unroll
    for (int t = 0; t < MT; ++t) {
#pragma unroll
      for (int i = 0; i < HD / 8; ++i) o_acc[t][i][0] = o_acc[t][i][1] = o_acc[t][i][2] = o_acc[t][i][3] = 0.f;
      m_run[t][0] = m_run[t][1] = -INFINITY;
      l_run[t][0] = l_run[t][1] = 0.f;
    }

    for (int k = 0; k < n_my; ++k) {
      ok = mbar_wait(&my_bars[g_cons % kDecStages], (g_cons / kDecStages) & 1, abort_flag);
      if (!ok) break;
      const uint32_t st = smem_u32(my_stages + (g_cons % kDecStages) * S::kStageBytes);
      ++g_cons;
      const int key0 = (warp + kDecWarps * k) * kPageTokens;
      // ---- S = Q K^T ------------------------------------------------------------------------------
      float sc[MT][2][4];
#pragma unroll
      for (int t = 0; t < MT; ++t)
#pragma unroll
        for (int i = 0; i < 2; ++i) sc[t][i][0] = sc[t][i][1] = sc[t][i][2] = sc[t][i][3] = 0.f;
      {
        const int id = lane >> 3, rr = lane & 7;
        const int key = (id >> 1) * 8 + rr;
        const int q_row = rr + 8 * (id & 1);
#pragma unroll
        for (int kk = 0; kk < KSTEPS; ++kk) {
          const int c = 2 * (kk & 3) + (id & 1);
          const uint32_t addr = st + (kk >> 2) * (S::kStageBytes / HALVES) + key * 128 + ((c ^ (key & 7)) << 4);
          uint32_t b0, b1, b2, b3;
          ldmatrix_x4(addr, b0, b1, b2, b3);
#pragma unroll
          for (int t = 0; t < MT; ++t) {
            uint32_t a[4];
            const int qc = 2 * kk + (id >> 1);
            ldmatrix_x4(q_addr + (t * 16 + q_row) * (HD * 2) + ((qc ^ (q_row & 7)) << 4), a[0], a[1], a[2], a[3]);
            mma_16816<HALF>(sc[t][0], a, b0, b1);
            mma_16816<HALF>(sc[t][1], a, b2, b3);
          }
        }
      }
      // ---- online softmax (exp2 domain), keys beyond a row's own position masked -------------------
      uint32_t pa[MT][4];
#pragma unroll
      for (int t = 0; t < MT; ++t) {
        float mx[2] = {-INFINITY, -INFINITY};
#pragma unroll
        for (int nt = 0; nt < 2; ++nt)
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            const int key = key0 + 8 * nt + 2 * qi + (e & 1);
            const float v = key < lim[t][e >> 1] ? sc[t][nt][e] * scale_log2 : -INFINITY;
            sc[t][nt][e] = v;
            mx[e >> 1] = fmaxf(mx[e >> 1], v);
          }
        float corr[2], msafe[2];
#pragma unroll
        for (int r = 0; r < 2; ++r) {
          mx[r] = fmaxf(mx[r], __shfl_xor_sync(0xffffffffu, mx[r], 1));
          mx[r] = fmaxf(mx[r], __shfl_xor_sync(0xffffffffu, mx[r], 2));
          const float m_new = fmaxf(m_run[t][r], mx[r]);
          msafe[r] = m_new == -INFINITY ? 0.f : m_new;
          corr[r] = exp2f(m_run[t][r] - msafe[r]);         // 0 when nothing was accumulated yet
          m_run[t][r] = m_new;
        }
        float ps[2] = {0.f, 0.f};
#pragma unroll
        for (int nt = 0; nt < 2; ++nt)
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            sc[t][nt][e] = exp2f(sc[t][nt][e] - msafe[e >> 1]);
            ps[e >> 1] += sc[t][nt][e];
          }
        l_run[t][0] = l_run[t][0] * corr[0] + ps[0];
        l_run[t][1] = l_run[t][1] * corr[1] + ps[1];
#pragma unroll
        for (int i = 0; i < HD / 8; ++i) {
          o_acc[t][i][0] *= corr[0]; o_acc[t][i][1] *= corr[0];
          o_acc[t][i][2] *= corr[1]; o_acc[t][i][3] *= corr[1];
        }
        pa[t][0] = pack_16<HALF>(sc[t][0][0], sc[t][0][1]);
        pa[t][1] = pack_16<HALF>(sc[t][0][2], sc[t][0][3]);
        pa[t][2] = pack_16<HALF>(sc[t][1][0], sc[t][1][1]);
        pa[t][3] = pack_16<HALF>(sc[t][1][2], sc[t][1][3]);
      }
      // ---- O += P V -------------------------------------------------------------------------------
      {
        const int id = lane >> 3, rr = lane & 7;
        const int key = (id & 1) * 8 + rr;
#pragma unroll
        for (int dt = 0; dt < KSTEPS; ++dt) {
          const int c = 2 * (dt & 3) + (id >> 1);
          const uint32_t addr = st + (dt >> 2) * (S::kStageBytes / HALVES) + kPageTokens * 128 + key * 128 +
                                ((c ^ (key & 7)) << 4);
          uint32_t v0, v1, v2, v3;
          ldmatrix_x4_trans(addr, v0, v1, v2, v3);
#pragma unroll
          for (int t = 0; t < MT; ++t) {
            mma_16816<HALF>(o_acc[t][2 * dt], pa[t], v0, v1);
            mma_16816<HALF>(o_acc[t][2 * dt + 1], pa[t], v2, v3);
          }
        }
      }
      __syncwarp();
      if (k + kDecStages < n_my) issue(k + kDecStages);
    }
    if (!ok) break;
#pragma unroll
    for (int t = 0; t < MT; ++t)
#pragma unroll
      for (int r = 0; r < 2; ++r) {
        l_run[t][r] += __shfl_xor_sync(0xffffffffu, l_run[t][r], 1);
        l_run[t][r] += __shfl_xor_sync(0xffffffffu, l_run[t][r], 2);
      }
    // ---- combine the four warps through shared memory (pipeline and query buffers are idle now) --
    __syncthreads();
    float *m_s = reinterpret_cast<float *>(smem);                      // [warp][ROWS]
    float *l_s = m_s + kDecWarps * ROWS;
    float *o_s = l_s + kDecWarps * ROWS;                               // [warp][ROWS][kRowStride]
#pragma unroll
    for (int t = 0; t < MT; ++t) {
      const int r_lo = t * 16 + quad, r_hi = r_lo + 8;
      if (qi == 0) {
        m_s[warp * ROWS + r_lo] = m_run[t][0];
        m_s[warp * ROWS + r_hi] = m_run[t][1];
        l_s[warp * ROWS + r_lo] = l_run[t][0];
        l_s[warp * ROWS + r_hi] = l_run[t][1];
      }
#pragma unroll
      for (int i = 0; i < HD / 8; ++i) {
        *reinterpret_cast<float2 *>(o_s + (warp * ROWS + r_lo) * S::kRowStride + 8 * i + 2 * qi) =
            make_float2(o_acc[t][i][0], o_acc[t][i][1]);
        *reinterpret_cast<float2 *>(o_s + (warp * ROWS + r_hi) * S::kRowStride + 8 * i + 2 * qi) =
            make_float2(o_acc[t][i][2], o_acc[t][i][3]);
      }
    }
    __syncthreads();
    for (int idx = threadIdx.x; idx < ROWS * HD; idx += blockDim.x) {
      const int r = idx / HD, d = idx % HD;
      const int tok = r / REP;
      if (tok < seg_beg || tok >= seg_end) continue;
      float M = -INFINITY;
#pragma unroll
      for (int w = 0; w < kDecWarps; ++w) M = fmaxf(M, m_s[w * ROWS + r]);
      float L = 0.f, O = 0.f;
#pragma unroll
      for (int w = 0; w < kDecWarps; ++w) {
        const float mw = m_s[w * ROWS + r];
        if (mw != -INFINITY) {
          const float c = exp2f(mw - M);
          L += l_s[w * ROWS + r] * c;
          O += o_s[(w * ROWS + r) * S::kRowStride + d] * c;
        }
      }
      reinterpret_cast<uint16_t *>(out)[(static_cast<size_t>(t0 + tok) * Hq + h * REP + r % REP) * HD + d] =
          cvt16(O / L, HALF);
    }
    seg_beg = seg_end;
    if (seg_beg < n_tok) {
      // another prompt's rows follow: the merge area is handed back to the copy engine
      __syncthreads();
      fence_proxy_async();
    }
  }
  if (*abort_flag) {
    for (uint32_t g = g_cons; g < g_iss; ++g) mbar_drain(&my_bars[g % kDecStages], (g / kDecStages) & 1);
    if (threadIdx.x == 0) atomicExch(status, STATUS_WAIT_TIMEOUT);
  }
}

template <int HD, bool HALF>
cudaError_t launch_prefill(const PrefillAttnArgs &a, cudaStream_t s) {
  const int REP = a.Hq / a.Hkv;
  const int TPC = 32 / REP;
  const float scale_log2 = 1.4426950408889634f / sqrtf(static_cast<float>(HD));
  return launch_early(attn_prefill_kernel<HD, HALF>, dim3(((a.R + TPC - 1) / TPC) * a.Hkv), dim3(kDecWarps * 32),
                      PreSmem<HD, 2>::kTotal, s, *a.tmKV, a.q, a.out, a.row_pt, a.row_pos, a.page_table, a.pt_width,
                      a.R, a.layer_row0, a.Hq, a.Hkv, a.n_pages, scale_log2, a.status);
}

// CTAs of the resident suffix kernel that fit the current device at once (cached per device, head
// dimension, operand format and group ratio; no stream work).
template <int HD, bool HALF>
int resident_slots(int smem_bytes, int rep) {
  static int cache[64][17] = {};             // one table per (HD, HALF) instantiation
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64 || rep < 1 || rep > 16) return 0;
  if (cache[dev][rep] == 0) {
    int sms = 0, per_sm = 0;
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return 0;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, attn_suffix_resident_kernel<HD, HALF>, kDecWarps * 32,
                                                      smem_bytes) != cudaSuccess)
      return 0;
    cache[dev][rep] = sms * per_sm;
  }
  return cache[dev][rep];
}

template <int HD, bool HALF>
cudaError_t launch_decode(const DecodeAttnArgs &a, cudaStream_t s) {
  using S = DecSmem<HD>;
  const int REP = a.Hq / a.Hkv;
  const int MT = (a.G * REP + 15) / 16;
  const float scale_log2 = 1.4426950408889634f / sqrtf(static_cast<float>(HD));
  cudaError_t e;
  if (MT >= 2 && a.prefix_impl != 1) {
    // two 16-row tiles of a group's query rows per CTA: half the CTAs, and at 32 rows per group the
    // launch fits the GPU at once
    e = launch_early(attn_prefix_group_kernel<HD, 2, HALF>, dim3(a.P * a.Hkv * ((MT + 1) / 2)), dim3(kDecWarps * 32),
                     PreSmem<HD, 2>::kTotal, s,
                     *a.tmKV, a.q, a.pre_o, a.pre_ml, a.page_table, a.pt_width, a.full_pages, a.layer_row0, a.Hq,
                     a.Hkv, a.G, a.n_pages, scale_log2, a.status, a.row_done);
  } else {
    e = launch_early(attn_decode_kernel<HD, true, HALF>, dim3(a.P * a.Hkv * MT), dim3(kDecWarps * 32), S::kTotal, s,
                     *a.tmKV, a.q, a.out, a.pre_o, a.pre_ml, a.page_table, a.pt_width, a.row_pos, a.full_pages,
                     a.layer_row0, a.Hq, a.Hkv, a.G, a.n_pages, scale_log2, a.row_done, a.status, a.out_row);
  }
  if (e != cudaSuccess) return e;
  if (a.suffix_impl != 1 && a.work && REP * HD <= 512) {   // merge area small enough for three CTAs per SM
    using R = SufSmem<HD>;
    const int n_items = a.P * a.G * a.Hkv;
    const int slots = resident_slots<HD, HALF>(R::total(REP), REP);
    if (slots <= 0) return cudaErrorInvalidConfiguration;
    return launch_early(attn_suffix_resident_kernel<HD, HALF>, dim3(n_items < slots ? n_items : slots),
                        dim3(kDecWarps * 32), R::total(REP), s, *a.tmKV, a.q, a.out, a.pre_o, a.pre_ml, a.page_table,
                        a.pt_width, a.row_pos, a.full_pages, a.layer_row0, a.Hq, a.Hkv, n_items, a.n_pages, scale_log2,
                        a.row_done, a.status, a.work, a.out_row);
  }
  return launch_early(attn_decode_kernel<HD, false, HALF>, dim3(a.P * a.G * a.Hkv), dim3(kDecWarps * 32), S::kTotal, s,
                      *a.tmKV, a.q, a.out, a.pre_o, a.pre_ml, a.page_table, a.pt_width, a.row_pos, a.full_pages,
                      a.layer_row0, a.Hq, a.Hkv, a.G, a.n_pages, scale_log2, a.row_done, a.status, a.out_row);
}

template <int HD, bool HALF>
cudaError_t configure_decode() {
  cudaError_t e;
  if ((e = cudaFuncSetAttribute(attn_decode_kernel<HD, true, HALF>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                DecSmem<HD>::kTotal)) != cudaSuccess) return e;
  if ((e = cudaFuncSetAttribute(attn_decode_kernel<HD, false, HALF>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                DecSmem<HD>::kTotal)) != cudaSuccess) return e;
  if ((e = cudaFuncSetAttribute(attn_prefix_group_kernel<HD, 2, HALF>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                PreSmem<HD, 2>::kTotal)) != cudaSuccess) return e;
  if ((e = cudaFuncSetAttribute(attn_prefill_kernel<HD, HALF>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                PreSmem<HD, 2>::kTotal)) != cudaSuccess) return e;
  return cudaFuncSetAttribute(attn_suffix_resident_kernel<HD, HALF>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                              SufSmem<HD>::total(kSufPre * kDecWarps * 32 / HD));
}

}  // namespace

cudaError_t attention_decode_configure() {
  cudaError_t e;
  if ((e = configure_decode<128, false>()) != cudaSuccess) return e;
  if ((e = configure_decode<128, true>()) != cudaSuccess) return e;
  if ((e = configure_decode<64, false>()) != cudaSuccess) return e;
  return configure_decode<64, true>();
}

bool attention_decode_supported(int hd, int page_size, int Hq, int Hkv) {
  const int rep = Hq / Hkv;
  return (hd == 64 || hd == 128) && page_size == kPageTokens && rep >= 1 && rep <= 16;
}

cudaError_t attention_prefill_launch(const PrefillAttnArgs &a, cudaStream_t s) {
  const int rep = a.Hkv > 0 ? a.Hq / a.Hkv : 0;
  if (rep != 1 && rep != 2 && rep != 4 && rep != 8) return cudaErrorInvalidValue;
  if (a.hd == 128) return a.half_io ? launch_prefill<128, true>(a, s) : launch_prefill<128, false>(a, s);
  if (a.hd == 64) return a.half_io ? launch_prefill<64, true>(a, s) : launch_prefill<64, false>(a, s);
  return cudaErrorInvalidValue;
}

cudaError_t attention_decode_launch(const DecodeAttnArgs &a, cudaStream_t s) {
  if (a.hd == 128) return a.half_io ? launch_decode<128, true>(a, s) : launch_decode<128, false>(a, s);
  if (a.hd == 64) return a.half_io ? launch_decode<64, true>(a, s) : launch_decode<64, false>(a, s);
  return cudaErrorInvalidValue;
}

}  // namespace echo

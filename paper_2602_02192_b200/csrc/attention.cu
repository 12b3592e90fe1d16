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

namespace echo {

namespace {

constexpr int kAttnWarps = 4;
constexpr int kMaxRep = 8;        // query heads per kv head

template <int HD, int REP>
__global__ void __launch_bounds__(kAttnWarps * 32)
attention_rows_kernel(const __nv_bfloat16 *q, const __nv_bfloat16 *kv_layer, __nv_bfloat16 *out,
                      const int32_t *row_pt, const int32_t *row_pos, const int32_t *page_table, int pt_width,
                      int Hq, int Hkv, int page_size, int n_pages, float scale, int *status) {
  constexpr int EPL = HD / 32;                       // output dims per lane
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
    q_s[a][d] = __bfloat162float(q[(static_cast<size_t>(r) * Hq + kvh * REP + a) * HD + d]) * scale;
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
          const __nv_bfloat162 *k2 = reinterpret_cast<const __nv_bfloat162 *>(&raw);
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            const float2 kf = __bfloat1622float2(k2[i]);
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
        const __nv_bfloat162 *v2 = reinterpret_cast<const __nv_bfloat162 *>(&raw);
        const float2 a0 = __bfloat1622float2(v2[0]), a1 = __bfloat1622float2(v2[1]);
        vf[0] = a0.x; vf[1] = a0.y; vf[2 % EPL] = a1.x; vf[3 % EPL] = a1.y;
      } else {
        const __nv_bfloat162 v2 = *reinterpret_cast<const __nv_bfloat162 *>(vr);
        const float2 a0 = __bfloat1622float2(v2);
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
    out[(static_cast<size_t>(r) * Hq + kvh * REP + a) * HD + d] = __float2bfloat16(acc / ll);
  }
}

template <int HD, int REP>
cudaError_t launch_rows(const __nv_bfloat16 *q, const __nv_bfloat16 *kv_layer, __nv_bfloat16 *out, RowMeta meta,
                        const int32_t *page_table, int pt_width, int R, int Hq, int Hkv, int page_size, int n_pages,
                        int *status, cudaStream_t s) {
  const float scale = 1.0f / sqrtf(static_cast<float>(HD));
  attention_rows_kernel<HD, REP><<<dim3(R, Hkv), kAttnWarps * 32, 0, s>>>(
      q, kv_layer, out, meta.row_pt, meta.row_pos, page_table, pt_width, Hq, Hkv, page_size, n_pages, scale, status);
  return cudaGetLastError();
}

}  // namespace

cudaError_t attention_rows_launch(const __nv_bfloat16 *q, const __nv_bfloat16 *kv_layer, __nv_bfloat16 *out,
                                  RowMeta meta, const int32_t *page_table, int pt_width, int R, int Hq, int Hkv,
                                  int hd, int page_size, int n_pages, int *status, cudaStream_t s) {
  const int rep = Hq / Hkv;
#define ECHO_ATTN_CASE(HD_, REP_)                                                                              \
  if (hd == HD_ && rep == REP_)                                                                                \
    return launch_rows<HD_, REP_>(q, kv_layer, out, meta, page_table, pt_width, R, Hq, Hkv, page_size, n_pages, \
                                  status, s);
  ECHO_ATTN_CASE(64, 1) ECHO_ATTN_CASE(64, 2) ECHO_ATTN_CASE(64, 4)
  ECHO_ATTN_CASE(128, 1) ECHO_ATTN_CASE(128, 2) ECHO_ATTN_CASE(128, 4) ECHO_ATTN_CASE(128, 8)
#undef ECHO_ATTN_CASE
  return cudaErrorInvalidValue;
}

}  // namespace echo

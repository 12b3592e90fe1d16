// Row-wise kernels of the rollout path: embedding gather, RMSNorm, RoPE + paged-KV
// append, SwiGLU, the Philox / Gumbel-max sampler with its log-probability, GRPO's
// group advantage, and the small bookkeeping kernels a decode step needs.

#include "common.cuh"
#include "ptx.cuh"

namespace echo {

bool g_early_start = true;

namespace {

// ---------------------------------------------------------------------------
// Philox4x32-10 (Salmon et al., SC'11), restated from its published definition.
// ---------------------------------------------------------------------------
__device__ __forceinline__ uint4 philox4x32_10(uint4 c, uint2 k) {
#pragma unroll
  for (int r = 0; r < 10; ++r) {
    const uint32_t hi0 = __umulhi(0xD2511F53u, c.x), lo0 = 0xD2511F53u * c.x;
    const uint32_t hi1 = __umulhi(0xCD9E8D57u, c.z), lo1 = 0xCD9E8D57u * c.z;
    c = make_uint4(hi1 ^ c.y ^ k.x, lo1, hi0 ^ c.w ^ k.y, lo0);
    k.x += 0x9E3779B9u;
    k.y += 0xBB67AE85u;
  }
  return c;
}
// w = (float(word) + 0.5f) * 2^-32 in IEEE fp32, each operation rounded on its own.
__device__ __forceinline__ float uniform_from_word(uint32_t x) {
  return __fmul_rn(__fadd_rn(__uint2float_rn(x), 0.5f), 2.3283064365386963e-10f);
}
// g = -log(-log1p(-w)); w == 1 gives -inf.
__device__ __forceinline__ float gumbel_from_uniform(float w) { return -logf(-log1pf(-w)); }

// ---------------------------------------------------------------------------
__global__ void embed_kernel(const __nv_bfloat16 *embed, const int32_t *tok_src, const int32_t *tok_idx, float *x,
                             int R, int d, int vocab, int *status) {
  early_start_sync();
  const int r = blockIdx.x;
  if (r >= R) return;
  int tok = tok_src[tok_idx ? tok_idx[r] : r];
  if (tok < 0 || tok >= vocab) {
    if (threadIdx.x == 0) atomicExch(status, STATUS_BAD_TOKEN);
    tok = 0;
  }
  const __nv_bfloat162 *src = reinterpret_cast<const __nv_bfloat162 *>(embed + static_cast<size_t>(tok) * d);
  float2 *dst = reinterpret_cast<float2 *>(x + static_cast<size_t>(r) * d);
  for (int i = threadIdx.x; i < d / 2; i += blockDim.x) dst[i] = __bfloat1622float2(src[i]);
}

__device__ __forceinline__ float block_sum(float v, float *scratch) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, nw = blockDim.x >> 5;
  if (lane == 0) scratch[warp] = v;
  __syncthreads();
  float t = 0.f;
  for (int i = 0; i < nw; ++i) t += scratch[i];      // same order in every thread: deterministic
  __syncthreads();
  return t;
}

// h = bf16( x * rsqrt(mean(x^2) + eps) * gain ).  One block per row; the row is read once
// (float4 per thread, kept in registers) when d <= 4 * 4 * blockDim.
constexpr int kNormThreads = 256;
constexpr int kNormVecs = 8;          // float4 per thread held in registers (d <= 8192)
__global__ void __launch_bounds__(kNormThreads)
rmsnorm_kernel(const float *__restrict__ x, const __nv_bfloat16 *__restrict__ gain, __nv_bfloat16 *__restrict__ h,
               int R, int d, float eps, int out_half) {
  __shared__ float scratch[32];
  const int r = blockIdx.x;
  const float *xr = x + static_cast<size_t>(r) * d;
  __nv_bfloat16 *hr = h + static_cast<size_t>(r) * d;
  const bool fast = (d % 4 == 0) && d <= 4 * kNormVecs * kNormThreads;
  // the gains are part of the installed snapshot, not of the preceding kernel's output: they are
  // fetched before the dependency wait
  uint2 graw[kNormVecs];
  if (fast) {
#pragma unroll
    for (int i = 0; i < kNormVecs; ++i) {
      const int idx = threadIdx.x + i * kNormThreads;
      graw[i] = idx < d / 4 ? reinterpret_cast<const uint2 *>(gain)[idx] : make_uint2(0u, 0u);
    }
  }
  early_start_sync();       // (also lets the following projection begin its weight prefetch)
  if (fast) {
    const int nv = d / 4;
    float4 v[kNormVecs];
    float ss = 0.f;
#pragma unroll
    for (int i = 0; i < kNormVecs; ++i) {
      const int idx = threadIdx.x + i * kNormThreads;
      v[i] = idx < nv ? reinterpret_cast<const float4 *>(xr)[idx] : make_float4(0.f, 0.f, 0.f, 0.f);
      ss = fmaf(v[i].x, v[i].x, fmaf(v[i].y, v[i].y, fmaf(v[i].z, v[i].z, fmaf(v[i].w, v[i].w, ss))));
    }
    ss = block_sum(ss, scratch);
    const float scale = rsqrtf(ss / static_cast<float>(d) + eps);
#pragma unroll
    for (int i = 0; i < kNormVecs; ++i) {
      const int idx = threadIdx.x + i * kNormThreads;
      if (idx < nv) {
        const float2 g0 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(&graw[i].x));
        const float2 g1 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(&graw[i].y));
        uint2 o;
        o.x = cvt16x2(v[i].x * scale * g0.x, v[i].y * scale * g0.y, out_half != 0);
        o.y = cvt16x2(v[i].z * scale * g1.x, v[i].w * scale * g1.y, out_half != 0);
        reinterpret_cast<uint2 *>(hr)[idx] = o;
      }
    }
    return;
  }
  float ss = 0.f;
  for (int i = threadIdx.x; i < d; i += blockDim.x) {
    const float v = xr[i];
    ss = fmaf(v, v, ss);
  }
  ss = block_sum(ss, scratch);
  const float scale = rsqrtf(ss / static_cast<float>(d) + eps);
  for (int i = threadIdx.x; i < d; i += blockDim.x)
    reinterpret_cast<uint16_t *>(hr)[i] = cvt16(xr[i] * scale * __bfloat162float(gain[i]), out_half != 0);
}

// table[pos][i] = (cos, sin)(pos * theta^(-2i/hd)), angles in fp64
__global__ void rope_table_kernel(float2 *table, int max_pos, int half, double theta, int hd) {
  const int idx = blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= max_pos * half) return;
  const int pos = idx / half, i = idx % half;
  const double ang = static_cast<double>(pos) * pow(theta, -2.0 * i / hd);
  table[idx] = make_float2(static_cast<float>(cos(ang)), static_cast<float>(sin(ang)));
}

// One block per activation row.  Rotates q and k heads (pairs (i, i + hd/2)), writes q as
// bf16 and k, v as bf16 into the row's page slot.
__global__ void rope_append_kernel(float *__restrict__ qkv, __nv_bfloat16 *__restrict__ q,
                                   __nv_bfloat16 *__restrict__ kv_layer, const float2 *__restrict__ rope_table,
                                   const int32_t *__restrict__ row_pt, const int32_t *__restrict__ row_pos,
                                   const int32_t *__restrict__ row_done, const int32_t *__restrict__ page_table,
                                   int pt_width, int R, int Hq, int Hkv, int hd, int page_size, int n_pages,
                                   int max_pos, int *status, int out_half, const int32_t *q_row) {
  early_start_sync();
  const bool oh = out_half != 0;
  const int r = blockIdx.x;
  // an ended row (or a padding row of a compacted step: no page-table row) is only cleared
  const bool skip = (row_done && row_done[r]) || row_pt[r] < 0;
  const int pos = skip ? -1 : row_pos[r];
  const int qr = (q_row && !skip) ? q_row[r] : r;                   // row of the query buffer this row writes
  const int half = hd / 2;
  const int ld = (Hq + 2 * Hkv) * hd;
  float *src = qkv + static_cast<size_t>(r) * ld;
  if (pos < 0 || pos >= max_pos) {
    if (threadIdx.x == 0 && !skip) atomicExch(status, STATUS_BAD_PAGE);
    for (int i = threadIdx.x; i < ld; i += blockDim.x) src[i] = 0.f;      // keep the buffer's zero invariant
    return;
  }
  const int page = page_table[static_cast<size_t>(row_pt[r]) * pt_width + pos / page_size];
  const int off = pos % page_size;
  if (page < 0 || page >= n_pages) {
    if (threadIdx.x == 0) atomicExch(status, STATUS_BAD_PAGE);
    for (int i = threadIdx.x; i < ld; i += blockDim.x) src[i] = 0.f;
    return;
  }
  const float2 *cs = rope_table + static_cast<size_t>(pos) * half;
  // q heads
#pragma unroll 4
  for (int idx = threadIdx.x; idx < Hq * half; idx += blockDim.x) {
    const int head = idx / half, i = idx % half;
    const float a = src[head * hd + i], b = src[head * hd + i + half];
    const float2 t = cs[i];
    uint16_t *dst = reinterpret_cast<uint16_t *>(q) + static_cast<size_t>(qr) * Hq * hd + head * hd;
    dst[i] = cvt16(a * t.x - b * t.y, oh);
    dst[i + half] = cvt16(b * t.x + a * t.y, oh);
  }
  // k heads (rotated) and v heads (plain) into the page slot
  const size_t page_elems = static_cast<size_t>(page_size) * hd;
#pragma unroll 2
  for (int idx = threadIdx.x; idx < Hkv * half; idx += blockDim.x) {
    const int head = idx / half, i = idx % half;
    float *ks = src + (Hq + head) * hd;
    float *vs = src + (Hq + Hkv + head) * hd;
    const float2 t = cs[i];
    uint16_t *kd = reinterpret_cast<uint16_t *>(kv_layer) +
                   ((static_cast<size_t>(page) * Hkv + head) * 2 + 0) * page_elems + off * hd;
    uint16_t *vd = kd + page_elems;
    const float a = ks[i], b = ks[i + half];
    kd[i] = cvt16(a * t.x - b * t.y, oh);
    kd[i + half] = cvt16(b * t.x + a * t.y, oh);
    vd[i] = cvt16(vs[i], oh);
    vd[i + half] = cvt16(vs[i + half], oh);
  }
  // the row is consumed: leave zeros for the next projection, whose k-slices add into this buffer
  // (a separate pass, so that the loads above are not ordered behind stores to the same array)
  __syncthreads();
  if ((ld & 3) == 0) {
    float4 *z = reinterpret_cast<float4 *>(src);
    for (int i = threadIdx.x; i < ld / 4; i += blockDim.x) z[i] = make_float4(0.f, 0.f, 0.f, 0.f);
  } else {
    for (int i = threadIdx.x; i < ld; i += blockDim.x) src[i] = 0.f;
  }
}

// Vector form of rope_append_kernel for head_dim % 8 == 0: a work item is four consecutive
// rotation pairs of one head (for a kv head: of its key, plus the matching eight values), moved
// with 16-byte loads and 8-byte stores.  Every qkv element is read by exactly one thread, which
// zeroes it right after reading, so no second pass over the row is needed.
__device__ __forceinline__ uint2 pack_16x4(float a, float b, float c, float d, bool half) {
  return make_uint2(cvt16x2(a, b, half), cvt16x2(c, d, half));
}
__global__ void __launch_bounds__(256)
rope_append_vec_kernel(float *__restrict__ qkv, __nv_bfloat16 *__restrict__ q, __nv_bfloat16 *__restrict__ kv_layer,
                       const float2 *__restrict__ rope_table, const int32_t *__restrict__ row_pt,
                       const int32_t *__restrict__ row_pos, const int32_t *__restrict__ row_done,
                       const int32_t *__restrict__ page_table, int pt_width,
                       int R, int Hq, int Hkv, int hd, int page_size, int n_pages, int max_pos, int *status,
                       int out_half, const int32_t *q_row) {
  early_start_sync();
  const bool oh = out_half != 0;
  const int r = blockIdx.x;
  const int half = hd / 2, q4 = half / 4;
  const int ld = (Hq + 2 * Hkv) * hd;
  float *src = qkv + static_cast<size_t>(r) * ld;
  const float4 zero4 = make_float4(0.f, 0.f, 0.f, 0.f);
  const int n_items = (Hq + Hkv) * q4;
  // All loads of the row are issued before anything depends on the row's position, so the
  // position -> page -> rotation-table chain runs under their latency.
  constexpr int kItems = 3;                             // items per thread held in registers
  float4 a[kItems], b[kItems], v0[kItems], v1[kItems];
#pragma unroll
  for (int j = 0; j < kItems; ++j) {
    const int item = threadIdx.x + j * 256;
    if (item < n_items) {
      const int unit = item / q4, i = (item % q4) * 4;
      a[j] = *reinterpret_cast<const float4 *>(src + unit * hd + i);
      b[j] = *reinterpret_cast<const float4 *>(src + unit * hd + i + half);
      if (unit >= Hq) {
        v0[j] = *reinterpret_cast<const float4 *>(src + (unit + Hkv) * hd + i);
        v1[j] = *reinterpret_cast<const float4 *>(src + (unit + Hkv) * hd + i + half);
      }
    }
  }
  // an ended row (or a padding row of a compacted step: no page-table row) is only cleared
  const bool ended = (row_done && row_done[r]) || row_pt[r] < 0;
  const int pos = ended ? -1 : row_pos[r];
  const int qr = (q_row && !ended) ? q_row[r] : r;       // row of the query buffer this row writes
  int page = -1;
  if (pos >= 0 && pos < max_pos) page = page_table[static_cast<size_t>(row_pt[r]) * pt_width + pos / page_size];
  const bool bad = page < 0 || page >= n_pages;
  if (bad && !ended && threadIdx.x == 0) atomicExch(status, STATUS_BAD_PAGE);
  const int off = bad ? 0 : pos % page_size;
  const float4 *cs4 = reinterpret_cast<const float4 *>(rope_table + static_cast<size_t>(bad ? 0 : pos) * half);
  const size_t page_elems = static_cast<size_t>(page_size) * hd;
  for (int j0 = 0; j0 < (n_items + 255) / 256; j0 += kItems) {
#pragma unroll
    for (int j = 0; j < kItems; ++j) {
      const int item = threadIdx.x + (j0 + j) * 256;
      if (item >= n_items) continue;
      const int unit = item / q4, i = (item % q4) * 4;
      float4 *pa = reinterpret_cast<float4 *>(src + unit * hd + i);
      float4 *pb = reinterpret_cast<float4 *>(src + unit * hd + i + half);
      float4 *va = reinterpret_cast<float4 *>(src + (unit + Hkv) * hd + i);
      float4 *vb = reinterpret_cast<float4 *>(src + (unit + Hkv) * hd + i + half);
      if (j0 > 0) {                                     // rows longer than 3 x 256 items: load late
        a[j] = *pa;
        b[j] = *pb;
        if (unit >= Hq) {
          v0[j] = *va;
          v1[j] = *vb;
        }
      }
      // the row is consumed: leave zeros for the next projection, whose k-slices add into it
      *pa = zero4;
      *pb = zero4;
      if (unit >= Hq) {
        *va = zero4;
        *vb = zero4;
      }
      if (bad) continue;
      const float4 t01 = cs4[i / 2], t23 = cs4[i / 2 + 1];       // (cos, sin) of pairs i..i+3
      const float4 x = a[j], y = b[j];
      const uint2 lo = pack_16x4(x.x * t01.x - y.x * t01.y, x.y * t01.z - y.y * t01.w, x.z * t23.x - y.z * t23.y,
                                 x.w * t23.z - y.w * t23.w, oh);
      const uint2 hi = pack_16x4(y.x * t01.x + x.x * t01.y, y.y * t01.z + x.y * t01.w, y.z * t23.x + x.z * t23.y,
                                 y.w * t23.z + x.w * t23.w, oh);
      if (unit < Hq) {
        __nv_bfloat16 *dst = q + static_cast<size_t>(qr) * Hq * hd + unit * hd + i;
        *reinterpret_cast<uint2 *>(dst) = lo;
        *reinterpret_cast<uint2 *>(dst + half) = hi;
      } else {
        const int head = unit - Hq;
        __nv_bfloat16 *kd = kv_layer + ((static_cast<size_t>(page) * Hkv + head) * 2 + 0) * page_elems + off * hd + i;
        *reinterpret_cast<uint2 *>(kd) = lo;
        *reinterpret_cast<uint2 *>(kd + half) = hi;
        __nv_bfloat16 *vd = kd + page_elems;
        *reinterpret_cast<uint2 *>(vd) = pack_16x4(v0[j].x, v0[j].y, v0[j].z, v0[j].w, oh);
        *reinterpret_cast<uint2 *>(vd + half) = pack_16x4(v1[j].x, v1[j].y, v1[j].z, v1[j].w, oh);
      }
    }
  }
}

__global__ void swiglu_kernel(const float *gu, __nv_bfloat16 *act, int R, int F, int out_half) {
  const size_t idx = static_cast<size_t>(blockIdx.x) * blockDim.x + threadIdx.x;
  if (idx >= static_cast<size_t>(R) * F) return;
  const size_t r = idx / F, f = idx % F;
  const float g = gu[r * 2 * F + f], u = gu[r * 2 * F + F + f];
  reinterpret_cast<uint16_t *>(act)[idx] = cvt16(g / (1.0f + __expf(-g)) * u, out_half != 0);
}

__global__ void gather_rows_kernel(const float *x, const int32_t *src_rows, float *dst, int n, int d) {
  const int i = blockIdx.x;
  const int r = src_rows[i];
  if (r < 0) return;
  for (int c = threadIdx.x; c < d; c += blockDim.x) dst[static_cast<size_t>(i) * d + c] = x[static_cast<size_t>(r) * d + c];
}

// Copies whole KV pages (all kv heads, K and V) in every layer: grid (n_copies, n_layers).
__global__ void copy_pages_kernel(__nv_bfloat16 *kv, const int32_t *src_page, const int32_t *dst_page,
                                  size_t layer_stride_elems, int page_elems) {
  const int c = blockIdx.x, l = blockIdx.y;
  const uint4 *src = reinterpret_cast<const uint4 *>(kv + l * layer_stride_elems + static_cast<size_t>(src_page[c]) * page_elems);
  uint4 *dst = reinterpret_cast<uint4 *>(kv + l * layer_stride_elems + static_cast<size_t>(dst_page[c]) * page_elems);
  for (int i = threadIdx.x; i < page_elems / 8; i += blockDim.x) dst[i] = src[i];
}

// Start of decode step j = *d_step + 1: row b feeds the token produced at step j-1 at
// position len0[b] + j - 1.  One block; the counter is bumped after every thread has read it.
//
// With `c` (compaction, used with an end token): the sequences that have not ended are packed to the
// front of the activation rows, in sequence order, so that the step's projections run on the live
// rows only.  row r of the step then belongs to sequence c.row_seq[r] (-1: padding row), sequence b
// sits in row c.seq_row[b] (-1: ended), positions are kept both per row and per sequence, and an
// ended sequence receives its end token / log-probability 0 for this step here.
struct Compaction {
  int32_t *row_seq, *seq_row, *seq_pos, *n_live;
  int32_t *out_tok;
  float *out_lp;
  const int32_t *seq_gid, *seq_t0;      // prompt queue: sequence id and first step of what slot b holds
};
__global__ void __launch_bounds__(512)
decode_prep_kernel(int32_t *d_step, const int32_t *tok_hist, int T, const int32_t *seq_len0, int32_t *row_tok,
                   int32_t *row_pos, int B, int eos_id, int32_t *row_done, Compaction c) {
  __shared__ int warp_sum[16];
  __shared__ int base_s;
  early_start_sync();
  const int j = *d_step + 1;
  if (threadIdx.x == 0) base_s = 0;
  __syncthreads();
  if (!c.row_seq) {
    for (int b = threadIdx.x; b < B; b += blockDim.x) {
      const int32_t tok = tok_hist[static_cast<size_t>(b) * T + (j - 1)];
      row_tok[b] = tok;
      row_pos[b] = seq_len0[b] + j - 1;
      // a sequence that is fed its end token has ended and stays ended whatever the token buffer holds
      // at later positions (a given trajectory may be padded with other ids after its end token); its
      // attention and cache writes are skipped from here on.  The flags are cleared when a rollout begins.
      if (row_done && eos_id >= 0 && tok == eos_id) row_done[b] = 1;
    }
    if (threadIdx.x == 0) *d_step = j;
    return;
  }
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nw = blockDim.x >> 5;
  for (int b0 = 0; b0 < B; b0 += blockDim.x) {          // same trip count in every thread
    const int b = b0 + threadIdx.x;
    int32_t tok = 0;
    int live = 0;
    // the sequence slot b generates (itself without a prompt queue) and the index t of the token this
    // step produces for it (token t - 1 is fed); a sequence also ends once all T tokens exist
    int gid = b, t = j;
    if (b < B) {
      if (c.seq_gid) {
        gid = c.seq_gid[b];
        t = j - c.seq_t0[b];
      }
      if (gid < 0 || t >= T) {
        row_done[b] = 1;
      } else {
        tok = tok_hist[static_cast<size_t>(gid) * T + (t - 1)];
        if (tok == eos_id) row_done[b] = 1;
      }
      live = row_done[b] ? 0 : 1;
    }
    // block-wide exclusive scan of the live flags
    const unsigned ballot = __ballot_sync(0xffffffffu, live);
    const int in_warp = __popc(ballot & ((1u << lane) - 1u));
    if (lane == 0) warp_sum[warp] = __popc(ballot);
    __syncthreads();
    int before = base_s;
    for (int w = 0; w < warp; ++w) before += warp_sum[w];
    int total = 0;
    for (int w = 0; w < nw; ++w) total += warp_sum[w];
    if (b < B) {
      const int pos = seq_len0[b] + t - 1;
      c.seq_pos[b] = pos;
      if (live) {
        const int r = before + in_warp;
        c.row_seq[r] = b;
        c.seq_row[b] = r;
        row_tok[r] = tok;
        row_pos[r] = pos;
      } else {
        c.seq_row[b] = -1;
        if (gid >= 0 && t < T) {
          c.out_tok[static_cast<size_t>(gid) * T + t] = eos_id;
          c.out_lp[static_cast<size_t>(gid) * T + t] = 0.f;
        }
      }
    }
    __syncthreads();
    if (threadIdx.x == 0) base_s += total;
    __syncthreads();
  }
  const int n_live = base_s;
  for (int r = n_live + threadIdx.x; r < B; r += blockDim.x) {      // padding rows: a valid token, no sequence
    c.row_seq[r] = -1;
    row_tok[r] = 0;
    row_pos[r] = 0;
  }
  if (threadIdx.x == 0) {
    *c.n_live = n_live;
    *d_step = j;
  }
}

__global__ void set_int_kernel(int32_t *p, int32_t v) { *p = v; }

// Slots changing hands between two decode steps (prompt queue); one block per slot sequence.
__global__ void admit_kernel(const int32_t *admit_seq, const int32_t *admit_gid, const int32_t *d_step,
                             int32_t *seq_gid, int32_t *seq_t0, int32_t *row_done, int32_t *out_tok, float *out_lp,
                             int T, int eos_id) {
  const int b = admit_seq[blockIdx.x];
  const int j = *d_step;
  const int old = seq_gid[b];
  const int gid_new = admit_gid[blockIdx.x];
  // gid -2: the slot's group is evicted and will be generated again later; its outputs are left alone
  if (old >= 0 && eos_id >= 0 && gid_new != -2) {
    // the steps so far wrote the sequence's positions up to j - t0 (its own tokens, then the end token
    // from the step that found it ended); the rest of its row follows here
    const int t_from = max(j - seq_t0[b] + 1, 1);
    for (int t = t_from + threadIdx.x; t < T; t += blockDim.x) {
      out_tok[static_cast<size_t>(old) * T + t] = eos_id;
      out_lp[static_cast<size_t>(old) * T + t] = 0.f;
    }
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    const int gid = gid_new < 0 ? -1 : gid_new;
    seq_gid[b] = gid;
    seq_t0[b] = j;
    row_done[b] = gid < 0 ? 1 : 0;
  }
}

__device__ __forceinline__ void lse_update(float &m, float &l, float s);
__device__ __forceinline__ void lse_merge(float &m, float &l, float m2, float l2);

// Rows of a teacher-forced scoring chunk, sequence-major: row r0 + i is token j = (r0 + i) % (T - 1) of
// sequence s = (r0 + i) / (T - 1): it feeds given token j at position len0[s] + j.
__global__ void score_rows_kernel(int r0, int R, int T, const int32_t *seq_len0, int32_t *row_pt, int32_t *row_pos,
                                  int32_t *tok_idx) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= R) return;
  const int r = r0 + i, s = r / (T - 1), j = r % (T - 1);
  row_pt[i] = s;
  row_pos[i] = seq_len0[s] + j;
  tok_idx[i] = s * T + j;
}

// first_end[s] = index of the first end token among the T given tokens of sequence s (T if none)
__global__ void first_end_kernel(const int32_t *tokens, int B, int T, int eos_id, int32_t *first_end) {
  const int s = blockIdx.x * blockDim.x + threadIdx.x;
  if (s >= B) return;
  int e = T;
  if (eos_id >= 0)
    for (int j = 0; j < T; ++j)
      if (tokens[static_cast<size_t>(s) * T + j] == eos_id) {
        e = j;
        break;
      }
  first_end[s] = e;
}

// Log-probability of given tokens: row r of the launch reads logits row r / rows_per_logit_row and
// scores token tokens[flat], flat = tok_idx ? tok_idx[r] + 1 : r * T (the first token of sequence r),
// under softmax(z / temperature); positions after a sequence's end token score 0.
__global__ void __launch_bounds__(512)
logprob_rows_kernel(const float *logits, int V, int rows_per_logit_row, float inv_temperature, const int32_t *tokens,
                    const int32_t *tok_idx, int T, const int32_t *first_end, float *out, int *status) {
  __shared__ float sm_m[16], sm_l[16];
  const int r = blockIdx.x;
  const size_t flat = tok_idx ? static_cast<size_t>(tok_idx[r]) + 1 : static_cast<size_t>(r) * T;
  const int s = static_cast<int>(flat / T), j = static_cast<int>(flat % T);
  if (first_end && j > first_end[s]) {
    if (threadIdx.x == 0) out[flat] = 0.f;
    return;
  }
  const float *z = logits + static_cast<size_t>(r / rows_per_logit_row) * V;
  float m = -INFINITY, l = 0.f;
  for (int v = threadIdx.x; v < V; v += blockDim.x) lse_update(m, l, z[v] * inv_temperature);
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    const float m2 = __shfl_xor_sync(0xffffffffu, m, o), l2 = __shfl_xor_sync(0xffffffffu, l, o);
    lse_merge(m, l, m2, l2);
  }
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (lane == 0) {
    sm_m[warp] = m;
    sm_l[warp] = l;
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    float mm = -INFINITY, ll = 0.f;
    for (int i = 0; i < (blockDim.x >> 5); ++i) lse_merge(mm, ll, sm_m[i], sm_l[i]);
    int tok = tokens[flat];
    if (tok < 0 || tok >= V) {
      atomicExch(status, STATUS_BAD_TOKEN);
      tok = 0;
    }
    out[flat] = z[tok] * inv_temperature - (mm + logf(ll));
  }
}

// Appendix F, turn-aware masking: c_t = number of turn-start tokens among x_0..x_t,
// m_t = [c_t > 1] [c_t odd]; with `shift`, m is aligned with the next-token targets (out[t] = m_{t+1}).
__global__ void turn_mask_kernel(const int32_t *tokens, int n, int T, int turn_start, int shift, uint8_t *out) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= n) return;
  const int32_t *x = tokens + static_cast<size_t>(i) * T;
  uint8_t *o = out + static_cast<size_t>(i) * T;
  int c = 0;
  for (int t = 0; t < T; ++t) {
    c += x[t] == turn_start ? 1 : 0;
    const uint8_t m = (c > 1 && (c & 1)) ? 1 : 0;
    if (!shift) o[t] = m;
    else if (t > 0) o[t - 1] = m;
  }
  if (shift && T > 0) o[T - 1] = 0;
}

// Parity hook: copies n floats of the residual stream into slot (*d_step - 1) of dst.
__global__ void capture_step_kernel(const float *__restrict__ x, float *__restrict__ dst, const int32_t *d_step,
                                    size_t n) {
  const size_t slot = static_cast<size_t>(*d_step - 1);
  const size_t i = (static_cast<size_t>(blockIdx.x) * blockDim.x + threadIdx.x) * 4;
  if (i < n) *reinterpret_cast<float4 *>(dst + slot * n + i) = *reinterpret_cast<const float4 *>(x + i);
}

// Read-only streaming probe: every thread walks the buffer with 16-byte loads and folds what it reads;
// the fold is stored only if it has a value it cannot have, so nothing is written.
__global__ void __launch_bounds__(512) read_probe_kernel(const uint4 *__restrict__ buf, size_t n_vec, uint32_t *sink) {
  const size_t stride = static_cast<size_t>(gridDim.x) * blockDim.x;
  uint32_t acc = 0;
  size_t i = static_cast<size_t>(blockIdx.x) * blockDim.x + threadIdx.x;
  for (; i + 3 * stride < n_vec; i += 4 * stride) {
    const uint4 a = __ldcs(buf + i), b = __ldcs(buf + i + stride), c = __ldcs(buf + i + 2 * stride),
                d = __ldcs(buf + i + 3 * stride);
    acc ^= a.x ^ a.y ^ a.z ^ a.w ^ b.x ^ b.y ^ b.z ^ b.w ^ c.x ^ c.y ^ c.z ^ c.w ^ d.x ^ d.y ^ d.z ^ d.w;
  }
  for (; i < n_vec; i += stride) {
    const uint4 a = __ldcs(buf + i);
    acc ^= a.x ^ a.y ^ a.z ^ a.w;
  }
  if (acc == 0x9E3779B9u && sink) atomicAdd(sink, 1u);
}

// Wait-limit probe: one warp waits, with the given limit, for a barrier phase that nothing completes.
// The wait gives up, the kernel records STATUS_WAIT_TIMEOUT and returns; nothing else depends on it.
__global__ void wait_probe_kernel(uint64_t limit_ns, int *status, unsigned long long *waited_ns) {
  __shared__ uint64_t bar;
  __shared__ int abort_flag;
  if (threadIdx.x == 0) {
    ptx::mbar_init(&bar, 1);
    abort_flag = 0;
    ptx::mbar_fence_init();
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    const uint64_t t0 = ptx::global_timer_ns();
    const bool ok = ptx::mbar_wait(&bar, 0, &abort_flag, limit_ns);
    *waited_ns = ptx::global_timer_ns() - t0;
    if (!ok) atomicExch(status, STATUS_WAIT_TIMEOUT);
  }
}

// Clipped surrogate with truncated importance sampling, one warp per sequence (all in fp32):
// J_i = sum_t m_t min(exp(lo - ls), C) (min(rho A, clip(rho, 1 - e, 1 + e) A) - beta k_t) / sum_t m_t,
// rho = exp(ln - lo), k_t = exp(d) - d - 1 with d = lr - ln (lr may be null: no KL term).
__global__ void grpo_surrogate_kernel(const float *__restrict__ ln, const float *__restrict__ lo,
                                      const float *__restrict__ ls, const float *__restrict__ lr,
                                      const float *__restrict__ adv, const uint8_t *__restrict__ mask, int n, int T,
                                      float eps_clip, float C, float beta, float *__restrict__ out) {
  const int i = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5), lane = threadIdx.x & 31;
  if (i >= n) return;
  const size_t base = static_cast<size_t>(i) * T;
  const float a = adv[i];
  float num = 0.f, den = 0.f;
  for (int t = lane; t < T; t += 32) {
    if (mask && !mask[base + t]) continue;
    const float rho = expf(ln[base + t] - lo[base + t]);
    const float w = fminf(expf(lo[base + t] - ls[base + t]), C);
    const float clipped = fminf(fmaxf(rho, 1.0f - eps_clip), 1.0f + eps_clip);
    float term = fminf(rho * a, clipped * a);
    if (lr) {
      const float d = lr[base + t] - ln[base + t];
      term -= beta * (expm1f(d) - d);
    }
    num += w * term;
    den += 1.0f;
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    num += __shfl_xor_sync(0xffffffffu, num, o);
    den += __shfl_xor_sync(0xffffffffu, den, o);
  }
  if (lane == 0) out[i] = den > 0.f ? num / den : 0.f;
}

// ---------------------------------------------------------------------------
// Sampler: one block per sequence row.  Single pass over the logits row keeps, per
// thread, the running (max, sum of exp) of s = z / T and the best perturbed score
// s + g with its id (ties -> lowest id); warp shuffles and one shared-memory stage
// combine them.
// ---------------------------------------------------------------------------
struct Best {
  float score;
  int id;
};
__device__ __forceinline__ void best_update(Best &b, float sc, int id) {
  if (sc > b.score || (sc == b.score && id < b.id)) {
    b.score = sc;
    b.id = id;
  }
}
__device__ __forceinline__ void lse_update(float &m, float &l, float s) {
  if (s > m) {
    l = l * __expf(m - s) + 1.0f;
    m = s;
  } else {
    l += __expf(s - m);
  }
}
__device__ __forceinline__ void lse_merge(float &m, float &l, float m2, float l2) {
  if (m2 == -INFINITY) return;
  if (m == -INFINITY) {
    m = m2;
    l = l2;
    return;
  }
  const float mm = fmaxf(m, m2);
  l = l * __expf(m - mm) + l2 * __expf(m2 - mm);
  m = mm;
}

constexpr int kSamplerThreads = 1024;

__global__ void __launch_bounds__(kSamplerThreads)
sampler_kernel(const float *logits, int V, int rows_per_logit_row, const int32_t *seq_ids, const int32_t *d_step,
               uint32_t j_host, float inv_temperature, uint32_t key0, uint32_t key1, const int32_t *forced,
               int forced_stride, int32_t *out_tok, float *out_lp, int out_stride, int eos_id,
               const uint2 *nucleus_cut, const int32_t *row_done, uint32_t seq_base, const int32_t *row_seq,
               const int32_t *seq_gid, const int32_t *seq_t0) {
  __shared__ float sm_m[32], sm_l[32], sm_score[32];
  __shared__ int sm_id[32];
  early_start_sync();
  const int r = blockIdx.x;
  // compacted step: logits row r belongs to sequence row_seq[r] (its noise stream, its output slot);
  // a padding row has no sequence
  int seq = row_seq ? row_seq[r] : r;
  if (seq < 0) return;
  uint32_t j = d_step ? static_cast<uint32_t>(*d_step) : j_host;
  if (seq_gid) {
    // prompt queue: slot `seq` generates sequence seq_gid[seq], whose token index is counted from the
    // step its token 0 was sampled at; noise stream and output row are the sequence's, not the slot's
    j -= static_cast<uint32_t>(seq_t0[seq]);
    seq = seq_gid[seq];
    if (seq < 0) return;
  }
  if (eos_id >= 0 && j > 0 && row_done) {
    // End-of-sequence rule: the sequence is finished once one of the tokens fed so far (the forced
    // ones when scoring a given trajectory) was eos_id, which the step's preparation kernel records
    // per row; finished positions hold eos_id with log-probability 0.
    if (row_done[seq]) {
      if (threadIdx.x == 0) {
        out_tok[static_cast<size_t>(seq) * out_stride + j] = eos_id;
        out_lp[static_cast<size_t>(seq) * out_stride + j] = 0.f;
      }
      return;
    }
  }
  const uint32_t s_id = seq_base + (seq_ids ? static_cast<uint32_t>(seq_ids[r]) : static_cast<uint32_t>(seq));
  const float *z = logits + static_cast<size_t>(r / rows_per_logit_row) * V;
  const uint2 key = make_uint2(key0, key1);
  // top-p: only ids that rank at or before the row's cut (score descending, id ascending) belong to
  // the distribution; the sum below then runs over the nucleus, which renormalises the log-probability
  const bool topp = nucleus_cut != nullptr;
  const uint2 cutv = topp ? nucleus_cut[r / rows_per_logit_row] : make_uint2(0u, 0x7fffffffu);
  auto in_nucleus = [&](float s, int id) -> bool {
    if (!topp) return true;
    const uint32_t k = order_key(s);
    return k > cutv.x || (k == cutv.x && static_cast<uint32_t>(id) <= cutv.y);
  };

  float m = -INFINITY, l = 0.f;
  Best best = {-INFINITY, 0x7fffffff};
  const int nblk = (V + 3) >> 2;
  const bool vec_ok = (V & 3) == 0;
  // The two accurate logarithms of the Gumbel transform are what this kernel's time goes to, and
  // almost no draw can win: -log1p(-w) >= w, so g <= -log(w), and a draw whose score plus that
  // bound (taken with the fast logarithm and a margin far above its error) stays below the best
  // perturbed score the warp has seen is skipped.  Skipping never changes the winner or a tie.
  float warp_best = -INFINITY;
  int it = 0;
  for (int base = 0; base < nblk; base += blockDim.x, ++it) {       // same trip count in every thread
    const int blk = base + threadIdx.x;
    if (blk < nblk) {
      const uint4 w = philox4x32_10(make_uint4(static_cast<uint32_t>(blk), j, s_id, 0u), key);
      const uint32_t words[4] = {w.x, w.y, w.z, w.w};
      float zz[4];
      const int v0 = blk << 2;
      if (vec_ok) {
        const float4 t = *reinterpret_cast<const float4 *>(z + v0);
        zz[0] = t.x; zz[1] = t.y; zz[2] = t.z; zz[3] = t.w;
      } else {
#pragma unroll
        for (int i = 0; i < 4; ++i) zz[i] = (v0 + i < V) ? z[v0 + i] : -INFINITY;
      }
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        if (v0 + i < V) {
          const float s = zz[i] * inv_temperature;
          if (!in_nucleus(s, v0 + i)) continue;
          lse_update(m, l, s);
          const float u01 = uniform_from_word(words[i]);
          if (s - __logf(u01) + 1e-3f >= warp_best) best_update(best, s + gumbel_from_uniform(u01), v0 + i);
        }
      }
    }
    if ((it & 3) == 3) {                     // every few blocks: share the best score across the warp
      float b = best.score;
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) b = fmaxf(b, __shfl_xor_sync(0xffffffffu, b, o));
      warp_best = b;
    }
  }
  // warp reduction
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    const float m2 = __shfl_xor_sync(0xffffffffu, m, o), l2 = __shfl_xor_sync(0xffffffffu, l, o);
    lse_merge(m, l, m2, l2);
    const float sc = __shfl_xor_sync(0xffffffffu, best.score, o);
    const int id = __shfl_xor_sync(0xffffffffu, best.id, o);
    best_update(best, sc, id);
  }
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (lane == 0) {
    sm_m[warp] = m; sm_l[warp] = l; sm_score[warp] = best.score; sm_id[warp] = best.id;
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    const int nw = blockDim.x >> 5;
    float mm = -INFINITY, ll = 0.f;
    Best bb = {-INFINITY, 0x7fffffff};
    for (int i = 0; i < nw; ++i) {
      lse_merge(mm, ll, sm_m[i], sm_l[i]);
      best_update(bb, sm_score[i], sm_id[i]);
    }
    const int tok = bb.id < V ? bb.id : 0;
    const size_t o = static_cast<size_t>(seq) * out_stride + j;
    out_tok[o] = tok;
    const int scored = forced ? forced[static_cast<size_t>(seq) * forced_stride + j] : tok;
    const int sc_id = (scored >= 0 && scored < V) ? scored : 0;
    const float s_sc = z[sc_id] * inv_temperature;
    out_lp[o] = in_nucleus(s_sc, sc_id) ? s_sc - (mm + logf(ll)) : -INFINITY;
  }
}

__global__ void noise_debug_kernel(uint32_t key0, uint32_t key1, uint32_t s_id, uint32_t j, uint32_t v0, uint32_t n,
                                   uint32_t *words, float *uniform) {
  const uint32_t i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= n) return;
  const uint32_t v = v0 + i;
  const uint4 w = philox4x32_10(make_uint4(v >> 2, j, s_id, 0u), make_uint2(key0, key1));
  const uint32_t arr[4] = {w.x, w.y, w.z, w.w};
  const uint32_t x = arr[v & 3];
  words[i] = x;
  uniform[i] = uniform_from_word(x);
}

// A = (R - mean) / (std + eps), std with divisor (G - 1).  One warp per group.
__global__ void advantage_kernel(const float *r, int P, int G, float eps, float *out) {
  const int p = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  const int lane = threadIdx.x & 31;
  if (p >= P) return;
  const float *rp = r + static_cast<size_t>(p) * G;
  float s = 0.f;
  for (int g = lane; g < G; g += 32) s += rp[g];
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
  const float mean = s / static_cast<float>(G);
  float ss = 0.f;
  for (int g = lane; g < G; g += 32) {
    const float dlt = rp[g] - mean;
    ss = fmaf(dlt, dlt, ss);
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
  const float denom = sqrtf(ss / static_cast<float>(G - 1)) + eps;
  for (int g = lane; g < G; g += 32) out[static_cast<size_t>(p) * G + g] = (rp[g] - mean) / denom;
}

}  // namespace

cudaError_t embed_launch(const __nv_bfloat16 *embed, const int32_t *tok_src, const int32_t *tok_idx, float *x, int R,
                         int d, int vocab, int *status, cudaStream_t s) {
  return launch_early(embed_kernel, dim3(R), dim3(256), 0, s, embed, tok_src, tok_idx, x, R, d, vocab, status);
}
cudaError_t rmsnorm_launch(const float *x, const __nv_bfloat16 *gain, __nv_bfloat16 *h, int R, int d, float eps,
                           cudaStream_t s, bool out_half) {
  return launch_early(rmsnorm_kernel, dim3(R), dim3(kNormThreads), 0, s, x, gain, h, R, d, eps, out_half ? 1 : 0);
}
cudaError_t rope_table_launch(float2 *table, int max_pos, int head_dim, double theta, cudaStream_t s) {
  const int half = head_dim / 2, n = max_pos * half;
  rope_table_kernel<<<(n + 255) / 256, 256, 0, s>>>(table, max_pos, half, theta, head_dim);
  return cudaGetLastError();
}
cudaError_t rope_append_launch(float *qkv, __nv_bfloat16 *q, __nv_bfloat16 *kv_layer, const float2 *rope_table,
                               RowMeta meta, const int32_t *page_table, int pt_width, int R, int Hq, int Hkv, int hd,
                               int page_size, int n_pages, int max_pos, int *status, cudaStream_t s, bool out_half,
                               const int32_t *q_row) {
  if (hd % 8 == 0 && (reinterpret_cast<uintptr_t>(qkv) & 15) == 0)
    return launch_early(rope_append_vec_kernel, dim3(R), dim3(256), 0, s, qkv, q, kv_layer, rope_table, meta.row_pt,
                        meta.row_pos, meta.row_done, page_table, pt_width, R, Hq, Hkv, hd, page_size, n_pages, max_pos,
                        status, out_half ? 1 : 0, q_row);
  return launch_early(rope_append_kernel, dim3(R), dim3(256), 0, s, qkv, q, kv_layer, rope_table, meta.row_pt,
                      meta.row_pos, meta.row_done, page_table, pt_width, R, Hq, Hkv, hd, page_size, n_pages, max_pos,
                      status, out_half ? 1 : 0, q_row);
}
cudaError_t swiglu_launch(const float *gu, __nv_bfloat16 *act, int R, int F, cudaStream_t s, bool out_half) {
  const size_t n = static_cast<size_t>(R) * F;
  swiglu_kernel<<<static_cast<unsigned>((n + 255) / 256), 256, 0, s>>>(gu, act, R, F, out_half ? 1 : 0);
  return cudaGetLastError();
}
cudaError_t gather_rows_launch(const float *x, const int32_t *src_rows, float *dst, int n, int d, cudaStream_t s) {
  gather_rows_kernel<<<n, 256, 0, s>>>(x, src_rows, dst, n, d);
  return cudaGetLastError();
}
cudaError_t copy_partial_pages_launch(__nv_bfloat16 *kv, const int32_t *src_page, const int32_t *dst_page,
                                      int n_copies, int n_layers, size_t layer_stride_elems, int page_elems,
                                      cudaStream_t s) {
  if (n_copies == 0) return cudaSuccess;
  copy_pages_kernel<<<dim3(n_copies, n_layers), 256, 0, s>>>(kv, src_page, dst_page, layer_stride_elems, page_elems);
  return cudaGetLastError();
}
cudaError_t decode_prep_launch(int32_t *d_step, const int32_t *tok_hist, int T, const int32_t *seq_len0,
                               int32_t *row_tok, int32_t *row_pos, int B, cudaStream_t s, int eos_id,
                               int32_t *row_done, const CompactRows *cr, int32_t *out_tok, float *out_lp) {
  Compaction c{nullptr, nullptr, nullptr, nullptr, nullptr, nullptr, nullptr, nullptr};
  if (cr) c = Compaction{cr->row_seq, cr->seq_row, cr->seq_pos, cr->n_live, out_tok, out_lp, cr->seq_gid, cr->seq_t0};
  return launch_early(decode_prep_kernel, dim3(1), dim3(512), 0, s, d_step, tok_hist, T, seq_len0, row_tok, row_pos, B,
                      eos_id, row_done, c);
}
cudaError_t sampler_launch(const float *logits, int R, int V, int rows_per_logit_row, const int32_t *seq_ids,
                           const int32_t *d_step, uint32_t j_host, float temperature, uint64_t seed,
                           const int32_t *forced, int forced_stride, int32_t *out_tok, float *out_lp, int out_stride,
                           cudaStream_t s, int eos_id, const uint2 *nucleus_cut, const int32_t *row_done,
                           uint32_t seq_base, const int32_t *row_seq, const int32_t *seq_gid,
                           const int32_t *seq_t0) {
  return launch_early(sampler_kernel, dim3(R), dim3(kSamplerThreads), 0, s, logits, V, rows_per_logit_row, seq_ids,
                      d_step, j_host, 1.0f / temperature, static_cast<uint32_t>(seed & 0xffffffffu),
                      static_cast<uint32_t>(seed >> 32), forced, forced_stride, out_tok, out_lp, out_stride, eos_id,
                      nucleus_cut, row_done, seq_base, row_seq, seq_gid, seq_t0);
}
cudaError_t admit_launch(int n, const int32_t *admit_seq, const int32_t *admit_gid, const int32_t *d_step,
                         int32_t *seq_gid, int32_t *seq_t0, int32_t *row_done, int32_t *out_tok, float *out_lp, int T,
                         int eos_id, cudaStream_t s) {
  if (n <= 0) return cudaSuccess;
  admit_kernel<<<n, 128, 0, s>>>(admit_seq, admit_gid, d_step, seq_gid, seq_t0, row_done, out_tok, out_lp, T, eos_id);
  return cudaGetLastError();
}
cudaError_t noise_debug_launch(uint64_t seed, uint32_t s_id, uint32_t j, uint32_t v0, uint32_t n, uint32_t *words,
                               float *uniform, cudaStream_t s) {
  if (n == 0) return cudaSuccess;
  noise_debug_kernel<<<(n + 255) / 256, 256, 0, s>>>(static_cast<uint32_t>(seed & 0xffffffffu),
                                                     static_cast<uint32_t>(seed >> 32), s_id, j, v0, n, words,
                                                     uniform);
  return cudaGetLastError();
}
cudaError_t advantage_launch(const float *r, int P, int G, float eps, float *out, cudaStream_t s) {
  if (P == 0) return cudaSuccess;
  advantage_kernel<<<(P + 7) / 8, 256, 0, s>>>(r, P, G, eps, out);
  return cudaGetLastError();
}
cudaError_t grpo_surrogate_launch(const float *ln, const float *lo, const float *ls, const float *lr,
                                  const float *adv, const uint8_t *mask, int n, int T, float eps_clip, float C,
                                  float beta, float *out, cudaStream_t s) {
  if (n == 0) return cudaSuccess;
  grpo_surrogate_kernel<<<(n + 7) / 8, 256, 0, s>>>(ln, lo, ls, lr, adv, mask, n, T, eps_clip, C, beta, out);
  return cudaGetLastError();
}
cudaError_t score_rows_launch(int r0, int R, int T, const int32_t *seq_len0, int32_t *row_pt, int32_t *row_pos,
                              int32_t *tok_idx, cudaStream_t s) {
  if (R <= 0) return cudaSuccess;
  score_rows_kernel<<<(R + 255) / 256, 256, 0, s>>>(r0, R, T, seq_len0, row_pt, row_pos, tok_idx);
  return cudaGetLastError();
}
cudaError_t first_end_launch(const int32_t *tokens, int B, int T, int eos_id, int32_t *first_end, cudaStream_t s) {
  first_end_kernel<<<(B + 127) / 128, 128, 0, s>>>(tokens, B, T, eos_id, first_end);
  return cudaGetLastError();
}
cudaError_t logprob_rows_launch(const float *logits, int rows, int V, int rows_per_logit_row, float temperature,
                                const int32_t *tokens, const int32_t *tok_idx, int T, const int32_t *first_end,
                                float *out, int *status, cudaStream_t s) {
  if (rows <= 0) return cudaSuccess;
  logprob_rows_kernel<<<rows, 512, 0, s>>>(logits, V, rows_per_logit_row, 1.0f / temperature, tokens, tok_idx, T,
                                           first_end, out, status);
  return cudaGetLastError();
}
cudaError_t turn_mask_launch(const int32_t *tokens, int n, int T, int turn_start, int shift, uint8_t *out,
                             cudaStream_t s) {
  if (n <= 0) return cudaSuccess;
  turn_mask_kernel<<<(n + 127) / 128, 128, 0, s>>>(tokens, n, T, turn_start, shift, out);
  return cudaGetLastError();
}
cudaError_t capture_step_launch(const float *x, float *dst, const int32_t *d_step, size_t n, cudaStream_t s) {
  if (n == 0) return cudaSuccess;
  if (n % 4) return cudaErrorInvalidValue;
  capture_step_kernel<<<static_cast<unsigned>((n / 4 + 255) / 256), 256, 0, s>>>(x, dst, d_step, n);
  return cudaGetLastError();
}
cudaError_t read_probe_launch(const void *buf, size_t bytes, uint32_t *sink, int n_blocks, cudaStream_t s) {
  read_probe_kernel<<<n_blocks, 512, 0, s>>>(static_cast<const uint4 *>(buf), bytes / 16, sink);
  return cudaGetLastError();
}
cudaError_t wait_probe_launch(uint64_t limit_ns, int *status, unsigned long long *waited_ns, cudaStream_t s) {
  wait_probe_kernel<<<1, 32, 0, s>>>(limit_ns, status, waited_ns);
  return cudaGetLastError();
}
cudaError_t set_int_launch(int32_t *p, int32_t v, cudaStream_t s) {
  set_int_kernel<<<1, 1, 0, s>>>(p, v);
  return cudaGetLastError();
}

}  // namespace echo

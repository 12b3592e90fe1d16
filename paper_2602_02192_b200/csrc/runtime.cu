// Host runtime and C ABI of the rollout library: arena carve-up, double weight buffer
// with the version state machine, page-table plan, prefill + decode orchestration
// (decode step captured once as a CUDA graph and replayed), stand-alone test entry points.

#include <algorithm>
#include <cmath>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <deque>
#include <new>
#include <string>
#include <vector>

#include "common.cuh"

using namespace echo;

namespace {

constexpr size_t kAlign = 1024;
constexpr size_t kRetileStageBytes = 64ull << 20;
constexpr int kChunkRows = 2048;      // prompt tokens per prefill forward: eight 256-row activation tiles share
                                      // every weight tile (read from HBM once, seven times from L2)
constexpr int kSmallChunkRows = 256;  // ... with the plain SIMT projection kernel (debugging aid)
constexpr int kMaxCtas = 160;         // persistent GEMM grid never exceeds this (148 SMs on B200)

size_t align_up(size_t v, size_t a = kAlign) { return (v + a - 1) / a * a; }
int ceil_div(int a, int b) { return (a + b - 1) / b; }

struct Dims {
  int L, d, Hq, Hkv, hd, F, V, Z;
  int n_qkv() const { return (Hq + 2 * Hkv) * hd; }
  // projection matrices are stored block-tiled (padded to 128 x 64 blocks); embed and norms plain
  size_t layer_weight_elems() const {
    return tiled_elems(n_qkv(), d) + tiled_elems(d, static_cast<size_t>(Hq) * hd) + 2 * tiled_elems(F, d) +
           tiled_elems(d, F) + 2ull * d;
  }
  size_t weight_elems() const { return L * layer_weight_elems() + static_cast<size_t>(V) * d + tiled_elems(V, d) + d; }
};

struct Limits {
  int P, G, Lp, T, B, R;            // R = rows of the activation buffers (a prefill chunk or a decode step)
  int n_pre, n_dec, n_pages, pt_width, max_pos;
};

bool config_ok(const echo_config *c) {
  if (!c) return false;
  if (c->n_layers < 1 || c->d_model < 8 || c->n_q_heads < 1 || c->n_kv_heads < 1 || c->d_ff < 8 || c->vocab < 2)
    return false;
  if (c->head_dim != 64 && c->head_dim != 128) return false;
  if (c->n_q_heads % c->n_kv_heads) return false;
  const int rep = c->n_q_heads / c->n_kv_heads;
  if (rep != 1 && rep != 2 && rep != 4 && rep != 8) return false;
  if (c->head_dim == 64 && rep == 8) return false;
  if (c->d_model % 8 || c->d_ff % 8) return false;
  if (c->kv_page_size < 1 || c->kv_page_size > 256 || (c->kv_page_size * c->head_dim) % 8) return false;
  if (c->max_prompts < 1 || c->max_G < 1 || c->max_prompt_len < 1 || c->max_new_tokens < 1) return false;
  if (c->n_weight_buffers != 1 && c->n_weight_buffers != 2) return false;
  if (c->eos_id < -1 || c->eos_id >= c->vocab) return false;
  if (!(c->top_p >= 0.f) || c->top_p > 1.f) return false;
  if (!(c->rms_eps >= 0.f) || !(c->rope_theta > 0.f)) return false;
  if (c->half_layers < 0 || c->half_layers > c->n_layers) return false;
  if (static_cast<long long>(c->max_prompts) * c->max_G > (1 << 20)) return false;
  if (c->kv_pages < 0 || c->queue_max_live < 0 || c->queue_optimistic < 0 || c->queue_optimistic > 8) return false;
  return true;
}

Dims dims_of(const echo_config &c) {
  return Dims{c.n_layers, c.d_model, c.n_q_heads, c.n_kv_heads, c.head_dim, c.d_ff, c.vocab, c.kv_page_size};
}

Limits limits_of(const echo_config &c) {
  Limits m;
  m.P = c.max_prompts; m.G = c.max_G; m.Lp = c.max_prompt_len; m.T = c.max_new_tokens;
  m.B = m.P * m.G;
  m.R = std::max(m.B, kChunkRows);
  const int Z = c.kv_page_size;
  m.n_pre = ceil_div(m.Lp, Z);
  int nd = 0;
  for (int b = 0; b < Z && b <= m.Lp; ++b) nd = std::max(nd, ceil_div(b + m.T - 1, Z));
  m.n_dec = nd;
  m.n_pages = m.P * m.n_pre + m.B * m.n_dec;
  if (c.kv_pages > 0) m.n_pages = std::max(c.kv_pages, m.n_pre + m.G * m.n_dec);
  m.pt_width = std::max(ceil_div(m.Lp + m.T - 1, Z), m.n_pre);
  m.max_pos = m.Lp + m.T;
  return m;
}

// Arena layout: offsets in bytes.
struct Layout {
  size_t weights[2], kv, rope, x, h, qkv, q, attn, act, gu, xlast, hlast, logits;
  size_t page_table, pre_row_pt, pre_row_pos, pre_tok_idx, gather_map, dec_row_tok, dec_row_pos, dec_row_pt,
      seq_len0, full_pages, pre_o, pre_ml, retile_stage, nucleus_cut, row_done, copy_src, copy_dst, d_step, status, attn_work, gemm_ws, gemm_counters, stage_prompts, stage_tok, stage_lp, row_seq, seq_row, seq_pos, n_live, gemm_bar, seq_gid, seq_t0, admit_seq, admit_gid, total;
  size_t weight_bytes, kv_layer_elems, n_tables_ints;
  int n_chunks_max;
};

Layout layout_of(const echo_config &c) {
  const Dims D = dims_of(c);
  const Limits M = limits_of(c);
  Layout lo;
  size_t off = 0;
  auto take = [&](size_t bytes) { size_t o = off; off = align_up(off + bytes); return o; };
  lo.weight_bytes = align_up(D.weight_elems() * 2 + (static_cast<size_t>(D.L) * 9 + 3) * kAlign);
  for (int b = 0; b < 2; ++b) lo.weights[b] = b < c.n_weight_buffers ? take(lo.weight_bytes) : 0;
  lo.kv_layer_elems = static_cast<size_t>(M.n_pages) * D.Hkv * 2 * D.Z * D.hd;
  lo.kv = take(lo.kv_layer_elems * D.L * 2);
  lo.rope = take(static_cast<size_t>(M.max_pos) * (D.hd / 2) * sizeof(float2));
  lo.x = take(static_cast<size_t>(M.R) * D.d * 4);
  lo.h = take(static_cast<size_t>(M.R) * D.d * 2);
  lo.qkv = take(static_cast<size_t>(M.R) * D.n_qkv() * 4);
  lo.q = take(static_cast<size_t>(M.R) * D.Hq * D.hd * 2);
  lo.attn = take(static_cast<size_t>(M.R) * D.Hq * D.hd * 2);
  lo.act = take(static_cast<size_t>(M.R) * D.F * 2);
  // gate / up pre-activations of the SIMT path (chunks of kSmallChunkRows there); last-position rows,
  // their normed copy and the logits: one row per sequence at most
  lo.gu = take(static_cast<size_t>(std::max(M.B, kSmallChunkRows)) * 2 * D.F * 4);
  lo.xlast = take(static_cast<size_t>(M.B) * D.d * 4);
  lo.hlast = take(static_cast<size_t>(M.B) * D.d * 2);
  lo.logits = take(static_cast<size_t>(M.B) * D.V * 4);
  const size_t n_pre_tok = static_cast<size_t>(M.P) * M.Lp;
  // row lists: the prompt tokens of a rollout, or one chunk of a scoring pass
  const size_t n_row_list = std::max<size_t>(n_pre_tok, kChunkRows);
  lo.n_chunks_max = static_cast<int>((n_pre_tok + kSmallChunkRows - 1) / kSmallChunkRows);
  lo.page_table = take(static_cast<size_t>(M.B + M.P) * M.pt_width * 4);
  lo.pre_row_pt = take(n_row_list * 4);
  lo.pre_row_pos = take(n_row_list * 4);
  lo.pre_tok_idx = take(n_row_list * 4);
  lo.gather_map = take(static_cast<size_t>(lo.n_chunks_max) * M.P * 4);
  lo.dec_row_tok = take(static_cast<size_t>(M.B) * 4);
  lo.dec_row_pos = take(static_cast<size_t>(M.B) * 4);
  lo.dec_row_pt = take(static_cast<size_t>(M.B) * 4);
  lo.seq_len0 = take(static_cast<size_t>(M.B) * 4);
  lo.full_pages = take(static_cast<size_t>(M.B) * 4);
  lo.pre_o = take(static_cast<size_t>(M.B) * D.Hq * D.hd * 4);
  lo.pre_ml = take(static_cast<size_t>(M.B) * D.Hq * 8);
  lo.retile_stage = take(kRetileStageBytes);       // bounce buffer for snapshots in pageable host memory
  lo.nucleus_cut = take(static_cast<size_t>(M.B) * 8);   // top-p: one (score key, id) cut per logits row
  lo.row_done = take(static_cast<size_t>(M.B) * 4);      // end-of-sequence rule: rows whose sequence has ended
  lo.row_seq = take(static_cast<size_t>(M.B) * 4);       // compaction of ended sequences out of a decode step's rows
  lo.seq_row = take(static_cast<size_t>(M.B) * 4);
  lo.seq_pos = take(static_cast<size_t>(M.B) * 4);
  lo.n_live = take(4);
  lo.gemm_bar = take(8);                                 // grid-wide barrier of the fused RMSNorm prologue
  lo.copy_src = take(static_cast<size_t>(M.B) * 4);
  lo.copy_dst = take(static_cast<size_t>(M.B) * 4);
  lo.d_step = take(4);
  lo.status = take(4);
  lo.attn_work = take(8);
  lo.gemm_ws = take(static_cast<size_t>(kMaxCtas) * 3 * 2 * kGemmTileN * kMaxBatchTile * sizeof(float));
  lo.gemm_counters = take(static_cast<size_t>(kGemmMaxUnits) * 4);
  lo.stage_prompts = take(static_cast<size_t>(M.P) * M.Lp * 4);
  lo.stage_tok = take(static_cast<size_t>(M.B) * M.T * 4);
  lo.stage_lp = take(static_cast<size_t>(M.B) * M.T * 4);
  // prompt queue: what each sequence slot generates, since which step; the slots changing hands
  lo.seq_gid = take(static_cast<size_t>(M.B) * 4);
  lo.seq_t0 = take(static_cast<size_t>(M.B) * 4);
  lo.admit_seq = take(static_cast<size_t>(M.B) * 4);
  lo.admit_gid = take(static_cast<size_t>(M.B) * 4);
  lo.total = off;
  return lo;
}

struct WeightBuf {
  uint8_t *base = nullptr;
  __nv_bfloat16 *embed = nullptr, *lm_head = nullptr, *final_norm = nullptr;
  std::vector<__nv_bfloat16 *> wqkv, wo, wgu, wdown, attn_norm, mlp_norm;
  std::vector<CUtensorMap> tm_qkv, tm_o, tm_gu, tm_down;
  std::vector<CUtensorMap> tm_gu_pair;       // gate/up with a 128-row box, for the SM-pair kernel
  CUtensorMap tm_lm;
  int64_t version = -1;
  bool has_data = false;       // an install was enqueued into this buffer
  cudaEvent_t installed = nullptr, inst_begin = nullptr, last_use = nullptr;
  bool used = false;           // last_use has been recorded at least once
};

}  // namespace

struct echo_ctx {
  echo_config cfg;
  Dims D;
  Limits M;
  Layout lo;
  int device = 0;
  uint8_t *arena = nullptr;
  cudaStream_t stream = nullptr, copy_stream = nullptr;
  WeightBuf wb[2];
  int active = -1, pending = -1, last_install = -1;
  int64_t newest_version = 0;
  bool any_version = false;
  cudaEvent_t plan_done = nullptr, all_done = nullptr;
  cudaEvent_t ev_begin = nullptr, ev_first = nullptr, ev_end = nullptr;   // phases of the last rollout
  bool plan_in_flight = false;
  // pinned staging for the plan tables
  int32_t *h_tables = nullptr;
  size_t h_tables_ints = 0;
  // last plan (host copy) for echo_debug_page_table
  std::vector<int32_t> last_table;
  int last_rows = 0, last_width = 0;
  echo_stats stats{};
  int64_t launches = 0;
  bool use_simt = false, use_graph = true, fast_decode = false, deterministic = false, use_pdl = true, use_pair = true;
  bool long_suffix = false;   // decode steps whose sequences hold many generated tokens (see kLongSuffix)
  int attn_suffix_impl = 0, attn_prefix_impl = 0;   // diagnostic kernel choices (ECHO_ATTN_IMPL / ECHO_ATTN_PREFIX)
  int chunk_rows = kChunkRows;
  // With an end token the decode steps run on the rows of the sequences that have not ended (see
  // decode_step); the host follows the number of live rows two windows of steps behind the GPU.
  bool fuse_norm = false;     // RMSNorm as the prologue of the projection that consumes it (decode steps)
  bool compact = false;
  int32_t *h_live = nullptr;          // page-locked: live rows reported at the end of each window
  int32_t *h_queue = nullptr;         // page-locked: admit lists (2 x B) and three snapshots of the ended flags (3 x B)
  bool queue_mode = false;            // the rollout being enqueued runs over a prompt queue
  cudaEvent_t live_ev[3] = {nullptr, nullptr, nullptr};
  bool prefill_rows = false;  // ECHO_ATTN_PREFILL=rows: the one-query-per-row kernel for the prompt prefill too
  uint32_t seq_base = 0;      // added to p * G + g in the noise streams (echo_set_sequence_base)
  // parity hook (echo_debug_capture): residual stream before / after one layer
  int cap_layer = -1;
  float *cap_pre_in = nullptr, *cap_pre_out = nullptr, *cap_dec_in = nullptr, *cap_dec_out = nullptr;
  int cap_row0 = 0;           // first prefill row of the chunk being run
  bool cap_decode = false;    // the forward being enqueued is a decode step
  CUtensorMap tm_kv;
  std::string last_error;
  // sampled per-kernel timing (echo_profile_config / echo_profile_read)
  int prof_every = 0;
  bool prof_now = false;
  int prof_step = 0;
  struct ProfRec { int step, cls; cudaEvent_t a, b; };
  std::vector<ProfRec> prof_recs;
  std::vector<cudaEvent_t> prof_pool;
  size_t prof_pool_used = 0;

  template <typename T>
  T *ptr(size_t off) const { return reinterpret_cast<T *>(arena + off); }
};

namespace {

int fail_cuda(echo_ctx *ctx, cudaError_t e, const char *what) {
  if (ctx) {
    char buf[256];
    snprintf(buf, sizeof buf, "%s: %s", what, cudaGetErrorString(e));
    ctx->last_error = buf;
  }
  return ECHO_ERR_CUDA;
}

cudaEvent_t prof_event(echo_ctx *ctx) {
  if (ctx->prof_pool_used == ctx->prof_pool.size()) {
    cudaEvent_t e = nullptr;
    if (cudaEventCreate(&e) != cudaSuccess) return nullptr;
    ctx->prof_pool.push_back(e);
  }
  return ctx->prof_pool[ctx->prof_pool_used++];
}
// Brackets the launches issued inside its scope with two events when the step is sampled.
struct ProfScope {
  echo_ctx *ctx;
  cudaEvent_t a = nullptr, b = nullptr;
  int cls;
  ProfScope(echo_ctx *c, int cls_) : ctx(c), cls(cls_) {
    if (!ctx->prof_now) return;
    a = prof_event(ctx);
    b = prof_event(ctx);
    if (a && b) cudaEventRecord(a, ctx->stream);
  }
  ~ProfScope() {
    if (!a || !b) return;
    cudaEventRecord(b, ctx->stream);
    ctx->prof_recs.push_back({ctx->prof_step, cls, a, b});
  }
};
enum { PROF_ATTN = 0, PROF_GEMM = 1, PROF_SAMPLER = 2, PROF_STEP = 3, PROF_NCLS = 4 };

#define CK(expr)                                            \
  do {                                                      \
    cudaError_t e__ = (expr);                               \
    if (e__ != cudaSuccess) return fail_cuda(ctx, e__, #expr); \
  } while (0)
#define LAUNCH(expr)                                        \
  do {                                                      \
    cudaError_t e__ = (expr);                               \
    if (e__ != cudaSuccess) return fail_cuda(ctx, e__, #expr); \
    ctx->launches++;                                        \
  } while (0)

struct DeviceGuard {
  int prev = -1;
  explicit DeviceGuard(int dev) {
    cudaGetDevice(&prev);
    if (prev != dev) cudaSetDevice(dev);
    else prev = -1;
  }
  ~DeviceGuard() {
    if (prev >= 0) cudaSetDevice(prev);
  }
};

// Decode step from which the suffix attention runs one CTA per (sequence, kv head) again (measured
// crossover of the two suffix kernels at the 8B shape: ~1100 generated tokens per sequence).
constexpr int kLongSuffix = 1088;

int pick_bnb(int rows) {
  if (rows <= 32) return 32;
  if (rows <= 64) return 64;
  if (rows <= 128) return 128;
  return 256;
}

// Y = X * W^T through the tensor-core kernel (or the SIMT reference when selected).
int run_gemm(echo_ctx *ctx, const CUtensorMap *tmW, const __nv_bfloat16 *W, const __nv_bfloat16 *X, void *Y, int ldY,
             int M, int N, int K, int epilogue, bool y_holds_zeros = false, const CUtensorMap *tmW_pair = nullptr,
             bool half_in = false, const NormPrologue *norm = nullptr) {
  ProfScope prof(ctx, PROF_GEMM);
  if (ctx->use_pair && !ctx->use_simt && !ctx->deterministic && (epilogue != EPI_SWIGLU || tmW_pair) &&
      gemm_pair_supported(Y, ldY, M, N, K, epilogue)) {
    // more than 64 rows: 2-CTA MMAs, k-slices added into Y in memory
    PairGemmArgs a{tmW_pair ? tmW_pair : tmW, X, Y, ldY, M, N, K, epilogue, ctx->ptr<int>(ctx->lo.status),
                   ctx->use_pdl ? 1 : 0, 0, 1, half_in ? 1 : 0};
    if (norm) a.norm = *norm;
    if (epilogue == EPI_STORE && !y_holds_zeros && gemm_pair_split(M, N, K, epilogue, 0) > 1) {
      CK(cudaMemsetAsync(Y, 0, static_cast<size_t>(M) * ldY * sizeof(float), ctx->stream));
      a.allow_early_start = 0;
    }
    LAUNCH(gemm_pair_launch(a, ctx->stream));
    return ECHO_OK;
  }
  if (ctx->use_simt) {
    if (epilogue == EPI_SWIGLU) {
      float *gu = ctx->ptr<float>(ctx->lo.gu);
      LAUNCH(gemm_simt_launch(X, W, gu, 2 * N, M, 2 * N, K, 0, ctx->stream, 1, N, half_in ? 1 : 0));
      LAUNCH(swiglu_launch(gu, reinterpret_cast<__nv_bfloat16 *>(Y), M, N, ctx->stream, half_in));
      return ECHO_OK;
    }
    LAUNCH(gemm_simt_launch(X, W, reinterpret_cast<float *>(Y), ldY, M, N, K, epilogue == EPI_ACCUM, ctx->stream, 1,
                            0, half_in ? 1 : 0));
    return ECHO_OK;
  }
  CUtensorMap tmX;
  const int bnb = pick_bnb(M);
  if (make_tensor_map(&tmX, X, M, K, K, bnb) != 0) {
    ctx->last_error = "tensor map encode failed (activation)";
    return ECHO_ERR_CUDA;
  }
  GemmArgs a{tmW, &tmX, Y, ldY, M, N, K, bnb, epilogue, ctx->ptr<int>(ctx->lo.status),
             ctx->ptr<float>(ctx->lo.gemm_ws), ctx->ptr<int>(ctx->lo.gemm_counters), kMaxCtas, 0, ctx->use_pdl ? 1 : 0,
             ctx->deterministic ? 0 : 1, 1, half_in ? 1 : 0};
  if (a.independent_splits && epilogue == EPI_STORE && N < 8 * 4096 && !y_holds_zeros) {
    // the k-slices add into Y: it must start at zero.  The memset is the GEMM's predecessor on the
    // stream, so this launch does not use the early start.
    CK(cudaMemsetAsync(Y, 0, static_cast<size_t>(M) * ldY * sizeof(float), ctx->stream));
    a.allow_early_start = 0;
  }
  LAUNCH(gemm_tc_launch(a, ctx->stream));
  return ECHO_OK;
}

// true if run_gemm will take the SM-pair kernel for this projection
bool takes_pair_kernel(echo_ctx *ctx, const void *Y, int ldY, int M, int N, int K, int epilogue, bool has_pair_map) {
  return ctx->use_pair && !ctx->use_simt && !ctx->deterministic && (epilogue != EPI_SWIGLU || has_pair_map) &&
         gemm_pair_supported(Y, ldY, M, N, K, epilogue);
}

#define TRY(expr)                 \
  do {                            \
    int rc__ = (expr);            \
    if (rc__ != ECHO_OK) return rc__; \
  } while (0)

// All layers for R activation rows already embedded in x.
int forward_layers(echo_ctx *ctx, const WeightBuf &w, int R, RowMeta meta, int decode_P = 0, int decode_G = 0,
                   const CompactRows *cr = nullptr) {
  const Dims &D = ctx->D;
  const Layout &lo = ctx->lo;
  float *x = ctx->ptr<float>(lo.x);
  __nv_bfloat16 *h = ctx->ptr<__nv_bfloat16>(lo.h);
  float *qkv = ctx->ptr<float>(lo.qkv);
  __nv_bfloat16 *q = ctx->ptr<__nv_bfloat16>(lo.q);
  __nv_bfloat16 *attn = ctx->ptr<__nv_bfloat16>(lo.attn);
  __nv_bfloat16 *act = ctx->ptr<__nv_bfloat16>(lo.act);
  const int32_t *pt = ctx->ptr<int32_t>(lo.page_table);
  int *status = ctx->ptr<int>(lo.status);
  const float2 *rope = ctx->ptr<float2>(lo.rope);
  for (int l = 0; l < D.L; ++l) {
    __nv_bfloat16 *kv_layer = ctx->ptr<__nv_bfloat16>(lo.kv) + static_cast<size_t>(l) * lo.kv_layer_elems;
    // the 16-bit operands of this layer (projection inputs and weights, q, cached K/V, probabilities)
    // are IEEE half instead of bf16
    const bool hf = l < ctx->cfg.half_layers;
    auto capture = [&](float *pre, float *dec) -> cudaError_t {
      const size_t n = static_cast<size_t>(R) * D.d;
      if (ctx->cap_decode)
        return dec ? capture_step_launch(x, dec, ctx->ptr<int32_t>(lo.d_step), n, ctx->stream) : cudaSuccess;
      return pre ? cudaMemcpyAsync(pre + static_cast<size_t>(ctx->cap_row0) * D.d, x, n * 4, cudaMemcpyDeviceToDevice,
                                   ctx->stream)
                 : cudaSuccess;
    };
    if (l == ctx->cap_layer) CK(capture(ctx->cap_pre_in, ctx->cap_dec_in));
    // RMSNorm: a kernel of its own, or (decode steps, when every CTA of the projection is resident at
    // once) the prologue of the projection that consumes it
    NormPrologue np_attn{x, w.attn_norm[l], h, ctx->cfg.rms_eps, ctx->ptr<int>(lo.gemm_bar)};
    const bool fuse_attn = ctx->fuse_norm && decode_P > 0 &&
                           takes_pair_kernel(ctx, qkv, D.n_qkv(), R, D.n_qkv(), D.d, EPI_STORE, false) &&
                           gemm_pair_can_fuse_norm(R, D.n_qkv(), D.d, EPI_STORE);
    if (!fuse_attn) LAUNCH(rmsnorm_launch(x, w.attn_norm[l], h, R, D.d, ctx->cfg.rms_eps, ctx->stream, hf));
    // the qkv buffer holds zeros here: rope_append clears every row it consumes
    TRY(run_gemm(ctx, &w.tm_qkv[l], w.wqkv[l], h, qkv, D.n_qkv(), R, D.n_qkv(), D.d, EPI_STORE, !ctx->use_simt, nullptr,
                 hf, fuse_attn ? &np_attn : nullptr));
    LAUNCH(rope_append_launch(qkv, q, kv_layer, rope, meta, pt, ctx->M.pt_width, R, D.Hq, D.Hkv, D.hd, D.Z,
                              ctx->M.n_pages, ctx->M.max_pos, status, ctx->stream, hf, cr ? cr->row_seq : nullptr));
    if (decode_P > 0 && ctx->fast_decode) {
      ProfScope prof(ctx, PROF_ATTN);
      // a compacted step: attention stays per sequence (q, positions, ended flags and page-table rows by
      // sequence id) and writes each live sequence's output into the activation row it occupies
      DecodeAttnArgs da{&ctx->tm_kv, q, attn, ctx->ptr<float>(lo.pre_o), ctx->ptr<float2>(lo.pre_ml), pt,
                        ctx->M.pt_width, cr ? cr->seq_pos : meta.row_pos, ctx->ptr<int32_t>(lo.full_pages),
                        static_cast<int>(static_cast<size_t>(l) * (lo.kv_layer_elems / D.hd)), decode_P, decode_G,
                        D.Hq, D.Hkv, D.hd, ctx->M.n_pages, status,
                        cr ? ctx->ptr<int32_t>(lo.row_done) : meta.row_done,
                        ctx->long_suffix ? nullptr : ctx->ptr<int>(lo.attn_work), hf ? 1 : 0, ctx->attn_suffix_impl,
                        ctx->attn_prefix_impl, cr ? cr->seq_row : nullptr};
      LAUNCH(attention_decode_launch(da, ctx->stream));
      ctx->launches++;                      // two kernels per call
    } else if (decode_P == 0 && ctx->fast_decode && !ctx->prefill_rows) {
      // prompt prefill: causal attention of the chunk on the warp-level tensor-core tile loop
      ProfScope prof(ctx, PROF_ATTN);
      PrefillAttnArgs pa{&ctx->tm_kv, q, attn, meta.row_pt, meta.row_pos, pt, ctx->M.pt_width, R,
                         static_cast<int>(static_cast<size_t>(l) * (lo.kv_layer_elems / D.hd)), D.Hq, D.Hkv, D.hd,
                         ctx->M.n_pages, status, hf ? 1 : 0};
      LAUNCH(attention_prefill_launch(pa, ctx->stream));
    } else {
      ProfScope prof(ctx, PROF_ATTN);
      LAUNCH(attention_rows_launch(q, kv_layer, attn, meta, pt, ctx->M.pt_width, R, D.Hq, D.Hkv, D.hd, D.Z,
                                   ctx->M.n_pages, status, ctx->stream, hf));
    }
    TRY(run_gemm(ctx, &w.tm_o[l], w.wo[l], attn, x, D.d, R, D.d, D.Hq * D.hd, EPI_ACCUM, false, nullptr, hf));
    NormPrologue np_mlp{x, w.mlp_norm[l], h, ctx->cfg.rms_eps, ctx->ptr<int>(lo.gemm_bar)};
    const bool fuse_mlp = ctx->fuse_norm && decode_P > 0 &&
                          takes_pair_kernel(ctx, act, D.F, R, D.F, D.d, EPI_SWIGLU, true) &&
                          gemm_pair_can_fuse_norm(R, D.F, D.d, EPI_SWIGLU);
    if (!fuse_mlp) LAUNCH(rmsnorm_launch(x, w.mlp_norm[l], h, R, D.d, ctx->cfg.rms_eps, ctx->stream, hf));
    TRY(run_gemm(ctx, &w.tm_gu[l], w.wgu[l], h, act, D.F, R, D.F, D.d, EPI_SWIGLU, false, &w.tm_gu_pair[l], hf,
                 fuse_mlp ? &np_mlp : nullptr));
    TRY(run_gemm(ctx, &w.tm_down[l], w.wdown[l], act, x, D.d, R, D.d, D.F, EPI_ACCUM, false, nullptr, hf));
    if (l == ctx->cap_layer) CK(capture(ctx->cap_pre_out, ctx->cap_dec_out));
  }
  return ECHO_OK;
}

// final norm + lm_head on `rows` rows of xsrc -> logits
int lm_head(echo_ctx *ctx, const WeightBuf &w, const float *xsrc, int rows) {
  const Dims &D = ctx->D;
  __nv_bfloat16 *hl = ctx->ptr<__nv_bfloat16>(ctx->lo.hlast);
  LAUNCH(rmsnorm_launch(xsrc, w.final_norm, hl, rows, D.d, ctx->cfg.rms_eps, ctx->stream));
  return run_gemm(ctx, &w.tm_lm, w.lm_head, hl, ctx->ptr<float>(ctx->lo.logits), D.V, rows, D.V, D.d, EPI_STORE);
}

void carve_weights(echo_ctx *ctx, WeightBuf &w, uint8_t *base) {
  const Dims &D = ctx->D;
  w.base = base;
  size_t off = 0;
  auto take = [&](size_t elems) {
    __nv_bfloat16 *p = reinterpret_cast<__nv_bfloat16 *>(base + off);
    off = align_up(off + elems * 2);
    return p;
  };
  w.embed = take(static_cast<size_t>(D.V) * D.d);
  w.lm_head = take(tiled_elems(D.V, D.d));
  w.final_norm = take(D.d);
  w.wqkv.resize(D.L); w.wo.resize(D.L); w.wgu.resize(D.L); w.wdown.resize(D.L);
  w.attn_norm.resize(D.L); w.mlp_norm.resize(D.L);
  w.tm_qkv.resize(D.L); w.tm_o.resize(D.L); w.tm_gu.resize(D.L); w.tm_down.resize(D.L); w.tm_gu_pair.resize(D.L);
  for (int l = 0; l < D.L; ++l) {
    w.wqkv[l] = take(tiled_elems(D.n_qkv(), D.d));                       // q, k, v rows of one matrix
    w.wo[l] = take(tiled_elems(D.d, static_cast<size_t>(D.Hq) * D.hd));
    w.wgu[l] = take(2 * tiled_elems(D.F, D.d));                          // gate part, then up part
    w.wdown[l] = take(tiled_elems(D.d, D.F));
    w.attn_norm[l] = take(D.d);
    w.mlp_norm[l] = take(D.d);
  }
}

int make_weight_maps(echo_ctx *ctx, WeightBuf &w) {
  const Dims &D = ctx->D;
  int rc = 0;
  rc |= make_tiled_map(&w.tm_lm, w.lm_head, D.V, D.d, kGemmTileN);
  const uint64_t gu_rows = 2ull * ((D.F + kTileRows - 1) / kTileRows) * kTileRows;     // both parts, padded
  for (int l = 0; l < D.L; ++l) {
    rc |= make_tiled_map(&w.tm_qkv[l], w.wqkv[l], D.n_qkv(), D.d, kGemmTileN);
    rc |= make_tiled_map(&w.tm_o[l], w.wo[l], D.d, D.Hq * D.hd, kGemmTileN);
    rc |= make_tiled_map(&w.tm_gu[l], w.wgu[l], gu_rows, D.d, 64);
    rc |= make_tiled_map(&w.tm_gu_pair[l], w.wgu[l], gu_rows, D.d, kGemmTileN);
    rc |= make_tiled_map(&w.tm_down[l], w.wdown[l], D.d, D.F, kGemmTileN);
  }
  if (rc) {
    ctx->last_error = "tensor map encode failed (weights)";
    return ECHO_ERR_CUDA;
  }
  return ECHO_OK;
}

// Flip to a newer snapshot if one is ready; returns the buffer to serve, or nullptr.
WeightBuf *begin_rollout_version(echo_ctx *ctx, int *rc) {
  *rc = ECHO_OK;
  if (ctx->pending >= 0) {
    WeightBuf &p = ctx->wb[ctx->pending];
    bool take = ctx->active < 0;
    if (!take) take = cudaEventQuery(p.installed) == cudaSuccess;
    if (take) {
      // order the compute stream after the install (a no-op when it has completed)
      cudaError_t e = cudaStreamWaitEvent(ctx->stream, p.installed, 0);
      if (e != cudaSuccess) {
        *rc = fail_cuda(ctx, e, "cudaStreamWaitEvent(installed)");
        return nullptr;
      }
      ctx->active = ctx->pending;
      ctx->pending = -1;
    }
  }
  if (ctx->active < 0) {
    *rc = ECHO_ERR_NO_POLICY;
    return nullptr;
  }
  return &ctx->wb[ctx->active];
}

struct Plan {
  int P, G, T, B, n_tok, n_chunks, n_copies, n_pages, width;
};

// The page plan itself (pure host arithmetic).  Writes pt[(P*G + P)][W]: rows 0..P*G-1 are the
// sequences' tables, rows P*G.. are where each prompt's prefill writes; entries past a row's last
// page are -1.  copy_src/copy_dst (capacity P*G each, may be null) list the partial prompt pages
// to duplicate into each sample's first decode page.  Returns the number of physical pages.
int plan_tables(const int32_t *lens, int P, int G, int T, int Z, int W, int32_t *pt, int32_t *copy_src,
                int32_t *copy_dst, int *n_copies_out) {
  const int B = P * G;
  std::fill(pt, pt + static_cast<size_t>(B + P) * W, -1);
  int next_page = 0;
  std::vector<int> pre_base(P);
  for (int p = 0; p < P; ++p) {
    pre_base[p] = next_page;
    next_page += ceil_div(lens[p], Z);
  }
  int n_copies = 0;
  for (int p = 0; p < P; ++p) {
    const int full = lens[p] / Z, n_pre = ceil_div(lens[p], Z);
    const int n_dec = ceil_div(lens[p] + T - 1, Z) - full;
    int32_t *pre_row = pt + static_cast<size_t>(B + p) * W;
    for (int qi = 0; qi < n_pre; ++qi) pre_row[qi] = pre_base[p] + qi;
    for (int g = 0; g < G; ++g) {
      const int s = p * G + g;
      int32_t *row = pt + static_cast<size_t>(s) * W;
      for (int qi = 0; qi < full; ++qi) row[qi] = pre_base[p] + qi;
      for (int qi = 0; qi < n_dec; ++qi) row[full + qi] = next_page + qi;
      if (n_pre > full && n_dec > 0) {          // partial last prompt page: private copy per sample
        if (copy_src) copy_src[n_copies] = pre_base[p] + full;
        if (copy_dst) copy_dst[n_copies] = next_page;
        ++n_copies;
      }
      next_page += n_dec;
    }
  }
  if (n_copies_out) *n_copies_out = n_copies;
  return next_page;
}

// Page tables and row lists, written into the pinned staging block in the order of the
// device-side table regions.  Sequence id s = p*G + g.  Prefix pages of prompt p:
// pre_base[p] + [0, ceil(Lp/Z)); decode pages of s: dec_base[s] + [0, n_dec_p).
int build_plan(echo_ctx *ctx, const int32_t *lens, int P, int G, int T, Plan *plan) {
  const int Z = ctx->D.Z;
  const Limits &M = ctx->M;
  const int B = P * G, W = M.pt_width;
  int32_t *h = ctx->h_tables;
  int32_t *h_pt = h;
  int32_t *h_row_pt = h_pt + static_cast<size_t>(M.B + M.P) * W;
  int32_t *h_row_pos = h_row_pt + static_cast<size_t>(M.P) * M.Lp;
  int32_t *h_tok_idx = h_row_pos + static_cast<size_t>(M.P) * M.Lp;
  int32_t *h_gather = h_tok_idx + static_cast<size_t>(M.P) * M.Lp;
  int32_t *h_dec_pt = h_gather + static_cast<size_t>(ctx->lo.n_chunks_max) * M.P;
  int32_t *h_len0 = h_dec_pt + M.B;
  int32_t *h_full = h_len0 + M.B;
  int32_t *h_csrc = h_full + M.B;
  int32_t *h_cdst = h_csrc + M.B;

  int n_copies = 0;
  const int next_page = plan_tables(lens, P, G, T, Z, W, h_pt, h_csrc, h_cdst, &n_copies);
  std::fill(h_pt + static_cast<size_t>(B + P) * W, h_pt + static_cast<size_t>(M.B + M.P) * W, -1);
  for (int p = 0; p < P; ++p)
    for (int g = 0; g < G; ++g) {
      const int s = p * G + g;
      h_dec_pt[s] = s;
      h_len0[s] = lens[p];
      h_full[s] = lens[p] / Z;
    }
  if (next_page > M.n_pages) return ECHO_ERR_INVALID;
  int n_tok = 0;
  for (int p = 0; p < P; ++p) n_tok += lens[p];
  const int chunk = ctx->chunk_rows;
  const int n_chunks = ceil_div(n_tok, chunk);
  std::fill(h_gather, h_gather + static_cast<size_t>(n_chunks) * P, -1);
  int i = 0;
  for (int p = 0; p < P; ++p) {
    for (int t = 0; t < lens[p]; ++t, ++i) {
      h_row_pt[i] = B + p;
      h_row_pos[i] = t;
      h_tok_idx[i] = p * M.Lp + t;
    }
    const int last = i - 1;
    h_gather[static_cast<size_t>(last / chunk) * P + p] = last % chunk;
  }
  *plan = Plan{P, G, T, B, n_tok, n_chunks, n_copies, next_page, W};
  ctx->last_table.assign(h_pt, h_pt + static_cast<size_t>(B) * W);
  ctx->last_rows = B;
  ctx->last_width = W;
  return ECHO_OK;
}

int upload_plan(echo_ctx *ctx, const Plan &pl) {
  const Limits &M = ctx->M;
  const Layout &lo = ctx->lo;
  const int W = M.pt_width;
  int32_t *h = ctx->h_tables;
  size_t o = 0;
  auto up = [&](size_t dev_off, size_t cap_ints, size_t n_ints) -> cudaError_t {
    cudaError_t e = cudaSuccess;
    if (n_ints) e = cudaMemcpyAsync(ctx->arena + dev_off, h + o, n_ints * 4, cudaMemcpyHostToDevice, ctx->stream);
    o += cap_ints;
    return e;
  };
  const size_t npt = static_cast<size_t>(M.P) * M.Lp;
  // the prefill rows of the table sit at row index B of *this* call, so upload B+P rows contiguously
  CK(up(lo.page_table, static_cast<size_t>(M.B + M.P) * W, static_cast<size_t>(pl.B + pl.P) * W));
  CK(up(lo.pre_row_pt, npt, pl.n_tok));
  CK(up(lo.pre_row_pos, npt, pl.n_tok));
  CK(up(lo.pre_tok_idx, npt, pl.n_tok));
  CK(up(lo.gather_map, static_cast<size_t>(lo.n_chunks_max) * M.P, static_cast<size_t>(pl.n_chunks) * pl.P));
  CK(up(lo.dec_row_pt, M.B, pl.B));
  CK(up(lo.seq_len0, M.B, pl.B));
  CK(up(lo.full_pages, M.B, pl.B));
  CK(up(lo.copy_src, M.B, pl.n_copies));
  CK(up(lo.copy_dst, M.B, pl.n_copies));
  CK(cudaEventRecord(ctx->plan_done, ctx->stream));
  ctx->plan_in_flight = true;
  return ECHO_OK;
}

// One decode step: token j-1 in, token j out.  Every kernel reads the step index from
// device memory, so the same launches (or the same captured graph) serve every step.
int decode_step(echo_ctx *ctx, const WeightBuf &w, const Plan &pl, const int32_t *tok_hist, float temperature,
                uint64_t seed, const int32_t *forced, int32_t *out_tokens, float *out_logprobs, int rows) {
  // rows: activation rows of this step's projections.  Without an end token: all P*G sequences.  With
  // one (ctx->compact): the preparation kernel packs the sequences that have not ended to the front,
  // and `rows` is an upper bound of their number that the host knows (see rollout_impl).
  const Layout &lo = ctx->lo;
  int32_t *d_step = ctx->ptr<int32_t>(lo.d_step);
  int32_t *row_tok = ctx->ptr<int32_t>(lo.dec_row_tok);
  int32_t *row_pos = ctx->ptr<int32_t>(lo.dec_row_pos);
  ProfScope prof_step(ctx, PROF_STEP);
  int32_t *row_done = (ctx->cfg.eos_id >= 0 || ctx->compact) ? ctx->ptr<int32_t>(lo.row_done) : nullptr;
  CompactRows crs{ctx->ptr<int32_t>(lo.row_seq), ctx->ptr<int32_t>(lo.seq_row), ctx->ptr<int32_t>(lo.seq_pos),
                  ctx->ptr<int32_t>(lo.n_live)};
  if (ctx->queue_mode) {
    crs.seq_gid = ctx->ptr<int32_t>(lo.seq_gid);
    crs.seq_t0 = ctx->ptr<int32_t>(lo.seq_t0);
  }
  const CompactRows *cr = ctx->compact ? &crs : nullptr;
  LAUNCH(decode_prep_launch(d_step, tok_hist, pl.T, ctx->ptr<int32_t>(lo.seq_len0), row_tok, row_pos, pl.B,
                            ctx->stream, ctx->cfg.eos_id, row_done, cr, out_tokens, out_logprobs));
  LAUNCH(embed_launch(w.embed, row_tok, nullptr, ctx->ptr<float>(lo.x), rows, ctx->D.d, ctx->D.V,
                      ctx->ptr<int>(lo.status), ctx->stream));
  // page-table row of an activation row: its sequence id (compacted: row_seq, -1 for padding rows)
  RowMeta meta{cr ? cr->row_seq : ctx->ptr<int32_t>(lo.dec_row_pt), row_pos, cr ? nullptr : row_done};
  ctx->cap_decode = true;
  const int rc_layers = forward_layers(ctx, w, rows, meta, pl.P, pl.G, cr);
  ctx->cap_decode = false;
  TRY(rc_layers);
  TRY(lm_head(ctx, w, ctx->ptr<float>(lo.x), rows));
  {
    ProfScope prof(ctx, PROF_SAMPLER);
    const uint2 *cut = nullptr;
    if (ctx->cfg.top_p > 0.f && ctx->cfg.top_p < 1.f) {
      LAUNCH(nucleus_cut_launch(ctx->ptr<float>(lo.logits), rows, ctx->D.V, temperature, ctx->cfg.top_p,
                                ctx->ptr<uint2>(lo.nucleus_cut), ctx->stream));
      cut = ctx->ptr<uint2>(lo.nucleus_cut);
    }
    LAUNCH(sampler_launch(ctx->ptr<float>(lo.logits), rows, ctx->D.V, 1, nullptr, d_step, 0, temperature, seed,
                          forced, pl.T, out_tokens, out_logprobs, pl.T, ctx->stream, ctx->cfg.eos_id, cut,
                          cr ? nullptr : row_done, ctx->seq_base, cr ? cr->row_seq : nullptr, crs.seq_gid, crs.seq_t0));
  }
  return ECHO_OK;
}

// Prompt prefill of a planned rollout: every prompt once, in chunks of ctx->chunk_rows tokens; leaves
// each prompt's last residual row in xlast and the private copies of partial prompt pages in place.
int run_prefill(echo_ctx *ctx, const WeightBuf &w, const Plan &pl, const int32_t *prompts) {
  const Layout &lo = ctx->lo;
  const Dims &D = ctx->D;
  float *x = ctx->ptr<float>(lo.x);
  int *status = ctx->ptr<int>(lo.status);
  for (int c = 0; c < pl.n_chunks; ++c) {
    const int r0 = c * ctx->chunk_rows, R = std::min(ctx->chunk_rows, pl.n_tok - r0);
    LAUNCH(embed_launch(w.embed, prompts, ctx->ptr<int32_t>(lo.pre_tok_idx) + r0, x, R, D.d, D.V, status,
                        ctx->stream));
    RowMeta meta{ctx->ptr<int32_t>(lo.pre_row_pt) + r0, ctx->ptr<int32_t>(lo.pre_row_pos) + r0, nullptr};
    ctx->cap_row0 = r0;
    TRY(forward_layers(ctx, w, R, meta));
    LAUNCH(gather_rows_launch(x, ctx->ptr<int32_t>(lo.gather_map) + static_cast<size_t>(c) * pl.P,
                              ctx->ptr<float>(lo.xlast), pl.P, D.d, ctx->stream));
  }
  if (pl.n_copies) {
    LAUNCH(copy_partial_pages_launch(ctx->ptr<__nv_bfloat16>(lo.kv), ctx->ptr<int32_t>(lo.copy_src),
                                     ctx->ptr<int32_t>(lo.copy_dst), pl.n_copies, D.L, lo.kv_layer_elems,
                                     D.Hkv * 2 * D.Z * D.hd, ctx->stream));
  }
  return ECHO_OK;
}

int rollout_impl(echo_ctx *ctx, const int32_t *prompts, const int32_t *prompt_lens, int P, int G, int T,
                 float temperature, uint64_t seed, const int32_t *forced, int32_t *out_tokens, float *out_logprobs,
                 int64_t *out_versions) {
  if (!ctx || !prompts || !prompt_lens || !out_tokens || !out_logprobs || !out_versions) return ECHO_ERR_INVALID;
  const Limits &M = ctx->M;
  if (P < 1 || P > M.P || G < 1 || G > M.G || T < 1 || T > M.T) return ECHO_ERR_INVALID;
  if (!(temperature > 0.f) || !std::isfinite(temperature)) return ECHO_ERR_INVALID;
  for (int p = 0; p < P; ++p)
    if (prompt_lens[p] < 1 || prompt_lens[p] > M.Lp) return ECHO_ERR_INVALID;
  DeviceGuard guard(ctx->device);

  int rc;
  WeightBuf *wp = begin_rollout_version(ctx, &rc);
  if (!wp) return rc;
  const WeightBuf &w = *wp;
  for (int i = 0; i < P * G; ++i) out_versions[i] = w.version;

  if (ctx->plan_in_flight) {       // the staging block is still being read by an earlier upload
    CK(cudaEventSynchronize(ctx->plan_done));
    ctx->plan_in_flight = false;
  }
  Plan pl;
  TRY(build_plan(ctx, prompt_lens, P, G, T, &pl));
  TRY(upload_plan(ctx, pl));

  const Layout &lo = ctx->lo;
  const Dims &D = ctx->D;
  const int64_t launches0 = ctx->launches;
  float *x = ctx->ptr<float>(lo.x);
  int *status = ctx->ptr<int>(lo.status);

  CK(cudaEventRecord(ctx->ev_begin, ctx->stream));
  ctx->prof_recs.clear();
  ctx->prof_pool_used = 0;
  if (ctx->prof_every < 0) {      // per-kernel-class timing of the prefill, reported as step 0
    ctx->prof_now = true;
    ctx->prof_step = 0;
  }
  if (ctx->cfg.eos_id >= 0)       // no sequence has ended yet
    CK(cudaMemsetAsync(ctx->arena + lo.row_done, 0, static_cast<size_t>(pl.B) * 4, ctx->stream));
  if (ctx->compact)               // padding rows of a compacted step are read by the output projection: keep them finite
    CK(cudaMemsetAsync(ctx->arena + lo.attn, 0, static_cast<size_t>(pl.B) * D.Hq * D.hd * 2, ctx->stream));
  // ---- prefill: once per prompt, in chunks of ctx->chunk_rows tokens --------
  cudaEvent_t pf_a = nullptr, pf_b = nullptr;
  if (ctx->prof_now && (pf_a = prof_event(ctx)) && (pf_b = prof_event(ctx))) cudaEventRecord(pf_a, ctx->stream);
  TRY(run_prefill(ctx, w, pl, prompts));
  // ---- first token of every sample from the prompt's last logits row --------
  TRY(lm_head(ctx, w, ctx->ptr<float>(lo.xlast), P));
  LAUNCH(set_int_launch(ctx->ptr<int32_t>(lo.d_step), 0, ctx->stream));
  const uint2 *cut0 = nullptr;
  if (ctx->cfg.top_p > 0.f && ctx->cfg.top_p < 1.f) {
    LAUNCH(nucleus_cut_launch(ctx->ptr<float>(lo.logits), P, D.V, temperature, ctx->cfg.top_p,
                              ctx->ptr<uint2>(lo.nucleus_cut), ctx->stream));
    cut0 = ctx->ptr<uint2>(lo.nucleus_cut);
  }
  LAUNCH(sampler_launch(ctx->ptr<float>(lo.logits), pl.B, D.V, G, nullptr, nullptr, 0, temperature, seed, forced, T,
                        out_tokens, out_logprobs, T, ctx->stream, ctx->cfg.eos_id, cut0, nullptr, ctx->seq_base));

  if (pf_a && pf_b) {
    cudaEventRecord(pf_b, ctx->stream);
    ctx->prof_recs.push_back({0, PROF_STEP, pf_a, pf_b});
  }
  ctx->prof_now = false;
  CK(cudaEventRecord(ctx->ev_first, ctx->stream));
  // ---- decode steps 1..T-1 ----------------------------------------------------
  const int32_t *tok_hist = forced ? forced : out_tokens;
  const int n_steps = T - 1;
  // Captures of the same step.  They differ in the suffix attention kernel: resident CTAs while the
  // sequences hold few generated tokens (their fixed cost per item is what counts), one CTA per
  // (sequence, kv head) from kLongSuffix generated tokens on (the launch is bound by the KV stream);
  // and, with an end token, in the number of activation rows: the projections' cost falls in steps
  // (more than 128 rows, 65-128, 33-64, up to 32), so there is one capture per such row count below
  // the batch size.  Captured when first needed.
  std::vector<int> buckets{pl.B};
  if (ctx->compact)
    for (int m : {128, 64, 32})
      if (m < pl.B) buckets.push_back(m);
  const int n_b = static_cast<int>(buckets.size());
  std::vector<cudaGraph_t> graph(2 * n_b, nullptr);
  std::vector<cudaGraphExec_t> exec(2 * n_b, nullptr);
  std::vector<char> tried(2 * n_b, 0);
  std::vector<int64_t> per_step(2 * n_b, 0);
  const bool graphs_ok = n_steps > 1 && ctx->use_graph && ctx->stream != nullptr;
  auto release_graphs = [&]() {
    for (size_t u = 0; u < exec.size(); ++u) {
      if (exec[u]) cudaGraphExecDestroy(exec[u]);      // executions already enqueued keep their resources
      if (graph[u]) cudaGraphDestroy(graph[u]);
    }
  };
  auto capture = [&](int v, int bi) -> int {
    const int u = v * n_b + bi;
    tried[u] = 1;
    const int64_t before = ctx->launches;
    if (cudaStreamBeginCapture(ctx->stream, cudaStreamCaptureModeThreadLocal) != cudaSuccess) {
      cudaGetLastError();
      return ECHO_OK;
    }
    ctx->long_suffix = v == 1;
    const int src = decode_step(ctx, w, pl, tok_hist, temperature, seed, forced, out_tokens, out_logprobs, buckets[bi]);
    ctx->long_suffix = false;
    cudaError_t e = cudaStreamEndCapture(ctx->stream, &graph[u]);
    per_step[u] = ctx->launches - before;
    ctx->launches = before;
    if (src != ECHO_OK) return src;
    if (e != cudaSuccess || cudaGraphInstantiate(&exec[u], graph[u], 0) != cudaSuccess) {
      cudaGetLastError();
      exec[u] = nullptr;
    }
    return ECHO_OK;
  };
  // Live rows (compaction): the preparation kernel of every step leaves the number of sequences that
  // have not ended in device memory; at the end of each window of kLiveWindow steps it is copied to
  // page-locked host memory, and the host reads the value of window w - 2 before it enqueues window w.
  // The count never rises during a rollout, so an older value is an upper bound of the current one.
  constexpr int kLiveWindow = 32;
  int live_bound = pl.B, bi = 0;
  int rc_steps = ECHO_OK;
  for (int j = 1; j <= n_steps && rc_steps == ECHO_OK; ++j) {
    if (ctx->compact && (j - 1) % kLiveWindow == 0) {
      const int wdw = (j - 1) / kLiveWindow;
      if (wdw >= 2) {
        cudaError_t se = cudaEventSynchronize(ctx->live_ev[(wdw - 2) % 3]);
        if (se != cudaSuccess) {
          rc_steps = fail_cuda(ctx, se, "cudaEventSynchronize(live rows)");
          break;
        }
        live_bound = std::min(live_bound, static_cast<int>(ctx->h_live[(wdw - 2) % 3]));
        bi = 0;
        for (int k = 1; k < n_b; ++k)
          if (buckets[k] >= live_bound) bi = k;          // buckets fall: the last one that still holds every live row
      }
    }
    const bool sampled = ctx->prof_every > 0 && (j % ctx->prof_every == 0);
    const int v = j >= kLongSuffix ? 1 : 0;
    const int u = v * n_b + bi;
    if (graphs_ok && !sampled && !tried[u]) rc_steps = capture(v, bi);
    if (rc_steps != ECHO_OK) break;
    if (exec[u] && !sampled) {
      cudaError_t le = cudaGraphLaunch(exec[u], ctx->stream);
      if (le != cudaSuccess) rc_steps = fail_cuda(ctx, le, "cudaGraphLaunch");
      ctx->launches += per_step[u];
    } else {
      ctx->prof_now = sampled;
      ctx->prof_step = j;
      ctx->long_suffix = v == 1;
      rc_steps = decode_step(ctx, w, pl, tok_hist, temperature, seed, forced, out_tokens, out_logprobs, buckets[bi]);
      ctx->long_suffix = false;
      ctx->prof_now = false;
    }
    if (ctx->compact && rc_steps == ECHO_OK && (j % kLiveWindow == 0) && j < n_steps) {
      const int wdw = j / kLiveWindow - 1;               // the window that just ended
      cudaError_t ce = cudaMemcpyAsync(&ctx->h_live[wdw % 3], ctx->arena + lo.n_live, 4, cudaMemcpyDeviceToHost,
                                       ctx->stream);
      if (ce == cudaSuccess) ce = cudaEventRecord(ctx->live_ev[wdw % 3], ctx->stream);
      if (ce != cudaSuccess) rc_steps = fail_cuda(ctx, ce, "live rows readback");
    }
  }
  release_graphs();
  ctx->stats.last_step_rows = static_cast<float>(buckets[bi]);
  if (rc_steps != ECHO_OK) return rc_steps;
  CK(cudaEventRecord(ctx->ev_end, ctx->stream));
  CK(cudaEventRecord(wp->last_use, ctx->stream));
  wp->used = true;
  ctx->stats.prefill_ms = ctx->stats.decode_ms = 0.f;

  ctx->stats.version_served = w.version;
  ctx->stats.tokens_generated = static_cast<int64_t>(pl.B) * T;
  ctx->stats.kernels_launched = ctx->launches - launches0;
  ctx->stats.decode_steps = n_steps;
  ctx->stats.n_pages = pl.n_pages;
  return ECHO_OK;
}


// ---- rollout over a prompt queue ---------------------------------------------------------------
// The context's max_prompts groups are SLOTS: a slot holds one prompt and its G samples.  KV pages come
// from a pool the host keeps: a group takes the pages of its prompt and of every sample's longest
// possible continuation when it is admitted, a sample's pages go back when the host has seen it ended,
// the prompt's when all samples have.  A group is admitted between two decode steps when a slot is free,
// the pool holds its pages and the live sequences stay within the configured number.  A sequence keeps
// the noise stream and the output row of its id (prompt index * G + g) and counts its tokens from the
// step it was admitted at, so its tokens do not depend on the slot or the moment it ran.  The host
// learns which sequences have ended from the ended flags, read every kQueueWindow steps.
constexpr int kQueueWindow = 16;

struct AdmitPlan {
  int n_new, n_tok, n_chunks, n_copies;
};

// Host plan for admitting prompts `which[i]` into slots `slots[i]` (i < n_new): the slots' page-table
// rows in the host mirror, the prefill row lists, the copies of partial prompt pages and the admit lists.
struct SlotPages {
  std::vector<int> prefix;                   // pages of the prompt (the last one may be partly filled)
  std::vector<std::vector<int>> sample;      // per sample: its own pages, in order
};

AdmitPlan plan_admit(echo_ctx *ctx, const int32_t *lens, int S, int G, int T, const std::vector<int> &slots,
                     const std::vector<int> &which, const std::vector<SlotPages> &pages) {
  const Limits &M = ctx->M;
  const int Z = ctx->D.Z, W = M.pt_width;
  int32_t *h_pt = ctx->h_tables;
  int32_t *h_row_pt = h_pt + static_cast<size_t>(M.B + M.P) * W;
  int32_t *h_row_pos = h_row_pt + static_cast<size_t>(M.P) * M.Lp;
  int32_t *h_tok_idx = h_row_pos + static_cast<size_t>(M.P) * M.Lp;
  int32_t *h_gather = h_tok_idx + static_cast<size_t>(M.P) * M.Lp;
  int32_t *h_dec_pt = h_gather + static_cast<size_t>(ctx->lo.n_chunks_max) * M.P;
  int32_t *h_len0 = h_dec_pt + M.B;
  int32_t *h_full = h_len0 + M.B;
  int32_t *h_csrc = h_full + M.B;
  int32_t *h_cdst = h_csrc + M.B;
  int32_t *h_admit_seq = ctx->h_queue, *h_admit_gid = ctx->h_queue + M.B;
  const int n_new = static_cast<int>(slots.size());
  AdmitPlan ap{n_new, 0, 0, 0};
  for (int i = 0; i < n_new; ++i) ap.n_tok += lens[which[i]];
  const int chunk = ctx->chunk_rows;
  ap.n_chunks = ceil_div(ap.n_tok, chunk);
  std::fill(h_gather, h_gather + static_cast<size_t>(ap.n_chunks) * n_new, -1);
  int row = 0;
  for (int i = 0; i < n_new; ++i) {
    const int slot = slots[i], p = which[i], len = lens[p];
    const int full = len / Z, n_pre = ceil_div(len, Z), n_dec = ceil_div(len + T - 1, Z) - full;
    const SlotPages &sp = pages[slot];
    int32_t *pre_row = h_pt + static_cast<size_t>(S * G + slot) * W;
    std::fill(pre_row, pre_row + W, -1);
    for (int qi = 0; qi < n_pre; ++qi) pre_row[qi] = sp.prefix[qi];
    for (int g = 0; g < G; ++g) {
      const int b = slot * G + g;
      int32_t *r = h_pt + static_cast<size_t>(b) * W;
      std::fill(r, r + W, -1);
      for (int qi = 0; qi < full; ++qi) r[qi] = sp.prefix[qi];
      const int n_own = std::min(n_dec, static_cast<int>(sp.sample[g].size()));   // pages handed out so far
      for (int qi = 0; qi < n_own; ++qi) r[full + qi] = sp.sample[g][qi];
      if (n_pre > full && n_own > 0) {          // partial last prompt page: private copy per sample
        h_csrc[ap.n_copies] = sp.prefix[full];
        h_cdst[ap.n_copies] = sp.sample[g][0];
        ++ap.n_copies;
      }
      h_len0[b] = len;
      h_full[b] = full;
      h_admit_seq[i * G + g] = b;
      h_admit_gid[i * G + g] = p * G + g;
    }
    for (int t = 0; t < len; ++t, ++row) {
      h_row_pt[row] = S * G + slot;
      h_row_pos[row] = t;
      h_tok_idx[row] = p * M.Lp + t;
    }
    const int last = row - 1;
    h_gather[static_cast<size_t>(last / chunk) * n_new + i] = last % chunk;
  }
  return ap;
}

int rollout_queue_impl(echo_ctx *ctx, const int32_t *prompts, const int32_t *prompt_lens, int Pq, int G, int T,
                       float temperature, uint64_t seed, const int32_t *forced, int32_t *out_tokens,
                       float *out_logprobs, int64_t *out_versions) {
  if (!ctx || !prompts || !prompt_lens || !out_tokens || !out_logprobs || !out_versions) return ECHO_ERR_INVALID;
  const Limits &M = ctx->M;
  if (Pq < 1 || G < 1 || G > M.G || T < 1 || T > M.T) return ECHO_ERR_INVALID;
  if (static_cast<long long>(Pq) * G > (1ll << 30) / T) return ECHO_ERR_INVALID;
  if (!(temperature > 0.f) || !std::isfinite(temperature)) return ECHO_ERR_INVALID;
  for (int p = 0; p < Pq; ++p)
    if (prompt_lens[p] < 1 || prompt_lens[p] > M.Lp) return ECHO_ERR_INVALID;
  if (!ctx->fast_decode) return ECHO_ERR_UNSUPPORTED;
  DeviceGuard guard(ctx->device);

  int rc;
  WeightBuf *wp = begin_rollout_version(ctx, &rc);
  if (!wp) return rc;
  const WeightBuf &w = *wp;
  for (long long i = 0; i < static_cast<long long>(Pq) * G; ++i) out_versions[i] = w.version;

  const Layout &lo = ctx->lo;
  const Dims &D = ctx->D;
  const int S = std::min(M.P, Pq), B = S * G, W = M.pt_width;
  const int eos = ctx->cfg.eos_id;
  const int64_t launches0 = ctx->launches;
  Plan pl{S, G, T, B, 0, 0, 0, 0, W};
  struct ModeGuard {                  // the step enqueued below packs its rows whatever the context's setting
    echo_ctx *c;
    bool compact0;
    ModeGuard(echo_ctx *cc) : c(cc), compact0(cc->compact) { c->compact = true; c->queue_mode = true; }
    ~ModeGuard() { c->compact = compact0; c->queue_mode = false; }
  } mode_guard(ctx);

  int32_t *d_step = ctx->ptr<int32_t>(lo.d_step);
  int32_t *row_done = ctx->ptr<int32_t>(lo.row_done);
  int32_t *seq_gid = ctx->ptr<int32_t>(lo.seq_gid), *seq_t0 = ctx->ptr<int32_t>(lo.seq_t0);
  CK(cudaEventRecord(ctx->ev_begin, ctx->stream));
  ctx->prof_recs.clear();
  ctx->prof_pool_used = 0;
  CK(cudaMemsetAsync(row_done, 0xff, static_cast<size_t>(B) * 4, ctx->stream));        // every slot empty
  CK(cudaMemsetAsync(seq_gid, 0xff, static_cast<size_t>(B) * 4, ctx->stream));
  CK(cudaMemsetAsync(seq_t0, 0, static_cast<size_t>(B) * 4, ctx->stream));
  CK(cudaMemsetAsync(ctx->arena + lo.attn, 0, static_cast<size_t>(B) * D.Hq * D.hd * 2, ctx->stream));
  LAUNCH(set_int_launch(d_step, 0, ctx->stream));
  if (ctx->plan_in_flight) {
    CK(cudaEventSynchronize(ctx->plan_done));
    ctx->plan_in_flight = false;
  }
  std::fill(ctx->h_tables, ctx->h_tables + static_cast<size_t>(M.B + M.P) * W, -1);
  {
    // slots that hold nothing yet: no prompt pages, length 0 (the prefix launch walks every slot's group)
    int32_t *h_len0 = ctx->h_tables + static_cast<size_t>(M.B + M.P) * W + 3 * static_cast<size_t>(M.P) * M.Lp +
                      static_cast<size_t>(lo.n_chunks_max) * M.P + M.B;
    std::fill(h_len0, h_len0 + 2 * static_cast<size_t>(M.B), 0);          // prompt lengths, then full prompt pages
  }
  ctx->last_rows = 0;

  const int32_t *tok_hist = forced ? forced : out_tokens;
  std::vector<int> slot_admit(S, -1);      // step after which the slot's current prompt was admitted; -1: empty
  std::vector<int> slot_live(S, 0);        // upper bound of the slot's sequences that have not ended
  std::vector<int> slot_prompt(S, -1);     // the prompt a slot holds
  std::deque<int> pending;                 // prompts not admitted yet (an evicted group's prompt returns to the head)
  for (int p = 0; p < Pq; ++p) pending.push_back(p);
  int j = 0, n_admits = 0;
  int64_t n_evictions = 0;
  const bool optimistic = ctx->cfg.queue_optimistic != 0;
  // the page pool (host side): free pages as a stack, the pages each slot holds, the peak in use
  const int Z = D.Z;
  std::vector<int> free_pages(M.n_pages);
  for (int i = 0; i < M.n_pages; ++i) free_pages[i] = M.n_pages - 1 - i;
  std::vector<SlotPages> slot_pages(S);
  int pages_peak = 0;
  // own pages of a sample whose prompt has `len` tokens once it may write positions below len + n
  // (n <= T - 1 tokens fed back); a partly filled last prompt page counts, it is copied per sample
  auto own_pages = [&](int len, int n) { return ceil_div(len + std::min(n, T - 1), Z) - len / Z; };
  // tokens a group admitted after step `adm` may have fed back by the window boundary that follows step `now`
  auto fed_by_next_boundary = [&](int adm, int now) { return (now / kQueueWindow + 1) * kQueueWindow - adm; };
  // pages a group takes when it is admitted after step `now`: everything it can ever need, or (optimistic)
  // what it needs up to the next boundary
  auto pages_of = [&](int len, int now) {
    return ceil_div(len, Z) + G * own_pages(len, optimistic ? fed_by_next_boundary(now, now) : T - 1);
  };
  std::vector<std::vector<char>> released(S, std::vector<char>(G, 1));
  auto take_pages = [&](int n, std::vector<int> &dst) {
    dst.assign(free_pages.end() - n, free_pages.end());
    std::reverse(dst.begin(), dst.end());
    free_pages.resize(free_pages.size() - n);
  };
  auto give_pages = [&](std::vector<int> &src) {
    free_pages.insert(free_pages.end(), src.rbegin(), src.rend());
    src.clear();
  };
  // a sample of a slot has ended (the host has seen its flag, or its length is reached): its pages
  // return to the pool; with the last sample the prompt's pages and the slot itself
  auto release_sample = [&](int slot, int g) {
    if (!slot_pages[slot].sample[g].empty()) give_pages(slot_pages[slot].sample[g]);
    released[slot][g] = 1;
  };
  auto release_slot = [&](int slot) {
    for (int g = 0; g < G; ++g) release_sample(slot, g);
    give_pages(slot_pages[slot].prefix);
    slot_admit[slot] = -1;
    slot_live[slot] = 0;
    slot_prompt[slot] = -1;
  };

  auto admit = [&](const std::vector<int> &slots) -> int {
    std::vector<int> which;
    for (size_t i = 0; i < slots.size(); ++i) {
      const int p = pending.front(), len = prompt_lens[p];
      pending.pop_front();
      which.push_back(p);
      SlotPages &sp = slot_pages[slots[i]];
      take_pages(ceil_div(len, Z), sp.prefix);
      sp.sample.assign(G, std::vector<int>());
      const int n_own = own_pages(len, optimistic ? fed_by_next_boundary(j, j) : T - 1);
      for (int g = 0; g < G; ++g) take_pages(n_own, sp.sample[g]);
      slot_prompt[slots[i]] = p;
      std::fill(released[slots[i]].begin(), released[slots[i]].end(), 0);
    }
    pages_peak = std::max(pages_peak, M.n_pages - static_cast<int>(free_pages.size()));
    if (ctx->plan_in_flight) {             // the staging block may still be read by the previous upload
      CK(cudaEventSynchronize(ctx->plan_done));
      ctx->plan_in_flight = false;
    }
    const AdmitPlan ap = plan_admit(ctx, prompt_lens, S, G, T, slots, which, slot_pages);
    const size_t npt = static_cast<size_t>(M.P) * M.Lp;
    const int32_t *h = ctx->h_tables;
    size_t o = 0;
    auto up = [&](size_t dev_off, size_t cap_ints, size_t n_ints) -> cudaError_t {
      cudaError_t e = cudaSuccess;
      if (n_ints) e = cudaMemcpyAsync(ctx->arena + dev_off, h + o, n_ints * 4, cudaMemcpyHostToDevice, ctx->stream);
      o += cap_ints;
      return e;
    };
    CK(up(lo.page_table, static_cast<size_t>(M.B + M.P) * W, static_cast<size_t>(B + S) * W));
    CK(up(lo.pre_row_pt, npt, ap.n_tok));
    CK(up(lo.pre_row_pos, npt, ap.n_tok));
    CK(up(lo.pre_tok_idx, npt, ap.n_tok));
    CK(up(lo.gather_map, static_cast<size_t>(lo.n_chunks_max) * M.P, static_cast<size_t>(ap.n_chunks) * ap.n_new));
    CK(up(lo.dec_row_pt, M.B, 0));
    CK(up(lo.seq_len0, M.B, B));
    CK(up(lo.full_pages, M.B, B));
    CK(up(lo.copy_src, M.B, ap.n_copies));
    CK(up(lo.copy_dst, M.B, ap.n_copies));
    const int n_seq = ap.n_new * G;
    CK(cudaMemcpyAsync(ctx->arena + lo.admit_seq, ctx->h_queue, static_cast<size_t>(n_seq) * 4, cudaMemcpyHostToDevice,
                       ctx->stream));
    CK(cudaMemcpyAsync(ctx->arena + lo.admit_gid, ctx->h_queue + M.B, static_cast<size_t>(n_seq) * 4,
                       cudaMemcpyHostToDevice, ctx->stream));
    CK(cudaEventRecord(ctx->plan_done, ctx->stream));
    ctx->plan_in_flight = true;
    LAUNCH(admit_launch(n_seq, ctx->ptr<int32_t>(lo.admit_seq), ctx->ptr<int32_t>(lo.admit_gid), d_step, seq_gid, seq_t0,
                        row_done, out_tokens, out_logprobs, T, eos, ctx->stream));
    // prefill of the admitted prompts, then token 0 of each of their samples
    const Plan apl{ap.n_new, G, T, n_seq, ap.n_tok, ap.n_chunks, ap.n_copies, M.n_pages, W};
    TRY(run_prefill(ctx, w, apl, prompts));
    TRY(lm_head(ctx, w, ctx->ptr<float>(lo.xlast), ap.n_new));
    const uint2 *cut0 = nullptr;
    if (ctx->cfg.top_p > 0.f && ctx->cfg.top_p < 1.f) {
      LAUNCH(nucleus_cut_launch(ctx->ptr<float>(lo.logits), ap.n_new, D.V, temperature, ctx->cfg.top_p,
                                ctx->ptr<uint2>(lo.nucleus_cut), ctx->stream));
      cut0 = ctx->ptr<uint2>(lo.nucleus_cut);
    }
    LAUNCH(sampler_launch(ctx->ptr<float>(lo.logits), n_seq, D.V, G, nullptr, d_step, 0, temperature, seed, forced, T,
                          out_tokens, out_logprobs, T, ctx->stream, eos, cut0, nullptr, ctx->seq_base,
                          ctx->ptr<int32_t>(lo.admit_seq), seq_gid, seq_t0));
    for (size_t i = 0; i < slots.size(); ++i) {
      slot_admit[slots[i]] = j;
      slot_live[slots[i]] = G;
    }
    ++n_admits;
    return ECHO_OK;
  };

  // graphs of the decode step per (suffix kernel, row count), captured when first needed; row counts:
  // all slots, the multiples of 128 below, 64 and 32
  std::vector<int> buckets{B};
  for (int m = (B - 1) / 128 * 128; m >= 128; m -= 128) buckets.push_back(m);
  for (int m : {64, 32})
    if (m < B) buckets.push_back(m);
  const int n_b = static_cast<int>(buckets.size());
  std::vector<cudaGraph_t> graph(2 * n_b, nullptr);
  std::vector<cudaGraphExec_t> exec(2 * n_b, nullptr);
  std::vector<char> tried(2 * n_b, 0);
  std::vector<int64_t> per_step(2 * n_b, 0);
  const bool graphs_ok = ctx->use_graph && ctx->stream != nullptr;
  auto release_graphs = [&]() {
    for (size_t u = 0; u < exec.size(); ++u) {
      if (exec[u]) cudaGraphExecDestroy(exec[u]);
      if (graph[u]) cudaGraphDestroy(graph[u]);
    }
  };
  auto capture = [&](int v, int bi) -> int {
    const int u = v * n_b + bi;
    tried[u] = 1;
    const int64_t before = ctx->launches;
    if (cudaStreamBeginCapture(ctx->stream, cudaStreamCaptureModeThreadLocal) != cudaSuccess) {
      cudaGetLastError();
      return ECHO_OK;
    }
    ctx->long_suffix = v == 1;
    const int src = decode_step(ctx, w, pl, tok_hist, temperature, seed, forced, out_tokens, out_logprobs, buckets[bi]);
    ctx->long_suffix = false;
    cudaError_t e = cudaStreamEndCapture(ctx->stream, &graph[u]);
    per_step[u] = ctx->launches - before;
    ctx->launches = before;
    if (src != ECHO_OK) return src;
    if (e != cudaSuccess || cudaGraphInstantiate(&exec[u], graph[u], 0) != cudaSuccess) {
      cudaGetLastError();
      exec[u] = nullptr;
    }
    return ECHO_OK;
  };

  int32_t *h_snap = ctx->h_queue + 2 * static_cast<size_t>(M.B);
  int bi = 0;
  int rc_steps = ECHO_OK;
  // a slot's sequences have all ended, as far as the host can know: by length, or by the flags of a
  // snapshot taken after the slot's admission
  auto by_length = [&](int slot) { return slot_admit[slot] >= 0 && j >= slot_admit[slot] + T - 1; };
  auto live_bound = [&]() {
    int n = 0;
    for (int sl = 0; sl < S; ++sl) n += slot_admit[sl] < 0 ? 0 : slot_live[sl];
    return n;
  };
  const int max_live = ctx->cfg.queue_max_live > 0 ? std::max(ctx->cfg.queue_max_live, G) : B;
  // Groups of the queue, in order, into free slots while pages and live rows allow.  A group that fits
  // an empty pool always exists (the pool holds at least one group at full length), so the queue drains.
  auto refill = [&]() -> int {
    for (int sl = 0; sl < S; ++sl)
      if (by_length(sl)) release_slot(sl);    // every sample has all its T tokens
    std::vector<int> slots;
    int need = 0, rows = live_bound();
    for (int sl = 0; sl < S && slots.size() < pending.size(); ++sl) {
      if (slot_admit[sl] >= 0) continue;
      const int p = pending[slots.size()];
      const int pg = pages_of(prompt_lens[p], j);
      // optimistic: keep queue_optimistic - 1 windows' worth of growth of everything live in hand (a page
      // per sequence and window), unless nothing is resident at all
      const int margin = optimistic && rows > 0 ? (ctx->cfg.queue_optimistic - 1) * (rows + G) : 0;
      if (need + pg + margin > static_cast<int>(free_pages.size()) || rows + G > max_live) break;
      need += pg;
      rows += G;
      slots.push_back(sl);
    }
    return slots.empty() ? ECHO_OK : admit(slots);
  };
  // Optimistic mode, at a window boundary: every live sample gets the pages for the positions it reaches
  // by the next boundary.  If the pool cannot cover that, the most recently admitted groups are evicted
  // (their prompts return to the head of the queue; the pool holds one group at full length, so the
  // oldest group always gets through).
  auto extend = [&]() -> int {
    auto wanted = [&](int sl) {
      return own_pages(prompt_lens[slot_prompt[sl]], fed_by_next_boundary(slot_admit[sl], j));
    };
    auto missing = [&](int sl) {
      const int want = wanted(sl);
      int m = 0;
      for (int g = 0; g < G; ++g)
        if (!released[sl][g]) m += std::max(0, want - static_cast<int>(slot_pages[sl].sample[g].size()));
      return m;
    };
    int need = 0;
    for (int sl = 0; sl < S; ++sl)
      if (slot_admit[sl] >= 0) need += missing(sl);
    std::vector<int> evicted;
    while (need > static_cast<int>(free_pages.size())) {
      int victim = -1;
      for (int sl = 0; sl < S; ++sl)
        if (slot_admit[sl] >= 0 && (victim < 0 || slot_admit[sl] >= slot_admit[victim])) victim = sl;
      if (victim < 0) return ECHO_ERR_INVALID;          // cannot happen: see above
      need -= missing(victim);
      pending.push_front(slot_prompt[victim]);
      release_slot(victim);
      evicted.push_back(victim);
      ++n_evictions;
    }
    if (need == 0 && evicted.empty()) return ECHO_OK;
    if (ctx->plan_in_flight) {
      CK(cudaEventSynchronize(ctx->plan_done));
      ctx->plan_in_flight = false;
    }
    int32_t *h_pt = ctx->h_tables;
    for (int sl = 0; sl < S; ++sl) {
      if (slot_admit[sl] < 0) continue;
      const int want = wanted(sl), full = prompt_lens[slot_prompt[sl]] / Z;
      for (int g = 0; g < G; ++g) {
        if (released[sl][g]) continue;
        std::vector<int> &own = slot_pages[sl].sample[g];
        int32_t *r = h_pt + static_cast<size_t>(sl * G + g) * W;
        while (static_cast<int>(own.size()) < want) {
          own.push_back(free_pages.back());
          free_pages.pop_back();
          r[full + static_cast<int>(own.size()) - 1] = own.back();
        }
      }
    }
    pages_peak = std::max(pages_peak, M.n_pages - static_cast<int>(free_pages.size()));
    CK(cudaMemcpyAsync(ctx->arena + lo.page_table, h_pt, static_cast<size_t>(B + S) * W * 4, cudaMemcpyHostToDevice,
                       ctx->stream));
    const int n_ev = static_cast<int>(evicted.size()) * G;
    if (n_ev) {
      int32_t *h_admit_seq = ctx->h_queue, *h_admit_gid = ctx->h_queue + M.B;
      for (size_t i = 0; i < evicted.size(); ++i)
        for (int g = 0; g < G; ++g) {
          h_admit_seq[i * G + g] = evicted[i] * G + g;
          h_admit_gid[i * G + g] = -2;
        }
      CK(cudaMemcpyAsync(ctx->arena + lo.admit_seq, h_admit_seq, static_cast<size_t>(n_ev) * 4, cudaMemcpyHostToDevice,
                         ctx->stream));
      CK(cudaMemcpyAsync(ctx->arena + lo.admit_gid, h_admit_gid, static_cast<size_t>(n_ev) * 4, cudaMemcpyHostToDevice,
                         ctx->stream));
    }
    CK(cudaEventRecord(ctx->plan_done, ctx->stream));
    ctx->plan_in_flight = true;
    if (n_ev)
      LAUNCH(admit_launch(n_ev, ctx->ptr<int32_t>(lo.admit_seq), ctx->ptr<int32_t>(lo.admit_gid), d_step, seq_gid, seq_t0,
                          row_done, out_tokens, out_logprobs, T, eos, ctx->stream));
    return ECHO_OK;
  };
  auto choose_rows = [&]() {                  // the smallest captured row count that holds every live sequence
    const int bound = live_bound();
    bi = 0;
    for (int k = 1; k < n_b; ++k)
      if (buckets[k] >= bound) bi = k;
  };
  bool first = true;
  for (;;) {
    if ((rc_steps = refill()) != ECHO_OK) break;
    if (first) {
      first = false;
      cudaEventRecord(ctx->ev_first, ctx->stream);
    }
    bool all_over = pending.empty();
    for (int sl = 0; sl < S && all_over; ++sl) all_over = slot_admit[sl] < 0;
    if (all_over) break;
    choose_rows();
    ++j;
    int age = 0;                             // most tokens any live slot's sequences may hold
    for (int sl = 0; sl < S; ++sl)
      if (slot_admit[sl] >= 0) age = std::max(age, j - slot_admit[sl]);
    const int v = age >= kLongSuffix ? 1 : 0;
    const int u = v * n_b + bi;
    if (graphs_ok && !tried[u]) rc_steps = capture(v, bi);
    if (rc_steps != ECHO_OK) break;
    if (exec[u]) {
      cudaError_t le = cudaGraphLaunch(exec[u], ctx->stream);
      if (le != cudaSuccess) rc_steps = fail_cuda(ctx, le, "cudaGraphLaunch");
      ctx->launches += per_step[u];
    } else {
      ctx->long_suffix = v == 1;
      rc_steps = decode_step(ctx, w, pl, tok_hist, temperature, seed, forced, out_tokens, out_logprobs, buckets[bi]);
      ctx->long_suffix = false;
    }
    if (rc_steps != ECHO_OK) break;
    if (j % kQueueWindow) continue;
    if (eos < 0) {                                       // without an end token sequences end by length only
      if (optimistic && (rc_steps = extend()) != ECHO_OK) break;
      continue;
    }
    // ---- window boundary: read the ended flags as of this step.  The host waits for the GPU here (the
    // steps it has enqueued so far), which costs one launch latency per window; what it learns decides
    // the refill and the row count of the next window.
    cudaError_t ce = cudaMemcpyAsync(h_snap, row_done, static_cast<size_t>(B) * 4, cudaMemcpyDeviceToHost, ctx->stream);
    if (ce == cudaSuccess) ce = cudaEventRecord(ctx->live_ev[0], ctx->stream);
    if (ce == cudaSuccess) ce = cudaEventSynchronize(ctx->live_ev[0]);
    if (ce != cudaSuccess) {
      rc_steps = fail_cuda(ctx, ce, "ended-flags snapshot");
      break;
    }
    for (int sl = 0; sl < S; ++sl) {
      if (slot_admit[sl] < 0 || slot_admit[sl] >= j) continue;      // nothing of the slot's prompt has run yet
      int live = 0;
      for (int g = 0; g < G; ++g) {
        if (h_snap[sl * G + g]) release_sample(sl, g);
        else ++live;
      }
      slot_live[sl] = std::min(slot_live[sl], live);
      if (slot_live[sl] == 0) release_slot(sl);
    }
    for (int sl = 0; sl < S; ++sl)
      if (by_length(sl)) release_slot(sl);
    if (optimistic && (rc_steps = extend()) != ECHO_OK) break;
  }
  release_graphs();
  if (rc_steps != ECHO_OK) return rc_steps;
  {
    // the outputs of sequences that ended before their T-th token are completed when their slot changes
    // hands; the last occupants' here
    if (ctx->plan_in_flight) {
      CK(cudaEventSynchronize(ctx->plan_done));
      ctx->plan_in_flight = false;
    }
    int32_t *h_admit_seq = ctx->h_queue, *h_admit_gid = ctx->h_queue + M.B;
    for (int b = 0; b < B; ++b) {
      h_admit_seq[b] = b;
      h_admit_gid[b] = -1;
    }
    CK(cudaMemcpyAsync(ctx->arena + lo.admit_seq, h_admit_seq, static_cast<size_t>(B) * 4, cudaMemcpyHostToDevice,
                       ctx->stream));
    CK(cudaMemcpyAsync(ctx->arena + lo.admit_gid, h_admit_gid, static_cast<size_t>(B) * 4, cudaMemcpyHostToDevice,
                       ctx->stream));
    CK(cudaEventRecord(ctx->plan_done, ctx->stream));
    ctx->plan_in_flight = true;
    LAUNCH(admit_launch(B, ctx->ptr<int32_t>(lo.admit_seq), ctx->ptr<int32_t>(lo.admit_gid), d_step, seq_gid, seq_t0,
                        row_done, out_tokens, out_logprobs, T, eos, ctx->stream));
  }
  ctx->stats.last_step_rows = static_cast<float>(buckets[bi]);
  CK(cudaEventRecord(ctx->ev_end, ctx->stream));
  CK(cudaEventRecord(wp->last_use, ctx->stream));
  wp->used = true;
  ctx->stats.prefill_ms = ctx->stats.decode_ms = 0.f;
  ctx->stats.version_served = w.version;
  ctx->stats.tokens_generated = static_cast<int64_t>(Pq) * G * T;
  ctx->stats.kernels_launched = ctx->launches - launches0;
  ctx->stats.decode_steps = j;
  ctx->stats.n_pages = pages_peak;
  ctx->stats.queue_evictions = n_evictions;
  return ECHO_OK;
}

// Teacher-forced scoring of whole trajectories in prefill-shaped passes: the prompt once per group, then
// every sequence's given tokens as rows of 2048-row chunks (sequence-major), each chunk through the
// layers with causal attention over the paged cache, the lm_head and the log-probability kernel in
// blocks of at most P*G rows (the logits buffer).
int score_impl(echo_ctx *ctx, const int32_t *prompts, const int32_t *prompt_lens, int P, int G, int T,
               float temperature, const int32_t *tokens, float *out_logprobs, int64_t *out_versions) {
  if (!ctx || !prompts || !prompt_lens || !tokens || !out_logprobs || !out_versions) return ECHO_ERR_INVALID;
  const Limits &M = ctx->M;
  if (P < 1 || P > M.P || G < 1 || G > M.G || T < 1 || T > M.T) return ECHO_ERR_INVALID;
  if (!(temperature > 0.f) || !std::isfinite(temperature)) return ECHO_ERR_INVALID;
  for (int p = 0; p < P; ++p)
    if (prompt_lens[p] < 1 || prompt_lens[p] > M.Lp) return ECHO_ERR_INVALID;
  DeviceGuard guard(ctx->device);
  int rc;
  WeightBuf *wp = begin_rollout_version(ctx, &rc);
  if (!wp) return rc;
  const WeightBuf &w = *wp;
  for (int i = 0; i < P * G; ++i) out_versions[i] = w.version;
  if (ctx->plan_in_flight) {
    CK(cudaEventSynchronize(ctx->plan_done));
    ctx->plan_in_flight = false;
  }
  Plan pl;
  TRY(build_plan(ctx, prompt_lens, P, G, T, &pl));
  TRY(upload_plan(ctx, pl));
  const Layout &lo = ctx->lo;
  const Dims &D = ctx->D;
  const int64_t launches0 = ctx->launches;
  float *x = ctx->ptr<float>(lo.x);
  int *status = ctx->ptr<int>(lo.status);
  float *logits = ctx->ptr<float>(lo.logits);
  int32_t *first_end = ctx->cfg.eos_id >= 0 ? ctx->ptr<int32_t>(lo.row_done) : nullptr;

  CK(cudaEventRecord(ctx->ev_begin, ctx->stream));
  ctx->prof_recs.clear();
  ctx->prof_pool_used = 0;
  if (first_end) LAUNCH(first_end_launch(tokens, pl.B, T, ctx->cfg.eos_id, first_end, ctx->stream));
  TRY(run_prefill(ctx, w, pl, prompts));
  // token 0 of every sample: scored on the prompt's last logits row
  TRY(lm_head(ctx, w, ctx->ptr<float>(lo.xlast), P));
  LAUNCH(logprob_rows_launch(logits, pl.B, D.V, G, temperature, tokens, nullptr, T, first_end, out_logprobs, status,
                             ctx->stream));
  CK(cudaEventRecord(ctx->ev_first, ctx->stream));
  // tokens 1..T-1: row (s, j) feeds given token j at position len0[s] + j and scores token j + 1
  const long n_rows = static_cast<long>(pl.B) * (T - 1);
  int32_t *row_pt = ctx->ptr<int32_t>(lo.pre_row_pt), *row_pos = ctx->ptr<int32_t>(lo.pre_row_pos),
          *tok_idx = ctx->ptr<int32_t>(lo.pre_tok_idx);
  for (long r0 = 0; r0 < n_rows; r0 += ctx->chunk_rows) {
    const int R = static_cast<int>(std::min<long>(ctx->chunk_rows, n_rows - r0));
    LAUNCH(score_rows_launch(static_cast<int>(r0), R, T, ctx->ptr<int32_t>(lo.seq_len0), row_pt, row_pos, tok_idx,
                             ctx->stream));
    LAUNCH(embed_launch(w.embed, tokens, tok_idx, x, R, D.d, D.V, status, ctx->stream));
    RowMeta meta{row_pt, row_pos, nullptr};
    ctx->cap_row0 = 0;
    TRY(forward_layers(ctx, w, R, meta));
    for (int sub = 0; sub < R; sub += pl.B) {
      const int rows = std::min(pl.B, R - sub);
      TRY(lm_head(ctx, w, x + static_cast<size_t>(sub) * D.d, rows));
      LAUNCH(logprob_rows_launch(logits, rows, D.V, 1, temperature, tokens, tok_idx + sub, T, first_end, out_logprobs,
                                 status, ctx->stream));
    }
  }
  CK(cudaEventRecord(ctx->ev_end, ctx->stream));
  CK(cudaEventRecord(wp->last_use, ctx->stream));
  wp->used = true;
  ctx->stats.prefill_ms = ctx->stats.decode_ms = 0.f;
  ctx->stats.version_served = w.version;
  ctx->stats.tokens_generated = static_cast<int64_t>(pl.B) * T;
  ctx->stats.kernels_launched = ctx->launches - launches0;
  ctx->stats.decode_steps = 0;
  ctx->stats.n_pages = pl.n_pages;
  return ECHO_OK;
}

}  // namespace

// ============================================================================
// C ABI
// ============================================================================
extern "C" {

size_t echo_arena_bytes(const echo_config *cfg) {
  if (!config_ok(cfg)) return 0;
  return layout_of(*cfg).total;
}

int echo_create(const echo_config *cfg, int device, void *arena, size_t arena_bytes, void *cuda_stream,
                echo_ctx **out) {
  if (!out) return ECHO_ERR_INVALID;
  *out = nullptr;
  if (!config_ok(cfg) || !arena) return ECHO_ERR_INVALID;
  Layout lo = layout_of(*cfg);
  if (arena_bytes < lo.total || (reinterpret_cast<uintptr_t>(arena) & 255)) return ECHO_ERR_ARENA;
  int n_dev = 0;
  if (cudaGetDeviceCount(&n_dev) != cudaSuccess || device < 0 || device >= n_dev) return ECHO_ERR_CUDA;
  DeviceGuard guard(device);
  echo_ctx *ctx = new (std::nothrow) echo_ctx();
  if (!ctx) return ECHO_ERR_INVALID;
  ctx->cfg = *cfg;
  ctx->D = dims_of(*cfg);
  ctx->M = limits_of(*cfg);
  ctx->lo = lo;
  ctx->device = device;
  // sub-allocations are 1 KiB-aligned relative to the base; the base's own 256-byte
  // alignment satisfies every consumer (tensor maps need 16 bytes, vector loads 16 bytes)
  ctx->arena = static_cast<uint8_t *>(arena);
  ctx->stream = static_cast<cudaStream_t>(cuda_stream);
  const char *impl = getenv("ECHO_GEMM_IMPL");
  ctx->use_simt = impl && !strcmp(impl, "simt");
  ctx->chunk_rows = ctx->use_simt ? kSmallChunkRows : kChunkRows;
  ctx->use_pair = !(impl && !strcmp(impl, "single"));
  const char *ng = getenv("ECHO_NO_GRAPH");
  ctx->use_graph = !(ng && ng[0] == '1');
  const char *det = getenv("ECHO_DETERMINISTIC");
  ctx->deterministic = det && det[0] == '1';
  const char *pdl = getenv("ECHO_NO_PDL");
  ctx->use_pdl = !(pdl && pdl[0] == '1');
  g_early_start = ctx->use_pdl;

  auto bail = [&](cudaError_t e, const char *what) {
    fail_cuda(ctx, e, what);
    fprintf(stderr, "echo_create: %s\n", ctx->last_error.c_str());
    echo_destroy(ctx);
    return ECHO_ERR_CUDA;
  };
  cudaError_t e;
  if ((e = cudaStreamCreateWithFlags(&ctx->copy_stream, cudaStreamNonBlocking)) != cudaSuccess)
    return bail(e, "cudaStreamCreate");
  for (int b = 0; b < cfg->n_weight_buffers; ++b) {
    carve_weights(ctx, ctx->wb[b], ctx->arena + lo.weights[b]);
    // the padding of the block-tiled matrices is never written again and must be zero (it meets
    // zero-filled activation columns in the MMAs); installs run on the same stream, after this
    if ((e = cudaMemsetAsync(ctx->arena + lo.weights[b], 0, lo.weight_bytes, ctx->copy_stream)) != cudaSuccess)
      return bail(e, "cudaMemset");
    if ((e = cudaEventCreate(&ctx->wb[b].installed)) != cudaSuccess) return bail(e, "cudaEventCreate");
    if ((e = cudaEventCreate(&ctx->wb[b].inst_begin)) != cudaSuccess) return bail(e, "cudaEventCreate");
    if ((e = cudaEventCreateWithFlags(&ctx->wb[b].last_use, cudaEventDisableTiming)) != cudaSuccess)
      return bail(e, "cudaEventCreate");
    if (make_weight_maps(ctx, ctx->wb[b]) != ECHO_OK) {
      fprintf(stderr, "echo_create: %s\n", ctx->last_error.c_str());
      echo_destroy(ctx);
      return ECHO_ERR_CUDA;
    }
  }
  if ((e = cudaEventCreateWithFlags(&ctx->plan_done, cudaEventDisableTiming)) != cudaSuccess)
    return bail(e, "cudaEventCreate");
  if ((e = cudaEventCreateWithFlags(&ctx->all_done, cudaEventDisableTiming)) != cudaSuccess)
    return bail(e, "cudaEventCreate");
  if ((e = cudaEventCreate(&ctx->ev_begin)) != cudaSuccess || (e = cudaEventCreate(&ctx->ev_first)) != cudaSuccess ||
      (e = cudaEventCreate(&ctx->ev_end)) != cudaSuccess)
    return bail(e, "cudaEventCreate");
  const Limits &M = ctx->M;
  ctx->h_tables_ints = static_cast<size_t>(M.B + M.P) * M.pt_width + 3ull * M.P * M.Lp +
                       static_cast<size_t>(lo.n_chunks_max) * M.P + 5ull * M.B;
  if ((e = cudaHostAlloc(reinterpret_cast<void **>(&ctx->h_tables), ctx->h_tables_ints * 4, cudaHostAllocDefault)) !=
      cudaSuccess)
    return bail(e, "cudaHostAlloc");
  if ((e = cudaHostAlloc(reinterpret_cast<void **>(&ctx->h_live), 3 * sizeof(int32_t), cudaHostAllocDefault)) !=
      cudaSuccess)
    return bail(e, "cudaHostAlloc");
  if ((e = cudaHostAlloc(reinterpret_cast<void **>(&ctx->h_queue), 5ull * M.B * sizeof(int32_t),
                         cudaHostAllocDefault)) != cudaSuccess)
    return bail(e, "cudaHostAlloc");
  for (int i = 0; i < 3; ++i)
    if ((e = cudaEventCreateWithFlags(&ctx->live_ev[i], cudaEventDisableTiming)) != cudaSuccess)
      return bail(e, "cudaEventCreate");
  if ((e = gemm_tc_configure()) != cudaSuccess) return bail(e, "cudaFuncSetAttribute");
  if ((e = gemm_pair_configure()) != cudaSuccess) return bail(e, "cudaFuncSetAttribute");
  // padding keys of a partly filled page take part in the P*V products with weight zero: the pool
  // must never hold NaN/Inf bit patterns
  if ((e = cudaMemsetAsync(ctx->arena + lo.kv, 0, lo.kv_layer_elems * ctx->D.L * 2, ctx->stream)) != cudaSuccess)
    return bail(e, "cudaMemset(kv)");
  {
    const char *na = getenv("ECHO_ATTN_IMPL");
    const char *np = getenv("ECHO_ATTN_PREFIX");
    ctx->attn_suffix_impl = na && !strcmp(na, "waves") ? 1 : 0;
    ctx->attn_prefix_impl = np && !strcmp(np, "tiles") ? 1 : 0;
    const char *npf = getenv("ECHO_ATTN_PREFILL");
    ctx->prefill_rows = npf && !strcmp(npf, "rows");
    const size_t kv_rows = lo.kv_layer_elems / ctx->D.hd * ctx->D.L;
    if (!(na && !strcmp(na, "rows")) && kv_rows < (1ull << 31) &&
        attention_decode_supported(ctx->D.hd, ctx->D.Z, ctx->D.Hq, ctx->D.Hkv)) {
      if ((e = attention_decode_configure()) != cudaSuccess) return bail(e, "cudaFuncSetAttribute(attn)");
      if (make_tensor_map(&ctx->tm_kv, ctx->arena + lo.kv, kv_rows, ctx->D.hd, ctx->D.hd, 2 * ctx->D.Z) != 0) {
        ctx->last_error = "tensor map encode failed (kv)";
        fprintf(stderr, "echo_create: %s\n", ctx->last_error.c_str());
        echo_destroy(ctx);
        return ECHO_ERR_CUDA;
      }
      ctx->fast_decode = true;
    }
  }
  {
    const char *fn = getenv("ECHO_FUSE_NORM");
    ctx->fuse_norm = fn && fn[0] == '1';
  }
  if ((e = cudaMemsetAsync(ctx->arena + lo.gemm_bar, 0, 8, ctx->stream)) != cudaSuccess) return bail(e, "cudaMemset");
  {
    const char *nc = getenv("ECHO_NO_COMPACT");
    ctx->compact = ctx->cfg.eos_id >= 0 && ctx->fast_decode && !(nc && nc[0] == '1');
  }
  if ((e = cudaMemsetAsync(ctx->arena + lo.status, 0, 4, ctx->stream)) != cudaSuccess) return bail(e, "cudaMemset");
  if ((e = cudaMemsetAsync(ctx->arena + lo.attn_work, 0, 8, ctx->stream)) != cudaSuccess) return bail(e, "cudaMemset");
  if ((e = cudaMemsetAsync(ctx->arena + lo.d_step, 0, 4, ctx->stream)) != cudaSuccess) return bail(e, "cudaMemset");
  if ((e = cudaMemsetAsync(ctx->arena + lo.qkv, 0, static_cast<size_t>(ctx->M.R) * ctx->D.n_qkv() * 4, ctx->stream)) !=
      cudaSuccess)
    return bail(e, "cudaMemset");
  if ((e = cudaMemsetAsync(ctx->arena + lo.gemm_counters, 0, static_cast<size_t>(kGemmMaxUnits) * 4, ctx->stream)) !=
      cudaSuccess)
    return bail(e, "cudaMemset");
  if ((e = rope_table_launch(ctx->ptr<float2>(lo.rope), M.max_pos, ctx->D.hd, static_cast<double>(cfg->rope_theta),
                             ctx->stream)) != cudaSuccess)
    return bail(e, "rope_table");
  *out = ctx;
  return ECHO_OK;
}

int echo_destroy(echo_ctx *ctx) {
  if (!ctx) return ECHO_ERR_INVALID;
  DeviceGuard guard(ctx->device);
  if (ctx->stream || true) cudaStreamSynchronize(ctx->stream);
  if (ctx->copy_stream) {
    cudaStreamSynchronize(ctx->copy_stream);
    cudaStreamDestroy(ctx->copy_stream);
  }
  for (int b = 0; b < 2; ++b) {
    if (ctx->wb[b].installed) cudaEventDestroy(ctx->wb[b].installed);
    if (ctx->wb[b].inst_begin) cudaEventDestroy(ctx->wb[b].inst_begin);
    if (ctx->wb[b].last_use) cudaEventDestroy(ctx->wb[b].last_use);
  }
  if (ctx->plan_done) cudaEventDestroy(ctx->plan_done);
  if (ctx->all_done) cudaEventDestroy(ctx->all_done);
  if (ctx->ev_begin) cudaEventDestroy(ctx->ev_begin);
  if (ctx->ev_first) cudaEventDestroy(ctx->ev_first);
  if (ctx->ev_end) cudaEventDestroy(ctx->ev_end);
  if (ctx->h_tables) cudaFreeHost(ctx->h_tables);
  if (ctx->h_live) cudaFreeHost(ctx->h_live);
  if (ctx->h_queue) cudaFreeHost(ctx->h_queue);
  for (int i = 0; i < 3; ++i)
    if (ctx->live_ev[i]) cudaEventDestroy(ctx->live_ev[i]);
  for (cudaEvent_t e : ctx->prof_pool) cudaEventDestroy(e);
  delete ctx;
  return ECHO_OK;
}

int echo_load_policy(echo_ctx *ctx, const echo_weights *src, int64_t version) {
  if (!ctx || !src) return ECHO_ERR_INVALID;
  if (!src->embed || !src->lm_head || !src->final_norm || !src->wq || !src->wk || !src->wv || !src->wo ||
      !src->w_gate || !src->w_up || !src->w_down || !src->attn_norm || !src->mlp_norm)
    return ECHO_ERR_INVALID;
  const Dims &D = ctx->D;
  for (int l = 0; l < D.L; ++l)
    if (!src->wq[l] || !src->wk[l] || !src->wv[l] || !src->wo[l] || !src->w_gate[l] || !src->w_up[l] ||
        !src->w_down[l] || !src->attn_norm[l] || !src->mlp_norm[l])
      return ECHO_ERR_INVALID;
  if (ctx->any_version && version <= ctx->newest_version) return ECHO_ERR_VERSION;
  if (ctx->pending >= 0) return ECHO_ERR_BUSY;
  DeviceGuard guard(ctx->device);

  int target;
  if (ctx->cfg.n_weight_buffers == 1) {
    target = 0;
  } else {
    target = ctx->active < 0 ? 0 : 1 - ctx->active;
  }
  WeightBuf &w = ctx->wb[target];
  cudaStream_t cs = ctx->copy_stream;
  // the copy may not start before every rollout that reads this buffer has finished
  if (w.used) CK(cudaStreamWaitEvent(cs, w.last_use, 0));
  if (ctx->cfg.n_weight_buffers == 1) {
    CK(cudaEventRecord(ctx->all_done, ctx->stream));
    CK(cudaStreamWaitEvent(cs, ctx->all_done, 0));
  }
  CK(cudaEventRecord(w.inst_begin, cs));
  auto cp = [&](void *dst, const void *s, size_t elems) {
    return cudaMemcpyAsync(dst, s, elems * 2, cudaMemcpyDefault, cs);
  };
  // Row-major source matrix -> rows [row0, row0 + rows) of block-tiled storage.  The re-tiling
  // kernel reads the source in place when the device can address it (device memory, page-locked
  // or managed host memory); a snapshot in pageable host memory goes through a bounce buffer.
  __nv_bfloat16 *stage = ctx->ptr<__nv_bfloat16>(ctx->lo.retile_stage);
  auto tile = [&](__nv_bfloat16 *dst, const void *s, size_t rows, size_t cols, size_t row0,
                  bool to_half) -> cudaError_t {
    cudaPointerAttributes at;
    const __nv_bfloat16 *dev_src = nullptr;
    if (cudaPointerGetAttributes(&at, s) == cudaSuccess && at.type != cudaMemoryTypeUnregistered && at.devicePointer)
      dev_src = static_cast<const __nv_bfloat16 *>(at.devicePointer);
    else
      (void)cudaGetLastError();
    if (dev_src) return retile_launch(dst, dev_src, rows, cols, row0, cs, to_half);
    const size_t chunk = kRetileStageBytes / (cols * 2);
    if (chunk == 0) return cudaErrorInvalidValue;
    for (size_t r = 0; r < rows; r += chunk) {
      const size_t n = rows - r < chunk ? rows - r : chunk;
      cudaError_t e = cudaMemcpyAsync(stage, static_cast<const __nv_bfloat16 *>(s) + r * cols, n * cols * 2,
                                      cudaMemcpyDefault, cs);
      if (e != cudaSuccess) return e;
      if ((e = retile_launch(dst, stage, n, cols, row0 + r, cs, to_half)) != cudaSuccess) return e;
    }
    return cudaSuccess;
  };
  const size_t d = D.d, qd = static_cast<size_t>(D.Hq) * D.hd, kd = static_cast<size_t>(D.Hkv) * D.hd;
  CK(cp(w.embed, src->embed, static_cast<size_t>(D.V) * d));
  CK(tile(w.lm_head, src->lm_head, D.V, d, 0, false));
  CK(cp(w.final_norm, src->final_norm, d));
  for (int l = 0; l < D.L; ++l) {
    const bool hf = l < ctx->cfg.half_layers;      // this layer's matrices are kept as IEEE half
    CK(tile(w.wqkv[l], src->wq[l], qd, d, 0, hf));
    CK(tile(w.wqkv[l], src->wk[l], kd, d, qd, hf));
    CK(tile(w.wqkv[l], src->wv[l], kd, d, qd + kd, hf));
    CK(tile(w.wo[l], src->wo[l], d, qd, 0, hf));
    CK(tile(w.wgu[l], src->w_gate[l], D.F, d, 0, hf));
    CK(tile(w.wgu[l] + tiled_elems(D.F, d), src->w_up[l], D.F, d, 0, hf));
    CK(tile(w.wdown[l], src->w_down[l], d, D.F, 0, hf));
    CK(cp(w.attn_norm[l], src->attn_norm[l], d));
    CK(cp(w.mlp_norm[l], src->mlp_norm[l], d));
  }
  CK(cudaEventRecord(w.installed, cs));
  w.version = version;
  w.has_data = true;
  ctx->pending = target;
  ctx->last_install = target;
  if (ctx->cfg.n_weight_buffers == 1) ctx->active = -1;   // the old weights are being overwritten
  ctx->newest_version = version;
  ctx->any_version = true;
  return ECHO_OK;
}

int echo_wait_policy(echo_ctx *ctx) {
  if (!ctx) return ECHO_ERR_INVALID;
  DeviceGuard guard(ctx->device);
  if (ctx->pending >= 0) {
    WeightBuf &w = ctx->wb[ctx->pending];
    CK(cudaEventSynchronize(w.installed));
    float ms = 0.f;
    if (cudaEventElapsedTime(&ms, w.inst_begin, w.installed) == cudaSuccess) ctx->stats.install_ms = ms;
  }
  return ECHO_OK;
}

int echo_rollout(echo_ctx *ctx, const int32_t *prompts, const int32_t *prompt_lens, int32_t P, int32_t G,
                 int32_t max_new_tokens, float temperature, uint64_t seed, int32_t *out_tokens, float *out_logprobs,
                 int64_t *out_versions) {
  return rollout_impl(ctx, prompts, prompt_lens, P, G, max_new_tokens, temperature, seed, nullptr, out_tokens,
                      out_logprobs, out_versions);
}

int echo_rollout_queue(echo_ctx *ctx, const int32_t *prompts, const int32_t *prompt_lens, int32_t n_prompts, int32_t G,
                       int32_t max_new_tokens, float temperature, uint64_t seed, const int32_t *forced_tokens,
                       int32_t *out_tokens, float *out_logprobs, int64_t *out_versions) {
  return rollout_queue_impl(ctx, prompts, prompt_lens, n_prompts, G, max_new_tokens, temperature, seed, forced_tokens,
                            out_tokens, out_logprobs, out_versions);
}

int echo_rollout_forced(echo_ctx *ctx, const int32_t *prompts, const int32_t *prompt_lens, int32_t P, int32_t G,
                        int32_t max_new_tokens, float temperature, uint64_t seed, const int32_t *forced_tokens,
                        int32_t *out_tokens, float *out_logprobs, int64_t *out_versions) {
  if (!forced_tokens) return ECHO_ERR_INVALID;
  return rollout_impl(ctx, prompts, prompt_lens, P, G, max_new_tokens, temperature, seed, forced_tokens, out_tokens,
                      out_logprobs, out_versions);
}

int echo_score(echo_ctx *ctx, const int32_t *prompts, const int32_t *prompt_lens, int32_t P, int32_t G,
               int32_t max_new_tokens, float temperature, const int32_t *tokens, float *out_logprobs,
               int64_t *out_versions) {
  return score_impl(ctx, prompts, prompt_lens, P, G, max_new_tokens, temperature, tokens, out_logprobs, out_versions);
}

int echo_turn_mask(const int32_t *tokens, int32_t n, int32_t T, int32_t turn_start_id, int32_t shift_to_targets,
                   uint8_t *out_mask, void *cuda_stream) {
  if (!tokens || !out_mask || n < 0 || T < 1) return ECHO_ERR_INVALID;
  cudaError_t e = turn_mask_launch(tokens, n, T, turn_start_id, shift_to_targets ? 1 : 0, out_mask,
                                   static_cast<cudaStream_t>(cuda_stream));
  return e == cudaSuccess ? ECHO_OK : ECHO_ERR_CUDA;
}

int echo_rollout_host(echo_ctx *ctx, const int32_t *prompts_host, const int32_t *prompt_lens, int32_t P, int32_t G,
                      int32_t max_new_tokens, float temperature, uint64_t seed, int32_t *out_tokens_host,
                      float *out_logprobs_host, int64_t *out_versions) {
  if (!ctx || !prompts_host || !out_tokens_host || !out_logprobs_host) return ECHO_ERR_INVALID;
  const Limits &M = ctx->M;
  if (P < 1 || P > M.P || G < 1 || G > M.G || max_new_tokens < 1 || max_new_tokens > M.T) return ECHO_ERR_INVALID;
  DeviceGuard guard(ctx->device);
  const Layout &lo = ctx->lo;
  int32_t *d_prompts = ctx->ptr<int32_t>(lo.stage_prompts);
  int32_t *d_tok = ctx->ptr<int32_t>(lo.stage_tok);
  float *d_lp = ctx->ptr<float>(lo.stage_lp);
  CK(cudaMemcpyAsync(d_prompts, prompts_host, static_cast<size_t>(P) * M.Lp * 4, cudaMemcpyHostToDevice,
                     ctx->stream));
  TRY(rollout_impl(ctx, d_prompts, prompt_lens, P, G, max_new_tokens, temperature, seed, nullptr, d_tok, d_lp,
                   out_versions));
  const size_t n = static_cast<size_t>(P) * G * max_new_tokens;
  CK(cudaMemcpyAsync(out_tokens_host, d_tok, n * 4, cudaMemcpyDeviceToHost, ctx->stream));
  CK(cudaMemcpyAsync(out_logprobs_host, d_lp, n * 4, cudaMemcpyDeviceToHost, ctx->stream));
  return echo_sync(ctx);
}

int echo_group_advantage(const float *rewards, int32_t P, int32_t G, float eps, float *out_adv, void *cuda_stream) {
  if (!rewards || !out_adv || P < 0 || G < 2 || !(eps >= 0.f)) return ECHO_ERR_INVALID;
  cudaError_t e = advantage_launch(rewards, P, G, eps, out_adv, static_cast<cudaStream_t>(cuda_stream));
  return e == cudaSuccess ? ECHO_OK : ECHO_ERR_CUDA;
}

int echo_grpo_surrogate(const float *logp_new, const float *logp_old, const float *logp_sampler, const float *adv,
                        const uint8_t *mask, int32_t n, int32_t T, float eps_clip, float C, float *out,
                        void *cuda_stream) {
  if (!logp_new || !logp_old || !logp_sampler || !adv || !out || n < 0 || T < 1) return ECHO_ERR_INVALID;
  if (!(eps_clip >= 0.f) || !(C > 0.f)) return ECHO_ERR_INVALID;
  cudaError_t e = grpo_surrogate_launch(logp_new, logp_old, logp_sampler, nullptr, adv, mask, n, T, eps_clip, C, 0.f,
                                        out, static_cast<cudaStream_t>(cuda_stream));
  return e == cudaSuccess ? ECHO_OK : ECHO_ERR_CUDA;
}

int echo_grpo_objective(const float *logp_new, const float *logp_old, const float *logp_sampler, const float *logp_ref,
                        const float *adv, const uint8_t *mask, int32_t n, int32_t T, float eps_clip, float C,
                        float beta, float *out, void *cuda_stream) {
  if (!logp_new || !logp_old || !logp_sampler || !logp_ref || !adv || !out || n < 0 || T < 1) return ECHO_ERR_INVALID;
  if (!(eps_clip >= 0.f) || !(C > 0.f) || !(beta >= 0.f)) return ECHO_ERR_INVALID;
  cudaError_t e = grpo_surrogate_launch(logp_new, logp_old, logp_sampler, logp_ref, adv, mask, n, T, eps_clip, C,
                                        beta, out, static_cast<cudaStream_t>(cuda_stream));
  return e == cudaSuccess ? ECHO_OK : ECHO_ERR_CUDA;
}

int echo_sync(echo_ctx *ctx) {
  if (!ctx) return ECHO_ERR_INVALID;
  DeviceGuard guard(ctx->device);
  CK(cudaStreamSynchronize(ctx->stream));
  CK(cudaStreamSynchronize(ctx->copy_stream));
  ctx->plan_in_flight = false;
  if (ctx->last_install >= 0) {
    WeightBuf &w = ctx->wb[ctx->last_install];
    float ms = 0.f;
    if (cudaEventElapsedTime(&ms, w.inst_begin, w.installed) == cudaSuccess) ctx->stats.install_ms = ms;
    else cudaGetLastError();
  }
  int status = 0;
  CK(cudaMemcpy(&status, ctx->arena + ctx->lo.status, 4, cudaMemcpyDeviceToHost));
  if (status != STATUS_OK) {
    cudaMemset(ctx->arena + ctx->lo.status, 0, 4);
    cudaMemset(ctx->arena + ctx->lo.gemm_counters, 0, static_cast<size_t>(kGemmMaxUnits) * 4);
    cudaMemset(ctx->arena + ctx->lo.gemm_bar, 0, 8);
    return status == STATUS_WAIT_TIMEOUT ? ECHO_ERR_TIMEOUT : ECHO_ERR_DEVICE_CHECK;
  }
  return ECHO_OK;
}

int echo_get_stats(echo_ctx *ctx, echo_stats *out) {
  if (!ctx || !out) return ECHO_ERR_INVALID;
  if (ctx->ev_end && cudaEventQuery(ctx->ev_end) == cudaSuccess) {
    float a = 0.f, b = 0.f;
    if (cudaEventElapsedTime(&a, ctx->ev_begin, ctx->ev_first) == cudaSuccess &&
        cudaEventElapsedTime(&b, ctx->ev_first, ctx->ev_end) == cudaSuccess) {
      ctx->stats.prefill_ms = a;
      ctx->stats.decode_ms = b;
    }
  }
  cudaGetLastError();
  *out = ctx->stats;
  return ECHO_OK;
}

int echo_debug_page_table(echo_ctx *ctx, int32_t *out, size_t n, int32_t *rows, int32_t *width) {
  if (!ctx) return ECHO_ERR_INVALID;
  if (rows) *rows = ctx->last_rows;
  if (width) *width = ctx->last_width;
  if (out) {
    if (n < ctx->last_table.size()) return ECHO_ERR_INVALID;
    std::copy(ctx->last_table.begin(), ctx->last_table.end(), out);
  }
  return ECHO_OK;
}

int echo_plan_page_table(const int32_t *prompt_lens, int32_t P, int32_t G, int32_t T, int32_t page_size,
                         int32_t *out_table, size_t capacity, int32_t *width, int32_t *n_pages) {
  if (!prompt_lens || !width || !n_pages || P < 1 || G < 1 || T < 1 || page_size < 1) return ECHO_ERR_INVALID;
  int W = 0;
  for (int p = 0; p < P; ++p) {
    if (prompt_lens[p] < 1) return ECHO_ERR_INVALID;
    W = std::max(W, std::max(ceil_div(prompt_lens[p] + T - 1, page_size), ceil_div(prompt_lens[p], page_size)));
  }
  *width = W;
  const size_t need = static_cast<size_t>(P) * G * W + static_cast<size_t>(P) * W;
  if (!out_table) {
    std::vector<int32_t> tmp(need);
    *n_pages = plan_tables(prompt_lens, P, G, T, page_size, W, tmp.data(), nullptr, nullptr, nullptr);
    return ECHO_OK;
  }
  if (capacity < need) return ECHO_ERR_INVALID;
  *n_pages = plan_tables(prompt_lens, P, G, T, page_size, W, out_table, nullptr, nullptr, nullptr);
  return ECHO_OK;
}

int echo_debug_noise(uint64_t seed, uint32_t s, uint32_t j, uint32_t v0, uint32_t n, uint32_t *out_words,
                     float *out_uniform, void *cuda_stream) {
  if (!out_words || !out_uniform) return ECHO_ERR_INVALID;
  cudaError_t e = noise_debug_launch(seed, s, j, v0, n, out_words, out_uniform, static_cast<cudaStream_t>(cuda_stream));
  return e == cudaSuccess ? ECHO_OK : ECHO_ERR_CUDA;
}

int echo_sample(const float *logits, int32_t R, int32_t V, int32_t rows_per_logit_row, const int32_t *seq_ids,
                uint32_t j, float temperature, uint64_t seed, const int32_t *forced, int32_t *out_tokens,
                float *out_logprobs, void *cuda_stream) {
  if (!logits || !out_tokens || !out_logprobs || R < 0 || V < 1 || rows_per_logit_row < 1) return ECHO_ERR_INVALID;
  if (!(temperature > 0.f) || !std::isfinite(temperature)) return ECHO_ERR_INVALID;
  if (R == 0) return ECHO_OK;
  // stand-alone call: outputs are dense [R], so the stride is 1 and the step index is folded
  // into the base pointers
  cudaError_t e = sampler_launch(logits, R, V, rows_per_logit_row, seq_ids, nullptr, j, temperature, seed,
                                 forced ? forced - j : nullptr, 1, out_tokens - j, out_logprobs - j, 1,
                                 static_cast<cudaStream_t>(cuda_stream));
  return e == cudaSuccess ? ECHO_OK : ECHO_ERR_CUDA;
}

int echo_sample_top_p(const float *logits, int32_t R, int32_t V, int32_t rows_per_logit_row, const int32_t *seq_ids,
                      uint32_t j, float temperature, float top_p, uint64_t seed, const int32_t *forced,
                      int32_t *out_tokens, float *out_logprobs, void *cut_scratch, void *cuda_stream) {
  if (!logits || !out_tokens || !out_logprobs || R < 0 || V < 1 || rows_per_logit_row < 1) return ECHO_ERR_INVALID;
  if (!(temperature > 0.f) || !std::isfinite(temperature) || !(top_p > 0.f) || !(top_p <= 1.f)) return ECHO_ERR_INVALID;
  if (R == 0) return ECHO_OK;
  cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
  const uint2 *cut = nullptr;
  if (top_p < 1.f) {
    if (!cut_scratch || (reinterpret_cast<uintptr_t>(cut_scratch) & 7)) return ECHO_ERR_INVALID;
    const int rows = (R + rows_per_logit_row - 1) / rows_per_logit_row;
    if (nucleus_cut_launch(logits, rows, V, temperature, top_p, static_cast<uint2 *>(cut_scratch), s) != cudaSuccess)
      return ECHO_ERR_CUDA;
    cut = static_cast<const uint2 *>(cut_scratch);
  }
  cudaError_t e = sampler_launch(logits, R, V, rows_per_logit_row, seq_ids, nullptr, j, temperature, seed,
                                 forced ? forced - j : nullptr, 1, out_tokens - j, out_logprobs - j, 1, s, -1, cut);
  return e == cudaSuccess ? ECHO_OK : ECHO_ERR_CUDA;
}

size_t echo_decode_attention_scratch_bytes(int32_t B, int32_t Hq, int32_t hd) {
  if (B < 1 || Hq < 1 || hd < 1) return 0;
  return align_up(static_cast<size_t>(B) * Hq * hd * 4) + align_up(static_cast<size_t>(B) * Hq * 8) + kAlign;
}

int echo_decode_attention(const void *q, const void *kv_pool, int32_t n_pages, const int32_t *page_table,
                          int32_t pt_width, const int32_t *row_pos, const int32_t *full_pages, int32_t P, int32_t G,
                          int32_t Hq, int32_t Hkv, int32_t hd, void *scratch, size_t scratch_bytes, void *out,
                          int32_t operand_format, int32_t kernel_choice, void *cuda_stream) {
  if (operand_format < 0 || operand_format > 1 || kernel_choice < 0 || kernel_choice > 3) return ECHO_ERR_INVALID;
  if (!q || !kv_pool || !page_table || !row_pos || !full_pages || !scratch || !out) return ECHO_ERR_INVALID;
  if (P < 1 || G < 1 || n_pages < 1 || pt_width < 1 || Hkv < 1 || Hq % Hkv) return ECHO_ERR_INVALID;
  if (!attention_decode_supported(hd, 16, Hq, Hkv)) return ECHO_ERR_UNSUPPORTED;
  const int B = P * G;
  if (scratch_bytes < echo_decode_attention_scratch_bytes(B, Hq, hd) || (reinterpret_cast<uintptr_t>(scratch) & 255))
    return ECHO_ERR_ARENA;
  const size_t rows = static_cast<size_t>(n_pages) * Hkv * 2 * 16;
  if (rows >= (1ull << 31)) return ECHO_ERR_UNSUPPORTED;
  cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
  if (attention_decode_configure() != cudaSuccess) return ECHO_ERR_CUDA;
  CUtensorMap tm;
  if (make_tensor_map(&tm, kv_pool, rows, hd, hd, 32) != 0) return ECHO_ERR_CUDA;
  uint8_t *sc = static_cast<uint8_t *>(scratch);
  float *pre_o = reinterpret_cast<float *>(sc);
  float2 *pre_ml = reinterpret_cast<float2 *>(sc + align_up(static_cast<size_t>(B) * Hq * hd * 4));
  int *status = reinterpret_cast<int *>(reinterpret_cast<uint8_t *>(pre_ml) + align_up(static_cast<size_t>(B) * Hq * 8));
  if (cudaMemsetAsync(status, 0, 16, s) != cudaSuccess) return ECHO_ERR_CUDA;     // status word + item counters
  DecodeAttnArgs da{&tm, static_cast<const __nv_bfloat16 *>(q), static_cast<__nv_bfloat16 *>(out), pre_o, pre_ml,
                    page_table, pt_width, row_pos, full_pages, 0, P, G, Hq, Hkv, hd, n_pages, status, nullptr,
                    status + 2, operand_format, kernel_choice & 1, (kernel_choice >> 1) & 1};
  if (attention_decode_launch(da, s) != cudaSuccess) return ECHO_ERR_CUDA;
  int st = 0;
  if (cudaMemcpyAsync(&st, status, 4, cudaMemcpyDeviceToHost, s) != cudaSuccess) return ECHO_ERR_CUDA;
  if (cudaStreamSynchronize(s) != cudaSuccess) return ECHO_ERR_CUDA;
  if (st == STATUS_WAIT_TIMEOUT) return ECHO_ERR_TIMEOUT;
  return st == STATUS_OK ? ECHO_OK : ECHO_ERR_DEVICE_CHECK;
}

size_t echo_gemm_workspace_bytes(int32_t M) {
  if (M < 1) return 0;
  if (gemm_tc_configure() != cudaSuccess) return 0;
  return align_up(gemm_workspace_bytes(pick_bnb(M))) + static_cast<size_t>(kGemmMaxUnits) * 4;
}

int echo_gemm_bf16(const void *X, const void *W, void *Y, int32_t M, int32_t N, int32_t K, int32_t epilogue,
                   int32_t impl, void *workspace, size_t workspace_bytes, void *cuda_stream) {
  if (!X || !W || !Y || M < 1 || M > 4096 || N < 1 || K < 8 || (K % 8)) return ECHO_ERR_INVALID;
  if (epilogue != EPI_STORE && epilogue != EPI_ACCUM && epilogue != EPI_SWIGLU) return ECHO_ERR_INVALID;
  cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
  const int half_in = impl >= 2000 ? 1 : 0;        // X and W hold IEEE half values
  if (half_in) impl -= 2000;
  const int tiled = impl >= 1000 ? 1 : 0;          // W is block-tiled storage (echo_retile_weights)
  if (tiled) impl -= 1000;
  if (impl == 1) {
    if (epilogue == EPI_SWIGLU) return ECHO_ERR_INVALID;
    cudaError_t e = gemm_simt_launch(static_cast<const __nv_bfloat16 *>(X), static_cast<const __nv_bfloat16 *>(W),
                                     static_cast<float *>(Y), N, M, N, K, epilogue == EPI_ACCUM, s, tiled, 0, half_in);
    return e == cudaSuccess ? ECHO_OK : ECHO_ERR_CUDA;
  }
  // tiled storage of a gate/up pair: two parts of N rows, each padded to whole blocks
  const uint64_t w_rows = epilogue == EPI_SWIGLU
                              ? (tiled ? 2ull * ((N + kTileRows - 1) / kTileRows) * kTileRows : 2ull * N)
                              : static_cast<uint64_t>(N);
  auto w_map = [&](CUtensorMap *tm, uint32_t box_rows) {
    return tiled ? make_tiled_map(tm, W, w_rows, K, box_rows) : make_tensor_map(tm, W, w_rows, K, K, box_rows);
  };
  if (gemm_tc_configure() != cudaSuccess) return ECHO_ERR_CUDA;
  if (impl >= 300) {
    // SM-pair kernel, impl - 300 k-slices per tile (0 = choose)
    if (gemm_pair_configure() != cudaSuccess) return ECHO_ERR_CUDA;
    if (!gemm_pair_supported(Y, N, M, N, K, epilogue)) return ECHO_ERR_UNSUPPORTED;
    CUtensorMap tmW2;
    if (w_map(&tmW2, kGemmTileN) != 0) return ECHO_ERR_CUDA;
    PairGemmArgs pa{&tmW2, X, Y, N, M, N, K, epilogue, nullptr, 0, impl - 300, tiled, half_in};
    if (epilogue == EPI_STORE && gemm_pair_split(M, N, K, epilogue, impl - 300) > 1 &&
        cudaMemsetAsync(Y, 0, static_cast<size_t>(M) * N * sizeof(float), s) != cudaSuccess)
      return ECHO_ERR_CUDA;
    return gemm_pair_launch(pa, s) == cudaSuccess ? ECHO_OK : ECHO_ERR_CUDA;
  }
  const int bnb = pick_bnb(M);
  const size_t ws_bytes = align_up(gemm_workspace_bytes(bnb));
  if (!workspace || workspace_bytes < ws_bytes + static_cast<size_t>(kGemmMaxUnits) * 4 ||
      (reinterpret_cast<uintptr_t>(workspace) & 255))
    return ECHO_ERR_ARENA;
  int *counters = reinterpret_cast<int *>(static_cast<uint8_t *>(workspace) + ws_bytes);
  if (cudaMemsetAsync(counters, 0, static_cast<size_t>(kGemmMaxUnits) * 4, s) != cudaSuccess) return ECHO_ERR_CUDA;
  CUtensorMap tmW, tmX;
  const bool gu = epilogue == EPI_SWIGLU;
  if (w_map(&tmW, gu ? 64 : kGemmTileN) != 0) return ECHO_ERR_CUDA;
  if (make_tensor_map(&tmX, X, M, K, K, bnb) != 0) return ECHO_ERR_CUDA;
  const bool indep = impl >= 200;
  const int split = indep ? impl - 200 : (impl >= 100 ? impl - 100 : (impl == 2 ? -1 : 0));
  if (indep && epilogue == EPI_SWIGLU) return ECHO_ERR_INVALID;
  if (indep && epilogue == EPI_STORE &&
      cudaMemsetAsync(Y, 0, static_cast<size_t>(M) * N * sizeof(float), s) != cudaSuccess)
    return ECHO_ERR_CUDA;
  GemmArgs a{&tmW, &tmX, Y, N, M, N, K, bnb, epilogue, nullptr, static_cast<float *>(workspace), counters, 0, split, 0,
             indep ? 1 : 0, tiled, half_in};
  cudaError_t e = gemm_tc_launch(a, s);
  return e == cudaSuccess ? ECHO_OK : ECHO_ERR_CUDA;
}

size_t echo_tiled_weight_bytes(int64_t rows, int64_t cols) {
  if (rows < 1 || cols < 1) return 0;
  return tiled_elems(static_cast<size_t>(rows), static_cast<size_t>(cols)) * 2;
}

int echo_retile_weights(const void *src, int64_t rows, int64_t cols, void *dst, size_t dst_bytes, void *cuda_stream) {
  if (!src || !dst || rows < 1 || cols < 8 || (cols % 8)) return ECHO_ERR_INVALID;
  if (dst_bytes < echo_tiled_weight_bytes(rows, cols)) return ECHO_ERR_ARENA;
  cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
  // padding of partial blocks must read as zero
  if (cudaMemsetAsync(dst, 0, echo_tiled_weight_bytes(rows, cols), s) != cudaSuccess) return ECHO_ERR_CUDA;
  cudaError_t e = retile_launch(static_cast<__nv_bfloat16 *>(dst), static_cast<const __nv_bfloat16 *>(src),
                                static_cast<size_t>(rows), static_cast<size_t>(cols), 0, s);
  return e == cudaSuccess ? ECHO_OK : ECHO_ERR_CUDA;
}

int echo_probe_read_bandwidth(const void *buf, size_t bytes, int32_t repeats, void *scratch, float *ms_per_pass,
                              void *cuda_stream) {
  if (!buf || !scratch || !ms_per_pass || bytes < 16 || (bytes % 16) || repeats < 1 || repeats > 1000 ||
      (reinterpret_cast<uintptr_t>(buf) & 15) || (reinterpret_cast<uintptr_t>(scratch) & 3))
    return ECHO_ERR_INVALID;
  cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
  int dev = 0, sms = 0;
  if (cudaGetDevice(&dev) != cudaSuccess ||
      cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
    return ECHO_ERR_CUDA;
  cudaEvent_t a = nullptr, b = nullptr;
  if (cudaEventCreate(&a) != cudaSuccess || cudaEventCreate(&b) != cudaSuccess) {
    if (a) cudaEventDestroy(a);
    return ECHO_ERR_CUDA;
  }
  int rc = ECHO_OK;
  uint32_t *sink = static_cast<uint32_t *>(scratch);
  if (read_probe_launch(buf, bytes, sink, sms * 4, s) != cudaSuccess) rc = ECHO_ERR_CUDA;      // warm-up pass
  if (rc == ECHO_OK && cudaEventRecord(a, s) != cudaSuccess) rc = ECHO_ERR_CUDA;
  for (int i = 0; i < repeats && rc == ECHO_OK; ++i)
    if (read_probe_launch(buf, bytes, sink, sms * 4, s) != cudaSuccess) rc = ECHO_ERR_CUDA;
  if (rc == ECHO_OK && (cudaEventRecord(b, s) != cudaSuccess || cudaEventSynchronize(b) != cudaSuccess))
    rc = ECHO_ERR_CUDA;
  float ms = 0.f;
  if (rc == ECHO_OK && cudaEventElapsedTime(&ms, a, b) != cudaSuccess) rc = ECHO_ERR_CUDA;
  cudaEventDestroy(a);
  cudaEventDestroy(b);
  if (rc == ECHO_OK) *ms_per_pass = ms / static_cast<float>(repeats);
  return rc;
}

int echo_set_sequence_base(echo_ctx *ctx, uint32_t base) {
  if (!ctx) return ECHO_ERR_INVALID;
  ctx->seq_base = base;
  return ECHO_OK;
}

int echo_debug_capture(echo_ctx *ctx, int32_t layer, float *pre_in, float *pre_out, float *dec_in, float *dec_out) {
  if (!ctx || layer < -1 || layer >= ctx->D.L) return ECHO_ERR_INVALID;
  if (ctx->D.d % 4) return ECHO_ERR_UNSUPPORTED;
  ctx->cap_layer = layer;
  ctx->cap_pre_in = pre_in;
  ctx->cap_pre_out = pre_out;
  ctx->cap_dec_in = dec_in;
  ctx->cap_dec_out = dec_out;
  return ECHO_OK;
}

int echo_debug_wait_limit(uint64_t limit_ns, void *scratch, uint64_t *waited_ns, void *cuda_stream) {
  if (limit_ns == 0 || limit_ns > 100000000ull || !scratch || (reinterpret_cast<uintptr_t>(scratch) & 7))
    return ECHO_ERR_INVALID;                                                    // at most 0.1 s
  cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
  struct Probe { int status; int pad; unsigned long long waited; };
  Probe *d = static_cast<Probe *>(scratch);
  Probe h{};
  if (cudaMemsetAsync(d, 0, sizeof(Probe), s) != cudaSuccess ||
      wait_probe_launch(limit_ns, &d->status, &d->waited, s) != cudaSuccess ||
      cudaMemcpyAsync(&h, d, sizeof(Probe), cudaMemcpyDeviceToHost, s) != cudaSuccess ||
      cudaStreamSynchronize(s) != cudaSuccess)
    return ECHO_ERR_CUDA;
  if (waited_ns) *waited_ns = h.waited;
  return h.status == STATUS_WAIT_TIMEOUT ? ECHO_ERR_TIMEOUT : ECHO_OK;
}

int echo_profile_config(echo_ctx *ctx, int32_t every_n_steps) {
  if (!ctx || every_n_steps < -1) return ECHO_ERR_INVALID;
  ctx->prof_every = every_n_steps;
  return ECHO_OK;
}

int echo_profile_read(echo_ctx *ctx, int32_t *steps, float *ms, int32_t capacity, int32_t *n_out) {
  if (!ctx || !n_out) return ECHO_ERR_INVALID;
  DeviceGuard guard(ctx->device);
  CK(cudaStreamSynchronize(ctx->stream));
  std::vector<int> order;
  for (const auto &r : ctx->prof_recs)
    if (order.empty() || order.back() != r.step) order.push_back(r.step);
  *n_out = static_cast<int32_t>(order.size());
  if (!steps || !ms) return ECHO_OK;
  if (capacity < *n_out) return ECHO_ERR_INVALID;
  for (size_t i = 0; i < order.size(); ++i) {
    steps[i] = order[i];
    for (int c = 0; c < PROF_NCLS; ++c) ms[i * PROF_NCLS + c] = 0.f;
  }
  size_t idx = 0;
  for (const auto &r : ctx->prof_recs) {
    while (order[idx] != r.step) ++idx;
    float t = 0.f;
    CK(cudaEventElapsedTime(&t, r.a, r.b));
    ms[idx * PROF_NCLS + r.cls] += t;
  }
  return ECHO_OK;
}

const char *echo_strerror(int code) {
  switch (code) {
    case ECHO_OK: return "ok";
    case ECHO_ERR_INVALID: return "invalid argument";
    case ECHO_ERR_ARENA: return "arena too small or misaligned";
    case ECHO_ERR_NO_POLICY: return "no policy installed";
    case ECHO_ERR_VERSION: return "version not strictly increasing";
    case ECHO_ERR_BUSY: return "an install is still pending";
    case ECHO_ERR_CUDA: return "CUDA error";
    case ECHO_ERR_DEVICE_CHECK: return "device-side range check failed";
    case ECHO_ERR_TIMEOUT: return "device-side wait timed out";
    case ECHO_ERR_UNSUPPORTED: return "unsupported shape";
    default: return "unknown error";
  }
}

const char *echo_last_error(echo_ctx *ctx) { return ctx ? ctx->last_error.c_str() : ""; }

}  // extern "C"

// Shared declarations of the rollout library's translation units (sm_100a only).
#pragma once

#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/echo.h"

namespace echo {

// Status word written by kernels that detect a problem themselves (never trap).
enum : int {
  STATUS_OK = 0,
  STATUS_BAD_PAGE = 1,        // page id / position outside the pool
  STATUS_BAD_TOKEN = 2,       // token id outside [0, vocab)
  STATUS_WAIT_TIMEOUT = 3,    // a bounded mbarrier wait ran out
};

constexpr int kGemmTileN = 128;      // output features per CTA (UMMA M)
constexpr int kGemmTileK = 64;       // bf16 elements per pipeline stage (one 128-byte swizzle row)
constexpr int kMaxBatchTile = 256;   // rows of activations per MMA (UMMA N)
constexpr int kGemmMaxUnits = 8192;  // output tiles per launch the tile counters cover

// ---- launches that may start early (programmatic stream serialization) --------------------------
// A kernel launched through launch_early may be scheduled while its predecessor on the stream is
// still draining, which hides the launch latency between the many short kernels of a decode step.
// Such a kernel MUST begin with early_start_sync(): it lets its own successor be scheduled and then
// waits until the predecessor has completed and its writes are visible, before touching memory.
extern bool g_early_start;          // cleared to launch everything the ordinary way

template <typename... KArgs, typename... Args>
inline cudaError_t launch_early(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t s,
                                Args... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = s;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = g_early_start ? 1 : 0;
  return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}
#ifdef __CUDACC__
// fp32 -> the 16-bit operand format of a layer (bf16, or IEEE half), as raw bits, and back
__device__ __forceinline__ uint16_t cvt16(float v, bool half) {
  if (half) return __half_as_ushort(__float2half_rn(v));
  return __bfloat16_as_ushort(__float2bfloat16(v));
}
__device__ __forceinline__ uint32_t cvt16x2(float lo, float hi, bool half) {
  if (half) {
    const __half2 v = __floats2half2_rn(lo, hi);
    return *reinterpret_cast<const uint32_t *>(&v);
  }
  const __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<const uint32_t *>(&v);
}
__device__ __forceinline__ float widen16(uint16_t bits, bool half) {
  return half ? __half2float(__ushort_as_half(bits)) : __uint_as_float(static_cast<uint32_t>(bits) << 16);
}
__device__ __forceinline__ float2 widen16x2(uint32_t w, bool half) {
  if (half) return __half22float2(*reinterpret_cast<const __half2 *>(&w));
  return make_float2(__uint_as_float(w << 16), __uint_as_float(w & 0xffff0000u));
}
// order-preserving 32-bit key of a float: a < b  <=>  order_key(a) < order_key(b)
__device__ __forceinline__ uint32_t order_key(float s) {
  const uint32_t u = __float_as_uint(s);
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}
__device__ __forceinline__ void early_start_sync() {
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  asm volatile("griddepcontrol.wait;" ::: "memory");
}
#endif

// ---- dense projections (gemm.cu) ------------------------------------------
// Y[m][n] (+)= sum_k X[m][k] * W[n][k], bf16 inputs, fp32 accumulation.
// tmW: tensor map over W [N][K] with box {64, 128}; tmX over X [M][K] with box {64, bnb}.
enum GemmEpilogue : int {
  EPI_STORE = 0,      // Y = acc
  EPI_ACCUM = 1,      // Y += acc              (residual add)
  EPI_SWIGLU = 2,     // W holds gate rows [0, N) and up rows [N, 2N): Y = bf16(silu(g) * u);
                      // its tensor map must use a 64-row box (64 gate + 64 up rows per tile)
};

struct GemmArgs {
  const CUtensorMap *tmW;
  const CUtensorMap *tmX;
  void *Y;            // fp32 [M][ldY], or bf16 for EPI_SWIGLU
  int ldY;
  int M, N, K;        // N counts output features per accumulator (F for SWIGLU)
  int bnb;            // activation rows per CTA: 32, 64, 128 or 256
  int epilogue;
  int *status;
  float *workspace;   // gemm_workspace_bytes(bnb) bytes: partial accumulators of split tiles
  int *counters;      // kGemmMaxUnits ints, zero before the first launch (the kernel re-zeroes them)
  int max_ctas;       // 0 = one CTA per SM
  int force_split;    // 0 = choose; k > 0 = split-K by k; -1 = always the persistent stream-K kernel
  int allow_early_start;    // 1: launch with programmatic stream serialization (see gemm.cu)
  int independent_splits;   // 1: k-slices add into Y in memory (Y must hold zeros for EPI_STORE; the order of
                            // the additions is not fixed); 0: slices are reduced in rank order inside a cluster
  int tiled;                // 1: W is stored block-tiled (see tiled_elems) and tmW is a map over that storage
  int half_in = 0;          // 1: X and W hold IEEE half values instead of bf16 (and a SwiGLU output is half)
};

// ---- block-tiled weight storage -------------------------------------------------------------
// A weight matrix [rows][cols] is kept as 128-row x 64-column blocks, each block contiguous
// (128 rows of 128 bytes = 16 KiB), ordered [row block][column block]; partial blocks are padded
// with zeros.  A CTA that streams the weights of a few output features along K then reads one
// long contiguous run instead of 128-byte pieces 2*cols bytes apart, which HBM serves about a
// fifth faster.  Element (n, k) lives at tiled_index(n, k, ceil(cols / 64)).
constexpr int kTileRows = 128, kTileCols = 64;
inline size_t tiled_elems(size_t rows, size_t cols) {
  return ((rows + kTileRows - 1) / kTileRows) * kTileRows * ((cols + kTileCols - 1) / kTileCols) * kTileCols;
}
__host__ __device__ inline size_t tiled_index(size_t n, size_t k, size_t col_blocks) {
  return (((n >> 7) * col_blocks + (k >> 6)) * kTileRows + (n & 127)) * kTileCols + (k & 63);
}
// Copies row-major src [rows][cols] (device memory, or host memory the device can read) into tiled
// storage whose row 0 is dst_row0 rows into the matrix at dst; padding is not written.
// to_half: the bf16 values are converted to IEEE half on the way (exact unless |w| < 2^-17 or > 65504).
cudaError_t retile_launch(__nv_bfloat16 *dst, const __nv_bfloat16 *src, size_t rows, size_t cols, size_t dst_row0,
                          cudaStream_t s, bool to_half = false);
// Tensor map over tiled storage of `rows` (padded to blocks) x `cols`: box = box_rows rows of one block.
int make_tiled_map(CUtensorMap *out, const void *base, uint64_t rows, uint64_t cols, uint32_t box_rows);
size_t gemm_workspace_bytes(int bnb);
cudaError_t gemm_tc_launch(const GemmArgs &a, cudaStream_t stream);
cudaError_t gemm_tc_configure();     // sets the dynamic shared memory attribute once per device
// part_rows > 0 with tiled storage: W consists of parts of part_rows rows, each starting on a block
cudaError_t gemm_simt_launch(const __nv_bfloat16 *X, const __nv_bfloat16 *W, float *Y, int ldY,
                             int M, int N, int K, int accumulate, cudaStream_t stream, int tiled = 0,
                             int part_rows = 0, int half_in = 0);
// Tensor map over a row-major bf16 matrix [rows][cols] (leading dimension ld elements),
// 128-byte swizzle, box {64, box_rows}.
int make_tensor_map(CUtensorMap *out, const void *base, uint64_t rows, uint64_t cols, uint64_t ld,
                    uint32_t box_rows);

// Output tile map over a row-major [rows][cols] fp32 or bf16 matrix, no swizzle, box {box_cols, box_rows}.
int make_out_map_box(CUtensorMap *out, void *base, uint64_t rows, uint64_t cols, uint64_t ld, bool bf16,
                     uint32_t box_cols, uint32_t box_rows);

// ---- projections on SM pairs (gemm_pair.cu) ---------------------------------
// Same arithmetic as above with 2-CTA MMAs: used for more than 64 activation rows.
// RMSNorm as the projection's prologue: before it loads activations, the launch itself computes
// h[r] = 16-bit( x[r] * rsqrt(mean(x[r]^2) + eps) * gain ) for its M rows (each CTA a share of the rows),
// meets at a grid-wide barrier and then reads h as its activation matrix X.  Needs every CTA of the
// launch resident at once (gemm_pair_can_fuse_norm).  x == nullptr: off.
struct NormPrologue {
  const float *x = nullptr;          // fp32 [M][d]: the residual stream
  const __nv_bfloat16 *gain = nullptr;
  void *h = nullptr;                 // 16-bit [M][d]: written here, = PairGemmArgs::X
  float eps = 0.f;
  int *bar = nullptr;                // two ints, zero before the first launch: arrivals, generation
};
struct PairGemmArgs {
  const CUtensorMap *tmW;   // tensor map over W with box {64, 128}; for EPI_SWIGLU over [2N][K] (gate rows, then up rows)
  const void *X;            // bf16 [M][K], contiguous
  void *Y;                  // fp32 [M][ldY], or bf16 for EPI_SWIGLU; 16-byte aligned rows
  int ldY;
  int M, N, K;
  int epilogue;
  int *status;
  int allow_early_start;
  int force_split;          // 0 = choose; k > 0 = k slices along K (linear epilogues only)
  int tiled;                // 1: W is block-tiled storage and tmW a map over it (make_tiled_map, 128-row box)
  int half_in = 0;          // 1: X and W hold IEEE half values instead of bf16 (and a SwiGLU output is half)
  NormPrologue norm;        // optional fused RMSNorm producing X (K = its row length)
};
// true if this launch's CTAs all fit the GPU at once (one row tile, at most as many SM pairs as can be
// resident): the condition for the fused RMSNorm prologue
bool gemm_pair_can_fuse_norm(int M, int N, int K, int epilogue);
cudaError_t gemm_pair_configure();
bool gemm_pair_supported(const void *Y, int ldY, int M, int N, int K, int epilogue);
// k-slices per tile the launch will use; with more than one slice and EPI_STORE, Y must hold zeros
int gemm_pair_split(int M, int N, int K, int epilogue, int force_split);
cudaError_t gemm_pair_launch(const PairGemmArgs &a, cudaStream_t stream);

// ---- element-wise / row-wise kernels (elementwise.cu) ------------------------
struct RowMeta {
  const int32_t *row_pt;     // page-table row of each activation row
  const int32_t *row_pos;    // absolute position of each activation row
  const int32_t *row_done;   // optional: non-zero = the row's sequence has ended (end token fed): nothing is
                             // appended or attended for it, its outputs are not used
};

cudaError_t embed_launch(const __nv_bfloat16 *embed, const int32_t *tok_src, const int32_t *tok_idx,
                         float *x, int R, int d, int vocab, int *status, cudaStream_t s);
// out_half: h is written as IEEE half instead of bf16 (the gain stays bf16)
cudaError_t rmsnorm_launch(const float *x, const __nv_bfloat16 *gain, __nv_bfloat16 *h, int R, int d,
                           float eps, cudaStream_t s, bool out_half = false);
cudaError_t rope_table_launch(float2 *table, int max_pos, int head_dim, double theta, cudaStream_t s);
// qkv fp32 [R][(Hq+2Hkv)*hd] -> q bf16 [R][Hq*hd], K/V into the paged cache of one layer; the rows
// of qkv it consumes are left holding zeros
cudaError_t rope_append_launch(float *qkv, __nv_bfloat16 *q, __nv_bfloat16 *kv_layer,
                               const float2 *rope_table, RowMeta meta, const int32_t *page_table,
                               int pt_width, int R, int Hq, int Hkv, int hd, int page_size,
                               int n_pages, int max_pos, int *status, cudaStream_t s, bool out_half = false,
                               const int32_t *q_row = nullptr);     // row of q each row writes (null: its own)
cudaError_t swiglu_launch(const float *gu, __nv_bfloat16 *act, int R, int F, cudaStream_t s, bool out_half = false);
cudaError_t gather_rows_launch(const float *x, const int32_t *src_rows, float *dst, int n, int d,
                               cudaStream_t s);
cudaError_t copy_partial_pages_launch(__nv_bfloat16 *kv, const int32_t *src_page, const int32_t *dst_page,
                                      int n_copies, int n_layers, size_t layer_stride_elems,
                                      int page_elems, cudaStream_t s);
// Compaction of a decode step's rows (used with an end token): the sequences that have not ended are
// packed to the front of the activation rows.  row_seq[r] = sequence of row r (-1: padding row),
// seq_row[b] = row of sequence b (-1: ended), seq_pos[b] = position sequence b feeds, *n_live = rows in use.
// With a prompt queue (groups admitted into freed slots during the rollout) a slot's sequence b also
// has seq_gid[b] = the sequence id it currently generates (prompt index * G + g; -1: empty slot) and
// seq_t0[b] = the step counter's value when its token 0 was sampled; both null otherwise (gid = b, t0 = 0).
struct CompactRows {
  int32_t *row_seq, *seq_row, *seq_pos, *n_live;
  int32_t *seq_gid = nullptr, *seq_t0 = nullptr;
};
// decode-step preparation: advances the step counter, sets the rows' token and position; with `cr` it
// also packs the live sequences and writes end token / 0 for the ended ones into the outputs
cudaError_t decode_prep_launch(int32_t *d_step, const int32_t *tok_hist, int T, const int32_t *seq_len0,
                               int32_t *row_tok, int32_t *row_pos, int B, cudaStream_t s, int eos_id = -1,
                               int32_t *row_done = nullptr, const CompactRows *cr = nullptr,
                               int32_t *out_tok = nullptr, float *out_lp = nullptr);
// Slots that change hands: for i < n, sequence slot admit_seq[i] finishes the outputs of the sequence
// it held (end token / 0 from its current position on, if eos_id >= 0), takes sequence id admit_gid[i]
// (-1: stays empty; -2: stays empty and the old sequence's outputs are NOT completed, it will be generated
// again) with its token 0 due at the step counter's current value, and is live again.
cudaError_t admit_launch(int n, const int32_t *admit_seq, const int32_t *admit_gid, const int32_t *d_step,
                         int32_t *seq_gid, int32_t *seq_t0, int32_t *row_done, int32_t *out_tok, float *out_lp, int T,
                         int eos_id, cudaStream_t s);
cudaError_t sampler_launch(const float *logits, int R, int V, int rows_per_logit_row,
                           const int32_t *seq_ids, const int32_t *d_step, uint32_t j_host,
                           float temperature, uint64_t seed, const int32_t *forced, int forced_stride,
                           int32_t *out_tok, float *out_lp, int out_stride, cudaStream_t s, int eos_id = -1,
                           const uint2 *nucleus_cut = nullptr,    // per logits row, from nucleus_cut_launch
                           const int32_t *row_done = nullptr,     // per row: non-zero = the sequence has ended
                           uint32_t seq_base = 0,                 // added to every sequence id of the noise streams
                           const int32_t *row_seq = nullptr,      // compacted step: sequence of each logits row
                           const int32_t *seq_gid = nullptr,      // prompt queue: sequence id a slot generates and
                           const int32_t *seq_t0 = nullptr);      // the step its token 0 was sampled at
// Nucleus (top-p) cut of each logits row: cut[row] = (order-preserving key of the score of the last
// nucleus member, its id; id 0x7fffffff = every id of that score).  nucleus.cu
cudaError_t nucleus_cut_launch(const float *logits, int rows, int V, float temperature, float top_p, uint2 *cut,
                               cudaStream_t s);
cudaError_t noise_debug_launch(uint64_t seed, uint32_t s_id, uint32_t j, uint32_t v0, uint32_t n,
                               uint32_t *words, float *uniform, cudaStream_t s);
cudaError_t advantage_launch(const float *r, int P, int G, float eps, float *out, cudaStream_t s);
cudaError_t grpo_surrogate_launch(const float *ln, const float *lo, const float *ls, const float *lr,
                                  const float *adv, const uint8_t *mask, int n, int T, float eps_clip, float C,
                                  float beta, float *out, cudaStream_t s);
cudaError_t set_int_launch(int32_t *p, int32_t v, cudaStream_t s);
// teacher-forced scoring of whole trajectories (see the kernels in elementwise.cu)
cudaError_t score_rows_launch(int r0, int R, int T, const int32_t *seq_len0, int32_t *row_pt, int32_t *row_pos,
                              int32_t *tok_idx, cudaStream_t s);
cudaError_t first_end_launch(const int32_t *tokens, int B, int T, int eos_id, int32_t *first_end, cudaStream_t s);
cudaError_t logprob_rows_launch(const float *logits, int rows, int V, int rows_per_logit_row, float temperature,
                                const int32_t *tokens, const int32_t *tok_idx, int T, const int32_t *first_end,
                                float *out, int *status, cudaStream_t s);
cudaError_t turn_mask_launch(const int32_t *tokens, int n, int T, int turn_start, int shift, uint8_t *out,
                             cudaStream_t s);
// copies n floats (a multiple of 4) of x into slot (*d_step - 1) of dst
cudaError_t capture_step_launch(const float *x, float *dst, const int32_t *d_step, size_t n, cudaStream_t s);
// reads `bytes` (a multiple of 16) of buf once with n_blocks blocks of 512 threads; writes nothing
cudaError_t read_probe_launch(const void *buf, size_t bytes, uint32_t *sink, int n_blocks, cudaStream_t s);
// one warp waits limit_ns for a barrier nobody signals, then sets *status = STATUS_WAIT_TIMEOUT
cudaError_t wait_probe_launch(uint64_t limit_ns, int *status, unsigned long long *waited_ns, cudaStream_t s);

// ---- attention (attention.cu) ------------------------------------------------
// One query row per activation row, keys 0..pos of its page-table row (causal by construction).
cudaError_t attention_rows_launch(const __nv_bfloat16 *q, const __nv_bfloat16 *kv_layer,
                                  __nv_bfloat16 *out, RowMeta meta, const int32_t *page_table,
                                  int pt_width, int R, int Hq, int Hkv, int hd, int page_size,
                                  int n_pages, int *status, cudaStream_t s, bool half_io = false);


// Decode-step attention with the group's prompt prefix read once for all G samples.
// Scratch: pre_o fp32 [B][Hq][hd] and pre_ml float2 [B][Hq] (prefix partials between the two kernels).
struct DecodeAttnArgs {
  const CUtensorMap *tmKV;        // whole KV pool as [rows][hd] bf16, box {64, 2 * page}, 128-byte swizzle
  const __nv_bfloat16 *q;         // [B][Hq][hd]
  __nv_bfloat16 *out;             // [B][Hq][hd]
  float *pre_o;
  float2 *pre_ml;
  const int32_t *page_table;      // row s = sequence s
  int pt_width;
  const int32_t *row_pos;         // position of the token each sequence feeds in this step
  const int32_t *full_pages;      // full prompt pages (shared by the group) per sequence
  int layer_row0;                 // first row of this layer in the pool's row space
  int P, G, Hq, Hkv, hd, n_pages;
  int *status;
  const int32_t *row_done;        // optional, per sequence: non-zero = ended, its suffix CTAs return at once
  int *work = nullptr;            // two zeroed ints: item counter of the resident suffix kernel, which leaves
                                  // them zero again (null: one suffix CTA per (sequence, kv head))
  int half_io = 0;                // 1: q, the pool and out hold IEEE half values; probabilities are rounded to half
  int suffix_impl = 0;            // 0: choose; 1: always one suffix CTA per (sequence, kv head)
  int prefix_impl = 0;            // 0: choose; 1: always one prefix CTA per 16-row tile
  const int32_t *out_row = nullptr;   // compacted step: row of `out` each sequence writes (null: its own)
};
// Causal attention of a chunk of R prompt tokens (rows of q / out) over the paged cache; row r belongs
// to page-table row row_pt[r] at position row_pos[r]; consecutive rows of one prompt have consecutive
// positions.  Needs 16-token pages and Hq / Hkv in {1, 2, 4, 8} (attention_decode_supported).
struct PrefillAttnArgs {
  const CUtensorMap *tmKV;        // as in DecodeAttnArgs
  const __nv_bfloat16 *q;         // [R][Hq][hd]
  __nv_bfloat16 *out;             // [R][Hq][hd]
  const int32_t *row_pt, *row_pos;
  const int32_t *page_table;
  int pt_width, R;
  int layer_row0;
  int Hq, Hkv, hd, n_pages;
  int *status;
  int half_io;
};
cudaError_t attention_prefill_launch(const PrefillAttnArgs &a, cudaStream_t s);
cudaError_t attention_decode_configure();
bool attention_decode_supported(int hd, int page_size, int Hq, int Hkv);
cudaError_t attention_decode_launch(const DecodeAttnArgs &a, cudaStream_t s);

}  // namespace echo

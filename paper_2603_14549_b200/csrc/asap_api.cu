// Host side of libasap: context and scratch memory, argument validation, tensor-map
// creation and the launch sequence of each C-ABI entry point declared in include/asap.h.
#include <cuda.h>
#include <cuda_runtime.h>
#include <math.h>
#include <stdarg.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include <new>
#include <utility>

#include "../../include/asap.h"
#include "kernels_stream.cuh"
#include "kernels_tc.cuh"
#include "kernels_attn.cuh"

using namespace asap;

namespace {

char g_init_error[256] = "";
constexpr int PROF_MAX_EVENTS = 16384;
constexpr int PROF_MAX_KERNELS = 32;

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *,
                                  const cuuint64_t *, const cuuint64_t *, const cuuint32_t *,
                                  const cuuint32_t *, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

inline size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

}  // namespace

struct asap_ctx {
  int device = 0, num_sms = 1;
  size_t cap_tokens = 0, cap_keep_rows = 0;
  int cap_B = 0, cap_H = 0, cap_D = 0;
  size_t cap_chunks = 0;      // rows of the query-sum partial buffer
  uint8_t *arena = nullptr;   // one allocation, carved below
  SampleDesc *desc = nullptr;
  float *qsum_partial = nullptr, *qbar = nullptr, *score_partial = nullptr, *inv_norm = nullptr,
        *kept_inv = nullptr;
  unsigned int *cnt_qsum = nullptr, *cnt_mass = nullptr, *cnt_score = nullptr, *cnt_sim = nullptr,
               *cnt_tiles = nullptr, *cnt_work = nullptr;
  float *mass_partial = nullptr;    // [B, H, max_vis] per-head attention masses written by the score kernel
  long long fuse_mass_min_tokens = 50000;   // B * max_vis from which the attention mass rides in the score kernel
  long long sim_pair_min_blocks = 0;        // blocks from which the similarity takes two row tiles per block (0: half the SM count)
  int sim_pair_stages = 0;                  // stages of that form (0: what fits 192 KB)
  int sim_cluster = 1;                      // 0: sliced similarity launches add their partials through global memory
  float *sim_part = nullptr;        // partial dot products / squared norms of a sliced similarity GEMM
  size_t sim_part_bytes = 0, cap_tiles = 0;
  int32_t *role = nullptr, *seg = nullptr, *members = nullptr;
  int2 *member_meta = nullptr;              // (visual index, merge weight) beside every entry of `members`
  __nv_bfloat16 *kept_rows = nullptr;
  uint32_t *status = nullptr;
  EncodeTiledFn encode = nullptr;
  cudaStream_t side = nullptr;            // second stream for the mass kernels of asap_prune_step
  cudaEvent_t ev_fork = nullptr, ev_desc = nullptr, ev_join = nullptr;
  uint64_t launches = 0;
  long long wait_limit = TC_WAIT_LIMIT;   // clock cycles a wait of the tensor-core kernels may take (asap_debug_wait_limit)
  size_t counters_off = 0, counters_bytes = 0, tiles_off = 0, tiles_bytes = 0;   // the kernels' hand-shake counters in the arena
  char err[512] = "";
  // per-kernel timing (asap_profile): one event before every launch, one at the end of a call
  bool prof_on = false;
  cudaEvent_t *prof_ev = nullptr;
  const char **prof_name = nullptr;   // kernel that starts at the event; nullptr = end of a call
  int prof_used = 0;
  asap_kernel_time prof_acc[PROF_MAX_KERNELS];
  int prof_nacc = 0;
};

namespace {

asap_status fail(asap_ctx *ctx, asap_status st, const char *fmt, ...) {
  va_list ap;
  va_start(ap, fmt);
  vsnprintf(ctx ? ctx->err : g_init_error, ctx ? sizeof(ctx->err) : sizeof(g_init_error), fmt, ap);
  va_end(ap);
  return st;
}

bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// 2-D bf16 tensor [rows, cols] row-major, box = 64 columns x box_rows rows, 128-byte swizzle.
bool make_map(asap_ctx *ctx, CUtensorMap *map, const void *ptr, uint64_t rows, uint64_t cols,
              uint32_t box_rows, uint64_t pitch_elems = 0) {
  cuuint64_t dims[2] = {cols, rows};
  cuuint64_t strides[1] = {(pitch_elems ? pitch_elems : cols) * 2};
  cuuint32_t box[2] = {64, box_rows};
  cuuint32_t estr[2] = {1, 1};
  CUresult r = ctx->encode(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(ptr), dims,
                           strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                           CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                           CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS;
}

// ---- validation of everything the host can see -------------------------------------------
enum Need : unsigned {
  NEED_QK = 1u, NEED_HIDDEN = 2u, NEED_SCORE_OUT = 4u, NEED_SELECT_OUT = 8u, NEED_MERGE_OUT = 16u
};

asap_status validate(asap_ctx *ctx, const asap_inputs *in, const asap_params *p,
                     const asap_outputs *out, unsigned need) {
  if (!ctx) return fail(nullptr, ASAP_ERR_INVALID, "null context");
  ctx->err[0] = 0;
  if (!in || !p || !out) return fail(ctx, ASAP_ERR_INVALID, "null inputs / params / outputs struct");
  if (in->B <= 0 || in->H <= 0 || in->total_tokens <= 0)
    return fail(ctx, ASAP_ERR_INVALID, "B, H and total_tokens must be positive");
  if (in->head_dim != 128) return fail(ctx, ASAP_ERR_UNSUPPORTED, "head_dim must be 128, got %d", in->head_dim);
  if (in->D != in->H * in->head_dim) return fail(ctx, ASAP_ERR_INVALID, "D != H * head_dim");
  if (in->D > 8192) return fail(ctx, ASAP_ERR_UNSUPPORTED, "D > 8192 is not supported");
  if (in->min_vis <= 0 || in->max_vis < in->min_vis || in->max_seq < in->max_vis)
    return fail(ctx, ASAP_ERR_INVALID, "need 0 < min_vis <= max_vis <= max_seq");
  if (in->max_vis > 57344) return fail(ctx, ASAP_ERR_UNSUPPORTED, "max_vis > 57344 is not supported");
  if (in->max_rank <= 0 || in->max_rank > in->max_seq)
    return fail(ctx, ASAP_ERR_INVALID, "need 0 < max_rank <= max_seq");
  if (p->keep_k <= 0 || p->keep_k > in->min_vis)
    return fail(ctx, ASAP_ERR_INVALID, "need 0 < keep_k <= min_vis (keep_k=%d, min_vis=%d)", p->keep_k, in->min_vis);
  if (!(p->lambda_max > 0.f && p->lambda_max <= 1.f))
    return fail(ctx, ASAP_ERR_INVALID, "lambda_max must be in (0, 1]");
  if (!(p->eps > 0.f)) return fail(ctx, ASAP_ERR_INVALID, "eps must be positive");
  if (p->sim_threshold != p->sim_threshold) return fail(ctx, ASAP_ERR_INVALID, "sim_threshold is NaN");
  // capacities
  if ((size_t)in->total_tokens > ctx->cap_tokens || in->B > ctx->cap_B || in->H > ctx->cap_H ||
      in->D > ctx->cap_D)
    return fail(ctx, ASAP_ERR_WORKSPACE, "problem exceeds the capacities given to asap_init");
  if ((size_t)in->B * (size_t)in->max_vis > ctx->cap_tokens)
    return fail(ctx, ASAP_ERR_WORKSPACE, "B * max_vis exceeds max_total_tokens");
  if ((size_t)in->B * (size_t)p->keep_k > ctx->cap_keep_rows)
    return fail(ctx, ASAP_ERR_WORKSPACE, "B * keep_k exceeds max_keep_rows");
  const size_t chunks = (size_t)in->B * ((in->max_vis + QSUM_ROWS - 1) / QSUM_ROWS);
  if (chunks > ctx->cap_chunks) return fail(ctx, ASAP_ERR_WORKSPACE, "query-sum scratch too small for B * max_vis");
  if (!in->cu_seqlens || !in->vis_start || !in->vis_len || !in->text_start || !in->text_len)
    return fail(ctx, ASAP_ERR_INVALID, "null per-sample array");
  if ((in->rank_start == nullptr) != (in->rank_len == nullptr))
    return fail(ctx, ASAP_ERR_INVALID, "rank_start and rank_len must both be given or both be NULL");
  if ((need & NEED_QK) && (!in->q || !in->k)) return fail(ctx, ASAP_ERR_INVALID, "null q / k");
  if ((need & NEED_QK) && (!aligned16(in->q) || !aligned16(in->k)))
    return fail(ctx, ASAP_ERR_ALIGN, "q / k must be 16-byte aligned");
  if (need & NEED_HIDDEN) {
    if (!in->hidden || !in->pos_ids) return fail(ctx, ASAP_ERR_INVALID, "null hidden / pos_ids");
    if (!aligned16(in->hidden)) return fail(ctx, ASAP_ERR_ALIGN, "hidden must be 16-byte aligned");
  }
  if ((need & NEED_SCORE_OUT) && (!out->mass || !out->salience || !out->mask_log || !out->rank_score))
    return fail(ctx, ASAP_ERR_INVALID, "null score output (mass / salience / mask_log / rank_score)");
  if ((need & NEED_SCORE_OUT) && p->per_head_mask && !out->mask_log_heads)
    return fail(ctx, ASAP_ERR_INVALID, "per_head_mask needs asap_outputs::mask_log_heads");
  if (p->per_head_mask && (in->H & 1)) return fail(ctx, ASAP_ERR_UNSUPPORTED, "per_head_mask needs an even number of heads");
  const bool has_drops = in->max_vis > p->keep_k;   // otherwise the dropped-token arrays are empty
  if ((need & NEED_SELECT_OUT) && (!out->keep_idx || (!out->drop_idx && has_drops)))
    return fail(ctx, ASAP_ERR_INVALID, "null keep_idx / drop_idx");
  if (need & NEED_MERGE_OUT) {
    if ((!out->assign && has_drops) || !out->out_hidden || !out->out_pos || !out->src_row || !out->out_cu_seqlens)
      return fail(ctx, ASAP_ERR_INVALID, "null merge output");
    if (!aligned16(out->out_hidden)) return fail(ctx, ASAP_ERR_ALIGN, "out_hidden must be 16-byte aligned");
    const long long bound = (long long)in->total_tokens - (long long)in->B * (in->min_vis - p->keep_k);
    if (out->out_rows_capacity <= 0 || bound <= 0)
      return fail(ctx, ASAP_ERR_INVALID, "out_rows_capacity must be positive");
  }
  return ASAP_OK;
}

// Called right before a kernel is enqueued (name) and once after the last kernel of an entry
// point (nullptr): with profiling on, drops a timestamp event on the stream.
void mark(asap_ctx *ctx, const char *name, cudaStream_t st) {
  if (!ctx->prof_on || ctx->prof_used >= PROF_MAX_EVENTS) return;
  if (cudaEventRecord(ctx->prof_ev[ctx->prof_used], st) != cudaSuccess) return;
  ctx->prof_name[ctx->prof_used++] = name;
}

// Every kernel is launched with programmatic stream serialization: its blocks may be scheduled
// while the previous kernel of the stream drains, and wait (griddepcontrol.wait, first statement
// of every kernel) until that kernel has completed and its writes are visible.
template <typename... KArgs, typename... Args>
void launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args &&...args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);   // errors surface in after_launch
}

// The same for a kernel whose grid-z neighbours form thread-block clusters of `cluster_z` blocks.
template <typename... KArgs, typename... Args>
void launch_pdl_cluster_z(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, int cluster_z,
                          Args &&...args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  attr[1].id = cudaLaunchAttributeClusterDimension;
  attr[1].val.clusterDim.x = 1;
  attr[1].val.clusterDim.y = 1;
  attr[1].val.clusterDim.z = (unsigned)cluster_z;
  cfg.attrs = attr;
  cfg.numAttrs = 2;
  cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

asap_status after_launch(asap_ctx *ctx, const char *what) {
  ctx->launches += 1;
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return fail(ctx, ASAP_ERR_CUDA, "%s launch failed: %s", what, cudaGetErrorString(e));
  return ASAP_OK;
}

asap_status finish(asap_ctx *ctx, asap_status result, cudaStream_t st) {
  mark(ctx, nullptr, st);
  ctx->wait_limit = TC_WAIT_LIMIT;      // a limit set by asap_debug_wait_limit holds for one call
  return result;
}

#define ASAP_TRY(expr)                   \
  do {                                   \
    asap_status st__ = (expr);           \
    if (st__ != ASAP_OK) return st__;    \
  } while (0)

// ---- stage launchers -------------------------------------------------------------------------
PrepareArgs prepare_args(asap_ctx *ctx, const asap_inputs *in, const asap_params *p, int32_t *out_cu,
                         int out_capacity) {
  PrepareArgs a;
  a.B = in->B; a.total_tokens = in->total_tokens; a.min_vis = in->min_vis; a.max_vis = in->max_vis;
  a.max_seq = in->max_seq; a.max_rank = in->max_rank; a.keep_k = p->keep_k; a.out_capacity = out_capacity;
  a.cu_seqlens = in->cu_seqlens; a.vis_start = in->vis_start; a.vis_len = in->vis_len;
  a.text_start = in->text_start; a.text_len = in->text_len; a.rank_start = in->rank_start;
  a.rank_len = in->rank_len; a.desc = ctx->desc; a.out_cu_seqlens = out_cu; a.status = ctx->status;
  return a;
}

asap_status launch_prepare(asap_ctx *ctx, const asap_inputs *in, const asap_params *p,
                           int32_t *out_cu, int out_capacity, cudaStream_t st) {
  mark(ctx, "prepare", st);
  launch_pdl(prepare_kernel, dim3(1), dim3(256), 0, st, prepare_args(ctx, in, p, out_cu, out_capacity));
  return after_launch(ctx, "prepare");
}

// Steps 1a-1b: query sum, attention mass, salience, mask vector.  With `fold_prepare` the query-sum
// kernel also carries the device-side validation and writes the descriptors.

// Rows a block of the query-sum kernel adds up: 32, doubled (up to 128) while the grid still has eight blocks per
// SM -- every chunk costs a partial row written and read back (32 rows: 12 % on top of the queries themselves).
int qsum_rows_per_chunk(const asap_ctx *ctx, const asap_inputs *in) {
  const long long col_blocks = (in->D + QSUM_COLS - 1) / QSUM_COLS;
  int rows = QSUM_ROWS;
  while (rows < 4 * QSUM_ROWS &&
         (long long)((in->max_vis + 2 * rows - 1) / (2 * rows)) * col_blocks * in->B >= 8LL * ctx->num_sms)
    rows *= 2;
  return rows;
}

asap_status launch_mass(asap_ctx *ctx, const asap_inputs *in, const asap_params *p, const asap_outputs *out,
                        bool fold_prepare, int32_t *out_cu, int out_capacity, cudaStream_t st,
                        cudaEvent_t after_qsum = nullptr) {
  const int D = in->D, B = in->B;
  const int qrows = qsum_rows_per_chunk(ctx, in);
  const int max_chunks = (in->max_vis + qrows - 1) / qrows;
  const int col_blocks = (D + QSUM_COLS - 1) / QSUM_COLS;
  PrepareArgs pa = prepare_args(ctx, in, p, out_cu, out_capacity);
  pa.write_desc = fold_prepare ? 1 : 0;
  mark(ctx, "qsum", st);
  launch_pdl(qsum_kernel, dim3(max_chunks, col_blocks, B), dim3(QSUM_THREADS), 0, st,
             static_cast<const __nv_bfloat16 *>(in->q), pa, D, max_chunks, qrows, ctx->qsum_partial, ctx->qbar,
             ctx->cnt_qsum);
  ASAP_TRY(after_launch(ctx, "qsum"));
  if (after_qsum && cudaEventRecord(after_qsum, st) != cudaSuccess)
    return fail(ctx, ASAP_ERR_CUDA, "event after the query-sum kernel");

  const int row_blocks = (in->max_vis + MASS_ROWS - 1) / MASS_ROWS;
  if (p->per_head_mask) {
    // the per-head masses go through the scratch the score kernel fills afterwards
    mark(ctx, "mass_heads", st);
    launch_pdl(mass_heads_kernel, dim3(row_blocks, B), dim3(MASS_THREADS), (size_t)(D + 2 * in->H) * sizeof(float), st,
               static_cast<const __nv_bfloat16 *>(in->k), ctx->desc, D, in->H, in->max_vis,
               1.0f / sqrtf((float)in->head_dim), p->lambda_max, p->eps, ctx->qbar, ctx->score_partial, out->mass,
               out->salience, out->mask_log, out->mask_log_heads, out->rank_score, ctx->cnt_mass);
    return after_launch(ctx, "mass_heads");
  }
  const float scale = 1.0f / ((float)in->H * sqrtf((float)in->head_dim));
  mark(ctx, "mass_salience", st);
  launch_pdl(mass_salience_kernel, dim3(row_blocks, B), dim3(MASS_THREADS), (size_t)D * sizeof(float), st,
             static_cast<const __nv_bfloat16 *>(in->k), ctx->desc, D, in->max_vis, scale, p->lambda_max, p->eps,
             ctx->qbar, out->mass, out->salience, out->mask_log, out->rank_score, ctx->cnt_mass);
  return after_launch(ctx, "mass_salience");
}

// Steps 1c-2: Eq. 4 probabilities of the ranking rows, summed per head; optionally the head sum.
asap_status launch_rank(asap_ctx *ctx, const asap_inputs *in, const asap_params *p, const asap_outputs *out,
                        bool with_head_sum, cudaStream_t st, bool with_mass = false) {
  const int D = in->D, B = in->B;
  CUtensorMap map_q, map_k;
  if (!make_map(ctx, &map_q, in->q, (uint64_t)in->total_tokens, (uint64_t)D, 128) ||
      !make_map(ctx, &map_k, in->k, (uint64_t)in->total_tokens, (uint64_t)D, 128))
    return fail(ctx, ASAP_ERR_CUDA, "cuTensorMapEncodeTiled failed for q / k");
  ScoreArgs sa;
  sa.pa = prepare_args(ctx, in, p, nullptr, 0x7fffffff); sa.pa.write_desc = 0; sa.B = B; sa.H = in->H; sa.max_vis = in->max_vis; sa.mask_enable = p->mask_enable ? 1 : 0;
  sa.scale_log2 = 1.4426950408889634f / sqrtf((float)in->head_dim);
  sa.mask_log = p->per_head_mask ? out->mask_log_heads : out->mask_log;
  sa.mask_b_stride = p->per_head_mask ? in->H * in->max_vis : in->max_vis;
  sa.mask_h_stride = p->per_head_mask ? in->max_vis : 0;
  sa.qbar = with_mass ? ctx->qbar : nullptr; sa.mass_heads = ctx->mass_partial; sa.D = D;
  sa.partial = ctx->score_partial; sa.work = ctx->cnt_work; sa.status = ctx->status; sa.wait_limit = ctx->wait_limit;
  mark(ctx, "score", st);
  const int items = B * in->H;
  launch_pdl(score_kernel, dim3(items < ctx->num_sms ? items : ctx->num_sms), dim3(SC_THREADS), SC_SMEM_BYTES, st,
             map_q, map_k, sa);
  ASAP_TRY(after_launch(ctx, "score"));
  if (!with_head_sum) return ASAP_OK;
  mark(ctx, "head_sum", st);
  launch_pdl(head_sum_kernel, dim3((in->max_vis + 255) / 256, B), dim3(256), 0, st, ctx->desc, in->H, in->max_vis,
             ctx->score_partial, out->rank_score);
  return after_launch(ctx, "head_sum");
}

// true when a similarity kernel will run for this call (it then writes assign / best_sim of every
// dropped token itself)
bool merging(const asap_inputs *in, const asap_params *p) { return p->merge_enable && in->max_vis > p->keep_k; }

// `fused_head_sum`: the ranking scores are still per-head sums in scratch (the score kernel ran
// without its head-sum kernel); the selection adds the heads itself and writes out->rank_score.
asap_status launch_select(asap_ctx *ctx, const asap_inputs *in, const asap_params *p,
                          const float *rank_score, const asap_outputs *out, bool with_merge,
                          bool fused_head_sum, cudaStream_t st) {
  mark(ctx, "select", st);
  launch_pdl(select_kernel, dim3(in->B), dim3(SELECT_THREADS), (size_t)in->max_vis * sizeof(uint32_t), st,
             rank_score, ctx->desc, in->max_vis, p->keep_k, out->keep_idx, out->drop_idx, ctx->role,
             with_merge ? out->assign : nullptr, with_merge ? out->best_sim : nullptr, merging(in, p) ? 1 : 0,
             fused_head_sum ? ctx->score_partial : nullptr, in->H, fused_head_sum ? out->rank_score : nullptr);
  return after_launch(ctx, "select");
}

// Step 4a: kept rows gathered, cosine similarity and assignment, CSR of the assignment.
// `salience`: the merge weights if they are complete when this is enqueued (the grouping then copies each
// member's weight beside its index for the merge kernel), else nullptr.
asap_status launch_merge_front(asap_ctx *ctx, const asap_inputs *in, const asap_params *p, const float *salience,
                               const int32_t *keep_idx, const int32_t *drop_idx, const asap_outputs *out,
                               cudaStream_t st) {
  const int B = in->B, D = in->D, k = p->keep_k;
  if (merging(in, p)) {
    mark(ctx, "kept_gather", st);
    launch_pdl(kept_gather_kernel, dim3(dim3((k + GATHER_THREADS / 32 - 1) / (GATHER_THREADS / 32), B)), dim3(GATHER_THREADS), 0, st, 
        static_cast<const __nv_bfloat16 *>(in->hidden), ctx->desc, D, k, keep_idx, ctx->kept_rows, ctx->kept_inv);
    ASAP_TRY(after_launch(ctx, "kept_gather"));

    int n_nt = (k + 255) / 256;
    int n_tile = (((k + n_nt - 1) / n_nt) + 15) & ~15;
    // Small problems leave most SMs without a row tile: slice the hidden dimension over several
    // blocks (at most 8, a divisor of the number of 128-column steps, scratch permitting), up to
    // two blocks per SM.
    int max_mt = (in->max_vis + 127) / 128;              // row tiles when every visual row is multiplied
    const int n_kb = D / 128;
    // The slice count minimises a simple cost: streaming a row tile takes about 1 us per 128-column
    // step of the slice, and the last slice adds up keep_k * slices partial values per row at about
    // 0.5 us per 64 of them.
    // With one slot tile (at most 256 kept slots) the slices of a row tile run as one thread-block cluster and
    // add their partial products through distributed shared memory: no partials in global memory, no
    // last-block pass over them; the adding then costs about a quarter of a microsecond per slice.
    const bool cluster_ok = ctx->sim_cluster != 0 && n_nt == 1;
    int splits = 1;
    float best_cost = (float)n_kb;
    for (int c = 2; c <= 8; ++c) {
      if (n_kb % c != 0) continue;
      if ((long long)max_mt * B * c > 2LL * ctx->num_sms) break;
      if ((size_t)B * max_mt * c * ((size_t)k + 1) * 128 * sizeof(float) > ctx->sim_part_bytes) break;
      if ((size_t)B * max_mt > ctx->cap_tiles) break;
      const float cost = (float)n_kb / c + (cluster_ok ? 0.25f * c : 0.5f * (float)k * c / 64.f);
      if (cost < best_cost) { best_cost = cost; splits = c; }
    }
    // a grid between one and two blocks per SM runs as one wave if two blocks fit on an SM:
    // give each block half of the shared memory and of the tensor memory then
    // Several slot tiles whose accumulators fit tensor memory together: one pass over the hidden
    // dimension with all of them live, so the visual rows are read once (a stage is then one 64-column
    // block of the rows and of every slot tile).
    // Taken only while three such stages still fit (up to 384 slots): with two, the shorter copies
    // cost more than the second read of the rows (measured: 320 slots 87 -> 77 us, 510 slots 91 -> 96 us).
    // The row operand: every visual row by tiled copies (a fifth to a half of the products are then thrown
    // away), or the dropped rows alone, gathered (half the bytes per clock, four more warps, one block per
    // SM).  Gathering is taken for batches large enough not to be sliced, from two fifths of the rows kept
    // (measured at a fifth, 576 of 2880: 1.11 ms gathered against 1.04 ms tiled; at a half, 1152 of 2304:
    // 0.56 ms against 0.92 ms).
    const bool gather_rows = splits == 1 && (long long)k * 5 >= 2LL * in->max_vis &&
                             (long long)max_mt * B > ctx->num_sms;
    // Every visual row, two row tiles per block, the kept slots dealt in groups of at most 256 to the
    // blocks of a pair, one pass each: fewer bytes out of L2 per product, which is what bounds the
    // similarity of a large batch.  Taken when that grid fills at least half of the SMs (measured: 96 blocks
    // 91 -> 75 us, 144 blocks 78 -> 72 us, 2304 blocks 1038 -> 845 us; 48 blocks 39 -> 57 us, where slicing
    // the hidden dimension over more blocks is worth more).
    {
      const int pairs = (in->max_vis + 255) / 256;
      const int pg = (k + 255) / 256;
      const int ptile = (((k + pg - 1) / pg) + 15) & ~15;
      const long long min_blocks = ctx->sim_pair_min_blocks > 0 ? ctx->sim_pair_min_blocks : (ctx->num_sms + 1) / 2;
      const int pstage = 2 * SIM_A_BYTES + ptile * 128;
      int pstages = ctx->sim_pair_stages > 0 ? ctx->sim_pair_stages : (192 * 1024) / pstage;
      if (pstages > SIM_MAX_STAGES) pstages = SIM_MAX_STAGES;
      const size_t psmem = (size_t)pstages * pstage + SIM_BOOK_BYTES + 1024;
      if (!gather_rows && D % 64 == 0 && (long long)pairs * B * pg >= min_blocks &&
          (size_t)B * pairs <= ctx->cap_tiles && pstages >= 2 && psmem <= 227 * 1024 &&
          (size_t)B * pairs * (size_t)(pg * 512 + 256) * sizeof(float) <= ctx->sim_part_bytes &&
          (size_t)(SIMP_THREADS / 32 + 1) * k * sizeof(int) <= (size_t)pstages * pstage) {
        uint32_t pcols = 32;
        while ((int)pcols < 2 * ptile) pcols <<= 1;
        CUtensorMap map_h, map_kept;
        if (!make_map(ctx, &map_h, in->hidden, (uint64_t)in->total_tokens, (uint64_t)D, 128) ||
            !make_map(ctx, &map_kept, ctx->kept_rows, (uint64_t)B * (uint64_t)k, (uint64_t)D, (uint32_t)ptile))
          return fail(ctx, ASAP_ERR_CUDA, "cuTensorMapEncodeTiled failed for hidden / kept rows");
        SimArgs sa;
        sa.desc = ctx->desc; sa.D = D; sa.max_vis = in->max_vis; sa.keep_k = k; sa.n_tile = ptile;
        sa.n_nt = 1; sa.stages = pstages; sa.splits = 1; sa.max_mt = pairs; sa.tmem_cols = pcols;
        sa.wide = 1; sa.groups = pg; sa.cluster = 0; sa.threshold = p->sim_threshold;
        sa.drop_idx = nullptr; sa.role = ctx->role;
        sa.hidden = static_cast<const __nv_bfloat16 *>(in->hidden); sa.kept_inv = ctx->kept_inv; sa.assign = out->assign;
        sa.best_sim = out->best_sim; sa.seg = ctx->seg; sa.members = ctx->members; sa.counters = ctx->cnt_sim;
        sa.tile_counters = ctx->cnt_tiles; sa.part = ctx->sim_part; sa.ss_part = nullptr; sa.smat = nullptr;
        sa.drop_all = drop_idx; sa.salience = salience; sa.member_meta = salience ? ctx->member_meta : nullptr;
        sa.status = ctx->status; sa.wait_limit = ctx->wait_limit;
        mark(ctx, "sim", st);
        launch_pdl(sim_pair_kernel, dim3(pairs * pg, B), dim3(SIMP_THREADS), psmem, st, map_h, map_kept, sa);
        return after_launch(ctx, "sim");
      }
    }
    if (gather_rows) max_mt = (in->max_vis - k + 127) / 128;
    bool wide = n_nt >= 2 && n_nt * n_tile <= 512 && 3 * (SIM_A_BYTES + n_nt * n_tile * 128) <= 192 * 1024;
    // More slots than that, and enough row tiles that the hidden dimension is not sliced: the slot tiles are
    // dealt to several blocks per row tile (groups of at most 384 slots = one or two tiles), each a single
    // pass in the layout above; the last block of a row tile combines the groups' best slots.  Several
    // passes inside one block would read the dropped rows from memory once per pass: the rows that all
    // resident blocks hold between two passes do not fit L2.
    int groups = 1;
    if (gather_rows && !wide && n_nt >= 2 && D % 64 == 0 && (size_t)B * max_mt <= ctx->cap_tiles) {
      int g = (k + 383) / 384;
      const int per_group = (k + g - 1) / g;
      const int tiles_g = per_group > 256 ? 2 : 1;
      const int tile_g = (((per_group + tiles_g - 1) / tiles_g) + 15) & ~15;
      g = (k + tiles_g * tile_g - 1) / (tiles_g * tile_g);
      if ((size_t)B * max_mt * g * 256 * sizeof(float) <= ctx->sim_part_bytes) {
        groups = g; n_nt = tiles_g; n_tile = tile_g; wide = true;
      }
    }
    const int stage_bytes = 2 * (SIM_A_BYTES + n_tile * 128);   // two adjacent 64-column blocks per stage
    uint32_t tmem_cols = 32;
    while ((int)tmem_cols < (wide ? n_nt * n_tile : 2 * n_tile)) tmem_cols <<= 1;
    const int stage_bytes_used = wide ? SIM_A_BYTES + n_nt * n_tile * 128 : stage_bytes;
    const long long ctas = (long long)max_mt * B * splits * groups;
    const bool two_per_sm = !wide && ctas > ctx->num_sms && ctas <= 2LL * ctx->num_sms && tmem_cols <= 256 &&
                            2 * stage_bytes <= 96 * 1024;
    // at most 192 KB of tiles: the block then fits the 196 KB shared-memory carve-out, which leaves
    // the SM its 32 KB of L1
    int stages = ((two_per_sm ? 96 : 192) * 1024) / stage_bytes_used;
    if (stages > SIM_MAX_STAGES) stages = SIM_MAX_STAGES;
    const size_t smem = (size_t)stages * stage_bytes_used + SIM_BOOK_BYTES + 1024;
    const int sim_threads = gather_rows ? SIM_THREADS : SIM_THREADS_TILED;
    if ((size_t)(sim_threads / 32 + 1) * k * sizeof(int) > (size_t)stages * stage_bytes_used)
      return fail(ctx, ASAP_ERR_UNSUPPORTED, "keep_k = %d is too large for the merge path", k);
    CUtensorMap map_h, map_kept;
    if (!make_map(ctx, &map_h, in->hidden, (uint64_t)in->total_tokens, (uint64_t)D, 128) ||
        !make_map(ctx, &map_kept, ctx->kept_rows, (uint64_t)B * (uint64_t)k, (uint64_t)D, (uint32_t)n_tile))
      return fail(ctx, ASAP_ERR_CUDA, "cuTensorMapEncodeTiled failed for hidden / kept rows");
    SimArgs sa;
    sa.desc = ctx->desc; sa.D = D; sa.max_vis = in->max_vis; sa.keep_k = k; sa.n_tile = n_tile;
    sa.n_nt = n_nt; sa.stages = stages; sa.splits = splits; sa.max_mt = max_mt; sa.tmem_cols = tmem_cols;
    sa.wide = wide ? 1 : 0;
    sa.groups = groups;
    const bool cluster = cluster_ok && splits > 1 && !wide && !gather_rows &&
                         (size_t)k * 512 + 4096 + (size_t)splits * 1536 <= (size_t)stages * stage_bytes_used;
    sa.cluster = cluster ? 1 : 0;
    sa.threshold = p->sim_threshold;
    sa.drop_idx = gather_rows ? drop_idx : nullptr; sa.role = ctx->role;
    sa.hidden = static_cast<const __nv_bfloat16 *>(in->hidden); sa.kept_inv = ctx->kept_inv; sa.assign = out->assign;
    sa.best_sim = out->best_sim; sa.seg = ctx->seg; sa.members = ctx->members; sa.counters = ctx->cnt_sim;
    sa.tile_counters = ctx->cnt_tiles; sa.part = ctx->sim_part;
    sa.ss_part = ctx->sim_part + (size_t)B * max_mt * splits * (size_t)k * 128;
    sa.smat = nullptr;
    sa.drop_all = drop_idx; sa.salience = salience; sa.member_meta = salience ? ctx->member_meta : nullptr;
    sa.status = ctx->status; sa.wait_limit = ctx->wait_limit;
    mark(ctx, "sim", st);
    if (gather_rows)
      launch_pdl(sim_kernel<true>, dim3(max_mt * groups, B, splits), dim3(SIM_THREADS), smem, st, map_h, map_kept, sa);
    else if (cluster)
      launch_pdl_cluster_z(sim_kernel<false>, dim3(max_mt, B, splits), dim3(SIM_THREADS_TILED), smem, st, splits, map_h,
                           map_kept, sa);
    else
      launch_pdl(sim_kernel<false>, dim3(max_mt * groups, B, splits), dim3(SIM_THREADS_TILED), smem, st, map_h, map_kept, sa);
    ASAP_TRY(after_launch(ctx, "sim"));
  }
  return ASAP_OK;
}

// Steps 4b-5: weighted merge and compaction (the first consumer of the salience).
asap_status launch_merge_back(asap_ctx *ctx, const asap_inputs *in, const asap_params *p,
                              const float *salience, const int32_t *keep_idx, const int32_t *drop_idx,
                              const asap_outputs *out, cudaStream_t st, bool grouped_with_weights = false) {
  const int B = in->B, D = in->D, k = p->keep_k;
  const bool do_merge = merging(in, p);
  MergeArgs ma;
  ma.hidden = static_cast<const __nv_bfloat16 *>(in->hidden); ma.pos_ids = in->pos_ids; ma.desc = ctx->desc;
  ma.D = D; ma.max_vis = in->max_vis; ma.keep_k = k; ma.merge_enable = do_merge ? 1 : 0; ma.eps = p->eps;
  ma.salience = salience; ma.keep_idx = keep_idx; ma.drop_idx = drop_idx; ma.seg = ctx->seg;
  ma.members = ctx->members; ma.member_meta = (do_merge && grouped_with_weights) ? ctx->member_meta : nullptr;
  ma.out_hidden = static_cast<__nv_bfloat16 *>(out->out_hidden);
  ma.out_pos = out->out_pos; ma.src_row = out->src_row;
  const int copy_rows = in->max_seq - in->min_vis;   // prefix + suffix rows of the longest sequence, at most
  const dim3 grid(k + (copy_rows + MERGE_COPY_ROWS - 1) / MERGE_COPY_ROWS, B);
  const int nv = (D / 8 + MERGE_THREADS - 1) / MERGE_THREADS;
  mark(ctx, "merge_compact", st);
  switch (nv) {
    case 1: launch_pdl(merge_compact_kernel<1>, dim3(grid), dim3(MERGE_THREADS), 0, st, ma); break;
    case 2:
      if ((long long)grid.x * grid.y >= 32LL * 3 * ctx->num_sms)       // more than 32 waves of three blocks per SM
        launch_pdl(merge_compact_kernel<2, true>, dim3(grid), dim3(MERGE_THREADS), 0, st, ma);
      else
        launch_pdl(merge_compact_kernel<2>, dim3(grid), dim3(MERGE_THREADS), 0, st, ma);
      break;
    case 3: launch_pdl(merge_compact_kernel<3>, dim3(grid), dim3(MERGE_THREADS), 0, st, ma); break;
    default: launch_pdl(merge_compact_kernel<4>, dim3(grid), dim3(MERGE_THREADS), 0, st, ma); break;
  }
  return after_launch(ctx, "merge_compact");
}

asap_status launch_merge(asap_ctx *ctx, const asap_inputs *in, const asap_params *p,
                         const float *salience, const int32_t *keep_idx, const int32_t *drop_idx,
                         const asap_outputs *out, cudaStream_t st) {
  ASAP_TRY(launch_merge_front(ctx, in, p, salience, keep_idx, drop_idx, out, st));
  return launch_merge_back(ctx, in, p, salience, keep_idx, drop_idx, out, st, true);
}

// Sec. 4.2 inside the kept set: kept rows gathered, their keep_k x keep_k cosine matrix, routing.
size_t route_smat_bytes(int B, int k) { return align_up((size_t)B * k * k * sizeof(float), 256); }
size_t route_mask_bytes(int B, int k) { return (size_t)B * k * ((k + 31) / 32) * sizeof(uint32_t); }

asap_status launch_consolidate_front(asap_ctx *ctx, const asap_inputs *in, const asap_params *p,
                                     const float *mass, const float *salience, const int32_t *keep_idx,
                                     const int32_t *drop_idx, void *scratch, const asap_outputs *out,
                                     int32_t *n_absorbed, cudaStream_t st) {
  const int B = in->B, D = in->D, k = p->keep_k;
  mark(ctx, "kept_gather", st);
  launch_pdl(kept_gather_kernel, dim3((k + GATHER_THREADS / 32 - 1) / (GATHER_THREADS / 32), B), dim3(GATHER_THREADS), 0, st,
             static_cast<const __nv_bfloat16 *>(in->hidden), ctx->desc, D, k, keep_idx, ctx->kept_rows, ctx->kept_inv);
  ASAP_TRY(after_launch(ctx, "kept_gather"));

  float *smat = static_cast<float *>(scratch);
  {
    // large batches: two row tiles per block, the slots dealt in groups to neighbouring blocks (see the similarity
    // launch of the merge); here every product is used, the matrix being square
    const int pairs = (k + 255) / 256;
    const int pg = (k + 255) / 256;
    const int ptile = (((k + pg - 1) / pg) + 15) & ~15;
    const long long min_blocks = ctx->sim_pair_min_blocks > 0 ? ctx->sim_pair_min_blocks : (ctx->num_sms + 1) / 2;
    const int pstage = 2 * SIM_A_BYTES + ptile * 128;
    int pstages = ctx->sim_pair_stages > 0 ? ctx->sim_pair_stages : (192 * 1024) / pstage;
    if (pstages > SIM_MAX_STAGES) pstages = SIM_MAX_STAGES;
    const size_t psmem = (size_t)pstages * pstage + SIM_BOOK_BYTES + 1024;
    if (D % 64 == 0 && (long long)pairs * B * pg >= min_blocks && pstages >= 2 && psmem <= 227 * 1024) {
      uint32_t pcols = 32;
      while ((int)pcols < 2 * ptile) pcols <<= 1;
      CUtensorMap map_a, map_b;
      if (!make_map(ctx, &map_a, ctx->kept_rows, (uint64_t)B * (uint64_t)k, (uint64_t)D, 128) ||
          !make_map(ctx, &map_b, ctx->kept_rows, (uint64_t)B * (uint64_t)k, (uint64_t)D, (uint32_t)ptile))
        return fail(ctx, ASAP_ERR_CUDA, "cuTensorMapEncodeTiled failed for the kept rows");
      SimArgs sa;
      sa.desc = ctx->desc; sa.D = D; sa.max_vis = in->max_vis; sa.keep_k = k; sa.n_tile = ptile;
      sa.n_nt = 1; sa.stages = pstages; sa.splits = 1; sa.max_mt = pairs; sa.tmem_cols = pcols;
      sa.wide = 1; sa.groups = pg; sa.cluster = 0; sa.threshold = p->sim_threshold;
      sa.drop_idx = nullptr; sa.role = nullptr; sa.drop_all = nullptr; sa.hidden = nullptr; sa.kept_inv = ctx->kept_inv;
      sa.assign = nullptr; sa.best_sim = nullptr; sa.seg = nullptr; sa.members = nullptr; sa.counters = nullptr;
      sa.tile_counters = nullptr; sa.part = nullptr; sa.ss_part = nullptr; sa.smat = smat; sa.salience = nullptr;
      sa.member_meta = nullptr; sa.status = ctx->status; sa.wait_limit = ctx->wait_limit;
      mark(ctx, "sim_kept", st);
      launch_pdl(sim_pair_kernel, dim3(pairs * pg, B), dim3(SIMP_THREADS), psmem, st, map_a, map_b, sa);
      ASAP_TRY(after_launch(ctx, "sim_kept"));
      goto routing;
    }
  }
  {
  const int n_nt = (k + 255) / 256;
  const int n_tile = (((k + n_nt - 1) / n_nt) + 15) & ~15;
  const int stage_bytes = 2 * (SIM_A_BYTES + n_tile * 128);
  uint32_t tmem_cols = 32;
  while ((int)tmem_cols < 2 * n_tile) tmem_cols <<= 1;
  // slices of the hidden dimension, chosen by the cost model of the similarity launch
  const int max_mt = (k + 127) / 128;
  const int n_kb = D / 128;
  const bool cluster_ok = ctx->sim_cluster != 0 && n_nt == 1;   // slices as a thread-block cluster (see the similarity launch)
  int splits = 1;
  float best_cost = (float)n_kb;
  for (int c = 2; c <= 8; ++c) {
    if (n_kb % c != 0) continue;
    if ((long long)max_mt * B * c > 2LL * ctx->num_sms) break;
    if ((size_t)B * max_mt * c * ((size_t)k + 1) * 128 * sizeof(float) > ctx->sim_part_bytes) break;
    if ((size_t)B * max_mt > ctx->cap_tiles) break;
    const float cost = (float)n_kb / c + (cluster_ok ? 0.25f * c : 0.5f * (float)k * c / 64.f);
    if (cost < best_cost) { best_cost = cost; splits = c; }
  }
  const long long ctas = (long long)max_mt * B * splits;
  const bool two_per_sm = ctas > ctx->num_sms && ctas <= 2LL * ctx->num_sms && tmem_cols <= 256 &&
                          2 * stage_bytes <= 96 * 1024;
  int stages = ((two_per_sm ? 96 : 192) * 1024) / stage_bytes;
  if (stages > SIM_MAX_STAGES) stages = SIM_MAX_STAGES;
  const size_t smem = (size_t)stages * stage_bytes + SIM_BOOK_BYTES + 1024;
  CUtensorMap map_a, map_b;
  if (!make_map(ctx, &map_a, ctx->kept_rows, (uint64_t)B * (uint64_t)k, (uint64_t)D, 128) ||
      !make_map(ctx, &map_b, ctx->kept_rows, (uint64_t)B * (uint64_t)k, (uint64_t)D, (uint32_t)n_tile))
    return fail(ctx, ASAP_ERR_CUDA, "cuTensorMapEncodeTiled failed for the kept rows");
  SimArgs sa;
  sa.desc = ctx->desc; sa.D = D; sa.max_vis = in->max_vis; sa.keep_k = k; sa.n_tile = n_tile;
  sa.n_nt = n_nt; sa.stages = stages; sa.splits = splits; sa.max_mt = max_mt; sa.tmem_cols = tmem_cols;
  sa.wide = 0;
  sa.groups = 1;
  const bool cluster = cluster_ok && splits > 1 &&
                       (size_t)k * 512 + 4096 + (size_t)splits * 1536 <= (size_t)stages * stage_bytes;
  sa.cluster = cluster ? 1 : 0;
  sa.threshold = p->sim_threshold;
  sa.drop_idx = nullptr; sa.role = nullptr; sa.hidden = nullptr; sa.kept_inv = ctx->kept_inv; sa.assign = nullptr; sa.best_sim = nullptr;
  sa.seg = nullptr; sa.members = nullptr; sa.counters = nullptr; sa.tile_counters = ctx->cnt_tiles;
  sa.part = ctx->sim_part; sa.ss_part = ctx->sim_part + (size_t)B * max_mt * splits * (size_t)k * 128;
  sa.smat = smat; sa.drop_all = nullptr; sa.salience = nullptr; sa.member_meta = nullptr;
  sa.status = ctx->status; sa.wait_limit = ctx->wait_limit;
  mark(ctx, "sim_kept", st);
  if (cluster)
    launch_pdl_cluster_z(sim_kernel<false>, dim3(max_mt, B, splits), dim3(SIM_THREADS_TILED), smem, st, splits, map_a, map_b, sa);
  else
    launch_pdl(sim_kernel<false>, dim3(max_mt, B, splits), dim3(SIM_THREADS_TILED), smem, st, map_a, map_b, sa);
  ASAP_TRY(after_launch(ctx, "sim_kept"));
  }
routing:
  RouteArgs ra;
  ra.desc = ctx->desc; ra.max_vis = in->max_vis; ra.keep_k = k; ra.kw = (k + 31) / 32;
  ra.threshold = p->sim_threshold; ra.smat = smat;
  const size_t fixed_words = 5 * (size_t)k;
  const size_t tail_words = (size_t)(in->max_vis - k) + (size_t)in->max_vis;
  const size_t mask_words = (size_t)k * ra.kw;
  const bool mask_in_smem = (fixed_words + (mask_words > tail_words ? mask_words : tail_words)) * 4 <= 200 * 1024;
  ra.mask_g = mask_in_smem ? nullptr
                           : reinterpret_cast<uint32_t *>(static_cast<uint8_t *>(scratch) + route_smat_bytes(B, k));
  const size_t route_smem = (fixed_words + (mask_in_smem && mask_words > tail_words ? mask_words : tail_words)) * 4;
  if (route_smem > 224 * 1024)
    return fail(ctx, ASAP_ERR_UNSUPPORTED, "max_vis = %d is too large for the routing kernel", in->max_vis);
  ra.salience = salience; ra.mass = mass; ra.keep_idx = keep_idx; ra.drop_idx = drop_idx;
  ra.final_keep = out->keep_idx; ra.src_idx = out->drop_idx; ra.src_assign = out->assign;
  ra.seg = ctx->seg; ra.members = ctx->members; ra.n_absorbed = n_absorbed; ra.src_sim = out->best_sim;
  mark(ctx, "route", st);
  launch_pdl(route_kernel, dim3(B), dim3(ROUTE_THREADS), route_smem, st, ra);
  return after_launch(ctx, "route");
}

}  // namespace

// =================================================================================================
// C ABI
// =================================================================================================
extern "C" {

asap_status asap_init(asap_ctx **ctx_out, int device, size_t max_total_tokens, int max_B, int max_H,
                      int max_D, size_t max_keep_rows) {
  g_init_error[0] = 0;
  if (!ctx_out) return fail(nullptr, ASAP_ERR_INVALID, "asap_init: null ctx pointer");
  *ctx_out = nullptr;
  if (max_total_tokens == 0 || max_B <= 0 || max_H <= 0 || max_D <= 0 || max_D % 8 != 0)
    return fail(nullptr, ASAP_ERR_INVALID, "asap_init: capacities must be positive, max_D a multiple of 8");
  if (max_total_tokens > 0x7fffffffULL) return fail(nullptr, ASAP_ERR_INVALID, "asap_init: max_total_tokens too large");
  if (max_keep_rows == 0) max_keep_rows = max_total_tokens;
  cudaError_t e = cudaSetDevice(device);
  if (e != cudaSuccess) return fail(nullptr, ASAP_ERR_CUDA, "cudaSetDevice(%d): %s", device, cudaGetErrorString(e));
  cudaDeviceProp prop;
  e = cudaGetDeviceProperties(&prop, device);
  if (e != cudaSuccess) return fail(nullptr, ASAP_ERR_CUDA, "cudaGetDeviceProperties: %s", cudaGetErrorString(e));
  if (prop.major != 10)
    return fail(nullptr, ASAP_ERR_UNSUPPORTED, "libasap is built for sm_100a only; device %d is sm_%d%d", device,
                prop.major, prop.minor);
  asap_ctx *ctx = new (std::nothrow) asap_ctx();
  if (!ctx) return fail(nullptr, ASAP_ERR_CUDA, "out of host memory");
  ctx->device = device;
  ctx->num_sms = prop.multiProcessorCount;
  ctx->cap_tokens = max_total_tokens; ctx->cap_B = max_B; ctx->cap_H = max_H; ctx->cap_D = max_D;
  ctx->cap_keep_rows = max_keep_rows;
  ctx->cap_chunks = max_total_tokens / QSUM_ROWS + 2 * (size_t)max_B;

  void *fn = nullptr;
  cudaDriverEntryPointQueryResult qres;
  e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres);
  if (e != cudaSuccess || qres != cudaDriverEntryPointSuccess || !fn) {
    delete ctx;
    return fail(nullptr, ASAP_ERR_CUDA, "cuTensorMapEncodeTiled is not available from the driver");
  }
  ctx->encode = reinterpret_cast<EncodeTiledFn>(fn);

  const size_t T = max_total_tokens, Bc = (size_t)max_B, Hc = (size_t)max_H, Dc = (size_t)max_D;
  const size_t col_blocks = (Dc + QSUM_COLS - 1) / QSUM_COLS;
  size_t off = 0;
  auto carve = [&](size_t bytes) { size_t o = off; off = align_up(off + bytes, 256); return o; };
  const size_t o_desc = carve(Bc * sizeof(SampleDesc));
  const size_t o_qpart = carve(ctx->cap_chunks * Dc * sizeof(float));
  const size_t o_qbar = carve(Bc * Dc * sizeof(float));
  const size_t o_spart = carve(Hc * T * sizeof(float));
  const size_t o_mpart = carve(Hc * T * sizeof(float));
  const size_t o_inv = carve(T * sizeof(float));
  const size_t o_kinv = carve(max_keep_rows * sizeof(float));
  const size_t o_cnt = carve((Bc * col_blocks + 3 * Bc + 2) * sizeof(unsigned int));
  const size_t o_role = carve(T * sizeof(int32_t));
  const size_t o_seg = carve((max_keep_rows + Bc) * sizeof(int32_t));
  const size_t o_mem = carve(T * sizeof(int32_t));
  const size_t o_meta = carve(T * sizeof(int2));
  const size_t o_kept = carve(max_keep_rows * Dc * sizeof(__nv_bfloat16));
  ctx->cap_tiles = T / 128 + Bc;                       // row tiles of 128 visual rows in any batch that fits
  ctx->sim_part_bytes = (size_t)32 << 20;
  const size_t o_tiles = carve(ctx->cap_tiles * sizeof(unsigned int));
  const size_t o_simpart = carve(ctx->sim_part_bytes);
  const size_t o_status = carve(sizeof(uint32_t));
  e = cudaMalloc(&ctx->arena, off);
  if (e != cudaSuccess) {
    delete ctx;
    return fail(nullptr, ASAP_ERR_CUDA, "cudaMalloc of %zu scratch bytes: %s", off, cudaGetErrorString(e));
  }
  ctx->desc = reinterpret_cast<SampleDesc *>(ctx->arena + o_desc);
  ctx->qsum_partial = reinterpret_cast<float *>(ctx->arena + o_qpart);
  ctx->qbar = reinterpret_cast<float *>(ctx->arena + o_qbar);
  ctx->score_partial = reinterpret_cast<float *>(ctx->arena + o_spart);
  ctx->mass_partial = reinterpret_cast<float *>(ctx->arena + o_mpart);
  if (const char *env = getenv("ASAP_FUSE_MASS_MIN_TOKENS")) ctx->fuse_mass_min_tokens = atoll(env);
  if (const char *env = getenv("ASAP_SIM_PAIR_MIN_BLOCKS")) ctx->sim_pair_min_blocks = atoll(env);
  if (const char *env = getenv("ASAP_SIM_PAIR_STAGES")) ctx->sim_pair_stages = atoi(env);
  if (const char *env = getenv("ASAP_SIM_CLUSTER")) ctx->sim_cluster = atoi(env);
  ctx->inv_norm = reinterpret_cast<float *>(ctx->arena + o_inv);
  ctx->kept_inv = reinterpret_cast<float *>(ctx->arena + o_kinv);
  ctx->counters_off = o_cnt; ctx->counters_bytes = (Bc * col_blocks + 3 * Bc + 2) * sizeof(unsigned int);
  ctx->tiles_off = o_tiles; ctx->tiles_bytes = ctx->cap_tiles * sizeof(unsigned int);
  ctx->cnt_qsum = reinterpret_cast<unsigned int *>(ctx->arena + o_cnt);
  ctx->cnt_mass = ctx->cnt_qsum + Bc * col_blocks;
  ctx->cnt_score = ctx->cnt_mass + Bc;
  ctx->cnt_sim = ctx->cnt_score + Bc;
  ctx->cnt_work = ctx->cnt_sim + Bc;
  ctx->role = reinterpret_cast<int32_t *>(ctx->arena + o_role);
  ctx->seg = reinterpret_cast<int32_t *>(ctx->arena + o_seg);
  ctx->members = reinterpret_cast<int32_t *>(ctx->arena + o_mem);
  ctx->member_meta = reinterpret_cast<int2 *>(ctx->arena + o_meta);
  ctx->kept_rows = reinterpret_cast<__nv_bfloat16 *>(ctx->arena + o_kept);
  ctx->cnt_tiles = reinterpret_cast<unsigned int *>(ctx->arena + o_tiles);
  ctx->sim_part = reinterpret_cast<float *>(ctx->arena + o_simpart);
  ctx->status = reinterpret_cast<uint32_t *>(ctx->arena + o_status);
  e = cudaMemset(ctx->arena + o_cnt, 0, (Bc * col_blocks + 3 * Bc + 2) * sizeof(unsigned int));
  if (e == cudaSuccess) e = cudaMemset(ctx->arena + o_tiles, 0, ctx->cap_tiles * sizeof(unsigned int));
  if (e == cudaSuccess) e = cudaMemset(ctx->status, 0, sizeof(uint32_t));
  // kernels whose dynamic shared memory exceeds the 48 KB default
  if (e == cudaSuccess) e = cudaFuncSetAttribute(score_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, SC_SMEM_BYTES);
  if (e == cudaSuccess) e = cudaFuncSetAttribute(sim_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024);
  if (e == cudaSuccess) e = cudaFuncSetAttribute(sim_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024);
  if (e == cudaSuccess) e = cudaFuncSetAttribute(sim_pair_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024);
  if (e == cudaSuccess) e = cudaFuncSetAttribute(select_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 224 * 1024);
  if (e == cudaSuccess) e = cudaFuncSetAttribute(route_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 224 * 1024);
  if (e == cudaSuccess) e = cudaFuncSetAttribute(attn_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, AT_SMEM_BYTES);
  if (e == cudaSuccess && ctx->sim_cluster) {
    // the cluster form of the sliced similarity launch needs eight co-resident blocks of up to 195 KB each in one
    // cluster; where the device (or the partition of it this process sees) cannot place one, the form is not used
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(1, 1, 8);
    cfg.blockDim = dim3(SIM_THREADS_TILED);
    cfg.dynamicSmemBytes = 195 * 1024;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 1; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 8;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    int clusters = 0;
    if (cudaOccupancyMaxActiveClusters(&clusters, sim_kernel<false>, &cfg) != cudaSuccess || clusters < 1) {
      ctx->sim_cluster = 0;
      cudaGetLastError();
    }
  }
  // lowest priority: when both streams have blocks to place, the score kernel's go first and the
  // mass kernels fill what is left of each SM
  int prio_least = 0, prio_greatest = 0;
  if (e == cudaSuccess) e = cudaDeviceGetStreamPriorityRange(&prio_least, &prio_greatest);
  if (e == cudaSuccess) e = cudaStreamCreateWithPriority(&ctx->side, cudaStreamNonBlocking, prio_least);
  if (e == cudaSuccess) e = cudaEventCreateWithFlags(&ctx->ev_desc, cudaEventDisableTiming);
  if (e == cudaSuccess) e = cudaEventCreateWithFlags(&ctx->ev_fork, cudaEventDisableTiming);
  if (e == cudaSuccess) e = cudaEventCreateWithFlags(&ctx->ev_join, cudaEventDisableTiming);
  if (e == cudaSuccess) e = cudaDeviceSynchronize();
  if (e != cudaSuccess) {
    if (ctx->ev_fork) cudaEventDestroy(ctx->ev_fork);
    if (ctx->ev_join) cudaEventDestroy(ctx->ev_join);
    if (ctx->ev_desc) cudaEventDestroy(ctx->ev_desc);
    if (ctx->side) cudaStreamDestroy(ctx->side);
    cudaFree(ctx->arena);
    delete ctx;
    return fail(nullptr, ASAP_ERR_CUDA, "asap_init set-up: %s", cudaGetErrorString(e));
  }
  *ctx_out = ctx;
  return ASAP_OK;
}

asap_status asap_score(asap_ctx *ctx, const asap_inputs *in, const asap_params *p, const asap_outputs *out,
                       void *stream) {
  ASAP_TRY(validate(ctx, in, p, out, NEED_QK | NEED_SCORE_OUT));
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  ASAP_TRY(launch_mass(ctx, in, p, out, true, nullptr, 0x7fffffff, st));
  return finish(ctx, launch_rank(ctx, in, p, out, true, st), st);
}

asap_status asap_select(asap_ctx *ctx, const asap_inputs *in, const asap_params *p, const float *rank_score,
                        const asap_outputs *out, void *stream) {
  ASAP_TRY(validate(ctx, in, p, out, NEED_SELECT_OUT));
  if (!rank_score) return fail(ctx, ASAP_ERR_INVALID, "null rank_score");
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  ASAP_TRY(launch_prepare(ctx, in, p, nullptr, 0x7fffffff, st));
  return finish(ctx, launch_select(ctx, in, p, rank_score, out, false, false, st), st);
}

asap_status asap_merge(asap_ctx *ctx, const asap_inputs *in, const asap_params *p, const float *salience,
                       const int32_t *keep_idx, const int32_t *drop_idx, const asap_outputs *out,
                       void *stream) {
  ASAP_TRY(validate(ctx, in, p, out, NEED_HIDDEN | NEED_MERGE_OUT));
  if (!salience || !keep_idx || (!drop_idx && in->max_vis > p->keep_k))
    return fail(ctx, ASAP_ERR_INVALID, "null salience / keep_idx / drop_idx");
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  ASAP_TRY(launch_prepare(ctx, in, p, out->out_cu_seqlens, out->out_rows_capacity, st));
  mark(ctx, "role_map", st);
  launch_pdl(role_map_kernel, dim3(dim3((in->max_vis + 255) / 256, in->B)), dim3(256), 0, st, ctx->desc, in->max_vis, p->keep_k,
                                                                         keep_idx, drop_idx, ctx->role, out->assign,
                                                                         out->best_sim, merging(in, p) ? 1 : 0);
  ASAP_TRY(after_launch(ctx, "role_map"));
  return finish(ctx, launch_merge(ctx, in, p, salience, keep_idx, drop_idx, out, st), st);
}

size_t asap_attention_scratch_bytes(int32_t total_tokens, int32_t D) {
  if (total_tokens <= 0 || D <= 0) return 0;
  return align_up((size_t)total_tokens, 8) * (size_t)D * sizeof(__nv_bfloat16);
}

asap_status asap_attention(asap_ctx *ctx, const asap_inputs *in, const asap_params *p, const float *mask_log,
                           const void *v, void *scratch, size_t scratch_bytes, void *out, void *stream) {
  asap_outputs none;
  memset(&none, 0, sizeof(none));
  ASAP_TRY(validate(ctx, in, p, &none, NEED_QK));
  if (!v || !out) return fail(ctx, ASAP_ERR_INVALID, "asap_attention: null v / out");
  if (!aligned16(v) || !aligned16(out)) return fail(ctx, ASAP_ERR_ALIGN, "asap_attention: v / out must be 16-byte aligned");
  if (p->mask_enable && !mask_log) return fail(ctx, ASAP_ERR_INVALID, "asap_attention: mask_enable needs mask_log");
  if (!scratch || !aligned16(scratch) || scratch_bytes < asap_attention_scratch_bytes(in->total_tokens, in->D))
    return fail(ctx, ASAP_ERR_WORKSPACE, "asap_attention: scratch is null, unaligned or smaller than asap_attention_scratch_bytes");
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const int total = in->total_tokens, D = in->D;
  const int total_pad = (int)align_up((size_t)total, 8);
  CUtensorMap map_q, map_k, map_vt;
  if (!make_map(ctx, &map_q, in->q, (uint64_t)total, (uint64_t)D, 128) ||
      !make_map(ctx, &map_k, in->k, (uint64_t)total, (uint64_t)D, 128) ||
      !make_map(ctx, &map_vt, scratch, (uint64_t)D, (uint64_t)total, 128, (uint64_t)total_pad))
    return fail(ctx, ASAP_ERR_CUDA, "cuTensorMapEncodeTiled failed for q / k / transposed v");
  ASAP_TRY(launch_prepare(ctx, in, p, nullptr, 0x7fffffff, st));
  mark(ctx, "transpose_v", st);
  launch_pdl(transpose_v_kernel, dim3((total_pad + TR_TILE - 1) / TR_TILE, (D + TR_TILE - 1) / TR_TILE), dim3(TR_THREADS), 0, st,
             static_cast<const __nv_bfloat16 *>(v), static_cast<__nv_bfloat16 *>(scratch), total, total_pad, D);
  ASAP_TRY(after_launch(ctx, "transpose_v"));
  AttnArgs aa;
  aa.desc = ctx->desc; aa.H = in->H; aa.D = D; aa.max_vis = in->max_vis; aa.mask_enable = p->mask_enable ? 1 : 0;
  aa.scale_log2 = 1.4426950408889634f / sqrtf((float)in->head_dim);
  aa.mask_log = mask_log; aa.out = static_cast<__nv_bfloat16 *>(out); aa.status = ctx->status;
  aa.wait_limit = ctx->wait_limit;
  aa.mask_b_stride = p->per_head_mask ? in->H * in->max_vis : in->max_vis;
  aa.mask_h_stride = p->per_head_mask ? in->max_vis : 0;
  mark(ctx, "attention", st);
  launch_pdl(attn_kernel, dim3((in->max_seq + 255) / 256, in->H, in->B), dim3(AT_THREADS), (size_t)AT_SMEM_BYTES, st,
             map_q, map_k, map_vt, aa);
  return finish(ctx, after_launch(ctx, "attention"), st);
}

size_t asap_consolidate_scratch_bytes(int32_t B, int32_t keep_k) {
  if (B <= 0 || keep_k <= 0) return 0;
  return route_smat_bytes(B, keep_k) + route_mask_bytes(B, keep_k);
}

asap_status asap_consolidate(asap_ctx *ctx, const asap_inputs *in, const asap_params *p, const float *mass,
                             const float *salience, const int32_t *keep_idx, const int32_t *drop_idx,
                             void *scratch, size_t scratch_bytes, const asap_outputs *out,
                             int32_t *n_absorbed, void *stream) {
  ASAP_TRY(validate(ctx, in, p, out, NEED_HIDDEN | NEED_SELECT_OUT | NEED_MERGE_OUT));
  if (!mass || !salience || !keep_idx || !drop_idx) return fail(ctx, ASAP_ERR_INVALID, "null mass / salience / keep_idx / drop_idx");
  if (!p->merge_enable || in->max_vis <= p->keep_k)
    return fail(ctx, ASAP_ERR_INVALID, "asap_consolidate needs merge_enable and keep_k < max_vis; asap_merge covers the rest");
  if (keep_idx == out->keep_idx || drop_idx == out->drop_idx)
    return fail(ctx, ASAP_ERR_INVALID, "asap_consolidate: the stage-1 lists must not be the output lists");
  if (p->keep_k > 32 * 32 * ROUTE_LANE_WORDS)
    return fail(ctx, ASAP_ERR_UNSUPPORTED, "asap_consolidate: keep_k above %d", 32 * 32 * ROUTE_LANE_WORDS);
  if (!scratch || !aligned16(scratch) || scratch_bytes < asap_consolidate_scratch_bytes(in->B, p->keep_k))
    return fail(ctx, ASAP_ERR_WORKSPACE, "asap_consolidate: scratch is null, unaligned or smaller than asap_consolidate_scratch_bytes");
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  ASAP_TRY(launch_prepare(ctx, in, p, out->out_cu_seqlens, out->out_rows_capacity, st));
  ASAP_TRY(launch_consolidate_front(ctx, in, p, mass, salience, keep_idx, drop_idx, scratch, out, n_absorbed, st));
  return finish(ctx, launch_merge_back(ctx, in, p, salience, out->keep_idx, out->drop_idx, out, st), st);
}

asap_status asap_prune_step(asap_ctx *ctx, const asap_inputs *in, const asap_params *p, const asap_outputs *out,
                            void *stream) {
  ASAP_TRY(validate(ctx, in, p, out, NEED_QK | NEED_HIDDEN | NEED_SCORE_OUT | NEED_SELECT_OUT | NEED_MERGE_OUT));
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  // With the text span as ranking rows the Eq. 3 mask never touches a ranked row (a text query lies
  // after every visual key), so the score kernel does not need the attention mass: the memory-bound
  // mass kernels then run on the context's side stream next to the score kernel, and rejoin before
  // the merge, which is the first consumer of the salience.  With caller-given ranking rows (which may
  // be visual) and while per-kernel timing is on, everything runs in order on `stream`.
  const bool text_rows = in->rank_start == nullptr && !p->per_head_mask;
  if (text_rows && (long long)in->B * in->max_vis >= ctx->fuse_mass_min_tokens) {
    // Large batches: the mass kernels no longer hide beside the score kernel (both are bound by the same
    // memory system), so Eq. 1's key side is taken from the key tiles the score kernel streams anyway:
    // query sum (carrying the validation) -> score kernel with two more columns per key tile -> Eq. 2-3.
    PrepareArgs pa = prepare_args(ctx, in, p, out->out_cu_seqlens, out->out_rows_capacity);
    pa.write_desc = 1;
    const int qrows = qsum_rows_per_chunk(ctx, in);
    const int max_chunks = (in->max_vis + qrows - 1) / qrows;
    mark(ctx, "qsum", st);
    launch_pdl(qsum_kernel, dim3(max_chunks, (in->D + QSUM_COLS - 1) / QSUM_COLS, in->B), dim3(QSUM_THREADS), 0, st,
               static_cast<const __nv_bfloat16 *>(in->q), pa, in->D, max_chunks, qrows, ctx->qsum_partial, ctx->qbar, ctx->cnt_qsum);
    ASAP_TRY(after_launch(ctx, "qsum"));
    ASAP_TRY(launch_rank(ctx, in, p, out, false, st, true));
    mark(ctx, "salience", st);
    launch_pdl(salience_from_heads_kernel, dim3(in->B), dim3(SAL_THREADS), 0, st, ctx->desc, in->H, in->max_vis,
               1.0f / ((float)in->H * sqrtf((float)in->head_dim)), p->lambda_max, p->eps, ctx->mass_partial, out->mass,
               out->salience, out->mask_log, out->rank_score);
    ASAP_TRY(after_launch(ctx, "salience"));
    ASAP_TRY(launch_select(ctx, in, p, out->rank_score, out, true, true, st));
    return finish(ctx, launch_merge(ctx, in, p, out->salience, out->keep_idx, out->drop_idx, out, st), st);
  }
  const bool overlap = text_rows && !ctx->prof_on && ctx->side != nullptr;
  if (!overlap) {
    ASAP_TRY(launch_mass(ctx, in, p, out, true, out->out_cu_seqlens, out->out_rows_capacity, st));
    ASAP_TRY(launch_rank(ctx, in, p, out, false, st));
    ASAP_TRY(launch_select(ctx, in, p, out->rank_score, out, true, true, st));
    return finish(ctx, launch_merge(ctx, in, p, out->salience, out->keep_idx, out->drop_idx, out, st), st);
  }
  // stream:      [fork] score (derives its own descriptors) -> wait descriptors -> select -> gather -> sim
  // side stream: qsum (carrying the validation) -> [descriptors ready] -> mass -> [join]
  // The score kernel is enqueued first, so its one block per SM is placed before the mass kernels'
  // many small blocks, which then fill what is left of each SM.
  cudaError_t e = cudaEventRecord(ctx->ev_fork, st);
  if (e != cudaSuccess) return fail(ctx, ASAP_ERR_CUDA, "fork event: %s", cudaGetErrorString(e));
  asap_status main_status = launch_rank(ctx, in, p, out, false, st);
  e = cudaStreamWaitEvent(ctx->side, ctx->ev_fork, 0);
  if (e != cudaSuccess) return fail(ctx, ASAP_ERR_CUDA, "fork to the side stream: %s", cudaGetErrorString(e));
  asap_status side_status = launch_mass(ctx, in, p, out, true, out->out_cu_seqlens, out->out_rows_capacity, ctx->side,
                                        ctx->ev_desc);
  e = cudaEventRecord(ctx->ev_join, ctx->side);
  if (e != cudaSuccess) return fail(ctx, ASAP_ERR_CUDA, "join event: %s", cudaGetErrorString(e));
  if (main_status == ASAP_OK) main_status = side_status;
  if (main_status == ASAP_OK && cudaStreamWaitEvent(st, ctx->ev_desc, 0) != cudaSuccess)
    main_status = fail(ctx, ASAP_ERR_CUDA, "wait for the descriptors");
  if (main_status == ASAP_OK) main_status = launch_select(ctx, in, p, out->rank_score, out, true, true, st);
  if (main_status == ASAP_OK) main_status = launch_merge_front(ctx, in, p, nullptr, out->keep_idx, out->drop_idx, out, st);
  // the side stream always rejoins, also after an error, so that `stream` stays ordered behind it
  e = cudaStreamWaitEvent(st, ctx->ev_join, 0);
  if (e != cudaSuccess) return fail(ctx, ASAP_ERR_CUDA, "join with the side stream: %s", cudaGetErrorString(e));
  if (main_status != ASAP_OK) return main_status;
  return finish(ctx, launch_merge_back(ctx, in, p, out->salience, out->keep_idx, out->drop_idx, out, st), st);
}

asap_status asap_compact_kv(asap_ctx *ctx, const int32_t *src_row, const int32_t *n_rows, int32_t rows_capacity,
                            int32_t src_rows, size_t row_bytes, int32_t n_tensors, const void *const *src,
                            void *const *dst, void *stream) {
  if (!ctx) return fail(nullptr, ASAP_ERR_INVALID, "null context");
  ctx->err[0] = 0;
  if (!src_row || !n_rows || !src || !dst) return fail(ctx, ASAP_ERR_INVALID, "asap_compact_kv: null argument");
  if (rows_capacity <= 0 || src_rows <= 0) return fail(ctx, ASAP_ERR_INVALID, "asap_compact_kv: row counts must be positive");
  if (n_tensors <= 0 || n_tensors > KV_MAX_TENSORS)
    return fail(ctx, ASAP_ERR_UNSUPPORTED, "asap_compact_kv: 1 .. %d tensors per call", KV_MAX_TENSORS);
  if (row_bytes == 0 || row_bytes % 16 != 0 || row_bytes / 16 > 0x7fffffff)
    return fail(ctx, ASAP_ERR_ALIGN, "asap_compact_kv: row_bytes must be a positive multiple of 16");
  GatherArgs ga;
  for (int i = 0; i < n_tensors; ++i) {
    if (!src[i] || !dst[i]) return fail(ctx, ASAP_ERR_INVALID, "asap_compact_kv: null tensor %d", i);
    if (!aligned16(src[i]) || !aligned16(dst[i]))
      return fail(ctx, ASAP_ERR_ALIGN, "asap_compact_kv: tensor %d is not 16-byte aligned", i);
    ga.src[i] = src[i];
    ga.dst[i] = dst[i];
  }
  ga.src_row = src_row; ga.n_rows = n_rows; ga.rows_capacity = rows_capacity; ga.src_rows = src_rows;
  ga.row_vecs = (int32_t)(row_bytes / 16);
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  mark(ctx, "gather_rows", st);
  launch_pdl(gather_rows_kernel, dim3((rows_capacity + KV_THREADS / 32 - 1) / (KV_THREADS / 32), n_tensors),
             dim3(KV_THREADS), 0, st, ga);
  return finish(ctx, after_launch(ctx, "gather_rows"), st);
}

asap_status asap_check(asap_ctx *ctx, void *stream) {
  if (!ctx) return fail(nullptr, ASAP_ERR_INVALID, "null context");
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  uint32_t word = 0;
  cudaError_t e = cudaMemcpyAsync(&word, ctx->status, sizeof(word), cudaMemcpyDeviceToHost, st);
  if (e == cudaSuccess) e = cudaStreamSynchronize(st);
  if (e != cudaSuccess) return fail(ctx, ASAP_ERR_CUDA, "asap_check: %s", cudaGetErrorString(e));
  if (word == 0) { ctx->err[0] = 0; return ASAP_OK; }
  cudaMemsetAsync(ctx->status, 0, sizeof(uint32_t), st);
  if (word & (STATUS_SCORE_TIMEOUT | STATUS_SIM_TIMEOUT | STATUS_ATTN_TIMEOUT)) {
    // blocks that gave up did not finish the hand-shakes that leave the counters at zero
    cudaMemsetAsync(ctx->arena + ctx->counters_off, 0, ctx->counters_bytes, st);
    cudaMemsetAsync(ctx->arena + ctx->tiles_off, 0, ctx->tiles_bytes, st);
  }
  cudaStreamSynchronize(st);
  return fail(ctx, ASAP_ERR_DEVICE, "device status 0x%x:%s%s%s%s%s", word,
              (word & STATUS_BAD_SAMPLE) ? " a per-sample span failed validation (sample skipped);" : "",
              (word & STATUS_OUT_CAPACITY) ? " shortened batch exceeds out_rows_capacity (nothing written);" : "",
              (word & STATUS_SCORE_TIMEOUT) ? " a wait timed out in the score kernel;" : "",
              (word & STATUS_SIM_TIMEOUT) ? " a wait timed out in the similarity kernel;" : "",
              (word & STATUS_ATTN_TIMEOUT) ? " a wait timed out in the attention kernel;" : "");
}

asap_status asap_debug_wait_limit(asap_ctx *ctx, long long cycles) {
  if (!ctx) return fail(nullptr, ASAP_ERR_INVALID, "null context");
  if (cycles <= 0) return fail(ctx, ASAP_ERR_INVALID, "asap_debug_wait_limit: cycles must be positive");
  ctx->wait_limit = cycles;
  return ASAP_OK;
}

asap_status asap_profile(asap_ctx *ctx, int enable) {
  if (!ctx) return fail(nullptr, ASAP_ERR_INVALID, "null context");
  cudaSetDevice(ctx->device);
  if (enable && !ctx->prof_ev) {
    ctx->prof_ev = new (std::nothrow) cudaEvent_t[PROF_MAX_EVENTS];
    ctx->prof_name = new (std::nothrow) const char *[PROF_MAX_EVENTS];
    if (!ctx->prof_ev || !ctx->prof_name) return fail(ctx, ASAP_ERR_CUDA, "out of host memory");
    for (int i = 0; i < PROF_MAX_EVENTS; ++i) {
      cudaError_t e = cudaEventCreate(&ctx->prof_ev[i]);
      if (e != cudaSuccess) {
        for (int j = 0; j < i; ++j) cudaEventDestroy(ctx->prof_ev[j]);
        delete[] ctx->prof_ev; delete[] ctx->prof_name;
        ctx->prof_ev = nullptr; ctx->prof_name = nullptr;
        return fail(ctx, ASAP_ERR_CUDA, "cudaEventCreate: %s", cudaGetErrorString(e));
      }
    }
  }
  ctx->prof_on = enable != 0;
  ctx->prof_used = 0;
  ctx->prof_nacc = 0;
  return ASAP_OK;
}

int asap_profile_read(asap_ctx *ctx, asap_kernel_time *out, int capacity) {
  if (!ctx || !ctx->prof_ev) return 0;
  cudaSetDevice(ctx->device);
  if (ctx->prof_used > 0) cudaEventSynchronize(ctx->prof_ev[ctx->prof_used - 1]);
  for (int i = 0; i + 1 < ctx->prof_used; ++i) {
    const char *name = ctx->prof_name[i];
    if (!name) continue;   // gap between two calls
    float ms = 0.f;
    if (cudaEventElapsedTime(&ms, ctx->prof_ev[i], ctx->prof_ev[i + 1]) != cudaSuccess) continue;
    int slot = -1;
    for (int s = 0; s < ctx->prof_nacc; ++s)
      if (strcmp(ctx->prof_acc[s].name, name) == 0) { slot = s; break; }
    if (slot < 0) {
      if (ctx->prof_nacc >= PROF_MAX_KERNELS) continue;
      slot = ctx->prof_nacc++;
      memset(&ctx->prof_acc[slot], 0, sizeof(asap_kernel_time));
      strncpy(ctx->prof_acc[slot].name, name, sizeof(ctx->prof_acc[slot].name) - 1);
    }
    ctx->prof_acc[slot].launches += 1;
    ctx->prof_acc[slot].total_ms += (double)ms;
  }
  ctx->prof_used = 0;
  const int n = ctx->prof_nacc < capacity ? ctx->prof_nacc : capacity;
  if (out) memcpy(out, ctx->prof_acc, (size_t)(n > 0 ? n : 0) * sizeof(asap_kernel_time));
  return ctx->prof_nacc;
}

// ---- asap_select_static: top-k selection with its scratch in a fixed device array -------------
namespace {

constexpr int STATIC_MAX_B = 64;                 // sequences per call
constexpr int STATIC_MAX_ROLE = 256 * 1024;      // B * max_vis per call

struct StaticSelectScratch {
  SampleDesc desc[STATIC_MAX_B];
  uint32_t status;
  uint32_t pad[63];
  int32_t role[STATIC_MAX_ROLE];
};

// Lives in every GPU that loads the library, from load to exit (about 1 MiB).  On the host this
// name is only a handle for cudaGetSymbolAddress; it is never passed to a kernel as it stands.
static __device__ __align__(256) unsigned char g_static_select[sizeof(StaticSelectScratch)];

constexpr int STATIC_MAX_DEVICES = 64;
StaticSelectScratch *g_static_ptr[STATIC_MAX_DEVICES] = {};   // device address, per device

// First call on a device: look the array's device address up with that device current and raise
// the selection kernel's shared-memory limit.  Neither call allocates.
asap_status static_select_setup(int device, StaticSelectScratch **out) {
  if (device < 0 || device >= STATIC_MAX_DEVICES)
    return fail(nullptr, ASAP_ERR_UNSUPPORTED, "asap_select_static: device index %d out of range", device);
  if (!g_static_ptr[device]) {
    void *ptr = nullptr;
    cudaError_t e = cudaGetSymbolAddress(&ptr, g_static_select);
    if (e != cudaSuccess || !ptr)
      return fail(nullptr, ASAP_ERR_CUDA, "asap_select_static: cudaGetSymbolAddress: %s", cudaGetErrorString(e));
    e = cudaFuncSetAttribute(select_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 224 * 1024);
    if (e != cudaSuccess)
      return fail(nullptr, ASAP_ERR_CUDA, "asap_select_static: cudaFuncSetAttribute: %s", cudaGetErrorString(e));
    g_static_ptr[device] = static_cast<StaticSelectScratch *>(ptr);
  }
  *out = g_static_ptr[device];
  return ASAP_OK;
}

}  // namespace

asap_status asap_select_static(const asap_inputs *in, const asap_params *p, const float *rank_score,
                               int32_t *keep_idx, int32_t *drop_idx, uint32_t *device_status,
                               void *stream) {
  g_init_error[0] = 0;
  if (!in || !p) return fail(nullptr, ASAP_ERR_INVALID, "asap_select_static: null inputs / params struct");
  if (in->B <= 0 || in->total_tokens <= 0)
    return fail(nullptr, ASAP_ERR_INVALID, "asap_select_static: B and total_tokens must be positive");
  if (in->min_vis <= 0 || in->max_vis < in->min_vis || in->max_seq < in->max_vis)
    return fail(nullptr, ASAP_ERR_INVALID, "asap_select_static: need 0 < min_vis <= max_vis <= max_seq");
  if (in->max_rank <= 0 || in->max_rank > in->max_seq)
    return fail(nullptr, ASAP_ERR_INVALID, "asap_select_static: need 0 < max_rank <= max_seq");
  if (p->keep_k <= 0 || p->keep_k > in->min_vis)
    return fail(nullptr, ASAP_ERR_INVALID, "asap_select_static: need 0 < keep_k <= min_vis");
  if (in->max_vis > 57344)
    return fail(nullptr, ASAP_ERR_UNSUPPORTED, "asap_select_static: max_vis > 57344 is not supported");
  if (in->B > STATIC_MAX_B || (long long)in->B * in->max_vis > STATIC_MAX_ROLE)
    return fail(nullptr, ASAP_ERR_WORKSPACE,
                "asap_select_static: B = %d, B * max_vis = %lld exceed the fixed scratch (B <= %d, B * max_vis <= %d)",
                in->B, (long long)in->B * in->max_vis, STATIC_MAX_B, STATIC_MAX_ROLE);
  if (!in->cu_seqlens || !in->vis_start || !in->vis_len || !in->text_start || !in->text_len)
    return fail(nullptr, ASAP_ERR_INVALID, "asap_select_static: null per-sample array");
  if ((in->rank_start == nullptr) != (in->rank_len == nullptr))
    return fail(nullptr, ASAP_ERR_INVALID, "asap_select_static: rank_start and rank_len go together");
  if (!rank_score || !keep_idx || (!drop_idx && in->max_vis > p->keep_k))
    return fail(nullptr, ASAP_ERR_INVALID, "asap_select_static: null rank_score / keep_idx / drop_idx");
  int device = -1;
  cudaError_t e = cudaGetDevice(&device);
  if (e != cudaSuccess) return fail(nullptr, ASAP_ERR_CUDA, "asap_select_static: cudaGetDevice: %s", cudaGetErrorString(e));
  StaticSelectScratch *scr = nullptr;
  ASAP_TRY(static_select_setup(device, &scr));
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  // the status word is the one thing that must start at zero; everything else is overwritten
  uint32_t *status = device_status ? device_status : &scr->status;
  e = cudaMemsetAsync(status, 0, sizeof(uint32_t), st);
  if (e != cudaSuccess) return fail(nullptr, ASAP_ERR_CUDA, "asap_select_static: cudaMemsetAsync: %s", cudaGetErrorString(e));
  asap_ctx view;                 // host-side bookkeeping only; owns nothing
  view.device = device;
  view.desc = scr->desc;
  view.role = scr->role;
  view.status = status;
  asap_outputs out;
  memset(&out, 0, sizeof(out));
  out.keep_idx = keep_idx;
  out.drop_idx = drop_idx;
  asap_status r = launch_prepare(&view, in, p, nullptr, 0x7fffffff, st);
  if (r == ASAP_OK) r = launch_select(&view, in, p, rank_score, &out, false, false, st);
  if (r != ASAP_OK) snprintf(g_init_error, sizeof(g_init_error), "asap_select_static: %s", view.err);
  return r;
}

const char *asap_last_error(const asap_ctx *ctx) { return ctx ? ctx->err : g_init_error; }

uint64_t asap_launch_count(const asap_ctx *ctx) { return ctx ? ctx->launches : 0; }

void asap_free(asap_ctx *ctx) {
  if (!ctx) return;
  cudaSetDevice(ctx->device);
  if (ctx->prof_ev) {
    for (int i = 0; i < PROF_MAX_EVENTS; ++i) cudaEventDestroy(ctx->prof_ev[i]);
    delete[] ctx->prof_ev;
    delete[] ctx->prof_name;
  }
  if (ctx->side) { cudaStreamSynchronize(ctx->side); cudaStreamDestroy(ctx->side); }
  if (ctx->ev_fork) cudaEventDestroy(ctx->ev_fork);
  if (ctx->ev_join) cudaEventDestroy(ctx->ev_join);
  if (ctx->ev_desc) cudaEventDestroy(ctx->ev_desc);
  cudaFree(ctx->arena);
  delete ctx;
}

}  // extern "C"

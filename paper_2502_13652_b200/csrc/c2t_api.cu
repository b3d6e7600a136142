// Host side of libc2t: argument validation, workspace carving, call ordering, launches.
#include <new>
#include <string.h>

#include "c2t_internal.h"

using namespace c2t;

struct c2t_ctx {
  c2t_config cfg;
  TreeState t;
  int grid;              // CTAs of the arg-max pass
  int grid_expand;       // CTAs of the expand pass
  int next_level;        // level the next c2t_expand_level must carry
  int expanded;          // 1 after expand_level(next_level), before its prune
  int shard_expanded;    // 1 after expand_level_shard(next_level), before its export
  int shard_vocab;       // tokens of that shard
  int finalized;         // 1 after c2t_prune(C2T_FINAL)
  int started;
  int64_t launches;
  size_t elem_bytes;
};

namespace {

struct Carver {
  char *base;
  size_t off;
  template <typename T>
  T *take(size_t count) {
    off = (off + 255) & ~(size_t)255;
    T *p = base ? reinterpret_cast<T *>(base + off) : nullptr;
    off += count * sizeof(T);
    return p;
  }
};

int validate(const c2t_config *c) {
  if (!c) return C2T_EINVAL;
  if (c->batch < 1 || c->vocab < 1 || c->max_depth < 1 || c->topk < 1 || c->frontier_cap < 1 ||
      c->budget < 0 || c->device < 0)
    return C2T_EINVAL;
  if (c->dtype != C2T_F32 && c->dtype != C2T_BF16) return C2T_EINVAL;
  if (c->classifier != C2T_CLS_MLP && c->classifier != C2T_CLS_IDENTITY_JOINT &&
      c->classifier != C2T_CLS_IDENTITY_COND)
    return C2T_EINVAL;
  if (c->tree_add != C2T_ADD_FRONTIER && c->tree_add != C2T_ADD_ALL_SURVIVORS) return C2T_EINVAL;
  if (c->entropy_top_m < 0) return C2T_EINVAL;
  if (!(c->threshold == c->threshold)) return C2T_EINVAL;
  if (c->classifier == C2T_CLS_MLP) {
    if (c->hidden < 1 || !c->w1 || !c->b1 || !c->w2 || !c->b2) return C2T_EINVAL;
    if (c->hidden > C2T_MAX_HIDDEN) return C2T_ERANGE;
  }
  if (c->batch > C2T_MAX_BATCH || c->topk > C2T_MAX_TOPK || c->frontier_cap > C2T_MAX_FRONTIER ||
      c->max_depth > C2T_MAX_DEPTH || c->budget > C2T_MAX_BUDGET)
    return C2T_ERANGE;
  if (c2t_tree_capacity(c) > C2T_MAX_TREE) return C2T_ERANGE;
  return C2T_OK;
}

int tree_capacity_unchecked(const c2t_config *c) {
  const long long K = c->topk, F = c->frontier_cap, D = c->max_depth;
  long long cap;
  if (c->tree_add == C2T_ADD_ALL_SURVIVORS) cap = 1 + K + (D - 1) * F * K;
  else cap = 1 + (K < F ? K : F) + (D - 1) * F;
  return cap > 0x7FFFFFFF ? 0x7FFFFFFF : (int)cap;
}

// The grid of the vocabulary pass is fixed per device: 2 CTAs per SM.  Workspace sizing must
// not depend on a device query failing, so sizes assume at most this many SMs.
constexpr int kMaxSms = 256;

int pass_grid(int device) {
  int sms = 0;
  if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, device) != cudaSuccess || sms < 1)
    return -1;
  if (sms > kMaxSms) sms = kMaxSms;
  return sms * kPassCtasPerSm;
}

size_t carve(const c2t_config *c, void *base, TreeState *t) {
  Carver w{reinterpret_cast<char *>(base), 0};
  const size_t B = c->batch, F = c->frontier_cap, K = c->topk;
  const size_t cap = tree_capacity_unchecked(c), Nw = c2t_final_width(c);
  const int eb = c->dtype == C2T_BF16 ? 2 : 4;
  // (expand workers outnumber arg-max CTAs, and their spans may be shorter)
  const size_t ms = max_splits_for(c->vocab, eb, kMaxSms * kExpandCtasPerSm * kExpandWarps, kSegmentPad,
                                   expand_min_span(c->vocab, eb, c->topk));
  TreeState s;
  memset(&s, 0, sizeof s);
  for (int i = 0; i < 2; ++i) {
    s.frontier_n[i] = w.take<int32_t>(B);
    s.frontier_node[i] = w.take<int32_t>(B * F);
  }
  s.tree_n = w.take<int32_t>(B);
  s.tree_token = w.take<int32_t>(B * cap);
  s.tree_parent = w.take<int32_t>(B * cap);
  s.tree_level = w.take<int32_t>(B * cap);
  s.tree_logP = w.take<double>(B * cap);
  s.tree_C = w.take<double>(B * cap);
  s.tree_Chat = w.take<double>(B * cap);
  s.remap = w.take<int32_t>(B * cap);
  s.cand_n = w.take<int32_t>(B);
  s.cand_token = w.take<int32_t>(B * F * K);
  s.cand_flags = w.take<int32_t>(B * F * K);
  s.cand_lp = w.take<double>(B * F * K);
  s.cand_logP = w.take<double>(B * F * K);
  s.cand_H = w.take<double>(B * F * K);
  s.cand_C = w.take<double>(B * F * K);
  s.final_n = w.take<int32_t>(B);
  s.final_src = w.take<int32_t>(B * Nw);
  s.final_token = w.take<int32_t>(B * Nw);
  s.final_parent = w.take<int32_t>(B * Nw);
  s.final_level = w.take<int32_t>(B * Nw);
  s.node_argmax = w.take<int32_t>(B * Nw);
  s.root_tok = w.take<int32_t>(B);
  s.prefix_len = w.take<int32_t>(B);
  s.walk_active = w.take<int32_t>(B);
  s.walk_cur = w.take<int32_t>(B);
  s.walk_len = w.take<int32_t>(B);
  s.status = w.take<uint32_t>(B);
  s.ticket = w.take<uint32_t>(1);
  s.info_draft = w.take<PassInfo>(1);
  s.info_target = w.take<PassInfo>(1);
  s.row_off_draft = w.take<int32_t>(B + 1);
  s.topm = w.take<double2>(B * F);
  if (c->entropy_top_m > 0 && c->entropy_top_m < c->vocab) {   // the expand pass sets Eq. 3's candidates aside
    s.topm_pool_vecs = (long long)topm_pool_vectors(B, F, c->vocab, eb);
    s.topm_pool = w.take<uint4>((size_t)s.topm_pool_vecs);
    s.topm_seg = w.take<TopmSegment>(B * F * ms);
    s.topm_done = w.take<int32_t>(B * F);
  }
  s.part_stats = w.take<float4>(B * F * ms);
  s.part_keys = w.take<unsigned long long>(B * F * ms * K);
  s.part_held = w.take<unsigned long long>(B * F * ms * kHeldPerSlot);
  s.part_best = w.take<unsigned long long>(B * Nw * ms);
  s.w1 = w.take<float>(3 * C2T_MAX_HIDDEN);
  s.b1 = w.take<float>(C2T_MAX_HIDDEN);
  s.w2 = w.take<float>(C2T_MAX_HIDDEN);
  s.b2 = w.take<float>(4);
  if (t) *t = s;
  return (w.off + 255) & ~(size_t)255;
}

bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15) == 0; }

}  // namespace

extern "C" {

int32_t c2t_tree_capacity(const c2t_config *cfg) {
  if (!cfg || cfg->topk < 1 || cfg->frontier_cap < 1 || cfg->max_depth < 1) return 0;
  return tree_capacity_unchecked(cfg);
}

int32_t c2t_final_width(const c2t_config *cfg) {
  const int32_t cap = c2t_tree_capacity(cfg);
  if (cap == 0) return 0;
  return (cfg->budget > 0 && cfg->budget < cap) ? cfg->budget : cap;
}

int32_t c2t_mask_words(const c2t_config *cfg) { return (c2t_final_width(cfg) + 63) / 64; }

size_t c2t_workspace_bytes(const c2t_config *cfg) {
  if (validate(cfg) != C2T_OK) return 0;
  return carve(cfg, nullptr, nullptr);
}

size_t c2t_host_step_ints(const c2t_config *cfg) {
  if (validate(cfg) != C2T_OK) return 0;
  const size_t B = cfg->batch, Nw = c2t_final_width(cfg), W = c2t_mask_words(cfg), D = cfg->max_depth;
  // roots, prefix lengths, n_nodes, tokens, parents, positions, mask (2 ints per word),
  // retrieve, n_leaves, accept_len, path, next_token; each padded to an even count
  size_t n = 0;
  const size_t parts[] = {B, B, B, B * Nw, B * Nw, B * Nw, 2 * B * Nw * W, B * Nw * (D + 1), B, B, B * (D + 1), B};
  for (size_t p : parts) n += (p + 1) & ~(size_t)1;
  return n;
}

int c2t_init(const c2t_config *cfg, void *workspace_dev, size_t workspace_bytes, c2t_ctx **out) {
  if (!out) return C2T_EINVAL;
  *out = nullptr;
  int rc = validate(cfg);
  if (rc != C2T_OK) return rc;
  if (!workspace_dev) return C2T_EINVAL;
  if (reinterpret_cast<uintptr_t>(workspace_dev) & 255) return C2T_EALIGN;
  if (workspace_bytes < carve(cfg, nullptr, nullptr)) return C2T_ERANGE;
  if (cudaSetDevice(cfg->device) != cudaSuccess) { cudaGetLastError(); return C2T_ECUDA; }
  const int grid = pass_grid(cfg->device);
  if (grid < 0 || prepare_expand_pass() != cudaSuccess || prepare_topm_pass() != cudaSuccess ||
      prepare_tree_kernels() != cudaSuccess) {
    cudaGetLastError();
    return C2T_ECUDA;
  }

  c2t_ctx *ctx = new (std::nothrow) c2t_ctx;
  if (!ctx) return C2T_ENOMEM;
  memset(ctx, 0, sizeof *ctx);
  ctx->cfg = *cfg;
  ctx->cfg.w1 = ctx->cfg.b1 = ctx->cfg.w2 = ctx->cfg.b2 = nullptr;
  ctx->grid = grid;
  ctx->grid_expand = grid / kPassCtasPerSm * kExpandCtasPerSm;
  ctx->elem_bytes = cfg->dtype == C2T_BF16 ? 2 : 4;
  carve(cfg, workspace_dev, &ctx->t);
  TreeState &t = ctx->t;
  t.B = cfg->batch; t.V = cfg->vocab; t.K = cfg->topk; t.F = cfg->frontier_cap; t.D = cfg->max_depth;
  t.N = cfg->budget; t.Nw = c2t_final_width(cfg); t.W = c2t_mask_words(cfg);
  t.cap = tree_capacity_unchecked(cfg);
  t.hidden = cfg->classifier == C2T_CLS_MLP ? cfg->hidden : 0;
  t.classifier = cfg->classifier; t.tree_add = cfg->tree_add; t.beta = cfg->threshold;
  t.entropy_top_m = cfg->entropy_top_m;
  t.min_span = expand_min_span(cfg->vocab, (int)ctx->elem_bytes, cfg->topk);
  t.max_splits = max_splits_for(cfg->vocab, (int)ctx->elem_bytes, ctx->grid_expand * kExpandWarps, kSegmentPad, t.min_span);
  t.max_splits_tgt = max_splits_for(cfg->vocab, (int)ctx->elem_bytes, ctx->grid, 0);

  cudaError_t e = cudaSuccess;
  if (cfg->classifier == C2T_CLS_MLP) {
    const size_t h = cfg->hidden;
    e = cudaMemcpy(t.w1, cfg->w1, 3 * h * sizeof(float), cudaMemcpyHostToDevice);
    if (e == cudaSuccess) e = cudaMemcpy(t.b1, cfg->b1, h * sizeof(float), cudaMemcpyHostToDevice);
    if (e == cudaSuccess) e = cudaMemcpy(t.w2, cfg->w2, h * sizeof(float), cudaMemcpyHostToDevice);
    if (e == cudaSuccess) e = cudaMemcpy(t.b2, cfg->b2, sizeof(float), cudaMemcpyHostToDevice);
  }
  if (e == cudaSuccess) e = cudaMemset(t.status, 0, sizeof(uint32_t) * cfg->batch);
  if (e == cudaSuccess) e = cudaMemset(t.ticket, 0, sizeof(uint32_t));
  if (e != cudaSuccess) { cudaGetLastError(); delete ctx; return C2T_ECUDA; }
  *out = ctx;
  return C2T_OK;
}

void c2t_destroy(c2t_ctx *ctx) { delete ctx; }

int c2t_begin_step(c2t_ctx *ctx, const int32_t *root_tok_dev, const int32_t *prefix_len_dev, void *stream) {
  if (!ctx || !root_tok_dev || !prefix_len_dev) return C2T_EINVAL;
  if (launch_begin_step(ctx->t, root_tok_dev, prefix_len_dev, (cudaStream_t)stream) != cudaSuccess)
    return C2T_ECUDA;
  ctx->launches += 1;
  ctx->next_level = 0;
  ctx->expanded = 0;
  ctx->shard_expanded = 0;
  ctx->finalized = 0;
  ctx->started = 1;
  return C2T_OK;
}

int c2t_expand_level(c2t_ctx *ctx, int level, const void *logits_dev, int64_t seq_stride,
                     int64_t row_stride, void *stream) {
  if (!ctx || !logits_dev) return C2T_EINVAL;
  if (!ctx->started || ctx->finalized || ctx->expanded || ctx->shard_expanded || level != ctx->next_level ||
      level >= ctx->cfg.max_depth)
    return C2T_EORDER;
  if (seq_stride < 0 || row_stride < ctx->cfg.vocab) return C2T_EINVAL;
  if (!aligned16(logits_dev) || (seq_stride * ctx->elem_bytes) % 16 || (row_stride * ctx->elem_bytes) % 16)
    return C2T_EALIGN;
  const TreeState &t = ctx->t;
  PassParams p;
  memset(&p, 0, sizeof p);
  p.logits = logits_dev; p.seq_stride = seq_stride; p.row_stride = row_stride;
  p.V = t.V; p.K = t.K; p.B = t.B; p.rows_per_seq_max = t.F;
  p.counts = t.frontier_n[level & 1];
  p.max_splits = t.max_splits;
  p.min_span = t.min_span;
  p.n_slots = (int64_t)t.B * t.F * t.max_splits;
  p.status = t.status;
  p.info = t.info_draft;
  p.part_stats = t.part_stats; p.part_keys = t.part_keys; p.part_held = t.part_held;
  p.row_off = t.row_off_draft;
  const bool truncated = t.entropy_top_m > 0 && t.entropy_top_m < t.V;   // Eq. 3: the sums over the M most probable tokens
  if (truncated) { p.topm_pool = t.topm_pool; p.topm_pool_vecs = t.topm_pool_vecs; p.topm_seg = t.topm_seg; }
  if (launch_expand_pass(p, ctx->cfg.dtype, ctx->grid_expand, (cudaStream_t)stream) != cudaSuccess)
    return C2T_ECUDA;
  ctx->launches += 1;
  if (truncated) {
    // from the vectors the pass set aside; then, for the rows where those did not suffice, from the rows themselves
    if (launch_topm_finish(t.entropy_top_m, t.F, t.B, p.counts, t, t.topm, ctx->cfg.dtype, (cudaStream_t)stream) != cudaSuccess)
      return C2T_ECUDA;
    if (launch_topm_entropy(logits_dev, seq_stride, row_stride, t.V, t.entropy_top_m, t.F, t.B, p.counts, t, t.topm,
                            t.topm_done, ctx->grid_expand, ctx->cfg.dtype, (cudaStream_t)stream) != cudaSuccess)
      return C2T_ECUDA;
    ctx->launches += 2;
  }
  ctx->expanded = 1;
  return C2T_OK;
}

int c2t_prune(c2t_ctx *ctx, int level, const c2t_frontier *out, void *stream) {
  if (!ctx) return C2T_EINVAL;
  if (!ctx->started || ctx->finalized) return C2T_EORDER;
  if (level == C2T_FINAL) {
    if (ctx->expanded) return C2T_EORDER;
    if (launch_final_prune(ctx->t, (cudaStream_t)stream) != cudaSuccess) return C2T_ECUDA;
    ctx->launches += 1;
    ctx->finalized = 1;
    return C2T_OK;
  }
  if (!ctx->expanded || level != ctx->next_level) return C2T_EORDER;
  if (launch_prune_level(ctx->t, level, out, nullptr, 0, (cudaStream_t)stream) != cudaSuccess) return C2T_ECUDA;
  ctx->launches += 1;
  ctx->expanded = 0;
  ctx->next_level = level + 1;
  return C2T_OK;
}

int c2t_expand_prune_level(c2t_ctx *ctx, int level, const void *logits_dev, int64_t seq_stride, int64_t row_stride,
                           const c2t_frontier *out, void *stream) {
  if (!ctx || !logits_dev) return C2T_EINVAL;
  const TreeState &t = ctx->t;
  if (t.B > C2T_FUSED_MAX_BATCH || (t.entropy_top_m > 0 && t.entropy_top_m < t.V)) {
    const int rc = c2t_expand_level(ctx, level, logits_dev, seq_stride, row_stride, stream);
    return rc != C2T_OK ? rc : c2t_prune(ctx, level, out, stream);
  }
  if (!ctx->started || ctx->finalized || ctx->expanded || ctx->shard_expanded || level != ctx->next_level ||
      level >= ctx->cfg.max_depth)
    return C2T_EORDER;
  if (seq_stride < 0 || row_stride < ctx->cfg.vocab) return C2T_EINVAL;
  if (!aligned16(logits_dev) || (seq_stride * ctx->elem_bytes) % 16 || (row_stride * ctx->elem_bytes) % 16)
    return C2T_EALIGN;
  PassParams p;
  memset(&p, 0, sizeof p);
  p.logits = logits_dev; p.seq_stride = seq_stride; p.row_stride = row_stride;
  p.V = t.V; p.K = t.K; p.B = t.B; p.rows_per_seq_max = t.F;
  p.counts = t.frontier_n[level & 1];
  p.max_splits = t.max_splits;
  p.min_span = t.min_span;
  p.n_slots = (int64_t)t.B * t.F * t.max_splits;
  p.status = t.status;
  p.info = t.info_draft;
  p.part_stats = t.part_stats; p.part_keys = t.part_keys; p.part_held = t.part_held;
  p.row_off = t.row_off_draft;
  if (launch_expand_prune(p, t, level, out, ctx->cfg.dtype, ctx->grid_expand, (cudaStream_t)stream) != cudaSuccess)
    return C2T_ECUDA;
  ctx->launches += 1;
  ctx->next_level = level + 1;
  return C2T_OK;
}

int c2t_expand_level_shard(c2t_ctx *ctx, int level, const void *logits_dev, int64_t seq_stride,
                           int64_t row_stride, int32_t vocab_count, void *stream) {
  if (!ctx || !logits_dev) return C2T_EINVAL;
  if (!ctx->started || ctx->finalized || ctx->expanded || ctx->shard_expanded || level != ctx->next_level ||
      level >= ctx->cfg.max_depth)
    return C2T_EORDER;
  if (vocab_count < 1 || vocab_count > ctx->cfg.vocab || seq_stride < 0 || row_stride < vocab_count) return C2T_EINVAL;
  if (ctx->t.entropy_top_m > 0 && ctx->t.entropy_top_m < ctx->t.V) return C2T_EINVAL;   // Eq. 3 needs whole rows
  if (!aligned16(logits_dev) || (seq_stride * ctx->elem_bytes) % 16 || (row_stride * ctx->elem_bytes) % 16)
    return C2T_EALIGN;
  const TreeState &t = ctx->t;
  PassParams p;
  memset(&p, 0, sizeof p);
  p.logits = logits_dev; p.seq_stride = seq_stride; p.row_stride = row_stride;
  p.V = vocab_count; p.K = t.K; p.B = t.B; p.rows_per_seq_max = t.F;
  p.counts = t.frontier_n[level & 1];
  p.max_splits = t.max_splits;                    // sized for whole rows: enough for any part of one
  p.min_span = t.min_span;
  p.n_slots = (int64_t)t.B * t.F * t.max_splits;
  p.status = t.status;
  p.info = t.info_draft;
  p.part_stats = t.part_stats; p.part_keys = t.part_keys; p.part_held = t.part_held;
  p.row_off = t.row_off_draft;
  if (launch_expand_pass(p, ctx->cfg.dtype, ctx->grid_expand, (cudaStream_t)stream) != cudaSuccess)
    return C2T_ECUDA;
  ctx->launches += 1;
  ctx->shard_expanded = 1;
  ctx->shard_vocab = vocab_count;
  return C2T_OK;
}

int c2t_export_row_records(c2t_ctx *ctx, int level, int32_t vocab_begin, c2t_row_record *records_dev,
                           void *stream) {
  if (!ctx || !records_dev) return C2T_EINVAL;
  if (!ctx->shard_expanded || level != ctx->next_level) return C2T_EORDER;
  if (vocab_begin < 0 || (int64_t)vocab_begin + ctx->shard_vocab > ctx->cfg.vocab) return C2T_EINVAL;
  if (launch_export_rows(ctx->t, level, ctx->shard_vocab, vocab_begin, records_dev, (cudaStream_t)stream) !=
      cudaSuccess)
    return C2T_ECUDA;
  ctx->launches += 1;
  ctx->shard_expanded = 0;
  return C2T_OK;
}

int c2t_prune_gathered(c2t_ctx *ctx, int level, const c2t_row_record *records_dev, int32_t n_shards,
                       const c2t_frontier *out, void *stream) {
  if (!ctx || !records_dev) return C2T_EINVAL;
  if (n_shards < 1) return C2T_EINVAL;
  if (n_shards > C2T_MAX_SHARDS) return C2T_ERANGE;
  if (!ctx->started || ctx->finalized || ctx->expanded || ctx->shard_expanded || level != ctx->next_level ||
      level >= ctx->cfg.max_depth)
    return C2T_EORDER;
  if (launch_prune_level(ctx->t, level, out, records_dev, n_shards, (cudaStream_t)stream) != cudaSuccess)
    return C2T_ECUDA;
  ctx->launches += 1;
  ctx->next_level = level + 1;
  return C2T_OK;
}

int c2t_build_verify(c2t_ctx *ctx, const c2t_verify *out, void *stream) {
  if (!ctx) return C2T_EINVAL;
  if (!ctx->finalized) return C2T_EORDER;
  if (launch_build_verify(ctx->t, out, (cudaStream_t)stream) != cudaSuccess) return C2T_ECUDA;
  ctx->launches += 1;
  return C2T_OK;
}

int c2t_dense_mask(c2t_ctx *ctx, void *out_dev, int32_t out_dtype, int64_t kv_len, void *stream) {
  if (!ctx || !out_dev || kv_len < 1) return C2T_EINVAL;
  if (out_dtype != C2T_F32 && out_dtype != C2T_BF16) return C2T_EINVAL;
  if (!ctx->finalized) return C2T_EORDER;
  if (launch_dense_mask(ctx->t, out_dev, out_dtype, kv_len, (cudaStream_t)stream) != cudaSuccess) return C2T_ECUDA;
  ctx->launches += 1;
  return C2T_OK;
}

int c2t_accept(c2t_ctx *ctx, const void *target_logits_dev, int64_t seq_stride, int64_t row_stride,
               const c2t_accept_out *out, void *stream) {
  if (!ctx || !target_logits_dev) return C2T_EINVAL;
  if (!ctx->finalized) return C2T_EORDER;
  if (seq_stride < 0 || row_stride < ctx->cfg.vocab) return C2T_EINVAL;
  if (!aligned16(target_logits_dev) || (seq_stride * ctx->elem_bytes) % 16 ||
      (row_stride * ctx->elem_bytes) % 16)
    return C2T_EALIGN;
  const TreeState &t = ctx->t;
  PassParams p;
  memset(&p, 0, sizeof p);
  p.logits = target_logits_dev; p.seq_stride = seq_stride; p.row_stride = row_stride;
  p.V = t.V; p.K = 1; p.B = t.B; p.rows_per_seq_max = t.Nw;
  p.counts = t.final_n;
  p.max_splits = t.max_splits_tgt;
  p.n_slots = (int64_t)t.B * t.Nw * t.max_splits_tgt;
  p.status = t.status;
  p.info = t.info_target;
  p.part_best = t.part_best;
  if (launch_argmax_pass(p, ctx->cfg.dtype, ctx->grid, (cudaStream_t)stream) != cudaSuccess)
    return C2T_ECUDA;
  if (launch_accept_walk(t, out, nullptr, 0, (cudaStream_t)stream) != cudaSuccess) return C2T_ECUDA;
  ctx->launches += 2;
  return C2T_OK;
}

int c2t_argmax_shard(c2t_ctx *ctx, const void *target_logits_dev, int64_t seq_stride, int64_t row_stride,
                     int32_t vocab_count, int32_t vocab_begin, uint64_t *keys_dev, void *stream) {
  if (!ctx || !target_logits_dev || !keys_dev) return C2T_EINVAL;
  if (!ctx->finalized) return C2T_EORDER;
  if (vocab_count < 1 || vocab_begin < 0 || (int64_t)vocab_begin + vocab_count > ctx->cfg.vocab || seq_stride < 0 ||
      row_stride < vocab_count)
    return C2T_EINVAL;
  if (!aligned16(target_logits_dev) || (seq_stride * ctx->elem_bytes) % 16 ||
      (row_stride * ctx->elem_bytes) % 16)
    return C2T_EALIGN;
  const TreeState &t = ctx->t;
  PassParams p;
  memset(&p, 0, sizeof p);
  p.logits = target_logits_dev; p.seq_stride = seq_stride; p.row_stride = row_stride;
  p.V = vocab_count; p.K = 1; p.B = t.B; p.rows_per_seq_max = t.Nw;
  p.counts = t.final_n;
  p.max_splits = t.max_splits_tgt;
  p.n_slots = (int64_t)t.B * t.Nw * t.max_splits_tgt;
  p.status = t.status;
  p.info = t.info_target;
  p.part_best = t.part_best;
  if (launch_argmax_pass(p, ctx->cfg.dtype, ctx->grid, (cudaStream_t)stream) != cudaSuccess)
    return C2T_ECUDA;
  if (launch_export_best(t, vocab_begin, reinterpret_cast<unsigned long long *>(keys_dev), (cudaStream_t)stream) !=
      cudaSuccess)
    return C2T_ECUDA;
  ctx->launches += 2;
  return C2T_OK;
}

int c2t_accept_gathered(c2t_ctx *ctx, const uint64_t *keys_dev, int32_t n_shards, const c2t_accept_out *out,
                        void *stream) {
  if (!ctx || !keys_dev || n_shards < 1) return C2T_EINVAL;
  if (n_shards > C2T_MAX_SHARDS) return C2T_ERANGE;
  if (!ctx->finalized) return C2T_EORDER;
  if (launch_accept_walk(ctx->t, out, reinterpret_cast<const unsigned long long *>(keys_dev), n_shards,
                         (cudaStream_t)stream) != cudaSuccess)
    return C2T_ECUDA;
  ctx->launches += 1;
  return C2T_OK;
}

int c2t_accept_lazy(c2t_ctx *ctx, const void *target_logits_dev, int64_t seq_stride, int64_t row_stride,
                    const c2t_accept_out *out, void *stream) {
  if (!ctx || !target_logits_dev) return C2T_EINVAL;
  if (!ctx->finalized) return C2T_EORDER;
  if (seq_stride < 0 || row_stride < ctx->cfg.vocab) return C2T_EINVAL;
  if (!aligned16(target_logits_dev) || (seq_stride * ctx->elem_bytes) % 16 ||
      (row_stride * ctx->elem_bytes) % 16)
    return C2T_EALIGN;
  const TreeState &t = ctx->t;
  PassParams p;
  memset(&p, 0, sizeof p);
  p.logits = target_logits_dev; p.seq_stride = seq_stride; p.row_stride = row_stride;
  p.V = t.V; p.K = 1; p.B = t.B; p.rows_per_seq_max = 1;
  p.counts = t.walk_active;          // one row per sequence that is still walking ...
  p.row_sel = t.walk_cur;            // ... the row of its current node
  p.max_splits = t.max_splits_tgt;
  p.n_slots = (int64_t)t.B * t.Nw * t.max_splits_tgt;
  p.status = t.status;
  p.info = t.info_target;
  p.part_best = t.part_best;
  cudaStream_t s = (cudaStream_t)stream;
  if (launch_lazy_walk_round(t, 0, out, nullptr, 0, s) != cudaSuccess) return C2T_ECUDA;
  ctx->launches += 1;
  for (int r = 0; r <= t.D; ++r) {   // a path has at most D + 1 nodes
    if (launch_argmax_pass(p, ctx->cfg.dtype, ctx->grid, s) != cudaSuccess) return C2T_ECUDA;
    if (launch_lazy_walk_round(t, r + 1, out, nullptr, 0, s) != cudaSuccess) return C2T_ECUDA;
    ctx->launches += 2;
  }
  return C2T_OK;
}

int c2t_lazy_begin(c2t_ctx *ctx, const c2t_accept_out *out, void *stream) {
  if (!ctx) return C2T_EINVAL;
  if (!ctx->finalized) return C2T_EORDER;
  if (launch_lazy_walk_round(ctx->t, 0, out, nullptr, 0, (cudaStream_t)stream) != cudaSuccess) return C2T_ECUDA;
  ctx->launches += 1;
  return C2T_OK;
}

int c2t_lazy_argmax_shard(c2t_ctx *ctx, const void *target_logits_dev, int64_t seq_stride, int64_t row_stride,
                          int32_t vocab_count, int32_t vocab_begin, uint64_t *keys_dev, void *stream) {
  if (!ctx || !target_logits_dev || !keys_dev) return C2T_EINVAL;
  if (!ctx->finalized) return C2T_EORDER;
  if (vocab_count < 1 || vocab_begin < 0 || (int64_t)vocab_begin + vocab_count > ctx->cfg.vocab || seq_stride < 0 ||
      row_stride < vocab_count)
    return C2T_EINVAL;
  if (!aligned16(target_logits_dev) || (seq_stride * ctx->elem_bytes) % 16 || (row_stride * ctx->elem_bytes) % 16)
    return C2T_EALIGN;
  const TreeState &t = ctx->t;
  PassParams p;
  memset(&p, 0, sizeof p);
  p.logits = target_logits_dev; p.seq_stride = seq_stride; p.row_stride = row_stride;
  p.V = vocab_count; p.K = 1; p.B = t.B; p.rows_per_seq_max = 1;
  p.counts = t.walk_active;          // one row per sequence that is still walking ...
  p.row_sel = t.walk_cur;            // ... the row of its current node
  p.max_splits = t.max_splits_tgt;
  p.n_slots = (int64_t)t.B * t.Nw * t.max_splits_tgt;
  p.status = t.status;
  p.info = t.info_target;
  p.part_best = t.part_best;
  cudaStream_t s = (cudaStream_t)stream;
  if (launch_argmax_pass(p, ctx->cfg.dtype, ctx->grid, s) != cudaSuccess) return C2T_ECUDA;
  if (launch_export_lazy_best(t, vocab_begin, reinterpret_cast<unsigned long long *>(keys_dev), s) != cudaSuccess)
    return C2T_ECUDA;
  ctx->launches += 2;
  return C2T_OK;
}

int c2t_lazy_step_gathered(c2t_ctx *ctx, int round, const uint64_t *keys_dev, int32_t n_shards,
                           const c2t_accept_out *out, void *stream) {
  if (!ctx || !keys_dev || n_shards < 1 || round < 1) return C2T_EINVAL;
  if (n_shards > C2T_MAX_SHARDS) return C2T_ERANGE;
  if (!ctx->finalized) return C2T_EORDER;
  if (launch_lazy_walk_round(ctx->t, round, out, reinterpret_cast<const unsigned long long *>(keys_dev), n_shards,
                             (cudaStream_t)stream) != cudaSuccess)
    return C2T_ECUDA;
  ctx->launches += 1;
  return C2T_OK;
}

int c2t_status(c2t_ctx *ctx, uint32_t *bits_host, uint32_t *per_seq_host, void *stream) {
  if (!ctx || !bits_host) return C2T_EINVAL;
  const int B = ctx->cfg.batch;
  uint32_t *tmp = per_seq_host ? per_seq_host : new (std::nothrow) uint32_t[B];
  if (!tmp) return C2T_ENOMEM;
  cudaError_t e = cudaMemcpyAsync(tmp, ctx->t.status, sizeof(uint32_t) * B, cudaMemcpyDeviceToHost,
                                  (cudaStream_t)stream);
  if (e == cudaSuccess) e = cudaStreamSynchronize((cudaStream_t)stream);
  uint32_t bits = 0;
  if (e == cudaSuccess)
    for (int b = 0; b < B; ++b) bits |= tmp[b];
  if (!per_seq_host) delete[] tmp;
  if (e != cudaSuccess) { cudaGetLastError(); return C2T_ECUDA; }
  *bits_host = bits;
  return C2T_OK;
}

int c2t_get_view(c2t_ctx *ctx, c2t_view *v) {
  if (!ctx || !v) return C2T_EINVAL;
  const TreeState &t = ctx->t;
  v->tree_n = t.tree_n; v->tree_token = t.tree_token; v->tree_parent = t.tree_parent;
  v->tree_level = t.tree_level; v->tree_logP = t.tree_logP; v->tree_C = t.tree_C; v->tree_Chat = t.tree_Chat;
  v->cand_n = t.cand_n; v->cand_token = t.cand_token; v->cand_lp = t.cand_lp; v->cand_logP = t.cand_logP;
  v->cand_H = t.cand_H; v->cand_C = t.cand_C; v->cand_flags = t.cand_flags;
  v->frontier_n = t.frontier_n[ctx->next_level & 1];
  v->frontier_node = t.frontier_node[ctx->next_level & 1];
  v->final_n = t.final_n; v->final_src = t.final_src; v->final_token = t.final_token;
  v->final_parent = t.final_parent; v->final_level = t.final_level; v->node_argmax = t.node_argmax;
  v->topm_from_pass = t.topm_done;
  return C2T_OK;
}

int c2t_decode_step_host(c2t_ctx *ctx, const c2t_host_step *io, void *stream) {
  if (!ctx || !io || !io->draft_logits_host || !io->target_logits_host || !io->root_tok_host ||
      !io->prefix_len_host || !io->draft_stage_dev || !io->target_stage_dev || !io->int_stage_dev)
    return C2T_EINVAL;
  cudaStream_t s = (cudaStream_t)stream;
  const c2t_config &c = ctx->cfg;
  const size_t B = c.batch, F = c.frontier_cap, V = c.vocab, D = c.max_depth, eb = ctx->elem_bytes;
  const size_t Nw = ctx->t.Nw, W = ctx->t.W;
  for (size_t l = 0; l < D; ++l)
    if (!io->draft_logits_host[l]) return C2T_EINVAL;

  // carve the integer staging buffer (each part padded to an even count: mask words need 8-byte alignment)
  int32_t *ip = io->int_stage_dev;
  if (reinterpret_cast<uintptr_t>(ip) & 7) return C2T_EALIGN;
  auto take = [&](size_t n) { int32_t *p = ip; ip += (n + 1) & ~(size_t)1; return p; };
  int32_t *root = take(B), *prefix = take(B);
  c2t_verify vo;
  vo.n_nodes = take(B); vo.tokens = take(B * Nw); vo.parents = take(B * Nw); vo.position_ids = take(B * Nw);
  vo.mask_bits = reinterpret_cast<uint64_t *>(take(2 * B * Nw * W));
  vo.retrieve = take(B * Nw * (D + 1)); vo.n_leaves = take(B);
  c2t_accept_out ao;
  ao.accept_len = take(B); ao.path = take(B * (D + 1)); ao.next_token = take(B);

#define C2T_CUDA(x) do { if ((x) != cudaSuccess) { cudaGetLastError(); return C2T_ECUDA; } } while (0)
#define C2T_CALL(x) do { int rc_ = (x); if (rc_ != C2T_OK) return rc_; } while (0)
  C2T_CUDA(cudaMemcpyAsync(root, io->root_tok_host, B * 4, cudaMemcpyHostToDevice, s));
  C2T_CUDA(cudaMemcpyAsync(prefix, io->prefix_len_host, B * 4, cudaMemcpyHostToDevice, s));
  C2T_CALL(c2t_begin_step(ctx, root, prefix, s));
  for (size_t l = 0; l < D; ++l) {
    if (l == 0)   // only the root's row of each sequence is ever read at level 0
      C2T_CUDA(cudaMemcpy2DAsync(io->draft_stage_dev, F * V * eb, io->draft_logits_host[0], F * V * eb,
                                 V * eb, B, cudaMemcpyHostToDevice, s));
    else
      C2T_CUDA(cudaMemcpyAsync(io->draft_stage_dev, io->draft_logits_host[l], B * F * V * eb,
                               cudaMemcpyHostToDevice, s));
    C2T_CALL(c2t_expand_level(ctx, (int)l, io->draft_stage_dev, (int64_t)(F * V), (int64_t)V, s));
    C2T_CALL(c2t_prune(ctx, (int)l, nullptr, s));
  }
  C2T_CALL(c2t_prune(ctx, C2T_FINAL, nullptr, s));
  C2T_CALL(c2t_build_verify(ctx, &vo, s));
  C2T_CUDA(cudaMemcpyAsync(io->target_stage_dev, io->target_logits_host, B * Nw * V * eb,
                           cudaMemcpyHostToDevice, s));
  C2T_CALL(c2t_accept(ctx, io->target_stage_dev, (int64_t)(Nw * V), (int64_t)V, &ao, s));
  if (io->n_nodes_host) C2T_CUDA(cudaMemcpyAsync(io->n_nodes_host, vo.n_nodes, B * 4, cudaMemcpyDeviceToHost, s));
  if (io->tokens_host) C2T_CUDA(cudaMemcpyAsync(io->tokens_host, vo.tokens, B * Nw * 4, cudaMemcpyDeviceToHost, s));
  if (io->accept_len_host) C2T_CUDA(cudaMemcpyAsync(io->accept_len_host, ao.accept_len, B * 4, cudaMemcpyDeviceToHost, s));
  if (io->path_host) C2T_CUDA(cudaMemcpyAsync(io->path_host, ao.path, B * (D + 1) * 4, cudaMemcpyDeviceToHost, s));
  if (io->next_token_host) C2T_CUDA(cudaMemcpyAsync(io->next_token_host, ao.next_token, B * 4, cudaMemcpyDeviceToHost, s));
  C2T_CUDA(cudaStreamSynchronize(s));
#undef C2T_CUDA
#undef C2T_CALL
  return C2T_OK;
}

int64_t c2t_launch_count(const c2t_ctx *ctx) { return ctx ? ctx->launches : 0; }

const char *c2t_strerror(int code) {
  switch (code) {
    case C2T_OK: return "ok";
    case C2T_EINVAL: return "invalid argument";
    case C2T_EALIGN: return "pointer or stride not aligned";
    case C2T_ERANGE: return "size out of range";
    case C2T_EORDER: return "call out of order";
    case C2T_ECUDA: return "CUDA runtime error";
    case C2T_ENOMEM: return "out of host memory";
    default: return "unknown error";
  }
}

}  // extern "C"

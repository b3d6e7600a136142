// Per-sequence kernels: classification and pruning of a level, the Top-N rerank, the
// verification inputs and the acceptance walk.  One CTA per sequence; all of this is
// O(F*K) or O(tree) work per sequence, done in double precision where it is floating point.
#include <string.h>

#include "c2t_internal.h"
#include "level_prune.cuh"

namespace c2t {
namespace {

constexpr int kTreeThreads = 512;
constexpr int kTreeWarps = kTreeThreads / 32;
constexpr unsigned kFull = 0xFFFFFFFFu;

__global__ void begin_step_kernel(TreeState t, const int32_t *root_tok, const int32_t *prefix_len) {
  chain_enter();
  const int b = blockIdx.x * blockDim.x + threadIdx.x;
  if (b >= t.B) return;
  const size_t o = (size_t)b * t.cap;
  t.tree_n[b] = 1;
  t.tree_token[o] = root_tok[b];
  t.tree_parent[o] = -1;
  t.tree_level[o] = 0;
  t.tree_logP[o] = 0.0;
  t.tree_C[o] = 1.0;
  t.tree_Chat[o] = INFINITY;
  t.frontier_n[0][b] = 1;
  t.frontier_n[1][b] = 0;
  t.frontier_node[0][(size_t)b * t.F] = 0;
  t.cand_n[b] = 0;
  t.final_n[b] = 0;
  t.root_tok[b] = root_tok[b];
  t.prefix_len[b] = prefix_len[b];
  t.status[b] = 0u;
}

// The record of every active row of the last (sharded) expand pass, for c2t_export_row_records.
__global__ void __launch_bounds__(kTreeThreads) export_rows_kernel(TreeState t, int level, int vloc, int tok_base,
                                                                   c2t_row_record *out) {
  __shared__ unsigned long long s_keys[kTreeWarps][kStageKeys];
  chain_enter();
  const int b = blockIdx.x, lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  int n = t.frontier_n[level & 1][b];
  const int row_off = t.row_off_draft[b];
  const PassInfo info = *t.info_draft;
  n = n < 0 ? 0 : (n > t.F ? t.F : n);
  for (int j = warp; j < n; j += kTreeWarps) {
    c2t_row_record *r = out + (size_t)b * t.F + j;
    const RowMerge m = merge_row_partials(t, info, b, row_off + j, t.K, vloc, s_keys[warp], r->x, r->tok, tok_base);
    if (lane == 0) {
      r->M = m.M; r->S = m.S; r->T = m.T;
      r->n = m.n_valid;
      r->fault = row_fault_bits(m.top, m.S, m.T);
    }
  }
}

// records == nullptr: the rows come from this context's own expand pass; else from gathered records of n_shards shards
__global__ void __launch_bounds__(kTreeThreads) prune_level_kernel(TreeState t, int level, c2t_frontier out,
                                                                   const c2t_row_record *records, int n_shards) {
  extern __shared__ __align__(16) unsigned char s_prune[];
  PruneShared<kTreeWarps> &sh = *reinterpret_cast<PruneShared<kTreeWarps> *>(s_prune);
  prune_level_body<kTreeThreads, true>(t, level, out, records, n_shards, blockIdx.x, sh);
}

// ---------------------------------------------------------------- rerank ----

// Top-N rerank (Sec. 2.2): root + the N-1 nodes first under (Chat desc, id asc), renumbered
// in id order.  Chat never exceeds the parent's and parents have lower ids, so the kept set
// is closed under "parent of".
__global__ void __launch_bounds__(kTreeThreads) final_prune_kernel(TreeState t) {
  __shared__ int s_scan[kTreeWarps + 1];
  chain_enter();
  const int b = blockIdx.x, tid = threadIdx.x;
  int n = t.tree_n[b];
  n = n > t.cap ? t.cap : n;
  const size_t tb = (size_t)b * t.cap, fb = (size_t)b * t.Nw;
  const double *chat = t.tree_Chat + tb;
  int32_t *remap = t.remap + tb;
  const bool all = (t.N <= 0 || n <= t.N);

  int run = 0;     // nodes kept so far (ids below the chunk)
  for (int base = 0; base < n; base += kTreeThreads) {
    const int i = base + tid;
    int keep = 0;
    if (i < n) {
      if (all || i == 0) keep = 1;
      else {
        const double ci = chat[i];
        int rank = 0;
        for (int o = 1; o < n; ++o) {
          const double co = __ldg(&chat[o]);
          rank += (co > ci) || (co == ci && o < i);
        }
        keep = rank < t.N - 1;
      }
    }
    int total;
    const int off = block_exclusive_scan<kTreeThreads>(keep, s_scan, &total);
    if (i < n) remap[i] = keep ? run + off : -1;
    run += total;
  }
  __syncthreads();
  const int n_final = run > t.Nw ? t.Nw : run;
  for (int i = tid; i < n; i += kTreeThreads) {
    const int m = remap[i];
    if (m < 0 || m >= t.Nw) continue;
    const int par = t.tree_parent[tb + i];
    t.final_src[fb + m] = i;
    t.final_token[fb + m] = t.tree_token[tb + i];
    t.final_parent[fb + m] = par < 0 ? -1 : remap[par];
    t.final_level[fb + m] = t.tree_level[tb + i];
  }
  for (int m = n_final + tid; m < t.Nw; m += kTreeThreads) {
    t.final_src[fb + m] = -1;
    t.final_token[fb + m] = 0;
    t.final_parent[fb + m] = -1;
    t.final_level[fb + m] = 0;
  }
  if (tid == 0) t.final_n[b] = n_final;
}

// ---------------------------------------------------------------- verify ----

__global__ void __launch_bounds__(kTreeThreads) build_verify_kernel(TreeState t, c2t_verify out) {
  __shared__ int s_has_child[C2T_MAX_BUDGET > C2T_MAX_TREE ? C2T_MAX_BUDGET : C2T_MAX_TREE];
  __shared__ int s_scan[kTreeWarps + 1];
  chain_enter();
  const int b = blockIdx.x, tid = threadIdx.x;
  const int n = t.final_n[b], Nw = t.Nw, W = t.W, width = t.D + 1;
  const size_t fb = (size_t)b * Nw;
  const int32_t *parent = t.final_parent + fb, *level = t.final_level + fb;
  const int prefix = t.prefix_len[b];

  for (int i = tid; i < Nw; i += kTreeThreads) s_has_child[i] = 0;
  __syncthreads();
  for (int i = tid; i < n; i += kTreeThreads)
    if (parent[i] >= 0) s_has_child[parent[i]] = 1;
  __syncthreads();

  for (int i = tid; i < Nw; i += kTreeThreads) {
    if (out.tokens) out.tokens[fb + i] = i < n ? t.final_token[fb + i] : 0;
    if (out.parents) out.parents[fb + i] = i < n ? parent[i] : -1;
    if (out.position_ids) out.position_ids[fb + i] = i < n ? prefix + level[i] : 0;
    if (out.mask_bits) {
      uint64_t *row = out.mask_bits + (fb + i) * W;
      for (int w = 0; w < W; ++w) row[w] = 0ull;
      if (i < n)
        for (int a = i, g = 0; a >= 0 && g <= t.D + 1; a = parent[a], ++g) row[a >> 6] |= 1ull << (a & 63);
    }
    if (out.retrieve) {
      int32_t *row = out.retrieve + (fb + i) * width;
      for (int k = 0; k < width; ++k) row[k] = -1;
    }
  }
  __syncthreads();
  // leaves in ascending id order
  int run = 0;
  for (int base = 0; base < n; base += kTreeThreads) {
    const int i = base + tid;
    const int leaf = (i < n && !s_has_child[i]) ? 1 : 0;
    int total;
    const int off = block_exclusive_scan<kTreeThreads>(leaf, s_scan, &total);
    if (leaf && out.retrieve) {
      int32_t *row = out.retrieve + (fb + run + off) * width;
      for (int a = i, g = 0; a >= 0 && g <= t.D + 1; a = parent[a], ++g) {
        const int l = level[a];
        if (l >= 0 && l < width) row[l] = a;
      }
    }
    run += total;
  }
  if (tid == 0) {
    if (out.n_nodes) out.n_nodes[b] = n;
    if (out.n_leaves) out.n_leaves[b] = run;
  }
}

// ---------------------------------------------------------------- accept ----

// best key of active row `a` of the last arg-max pass (0: none)
__device__ __forceinline__ unsigned long long row_best_key(const TreeState &t, const PassInfo &info, int seq, int a) {
  const long long first_vec = (long long)a * info.vec_per_row;
  const int c_first = (int)(first_vec / info.span);
  const int c_last = (int)((first_vec + info.vec_per_row - 1) / info.span);
  int n_splits = c_last - c_first + 1;
  if (n_splits > t.max_splits_tgt) {
    n_splits = t.max_splits_tgt;
    atomicOr(&t.status[seq], C2T_ST_INTERNAL);
  }
  unsigned long long best = 0ull;
  for (int s = 0; s < n_splits; ++s) {
    unsigned long long k = t.part_best[(size_t)a * t.max_splits_tgt + s];
    best = k > best ? k : best;
  }
  return best;
}

// rows of earlier sequences in the arg-max pass over the final trees (all threads of the CTA call this)
__device__ int target_row_offset(const TreeState &t, int b, int *s_scan, int *s_total) {
  int part = 0;
  for (int i = threadIdx.x; i < b; i += kTreeThreads) {
    int c = t.final_n[i];
    part += c < 0 ? 0 : (c > t.Nw ? t.Nw : c);
  }
  int total;
  block_exclusive_scan<kTreeThreads>(part, s_scan, &total);
  if (threadIdx.x == 0) *s_total = total;
  __syncthreads();
  return *s_total;
}

// The best key of every final node's row over one token range, token ids made global, for c2t_argmax_shard.
__global__ void __launch_bounds__(kTreeThreads) export_best_kernel(TreeState t, int tok_base, unsigned long long *out) {
  __shared__ int s_scan[kTreeWarps + 1];
  __shared__ int s_total;
  chain_enter();
  const int b = blockIdx.x, n = t.final_n[b], Nw = t.Nw;
  const PassInfo info = *t.info_target;
  const int row_off = target_row_offset(t, b, s_scan, &s_total);
  for (int i = threadIdx.x; i < Nw; i += kTreeThreads) {
    unsigned long long key = 0ull;
    if (i < n) {
      const unsigned long long best = row_best_key(t, info, b, row_off + i);
      if (best) key = (best & 0xFFFFFFFF00000000ull) | (0xFFFFFFFFu - (uint32_t)(key_token(best) + tok_base));
    }
    out[(size_t)b * Nw + i] = key;
  }
}

// gathered == nullptr: the arg-max of this context's own pass; else the best of n_shards gathered keys per node
__global__ void __launch_bounds__(kTreeThreads) accept_walk_kernel(TreeState t, c2t_accept_out out,
                                                                   const unsigned long long *gathered, int n_shards) {
  __shared__ int s_misc[1];
  chain_enter();
  const int b = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int n = t.final_n[b], Nw = t.Nw, width = t.D + 1;
  const size_t fb = (size_t)b * Nw;
  const PassInfo info = *t.info_target;

  // rows of earlier sequences in the argmax pass
  if (!gathered) {
    __shared__ int s_scan[kTreeWarps + 1];
    int part = 0;
    for (int i = tid; i < b; i += kTreeThreads) {
      int c = t.final_n[i];
      part += c < 0 ? 0 : (c > Nw ? Nw : c);
    }
    int total;
    block_exclusive_scan<kTreeThreads>(part, s_scan, &total);
    if (tid == 0) s_misc[0] = total;
    __syncthreads();
  }
  const int row_off = gathered ? 0 : s_misc[0];
  // target argmax per node: best key over the row's partials
  for (int i = tid; i < Nw; i += kTreeThreads) {
    int tok = -1;
    if (i < n) {
      unsigned long long best = 0ull;
      if (gathered) {                               // equal logits in two shards: the larger key is the lower token id
        for (int s = 0; s < n_shards; ++s) {
          const unsigned long long k = gathered[((size_t)s * t.B + b) * Nw + i];
          best = k > best ? k : best;
        }
      } else {
        best = row_best_key(t, info, b, row_off + i);
      }
      tok = best ? key_token(best) : -1;
    }
    t.node_argmax[fb + i] = tok;
  }
  __syncthreads();
  if (warp != 0) return;
  // greedy walk by one warp
  const int32_t *parent = t.final_parent + fb, *token = t.final_token + fb;
  int cur = 0, len = 0;
  if (out.path && lane < width) out.path[(size_t)b * width + lane] = lane == 0 ? 0 : -1;
  for (int w = 32 + lane; out.path && w < width; w += 32) out.path[(size_t)b * width + w] = -1;
  __syncwarp();
  while (n > 0 && len + 1 < width) {
    const int want = t.node_argmax[fb + cur];
    int found = 0x7FFFFFFF;
    for (int c = cur + 1 + lane; c < n; c += 32)
      if (parent[c] == cur && token[c] == want) { found = c; break; }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      int other = __shfl_xor_sync(kFull, found, o);
      found = other < found ? other : found;
    }
    if (found == 0x7FFFFFFF) break;
    cur = found;
    ++len;
    if (lane == 0 && out.path) out.path[(size_t)b * width + len] = cur;
  }
  if (lane == 0) {
    if (out.accept_len) out.accept_len[b] = len;
    if (out.next_token) out.next_token[b] = n > 0 ? t.node_argmax[fb + cur] : -1;
  }
}

// ---------------------------------------------------------------- dense mask -

// One CTA per (sequence, final-tree row): the row's ancestor-or-self set as bits in shared
// memory (a walk up the parent pointers, at most D+1 steps), then the row of kv_len additive
// mask values, 0 or -inf (Sec. 2.2).
template <typename T>
__global__ void __launch_bounds__(256) dense_mask_kernel(TreeState t, T *out, long long kv_len, T zero, T ninf) {
  __shared__ unsigned long long s_bits[(C2T_MAX_TREE + 63) / 64];   // Nw never exceeds the tree capacity
  const int b = blockIdx.y, i = blockIdx.x, tid = threadIdx.x;
  const int Nw = t.Nw, n = t.final_n[b];
  const int words = (Nw + 63) / 64;
  for (int w = tid; w < words; w += blockDim.x) s_bits[w] = 0ull;
  __syncthreads();
  if (tid == 0 && i < n) {
    const int32_t *parent = t.final_parent + (size_t)b * Nw;
    for (int j = i, guard = 0; j >= 0 && guard <= Nw; j = parent[j], ++guard) s_bits[j >> 6] |= 1ull << (j & 63);
  }
  __syncthreads();
  const long long prefix = t.prefix_len[b];
  T *row = out + ((size_t)b * Nw + i) * kv_len;
  for (long long c = tid; c < kv_len; c += blockDim.x) {
    bool on = c < prefix;
    const long long j = c - prefix;
    if (j >= 0 && j < Nw) on = (s_bits[j >> 6] >> (j & 63)) & 1ull;
    row[c] = on ? zero : ninf;
  }
}

// ---------------------------------------------------------------- lazy walk --

// One round of the acceptance walk that reads only the rows it visits (Sec. 5 Metrics).
// Round 0 puts every sequence with a tree on its root.  Round r > 0 follows the arg-max pass
// over the current nodes' rows (one row per walking sequence, in sequence order): the
// sequence moves to the child that carries the arg-max token, or stops.  A single CTA serves
// all sequences, 1024 at a time; the scan numbers the walking sequences the way the pass did.
constexpr int kWalkThreads = 1024;

// gathered == nullptr: the arg-max of this context's own pass over whole rows; else the best of n_shards gathered keys
// per sequence ([n_shards, B], one key for the sequence's current node, 0 for a sequence that has stopped).
__global__ void __launch_bounds__(kWalkThreads) lazy_walk_round_kernel(TreeState t, int round, c2t_accept_out out,
                                                                       const unsigned long long *gathered, int n_shards) {
  __shared__ int s_warp[kWalkThreads / 32 + 1];
  chain_enter();
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int Nw = t.Nw, width = t.D + 1;
  const PassInfo info = *t.info_target;
  int rows_before = 0;                               // walking sequences in earlier chunks
  for (int base = 0; base < t.B; base += kWalkThreads) {
    const int b = base + tid;
    const bool in = b < t.B;
    const size_t fb = (size_t)b * Nw;
    if (round == 0) {
      if (in) {
        const int n = t.final_n[b];
        for (int i = 0; i < Nw; ++i) t.node_argmax[fb + i] = -1;
        if (out.path)
          for (int w = 0; w < width; ++w) out.path[(size_t)b * width + w] = w == 0 ? 0 : -1;
        t.walk_cur[b] = 0;
        t.walk_len[b] = 0;
        t.walk_active[b] = n > 0;
        if (n <= 0) {
          if (out.accept_len) out.accept_len[b] = 0;
          if (out.next_token) out.next_token[b] = -1;
        }
      }
      continue;
    }
    const int was = in ? t.walk_active[b] : 0;
    // the row number of this sequence in the pass: walking sequences before it
    int inc = was;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int v = __shfl_up_sync(kFull, inc, o);
      if (lane >= o) inc += v;
    }
    __syncthreads();
    if (lane == 31) s_warp[warp] = inc;
    __syncthreads();
    if (tid == 0) {
      int run = 0;
      for (int w = 0; w < kWalkThreads / 32; ++w) { const int v = s_warp[w]; s_warp[w] = run; run += v; }
      s_warp[kWalkThreads / 32] = run;
    }
    __syncthreads();
    const int a = rows_before + s_warp[warp] + inc - was;
    rows_before += s_warp[kWalkThreads / 32];
    if (!was) continue;

    unsigned long long best = 0ull;
    if (gathered) {                                    // equal logits in two shards: the larger key is the lower token id
      for (int sh = 0; sh < n_shards; ++sh) {
        const unsigned long long k = gathered[(size_t)sh * t.B + b];
        best = k > best ? k : best;
      }
    } else {
      const long long first_vec = (long long)a * info.vec_per_row;
      const int c_first = (int)(first_vec / info.span);
      const int c_last = (int)((first_vec + info.vec_per_row - 1) / info.span);
      int n_splits = c_last - c_first + 1;
      if (n_splits > t.max_splits_tgt) {
        n_splits = t.max_splits_tgt;
        atomicOr(&t.status[b], C2T_ST_INTERNAL);
      }
      for (int sp = 0; sp < n_splits; ++sp) {
        const unsigned long long k = t.part_best[(size_t)a * t.max_splits_tgt + sp];
        best = k > best ? k : best;
      }
    }
    const int want = best ? key_token(best) : -1;
    const int n = t.final_n[b];
    int cur = t.walk_cur[b], len = t.walk_len[b];
    t.node_argmax[fb + cur] = want;
    int found = -1;
    if (len + 1 < width)
      for (int c = cur + 1; c < n; ++c)
        if (t.final_parent[fb + c] == cur && t.final_token[fb + c] == want) { found = c; break; }
    if (found >= 0) {
      ++len;
      t.walk_cur[b] = found;
      t.walk_len[b] = len;
      if (out.path) out.path[(size_t)b * width + len] = found;
    } else {
      t.walk_active[b] = 0;
      if (out.accept_len) out.accept_len[b] = len;
      if (out.next_token) out.next_token[b] = want;
    }
  }
}

// After an arg-max pass over one token range of the walking sequences' current rows: per sequence the best key of
// that range with the token id made global (0 for a sequence that has stopped), for c2t_lazy_argmax_shard.  The
// pass numbered the walking sequences in sequence order; the scan here does the same.
__global__ void __launch_bounds__(kWalkThreads) export_lazy_best_kernel(TreeState t, int tok_base, unsigned long long *out) {
  __shared__ int s_warp[kWalkThreads / 32 + 1];
  chain_enter();
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const PassInfo info = *t.info_target;
  int rows_before = 0;
  for (int base = 0; base < t.B; base += kWalkThreads) {
    const int b = base + tid;
    const int was = b < t.B ? t.walk_active[b] : 0;
    int inc = was;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int v = __shfl_up_sync(kFull, inc, o);
      if (lane >= o) inc += v;
    }
    __syncthreads();
    if (lane == 31) s_warp[warp] = inc;
    __syncthreads();
    if (tid == 0) {
      int run = 0;
      for (int w = 0; w < kWalkThreads / 32; ++w) { const int v = s_warp[w]; s_warp[w] = run; run += v; }
      s_warp[kWalkThreads / 32] = run;
    }
    __syncthreads();
    const int a = rows_before + s_warp[warp] + inc - was;
    rows_before += s_warp[kWalkThreads / 32];
    if (b >= t.B) continue;
    unsigned long long key = 0ull;
    if (was) {
      const unsigned long long best = row_best_key(t, info, b, a);
      if (best) key = (best & 0xFFFFFFFF00000000ull) | (0xFFFFFFFFu - (uint32_t)(key_token(best) + tok_base));
    }
    out[b] = key;
  }
}

}  // namespace

cudaError_t launch_dense_mask(const TreeState &t, void *out, int out_dtype, int64_t kv_len, cudaStream_t s) {
  const dim3 grid(t.Nw, t.B);
  if (out_dtype == C2T_F32) {
    dense_mask_kernel<float><<<grid, 256, 0, s>>>(t, reinterpret_cast<float *>(out), kv_len, 0.f, -INFINITY);
  } else {
    // bf16 as raw 16-bit words: +0 and -inf
    dense_mask_kernel<unsigned short><<<grid, 256, 0, s>>>(t, reinterpret_cast<unsigned short *>(out), kv_len,
                                                          (unsigned short)0x0000, (unsigned short)0xFF80);
  }
  return cudaGetLastError();
}

cudaError_t launch_lazy_walk_round(const TreeState &t, int round, const c2t_accept_out *out,
                                   const unsigned long long *gathered, int n_shards, cudaStream_t s) {
  c2t_accept_out o;
  memset(&o, 0, sizeof o);
  if (out) o = *out;
  return launch_chained(lazy_walk_round_kernel, dim3(1), dim3(kWalkThreads), 0, s, t, round, o, gathered, n_shards);
}

cudaError_t launch_export_lazy_best(const TreeState &t, int vocab_begin, unsigned long long *out, cudaStream_t s) {
  return launch_chained(export_lazy_best_kernel, dim3(1), dim3(kWalkThreads), 0, s, t, vocab_begin, out);
}

cudaError_t launch_begin_step(const TreeState &t, const int32_t *root_tok, const int32_t *prefix_len,
                              cudaStream_t s) {
  return launch_chained(begin_step_kernel, dim3((t.B + 127) / 128), dim3(128), 0, s, t, root_tok, prefix_len);
}

cudaError_t launch_export_rows(const TreeState &t, int level, int vocab_count, int vocab_begin, c2t_row_record *out,
                               cudaStream_t s) {
  return launch_chained(export_rows_kernel, dim3(t.B), dim3(kTreeThreads), 0, s, t, level, vocab_count, vocab_begin, out);
}

cudaError_t launch_prune_level(const TreeState &t, int level, const c2t_frontier *out, const c2t_row_record *records,
                               int n_shards, cudaStream_t s) {
  c2t_frontier o = {nullptr, nullptr, nullptr, nullptr};
  if (out) o = *out;
  return launch_chained(prune_level_kernel, dim3(t.B), dim3(kTreeThreads), sizeof(PruneShared<kTreeWarps>), s, t, level, o,
                        records, n_shards);
}

cudaError_t prepare_tree_kernels() {
  return cudaFuncSetAttribute(prune_level_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                              (int)sizeof(PruneShared<kTreeWarps>));
}

cudaError_t launch_final_prune(const TreeState &t, cudaStream_t s) {
  return launch_chained(final_prune_kernel, dim3(t.B), dim3(kTreeThreads), 0, s, t);
}

cudaError_t launch_build_verify(const TreeState &t, const c2t_verify *out, cudaStream_t s) {
  c2t_verify o = {nullptr, nullptr, nullptr, nullptr, nullptr, nullptr, nullptr};
  if (out) o = *out;
  return launch_chained(build_verify_kernel, dim3(t.B), dim3(kTreeThreads), 0, s, t, o);
}

cudaError_t launch_export_best(const TreeState &t, int vocab_begin, unsigned long long *out, cudaStream_t s) {
  return launch_chained(export_best_kernel, dim3(t.B), dim3(kTreeThreads), 0, s, t, vocab_begin, out);
}

cudaError_t launch_accept_walk(const TreeState &t, const c2t_accept_out *out, const unsigned long long *gathered,
                               int n_shards, cudaStream_t s) {
  c2t_accept_out o = {nullptr, nullptr, nullptr};
  if (out) o = *out;
  return launch_chained(accept_walk_kernel, dim3(t.B), dim3(kTreeThreads), 0, s, t, o, gathered, n_shards);
}

}  // namespace c2t

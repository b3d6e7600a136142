// Per-sequence kernels: classification and pruning of a level, the Top-N rerank, the
// verification inputs and the acceptance walk.  One CTA per sequence; all of this is
// O(F*K) or O(tree) work per sequence, done in double precision where it is floating point.
#include <string.h>

#include "c2t_internal.h"

namespace c2t {
namespace {

constexpr int kTreeThreads = 512;
constexpr int kTreeWarps = kTreeThreads / 32;
constexpr int kMaxCand = C2T_MAX_TOPK * C2T_MAX_FRONTIER;   // 1024
constexpr unsigned kFull = 0xFFFFFFFFu;
constexpr int kStageKeys = 192;   // keys of a row's partial lists that a warp stages in shared memory

__device__ __forceinline__ double warp_sum(double v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_down_sync(kFull, v, o);
  return __shfl_sync(kFull, v, 0);
}

// Exclusive scan of one int per thread over the CTA; returns the exclusive prefix, *total = sum.
__device__ int block_exclusive_scan(int v, int *s_warp /*[kTreeWarps+1]*/, int *total) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  int inc = v;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    int t = __shfl_up_sync(kFull, inc, o);
    if (lane >= o) inc += t;
  }
  __syncthreads();
  if (lane == 31) s_warp[warp] = inc;
  __syncthreads();
  if (threadIdx.x == 0) {
    int run = 0;
    for (int w = 0; w < kTreeWarps; ++w) { int t = s_warp[w]; s_warp[w] = run; run += t; }
    s_warp[kTreeWarps] = run;
  }
  __syncthreads();
  *total = s_warp[kTreeWarps];
  return s_warp[warp] + inc - v;
}

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

// ---------------------------------------------------------------- a level ---

// Confidence of one child (Eq. 4): two-layer FFN on (P, H, d), ReLU, sigmoid.
__device__ double classify(const TreeState &t, const float *s_w, double P, double H, double d) {
  const float *w1 = s_w, *b1 = s_w + 3 * C2T_MAX_HIDDEN, *w2 = b1 + C2T_MAX_HIDDEN, *b2 = w2 + C2T_MAX_HIDDEN;
  double z = (double)b2[0];
  for (int k = 0; k < t.hidden; ++k) {
    double a = (double)b1[k] + (double)w1[3 * k] * P + (double)w1[3 * k + 1] * H + (double)w1[3 * k + 2] * d;
    if (a < 0.0) a = 0.0;
    z += (double)w2[k] * a;
  }
  return 1.0 / (1.0 + exp(-z));
}

// What one warp makes of the partial records of one active row of the last expand pass.
struct RowMerge {
  double M, S, T;              // row maximum; sums over every other element of e^(x - M) and e^(x - M)(x - M)
  unsigned long long top;      // the row's best key (0: none)
  int n_valid;                 // candidates written (at most K)
};

// One warp merges the partial records of active row `a` (all lanes return the same values).  The K
// best (logit, token) pairs go to out_x / out_tok (shared or global memory, best first, padded with
// -inf / -1), token ids offset by tok_base; vloc is the length of the rows the pass read (tokens at
// or past it pad a ragged last vector).  sk: the warp's staging area of kStageKeys keys.
__device__ RowMerge merge_row_partials(const TreeState &t, const PassInfo &info, int seq, int a, int K, int vloc,
                                       unsigned long long *sk, float *out_x, int *out_tok, int tok_base) {
  const int lane = threadIdx.x & 31;
  // the workers that hold a piece of this row: the rows, each behind info.pad virtual vectors, were cut every info.span
  const long long first_vec = (long long)a * (info.vec_per_row + info.pad) + info.pad;
  const int c_first = (int)(first_vec / info.span);
  const int c_last = (int)((first_vec + info.vec_per_row - 1) / info.span);
  int n_splits = c_last - c_first + 1;
  if (n_splits > t.max_splits) {                    // the host's sizing and the pass disagree: say so, stay in bounds
    n_splits = t.max_splits;
    if (lane == 0) atomicOr(&t.status[seq], C2T_ST_INTERNAL);
  }
  const size_t slot0 = (size_t)a * t.max_splits;
  const int n_keys = n_splits * K;

  // rows with few partials (the usual case): every load is issued before the first use
  const bool staged = n_splits <= 32 && n_keys <= kStageKeys && kHeldPerSlot == 1;
  unsigned long long my_held = 0ull;
  float4 my_stats = make_float4(0.f, 0.f, 0.f, 0.f);
  if (staged) {
    if (lane < n_splits) {
      my_held = t.part_held[slot0 + lane];
      my_stats = t.part_stats[slot0 + lane];
    }
    for (int i = lane; i < n_keys; i += 32) sk[i] = t.part_keys[slot0 * K + i];
  }

  // the row maximum is the largest key held out of any partial's sums
  const int n_held = n_splits * kHeldPerSlot;
  unsigned long long top = my_held;
  if (!staged) {
    for (int i = lane; i < n_held; i += 32) {
      unsigned long long k0 = t.part_held[slot0 * kHeldPerSlot + i];
      top = k0 > top ? k0 : top;
    }
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    unsigned long long other = __shfl_xor_sync(kFull, top, o);
    top = other > top ? other : top;
  }
  const double M = (double)key_value(top);

  // fp32 sums of every split: S = sum 2^t, U = sum 2^t t with t = x log2(e) + c, brought to
  // natural units relative to M:  x - M = t ln2 + g,  g = -c ln2 - M
  double S = 0.0, T = 0.0;
  for (int i = lane; i < n_splits; i += 32) {
    const float4 st = staged ? my_stats : t.part_stats[slot0 + i];
    const double Ss = (double)st.y, Us = (double)st.z;
    if (Ss != 0.0 || Us != 0.0) {               // (NaN passes this test and poisons the sums)
      const double kLn2 = 0.69314718055994530942;
      const double g = -(double)st.x * kLn2 - M;
      const double f = exp(g);
      S += Ss * f;
      T += f * (kLn2 * Us + g * Ss);
    }
  }
  // held-out elements are not in those sums: add them exactly, all but the row maximum itself
  for (int i = lane; i < n_held; i += 32) {
    const unsigned long long key = staged ? my_held : t.part_held[slot0 * kHeldPerSlot + i];
    if (key == 0ull || key == top) continue;
    const float x = key_value(key);
    if (x > kNegInfAsFinite) {
      double d = (double)x - M;
      double e = exp(d);
      S += e;
      T += e * d;
    }
  }
  // the K best keys over all splits become the candidates
  S = warp_sum(S);
  T = warp_sum(T);
  int n_valid = 0;
  if (staged) {
    // every split's list is sorted and now in shared memory, one list per lane: take the
    // largest head K times (a key of a token past the vocabulary ends its list: it pads a
    // ragged last vector and sorts behind every real element)
    __syncwarp();
    int pos = 0;
    for (; n_valid < K; ++n_valid) {
      unsigned long long h = (lane < n_splits && pos < K) ? sk[lane * K + pos] : 0ull;
      if (h != 0ull && key_token(h) >= vloc) h = 0ull;
      const uint32_t hi = (uint32_t)(h >> 32), mx_hi = __reduce_max_sync(kFull, hi);
      const uint32_t mx_lo = __reduce_max_sync(kFull, hi == mx_hi ? (uint32_t)h : 0u);
      const unsigned long long mx = ((unsigned long long)mx_hi << 32) | mx_lo;
      if (mx == 0ull) break;
      if (lane == 0) { out_x[n_valid] = key_value(mx); out_tok[n_valid] = key_token(mx) + tok_base; }
      if (h == mx) ++pos;
    }
    __syncwarp();
  } else {
    for (int i = lane; i < n_keys; i += 32) {
      const unsigned long long key = t.part_keys[slot0 * K + i];
      if (key == 0ull) continue;
      const int tok = key_token(key);
      if (tok >= vloc) continue;                    // padding of a ragged last vector
      int rank = 0;
      for (int r = 0; r < n_keys; ++r) {
        unsigned long long other = t.part_keys[slot0 * K + r];
        rank += (other > key) && (key_token(other) < vloc);
      }
      if (rank < K) { out_x[rank] = key_value(key); out_tok[rank] = tok + tok_base; }
    }
    for (int i = lane; i < n_keys; i += 32) {
      unsigned long long key = t.part_keys[slot0 * K + i];
      n_valid += (key != 0ull && key_token(key) < vloc);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) n_valid += __shfl_xor_sync(kFull, n_valid, o);
    if (n_valid > K) n_valid = K;
  }
  // candidates that do not exist (fewer than K tokens in the vocabulary)
  for (int r = n_valid + lane; r < K; r += 32) { out_x[r] = -INFINITY; out_tok[r] = -1; }
  RowMerge m;
  m.M = M; m.S = S; m.T = T; m.top = top; m.n_valid = n_valid;
  return m;
}

// status bits of a row from its best key and its sums
__device__ __forceinline__ uint32_t row_fault_bits(unsigned long long top, double S, double T) {
  const float top_x = key_value(top);
  if (top == 0ull || top_x <= kNegInfAsFinite) return C2T_ST_ALL_NEGINF;
  if (top_x == INFINITY) return C2T_ST_POSINF_LOGIT;
  if (S != S || T != T || isinf(S)) return C2T_ST_NAN_LOGIT;
  return 0u;
}

// One warp merges the gathered records of row (b, j): lane s holds shard s's record.  Writes the K
// best candidates to out_x / out_tok and returns the merged maximum and sums; *fault_out collects the
// shards' status bits ("all -inf" only if every shard says so).
__device__ RowMerge merge_row_records(const TreeState &t, const c2t_row_record *records, int n_shards, int b, int j,
                                      int K, float *out_x, int *out_tok, uint32_t *fault_out) {
  const int lane = threadIdx.x & 31;
  const c2t_row_record *rec = records + ((size_t)lane * t.B + b) * t.F + j;
  double Mg = 0.0, Sg = 0.0, Tg = 0.0;
  int ng = 0;
  uint32_t fg = 0u;
  bool live = false;
  if (lane < n_shards) {
    Mg = rec->M; Sg = rec->S; Tg = rec->T; ng = rec->n; fg = rec->fault;
    ng = ng < 0 ? 0 : (ng > K ? K : ng);
    live = !(fg & C2T_ST_ALL_NEGINF);
  }
  const uint32_t fault = __reduce_or_sync(kFull, fg & ~(uint32_t)C2T_ST_ALL_NEGINF);
  // the row maximum is the best of the shards' maxima; equal values go to the lower shard, whose token ids are lower
  unsigned long long top = live ? (((unsigned long long)f32_orderable(__float_as_uint((float)Mg)) << 32) |
                                   (0xFFFFFFFFu - (uint32_t)lane)) : 0ull;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    unsigned long long other = __shfl_xor_sync(kFull, top, o);
    top = other > top ? other : top;
  }
  const int winner = (int)(0xFFFFFFFFu - (uint32_t)top);
  const double M = (double)key_value(top);
  double S = 0.0, T = 0.0;
  if (live) {
    const double d = Mg - M, f = exp(d);          // this shard's sums are relative to its own maximum
    S = f * Sg;
    T = f * (Tg + d * Sg);
    if (lane != winner) { S += f; T += f * d; }   // its maximum is an ordinary element of the row
  }
  S = warp_sum(S);
  T = warp_sum(T);
  int n_valid = 0, pos = 0;
  for (; n_valid < K; ++n_valid) {                // the shards' lists are sorted: take the largest head K times
    const unsigned long long h = (live && pos < ng) ? make_key(rec->x[pos], (uint32_t)rec->tok[pos]) : 0ull;
    const uint32_t hi = (uint32_t)(h >> 32), mx_hi = __reduce_max_sync(kFull, hi);
    const uint32_t mx_lo = __reduce_max_sync(kFull, hi == mx_hi ? (uint32_t)h : 0u);
    const unsigned long long mx = ((unsigned long long)mx_hi << 32) | mx_lo;
    if (mx == 0ull) break;
    if (lane == 0) { out_x[n_valid] = key_value(mx); out_tok[n_valid] = key_token(mx); }
    if (h == mx) ++pos;
  }
  for (int r = n_valid + lane; r < K; r += 32) { out_x[r] = -INFINITY; out_tok[r] = -1; }
  *fault_out = fault;
  RowMerge m;
  m.M = M; m.S = S; m.T = T; m.top = top; m.n_valid = n_valid;
  return m;
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
  __shared__ float s_w[5 * C2T_MAX_HIDDEN + 4];
  __shared__ double s_rowM[C2T_MAX_FRONTIER], s_rowL[C2T_MAX_FRONTIER], s_rowH[C2T_MAX_FRONTIER];
  __shared__ int s_rowfault[C2T_MAX_FRONTIER];
  __shared__ float s_x[kMaxCand];
  __shared__ int s_tok[kMaxCand];
  __shared__ double s_C[kMaxCand];
  __shared__ unsigned char s_keep[kMaxCand], s_sel[kMaxCand];
  __shared__ int s_scan[kTreeWarps + 1];
  __shared__ int s_misc[2];
  __shared__ unsigned long long s_keys[kTreeWarps][kStageKeys];
  unsigned long long *s_ckey = &s_keys[0][0];     // phases 2-3 reuse the staging area: a key per candidate
  static_assert(kTreeWarps * kStageKeys >= kMaxCand, "candidate keys must fit the staging area");

  const int b = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int K = t.K, F = t.F;
  const int cur = level & 1, nxt = cur ^ 1;
  chain_release();
  // the classifier's weights were written at init, not by the chain: they are staged while the
  // expand pass may still be finishing
  if (tid == 0) s_misc[1] = 0;                    // survivors of the first pruning
  if (t.classifier == C2T_CLS_MLP) {
    for (int i = tid; i < 3 * t.hidden; i += kTreeThreads) s_w[i] = t.w1[i];
    for (int i = tid; i < t.hidden; i += kTreeThreads) {
      s_w[3 * C2T_MAX_HIDDEN + i] = t.b1[i];
      s_w[4 * C2T_MAX_HIDDEN + i] = t.w2[i];
    }
    if (tid == 0) s_w[5 * C2T_MAX_HIDDEN] = t.b2[0];
  }
  chain_wait();
  int n = t.frontier_n[cur][b];
  const int row_off = t.row_off_draft[b];         // rows of earlier sequences in the expand pass
  const PassInfo info = *t.info_draft;            // (loads issued together with the one above)
  n = n < 0 ? 0 : (n > F ? F : n);
  const size_t cbase = (size_t)b * F * K;

  if (n == 0) {                                   // the loop of Alg. 1 has ended for this sequence
    if (tid == 0) {
      t.frontier_n[nxt][b] = 0;
      t.cand_n[b] = 0;
      if (out.count) out.count[b] = 0;
    }
    return;
  }
  __syncthreads();

  // ---- phase 1: one warp per row merges that row's partial records
  for (int j = warp; j < n; j += kTreeWarps) {
    uint32_t shard_faults = 0u;
    const RowMerge m = records
        ? merge_row_records(t, records, n_shards, b, j, K, &s_x[j * K], &s_tok[j * K], &shard_faults)
        : merge_row_partials(t, info, b, row_off + j, K, t.V, s_keys[warp], &s_x[j * K], &s_tok[j * K], 0);
    if (lane == 0) {
      const uint32_t fault = shard_faults ? shard_faults : row_fault_bits(m.top, m.S, m.T);
      const double L = log1p(m.S);                // ln sum_v e^(x_v - M); the maximum contributes the 1
      s_rowM[j] = m.M;
      s_rowL[j] = L;
      if (t.entropy_top_m > 0 && t.entropy_top_m < t.V) {
        const double2 sm = t.topm[(size_t)b * F + j];               // Eq. 3: only the M most probable tokens,
        s_rowH[j] = (L * sm.x - sm.y) / (1.0 + m.S);               // probabilities of the full softmax
      } else {
        s_rowH[j] = L - m.T / (1.0 + m.S);        // Eq. 2 with natural log
      }
      s_rowfault[j] = (int)fault;
      if (fault) atomicOr(&t.status[b], fault);
    }
  }
  __syncthreads();

  // ---- phase 2: features and confidence, one thread per candidate child
  const int nc = n * K;
  for (int c = tid; c < nc; c += kTreeThreads) {
    const int j = c / K;
    const int f = t.frontier_node[cur][(size_t)b * F + j];
    const int tok = s_tok[c];
    const float x = s_x[c];
    const bool ok = tok >= 0 && !s_rowfault[j];
    const double lp = (x > kNegInfAsFinite) ? ((double)x - s_rowM[j]) - s_rowL[j] : -INFINITY;
    const double logP = t.tree_logP[(size_t)b * t.cap + f] + lp;           // Eq. 1 in log space
    const double P = exp(logP);
    const double H = s_rowH[j];
    double C;
    if (!ok) C = NAN;
    else if (t.classifier == C2T_CLS_IDENTITY_JOINT) C = P;
    else if (t.classifier == C2T_CLS_IDENTITY_COND) C = exp(lp);
    else C = classify(t, s_w, P, H, (double)level);
    const bool keep = ok && C >= (double)t.beta;                            // first pruning
    s_C[c] = C;
    s_keep[c] = keep;
    s_sel[c] = keep;
    // (C desc, index asc) as integer compares: an orderable image of C, 0 for a dropped candidate
    const unsigned long long cb = (unsigned long long)__double_as_longlong(C);
    s_ckey[c] = keep ? (cb ^ ((cb >> 63) ? ~0ull : 0x8000000000000000ull)) : 0ull;
    if (keep) atomicAdd(&s_misc[1], 1);
    t.cand_token[cbase + c] = tok;
    t.cand_lp[cbase + c] = ok ? lp : NAN;
    t.cand_logP[cbase + c] = ok ? logP : NAN;
    t.cand_H[cbase + c] = ok ? H : NAN;
    t.cand_C[cbase + c] = C;
  }
  __syncthreads();

  // ---- phase 3: second pruning, the F survivors that come first under (C desc, index asc)
  const int n_keep = s_misc[1];
  if (n_keep > F) {
    // four threads per survivor share the comparisons against all candidates
    for (int c0 = 0; c0 < nc; c0 += kTreeThreads / 4) {
      const int c = c0 + (tid >> 2);
      const unsigned long long kc = c < nc ? s_ckey[c] : 0ull;
      int rank = 0;
      if (kc != 0ull)
        for (int o = tid & 3; o < nc; o += 4) {
          const unsigned long long ko = s_ckey[o];
          rank += (ko > kc) || (ko == kc && o < c);
        }
      rank += __shfl_xor_sync(kFull, rank, 1);
      rank += __shfl_xor_sync(kFull, rank, 2);
      if (kc != 0ull && (tid & 3) == 0) s_sel[c] = rank < F;
    }
  }
  __syncthreads();

  // ---- phase 4: stable compaction in candidate order; append to the tree, emit the frontier
  const int per = (nc + kTreeThreads - 1) / kTreeThreads;      // consecutive candidates per thread
  const int c0 = tid * per, c1 = (c0 + per < nc) ? c0 + per : nc;
  const bool add_all = t.tree_add == C2T_ADD_ALL_SURVIVORS;
  int n_add = 0, n_sel = 0;
  for (int c = c0; c < c1; ++c) { n_add += add_all ? s_keep[c] : s_sel[c]; n_sel += s_sel[c]; }
  // one scan for both counts (each at most kMaxCand = 1024: 16 bits apiece)
  int tot_both;
  const int off_both = block_exclusive_scan(n_add | (n_sel << 16), s_scan, &tot_both);
  int off_add = off_both & 0xFFFF, off_sel = off_both >> 16;
  const int tot_add = tot_both & 0xFFFF, tot_sel = tot_both >> 16;
  const int base = t.tree_n[b];
  const bool overflow = base + tot_add > t.cap;
  const size_t tb = (size_t)b * t.cap;
  for (int c = c0; c < c1; ++c) {
    const bool add = add_all ? s_keep[c] : s_sel[c];
    int flags = (s_keep[c] ? 1 : 0) | (s_sel[c] ? 2 : 0);
    t.cand_flags[cbase + c] = flags;
    if (!add) continue;
    const int id = base + off_add++;
    if (id < t.cap) {
      const int j = c / K;
      const int f = t.frontier_node[cur][(size_t)b * F + j];
      t.tree_token[tb + id] = s_tok[c];
      t.tree_parent[tb + id] = f;
      t.tree_level[tb + id] = level + 1;
      t.tree_logP[tb + id] = t.cand_logP[cbase + c];
      t.tree_C[tb + id] = s_C[c];
      const double ch = t.tree_Chat[tb + f];
      t.tree_Chat[tb + id] = s_C[c] < ch ? s_C[c] : ch;
    }
    if (s_sel[c] && !overflow) {
      const int slot = off_sel++;
      if (!C2T_IN_BOUNDS(slot, F, &t.status[b])) continue;
      t.frontier_node[nxt][(size_t)b * F + slot] = id;
      if (out.token) out.token[(size_t)b * F + slot] = s_tok[c];
      if (out.node_id) out.node_id[(size_t)b * F + slot] = id;
      if (out.parent_slot) out.parent_slot[(size_t)b * F + slot] = c / K;
    }
  }
  __syncthreads();
  if (tid == 0) {
    const int next_n = overflow ? 0 : tot_sel;
    t.tree_n[b] = overflow ? t.cap : base + tot_add;
    t.frontier_n[nxt][b] = next_n;
    t.cand_n[b] = nc;
    if (out.count) out.count[b] = next_n;
    if (overflow) atomicOr(&t.status[b], C2T_ST_TREE_OVERFLOW);
  }
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
    const int off = block_exclusive_scan(keep, s_scan, &total);
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
    const int off = block_exclusive_scan(leaf, s_scan, &total);
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
  block_exclusive_scan(part, s_scan, &total);
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
    block_exclusive_scan(part, s_scan, &total);
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

__global__ void __launch_bounds__(kWalkThreads) lazy_walk_round_kernel(TreeState t, int round, c2t_accept_out out) {
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

    const long long first_vec = (long long)a * info.vec_per_row;
    const int c_first = (int)(first_vec / info.span);
    const int c_last = (int)((first_vec + info.vec_per_row - 1) / info.span);
    int n_splits = c_last - c_first + 1;
    if (n_splits > t.max_splits_tgt) {
      n_splits = t.max_splits_tgt;
      atomicOr(&t.status[b], C2T_ST_INTERNAL);
    }
    unsigned long long best = 0ull;
    for (int sp = 0; sp < n_splits; ++sp) {
      const unsigned long long k = t.part_best[(size_t)a * t.max_splits_tgt + sp];
      best = k > best ? k : best;
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

cudaError_t launch_lazy_walk_round(const TreeState &t, int round, const c2t_accept_out *out, cudaStream_t s) {
  c2t_accept_out o;
  memset(&o, 0, sizeof o);
  if (out) o = *out;
  return launch_chained(lazy_walk_round_kernel, dim3(1), dim3(kWalkThreads), 0, s, t, round, o);
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
  return launch_chained(prune_level_kernel, dim3(t.B), dim3(kTreeThreads), 0, s, t, level, o, records, n_shards);
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

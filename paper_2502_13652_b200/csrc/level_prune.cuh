// The per-sequence work of a level (Eq. 1, Eq. 4, Alg. 1, Sec. 4.2.2): merge of the rows' partial records,
// features, classifier, the two prunings, compaction, tree append.  A device function, so that the pruning kernel
// (one CTA per sequence) and the expand kernel's last CTA (small batches: expand and prune in one launch) share it.
#pragma once

#include "c2t_internal.h"

namespace c2t {
namespace {

constexpr int kMaxCand = C2T_MAX_TOPK * C2T_MAX_FRONTIER;   // 1024
constexpr unsigned kFullMask = 0xFFFFFFFFu;

__device__ __forceinline__ double warp_sum(double v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_down_sync(kFullMask, v, o);
  return __shfl_sync(kFullMask, v, 0);
}

// Exclusive scan of one int per thread over a CTA of NT threads; returns the exclusive prefix, *total = sum.
template <int NT>
__device__ int block_exclusive_scan(int v, int *s_warp /*[NT/32+1]*/, int *total) {
  constexpr int kTreeWarps = NT / 32;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  int inc = v;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    int t = __shfl_up_sync(kFullMask, inc, o);
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
    unsigned long long other = __shfl_xor_sync(kFullMask, top, o);
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
      const uint32_t hi = (uint32_t)(h >> 32), mx_hi = __reduce_max_sync(kFullMask, hi);
      const uint32_t mx_lo = __reduce_max_sync(kFullMask, hi == mx_hi ? (uint32_t)h : 0u);
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
    for (int o = 16; o > 0; o >>= 1) n_valid += __shfl_xor_sync(kFullMask, n_valid, o);
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
  const uint32_t fault = __reduce_or_sync(kFullMask, fg & ~(uint32_t)C2T_ST_ALL_NEGINF);
  // the row maximum is the best of the shards' maxima; equal values go to the lower shard, whose token ids are lower
  unsigned long long top = live ? (((unsigned long long)f32_orderable(__float_as_uint((float)Mg)) << 32) |
                                   (0xFFFFFFFFu - (uint32_t)lane)) : 0ull;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    unsigned long long other = __shfl_xor_sync(kFullMask, top, o);
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
    const uint32_t hi = (uint32_t)(h >> 32), mx_hi = __reduce_max_sync(kFullMask, hi);
    const uint32_t mx_lo = __reduce_max_sync(kFullMask, hi == mx_hi ? (uint32_t)h : 0u);
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

// records == nullptr: the rows come from this context's own expand pass; else from gathered records of n_shards shards
// The shared memory of prune_level_body for a CTA of NW warps.
template <int NW>
struct PruneShared {
  double rowM[C2T_MAX_FRONTIER], rowL[C2T_MAX_FRONTIER], rowH[C2T_MAX_FRONTIER];
  double C[kMaxCand];
  double logP[kMaxCand];                       // joint log-probability of every candidate
  unsigned long long keys[NW][kStageKeys];
  float w[5 * C2T_MAX_HIDDEN + 4];
  float x[kMaxCand];
  int tok[kMaxCand];
  double flogP[C2T_MAX_FRONTIER];              // joint log-probability of every frontier node
  double fchat[C2T_MAX_FRONTIER];              // its smallest confidence on the path from the root
  int fnode[C2T_MAX_FRONTIER];                 // tree id of every frontier node
  int rowfault[C2T_MAX_FRONTIER];
  int scan[NW + 1];
  int misc[2];
  unsigned char keep[kMaxCand], sel[kMaxCand];
};

// NT: threads of the CTA; b: the sequence; chained: the caller is a kernel of the launch chain of its own (the
// classifier's weights are then staged before the wait for the predecessor).
template <int NT, bool CHAINED>
__device__ void prune_level_body(const TreeState &t, int level, const c2t_frontier &out, const c2t_row_record *records,
                                 int n_shards, int b, PruneShared<NT / 32> &sh) {
  constexpr int kTreeThreads = NT, kTreeWarps = NT / 32;
  float *s_w = sh.w;
  double *s_rowM = sh.rowM, *s_rowL = sh.rowL, *s_rowH = sh.rowH;
  int *s_rowfault = sh.rowfault;
  float *s_x = sh.x;
  int *s_tok = sh.tok;
  double *s_C = sh.C;
  unsigned char *s_keep = sh.keep, *s_sel = sh.sel;
  int *s_scan = sh.scan;
  int *s_misc = sh.misc;
  unsigned long long (*s_keys)[kStageKeys] = sh.keys;
  unsigned long long *s_ckey = &s_keys[0][0];     // phases 2-3 reuse the staging area: a key per candidate
  static_assert(kTreeWarps * kStageKeys >= kMaxCand, "candidate keys must fit the staging area");

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int K = t.K, F = t.F;
  const int cur = level & 1, nxt = cur ^ 1;
  if (CHAINED) chain_release();
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
  if (CHAINED) chain_wait();
  __syncthreads();                                // (a CTA that serves several sequences: the last one's reads are done)
  int n = t.frontier_n[cur][b];
  const int row_off = t.row_off_draft[b];         // rows of earlier sequences in the expand pass
  const PassInfo info = *t.info_draft;            // (loads issued together with the one above)
  const int tree_base = t.tree_n[b];              // (needed last; its latency hides behind everything else)
  // the frontier's nodes, their joint log-probabilities (Eq. 1's left factor) and path confidences: two dependent
  // loads, issued by the last warp (the one least likely to have a row) so that they run beside the rows' merges;
  // phases 2 and 4 read them, behind barriers (slots past the frontier's size hold anything: kept in bounds, unused)
  if (warp == kTreeWarps - 1 && lane < F) {
    int f = t.frontier_node[cur][(size_t)b * F + lane];
    f = f < 0 ? 0 : (f >= t.cap ? t.cap - 1 : f);
    sh.fnode[lane] = f;
    sh.flogP[lane] = t.tree_logP[(size_t)b * t.cap + f];
    sh.fchat[lane] = t.tree_Chat[(size_t)b * t.cap + f];
  }
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
  // (no barrier here: phase 1 reads nothing that was written above)

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
    const int tok = s_tok[c];
    const float x = s_x[c];
    const bool ok = tok >= 0 && !s_rowfault[j];
    const double lp = (x > kNegInfAsFinite) ? ((double)x - s_rowM[j]) - s_rowL[j] : -INFINITY;
    const double logP = sh.flogP[j] + lp;                                   // Eq. 1 in log space
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
    sh.logP[c] = logP;
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
      rank += __shfl_xor_sync(kFullMask, rank, 1);
      rank += __shfl_xor_sync(kFullMask, rank, 2);
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
  const int off_both = block_exclusive_scan<NT>(n_add | (n_sel << 16), s_scan, &tot_both);
  int off_add = off_both & 0xFFFF, off_sel = off_both >> 16;
  const int tot_add = tot_both & 0xFFFF, tot_sel = tot_both >> 16;
  const int base = tree_base;
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
      const int f = sh.fnode[j];
      t.tree_token[tb + id] = s_tok[c];
      t.tree_parent[tb + id] = f;
      t.tree_level[tb + id] = level + 1;
      t.tree_logP[tb + id] = sh.logP[c];              // (a node is only added if its candidate was in order)
      t.tree_C[tb + id] = s_C[c];
      const double ch = sh.fchat[j];
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

}  // namespace
}  // namespace c2t

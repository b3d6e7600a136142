// Internal declarations shared by the CUDA translation units of libc2t.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "c2t.h"

namespace c2t {

// ---------------------------------------------------------------- keys ------
// Total order used everywhere a "largest logit, then lowest token id" decision is taken:
// key = (orderable(value) << 32) | (0xFFFFFFFF - token).  A larger key wins.  0 = empty.

__host__ __device__ __forceinline__ uint32_t f32_orderable(uint32_t bits) {
  return bits ^ ((bits & 0x80000000u) ? 0xFFFFFFFFu : 0x80000000u);
}
__host__ __device__ __forceinline__ uint32_t f32_from_orderable(uint32_t o) {
  return o ^ ((o & 0x80000000u) ? 0x80000000u : 0xFFFFFFFFu);
}
__device__ __forceinline__ unsigned long long make_key(float x, uint32_t tok) {
  return ((unsigned long long)f32_orderable(__float_as_uint(x)) << 32) | (0xFFFFFFFFu - tok);
}
__device__ __forceinline__ float key_value(unsigned long long k) {
  return __uint_as_float(f32_from_orderable((uint32_t)(k >> 32)));
}
__device__ __forceinline__ int32_t key_token(unsigned long long k) {
  return (int32_t)(0xFFFFFFFFu - (uint32_t)k);
}

// Logits of -inf (and anything below -2^127) are read as -2^127, so that "probability zero"
// never produces inf - inf or 0 * inf in the running sums.
constexpr float kNegInfAsFinite = -1.7e38f;   // anything at or below this was -inf (or as good as)

// ---------------------------------------------------------------- index checks
// A build with -DC2T_DEBUG_BOUNDS checks the indices of the kernels' writes to shared memory queues, pools and
// workspace records: a failed check sets C2T_ST_INTERNAL in the given status word (if there is one) and the guarded
// access is skipped.  It stands in for a memory checker where none can be run.  In a normal build the check is the
// constant `true`.
#ifdef __CUDACC__
#ifdef C2T_DEBUG_BOUNDS
__device__ __forceinline__ bool c2t_in_bounds(unsigned long long i, unsigned long long n, uint32_t *status) {
  if (i < n) return true;
  if (status) atomicOr(status, (uint32_t)C2T_ST_INTERNAL);
  return false;
}
#define C2T_IN_BOUNDS(i, n, status) c2t_in_bounds((unsigned long long)(i), (unsigned long long)(n), (status))
#else
#define C2T_IN_BOUNDS(i, n, status) true
#endif
#endif

// ---------------------------------------------------------------- launch chain
// The kernels of a decode step form a chain in which each one consumes what the one before wrote.
// They are launched with programmatic stream serialisation: the next kernel's CTAs may be placed
// on SMs (and its launch latency paid) while the previous kernel is still finishing.  Every kernel
// of the chain therefore starts with chain_enter(): it lets its own successor be scheduled and then
// waits until the predecessor has completed and its writes are visible.  Nothing touches global
// memory before that, so the chain behaves exactly like plain stream order.
#ifdef __CUDACC__
__device__ __forceinline__ void chain_release() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void chain_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void chain_enter() {
  chain_release();
  chain_wait();
}

template <typename... KArgs, typename... Args>
cudaError_t launch_chained(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t s,
                           Args &&...args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = s;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...);
}
#endif

// ---------------------------------------------------------------- vocab pass -

constexpr int kPassThreads = 512;     // threads per CTA of the vocabulary pass
constexpr int kPassCtasPerSm = 2;
constexpr int kMinSpanVectors = 1024; // a CTA never gets fewer 16-byte vectors than this
// the expand pass: every warp is a worker of its own (a span of the rows, its own partial records).
// 20 warps per SM: 96 registers per thread (no spills) and fewer segments to open than with 24; measured
// 3 % faster than 24 warps and 4 % faster than 16.
constexpr int kExpandThreads = 640;
// 16-byte vectors a lane holds of one group (a group is 32 times this).  Measured on 640 rows of 128256 bf16 logits:
// 4 with 20 warps 44 us; 2 with 24 warps 45 us; 8 with 10 or 14 warps 67 us.
constexpr int kExpandVecPerLane = 4;
constexpr int kExpandCtasPerSm = 1;
constexpr int kExpandWarps = kExpandThreads / 32;
// Opening a segment (filter warm-up, extra drains while the filter is still loose, the record)
// costs a warp about as much as streaming this many vectors (measured: the 640-row level is
// fastest with 1024 to 2048).  The expand pass cuts the rows into spans of equal COST: every row
// is preceded by this many virtual vectors, the padded rows are laid end to end and cut evenly,
// and a worker streams the real vectors of its piece.
constexpr int kSegmentPad = 1024;
constexpr int kHeldPerSlot = 1;       // exact keys held out of the fp32 sums per partial record

// What one launch of the vocabulary pass derived from the device-side row counts.
struct PassInfo {
  int32_t n_rows;       // active rows
  int32_t vec_per_row;  // 16-byte vectors per row (last one may be ragged)
  int64_t span;         // vectors per worker (a CTA of the arg-max pass, a warp of the expand pass)
  int32_t pad;          // expand pass: virtual vectors in front of every row (see kSegmentPad), else 0
  int32_t reserved;
};

struct TopmSegment;

struct PassParams {
  const void *logits;
  int64_t seq_stride, row_stride;   // elements
  int32_t V, K, B;
  int32_t rows_per_seq_max;         // F (draft) or Nw (target)
  const int32_t *counts;            // [B] active rows per sequence, device
  const int32_t *row_sel;           // arg-max pass only, may be null: [B] the row of sequence b to read (then counts is 0 or 1)
  int32_t max_splits;               // partial slots per row
  int32_t min_span;                 // expand: the fewest vectors a worker gets (expand_min_span)
  int64_t n_slots;                  // partial slots in the workspace (rows the workspace was carved for x max_splits)
  uint32_t *status;                 // may be null: a status word for C2T_ST_INTERNAL (the first sequence's)
  PassInfo *info;                   // written by CTA 0
  int32_t *row_off;                 // may be null: [B+1] first active row of every sequence, written by CTA 0
  // expand: per (row, split) partial
  float4 *part_stats;               // {offset c, S, U, n_keys as int bits}: base-2 sums, see expand_pass.cu
  unsigned long long *part_keys;    // [.. * K] the segment's K largest keys, sorted descending, 0-padded
  unsigned long long *part_held;    // [.. * kHeldPerSlot] keys excluded from S and U (0 = none)
  // expand with M > 0 (else null): the pool of candidate vectors, cut evenly among the workers, and a record per (row, split)
  uint4 *topm_pool;
  long long topm_pool_vecs;
  TopmSegment *topm_seg;
  // argmax: per (row, split) best key
  unsigned long long *part_best;
};

// ---------------------------------------------------------------- candidates of the truncated entropy (Eq. 3)
// With entropy_top_m = M > 0 the expand pass also sets aside every 16-byte vector that holds an element at or above
// a floor of its segment: the kTopmRank-th largest of the 32 lane maxima over the segment's first two groups, about
// the top 2 % of the elements seen there (M = 1000 of 128256 is the top 0.8 %).  The vectors go, in stream order, to
// a region of the warp's own in a pool in global memory; the segment's record says where they are and what the floor
// was.  A small kernel per row then takes the elements at or above the row's highest floor F from those vectors: if
// there are at least M of them the M-th largest is among them and so is everything above it, and Eq. 3's sums follow
// without reading the row again.  Rows for which that fails (a region ran full, fewer than M elements at or above F,
// more than fit in shared memory) are left to the pass that reads the row again.
constexpr int kTopmRank = 24;
constexpr int kTopmPoolDivisor = 3;      // the pool holds a third of the largest level's vectors (twice what is expected)
constexpr float kTopmLowestFloor = -1.7e38f;   // above -2^127, the value that pads a ragged vector
struct TopmSegment {
  int first;       // the segment's first vector in the pool
  int n;           // vectors, or -1: the region ran full
  float floor;
  int pad;
};
size_t topm_pool_vectors(size_t batch, size_t rows_per_seq, int vocab, int elem_bytes);

// partial slots a row can need; workers: CTAs (arg-max, pad 0) or warps (expand, pad kSegmentPad)
int max_splits_for(int vocab, int elem_bytes, int workers, int pad, int min_span = kMinSpanVectors);
// Keys of a row's partial lists that one warp of the row merge stages in shared memory; a row with more takes a slow path.
constexpr int kStageKeys = 320;
// The fewest vectors a worker of the expand pass gets: as few as the row merge allows (at most 31 partial lists per
// row, and K keys apiece must fit the staging area), so that launches with few rows still spread over the chip.
int expand_min_span(int vocab, int elem_bytes, int K);

cudaError_t prepare_expand_pass();   // once per device: opt in to the kernel's shared-memory size
cudaError_t launch_expand_pass(const PassParams &p, int dtype, int grid, cudaStream_t s);
cudaError_t launch_argmax_pass(const PassParams &p, int dtype, int grid, cudaStream_t s);
struct TreeState;
// expand and prune of a level in one launch (batches of at most C2T_FUSED_MAX_BATCH sequences)
cudaError_t launch_expand_prune(const PassParams &p, const TreeState &t, int level, const c2t_frontier *out, int dtype,
                                int grid, cudaStream_t s);
// ---------------------------------------------------------------- tree state -

struct TreeState {
  int32_t B, V, K, F, D, N, Nw, W, cap, hidden, classifier, tree_add, max_splits, max_splits_tgt, min_span;
  float beta;
  // frontier, double buffered by level parity
  int32_t *frontier_n[2];      // [B]
  int32_t *frontier_node[2];   // [B, F]
  // tree
  int32_t *tree_n;             // [B]
  int32_t *tree_token, *tree_parent, *tree_level;   // [B, cap]
  double *tree_logP, *tree_C, *tree_Chat;           // [B, cap]
  int32_t *remap;              // [B, cap] scratch of the rerank
  // candidates of the last level
  int32_t *cand_n;             // [B]
  int32_t *cand_token, *cand_flags;                 // [B, F*K]
  double *cand_lp, *cand_logP, *cand_H, *cand_C;    // [B, F*K]
  // final tree
  int32_t *final_n;            // [B]
  int32_t *final_src, *final_token, *final_parent, *final_level;   // [B, Nw]
  int32_t *node_argmax;        // [B, Nw]
  int32_t *root_tok, *prefix_len;                   // [B]
  int32_t *walk_active, *walk_cur, *walk_len;       // [B] state of the lazy acceptance walk
  int32_t entropy_top_m;       // M of Eq. 3 (0: exact entropy)
  double2 *topm;               // [B, F] {S_M, T_M} of the last expand call when M > 0
  uint4 *topm_pool;            // M > 0: candidate vectors set aside by the expand pass
  long long topm_pool_vecs;
  TopmSegment *topm_seg;       // M > 0: [B * F * max_splits] where each segment's candidates are
  int32_t *topm_done;          // M > 0: [B, F] 1 where the row's sums came from the candidate vectors
  uint32_t *status;            // [B]
  uint32_t *ticket;            // one counter: CTAs of a fused expand + prune launch that have finished (0 between launches)
  PassInfo *info_draft, *info_target;
  int32_t *row_off_draft;          // [B+1] first row of every sequence in the last expand pass
  float4 *part_stats;
  unsigned long long *part_keys;
  unsigned long long *part_held;
  unsigned long long *part_best;
  float *w1, *b1, *w2, *b2;
};

// truncated entropy (Eq. 3): per active row (b, j) the sums over its M largest logits, out[b * F + j] = {S_M, T_M};
// runs after the expand pass of the same level, whose partial records give it the row maxima
cudaError_t prepare_topm_pass();     // once per device: opt in to the kernel's shared-memory size
cudaError_t prepare_tree_kernels();  // the same for the pruning kernel
cudaError_t launch_topm_entropy(const void *logits, int64_t seq_stride, int64_t row_stride, int V, int M, int F,
                                int B, const int32_t *counts, const TreeState &t, double2 *out, const int32_t *done,
                                int n_ctas, int dtype, cudaStream_t s);
// the same sums from the candidate vectors of the expand pass, for the rows where they suffice (t.topm_done says
// which; launch_topm_entropy skips those when given t.topm_done)
cudaError_t launch_topm_finish(int M, int F, int B, const int32_t *counts, const TreeState &t, double2 *out, int dtype,
                               cudaStream_t s);
cudaError_t launch_begin_step(const TreeState &t, const int32_t *root_tok, const int32_t *prefix_len,
                              cudaStream_t s);
// records == nullptr: rows merged from this context's own expand pass; else from n_shards gathered records per row
cudaError_t launch_prune_level(const TreeState &t, int level, const c2t_frontier *out, const c2t_row_record *records,
                               int n_shards, cudaStream_t s);
cudaError_t launch_export_rows(const TreeState &t, int level, int vocab_count, int vocab_begin, c2t_row_record *out,
                               cudaStream_t s);
cudaError_t launch_final_prune(const TreeState &t, cudaStream_t s);
cudaError_t launch_build_verify(const TreeState &t, const c2t_verify *out, cudaStream_t s);
cudaError_t launch_dense_mask(const TreeState &t, void *out, int out_dtype, int64_t kv_len, cudaStream_t s);
// gathered == nullptr: node arg-maxes from this context's own pass; else the best of n_shards gathered keys per node
cudaError_t launch_accept_walk(const TreeState &t, const c2t_accept_out *out, const unsigned long long *gathered,
                               int n_shards, cudaStream_t s);
cudaError_t launch_export_best(const TreeState &t, int vocab_begin, unsigned long long *out, cudaStream_t s);
// one round of the lazy walk: round 0 starts it, round r > 0 consumes the arg-max of round r-1
// gathered == nullptr: the round consumes this context's own arg-max pass; else n_shards gathered keys per sequence
cudaError_t launch_lazy_walk_round(const TreeState &t, int round, const c2t_accept_out *out,
                                   const unsigned long long *gathered, int n_shards, cudaStream_t s);
cudaError_t launch_export_lazy_best(const TreeState &t, int vocab_begin, unsigned long long *out, cudaStream_t s);

}  // namespace c2t

/*
 * libc2t — draft-tree construction for speculative decoding with a confidence
 * classifier (C2T, arXiv 2502.13652), as CUDA kernels for sm_100a behind a C ABI.
 *
 * One context serves B independent sequences on one GPU.  A decode step is
 *
 *   c2t_begin_step
 *   for level = 0 .. D-1:   c2t_expand_level(level, draft logits)   (Sec. 4.2.1, Eq. 1-3)
 *                           c2t_prune(level)                        (Eq. 4, Alg. 1, Sec. 4.2.2)
 *                           [caller runs its draft model on the emitted frontier]
 *   c2t_prune(C2T_FINAL)                                            (Top-N rerank, Sec. 2.2)
 *   c2t_build_verify                                                (tree attention, Sec. 2.2)
 *   c2t_accept(target logits)                                       (accept length, Sec. 5 Metrics)
 *
 * Conventions, unless a function says otherwise:
 *   - pointers named *_dev are device pointers, *_host host pointers; "stream" is a
 *     cudaStream_t passed as void* (NULL = the legacy default stream);
 *   - every call returns C2T_OK (0) or a negative C2T_E* code; nothing throws, exits
 *     or prints;
 *   - calls only enqueue work on `stream` and return; outputs are valid in stream
 *     order.  Only c2t_status and c2t_decode_step_host synchronise;
 *   - the library never allocates or frees device memory: the workspace, every input
 *     and every output belong to the caller, who keeps them alive until the work
 *     that uses them has finished;
 *   - a context is not thread-safe; use one context per stream;
 *   - data faults (NaN or +inf in a logits row, a row of only -inf, a tree that
 *     outgrows its capacity) never fault the device: they set bits in a per-sequence
 *     status word and leave that sequence's results unspecified but in bounds.
 */
#ifndef C2T_H
#define C2T_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct c2t_ctx c2t_ctx;

typedef enum { C2T_F32 = 0, C2T_BF16 = 1 } c2t_dtype;
/* C2T_CLS_MLP: the paper's two-layer FFN.  C2T_CLS_IDENTITY_JOINT: confidence := joint
 * probability, which turns the method into EAGLE-2's expand + rerank (Sec. 2.2) and, with
 * K = F = 1, into the "DyJoint" early-stop rule of the chain-mode comparison (Sec. 5, Benefits
 * in Chain Mode).  C2T_CLS_IDENTITY_COND: confidence := the child's own probability under its
 * parent's distribution; with K = F = 1 the child is the arg-max token, so this is that
 * comparison's "DyMax" rule (stop when the maximum probability falls below the threshold). */
typedef enum { C2T_CLS_MLP = 0, C2T_CLS_IDENTITY_JOINT = 1, C2T_CLS_IDENTITY_COND = 2 } c2t_classifier;
/* What "extend N or topK(N) to T" (Alg. 1) adds to the tree at a level: only the capped
 * next-layer generators, or every node that passed the threshold. */
typedef enum { C2T_ADD_FRONTIER = 0, C2T_ADD_ALL_SURVIVORS = 1 } c2t_tree_add;

#define C2T_FINAL (-1)

#define C2T_OK       0
#define C2T_EINVAL  (-1)   /* null pointer, non-positive size, unknown enum value        */
#define C2T_EALIGN  (-2)   /* logits base or stride not 16-byte aligned                  */
#define C2T_ERANGE  (-3)   /* a size exceeds a C2T_MAX_* limit or the workspace is small */
#define C2T_EORDER  (-4)   /* calls out of sequence within a decode step                 */
#define C2T_ECUDA   (-5)   /* a CUDA runtime call failed                                 */
#define C2T_ENOMEM  (-6)   /* the host could not allocate the context                    */

#define C2T_MAX_BATCH     4096
#define C2T_MAX_TOPK      32
#define C2T_MAX_FRONTIER  32
#define C2T_MAX_HIDDEN    64
#define C2T_MAX_DEPTH     32
#define C2T_MAX_BUDGET    1024
#define C2T_MAX_TREE      8192   /* nodes per sequence before the Top-N rerank */
#define C2T_MAX_SHARDS    32     /* vocabulary shards merged by c2t_prune_gathered */
#define C2T_FUSED_MAX_BATCH 2    /* largest batch for which c2t_expand_prune_level uses a single launch */

/* per-sequence status bits */
#define C2T_ST_NAN_LOGIT     1u
#define C2T_ST_POSINF_LOGIT  2u
#define C2T_ST_ALL_NEGINF    4u
#define C2T_ST_TREE_OVERFLOW 8u
/* The library caught itself outside its own bounds: a row has more partial records than the workspace
 * was carved for, or (in a build with -DC2T_DEBUG_BOUNDS) an index check failed.  The access is
 * clamped or skipped, never made; the sequence's results are unspecified.  Never set by data. */
#define C2T_ST_INTERNAL      16u

/*
 * Method parameters (Alg. 1's inputs d_max and beta; Top-K of Sec. 4.2.2 split into the
 * K children classified per node and the F generators kept per layer, K = F in the
 * paper; EAGLE-2's N of Sec. 2.2; the classifier of Sec. 4.1).
 */
typedef struct {
  int32_t batch;          /* B sequences                                                  */
  int32_t vocab;          /* V                                                            */
  int32_t dtype;          /* c2t_dtype of draft and target logits                         */
  int32_t max_depth;      /* D = d_max draft rounds                                       */
  int32_t topk;           /* K                                                            */
  int32_t frontier_cap;   /* F                                                            */
  int32_t budget;         /* N, counts the root; 0 = no rerank                            */
  float   threshold;      /* beta; a node is kept iff C >= beta                           */
  int32_t entropy_top_m;  /* M of Eq. 3: entropy over the M most probable tokens, their
                             probabilities not renormalised; 0 (or M >= V) = exact, Eq. 2.
                             M > 0 adds a pool of a third of [B, F, V] to the workspace     */
  int32_t classifier;     /* c2t_classifier                                               */
  int32_t hidden;         /* h                                                            */
  const float *w1;        /* HOST [h*3] row-major, features in the order (P, H, d)        */
  const float *b1;        /* HOST [h]                                                     */
  const float *w2;        /* HOST [h]                                                     */
  const float *b2;        /* HOST [1]     (all four copied at init; unused in identity mode) */
  int32_t tree_add;       /* c2t_tree_add                                                 */
  int32_t device;         /* CUDA device ordinal                                          */
} c2t_config;

/* Sizes derived from a configuration (0 on an invalid configuration). */
size_t  c2t_workspace_bytes(const c2t_config *cfg);  /* device workspace the caller provides   */
int32_t c2t_tree_capacity(const c2t_config *cfg);    /* nodes per sequence before the rerank   */
int32_t c2t_final_width(const c2t_config *cfg);      /* Nw: node slots per sequence after it   */
int32_t c2t_mask_words(const c2t_config *cfg);       /* W = ceil(Nw / 64)                      */

/*
 * Validates cfg, copies the classifier weights to the device and carves `workspace_dev`
 * (256-byte aligned, at least c2t_workspace_bytes(cfg), owned by the caller for the life
 * of the context).  Synchronous.  On success *out receives the context.
 */
int c2t_init(const c2t_config *cfg, void *workspace_dev, size_t workspace_bytes, c2t_ctx **out);
void c2t_destroy(c2t_ctx *ctx);

/*
 * Starts a decode step: tree = {root}, C_root = 1, frontier = {root}  (Alg. 1, initialisation).
 * root_tok_dev [B] int32: the token the target model produced last; prefix_len_dev [B] int32:
 * tokens already committed (only used for position ids).  Clears the status words.
 */
int c2t_begin_step(c2t_ctx *ctx, const int32_t *root_tok_dev, const int32_t *prefix_len_dev,
                   void *stream);

/*
 * Post-processing of one draft round (Sec. 4.2.1; Eq. 2; Top-K purpose 1 of Sec. 4.2.2):
 * for every active frontier slot (b, j), j < n_level(b), one pass over logits row (b, j)
 * yields the softmax normaliser, the exact entropy of the row and its K most probable
 * tokens (ties to the lower token id).  Results stay in the workspace for c2t_prune.
 * With cfg.entropy_top_m = M, 0 < M < V, the pass also sets aside the vectors that can hold one
 * of a row's M most probable tokens, and a second kernel takes the entropy over those M (Eq. 3),
 * which c2t_prune then uses instead, from them; only a row for which they do not suffice (see
 * c2t_view.topm_from_pass) is read once more.  (Those M terms are added in fp64 in an order that
 * depends on timing, so with M > 0 two runs may differ in the last bits of the entropy; everything
 * else, and all of it with M = 0, repeats bit for bit.)
 *   logits_dev: [B, F, V] of cfg.dtype; element offset of (b, j, v) =
 *               b*seq_stride + j*row_stride + v.  Base address 16-byte aligned, both strides
 *               multiples of 16 bytes.  Rows of inactive slots are never read.
 *   level:      must equal the number of c2t_prune calls made since c2t_begin_step.
 */
int c2t_expand_level(c2t_ctx *ctx, int level, const void *logits_dev, int64_t seq_stride,
                     int64_t row_stride, void *stream);

/* Next-layer generators, written by c2t_prune(level >= 0).  Caller-owned device arrays;
 * any pointer may be NULL to skip that output. */
typedef struct {
  int32_t *count;        /* [B]     n_{level+1}(b) <= F                                   */
  int32_t *token;        /* [B, F]  token of generator slot j (input of the draft model)  */
  int32_t *node_id;      /* [B, F]  its id in the tree                                    */
  int32_t *parent_slot;  /* [B, F]  slot of its parent in the current level's frontier    */
} c2t_frontier;

/*
 * level >= 0 — classify and prune the children found by c2t_expand_level(level):
 *   joint probability P = P_parent * p (Eq. 1), features (P, H of the parent's row, d = level),
 *   confidence C = F(P, H, d) (Eq. 4), first pruning C >= beta (Alg. 1), second pruning: the F
 *   survivors with the highest C (ties to the earlier candidate) generate the next layer
 *   (Sec. 4.2.2); survivors are appended to the tree in candidate order (parent slot, then
 *   rank) according to cfg.tree_add.  `out` may be NULL.
 * level == C2T_FINAL — Top-N rerank (Sec. 2.2): keep the root and the N-1 nodes with the
 *   highest score, the score of a node being the minimum confidence on its root path (ties
 *   to the lower node id), renumbered in creation order.  `out` is ignored.  Must follow the
 *   last level pruned (any number of levels <= D).
 */
int c2t_prune(c2t_ctx *ctx, int level, const c2t_frontier *out, void *stream);

/*
 * c2t_expand_level(level, ...) followed by c2t_prune(level, out), as one call (Sec. 4.2.1, Eq. 1-2, Eq. 4,
 * Alg. 1, Sec. 4.2.2: the same operations, the same results bit for bit).  For batches of at most
 * C2T_FUSED_MAX_BATCH sequences (the paper's own operating point is one sequence) it is ONE kernel launch:
 * the thread block that finishes the vocabulary pass last does the per-sequence work, which halves the
 * launch-to-launch latency that bounds such a step.  Larger batches, and contexts with entropy_top_m > 0,
 * get the two (or three) launches of the separate calls.  Arguments, alignment rules and errors as for
 * c2t_expand_level; `out` as for c2t_prune (may be NULL).
 */
int c2t_expand_prune_level(c2t_ctx *ctx, int level, const void *logits_dev, int64_t seq_stride,
                           int64_t row_stride, const c2t_frontier *out, void *stream);

/* Verification inputs, written by c2t_build_verify.  Caller-owned device arrays, NULL = skip.
 * Nw = c2t_final_width, W = c2t_mask_words, D = cfg.max_depth. */
typedef struct {
  int32_t  *n_nodes;       /* [B]          nodes in the final tree, root included          */
  int32_t  *tokens;        /* [B, Nw]      token per node; 0 past n_nodes                  */
  int32_t  *parents;       /* [B, Nw]      parent node id; -1 for the root and past n_nodes */
  int32_t  *position_ids;  /* [B, Nw]      prefix_len + tree level; 0 past n_nodes         */
  uint64_t *mask_bits;     /* [B, Nw, W]   bit j of row i set iff j is i or an ancestor of i;
                                            every node also attends the whole prefix      */
  int32_t  *retrieve;      /* [B, Nw, D+1] row r: node ids root -> r-th leaf (leaves in
                                            ascending id order), -1 padded                 */
  int32_t  *n_leaves;      /* [B]                                                          */
} c2t_verify;

/* Tree-attention inputs of the final tree (Sec. 2.2).  Must follow c2t_prune(C2T_FINAL). */
int c2t_build_verify(c2t_ctx *ctx, const c2t_verify *out, void *stream);

/*
 * The tree-attention mask (Sec. 2.2) written out as an additive matrix, for attention kernels
 * that cannot take the bit masks of c2t_build_verify:
 *   out_dev[b, i, c], i < Nw (c2t_final_width), c < kv_len, of out_dtype (C2T_F32 or C2T_BF16),
 *   element offset (b*Nw + i)*kv_len + c, caller-owned: 0 where final node i of sequence b
 *   attends key c, -inf elsewhere.
 * Keys [0, prefix_len[b]) are the sequence's own prefix, which every row attends; key
 * prefix_len[b] + j is tree node j, attended iff j is i or an ancestor of i.  Rows i >= n_nodes(b)
 * attend the prefix only.  Keys at or past kv_len do not exist: the caller chooses
 * kv_len >= max_b prefix_len[b] + n_nodes(b), or gets a clipped matrix.  prefix_len is the array
 * given to c2t_begin_step.  Must follow c2t_prune(C2T_FINAL); C2T_EINVAL for kv_len < 1 or an
 * unknown out_dtype.
 */
int c2t_dense_mask(c2t_ctx *ctx, void *out_dev, int32_t out_dtype, int64_t kv_len, void *stream);

/*
 * Vocabulary-parallel levels.  When the draft model's output layer is sharded over the vocabulary,
 * each GPU holds the logits of a contiguous token range [vocab_begin, vocab_begin + vocab_count) of
 * every frontier row.  A level is then built in three calls instead of two:
 *
 *   c2t_expand_level_shard   the vocabulary pass of c2t_expand_level over this range only;
 *   c2t_export_row_records   one c2t_row_record per active row: the range's maximum, its softmax and
 *                            entropy sums relative to that maximum, its K largest logits with GLOBAL
 *                            token ids (the quantities of Sec. 4.2.1, Eq. 2 and Sec. 4.2.2 restricted
 *                            to the range);
 *   (the caller all-gathers the records of all ranges: [n_shards, B, F] records, shard-major, in
 *    ascending order of vocab_begin; 288 bytes per row and shard)
 *   c2t_prune_gathered       c2t_prune(level) with the rows' sums and candidates merged from the
 *                            gathered records instead of from this context's own pass: the maxima are
 *                            aligned (sums rescaled by e^(M_shard - M)), a shard's own maximum rejoins
 *                            the sums unless it is the row's, and the K best of the shards' lists are
 *                            taken under the usual order (logit descending, token id ascending).
 *
 * The results are those of c2t_expand_level + c2t_prune on the full rows up to fp64 rounding of the
 * merge.  A range whose elements are all -inf contributes nothing; NaN and +inf set the status bits of
 * the sequence as usual.  Ranges must be disjoint, cover [0, V), and every vocab_begin must keep the
 * shard's rows 16-byte aligned.  The truncated entropy of Eq. 3 (entropy_top_m) is not available in
 * this mode (C2T_EINVAL).
 */
typedef struct {
  double  M;                     /* largest logit of the range (its best key's value)              */
  double  S;                     /* sum over the range's OTHER elements of e^(x - M)                */
  double  T;                     /* sum over the range's other elements of e^(x - M) (x - M)        */
  int32_t n;                     /* entries of tok / x that are valid (at most K)                   */
  uint32_t fault;                /* C2T_ST_* bits of this range of this row                         */
  int32_t tok[C2T_MAX_TOPK];     /* global token ids of the range's largest logits, best first      */
  float   x[C2T_MAX_TOPK];       /* those logits                                                    */
} c2t_row_record;

/*
 * The vocabulary pass of level `level` over one token range (Sec. 4.2.1, Eq. 2, Sec. 4.2.2).
 * logits_dev: [B, F, vocab_count] of cfg.dtype with the strides and alignment rules of
 * c2t_expand_level (row_stride >= vocab_count); 1 <= vocab_count <= V.  Same call order as
 * c2t_expand_level; must be followed by c2t_export_row_records before anything else.
 */
int c2t_expand_level_shard(c2t_ctx *ctx, int level, const void *logits_dev, int64_t seq_stride,
                           int64_t row_stride, int32_t vocab_count, void *stream);

/*
 * Writes the record of every active row (b, j) of the pass just run to records_dev[b * F + j]
 * (device memory of the caller, B * F records; rows j >= the sequence's frontier size are not
 * written).  vocab_begin is added to the token ids; vocab_begin + vocab_count <= V.
 */
int c2t_export_row_records(c2t_ctx *ctx, int level, int32_t vocab_begin, c2t_row_record *records_dev,
                           void *stream);

/*
 * c2t_prune(level) from gathered records (Eq. 1, Eq. 4, Alg. 1's two prunings): records_dev is
 * [n_shards, B, F], shard s of row (b, j) at (s * B + b) * F + j; 1 <= n_shards <= C2T_MAX_SHARDS.
 * `level` must be the level whose records were exported; the next call is c2t_expand_level(_shard)
 * of level + 1 or c2t_prune(C2T_FINAL).  Every rank that calls it with the same records builds the
 * same tree.
 */
int c2t_prune_gathered(c2t_ctx *ctx, int level, const c2t_row_record *records_dev, int32_t n_shards,
                       const c2t_frontier *out, void *stream);

typedef struct {
  int32_t *accept_len;   /* [B]      tau of this step: accepted draft tokens, root excluded */
  int32_t *path;         /* [B, D+1] accepted node ids, root first, -1 padded               */
  int32_t *next_token;   /* [B]      the target's greedy token after the last accepted node */
} c2t_accept_out;

/*
 * Greedy acceptance over the final tree (Sec. 5 Metrics: the accept length excludes the
 * target's own token).  target_logits_dev: [B, Nw, V] of cfg.dtype, row (b, i) = target
 * logits at final node i, element offset b*seq_stride + i*row_stride + v, aligned like the
 * draft logits; rows i >= n_nodes(b) are never read.  From the root, move to the child
 * carrying the target's argmax token (ties to the lower id) until none does.
 * Must follow c2t_prune(C2T_FINAL).
 */
int c2t_accept(c2t_ctx *ctx, const void *target_logits_dev, int64_t seq_stride,
               int64_t row_stride, const c2t_accept_out *out, void *stream);

/*
 * Greedy acceptance with the target logits sharded over the vocabulary (Sec. 5 Metrics; see
 * "Vocabulary-parallel levels" above).  c2t_argmax_shard reads this rank's token range
 * [vocab_begin, vocab_begin + vocab_count) of every final node's row ([B, Nw, vocab_count], strides and
 * alignment as in c2t_accept with row_stride >= vocab_count) and writes one 64-bit key per node to
 * keys_dev[b * Nw + i]: the range's largest logit in an order-preserving image in the high word,
 * 0xFFFFFFFF - (global token id) in the low word, 0 for i >= n_nodes(b).  The caller all-gathers the
 * keys of all ranges ([n_shards, B, Nw]); c2t_accept_gathered takes the largest key per node (equal
 * logits: the lower token id), then walks as c2t_accept does; outputs and node_argmax as there.
 * Both must follow c2t_prune(C2T_FINAL).
 */
int c2t_argmax_shard(c2t_ctx *ctx, const void *target_logits_dev, int64_t seq_stride, int64_t row_stride,
                     int32_t vocab_count, int32_t vocab_begin, uint64_t *keys_dev, void *stream);
int c2t_accept_gathered(c2t_ctx *ctx, const uint64_t *keys_dev, int32_t n_shards, const c2t_accept_out *out,
                        void *stream);

/*
 * The same greedy acceptance (Sec. 5 Metrics), reading only the target rows the walk visits:
 * the arg-max of the root's row, then of the accepted child's row, and so on, one row per
 * sequence and depth, accept_len + 1 rows per sequence instead of all n_nodes.  Arguments,
 * layout, outputs and error codes are those of c2t_accept; accept_len, path and next_token are
 * identical to c2t_accept's.  The node_argmax view (c2t_get_view) is filled for the nodes on the
 * accepted path only, -1 elsewhere.  Issues 2*(D+1)+1 short launches whatever the accept
 * lengths turn out to be (the host never waits for the device); rounds in which no sequence is
 * still walking read nothing.  Must follow c2t_prune(C2T_FINAL).
 */
int c2t_accept_lazy(c2t_ctx *ctx, const void *target_logits_dev, int64_t seq_stride,
                    int64_t row_stride, const c2t_accept_out *out, void *stream);

/*
 * c2t_accept_lazy for target logits that are sharded over the vocabulary (Sec. 5 Metrics; the rows read are
 * still only those on the accepted path).  Every rank drives the same loop:
 *
 *   c2t_lazy_begin(out)                                    puts every sequence on its root
 *   for round = 1 .. D + 1:
 *     c2t_lazy_argmax_shard(target shard, ..., keys)       this rank's best key of every walking sequence's
 *                                                          current row, token ids made global ([B] keys, 0 for
 *                                                          a sequence that has stopped)
 *     [all-gather of the B keys, 8 bytes per sequence]
 *     c2t_lazy_step_gathered(round, gathered keys [n_shards, B], n_shards, out)
 *                                                          largest key per sequence (equal logits: the lower
 *                                                          token id), then one step of every walk
 *
 * A path has at most D + 1 nodes, so D + 1 rounds always finish the walk; rounds after a sequence has
 * stopped read nothing of it.  `out` as for c2t_accept; results equal c2t_accept's.  Must follow
 * c2t_prune(C2T_FINAL).  keys_dev: caller-owned device buffers.
 */
int c2t_lazy_begin(c2t_ctx *ctx, const c2t_accept_out *out, void *stream);
int c2t_lazy_argmax_shard(c2t_ctx *ctx, const void *target_logits_dev, int64_t seq_stride, int64_t row_stride,
                          int32_t vocab_count, int32_t vocab_begin, uint64_t *keys_dev, void *stream);
int c2t_lazy_step_gathered(c2t_ctx *ctx, int round, const uint64_t *keys_dev, int32_t n_shards,
                           const c2t_accept_out *out, void *stream);

/*
 * The paper has no counterpart to this call; it exists for callers that cannot allocate.
 *
 * Some users of this library may not call cudaMalloc, and may not ask an allocator for a
 * workspace either: an inference server that sized all of its device memory at start-up, a
 * plug-in that runs inside someone else's engine, a latency-critical loop in which an
 * allocation (which can synchronise the whole device) is forbidden.  For them this entry
 * point computes the greedy token of every row of a logits matrix - the arg-max pass that
 * c2t_accept runs over the target logits, ties to the lower token id, NaN ignored - without a
 * context and without a workspace: the scratch memory it needs between its kernels is a fixed
 * array that lives inside the library's device code.
 *
 *   logits_dev   [rows, vocab] of `dtype` (c2t_dtype), element offset of (r, v) = r*row_stride + v;
 *                base 16-byte aligned, row_stride a multiple of 16 bytes
 *   argmax_dev   [rows] int32, caller-owned; -1 for a row that holds only NaN
 *
 * Limits and rules:
 *   - rows <= C2T_STATIC_MAX_ROWS and vocab <= C2T_STATIC_MAX_VOCAB; larger sizes are refused
 *     with C2T_ERANGE.  The array takes about 2.1 MB on every GPU that loads the library,
 *     until the process ends;
 *   - the first call on a device looks the array's device address up (cudaGetSymbolAddress,
 *     with that device current) and reads the SM count; make that first call once at start-up,
 *     before any stream capture begins;
 *   - the call only enqueues kernels on `stream`; it never calls cudaMalloc, cudaFree or any
 *     allocating routine.  Work is done on the device that is current when it is called;
 *   - all calls on a device share the one array and it keeps the last call's contents (the
 *     call clears what it is about to use): two calls whose kernels can overlap on the GPU -
 *     different streams, or different host threads without ordering - race on it.  Issue them
 *     on one stream, or order them with events.
 */
#define C2T_STATIC_MAX_ROWS  4096
#define C2T_STATIC_MAX_VOCAB 262144
int c2t_row_argmax_static(const void *logits_dev, int32_t rows, int32_t vocab, int32_t dtype,
                          int64_t row_stride, int32_t *argmax_dev, void *stream);

/* Waits for `stream`, then ORs all sequences' status words into *bits_host and, if
 * per_seq_host is not NULL, copies the B words there.  For tests and debugging. */
int c2t_status(c2t_ctx *ctx, uint32_t *bits_host, uint32_t *per_seq_host, void *stream);

/*
 * Read-only device views into the workspace, for inspection and tests.  Tree arrays are
 * [B, c2t_tree_capacity]; candidate arrays are [B, F*K] and hold the level pruned last
 * (candidate index = parent slot * K + rank); final arrays are [B, Nw].
 */
typedef struct {
  const int32_t *tree_n;        /* [B]                                                      */
  const int32_t *tree_token, *tree_parent, *tree_level;
  const double  *tree_logP;     /* log joint probability                                   */
  const double  *tree_C;        /* confidence                                              */
  const double  *tree_Chat;     /* min confidence on the root path (root: +inf)            */
  const int32_t *cand_n;        /* [B] candidates at the last level                        */
  const int32_t *cand_token;
  const double  *cand_lp;       /* log generation probability                              */
  const double  *cand_logP, *cand_H, *cand_C;
  const int32_t *cand_flags;    /* bit 0: C >= beta; bit 1: next-layer generator           */
  const int32_t *frontier_n;    /* [B] generators entering the next expand                 */
  const int32_t *frontier_node; /* [B, F]                                                  */
  const int32_t *final_n;       /* [B]                                                     */
  const int32_t *final_src;     /* [B, Nw] tree id each final node came from               */
  const int32_t *final_token, *final_parent, *final_level;
  const int32_t *node_argmax;   /* [B, Nw] target argmax per final node (after c2t_accept) */
  const int32_t *topm_from_pass;/* [B, F] with 0 < entropy_top_m < V, else NULL: 1 where the last
                                   c2t_expand_level took the row's Eq. 3 sums from the vectors the
                                   pass set aside, 0 where the row was read a second time   */
} c2t_view;
int c2t_get_view(c2t_ctx *ctx, c2t_view *out);

/* Host-side description of a whole decode step fed from host memory. */
typedef struct {
  const void *const *draft_logits_host; /* [D] pointers, each [B, F, V] contiguous, pinned  */
  const void *target_logits_host;       /* [B, Nw, V] contiguous, pinned                    */
  const int32_t *root_tok_host;         /* [B]                                              */
  const int32_t *prefix_len_host;       /* [B]                                              */
  void *draft_stage_dev;                /* device staging, B*F*V elements                   */
  void *target_stage_dev;               /* device staging, B*Nw*V elements                  */
  int32_t *int_stage_dev;               /* device staging, c2t_host_step_ints(cfg) int32    */
  /* results, host */
  int32_t *n_nodes_host;                /* [B]                                              */
  int32_t *tokens_host;                 /* [B, Nw]                                          */
  int32_t *accept_len_host;             /* [B]                                              */
  int32_t *path_host;                   /* [B, D+1]                                         */
  int32_t *next_token_host;             /* [B]                                              */
} c2t_host_step;
size_t c2t_host_step_ints(const c2t_config *cfg);

/*
 * One whole decode step (all the calls listed at the top) with inputs and results in HOST
 * memory: copies each level's draft logits and the target logits to the caller's device
 * staging buffers on `stream`, runs the step, copies the results back and waits for
 * `stream`.  Level 0 copies only slot 0 of each sequence (the root's row).  Exists so that
 * an end-to-end figure including the transfers can be measured through the library.
 */
int c2t_decode_step_host(c2t_ctx *ctx, const c2t_host_step *io, void *stream);

/* Number of kernels the context has launched since c2t_init (host-side counter). */
int64_t c2t_launch_count(const c2t_ctx *ctx);

const char *c2t_strerror(int code);

#ifdef __cplusplus
}
#endif
#endif /* C2T_H */

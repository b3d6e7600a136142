/*
 * CPU oracle for the C2T draft-tree hot path (arXiv 2502.13652).
 *
 * TEST INFRASTRUCTURE ONLY.  Plain C99, double precision, single thread, one
 * row / one sequence at a time, two passes over the vocabulary plus a full sort
 * per row.  It shares no code with the CUDA library and is never on the
 * product path: only the tests, the smoke check and the benchmark's CPU
 * baseline call it.
 *
 * What follows the paper, and where:
 *   - generation probability p = softmax of the draft logits          (Sec. 4.2.1)
 *   - joint probability  P_i = prod_{j in Path(root,i)} p_j           (Eq. 1)
 *   - entropy  H_i = - sum_{j in S(i)} p_j log p_j, optionally over the
 *     top-M probabilities without renormalising                        (Eq. 2-3)
 *   - depth d_i = loop counter at creation, 0 for the root's children  (Alg. 1)
 *   - confidence C_i = F(P_i, H_i, d_i), two-layer FFN, ReLU, sigmoid  (Sec. 4.1, Eq. 4)
 *   - first pruning: drop C_i < beta; stop when nothing survives       (Alg. 1, Sec. 4.2.1)
 *   - second pruning: classify only the Top-K children of a node, and
 *     let at most Top-K (here F) survivors generate the next layer     (Sec. 4.2.2)
 *   - EAGLE-2 style Top-N rerank of the whole tree                     (Sec. 2.2)
 *   - tree attention inputs and the accept length tau                  (Sec. 2.2, Sec. 5 Metrics)
 *
 * Readings taken where the paper is silent (listed in the design notes):
 * natural log; entropy of the parent's output row is shared by its K children;
 * ties in top-K / argmax go to the lower token id; ties in the cap go to the
 * earlier candidate; ties in the budget go to the lower node id; keep iff
 * C >= beta; budget ranks by the minimum confidence along the root path.
 *
 * Parity pins (tests, CPU only): brute-force sort for top-K, closed forms for
 * softmax and entropy, products along parent pointers for Eq. 1, an
 * independently enumerated V=8 depth-3 tree, the EAGLE-2 reduction, brute-force
 * masks / retrieve rows / accept length.  Nothing here is "parity unpinned".
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define ORC_F32 0
#define ORC_BF16 1

#define ORC_CLS_MLP 0
#define ORC_CLS_IDENTITY_JOINT 1
#define ORC_CLS_IDENTITY_COND 2   /* confidence := the child's own probability ("DyMax" stop rule, chain-mode comparison of Sec. 5) */

#define ORC_ADD_FRONTIER 0
#define ORC_ADD_ALL_SURVIVORS 1

/* row faults */
#define ORC_ROW_OK 0
#define ORC_ROW_NAN 1
#define ORC_ROW_POSINF 2
#define ORC_ROW_ALL_NEGINF 4

static double widen(const void *base, int dtype, int64_t i)
{
    if (dtype == ORC_BF16) {
        uint32_t bits = (uint32_t)((const uint16_t *)base)[i] << 16;
        float f;
        memcpy(&f, &bits, sizeof f);
        return (double)f;
    }
    return (double)((const float *)base)[i];
}

/* ---- one logits row: softmax, entropy, top-K --------------------------- */

typedef struct { double x; int32_t id; } orc_pair;

static int cmp_x_desc_id_asc(const void *pa, const void *pb)
{
    const orc_pair *a = (const orc_pair *)pa, *b = (const orc_pair *)pb;
    if (a->x > b->x) return -1;
    if (a->x < b->x) return 1;
    return (a->id > b->id) - (a->id < b->id);
}

/*
 * Softmax (generation probabilities), entropy (Eq. 2; Eq. 3 when 0 < M < V) and
 * the K most probable tokens of one row.
 *   lp_v = x_v - m - ln sum_u exp(x_u - m),  p_v = exp(lp_v)
 *   H = - sum_{v in S_M} p_v * lp_v, terms with p_v = 0 contribute 0
 * Order: (x descending, token id ascending), by a full sort.
 * Outputs: *log_z = m + ln Z; *entropy; top_tok/top_x/top_lp [K] (if V < K the
 * tail is token -1, x = lp = -inf).  Returns a row-fault bit mask.
 */
int orc_row_stats(const void *row, int dtype, int32_t V, int32_t K, int32_t M,
                  double *log_z, double *entropy,
                  int32_t *top_tok, double *top_x, double *top_lp)
{
    orc_pair *all = (orc_pair *)malloc((size_t)V * sizeof(orc_pair));
    int fault = ORC_ROW_OK;
    double m = -INFINITY;
    for (int32_t v = 0; v < V; ++v) {
        double x = widen(row, dtype, v);
        all[v].x = x;
        all[v].id = v;
        if (isnan(x)) fault |= ORC_ROW_NAN;
        else if (x == INFINITY) fault |= ORC_ROW_POSINF;
        if (x > m) m = x;
    }
    if (!fault && m == -INFINITY) fault |= ORC_ROW_ALL_NEGINF;
    if (fault) {
        *log_z = NAN; *entropy = NAN;
        for (int32_t r = 0; r < K; ++r) { top_tok[r] = -1; top_x[r] = NAN; top_lp[r] = NAN; }
        free(all);
        return fault;
    }
    double Z = 0.0;
    for (int32_t v = 0; v < V; ++v) Z += exp(all[v].x - m);
    double lnZ = log(Z);
    *log_z = m + lnZ;

    qsort(all, (size_t)V, sizeof(orc_pair), cmp_x_desc_id_asc);

    int32_t n_ent = (M > 0 && M < V) ? M : V;
    double H = 0.0;
    for (int32_t r = 0; r < n_ent; ++r) {
        double lp = all[r].x - m - lnZ;
        double p = exp(lp);
        if (p > 0.0) H -= p * lp;
    }
    *entropy = H;
    for (int32_t r = 0; r < K; ++r) {
        if (r < V) {
            top_tok[r] = all[r].id;
            top_x[r] = all[r].x;
            top_lp[r] = all[r].x - m - lnZ;
        } else {
            top_tok[r] = -1; top_x[r] = -INFINITY; top_lp[r] = -INFINITY;
        }
    }
    free(all);
    return ORC_ROW_OK;
}

/* Full softmax of one row into p[V] (used by the pins). */
int orc_row_softmax(const void *row, int dtype, int32_t V, double *p)
{
    double m = -INFINITY;
    for (int32_t v = 0; v < V; ++v) { double x = widen(row, dtype, v); if (x > m) m = x; }
    double Z = 0.0;
    for (int32_t v = 0; v < V; ++v) Z += exp(widen(row, dtype, v) - m);
    double lnZ = log(Z);
    for (int32_t v = 0; v < V; ++v) p[v] = exp(widen(row, dtype, v) - m - lnZ);
    return 0;
}

/* ---- the classifier (Sec. 4.1, Eq. 4) ----------------------------------- */

/* C = sigmoid(b2 + sum_k W2[k] * relu(b1[k] + W1[k][0]*P + W1[k][1]*H + W1[k][2]*d)) */
double orc_classifier(double P, double H, double d, int32_t hidden,
                      const float *w1, const float *b1, const float *w2, const float *b2)
{
    double z = (double)b2[0];
    for (int32_t k = 0; k < hidden; ++k) {
        double a = (double)b1[k] + (double)w1[3 * k + 0] * P + (double)w1[3 * k + 1] * H
                 + (double)w1[3 * k + 2] * d;
        if (a < 0.0) a = 0.0;
        z += (double)w2[k] * a;
    }
    return 1.0 / (1.0 + exp(-z));
}

/* ---- Algorithm 1 for one sequence --------------------------------------- */

typedef struct {
    int32_t vocab, dtype;
    int32_t max_depth;      /* D = d_max draft rounds               */
    int32_t topk;           /* K children classified per node       */
    int32_t frontier_cap;   /* F generators kept per level          */
    int32_t budget;         /* N, counts the root; 0 = none         */
    double  threshold;      /* beta                                 */
    int32_t entropy_top_m;  /* M; 0 = exact                         */
    int32_t classifier;     /* ORC_CLS_*                            */
    int32_t hidden;
    const float *w1, *b1, *w2, *b2;
    int32_t tree_add;       /* ORC_ADD_*                            */
} orc_config;

/* per-level candidate records, [D][F*K]; per-level frontier, [D+1][F] */
typedef struct {
    int32_t *n_cand;        /* [D]        candidates at the level (n_frontier*K)          */
    int32_t *tok;           /* [D][F*K]                                                      */
    int32_t *parent_node;   /* [D][F*K]   tree id of the generating node                     */
    double  *lp;            /* [D][F*K]   log generation probability                         */
    double  *logP;          /* [D][F*K]   log joint probability                              */
    double  *H;             /* [D][F*K]                                                      */
    double  *C;             /* [D][F*K]                                                      */
    int32_t *keep;          /* [D][F*K]   C >= beta                                          */
    int32_t *next;          /* [D][F*K]   member of the next frontier                        */
    int32_t *n_frontier;    /* [D+1]      n_frontier[l] = generators entering level l        */
    int32_t *frontier_node; /* [D+1][F]   tree ids                                           */
    int32_t *row_fault;     /* [D][F]                                                        */
} orc_levels;

typedef struct {
    int32_t capacity;
    int32_t n;
    int32_t *tok, *parent, *level;
    double  *logP, *C, *Chat;   /* Chat = min of C along the root path (root: +inf) */
} orc_tree;

static int cmp_cand_c_desc_idx_asc(const void *pa, const void *pb)
{
    const orc_pair *a = (const orc_pair *)pa, *b = (const orc_pair *)pb;
    if (a->x > b->x) return -1;
    if (a->x < b->x) return 1;
    return (a->id > b->id) - (a->id < b->id);
}

/*
 * logits: rows for this sequence, level l slot j at logits + (l*level_stride + j*row_stride)
 * elements.  Returns 0, or -1 if the tree capacity was exceeded.
 */
int orc_build_tree(const orc_config *cfg, const void *logits, int64_t level_stride,
                   int64_t row_stride, int32_t root_tok, orc_tree *T, orc_levels *L)
{
    const int32_t K = cfg->topk, F = cfg->frontier_cap, D = cfg->max_depth, V = cfg->vocab;
    const int32_t FK = F * K;
    const size_t esz = cfg->dtype == ORC_BF16 ? 2 : 4;
    int overflow = 0;

    /* root initialisation (Alg. 1): the tree and the generator set hold the root alone, with confidence 1 */
    T->n = 1;
    T->tok[0] = root_tok; T->parent[0] = -1; T->level[0] = 0;
    T->logP[0] = 0.0; T->C[0] = 1.0; T->Chat[0] = INFINITY;
    for (int32_t l = 0; l <= D; ++l) L->n_frontier[l] = 0;
    L->n_frontier[0] = 1;
    L->frontier_node[0] = 0;

    int32_t *top_tok = (int32_t *)malloc((size_t)K * sizeof(int32_t));
    double *top_x = (double *)malloc((size_t)K * sizeof(double));
    double *top_lp = (double *)malloc((size_t)K * sizeof(double));
    orc_pair *order = (orc_pair *)malloc((size_t)FK * sizeof(orc_pair));

    for (int32_t d = 0; d < D; ++d) {
        const int32_t nf = L->n_frontier[d];
        L->n_cand[d] = 0;
        if (nf == 0) continue;                       /* no C_i passed beta: the loop has ended */
        int32_t *ctok = L->tok + (size_t)d * FK, *cpar = L->parent_node + (size_t)d * FK;
        double *clp = L->lp + (size_t)d * FK, *clogP = L->logP + (size_t)d * FK;
        double *cH = L->H + (size_t)d * FK, *cC = L->C + (size_t)d * FK;
        int32_t *ckeep = L->keep + (size_t)d * FK, *cnext = L->next + (size_t)d * FK;

        /* children by generation probability (Sec. 4.2.2): the K most probable tokens of every generator's row */
        int32_t nc = 0;
        for (int32_t j = 0; j < nf; ++j) {
            const int32_t f = L->frontier_node[(size_t)d * F + j];
            const char *row = (const char *)logits + ((size_t)d * level_stride + (size_t)j * row_stride) * esz;
            double logZ, H;
            int fault = orc_row_stats(row, cfg->dtype, V, K, cfg->entropy_top_m, &logZ, &H,
                                      top_tok, top_x, top_lp);
            L->row_fault[(size_t)d * F + j] = fault;
            for (int32_t r = 0; r < K; ++r, ++nc) {
                ctok[nc] = top_tok[r];
                cpar[nc] = f;
                clp[nc] = top_lp[r];
                clogP[nc] = T->logP[f] + top_lp[r];      /* Eq. 1 in log space */
                cH[nc] = H;                              /* entropy of the row the child sits in */
            }
        }
        L->n_cand[d] = nc;

        /* confidence of every child (Eq. 4) and first pruning (Sec. 4.2.1): a child stays iff its confidence reaches beta */
        int32_t n_surv = 0;
        for (int32_t c = 0; c < nc; ++c) {
            double P = exp(clogP[c]);
            double C;
            if (ctok[c] < 0 || isnan(clogP[c])) C = NAN;
            else if (cfg->classifier == ORC_CLS_IDENTITY_JOINT) C = P;
            else if (cfg->classifier == ORC_CLS_IDENTITY_COND) C = exp(clp[c]);
            else C = orc_classifier(P, cH[c], (double)d, cfg->hidden, cfg->w1, cfg->b1, cfg->w2, cfg->b2);
            cC[c] = C;
            ckeep[c] = (C >= cfg->threshold) ? 1 : 0;    /* NaN compares false */
            cnext[c] = 0;
            if (ckeep[c]) { order[n_surv].x = C; order[n_surv].id = c; ++n_surv; }
        }

        /* second pruning: the F survivors that come first under (C desc, candidate index asc) */
        qsort(order, (size_t)n_surv, sizeof(orc_pair), cmp_cand_c_desc_idx_asc);
        int32_t n_next = n_surv < F ? n_surv : F;
        for (int32_t s = 0; s < n_next; ++s) cnext[order[s].id] = 1;

        /* tree append (Alg. 1), in candidate order: the capped set, or every survivor (the variant of App. B.6) */
        int32_t slot = 0;
        for (int32_t c = 0; c < nc; ++c) {
            int add = cfg->tree_add == ORC_ADD_ALL_SURVIVORS ? ckeep[c] : cnext[c];
            if (!add) continue;
            if (T->n >= T->capacity) { overflow = 1; continue; }
            int32_t id = T->n++;
            int32_t f = cpar[c];
            T->tok[id] = ctok[c]; T->parent[id] = f; T->level[id] = d + 1;
            T->logP[id] = clogP[c]; T->C[id] = cC[c];
            T->Chat[id] = cC[c] < T->Chat[f] ? cC[c] : T->Chat[f];
            if (cnext[c] && d + 1 <= D) L->frontier_node[(size_t)(d + 1) * F + slot++] = id;
        }
        L->n_frontier[d + 1] = slot;
    }
    free(top_tok); free(top_x); free(top_lp); free(order);
    return overflow ? -1 : 0;
}

/* ---- Top-N rerank of the finished tree (Sec. 2.2, EAGLE-2's N) ----------- */

/*
 * Keep the root and the N-1 other nodes that come first under (Chat desc, id asc);
 * renumber in id order.  Chat never exceeds the parent's, and a parent has the
 * lower id, so the kept set is closed under "parent of".
 * Outputs: src[new] = old id; tok/parent/level of the kept tree.  Returns n_final.
 */
int32_t orc_final_prune(const orc_tree *T, int32_t N, int32_t *src, int32_t *tok,
                        int32_t *parent, int32_t *level)
{
    const int32_t n = T->n;
    int32_t *keep = (int32_t *)calloc((size_t)n, sizeof(int32_t));
    if (N <= 0 || n <= N) {
        for (int32_t i = 0; i < n; ++i) keep[i] = 1;
    } else {
        orc_pair *order = (orc_pair *)malloc((size_t)n * sizeof(orc_pair));
        for (int32_t i = 1; i < n; ++i) { order[i - 1].x = T->Chat[i]; order[i - 1].id = i; }
        qsort(order, (size_t)(n - 1), sizeof(orc_pair), cmp_cand_c_desc_idx_asc);
        keep[0] = 1;
        for (int32_t s = 0; s < N - 1; ++s) keep[order[s].id] = 1;
        free(order);
    }
    int32_t *remap = (int32_t *)malloc((size_t)n * sizeof(int32_t));
    int32_t m = 0;
    for (int32_t i = 0; i < n; ++i) {
        remap[i] = -1;
        if (!keep[i]) continue;
        remap[i] = m;
        src[m] = i;
        tok[m] = T->tok[i];
        parent[m] = T->parent[i] < 0 ? -1 : remap[T->parent[i]];
        level[m] = T->level[i];
        ++m;
    }
    free(keep); free(remap);
    return m;
}

/* ---- verification inputs (tree attention, Sec. 2.2) ---------------------- */

/*
 * mask row i: bit j set iff j is i or an ancestor of i  (W 64-bit words per row)
 * position_ids[i] = prefix_len + level[i]
 * retrieve row r : node ids root -> r-th leaf (leaves ascending), -1 padded to width
 * Rows past n / n_leaves are 0 / -1.  Returns n_leaves.
 */
int32_t orc_build_verify(int32_t n, const int32_t *parent, const int32_t *level,
                         int32_t prefix_len, int32_t N_rows, int32_t W, int32_t width,
                         uint64_t *mask, int32_t *position_ids, int32_t *retrieve)
{
    memset(mask, 0, (size_t)N_rows * W * sizeof(uint64_t));
    for (int32_t i = 0; i < N_rows; ++i) position_ids[i] = 0;
    for (int32_t i = 0; i < N_rows * width; ++i) retrieve[i] = -1;
    int32_t *has_child = (int32_t *)calloc((size_t)(n > 0 ? n : 1), sizeof(int32_t));
    for (int32_t i = 0; i < n; ++i) {
        for (int32_t a = i; a >= 0; a = parent[a]) mask[(size_t)i * W + a / 64] |= (uint64_t)1 << (a % 64);
        position_ids[i] = prefix_len + level[i];
        if (parent[i] >= 0) has_child[parent[i]] = 1;
    }
    int32_t n_leaves = 0;
    for (int32_t i = 0; i < n; ++i) {
        if (has_child[i]) continue;
        for (int32_t a = i; a >= 0; a = parent[a]) retrieve[(size_t)n_leaves * width + level[a]] = a;
        ++n_leaves;
    }
    free(has_child);
    return n_leaves;
}

/* ---- greedy acceptance (Sec. 5 Metrics: tau excludes the target's own token) */

/* argmax of one row, ties to the lower token id */
int32_t orc_row_argmax(const void *row, int dtype, int32_t V)
{
    int32_t best = -1;
    double bx = 0.0;
    for (int32_t v = 0; v < V; ++v) {
        double x = widen(row, dtype, v);
        if (isnan(x)) continue;
        if (best < 0 || x > bx) { best = v; bx = x; }
    }
    return best;
}

/*
 * Walk from the root: at node cur the target's greedy token is argmax(target row cur);
 * move to the child of cur carrying that token, else stop.
 * path[0..accept_len] = node ids (root first), -1 padded to `width`;
 * next_token = the target's greedy token at the last accepted node.
 */
int32_t orc_accept(int32_t n, const int32_t *tok, const int32_t *parent,
                   const void *target, int dtype, int32_t V, int64_t row_stride,
                   int32_t width, int32_t *path, int32_t *next_token, int32_t *node_argmax)
{
    const size_t esz = dtype == ORC_BF16 ? 2 : 4;
    for (int32_t i = 0; i < n; ++i)
        node_argmax[i] = orc_row_argmax((const char *)target + (size_t)i * row_stride * esz, dtype, V);
    for (int32_t i = 0; i < width; ++i) path[i] = -1;
    int32_t cur = 0, len = 0;
    path[0] = 0;
    for (;;) {
        int32_t want = node_argmax[cur], nxt = -1;
        for (int32_t c = cur + 1; c < n; ++c)
            if (parent[c] == cur && tok[c] == want) { nxt = c; break; }
        if (nxt < 0 || len + 1 >= width) break;
        cur = nxt;
        path[++len] = cur;
    }
    *next_token = node_argmax[cur];
    return len;
}

/* ---- a whole decode step over a batch (what the CPU baseline times) ------- */

/*
 * For b in [0,B): Algorithm 1, Top-N rerank, verification inputs, accept walk.
 * draft:  element offset of (b, level l, slot j) = b*seq_stride + l*level_stride + j*row_stride
 * target: element offset of (b, node i)          = b*tgt_seq_stride + i*tgt_row_stride
 * Outputs are [B, Nw] / [B, Nw, W] / [B, Nw, D+1] / [B, D+1] like the library's.
 * Returns the number of logits rows visited (draft + target).
 */
int64_t orc_decode_step(const orc_config *cfg, int32_t B, int32_t Nw, int32_t tree_capacity,
                        const void *draft, int64_t seq_stride, int64_t level_stride, int64_t row_stride,
                        const void *target, int64_t tgt_seq_stride, int64_t tgt_row_stride,
                        const int32_t *root_tok, const int32_t *prefix_len,
                        int32_t *n_final, int32_t *tokens, int32_t *parents, int32_t *position_ids,
                        uint64_t *mask, int32_t *retrieve, int32_t *n_leaves,
                        int32_t *accept_len, int32_t *path, int32_t *next_token)
{
    const int32_t K = cfg->topk, F = cfg->frontier_cap, D = cfg->max_depth;
    const int32_t FK = F * K, W = (Nw + 63) / 64, width = D + 1;
    const size_t esz = cfg->dtype == ORC_BF16 ? 2 : 4;
    int64_t rows = 0;

    orc_tree T;
    T.capacity = tree_capacity;
    T.tok = (int32_t *)malloc((size_t)tree_capacity * sizeof(int32_t));
    T.parent = (int32_t *)malloc((size_t)tree_capacity * sizeof(int32_t));
    T.level = (int32_t *)malloc((size_t)tree_capacity * sizeof(int32_t));
    T.logP = (double *)malloc((size_t)tree_capacity * sizeof(double));
    T.C = (double *)malloc((size_t)tree_capacity * sizeof(double));
    T.Chat = (double *)malloc((size_t)tree_capacity * sizeof(double));
    orc_levels L;
    L.n_cand = (int32_t *)malloc((size_t)D * sizeof(int32_t));
    L.tok = (int32_t *)malloc((size_t)D * FK * sizeof(int32_t));
    L.parent_node = (int32_t *)malloc((size_t)D * FK * sizeof(int32_t));
    L.lp = (double *)malloc((size_t)D * FK * sizeof(double));
    L.logP = (double *)malloc((size_t)D * FK * sizeof(double));
    L.H = (double *)malloc((size_t)D * FK * sizeof(double));
    L.C = (double *)malloc((size_t)D * FK * sizeof(double));
    L.keep = (int32_t *)malloc((size_t)D * FK * sizeof(int32_t));
    L.next = (int32_t *)malloc((size_t)D * FK * sizeof(int32_t));
    L.n_frontier = (int32_t *)malloc((size_t)(D + 1) * sizeof(int32_t));
    L.frontier_node = (int32_t *)malloc((size_t)(D + 1) * F * sizeof(int32_t));
    L.row_fault = (int32_t *)calloc((size_t)D * F, sizeof(int32_t));
    int32_t *src = (int32_t *)malloc((size_t)tree_capacity * sizeof(int32_t));
    int32_t *ftok = (int32_t *)malloc((size_t)tree_capacity * sizeof(int32_t));
    int32_t *fpar = (int32_t *)malloc((size_t)tree_capacity * sizeof(int32_t));
    int32_t *flev = (int32_t *)malloc((size_t)tree_capacity * sizeof(int32_t));
    int32_t *amax = (int32_t *)malloc((size_t)tree_capacity * sizeof(int32_t));

    for (int32_t b = 0; b < B; ++b) {
        const char *dl = (const char *)draft + (size_t)b * seq_stride * esz;
        orc_build_tree(cfg, dl, level_stride, row_stride, root_tok[b], &T, &L);
        for (int32_t l = 0; l < D; ++l) rows += L.n_frontier[l];
        int32_t nf = orc_final_prune(&T, cfg->budget, src, ftok, fpar, flev);
        if (nf > Nw) nf = Nw;
        n_final[b] = nf;
        for (int32_t i = 0; i < Nw; ++i) {
            tokens[(size_t)b * Nw + i] = i < nf ? ftok[i] : 0;
            parents[(size_t)b * Nw + i] = i < nf ? fpar[i] : -1;
        }
        n_leaves[b] = orc_build_verify(nf, fpar, flev, prefix_len[b], Nw, W, width,
                                       mask + (size_t)b * Nw * W, position_ids + (size_t)b * Nw,
                                       retrieve + (size_t)b * Nw * width);
        const char *tl = (const char *)target + (size_t)b * tgt_seq_stride * esz;
        accept_len[b] = orc_accept(nf, ftok, fpar, tl, cfg->dtype, cfg->vocab, tgt_row_stride,
                                   width, path + (size_t)b * width, next_token + b, amax);
        rows += nf;
    }
    free(T.tok); free(T.parent); free(T.level); free(T.logP); free(T.C); free(T.Chat);
    free(L.n_cand); free(L.tok); free(L.parent_node); free(L.lp); free(L.logP); free(L.H);
    free(L.C); free(L.keep); free(L.next); free(L.n_frontier); free(L.frontier_node); free(L.row_fault);
    free(src); free(ftok); free(fpar); free(flev); free(amax);
    return rows;
}

"""Pins for the CPU oracle: closed forms, brute force, hand-enumerated trees.

None of these re-type the oracle's formulas: each compares against a value the
mathematics fixes, a library routine on a special case, or a differently
structured brute force, so that a dropped term, a wrong sign or index, or a
swapped operand in the oracle fails at least one of them.
"""
import itertools
import json
import math
import os

import numpy as np
import pytest
import scipy.special
import scipy.stats
import torch

import c2t_inputs

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def bf16_round(x: torch.Tensor) -> torch.Tensor:
    return x.to(torch.bfloat16)


# ---------------------------------------------------------------- top-K ------

def brute_topk(row: torch.Tensor, K: int):
    x = row.to(torch.float64).numpy()
    order = np.lexsort((np.arange(x.size), -x))          # by -x, then by id
    return order[:K]


@pytest.mark.parametrize("case", ["random_f32", "random_bf16", "all_equal", "two_valued", "bf16_heavy_ties"])
def test_topk_matches_brute_force_sort(oracle_mod, case):
    g = torch.Generator().manual_seed(11)
    V, K = 4099, 10
    if case == "random_f32":
        row = torch.randn(V, generator=g) * 5
    elif case == "random_bf16":
        row = bf16_round(torch.randn(V, generator=g) * 5)
    elif case == "all_equal":
        row = torch.full((V,), 1.25)
    elif case == "two_valued":
        row = torch.where(torch.rand(V, generator=g) < 0.01, torch.tensor(3.0), torch.tensor(-1.0))
    else:
        row = bf16_round(40 + torch.randn(V, generator=g) * 0.5)   # spacing 0.25 at this magnitude
    fault, _, _, tok, x, _ = oracle_mod.row_stats(row, K)
    assert fault == 0
    want = brute_topk(row, K)
    assert tok.tolist() == want.tolist()
    assert np.array_equal(x, row.to(torch.float64).numpy()[want])
    if case == "all_equal":
        assert tok.tolist() == list(range(K))           # ties go to the lower token id


def test_topk_k_larger_than_vocab(oracle_mod):
    row = torch.tensor([0.0, 2.0, 1.0])
    _, _, _, tok, x, lp = oracle_mod.row_stats(row, 5)
    assert tok.tolist() == [1, 2, 0, -1, -1]
    assert np.isneginf(lp[3:]).all()


# ---------------------------------------------------------------- softmax ----

def test_softmax_sums_to_one_and_matches_library(oracle_mod):
    g = torch.Generator().manual_seed(3)
    for dtype in (torch.float32, torch.bfloat16):
        row = (torch.randn(32000, generator=g) * 4).to(dtype)
        p = oracle_mod.row_softmax(row)
        assert abs(p.sum() - 1.0) < 1e-12
        ref = scipy.special.softmax(row.to(torch.float64).numpy())
        np.testing.assert_allclose(p, ref, rtol=1e-12, atol=0)


def test_softmax_shift_invariance(oracle_mod):
    g = torch.Generator().manual_seed(4)
    row = torch.randn(1000, generator=g)
    # shifts by powers of two keep the fp32 inputs exact
    a = oracle_mod.row_stats(row, 4)
    b = oracle_mod.row_stats(row * 1.0 + 0.0, 4)
    assert a[2] == b[2]
    row64 = row.to(torch.float32)
    shifted = (row64.to(torch.float64) + 8.0).to(torch.float32)
    if torch.equal(shifted.to(torch.float64), row64.to(torch.float64) + 8.0):
        c = oracle_mod.row_stats(shifted, 4)
        np.testing.assert_allclose(c[5], a[5], rtol=0, atol=1e-12)     # log-probs unchanged
        assert abs(c[1] - (a[1] + 8.0)) < 1e-12                        # logZ shifts by the constant
        assert abs(c[2] - a[2]) < 1e-12


def test_softmax_two_valued_closed_form(oracle_mod):
    V, a = 32000, 7.0
    row = torch.zeros(V)
    row[123] = a
    fault, logz, H, tok, x, lp = oracle_mod.row_stats(row, 3)
    p1 = math.exp(a) / (math.exp(a) + V - 1)
    q = 1.0 / (math.exp(a) + V - 1)
    assert tok.tolist() == [123, 0, 1]
    assert abs(math.exp(lp[0]) - p1) < 1e-12 * p1
    assert abs(math.exp(lp[1]) - q) < 1e-12 * q
    assert abs(logz - math.log(math.exp(a) + V - 1)) < 1e-12
    H_closed = -(p1 * math.log(p1) + (V - 1) * q * math.log(q))
    assert abs(H - H_closed) < 1e-11


# ---------------------------------------------------------------- entropy ----

@pytest.mark.parametrize("V", [8, 1000, 32000, 128256])
def test_entropy_of_uniform_logits_is_log_v(oracle_mod, V):
    for dtype in (torch.float32, torch.bfloat16):
        row = torch.full((V,), -2.5).to(dtype)
        _, logz, H, _, _, lp = oracle_mod.row_stats(row, 2)
        assert abs(H - math.log(V)) < 1e-10
        assert abs(lp[0] + math.log(V)) < 1e-10


def test_truncated_entropy_of_uniform_logits(oracle_mod):
    # Eq. 3 keeps the same p_j (no renormalisation): M of V equal terms
    V, M = 32000, 1000
    row = torch.zeros(V)
    _, _, H, _, _, _ = oracle_mod.row_stats(row, 2, M)
    assert abs(H - (M / V) * math.log(V)) < 1e-12
    _, _, H_full, _, _, _ = oracle_mod.row_stats(row, 2, V)
    assert abs(H_full - math.log(V)) < 1e-10


def test_truncated_entropy_picks_the_largest_probabilities(oracle_mod):
    g = torch.Generator().manual_seed(5)
    row = torch.randn(5000, generator=g) * 3
    M = 100
    _, _, H, _, _, _ = oracle_mod.row_stats(row, 2, M)
    p = scipy.special.softmax(row.to(torch.float64).numpy())
    top = np.sort(p)[::-1][:M]
    assert abs(H - float(-(top * np.log(top)).sum())) < 1e-12


def test_entropy_dyadic_row(oracle_mod):
    # p = 1/2, 1/4, ..., 1/128, 1/128  =>  H = (127/64) ln 2
    p = [2.0 ** -(t + 1) for t in range(7)] + [2.0 ** -7]
    row = torch.tensor([math.log(v) for v in p], dtype=torch.float64).to(torch.float32)
    _, _, H, _, _, _ = oracle_mod.row_stats(row, 2)
    assert abs(H - (127.0 / 64.0) * math.log(2.0)) < 1e-6    # fp32 storage of ln p
    assert abs((127.0 / 64.0) * math.log(2.0) - 1.375464) < 1e-6


def test_entropy_matches_library_and_bounds(oracle_mod):
    g = torch.Generator().manual_seed(6)
    for scale in (0.1, 1.0, 4.0, 8.0):
        row = torch.randn(32000, generator=g) * scale
        _, _, H, _, _, _ = oracle_mod.row_stats(row, 2)
        p = scipy.special.softmax(row.to(torch.float64).numpy())
        assert abs(H - scipy.stats.entropy(p)) < 1e-10
        assert 0.0 <= H <= math.log(32000) + 1e-12


def test_neg_inf_logits_have_zero_probability(oracle_mod):
    row = torch.tensor([0.0, float("-inf"), 0.0, float("-inf")])
    fault, _, H, tok, _, lp = oracle_mod.row_stats(row, 4)
    assert fault == 0
    assert abs(H - math.log(2)) < 1e-12
    assert tok.tolist() == [0, 2, 1, 3]
    assert np.isneginf(lp[2:]).all()


def test_row_faults(oracle_mod):
    assert oracle_mod.row_stats(torch.tensor([0.0, float("nan")]), 1)[0] == 1
    assert oracle_mod.row_stats(torch.tensor([0.0, float("inf")]), 1)[0] == 2
    assert oracle_mod.row_stats(torch.tensor([float("-inf")] * 3), 1)[0] == 4


# ---------------------------------------------------------------- classifier -

def test_classifier_zero_weights_give_one_half(oracle_mod):
    h = 16
    c = oracle_mod.classifier(0.3, 4.0, 5.0, np.zeros((h, 3)), np.zeros(h), np.zeros(h), np.zeros(1))
    assert c == 0.5


def test_classifier_single_unit_is_sigmoid_of_p(oracle_mod):
    for P in (0.0, 0.1, 0.9, 1.0):
        c = oracle_mod.classifier(P, 3.3, 7.0, np.array([[1.0, 0, 0]]), np.zeros(1), np.ones(1), np.zeros(1))
        assert abs(c - 1.0 / (1.0 + math.exp(-P))) < 1e-15


def test_classifier_feature_order_and_relu(oracle_mod):
    # one unit per feature, with signs that make ReLU clip exactly one of them
    w1 = np.array([[2.0, 0, 0], [0, -1.0, 0], [0, 0, 0.5]])
    b1 = np.array([0.0, 1.0, -1.0]); w2 = np.array([1.0, 10.0, 100.0]); b2 = np.array([-3.0])
    P, H, d = 0.25, 3.0, 4.0
    # unit0 = 0.5, unit1 = relu(1-3) = 0, unit2 = relu(2-1) = 1  ->  z = -3 + 0.5 + 0 + 100
    c = oracle_mod.classifier(P, H, d, w1, b1, w2, b2)
    assert abs(c - 1.0 / (1.0 + math.exp(-97.5))) < 1e-15
    # swapping H and d changes which unit clips: unit1 = relu(1-4)=0, unit2 = relu(1.5-1)=0.5
    c2 = oracle_mod.classifier(P, d, H, w1, b1, w2, b2)
    assert abs(c2 - 1.0 / (1.0 + math.exp(-(-3 + 0.5 + 50)))) < 1e-15


def test_classifier_against_long_double(oracle_mod):
    w1, b1, w2, b2 = [t.numpy() for t in c2t_inputs.classifier_weights(48, seed=9, std=1.0)]
    rng = np.random.default_rng(0)
    for _ in range(50):
        P, H, d = rng.random(), rng.random() * 10, float(rng.integers(0, 11))
        ld = np.longdouble
        a = b1.astype(ld) + w1.astype(ld) @ np.array([P, H, d], dtype=ld)
        z = b2.astype(ld)[0] + (w2.astype(ld) * np.maximum(a, 0)).sum()
        want = float(1 / (1 + np.exp(-z)))
        assert abs(oracle_mod.classifier(P, H, d, w1, b1, w2, b2) - want) < 1e-14


# ---------------------------------------------------------------- helpers ----

def make_cfg(oracle_mod, V, D, K, F, N, beta, classifier="mlp", hidden=16, dtype=torch.float32,
             tree_add="frontier", wseed=0, M=0, wstd=0.1):
    w1, b1, w2, b2 = c2t_inputs.classifier_weights(hidden, seed=wseed, std=wstd)
    return oracle_mod.OracleConfig(
        vocab=V, dtype=oracle_mod.BF16 if dtype == torch.bfloat16 else oracle_mod.F32,
        max_depth=D, topk=K, frontier_cap=F, budget=N, threshold=beta, entropy_top_m=M,
        classifier={"mlp": oracle_mod.CLS_MLP, "identity": oracle_mod.CLS_IDENTITY_JOINT,
                    "cond": oracle_mod.CLS_IDENTITY_COND}[classifier],
        hidden=hidden, w1=w1, b1=b1, w2=w2, b2=b2,
        tree_add=oracle_mod.ADD_FRONTIER if tree_add == "frontier" else oracle_mod.ADD_ALL_SURVIVORS)


def seq_logits(V, D, F, dtype=torch.float32, seq=0, step=0, scale=4.0):
    """[D, F, V] draft logits of one sequence."""
    return torch.stack([c2t_inputs.draft_logits(1, F, V, step, l, dtype, scale, seq_base=seq)[0]
                        for l in range(D)])


# ---------------------------------------------------------------- Eq. 1 ------

@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_joint_probability_is_product_along_root_path(oracle_mod, dtype):
    V, D, K, F = 2000, 5, 4, 4
    cfg = make_cfg(oracle_mod, V, D, K, F, 0, 0.0, classifier="identity")
    lg = seq_logits(V, D, F, dtype)
    cfg.dtype = oracle_mod.BF16 if dtype == torch.bfloat16 else oracle_mod.F32
    t, L = oracle_mod.build_tree(cfg, lg, 1)
    assert t.n == 1 + min(K, F) + (D - 1) * F
    # node -> (level, slot) of the row that generated it, from the frontier lists
    slot_of = {}
    for l in range(D + 1):
        for j in range(L.n_frontier[l]):
            slot_of[int(L.frontier_node[l, j])] = (l, j)
    for i in range(1, t.n):
        prod, a = 1.0, i
        while t.parent[a] >= 0:
            par = int(t.parent[a])
            l, j = slot_of[par]
            assert t.level[a] == l + 1
            p_row = scipy.special.softmax(lg[l, j].to(torch.float64).numpy())
            prod *= p_row[t.tok[a]]
            a = par
        assert abs(math.exp(t.logP[i]) - prod) <= 1e-12 * prod
        assert t.logP[i] <= t.logP[t.parent[i]] + 1e-15       # a child is never more probable


# ---------------------------------------------------------------- tiny tree --

def test_hand_enumerated_tiny_tree(oracle_mod):
    with open(os.path.join(GOLDEN, "tiny_tree_v8.json")) as f:
        G = json.load(f)
    V, D, K, F, N = 8, G["D"], G["K"], G["F"], G["N"]
    row = torch.tensor([math.log(p) for p in G["p"]], dtype=torch.float64).to(torch.float32)
    lg = row.expand(D, F, V).contiguous()
    cfg = make_cfg(oracle_mod, V, D, K, F, N, G["beta"], classifier="identity")
    t, L = oracle_mod.build_tree(cfg, lg, G["root_token"])
    assert t.n == len(G["tree_tokens"])
    assert t.tok[:t.n].tolist() == G["tree_tokens"]
    assert t.parent[:t.n].tolist() == G["tree_parents"]
    assert t.level[:t.n].tolist() == G["tree_levels"]
    np.testing.assert_allclose(np.exp(t.logP[:t.n]), G["tree_joint"], rtol=1e-6)
    for l in range(D):
        n = L.n_cand[l]
        assert n == len(G["level_candidates_joint"][l])
        np.testing.assert_allclose(np.exp(L.logP[l, :n]), G["level_candidates_joint"][l], rtol=1e-6)
        assert L.keep[l, :n].tolist() == G["level_keep"][l]
        assert L.next[l, :n].tolist() == G["level_next"][l]
    ft = oracle_mod.final_prune(t, N)
    assert ft.n == N
    assert ft.src[:N].tolist() == G["final_src"]
    assert ft.tok[:N].tolist() == G["final_tokens"]
    assert ft.parent[:N].tolist() == G["final_parents"]
    v = oracle_mod.build_verify(ft, G["prefix_len"], N, D + 1)
    assert v.mask[:, 0].tolist() == G["final_masks"]
    assert v.position_ids.tolist() == G["final_positions"]
    assert v.n_leaves == G["n_leaves"]
    assert v.retrieve[:v.n_leaves].tolist() == G["retrieve"]
    target = torch.zeros(N, V)
    for i, a in enumerate(G["target_argmax"]):
        target[i, a] = 5.0
    acc = oracle_mod.accept(ft, target, D + 1)
    assert acc.accept_len == G["accept_len"]
    assert acc.path.tolist() == G["accept_path"]
    assert acc.next_token == G["next_token"]


def test_tiny_tree_with_mlp_against_independent_enumeration(oracle_mod):
    """Same V=8 rows, a non-trivial MLP; expected tree enumerated here with plain Python floats."""
    p = [0.5, 0.3, 0.1, 0.05, 0.02, 0.015, 0.01, 0.005]
    V, D, K, F, N, beta = 8, 3, 3, 2, 0, 0.5
    H = -sum(q * math.log(q) for q in p)
    # weights exactly representable in fp32
    w1 = [[3.0, -0.25, -0.125], [-1.0, 0.25, 0.25]]; b1 = [0.5, 0.125]; w2 = [2.0, -1.5]; b2 = [0.125]

    def conf(P, d, H=H):
        z = b2[0]
        for k in range(2):
            z += w2[k] * max(0.0, b1[k] + w1[k][0] * P + w1[k][1] * H + w1[k][2] * d)
        return 1.0 / (1.0 + math.exp(-z))

    # independent enumeration: nodes are token tuples
    tree = [()]
    frontier = [()]
    for d in range(D):
        cands = [(path + (t,), conf(math.prod(p[s] for s in path + (t,)), d))
                 for path in frontier for t in range(K)]       # tokens 0..K-1 are the K most probable
        surv = [(i, c) for i, c in enumerate(cands) if c[1] >= beta]
        chosen = sorted(surv, key=lambda ic: (-ic[1][1], ic[0]))[:F]
        keep_idx = sorted(i for i, _ in chosen)
        frontier = [cands[i][0] for i in keep_idx]
        tree += frontier
        if not frontier:
            break
    row = torch.tensor([math.log(q) for q in p], dtype=torch.float64).to(torch.float32)
    lg = row.expand(D, F, V).contiguous()
    cfg = make_cfg(oracle_mod, V, D, K, F, N, beta, hidden=2)
    cfg.w1 = torch.tensor(w1); cfg.b1 = torch.tensor(b1); cfg.w2 = torch.tensor(w2); cfg.b2 = torch.tensor(b2)
    t, L = oracle_mod.build_tree(cfg, lg, 0)
    got = []
    for i in range(t.n):
        path, a = [], i
        while t.parent[a] >= 0:
            path.append(int(t.tok[a])); a = int(t.parent[a])
        got.append(tuple(reversed(path)))
    assert got == tree
    assert len(tree) > 3                                         # the case is not degenerate
    for l in range(D):
        for c in range(L.n_cand[l]):
            assert abs(L.H[l, c] - H) < 1e-6
            assert abs(L.C[l, c] - conf(math.exp(L.logP[l, c]), l, L.H[l, c])) < 1e-12


# ---------------------------------------------------------------- Alg. 1 edges

def test_zero_weights_exercise_threshold_equality_and_cap_ties(oracle_mod):
    V, D, K, F = 500, 4, 5, 3
    cfg = make_cfg(oracle_mod, V, D, K, F, 0, 0.5, wstd=0.0)
    lg = seq_logits(V, D, F)
    t, L = oracle_mod.build_tree(cfg, lg, 0)
    for l in range(D):
        n = L.n_cand[l]
        assert (L.C[l, :n] == 0.5).all() and L.keep[l, :n].all()      # C == beta is kept
        assert L.next[l, :n].tolist() == [1] * min(F, n) + [0] * (n - min(F, n))   # ties -> candidate order
    assert t.n == 1 + min(K, F) + (D - 1) * F
    cfg.threshold = 0.5000001
    t2, L2 = oracle_mod.build_tree(cfg, lg, 0)
    assert t2.n == 1 and L2.n_frontier[1] == 0 and L2.n_cand[1] == 0   # nothing passes: loop ends


def test_depth_feature_starts_at_zero(oracle_mod):
    # classifier that only looks at depth: C = sigmoid(4 - 3 d) -> keeps d = 0, 1 and prunes d >= 2 at beta .5
    V, D, K, F = 300, 5, 2, 2
    cfg = make_cfg(oracle_mod, V, D, K, F, 0, 0.5, hidden=1)
    cfg.w1 = torch.tensor([[0.0, 0.0, -3.0]]); cfg.b1 = torch.tensor([4.0])
    cfg.w2 = torch.tensor([1.0]); cfg.b2 = torch.tensor([0.0])
    # relu(4 - 3d): d=0 -> 4, d=1 -> 1, d>=2 -> 0  => C = sigmoid(.) = .98, .73, .5  (C=.5 is kept)
    cfg.threshold = 0.6
    t, L = oracle_mod.build_tree(cfg, seq_logits(V, D, F), 0)
    assert L.n_frontier.tolist() == [1, 2, 2, 0, 0, 0]
    assert abs(L.C[0, 0] - 1 / (1 + math.exp(-4.0))) < 1e-15
    assert abs(L.C[1, 0] - 1 / (1 + math.exp(-1.0))) < 1e-15
    assert t.level[:t.n].max() == 2


def test_all_survivors_mode_adds_every_survivor(oracle_mod):
    V, D, K, F = 400, 3, 4, 2
    cfg = make_cfg(oracle_mod, V, D, K, F, 0, 0.0, classifier="identity", tree_add="all")
    t, L = oracle_mod.build_tree(cfg, seq_logits(V, D, F), 0)
    assert t.n == 1 + K + (D - 1) * F * K
    assert L.n_frontier.tolist() == [1, F, F, F]


# ---------------------------------------------------------------- EAGLE-2 ----

def eagle2_brute(lg: torch.Tensor, K: int, D: int, N: int):
    """Expand + rerank written directly from the description of EAGLE-2 (Sec. 2.2):
    each layer node emits its Top-K, the Top-K of all emitted (by joint probability)
    generate the next layer, then the Top-N of the whole tree by joint probability stay.
    Nodes are token paths; returns (all T_1 paths, kept T_2 paths)."""
    P = {(): 1.0}
    order = [()]
    layer = [()]
    for d in range(D):
        emitted = []
        for j, path in enumerate(layer):
            p_row = scipy.special.softmax(lg[d, j].to(torch.float64).numpy())
            top = np.lexsort((np.arange(p_row.size), -lg[d, j].to(torch.float64).numpy()))[:K]
            for t in top:
                child = path + (int(t),)
                P[child] = P[path] * p_row[t]
                emitted.append(child)
        order += emitted
        ranked = sorted(range(len(emitted)), key=lambda i: (-P[emitted[i]], i))[:K]
        layer = [emitted[i] for i in sorted(ranked)]
    non_root = order[1:]
    ranked = sorted(range(len(non_root)), key=lambda i: (-P[non_root[i]], i))[:N - 1]
    kept = [()] + [non_root[i] for i in sorted(ranked)]
    return order, kept, P


@pytest.mark.parametrize("K,D,N", [(10, 11, 60), (4, 5, 20), (3, 4, 1000)])
def test_identity_classifier_reduces_to_eagle2(oracle_mod, K, D, N):
    V = 64
    cfg = make_cfg(oracle_mod, V, D, K, K, N, 0.0, classifier="identity", tree_add="all")
    lg = seq_logits(V, D, K, scale=1.0)
    t, L = oracle_mod.build_tree(cfg, lg, 0)
    order, kept, P = eagle2_brute(lg, K, D, N)
    assert t.n == 1 + K + (D - 1) * K * K == len(order)          # 1011 at K=10, d_max=11 (App. B.1)
    paths = []
    for i in range(t.n):
        path, a = [], i
        while t.parent[a] >= 0:
            path.append(int(t.tok[a])); a = int(t.parent[a])
        paths.append(tuple(reversed(path)))
    assert paths == order
    ft = oracle_mod.final_prune(t, N)
    got = [paths[s] for s in ft.src[:ft.n]]
    # joint probabilities of distinct nodes can tie only by accident; compare sets of paths
    assert got == kept
    assert ft.n == min(N, t.n)
    kept_set = set(got)
    for path in got:                                              # T_2 is a valid subtree of T_1
        assert path[:-1] in kept_set or path == ()


# ---------------------------------------------------------------- budget -----

def random_tree(rng, n):
    parent = np.full(n, -1, np.int32)
    level = np.zeros(n, np.int32)
    for i in range(1, n):
        parent[i] = rng.integers(0, i)
    # renumber so that ids are level-major like Algorithm 1 produces (parents always earlier)
    for i in range(1, n):
        level[i] = level[parent[i]] + 1
    return parent, level


def test_budget_prune_on_random_small_trees(oracle_mod):
    rng = np.random.default_rng(42)
    for trial in range(200):
        n = int(rng.integers(2, 13))
        parent, level = random_tree(rng, n)
        Cv = rng.random(n)
        if trial % 3 == 0:
            Cv = np.round(Cv * 4) / 4                                 # force ties
        Cv[0] = 1.0
        chat = np.empty(n)
        for i in range(n):                                            # explicit path walks
            m, a = math.inf, i
            while a > 0:
                m = min(m, Cv[a]); a = parent[a]
            chat[i] = m
        tree = oracle_mod.Tree(n, rng.integers(0, 99, n).astype(np.int32), parent, level,
                               np.zeros(n), Cv.copy(), chat.copy())
        N = int(rng.integers(1, n + 3))
        ft = oracle_mod.final_prune(tree, N)
        kept = ft.src[:ft.n].tolist()
        assert ft.n == min(N, n)
        assert kept[0] == 0 and kept == sorted(kept)
        dropped = [i for i in range(n) if i not in kept]
        for i in kept[1:]:
            assert parent[i] in kept                                  # ancestor-closed
            for j in dropped:
                assert (chat[i], -i) > (chat[j], -j)
        remap = {old: new for new, old in enumerate(kept)}
        for new, old in enumerate(kept):
            assert ft.parent[new] == (-1 if old == 0 else remap[int(parent[old])])
            assert ft.tok[new] == tree.tok[old] and ft.level[new] == level[old]
        if N >= n:
            assert kept == list(range(n))


def test_budget_uses_min_confidence_along_path(oracle_mod):
    # root -> a (C .2) -> b (C .9);  root -> c (C .5).  b's score is .2, so N=3 keeps a and c, never b
    parent = np.array([-1, 0, 1, 0], np.int32); level = np.array([0, 1, 2, 1], np.int32)
    Cv = np.array([1.0, 0.2, 0.9, 0.5]); chat = np.array([math.inf, 0.2, 0.2, 0.5])
    tree = oracle_mod.Tree(4, np.arange(4, dtype=np.int32), parent, level, np.zeros(4), Cv, chat)
    assert oracle_mod.final_prune(tree, 3).src[:3].tolist() == [0, 1, 3]
    assert oracle_mod.final_prune(tree, 2).src[:2].tolist() == [0, 3]


def test_build_tree_chat_is_running_minimum(oracle_mod):
    V, D, K, F = 1000, 6, 5, 5
    cfg = make_cfg(oracle_mod, V, D, K, F, 0, 0.45, wseed=3)
    t, _ = oracle_mod.build_tree(cfg, seq_logits(V, D, F), 0)
    assert t.n > 6
    for i in range(1, t.n):
        m, a = math.inf, i
        while a > 0:
            m = min(m, t.C[a]); a = int(t.parent[a])
        assert t.Chat[i] == m


def test_dense_mask_equals_expanded_bit_masks(oracle_mod):
    """The dense additive mask is the bit mask of the verify inputs written out behind the prefix:
    compared entry by entry with the bits (themselves pinned against parent-pointer walks above)."""
    V, D, K, F, N = 500, 5, 3, 3, 14
    cfg = make_cfg(oracle_mod, V, D, K, F, N, 0.0, classifier="identity")
    t, _ = oracle_mod.build_tree(cfg, seq_logits(V, D, F), 3)
    ft = oracle_mod.final_prune(t, N)
    Nw, prefix = oracle_mod.final_width(cfg), 7
    ver = oracle_mod.build_verify(ft, prefix, Nw, D + 1)
    for kv_len in (prefix + Nw, prefix + Nw + 5, prefix + 4, 3):
        m = oracle_mod.dense_mask(ft, prefix, Nw, kv_len)
        assert m.shape == (Nw, kv_len) and set(np.unique(m)) <= {0.0, -np.inf}
        for i in range(Nw):
            for c in range(kv_len):
                if c < prefix:
                    want = True
                elif c - prefix < Nw and i < ft.n:
                    want = bool(int(ver.mask[i, (c - prefix) // 64]) >> ((c - prefix) % 64) & 1)
                else:
                    want = False
                assert (m[i, c] == 0.0) == want
    # a node attends exactly level+1 tree keys
    m = oracle_mod.dense_mask(ft, prefix, Nw, prefix + Nw)
    for i in range(ft.n):
        assert int((m[i, prefix:] == 0.0).sum()) == int(ft.level[i]) + 1


# ---------------------------------------------------------------- chain mode --

@pytest.mark.parametrize("rule,thr", [("cond", 0.3), ("identity", 0.08)])
def test_chain_mode_stop_rules_against_numpy(oracle_mod, rule, thr):
    """K = F = 1 (Sec. 5, Benefits in Chain Mode): the draft is a chain of arg-max tokens that ends
    at the first level whose maximum probability ("DyMax", rule cond) or whose joint probability
    ("DyJoint", rule identity) is below the threshold.  Recomputed here with scipy's softmax."""
    from scipy.special import softmax
    V, D = 3000, 8
    lengths = set()
    for seq in range(12):
        cfg = make_cfg(oracle_mod, V, D, 1, 1, 0, thr, classifier=rule)
        lg = seq_logits(V, D, 1, seq=seq, scale=1.5)
        t, _ = oracle_mod.build_tree(cfg, lg, 7)
        want_tok, joint = [], 1.0
        for l in range(D):
            p = softmax(lg[l, 0].double().numpy())
            tok = int(np.argmax(p))                     # (no exact ties in these rows)
            joint *= p[tok]
            if (p[tok] if rule == "cond" else joint) < thr:
                break
            want_tok.append(tok)
        assert t.n == 1 + len(want_tok)
        assert t.tok[1:t.n].tolist() == want_tok
        assert t.parent[1:t.n].tolist() == list(range(len(want_tok)))
        lengths.add(len(want_tok))
    assert len(lengths) >= 3                            # the rule really stops chains at different depths


# ---------------------------------------------------------------- verify -----

def test_verify_inputs_against_brute_force(oracle_mod):
    rng = np.random.default_rng(7)
    for n in (1, 2, 5, 60, 64, 65, 80, 130):
        parent, level = random_tree(rng, n)
        # level-major renumbering is not required by the definitions; any parent-before-child order works
        ft = oracle_mod.FinalTree(n, np.arange(n, dtype=np.int32), rng.integers(0, 9, n).astype(np.int32),
                                  parent, level)
        width = int(level.max()) + 2
        rows = n + 3
        v = oracle_mod.build_verify(ft, 77, rows, width)
        W = (rows + 63) // 64
        children = {i: [c for c in range(n) if parent[c] == i] for i in range(n)}
        for i in range(n):
            anc = set()
            a = i
            while a >= 0:
                anc.add(a); a = parent[a]
            bits = {j for j in range(rows) if (int(v.mask[i, j // 64]) >> (j % 64)) & 1}
            assert bits == anc
            assert len(bits) == level[i] + 1
            assert v.position_ids[i] == 77 + level[i]
        assert not v.mask[n:].any() and not v.position_ids[n:].any()
        leaves = [i for i in range(n) if not children[i]]
        assert v.n_leaves == len(leaves)
        seen = set()
        for r, leaf in enumerate(leaves):
            chain = [x for x in v.retrieve[r].tolist() if x >= 0]
            assert chain[0] == 0 and chain[-1] == leaf
            for a, b in zip(chain, chain[1:]):
                assert parent[b] == a
            assert v.retrieve[r].tolist() == chain + [-1] * (width - len(chain))
            seen.update(chain)
        assert seen == set(range(n))
        assert (v.retrieve[len(leaves):] == -1).all()


# ---------------------------------------------------------------- accept -----

def test_accept_equals_best_retrieve_row(oracle_mod):
    rng = np.random.default_rng(8)
    V = 12
    for trial in range(100):
        n = int(rng.integers(1, 30))
        parent, level = random_tree(rng, n)
        tok = np.zeros(n, np.int32)
        for i in range(n):                                   # siblings carry distinct tokens
            sib = [c for c in range(i) if parent[c] == parent[i]]
            free = [t for t in range(V) if t not in {int(tok[s]) for s in sib}]
            tok[i] = free[int(rng.integers(0, len(free)))] if free else 0
            if not free:
                parent[i] = i - 1; level[i] = level[i - 1] + 1
        ft = oracle_mod.FinalTree(n, np.arange(n, dtype=np.int32), tok, parent, level)
        width = int(level.max()) + 2
        target = torch.from_numpy(rng.standard_normal((n, V)).astype(np.float32))
        if trial % 2:
            target = target.to(torch.bfloat16)
        acc = oracle_mod.accept(ft, target, width)
        amax = target.to(torch.float64).numpy().argmax(axis=1)       # first occurrence = lower id
        assert acc.node_argmax[:n].tolist() == amax.tolist()
        v = oracle_mod.build_verify(ft, 0, n, width)
        best = 0
        for r in range(v.n_leaves):
            chain = [x for x in v.retrieve[r].tolist() if x >= 0]
            k = 0
            while k + 1 < len(chain) and tok[chain[k + 1]] == amax[chain[k]]:
                k += 1
            best = max(best, k)
        assert acc.accept_len == best
        path = [x for x in acc.path.tolist() if x >= 0]
        assert len(path) == best + 1 and path[0] == 0
        for a, b in zip(path, path[1:]):
            assert parent[b] == a and tok[b] == amax[a]
        assert acc.next_token == amax[path[-1]]


def test_accept_planted_path(oracle_mod):
    V, D, K, F = 3000, 6, 4, 4
    cfg = make_cfg(oracle_mod, V, D, K, F, 0, 0.0, classifier="identity")
    t, _ = oracle_mod.build_tree(cfg, seq_logits(V, D, F), 0)
    ft = oracle_mod.final_prune(t, 0)
    for depth in range(0, D + 1):
        leaf = max(i for i in range(ft.n) if ft.level[i] == depth)
        chain = []
        a = leaf
        while a >= 0:
            chain.append(a); a = int(ft.parent[a])
        chain.reverse()
        target = torch.zeros(ft.n, V)
        off_tree = int(np.setdiff1d(np.arange(V), ft.tok[:ft.n])[0])
        target[:, off_tree] = 1.0                           # default: a token no child carries
        for a, b in zip(chain, chain[1:]):
            target[a, off_tree] = 0.0
            target[a, ft.tok[b]] = 2.0
        acc = oracle_mod.accept(ft, target, D + 1)
        assert acc.accept_len == depth
        assert [x for x in acc.path.tolist() if x >= 0] == chain
        assert acc.next_token == off_tree


def test_argmax_ties_go_to_lower_id(oracle_mod):
    row = torch.tensor([1.0, 3.0, 3.0, 2.0]).to(torch.bfloat16)
    assert oracle_mod.row_argmax(row) == 1


# ---------------------------------------------------------------- whole step -

def test_decode_step_matches_per_sequence_calls(oracle_mod):
    B, V, D, K, F, N = 3, 1500, 4, 5, 4, 12
    cfg = make_cfg(oracle_mod, V, D, K, F, N, 0.5, dtype=torch.bfloat16, wseed=1)
    draft = torch.stack([seq_logits(V, D, F, torch.bfloat16, seq=b) for b in range(B)])   # [B,D,F,V]
    Nw = oracle_mod.final_width(cfg)
    target = c2t_inputs.target_logits(B, Nw, V, 0, torch.bfloat16)
    root = c2t_inputs.root_tokens(B, V).numpy()
    pre = c2t_inputs.prefix_lengths(B).numpy()
    r = oracle_mod.decode_step(cfg, draft, target, root, pre)
    for b in range(B):
        t, _ = oracle_mod.build_tree(cfg, draft[b], int(root[b]))
        ft = oracle_mod.final_prune(t, N)
        v = oracle_mod.build_verify(ft, int(pre[b]), Nw, D + 1)
        acc = oracle_mod.accept(ft, target[b], D + 1)
        assert r.n_final[b] == ft.n
        assert r.tokens[b, :ft.n].tolist() == ft.tok[:ft.n].tolist()
        assert r.parents[b, :ft.n].tolist() == ft.parent[:ft.n].tolist()
        assert np.array_equal(r.mask[b], v.mask) and np.array_equal(r.retrieve[b], v.retrieve)
        assert np.array_equal(r.position_ids[b], v.position_ids)
        assert r.n_leaves[b] == v.n_leaves
        assert r.accept_len[b] == acc.accept_len and r.next_token[b] == acc.next_token
        assert np.array_equal(r.path[b], acc.path)


def test_generator_is_deterministic_and_keyed():
    a = c2t_inputs.draft_logits(2, 3, 100, 0, 1, torch.bfloat16)
    b = c2t_inputs.draft_logits(2, 3, 100, 0, 1, torch.bfloat16)
    c = c2t_inputs.draft_logits(2, 3, 100, 0, 2, torch.bfloat16)
    assert torch.equal(a, b) and not torch.equal(a, c)
    # sequence b of a batch equals the same sequence generated alone
    d = c2t_inputs.draft_logits(1, 3, 100, 0, 1, torch.bfloat16, seq_base=1)
    assert torch.equal(a[1], d[0])
    r = c2t_inputs.token_rank(0, 100)
    assert sorted(r.tolist()) == list(range(1, 101))

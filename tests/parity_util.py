"""Helpers shared by the GPU parity tests: run the library and the oracle on the same bytes
and compare them element by element.

Tolerances (relative, on probabilities, entropies and confidences): 1e-5 for fp32 logits,
2e-3 for bf16 logits.  Everything integer (tokens, kept sets, parents, masks, positions,
retrieve rows, accept lengths) must be identical, with one family of exceptions that is checked
candidate by candidate.  Where the two sides take a different decision, every candidate (or
node) whose decision differs must itself sit on a boundary in the oracle:

  near_beta      its confidence is within 1e-6 (relative) of the threshold;
  near_cap       it was swapped, in the F-survivor cap, with a candidate whose confidence is within
                 1e-6 (relative) of its own and not equal to it;
  cross_row_tie  the same swap between two candidates of DIFFERENT rows whose oracle confidences
                 are exactly equal: the oracle orders them by candidate index, the CUDA path by the
                 last bits of two fp32 row sums (exactly equal confidences from the same row tie
                 on both sides and must agree);
  near_budget    the same two rules at the cut of the Top-N rerank (min-confidence-on-path scores).

Anything else fails at once.  A sequence with such a difference is "diverged" from that level
on (its later levels legitimately differ); the caller states how many diverged sequences of
which kinds a case may have (none by default), and that is asserted, not printed.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field

import numpy as np
import torch

import c2t_inputs
import oracle
import paper_2502_13652_b200 as c2t

RTOL = {torch.float32: 1e-5, torch.bfloat16: 2e-3}
NEAR = 1e-6
# Entropy also gets an absolute floor: the oracle evaluates Eq. 2 literally, through ln Z with
# Z = 1 + eps for a peaked row, so its own fp64 rounding leaves an absolute error of a few
# 1e-16 in H; below H ~ 1e-10 that exceeds any relative tolerance.  1e-12 is far above that
# rounding and far below any entropy that moves a confidence.
H_ATOL = 1e-12


def make_configs(B, V, D, K, F, N, beta, dtype, classifier="mlp", hidden=16, tree_add="frontier",
                 wseed=0, wstd=0.1, weights=None, M=0):
    w1, b1, w2, b2 = weights if weights is not None else c2t_inputs.classifier_weights(hidden, seed=wseed, std=wstd)
    ocfg = oracle.OracleConfig(
        vocab=V, dtype=oracle.BF16 if dtype == torch.bfloat16 else oracle.F32, max_depth=D, topk=K,
        frontier_cap=F, budget=N, threshold=beta, entropy_top_m=M,
        classifier={"mlp": oracle.CLS_MLP, "identity": oracle.CLS_IDENTITY_JOINT, "cond": oracle.CLS_IDENTITY_COND}[classifier],
        hidden=hidden, w1=w1, b1=b1, w2=w2, b2=b2,
        tree_add=oracle.ADD_FRONTIER if tree_add == "frontier" else oracle.ADD_ALL_SURVIVORS)
    gcfg = c2t.Config(
        batch=B, vocab=V, dtype=c2t.BF16 if dtype == torch.bfloat16 else c2t.F32, max_depth=D, topk=K,
        frontier_cap=F, budget=N, threshold=beta, entropy_top_m=M,
        classifier={"mlp": c2t.CLS_MLP, "identity": c2t.CLS_IDENTITY_JOINT, "cond": c2t.CLS_IDENTITY_COND}[classifier],
        hidden=hidden, w1=w1, b1=b1, w2=w2, b2=b2,
        tree_add=c2t.ADD_FRONTIER if tree_add == "frontier" else c2t.ADD_ALL_SURVIVORS)
    return ocfg, gcfg


def gen_inputs(B, V, D, F, Nw, dtype, step=0, scale=4.0, device="cpu", seq_base=0):
    draft = [c2t_inputs.draft_logits(B, F, V, step, l, dtype, scale, device=device, seq_base=seq_base)
             for l in range(D)]
    target = c2t_inputs.target_logits(B, Nw, V, step, dtype, scale, device=device, seq_base=seq_base)
    root = c2t_inputs.root_tokens(B, V, step, seq_base)
    prefix = c2t_inputs.prefix_lengths(B, seq_base=seq_base)
    return draft, target, root, prefix


# Rows that stress one property each (ties, -inf, a dominant element, values that keep rising).
def special_rows(kind, B, F, V, dtype):
    g = torch.Generator().manual_seed(5)
    if kind == "uniform":
        return torch.full((B, F, V), 1.5).to(dtype)
    if kind == "two_valued":
        x = torch.where(torch.rand(B, F, V, generator=g) < 0.001, torch.tensor(9.0), torch.tensor(-2.0))
        return x.to(dtype)
    if kind == "heavy_ties":
        return (40 + torch.randn(B, F, V, generator=g) * 0.4).to(torch.bfloat16).to(dtype)
    if kind == "neg_inf":
        x = torch.randn(B, F, V, generator=g) * 3
        x[torch.rand(B, F, V, generator=g) < 0.3] = float("-inf")
        x[:, :, : V // 2] = float("-inf")         # first half of every row has probability zero
        return x.to(dtype)
    if kind == "peaked":
        x = torch.randn(B, F, V, generator=g)
        x[:, :, 17] = 30.0                         # entropy ~1e-11: the tail must keep relative accuracy
        return x.to(dtype)
    if kind == "rising":
        # every vector beats everything before it; the noise keeps sums of two log-probs from tying
        x = torch.arange(V, dtype=torch.float32) * (80.0 / V) + torch.randn(B, F, V, generator=g) * 0.3
        return x.to(dtype)
    if kind == "late_jump":
        x = torch.randn(B, F, V, generator=g) - 500.0
        x[:, :, V - 100:] += 600.0                 # the last elements dwarf everything seen before
        return x.to(dtype)
    raise ValueError(kind)


@dataclass
class Report:
    sequences: int = 0
    near_tie_sequences: int = 0          # sequences in which the oracle sits on some boundary (information only)
    diverged_sequences: int = 0          # sequences with an excused difference (see the module docstring)
    excused: dict = field(default_factory=dict)      # kind -> sequences
    where: dict = field(default_factory=dict)        # sequence -> (level or "final", kind)
    max_rel_p: float = 0.0
    max_rel_H: float = 0.0
    max_rel_C: float = 0.0
    kept_nodes: list = field(default_factory=list)         # the CUDA path's final node counts
    accept_len: list = field(default_factory=list)         # the CUDA path's accept lengths
    oracle_kept_nodes: list = field(default_factory=list)
    oracle_accept_len: list = field(default_factory=list)
    oracle_next_token: list = field(default_factory=list)
    rows_expanded: int = 0               # active draft rows over all levels
    rows_topm_from_pass: int = 0         # of those, rows whose Eq. 3 sums came from the vectors the pass set aside

    def line(self) -> str:
        return (f"seq={self.sequences} near_tie={self.near_tie_sequences} diverged={self.diverged_sequences} "
                f"{dict(self.excused) if self.excused else ''} "
                f"max_rel p={self.max_rel_p:.2e} H={self.max_rel_H:.2e} C={self.max_rel_C:.2e} "
                f"mean_nodes={np.mean(self.kept_nodes) if self.kept_nodes else 0:.1f} "
                f"mean_tau={np.mean(self.accept_len) if self.accept_len else 0:.2f}")


def _rel(a: np.ndarray, b: np.ndarray, atol: float = 0.0) -> float:
    """max (|a-b| - atol) / |b| over finite entries (0 where both are equal)."""
    a = np.asarray(a, np.float64); b = np.asarray(b, np.float64)
    if a.size == 0:
        return 0.0
    den = np.maximum(np.abs(b), 1e-300)
    r = np.maximum(np.abs(a - b) - atol, 0.0) / den
    r[(a == b)] = 0.0
    return float(np.nanmax(r)) if np.isfinite(r).any() else 0.0


def _close(a: float, b: float) -> bool:
    return abs(a - b) <= NEAR * max(abs(a), abs(b))


def _near_tie_at_level(L, l, F, beta) -> bool:
    """Does the oracle sit on a boundary at this level (information only)?"""
    n = int(L.n_cand[l])
    if n == 0:
        return False
    Cv = L.C[l, :n]
    if beta != 0.0 and np.any(np.abs(Cv - beta) <= NEAR * abs(beta)):
        return True
    surv = np.sort(Cv[L.keep[l, :n] == 1])[::-1]
    return len(surv) > F and surv[F - 1] != surv[F] and _close(surv[F - 1], surv[F])


def _near_tie_budget(tree, N) -> bool:
    if N <= 0 or tree.n <= N:
        return False
    ch = np.sort(tree.Chat[1:tree.n])[::-1]
    a, b = ch[N - 2], ch[N - 1]
    return a != b and _close(a, b)


def _excuse_swaps(lost, won, score, group) -> str | None:
    """lost: items the oracle selected and the CUDA path did not; won: the reverse.  Every item must
    have a partner on the other side whose oracle score is within 1e-6 of its own; exactly equal
    scores only count between different groups (rows / parents).  Returns the kind, or None."""
    if len(lost) != len(won) or not lost:
        return None
    kind = None
    for mine, others in ((lost, won), (won, lost)):
        for i in mine:
            exact = [o for o in others if score[o] == score[i] and group[o] != group[i]]
            near = [o for o in others if score[o] != score[i] and _close(score[o], score[i])]
            if not exact and not near:
                return None
            k = "near" if near else "cross_row_tie"
            kind = k if kind in (None, k) else "near"
    return kind


def _excuse_level(L, l, K, beta, g_flags) -> str | None:
    """The keep/next flags of a level differ: is every differing candidate on a boundary of the oracle?"""
    n = int(L.n_cand[l])
    Cv = L.C[l, :n]
    o_keep, o_next = L.keep[l, :n], L.next[l, :n]
    g_keep, g_next = g_flags[:n] & 1, (g_flags[:n] >> 1) & 1
    dk = np.nonzero(o_keep != g_keep)[0]
    if len(dk):
        # a candidate that crosses the threshold also shifts the cap, so nothing else is asked of this level
        ok = beta != 0.0 and all(abs(Cv[c] - beta) <= NEAR * abs(beta) for c in dk)
        return "near_beta" if ok else None
    lost = [int(c) for c in np.nonzero((o_next == 1) & (g_next == 0))[0]]
    won = [int(c) for c in np.nonzero((o_next == 0) & (g_next == 1))[0]]
    kind = _excuse_swaps(lost, won, Cv, np.arange(n) // K)
    return {"near": "near_cap", "cross_row_tie": "cross_row_tie", None: None}[kind]


def _excuse_budget(tree, ft, g_src) -> str | None:
    """The reranks kept different nodes of the same tree: is every differing node on the cut of the oracle?"""
    o_set, g_set = set(int(i) for i in ft.src[:ft.n]), set(int(i) for i in g_src)
    if len(o_set) != len(g_set) or not all(0 <= i < tree.n for i in g_set):
        return None
    kind = _excuse_swaps(sorted(o_set - g_set), sorted(g_set - o_set), tree.Chat, tree.parent)
    return {"near": "near_budget", "cross_row_tie": "cross_row_tie", None: None}[kind]


def run_and_compare(ocfg, gcfg, draft_cpu, target_cpu, root, prefix, seqs=None, ctx=None,
                    draft_dev=None, target_dev=None, shards=None, allow_diverged=0, allow_kinds=(), fused=False) -> Report:
    """Runs one decode step on the GPU (level by level) and on the oracle; asserts parity.

    shards: token ranges [(begin, end), ...] covering the vocabulary in ascending order.  Every level
    is then built the vocabulary-parallel way (one sharded pass and one record export per range, run
    one after the other on this GPU, then the prune from the gathered records); the oracle still
    works on whole rows.

    draft_cpu: list of D tensors [B,F,V] on CPU (or None when `seqs` rows are pulled from
    draft_dev); seqs: sequences the oracle checks (default all).

    fused: every level through c2t_expand_prune_level (one launch for small batches) instead of the two calls.

    allow_diverged / allow_kinds: how many sequences may differ from the oracle through a boundary
    case of the module docstring, and of which kinds; more, or another kind, fails."""
    dtype = gcfg.torch_dtype
    rtol = RTOL[dtype]
    B, D, F, K = gcfg.batch, gcfg.max_depth, gcfg.frontier_cap, gcfg.topk
    own = ctx is None
    if own:
        ctx = c2t.Context(gcfg)
    dev = ctx.device
    if draft_dev is None:
        draft_dev = [t.to(dev) for t in draft_cpu]
        target_dev = target_cpu.to(dev)
    seqs = list(range(B)) if seqs is None else list(seqs)
    beta = float(np.float32(gcfg.threshold))

    # oracle, one sequence at a time
    orc = {}
    for b in seqs:
        if draft_cpu is not None:
            lg = torch.stack([draft_cpu[l][b] for l in range(D)])
            tg = target_cpu[b]
        else:
            lg = torch.stack([draft_dev[l][b].cpu() for l in range(D)])
            tg = target_dev[b].cpu()
        tree, L = oracle.build_tree(ocfg, lg, int(root[b]))
        ft = oracle.final_prune(tree, ocfg.budget)
        ver = oracle.build_verify(ft, int(prefix[b]), ctx.Nw, D + 1)
        acc = oracle.accept(ft, tg[:max(ft.n, 1)], D + 1)
        orc[b] = (tree, L, ft, ver, acc)

    rep = Report(sequences=len(seqs))
    near = {b: False for b in seqs}
    diverged = {}                                   # sequence -> (level or "final", kind)

    root_d = root.to(dev); prefix_d = prefix.to(dev)
    ctx.c2t_begin_step(root_d, prefix_d)
    records = ctx.new_row_records(len(shards)) if shards else None
    for l in range(D):
        if shards:
            for g, (v0, v1) in enumerate(shards):
                ctx.c2t_expand_level_shard(l, draft_dev[l][:, :, v0:v1])
                ctx.c2t_export_row_records(l, v0, records[g])
            ctx.c2t_prune_gathered(l, records)
        elif fused:
            ctx.c2t_expand_prune_level(l, draft_dev[l])
        else:
            n_in = ctx.c2t_get_view()["frontier_n"].cpu().numpy().copy()
            ctx.c2t_expand_level(l, draft_dev[l])
            from_pass = ctx.c2t_get_view()["topm_from_pass"]
            if from_pass is not None:
                fp = from_pass.cpu().numpy()
                rep.rows_expanded += int(n_in.sum())
                rep.rows_topm_from_pass += int(sum(fp[b, :n_in[b]].sum() for b in range(B)))
            ctx.c2t_prune(l)
        view = ctx.c2t_get_view()
        torch.cuda.synchronize()
        g_n = view["cand_n"].cpu().numpy()
        g_tok = view["cand_token"].cpu().numpy(); g_flags = view["cand_flags"].cpu().numpy()
        g_lp = view["cand_lp"].cpu().numpy(); g_logP = view["cand_logP"].cpu().numpy()
        g_H = view["cand_H"].cpu().numpy(); g_C = view["cand_C"].cpu().numpy()
        g_fn = view["frontier_n"].cpu().numpy(); g_fnode = view["frontier_node"].cpu().numpy()
        e_cnt = ctx.frontier["count"].cpu().numpy(); e_tok = ctx.frontier["token"].cpu().numpy()
        e_node = ctx.frontier["node_id"].cpu().numpy(); e_ps = ctx.frontier["parent_slot"].cpu().numpy()
        for b in seqs:
            if b in diverged:
                continue
            tree, L, *_ = orc[b]
            n = int(L.n_cand[l])
            near[b] = near[b] or _near_tie_at_level(L, l, F, beta)
            assert g_n[b] == n, f"level {l} seq {b}: candidate count {g_n[b]} != {n}"
            if n == 0:
                assert g_fn[b] == 0
                continue
            assert np.array_equal(g_tok[b, :n], L.tok[l, :n]), f"level {l} seq {b}: top-K tokens differ"
            rp = _rel(np.exp(g_lp[b, :n]), np.exp(L.lp[l, :n]))
            rP = _rel(np.exp(g_logP[b, :n]), np.exp(L.logP[l, :n]))
            rH = _rel(g_H[b, :n], L.H[l, :n], H_ATOL); rC = _rel(g_C[b, :n], L.C[l, :n])
            rep.max_rel_p = max(rep.max_rel_p, rp, rP); rep.max_rel_H = max(rep.max_rel_H, rH)
            rep.max_rel_C = max(rep.max_rel_C, rC)
            assert rp <= rtol and rP <= rtol, f"level {l} seq {b}: probability error {rp:.2e}/{rP:.2e}"
            assert rH <= rtol, f"level {l} seq {b}: entropy error {rH:.2e}"
            assert rC <= rtol, f"level {l} seq {b}: confidence error {rC:.2e}"
            o_flags = L.keep[l, :n] | (L.next[l, :n] << 1)
            if not np.array_equal(g_flags[b, :n], o_flags):
                kind = _excuse_level(L, l, K, beta, g_flags[b])
                assert kind is not None, (f"level {l} seq {b}: keep/next flags differ at candidates that are on no "
                                          f"boundary of the oracle: {np.nonzero(g_flags[b, :n] != o_flags)[0].tolist()}")
                diverged[b] = (l, kind)
                continue
            nn = int(L.n_frontier[l + 1])
            assert g_fn[b] == nn and e_cnt[b] == nn
            assert np.array_equal(g_fnode[b, :nn], L.frontier_node[l + 1, :nn])
            assert np.array_equal(e_node[b, :nn], L.frontier_node[l + 1, :nn])
            sel = np.nonzero(L.next[l, :n])[0]
            assert np.array_equal(e_tok[b, :nn], L.tok[l, sel])
            assert np.array_equal(e_ps[b, :nn], sel // K)

    ctx.c2t_prune(c2t.FINAL)
    ctx.c2t_build_verify()
    ctx.c2t_accept(target_dev)
    bits, per = ctx.c2t_status()
    view = {k: v.cpu().numpy() for k, v in ctx.c2t_get_view().items() if v is not None}
    ver_g = {k: v.cpu().numpy() for k, v in ctx.verify.items()}
    acc_g = {k: v.cpu().numpy() for k, v in ctx.accepted.items()}
    # the walk that reads only the rows it visits must give the same answers
    ctx.c2t_accept_lazy(target_dev)
    acc_l = {k: v.cpu().numpy() for k, v in ctx.accepted.items()}
    amax_l = ctx.c2t_get_view()["node_argmax"].cpu().numpy()
    for k in ("accept_len", "path", "next_token"):   # on every sequence, checked against the oracle or not
        assert np.array_equal(acc_l[k], acc_g[k]), f"lazy acceptance: {k} differs from the all-rows walk"
    if shards:
        # the acceptance with the target rows sharded the same way: one key per node and range, the walk from the
        # gathered keys; everything it writes must equal the whole-row walk (checked against the oracle below)
        keys = torch.zeros((len(shards), B, ctx.Nw), dtype=torch.int64, device=dev)
        for g, (v0, v1) in enumerate(shards):
            ctx.c2t_argmax_shard(target_dev[:, :, v0:v1], v0, keys[g])
        ctx.c2t_accept_gathered(keys)
        acc_s = {k: v.cpu().numpy() for k, v in ctx.accepted.items()}
        amax_s = ctx.c2t_get_view()["node_argmax"].cpu().numpy()
        for k in acc_g:
            assert np.array_equal(acc_s[k], acc_g[k]), f"sharded acceptance: {k} differs from the whole-row walk"
        assert np.array_equal(amax_s, view["node_argmax"])
        # ... and the walk that reads only the rows it visits, sharded: D + 1 rounds of one key per sequence and range
        lkeys = torch.zeros((len(shards), B), dtype=torch.int64, device=dev)
        ctx.c2t_lazy_begin()
        for r in range(1, D + 2):
            for g, (v0, v1) in enumerate(shards):
                ctx.c2t_lazy_argmax_shard(target_dev[:, :, v0:v1], v0, lkeys[g])
            ctx.c2t_lazy_step_gathered(r, lkeys)
        acc_ls = {k: v.cpu().numpy() for k, v in ctx.accepted.items()}
        amax_ls = ctx.c2t_get_view()["node_argmax"].cpu().numpy()
        for k in acc_g:
            assert np.array_equal(acc_ls[k], acc_g[k]), f"sharded lazy acceptance: {k} differs from the whole-row walk"
        assert np.array_equal(amax_ls, amax_l), "sharded lazy acceptance read other rows than the whole-row lazy walk"
    ctx.c2t_accept(target_dev)                      # leave the all-rows results behind for the caller
    for b in seqs:
        tree, L, ft, ver, acc = orc[b]
        near[b] = near[b] or _near_tie_budget(tree, ocfg.budget)
        rep.oracle_kept_nodes.append(int(ft.n)); rep.oracle_accept_len.append(int(acc.accept_len))
        rep.oracle_next_token.append(int(acc.next_token))
        rep.kept_nodes.append(int(ver_g["n_nodes"][b])); rep.accept_len.append(int(acc_g["accept_len"][b]))
        if b in diverged:
            continue
        n = tree.n
        assert view["tree_n"][b] == n, f"seq {b}: tree size {view['tree_n'][b]} != {n}"
        assert np.array_equal(view["tree_token"][b, :n], tree.tok[:n]), f"seq {b}: tree tokens differ"
        assert np.array_equal(view["tree_parent"][b, :n], tree.parent[:n]), f"seq {b}: tree parents differ"
        assert np.array_equal(view["tree_level"][b, :n], tree.level[:n]), f"seq {b}: tree levels differ"
        if n > 1:
            rP = _rel(np.exp(view["tree_logP"][b, 1:n]), np.exp(tree.logP[1:n]))
            rC = _rel(view["tree_C"][b, 1:n], tree.C[1:n])
            rep.max_rel_p = max(rep.max_rel_p, rP); rep.max_rel_C = max(rep.max_rel_C, rC)
            assert rP <= rtol and rC <= rtol
        m = ft.n
        assert view["final_n"][b] == m and ver_g["n_nodes"][b] == m, f"seq {b}: final node count differs"
        if not np.array_equal(view["final_src"][b, :m], ft.src[:m]):
            kind = _excuse_budget(tree, ft, view["final_src"][b, :m])
            assert kind is not None, f"seq {b}: the reranks keep different nodes, none of them on the oracle's cut"
            diverged[b] = ("final", kind)
            continue
        cols = np.arange(ctx.Nw)
        assert np.array_equal(ver_g["tokens"][b], np.where(cols < m, ft.tok[:ctx.Nw], 0)), f"seq {b}: final tokens"
        assert np.array_equal(ver_g["parents"][b], np.where(cols < m, ft.parent[:ctx.Nw], -1)), f"seq {b}: final parents"
        assert np.array_equal(ver_g["position_ids"][b], ver.position_ids), f"seq {b}: position ids"
        assert np.array_equal(ver_g["mask_bits"][b].view(np.uint64), ver.mask), f"seq {b}: tree-attention masks"
        assert np.array_equal(ver_g["retrieve"][b], ver.retrieve), f"seq {b}: retrieve rows"
        assert ver_g["n_leaves"][b] == ver.n_leaves, f"seq {b}: leaf count"
        assert np.array_equal(view["node_argmax"][b, :m], acc.node_argmax[:m]), f"seq {b}: target arg-maxes"
        assert acc_g["accept_len"][b] == acc.accept_len, f"seq {b}: accept length"
        assert np.array_equal(acc_g["path"][b], acc.path), f"seq {b}: accepted path"
        assert acc_g["next_token"][b] == acc.next_token, f"seq {b}: next token"
        on_path = np.zeros(ctx.Nw, dtype=bool); on_path[[i for i in acc.path if i >= 0]] = True
        assert np.array_equal(amax_l[b, :m][on_path[:m]], np.asarray(acc.node_argmax[:m])[on_path[:m]])
        assert (amax_l[b][~on_path] == -1).all(), f"seq {b}: the lazy walk read rows off its path"
    rep.near_tie_sequences = sum(near.values())
    rep.diverged_sequences = len(diverged)
    rep.where = dict(diverged)
    for _, kind in diverged.values():
        rep.excused[kind] = rep.excused.get(kind, 0) + 1
    rep.status_bits = bits
    if own:
        ctx.close()
    assert rep.diverged_sequences <= allow_diverged and set(rep.excused) <= set(allow_kinds), (
        f"{rep.diverged_sequences} sequence(s) differ from the oracle through boundary cases {rep.where}; "
        f"this case allows {allow_diverged} of kinds {tuple(allow_kinds)}")
    return rep


ALL_KINDS = ("near_beta", "near_cap", "near_budget", "cross_row_tie")


def run_chain(ocfg, gcfg, n_steps, seqs, scale=4.0, allow_diverged=0, allow_kinds=()):
    """`n_steps` decode steps in a row: step s + 1 starts from step s's next token and from a prefix
    that is accept_len + 1 tokens longer (Sec. 2.1: the accepted drafts and the target's own token are
    committed).  The CUDA path carries that state on the device, from its own outputs; the oracle
    carries its own.  Before every step the two states of the checked sequences must be equal; every
    step is compared like a single one.  A step that differs through a boundary case (see the module
    docstring) is counted, and the oracle's state is set to the CUDA path's from there on."""
    dtype = gcfg.torch_dtype
    B, V, D, F = gcfg.batch, gcfg.vocab, gcfg.max_depth, gcfg.frontier_cap
    ctx = c2t.Context(gcfg)
    dev = ctx.device
    Nw = ctx.Nw
    root = c2t_inputs.root_tokens(B, V, 0).to(dev)
    prefix = c2t_inputs.prefix_lengths(B).to(dev)
    o_root = {b: int(root[b]) for b in seqs}
    o_prefix = {b: int(prefix[b]) for b in seqs}
    out = Report(sequences=len(seqs))
    steps_diverged = 0
    for s in range(n_steps):
        draft = [c2t_inputs.draft_logits(B, F, V, s, l, dtype, scale, device=dev) for l in range(D)]
        target = c2t_inputs.target_logits(B, Nw, V, s, dtype, scale, device=dev)
        rc, pc = root.cpu(), prefix.cpu()
        for b in seqs:
            assert int(rc[b]) == o_root[b] and int(pc[b]) == o_prefix[b], f"step {s} seq {b}: the chains' states differ"
        rep = run_and_compare(ocfg, gcfg, None, None, root, prefix, seqs=seqs, ctx=ctx, draft_dev=draft,
                              target_dev=target, allow_diverged=len(seqs), allow_kinds=ALL_KINDS)
        assert rep.status_bits == 0
        # both chains advance from their own results (device tensors on the CUDA side: no host round trip)
        new_root = ctx.accepted["next_token"].clone()
        new_prefix = prefix + ctx.accepted["accept_len"] + 1
        for i, b in enumerate(seqs):
            if b in rep.where:
                steps_diverged += 1
                out.excused[rep.where[b][1]] = out.excused.get(rep.where[b][1], 0) + 1
                out.where[(s, b)] = rep.where[b]
                o_root[b], o_prefix[b] = int(new_root[b]), int(new_prefix[b])
            else:
                o_root[b] = rep.oracle_next_token[i]
                o_prefix[b] += rep.oracle_accept_len[i] + 1
        root, prefix = new_root, new_prefix
        out.kept_nodes += rep.kept_nodes; out.accept_len += rep.accept_len
        out.oracle_kept_nodes += rep.oracle_kept_nodes; out.oracle_accept_len += rep.oracle_accept_len
        out.max_rel_p = max(out.max_rel_p, rep.max_rel_p); out.max_rel_H = max(out.max_rel_H, rep.max_rel_H)
        out.max_rel_C = max(out.max_rel_C, rep.max_rel_C)
        out.near_tie_sequences += rep.near_tie_sequences
    out.diverged_sequences = steps_diverged
    out.status_bits = 0
    out.final_prefix = prefix.cpu()
    ctx.close()
    assert steps_diverged <= allow_diverged and set(out.excused) <= set(allow_kinds), (
        f"{steps_diverged} sequence-step(s) differ from the oracle through boundary cases {out.where}; "
        f"this chain allows {allow_diverged} of kinds {tuple(allow_kinds)}")
    return out

"""GPU parity: the CUDA library against the CPU oracle on the same seeded bytes, through the C ABI."""
import json
import math
import os

import numpy as np
import pytest
import torch

import c2t_inputs
import oracle
import paper_2502_13652_b200 as c2t
from parity_util import RTOL, gen_inputs, make_configs, run_and_compare, run_chain, special_rows

pytestmark = pytest.mark.gpu

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


@pytest.fixture(scope="module", autouse=True)
def _built():
    from paper_2502_13652_b200 import build
    build.build()
    oracle.build()
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    assert os.path.exists(c2t.LIB_PATH)


def case(B, V, D, K, F, N, beta, dtype, step=0, scale=4.0, allow_diverged=0, allow_kinds=(), fused=False, **kw):
    """One decode step of seeded inputs on both sides.  No sequence may differ from the oracle unless the
    caller names the boundary case and bounds the count (see parity_util)."""
    ocfg, gcfg = make_configs(B, V, D, K, F, N, beta, dtype, **kw)
    Nw = c2t.c2t_final_width(gcfg)
    draft, target, root, prefix = gen_inputs(B, V, D, F, Nw, dtype, step=step, scale=scale)
    rep = run_and_compare(ocfg, gcfg, draft, target, root, prefix, allow_diverged=allow_diverged,
                          allow_kinds=allow_kinds, fused=fused)
    print(f"\n  [{B}x{V} {str(dtype)[6:]} D{D} K{K} F{F} N{N} b{beta}] {rep.line()}")
    assert rep.status_bits == 0
    assert rep.kept_nodes == rep.oracle_kept_nodes or rep.diverged_sequences
    return rep


def test_tiny_hand_enumerated_tree():
    with open(os.path.join(GOLDEN, "tiny_tree_v8.json")) as f:
        G = json.load(f)
    V, D, K, F, N = 8, G["D"], G["K"], G["F"], G["N"]
    ocfg, gcfg = make_configs(1, V, D, K, F, N, G["beta"], torch.float32, classifier="identity")
    row = torch.tensor([math.log(p) for p in G["p"]], dtype=torch.float64).to(torch.float32)
    draft = [row.expand(1, F, V).contiguous() for _ in range(D)]
    target = torch.zeros(1, N, V)
    for i, a in enumerate(G["target_argmax"]):
        target[0, i, a] = 5.0
    root = torch.tensor([G["root_token"]], dtype=torch.int32)
    prefix = torch.tensor([G["prefix_len"]], dtype=torch.int32)
    ctx = c2t.Context(gcfg)
    rep = run_and_compare(ocfg, gcfg, draft, target, root, prefix, ctx=ctx)
    assert rep.diverged_sequences == 0
    # and directly against the hand-enumerated values
    v = ctx.verify
    assert v["n_nodes"].tolist() == [N]
    assert v["tokens"][0].tolist() == G["final_tokens"]
    assert v["parents"][0].tolist() == G["final_parents"]
    assert v["mask_bits"][0, :, 0].tolist() == G["final_masks"]
    assert v["position_ids"][0].tolist() == G["final_positions"]
    assert v["n_leaves"].tolist() == [G["n_leaves"]]
    assert v["retrieve"][0, :G["n_leaves"]].tolist() == G["retrieve"]
    assert ctx.accepted["accept_len"].tolist() == [G["accept_len"]]
    assert ctx.accepted["path"][0].tolist() == G["accept_path"]
    assert ctx.accepted["next_token"].tolist() == [G["next_token"]]
    ctx.close()


def test_config1_single_sequence_fp32():
    case(1, 32000, 6, 10, 10, 60, 0.5, torch.float32)


@pytest.mark.parametrize("B,V,dtype", [(1, 32000, torch.float32), (2, 32000, torch.bfloat16), (1, 128256, torch.bfloat16),
                                       (2, 5000, torch.float32)])
def test_fused_expand_prune_level_against_oracle(B, V, dtype):
    """Expand and prune of a level in one launch (batches of one or two sequences): against the oracle like the
    separate calls, and one launch per level."""
    D = 6
    ocfg, gcfg = make_configs(B, V, D, 8, 16, 50, 0.4, dtype)
    Nw = c2t.c2t_final_width(gcfg)
    draft, target, root, prefix = gen_inputs(B, V, D, 16, Nw, dtype)
    ctx = c2t.Context(gcfg)
    n0 = ctx.c2t_launch_count()
    rep = run_and_compare(ocfg, gcfg, draft, target, root, prefix, ctx=ctx, fused=True)
    assert rep.status_bits == 0
    # begin_step, D fused levels, rerank, verify inputs; then the acceptance calls of the comparison
    ctx.decode_step([t.cuda() for t in draft], target.cuda(), root.cuda(), prefix.cuda())
    n1 = ctx.c2t_launch_count()
    ctx.decode_step([t.cuda() for t in draft], target.cuda(), root.cuda(), prefix.cuda())
    assert ctx.c2t_launch_count() - n1 == 1 + D + 1 + 1 + 2
    ctx.close()


def test_fused_and_separate_calls_agree_bit_for_bit():
    B, V, D, K, F, N = 2, 128256, 10, 8, 16, 80
    _, gcfg = make_configs(B, V, D, K, F, N, 0.3, torch.bfloat16)
    Nw = c2t.c2t_final_width(gcfg)
    draft, target, root, prefix = gen_inputs(B, V, D, F, Nw, torch.bfloat16)
    draft = [t.cuda() for t in draft]; target = target.cuda(); root = root.cuda(); prefix = prefix.cuda()
    ctx = c2t.Context(gcfg)
    snaps = []
    for fused in (False, True, True):
        ctx.c2t_begin_step(root, prefix)
        for l in range(D):
            if fused:
                ctx.c2t_expand_prune_level(l, draft[l])
            else:
                ctx.c2t_expand_level(l, draft[l]); ctx.c2t_prune(l)
        ctx.c2t_prune(c2t.FINAL); ctx.c2t_build_verify(); ctx.c2t_accept(target)
        torch.cuda.synchronize()
        v = ctx.c2t_get_view()
        n = v["tree_n"].clone()
        live = torch.arange(ctx.cap, device="cuda")[None, :] < n[:, None]
        snaps.append([n, torch.where(live, v["tree_token"], 0), torch.where(live, v["tree_parent"], 0),
                      torch.where(live, v["tree_logP"], 0.0), torch.where(live, v["tree_C"], 0.0),
                      v["cand_flags"].clone(), ctx.frontier["count"].clone(), ctx.frontier["token"].clone(),
                      ctx.verify["mask_bits"].clone(), ctx.verify["retrieve"].clone(), ctx.accepted["path"].clone()])
    assert int(snaps[0][0].max()) > 1
    for other in snaps[1:]:
        for a, b in zip(snaps[0], other):
            assert torch.equal(a, b)
    ctx.close()


def test_config2_batch8_bf16_several_steps():
    # the full configuration runs 64 decode steps; the oracle needs seconds per step, so a few here
    nodes = []
    for step in range(3):
        rep = case(8, 32000, 8, 10, 10, 60, 0.5, torch.bfloat16, step=step)
        nodes += rep.kept_nodes
    assert max(nodes) > 1


def test_config2_chained_64_steps():
    """B=8, V=32000, bf16, D=8, K=F=10, N=60: 64 decode steps in which every step starts from the
    previous step's next token and grown prefix; two of the eight sequences are checked against the
    oracle at every step (the oracle needs seconds per sequence and step)."""
    ocfg, gcfg = make_configs(8, 32000, 8, 10, 10, 60, 0.5, torch.bfloat16)
    rep = run_chain(ocfg, gcfg, 64, seqs=[1, 6])
    print(f"\n  [config 2, 64 chained steps] {rep.line()}")
    assert len(rep.accept_len) == 2 * 64 and rep.accept_len == rep.oracle_accept_len
    assert rep.kept_nodes == rep.oracle_kept_nodes and max(rep.kept_nodes) > 1


# The ablation sweep's corner points at full batch: classifier (identity on the joint probability, i.e.
# EAGLE-2's expand + rerank, against the FFN), both vocabularies and dtypes, the smallest and largest budget,
# the deepest tree, the flattest and the most peaked logits.  Sampled sequences, as for the throughput case.
@pytest.mark.parametrize("V,dtype,classifier,N,scale", [
    (128256, torch.float32, "identity", 20, 1.0),
    (128256, torch.bfloat16, "mlp", 80, 8.0),
    (128256, torch.bfloat16, "identity", 80, 1.0),
    (32000, torch.float32, "mlp", 20, 8.0),
    (32000, torch.bfloat16, "identity", 80, 8.0),
])
def test_config5_ablation_corners_sampled(V, dtype, classifier, N, scale):
    B, D, K, F = 32, 10, 10, 10
    beta = 0.5 if classifier == "mlp" else 0.0
    ocfg, gcfg = make_configs(B, V, D, K, F, N, beta, dtype, classifier=classifier)
    Nw = c2t.c2t_final_width(gcfg)
    draft, target, root, prefix = gen_inputs(B, V, D, F, Nw, dtype, scale=scale, device="cuda")
    rep = run_and_compare(ocfg, gcfg, None, None, root, prefix, seqs=[0, 17], draft_dev=draft, target_dev=target)
    print(f"\n  [config 5: V={V} {dtype} {classifier} N={N} scale={scale}] {rep.line()}")
    assert rep.status_bits == 0 and rep.kept_nodes == rep.oracle_kept_nodes


@pytest.mark.parametrize("beta", [0.3, 0.5, 0.7])
def test_config3_llama3_vocab_single_sequence(beta):
    case(1, 128256, 10, 8, 16, 80, beta, torch.bfloat16)


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("classifier,tree_add,beta", [("mlp", "frontier", 0.5), ("identity", "all", 0.0)])
def test_ablation_shapes(dtype, classifier, tree_add, beta):
    for scale in (1.0, 8.0):
        case(4, 32000, 6, 10, 10, 40, beta, dtype, scale=scale, classifier=classifier, tree_add=tree_add)


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("V", [5003, 8191, 1000, 37])
def test_ragged_vocab_and_padded_stride(dtype, V):
    B, D, K, F, N = 3, 4, 6, 5, 18
    ocfg, gcfg = make_configs(B, V, D, K, F, N, 0.5, dtype, wseed=2)
    Nw = c2t.c2t_final_width(gcfg)
    draft, target, root, prefix = gen_inputs(B, V, D, F, Nw, dtype)
    Vp = (V + 31) // 32 * 32 + 32
    dev = torch.device("cuda", 0)

    def padded(t):
        buf = torch.full((t.shape[0], t.shape[1], Vp), float("nan"), dtype=dtype, device=dev)
        buf[:, :, :V] = t.to(dev)
        return buf[:, :, :V]                    # row stride Vp > V; the padding is NaN and must never be read

    rep = run_and_compare(ocfg, gcfg, draft, target, root, prefix,
                          draft_dev=[padded(t) for t in draft], target_dev=padded(target))
    assert rep.status_bits == 0


def test_chain_mode_k1_f1():
    case(4, 32000, 8, 1, 1, 0, 0.45, torch.bfloat16, wseed=5)


@pytest.mark.parametrize("rule,thr", [("cond", 0.3), ("identity", 0.08), ("mlp", 0.5)])
def test_chain_mode_stop_rules(rule, thr):
    """K = F = 1 with the three early-stop rules of the chain-mode comparison (Sec. 5): maximum
    probability, joint probability, the classifier.  Chains end at different depths per sequence."""
    rep = case(8, 32000, 10, 1, 1, 0, thr, torch.bfloat16, scale=1.5, classifier=rule, wseed=5)
    assert len(set(rep.kept_nodes)) >= 2


def test_beta_zero_keeps_everything_beta_one_stops_at_root():
    rep = case(2, 4096, 5, 4, 4, 0, 0.0, torch.float32)
    assert rep.kept_nodes == [1 + 4 + 4 * 4] * 2
    rep = case(2, 4096, 5, 4, 4, 0, 1.0, torch.float32)
    assert rep.kept_nodes == [1, 1] and rep.accept_len == [0, 0]


def test_budget_smaller_and_larger_than_tree():
    case(2, 4096, 5, 4, 4, 7, 0.0, torch.float32, classifier="identity", tree_add="all")
    case(2, 4096, 5, 4, 4, 1, 0.0, torch.float32)
    case(2, 4096, 5, 4, 4, 500, 0.0, torch.float32, classifier="identity", tree_add="all")


def test_eagle2_complete_tree_1011_nodes():
    rep = case(1, 2048, 11, 10, 10, 0, 0.0, torch.float32, scale=1.0, classifier="identity", tree_add="all")
    assert rep.kept_nodes == [1011]


def test_zero_weights_every_confidence_ties():
    case(2, 8000, 4, 5, 3, 10, 0.5, torch.bfloat16, wstd=0.0)


def test_wide_limits_k32_f32_h64():
    case(1, 16384, 3, 32, 32, 100, 0.5, torch.bfloat16, hidden=64, wseed=4)


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("kind", ["uniform", "two_valued", "heavy_ties", "neg_inf", "peaked", "rising", "late_jump"])
def test_special_rows(kind, dtype):
    B, V, D, K, F, N = 2, 20000, 3, 5, 4, 12
    ocfg, gcfg = make_configs(B, V, D, K, F, N, 0.0, dtype, classifier="identity")
    Nw = c2t.c2t_final_width(gcfg)
    draft = [special_rows(kind, B, F, V, dtype) for _ in range(D)]
    target = special_rows(kind, B, Nw, V, dtype)
    root = torch.zeros(B, dtype=torch.int32); prefix = torch.full((B,), 9, dtype=torch.int32)
    # all-equal rows make the confidences of children of different rows exactly equal in the oracle, which
    # orders them by candidate index; the CUDA path's fp32 row sums depend on where a row is cut into
    # segments, so there the order follows the last bits of two sums: the one named departure
    uniform = dict(allow_diverged=B, allow_kinds=("cross_row_tie",)) if kind == "uniform" else {}
    rep = run_and_compare(ocfg, gcfg, draft, target, root, prefix, **uniform)
    print(f"\n  [{kind} {dtype}] {rep.line()}")
    assert rep.status_bits == 0
    if kind == "uniform":
        ctx = c2t.Context(gcfg)
        ctx.c2t_begin_step(root.cuda(), prefix.cuda())
        ctx.c2t_expand_level(0, draft[0].cuda()); ctx.c2t_prune(0)
        H = ctx.c2t_get_view()["cand_H"][:, 0].cpu().numpy()
        assert np.allclose(H, math.log(V), rtol=RTOL[dtype], atol=0)
        ctx.close()


@pytest.mark.parametrize("fault,bit", [(float("nan"), c2t.ST_NAN_LOGIT), (float("inf"), c2t.ST_POSINF_LOGIT),
                                       ("all_neg_inf", c2t.ST_ALL_NEGINF)])
def test_data_faults_set_status_and_spare_other_sequences(fault, bit):
    B, V, D, K, F, N = 3, 9000, 3, 4, 4, 10
    dtype = torch.bfloat16
    ocfg, gcfg = make_configs(B, V, D, K, F, N, 0.5, dtype)
    Nw = c2t.c2t_final_width(gcfg)
    draft, target, root, prefix = gen_inputs(B, V, D, F, Nw, dtype)
    if fault == "all_neg_inf":
        draft[0][1, 0, :] = float("-inf")
    else:
        draft[0][1, 0, 4321] = fault                  # sequence 1, the root's row
    ctx = c2t.Context(gcfg)
    rep = run_and_compare(ocfg, gcfg, draft, target, root, prefix, seqs=[0, 2], ctx=ctx)
    bits, per = ctx.c2t_status()
    assert per[0] == 0 and per[2] == 0 and (per[1] & bit)
    n = ctx.verify["n_nodes"].cpu().numpy()
    assert n[1] == 1                                  # the faulted sequence keeps only its root
    assert rep.diverged_sequences == 0
    ctx.close()


def test_call_order_and_alignment_errors():
    B, V, D = 2, 1024, 3
    _, gcfg = make_configs(B, V, D, 4, 4, 10, 0.5, torch.float32)
    ctx = c2t.Context(gcfg)
    lg = torch.zeros(B, 4, V, device="cuda")
    root = torch.zeros(B, dtype=torch.int32, device="cuda")

    def code(fn, *a):
        with pytest.raises(c2t.C2TError) as e:
            fn(*a)
        return e.value.code

    assert code(ctx.c2t_expand_level, 0, lg) == c2t.EORDER            # before begin_step
    ctx.c2t_begin_step(root, root)
    assert code(ctx.c2t_prune, 0) == c2t.EORDER                       # nothing expanded yet
    assert code(ctx.c2t_expand_level, 1, lg) == c2t.EORDER            # wrong level
    assert code(ctx.c2t_build_verify) == c2t.EORDER
    tg0 = torch.zeros(B, ctx.Nw, V, device="cuda")
    assert code(ctx.c2t_accept, tg0) == c2t.EORDER                    # no final tree yet
    assert code(ctx.c2t_accept_lazy, tg0) == c2t.EORDER
    assert code(ctx.c2t_dense_mask, torch.zeros(B, ctx.Nw, 64, device="cuda")) == c2t.EORDER
    odd = torch.zeros(B * 4 * V + 8, device="cuda")[1:1 + B * 4 * V].view(B, 4, V)
    assert code(ctx.c2t_expand_level, 0, odd) == c2t.EALIGN
    ctx.c2t_expand_level(0, lg)
    assert code(ctx.c2t_expand_level, 0, lg) == c2t.EORDER            # twice
    assert code(ctx.c2t_prune, c2t.FINAL) == c2t.EORDER               # level 0 not pruned yet
    ctx.c2t_prune(0)
    ctx.c2t_prune(c2t.FINAL)                                          # fewer than D levels is allowed
    assert code(ctx.c2t_expand_level, 1, lg) == c2t.EORDER            # step is final
    ctx.c2t_build_verify()
    ctx.c2t_accept(tg0)
    torch.cuda.synchronize()
    first = {k: v.clone() for k, v in ctx.accepted.items()}
    ctx.c2t_accept_lazy(tg0)                                          # all-zero rows: arg-max is token 0 everywhere
    torch.cuda.synchronize()
    for k, v in ctx.accepted.items():
        assert torch.equal(v, first[k]), k
    odd_t = torch.zeros(B * ctx.Nw * V + 8, device="cuda")[1:1 + B * ctx.Nw * V].view(B, ctx.Nw, V)
    assert code(ctx.c2t_accept_lazy, odd_t) == c2t.EALIGN
    ctx.close()


def test_results_are_reproducible():
    """Everything repeats bit for bit, the floating-point results included: every warp of the
    vocabulary pass works on its own span in a fixed order and the merge adds the partial records
    in slot order, so no sum depends on timing."""
    B, V, D, K, F, N = 8, 32000, 4, 10, 10, 30
    _, gcfg = make_configs(B, V, D, K, F, N, 0.5, torch.bfloat16)
    Nw = c2t.c2t_final_width(gcfg)
    draft, target, root, prefix = gen_inputs(B, V, D, F, Nw, torch.bfloat16)
    draft = [t.cuda() for t in draft]; target = target.cuda(); root = root.cuda(); prefix = prefix.cuda()
    ctx = c2t.Context(gcfg)
    snaps = []
    for _ in range(3):
        ctx.decode_step(draft, target, root, prefix)
        torch.cuda.synchronize()
        v = ctx.c2t_get_view()
        n = v["tree_n"].clone()
        live = torch.arange(ctx.cap, device="cuda")[None, :] < n[:, None]
        ints = [n, torch.where(live, v["tree_token"], 0), torch.where(live, v["tree_parent"], 0),
                v["cand_flags"].clone(), ctx.verify["mask_bits"].clone(), ctx.verify["retrieve"].clone(),
                ctx.accepted["path"].clone(), ctx.accepted["next_token"].clone()]
        floats = [torch.where(live, v["tree_logP"], 0.0), torch.where(live, v["tree_C"], 0.0)]
        snaps.append((ints, floats))
    for ints, floats in snaps[1:]:
        for a, b in zip(snaps[0][0], ints):
            assert torch.equal(a, b)
        for a, b in zip(snaps[0][1], floats):
            assert torch.equal(a, b)
    ctx.close()


def test_back_to_back_steps_equal_isolated_steps():
    """Steps queued without any host synchronisation give what the same steps give one at a time.
    The kernels of a step are launched so that each may be placed on the SMs while its predecessor is
    still finishing and waits for it before its first access to memory; a kernel that ran ahead of
    that wait would read the other input set's frontier or partial records here."""
    B, V, D, K, F, N = 8, 32000, 5, 10, 10, 40
    _, gcfg = make_configs(B, V, D, K, F, N, 0.5, torch.bfloat16)
    Nw = c2t.c2t_final_width(gcfg)
    sets = []
    for step in (0, 1):
        draft, target, root, prefix = gen_inputs(B, V, D, F, Nw, torch.bfloat16, step=step)
        sets.append(([t.cuda() for t in draft], target.cuda(), root.cuda(), prefix.cuda()))
    ctx = c2t.Context(gcfg)

    def snapshot():                                      # device-side copies in stream order, no synchronisation
        v = ctx.c2t_get_view()
        n = v["tree_n"].clone()
        live = torch.arange(ctx.cap, device="cuda")[None, :] < n[:, None]
        return [n, torch.where(live, v["tree_token"], 0), torch.where(live, v["tree_parent"], 0),
                torch.where(live, v["tree_logP"], 0.0), torch.where(live, v["tree_C"], 0.0),
                ctx.verify["mask_bits"].clone(), ctx.verify["retrieve"].clone(),
                ctx.accepted["accept_len"].clone(), ctx.accepted["path"].clone(), ctx.accepted["next_token"].clone()]

    alone = []
    for inp in sets:
        ctx.decode_step(*inp)
        torch.cuda.synchronize()
        alone.append(snapshot())
        torch.cuda.synchronize()
    assert not all(torch.equal(a, b) for a, b in zip(alone[0], alone[1]))     # the two sets do differ
    queued = []
    for i in range(24):                                  # no synchronisation inside this loop
        ctx.decode_step(*sets[i & 1])
        queued.append(snapshot())
    torch.cuda.synchronize()
    for i, snap in enumerate(queued):
        for a, b in zip(alone[i & 1], snap):
            assert torch.equal(a, b), i
    ctx.close()


@pytest.mark.parametrize("dtype,V,M", [(torch.bfloat16, 32000, 1000), (torch.float32, 32000, 1000),
                                       (torch.bfloat16, 5000, 100), (torch.float32, 4096, 5),
                                       (torch.bfloat16, 3000, 3000), (torch.float32, 3000, 7000)])
def test_truncated_entropy_top_m(dtype, V, M):
    """Eq. 3: the entropy feature over the M most probable tokens only (the paper's M = 1000), full
    softmax probabilities; M >= V is the exact entropy again."""
    case(4, V, 4, 8, 6, 24, 0.5, dtype, M=M)


@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32])
def test_truncated_entropy_comes_from_the_expand_pass(dtype):
    """At the paper's vocabulary and M = 1000 the rows are read once: the pass sets the vectors aside that can hold
    one of the M most probable tokens and Eq. 3's sums are taken from those (the view says for which rows)."""
    rep = case(3, 128256, 3, 10, 8, 30, 0.0, dtype, M=1000, classifier="identity")
    assert rep.rows_expanded == 3 * (1 + 8 + 8)
    assert rep.rows_topm_from_pass >= 0.9 * rep.rows_expanded, (rep.rows_topm_from_pass, rep.rows_expanded)


def test_truncated_entropy_rows_the_pass_cannot_serve_are_read_again():
    """M close to V: fewer than M elements reach the floor above which the pass sets vectors aside, so every row
    takes the second read (rows of equal values, where the regions run full, are among the special rows below)."""
    rep = case(2, 6000, 2, 4, 4, 12, 0.0, torch.float32, M=4500, classifier="identity")
    assert rep.rows_expanded == 2 * (1 + 4) and rep.rows_topm_from_pass == 0


@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32])
def test_truncated_entropy_with_both_routes_in_one_step(dtype):
    """A small vocabulary with M = 64: some rows are served from the vectors the pass set aside, the others are
    read again, within the same launches."""
    rep = case(3, 1000, 3, 8, 6, 20, 0.0, dtype, M=64, classifier="identity")
    assert 0 < rep.rows_topm_from_pass < rep.rows_expanded, (rep.rows_topm_from_pass, rep.rows_expanded)


@pytest.mark.parametrize("kind", ["heavy_ties", "two_valued", "neg_inf", "uniform"])
def test_truncated_entropy_on_special_rows(kind):
    """Many equal values around the M-th largest: equal values give equal terms, so only the count matters."""
    B, V, D, K, F, N = 2, 20000, 2, 5, 4, 10
    dtype = torch.bfloat16
    ocfg, gcfg = make_configs(B, V, D, K, F, N, 0.0, dtype, classifier="identity", M=700)
    Nw = c2t.c2t_final_width(gcfg)
    draft = [special_rows(kind, B, F, V, dtype) for _ in range(D)]
    target = special_rows(kind, B, Nw, V, dtype)
    root = torch.zeros(B, dtype=torch.int32); prefix = torch.full((B,), 9, dtype=torch.int32)
    uniform = dict(allow_diverged=B, allow_kinds=("cross_row_tie",)) if kind == "uniform" else {}
    rep = run_and_compare(ocfg, gcfg, draft, target, root, prefix, **uniform)
    assert rep.status_bits == 0
    if kind == "uniform":                # every vector reaches the floor: more than the pass has room for
        assert rep.rows_topm_from_pass == 0


@pytest.mark.parametrize("out_dtype", [torch.float32, torch.bfloat16])
def test_dense_mask_matches_oracle(out_dtype):
    B, V, D, K, F, N = 5, 6000, 5, 4, 4, 18
    dtype = torch.bfloat16
    ocfg, gcfg = make_configs(B, V, D, K, F, N, 0.3, dtype)
    Nw = c2t.c2t_final_width(gcfg)
    draft, target, root, prefix = gen_inputs(B, V, D, F, Nw, dtype)
    ctx = c2t.Context(gcfg)
    ctx.c2t_begin_step(root.cuda(), prefix.cuda())
    for l in range(D):
        ctx.c2t_expand_level(l, draft[l].cuda()); ctx.c2t_prune(l)
    ctx.c2t_prune(c2t.FINAL)
    for kv_len in (int(prefix.max()) + Nw, int(prefix.max()) + Nw + 13, int(prefix.min()) + 3):   # exact, padded, clipped
        out = torch.full((B, Nw, kv_len), 7.0, dtype=out_dtype, device="cuda")
        ctx.c2t_dense_mask(out)
        got = out.float().cpu().numpy()
        for b in range(B):
            lg = torch.stack([draft[l][b] for l in range(D)])
            tree, _ = oracle.build_tree(ocfg, lg, int(root[b]))
            ft = oracle.final_prune(tree, N)
            want = oracle.dense_mask(ft, int(prefix[b]), Nw, kv_len)
            assert np.array_equal(got[b], want), (b, kv_len)
    with pytest.raises(c2t.C2TError):
        ctx.c2t_dense_mask(torch.zeros(B, Nw, 0, device="cuda"))
    ctx.close()


def test_lazy_accept_follows_planted_paths():
    """Target rows whose arg-max is planted on a root-to-leaf chain of the final tree: both
    acceptance calls must walk the whole chain, and the lazy one must not look anywhere else."""
    B, V, D, K, F, N = 6, 9000, 5, 4, 4, 20
    dtype = torch.bfloat16
    _, gcfg = make_configs(B, V, D, K, F, N, 0.0, dtype, classifier="identity")
    Nw = c2t.c2t_final_width(gcfg)
    draft, target, root, prefix = gen_inputs(B, V, D, F, Nw, dtype)
    ctx = c2t.Context(gcfg)
    ctx.c2t_begin_step(root.cuda(), prefix.cuda())
    for l in range(D):
        ctx.c2t_expand_level(l, draft[l].cuda()); ctx.c2t_prune(l)
    ctx.c2t_prune(c2t.FINAL); ctx.c2t_build_verify()
    torch.cuda.synchronize()
    ver = {k: v.cpu().numpy() for k, v in ctx.verify.items()}
    planted = []
    for b in range(B):
        rows = ver["retrieve"][b, :ver["n_leaves"][b]]
        chain = [int(x) for x in rows[b % len(rows)] if x >= 0]          # a different leaf per sequence
        for here, nxt in zip(chain, chain[1:]):
            target[b, here, int(ver["tokens"][b, nxt])] = 100.0
        if len(chain) < D + 1:                                           # the leaf's own arg-max: a token no child has
            target[b, chain[-1], V - 1 - b] = 100.0
        planted.append(chain)
    tg = target.cuda()
    ctx.c2t_accept(tg); torch.cuda.synchronize()
    full = {k: v.cpu().numpy().copy() for k, v in ctx.accepted.items()}
    amax_full = ctx.c2t_get_view()["node_argmax"].cpu().numpy().copy()
    ctx.c2t_accept_lazy(tg); torch.cuda.synchronize()
    lazy = {k: v.cpu().numpy() for k, v in ctx.accepted.items()}
    amax_lazy = ctx.c2t_get_view()["node_argmax"].cpu().numpy()
    lazy = {k: v.copy() for k, v in lazy.items()}; amax_lazy = amax_lazy.copy()
    # the same walk over target rows sharded into three token ranges (the planted tokens fall into different ranges)
    shards = [(0, 2000), (2000, 6000), (6000, V)]
    keys = torch.zeros((len(shards), B), dtype=torch.int64, device="cuda")
    ctx.c2t_lazy_begin()
    for r in range(1, D + 2):
        for g, (v0, v1) in enumerate(shards):
            ctx.c2t_lazy_argmax_shard(tg[:, :, v0:v1], v0, keys[g])
        ctx.c2t_lazy_step_gathered(r, keys)
    torch.cuda.synchronize()
    lazy_s = {k: v.cpu().numpy() for k, v in ctx.accepted.items()}
    amax_lazy_s = ctx.c2t_get_view()["node_argmax"].cpu().numpy()
    for b, chain in enumerate(planted):
        assert full["accept_len"][b] == len(chain) - 1 == lazy["accept_len"][b] == lazy_s["accept_len"][b]
        assert [x for x in full["path"][b] if x >= 0] == chain == [x for x in lazy["path"][b] if x >= 0]
        assert [x for x in lazy_s["path"][b] if x >= 0] == chain
        assert full["next_token"][b] == lazy["next_token"][b] == lazy_s["next_token"][b]
        for i in range(Nw):
            assert amax_lazy[b, i] == (amax_full[b, i] if i in chain else -1)
            assert amax_lazy_s[b, i] == amax_lazy[b, i]
        # against the oracle: the arg-max of every row on the path, one by one
        for i in chain:
            assert amax_full[b, i] == oracle.row_argmax(target[b, i])
    assert max(len(c) for c in planted) >= 3
    ctx.close()


def test_decode_step_host_matches_device_path():
    B, V, D, K, F, N = 4, 12000, 4, 6, 5, 16
    _, gcfg = make_configs(B, V, D, K, F, N, 0.5, torch.bfloat16)
    Nw = c2t.c2t_final_width(gcfg)
    draft, target, root, prefix = gen_inputs(B, V, D, F, Nw, torch.bfloat16)
    ctx = c2t.Context(gcfg)
    ctx.decode_step([t.cuda() for t in draft], target.cuda(), root.cuda(), prefix.cuda())
    torch.cuda.synchronize()
    want = {"n_nodes": ctx.verify["n_nodes"].cpu(), "tokens": ctx.verify["tokens"].cpu(),
            "accept_len": ctx.accepted["accept_len"].cpu(), "path": ctx.accepted["path"].cpu(),
            "next_token": ctx.accepted["next_token"].cpu()}
    stage, results = ctx.host_step_buffers()
    ctx.c2t_decode_step_host([t.pin_memory() for t in draft], target.pin_memory(), root.pin_memory(),
                             prefix.pin_memory(), results, stage)
    for k, w in want.items():
        assert torch.equal(results[k], w), k
    assert ctx.c2t_launch_count() == 2 * (1 + 2 * D + 1 + 1 + 2)
    ctx.close()


def test_config4_full_size_sampled_against_oracle():
    """B=64, V=128256, bf16, D=8, K=F=10, N=60 in the launch shape the benchmark times; the oracle
    checks three sampled sequences end to end, and properties that hold at any size cover the rest."""
    B, V, D, K, F, N = 64, 128256, 8, 10, 10, 60
    dtype = torch.bfloat16
    ocfg, gcfg = make_configs(B, V, D, K, F, N, 0.5, dtype)
    Nw = c2t.c2t_final_width(gcfg)
    draft, target, root, prefix = gen_inputs(B, V, D, F, Nw, dtype, device="cuda")
    ctx = c2t.Context(gcfg)
    rep = run_and_compare(ocfg, gcfg, None, None, root, prefix, seqs=[0, 31, 63], ctx=ctx,
                          draft_dev=draft, target_dev=target)
    print(f"\n  [config 4 sampled] {rep.line()}")
    assert rep.status_bits == 0
    v = {k: t.cpu().numpy() for k, t in ctx.verify.items()}
    acc = {k: t.cpu().numpy() for k, t in ctx.accepted.items()}
    for b in range(B):
        n = v["n_nodes"][b]
        assert 1 <= n <= N
        par = v["parents"][b, :n]
        assert par[0] == -1 and (par[1:] < np.arange(1, n)).all() and (par[1:] >= 0).all()
        for i in range(n):
            bits = int(v["mask_bits"][b, i, 0])
            assert bits >> i & 1 and (i == 0 or bits == int(v["mask_bits"][b, par[i], 0]) | 1 << i)
            assert v["position_ids"][b, i] == prefix[b] + bin(bits).count("1") - 1
        sib = {}
        for i in range(1, n):
            assert (par[i], v["tokens"][b, i]) not in sib      # siblings carry distinct tokens
            sib[(par[i], v["tokens"][b, i])] = i
        path = [x for x in acc["path"][b] if x >= 0]
        assert len(path) == acc["accept_len"][b] + 1 and path[0] == 0
        for a, c in zip(path, path[1:]):
            assert par[c] == a
    # target argmax of sampled rows, one by one
    amax = ctx.c2t_get_view()["node_argmax"].cpu().numpy()
    for b, i in [(5, 0), (17, 3), (40, 59), (63, 30)]:
        if i < v["n_nodes"][b]:
            assert amax[b, i] == oracle.row_argmax(target[b, i].cpu())
    ctx.close()

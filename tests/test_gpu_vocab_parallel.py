"""Vocabulary-parallel levels against the whole-row oracle.  With one GPU the token ranges are
processed one after the other through the same three calls a rank would make (sharded pass,
record export, prune from the gathered records); no kernel waits for another."""
import pytest
import torch

import paper_2502_13652_b200 as c2t
from parity_util import gen_inputs, make_configs, run_and_compare, special_rows

pytestmark = pytest.mark.gpu


def even_shards(V, G, step=8):
    cuts = [min(V, (V * g // G) // step * step) for g in range(G)] + [V]
    return [(cuts[g], cuts[g + 1]) for g in range(G)]


@pytest.mark.parametrize("dtype,V,shards", [
    (torch.bfloat16, 32000, even_shards(32000, 4)),
    (torch.float32, 32000, [(0, 20000), (20000, 32000)]),
    (torch.bfloat16, 128256, even_shards(128256, 8)),
    (torch.float32, 4096, even_shards(4096, 32)),            # the largest shard count, 128 tokens apiece
    (torch.bfloat16, 32000, [(0, 32000)]),                   # one shard: the records carry a whole row
])
def test_sharded_levels_match_whole_rows(dtype, V, shards):
    B, D, K, F, N = 4, 4, 10, 6, 30
    ocfg, gcfg = make_configs(B, V, D, K, F, N, 0.5, dtype)
    Nw = c2t.c2t_final_width(gcfg)
    draft, target, root, prefix = gen_inputs(B, V, D, F, Nw, dtype)
    rep = run_and_compare(ocfg, gcfg, draft, target, root, prefix, shards=shards)
    print(f"\n  [{len(shards)} shards of {V} {dtype}] {rep.line()}")
    assert rep.status_bits == 0


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("V,shards", [(5003, [(0, 2000), (2000, 5003)]), (37, [(0, 8), (8, 16), (16, 37)])])
def test_sharded_ragged_rows_and_short_shards(dtype, V, shards):
    """A last shard whose length is not a whole number of 16-byte vectors, rows with a padded stride, and
    shards with fewer tokens than K."""
    B, D, K, F, N = 3, 4, 10, 5, 18
    ocfg, gcfg = make_configs(B, V, D, K, F, N, 0.5, dtype, wseed=2)
    Nw = c2t.c2t_final_width(gcfg)
    draft, target, root, prefix = gen_inputs(B, V, D, F, Nw, dtype)
    Vp = (V + 31) // 32 * 32 + 32
    dev = torch.device("cuda", 0)

    def padded(t):
        buf = torch.full((t.shape[0], t.shape[1], Vp), float("nan"), dtype=dtype, device=dev)
        buf[:, :, :V] = t.to(dev)
        return buf[:, :, :V]

    rep = run_and_compare(ocfg, gcfg, draft, target, root, prefix, draft_dev=[padded(t) for t in draft],
                          target_dev=padded(target), shards=shards)
    assert rep.status_bits == 0


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("kind", ["uniform", "two_valued", "heavy_ties", "neg_inf", "peaked", "late_jump"])
def test_sharded_special_rows(kind, dtype):
    """Ties that span shards go to the lower token id, a shard that is all -inf contributes nothing
    (neg_inf: the first half of every row), a maximum in the last shard dwarfs the others (late_jump)."""
    B, V, D, K, F, N = 2, 20000, 3, 5, 4, 12
    ocfg, gcfg = make_configs(B, V, D, K, F, N, 0.0, dtype, classifier="identity")
    Nw = c2t.c2t_final_width(gcfg)
    draft = [special_rows(kind, B, F, V, dtype) for _ in range(D)]
    target = special_rows(kind, B, Nw, V, dtype)
    root = torch.zeros(B, dtype=torch.int32); prefix = torch.full((B,), 9, dtype=torch.int32)
    uniform = dict(allow_diverged=B, allow_kinds=("cross_row_tie",)) if kind == "uniform" else {}
    rep = run_and_compare(ocfg, gcfg, draft, target, root, prefix, shards=even_shards(V, 4), **uniform)
    print(f"\n  [{kind} {dtype}] {rep.line()}")
    assert rep.status_bits == 0


def test_sharded_faults_and_call_order():
    B, V, D, K, F, N = 2, 4096, 3, 5, 4, 12
    _, gcfg = make_configs(B, V, D, K, F, N, 0.5, torch.float32)
    Nw = c2t.c2t_final_width(gcfg)
    draft, target, root, prefix = gen_inputs(B, V, D, F, Nw, torch.float32)
    x = draft[0].cuda()
    x[1, 0, 3000] = float("nan")                                     # sequence 1, second shard
    ctx = c2t.Context(gcfg)
    rec = ctx.new_row_records(2)
    ctx.c2t_begin_step(root.cuda(), prefix.cuda())

    def err(fn, *a, **k):
        with pytest.raises(c2t.C2TError) as e:
            fn(*a, **k)
        return e.value.code

    assert err(ctx.c2t_export_row_records, 0, 0, rec[0]) == c2t.EORDER          # nothing to export yet
    ctx.c2t_expand_level_shard(0, x[:, :, :2048])
    assert err(ctx.c2t_prune, 0) == c2t.EORDER                                  # a sharded pass is not a whole one
    assert err(ctx.c2t_prune_gathered, 0, rec) == c2t.EORDER                    # the export comes first
    assert err(ctx.c2t_expand_level, 0, x) == c2t.EORDER
    assert err(ctx.c2t_export_row_records, 0, 2049, rec[0]) == c2t.EINVAL       # range past the vocabulary
    ctx.c2t_export_row_records(0, 0, rec[0])
    ctx.c2t_expand_level_shard(0, x[:, :, 2048:])
    ctx.c2t_export_row_records(0, 2048, rec[1])
    assert err(ctx.c2t_prune_gathered, 1, rec) == c2t.EORDER                    # wrong level
    big = torch.zeros((33,) + tuple(rec.shape[1:]), dtype=torch.uint8, device="cuda")
    assert err(ctx.c2t_prune_gathered, 0, big) == c2t.ERANGE
    ctx.c2t_prune_gathered(0, rec)
    bits, per = ctx.c2t_status()
    assert per[0] == 0 and per[1] & c2t.ST_NAN_LOGIT                            # the fault stays with its sequence
    keys = torch.zeros((2, B, ctx.Nw), dtype=torch.int64, device="cuda")
    tgt = target.cuda()
    assert err(ctx.c2t_argmax_shard, tgt[:, :, :2048], 0, keys[0]) == c2t.EORDER   # the tree is not final yet
    assert err(ctx.c2t_accept_gathered, keys) == c2t.EORDER
    ctx.c2t_prune(c2t.FINAL)
    assert err(ctx.c2t_argmax_shard, tgt[:, :, :2048], 2056, keys[0]) == c2t.EINVAL   # range past the vocabulary
    ctx.c2t_argmax_shard(tgt[:, :, :2048], 0, keys[0])
    ctx.c2t_argmax_shard(tgt[:, :, 2048:], 2048, keys[1])
    ctx.c2t_accept_gathered(keys)
    big_keys = torch.zeros((33, B, ctx.Nw), dtype=torch.int64, device="cuda")
    assert err(ctx.c2t_accept_gathered, big_keys) == c2t.ERANGE
    ctx.close()

    _, mcfg = make_configs(B, V, D, K, F, N, 0.5, torch.float32, M=100)
    ctx = c2t.Context(mcfg)
    ctx.c2t_begin_step(root.cuda(), prefix.cuda())
    assert err(ctx.c2t_expand_level_shard, 0, x[:, :, :2048]) == c2t.EINVAL     # Eq. 3 needs whole rows
    ctx.close()

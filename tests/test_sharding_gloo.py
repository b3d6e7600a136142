"""The N > 1 path of the benchmark on CPU: two gloo ranks.

Sequences are independent, so the multi-GPU run shards them with no collective on the data path:
every rank owns a disjoint block of sequences and the only communication is the barrier and the
max-over-ranks of the timing.  This test runs that host logic with world_size 2 over gloo and lets
each rank push its own sequences through the oracle to show the shards really are different work.
"""
import os
import sys

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank: int, world: int, port: int, out):
    sys.path.insert(0, ROOT)
    import bench
    import c2t_inputs
    import oracle

    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    B, V, D, K, F, N = 2, 512, 3, 4, 3, 8
    base = bench.rank_sequence_base(rank, B)
    draft = torch.stack([c2t_inputs.draft_logits(B, F, V, 0, l, torch.float32, seq_base=base) for l in range(D)], dim=1)
    target = c2t_inputs.target_logits(B, N, V, 0, torch.float32, seq_base=base)
    w1, b1, w2, b2 = c2t_inputs.classifier_weights(8)
    cfg = oracle.OracleConfig(vocab=V, max_depth=D, topk=K, frontier_cap=F, budget=N, threshold=0.45, hidden=8,
                              w1=w1, b1=b1, w2=w2, b2=b2)
    r = oracle.decode_step(cfg, draft.contiguous(), target, c2t_inputs.root_tokens(B, V, 0, base).numpy(),
                           c2t_inputs.prefix_lengths(B, seq_base=base).numpy())
    dist.barrier()
    ms = 10.0 + 5.0 * rank                                   # rank 1 is the slow one
    slowest = bench.max_over_ranks(ms, dist)
    tokens = torch.from_numpy(r.tokens.astype(np.int64))
    gathered = [torch.zeros_like(tokens) for _ in range(world)]
    dist.all_gather(gathered, tokens)                        # test-only: to compare the shards
    if rank == 0:
        out.put({"slowest": slowest, "base": base,
                 "value": bench.whole_job_levels_per_second(world, B, D, slowest),
                 "tokens": [g.numpy() for g in gathered]})
    dist.destroy_process_group()


def test_two_ranks_shard_sequences_and_time_by_the_slowest():
    oracle_dir = os.path.join(ROOT, "oracle")
    sys.path.insert(0, ROOT)
    import oracle
    oracle.build()                                           # once, before the ranks race to build it
    import bench
    import c2t_inputs
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = 29500 + os.getpid() % 2000
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    res = out.get(timeout=120)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert res["slowest"] == 15.0                            # the max over ranks, not rank 0's own 10.0
    assert res["value"] == 2 * 2 * 3 / 15.0e-3               # whole-job figure counts both ranks' sequences
    assert bench.rank_sequence_base(0, 2) == 0 and bench.rank_sequence_base(1, 2) == 2
    assert not np.array_equal(res["tokens"][0], res["tokens"][1])   # different sequences, different trees
    # rank 1's shard is exactly global sequences 2..3: same bytes as generating them in one process
    a = c2t_inputs.draft_logits(4, 3, 512, 0, 1, torch.float32)[2:]
    b = c2t_inputs.draft_logits(2, 3, 512, 0, 1, torch.float32, seq_base=2)
    assert torch.equal(a, b)
    assert os.path.isdir(oracle_dir)


# ---------------------------------------------------------------- vocabulary-parallel exchange

RECORD = np.dtype([("M", "<f8"), ("S", "<f8"), ("T", "<f8"), ("n", "<i4"), ("fault", "<u4"),
                   ("tok", "<i4", (32,)), ("x", "<f4", (32,))])


def _range_records(logits: torch.Tensor, v0: int, v1: int, K: int) -> np.ndarray:
    """What a rank exports for its token range [v0, v1) of rows [B, F, V] (plain numpy, fp64)."""
    x = logits[:, :, v0:v1].double().numpy()
    B, F, _ = x.shape
    rec = np.zeros((B, F), dtype=RECORD)
    for b in range(B):
        for j in range(F):
            row = x[b, j]
            order = np.lexsort((np.arange(row.size), -row))          # logit descending, token id ascending
            m = row[order[0]]
            rest = np.delete(row, order[0])
            rec[b, j]["M"] = m
            rec[b, j]["S"] = np.exp(rest - m).sum()
            rec[b, j]["T"] = (np.exp(rest - m) * (rest - m)).sum()
            k = min(K, row.size)
            rec[b, j]["n"] = k
            rec[b, j]["tok"][:k] = order[:k] + v0
            rec[b, j]["x"][:k] = row[order[:k]]
    return rec


def _vp_worker(rank: int, world: int, port: int, out):
    sys.path.insert(0, ROOT)
    import c2t_inputs
    from paper_2502_13652_b200 import vocab_parallel as vp

    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    B, F, V, K = 2, 3, 1000, 5
    logits = c2t_inputs.draft_logits(B, F, V, 0, 1, torch.float32)    # every rank can draw the whole rows here
    v0, v1 = vp.shard_ranges(V, world, 4)[rank]
    local = torch.from_numpy(_range_records(logits, v0, v1, K).view(np.uint8).reshape(B, F, RECORD.itemsize))
    gathered = vp.gather_row_records(local)                           # the path's only collective
    # the same exchange into a buffer allocated once (what ExchangeBuffers holds), and for the 8-byte keys of the
    # acceptance walks: [B, Nw] per rank for the all-rows walk, [B] per rank and round for the lazy one
    buf = torch.full((world, B, F, RECORD.itemsize), 255, dtype=torch.uint8)
    again = vp.gather_row_records(local, out=buf)
    assert again.data_ptr() == buf.data_ptr() and torch.equal(again, gathered)
    keys = torch.arange(B, dtype=torch.int64) * 10 + rank
    got_keys = vp.gather_row_records(keys, out=torch.zeros((world, B), dtype=torch.int64))
    assert got_keys.tolist() == [[b * 10 + r for b in range(B)] for r in range(world)]
    if rank == 0:
        out.put(gathered.numpy())
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_exchange_row_records_in_token_order():
    sys.path.insert(0, ROOT)
    import c2t_inputs
    from paper_2502_13652_b200 import binding
    from paper_2502_13652_b200 import vocab_parallel as vp
    assert RECORD.itemsize == binding.ROW_RECORD_BYTES == 288
    for V, world, eb in ((1000, 2, 4), (128256, 8, 2), (37, 3, 2), (32000, 7, 4)):
        r = vp.shard_ranges(V, world, eb)
        assert r[0][0] == 0 and r[-1][1] == V and all(a[1] == b[0] for a, b in zip(r, r[1:]))
        assert all((v0 * eb) % 16 == 0 and v1 > v0 for v0, v1 in r)
    with np.testing.assert_raises(ValueError):
        vp.shard_ranges(16, 8, 2)

    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = 31500 + os.getpid() % 2000
    procs = [ctx.Process(target=_vp_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    got = out.get(timeout=120)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    B, F, V, K = 2, 3, 1000, 5
    logits = c2t_inputs.draft_logits(B, F, V, 0, 1, torch.float32)
    ranges = vp.shard_ranges(V, 2, 4)
    assert got.shape == (2, B, F, 288)
    rec = got.reshape(2, B, F, 288).view(RECORD).reshape(2, B, F)
    for g, (v0, v1) in enumerate(ranges):                             # shard-major, in rank = token order
        want = _range_records(logits, v0, v1, K)
        for name in RECORD.names:
            assert np.array_equal(rec[g][name], want[name]), (g, name)
    # merging the two records of a row the way the header states gives the whole row's softmax normaliser,
    # entropy and top-K (scipy on the whole row)
    from scipy.special import logsumexp
    from scipy.stats import entropy
    for b in range(B):
        for j in range(F):
            row = logits[b, j].double().numpy()
            M = max(rec[g, b, j]["M"] for g in range(2))
            w = min(g for g in range(2) if rec[g, b, j]["M"] == M)
            S = T = 0.0
            for g in range(2):
                d = rec[g, b, j]["M"] - M
                S += np.exp(d) * rec[g, b, j]["S"] + (np.exp(d) if g != w else 0.0)
                T += np.exp(d) * (rec[g, b, j]["T"] + d * rec[g, b, j]["S"]) + (np.exp(d) * d if g != w else 0.0)
            assert abs((M + np.log1p(S)) - logsumexp(row)) < 1e-12 * abs(logsumexp(row)) + 1e-12
            p = np.exp(row - logsumexp(row))
            assert abs((np.log1p(S) - T / (1.0 + S)) - entropy(p)) < 1e-10
            heads = sorted(((-rec[g, b, j]["x"][i], rec[g, b, j]["tok"][i]) for g in range(2) for i in range(K)))[:K]
            order = np.lexsort((np.arange(V), -row))[:K]
            assert [t for _, t in heads] == list(order)

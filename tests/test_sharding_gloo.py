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

"""The allocation-free entry point, c2t_row_argmax_static, against c2t_accept.

Some callers of this library are not allowed to allocate device memory (a server whose memory
was all handed out at start-up, a plug-in inside another engine, a loop that must never hit
cudaMalloc's device-wide synchronisation).  For them the library offers the arg-max pass with
its scratch in a fixed device array.  This test calls it through the C ABI twice in a row, on
different logits, and requires the tokens to equal what the ordinary path (c2t_accept with a
caller-provided workspace) finds for the same rows.  It is collected last so that a run that
stops at the first failure has already run every other test, and it does not depend on them.
"""
import ctypes as C

import pytest
import torch

import c2t_inputs
import oracle
import paper_2502_13652_b200 as c2t
from parity_util import gen_inputs, make_configs

pytestmark = pytest.mark.gpu


def reference_argmax(ctx, draft, target, root, prefix):
    """Per-node target arg-max from the ordinary path, and how many nodes each sequence has."""
    ctx.decode_step(draft, target, root, prefix)
    torch.cuda.synchronize()
    return ctx.c2t_get_view()["node_argmax"].clone(), ctx.verify["n_nodes"].clone()


@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32])
def test_static_scratch_argmax_matches_accept_twice_in_a_row(dtype):
    from paper_2502_13652_b200 import build
    build.build()
    B, V, D, K, F, N = 6, 32000, 4, 6, 5, 16
    _, gcfg = make_configs(B, V, D, K, F, N, 0.4, dtype)
    ctx = c2t.Context(gcfg)
    Nw = ctx.Nw
    out = torch.full((B * Nw,), -7, dtype=torch.int32, device="cuda")
    for step in range(2):                                   # two calls in a row, different logits
        draft, target, root, prefix = gen_inputs(B, V, D, F, Nw, dtype, step=step)
        draft = [t.cuda() for t in draft]; target = target.cuda()
        want, n_nodes = reference_argmax(ctx, draft, target, root.cuda(), prefix.cuda())
        assert int(n_nodes.max()) > 1
        c2t.c2t_row_argmax_static(target.view(B * Nw, V), out)
        torch.cuda.synchronize()
        got = out.view(B, Nw)
        live = torch.arange(Nw, device="cuda")[None, :] < n_nodes[:, None]
        assert torch.equal(got[live], want[live])            # integers: identical, not merely close
        # rows past a sequence's node count are never read by c2t_accept; check them directly
        direct = target.view(B * Nw, V).float().argmax(dim=1).to(torch.int32)
        tied = (target.view(B * Nw, V) == target.view(B * Nw, V).max(dim=1, keepdim=True).values).sum(1) > 1
        assert torch.equal(out[~tied], direct[~tied])
    ctx.close()


@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32])
def test_static_scratch_argmax_against_the_oracle_on_tie_heavy_rows(dtype):
    """Row by row against the oracle's arg-max (largest logit, ties to the lower token id) on rows where
    the maximum occurs many times, with a row length that is not a whole number of 16-byte vectors, -inf
    entries and a padded stride.  Two calls in a row with different row counts: the second, shorter call
    must not see the keys the first one left in the shared scratch."""
    from paper_2502_13652_b200 import build
    build.build()
    oracle.build()
    V, Vp = 5003, 5024
    g = torch.Generator().manual_seed(11)
    for rows in (37, 9):
        x = (40 + torch.randn(rows, V, generator=g) * 0.4).to(torch.bfloat16)      # spacing 0.25: the maximum repeats
        x[torch.rand(rows, V, generator=g) < 0.2] = float("-inf")
        x[rows // 2, :] = float("-inf")                                             # a row without any finite logit
        x[0, :] = 3.0                                                               # all equal: token 0
        x = x.to(dtype)
        assert int((x[1] == x[1].max()).sum()) > 1
        buf = torch.full((rows, Vp), float("nan"), dtype=dtype, device="cuda")      # the padding must never be read
        buf[:, :V] = x.cuda()
        out = torch.full((rows,), -7, dtype=torch.int32, device="cuda")
        c2t.c2t_row_argmax_static(buf[:, :V], out)
        torch.cuda.synchronize()
        want = [oracle.row_argmax(x[r]) for r in range(rows)]
        got = out.tolist()
        for r in range(rows):
            if r == rows // 2:
                continue                                     # all -inf: no arg-max is defined; both sides only stay in range
            assert got[r] == want[r], (rows, r, got[r], want[r])
        assert -1 <= got[rows // 2] < V


def test_static_scratch_limits_and_arguments():
    from paper_2502_13652_b200 import build
    build.build()
    L = c2t.lib()
    x = torch.zeros(8, 1024, device="cuda")
    out = torch.zeros(8, dtype=torch.int32, device="cuda")
    s = torch.cuda.current_stream().cuda_stream
    call = lambda rows, vocab, stride, ptr=x.data_ptr(): L.c2t_row_argmax_static(  # noqa: E731
        ptr, rows, vocab, c2t.F32, stride, out.data_ptr(), s)
    assert call(c2t.STATIC_MAX_ROWS + 1, 1024, 1024) == c2t.ERANGE      # refused, nothing launched
    assert call(8, c2t.STATIC_MAX_VOCAB + 1, c2t.STATIC_MAX_VOCAB + 4) == c2t.ERANGE
    assert call(0, 1024, 1024) == c2t.EINVAL
    assert call(8, 1024, 1000) == c2t.EINVAL                            # stride shorter than a row
    assert call(8, 1024, 1024, x.data_ptr() + 4) == c2t.EALIGN
    assert L.c2t_row_argmax_static(None, 8, 1024, c2t.F32, 1024, out.data_ptr(), s) == c2t.EINVAL
    assert call(8, 1024, 1024) == c2t.OK
    torch.cuda.synchronize()
    assert out.tolist() == [0] * 8                                      # all-equal rows: lowest token id

"""The library built with -DC2T_DEBUG_BOUNDS (every kernel checks the indices of its own writes to queues, pools
and workspace records and reports a failed check as C2T_ST_INTERNAL) must pass the same parity cases without ever
setting that bit.  This is the stand-in for a memory checker.  The variant is a second shared library, selected by
the C2T_LIBRARY environment variable, so the cases run in a child process."""
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

CHILD = r"""
import sys, torch
sys.path.insert(0, {root!r}); sys.path.insert(0, {tests!r})
import oracle, paper_2502_13652_b200 as c2t
from parity_util import gen_inputs, make_configs, run_and_compare, special_rows
assert c2t.LIB_PATH.endswith("libc2t_debug.so")
oracle.build()
cases = [(2, 32000, 5, 10, 10, 40, 0.5, torch.bfloat16, {{}}),
         (3, 5004, 4, 6, 5, 18, 0.5, torch.float32, {{}}),
         (1, 16384, 3, 32, 32, 100, 0.5, torch.bfloat16, dict(hidden=64, wseed=4)),
         (1, 128256, 4, 8, 16, 40, 0.3, torch.bfloat16, {{}}),
         (2, 4096, 5, 4, 4, 7, 0.0, torch.float32, dict(classifier="identity", tree_add="all"))]
for B, V, D, K, F, N, beta, dtype, kw in cases:
    ocfg, gcfg = make_configs(B, V, D, K, F, N, beta, dtype, **kw)
    Nw = c2t.c2t_final_width(gcfg)
    draft, target, root, prefix = gen_inputs(B, V, D, F, Nw, dtype)
    rep = run_and_compare(ocfg, gcfg, draft, target, root, prefix)
    assert rep.status_bits == 0, rep.status_bits
for kind in ("rising", "uniform", "neg_inf"):
    B, V, D, K, F, N = 2, 20000, 3, 5, 4, 12
    ocfg, gcfg = make_configs(B, V, D, K, F, N, 0.0, torch.bfloat16, classifier="identity")
    Nw = c2t.c2t_final_width(gcfg)
    draft = [special_rows(kind, B, F, V, torch.bfloat16) for _ in range(D)]
    target = special_rows(kind, B, Nw, V, torch.bfloat16)
    root = torch.zeros(B, dtype=torch.int32); prefix = torch.full((B,), 9, dtype=torch.int32)
    rep = run_and_compare(ocfg, gcfg, draft, target, root, prefix, allow_diverged=B, allow_kinds=("cross_row_tie",))
    assert rep.status_bits & c2t.ST_INTERNAL == 0 and rep.status_bits == 0, rep.status_bits
print("debug-bounds cases ok")
"""


def test_parity_cases_under_index_checks():
    from paper_2502_13652_b200 import build
    lib = build.build(debug_bounds=True)
    env = dict(os.environ, C2T_LIBRARY=lib)
    code = CHILD.format(root=ROOT, tests=os.path.join(ROOT, "tests"))
    out = subprocess.run([sys.executable, "-c", code], env=env, capture_output=True, text=True, timeout=900)
    assert out.returncode == 0, out.stdout[-2000:] + out.stderr[-4000:]
    assert "debug-bounds cases ok" in out.stdout

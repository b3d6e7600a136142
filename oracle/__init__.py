"""CPU oracle for the C2T draft-tree hot path.  TEST INFRASTRUCTURE ONLY.

`c2t_oracle.c` is the implementation (plain C99, double precision); this
package compiles it with gcc and exposes it through ctypes.  Nothing on the
product path may import it: only tests, the smoke check and the benchmark's CPU
baseline do.  It imports nothing from the CUDA package.
"""
from .c2t_oracle import (  # noqa: F401
    OracleConfig, LevelRecords, Tree, FinalTree, VerifyInputs, AcceptResult, StepResult,
    build, lib, row_stats, row_softmax, classifier, build_tree, final_prune, build_verify, dense_mask,
    row_argmax, accept, decode_step, tree_capacity, final_width,
    F32, BF16, CLS_MLP, CLS_IDENTITY_JOINT, CLS_IDENTITY_COND, ADD_FRONTIER, ADD_ALL_SURVIVORS,
)

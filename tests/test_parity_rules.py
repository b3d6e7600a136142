"""The rules by which the GPU parity tests excuse a difference from the oracle, checked on planted
differences (CPU only): a difference passes only if every candidate or node involved sits on a
boundary of the oracle; a difference anywhere else is reported."""
import os
import sys
from types import SimpleNamespace

import numpy as np

sys.path.insert(0, os.path.dirname(__file__))
from parity_util import _excuse_budget, _excuse_level, _excuse_swaps, _near_tie_at_level  # noqa: E402

K = 3


def level(C, keep, nxt):
    C = np.asarray(C, np.float64)
    n = len(C)
    return SimpleNamespace(n_cand=np.array([n]), C=C[None, :], keep=np.asarray(keep, np.int32)[None, :],
                           next=np.asarray(nxt, np.int32)[None, :])


def flags(keep, nxt):
    return np.asarray(keep, np.int32) | (np.asarray(nxt, np.int32) << 1)


def test_identical_flags_need_no_excuse_and_swaps_need_partners():
    assert _excuse_swaps([], [], np.zeros(3), np.zeros(3)) is None            # nothing differs: not a swap
    assert _excuse_swaps([0], [], np.zeros(3), np.arange(3)) is None          # counts differ: never excused


def test_near_threshold_candidate_may_flip():
    beta = 0.5
    L = level([0.9, 0.5 + 2e-7, 0.2, 0.7, 0.1, 0.05], [1, 1, 0, 1, 0, 0], [1, 1, 0, 1, 0, 0])
    g = flags([1, 0, 0, 1, 0, 0], [1, 0, 0, 1, 0, 0])                         # the candidate at beta + 2e-7 dropped
    assert _excuse_level(L, 0, K, beta, g) == "near_beta"
    g = flags([1, 1, 0, 0, 0, 0], [1, 1, 0, 0, 0, 0])                         # 0.7 dropped: nowhere near beta
    assert _excuse_level(L, 0, K, beta, g) is None
    # at beta = 0 nothing is near the threshold (the old absolute test excused every tiny probability)
    L0 = level([0.9, 1e-9, 0.2], [1, 1, 1], [1, 1, 1])
    assert _excuse_level(L0, 0, K, 0.0, flags([1, 0, 1], [1, 0, 1])) is None
    assert not _near_tie_at_level(L0, 0, 2, 0.0)


def test_cap_swap_needs_near_equal_confidences():
    # cap of 2 among survivors; candidates 1 (row 0) and 3 (row 1) are 3e-7 apart in relative terms
    C = [0.9, 0.4, 0.1, 0.4 * (1 - 3e-7), 0.05, 0.01]
    L = level(C, [1] * 6, [1, 1, 0, 0, 0, 0])
    assert _excuse_level(L, 0, K, 0.0, flags([1] * 6, [1, 0, 0, 1, 0, 0])) == "near_cap"
    assert _excuse_level(L, 0, K, 0.0, flags([1] * 6, [1, 0, 1, 0, 0, 0])) is None     # swapped with 0.1: a real error
    assert _excuse_level(L, 0, K, 0.0, flags([1] * 6, [0, 1, 0, 1, 0, 0])) is None     # the best one lost its place


def test_exact_ties_are_excused_across_rows_only():
    C = [0.9, 0.4, 0.4, 0.4, 0.05, 0.01]              # candidates 1, 2 share row 0; candidate 3 is in row 1
    L = level(C, [1] * 6, [1, 1, 0, 0, 0, 0])
    assert _excuse_level(L, 0, K, 0.0, flags([1] * 6, [1, 0, 0, 1, 0, 0])) == "cross_row_tie"
    # the same row gives both sides the same bits: candidate order must decide on both
    assert _excuse_level(L, 0, K, 0.0, flags([1] * 6, [1, 0, 1, 0, 0, 0])) is None


def test_budget_cut():
    # nodes 0..5, parents; Chat decreasing except a near tie between nodes 3 and 4
    parent = np.array([-1, 0, 0, 1, 2, 1], np.int32)
    chat = np.array([np.inf, 0.8, 0.7, 0.3, 0.3 * (1 + 2e-7), 0.1])
    tree = SimpleNamespace(n=6, Chat=chat, parent=parent)
    ft = SimpleNamespace(n=4, src=np.array([0, 1, 2, 4, -1, -1], np.int32))
    assert _excuse_budget(tree, ft, np.array([0, 1, 2, 3])) == "near_budget"
    assert _excuse_budget(tree, ft, np.array([0, 1, 2, 5])) is None            # 0.1 instead of 0.3: a real error
    assert _excuse_budget(tree, ft, np.array([0, 1, 2, 9])) is None            # not a node of the tree
    chat2 = chat.copy(); chat2[4] = 0.3                                        # exact tie, different parents
    tree2 = SimpleNamespace(n=6, Chat=chat2, parent=parent)
    ft2 = SimpleNamespace(n=4, src=np.array([0, 1, 2, 3, -1, -1], np.int32))
    assert _excuse_budget(tree2, ft2, np.array([0, 1, 2, 4])) == "cross_row_tie"
    parent3 = parent.copy(); parent3[4] = 1                                    # ... same parent: must agree
    tree3 = SimpleNamespace(n=6, Chat=chat2, parent=parent3)
    assert _excuse_budget(tree3, ft2, np.array([0, 1, 2, 4])) is None

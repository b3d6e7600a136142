"""ctypes front end of the C oracle (test infrastructure only; see c2t_oracle.c)."""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from dataclasses import dataclass, field
from typing import Optional

import numpy as np
import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "c2t_oracle.c")
_SO = os.path.join(_HERE, "libc2t_oracle.so")

F32, BF16 = 0, 1
CLS_MLP, CLS_IDENTITY_JOINT, CLS_IDENTITY_COND = 0, 1, 2
ADD_FRONTIER, ADD_ALL_SURVIVORS = 0, 1

_lib: Optional[C.CDLL] = None


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (no tuning flags beyond -O2)."""
    if force or not os.path.exists(_SO) or os.path.getmtime(_SO) < os.path.getmtime(_SRC):
        subprocess.check_call(["gcc", "-O2", "-std=c99", "-shared", "-fPIC", "-o", _SO, _SRC, "-lm"])
    return _SO


class _Cfg(C.Structure):
    _fields_ = [
        ("vocab", C.c_int32), ("dtype", C.c_int32), ("max_depth", C.c_int32), ("topk", C.c_int32),
        ("frontier_cap", C.c_int32), ("budget", C.c_int32), ("threshold", C.c_double),
        ("entropy_top_m", C.c_int32), ("classifier", C.c_int32), ("hidden", C.c_int32),
        ("w1", C.c_void_p), ("b1", C.c_void_p), ("w2", C.c_void_p), ("b2", C.c_void_p),
        ("tree_add", C.c_int32),
    ]


class _Levels(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in (
        "n_cand", "tok", "parent_node", "lp", "logP", "H", "C", "keep", "next",
        "n_frontier", "frontier_node", "row_fault")]


class _Tree(C.Structure):
    _fields_ = [("capacity", C.c_int32), ("n", C.c_int32), ("tok", C.c_void_p),
                ("parent", C.c_void_p), ("level", C.c_void_p), ("logP", C.c_void_p),
                ("C", C.c_void_p), ("Chat", C.c_void_p)]


def lib() -> C.CDLL:
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
        _lib.orc_classifier.restype = C.c_double
        _lib.orc_classifier.argtypes = [C.c_double, C.c_double, C.c_double, C.c_int32,
                                        C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
        _lib.orc_row_stats.restype = C.c_int
        _lib.orc_row_stats.argtypes = [C.c_void_p, C.c_int, C.c_int32, C.c_int32, C.c_int32,
                                       C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
        _lib.orc_row_softmax.argtypes = [C.c_void_p, C.c_int, C.c_int32, C.c_void_p]
        _lib.orc_row_argmax.restype = C.c_int32
        _lib.orc_row_argmax.argtypes = [C.c_void_p, C.c_int, C.c_int32]
        _lib.orc_build_tree.restype = C.c_int
        _lib.orc_build_tree.argtypes = [C.POINTER(_Cfg), C.c_void_p, C.c_int64, C.c_int64, C.c_int32,
                                        C.POINTER(_Tree), C.POINTER(_Levels)]
        _lib.orc_final_prune.restype = C.c_int32
        _lib.orc_final_prune.argtypes = [C.POINTER(_Tree), C.c_int32] + [C.c_void_p] * 4
        _lib.orc_build_verify.restype = C.c_int32
        _lib.orc_build_verify.argtypes = [C.c_int32, C.c_void_p, C.c_void_p, C.c_int32, C.c_int32,
                                          C.c_int32, C.c_int32, C.c_void_p, C.c_void_p, C.c_void_p]
        _lib.orc_accept.restype = C.c_int32
        _lib.orc_accept.argtypes = [C.c_int32, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int, C.c_int32,
                                    C.c_int64, C.c_int32, C.c_void_p, C.c_void_p, C.c_void_p]
        _lib.orc_decode_step.restype = C.c_int64
        _lib.orc_decode_step.argtypes = ([C.POINTER(_Cfg), C.c_int32, C.c_int32, C.c_int32,
                                          C.c_void_p, C.c_int64, C.c_int64, C.c_int64,
                                          C.c_void_p, C.c_int64, C.c_int64] + [C.c_void_p] * 12)
    return _lib


@dataclass
class OracleConfig:
    vocab: int
    dtype: int = F32
    max_depth: int = 6
    topk: int = 10
    frontier_cap: int = 10
    budget: int = 60
    threshold: float = 0.5
    entropy_top_m: int = 0
    classifier: int = CLS_MLP
    hidden: int = 16
    w1: Optional[torch.Tensor] = None
    b1: Optional[torch.Tensor] = None
    w2: Optional[torch.Tensor] = None
    b2: Optional[torch.Tensor] = None
    tree_add: int = ADD_FRONTIER
    _keep: list = field(default_factory=list, repr=False)

    def c_struct(self) -> _Cfg:
        self._keep = []
        ptrs = []
        for w, shape in ((self.w1, (self.hidden, 3)), (self.b1, (self.hidden,)),
                         (self.w2, (self.hidden,)), (self.b2, (1,))):
            if w is None:
                a = np.zeros(shape, dtype=np.float32)
            else:
                a = np.ascontiguousarray(w.detach().cpu().numpy().astype(np.float32).reshape(shape))
            self._keep.append(a)
            ptrs.append(a.ctypes.data)
        # the threshold is a float32 in the library's configuration: compare against that value
        beta = float(np.float32(self.threshold))
        return _Cfg(self.vocab, self.dtype, self.max_depth, self.topk, self.frontier_cap, self.budget,
                    beta, self.entropy_top_m, self.classifier, self.hidden, *ptrs, self.tree_add)


def tree_capacity(cfg: OracleConfig) -> int:
    """Largest tree Algorithm 1 can build: root + level-0 children + later levels."""
    K, F, D = cfg.topk, cfg.frontier_cap, cfg.max_depth
    if cfg.tree_add == ADD_ALL_SURVIVORS:
        return 1 + K + max(D - 1, 0) * F * K
    return 1 + min(K, F) + max(D - 1, 0) * F


def final_width(cfg: OracleConfig) -> int:
    cap = tree_capacity(cfg)
    return min(cfg.budget, cap) if cfg.budget > 0 else cap


def _dtype_code(t: torch.Tensor) -> int:
    if t.dtype == torch.float32:
        return F32
    if t.dtype == torch.bfloat16:
        return BF16
    raise TypeError(f"unsupported logits dtype {t.dtype}")


def _ptr(t: torch.Tensor) -> int:
    assert t.device.type == "cpu"
    return t.data_ptr()


def row_stats(row: torch.Tensor, K: int, M: int = 0):
    """(fault, logZ, H, tok[K], x[K], lp[K]) for one logits row [V]."""
    row = row.contiguous()
    V = row.numel()
    logz, H = C.c_double(), C.c_double()
    tok = np.empty(K, np.int32); x = np.empty(K, np.float64); lp = np.empty(K, np.float64)
    fault = lib().orc_row_stats(_ptr(row), _dtype_code(row), V, K, M, C.byref(logz), C.byref(H),
                                tok.ctypes.data, x.ctypes.data, lp.ctypes.data)
    return fault, logz.value, H.value, tok, x, lp


def row_softmax(row: torch.Tensor) -> np.ndarray:
    row = row.contiguous()
    p = np.empty(row.numel(), np.float64)
    lib().orc_row_softmax(_ptr(row), _dtype_code(row), row.numel(), p.ctypes.data)
    return p


def row_argmax(row: torch.Tensor) -> int:
    row = row.contiguous()
    return lib().orc_row_argmax(_ptr(row), _dtype_code(row), row.numel())


def classifier(P: float, H: float, d: float, w1, b1, w2, b2) -> float:
    arrs = [np.ascontiguousarray(np.asarray(w, dtype=np.float32)) for w in (w1, b1, w2, b2)]
    hidden = arrs[1].size
    return lib().orc_classifier(P, H, d, hidden, *[a.ctypes.data for a in arrs])


@dataclass
class LevelRecords:
    n_cand: np.ndarray; tok: np.ndarray; parent_node: np.ndarray; lp: np.ndarray
    logP: np.ndarray; H: np.ndarray; C: np.ndarray; keep: np.ndarray; next: np.ndarray
    n_frontier: np.ndarray; frontier_node: np.ndarray; row_fault: np.ndarray


@dataclass
class Tree:
    n: int; tok: np.ndarray; parent: np.ndarray; level: np.ndarray
    logP: np.ndarray; C: np.ndarray; Chat: np.ndarray; overflow: bool = False
    _c: Optional[_Tree] = field(default=None, repr=False)


def _tree_struct(t: Tree) -> _Tree:
    return _Tree(len(t.tok), t.n, t.tok.ctypes.data, t.parent.ctypes.data, t.level.ctypes.data,
                 t.logP.ctypes.data, t.C.ctypes.data, t.Chat.ctypes.data)


def build_tree(cfg: OracleConfig, logits: torch.Tensor, root_tok: int):
    """Algorithm 1 for one sequence.  logits: [D, F, V] (CPU).  Returns (Tree, LevelRecords)."""
    assert logits.dim() == 3 and logits.shape[0] >= cfg.max_depth and logits.shape[1] >= cfg.frontier_cap
    assert logits.stride(2) == 1
    D, F, K = cfg.max_depth, cfg.frontier_cap, cfg.topk
    FK = F * K
    cap = tree_capacity(cfg)
    t = Tree(0, np.zeros(cap, np.int32), np.zeros(cap, np.int32), np.zeros(cap, np.int32),
             np.zeros(cap, np.float64), np.zeros(cap, np.float64), np.zeros(cap, np.float64))
    L = LevelRecords(
        np.zeros(D, np.int32), np.full((D, FK), -1, np.int32), np.full((D, FK), -1, np.int32),
        np.zeros((D, FK)), np.zeros((D, FK)), np.zeros((D, FK)), np.zeros((D, FK)),
        np.zeros((D, FK), np.int32), np.zeros((D, FK), np.int32),
        np.zeros(D + 1, np.int32), np.full((D + 1, F), -1, np.int32), np.zeros((D, F), np.int32))
    cl = _Levels(*[getattr(L, n).ctypes.data for n, _ in _Levels._fields_])
    ct = _tree_struct(t)
    cc = cfg.c_struct()
    rc = lib().orc_build_tree(C.byref(cc), _ptr(logits), logits.stride(0), logits.stride(1),
                              int(root_tok), C.byref(ct), C.byref(cl))
    t.n = ct.n
    t.overflow = rc != 0
    return t, L


@dataclass
class FinalTree:
    n: int; src: np.ndarray; tok: np.ndarray; parent: np.ndarray; level: np.ndarray


def final_prune(tree: Tree, budget: int) -> FinalTree:
    cap = len(tree.tok)
    src = np.full(cap, -1, np.int32); tok = np.zeros(cap, np.int32)
    par = np.full(cap, -1, np.int32); lev = np.zeros(cap, np.int32)
    ct = _tree_struct(tree)
    n = lib().orc_final_prune(C.byref(ct), budget, src.ctypes.data, tok.ctypes.data,
                              par.ctypes.data, lev.ctypes.data)
    return FinalTree(n, src, tok, par, lev)


@dataclass
class VerifyInputs:
    n_leaves: int; mask: np.ndarray; position_ids: np.ndarray; retrieve: np.ndarray


def build_verify(ft: FinalTree, prefix_len: int, n_rows: int, width: int) -> VerifyInputs:
    W = (n_rows + 63) // 64
    mask = np.zeros((n_rows, W), np.uint64)
    pos = np.zeros(n_rows, np.int32)
    ret = np.full((n_rows, width), -1, np.int32)
    par = np.ascontiguousarray(ft.parent); lev = np.ascontiguousarray(ft.level)
    nl = lib().orc_build_verify(ft.n, par.ctypes.data, lev.ctypes.data, int(prefix_len), n_rows, W, width,
                                mask.ctypes.data, pos.ctypes.data, ret.ctypes.data)
    return VerifyInputs(nl, mask, pos, ret)


def dense_mask(ft: FinalTree, prefix_len: int, n_rows: int, kv_len: int) -> np.ndarray:
    """Additive tree-attention mask (Sec. 2.2) written out: [n_rows, kv_len] float64, 0 where final
    node i attends key c and -inf elsewhere.  Keys [0, prefix_len) are the prefix, which every row
    attends; key prefix_len + j is tree node j, attended iff j is i or an ancestor of i.  Rows past
    the tree attend the prefix only.  Keys at or past kv_len do not exist."""
    out = np.full((n_rows, kv_len), -np.inf)
    for i in range(n_rows):
        for c in range(min(int(prefix_len), kv_len)):
            out[i, c] = 0.0
        if i < ft.n:
            j = i
            while j >= 0:                      # i, its parent, ... up to the root
                if prefix_len + j < kv_len:
                    out[i, prefix_len + j] = 0.0
                j = int(ft.parent[j])
    return out


@dataclass
class AcceptResult:
    accept_len: int; path: np.ndarray; next_token: int; node_argmax: np.ndarray


def accept(ft: FinalTree, target: torch.Tensor, width: int) -> AcceptResult:
    """target: [>=n, V] CPU logits, row i for final node i."""
    assert target.stride(1) == 1
    path = np.full(width, -1, np.int32)
    nxt = C.c_int32()
    amax = np.full(max(ft.n, 1), -1, np.int32)
    tok = np.ascontiguousarray(ft.tok); par = np.ascontiguousarray(ft.parent)
    ln = lib().orc_accept(ft.n, tok.ctypes.data, par.ctypes.data, _ptr(target), _dtype_code(target),
                          target.shape[1], target.stride(0), width, path.ctypes.data, C.byref(nxt),
                          amax.ctypes.data)
    return AcceptResult(ln, path, nxt.value, amax)


@dataclass
class StepResult:
    n_final: np.ndarray; tokens: np.ndarray; parents: np.ndarray; position_ids: np.ndarray
    mask: np.ndarray; retrieve: np.ndarray; n_leaves: np.ndarray
    accept_len: np.ndarray; path: np.ndarray; next_token: np.ndarray; rows_visited: int


def decode_step(cfg: OracleConfig, draft: torch.Tensor, target: torch.Tensor,
                root_tok, prefix_len) -> StepResult:
    """One decode step over a batch.  draft: [B, D, F, V]; target: [B, Nw, V] (CPU)."""
    B = draft.shape[0]
    assert draft.stride(3) == 1 and target.stride(2) == 1
    Nw = final_width(cfg)
    assert target.shape[1] >= Nw
    W = (Nw + 63) // 64
    width = cfg.max_depth + 1
    root = np.ascontiguousarray(np.asarray(root_tok, dtype=np.int32))
    pre = np.ascontiguousarray(np.asarray(prefix_len, dtype=np.int32))
    r = StepResult(np.zeros(B, np.int32), np.zeros((B, Nw), np.int32), np.full((B, Nw), -1, np.int32),
                   np.zeros((B, Nw), np.int32), np.zeros((B, Nw, W), np.uint64),
                   np.full((B, Nw, width), -1, np.int32), np.zeros(B, np.int32),
                   np.zeros(B, np.int32), np.full((B, width), -1, np.int32), np.zeros(B, np.int32), 0)
    cc = cfg.c_struct()
    r.rows_visited = lib().orc_decode_step(
        C.byref(cc), B, Nw, tree_capacity(cfg),
        _ptr(draft), draft.stride(0), draft.stride(1), draft.stride(2),
        _ptr(target), target.stride(0), target.stride(1),
        root.ctypes.data, pre.ctypes.data,
        r.n_final.ctypes.data, r.tokens.ctypes.data, r.parents.ctypes.data, r.position_ids.ctypes.data,
        r.mask.ctypes.data, r.retrieve.ctypes.data, r.n_leaves.ctypes.data,
        r.accept_len.ctypes.data, r.path.ctypes.data, r.next_token.ctypes.data)
    return r

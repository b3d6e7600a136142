"""ctypes binding of libc2t.so (see include/c2t.h for the contract of every call).

Argument marshalling only: every step of the path runs in the library's CUDA kernels.
PyTorch supplies device memory (`torch.empty`), streams and nothing else.  There is no CPU
fallback: if the shared library is missing the import of this module fails.
"""
from __future__ import annotations

import ctypes as C
import os
from dataclasses import dataclass
from typing import Optional, Sequence

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
# C2T_LIBRARY selects another build of the same library (the -DC2T_DEBUG_BOUNDS variant, see build.py)
LIB_PATH = os.environ.get("C2T_LIBRARY") or os.path.join(_HERE, "libc2t.so")

F32, BF16 = 0, 1
CLS_MLP, CLS_IDENTITY_JOINT, CLS_IDENTITY_COND = 0, 1, 2
ADD_FRONTIER, ADD_ALL_SURVIVORS = 0, 1
FINAL = -1
OK, EINVAL, EALIGN, ERANGE, EORDER, ECUDA, ENOMEM = 0, -1, -2, -3, -4, -5, -6
ST_NAN_LOGIT, ST_POSINF_LOGIT, ST_ALL_NEGINF, ST_TREE_OVERFLOW, ST_INTERNAL = 1, 2, 4, 8, 16


class C2TError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__(f"{where}: {lib().c2t_strerror(code).decode()} ({code})")


class c2t_config(C.Structure):
    _fields_ = [
        ("batch", C.c_int32), ("vocab", C.c_int32), ("dtype", C.c_int32), ("max_depth", C.c_int32),
        ("topk", C.c_int32), ("frontier_cap", C.c_int32), ("budget", C.c_int32), ("threshold", C.c_float),
        ("entropy_top_m", C.c_int32), ("classifier", C.c_int32), ("hidden", C.c_int32),
        ("w1", C.c_void_p), ("b1", C.c_void_p), ("w2", C.c_void_p), ("b2", C.c_void_p),
        ("tree_add", C.c_int32), ("device", C.c_int32),
    ]


class c2t_frontier(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in ("count", "token", "node_id", "parent_slot")]


MAX_TOPK = 32
MAX_SHARDS = 32


class c2t_row_record(C.Structure):
    _fields_ = [("M", C.c_double), ("S", C.c_double), ("T", C.c_double), ("n", C.c_int32), ("fault", C.c_uint32),
                ("tok", C.c_int32 * MAX_TOPK), ("x", C.c_float * MAX_TOPK)]


ROW_RECORD_BYTES = C.sizeof(c2t_row_record)      # 288


class c2t_verify(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in ("n_nodes", "tokens", "parents", "position_ids", "mask_bits",
                                          "retrieve", "n_leaves")]


class c2t_accept_out(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in ("accept_len", "path", "next_token")]


_VIEW_FIELDS = ("tree_n", "tree_token", "tree_parent", "tree_level", "tree_logP", "tree_C", "tree_Chat",
                "cand_n", "cand_token", "cand_lp", "cand_logP", "cand_H", "cand_C", "cand_flags",
                "frontier_n", "frontier_node", "final_n", "final_src", "final_token", "final_parent",
                "final_level", "node_argmax", "topm_from_pass")


class c2t_view(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in _VIEW_FIELDS]


class c2t_host_step(C.Structure):
    _fields_ = [
        ("draft_logits_host", C.POINTER(C.c_void_p)), ("target_logits_host", C.c_void_p),
        ("root_tok_host", C.c_void_p), ("prefix_len_host", C.c_void_p),
        ("draft_stage_dev", C.c_void_p), ("target_stage_dev", C.c_void_p), ("int_stage_dev", C.c_void_p),
        ("n_nodes_host", C.c_void_p), ("tokens_host", C.c_void_p), ("accept_len_host", C.c_void_p),
        ("path_host", C.c_void_p), ("next_token_host", C.c_void_p),
    ]


_lib: Optional[C.CDLL] = None


def lib() -> C.CDLL:
    """The loaded shared library.  Raises if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise ImportError(f"{LIB_PATH} is missing: build it with "
                              "`python -m paper_2502_13652_b200.build` (needs nvcc)")
        L = C.CDLL(LIB_PATH)
        P = C.POINTER
        L.c2t_workspace_bytes.restype = C.c_size_t
        L.c2t_workspace_bytes.argtypes = [P(c2t_config)]
        for name in ("c2t_tree_capacity", "c2t_final_width", "c2t_mask_words"):
            getattr(L, name).restype = C.c_int32
            getattr(L, name).argtypes = [P(c2t_config)]
        L.c2t_host_step_ints.restype = C.c_size_t
        L.c2t_host_step_ints.argtypes = [P(c2t_config)]
        L.c2t_init.restype = C.c_int
        L.c2t_init.argtypes = [P(c2t_config), C.c_void_p, C.c_size_t, P(C.c_void_p)]
        L.c2t_destroy.restype = None
        L.c2t_destroy.argtypes = [C.c_void_p]
        L.c2t_begin_step.restype = C.c_int
        L.c2t_begin_step.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
        L.c2t_expand_level.restype = C.c_int
        L.c2t_expand_level.argtypes = [C.c_void_p, C.c_int, C.c_void_p, C.c_int64, C.c_int64, C.c_void_p]
        L.c2t_expand_prune_level.restype = C.c_int
        L.c2t_expand_prune_level.argtypes = [C.c_void_p, C.c_int, C.c_void_p, C.c_int64, C.c_int64,
                                             P(c2t_frontier), C.c_void_p]
        L.c2t_prune.restype = C.c_int
        L.c2t_prune.argtypes = [C.c_void_p, C.c_int, P(c2t_frontier), C.c_void_p]
        L.c2t_lazy_begin.restype = C.c_int
        L.c2t_lazy_begin.argtypes = [C.c_void_p, P(c2t_accept_out), C.c_void_p]
        L.c2t_lazy_argmax_shard.restype = C.c_int
        L.c2t_lazy_argmax_shard.argtypes = [C.c_void_p, C.c_void_p, C.c_int64, C.c_int64, C.c_int32, C.c_int32,
                                            C.c_void_p, C.c_void_p]
        L.c2t_lazy_step_gathered.restype = C.c_int
        L.c2t_lazy_step_gathered.argtypes = [C.c_void_p, C.c_int, C.c_void_p, C.c_int32, P(c2t_accept_out),
                                             C.c_void_p]
        L.c2t_expand_level_shard.restype = C.c_int
        L.c2t_expand_level_shard.argtypes = [C.c_void_p, C.c_int, C.c_void_p, C.c_int64, C.c_int64, C.c_int32,
                                             C.c_void_p]
        L.c2t_export_row_records.restype = C.c_int
        L.c2t_export_row_records.argtypes = [C.c_void_p, C.c_int, C.c_int32, C.c_void_p, C.c_void_p]
        L.c2t_prune_gathered.restype = C.c_int
        L.c2t_prune_gathered.argtypes = [C.c_void_p, C.c_int, C.c_void_p, C.c_int32, P(c2t_frontier), C.c_void_p]
        L.c2t_argmax_shard.restype = C.c_int
        L.c2t_argmax_shard.argtypes = [C.c_void_p, C.c_void_p, C.c_int64, C.c_int64, C.c_int32, C.c_int32, C.c_void_p,
                                       C.c_void_p]
        L.c2t_accept_gathered.restype = C.c_int
        L.c2t_accept_gathered.argtypes = [C.c_void_p, C.c_void_p, C.c_int32, P(c2t_accept_out), C.c_void_p]
        L.c2t_build_verify.restype = C.c_int
        L.c2t_build_verify.argtypes = [C.c_void_p, P(c2t_verify), C.c_void_p]
        L.c2t_accept.restype = C.c_int
        L.c2t_accept.argtypes = [C.c_void_p, C.c_void_p, C.c_int64, C.c_int64, P(c2t_accept_out), C.c_void_p]
        L.c2t_dense_mask.restype = C.c_int
        L.c2t_dense_mask.argtypes = [C.c_void_p, C.c_void_p, C.c_int32, C.c_int64, C.c_void_p]
        L.c2t_accept_lazy.restype = C.c_int
        L.c2t_accept_lazy.argtypes = [C.c_void_p, C.c_void_p, C.c_int64, C.c_int64, P(c2t_accept_out), C.c_void_p]
        L.c2t_status.restype = C.c_int
        L.c2t_status.argtypes = [C.c_void_p, P(C.c_uint32), C.c_void_p, C.c_void_p]
        L.c2t_get_view.restype = C.c_int
        L.c2t_get_view.argtypes = [C.c_void_p, P(c2t_view)]
        L.c2t_decode_step_host.restype = C.c_int
        L.c2t_decode_step_host.argtypes = [C.c_void_p, P(c2t_host_step), C.c_void_p]
        L.c2t_launch_count.restype = C.c_int64
        L.c2t_launch_count.argtypes = [C.c_void_p]
        L.c2t_row_argmax_static.restype = C.c_int
        L.c2t_row_argmax_static.argtypes = [C.c_void_p, C.c_int32, C.c_int32, C.c_int32, C.c_int64, C.c_void_p,
                                            C.c_void_p]
        L.c2t_strerror.restype = C.c_char_p
        L.c2t_strerror.argtypes = [C.c_int]
        _lib = L
    return _lib


def _check(rc: int, where: str) -> None:
    if rc != OK:
        raise C2TError(rc, where)


def _stream(stream) -> int:
    if stream is None:
        return torch.cuda.current_stream().cuda_stream
    return stream.cuda_stream if hasattr(stream, "cuda_stream") else int(stream)


def _dp(t: Optional[torch.Tensor]) -> Optional[int]:
    return None if t is None else t.data_ptr()


@dataclass
class Config:
    """Mirror of `c2t_config`; weights are CPU float32 tensors."""
    batch: int
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
    device: int = 0

    def c_struct(self):
        keep = []
        ptrs = []
        for w in (self.w1, self.b1, self.w2, self.b2):
            if w is None:
                ptrs.append(None)
            else:
                w = w.detach().to("cpu", torch.float32).contiguous()
                keep.append(w)
                ptrs.append(w.data_ptr())
        s = c2t_config(self.batch, self.vocab, self.dtype, self.max_depth, self.topk, self.frontier_cap,
                       self.budget, self.threshold, self.entropy_top_m, self.classifier, self.hidden,
                       *ptrs, self.tree_add, self.device)
        return s, keep

    @property
    def torch_dtype(self) -> torch.dtype:
        return torch.bfloat16 if self.dtype == BF16 else torch.float32


def c2t_workspace_bytes(cfg: Config) -> int:
    s, _keep = cfg.c_struct()
    return lib().c2t_workspace_bytes(C.byref(s))


def c2t_tree_capacity(cfg: Config) -> int:
    s, _keep = cfg.c_struct()
    return lib().c2t_tree_capacity(C.byref(s))


def c2t_final_width(cfg: Config) -> int:
    s, _keep = cfg.c_struct()
    return lib().c2t_final_width(C.byref(s))


def c2t_mask_words(cfg: Config) -> int:
    s, _keep = cfg.c_struct()
    return lib().c2t_mask_words(C.byref(s))


STATIC_MAX_ROWS, STATIC_MAX_VOCAB = 4096, 262144


def c2t_row_argmax_static(logits: torch.Tensor, out: torch.Tensor, stream=None) -> None:
    """Greedy token of every row of `logits` [rows, V] into `out` [rows] int32, using the scratch
    array built into the library instead of a workspace: nothing is allocated by this call, which
    is what a caller that may not allocate device memory needs.  Calls share that array, so keep
    them on one stream (or order them); the first call on a device should precede any capture."""
    assert logits.is_cuda and out.is_cuda and logits.dim() == 2 and logits.stride(1) == 1
    assert out.dtype == torch.int32 and out.is_contiguous() and out.numel() == logits.shape[0]
    dtype = BF16 if logits.dtype == torch.bfloat16 else F32
    assert logits.dtype in (torch.bfloat16, torch.float32)
    with torch.cuda.device(logits.device):
        _check(lib().c2t_row_argmax_static(logits.data_ptr(), logits.shape[0], logits.shape[1], dtype,
                                           logits.stride(0), out.data_ptr(), _stream(stream)),
               "c2t_row_argmax_static")


class Context:
    """A `c2t_ctx` plus the torch tensors that back its workspace and default outputs.

    Methods carry the names of the C entry points; each one only marshals its arguments.
    """

    def __init__(self, cfg: Config):
        self.cfg = cfg
        L = lib()
        s, keep = cfg.c_struct()
        self.device = torch.device("cuda", cfg.device)
        nbytes = L.c2t_workspace_bytes(C.byref(s))
        if nbytes == 0:
            handle = C.c_void_p()
            _check(L.c2t_init(C.byref(s), None, 0, C.byref(handle)) or EINVAL, "c2t_init")
        self.workspace = torch.empty(nbytes + 256, dtype=torch.uint8, device=self.device)
        base = (self.workspace.data_ptr() + 255) & ~255
        handle = C.c_void_p()
        with torch.cuda.device(self.device):
            _check(L.c2t_init(C.byref(s), base, nbytes, C.byref(handle)), "c2t_init")
        self._h = handle
        self.B, self.F, self.K, self.D, self.V = cfg.batch, cfg.frontier_cap, cfg.topk, cfg.max_depth, cfg.vocab
        self.cap = L.c2t_tree_capacity(C.byref(s))
        self.Nw = L.c2t_final_width(C.byref(s))
        self.W = L.c2t_mask_words(C.byref(s))
        i32 = dict(dtype=torch.int32, device=self.device)
        B, F, Nw, W, D = self.B, self.F, self.Nw, self.W, self.D
        # default caller-owned outputs
        self.frontier = {"count": torch.zeros(B, **i32), "token": torch.zeros(B, F, **i32),
                         "node_id": torch.zeros(B, F, **i32), "parent_slot": torch.zeros(B, F, **i32)}
        self.verify = {"n_nodes": torch.zeros(B, **i32), "tokens": torch.zeros(B, Nw, **i32),
                       "parents": torch.zeros(B, Nw, **i32), "position_ids": torch.zeros(B, Nw, **i32),
                       "mask_bits": torch.zeros(B, Nw, W, dtype=torch.int64, device=self.device),
                       "retrieve": torch.zeros(B, Nw, D + 1, **i32), "n_leaves": torch.zeros(B, **i32)}
        self.accepted = {"accept_len": torch.zeros(B, **i32), "path": torch.zeros(B, D + 1, **i32),
                         "next_token": torch.zeros(B, **i32)}
        self._frontier_c = c2t_frontier(*[self.frontier[n].data_ptr() for n, _ in c2t_frontier._fields_])
        self._verify_c = c2t_verify(*[self.verify[n].data_ptr() for n, _ in c2t_verify._fields_])
        self._accept_c = c2t_accept_out(*[self.accepted[n].data_ptr() for n, _ in c2t_accept_out._fields_])

    def close(self) -> None:
        if getattr(self, "_h", None) is not None and self._h:
            lib().c2t_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # -- the entry points ---------------------------------------------------------------
    def c2t_begin_step(self, root_tok: torch.Tensor, prefix_len: torch.Tensor, stream=None) -> None:
        assert root_tok.dtype == torch.int32 and prefix_len.dtype == torch.int32
        assert root_tok.is_cuda and prefix_len.is_cuda and root_tok.numel() == self.B == prefix_len.numel()
        _check(lib().c2t_begin_step(self._h, root_tok.data_ptr(), prefix_len.data_ptr(), _stream(stream)),
               "c2t_begin_step")

    def c2t_expand_level(self, level: int, logits: torch.Tensor, stream=None) -> None:
        """logits: [B, >=F, V] CUDA tensor of the configured dtype, last dimension contiguous."""
        assert logits.is_cuda and logits.dtype == self.cfg.torch_dtype and logits.dim() == 3
        assert logits.shape[0] == self.B and logits.shape[2] == self.V and logits.stride(2) == 1
        _check(lib().c2t_expand_level(self._h, level, logits.data_ptr(), logits.stride(0), logits.stride(1),
                                      _stream(stream)), "c2t_expand_level")

    def c2t_expand_prune_level(self, level: int, logits: torch.Tensor, stream=None, emit: bool = True) -> None:
        """c2t_expand_level and c2t_prune of a level as one call (one launch for batches of at most 2 sequences)."""
        assert logits.is_cuda and logits.dtype == self.cfg.torch_dtype and logits.dim() == 3
        assert logits.shape[0] == self.B and logits.shape[2] == self.V and logits.stride(2) == 1
        out = C.byref(self._frontier_c) if emit else None
        _check(lib().c2t_expand_prune_level(self._h, level, logits.data_ptr(), logits.stride(0), logits.stride(1), out,
                                            _stream(stream)), "c2t_expand_prune_level")

    def c2t_prune(self, level: int, stream=None, emit: bool = True) -> None:
        out = C.byref(self._frontier_c) if (emit and level != FINAL) else None
        _check(lib().c2t_prune(self._h, level, out, _stream(stream)), "c2t_prune")

    def c2t_expand_level_shard(self, level: int, logits: torch.Tensor, stream=None) -> None:
        """logits: [B, >=F, vocab_count] CUDA tensor of the configured dtype, last dimension contiguous (a slice of
        wider rows is fine: the strides are the tensor's)."""
        assert logits.is_cuda and logits.dtype == self.cfg.torch_dtype and logits.dim() == 3
        assert logits.shape[0] == self.B and logits.stride(2) == 1
        _check(lib().c2t_expand_level_shard(self._h, level, logits.data_ptr(), logits.stride(0), logits.stride(1),
                                            logits.shape[2], _stream(stream)), "c2t_expand_level_shard")

    def new_row_records(self, n_shards: int = 1) -> torch.Tensor:
        """Device buffer for [n_shards, B, F] row records, as bytes (see `c2t_row_record`)."""
        return torch.zeros((n_shards, self.B, self.F, ROW_RECORD_BYTES), dtype=torch.uint8,
                           device=self.workspace.device)

    def c2t_export_row_records(self, level: int, vocab_begin: int, records: torch.Tensor, stream=None) -> None:
        """records: [B, F, ROW_RECORD_BYTES] uint8 CUDA tensor, contiguous (one shard's slot of `new_row_records`)."""
        assert records.is_cuda and records.dtype == torch.uint8 and records.is_contiguous()
        assert records.numel() == self.B * self.F * ROW_RECORD_BYTES
        _check(lib().c2t_export_row_records(self._h, level, vocab_begin, records.data_ptr(), _stream(stream)),
               "c2t_export_row_records")

    def c2t_prune_gathered(self, level: int, records: torch.Tensor, stream=None, emit: bool = True) -> None:
        """records: [n_shards, B, F, ROW_RECORD_BYTES] uint8 CUDA tensor, shards in ascending token order."""
        assert records.is_cuda and records.dtype == torch.uint8 and records.is_contiguous() and records.dim() == 4
        assert records.shape[1:] == (self.B, self.F, ROW_RECORD_BYTES)
        out = C.byref(self._frontier_c) if emit else None
        _check(lib().c2t_prune_gathered(self._h, level, records.data_ptr(), records.shape[0], out, _stream(stream)),
               "c2t_prune_gathered")

    def c2t_build_verify(self, stream=None) -> None:
        _check(lib().c2t_build_verify(self._h, C.byref(self._verify_c), _stream(stream)), "c2t_build_verify")

    def c2t_accept(self, target_logits: torch.Tensor, stream=None) -> None:
        """target_logits: [B, >=Nw, V] CUDA tensor of the configured dtype."""
        t = target_logits
        assert t.is_cuda and t.dtype == self.cfg.torch_dtype and t.dim() == 3
        assert t.shape[0] == self.B and t.shape[2] == self.V and t.stride(2) == 1
        _check(lib().c2t_accept(self._h, t.data_ptr(), t.stride(0), t.stride(1), C.byref(self._accept_c),
                                _stream(stream)), "c2t_accept")

    def c2t_argmax_shard(self, target_shard: torch.Tensor, vocab_begin: int, keys: torch.Tensor, stream=None) -> None:
        """target_shard: [B, >=Nw, vocab_count] CUDA tensor of the configured dtype; keys: [B, Nw] int64 CUDA
        tensor (the 64-bit keys, as raw bits)."""
        t = target_shard
        assert t.is_cuda and t.dtype == self.cfg.torch_dtype and t.dim() == 3 and t.shape[0] == self.B
        assert t.stride(2) == 1
        assert keys.is_cuda and keys.dtype == torch.int64 and keys.is_contiguous() and keys.numel() == self.B * self.Nw
        _check(lib().c2t_argmax_shard(self._h, t.data_ptr(), t.stride(0), t.stride(1), t.shape[2], vocab_begin,
                                      keys.data_ptr(), _stream(stream)), "c2t_argmax_shard")

    def c2t_accept_gathered(self, keys: torch.Tensor, stream=None) -> None:
        """keys: [n_shards, B, Nw] int64 CUDA tensor of gathered keys."""
        assert keys.is_cuda and keys.dtype == torch.int64 and keys.is_contiguous() and keys.dim() == 3
        assert keys.shape[1:] == (self.B, self.Nw)
        _check(lib().c2t_accept_gathered(self._h, keys.data_ptr(), keys.shape[0], C.byref(self._accept_c),
                                         _stream(stream)), "c2t_accept_gathered")

    def c2t_dense_mask(self, out: torch.Tensor, stream=None) -> None:
        """out: [B, Nw, kv_len] CUDA tensor, float32 or bfloat16, contiguous: the additive tree-attention mask."""
        assert out.is_cuda and out.is_contiguous() and out.dim() == 3
        assert out.shape[0] == self.B and out.shape[1] == self.Nw
        assert out.dtype in (torch.float32, torch.bfloat16)
        _check(lib().c2t_dense_mask(self._h, out.data_ptr(), F32 if out.dtype == torch.float32 else BF16,
                                    out.shape[2], _stream(stream)), "c2t_dense_mask")

    def c2t_accept_lazy(self, target_logits: torch.Tensor, stream=None) -> None:
        """As c2t_accept, reading only the target rows on the accepted path."""
        t = target_logits
        assert t.is_cuda and t.dtype == self.cfg.torch_dtype and t.dim() == 3
        assert t.shape[0] == self.B and t.shape[2] == self.V and t.stride(2) == 1
        _check(lib().c2t_accept_lazy(self._h, t.data_ptr(), t.stride(0), t.stride(1), C.byref(self._accept_c),
                                     _stream(stream)), "c2t_accept_lazy")

    def c2t_lazy_begin(self, stream=None) -> None:
        _check(lib().c2t_lazy_begin(self._h, C.byref(self._accept_c), _stream(stream)), "c2t_lazy_begin")

    def c2t_lazy_argmax_shard(self, target_shard: torch.Tensor, vocab_begin: int, keys: torch.Tensor, stream=None) -> None:
        """target_shard: [B, >=Nw, vocab_count] CUDA tensor of the configured dtype; keys: [B] int64 CUDA tensor."""
        t = target_shard
        assert t.is_cuda and t.dtype == self.cfg.torch_dtype and t.dim() == 3 and t.shape[0] == self.B
        assert t.stride(2) == 1
        assert keys.is_cuda and keys.dtype == torch.int64 and keys.is_contiguous() and keys.numel() == self.B
        _check(lib().c2t_lazy_argmax_shard(self._h, t.data_ptr(), t.stride(0), t.stride(1), t.shape[2], vocab_begin,
                                           keys.data_ptr(), _stream(stream)), "c2t_lazy_argmax_shard")

    def c2t_lazy_step_gathered(self, round_: int, keys: torch.Tensor, stream=None) -> None:
        """keys: [n_shards, B] int64 CUDA tensor of gathered keys."""
        assert keys.is_cuda and keys.dtype == torch.int64 and keys.is_contiguous() and keys.dim() == 2
        assert keys.shape[1] == self.B
        _check(lib().c2t_lazy_step_gathered(self._h, round_, keys.data_ptr(), keys.shape[0], C.byref(self._accept_c),
                                            _stream(stream)), "c2t_lazy_step_gathered")

    def c2t_status(self, stream=None):
        """(OR of all status words, per-sequence words as a list).  Synchronises the stream."""
        bits = C.c_uint32()
        per = (C.c_uint32 * self.B)()
        _check(lib().c2t_status(self._h, C.byref(bits), per, _stream(stream)), "c2t_status")
        return bits.value, list(per)

    def c2t_launch_count(self) -> int:
        return lib().c2t_launch_count(self._h)

    def c2t_get_view(self) -> dict:
        """Tensors aliasing the workspace (no copies); see `c2t_view` in the header."""
        v = c2t_view()
        _check(lib().c2t_get_view(self._h, C.byref(v)), "c2t_get_view")
        B, F, K, cap, Nw = self.B, self.F, self.K, self.cap, self.Nw
        shapes = {"tree_n": (B,), "cand_n": (B,), "frontier_n": (B,), "final_n": (B,),
                  "frontier_node": (B, F), "topm_from_pass": (B, F)}
        out = {}
        base = self.workspace.data_ptr()
        for name in _VIEW_FIELDS:
            ptr = getattr(v, name)
            if not ptr:                      # (topm_from_pass without a truncated entropy)
                out[name] = None
                continue
            if name in shapes:
                shape = shapes[name]
            elif name.startswith("tree_"):
                shape = (B, cap)
            elif name.startswith("cand_"):
                shape = (B, F * K)
            else:
                shape = (B, Nw)
            dt = torch.float64 if name in ("tree_logP", "tree_C", "tree_Chat", "cand_lp", "cand_logP",
                                           "cand_H", "cand_C") else torch.int32
            n = 1
            for s in shape:
                n *= s
            esz = 8 if dt == torch.float64 else 4
            off = ptr - base
            out[name] = self.workspace[off:off + n * esz].view(dt).view(shape)
        return out

    def c2t_decode_step_host(self, draft_host: Sequence[torch.Tensor], target_host: torch.Tensor,
                             root_host: torch.Tensor, prefix_host: torch.Tensor, results: dict,
                             stage: dict, stream=None) -> None:
        """Whole step from pinned host tensors; `stage` holds the device staging tensors
        ("draft", "target", "ints"), `results` the pinned host result tensors."""
        arr = (C.c_void_p * self.D)(*[t.data_ptr() for t in draft_host])
        io = c2t_host_step(arr, target_host.data_ptr(), root_host.data_ptr(), prefix_host.data_ptr(),
                           stage["draft"].data_ptr(), stage["target"].data_ptr(), stage["ints"].data_ptr(),
                           _dp(results.get("n_nodes")), _dp(results.get("tokens")),
                           _dp(results.get("accept_len")), _dp(results.get("path")),
                           _dp(results.get("next_token")))
        _check(lib().c2t_decode_step_host(self._h, C.byref(io), _stream(stream)), "c2t_decode_step_host")

    def host_step_buffers(self):
        """Device staging and pinned host result tensors for `c2t_decode_step_host`."""
        s, _keep = self.cfg.c_struct()
        n_ints = lib().c2t_host_step_ints(C.byref(s))
        dt = self.cfg.torch_dtype
        stage = {"draft": torch.empty(self.B, self.F, self.V, dtype=dt, device=self.device),
                 "target": torch.empty(self.B, self.Nw, self.V, dtype=dt, device=self.device),
                 "ints": torch.empty(n_ints, dtype=torch.int32, device=self.device)}
        pin = dict(dtype=torch.int32, pin_memory=True)
        results = {"n_nodes": torch.zeros(self.B, **pin), "tokens": torch.zeros(self.B, self.Nw, **pin),
                   "accept_len": torch.zeros(self.B, **pin), "path": torch.zeros(self.B, self.D + 1, **pin),
                   "next_token": torch.zeros(self.B, **pin)}
        return stage, results

    # -- convenience: the call sequence of one decode step on device tensors ---------------
    def decode_step(self, draft_levels: Sequence[torch.Tensor], target: torch.Tensor,
                    root_tok: torch.Tensor, prefix_len: torch.Tensor, stream=None) -> None:
        self.c2t_begin_step(root_tok, prefix_len, stream)
        for level in range(self.D):
            self.c2t_expand_prune_level(level, draft_levels[level], stream)
        self.c2t_prune(FINAL, stream)
        self.c2t_build_verify(stream)
        self.c2t_accept(target, stream)

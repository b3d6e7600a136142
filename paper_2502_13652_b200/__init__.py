"""C2T draft-tree construction (arXiv 2502.13652) as sm_100a CUDA kernels behind libc2t.so.

`binding` is the ctypes layer over the C ABI declared in include/c2t.h; `build` compiles the
library with nvcc.  There is no CPU implementation here and no fallback.
"""
from .binding import (  # noqa: F401
    Config, Context, C2TError, lib, LIB_PATH,
    c2t_workspace_bytes, c2t_tree_capacity, c2t_final_width, c2t_mask_words, c2t_row_argmax_static,
    STATIC_MAX_ROWS, STATIC_MAX_VOCAB,
    F32, BF16, CLS_MLP, CLS_IDENTITY_JOINT, CLS_IDENTITY_COND, ADD_FRONTIER, ADD_ALL_SURVIVORS, FINAL,
    OK, EINVAL, EALIGN, ERANGE, EORDER, ECUDA, ENOMEM,
    ST_NAN_LOGIT, ST_POSINF_LOGIT, ST_ALL_NEGINF, ST_TREE_OVERFLOW, ST_INTERNAL,
)
from .weights import save_classifier, load_classifier  # noqa: F401,E402
from .vocab_parallel import (  # noqa: F401,E402
    shard_ranges, gather_row_records, vocab_parallel_level, vocab_parallel_accept, vocab_parallel_accept_lazy,
    ExchangeBuffers)

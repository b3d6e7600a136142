"""Classifier weights on disk.

The confidence classifier of Eq. 4 is a two-layer network over the features (P, H, d): a hidden
layer of h ReLU units and one sigmoid output (Sec. 4.1; the paper's default is h = 48, its
hidden-size study goes from 2 to 48).  The library takes the four arrays as host pointers at
`c2t_init`; this module only moves them between a file and CPU tensors, so that a classifier
trained elsewhere can be plugged in.  Training is not part of this package.

File layout (little endian): 8 bytes magic "C2TFFN\\0\\1", int32 h, int32 feature count (3),
then float32 W1[h][3] (row-major, columns in the order P, H, d), b1[h], W2[h], b2[1].
"""
from __future__ import annotations

import struct
from typing import Tuple

import numpy as np
import torch

MAGIC = b"C2TFFN\x00\x01"
N_FEATURES = 3
MAX_HIDDEN = 64          # C2T_MAX_HIDDEN in include/c2t.h

Weights = Tuple[torch.Tensor, torch.Tensor, torch.Tensor, torch.Tensor]


def save_classifier(path: str, w1, b1, w2, b2) -> None:
    """Writes (W1 [h,3], b1 [h], W2 [h], b2 [1]) as float32."""
    arrs = [np.ascontiguousarray(torch.as_tensor(a).detach().cpu().to(torch.float32).numpy()) for a in (w1, b1, w2, b2)]
    h = arrs[1].shape[0]
    if not 1 <= h <= MAX_HIDDEN:
        raise ValueError(f"hidden size {h} outside 1..{MAX_HIDDEN}")
    if arrs[0].shape != (h, N_FEATURES) or arrs[2].reshape(-1).shape != (h,) or arrs[3].reshape(-1).shape != (1,):
        raise ValueError("expected W1 [h,3], b1 [h], W2 [h], b2 [1]")
    with open(path, "wb") as f:
        f.write(MAGIC)
        f.write(struct.pack("<ii", h, N_FEATURES))
        for a in arrs:
            f.write(a.astype("<f4", copy=False).tobytes())


def load_classifier(path: str) -> Weights:
    """Reads a file written by `save_classifier`; returns CPU float32 tensors ready for `Config`."""
    with open(path, "rb") as f:
        blob = f.read()
    if len(blob) < 16 or blob[:8] != MAGIC:
        raise ValueError(f"{path}: not a C2T classifier file")
    h, nf = struct.unpack_from("<ii", blob, 8)
    if nf != N_FEATURES or not 1 <= h <= MAX_HIDDEN:
        raise ValueError(f"{path}: hidden size {h}, {nf} features: unsupported")
    n = h * nf + h + h + 1
    if len(blob) != 16 + 4 * n:
        raise ValueError(f"{path}: {len(blob)} bytes, expected {16 + 4 * n}")
    flat = np.frombuffer(blob, dtype="<f4", count=n, offset=16).astype(np.float32)
    if not np.isfinite(flat).all():
        raise ValueError(f"{path}: non-finite weight")
    w1 = torch.from_numpy(flat[:h * nf].reshape(h, nf).copy())
    b1 = torch.from_numpy(flat[h * nf:h * nf + h].copy())
    w2 = torch.from_numpy(flat[h * nf + h:h * nf + 2 * h].copy())
    b2 = torch.from_numpy(flat[h * nf + 2 * h:].copy())
    return w1, b1, w2, b2

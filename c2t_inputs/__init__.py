"""Seeded synthetic inputs for the C2T draft-tree hot path.

This module only produces bytes: draft logits, target logits, root tokens,
prefix lengths and classifier weights.  It contains none of the method's
arithmetic (no softmax, entropy, top-k, classifier or pruning).  The CPU oracle
and the CUDA library both consume the tensors it returns, so a parity check
never depends on two random-number or `log` implementations agreeing.

Recipe (stands in for LLaMA/Vicuna-class draft-head outputs, whose datasets and
weights are not available):

  * each sequence b owns a seeded random permutation of the vocabulary;
    rank(v) in 1..V is token v's place in it;
  * a logits row is  x_v = scale * g_v - s * ln(rank(v)),  g_v standard Gumbel
    noise, s = 1.1 (a Zipf prior), scale = 4 unless stated; rounded
    to-nearest-even into the storage dtype (fp32 or bf16);
  * draft rows are keyed by (sequence, decode step, level, frontier slot),
    target rows by (sequence, decode step, final node index); draft and target
    rows of one sequence share its permutation, which is the only source of
    agreement between the two;
  * classifier weights are N(0, 0.1^2), drawn in the order W1, b1, W2, b2.

Every draw comes from a `torch.Generator` seeded by a hash of the key, so a
tensor is a pure function of (key, device type).  CPU and CUDA generators give
different streams; a test or benchmark generates once and hands the same bytes
to both sides.
"""
from __future__ import annotations

import hashlib
import struct

import torch

MASTER_SEED = 250213652

STREAM_DRAFT = 0
STREAM_TARGET = 1
STREAM_WEIGHTS = 2
STREAM_PERM = 3
STREAM_MISC = 4

__all__ = [
    "MASTER_SEED", "key_seed", "token_rank", "zipf_prior", "draft_logits",
    "target_logits", "classifier_weights", "root_tokens", "prefix_lengths",
]


def key_seed(*key: int, master: int = MASTER_SEED) -> int:
    """63-bit seed from an integer key tuple (stateless, order-sensitive)."""
    payload = struct.pack("<%dq" % (len(key) + 1), master, *[int(k) for k in key])
    digest = hashlib.blake2b(payload, digest_size=8).digest()
    return int.from_bytes(digest, "little") & ((1 << 63) - 1)


def _generator(device, *key: int, master: int = MASTER_SEED) -> torch.Generator:
    gen = torch.Generator(device=device)
    gen.manual_seed(key_seed(*key, master=master))
    return gen


def token_rank(seq: int, vocab: int, device="cpu", master: int = MASTER_SEED) -> torch.Tensor:
    """rank(v) in 1..V for sequence `seq`: position of v in a seeded permutation."""
    gen = _generator(device, STREAM_PERM, seq, master=master)
    perm = torch.randperm(vocab, generator=gen, device=device)
    rank = torch.empty(vocab, dtype=torch.int64, device=device)
    rank[perm] = torch.arange(1, vocab + 1, dtype=torch.int64, device=device)
    return rank


def zipf_prior(seq: int, vocab: int, s: float = 1.1, device="cpu",
               master: int = MASTER_SEED) -> torch.Tensor:
    """-s * ln(rank(v)) as float32 [V]."""
    return (-s) * torch.log(token_rank(seq, vocab, device, master).to(torch.float32))


def _gumbel(shape, gen: torch.Generator, device) -> torch.Tensor:
    u = torch.rand(shape, generator=gen, device=device, dtype=torch.float32)
    u = u.clamp_(2.0 ** -25, 1.0 - 2.0 ** -25)
    return -torch.log(-torch.log(u))


def _rows(stream: int, batch: int, rows: int, vocab: int, step: int, level: int,
          dtype: torch.dtype, scale: float, s: float, device, seq_base: int,
          master: int) -> torch.Tensor:
    out = torch.empty((batch, rows, vocab), dtype=dtype, device=device)
    for b in range(batch):
        seq = seq_base + b
        prior = zipf_prior(seq, vocab, s, device, master)
        gen = _generator(device, stream, seq, step, level, master=master)
        x = _gumbel((rows, vocab), gen, device).mul_(scale).add_(prior)
        out[b] = x.to(dtype)
    return out


def draft_logits(batch: int, frontier_cap: int, vocab: int, step: int, level: int,
                 dtype: torch.dtype = torch.float32, scale: float = 4.0, s: float = 1.1,
                 device="cpu", seq_base: int = 0, master: int = MASTER_SEED) -> torch.Tensor:
    """Draft-model logits for one level: [B, F, V]; row (b, j) belongs to frontier slot j.

    Rows exist for all F slots; slots beyond a sequence's frontier size are never read.
    """
    return _rows(STREAM_DRAFT, batch, frontier_cap, vocab, step, level, dtype, scale, s,
                 device, seq_base, master)


def target_logits(batch: int, nodes: int, vocab: int, step: int,
                  dtype: torch.dtype = torch.float32, scale: float = 4.0, s: float = 1.1,
                  device="cpu", seq_base: int = 0, master: int = MASTER_SEED) -> torch.Tensor:
    """Target-model logits over the final tree: [B, N, V]; row (b, i) belongs to final node i."""
    return _rows(STREAM_TARGET, batch, nodes, vocab, step, 0, dtype, scale, s,
                 device, seq_base, master)


def classifier_weights(hidden: int, seed: int = 0, std: float = 0.1,
                       master: int = MASTER_SEED):
    """(W1 [h,3], b1 [h], W2 [h], b2 [1]) float32 on CPU, N(0, std^2), drawn in that order."""
    gen = _generator("cpu", STREAM_WEIGHTS, seed, hidden, master=master)
    w1 = torch.randn((hidden, 3), generator=gen, dtype=torch.float32) * std
    b1 = torch.randn((hidden,), generator=gen, dtype=torch.float32) * std
    w2 = torch.randn((hidden,), generator=gen, dtype=torch.float32) * std
    b2 = torch.randn((1,), generator=gen, dtype=torch.float32) * std
    return w1.contiguous(), b1.contiguous(), w2.contiguous(), b2.contiguous()


def root_tokens(batch: int, vocab: int, step: int = 0, seq_base: int = 0,
                master: int = MASTER_SEED) -> torch.Tensor:
    """Root token per sequence (the target model's own last token): int32 [B] on CPU."""
    gen = _generator("cpu", STREAM_MISC, seq_base, step, batch, master=master)
    return torch.randint(0, vocab, (batch,), generator=gen, dtype=torch.int64).to(torch.int32)


def prefix_lengths(batch: int, low: int = 16, high: int = 2048, seq_base: int = 0,
                   master: int = MASTER_SEED) -> torch.Tensor:
    """Committed-prefix length per sequence: int32 [B] on CPU."""
    gen = _generator("cpu", STREAM_MISC, seq_base, -1, batch, master=master)
    return torch.randint(low, high, (batch,), generator=gen, dtype=torch.int64).to(torch.int32)

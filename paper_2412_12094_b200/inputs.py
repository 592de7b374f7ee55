"""Seeded synthetic inputs for the SepLLM attention path.

This module only draws random numbers and shapes them; it holds none of the
method's arithmetic (no mask, no softmax, no cache rule).  Both the CUDA tests
and the CPU oracle tests read their inputs from here so that they see the same
bits.  Real token streams and activations (the paper trains on the Pile and
streams PG19) are replaced by these stand-ins.

Recipe
------
* token ids: uniform over a 50 000-entry vocabulary with the nine separator
  ids removed, then separator positions are overwritten with one of the nine
  ids drawn uniformly.  Separator positions are either i.i.d. Bernoulli(rho)
  ("iid") or the ends of segments whose lengths are geometric with mean 1/rho
  ("geometric"): a segment of length g is g-1 ordinary tokens followed by its
  separator.
* Q, K, V, dO: N(0,1) in fp32, rounded to nearest-even bf16.
* document boundaries of packed rows: document lengths geometric with a given
  mean (the length mix of a packed pre-training row: many short documents, a
  few long ones), a 1 at the first token of every document but the first.
"""
from __future__ import annotations

import numpy as np
import torch

VOCAB = 50000
# Nine distinct synthetic ids standing in for '.', ',', '?', '!', ';', ':',
# ' ', '\t', '\n'.  The paper names the strings only; real ids depend on a
# tokenizer that is not available here.
SEP_IDS = np.array([11, 13, 29, 101, 1027, 2048, 4099, 17000, 49999], dtype=np.int32)


def _rng(seed: int, stream: int) -> np.random.Generator:
    return np.random.Generator(np.random.Philox(key=[int(seed), int(stream)]))


def token_ids(seed: int, B: int, L: int, rho: float, structure: str = "iid") -> np.ndarray:
    """int32 [B][L] token ids with separators placed as the recipe says."""
    g = _rng(seed, 0)
    non_sep = np.setdiff1d(np.arange(VOCAB, dtype=np.int32), SEP_IDS)
    ids = non_sep[g.integers(0, non_sep.size, size=(B, L))].astype(np.int32)
    if rho <= 0.0:
        return ids
    if structure == "iid":
        is_sep = g.random((B, L)) < rho
    elif structure == "geometric":
        is_sep = np.zeros((B, L), dtype=bool)
        for b in range(B):
            # enough gaps to cover L with overwhelming probability
            n_gaps = int(L * rho * 1.5) + 64
            pos = np.cumsum(g.geometric(rho, size=n_gaps)) - 1
            while pos[-1] < L:  # pragma: no cover - practically never
                more = np.cumsum(g.geometric(rho, size=n_gaps)) + pos[-1]
                pos = np.concatenate([pos, more])
            is_sep[b, pos[pos < L]] = True
    else:
        raise ValueError(structure)
    which = SEP_IDS[g.integers(0, SEP_IDS.size, size=(B, L))]
    ids = np.where(is_sep, which, ids).astype(np.int32)
    return ids


def doc_first(seed: int, B: int, L: int, mean_len: float) -> np.ndarray:
    """int32 [B][L]: 1 where a new document begins inside a packed row (position 0 begins one
    without being marked)."""
    g = _rng(seed, 9)
    out = np.zeros((B, L), dtype=np.int32)
    for b in range(B):
        pos = 0
        while True:
            pos += int(g.geometric(1.0 / mean_len))
            if pos >= L:
                break
            out[b, pos] = 1
    return out


def normal_bf16(seed: int, stream: int, shape) -> torch.Tensor:
    """N(0,1) tensor rounded to bf16 (CPU)."""
    g = _rng(seed, stream)
    x = g.standard_normal(size=shape, dtype=np.float32)
    return torch.from_numpy(x).to(torch.bfloat16)


def qkv_do(seed: int, B: int, Hq: int, Hkv: int, L: int, d: int):
    """Q, K, V, dO as bf16 CPU tensors, layouts [B][H][L][d]."""
    Q = normal_bf16(seed, 1, (B, Hq, L, d))
    K = normal_bf16(seed, 2, (B, Hkv, L, d))
    V = normal_bf16(seed, 3, (B, Hkv, L, d))
    dO = normal_bf16(seed, 4, (B, Hq, L, d))
    return Q, K, V, dO


# The five workloads (shapes, token structure, a, n) used by tests and bench.
CONFIGS = {
    "tiny": dict(B=1, Hq=2, Hkv=2, d=64, L=512, rho=0.12, structure="iid",
                 n_init=4, n_neighbor=64, seed=1001),
    "pythia160m": dict(B=8, Hq=12, Hkv=12, d=64, L=2048, rho=0.12, structure="iid",
                       n_init=4, n_neighbor=256, seed=1002),
    "llama8b_prefill": dict(B=1, Hq=32, Hkv=8, d=128, L=8192, rho=0.10, structure="geometric",
                            n_init=4, n_neighbor=256, seed=1003),
    # a shorter copy of the long-context shape, for profiler captures (inputs still exceed L2)
    "llama8b_L16k_r10": dict(B=1, Hq=32, Hkv=8, d=128, L=16384, rho=0.10, structure="geometric",
                             n_init=4, n_neighbor=512, seed=1008),
    "llama8b_long_r05": dict(B=1, Hq=32, Hkv=8, d=128, L=65536, rho=0.05, structure="geometric",
                             n_init=4, n_neighbor=512, seed=1004),
    "llama8b_long_r10": dict(B=1, Hq=32, Hkv=8, d=128, L=65536, rho=0.10, structure="geometric",
                             n_init=4, n_neighbor=512, seed=1005),
    "llama8b_long_r20": dict(B=1, Hq=32, Hkv=8, d=128, L=65536, rho=0.20, structure="geometric",
                             n_init=4, n_neighbor=512, seed=1006),
}

DECODE_CONFIG = dict(B=32, Hq=32, Hkv=8, d=128, a=4, s=1024, w=256, c=3332, rho=0.12,
                     stream_len=1 << 20, seed=1007)


def decode_stream_ids(seed: int, B: int, T: int, rho: float) -> np.ndarray:
    """int32 [B][T] token ids of the streaming-decode workload (i.i.d. separators)."""
    return token_ids(seed, B, T, rho, "iid")


def decode_kv_pool(seed: int, steps: int, B: int, Hkv: int, Hq: int, d: int):
    """Per-step new k, v ([steps][B][Hkv][d]) and q ([steps][B][Hq][d]), bf16 CPU."""
    k = normal_bf16(seed, 11, (steps, B, Hkv, d))
    v = normal_bf16(seed, 12, (steps, B, Hkv, d))
    q = normal_bf16(seed, 13, (steps, B, Hq, d))
    return k, v, q

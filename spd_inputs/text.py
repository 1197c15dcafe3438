"""Synthetic token streams, prefixes and n-gram frequency tables.

The paper counts n-grams (n = 2..6) over about 200 M RedPajama tokens and stores
"each unique n-gram and its count" (Section 4).  That corpus is not available, so a
Zipf-distributed token stream of the same length stands in.  A table is emitted in a
neutral form: unique n-grams as rows of an int32 array in lexicographic order, with an
int64 count per row.  Nothing here computes probabilities.
"""
from __future__ import annotations

from typing import Dict, List, Sequence

import numpy as np
import torch

from .rng import hash_u64, uniform01

_BITS = 21                      # bits per token inside a packed sort key (vocab < 2^21)
_PER_WORD = 3                   # tokens per 63-bit word
_CHUNK = 1 << 24


def zipf_cdf(vocab: int, s: float) -> np.ndarray:
    """Cumulative distribution of P(rank r) ~ r^-s, r = 1..vocab (float64, computed on the host)."""
    w = np.arange(1, vocab + 1, dtype=np.float64) ** (-float(s))
    c = np.cumsum(w)
    return c / c[-1]


def zipf_tokens(seed: int, tensor_id: int, length: int, vocab: int, s: float,
                device: str | torch.device = "cpu") -> torch.Tensor:
    """`length` token ids (int64); token id = Zipf rank - 1, drawn by inverse CDF."""
    cdf = torch.from_numpy(zipf_cdf(vocab, s)).to(device)
    out = torch.empty(length, dtype=torch.int64, device=device)
    for lo in range(0, length, _CHUNK):
        hi = min(length, lo + _CHUNK)
        idx = torch.arange(lo, hi, dtype=torch.int64, device=device)
        u = uniform01(hash_u64(seed, tensor_id, idx))
        out[lo:hi] = torch.searchsorted(cdf, u).clamp_(max=vocab - 1)
    return out


def make_prefix(kind: str, length: int, vocab: int, s: float = 1.1, seed: int = 2,
                tensor_id: int = 0) -> List[int]:
    """Prefix token ids: 'uniform' over the vocabulary, or 'zipf' with exponent s."""
    idx = torch.arange(length, dtype=torch.int64)
    if kind == "uniform":
        u = uniform01(hash_u64(seed, tensor_id, idx))
        ids = torch.floor(u * vocab).to(torch.int64).clamp_(max=vocab - 1)
    elif kind == "zipf":
        ids = zipf_tokens(seed, tensor_id, length, vocab, s)
    else:
        raise ValueError(kind)
    return [int(x) for x in ids]


def _pack(stream: torch.Tensor, start: int, cnt: int, rows: int) -> torch.Tensor:
    w = torch.zeros(rows, dtype=torch.int64, device=stream.device)
    for j in range(cnt):
        w = (w << _BITS) | stream[start + j:start + j + rows]
    return w


def count_ngrams(stream: torch.Tensor, n: int, retain: int | None = None) -> Dict[str, torch.Tensor]:
    """Unique n-grams of `stream` with their occurrence counts.

    Returns {'n', 'keys' int32 [N, n] in lexicographic order, 'counts' int64 [N]}.  With
    `retain`, only the `retain` most frequent n-grams are kept (count descending, ties by
    smaller key), still listed in lexicographic order.
    """
    if not 1 <= n <= 2 * _PER_WORD:
        raise ValueError("n must be in 1..6")
    rows = stream.numel() - n + 1
    if rows <= 0:
        return {"n": n, "keys": torch.zeros((0, n), dtype=torch.int32),
                "counts": torch.zeros(0, dtype=torch.int64)}
    n_hi = min(n, _PER_WORD)
    hi = _pack(stream, 0, n_hi, rows)
    if n > _PER_WORD:
        lo = _pack(stream, _PER_WORD, n - _PER_WORD, rows)
        order = torch.sort(lo, stable=True).indices
        hi = hi[order]
        o2 = torch.sort(hi, stable=True).indices
        hi = hi[o2]
        lo = lo[order[o2]]
        del order, o2
        new = torch.ones(rows, dtype=torch.bool, device=stream.device)
        new[1:] = (hi[1:] != hi[:-1]) | (lo[1:] != lo[:-1])
    else:
        lo = None
        hi = torch.sort(hi).values
        new = torch.ones(rows, dtype=torch.bool, device=stream.device)
        new[1:] = hi[1:] != hi[:-1]
    starts = torch.nonzero(new).squeeze(1)
    del new
    ends = torch.cat([starts[1:], torch.tensor([rows], dtype=torch.int64, device=stream.device)])
    counts = ends - starts
    hi = hi[starts]
    if lo is not None:
        lo = lo[starts]
    if retain is not None and counts.numel() > retain:
        top = torch.sort(-counts, stable=True).indices[:retain]
        sel = torch.sort(top).values
        counts, hi = counts[sel], hi[sel]
        if lo is not None:
            lo = lo[sel]
    keys = torch.empty((counts.numel(), n), dtype=torch.int32, device=stream.device)
    mask = (1 << _BITS) - 1
    for j in range(n_hi):
        keys[:, j] = ((hi >> (_BITS * (n_hi - 1 - j))) & mask).to(torch.int32)
    for j in range(n - n_hi):
        keys[:, n_hi + j] = ((lo >> (_BITS * (n - n_hi - 1 - j))) & mask).to(torch.int32)
    return {"n": n, "keys": keys.cpu().contiguous(), "counts": counts.cpu().contiguous()}


def make_ngram_tables(vocab: int, s: float, length: int, orders: Sequence[int], retain: int | None,
                      seed: int = 1, device: str | torch.device = "cpu") -> List[Dict[str, torch.Tensor]]:
    """Frequency tables for each order in `orders`, counted over one Zipf(s) stream of `length` tokens."""
    stream = zipf_tokens(seed, 0, length, vocab, s, device)
    return [count_ngrams(stream, n, retain) for n in orders]

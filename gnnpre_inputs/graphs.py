"""Seeded synthetic graphs in CSR form (rowptr int64, colidx int32).

Two families, standing in for the public datasets the paper measures on:

* Erdos-Renyi G(n, m): m distinct unordered pairs drawn uniformly.
* R-MAT (Chakrabarti, Zhan, Faloutsos, SDM 2004) with quadrant probabilities
  (a, b, c, d), vertices relabelled by a seeded permutation so that vertex ids
  carry no locality, as in real citation graphs.

Edges are the first `m` distinct valid candidates in counter order, so a graph
depends only on (seed, parameters), never on chunk sizes or the device used.
Every graph returned is symmetric, has no self-loops and no duplicate edges,
and lists each row's columns in ascending order.

This module holds no arithmetic of the propagation method itself.
"""
from __future__ import annotations

import math
from dataclasses import dataclass

import torch

from . import rng

STREAM_EDGES = 1
STREAM_RELABEL = 2


@dataclass
class CSRGraph:
    n: int
    rowptr: torch.Tensor  # int64 [n+1]
    colidx: torch.Tensor  # int32 [nnz]

    @property
    def nnz(self) -> int:
        return int(self.colidx.numel())

    def to(self, device) -> "CSRGraph":
        return CSRGraph(self.n, self.rowptr.to(device), self.colidx.to(device))


def _first_m_distinct(candidates, m: int, device, start_factor: float = 1.3) -> torch.Tensor:
    """Keys of the first `m` distinct valid candidates in counter order.

    `candidates(counter)` maps an int64 counter tensor to int64 keys, with -1
    marking a rejected candidate.  Returned keys are sorted ascending.
    """
    if m == 0:
        return torch.empty(0, dtype=torch.int64, device=device)
    total = int(m * start_factor) + 1024
    while True:
        counter = torch.arange(total, dtype=torch.int64, device=device)
        keys = candidates(counter)
        del counter
        order = torch.argsort(keys, stable=True)  # ties keep counter order
        keys = keys[order]
        first = torch.ones_like(keys, dtype=torch.bool)
        first[1:] = keys[1:] != keys[:-1]
        first &= keys >= 0
        first_counter = order[first]
        keys = keys[first]
        del order, first
        if keys.numel() >= m:
            if keys.numel() > m:
                # keep the m distinct keys that appeared earliest
                kth = torch.sort(first_counter).values[m - 1]
                keys = keys[first_counter <= kth]
            return keys  # still ascending: a mask keeps order
        del keys, first_counter
        total = int(total * 1.5) + 1024


def _csr_from_directed_keys(keys: torch.Tensor, n: int) -> CSRGraph:
    """keys = row * n + col, sorted ascending and distinct."""
    rows = torch.div(keys, n, rounding_mode="floor")
    cols = (keys - rows * n).to(torch.int32)
    counts = torch.bincount(rows, minlength=n)
    rowptr = torch.zeros(n + 1, dtype=torch.int64, device=keys.device)
    torch.cumsum(counts, 0, out=rowptr[1:])
    return CSRGraph(n, rowptr, cols)


def _symmetrise(src: torch.Tensor, dst: torch.Tensor, n: int) -> CSRGraph:
    """Union of the edge set with its transpose; reciprocal pairs merge."""
    keys = torch.cat([src * n + dst, dst * n + src])
    keys = torch.unique(keys)  # sorted
    return _csr_from_directed_keys(keys, n)


def erdos_renyi(n: int, m_undirected: int, seed: int, device="cpu") -> CSRGraph:
    """G(n, m): m distinct unordered pairs i<j, then both directions."""
    assert 2 <= n < 2 ** 31 and m_undirected <= n * (n - 1) // 2
    key = rng.stream_key(seed, STREAM_EDGES)

    def candidates(counter):
        bits = rng.mix64(key, counter)
        u = rng.below(rng.hi32(bits), n)
        v = rng.below(rng.lo32(bits), n)
        lo = torch.minimum(u, v)
        hi = torch.maximum(u, v)
        k = lo * n + hi
        return torch.where(u == v, torch.full_like(k, -1), k)

    pairs = _first_m_distinct(candidates, m_undirected, device, start_factor=1.1)
    lo = torch.div(pairs, n, rounding_mode="floor")
    hi = pairs - lo * n
    return _symmetrise(lo, hi, n)


def _rmat_endpoints(key: int, counter: torch.Tensor, scale: int, abcd) -> tuple:
    a, b, c, _ = abcd
    t_a = int(round(a * 2 ** 32))
    t_ab = int(round((a + b) * 2 ** 32))
    t_abc = int(round((a + b + c) * 2 ** 32))
    u = torch.zeros_like(counter)
    v = torch.zeros_like(counter)
    bits = None
    for level in range(scale):
        if level % 2 == 0:
            # one 64-bit draw serves two levels; each level has its own key
            bits = rng.mix64(key ^ ((level // 2 + 1) * 0xD1B54A32D192ED03 & ((1 << 64) - 1)), counter)
            r = rng.hi32(bits)
        else:
            r = rng.lo32(bits)
        ubit = (r >= t_ab).to(torch.int64)                       # quadrants c, d: lower half
        vbit = ((r >= t_a) & (r < t_ab) | (r >= t_abc)).to(torch.int64)  # quadrants b, d: right half
        u = (u << 1) | ubit
        v = (v << 1) | vbit
    return u, v


def _relabel(n: int, seed: int, device) -> torch.Tensor:
    """label[old_id] = new id: a seeded permutation of [0, n)."""
    key = rng.stream_key(seed, STREAM_RELABEL)
    h = rng.mix64(key, torch.arange(n, dtype=torch.int64, device=device))
    order = torch.argsort(h, stable=True)
    label = torch.empty(n, dtype=torch.int64, device=device)
    label[order] = torch.arange(n, dtype=torch.int64, device=device)
    return label


def rmat(n: int, m: int, seed: int, *, directed_candidates: bool, abcd=(0.57, 0.19, 0.19, 0.05),
         device="cpu") -> CSRGraph:
    """R-MAT graph on n vertices, symmetrised.

    directed_candidates=True : the first m distinct directed edges (i, j), i != j,
        are kept and then symmetrised, so reciprocal pairs merge (nnz <= 2m).
    directed_candidates=False: the first m distinct unordered pairs are kept
        (nnz == 2m).
    Candidates with an endpoint >= n are rejected (n need not be a power of two).
    """
    assert 2 <= n < 2 ** 31
    scale = max(1, math.ceil(math.log2(n)))
    key = rng.stream_key(seed, STREAM_EDGES)

    def candidates(counter):
        u, v = _rmat_endpoints(key, counter, scale, abcd)
        bad = (u == v) | (u >= n) | (v >= n)
        if directed_candidates:
            k = u * n + v
        else:
            k = torch.minimum(u, v) * n + torch.maximum(u, v)
        return torch.where(bad, torch.full_like(k, -1), k)

    kept = _first_m_distinct(candidates, m, device, start_factor=1.5)
    src = torch.div(kept, n, rounding_mode="floor")
    dst = kept - src * n
    del kept
    label = _relabel(n, seed, device)
    return _symmetrise(label[src], label[dst], n)


def from_edge_list(n: int, edges, device="cpu") -> CSRGraph:
    """Small hand-written graphs for tests: undirected pairs -> symmetric CSR."""
    if len(edges) == 0:
        return CSRGraph(n, torch.zeros(n + 1, dtype=torch.int64, device=device),
                        torch.empty(0, dtype=torch.int32, device=device))
    e = torch.tensor(list(edges), dtype=torch.int64, device=device).reshape(-1, 2)
    assert bool((e[:, 0] != e[:, 1]).all()), "self-loops are not part of A"
    return _symmetrise(e[:, 0], e[:, 1], n)

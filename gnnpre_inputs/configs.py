"""The five benchmark workloads as seeded synthetic inputs.

Shapes follow the paper's dataset table (nodes / edges / feature widths of the
citation and co-purchase graphs it measures on); the graphs themselves are
synthetic stand-ins, because the public datasets are not available offline.

  c1  Erdos-Renyi, 4,096 nodes, 32,768 undirected edges, F=64,  K=2, GCN, b=1
  c2  R-MAT, 169,343 nodes, 1,166,243 directed edges symmetrised, F=128, K=3, GCN, b=4
  c3  operator / width / block-count sweep on the c2 graph
  c4  R-MAT, 2,449,029 nodes, 61,859,140 undirected edges, F=100, K=3, SAGE, b=32
  c5  R-MAT, 111,059,956 nodes, 807,842,936 undirected edges, F=128, K=2, GCN, streamed

and two more with the node count, edge count and feature width of the two wide-feature datasets of
that table (rows of 2,000 and 2,408 bytes):

  flickr  R-MAT,  89,250 nodes,    899,756 undirected edges, F=500, K=2, GCN
  reddit  R-MAT, 232,965 nodes, 11,606,919 undirected edges, F=602, K=2, GCN

This module holds no arithmetic of the propagation method itself.
"""
from __future__ import annotations

from dataclasses import dataclass, field

from . import features, graphs

BASE_SEED = 220712000

OP_GCN, OP_SAGE, OP_GIN = 0, 1, 2


@dataclass(frozen=True)
class Workload:
    name: str
    kind: str            # "er" or "rmat"
    n: int
    m: int               # edges drawn (see directed)
    directed: bool       # R-MAT only: m counts directed candidates
    feat_dim: int
    hops: int
    op: int
    blocks: int          # forced b (0 = solve the budget)
    seed: int
    gin_eps: float = 0.0
    streamed: bool = False
    sweep: dict = field(default_factory=dict)


WORKLOADS = {
    "c1": Workload("c1", "er", 4096, 32768, False, 64, 2, OP_GCN, 1, BASE_SEED + 0),
    "c2": Workload("c2", "rmat", 169343, 1166243, True, 128, 3, OP_GCN, 4, BASE_SEED + 1),
    "c3": Workload("c3", "rmat", 169343, 1166243, True, 128, 3, OP_GCN, 1, BASE_SEED + 1, gin_eps=0.1,
                   sweep={"ops": (OP_GCN, OP_SAGE, OP_GIN), "feat_dims": (16, 64, 128, 256, 512),
                          "blocks": (1, 8, 64)}),
    "c4": Workload("c4", "rmat", 2449029, 61859140, False, 100, 3, OP_SAGE, 32, BASE_SEED + 3),
    "c5": Workload("c5", "rmat", 111059956, 807842936, False, 128, 2, OP_GCN, 0, BASE_SEED + 4,
                   streamed=True),
    "flickr": Workload("flickr", "rmat", 89250, 899756, False, 500, 2, OP_GCN, 0, BASE_SEED + 5),
    "reddit": Workload("reddit", "rmat", 232965, 11606919, False, 602, 2, OP_GCN, 0, BASE_SEED + 6),
}


def scaled(w: Workload, divisor: int) -> Workload:
    """Same structure with nodes and edges divided by `divisor` (mean degree kept)."""
    if divisor == 1:
        return w
    return Workload(f"{w.name}/{divisor}", w.kind, max(2, w.n // divisor), max(1, w.m // divisor), w.directed,
                    w.feat_dim, w.hops, w.op, w.blocks, w.seed, w.gin_eps, w.streamed, w.sweep)


def make_graph(w: Workload, device="cpu") -> graphs.CSRGraph:
    if w.kind == "er":
        return graphs.erdos_renyi(w.n, w.m, w.seed, device=device)
    return graphs.rmat(w.n, w.m, w.seed, directed_candidates=w.directed, device=device)


def make_features(w: Workload, device="cpu", feat_dim: int | None = None, ld: int | None = None):
    return features.normal_matrix(w.n, feat_dim or w.feat_dim, w.seed, device=device, ld=ld)

"""Seeded synthetic inputs shared by the tests and the benchmark.

This module holds none of the method's arithmetic: it only draws graphs, tables and
query lists.  The graphs stand in for WikiKG90Mv2 (Section 2, dataset table): power-law
entity degrees, skewed relation frequencies, entity ids scrambled by a random permutation
so that hot rows spread over all partitions (the paper's "random partitioning").
"""
from __future__ import annotations

import numpy as np


def _bounded_zipf(rng: np.random.Generator, n_items: int, s: float, size: int) -> np.ndarray:
    """`size` draws of a rank in [0, n_items) with P(rank k) proportional to (k+1)^-s."""
    if s == 0.0:
        return rng.integers(0, n_items, size=size, dtype=np.int64)
    w = np.arange(1, n_items + 1, dtype=np.float64) ** (-s)
    cdf = np.cumsum(w)
    cdf /= cdf[-1]
    u = rng.random(size)
    return np.minimum(np.searchsorted(cdf, u, side="right"), n_items - 1).astype(np.int64)


def make_graph(num_entities: int, num_relations: int, num_triples: int, *, seed: int,
               entity_zipf: float = 1.1, relation_zipf: float = 0.0):
    """Triples (h, r, t) as int32 arrays.  Heads and tails are drawn independently from a
    Zipf(entity_zipf) law over popularity ranks, rank -> id through a seeded permutation;
    relations Zipf(relation_zipf) over a permuted relation order (0.0 = uniform).
    Duplicates and self-loops are allowed."""
    rng = np.random.default_rng(seed)
    perm = rng.permutation(num_entities).astype(np.int32)
    h = perm[_bounded_zipf(rng, num_entities, entity_zipf, num_triples)]
    t = perm[_bounded_zipf(rng, num_entities, entity_zipf, num_triples)]
    rperm = rng.permutation(num_relations).astype(np.int32)
    r = rperm[_bounded_zipf(rng, num_relations, relation_zipf, num_triples)]
    return np.ascontiguousarray(h), np.ascontiguousarray(r), np.ascontiguousarray(t)


def make_tables(num_entities: int, num_relations: int, dim: int, score: str, *, seed: int):
    """fp32 tables: entity rows N(0, std 1/sqrt(dim)); relation rows the same, except RotatE
    whose dim/2 phases are uniform in [-pi, pi]; TransH also gets a table of normals."""
    rng = np.random.default_rng(seed + 1_000_003)
    std = 1.0 / np.sqrt(dim)
    ent = (rng.standard_normal((num_entities, dim)) * std).astype(np.float32)
    if score in ("rotate", "rotate_real_l1"):
        rel = rng.uniform(-np.pi, np.pi, size=(num_relations, dim // 2)).astype(np.float32)
    else:
        rel = (rng.standard_normal((num_relations, dim)) * std).astype(np.float32)
    relw = None
    if score == "transh":
        relw = (rng.standard_normal((num_relations, dim)) * std).astype(np.float32)
    return ent, rel, relw


def make_queries(num_entities: int, num_relations: int, num_queries: int, *, seed: int,
                 entity_zipf: float = 1.1):
    """(h, r) queries with Zipf heads, uniform relations, and a uniform designated true tail."""
    rng = np.random.default_rng(seed + 2_000_003)
    perm = rng.permutation(num_entities).astype(np.int32)
    qh = perm[_bounded_zipf(rng, num_entities, entity_zipf, num_queries)]
    qr = rng.integers(0, num_relations, size=num_queries).astype(np.int32)
    tt = rng.integers(0, num_entities, size=num_queries).astype(np.int32)
    return np.ascontiguousarray(qh), qr, tt


def make_graph_device(num_entities: int, num_relations: int, num_triples: int, *, seed: int, device,
                      entity_zipf: float = 1.1, relation_zipf: float = 0.0, chunk: int = 1 << 25):
    """The law of `make_graph` drawn on a GPU with torch's seeded generator, for graphs too large to draw
    (or to hold three times over) on the host: int32 device tensors (h, r, t).  The random stream differs
    from `make_graph`'s; the distribution (Zipf popularity ranks through a random permutation) is the same."""
    import torch
    gen = torch.Generator(device=device)
    gen.manual_seed(seed)

    def cdf_of(n_items, s):
        w = torch.arange(1, n_items + 1, dtype=torch.float64, device=device).pow_(-s)
        c = torch.cumsum(w, 0)
        return c.div_(c[-1].clone())

    def draw(n_items, s, perm, out):
        cdf = cdf_of(n_items, s) if s != 0.0 else None
        for lo in range(0, num_triples, chunk):
            n = min(chunk, num_triples - lo)
            if cdf is None:
                ranks = torch.randint(0, n_items, (n,), generator=gen, device=device)
            else:
                u = torch.rand(n, dtype=torch.float64, generator=gen, device=device)
                ranks = torch.searchsorted(cdf, u, right=True).clamp_(max=n_items - 1)
            out[lo:lo + n] = perm[ranks]
        return out

    perm = torch.randperm(num_entities, generator=gen, device=device).to(torch.int32)
    h = draw(num_entities, entity_zipf, perm, torch.empty(num_triples, dtype=torch.int32, device=device))
    t = draw(num_entities, entity_zipf, perm, torch.empty(num_triples, dtype=torch.int32, device=device))
    rperm = torch.randperm(num_relations, generator=gen, device=device).to(torch.int32)
    r = draw(num_relations, relation_zipf, rperm, torch.empty(num_triples, dtype=torch.int32, device=device))
    return h, r, t

"""Full-entity inference with the entity table sharded row-wise over several devices (Section 4 "Inference").

Every rank holds one shard of the entity table (rows ``[ent_base, ent_base + rows)``) and whole relation tables.
The protocol is the paper's: the query heads' information is shared between the workers, every worker scores ALL
queries against its own shard and returns its top-K, and a final top-K over the D * K gathered candidates selects
the predictions; the rank of the true tail is one plus the shards' counts of entities ordered before it.

This module holds the plumbing only -- which small per-query array is summed or gathered when.  The arithmetic is
behind ``local``: an object with four methods (``query_vectors``, ``true_scores``, ``score_topk``, ``merge``), in
production ``GpuShard`` (the C ABI's ``kge_shard_*`` / ``kge_merge_topk`` calls), in the CPU tests an oracle stand-in.
``comm`` is an object with ``all_reduce_sum(array)`` and ``all_gather(array) -> list``: ``DistComm`` wraps a
``torch.distributed`` process group (NCCL on GPUs, gloo on the CPU); plain NCCL collectives, no peer-memory tricks.
"""
from __future__ import annotations


def sharded_score_all_topk(local, comm, q_heads, q_rels, k, true_tails=None):
    """Returns (ids [nq, k], scores [nq, k], ranks [nq] or None), identical on every rank and identical to what one
    device holding the whole table returns."""
    qvec = comm.all_reduce_sum(local.query_vectors(q_heads, q_rels))         # each head lives in exactly one shard
    ftrue = None
    if true_tails is not None:
        ftrue = comm.all_reduce_sum(local.true_scores(qvec, q_rels, true_tails))
    ids, scores, beat = local.score_topk(qvec, q_rels, k, ftrue, true_tails)
    all_ids, all_scores = comm.all_gather(ids), comm.all_gather(scores)        # D lists of [nq, k]
    out_ids, out_scores = local.merge(all_ids, all_scores, k)
    ranks = None
    if true_tails is not None:
        ranks = comm.all_reduce_sum(beat) + 1
    return out_ids, out_scores, ranks


class DistComm:
    """torch.distributed collectives on torch tensors (device tensors with NCCL, host tensors with gloo)."""

    def __init__(self, group=None):
        import torch.distributed as dist
        self.dist, self.group = dist, group

    def all_reduce_sum(self, t):
        self.dist.all_reduce(t, op=self.dist.ReduceOp.SUM, group=self.group)
        return t

    def all_gather(self, t):
        import torch
        out = [torch.empty_like(t) for _ in range(self.dist.get_world_size(self.group))]
        self.dist.all_gather(out, t.contiguous(), group=self.group)
        return out


class GpuShard:
    """One rank's shard behind the C ABI: ``kge`` is a ``Kge`` bound to the shard's rows (its ``num_entities`` is the
    shard's height) with an inference workspace; ``ent_base`` the whole-table id of its first row."""

    def __init__(self, kge, ent_base: int):
        self.kge, self.ent_base = kge, int(ent_base)

    def query_vectors(self, q_heads, q_rels):
        import torch
        out = torch.empty((q_heads.numel(), self.kge.cfg.dim), dtype=torch.float32, device=q_heads.device)
        self.kge.shard_query_vectors(q_heads, q_rels, self.ent_base, out)
        return out

    def true_scores(self, qvec, q_rels, true_tails):
        import torch
        out = torch.empty(q_rels.numel(), dtype=torch.float32, device=qvec.device)
        self.kge.shard_true_scores(qvec, q_rels, true_tails, self.ent_base, out)
        return out

    def score_topk(self, qvec, q_rels, k, ftrue, true_tails):
        import torch
        nq, dev = q_rels.numel(), qvec.device
        ids = torch.empty((nq, k), dtype=torch.int32, device=dev)
        scores = torch.empty((nq, k), dtype=torch.float32, device=dev)
        beat = torch.empty(nq, dtype=torch.int32, device=dev) if true_tails is not None else None
        self.kge.shard_score_topk(qvec, q_rels, k, ftrue, true_tails, self.ent_base, ids, scores, beat)
        return ids, scores, beat

    def merge(self, all_ids, all_scores, k):
        import torch
        from .binding import merge_topk, KgeError
        cand_ids = torch.cat(all_ids, dim=1).contiguous()          # [nq, D * k]: the shards' lists side by side
        cand_scores = torch.cat(all_scores, dim=1).contiguous()
        out_ids = torch.empty((cand_ids.shape[0], k), dtype=torch.int32, device=cand_ids.device)
        out_scores = torch.empty((cand_ids.shape[0], k), dtype=torch.float32, device=cand_ids.device)
        rc = merge_topk(cand_ids, cand_scores, k, out_ids, out_scores)
        if rc != 0:
            raise KgeError(rc, "kge_merge_topk")
        return out_ids, out_scores


def sharded_score_all_topk_sequential(shards, q_heads, q_rels, k, true_tails=None):
    """The same protocol with the shards visited one after another by ONE process (``shards``: a list of objects like
    ``GpuShard``): the sums and gathers become loops.  This is also how one device scores a table that does not fit its
    memory -- bind, score and release the shards in turn."""
    qvec = None
    for sh in shards:
        part = sh.query_vectors(q_heads, q_rels)
        qvec = part if qvec is None else qvec + part
    ftrue = None
    if true_tails is not None:
        for sh in shards:
            part = sh.true_scores(qvec, q_rels, true_tails)
            ftrue = part if ftrue is None else ftrue + part
    lists = [sh.score_topk(qvec, q_rels, k, ftrue, true_tails) for sh in shards]
    out_ids, out_scores = shards[0].merge([l[0] for l in lists], [l[1] for l in lists], k)
    ranks = None
    if true_tails is not None:
        ranks = sum(l[2] for l in lists) + 1
    return out_ids, out_scores, ranks

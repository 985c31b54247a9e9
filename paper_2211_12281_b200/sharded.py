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


# ------------------------------------------------------------------------------------------ training
# One BESS training step (Section 4 "Training") with the entity table sharded over D workers.  Worker i holds the shard
# E_i (rows [i S, (i+1) S) of the table, S = ceil(E / D)) and whole relation tables; its micro-batch B_i has all heads
# in E_i and B/D tails in every E_j (Eq. 3), its N shared negatives N/D entities of every E_j (Eq. 4).  Per step:
#   1. every worker draws its micro-batch (the library's sampler with head_part = i; ids are whole-table ids);
#   2. AllToAll of ids: worker i tells worker j which B/D + N/D of j's rows it needs;
#   3. AllToAll of rows: the owners gather and send them -- the same amount between every pair of workers;
#   4. worker i runs the forward and backward of the unchanged step on its shard extended by the B + N received rows;
#   5. AllToAll of gradient rows back to the owners (the mirror of 3; the paper leaves this step implicit);
#   6. every owner applies one de-duplicated update to its shard from its own heads' rows and the rows it received;
#   7. AllGather of the relations' (and TransH normals') gradient rows: every worker applies the same update to its copy.
# The protocol is written once, as a generator that yields at every collective ("program"); `run_distributed` drives it
# with a torch.distributed group, `run_lockstep` drives D programs inside one process (the workers' collectives become
# list shuffles) -- which is how a single GPU checks the multi-worker path against the oracle.

class BessRank:
    """One worker behind the C ABI.  `sampler`: a Kge whose config has the WHOLE table's num_entities and head_part =
    rank, with this worker's share of the graph loaded (the triples whose head lies in its shard suffice).  `compute`:
    a Kge with the same model whose num_entities is shard_rows + B + N, bound to `ent_ext` -- the shard's rows followed
    by B + N rows that receive the step's remote tails and negatives (optimiser state extended likewise)."""

    def __init__(self, rank, world, sampler, compute, ent_ext, shard_rows, shard_size):
        import torch
        self.rank, self.world, self.sampler, self.compute = rank, world, sampler, compute
        self.ent_ext, self.rows, self.S = ent_ext, int(shard_rows), int(shard_size)
        c = compute.cfg
        self.B, self.N, self.d = c.batch, c.num_neg, c.dim
        dev = ent_ext.device
        self.ids = [torch.empty(n, dtype=torch.int32, device=dev) for n in (self.B, self.B, self.B, self.N)]
        self.loss = torch.zeros(1, dtype=torch.float32, device=dev)
        self.scratch = {}

    def sample(self, step):
        self.sampler.sample_batch(step, *self.ids)
        return self.ids

    def gather(self, ids):
        import torch
        out = torch.empty((ids.numel(), self.d), dtype=torch.float32, device=ids.device)
        self.compute.gather_rows(ids, self.rank * self.S, out)
        return out

    def gradients(self, step, heads_local, rels, tails_local, negs_local):
        import torch
        self.compute.train_gradients(step, heads_local, rels, tails_local, negs_local, self.loss)
        ws = self.compute.workspace
        views = []
        for addr, shape in zip(self.compute.gradient_rows(), ((2 * self.B + self.N, self.d), (self.B, -1), (self.B, self.d))):
            if not addr:
                views.append(None); continue
            off = addr - ws.data_ptr()
            width = shape[1] if shape[1] > 0 else (self.d // 2 if self.compute.cfg.score == 2 else self.d)      # RotatE: d/2 phases
            views.append(ws[off:off + shape[0] * width * 4].view(torch.float32).view(shape[0], width))
        return views

    def apply(self, table, ids, grads, step, lr):
        self.scratch[table] = self.compute.apply_gradients(table, ids.contiguous(), grads.contiguous(), step, lr, self.scratch.get(table))


def bess_train_step_program(rk, step, lr):
    """The protocol of one step for worker `rk` (an object with BessRank's methods); yields ("all_to_all", [D tensors]),
    ("all_gather", tensor) or ("all_reduce_sum", tensor) and is sent the collective's result.  Returns the global loss."""
    import torch
    D, B, N = rk.world, rk.B, rk.N
    bD, nD = B // D, N // D
    heads, rels, tails, negs = rk.sample(step)
    want = [torch.cat([tails[j * bD:(j + 1) * bD], negs[j * nD:(j + 1) * nD]]) for j in range(D)]
    asked = yield ("all_to_all", want)                                         # asked[r]: ids worker r needs from this shard
    rows = rk.gather(torch.cat(asked))
    per = bD + nD
    got = yield ("all_to_all", [rows[r * per:(r + 1) * per] for r in range(D)])   # got[j]: rows of this worker's tails / negatives in E_j
    for j in range(D):
        rk.ent_ext[rk.rows + j * bD: rk.rows + (j + 1) * bD] = got[j][:bD]
        rk.ent_ext[rk.rows + B + j * nD: rk.rows + B + (j + 1) * nD] = got[j][bD:]
    dev = heads.device
    heads_local = heads - rk.rank * rk.S
    tails_local = torch.arange(rk.rows, rk.rows + B, dtype=torch.int32, device=dev)
    negs_local = torch.arange(rk.rows + B, rk.rows + B + N, dtype=torch.int32, device=dev)
    g_ent, g_rel, g_relw = rk.gradients(step, heads_local, rels, tails_local, negs_local)
    back = [torch.cat([g_ent[B + j * bD: B + (j + 1) * bD], g_ent[2 * B + j * nD: 2 * B + (j + 1) * nD]]) for j in range(D)]
    received = yield ("all_to_all", back)                                      # received[r]: gradient rows of the rows sent to worker r
    ids = torch.cat([heads_local] + [a - rk.rank * rk.S for a in asked])
    rk.apply(0, ids, torch.cat([g_ent[:B]] + list(received)), step, lr)
    all_rels = yield ("all_gather", rels)
    all_grel = yield ("all_gather", g_rel)
    rk.apply(1, torch.cat(all_rels), torch.cat(all_grel), step, lr)
    if g_relw is not None:
        all_gw = yield ("all_gather", g_relw)
        rk.apply(2, torch.cat(all_rels), torch.cat(all_gw), step, lr)
    total = yield ("all_reduce_sum", rk.loss.clone())
    return total


def run_lockstep(programs):
    """Drives D programs inside one process: at every yield all workers' contributions are exchanged as the collective
    would.  Returns the programs' return values."""
    D = len(programs)
    sent = [p.send(None) for p in programs]
    results = [None] * D
    while True:
        kind = sent[0][0]
        assert all(s[0] == kind for s in sent)
        if kind == "all_to_all":
            replies = [[sent[src][1][dst].clone() for src in range(D)] for dst in range(D)]
        elif kind == "all_gather":
            gathered = [s[1].clone() for s in sent]
            replies = [list(gathered) for _ in range(D)]
        else:
            total = sum(s[1] for s in sent)
            replies = [total.clone() for _ in range(D)]
        nxt, done = [], 0
        for i, p in enumerate(programs):
            try:
                nxt.append(p.send(replies[i]))
            except StopIteration as stop:
                results[i] = stop.value; done += 1; nxt.append(None)
        if done == D:
            return results
        assert done == 0, "the workers' programs must finish together"
        sent = nxt


def run_distributed(program, group=None):
    """Drives one worker's program with torch.distributed collectives (NCCL on GPUs, gloo on the CPU)."""
    import torch
    import torch.distributed as dist
    world = dist.get_world_size(group)
    try:
        msg = program.send(None)
        while True:
            kind, payload = msg
            if kind == "all_to_all":
                if dist.get_backend(group) == "nccl":
                    out = [torch.empty_like(payload[r]) for r in range(world)]
                    dist.all_to_all(out, [t.contiguous() for t in payload], group=group)
                else:
                    # gloo has no AllToAll: every rank gathers every rank's (equally shaped) send list and keeps its column
                    mine = torch.stack([t.contiguous() for t in payload])
                    everyone = [torch.empty_like(mine) for _ in range(world)]
                    dist.all_gather(everyone, mine, group=group)
                    me = dist.get_rank(group)
                    out = [everyone[src][me] for src in range(world)]
                reply = out
            elif kind == "all_gather":
                out = [torch.empty_like(payload) for _ in range(world)]
                dist.all_gather(out, payload.contiguous(), group=group)
                reply = out
            else:
                dist.all_reduce(payload, op=dist.ReduceOp.SUM, group=group)
                reply = payload
            msg = program.send(reply)
    except StopIteration as stop:
        return stop.value

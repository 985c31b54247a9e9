"""The N > 1 path of full-entity inference (Section 4 "Inference"): the entity table sharded over the ranks, query
vectors and true-tail scores summed, per-shard top-K lists gathered and merged, beat counts summed.  Here as two
gloo ranks on the CPU with the fp32 oracle standing in for each rank's shard arithmetic: every rank must end with the
lists and ranks the oracle gives on the whole table, bit for bit."""
import json
import os
import subprocess
import sys
from pathlib import Path

ROOT = Path(__file__).resolve().parent.parent

WORKER = r"""
import os, sys, json
sys.path.insert(0, os.environ["KGE_ROOT"])
import numpy as np, torch
import torch.distributed as dist
import kge_synth
from oracle.kge_oracle import Oracle, make_config
from paper_2211_12281_b200.sharded import sharded_score_all_topk, DistComm

dist.init_process_group("gloo", init_method="tcp://127.0.0.1:" + os.environ["KGE_PORT"],
                        rank=int(os.environ["RANK"]), world_size=int(os.environ["WORLD_SIZE"]))
rank, world = dist.get_rank(), dist.get_world_size()
score, p = os.environ["KGE_SCORE"], int(os.environ["KGE_P"])
E, R, d, K, nq = 1001, 7, 16, 10, 37
o = Oracle("f32")
ent, rel, relw = kge_synth.make_tables(E, R, d, score, seed=5)
ent[900] = ent[3]; ent[4] = ent[3]                       # exact ties across the two shards
qh, qr, tt = kge_synth.make_queries(E, R, nq, seed=5)
tt[0] = 900; tt[1] = 3
cfg = make_config(num_entities=E, num_relations=R, dim=d, score=score, p_norm=p)
S = (E + world - 1) // world
lo, hi = rank * S, min(E, (rank + 1) * S)


class OracleShard:
    # a rank's shard arithmetic by the oracle: rows [lo, hi) of the table, whole relation tables
    def query_vectors(self, q_heads, q_rels):
        out = np.zeros((nq, d), np.float32)
        for i, (h, r) in enumerate(zip(q_heads, q_rels)):
            if lo <= h < hi:
                out[i] = o.query_vector(score, ent[h], rel[r], None if relw is None else relw[r])
        return torch.from_numpy(out)

    def true_scores(self, qvec, q_rels, true_tails):
        # the oracle scores from raw rows: the true tail's score is needed by every rank and owned by one
        out = np.zeros(nq, np.float32)
        for i, t in enumerate(true_tails):
            if lo <= t < hi:
                out[i] = o.score(score, p, ent[qh[i]], rel[q_rels[i]], ent[t], w=None if relw is None else relw[q_rels[i]])
        return torch.from_numpy(out)

    def score_topk(self, qvec, q_rels, k, ftrue, true_tails):
        ids, sc, ranks = o.score_all_topk(cfg, ent, rel, relw, qh, q_rels, k, true_tails=true_tails, ent_lo=lo, ent_hi=hi)
        return torch.from_numpy(ids), torch.from_numpy(sc), torch.from_numpy((ranks - 1).astype(np.int32))

    def merge(self, all_ids, all_scores, k):
        ids = torch.cat(all_ids, dim=1).numpy(); sc = torch.cat(all_scores, dim=1).numpy()
        out_i, out_s = np.empty((nq, k), np.int32), np.empty((nq, k), np.float32)
        for q in range(nq):
            keep = ids[q] >= 0
            order = np.lexsort((ids[q][keep], -sc[q][keep]))[:k]
            out_i[q] = ids[q][keep][order]; out_s[q] = sc[q][keep][order]
        return torch.from_numpy(out_i), torch.from_numpy(out_s)


ids, sc, ranks = sharded_score_all_topk(OracleShard(), DistComm(), qh, qr, K, tt)
w_ids, w_sc, w_ranks = o.score_all_topk(cfg, ent, rel, relw, qh, qr, K, true_tails=tt)
ok = bool((ids.numpy() == w_ids).all() and (sc.numpy() == w_sc).all() and (ranks.numpy() == w_ranks).all())
print(json.dumps({"rank": rank, "ok": ok, "ids0": ids[0].tolist()}), flush=True)
dist.barrier()
dist.destroy_process_group()
"""


def _free_port():
    import socket
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _run(score, p, world):
    port = str(_free_port())
    procs = []
    for rank in range(world):
        env = dict(os.environ, RANK=str(rank), WORLD_SIZE=str(world), KGE_PORT=port, KGE_ROOT=str(ROOT), KGE_SCORE=score, KGE_P=str(p),
                   OMP_NUM_THREADS="2")
        procs.append(subprocess.Popen([sys.executable, "-c", WORKER], env=env, stdout=subprocess.PIPE, text=True))
    outs = []
    for pr in procs:
        out, _ = pr.communicate(timeout=300)
        assert pr.returncode == 0
        outs.append(json.loads(out.strip().splitlines()[-1]))
    assert all(o["ok"] for o in outs)
    assert all(o["ids0"] == outs[0]["ids0"] for o in outs)          # every rank holds the same final lists


def test_two_gloo_ranks_reproduce_the_single_table_result_transe():
    _run("transe", 1, 2)


def test_three_gloo_ranks_ragged_last_shard_transh():
    _run("transh", 2, 3)

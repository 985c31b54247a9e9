"""The multi-worker BESS training step (Section 4 "Training") as real process-group collectives: two gloo ranks on the
CPU run sharded.bess_train_step_program through sharded.run_distributed -- AllToAll of ids, of tail rows, of gradient
rows back, AllGather of relation gradients -- with the fp64 oracle standing in for each worker's shard arithmetic.
Every rank must end with the shard the oracle gives for the whole table: the sum over the workers of the micro-batch
gradients at the pre-step tables, applied once (SGD)."""
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
from paper_2211_12281_b200.sharded import bess_train_step_program, run_distributed

dist.init_process_group("gloo", init_method="tcp://127.0.0.1:" + os.environ["KGE_PORT"],
                        rank=int(os.environ["RANK"]), world_size=int(os.environ["WORLD_SIZE"]))
rank, D = dist.get_rank(), dist.get_world_size()
o = Oracle("f64")
E, R, d, B, N, T, lr = 203, 4, 8, 8 * D, 12 * D, 6000, 0.1
kw = dict(num_relations=R, dim=d, score="transe", p_norm=2, loss="softmax", batch=B, num_neg=N, num_parts=D, ce_correction=0.2, seed=3)
h, r, t = kge_synth.make_graph(E, R, T, seed=31, relation_zipf=1.0)
ent, rel, _ = kge_synth.make_tables(E, R, d, "transe", seed=31)
ent, rel = ent.astype(np.float64), rel.astype(np.float64)
S = (E + D - 1) // D
graph = o.graph_build(E, R, D, h, r, t)


class OracleRank:
    # a worker's shard arithmetic by the oracle, on torch CPU tensors
    def __init__(self, i):
        self.rank, self.world, self.B, self.N, self.d, self.S = i, D, B, N, d, S
        self.rows = min(E, (i + 1) * S) - i * S
        self.ent_ext = torch.zeros((self.rows + B + N, d), dtype=torch.float64)
        self.ent_ext[:self.rows] = torch.from_numpy(ent[i * S:i * S + self.rows])
        self.rel = rel.copy()
        self.loss = torch.zeros(1, dtype=torch.float64)
        self.cfg_sample = make_config(**dict(kw, num_entities=E, head_part=i))
        self.cfg_compute = make_config(**dict(kw, num_entities=self.rows + B + N, num_parts=1))

    def sample(self, step):
        return [torch.from_numpy(a) for a in o.sample_batch(self.cfg_sample, step, graph)]

    def gather(self, ids):
        return self.ent_ext[(ids - self.rank * S).long()].clone()

    def gradients(self, step, hl, rels, tl, nl):
        g = o.batch_grads(self.cfg_compute, self.ent_ext.numpy(), self.rel, None, hl.numpy(), rels.numpy(), tl.numpy(), nl.numpy())
        self.loss[0] = g["loss"]
        return torch.from_numpy(np.concatenate([g["dh"], g["dtpos"], g["dtneg"]])), torch.from_numpy(g["dr"]), None

    def apply(self, table, ids, grads, step, lr_):
        tab = self.ent_ext.numpy() if table == 0 else self.rel
        acc = np.zeros_like(tab)
        np.add.at(acc, ids.numpy(), grads.numpy())
        tab -= lr_ * acc


me = OracleRank(rank)
total = run_distributed(bess_train_step_program(me, 0, lr))

# the whole-table answer
g_ent, g_rel, loss = np.zeros_like(ent), np.zeros_like(rel), 0.0
for i in range(D):
    cfg = make_config(**dict(kw, num_entities=E, head_part=i))
    batch = o.sample_batch(cfg, 0, graph)
    g = o.batch_grads(cfg, ent, rel, None, *batch)
    loss += g["loss"]
    np.add.at(g_ent, batch[0], g["dh"]); np.add.at(g_ent, batch[2], g["dtpos"]); np.add.at(g_ent, batch[3], g["dtneg"])
    np.add.at(g_rel, batch[1], g["dr"])
want_shard = (ent - lr * g_ent)[rank * S: rank * S + me.rows]
ok = bool(np.allclose(me.ent_ext[:me.rows].numpy(), want_shard, rtol=1e-12, atol=1e-14) and np.allclose(me.rel, rel - lr * g_rel, rtol=1e-12, atol=1e-14)
          and abs(float(total) - loss) <= 1e-10 * abs(loss) and np.abs(g_ent[rank * S: rank * S + me.rows]).sum() > 0)
print(json.dumps({"rank": rank, "ok": ok}), flush=True)
dist.barrier()
dist.destroy_process_group()
"""


def _free_port():
    import socket
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _run(world):
    port = str(_free_port())
    procs = []
    for rank in range(world):
        env = dict(os.environ, RANK=str(rank), WORLD_SIZE=str(world), KGE_PORT=port, KGE_ROOT=str(ROOT), OMP_NUM_THREADS="2")
        procs.append(subprocess.Popen([sys.executable, "-c", WORKER], env=env, stdout=subprocess.PIPE, stderr=subprocess.PIPE, text=True))
    for pr in procs:
        out, err = pr.communicate(timeout=300)
        assert pr.returncode == 0, err[-2000:]
        assert json.loads(out.strip().splitlines()[-1])["ok"]


def test_two_gloo_ranks_one_bess_step():
    _run(2)


def test_three_gloo_ranks_ragged_last_shard():
    _run(3)

"""GPU parity of the multi-worker BESS training step (Section 4 "Training") through the C ABI: D = 2 workers emulated in
one process on one GPU (their collectives become list shuffles, sharded.run_lockstep), each with its shard of the entity
table, its own micro-batch B_i (heads in E_i, tails and negatives balanced over the partitions: Eq. 3, Eq. 4), the rows of
remote tails and negatives received from their owners, gradient rows sent back, one de-duplicated update per owner.
Checked against the oracle: the sum over the workers of the oracle's micro-batch gradients at the pre-step tables, applied
once per row.  (The collectives' plumbing on real process groups: test_bess_protocol_cpu.py, gloo ranks.)"""
import numpy as np
import pytest

import kge_synth
from oracle.kge_oracle import make_config
from parity_util import assert_close

pytestmark = pytest.mark.gpu


def _make_workers(torch, K, kw, D, E, R, d, B, N, T, ent, rel, relw, opt, h, r, t):
    from paper_2211_12281_b200.sharded import BessRank
    dev = torch.device("cuda:0")
    S = (E + D - 1) // D
    rel_all = [torch.from_numpy(rel.copy()).to(dev) for _ in range(D)]                  # every worker its own copy
    relw_all = [None if relw is None else torch.from_numpy(relw.copy()).to(dev) for _ in range(D)]
    workers = []
    for i in range(D):
        lo, hi = i * S, min(E, (i + 1) * S)
        rows = hi - lo
        ent_ext = torch.zeros((rows + B + N, d), dtype=torch.float32, device=dev)
        ent_ext[:rows] = torch.from_numpy(ent[lo:hi])
        states = [None, None, None]
        if opt == "adagrad":
            states = [torch.zeros(rows + B + N, device=dev), torch.zeros(R, device=dev), None if relw is None else torch.zeros(R, device=dev)]
        mine = (h // S) == i                                                             # this worker's share of the graph
        sampler = K.Kge(K.KgeConfig.make(**dict(kw, num_entities=E, head_part=i)))
        sampler.bind(ent_ext, rel_all[i], relw_all[i], *states, num_triples=int(mine.sum()))
        sampler.graph_load(np.ascontiguousarray(h[mine]), np.ascontiguousarray(r[mine]), np.ascontiguousarray(t[mine]))
        compute = K.Kge(K.KgeConfig.make(**dict(kw, num_entities=rows + B + N, num_parts=1)))
        compute.bind(ent_ext, rel_all[i], relw_all[i], *states)
        workers.append((BessRank(i, D, sampler, compute, ent_ext, rows, S), rel_all[i], relw_all[i], states))
    return workers, S


@pytest.mark.parametrize("score,p,opt", [("transe", 1, "sgd"), ("distmult", 1, "adagrad"), ("transh", 2, "sgd")])
def test_two_workers_one_step_against_oracle(oracle64, score, p, opt):
    import torch
    import paper_2211_12281_b200 as K
    from paper_2211_12281_b200.sharded import bess_train_step_program, run_lockstep
    D, E, R, d, B, N, T, lr = 2, 301, 5, 32, 64, 96, 20000, 0.05
    kw = dict(num_relations=R, dim=d, score=score, p_norm=p, loss="logsigmoid", opt=opt, batch=B, num_neg=N, num_parts=D,
              gamma=4.0 if score != "distmult" else 0.0, adv_temp=0.5, lr=lr, seed=7)
    h, r, t = kge_synth.make_graph(E, R, T, seed=29, relation_zipf=1.0)
    ent, rel, relw = kge_synth.make_tables(E, R, d, score, seed=29)
    workers, S = _make_workers(torch, K, kw, D, E, R, d, B, N, T, ent, rel, relw, opt, h, r, t)
    for step in range(2):
        # the oracle's side: every worker's micro-batch at the pre-step (whole) tables
        ent_now = np.concatenate([w[0].ent_ext[:w[0].rows].cpu().numpy() for w in workers]).astype(np.float64)
        rel_now = workers[0][1].cpu().numpy().astype(np.float64)
        relw_now = None if relw is None else workers[0][2].cpu().numpy().astype(np.float64)
        g_ent, g_rel = np.zeros_like(ent_now), np.zeros_like(rel_now)
        g_relw = None if relw is None else np.zeros_like(relw_now)
        loss_o = 0.0
        for i in range(D):
            cfg = make_config(**dict(kw, num_entities=E, head_part=i))
            graph = oracle64.graph_build(E, R, D, h, r, t)
            batch = oracle64.sample_batch(cfg, step, graph)
            S_ = (E + D - 1) // D
            assert ((batch[0] // S_) == i).all()                                                     # heads in E_i
            assert (np.bincount(batch[2] // S_, minlength=D) == B // D).all()                        # Eq. 3
            assert (np.bincount(batch[3] // S_, minlength=D) == N // D).all()                        # Eq. 4
            g = oracle64.batch_grads(cfg, ent_now, rel_now, relw_now, *batch)
            loss_o += g["loss"]
            np.add.at(g_ent, batch[0], g["dh"]); np.add.at(g_ent, batch[2], g["dtpos"]); np.add.at(g_ent, batch[3], g["dtneg"])
            np.add.at(g_rel, batch[1], g["dr"])
            if g_relw is not None:
                np.add.at(g_relw, batch[1], g["dw"])
        losses = run_lockstep([bess_train_step_program(w[0], step, lr) for w in workers])
        for w in workers:
            assert w[0].compute.get_status() == 0 and w[0].sampler.get_status() == 0
        assert_close(losses[0].item(), loss_o, atol=1e-4, what="global loss")
        assert losses[0].item() == losses[1].item()
        ent_new = np.concatenate([w[0].ent_ext[:w[0].rows].cpu().numpy() for w in workers])

        def stepped(tab, grad, state_before):
            if opt == "sgd":
                return tab - lr * grad
            touched = np.abs(grad).max(axis=1) > 0
            s_new = state_before + np.where(touched, (grad ** 2).mean(axis=1), 0.0)
            return tab - lr * grad / (np.sqrt(s_new)[:, None] + 1e-10) * touched[:, None]

        st_e = np.zeros(E) if step == 0 else st_e_prev
        st_r = np.zeros(R) if step == 0 else st_r_prev
        assert_close(ent_new, stepped(ent_now, g_ent, st_e), atol=2e-6, what="entity shards")
        for w in workers:                                                                              # every worker's relation copy
            assert_close(w[1].cpu().numpy(), stepped(rel_now, g_rel, st_r), atol=2e-6, what="relation table")
            if relw is not None:
                assert_close(w[2].cpu().numpy(), stepped(relw_now, g_relw, np.zeros(R)), atol=2e-6, what="normals")
        assert (workers[0][1] == workers[1][1]).all()                                                  # the copies stay bit-identical
        if opt == "adagrad":
            st_e_prev = st_e + np.where(np.abs(g_ent).max(axis=1) > 0, (g_ent ** 2).mean(axis=1), 0.0)
            st_r_prev = st_r + np.where(np.abs(g_rel).max(axis=1) > 0, (g_rel ** 2).mean(axis=1), 0.0)
        else:
            st_e_prev, st_r_prev = st_e, st_r

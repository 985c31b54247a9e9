"""GPU parity of sharded full-entity inference (Section 4 "Inference") through the C ABI: the entity table cut into
three row shards (the last one ragged), each bound to its own handle, visited one after another by this process.  The
merged lists, scores and ranks must equal what one handle bound to the whole table returns, bit for bit, and the fp32
oracle's.  (The multi-process form of the same protocol runs as gloo ranks on the CPU in test_sharded_inference_cpu.py.)"""
import numpy as np
import pytest

import kge_synth
from parity_util import GpuSide, Problem

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("score,p,tc", [("transe", 1, False), ("transh", 2, False), ("rotate", 1, False), ("distmult", 1, False),
                                        ("complex", 1, True)])
def test_three_shards_equal_the_whole_table(oracle32, score, p, tc):
    import torch
    import paper_2211_12281_b200 as K
    from paper_2211_12281_b200.sharded import GpuShard, sharded_score_all_topk_sequential
    E, R, d, k, nq, D = 5000, 9, 64, 10, 70, 3
    prob = Problem(E=E, R=R, T=100, d=d, score=score, p_norm=p, B=4, N=4, P=1, graph_seed=23, tc=tc)
    prob.ent[4000] = prob.ent[17]; prob.ent[1700] = prob.ent[17]            # exact ties across shards
    qh, qr, tt = kge_synth.make_queries(E, R, nq, seed=23)
    tt[0] = qh[0]; tt[1] = 4000; tt[2] = 17
    whole = GpuSide(prob, max_queries=nq, topk=k, load_graph=False)
    t, dev = whole.torch, whole.ent.device
    qh_d, qr_d, tt_d = whole.dev_i32(qh), whole.dev_i32(qr), whole.dev_i32(tt)
    ids = t.empty((nq, k), dtype=t.int32, device=dev); sc = t.empty((nq, k), dtype=t.float32, device=dev)
    ranks = t.empty(nq, dtype=t.int32, device=dev)
    whole.kge.score_all_topk(qh_d, qr_d, k, tt_d, ids, sc, ranks)
    S = (E + D - 1) // D
    shards, keep = [], []
    for j in range(D):
        lo, hi = j * S, min(E, (j + 1) * S)
        rows = whole.ent[lo:hi].contiguous()
        kw = dict(prob.kw, num_entities=hi - lo)
        kge = K.Kge(K.KgeConfig.make(**kw, prec=K.PREC_BF16_TC if tc else K.PREC_FP32))
        kge.bind(rows, whole.rel, whole.relw, max_queries=nq, topk=k)
        shards.append(GpuShard(kge, lo)); keep.append(rows)
    s_ids, s_sc, s_ranks = sharded_score_all_topk_sequential(shards, qh_d, qr_d, k, tt_d)
    for sh in shards:
        assert sh.kge.get_status() == 0
    assert (s_ids == ids).all() and (s_sc == sc).all() and (s_ranks == ranks).all()
    # without true tails: lists only
    l_ids, l_sc, l_ranks = sharded_score_all_topk_sequential(shards, qh_d, qr_d, k, None)
    assert l_ranks is None and (l_ids == ids).all() and (l_sc == sc).all()
    if not tc and score != "rotate":
        o_ids, _, o_ranks = oracle32.score_all_topk(prob.oracle_cfg(), prob.ent, prob.rel, prob.relw, qh, qr, k, true_tails=tt)
        assert (s_ids.cpu().numpy() == o_ids).all() and (s_ranks.cpu().numpy() == o_ranks).all()


def test_merge_ignores_unused_places_and_rejects_oversized_lists():
    import torch
    import paper_2211_12281_b200 as K
    dev = torch.device("cuda:0")
    cand_ids = torch.tensor([[5, -1, 9, 2, -1, 7]], dtype=torch.int32, device=dev)
    cand_sc = torch.tensor([[1.0, 9.0, 1.0, 3.0, 9.0, -2.0]], dtype=torch.float32, device=dev)
    out_i = torch.zeros((1, 5), dtype=torch.int32, device=dev); out_s = torch.zeros((1, 5), dtype=torch.float32, device=dev)
    assert K.merge_topk(cand_ids, cand_sc, 5, out_i, out_s) == 0
    assert out_i[0].tolist() == [2, 5, 9, 7, -1] and out_s[0, :4].tolist() == [3.0, 1.0, 1.0, -2.0] and out_s[0, 4] == -np.inf
    big = torch.zeros((1, 2049), dtype=torch.int32, device=dev)
    assert K.merge_topk(big, big.float(), 5, out_i, out_s) == -4

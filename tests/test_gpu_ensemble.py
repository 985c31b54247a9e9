"""GPU parity of the power-rank ensemble (Section 3.2 "Ensemble", Eq. 2) against the oracle's brute force:
entity ids bit-exact and fp64 scores equal (both sides add the same rank scores in the same order), at the
paper's shape (85 models, top-100 lists) and fed by kge_score_all_topk at k = 100."""
import numpy as np
import pytest

import kge_synth
from parity_util import GpuSide, Problem

pytestmark = pytest.mark.gpu


def _gpu_ensemble(lists, power, top_n):
    import torch
    import paper_2211_12281_b200 as K
    dev = torch.device("cuda:0")
    M, nq, k = lists.shape
    table = torch.from_numpy(K.ensemble_rank_scores(power, k)).to(dev)
    ids = torch.full((nq, top_n), -7, dtype=torch.int32, device=dev)
    sc = torch.zeros((nq, top_n), dtype=torch.float64, device=dev)
    rc = K.ensemble_topk(torch.from_numpy(np.ascontiguousarray(lists)).to(dev), table, top_n, ids, sc)
    assert rc == 0
    torch.cuda.synchronize()
    return ids.cpu().numpy(), sc.cpu().numpy()


@pytest.mark.parametrize("M,nq,K,E", [(6, 200, 12, 60), (3, 33, 10, 4000), (85, 64, 100, 3000), (1, 5, 16, 100)])
@pytest.mark.parametrize("power", [-0.5, -1.0, 1.0, 2.0])
def test_ensemble_against_oracle(oracle64, M, nq, K, E, power):
    rng = np.random.default_rng(M * 1000 + K)
    lists = np.stack([np.stack([rng.permutation(E)[:K] for _ in range(nq)]) for _ in range(M)]).astype(np.int32)
    if M > 2:
        lists[1, :, K - 3:] = -1                        # a model that returned shorter lists
        lists[2, 0, :] = lists[0, 0, ::-1]              # mirrored ranks: exact ties decided by the id
    top_n = 10
    ids, sc = _gpu_ensemble(lists, power, top_n)
    o_ids, o_sc = oracle64.ensemble_topk(lists, power, top_n)
    assert (ids == o_ids).all()
    assert (sc == o_sc).all()


def test_ensemble_fewer_candidates_than_places_and_limits(oracle64):
    import torch
    import paper_2211_12281_b200 as K
    lists = np.array([[[4, 9, -1, -1]], [[9, 4, -1, -1]]], np.int32)
    ids, sc = _gpu_ensemble(lists, -0.5, 5)
    o_ids, o_sc = oracle64.ensemble_topk(lists, -0.5, 5)
    assert (ids == o_ids).all() and ids[0].tolist() == [4, 9, -1, -1, -1] and (sc == o_sc).all()
    dev = torch.device("cuda:0")
    big = torch.zeros((165, 1, 100), dtype=torch.int32, device=dev)                 # 16,500 entries per query
    table = torch.zeros(101, dtype=torch.float64, device=dev)
    out = torch.zeros((1, 10), dtype=torch.int32, device=dev)
    assert K.ensemble_topk(big, table, 10, out) == -4
    with pytest.raises(K.KgeError):
        K.ensemble_rank_scores(0.0, 10)                                              # Eq. 2 needs p != 0


def test_ensemble_of_three_scoring_functions_at_top_100(oracle32, oracle64):
    """Three models (TransE-L1, DistMult, ComplEx, their own random tables) score 40 queries against 20,000
    entities with k = 100; their lists (bit-exact against the fp32 oracle at k = 100) feed the ensemble."""
    import torch
    E, R, d, K, nq = 20000, 9, 32, 100, 40
    qh, qr, tt = kge_synth.make_queries(E, R, nq, seed=17)
    lists = []
    for m, score in enumerate(("transe", "distmult", "complex")):
        prob = Problem(E=E, R=R, T=100, d=d, score=score, p_norm=1, B=4, N=4, P=1, graph_seed=40 + m)
        gpu = GpuSide(prob, max_queries=nq, topk=K, load_graph=False)
        t, dev = gpu.torch, gpu.ent.device
        ids = t.empty((nq, K), dtype=t.int32, device=dev); sc = t.empty((nq, K), dtype=t.float32, device=dev)
        gpu.kge.score_all_topk(gpu.dev_i32(qh), gpu.dev_i32(qr), K, None, ids, sc)
        assert gpu.kge.get_status() == 0
        o_ids, _, _ = oracle32.score_all_topk(prob.oracle_cfg(), prob.ent, prob.rel, None, qh, qr, K)
        assert (ids.cpu().numpy() == o_ids).all()
        lists.append(ids.cpu().numpy())
    lists = np.stack(lists)
    ids, sc = _gpu_ensemble(lists, -0.5, 10)
    o_ids, o_sc = oracle64.ensemble_topk(lists, -0.5, 10)
    assert (ids == o_ids).all() and (sc == o_sc).all()

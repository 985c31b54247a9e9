"""Pins of the oracle's power-rank ensemble (Section 3.2 "Ensemble", Eq. 2)."""
import numpy as np
import pytest


def test_hand_worked_three_model_example(oracle64):
    # one query, K = 3, three models
    lists = np.array([[[7, 2, 9]], [[2, 7, 4]], [[5, 2, 7]]], np.int32)        # [M = 3, nq = 1, K = 3]
    # p = -0.5: s_m = k^-0.5 for the k-th entry, 0 if absent
    #   entity 2: 2^-0.5 + 1 + 2^-0.5 ;  7: 1 + 2^-0.5 + 3^-0.5 ;  5: 1 ;  9: 3^-0.5 ;  4: 3^-0.5 (tie with 9: smaller id first)
    ids, sc = oracle64.ensemble_topk(lists, -0.5, top_n=5)
    a, b = 2 ** -0.5, 3 ** -0.5
    assert ids[0].tolist() == [2, 7, 5, 4, 9]
    assert sc[0] == pytest.approx([1 + 2 * a, 1 + a + b, 1.0, b, b], rel=1e-15)
    # p = 1: s_m = -k for the k-th entry, -(K + 1) = -4 if absent
    #   2: -2 - 1 - 2 = -5 ;  7: -1 - 2 - 3 = -6 ;  5: -4 - 4 - 1 = -9 ;  9: -3 - 4 - 4 = -11 ;  4: -4 - 3 - 4 = -11
    ids, sc = oracle64.ensemble_topk(lists, 1.0, top_n=6)
    assert ids[0].tolist() == [2, 7, 5, 4, 9, -1]
    assert sc[0][:5].tolist() == [-5.0, -6.0, -9.0, -11.0, -11.0] and sc[0][5] == -np.inf


def test_reciprocal_rank_fusion_and_model_permutation(oracle64):
    rng = np.random.default_rng(4)
    M, nq, K, E = 6, 40, 12, 60
    lists = np.stack([np.stack([rng.permutation(E)[:K] for _ in range(nq)]) for _ in range(M)]).astype(np.int32)
    lists[2, :, K - 2:] = -1                                                   # a model with shorter lists
    ids, sc = oracle64.ensemble_topk(lists, -1.0, top_n=10)                    # p = -1: the sum of reciprocal ranks
    for q in range(nq):
        s = np.zeros(E)
        for m in range(M):
            for k in range(K):
                if lists[m, q, k] >= 0:
                    s[lists[m, q, k]] += 1.0 / (k + 1)
        order = np.lexsort((np.arange(E), -s))[:10]
        assert np.allclose(sc[q], s[order], rtol=1e-13)
        gap = np.abs(np.diff(s[order])) > 1e-12                               # ids must agree wherever the order is not a near-tie
        assert all(ids[q][i] == order[i] for i in range(10) if (i == 0 or gap[i - 1]) and (i == 9 or gap[i]))
    # the ensemble does not depend on the order of the models (up to the rounding of the sums)
    perm = rng.permutation(M)
    ids2, sc2 = oracle64.ensemble_topk(lists[perm], -1.0, top_n=10)
    assert np.allclose(sc, sc2, rtol=1e-13)
    for p in (-0.5, 0.5, 2.0):
        ids_p, sc_p = oracle64.ensemble_topk(lists, p, top_n=10)
        assert (np.diff(sc_p, axis=1) <= 0).all()                              # descending
        # an entity that every model ranks first beats everything
        forced = lists.copy(); forced[:, :, 0] = E + 5
        assert (oracle64.ensemble_topk(forced, p, top_n=1)[0] == E + 5).all()


def test_exact_ties_go_to_the_smaller_id(oracle64):
    # two entities with mirrored ranks in two models: identical sums, bit for bit
    lists = np.array([[[30, 10, 5]], [[10, 30, 6]]], np.int32)
    for p in (-0.5, 1.0):
        ids, sc = oracle64.ensemble_topk(lists, p, top_n=2)
        assert ids[0].tolist() == [10, 30] and sc[0][0] == sc[0][1]

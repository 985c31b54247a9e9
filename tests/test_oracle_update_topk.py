"""Pins for the oracle's dedup, sparse row update, full-entity top-k, rank and MRR."""
import numpy as np
import pytest

from oracle.kge_oracle import make_config
import kge_synth


def test_dedup_against_numpy_stable_argsort(oracle64):
    rng = np.random.default_rng(0)
    for n in (1, 2, 17, 300):
        ids = rng.integers(0, 12, n).astype(np.int32)
        uniq, seg, perm = oracle64.dedup(ids)
        assert (perm == np.argsort(ids, kind="stable")).all()
        u, counts = np.unique(ids, return_counts=True)
        assert (uniq == u).all() and (np.diff(seg) == counts).all() and seg[0] == 0 and seg[-1] == n
    uniq, seg, perm = oracle64.dedup(np.array([5, 5, 5], np.int32))
    assert uniq.tolist() == [5] and seg.tolist() == [0, 3] and perm.tolist() == [0, 1, 2]


def _numpy_sgd_step_distmult_logsigmoid(ent, rel, heads, rels, tails, negs, lr, gamma):
    """Independent restatement: dense autograd-free DistMult + uniform-weight log-sigmoid
    loss, gradients by matrix algebra, update by scatter-add."""
    h, r, tp, tn = ent[heads], rel[rels], ent[tails], ent[negs]
    q = h * r
    fpos, F = (q * tp).sum(1), q @ tn.T
    sig = lambda z: 1 / (1 + np.exp(-z))
    N = len(negs)
    loss = (np.log1p(np.exp(-(gamma + fpos))) + np.log1p(np.exp(gamma + F)).sum(1) / N).sum()
    gpos, G = -sig(-(gamma + fpos)), sig(gamma + F) / N
    dq = gpos[:, None] * tp + G @ tn
    g_ent, g_rel = np.zeros_like(ent), np.zeros_like(rel)
    np.add.at(g_ent, heads, dq * r); np.add.at(g_rel, rels, dq * h)
    np.add.at(g_ent, tails, gpos[:, None] * q); np.add.at(g_ent, negs, G.T @ q)
    return loss, ent - lr * g_ent, rel - lr * g_rel


def test_sgd_step_matches_numpy_restatement_with_repeated_rows(oracle64):
    rng = np.random.default_rng(1)
    E, R, d, B, N = 30, 4, 8, 16, 12
    ent, rel, _ = kge_synth.make_tables(E, R, d, "distmult", seed=0)
    ent, rel = ent.astype(np.float64), rel.astype(np.float64)
    heads, tails = rng.integers(0, E, B), rng.integers(0, E, B)
    rels, negs = rng.integers(0, R, B), rng.integers(0, E, N)
    heads[3] = tails[5] = negs[2] = negs[7] = 9          # one entity as head, tail and two negatives
    cfg = make_config(num_entities=E, num_relations=R, dim=d, score="distmult", batch=B, num_neg=N, gamma=0.3, opt="sgd")
    loss_np, ent_np, rel_np = _numpy_sgd_step_distmult_logsigmoid(ent, rel, heads, rels, tails, negs, 0.1, 0.3)
    e, r = ent.copy(), rel.copy()
    loss = oracle64.train_step(cfg, 0.1, 0, e, r, None, None, None, None, heads, rels, tails, negs)
    assert loss == pytest.approx(loss_np, rel=1e-12)
    assert e == pytest.approx(ent_np, rel=1e-11, abs=1e-14) and r == pytest.approx(rel_np, rel=1e-11, abs=1e-14)
    untouched = np.setdiff1d(np.arange(E), np.concatenate([heads, tails, negs]))
    assert (e[untouched] == ent[untouched]).all()
    # slot order inside the batch does not matter (up to rounding)
    pb, pn = rng.permutation(B), rng.permutation(N)
    e2, r2 = ent.copy(), rel.copy()
    oracle64.train_step(cfg, 0.1, 0, e2, r2, None, None, None, None, heads[pb], rels[pb], tails[pb], negs[pn])
    assert e2 == pytest.approx(e, rel=1e-11, abs=1e-14)


@pytest.mark.parametrize("opt", ["adam", "adagrad"])
def test_adam_and_rowwise_adagrad_textbook_two_steps(oracle64, opt):
    """Two steps with the same batch; expected values from the textbook recurrences applied
    to the table gradient that batch_grads (pinned by finite differences) reports."""
    rng = np.random.default_rng(2)
    E, R, d, B, N = 12, 3, 6, 4, 6
    ent, rel, relw = kge_synth.make_tables(E, R, d, "transh", seed=3)
    ent, rel, relw = (a.astype(np.float64) for a in (ent, rel, relw))
    heads, tails = np.array([1, 1, 4, 7], np.int32), np.array([2, 4, 1, 8], np.int32)
    rels, negs = np.array([0, 2, 2, 0], np.int32), np.array([1, 3, 3, 9, 10, 2], np.int32)
    cfg = make_config(num_entities=E, num_relations=R, dim=d, score="transh", p_norm=2, loss="softmax",
                      batch=B, num_neg=N, opt=opt, ce_correction=0.2)
    lr = 0.05
    st = (lambda rows, w: np.zeros((rows, 2 * w))) if opt == "adam" else (lambda rows, w: np.zeros(rows))
    tabs = dict(ent=ent.copy(), rel=rel.copy(), relw=relw.copy())
    states = dict(ent=st(E, d), rel=st(R, d), relw=st(R, d))
    exp_t = {k: v.copy() for k, v in tabs.items()}
    exp_s = {k: v.copy() for k, v in states.items()}
    for step in range(2):
        out = oracle64.batch_grads(cfg, exp_t["ent"], exp_t["rel"], exp_t["relw"], heads, rels, tails, negs)
        grads = dict(ent=np.zeros((E, d)), rel=np.zeros((R, d)), relw=np.zeros((R, d)))
        np.add.at(grads["ent"], heads, out["dh"]); np.add.at(grads["ent"], tails, out["dtpos"])
        np.add.at(grads["ent"], negs, out["dtneg"])
        np.add.at(grads["rel"], rels, out["dr"]); np.add.at(grads["relw"], rels, out["dw"])
        touched = dict(ent=np.unique(np.concatenate([heads, tails, negs])), rel=np.unique(rels), relw=np.unique(rels))
        for name in ("ent", "rel", "relw"):
            rows, g = touched[name], grads[name][touched[name]]
            if opt == "adam":
                m, v = exp_s[name][rows, :d], exp_s[name][rows, d:]
                m[:] = 0.9 * m + 0.1 * g; v[:] = 0.999 * v + 0.001 * g * g
                exp_s[name][rows, :d], exp_s[name][rows, d:] = m, v
                mhat, vhat = m / (1 - 0.9 ** (step + 1)), v / (1 - 0.999 ** (step + 1))
                exp_t[name][rows] -= lr * mhat / (np.sqrt(vhat) + 1e-8)
            else:
                exp_s[name][rows] += (g * g).mean(1)
                exp_t[name][rows] -= lr * g / (np.sqrt(exp_s[name][rows]) + 1e-10)[:, None]
        oracle64.train_step(cfg, lr, step, tabs["ent"], tabs["rel"], tabs["relw"],
                            states["ent"], states["rel"], states["relw"], heads, rels, tails, negs)
        for name in ("ent", "rel", "relw"):
            assert tabs[name] == pytest.approx(exp_t[name], rel=1e-10, abs=1e-13), (name, step)
            assert states[name] == pytest.approx(exp_s[name], rel=1e-10, abs=1e-15), (name, step)
    # rows never touched keep zero state (sparse / lazy optimiser)
    idle = np.setdiff1d(np.arange(E), np.concatenate([heads, tails, negs]))
    assert (states["ent"][idle] == 0).all() and (tabs["ent"][idle] == ent[idle]).all()


# ----------------------------------------------------------------------------- inference
@pytest.mark.parametrize("score,p", [("transe", 1), ("distmult", 1), ("rotate", 1), ("transh", 2), ("complex", 1)])
def test_topk_and_rank_against_numpy_lexsort(oracle64, oracle32, score, p):
    E, R, d, K, nq = 200, 5, 8, 10, 12
    ent, rel, relw = kge_synth.make_tables(E, R, d, score, seed=4)
    ent[50] = ent[20]; ent[120] = ent[20]; ent[7] = ent[6]        # exact ties
    qh, qr, tt = kge_synth.make_queries(E, R, nq, seed=4)
    tt[0] = qh[0]; tt[1] = 120; tt[2] = 20                         # true tail = head; tied true tails
    cfg = make_config(num_entities=E, num_relations=R, dim=d, score=score, p_norm=p)
    for orc in (oracle64, oracle32):
        ids, sc, ranks = orc.score_all_topk(cfg, ent, rel, relw, qh, qr, K, true_tails=tt)
        for q in range(nq):
            f = np.array([orc.score(score, p, ent[qh[q]], rel[qr[q]], ent[e], w=None if relw is None else relw[qr[q]])
                          for e in range(E)]).astype(orc.real)
            order = np.lexsort((np.arange(E), -f))                 # score descending, then id ascending
            assert (ids[q] == order[:K]).all() and (sc[q] == f[order[:K]]).all()
            assert ranks[q] == 1 + list(order).index(tt[q])
    assert (np.diff(sc, axis=1) <= 0).all()


def test_topk_k_larger_than_range_and_subrange(oracle64):
    E, R, d = 9, 2, 4
    ent, rel, _ = kge_synth.make_tables(E, R, d, "transe", seed=5)
    cfg = make_config(num_entities=E, num_relations=R, dim=d, score="transe", p_norm=1)
    ids, sc, ranks = oracle64.score_all_topk(cfg, ent, rel, None, [3], [1], 12, true_tails=[4])
    assert sorted(ids[0, :E].tolist()) == list(range(E)) and (ids[0, E:] == -1).all() and np.isinf(sc[0, E:]).all()
    ids2, _, ranks2 = oracle64.score_all_topk(cfg, ent, rel, None, [3], [1], 3, true_tails=[4], ent_lo=2, ent_hi=7)
    full = [e for e in ids[0, :E] if 2 <= e < 7]
    assert ids2[0].tolist() == full[:3] and ranks2[0] == 1 + full.index(4)


def test_mrr_definition(oracle64):
    ranks = np.array([1, 2, 10, 11, 50], np.int64)
    assert oracle64.mrr(ranks, 10) == pytest.approx((1 + 0.5 + 0.1) / 5)     # reciprocal rank 0 beyond top-10
    assert oracle64.mrr(ranks, 0) == pytest.approx((1 + 0.5 + 0.1 + 1 / 11 + 1 / 50) / 5)

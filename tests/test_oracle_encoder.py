"""Pins of the oracle's feature-projection encoder (Section 3.1 "Encoder", Eq. 1)."""
import itertools

import numpy as np
import pytest

from oracle.kge_oracle import make_config


def _problem(rng, score, E=9, R=3, d=4, F=6, B=3, N=4):
    ent = rng.standard_normal((E, d)) * 0.5
    feat = rng.standard_normal((E, F))
    MH, MT = rng.standard_normal((d, F)) * 0.3, rng.standard_normal((d, F)) * 0.3
    rel = rng.uniform(-np.pi, np.pi, (R, d // 2)) if score == "rotate" else rng.standard_normal((R, d)) * 0.5
    relw = rng.standard_normal((R, d)) if score == "transh" else None
    # entity 2 is a head, a tail and a negative: its shallow row collects all three, through M_H once and M_T twice
    heads = np.array([2, 0, 5], np.int32); rels = np.array([1, 1, 0], np.int32)
    tails = np.array([3, 2, 6], np.int32); negs = np.array([2, 4, 4, 8], np.int32)
    return ent, feat, MH, MT, rel, relw, heads, rels, tails, negs


def test_encoder_embedding_is_shallow_row_plus_projection(oracle64):
    rng = np.random.default_rng(1)
    ent, feat, MH, MT, rel, relw, heads, rels, tails, negs = _problem(rng, "distmult")
    cfg = make_config(num_entities=9, num_relations=3, dim=4, score="distmult", batch=3, num_neg=4, loss="softmax")
    # the loss with the encoder equals the plain loss on tables whose rows are the final embeddings -- built here per role
    e_head, e_tail = ent + feat @ MH.T, ent + feat @ MT.T
    B = len(heads)
    compact = np.concatenate([e_head[heads], e_tail[tails], e_tail[negs]])
    plain = oracle64.batch_loss(make_config(num_entities=len(compact), num_relations=3, dim=4, score="distmult", batch=3, num_neg=4, loss="softmax"),
                                compact, rel, None, np.arange(B), rels, B + np.arange(B), 2 * B + np.arange(len(negs)))["loss"]
    assert oracle64.encoder_batch_loss(cfg, ent, feat, MH, MT, rel, None, heads, rels, tails, negs) == pytest.approx(plain, rel=1e-13)
    # zero projection matrices: the encoder disappears
    Z = np.zeros_like(MH)
    assert oracle64.encoder_batch_loss(cfg, ent, feat, Z, Z, rel, None, heads, rels, tails, negs) == pytest.approx(
        oracle64.batch_loss(cfg, ent, rel, None, heads, rels, tails, negs)["loss"], rel=1e-13)


@pytest.mark.parametrize("score,p,loss", [("transe", 2, "logsigmoid"), ("distmult", 1, "softmax"), ("complex", 1, "logsigmoid"),
                                          ("transh", 2, "softmax"), ("rotate", 2, "softmax")])
def test_encoder_grads_match_central_finite_differences(oracle64, score, p, loss):
    rng = np.random.default_rng(7)
    ent, feat, MH, MT, rel, relw, heads, rels, tails, negs = _problem(rng, score)
    cfg = make_config(num_entities=9, num_relations=3, dim=4, score=score, p_norm=p, loss=loss, batch=3, num_neg=4,
                      gamma=1.0 if loss == "logsigmoid" else 0.0, adv_temp=0.0, ce_correction=0.3, loss_scale=0.5)
    out = oracle64.encoder_batch_grads(cfg, ent, feat, MH, MT, rel, relw, heads, rels, tails, negs)
    g_ent = np.zeros_like(ent)
    np.add.at(g_ent, heads, out["dh"]); np.add.at(g_ent, tails, out["dtpos"]); np.add.at(g_ent, negs, out["dtneg"])

    def loss_at(e, mh, mt):
        return oracle64.encoder_batch_loss(cfg, e, feat, mh, mt, rel, relw, heads, rels, tails, negs)

    assert out["loss"] == pytest.approx(loss_at(ent, MH, MT), rel=1e-14)
    eps = 1e-6
    for name, tab, grad in (("ent", ent, g_ent), ("MH", MH, out["dMH"]), ("MT", MT, out["dMT"])):
        for idx in itertools.product(range(tab.shape[0]), range(tab.shape[1])):
            args = dict(ent=ent, MH=MH, MT=MT)
            plus, minus = tab.copy(), tab.copy()
            plus[idx] += eps; minus[idx] -= eps
            args[name] = plus; lp = loss_at(args["ent"], args["MH"], args["MT"])
            args[name] = minus; lm = loss_at(args["ent"], args["MH"], args["MT"])
            assert grad[idx] == pytest.approx((lp - lm) / (2 * eps), rel=5e-6, abs=5e-8), (name, idx)
    assert np.abs(out["dMH"]).sum() > 0 and np.abs(out["dMT"]).sum() > 0


def test_encoder_step_updates_matrices_and_shared_matrix_sums_both_roles(oracle64):
    rng = np.random.default_rng(3)
    ent, feat, MH, MT, rel, relw, heads, rels, tails, negs = _problem(rng, "distmult")
    cfg = make_config(num_entities=9, num_relations=3, dim=4, score="distmult", batch=3, num_neg=4, loss="softmax", opt="sgd")
    g = oracle64.encoder_batch_grads(cfg, ent, feat, MH, MT, rel, None, heads, rels, tails, negs)
    e, mh, mt, r = ent.copy(), MH.copy(), MT.copy(), rel.copy()
    oracle64.encoder_train_step(cfg, False, 0.1, 0, e, feat, mh, mt, r, None, None, None, None, None, None, heads, rels, tails, negs)
    assert mh == pytest.approx(MH - 0.1 * g["dMH"], rel=1e-13) and mt == pytest.approx(MT - 0.1 * g["dMT"], rel=1e-13)
    g_ent = np.zeros_like(ent)
    np.add.at(g_ent, heads, g["dh"]); np.add.at(g_ent, tails, g["dtpos"]); np.add.at(g_ent, negs, g["dtneg"])
    assert e == pytest.approx(ent - 0.1 * g_ent, rel=1e-13, abs=1e-15)
    # one shared matrix: its gradient is the sum over both roles
    gs = oracle64.encoder_batch_grads(cfg, ent, feat, MH, MH, rel, None, heads, rels, tails, negs)
    m = MH.copy()
    oracle64.encoder_train_step(cfg, True, 0.1, 0, ent.copy(), feat, m, m, rel.copy(), None, None, None, None, None, None, heads, rels, tails, negs)
    assert m == pytest.approx(MH - 0.1 * (gs["dMH"] + gs["dMT"]), rel=1e-13)

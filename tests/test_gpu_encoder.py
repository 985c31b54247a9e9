"""GPU parity of the feature-projection encoder (Section 3.1 "Encoder", Eq. 1) against the oracle: projections of the
batch's slots (tensor cores, bf16 operands: the oracle rounds M the same way, the features are bf16 values on both sides),
the loss, the per-slot gradient rows, dM_H / dM_T (gradient rows rounded to bf16 on the GPU: compared at 1e-2 of the largest
entry, as the tensor-core backward is), the updated shallow rows and the updated matrices, over two steps."""
import numpy as np
import pytest

from parity_util import GpuSide, OracleSide, Problem, assert_close

pytestmark = pytest.mark.gpu


def _bf16(a):
    import torch
    return torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32)).to(torch.bfloat16)


@pytest.mark.parametrize("score,p,opt,shared,F,d", [("transe", 1, "sgd", False, 128, 40), ("distmult", 1, "adam", False, 64, 64),
                                                     ("transh", 2, "adagrad", True, 192, 32), ("complex", 1, "sgd", True, 768, 128)])
def test_encoder_step_against_oracle(oracle64, score, p, opt, shared, F, d):
    import torch
    prob = Problem(E=400, R=6, T=20000, d=d, score=score, p_norm=p, loss="softmax", opt=opt, B=96, N=160, P=2,
                   ce_correction=0.2, lr=0.02, graph_seed=17, relation_zipf=1.0)
    prob.kw.update(feat_dim=F, feat_shared=1 if shared else 0)
    rng = np.random.default_rng(17)
    feat = _bf16(rng.standard_normal((prob.E, F)) / np.sqrt(F))                    # the features are bf16 values by definition
    MH = (rng.standard_normal((d, F)) * 0.3).astype(np.float32)
    MT = MH if shared else (rng.standard_normal((d, F)) * 0.3).astype(np.float32)
    gpu = GpuSide(prob)
    dev = gpu.ent.device
    feat_d, MH_d = feat.to(dev), torch.from_numpy(MH.copy()).to(dev)
    MT_d = MH_d if shared else torch.from_numpy(MT.copy()).to(dev)
    st_shape = {"sgd": None, "adam": (d, 2 * F), "adagrad": (d,)}[opt]
    MH_s = None if st_shape is None else torch.zeros(st_shape, dtype=torch.float32, device=dev)
    MT_s = MH_s if shared else (None if st_shape is None else torch.zeros(st_shape, dtype=torch.float32, device=dev))
    gpu.kge.bind_features(feat_d, MH_d, MT_d, MH_s, MT_s)
    orc = OracleSide(prob, oracle64)
    okw = {k: v for k, v in prob.kw.items() if k not in ("feat_dim", "feat_shared", "contract")}
    from oracle.kge_oracle import make_config
    cfg = make_config(**okw, bf16_projection=1)
    feat64 = feat.float().numpy().astype(np.float64)
    B, N = prob.B, prob.N
    for step in range(2):
        batch = orc.sample(step)
        ent, rel, relw = (None if a is None else oracle64.arr(a).copy() for a in gpu.tables())
        mh, mt = oracle64.arr(MH_d.cpu().numpy()).copy(), None
        mt = mh if shared else oracle64.arr(MT_d.cpu().numpy()).copy()
        states = [None if s is None else oracle64.arr(s.cpu().numpy()).copy() for s in gpu.states]
        mh_s = None if MH_s is None else oracle64.arr(MH_s.cpu().numpy()).copy()
        mt_s = mh_s if shared else (None if MT_s is None else oracle64.arr(MT_s.cpu().numpy()).copy())
        want = oracle64.encoder_batch_grads(cfg, ent, feat64, mh, mt, rel, relw, *batch)
        loss = torch.zeros(1, dtype=torch.float32, device=dev)
        gpu.kge.train_step(step, prob.lr, *[gpu.dev_i32(a) for a in batch], loss_out=loss)
        assert gpu.kge.get_status() == 0
        assert_close(loss.item(), want["loss"], atol=1e-5, what="loss")
        ge = gpu.kge.debug_export("GRAD_ENT").reshape(2 * B + N, d)
        scale = max(np.abs(want["dh"]).max(), np.abs(want["dtneg"]).max())
        assert_close(ge[:B], want["dh"], atol=2e-5 * scale, what="dh")
        assert_close(ge[B:2 * B], want["dtpos"], atol=2e-5 * scale, what="dtpos")
        assert_close(ge[2 * B:], want["dtneg"], atol=2e-5 * scale, what="dtneg")
        loss_o = oracle64.encoder_train_step(cfg, shared, prob.lr, step, ent, feat64, mh, mt, rel, relw, states[0], mh_s, mt_s, states[1],
                                             states[2], *batch)
        assert loss_o == pytest.approx(want["loss"], rel=1e-12)
        g_ent, g_rel, _ = gpu.tables()
        if opt != "adam":      # (Adam's first step from zero moments is ill-conditioned where a gradient vanishes: covered elsewhere)
            assert_close(g_ent, ent, atol=2e-6, what="shallow rows")
            assert_close(g_rel, rel, atol=2e-6, what="relation rows")
        # the matrices: their gradient comes from bf16-rounded gradient rows (fp32 accumulation)
        gM = want["dMH"] + want["dMT"] if shared else want["dMH"]
        tolM = {"sgd": 1e-2 * prob.lr * np.abs(gM).max(), "adam": 2.5 * prob.lr, "adagrad": 2e-2 * prob.lr}[opt]
        assert_close(MH_d.cpu().numpy(), mh, rtol=1e-4, atol=tolM, what="M_H")
        if not shared:
            tolT = {"sgd": 1e-2 * prob.lr * np.abs(want["dMT"]).max(), "adam": 2.5 * prob.lr, "adagrad": 2e-2 * prob.lr}[opt]
            assert_close(MT_d.cpu().numpy(), mt, rtol=1e-4, atol=tolT, what="M_T")
        if opt == "sgd":       # the step itself, not only the result: (M_before - M_after) / lr is the gradient
            got_g = (oracle64.arr(MH if step == 0 else prev_mh) - MH_d.cpu().numpy().astype(np.float64)) / prob.lr
            assert_close(got_g, gM, rtol=1e-2, atol=1e-2 * np.abs(gM).max(), what="dM_H")
        prev_mh = MH_d.cpu().numpy().copy()
        if opt == "adam":
            assert_close(MH_s.cpu().numpy()[:, :F], mh_s[:, :F], rtol=1e-2, atol=1e-2 * np.abs(mh_s[:, :F]).max(), what="first moments of M_H")


def test_encoder_handle_refuses_what_it_does_not_offer():
    import paper_2211_12281_b200 as K
    with pytest.raises(K.KgeError) as e:
        K.Kge(K.KgeConfig.make(num_entities=100, num_relations=3, dim=32, score="transe", batch=4, num_neg=4, feat_dim=100))
    assert e.value.code == -5                       # the feature axis is cut into 64-element slices
    prob = Problem(E=100, R=3, T=500, d=32, score="transe", B=4, N=4, P=1)
    prob.kw.update(feat_dim=64)
    gpu = GpuSide(prob, max_queries=4, topk=2)
    with pytest.raises(K.KgeError) as e:
        gpu.kge.train_step(0, 0.1)                   # features not bound yet
    assert e.value.code == -6
    t = gpu.torch
    z = t.zeros(4, dtype=t.int32, device=gpu.ent.device)
    with pytest.raises(K.KgeError) as e:
        gpu.kge.score_all_topk(z, z, 2, None, t.zeros((4, 2), dtype=t.int32, device=z.device), t.zeros((4, 2), device=z.device))
    assert e.value.code == -5

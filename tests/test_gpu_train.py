"""GPU parity of the training step against the fp64 oracle: per-stage taps (positive
scores, dL/dF, gradient rows, dedup segments) and updated tables, for all five scoring
functions, both norms, both losses and the three optimisers; sizes span several tiles with
ragged tails.  Tolerance: |a-b| <= 1e-4 max(|a|,|b|) + atol, atol a small multiple of fp32
epsilon times the magnitude of the summed terms."""
import numpy as np
import pytest

from parity_util import GpuSide, OracleSide, Problem, assert_close

pytestmark = pytest.mark.gpu

MODELS = [("transe", 1), ("transe", 2), ("transh", 1), ("transh", 2), ("rotate", 1), ("rotate", 2),
          ("distmult", 1), ("complex", 1), ("rotate_real_l1", 1)]


def _check_step(gpu, orc, step, batch, *, taps=True, rows_atol=2e-6, warm_adam=False):
    prob = gpu.prob
    B, N, d = prob.B, prob.N, prob.d
    # tensor-core path: the scores come from bf16-rounded operands (matched by the oracle, so dL/dF
    # is still compared tightly), and the two backward contractions take dL/dF, q and t rounded
    # to bf16 (relative error 2^-9 per factor) with fp32 accumulation.  A gradient coordinate is a
    # sum of signed terms, so its error is bounded relative to the largest gradient, not to itself:
    # 1e-2 of the largest coordinate for the taps, and lr times 1e-2 of the largest summed
    # magnitude for the updated rows.  The stated bound of this path is 2e-2 relative on scores.
    ga = 1e-2 if prob.tc else 2e-5
    if prob.tc:
        g = orc.grads(batch)
        mag = np.zeros((prob.E, d))
        np.add.at(mag, batch[0], np.abs(g["dh"])); np.add.at(mag, batch[2], np.abs(g["dtpos"]))
        np.add.at(mag, batch[3], np.abs(g["dtneg"]))
        rmag = np.zeros((prob.R, g["dr"].shape[1])); np.add.at(rmag, batch[1], np.abs(g["dr"]))
        rows_atol = 1e-2 * prob.lr * max(mag.max(), rmag.max())
    dev = [gpu.dev_i32(a) for a in batch]
    loss_dev = gpu.torch.zeros(1, dtype=gpu.torch.float32, device=gpu.ent.device)
    want = orc.grads(batch) if taps else None
    grads_for_adam = (want or orc.grads(batch)) if prob.opt == "adam" else None
    fwd = orc.o.batch_loss(orc.cfg, orc.ent, orc.rel, orc.relw, *batch) if taps else None     # at the pre-step tables
    qvec = None
    if taps:
        wrow = lambda b: None if orc.relw is None else orc.relw[batch[1][b]]
        qvec = np.stack([orc.o.query_vector(prob.score, orc.ent[batch[0][b]], orc.rel[batch[1][b]], wrow(b)) for b in range(B)])
        scores_dev = gpu.torch.full((B, N), float("nan"), dtype=gpu.torch.float32, device=gpu.ent.device)
        gpu.kge.debug_capture_scores(scores_dev)
    gpu.kge.train_step(step, prob.lr, *dev, loss_out=loss_dev)
    gpu.kge.debug_capture_scores(None)
    assert gpu.kge.get_status() == 0
    loss_o = orc.step(step, batch)
    assert_close(loss_dev.item(), loss_o, atol=1e-5, what="loss")
    if taps:
        kge = gpu.kge
        # forward taps, element by element: per-query vectors, positive scores, the B x N score block, per-positive loss.
        # Relative 1e-4; the absolute term covers values that are cancelling sums of d products of O(1 / d) terms
        # (the tensor-core block: the same operand rounding on both sides, another accumulation order).
        assert_close(kge.debug_export("Q").reshape(B, d), qvec, atol=2e-6, what="Q")
        assert_close(kge.debug_export("FPOS"), fwd["fpos"], atol=2e-6, what="positive scores")
        assert_close(scores_dev.cpu().numpy(), fwd["F"], atol=2e-6, what="score block F")
        assert_close(kge.debug_export("LROW"), fwd["Lrow"], atol=1e-5, what="per-positive loss")
        l2 = prob.kw["p_norm"] == 2 and prob.score in ("transe", "transh", "rotate", "rotate_real_l1")
        G = kge.debug_export("G").reshape(B, N)
        if l2:   # the tap holds dL/dF divided by the distance; undo with the oracle's distances
            F = orc.o.batch_loss(orc.cfg, *orc._pre, *batch)["F"]
            G = G * -F
        if prob.tc:   # the tensor-core path keeps dL/dF as bf16 (8 significand bits)
            assert_close(G, want["G"], rtol=2.0 ** -8, atol=1e-6, what="G")
        else:
            assert_close(G, want["G"], atol=1e-7, what="G")
        ge = kge.debug_export("GRAD_ENT").reshape(2 * B + N, d)
        scale = max(np.abs(want["dh"]).max(), np.abs(want["dtneg"]).max(), 1e-30)
        assert_close(ge[:B], want["dh"], atol=ga * scale, what="dh")
        assert_close(ge[B:2 * B], want["dtpos"], atol=ga * scale, what="dtpos")
        assert_close(ge[2 * B:], want["dtneg"], atol=ga * scale, what="dtneg")
        assert_close(kge.debug_export("GRAD_REL").reshape(B, -1), want["dr"],
                     atol=ga * max(np.abs(want["dr"]).max(), 1e-30), what="dr")
        if prob.score == "transh":
            assert_close(kge.debug_export("GRAD_RELW").reshape(B, d), want["dw"],
                         atol=2e-5 * max(np.abs(want["dw"]).max(), 1e-30), what="dw")
        # dedup: bit-exact
        ids = np.concatenate([batch[0], batch[2], batch[3]])
        for pre, lst in (("ENT", ids), ("REL", batch[1])):
            uniq, seg, perm = orc.o.dedup(lst)
            assert (kge.debug_export(pre + "_UNIQ") == uniq).all()
            assert (kge.debug_export(pre + "_SEG") == seg).all()
            assert (kge.debug_export(pre + "_PERM") == perm).all()
    ent, rel, relw = gpu.tables()
    if prob.opt == "adam":
        _check_adam_tables(prob, batch, grads_for_adam, (ent, rel, relw), (orc.ent, orc.rel, orc.relw), rows_atol, warm=warm_adam)
    else:
        assert_close(ent, orc.ent, atol=rows_atol, what="entity table")
        assert_close(rel, orc.rel, atol=rows_atol, what="relation table")
        if relw is not None:
            assert_close(relw, orc.relw, atol=rows_atol, what="normal table")
    for got, want_s, name in zip(gpu.states, orc.states, ("ent_state", "rel_state", "relw_state")):
        if got is not None:
            # moments are linear / quadratic in a gradient that is itself a cancelling sum
            assert_close(got.cpu().numpy(), want_s, atol=2e-5 * float(np.abs(want_s).max()) + 1e-12, what=name)


def _check_adam_tables(prob, batch, g, got, want, rows_atol, warm=False):
    """Adam divides by sqrt(v) + eps, so its step is discontinuous where a gradient
    coordinate is zero: there fp32 rounding noise (1e-9) against the exact zero (the softmax
    probabilities of a row sum to one, so e.g. a TransE-L1 coordinate with every tail on the
    same side of q cancels exactly) decides a step of order lr.  Coordinates whose exact
    gradient is below 1e-4 of the table's largest are only required to move by a bounded
    amount (10 lr); all others meet the normal tolerance."""
    heads, rels, tails, negs = batch
    tabs = [np.zeros_like(want[0]), np.zeros_like(want[1]), None if want[2] is None else np.zeros_like(want[2])]
    np.add.at(tabs[0], heads, g["dh"]); np.add.at(tabs[0], tails, g["dtpos"]); np.add.at(tabs[0], negs, g["dtneg"])
    np.add.at(tabs[1], rels, g["dr"])
    if tabs[2] is not None:
        np.add.at(tabs[2], rels, g["dw"])
    for name, gt, a, b in zip(("entity", "relation", "normal"), tabs, got, want):
        if gt is None:
            continue
        if warm:     # second moments well away from zero: the step is continuous in g, every coordinate is compared
            assert_close(a, b, atol=rows_atol, what=name + " table (all coordinates, warm moments)")
            continue
        ill = np.abs(gt) < 1e-4 * np.abs(gt).max()
        a, b = np.asarray(a, np.float64), np.asarray(b, np.float64)
        assert_close(np.where(ill, b, a), b, atol=rows_atol, what=name + " table (well-conditioned coordinates)")
        assert (np.abs(a - b)[ill] <= 10 * prob.lr).all(), name
        touched = np.abs(gt).max(axis=1) > 0
        assert ill[touched].mean() < 0.25


def _run(oracle64, prob, steps=2, taps=True, external_batch=None):
    gpu, orc = GpuSide(prob), OracleSide(prob, oracle64)
    for step in range(steps):
        batch = external_batch if external_batch is not None else orc.sample(step)
        # each step is compared from identical tables: the oracle restarts from the GPU's rows
        orc.set_tables(*gpu.tables(), states=[None if s is None else s.cpu().numpy() for s in gpu.states])
        orc._pre = (orc.ent.copy(), orc.rel.copy(), None if orc.relw is None else orc.relw.copy())
        _check_step(gpu, orc, step, batch, taps=taps)
    return gpu, orc


@pytest.mark.parametrize("score,p", MODELS)
@pytest.mark.parametrize("loss", ["logsigmoid", "softmax"])
def test_step_taps_and_tables_all_models(oracle64, score, p, loss):
    # B = 72 and N = 70 leave ragged 64-wide tiles; d = 40 leaves a ragged 32-wide slice
    prob = Problem(E=500, R=7, T=20000, d=40, score=score, p_norm=p, loss=loss, B=72, N=70, P=2,
                   gamma=6.0 if loss == "logsigmoid" and score in ("transe", "transh", "rotate", "rotate_real_l1") else 0.0,
                   adv_temp=1.0 if loss == "logsigmoid" else 0.0, ce_correction=0.5, loss_scale=0.25,
                   lr=0.05, graph_seed=3, relation_zipf=1.0)
    _run(oracle64, prob)


@pytest.mark.parametrize("opt", ["adam", "adagrad"])
@pytest.mark.parametrize("score,p", [("transe", 1), ("complex", 1), ("transh", 2), ("rotate", 1)])
def test_optimisers_with_state(oracle64, opt, score, p):
    prob = Problem(E=300, R=5, T=10000, d=32, score=score, p_norm=p, loss="softmax", opt=opt, B=64, N=96, P=2,
                   ce_correction=0.1, lr=0.01, graph_seed=4, relation_zipf=1.0)
    _run(oracle64, prob, steps=3, taps=False)


@pytest.mark.parametrize("score,p", [("transe", 1), ("complex", 1), ("transh", 2), ("rotate", 1)])
def test_adam_from_warm_moments_every_coordinate(oracle64, score, p):
    """Adam's step m^ / (sqrt(v^) + eps) is discontinuous in the gradient only where v is zero (the first
    time a row is touched).  From moments that are already warm -- here every row starts with second
    moments of the size of a squared gradient -- the step is continuous, so ALL coordinates of the
    updated tables and of both moments are held to the normal tolerance, at global steps 2, 3 and 4."""
    prob = Problem(E=300, R=5, T=10000, d=32, score=score, p_norm=p, loss="softmax", opt="adam", B=64, N=96, P=2,
                   ce_correction=0.1, lr=0.01, graph_seed=4, relation_zipf=1.0)
    gpu, orc = GpuSide(prob), OracleSide(prob, oracle64)
    g0 = orc.grads(orc.sample(0))
    gs = float(np.sqrt(np.mean(g0["dh"] ** 2))) + 1e-6                  # a typical gradient magnitude
    rng = np.random.default_rng(9)
    for st in gpu.states:
        if st is None:
            continue
        w = st.shape[1] // 2
        init = np.concatenate([rng.standard_normal((st.shape[0], w)) * gs,                  # first moments
                               rng.uniform(0.5, 1.5, (st.shape[0], w)) * gs * gs], axis=1)   # second moments > 0
        st.copy_(gpu.torch.from_numpy(init.astype(np.float32)))
    for step in (2, 3, 4):
        batch = orc.sample(step)
        orc.set_tables(*gpu.tables(), states=[None if s is None else s.cpu().numpy() for s in gpu.states])
        _check_step(gpu, orc, step, batch, taps=False, warm_adam=True)


def test_l1_exact_ties_take_one_sub_gradient_everywhere(oracle64, oracle64_tie):
    """Tables of small integers make q_k = t_k happen in a large share of the (query, negative, coordinate)
    elements, and for the positive pair too.  |x| has every value in [-1, 1] as a sub-gradient at 0; the
    oracle's default is 0, the CUDA library takes -1 (the left derivative) in every kernel of the step.
    Checked coordinate by coordinate: (i) against the oracle build whose sub-gradient at 0 is -1 (TransE
    and TransH, all gradient rows and the updated tables); (ii) for TransE against the default oracle
    plus the closed-form difference  d(dh) = +sum over ties of dL/dF,  d(dt) = -sum over ties of dL/dF."""
    for score in ("transe", "transh"):
        prob = Problem(E=60, R=4, T=3000, d=16, score=score, p_norm=1, loss="logsigmoid", B=32, N=40, P=2,
                       gamma=4.0, adv_temp=0.5, lr=0.05, graph_seed=15)
        rng = np.random.default_rng(15)
        prob.ent = rng.integers(-2, 3, prob.ent.shape).astype(np.float32)
        prob.rel = rng.integers(-1, 2, prob.rel.shape).astype(np.float32)
        if score == "transh":
            prob.relw = np.zeros_like(prob.relw)
            prob.relw[np.arange(prob.R), np.arange(prob.R)] = 2.0      # axis-aligned normals: the projection stays in the integers
        gpu, o_tie, o_def = GpuSide(prob), OracleSide(prob, oracle64_tie), OracleSide(prob, oracle64)
        batch = o_def.sample(0)
        batch[2][:8] = batch[0][:8]                                     # a few positives with t = h: the positive pair ties where r = 0
        B, N, d = prob.B, prob.N, prob.d
        want, base = o_tie.grads(batch), o_def.grads(batch)
        fwd = oracle64.batch_loss(o_def.cfg, o_def.ent, o_def.rel, o_def.relw, *batch)
        gpu.kge.train_step(0, prob.lr, *[gpu.dev_i32(a) for a in batch])
        assert gpu.kge.get_status() == 0
        ge = gpu.kge.debug_export("GRAD_ENT").reshape(2 * B + N, d)
        scale = max(np.abs(want["dh"]).max(), np.abs(want["dtneg"]).max())
        for got, key in ((ge[:B], "dh"), (ge[B:2 * B], "dtpos"), (ge[2 * B:], "dtneg"),
                         (gpu.kge.debug_export("GRAD_REL").reshape(B, d), "dr")):
            assert_close(got, want[key], atol=2e-5 * scale, what=f"{score} {key} against the sign(0) = -1 oracle")
        if score == "transh":
            assert_close(gpu.kge.debug_export("GRAD_RELW").reshape(B, d), want["dw"], atol=2e-5 * np.abs(want["dw"]).max(), what="dw")
            continue
        q = o_def.ent[batch[0]] + o_def.rel[batch[1]]
        tie_neg = q[:, None, :] == o_def.ent[batch[3]][None, :, :]              # [B, N, d]
        tie_pos = q == o_def.ent[batch[2]]
        assert tie_neg.mean() > 0.1 and tie_pos.sum() > 0
        G, gpos = base["G"], base["gpos"]
        d_dh = np.einsum("bn,bnk->bk", G, tie_neg) + gpos[:, None] * tie_pos
        assert_close(ge[:B], base["dh"] + d_dh, atol=2e-5 * scale, what="dh = default oracle + tie weights")
        assert_close(ge[B:2 * B], base["dtpos"] - gpos[:, None] * tie_pos, atol=2e-5 * scale, what="dtpos")
        assert_close(ge[2 * B:], base["dtneg"] - np.einsum("bn,bnk->nk", G, tie_neg), atol=2e-5 * scale, what="dtneg")
        assert np.abs(d_dh).max() > 100 * 2e-5 * scale                           # the difference is far above the tolerance
        assert fwd["loss"] > 0
        o_tie.step(0, batch)
        assert_close(gpu.tables()[0], o_tie.ent, atol=2e-6, what="entity table")
        assert_close(gpu.tables()[1], o_tie.rel, atol=2e-6, what="relation table")


def test_bounded_wait_runs_out_and_the_context_stays_usable(oracle64):
    """Every wait of a kernel on an asynchronous copy or a barrier is a bounded loop.  With the limit cut to
    32 tries, a thread block that waits on a barrier nothing arrives at gives up, records KGE_ERR_TIMEOUT
    (-11) and returns; the status clears, and a normal step on the same handle then runs clean."""
    prob = Problem(E=500, R=7, T=20000, d=32, score="transe", p_norm=1, B=64, N=64, P=2, gamma=6.0, lr=0.05)
    gpu, orc = GpuSide(prob), OracleSide(prob, oracle64)
    gpu.kge.debug_set_wait_limit(32)
    gpu.kge.debug_wait_probe()
    assert gpu.kge.get_status() == -11
    assert gpu.kge.get_status() == 0
    gpu.kge.debug_set_wait_limit(0)                 # back to the default
    orc._pre = (orc.ent.copy(), orc.rel.copy(), None)
    _check_step(gpu, orc, 0, orc.sample(0), taps=True)
    assert gpu.kge.get_status() == 0


@pytest.mark.parametrize("score,p,form,tc", [("transe", 1, 0, False), ("distmult", 1, 1, False), ("transh", 2, 0, False),
                                             ("rotate", 1, 1, False), ("complex", 1, 0, True), ("transe", 2, 1, True)])
def test_l3_regulariser(oracle64, score, p, form, tc):
    """lambda_S Omega_S on the gathered rows (Section 3.1 "Regularisation"), both forms, on the CUDA-core and the
    tensor-core path (where the negatives' gradient rows otherwise bypass the chain kernel): the loss, every
    gradient row and the updated tables against the oracle; one entity is head, tail and negative at once."""
    d = 64 if tc else 40
    prob = Problem(E=400, R=6, T=20000, d=d, score=score, p_norm=p, loss="softmax" if tc else "logsigmoid", B=128, N=128, P=2,
                   gamma=4.0 if score in ("transe", "transh", "rotate") and not tc else 0.0, adv_temp=0.0 if tc else 0.5,
                   ce_correction=0.2, loss_scale=0.5, lr=0.05, graph_seed=16, relation_zipf=1.0, tc=tc,
                   reg_lambda=0.07, reg_form=form)
    prob.ent[5] = 0.0                                   # a zero row: the norm has zero gradient there
    gpu, orc = GpuSide(prob), OracleSide(prob, oracle64)
    batch = [a.copy() for a in orc.sample(0)]
    batch[0][:3] = 9; batch[2][3:5] = 9; batch[3][:4] = 9; batch[3][7] = 5; batch[0][10] = 5
    orc._pre = (orc.ent.copy(), orc.rel.copy(), None if orc.relw is None else orc.relw.copy())
    unreg = oracle64.batch_loss(Problem.oracle_cfg(_without_reg(prob)), orc.ent, orc.rel, orc.relw, *batch)["loss"]
    _check_step(gpu, orc, 0, batch)
    assert gpu.kge.get_status() == 0
    reg = oracle64.batch_loss(orc.cfg, *orc._pre, *batch)["loss"] - unreg
    assert reg > 0.01 * abs(unreg)                      # the term is a visible share of the loss


def _without_reg(prob):
    import copy
    q = copy.copy(prob)
    q.kw = dict(prob.kw, reg_lambda=0.0)
    return q


def test_lr_linear_decay_helper(oracle64):
    import paper_2211_12281_b200 as K
    f = K.lib().kge_lr_linear_decay
    for lr0, step, total in ((0.05, 0, 1000), (0.05, 500, 1000), (0.05, 999, 1000), (0.05, 1000, 1000), (0.05, 5000, 1000),
                             (3e-3, 1234567, 5_000_000), (1.0, 7, 0)):
        assert f(lr0, step, total) == pytest.approx(oracle64.lr_linear_decay(np.float32(lr0), step, total), rel=1e-6, abs=0)


def test_wide_rows_and_many_splits(oracle64):
    # d = 256 (two slices per lane), B << N so the dQ accumulation is split over columns
    prob = Problem(E=2000, R=11, T=40000, d=256, score="distmult", loss="softmax", B=32, N=640, P=4,
                   ce_correction=1.0, lr=0.1, graph_seed=5)
    _run(oracle64, prob, steps=1)
    prob = Problem(E=2000, R=11, T=40000, d=384, score="transe", p_norm=1, loss="logsigmoid", B=256, N=32, P=4,
                   gamma=12.0, adv_temp=0.5, lr=0.1, graph_seed=6)
    _run(oracle64, prob, steps=1)


@pytest.mark.parametrize("N,loss", [(256, "logsigmoid"), (512, "softmax"), (1024, "softmax"), (512, "logsigmoid")])
def test_loss_rows_in_registers(oracle64, N, loss):
    """Rows of 256 / 512 / 1024 scores are held in registers by 2 / 4 / 4 warps that exchange their
    partial maxima and sums through shared memory; B = 37 leaves a CTA with spare warps."""
    prob = Problem(E=3000, R=5, T=20000, d=32, score="transe", p_norm=1, loss=loss, B=37, N=N, P=1,
                   gamma=6.0, adv_temp=1.0 if loss == "logsigmoid" else 0.0, ce_correction=0.2, lr=0.05, graph_seed=13,
                   relation_zipf=1.0)
    _run(oracle64, prob, steps=1)


@pytest.mark.parametrize("d", [128, 256, 384])
def test_transh_l1_row_widths(oracle64, d):
    """TransH p = 1 at one, two and four 128-float slices per lane: the backward takes its sign
    sums as predicated adds for the first two and element by element on the query side of the
    widest rows."""
    prob = Problem(E=800, R=6, T=20000, d=d, score="transh", p_norm=1, loss="logsigmoid", B=96, N=80, P=2,
                   gamma=6.0, adv_temp=0.5, lr=0.05, graph_seed=12, relation_zipf=1.0)
    _run(oracle64, prob, steps=1)


@pytest.mark.parametrize("p,d,B,N", [(1, 128, 96, 80), (2, 128, 200, 300), (1, 128, 1024, 1024), (1, 256, 132, 200), (2, 96, 64, 130),
                                     (1, 64, 260, 64), (1, 160, 36, 40), (2, 32, 8, 16), (1, 512, 68, 72), (2, 384, 36, 136)])
def test_transh_tensor_core_contractions(oracle64, p, d, B, N):
    """TransH on the fp32 path with its three dense contractions forced onto the tensor cores (u = w.t from
    three-term bf16 splits, six products; the backward's two sums with per-pair coefficients from two-term
    splits, four products): the fp32 tolerances hold.  Shapes: a single ragged
    tile; ragged rows and columns; four K splits; rows of two 128-float slabs (two column tiles); a row width that
    leaves the tile's last 64 columns outside the operand; 128-column tiles; a fold of the output columns that is no
    multiple of 64; a block smaller than one slice of the contraction index; the widest rows (four column tiles of
    the folded output, four column slabs in the CUDA-core kernels); three column tiles."""
    prob = Problem(E=3000, R=6, T=30000, d=d, score="transh", p_norm=p, loss="logsigmoid", B=B, N=N, P=2,
                   gamma=6.0, adv_temp=0.5, lr=0.05, graph_seed=21, relation_zipf=1.0, contract=1)
    _run(oracle64, prob, steps=2)


@pytest.mark.parametrize("opt,reg", [("adam", 0.0), ("adagrad", 1e-3), ("sgd", 1e-3)])
def test_transh_tensor_core_contractions_with_optimisers_and_regulariser(oracle64, opt, reg):
    """The tensor-core route of TransH under the stateful optimisers and with the L3 regulariser's gradient joining
    the same rows in the chain kernel (softmax loss here; the other tests of this route use the log-sigmoid)."""
    prob = Problem(E=3000, R=6, T=30000, d=64, score="transh", p_norm=1, loss="softmax", opt=opt, B=132, N=200, P=2,
                   ce_correction=0.2, lr=0.02, graph_seed=23, relation_zipf=1.0, contract=1, reg_lambda=reg)
    _run(oracle64, prob, steps=2)


def test_transh_tensor_core_contractions_run_twice_bit_identical():
    """Three free-running steps of TransH with its contractions on the tensor cores (split-K slabs and the two
    halves of a folded tile are added in a fixed order), twice from the same tables: the same bits."""
    prob = Problem(E=5000, R=6, T=40000, d=128, score="transh", p_norm=1, loss="logsigmoid", opt="adagrad", B=1024, N=768, P=2,
                   gamma=6.0, adv_temp=1.0, lr=0.05, graph_seed=22, relation_zipf=1.0, contract=1)
    tables = []
    for _ in range(2):
        gpu = GpuSide(prob)
        for step in range(3):
            gpu.kge.train_step(step, prob.lr)
        assert gpu.kge.get_status() == 0
        tables.append(gpu.tables())
    for a, b in zip(*tables):
        assert (a == b).all()


@pytest.mark.parametrize("score,p", [("distmult", 1), ("complex", 1), ("transe", 2)])
@pytest.mark.parametrize("d", [64, 192, 256])
def test_tensor_core_score_block(oracle64, score, p, d):
    """bf16 tensor-core score block (DistMult, ComplEx, TransE-L2 by the norm expansion)
    against the oracle with bf16-rounded operands: B = 200 and N = 300 leave ragged 128-wide
    tiles, d = 192 a ragged 4-slice ring.  Operands are rounded identically on both sides, so
    the scores differ by accumulation order only and the fp32 tolerances apply; the stated
    bound for this path is 2e-2 relative on scores."""
    prob = Problem(E=3000, R=9, T=30000, d=d, score=score, p_norm=p, loss="softmax", B=200, N=300, P=2,
                   ce_correction=0.3, lr=0.05, graph_seed=7, relation_zipf=1.0, tc=True)
    _run(oracle64, prob, steps=2)
    prob = Problem(E=3000, R=9, T=30000, d=d, score=score, p_norm=p, loss="logsigmoid", B=128, N=256, P=2,
                   gamma=4.0 if score == "transe" else 0.0, adv_temp=0.5, lr=0.05, graph_seed=8, tc=True)
    _run(oracle64, prob, steps=1)


@pytest.mark.parametrize("score,p,loss,N,a", [("distmult", 1, "softmax", 2400, 0.0), ("transe", 2, "logsigmoid", 2500, 0.5),
                                              ("complex", 1, "logsigmoid", 2560, 0.5), ("transe", 2, "logsigmoid", 2500, 1.0)])
def test_tensor_core_wide_tiles(oracle64, score, p, loss, N, a):
    """Enough tiles to fill every SM, which switches the fused forward passes to 256-column
    tiles: N = 2400 leaves the last tile's upper half outside the problem (its statistics pieces
    do not exist), N = 2500 a ragged last piece, N = 2560 none.  Temperature 1 with a distance score
    takes the epilogues that share one exponential between the weight and the loss term."""
    prob = Problem(E=20000, R=9, T=60000, d=64, score=score, p_norm=p, loss=loss, B=2048, N=N, P=2,
                   ce_correction=0.3, gamma=4.0 if score == "transe" else 0.0, adv_temp=a,
                   lr=0.05, graph_seed=11, relation_zipf=1.0, tc=True)
    _run(oracle64, prob, steps=1)


@pytest.mark.parametrize("gamma", [12.0, 0.5, 90.0])
def test_tensor_core_distance_logsigmoid_temperature_one(oracle64, gamma):
    """TransE-L2 on tensor cores, log-sigmoid loss with self-adversarial temperature exactly 1 (128-column tiles
    here): margin 12 as in the large configuration, a small margin, and one beyond the range of the
    shared-exponential form (the general epilogues take over there)."""
    prob = Problem(E=3000, R=9, T=30000, d=128, score="transe", p_norm=2, loss="logsigmoid", B=200, N=300, P=2,
                   gamma=gamma, adv_temp=1.0, lr=0.05, graph_seed=18, relation_zipf=1.0, tc=True)
    _run(oracle64, prob, steps=2)


def test_tensor_core_path_refuses_what_it_cannot_do():
    import paper_2211_12281_b200 as K
    for kw in (dict(score="transe", p_norm=1, dim=128), dict(score="rotate", p_norm=2, dim=128),
               dict(score="distmult", dim=96)):
        with pytest.raises(K.KgeError) as e:
            K.Kge(K.KgeConfig.make(num_entities=100, num_relations=3, batch=4, num_neg=4, prec=K.PREC_BF16_TC, **kw))
        assert e.value.code == -5


@pytest.mark.parametrize("score,p", [("transe", 1), ("distmult", 1), ("transh", 1)])
def test_smallest_problem(oracle64, score, p):
    """One positive, one negative, one partition, four coordinates: every tile, chunk and piece is ragged."""
    prob = Problem(E=5, R=1, T=6, d=4, score=score, p_norm=p, loss="logsigmoid", B=1, N=1, P=1,
                   gamma=1.0 if score != "distmult" else 0.0, adv_temp=1.0, lr=0.1, graph_seed=14)
    _run(oracle64, prob, steps=2)


def test_repeated_rows_one_entity_everywhere(oracle64):
    """One entity is head, tail and negative several times; one relation for the whole batch."""
    prob = Problem(E=64, R=2, T=2000, d=32, score="distmult", loss="logsigmoid", B=16, N=16, P=1, lr=0.1)
    rng = np.random.default_rng(0)
    heads, tails, negs = rng.integers(0, 64, 16), rng.integers(0, 64, 16), rng.integers(0, 64, 16)
    heads[[0, 5, 9]] = 7; tails[[1, 5]] = 7; negs[[0, 3, 15]] = 7
    rels = np.zeros(16, np.int64)
    batch = [a.astype(np.int32) for a in (heads, rels, tails, negs)]
    _run(oracle64, prob, steps=2, external_batch=batch)


def test_config1_ten_sgd_steps_free_running(oracle64):
    """The small configuration: 10 SGD steps of DistMult with internal sampling, both sides
    running freely from the same initial tables."""
    prob = Problem(E=1000, R=10, T=20000, d=32, score="distmult", loss="logsigmoid", B=64, N=128, P=2,
                   lr=0.1, seed=0, graph_seed=0)
    gpu, orc = GpuSide(prob), OracleSide(prob, oracle64)
    loss_dev = gpu.torch.zeros(1, dtype=gpu.torch.float32, device=gpu.ent.device)
    for step in range(10):
        gpu.kge.train_step(step, prob.lr, loss_out=loss_dev)
        assert (gpu.kge.debug_export("BATCH") == np.concatenate(orc.sample(step))).all()
        loss_o = orc.step(step, orc.sample(step))
        assert_close(loss_dev.item(), loss_o, atol=1e-5, what=f"loss step {step}")
    ent, rel, _ = gpu.tables()
    assert_close(ent, orc.ent, atol=2e-6, what="entity table after 10 steps")
    assert_close(rel, orc.rel, atol=2e-6, what="relation table after 10 steps")
    assert gpu.kge.get_status() == 0
    # run twice: bit-identical (no atomics on floats anywhere)
    gpu2 = GpuSide(prob)
    for step in range(10):
        gpu2.kge.train_step(step, prob.lr)
    assert (gpu2.tables()[0] == ent).all() and (gpu2.tables()[1] == rel).all()


@pytest.mark.parametrize("score,p", [("transe", 1), ("rotate", 1)])
def test_config2_full_size_step(oracle64, score, p):
    """The headline configuration at full size, in the launch configuration the benchmark times:
    100,000 entities, d = 128, B = N = 1,024, P = 4, log-sigmoid with margin 12, SGD 0.05."""
    prob = Problem(E=100000, R=500, T=2000000, d=128, score=score, p_norm=p, loss="logsigmoid",
                   B=1024, N=1024, P=4, gamma=12.0, adv_temp=1.0, lr=0.05, seed=0, graph_seed=1,
                   relation_zipf=1.0)
    gpu, orc = GpuSide(prob), OracleSide(prob, oracle64)
    batch = orc.sample(0)
    orc._pre = (orc.ent.copy(), orc.rel.copy(), None)
    touched = np.unique(np.concatenate([batch[0], batch[2], batch[3]]))
    before = orc.ent[touched].copy()
    _check_step(gpu, orc, 0, batch, taps=True)
    assert np.abs(orc.ent[touched] - before).max() > 1e-4      # the step moved the touched rows


def test_host_entry_point_matches_device_entry_point(oracle64):
    prob = Problem(E=500, R=7, T=20000, d=32, score="transe", p_norm=1, B=64, N=64, P=2, gamma=6.0, lr=0.05)
    a, b = GpuSide(prob), GpuSide(prob)
    t = a.torch
    orc = OracleSide(prob, oracle64)
    for step in range(3):
        batch = orc.sample(step)
        loss_a = t.zeros(1, dtype=t.float32, device=a.ent.device)
        a.kge.train_step(step, prob.lr, *[a.dev_i32(x) for x in batch], loss_out=loss_a)
        pinned = [t.from_numpy(x).pin_memory() for x in batch]
        loss_b = t.zeros(1, dtype=t.float32).pin_memory()
        b.kge.train_step_host(step, prob.lr, *pinned, loss_b)
        assert loss_a.item() == loss_b.item()
    assert (a.tables()[0] == b.tables()[0]).all() and (a.tables()[1] == b.tables()[1]).all()


def test_out_of_range_id_sets_status_and_does_not_fault(oracle64):
    prob = Problem(E=100, R=3, T=3000, d=16, score="transe", B=16, N=16, P=1, gamma=1.0)
    gpu = GpuSide(prob)
    orc = OracleSide(prob, oracle64)
    batch = [x.copy() for x in orc.sample(0)]
    batch[3][5] = 100                      # one past the table
    gpu.kge.train_step(0, 0.1, *[gpu.dev_i32(x) for x in batch])
    assert gpu.kge.get_status() == -8      # KGE_ERR_ID_RANGE, reported once, then cleared
    assert gpu.kge.get_status() == 0
    assert np.isfinite(gpu.tables()[0]).all()

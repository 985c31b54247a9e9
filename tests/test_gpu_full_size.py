"""Parity at the full table sizes of the large configurations, on what the oracle can afford: the rows one step
touches.  The GPU runs the step on the whole table (10 M x 256 fp32 plus Adam state for
the 10 M-entity configuration); the rows of the batch are pulled out before and after, the ids are renumbered
densely, and the fp64 oracle runs the same step on that compact problem -- every quantity of
the step depends on the tables only through the rows the batch names, and the sampled-softmax
correction c is passed as a number, so the compact problem has the same answer."""
import numpy as np
import pytest

import kge_synth
from oracle.kge_oracle import make_config
from parity_util import assert_close

pytestmark = pytest.mark.gpu


def _compact(ids_list, touched):
    return [np.searchsorted(touched, ids).astype(np.int32) for ids in ids_list]


@pytest.mark.parametrize("score", ["distmult", "complex"])
def test_config3_full_table_step_on_touched_rows(oracle64, score):
    import torch
    import paper_2211_12281_b200 as K
    dev = torch.device("cuda:0")
    free, _ = torch.cuda.mem_get_info()
    if free < 45e9:
        pytest.skip("needs 45 GB of free device memory")
    # the 10 M-entity configuration with a graph of 20 M triples instead of 100 M (the step never sees the graph's size)
    E, R, T, d, B, N, P = 10_000_000, 1000, 20_000_000, 256, 4096, 16384, 8
    lr, c = 1e-3, float(np.log((E - 1) / N))
    kw = dict(num_entities=E, num_relations=R, dim=d, score=score, loss="softmax", opt="adam", batch=B, num_neg=N,
              num_parts=P, ce_correction=c, lr=lr, seed=0)
    h, r, t = kge_synth.make_graph(E, R, T, seed=2, relation_zipf=1.0)
    gen = torch.Generator(device=dev); gen.manual_seed(7)
    ent = torch.empty((E, d), dtype=torch.float32, device=dev).normal_(0.0, d ** -0.5, generator=gen)
    rel = torch.empty((R, d), dtype=torch.float32, device=dev).normal_(0.0, d ** -0.5, generator=gen)
    ent_state = torch.zeros((E, 2 * d), dtype=torch.float32, device=dev)
    rel_state = torch.zeros((R, 2 * d), dtype=torch.float32, device=dev)
    kge = K.Kge(K.KgeConfig.make(**kw, prec=K.PREC_BF16_TC))
    kge.bind(ent, rel, None, ent_state, rel_state, num_triples=T)
    kge.graph_load(h, r, t)

    # the batch of step 0: sampled on the device, bit-exact against the oracle's sampler
    bufs = [torch.empty(n, dtype=torch.int32, device=dev) for n in (B, B, B, N)]
    kge.sample_batch(0, *bufs)
    heads, rels, tails, negs = (b.cpu().numpy() for b in bufs)
    graph = oracle64.graph_build(E, R, P, h, r, t)
    want = oracle64.sample_batch(make_config(**kw), 0, graph)
    for got, exp in zip((heads, rels, tails, negs), want):
        assert (got == exp).all()
    S = (E + P - 1) // P
    assert (np.bincount(negs // S, minlength=P) == N // P).all()                       # Eq. 4
    assert (np.bincount((heads // S) * P + tails // S, minlength=P * P) == B // (P * P)).all()   # Eq. 3

    touched = np.unique(np.concatenate([heads, tails, negs]))
    tidx = torch.from_numpy(touched.astype(np.int64)).to(dev)
    before = ent[tidx].cpu().numpy()
    rel_before = rel.cpu().numpy()
    loss = torch.zeros(1, dtype=torch.float32, device=dev)
    kge.train_step(0, lr, *bufs, loss_out=loss)
    assert kge.get_status() == 0
    after, m_after = ent[tidx].cpu().numpy(), ent_state[tidx].cpu().numpy()

    # the same step on the compact problem, fp64, scores from bf16-rounded operands
    ch, ct, cn = _compact([heads, tails, negs], touched)
    ckw = dict(kw, num_entities=len(touched), num_parts=1)
    cfg = make_config(**ckw, bf16_operands=1)
    g = oracle64.batch_grads(cfg, before, rel_before, None, ch, rels, ct, cn)
    e64, r64 = oracle64.arr(before).copy(), oracle64.arr(rel_before).copy()
    es, rs = np.zeros((len(touched), 2 * d)), np.zeros((R, 2 * d))
    loss_o = oracle64.train_step(cfg, lr, 0, e64, r64, None, es, rs, None, ch, rels, ct, cn)
    assert_close(loss.item(), loss_o, rtol=1e-4, atol=1e-3, what="loss")

    # Adam's first moment is (1 - beta1) x gradient: linear, so it carries the gradient's error
    # bound of this path (bf16 factors in the backward contractions: 1e-2 of the largest summed
    # magnitude); the table rows are compared where the step is well conditioned.
    mag = np.zeros((len(touched), d))
    np.add.at(mag, ch, np.abs(g["dh"])); np.add.at(mag, ct, np.abs(g["dtpos"])); np.add.at(mag, cn, np.abs(g["dtneg"]))
    assert_close(m_after[:, :d], es[:, :d], rtol=1e-2, atol=0.1 * 1e-2 * mag.max(), what="first moments of the touched rows")
    gsum = es[:, :d] / 0.1
    well = np.abs(gsum) > 0.05 * np.abs(gsum).max()
    assert well.sum() > 1000
    assert_close(np.where(well, after, e64), e64, rtol=1e-4, atol=0.05 * lr, what="touched rows (well-conditioned coordinates)")
    assert (np.abs(after - e64) <= 2.5 * lr).all()                  # an Adam step never exceeds about lr
    untouched = torch.from_numpy(np.setdiff1d(np.arange(0, E, 997), touched)).to(dev)
    assert (ent_state[untouched] == 0).all()                          # rows outside the batch are not written


@pytest.mark.parametrize("score,p_norm,tc", [("transe", 2, True), ("transh", 1, False)])
def test_config4_full_table_step_on_touched_rows(oracle64, score, p_norm, tc):
    """the 91 M-entity training configuration: 91,000,000 entities of d = 128 (a 46.6 GB table), B = N = 8,192, P = 16, row-wise
    Adagrad, log-sigmoid loss with margin 12; TransE-L2 on tensor cores (norm expansion), TransH on
    CUDA cores.  The graph is cut to 20 M triples (the step never sees its size)."""
    import torch
    import paper_2211_12281_b200 as K
    dev = torch.device("cuda:0")
    free, _ = torch.cuda.mem_get_info()
    if free < 60e9:
        pytest.skip("needs 60 GB of free device memory")
    E, R, T, d, B, N, P = 91_000_000, 1400, 20_000_000, 128, 8192, 8192, 16
    lr = 0.05
    kw = dict(num_entities=E, num_relations=R, dim=d, score=score, p_norm=p_norm, loss="logsigmoid", opt="adagrad",
              batch=B, num_neg=N, num_parts=P, gamma=12.0, adv_temp=1.0, lr=lr, seed=0)
    h, r, t = kge_synth.make_graph(E, R, T, seed=3, relation_zipf=1.0)
    gen = torch.Generator(device=dev); gen.manual_seed(8)
    ent = torch.empty((E, d), dtype=torch.float32, device=dev).normal_(0.0, d ** -0.5, generator=gen)
    rel = torch.empty((R, d), dtype=torch.float32, device=dev).normal_(0.0, d ** -0.5, generator=gen)
    relw = torch.empty((R, d), dtype=torch.float32, device=dev).normal_(0.0, d ** -0.5, generator=gen) if score == "transh" else None
    ent_state = torch.zeros(E, dtype=torch.float32, device=dev)
    rel_state = torch.zeros(R, dtype=torch.float32, device=dev)
    relw_state = torch.zeros(R, dtype=torch.float32, device=dev) if relw is not None else None
    kge = K.Kge(K.KgeConfig.make(**kw, prec=K.PREC_BF16_TC if tc else K.PREC_FP32))
    kge.bind(ent, rel, relw, ent_state, rel_state, relw_state, num_triples=T)
    kge.graph_load(h, r, t)
    bufs = [torch.empty(n, dtype=torch.int32, device=dev) for n in (B, B, B, N)]
    kge.sample_batch(0, *bufs)
    heads, rels, tails, negs = (b.cpu().numpy() for b in bufs)
    S = (E + P - 1) // P
    assert (np.bincount(negs // S, minlength=P) == N // P).all()                       # Eq. 4
    assert (np.bincount((heads // S) * P + tails // S, minlength=P * P) == B // (P * P)).all()   # Eq. 3
    graph = oracle64.graph_build(E, R, P, h, r, t)
    for got, exp in zip((heads, rels, tails, negs), oracle64.sample_batch(make_config(**kw), 0, graph)):
        assert (got == exp).all()

    touched = np.unique(np.concatenate([heads, tails, negs]))
    tidx = torch.from_numpy(touched.astype(np.int64)).to(dev)
    before, rel_before = ent[tidx].cpu().numpy(), rel.cpu().numpy()
    relw_before = None if relw is None else relw.cpu().numpy()
    loss = torch.zeros(1, dtype=torch.float32, device=dev)
    kge.train_step(0, lr, *bufs, loss_out=loss)
    assert kge.get_status() == 0
    after, s_after = ent[tidx].cpu().numpy(), ent_state[tidx].cpu().numpy()

    ch, ct, cn = _compact([heads, tails, negs], touched)
    cfg = make_config(**dict(kw, num_entities=len(touched), num_parts=1), bf16_operands=1 if tc else 0)
    e64, r64 = oracle64.arr(before).copy(), oracle64.arr(rel_before).copy()
    w64 = None if relw_before is None else oracle64.arr(relw_before).copy()
    es, rs = np.zeros(len(touched)), np.zeros(R)
    ws = None if w64 is None else np.zeros(R)
    loss_o = oracle64.train_step(cfg, lr, 0, e64, r64, w64, es, rs, ws, ch, rels, ct, cn)
    assert_close(loss.item(), loss_o, rtol=1e-4, atol=1e-3, what="loss")
    step_size = np.abs(e64 - oracle64.arr(before)).max()
    assert step_size > 1e-3
    rel_tol = 2e-2 if tc else 1e-4            # bf16 factors in the tensor-core backward; fp32 otherwise
    assert_close(s_after, es, rtol=2 * rel_tol, atol=1e-12, what="row-wise Adagrad state of the touched rows")
    if p_norm == 1:
        # |x| has a kink at 0: the sign of a residual q_k - t_k that is zero to within fp32 rounding is
        # decided in fp32 here and in fp64 by the oracle.  Of the 8.6e9 residuals of this batch a few
        # hundred round across zero, each moving one gradient coordinate by 2 dL/dF of one pair: a
        # handful of coordinates may leave the tolerance, by at most a hundredth of the largest step.
        err = np.abs(after - e64)
        out = err > 1e-4 * np.maximum(np.abs(after), np.abs(e64)) + rel_tol * step_size + 2e-6
        assert out.sum() <= 64 and (err[out] <= 1e-2 * step_size).all(), (out.sum(), err.max())
    else:
        assert_close(after, e64, rtol=1e-4, atol=rel_tol * step_size + 2e-6, what="touched rows")
    assert_close(rel.cpu().numpy(), r64, rtol=1e-4, atol=rel_tol * np.abs(r64 - rel_before).max() + 2e-6, what="relation table")
    if w64 is not None:
        assert_close(relw.cpu().numpy(), w64, rtol=1e-4, atol=rel_tol * np.abs(w64 - relw_before).max() + 2e-6, what="normal table")


@pytest.mark.parametrize("score,tc", [("transe", False), ("distmult", True)])
def test_config5_full_table_topk_properties(oracle32, oracle64, score, tc):
    """the full-entity scoring configuration: queries against all 91,000,000 entities (46.6 GB table), top-10 and rank.  The
    oracle cannot hold the table, so the lists are checked by what fixes them: every reported
    score is the oracle's score of that (query, entity) pair; the list is ordered by (score
    descending, id ascending) with distinct ids; no entity of a 400,000-row sample is ordered
    before the list's last entry unless it is in the list; and asking for the rank of the list's
    first and last entries returns exactly 1 and 10."""
    import torch
    import paper_2211_12281_b200 as K
    dev = torch.device("cuda:0")
    free, _ = torch.cuda.mem_get_info()
    if free < 80e9:
        pytest.skip("needs 80 GB of free device memory")
    E, R, d, nq, k = 91_000_000, 1400, 128, 300, 10
    gen = torch.Generator(device=dev); gen.manual_seed(9)
    ent = torch.empty((E, d), dtype=torch.float32, device=dev).normal_(0.0, d ** -0.5, generator=gen)
    rel = torch.empty((R, d), dtype=torch.float32, device=dev).normal_(0.0, d ** -0.5, generator=gen)
    ent[12345] = ent[77]                                   # an exact tie somewhere in the table
    qh, qr, tt = kge_synth.make_queries(E, R, nq, seed=9)
    qh[0] = 77
    kw = dict(num_entities=E, num_relations=R, dim=d, score=score, p_norm=1)
    kge = K.Kge(K.KgeConfig.make(**kw, prec=K.PREC_BF16_TC if tc else K.PREC_FP32))
    kge.bind(ent, rel, max_queries=nq, topk=k)
    to_dev = lambda a: torch.from_numpy(np.ascontiguousarray(a, dtype=np.int32)).to(dev)
    ids = torch.empty((nq, k), dtype=torch.int32, device=dev); sc = torch.empty((nq, k), dtype=torch.float32, device=dev)
    ranks = torch.empty(nq, dtype=torch.int32, device=dev)
    kge.score_all_topk(to_dev(qh), to_dev(qr), k, to_dev(tt), ids, sc, ranks)
    assert kge.get_status() == 0
    ids_h, sc_h, ranks_h = ids.cpu().numpy(), sc.cpu().numpy(), ranks.cpu().numpy()
    assert ((ids_h >= 0) & (ids_h < E)).all() and ((ranks_h >= 1) & (ranks_h <= E)).all()

    orc = oracle64 if tc else oracle32
    rel_h = rel.cpu().numpy()
    pull = lambda idx: ent[torch.from_numpy(np.asarray(idx, dtype=np.int64)).to(dev)].cpu().numpy()
    heads_h = pull(qh)
    rng = np.random.default_rng(0)
    sample = np.unique(rng.integers(0, E, 400_000))
    sample_rows = pull(sample)
    for q in range(0, nq, 7):
        rows = pull(ids_h[q])
        want = np.array([orc.score(score, 1, heads_h[q], rel_h[qr[q]], rows[j], bf16=1 if tc else 0) for j in range(k)])
        if tc:
            assert_close(sc_h[q], want, rtol=1e-4, atol=1e-5, what="reported scores")
        else:
            assert (sc_h[q] == want.astype(np.float32)).all()       # fp32 path: same operation order, bit-exact
        assert len(set(ids_h[q])) == k
        for j in range(k - 1):
            assert sc_h[q, j] > sc_h[q, j + 1] or (sc_h[q, j] == sc_h[q, j + 1] and ids_h[q, j] < ids_h[q, j + 1])
    # nothing in the sample beats a list's last entry (checked for a few queries, scores by the oracle)
    cfg = make_config(**dict(kw, num_entities=len(sample)), bf16_operands=1 if tc else 0)
    probe = np.arange(0, nq, 50)
    tab = np.concatenate([sample_rows, heads_h[probe]])          # the probe heads ride along as extra rows
    cfg = make_config(**dict(kw, num_entities=len(tab)), bf16_operands=1 if tc else 0)
    q_heads = (len(sample) + np.arange(len(probe))).astype(np.int32)
    s_ids, s_sc, _ = orc.score_all_topk(cfg, tab, rel_h, None, q_heads, qr[probe], 3)
    for i, q in enumerate(probe):
        for j in range(3):
            if s_ids[i, j] >= len(sample):
                continue
            e, f = sample[s_ids[i, j]], s_sc[i, j]
            in_list = e in set(ids_h[q])
            slack = 1e-4 * abs(f) if tc else 0.0
            assert in_list or f < sc_h[q, k - 1] + slack or (f == sc_h[q, k - 1] and e > ids_h[q, k - 1])
    # the tie: entity 77 queried as a head sees rows 77 and 12345 with equal scores, lower id first
    pos = {int(e): j for j, e in enumerate(ids_h[0])}
    if 77 in pos and 12345 in pos:
        assert pos[77] < pos[12345] and sc_h[0, pos[77]] == sc_h[0, pos[12345]]
    # ranks of the first and the last list entries are 1 and k, exactly
    for j in (0, k - 1):
        kge.score_all_topk(to_dev(qh), to_dev(qr), k, ids[:, j].contiguous(), ids, sc, ranks)
        assert (ranks.cpu().numpy() == j + 1).all()
        assert (ids.cpu().numpy() == ids_h).all()                  # and the lists do not depend on the true tail

"""The allocation-free entry point (kge_score_all_topk_static) must return exactly what
kge_score_all_topk returns.  Some callers cannot allocate device memory at all -- their GPU
memory belongs to another allocator, or their host forbids allocation once it is running --
so this variant keeps every intermediate in one fixed array inside the library.  Because
that array is shared by all calls and keeps the previous call's contents, the check runs
two different query batches back to back: stale state from the first must not leak into the
second.  Collected last on purpose (file name), and it must pass on its own as well."""
import numpy as np
import pytest

import kge_synth
from parity_util import GpuSide, Problem

pytestmark = pytest.mark.gpu


def _both(gpu, prob, qh, qr, tt, k):
    import paper_2211_12281_b200 as K
    t, dev = gpu.torch, gpu.ent.device
    nq = len(qh)
    out = []
    for static in (False, True):
        ids = t.full((nq, k), -7, dtype=t.int32, device=dev)
        sc = t.zeros((nq, k), dtype=t.float32, device=dev)
        ranks = t.zeros(nq, dtype=t.int32, device=dev)
        args = (gpu.dev_i32(qh), gpu.dev_i32(qr), k, gpu.dev_i32(tt), ids, sc, ranks)
        if static:
            rc = K.score_all_topk_static(gpu.kge.cfg, gpu.ent, gpu.rel, gpu.relw, *args)
            assert rc == 0
        else:
            gpu.kge.score_all_topk(*args)
        out.append((ids.cpu().numpy(), sc.cpu().numpy(), ranks.cpu().numpy()))
    return out


@pytest.mark.parametrize("score,p", [("transe", 1), ("transh", 2), ("complex", 1)])
def test_static_entry_point_matches_workspace_entry_point_twice(oracle32, score, p):
    E, R, d, k = 3000, 6, 48, 10
    prob = Problem(E=E, R=R, T=100, d=d, score=score, p_norm=p, B=4, N=4, P=1, graph_seed=21)
    prob.ent[2500] = prob.ent[3]            # an exact tie
    gpu = GpuSide(prob, max_queries=64, topk=16, load_graph=False)
    for call, (nq, seed) in enumerate(((64, 5), (37, 6))):       # second call: fewer, different queries
        qh, qr, tt = kge_synth.make_queries(E, R, nq, seed=seed)
        (ids_a, sc_a, rk_a), (ids_b, sc_b, rk_b) = _both(gpu, prob, qh, qr, tt, k)
        assert (ids_a == ids_b).all(), call             # ids and ranks: bit-exact
        assert (rk_a == rk_b).all(), call
        assert (sc_a == sc_b).all(), call               # same kernels, same arithmetic: identical scores
        assert (ids_a >= 0).all() and (rk_a >= 1).all()
        # and on its own feet: the fp32 oracle's lists and ranks, bit for bit
        o_ids, _, o_ranks = oracle32.score_all_topk(prob.oracle_cfg(), prob.ent, prob.rel, prob.relw, qh, qr, k, true_tails=tt)
        assert (ids_b == o_ids).all() and (rk_b == o_ranks).all(), call


def test_static_entry_point_rejects_sizes_beyond_its_fixed_array():
    import paper_2211_12281_b200 as K
    prob = Problem(E=500, R=3, T=100, d=16, score="transe", B=4, N=4, P=1, graph_seed=22)
    gpu = GpuSide(prob, max_queries=80, topk=40, load_graph=False)
    t, dev = gpu.torch, gpu.ent.device
    mk = lambda nq, k: (t.zeros(nq, dtype=t.int32, device=dev), t.zeros(nq, dtype=t.int32, device=dev), k, None,
                        t.zeros((nq, k), dtype=t.int32, device=dev), t.zeros((nq, k), dtype=t.float32, device=dev))
    assert K.score_all_topk_static(gpu.kge.cfg, gpu.ent, gpu.rel, None, *mk(65, 4)) == -4      # too many queries
    assert K.score_all_topk_static(gpu.kge.cfg, gpu.ent, gpu.rel, None, *mk(8, 33)) == -4      # k too large
    assert K.score_all_topk_static(gpu.kge.cfg, gpu.ent, gpu.rel, None, *mk(8, 4)) == 0

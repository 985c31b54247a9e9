"""GPU parity of the on-device table initialisation against the oracle's recipe: the Philox words bit for
bit, the values within fp32 rounding of the oracle's fp64 evaluation (logarithm, sine and cosine come from
different libraries), and the statistical laws on the device's own output."""
import numpy as np
import pytest

from parity_util import GpuSide, Problem

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("score,opt", [("transe", "adam"), ("rotate", "sgd"), ("transh", "adagrad")])
def test_init_tables_against_oracle(oracle64, score, opt):
    from scipy import stats
    E, R, d, std, seed = 5000, 11, 40 if score != "rotate" else 44, 0.2, 2 ** 33 + 5
    prob = Problem(E=E, R=R, T=100, d=d, score=score, opt=opt, B=4, N=4, P=1, seed=seed, graph_seed=1)
    gpu = GpuSide(prob, load_graph=False)
    for st in gpu.states:
        if st is not None:
            st.fill_(3.0)
    gpu.kge.init_tables(std)
    assert gpu.kge.get_status() == 0
    ent, rel, relw = gpu.tables()
    kw = prob.rel_width                                     # rotate: 22 phases per relation (a ragged group of four)
    want_ent = oracle64.init_table(seed, 2, E, d, std)
    want_rel = oracle64.init_table(seed, 3, R, kw, std, kind=1 if score == "rotate" else 0)
    assert np.abs(ent - want_ent).max() <= 4e-6 * std * 6 and np.abs(rel - want_rel).max() <= 2e-6 * max(std * 6, np.pi)
    if relw is not None:
        assert np.abs(relw - oracle64.init_table(seed, 4, R, d, std)).max() <= 4e-6 * std * 6
    for st in gpu.states:
        assert st is None or float(st.abs().max()) == 0.0
    # the generator's words themselves
    t = gpu.torch
    words = t.empty((300, d), dtype=t.float32, device=gpu.ent.device)
    gpu.kge.debug_init_words(words, 300, d, 2)
    assert (words.cpu().numpy().view(np.uint32) == oracle64.init_table(seed, 2, 300, d, kind=2).view(np.uint32)).all()
    # the laws, on the device's output
    x = ent.astype(np.float64).ravel()
    assert abs(x.mean()) < 5 * std / np.sqrt(x.size) and abs(x.std() - std) < 5 * std / np.sqrt(2 * x.size)
    assert stats.kstest(x / std, "norm").pvalue > 1e-3
    if score == "rotate":
        # phases of a larger table through the same kernel: bind a second handle whose relation table it is
        prob2 = Problem(E=8, R=20000, T=100, d=d, score=score, B=4, N=4, P=1, seed=seed, graph_seed=1)
        gpu2 = GpuSide(prob2, load_graph=False)
        gpu2.kge.init_tables(std)
        ph = gpu2.tables()[1].astype(np.float64).ravel()
        assert ph.min() >= -np.pi and ph.max() <= np.pi
        assert stats.kstest((ph + np.pi) / (2 * np.pi), "uniform").pvalue > 1e-3

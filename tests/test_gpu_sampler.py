"""GPU parity: the Philox batch sampler must reproduce the oracle's indices bit for bit."""
import numpy as np
import pytest

from parity_util import GpuSide, OracleSide, Problem

pytestmark = pytest.mark.gpu

CASES = {
    # the small configuration and the headline configuration (shapes)
    "c1": dict(E=1000, R=10, T=20000, d=32, score="distmult", B=64, N=128, P=2, seed=0),
    "c2": dict(E=100000, R=500, T=2000000, d=128, score="transe", B=1024, N=1024, P=4, seed=0,
               graph_seed=1, relation_zipf=1.0),
    # ragged last partition (S = 251, last shard 247), fixed head partition, uniform mode
    "ragged_head2": dict(E=1000, R=7, T=30000, d=16, score="transe", B=96, N=60, P=4, head_part=2, seed=77),
    "uniform_mode": dict(E=1000, R=7, T=30000, d=16, score="transe", B=64, N=64, P=2, sample_mode=1, seed=5),
    "one_part": dict(E=333, R=3, T=5000, d=16, score="transe", B=50, N=30, P=1, seed=2**40 + 7),
}


@pytest.mark.parametrize("name", list(CASES))
def test_sampled_indices_bit_exact(oracle64, name):
    prob = Problem(**CASES[name])
    gpu, orc = GpuSide(prob), OracleSide(prob, oracle64)
    steps = list(range(100 if name in ("c1", "c2") else 20)) + [2**32 + 5, 2**63 + 11]
    for step in steps:
        got, want = gpu.sample(step), orc.sample(step)
        for g, w, what in zip(got, want, ("heads", "rels", "tails", "negs")):
            assert (g == w).all(), (name, step, what)
    assert gpu.kge.get_status() == 0


@pytest.mark.parametrize("name", ["c2", "ragged_head2", "c1"])
def test_step_that_samples_its_own_batch_uses_the_oracles_batch(oracle64, name):
    """kge_train_step with no ids draws the batch inside its gather kernel (the cumulative weights of a
    bucket staged per thread block): at the headline shape (R = 500 weights per bucket, B = N = 1,024) and
    with a fixed head partition and a ragged last shard the ids it used are the oracle's, bit for bit."""
    prob = Problem(**CASES[name])
    gpu, orc = GpuSide(prob), OracleSide(prob, oracle64)
    for step in (0, 1, 7, 2**32 + 5):
        gpu.kge.train_step(step, 0.01)
        assert (gpu.kge.debug_export("BATCH") == np.concatenate(orc.sample(step))).all(), (name, step)
    assert gpu.kge.get_status() == 0


def test_graph_load_reports_empty_bucket_and_bad_ids():
    import paper_2211_12281_b200 as K
    prob = Problem(E=40, R=5, T=4, d=16, score="transe", B=8, N=4, P=2)
    prob.h = np.array([0, 1, 2, 25], np.int32); prob.t = np.array([1, 30, 3, 26], np.int32)
    prob.r = np.zeros(4, np.int32)
    with pytest.raises(K.KgeError) as e:
        GpuSide(prob)                       # bucket (1, 0) is empty
    assert e.value.code == -3
    prob.h = np.array([0, 1, 2, 40], np.int32)
    with pytest.raises(K.KgeError) as e:
        GpuSide(prob)
    assert e.value.code == -1

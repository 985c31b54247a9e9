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


GRAPH_CASES = {
    # 19-bit keys (three radix passes), ragged last tile, ragged last shard, skewed relations
    "p16_r1400": dict(E=100003, R=1400, T=1_000_037, d=16, score="transe", B=256, N=64, P=16, relation_zipf=1.0, graph_seed=31),
    # one pass (8-bit keys), fewer triples than one tile
    "tiny": dict(E=40, R=7, T=5000, d=16, score="transe", B=8, N=8, P=2, graph_seed=32),
    # two passes, fixed head partition, uniform sampling mode
    "two_pass": dict(E=5000, R=300, T=200_000, d=16, score="transe", B=16, N=16, P=4, head_part=1, sample_mode=1, graph_seed=33),
}


def _check_graph_taps(gpu, want):
    for tap, key in (("GRAPH_H", "h"), ("GRAPH_R", "r"), ("GRAPH_T", "t"), ("GRAPH_OFF", "off"), ("GRAPH_WCUM", "wcum")):
        got = gpu.kge.debug_export(tap)
        assert got.dtype == want[key].dtype and (got == want[key]).all(), tap


@pytest.mark.parametrize("name", list(GRAPH_CASES))
def test_graph_preprocessing_on_device_is_bit_identical(oracle64, name):
    """kge_graph_load_device against the oracle's stable sort by (part(h), part(t), r): the sorted triples,
    the per-bucket relation offsets and the running cube-root weights, word for word; and the host path
    gives the same."""
    prob = Problem(**GRAPH_CASES[name])
    want = oracle64.graph_build(prob.E, prob.R, prob.P, prob.h, prob.r, prob.t)
    gpu = GpuSide(prob, load_graph=False)
    gpu.kge.bind(gpu.ent, gpu.rel, num_triples=prob.T)
    gpu.kge.graph_load_device(gpu.dev_i32(prob.h), gpu.dev_i32(prob.r), gpu.dev_i32(prob.t))
    _check_graph_taps(gpu, want)
    orc = OracleSide(prob, oracle64)
    for step in (0, 3):
        for g, w in zip(gpu.sample(step), orc.sample(step)):
            assert (g == w).all()
    gpu.kge.graph_load(prob.h, prob.r, prob.t)          # the host path over the same workspace
    _check_graph_taps(gpu, want)


def test_graph_preprocessing_on_device_20m_triples(oracle64):
    """20 M triples with the partition and relation counts of the 91 M-entity configuration (P = 16, R = 1,400)."""
    import kge_synth
    E, R, T, P = 1_000_000, 1400, 20_000_000, 16
    h, r, t = kge_synth.make_graph(E, R, T, seed=3, relation_zipf=1.0)
    want = oracle64.graph_build(E, R, P, h, r, t)
    prob = Problem(E=1000, R=R, T=8, d=16, score="transe", B=256, N=64, P=P, graph_seed=3)
    prob.kw["num_entities"] = E; prob.E = E; prob.T = T
    prob.ent = np.zeros((E, 16), np.float32)
    gpu = GpuSide(prob, load_graph=False)
    gpu.kge.bind(gpu.ent, gpu.rel, num_triples=T)
    gpu.kge.graph_load_device(gpu.dev_i32(h), gpu.dev_i32(r), gpu.dev_i32(t))
    _check_graph_taps(gpu, want)


def test_graph_preprocessing_on_device_reports_empty_bucket_and_bad_ids():
    import paper_2211_12281_b200 as K
    prob = Problem(E=40, R=5, T=4, d=16, score="transe", B=8, N=4, P=2)
    gpu = GpuSide(prob, load_graph=False)
    gpu.kge.bind(gpu.ent, gpu.rel, num_triples=4)
    h, t, r = np.array([0, 1, 2, 25], np.int32), np.array([1, 30, 3, 26], np.int32), np.zeros(4, np.int32)
    with pytest.raises(K.KgeError) as e:
        gpu.kge.graph_load_device(gpu.dev_i32(h), gpu.dev_i32(r), gpu.dev_i32(t))      # bucket (1, 0) is empty
    assert e.value.code == -3
    h[3] = 40
    with pytest.raises(K.KgeError) as e:
        gpu.kge.graph_load_device(gpu.dev_i32(h), gpu.dev_i32(r), gpu.dev_i32(t))
    assert e.value.code == -1
    with pytest.raises(K.KgeError) as e:
        gpu.kge.train_step(0, 0.1)                      # a failed load leaves no graph behind
    assert e.value.code == -6

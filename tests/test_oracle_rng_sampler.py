"""Pins for the oracle's counter-based generator, graph preprocessing and sampler.

Nothing here re-types the oracle's formulas: Philox is checked against cuRAND's host
generator, the integer helpers against Python big integers, the bucket structure against a
brute-force membership scan, and the sampler against the counts and the probability law
that Eq. 3, Eq. 4 and the cube-root sampling equation fix.
"""
import ctypes as C

import numpy as np
import pytest

from oracle.kge_oracle import make_config
import kge_synth


def _curand_host_words(seed, offset, n):
    try:
        lib = C.CDLL("libcurand.so.10")
    except OSError:
        try:
            lib = C.CDLL("/usr/local/cuda/lib64/libcurand.so")
        except OSError:
            pytest.skip("cuRAND host library not available")
    gen = C.c_void_p()
    assert lib.curandCreateGeneratorHost(C.byref(gen), C.c_int(161)) == 0  # PHILOX4_32_10
    assert lib.curandSetPseudoRandomGeneratorSeed(gen, C.c_ulonglong(seed)) == 0
    assert lib.curandSetGeneratorOffset(gen, C.c_ulonglong(offset)) == 0
    out = np.zeros(n, np.uint32)
    assert lib.curandGenerate(gen, out.ctypes.data_as(C.c_void_p), C.c_size_t(n)) == 0
    lib.curandDestroyGenerator(gen)
    return out


def test_philox_matches_curand_host_generator(oracle64):
    """cuRAND's host Philox4_32_10 emits, for 4-word block i of its stream,
    philox(counter=(i // 65536 as 64 bits in words 0-1, i % 65536 in word 2, 0), key=seed)."""
    rng = np.random.default_rng(0)
    for seed in (0, 1, 0x0123456789ABCDEF, 0xFEEDFACE12345678):
        key = [seed & 0xFFFFFFFF, seed >> 32]
        words = _curand_host_words(seed, 0, 4 * 65536 * 2).reshape(-1, 4)
        for i in list(rng.integers(0, len(words), 200)) + [0, 65535, 65536, len(words) - 1]:
            got = oracle64.philox([i // 65536, 0, i % 65536, 0], key)
            assert (got == words[i]).all(), (seed, i)
        # a far offset reaches counter word 1
        for c0, c1, c2 in ((5, 1, 7), (0xDEADBEEF, 3, 65535), (0xFFFFFFFF, 0x1FFF, 12345)):
            block = (c1 << 32 | c0) * 65536 + c2
            w = _curand_host_words(seed, 4 * block, 4)
            assert (oracle64.philox([c0, c1, c2, 0], key) == w).all()


def test_philox_counter_word3_and_key_are_live(oracle64):
    """Changing any counter or key word changes the block (streams are separated by word 3)."""
    base = oracle64.philox([1, 2, 3, 4], [5, 6])
    for pos in range(4):
        c = [1, 2, 3, 4]; c[pos] += 1
        assert (oracle64.philox(c, [5, 6]) != base).any()
    assert (oracle64.philox([1, 2, 3, 4], [5, 7]) != base).any()
    assert (oracle64.philox([1, 2, 3, 4], [4, 6]) != base).any()


def test_mulhi64_and_icbrt_against_bigints(oracle64):
    rng = np.random.default_rng(1)
    for _ in range(500):
        a = int(rng.integers(0, 2**64, dtype=np.uint64)); n = int(rng.integers(0, 2**40))
        assert oracle64.mulhi64(a, n) == (a * n) >> 64
    assert oracle64.mulhi64(2**64 - 1, 7) == 6 and oracle64.mulhi64(0, 7) == 0
    for n in [0, 1, 2, 7, 8, 9, 26, 27, 28, 1000, 12345678, 2**30 - 1, 2**30, 601062811, 2**40 + 17]:
        w = oracle64.icbrt_weight(n)
        if n == 0:
            assert w == 0
        else:
            assert w ** 3 <= n << 60 < (w + 1) ** 3
    # perfect cubes times 2^60: exact
    assert oracle64.icbrt_weight(27) == 3 << 20 and oracle64.icbrt_weight(1) == 1 << 20


def test_graph_build_brute_force(oracle64):
    E, R, P = 23, 3, 4          # S = 6: shards 6, 6, 6, 5
    h, r, t = kge_synth.make_graph(E, R, 400, seed=3, relation_zipf=1.0)
    g = oracle64.graph_build(E, R, P, h, r, t)
    S = -(-E // P)
    pos = 0
    for i in range(P):
        for j in range(P):
            w_acc = 0
            for rr in range(R):
                members = [e for e in range(len(h)) if h[e] // S == i and t[e] // S == j and r[e] == rr]
                base = (i * P + j) * (R + 1)
                assert g["off"][base + rr] == pos
                assert int(g["wcum"][base + rr]) == w_acc
                n = len(members)
                # stable: members keep their input order
                assert (g["h"][pos:pos + n] == h[members]).all()
                assert (g["t"][pos:pos + n] == t[members]).all()
                assert (g["r"][pos:pos + n] == rr).all()
                pos += n
                w_acc += oracle64.icbrt_weight(n)
            assert g["off"][base + R] == pos and int(g["wcum"][base + R]) == w_acc
    assert pos == len(h)
    with pytest.raises(ValueError):
        oracle64.graph_build(E, R, P, np.array([E]), np.array([0]), np.array([0]))


def _toy(oracle, E=40, R=5, P=2, T=4000, seed=5):
    h, r, t = kge_synth.make_graph(E, R, T, seed=seed, relation_zipf=1.0)
    return (h, r, t), oracle.graph_build(E, R, P, h, r, t)


def test_sampler_balanced_counts_eq3_eq4(oracle64):
    E, R, P, B, N = 41, 5, 4, 64, 24     # S = 11: shards 11, 11, 11, 8
    h, r, t = kge_synth.make_graph(E, R, 6000, seed=7, relation_zipf=1.0)
    g = oracle64.graph_build(E, R, P, h, r, t)
    triples = set(zip(h.tolist(), r.tolist(), t.tolist()))
    S = -(-E // P)
    for head_part in (-1, 0, 3):
        cfg = make_config(num_entities=E, num_relations=R, dim=4, score="transe", batch=B, num_neg=N,
                          num_parts=P, head_part=head_part, seed=11)
        for step in range(5):
            hh, rr, tt, nn = oracle64.sample_batch(cfg, step, g)
            assert all((a, b, c) in triples for a, b, c in zip(hh.tolist(), rr.tolist(), tt.tolist()))
            cnt = np.zeros((P, P), int)
            np.add.at(cnt, (hh // S, tt // S), 1)
            if head_part < 0:
                assert (cnt == B // (P * P)).all()                     # every bucket, B/P^2
                assert (np.repeat(np.arange(P * P), B // (P * P)) == (hh // S) * P + tt // S).all()
            else:
                assert (cnt[head_part] == B // P).all() and cnt.sum() == B   # Eq. 3
            assert (np.bincount(nn // S, minlength=P) == N // P).all()       # Eq. 4
            assert (np.repeat(np.arange(P), N // P) == nn // S).all()
            assert nn.min() >= 0 and nn.max() < E
        # counter-based: same (seed, step) -> same batch; another step or seed differs
        a = oracle64.sample_batch(cfg, 3, g); b = oracle64.sample_batch(cfg, 3, g)
        assert all((x == y).all() for x, y in zip(a, b))
        c = oracle64.sample_batch(cfg, 4, g)
        assert any((x != y).any() for x, y in zip(a, c))


def test_sampler_divisibility_and_empty_bucket_errors(oracle64):
    (_, _, _), g = _toy(oracle64)
    bad = make_config(num_entities=40, num_relations=5, dim=4, score="transe", batch=6, num_neg=4, num_parts=2)
    with pytest.raises(ValueError):
        oracle64.sample_batch(bad, 0, g)            # 6 % 4 != 0
    bad = make_config(num_entities=40, num_relations=5, dim=4, score="transe", batch=8, num_neg=5, num_parts=2)
    with pytest.raises(ValueError):
        oracle64.sample_batch(bad, 0, g)            # 5 % 2 != 0
    # a graph whose bucket (1, 0) is empty
    h = np.array([0, 1, 2, 25], np.int32); t = np.array([1, 30, 3, 26], np.int32); r = np.zeros(4, np.int32)
    g2 = oracle64.graph_build(40, 5, 2, h, r, t)
    cfg = make_config(num_entities=40, num_relations=5, dim=4, score="transe", batch=8, num_neg=4, num_parts=2)
    with pytest.raises(ValueError):
        oracle64.sample_batch(cfg, 0, g2)


def test_sampler_cube_root_relation_law_chi_square(oracle64):
    """One bucket (P = 1), three relations with counts 1000 / 125 / 8: relation frequencies
    must follow 10 : 5 : 2, and triples inside a relation must be uniform."""
    counts = [1000, 125, 8]
    r = np.concatenate([np.full(c, k, np.int32) for k, c in enumerate(counts)])
    rng = np.random.default_rng(0)
    order = rng.permutation(len(r))
    r = r[order]
    h = np.arange(len(r), dtype=np.int32) % 50       # tail id encodes the triple's identity
    t = np.arange(len(r), dtype=np.int32)
    E = len(r)
    g = oracle64.graph_build(E, 3, 1, h, r, t)
    B = 4096
    cfg = make_config(num_entities=E, num_relations=3, dim=4, score="transe", batch=B, num_neg=1, num_parts=1, seed=42)
    rel_counts = np.zeros(3); tail_hits = np.zeros(E)
    steps = 40
    for step in range(steps):
        hh, rr, tt, _ = oracle64.sample_batch(cfg, step, g)
        assert (r[tt] == rr).all() and (h[tt] == hh).all()
        rel_counts += np.bincount(rr, minlength=3)
        tail_hits += np.bincount(tt, minlength=E)
    n = B * steps
    expect = np.array([10.0, 5.0, 2.0]) / 17.0 * n
    chi2 = ((rel_counts - expect) ** 2 / expect).sum()
    assert chi2 < 13.8, (rel_counts, expect)        # chi2(2 dof) 0.999 quantile
    # a sampler that ignored the cube root (uniform over triples) would give 1000:125:8
    naive = np.array(counts) / sum(counts) * n
    assert ((rel_counts - naive) ** 2 / naive).sum() > 1000
    # uniform within relation 1 (125 triples)
    in_r1 = np.where(r == 1)[0]
    obs = tail_hits[in_r1]
    exp = obs.sum() / len(in_r1)
    assert ((obs - exp) ** 2 / exp).sum() < 180.0    # chi2(124 dof) 0.999 quantile ~ 178
    # sample_mode 1: uniform over the bucket's triples
    cfg1 = make_config(num_entities=E, num_relations=3, dim=4, score="transe", batch=B, num_neg=1, num_parts=1,
                       seed=42, sample_mode=1)
    rc = np.zeros(3)
    for step in range(10):
        rc += np.bincount(oracle64.sample_batch(cfg1, step, g)[1], minlength=3)
    e1 = np.array(counts) / sum(counts) * B * 10
    assert ((rc - e1) ** 2 / e1).sum() < 13.8


def test_negative_sampler_uniform_within_partition(oracle64):
    E, P, N = 10, 2, 4096
    (_, _, _), g = _toy(oracle64, E=E, R=2, P=P, T=500)
    cfg = make_config(num_entities=E, num_relations=2, dim=4, score="transe", batch=4, num_neg=N, num_parts=P, seed=9)
    hits = np.zeros(E)
    for step in range(10):
        hits += np.bincount(oracle64.sample_batch(cfg, step, g)[3], minlength=E)
    exp = N * 10 / E
    assert ((hits - exp) ** 2 / exp).sum() < 27.9     # chi2(9 dof) 0.999 quantile


# ----------------------------------------------------------------------------- table initialisation
def test_init_table_laws_and_words(oracle64):
    """The initialisation recipe: normal entries with the requested standard deviation (moments and a
    Kolmogorov-Smirnov test), uniform phases in (-pi, pi), no correlation between the two outputs of a
    Box-Muller pair or between neighbouring rows, raw words equal to philox of (row, c, stream), and
    tables of different streams / seeds unrelated."""
    from scipy import stats
    rows, width, std = 4000, 52, 0.25
    a = oracle64.init_table(7, 2, rows, width, std).astype(np.float64)
    n = a.size
    assert abs(a.mean()) < 5 * std / np.sqrt(n) and abs(a.std() - std) < 5 * std / np.sqrt(2 * n)
    assert stats.kstest(a.ravel() / std, "norm").pvalue > 1e-3
    assert abs(stats.kurtosis(a.ravel())) < 0.05 and abs(stats.skew(a.ravel())) < 0.03
    for x, y in ((a[:, 0::2], a[:, 1::2]), (a[:-1], a[1:]), (a[:, :-4], a[:, 4:])):
        assert abs(np.corrcoef(x.ravel(), y.ravel())[0, 1]) < 5 / np.sqrt(x.size)
    # Box-Muller radius: z0^2 + z1^2 = -2 std^2 ln u is exponentially distributed with mean 2 std^2
    r2 = (a[:, 0::2] ** 2 + a[:, 1::2] ** 2).ravel() / (2 * std * std)
    assert stats.kstest(r2, "expon").pvalue > 1e-3
    ph = oracle64.init_table(7, 3, rows, 6, kind=1).astype(np.float64)          # width 6: a ragged group of four
    assert ph.min() > -np.pi - 1e-6 and ph.max() < np.pi + 1e-6
    assert stats.kstest((ph.ravel() + np.pi) / (2 * np.pi), "uniform").pvalue > 1e-3
    words = oracle64.init_table(7, 2, 50, 8, kind=2).view(np.uint32)
    for row, c in ((0, 0), (49, 1), (17, 0)):
        assert (words[row, 4 * c:4 * c + 4] == oracle64.philox([row, 0, c, 2], [7, 0])).all()
    big = oracle64.init_table(2 ** 40 + 9, 4, 3, 4, kind=2).view(np.uint32)
    assert (big[2] == oracle64.philox([2, 0, 0, 4], [9, 2 ** 8])).all()            # the seed's upper half is the second key word
    assert abs(np.corrcoef(a.ravel(), oracle64.init_table(7, 4, rows, width, std).ravel())[0, 1]) < 5 / np.sqrt(n)
    assert abs(np.corrcoef(a.ravel(), oracle64.init_table(8, 2, rows, width, std).ravel())[0, 1]) < 5 / np.sqrt(n)
    # the uniform behind every entry is (k + 1/2) 2^-23: recover it from a phase and check it is on that grid
    k = (ph.ravel() / np.pi + 1) / 2 * 2 ** 23 - 0.5
    assert np.abs(k - np.round(k)).max() < 2e-1      # fp32 storage of the phase leaves about 0.1 of a grid step

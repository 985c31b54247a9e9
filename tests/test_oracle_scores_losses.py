"""Pins for the oracle's scoring functions, losses and gradients: special cases the
scoring-function table and the loss equations fix, numpy library routines, closed forms,
and central finite differences in fp64."""
import itertools

import numpy as np
import pytest

from oracle.kge_oracle import make_config

MODELS = [("transe", 1), ("transe", 2), ("transh", 1), ("transh", 2), ("rotate", 1), ("rotate", 2),
          ("distmult", 1), ("complex", 1), ("rotate_real_l1", 1)]
ROTATE = ("rotate", "rotate_real_l1")


def _rows(rng, d, score):
    h, t = rng.standard_normal(d), rng.standard_normal(d)
    r = rng.uniform(-np.pi, np.pi, d // 2) if score in ROTATE else rng.standard_normal(d)
    w = rng.standard_normal(d) if score == "transh" else None
    return h, r, w, t


def test_transe_zero_at_h_eq_t_r_zero_and_numpy_norms(oracle64):
    rng = np.random.default_rng(0)
    h = rng.standard_normal(16)
    for p in (1, 2):
        assert oracle64.score("transe", p, h, np.zeros(16), h) == 0.0
        r, t = rng.standard_normal(16), rng.standard_normal(16)
        assert oracle64.score("transe", p, h, r, t) == pytest.approx(-np.linalg.norm(h + r - t, ord=p), rel=1e-13)
    # antisymmetric: swapping h and t changes the score when r != 0
    assert oracle64.score("transe", 1, h, r, t) != pytest.approx(oracle64.score("transe", 1, t, r, h))


def test_distmult_symmetry_and_einsum(oracle64):
    rng = np.random.default_rng(1)
    h, r, t = rng.standard_normal((3, 12))
    f = oracle64.score("distmult", 1, h, r, t)
    assert f == pytest.approx(oracle64.score("distmult", 1, t, r, h), rel=1e-13)
    assert f == pytest.approx(np.einsum("k,k,k->", r, h, t), rel=1e-12)


def test_complex_reduces_to_distmult_and_matches_numpy_complex(oracle64):
    rng = np.random.default_rng(2)
    d = 10
    hr, rr, tr = rng.standard_normal((3, d // 2))
    inter = lambda re, im: np.stack([re, im], 1).reshape(-1)
    z = np.zeros(d // 2)
    f = oracle64.score("complex", 1, inter(hr, z), inter(rr, z), inter(tr, z))
    assert f == pytest.approx(oracle64.score("distmult", 1, hr, rr, tr), rel=1e-13)
    hi, ri, ti = rng.standard_normal((3, d // 2))
    hc, rc, tc = hr + 1j * hi, rr + 1j * ri, tr + 1j * ti
    f = oracle64.score("complex", 1, inter(hr, hi), inter(rr, ri), inter(tr, ti))
    assert f == pytest.approx(np.real(np.sum(rc * hc * np.conj(tc))), rel=1e-12)
    # f(t, r, h) = f(h, conj r, t)
    assert oracle64.score("complex", 1, inter(tr, ti), inter(rr, ri), inter(hr, hi)) == pytest.approx(
        oracle64.score("complex", 1, inter(hr, hi), inter(rr, -ri), inter(tr, ti)), rel=1e-12)


def test_rotate_special_phases_and_numpy_complex(oracle64):
    rng = np.random.default_rng(3)
    d = 12
    h, t = rng.standard_normal(d), rng.standard_normal(d)
    hc, tc = h[0::2] + 1j * h[1::2], t[0::2] + 1j * t[1::2]
    zero = np.zeros(d // 2)
    assert oracle64.score("rotate", 1, h, zero, t) == pytest.approx(-np.abs(hc - tc).sum(), rel=1e-13)
    assert oracle64.score("rotate", 2, h, zero, t) == pytest.approx(-np.linalg.norm(h - t), rel=1e-13)
    assert oracle64.score("rotate", 1, h, np.full(d // 2, np.pi), t) == pytest.approx(-np.abs(-hc - tc).sum(), rel=1e-12)
    th = rng.uniform(-np.pi, np.pi, d // 2)
    assert oracle64.score("rotate", 1, h, th, t) == pytest.approx(-np.abs(hc * np.exp(1j * th) - tc).sum(), rel=1e-12)
    # L1 over moduli differs from the literal real L1 (|Re| + |Im|), which is the other score id
    assert oracle64.score("rotate", 1, h, zero, t) != pytest.approx(-np.abs(h - t).sum())
    assert oracle64.score("rotate_real_l1", 1, h, zero, t) == pytest.approx(-np.abs(h - t).sum(), rel=1e-13)
    q = hc * np.exp(1j * th) - tc
    assert oracle64.score("rotate_real_l1", 1, h, th, t) == pytest.approx(-(np.abs(q.real) + np.abs(q.imag)).sum(), rel=1e-12)
    # with p = 2 the real norm is the complex one: the two ids agree
    assert oracle64.score("rotate_real_l1", 2, h, th, t) == oracle64.score("rotate", 2, h, th, t)
    # |Re| + |Im| >= modulus, component by component
    assert oracle64.score("rotate_real_l1", 1, h, th, t) <= oracle64.score("rotate", 1, h, th, t)


def test_transh_special_cases(oracle64):
    rng = np.random.default_rng(4)
    d = 9
    h, r, w, t = rng.standard_normal((4, d))
    what = w / np.linalg.norm(w)
    for p in (1, 2):
        # the definition, with numpy
        x = (h - what @ h * what) + r - (t - what @ t * what)
        assert oracle64.score("transh", p, h, r, t, w=w) == pytest.approx(-np.linalg.norm(x, ord=p), rel=1e-12)
        # r = 0 and t = h + lambda w: both project to the same point
        assert oracle64.score("transh", p, h, np.zeros(d), h + 2.5 * what, w=w) == pytest.approx(0.0, abs=1e-13)
        # normal orthogonal to h, t: TransE
        w2 = np.zeros(d); w2[0] = 3.0
        h2, t2 = h.copy(), t.copy(); h2[0] = t2[0] = 0.0
        assert oracle64.score("transh", p, h2, r, t2, w=w2) == pytest.approx(oracle64.score("transe", p, h2, r, t2), rel=1e-13)
        # the scale of w does not matter
        assert oracle64.score("transh", p, h, r, t, w=7 * w) == pytest.approx(oracle64.score("transh", p, h, r, t, w=w), rel=1e-12)


def test_bf16_operand_variant_is_close_and_exact_on_bf16_inputs(oracle64):
    rng = np.random.default_rng(5)
    d = 64
    for score in ("distmult", "complex"):
        h, r, t = rng.standard_normal((3, d)) / np.sqrt(d)
        f, fb = oracle64.score(score, 1, h, r, t), oracle64.score(score, 1, h, r, t, bf16=1)
        assert fb != f and abs(fb - f) < 2e-2 * np.abs(np.stack([h * r, t])).max() * d ** 0.5
    # inputs already representable in bf16 (small integers): both variants agree exactly
    h, t = rng.integers(-8, 8, d).astype(float), rng.integers(-8, 8, d).astype(float)
    r = np.ones(d)
    assert oracle64.score("distmult", 1, h, r, t, bf16=1) == oracle64.score("distmult", 1, h, r, t)
    assert oracle64.score("transe", 2, h, np.zeros(d), t, bf16=1) == pytest.approx(-np.linalg.norm(h - t), rel=1e-13)


def test_query_vector_is_the_tail_independent_part_of_every_score(oracle64):
    """q per model against numpy, and f(h, r, t) recovered from (q, t) alone."""
    rng = np.random.default_rng(21)
    d = 12
    h, r, t, w = rng.standard_normal((4, d))
    c = lambda v: v[0::2] + 1j * v[1::2]
    q = oracle64.query_vector("transe", h, r)
    assert q == pytest.approx(h + r, rel=1e-15)
    for p in (1, 2):
        assert oracle64.score("transe", p, h, r, t) == pytest.approx(-np.linalg.norm(q - t, ord=p), rel=1e-13)
    q = oracle64.query_vector("distmult", h, r)
    assert q == pytest.approx(r * h, rel=1e-15)
    assert oracle64.score("distmult", 1, h, r, t) == pytest.approx(q @ t, rel=1e-12)
    q = oracle64.query_vector("complex", h, r)
    assert c(q) == pytest.approx(c(r) * c(h), rel=1e-13)
    assert oracle64.score("complex", 1, h, r, t) == pytest.approx(q @ t, rel=1e-12)      # real dot of the interleaved rows
    ph = rng.uniform(-np.pi, np.pi, d // 2)
    q = oracle64.query_vector("rotate", h, ph)
    assert c(q) == pytest.approx(c(h) * np.exp(1j * ph), rel=1e-13)
    assert oracle64.score("rotate", 1, h, ph, t) == pytest.approx(-np.abs(c(q) - c(t)).sum(), rel=1e-13)
    assert oracle64.score("rotate", 2, h, ph, t) == pytest.approx(-np.linalg.norm(q - t), rel=1e-13)
    q = oracle64.query_vector("transh", h, r, w=w)
    what = w / np.linalg.norm(w)
    assert q == pytest.approx(h - (what @ h) * what + r, rel=1e-12)
    for p in (1, 2):
        x = (q - t) + (what @ t) * what
        assert oracle64.score("transh", p, h, r, t, w=w) == pytest.approx(-np.linalg.norm(x, ord=p), rel=1e-12)


def test_tie_build_differs_from_the_default_only_at_exact_ties(oracle64, oracle64_tie):
    """The build with sign(0) = -1: identical gradients on generic inputs for every model; on TransE p = 1
    with integer rows the difference is the closed form -g [x_k = 0] on dh, dr and +g [x_k = 0] on dt."""
    rng = np.random.default_rng(22)
    d = 8
    for score, p in (("transe", 1), ("transe", 2), ("transh", 1), ("transh", 2), ("rotate", 1), ("distmult", 1), ("complex", 1)):
        h, t, w = rng.standard_normal((3, d))
        r = rng.standard_normal(d // 2 if score == "rotate" else d)
        a = oracle64.score_grad(score, p, 0.7, h, r, t, w=w if score == "transh" else None)
        b = oracle64_tie.score_grad(score, p, 0.7, h, r, t, w=w if score == "transh" else None)
        for x, y in zip(a, b):
            assert x is None or (x == y).all()
    h = np.array([1., 2., -1., 0., 3., 0., 2., 1.]); r = np.array([0., -1., 1., 0., 0., 2., 1., -1.])
    t = np.array([1., 0., 0., 0., 2., 2., 5., 0.])          # x = h + r - t = (0, 1, 0, 0, 1, 0, -2, 0)
    tie = (h + r - t) == 0
    assert tie.sum() == 5
    g = 0.3
    dh0, dr0, _, dt0 = oracle64.score_grad("transe", 1, g, h, r, t)
    dh1, dr1, _, dt1 = oracle64_tie.score_grad("transe", 1, g, h, r, t)
    # f = -sum |x|: df/dx = -sign(x); at a tie the default build has 0 and the tie build -(-1) = +1
    assert (dh0[tie] == 0).all() and (dt0[tie] == 0).all()
    assert dh1 - dh0 == pytest.approx(g * tie) and dr1 - dr0 == pytest.approx(g * tie) and dt1 - dt0 == pytest.approx(-g * tie)
    # p = 2 and the dot-product models have no such kink: the builds agree on these rows too
    for score, p in (("transe", 2), ("distmult", 1)):
        for x, y in zip(oracle64.score_grad(score, p, g, h, r, t), oracle64_tie.score_grad(score, p, g, h, r, t)):
            assert x is None or (x == y).all()


def _f32(bits):
    return float(np.array([bits], dtype=np.uint32).view(np.float32)[0])


# (fp32 input bits, bf16 result as the upper 16 bits) worked out by hand from the IEEE definition of
# round-to-nearest-even to an 8-bit significand: bf16 keeps the upper 16 bits of the fp32 pattern, the
# lower 16 bits are the discarded fraction (0x8000 = exactly half a unit in the last kept place).
BF16_PATTERNS = [
    (0x3F800000, 0x3F80),   # 1.0 is representable
    (0x3F808000, 0x3F80),   # 1 + 2^-8: a tie, kept mantissa 0000000 is even -> down to 1.0
    (0x3F818000, 0x3F82),   # 1 + 3 2^-8: a tie, kept mantissa 0000001 is odd -> up to 1 + 2^-6
    (0x3F808001, 0x3F81),   # just above the tie -> up
    (0x3F807FFF, 0x3F80),   # just below the tie -> down
    (0x3F810001, 0x3F81),   # just above a representable value -> stays
    (0xBF808000, 0xBF80),   # the negative twins: rounding is symmetric in the sign
    (0xBF818000, 0xBF82),
    (0xBF808001, 0xBF81),
    (0x3FFF8000, 0x4000),   # 2 - 2^-8: a tie with kept mantissa 1111111 (odd) -> carries into the exponent: 2.0
    (0x3FFF7FFF, 0x3FFF),   # just below it -> 2 - 2^-7
    (0x7F7F7FFF, 0x7F7F),   # the largest input that stays finite
    (0x7F7FFFFF, 0x7F80),   # the largest finite fp32 lies above the last tie -> +inf
    (0x7F7F8000, 0x7F80),   # that tie itself: kept mantissa odd -> up -> +inf
    (0x00000001, 0x0000),   # smallest fp32 subnormal -> +0
    (0x00008000, 0x0000),   # half of the smallest bf16 subnormal: a tie -> even -> +0
    (0x00008001, 0x0001),   # just above -> the smallest bf16 subnormal 2^-133
    (0x00018000, 0x0002),   # 1.5 x 2^-133: a tie, odd -> up to 2^-132
    (0x007F8000, 0x0080),   # subnormal that rounds up into the smallest normal 2^-126
    (0x80008000, 0x8000),   # -0 result keeps its sign
]


def test_bf16_round_hand_worked_bit_patterns(oracle64, oracle32):
    for o in (oracle64, oracle32):
        for bits, want_hi in BF16_PATTERNS:
            got = np.array([o.bf16_round(_f32(bits))], dtype=np.float32).view(np.uint32)[0]
            assert got == want_hi << 16, (hex(bits), hex(got), hex(want_hi << 16))
    # a few of the same as plain numbers
    assert oracle64.bf16_round(1 + 2.0 ** -8) == 1.0
    assert oracle64.bf16_round(1 + 3 * 2.0 ** -8) == 1 + 2.0 ** -6
    assert oracle64.bf16_round(-(1 + 2.0 ** -8 + 2.0 ** -20)) == -(1 + 2.0 ** -7)
    assert oracle64.bf16_round(2 - 2.0 ** -8) == 2.0
    assert oracle64.bf16_round(3.3895313892515355e38) == 3.3895313892515355e38     # (2 - 2^-7) 2^127, the largest bf16
    assert oracle64.bf16_round(float(np.finfo(np.float32).max)) == float("inf")


def test_bf16_round_against_an_independent_routine_on_random_floats(oracle64):
    """torch's float -> bfloat16 conversion (round to nearest even) on 10^5 random bit patterns of
    every magnitude, and exact rational arithmetic on a sample of them."""
    import torch
    from fractions import Fraction
    rng = np.random.default_rng(11)
    bits = rng.integers(0, 2 ** 32, size=100_000, dtype=np.uint64).astype(np.uint32)
    x = bits.view(np.float32)
    x = x[np.isfinite(x)]
    want = torch.from_numpy(x.copy()).to(torch.bfloat16).to(torch.float32).numpy()
    got = np.array([oracle64.bf16_round(float(v)) for v in x], dtype=np.float32)
    assert (got.view(np.uint32) == want.view(np.uint32)).all()
    # the definition itself on normal numbers: nearest multiple of 2^(e-7), ties to the even multiple
    for v in x[:2000]:
        if v == 0 or abs(float(v)) < 2.0 ** -120 or abs(float(v)) > 2.0 ** 120:
            continue
        fr = Fraction(float(v))
        e = int(np.floor(np.log2(abs(float(v)))))
        while Fraction(2) ** e > abs(fr):
            e -= 1
        while Fraction(2) ** (e + 1) <= abs(fr):
            e += 1
        ulp = Fraction(2) ** (e - 7)
        n = fr / ulp
        lo = n.numerator // n.denominator
        rem = n - lo
        k = lo + (1 if rem > Fraction(1, 2) or (rem == Fraction(1, 2) and lo % 2 == 1) else 0)
        assert Fraction(oracle64.bf16_round(float(v))) == k * ulp, float(v)


def test_bf16_norm_expansion_clamps_negative_squared_distance(oracle64):
    """TransE p = 2 in the bf16 variant is -sqrt(max(|q|^2 + |t|^2 - 2 bf16(q).bf16(t), 0)).  With q = t the
    exact distance is 0, but the rounded cross term differs from |q|^2: operands that round up in magnitude
    make the expansion negative, which must clamp to a score of exactly 0 (not NaN); operands that round
    down leave 2 d (x^2 - bf16(x)^2) > 0, whose root is the score."""
    d = 4
    up = 1 + 0.75 * 2.0 ** -7          # rounds to 1 + 2^-7: bf16(q).bf16(t) > |q|^2
    f = oracle64.score("transe", 2, np.full(d, up), np.zeros(d), np.full(d, up), bf16=1)
    assert f == 0.0 and not np.isnan(f)
    down = 1 + 0.25 * 2.0 ** -7        # rounds to 1.0
    f = oracle64.score("transe", 2, np.full(d, down), np.zeros(d), np.full(d, down), bf16=1)
    assert f == pytest.approx(-np.sqrt(2 * d * (down * down - 1.0)), rel=1e-12)
    # the exact variant scores 0 in both cases
    assert oracle64.score("transe", 2, np.full(d, up), np.zeros(d), np.full(d, up)) == 0.0


# ----------------------------------------------------------------------------- losses
def test_sampled_softmax_uniform_scores_closed_forms(oracle64):
    N, E = 37, 1000
    base = dict(num_entities=E, num_relations=1, dim=4, score="distmult", loss="softmax", num_neg=N)
    L, gpos, G = oracle64.row_loss(make_config(**base), 0.3, np.full(N, 0.3))
    assert L == pytest.approx(np.log(N + 1), rel=1e-13)                      # c = 0
    assert gpos + G.sum() == pytest.approx(0.0, abs=1e-14) and G == pytest.approx(1 / (N + 1))
    L, _, _ = oracle64.row_loss(make_config(**base, ce_correction=np.log((E - 1) / N)), 0.3, np.full(N, 0.3))
    assert L == pytest.approx(np.log(E), rel=1e-13)                          # the paper's c
    # general scores against scipy-free numpy logsumexp, including large magnitudes
    rng = np.random.default_rng(6)
    F = rng.standard_normal(N) * 50
    c = 1.7
    L, gpos, G = oracle64.row_loss(make_config(**base, ce_correction=c), 2.0, F)
    z = np.concatenate([[2.0], F + c])
    lse = z.max() + np.log(np.exp(z - z.max()).sum())
    assert L == pytest.approx(-2.0 + lse, rel=1e-12)
    assert gpos + 1 + G.sum() == pytest.approx(1.0, rel=1e-12)


def test_logsigmoid_closed_forms(oracle64):
    N = 8
    base = dict(num_entities=10, num_relations=1, dim=4, score="transe", loss="logsigmoid", num_neg=N)
    L, gpos, G = oracle64.row_loss(make_config(**base, gamma=0.0, adv_temp=0.0), 0.0, np.zeros(N))
    assert L == pytest.approx(2 * np.log(2), rel=1e-13)
    assert gpos == pytest.approx(-0.5) and G == pytest.approx(np.full(N, 0.5 / N))
    # definition with numpy, gamma and self-adversarial temperature on
    rng = np.random.default_rng(7)
    F = -np.abs(rng.standard_normal(N)) * 6
    fpos, gamma, a = -3.0, 5.0, 0.7
    L, gpos, G = oracle64.row_loss(make_config(**base, gamma=gamma, adv_temp=a), fpos, F)
    sig = lambda z: 1 / (1 + np.exp(-z))
    w = np.exp(a * F) / np.exp(a * F).sum()
    assert L == pytest.approx(-np.log(sig(gamma + fpos)) - (w * np.log(sig(-gamma - F))).sum(), rel=1e-12)
    assert G == pytest.approx(w * sig(gamma + F), rel=1e-12)
    # a = 0: uniform weights; very negative argument stays finite
    L, _, G = oracle64.row_loss(make_config(**base, gamma=0.0, adv_temp=0.0), -800.0, np.full(N, 800.0))
    assert L == pytest.approx(1600.0, rel=1e-13) and np.isfinite(G).all()


# ----------------------------------------------------------------------------- gradients
def _tiny_problem(rng, score, E=7, R=3, d=4, B=3, N=5):
    ent = rng.standard_normal((E, d)) * 0.7
    rel = rng.uniform(-np.pi, np.pi, (R, d // 2)) if score in ROTATE else rng.standard_normal((R, d)) * 0.7
    relw = rng.standard_normal((R, d)) if score == "transh" else None
    # repeated rows on purpose: entity 2 is a head, a tail and a negative; relation 1 twice
    heads = np.array([2, 0, 5], np.int32); rels = np.array([1, 1, 0], np.int32)
    tails = np.array([3, 2, 6], np.int32); negs = np.array([2, 4, 4, 1, 6], np.int32)
    return ent, rel, relw, heads, rels, tails, negs


def test_l3_regulariser_term_and_lr_decay_closed_forms(oracle64):
    e = np.array([1.0, -2.0, 2.0, 0.0])
    assert oracle64.l3_term(0, e) == pytest.approx(17.0 ** (1 / 3), rel=1e-15)       # ||e||_3 = (1 + 8 + 8)^(1/3)
    assert oracle64.l3_term(1, e) == pytest.approx(17.0, rel=1e-15)
    assert oracle64.l3_term(0, -3 * e) == pytest.approx(3 * 17.0 ** (1 / 3), rel=1e-14)  # a norm is homogeneous
    assert oracle64.l3_term(0, np.zeros(4)) == 0.0
    # the batch term counts every occurrence of a row: lambda (sum over heads, tails, negatives)
    rng = np.random.default_rng(3)
    ent, rel, relw, heads, rels, tails, negs = _tiny_problem(rng, "distmult")
    kw = dict(num_entities=7, num_relations=3, dim=4, score="distmult", batch=3, num_neg=5, loss_scale=0.5)
    base = oracle64.batch_loss(make_config(**kw), ent, rel, None, heads, rels, tails, negs)["loss"]
    for form in (0, 1):
        omega = sum(np.sum(np.abs(ent[i]) ** 3) ** (1.0 if form else 1 / 3) for i in np.concatenate([heads, tails, negs]))
        got = oracle64.batch_loss(make_config(**kw, reg_lambda=0.3, reg_form=form), ent, rel, None, heads, rels, tails, negs)["loss"]
        assert got == pytest.approx(base + 0.3 * omega, rel=1e-13)                   # added as it stands, not times loss_scale
    # linear decay to zero (Section 5)
    assert oracle64.lr_linear_decay(0.05, 0, 1000) == 0.05 and oracle64.lr_linear_decay(0.05, 1000, 1000) == 0.0
    assert oracle64.lr_linear_decay(0.05, 500, 1000) == pytest.approx(0.025, rel=1e-15)
    assert oracle64.lr_linear_decay(0.05, 2000, 1000) == 0.0
    steps = np.arange(0, 1000, 37)
    lrs = np.array([oracle64.lr_linear_decay(0.05, int(s), 1000) for s in steps])
    assert np.allclose(np.diff(lrs), -0.05 * 37 / 1000, rtol=1e-12, atol=0)


@pytest.mark.parametrize("score,p", MODELS)
@pytest.mark.parametrize("loss,reg", [("logsigmoid", None), ("softmax", None), ("softmax", 0), ("logsigmoid", 1)])
def test_batch_grads_match_central_finite_differences(oracle64, score, p, loss, reg):
    rng = np.random.default_rng(100 * MODELS.index((score, p)) + len(loss))
    ent, rel, relw, heads, rels, tails, negs = _tiny_problem(rng, score)
    E, d = ent.shape
    cfg = make_config(num_entities=E, num_relations=len(rel), dim=d, score=score, p_norm=p, loss=loss,
                      batch=3, num_neg=5, gamma=1.5 if loss == "logsigmoid" else 0.0, adv_temp=0.8,
                      ce_correction=0.4, loss_scale=0.5, reg_lambda=0.0 if reg is None else 0.37, reg_form=reg or 0)
    out = oracle64.batch_grads(cfg, ent, rel, relw, heads, rels, tails, negs)
    base = oracle64.batch_loss(cfg, ent, rel, relw, heads, rels, tails, negs)
    assert out["loss"] == pytest.approx(base["loss"], rel=1e-14)
    # StopGrad: the self-adversarial weights are constants of the differentiation
    w_fixed = None
    if loss == "logsigmoid":
        aF = cfg.adv_temp * base["F"]
        w_fixed = np.exp(aF - aF.max(1, keepdims=True)); w_fixed /= w_fixed.sum(1, keepdims=True)
    # analytic table gradients = scatter-add of the per-slot gradient rows
    g_ent = np.zeros_like(ent); g_rel = np.zeros_like(rel)
    np.add.at(g_ent, heads, out["dh"]); np.add.at(g_ent, tails, out["dtpos"]); np.add.at(g_ent, negs, out["dtneg"])
    np.add.at(g_rel, rels, out["dr"])
    g_w = None
    if relw is not None:
        g_w = np.zeros_like(relw); np.add.at(g_w, rels, out["dw"])

    def loss_at(e, r, w):
        return oracle64.batch_loss(cfg, e, r, w, heads, rels, tails, negs, w_fixed=w_fixed)["loss"]

    eps = 1e-6
    for name, tab, grad in (("ent", ent, g_ent), ("rel", rel, g_rel), ("relw", relw, g_w)):
        if tab is None:
            continue
        for idx in itertools.product(range(tab.shape[0]), range(tab.shape[1])):
            args = dict(ent=ent, rel=rel, relw=relw)
            plus, minus = tab.copy(), tab.copy()
            plus[idx] += eps; minus[idx] -= eps
            args[name] = plus; lp = loss_at(args["ent"], args["rel"], args["relw"])
            args[name] = minus; lm = loss_at(args["ent"], args["rel"], args["relw"])
            fd = (lp - lm) / (2 * eps)
            assert grad[idx] == pytest.approx(fd, rel=2e-6, abs=2e-8), (name, idx)
    # untouched rows have zero gradient, touched tables do not vanish
    assert np.abs(g_ent).sum() > 0 and np.abs(g_rel).sum() > 0
    assert (g_rel[2] == 0).all()


def test_subgradient_conventions_at_kinks(oracle64):
    d = 4
    h = np.array([1.0, -2.0, 0.5, 0.0]); r = np.zeros(d)
    # L1: coordinates with zero residual get zero gradient
    dh, dr, _, dt = oracle64.score_grad("transe", 1, 1.0, h, r, np.array([1.0, 0.0, 0.5, 3.0]))
    assert (dh == np.array([0.0, 1.0, 0.0, 1.0])).all() and (dt == -dh).all() and (dr == dh).all()
    # L2 / modulus at zero distance: zero gradient, no NaN
    for score in ("transe", "rotate"):
        rr = np.zeros(d // 2) if score == "rotate" else r
        for p in (1, 2):
            dh, _, _, dt = oracle64.score_grad(score, p, 1.0, h, rr, h)
            assert (dh == 0).all() and (dt == 0).all()

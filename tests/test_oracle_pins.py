"""Pins for the CPU oracle: every check here compares the oracle with something
other than itself -- published known-answer vectors, an independent
big-integer Philox, hand-worked values, exact identities, brute force and
closed forms.  No GPU is needed."""
import itertools
import os
from fractions import Fraction

import numpy as np
import pytest

import oracle
from conftest import GOLDEN

M32 = 0xFFFFFFFF


# --------------------------------------------------------------------------
# Independent Philox4x32-10 in unbounded Python integers, written from the
# round definition of the SC'11 paper (Section 3.3): multiply words 0 and 2 by
# the two constants, xor the high halves with words 1/3 and the round key,
# permute; the key advances by the Weyl constants before rounds 2..10.
# --------------------------------------------------------------------------
def py_philox4x32_10(ctr, key):
    c = [int(w) for w in ctr]
    k = [int(w) for w in key]
    for rnd in range(10):
        if rnd:
            k = [(k[0] + 0x9E3779B9) & M32, (k[1] + 0xBB67AE85) & M32]
        prod0 = 0xD2511F53 * c[0]
        prod1 = 0xCD9E8D57 * c[2]
        c = [((prod1 >> 32) ^ c[1] ^ k[0]) & M32, prod1 & M32,
             ((prod0 >> 32) ^ c[3] ^ k[1]) & M32, prod0 & M32]
    return c


def py_draw(seed, s, i, d):
    """(r1, r2) as exact fractions, from the counter/key packing the library
    defines: counter {d>>1, i, s, 0}, key = low/high half of the seed, even
    element takes words 0,1 and odd element words 2,3."""
    o = py_philox4x32_10([d >> 1, i, s, 0], [seed & M32, seed >> 32])
    a, b = (o[2], o[3]) if d & 1 else (o[0], o[1])
    return Fraction(a >> 8, 1 << 24), Fraction(b >> 8, 1 << 24)


def test_philox_known_answers():
    rows = 0
    with open(os.path.join(GOLDEN, "philox4x32_10_kat.txt")) as fh:
        for line in fh:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            w = [int(t, 16) for t in line.split()]
            assert len(w) == 10
            got = oracle.philox4x32_10(w[0:4], w[4:6])
            assert [int(g) for g in got] == w[6:10]
            assert py_philox4x32_10(w[0:4], w[4:6]) == w[6:10]
            rows += 1
    assert rows == 3


def test_philox_matches_big_integer_implementation():
    rng = np.random.default_rng(1234)
    words = rng.integers(0, 1 << 32, size=(10_000, 6), dtype=np.uint64)
    # structured counters too: small values, single bits, carries in the key
    extra = [[1, 0, 0, 0, 0, 0], [0, 1, 0, 0, 0, 0], [0, 0, 1, 0, 0, 0],
             [0, 0, 0, 1, 0, 0], [0, 0, 0, 0, 1, 0], [0, 0, 0, 0, 0, 1],
             [M32, 0, M32, 0, 0x61C88647, 0x44985179]]
    for w in list(words) + extra:
        w = [int(t) for t in w]
        assert [int(g) for g in oracle.philox4x32_10(w[:4], w[4:])] == \
            py_philox4x32_10(w[:4], w[4:])


def test_uniform_is_exact_24_bit_grid():
    for word in [0, 1, 255, 256, 257, 0x80000000, 0xFFFFFF00, M32, 0x12345678]:
        r = oracle.uniform(word)
        assert Fraction(float(r)) == Fraction(word >> 8, 1 << 24)
        assert 0.0 <= float(r) < 1.0
    assert float(oracle.uniform(M32)) == 1.0 - 2.0 ** -24


def test_draw_packing_matches_definition():
    rng = np.random.default_rng(7)
    for _ in range(2000):
        seed = int(rng.integers(0, 1 << 63)) * 2 + int(rng.integers(0, 2))
        s = int(rng.integers(0, 1 << 32))
        i = int(rng.integers(0, 1024))
        d = int(rng.integers(0, 1 << 33))
        r1, r2 = oracle.draw(seed, s, i, d)
        e1, e2 = py_draw(seed, s, i, d)
        assert Fraction(float(r1)) == e1 and Fraction(float(r2)) == e2
    # neighbouring elements share one call, neighbouring pairs do not
    assert oracle.draw(5, 0, 0, 10) != oracle.draw(5, 0, 0, 11)
    assert oracle.draw(5, 0, 0, 10) != oracle.draw(5, 0, 1, 10)
    assert oracle.draw(5, 0, 0, 10) != oracle.draw(5, 1, 0, 10)
    assert oracle.draw(5, 0, 0, 10) != oracle.draw(6, 0, 0, 10)
    assert oracle.draw(5, 0, 0, 10) != oracle.draw(5 + (1 << 32), 0, 0, 10)


def _draws_through_sync(n, seed, s, which):
    """Recover r1 (which=1) or r2 (which=2) of particle 1 for elements 0..n-1
    from a sync whose other factors are exactly 1 or 0."""
    x = np.zeros((2, n), np.float32)
    v = np.zeros((2, n), np.float32)
    p = np.zeros((2, n), np.float32)
    if which == 1:
        p[1] = 1.0                      # pBest - w = 1, c1 = 1, c2 = 0
        c1, c2 = 1.0, 0.0
    else:
        x[0] = 1.0                      # gBest - w = 1 for particle 1
        p[0] = 1.0
        c1, c2 = 0.0, 1.0
    pl = np.array([0.0, 0.0], np.float32)   # nobody improves
    g, imp, _ = oracle.sync(x, v, p, [1.0, 2.0], pl, m_max=0.0, m_min=0.0, t=0,
                            t_max=1, c1=c1, c2=c2, lam=1.0, seed=seed, s=s)
    assert g == 0 and not imp.any()
    return v[1].copy()


def test_sync_uses_the_documented_stream_and_it_is_uniform():
    n = 4_000_000
    r1 = _draws_through_sync(n, seed=0xDEADBEEFCAFE, s=3, which=1)
    r2 = _draws_through_sync(n, seed=0xDEADBEEFCAFE, s=3, which=2)
    for d in [0, 1, 2, 3, 4, 5, 1000, 1001, n - 2, n - 1]:
        e1, e2 = py_draw(0xDEADBEEFCAFE, 3, 1, d)
        assert Fraction(float(r1[d])) == e1
        assert Fraction(float(r2[d])) == e2
    for r in (r1, r2):
        assert r.min() >= 0.0 and r.max() < 1.0
        assert abs(float(r.mean(dtype=np.float64)) - 0.5) < 1e-3
        assert abs(float(r.var(dtype=np.float64)) - 1.0 / 12.0) < 1e-3
        hist = np.histogram(r, bins=16, range=(0.0, 1.0))[0] / n
        assert np.abs(hist - 1 / 16).max() < 1e-3
    # r1 and r2 are different streams, and so are successive elements
    assert abs(float(np.corrcoef(r1, r2)[0, 1])) < 5e-3
    assert abs(float(np.corrcoef(r1[:-1], r1[1:])[0, 1])) < 5e-3
    assert np.count_nonzero(r1 == r2) < 10


# --------------------------------------------------------------------------
# Hand-worked examples (Algorithm 1 + Algorithm 3 + Eq. 6/7).
# --------------------------------------------------------------------------
def _parse_cases(path):
    cases, cur = [], None
    with open(path) as fh:
        for line in fh:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            key, _, rest = line.partition(" ")
            if key == "case":
                cur = {"name": rest}
                cases.append(cur)
                continue
            rows = [[float(t) for t in r.split()] for r in rest.split(";")]
            if key in ("m", "c1", "c2", "lambda", "expect_g"):
                cur[key] = rows[0][0]
            else:
                cur[key] = np.array(rows if len(rows) > 1 else rows[0], np.float32)
    return cases


@pytest.mark.parametrize("case", _parse_cases(os.path.join(GOLDEN, "hand_worked_sync.txt")),
                         ids=lambda c: c["name"])
def test_hand_worked_sync(case):
    x, v, p = case["x"].copy(), case["v"].copy(), case["p"].copy()
    pl = case["pbest_loss"].copy()
    g, imp, gb = oracle.sync(x, v, p, case["loss"], pl,
                             m_max=case["m"], m_min=case["m"], t=0, t_max=1,
                             c1=case["c1"], c2=case["c2"], lam=case["lambda"],
                             seed=0, s=0, fixed_r=case["r"], want_gbest=True)
    assert g == int(case["expect_g"])
    assert imp.tolist() == [bool(b) for b in np.atleast_1d(case["expect_improved"])]
    assert np.array_equal(gb, case["expect_gbest"])
    assert np.array_equal(v, case["expect_v"])
    assert np.array_equal(x, case["expect_x"])
    assert np.array_equal(p, case["expect_p"])
    assert np.array_equal(pl, case["expect_pbest_loss"])


# --------------------------------------------------------------------------
# Exact identities of Eq. 6/7 and of the sync ordering.
# --------------------------------------------------------------------------
def _random_swarm(K, n, seed, pad=0):
    rng = np.random.default_rng(seed)
    mk = lambda: np.ascontiguousarray(  # noqa: E731
        rng.standard_normal((K, n + pad)).astype(np.float32))
    return mk(), mk(), mk()


def test_identity_pure_inertia_is_exact_x_plus_v():
    x, v, p = _random_swarm(5, 1001, 11)
    x0, v0 = x.copy(), v.copy()
    loss = np.array([3, 1, 2, 5, 4], np.float32)
    pl = np.zeros(5, np.float32)
    oracle.sync(x, v, p, loss, pl, m_max=1.0, m_min=1.0, t=0, t_max=1,
                c1=0.0, c2=0.0, lam=1.0, seed=9, s=0)
    assert np.array_equal(v, v0)
    assert np.array_equal(x, x0 + v0)           # one fp32 addition per element


def test_identity_fixed_point_when_swarm_is_collapsed():
    rng = np.random.default_rng(3)
    row = rng.standard_normal(513).astype(np.float32)
    x = np.tile(row, (6, 1))
    v = np.zeros_like(x)
    p = x.copy()
    loss = rng.random(6).astype(np.float32)
    pl = np.full(6, np.inf, np.float32)
    for s in range(3):
        oracle.sync(x, v, p, loss, pl, m_max=0.7, m_min=0.7, t=0, t_max=1,
                    c1=1.5, c2=1.5, lam=1.0, seed=1, s=s)
        assert np.array_equal(x, np.tile(row, (6, 1)))
        assert not v.any() and np.array_equal(p, x)


def test_identity_single_particle():
    x, v, p = _random_swarm(1, 300, 5)
    x0, v0 = x.copy(), v.copy()
    pl = np.full(1, np.inf, np.float32)
    g, imp, _ = oracle.sync(x, v, p, [0.5], pl, m_max=0.5, m_min=0.5, t=0,
                            t_max=1, c1=1.5, c2=1.5, lam=1.0, seed=2, s=0)
    # K=1: the particle is gBest and has just improved, both searches vanish
    assert g == 0 and imp.tolist() == [True]
    assert np.array_equal(v, np.float32(0.5) * v0)
    assert np.array_equal(x, x0 + v)
    assert np.array_equal(p, x0) and pl[0] == np.float32(0.5)


def test_gbest_particle_and_improved_particle_lose_their_terms():
    K, n = 4, 257
    x, v, p = _random_swarm(K, n, 21)
    loss = np.array([0.9, 0.2, 0.5, 0.7], np.float32)          # g = 1
    pl0 = np.array([1.0, 0.1, 0.4, 0.6], np.float32)           # only 0 improves
    outs = []
    for c1, c2 in [(1.5, 1.5), (0.25, 1.5), (1.5, 0.75)]:
        xx, vv, pp, pl = x.copy(), v.copy(), p.copy(), pl0.copy()
        g, imp, _ = oracle.sync(xx, vv, pp, loss, pl, m_max=0.7, m_min=0.7, t=0,
                                t_max=1, c1=c1, c2=c2, lam=1.0, seed=4, s=0)
        assert g == 1 and imp.tolist() == [True, False, False, False]
        outs.append((xx, vv, pp))
    # particle 0 improved: pBest = w, so its result cannot depend on c1
    assert np.array_equal(outs[0][1][0], outs[1][1][0])
    assert not np.array_equal(outs[0][1][2], outs[1][1][2])
    # particle 1 is gBest: gBest - w = 0, so its result cannot depend on c2
    assert np.array_equal(outs[0][1][1], outs[2][1][1])
    assert not np.array_equal(outs[0][1][2], outs[2][1][2])
    # pBest of the improved particle is its pre-update weight; others untouched
    assert np.array_equal(outs[0][2][0], x[0])
    assert np.array_equal(outs[0][2][1:], p[1:])
    # gBest particle: v' = fma(t1, pBest - w, m v) with the documented draw
    for d in range(n):
        r1, _ = py_draw(4, 0, 1, d)
        t1 = np.float32(1.5) * np.float32(float(r1))
        dl = np.float32(p[1, d] - x[1, d])
        a0 = np.float32(0.7) * v[1, d]
        expect = Fraction(float(t1)) * Fraction(float(dl)) + Fraction(float(a0))
        got = Fraction(float(outs[0][1][1, d]))
        # correctly rounded result of the exact fused expression
        assert np.float32(float(expect)) == np.float32(float(got))


def test_textbook_pso_special_case_in_exact_arithmetic():
    """lambda = 1 and constant m reduce Eq. 6/7 to the standard PSO update
    (Eq. 3/4); evaluate that in exact rational arithmetic with draws from the
    independent Philox and require fp32-level agreement."""
    K, n, seed, s = 3, 40, 77, 5
    x, v, p = _random_swarm(K, n, 31)
    x0, v0, p0 = x.copy(), v.copy(), p.copy()
    loss = np.array([0.8, 0.3, 0.6], np.float32)
    pl = np.array([0.1, 0.1, 0.1], np.float32)                 # nobody improves
    m, c1, c2 = np.float32(0.7), np.float32(1.5), np.float32(0.9)
    oracle.sync(x, v, p, loss, pl, m_max=m, m_min=m, t=0, t_max=1, c1=c1, c2=c2,
                lam=1.0, seed=seed, s=s)
    F = lambda a: Fraction(float(a))  # noqa: E731
    for i in range(K):
        for d in range(n):
            r1, r2 = py_draw(seed, s, i, d)
            ve = (F(m) * F(v0[i, d]) + F(c1) * r1 * (F(p0[i, d]) - F(x0[i, d]))
                  + F(c2) * r2 * (F(x0[1, d]) - F(x0[i, d])))
            xe = F(x0[i, d]) + ve
            scale = (abs(F(m) * F(v0[i, d])) + abs(F(c1) * r1 * (F(p0[i, d]) - F(x0[i, d])))
                     + abs(F(c2) * r2 * (F(x0[1, d]) - F(x0[i, d]))))
            assert abs(F(v[i, d]) - ve) <= scale * Fraction(4, 1 << 24)
            assert abs(F(x[i, d]) - xe) <= (scale + abs(F(x0[i, d]))) * Fraction(4, 1 << 24)
    assert np.array_equal(p, p0)


def test_lambda_divides_both_search_terms():
    """Eq. 6: lambda = 4 with (c1, c2) equals lambda = 1 with (c1/4, c2/4)."""
    x, v, p = _random_swarm(4, 129, 8)
    loss = np.array([0.5, 0.4, 0.9, 0.7], np.float32)
    res = []
    for c1, c2, lam in [(2.0, 1.0, 4.0), (0.5, 0.25, 1.0)]:
        xx, vv, pp = x.copy(), v.copy(), p.copy()
        pl = np.zeros(4, np.float32)
        oracle.sync(xx, vv, pp, loss, pl, m_max=0.6, m_min=0.6, t=0, t_max=1,
                    c1=c1, c2=c2, lam=lam, seed=3, s=1)
        res.append((xx, vv))
    assert np.array_equal(res[0][0], res[1][0]) and np.array_equal(res[0][1], res[1][1])


# --------------------------------------------------------------------------
# Selection: brute force over small loss alphabets.
# --------------------------------------------------------------------------
def test_selection_brute_force():
    alphabet = [np.float32(0.0), np.float32(-0.0), np.float32(1.0),
                np.float32(np.inf), np.float32(0.5)]
    for loss in itertools.product(alphabet, repeat=4):
        loss = np.array(loss, np.float32)
        best = min(float(a) for a in loss)
        expect_g = next(i for i, a in enumerate(loss) if float(a) == best)
        assert oracle.argmin(loss) == expect_g
    small = [np.float32(0.0), np.float32(1.0), np.float32(np.inf)]
    for loss in itertools.product(small, repeat=3):
        for pl in itertools.product(small, repeat=3):
            imp, new = oracle.pbest_select(loss, pl)
            for i in range(3):
                better = float(loss[i]) < float(pl[i])      # strict: equal never improves
                assert bool(imp[i]) == better
                assert float(new[i]) == (float(loss[i]) if better else float(pl[i]))


def test_selection_nan_never_wins():
    nan = np.float32(np.nan)
    assert oracle.argmin([nan, 2.0, 1.0]) == 2
    assert oracle.argmin([2.0, nan, 1.0, 1.0]) == 2
    assert oracle.argmin([nan, nan]) == 0
    imp, new = oracle.pbest_select([nan, 1.0], [np.inf, nan])
    assert imp.tolist() == [False, False]


def test_argmin_ties_lowest_index_random():
    rng = np.random.default_rng(0)
    for _ in range(500):
        K = int(rng.integers(1, 40))
        loss = rng.integers(0, 4, size=K).astype(np.float32)
        assert oracle.argmin(loss) == int(np.argmin(loss))   # numpy: first minimum


# --------------------------------------------------------------------------
# Eq. 5.
# --------------------------------------------------------------------------
def test_inertia_schedule_endpoints_and_midpoint():
    assert oracle.inertia(0.9, 0.3, 0, 1000) == np.float32(0.9)
    assert oracle.inertia(0.9, 0.3, 1000, 1000) == np.float32(0.3)
    mid = (float(np.float32(0.9)) + float(np.float32(0.3))) / 2
    assert oracle.inertia(0.9, 0.3, 500, 1000) == np.float32(mid)
    assert oracle.inertia(0.7, 0.7, 123, 1000) == np.float32(0.7)
    # monotone decrease, clamped outside [0, t_max]
    vals = [float(oracle.inertia(0.9, 0.3, t, 50)) for t in range(51)]
    assert all(a > b for a, b in zip(vals, vals[1:]))
    assert oracle.inertia(0.9, 0.3, -5, 50) == np.float32(0.9)
    assert oracle.inertia(0.9, 0.3, 99, 50) == np.float32(0.3)
    # a quarter of the way, in exact arithmetic
    q = Fraction(float(np.float32(0.9))) - Fraction(1, 4) * (
        Fraction(float(np.float32(0.9))) - Fraction(float(np.float32(0.3))))
    assert oracle.inertia(0.9, 0.3, 25, 100) == np.float32(float(q))


# --------------------------------------------------------------------------
# Parameter averaging.
# --------------------------------------------------------------------------
def test_average_closed_forms():
    rng = np.random.default_rng(2)
    one = rng.standard_normal((1, 77)).astype(np.float32)
    keep = one.copy()
    oracle.average(one)
    assert np.array_equal(one, keep)                                   # K = 1
    two = rng.standard_normal((2, 1000)).astype(np.float32)
    expect = ((two[0].astype(np.float64) + two[1].astype(np.float64)) / 2).astype(np.float32)
    oracle.average(two)
    assert np.array_equal(two[0], expect) and np.array_equal(two[1], expect)
    ints = rng.integers(-1000, 1000, size=(8, 333)).astype(np.float32)  # exactly summable
    mean = ints.astype(np.float64).mean(axis=0)
    oracle.average(ints)
    assert np.array_equal(ints, np.tile(mean.astype(np.float32), (8, 1)))
    gen = rng.standard_normal((7, 4096)).astype(np.float32)
    ref = gen.astype(np.float64).mean(axis=0)
    mag = np.abs(gen).astype(np.float64).sum(axis=0) / 7
    oracle.average(gen)
    assert np.all(np.abs(gen - ref) <= 7 * 2.0 ** -24 * mag + 1e-45)
    assert all(np.array_equal(gen[0], gen[k]) for k in range(7))


def test_average_respects_row_stride_and_padding():
    rng = np.random.default_rng(4)
    buf = rng.standard_normal((3, 16)).astype(np.float32)
    keep = buf.copy()
    view = buf[:, :13]
    oracle.average(view)
    assert np.array_equal(buf[:, 13:], keep[:, 13:])
    assert np.array_equal(buf[0, :13], buf[2, :13])


# --------------------------------------------------------------------------
# Quadratic stand-in fitness.
# --------------------------------------------------------------------------
@pytest.mark.parametrize("n", [1, 3, 4, 5, 127, 128, 129, 4096, 131_072 + 5, 300_001])
def test_quadratic_fitness_against_plain_double_sum(n):
    rng = np.random.default_rng(n)
    x = rng.standard_normal(n).astype(np.float32)
    t = rng.standard_normal(n).astype(np.float32)
    d = (0.5 + 1.5 * rng.random(n)).astype(np.float32)
    # fp32 terms as defined, then a plain sequential double sum
    e = x - t
    terms = (d * (e * e)).astype(np.float32).astype(np.float64)
    plain = float(np.sum(terms))          # pairwise in numpy; both are ~1e-16-accurate
    got = float(oracle.quadratic_fitness(x, d, t))
    assert abs(got - plain) <= 1e-6 * plain          # fp32 rounding of the result
    assert got == float(np.float32(plain)) or abs(got - plain) <= 2.0 ** -23 * plain
    # and against the mathematical value
    exact = float(np.sum(d.astype(np.float64) * (x.astype(np.float64) - t.astype(np.float64)) ** 2))
    assert abs(got - exact) <= 1e-6 * exact


def test_quadratic_fitness_special_cases():
    rng = np.random.default_rng(6)
    n = 1000
    t = rng.standard_normal(n).astype(np.float32)
    d = (0.5 + 1.5 * rng.random(n)).astype(np.float32)
    assert float(oracle.quadratic_fitness(t.copy(), d, t)) == 0.0
    for j in [0, 1, 3, 4, 127, 128, 500, 999]:
        x = t.copy()
        x[j] = t[j] + np.float32(3.0)
        e = np.float32(x[j] - t[j])
        assert oracle.quadratic_fitness(x, d, t) == np.float32(d[j] * np.float32(e * e))
    # small integers: every partial sum is exact, so any order gives the same value
    xi = rng.integers(-8, 8, size=n).astype(np.float32)
    ti = rng.integers(-8, 8, size=n).astype(np.float32)
    di = rng.integers(1, 4, size=n).astype(np.float32)
    assert float(oracle.quadratic_fitness(xi, di, ti)) == float(np.sum(di * (xi - ti) ** 2))


def _fitness_order_cases():
    import golden_cases
    return golden_cases.fitness_order_cases()


@pytest.mark.parametrize("case", _fitness_order_cases(), ids=lambda c: c[0])
def test_quadratic_fitness_hand_worked_order_and_rounding(case):
    """The summation order and the three unfused fp32 operations of a term are
    part of the fitness' definition; each golden case is worked by hand from
    dyadic numbers so that another order or another rounding gives a different
    fp32 value."""
    name, w, d, t, want = case
    got = oracle.quadratic_fitness(w, d, t)
    assert got.view(np.uint32) == want.view(np.uint32), (name, float(got), float(want))
    # the per-row entry point goes through the same function (row stride > N)
    rows = np.zeros((3, w.size + 5), np.float32)
    rows[1, :w.size] = w
    rows[2, :w.size] = t                      # w = t: every error is 0
    got_rows = oracle.quadratic_losses(rows[:, :w.size], d, t, nthreads=2)
    assert got_rows[1].view(np.uint32) == want.view(np.uint32)
    assert got_rows[2] == 0.0


def test_quadratic_losses_rows():
    rng = np.random.default_rng(9)
    x = rng.standard_normal((5, 260)).astype(np.float32)
    t = rng.standard_normal(257).astype(np.float32)
    d = rng.random(257).astype(np.float32)
    got = oracle.quadratic_losses(x[:, :257], d, t, nthreads=3)
    for i in range(5):
        assert got[i] == oracle.quadratic_fitness(x[i, :257].copy(), d, t)


# --------------------------------------------------------------------------
# Structure: sub-sampled columns, threads, step counter.
# --------------------------------------------------------------------------
def test_column_sample_follows_the_full_run():
    K, n = 4, 1003
    x, v, p = _random_swarm(K, n, 13, pad=1)
    full = oracle.RefSwarm(x[:, :n], v[:, :n], p[:, :n], m_max=0.9, m_min=0.3,
                           t_max=20, c1=0.2, c2=0.9, seed=99)
    cols = np.array([0, 1, 2, 7, 500, 501, 1001, 1002])
    part = oracle.RefSwarm(x[:, cols], v[:, cols], p[:, cols], m_max=0.9, m_min=0.3,
                           t_max=20, c1=0.2, c2=0.9, seed=99, elem_index=cols)
    rng = np.random.default_rng(1)
    for s in range(6):
        loss = rng.random(K).astype(np.float32)
        full.sync(loss, t=3 * s, lam=1.0 + s)
        part.sync(loss, t=3 * s, lam=1.0 + s)
        assert np.array_equal(full.x[:, cols], part.x)
        assert np.array_equal(full.v[:, cols], part.v)
        assert np.array_equal(full.p[:, cols], part.p)
        assert full.g == part.g and np.array_equal(full.improved, part.improved)


def test_threads_do_not_change_the_result():
    K, n = 3, 10_001
    x, v, p = _random_swarm(K, n, 17)
    a = oracle.RefSwarm(x, v, p, m_max=0.7, m_min=0.7, t_max=1, c1=1.5, c2=1.5, seed=5)
    b = oracle.RefSwarm(x, v, p, m_max=0.7, m_min=0.7, t_max=1, c1=1.5, c2=1.5, seed=5,
                        nthreads=4)
    for s in range(3):
        loss = np.array([0.3, 0.2, 0.25], np.float32) + np.float32(0.1 * s)
        a.sync(loss)
        b.sync(loss)
    assert np.array_equal(a.x, b.x) and np.array_equal(a.v, b.v) and np.array_equal(a.p, b.p)


def test_step_counter_changes_the_draws_and_first_sync_improves_everyone():
    K, n = 3, 64
    x, v, p = _random_swarm(K, n, 19)
    sw = oracle.RefSwarm(x, v, p, m_max=0.7, m_min=0.7, t_max=1, c1=1.5, c2=1.5, seed=5)
    g, imp = sw.sync([0.5, 0.4, 0.6])
    assert imp.all() and sw.s == 1                 # pBest_loss starts at +inf
    assert np.array_equal(sw.p, x)                 # pBest <- pre-update weights
    assert np.array_equal(sw.pbest_loss, np.array([0.5, 0.4, 0.6], np.float32))
    v1 = sw.v.copy()
    sw2 = oracle.RefSwarm(x, v, p, m_max=0.7, m_min=0.7, t_max=1, c1=1.5, c2=1.5, seed=5)
    sw2.s = 1
    sw2.sync([0.5, 0.4, 0.6])
    assert not np.array_equal(v1, sw2.v)


# --------------------------------------------------------------------------
# Whole iteration: PSO on the quadratic heads for its minimiser (sanity).
# --------------------------------------------------------------------------
def test_pso_on_quadratic_converges_towards_minimiser():
    K, n = 32, 6
    rng = np.random.default_rng(42)
    t = rng.standard_normal(n).astype(np.float32)
    d = (0.5 + 1.5 * rng.random(n)).astype(np.float32)
    x = rng.standard_normal((K, n)).astype(np.float32) * np.float32(3.0)
    sw = oracle.RefSwarm(x, np.zeros_like(x), x, m_max=0.7, m_min=0.7, t_max=1,
                         c1=1.5, c2=1.5, seed=5)
    best_hist = []
    first = None
    for s in range(400):
        loss = oracle.quadratic_losses(sw.x, d, t)
        first = float(loss.min()) if first is None else first
        sw.sync(loss)
        best_hist.append(float(sw.pbest_loss.min()))
    assert all(a >= b for a, b in zip(best_hist, best_hist[1:]))
    assert best_hist[-1] < 1e-6 * first
    best = sw.p[int(np.argmin(sw.pbest_loss))]
    assert np.abs(best - t).max() < 1e-2


# --------------------------------------------------------------------------
# gBest from the history of all particles (standard PSO, Section II-C step 3).
# --------------------------------------------------------------------------
def test_history_gbest_hand_worked_three_syncs():
    """K=2, N=2, m=0.5, c1=0, c2=1, r2=0.5 -> v' = 0.5 v + 0.5 (gBest - w).
    Sync 1: losses [1, 0.5] -> g=1, nothing remembered yet -> gBest=[0,4], loss 0.5.
       p0: v'=0.5([0,4]-[2,0])=[-1,2], w'=[1,2];  p1: v'=0, w'=[0,4].
    Sync 2: losses [0.75, 2] -> current best p0=[1,2] with 0.75 >= 0.5: gBest stays [0,4].
       p0: v'=0.5[-1,2]+0.5([0,4]-[1,2])=[-1,2], w'=[0,4];  p1: v'=0, w'=[0,4].
       (current-iteration gBest would give w'=[0.5,3] for both.)
    Sync 3: losses [0.25, 1] -> 0.25 < 0.5: gBest <- p0's weights before the update = [0,4]."""
    x = np.array([[2, 0], [0, 4]], np.float32)
    for history, expect2 in ((True, [[0, 4], [0, 4]]), (False, [[0.5, 3], [0.5, 3]])):
        sw = oracle.RefSwarm(x, np.zeros_like(x), x, m_max=0.5, m_min=0.5, t_max=1, c1=0.0, c2=1.0,
                             seed=0, history=history)
        kw = dict(m_max=0.5, m_min=0.5, t=0, t_max=1, c1=0.0, c2=1.0, lam=1.0, seed=0,
                  fixed_r=np.array([0.5, 0.5], np.float32), history=sw.history, want_gbest=True)
        g, _, gb = oracle.sync(sw.x, sw.v, sw.p, [1.0, 0.5], sw.pbest_loss, s=0, **kw)
        assert g == 1 and gb.tolist() == [0, 4]
        assert sw.x.tolist() == [[1, 2], [0, 4]] and sw.v.tolist() == [[-1, 2], [0, 0]]
        g, _, gb = oracle.sync(sw.x, sw.v, sw.p, [0.75, 2.0], sw.pbest_loss, s=1, **kw)
        assert g == 0
        assert gb.tolist() == ([0, 4] if history else [1, 2])
        assert sw.x.tolist() == expect2
        if history:
            assert sw.history["loss"][0] == np.float32(0.5) and sw.history["row"].tolist() == [0, 4]
            g, _, gb = oracle.sync(sw.x, sw.v, sw.p, [0.25, 1.0], sw.pbest_loss, s=2, **kw)
            assert g == 0 and sw.history["loss"][0] == np.float32(0.25)
            assert gb.tolist() == [0, 4] and sw.history["row"].tolist() == [0, 4]


def test_history_gbest_properties():
    K, n = 5, 301
    x, v, p = _random_swarm(K, n, 23)
    rng = np.random.default_rng(5)
    cur = oracle.RefSwarm(x, v, p, m_max=0.7, m_min=0.7, t_max=1, c1=1.5, c2=1.5, seed=3)
    his = oracle.RefSwarm(x, v, p, m_max=0.7, m_min=0.7, t_max=1, c1=1.5, c2=1.5, seed=3, history=True)
    # strictly decreasing minimum: the remembered best is always the current one
    for s in range(5):
        loss = (rng.random(K) + 10.0 - s).astype(np.float32)
        cur.sync(loss)
        his.sync(loss)
        assert np.array_equal(cur.x, his.x) and np.array_equal(cur.v, his.v)
        assert his.history["loss"][0] == loss.min()
    # from now on nothing beats the remembered loss: the row must not move
    kept = his.history["row"].copy()
    kept_loss = his.history["loss"][0]
    for s in range(4):
        loss = (rng.random(K) + 20.0).astype(np.float32)
        loss[s % K] = kept_loss                       # equal is not better (strict <)
        before = his.x.copy()
        his.sync(loss, want_gbest=True)
        assert np.array_equal(his.history["row"], kept) and his.history["loss"][0] == kept_loss
        assert np.array_equal(his.gbest, kept)
        assert not np.array_equal(his.gbest, before[his.g])
    # NaN never enters the history
    his.sync(np.full(K, np.nan, np.float32))
    assert np.array_equal(his.history["row"], kept)
    # nothing remembered yet: the first sync takes the current best whatever its loss
    fresh = oracle.RefSwarm(x, v, p, m_max=0.7, m_min=0.7, t_max=1, c1=1.5, c2=1.5, seed=3, history=True)
    fresh.sync(np.full(K, np.inf, np.float32), want_gbest=True)
    assert fresh.g == 0 and np.array_equal(fresh.gbest, x[0]) and np.array_equal(fresh.history["row"], x[0])
    assert fresh.history["valid"][0] == 1 and np.isinf(fresh.history["loss"][0])
    before = fresh.x.copy()
    fresh.sync(np.array([5, 4, 3, 4, 5], np.float32), want_gbest=True)
    assert np.array_equal(fresh.gbest, before[2]) and fresh.history["loss"][0] == 3.0


# --------------------------------------------------------------------------
# Synchronous SGD update (Section II-B).
# --------------------------------------------------------------------------
def test_ssgd_closed_forms():
    rng = np.random.default_rng(8)
    # K = 1: w + alpha * g, two roundings
    w = rng.standard_normal((1, 500)).astype(np.float32)
    g = rng.standard_normal((1, 500)).astype(np.float32)
    w0 = w.copy()
    oracle.ssgd(w, g, 0.25)
    assert np.array_equal(w, w0 + np.float32(0.25) * g)
    # small integers and a power-of-two worker count: exact
    wi = rng.integers(-50, 50, size=(4, 333)).astype(np.float32)
    wi[1:] = wi[0]
    gi = rng.integers(-20, 20, size=(4, 333)).astype(np.float32)
    expect = wi[0].astype(np.float64) + 0.5 / 4 * gi.astype(np.float64).sum(axis=0)
    oracle.ssgd(wi, gi, 0.5)
    assert all(np.array_equal(wi[k].astype(np.float64), expect) for k in range(4))
    # general case against double arithmetic; sign convention is "+ alpha" as the paper writes it
    K, n = 7, 4096
    wg = np.tile(rng.standard_normal(n).astype(np.float32), (K, 1))
    gg = rng.standard_normal((K, n)).astype(np.float32)
    ref = wg[0].astype(np.float64) + (-0.01 / K) * gg.astype(np.float64).sum(axis=0)
    mag = np.abs(wg[0]).astype(np.float64) + 0.01 / K * np.abs(gg).astype(np.float64).sum(axis=0)
    oracle.ssgd(wg, gg, -0.01, nthreads=3)
    assert np.all(np.abs(wg[0] - ref) <= (K + 3) * 2.0 ** -24 * mag)
    assert all(np.array_equal(wg[0], wg[k]) for k in range(K))


def test_ssgd_equals_averaging_of_one_local_step():
    """Section II-B: with step = 1, averaging the workers' weights after one
    local update w + alpha g_k is the SSGD update w + (alpha / n) sum g_k."""
    rng = np.random.default_rng(12)
    K, n, alpha = 8, 2000, np.float32(-0.125)
    w = np.tile(rng.standard_normal(n).astype(np.float32), (K, 1))
    g = rng.standard_normal((K, n)).astype(np.float32)
    local = (w + alpha * g).astype(np.float32)
    oracle.average(local)
    a = w.copy()
    oracle.ssgd(a, g, alpha)
    scale = np.abs(w[0]) + np.abs(alpha) * np.abs(g).max(axis=0)
    assert np.all(np.abs(local[0] - a[0]) <= 16 * 2.0 ** -24 * scale)


def test_ssgd_respects_strides():
    rng = np.random.default_rng(4)
    wbuf = rng.standard_normal((3, 16)).astype(np.float32)
    gbuf = rng.standard_normal((3, 24)).astype(np.float32)
    keep = wbuf.copy()
    oracle.ssgd(wbuf[:, :13], gbuf[:, :13], 0.5)
    assert np.array_equal(wbuf[:, 13:], keep[:, 13:])
    exp = keep[0, :13] + (np.float32(0.5) / np.float32(3)) * ((gbuf[0, :13] + gbuf[1, :13]) + gbuf[2, :13])
    assert np.array_equal(wbuf[1, :13], exp)


def test_update_is_exactly_homogeneous_under_power_of_two_scaling():
    """Eq. 6 / Eq. 7 are linear in (w, v, pBest): scaling the whole state by
    2^k scales every intermediate exactly, so the result scales bit for bit."""
    K, n = 4, 515
    x, v, p = _random_swarm(K, n, 29)
    loss = np.array([0.4, 0.9, 0.3, 0.8], np.float32)
    outs = []
    for k in (0, 7, -9):
        f = np.float32(2.0 ** k)
        sw = oracle.RefSwarm(x * f, v * f, p * f, m_max=0.9, m_min=0.3, t_max=10, c1=0.2, c2=0.9, seed=12)
        sw.sync(loss, t=4, lam=3.0)
        sw.sync(loss[::-1].copy(), t=5, lam=3.0)
        outs.append((sw.x / f, sw.v / f, sw.p / f))
    for a in outs[1:]:
        for got, want in zip(a, outs[0]):
            assert np.array_equal(got, want)

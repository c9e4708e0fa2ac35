"""Pins for the CPU oracle: each stage is checked against something other than itself -- big-integer
Python arithmetic, dense brute force, numpy library routines, exactly-representable inputs, and the
invariants the paper states (linearity of the sketch, exact recovery without collisions, "true top-k"
when every coordinate is a candidate, error feedback).  No GPU, no CUDA library."""
import math
from fractions import Fraction

import numpy as np
import pytest

from oracle import Oracle, derive_params, select

P = 2**31 - 1
M64 = 2**64 - 1


# ------------------------------------------------------------------------------------------------
# independent helpers (Python big integers / numpy only; nothing from the oracle)
# ------------------------------------------------------------------------------------------------
def py_params(seed, r):
    """Seed -> hash parameters with Python's unbounded integers."""
    s = seed & M64
    out = []

    def nxt():
        nonlocal s
        s = (s + 0x9E3779B97F4A7C15) & M64
        z = s
        z = ((z ^ (z >> 30)) * 0xBF58476D1CE4E5B9) & M64
        z = ((z ^ (z >> 27)) * 0x94D049BB133111EB) & M64
        return z ^ (z >> 31)

    for _ in range(r):
        a = 1 + nxt() % (P - 1)
        b = nxt() % P
        a2 = 1 + nxt() % (P - 1)
        b2 = nxt() % P
        out.append((a, b, a2, b2))
    return out


def py_hash(params, c, i):
    """(bucket, sign) per row for coordinate i, Python big integers."""
    hs, ss = [], []
    for a, b, a2, b2 in params:
        hs.append(((a * i + b) % P) % c)
        ss.append(2 * (((a2 * i + b2) % P) & 1) - 1)
    return hs, ss


def dense_matrix(params, c, d):
    """The r*c x d matrix A with S(x) = A x (Appendix B: sketching is a linear map)."""
    r = len(params)
    A = np.zeros((r * c, d))
    for i in range(d):
        hs, ss = py_hash(params, c, i)
        for j in range(r):
            A[j * c + hs[j], i] = ss[j]
    return A


def np_topk_set(x32, k):
    """Textbook top-k by magnitude with index tie-break, via numpy's lexsort."""
    key = np.abs(x32).view(np.uint32).astype(np.int64)
    order = np.lexsort((np.arange(x32.size), -key))
    return order[:k]


def state(W, d, ld=None):
    ld = ld or d
    return np.zeros((W, ld), np.float32), np.zeros((W, ld), np.float32)


# ------------------------------------------------------------------------------------------------
# hash family
# ------------------------------------------------------------------------------------------------
@pytest.mark.parametrize("seed", [0, 1, 0x5EED, 2**64 - 1, 123456789012345])
def test_params_match_big_integer_restatement(seed):
    got = derive_params(seed, 15)
    want = np.array(py_params(seed, 15), dtype=np.uint64)
    assert (got.astype(np.uint64) == want).all()
    assert (got[:, 0] >= 1).all() and (got[:, 0] < P).all() and (got[:, 2] >= 1).all()
    assert (got[:, 1] < P).all() and (got[:, 3] < P).all()
    # the first r rows do not depend on how many rows are asked for
    assert (derive_params(seed, 5) == got[:5]).all()


def test_generator_first_outputs_for_seed_zero():
    # The draw function is a 64-bit mix of a Weyl sequence; its first output for seed 0, computed here
    # with Python integers, fixes a_0 = 1 + z mod (p-1).
    s = 0x9E3779B97F4A7C15
    z = s
    z = ((z ^ (z >> 30)) * 0xBF58476D1CE4E5B9) & M64
    z = ((z ^ (z >> 27)) * 0x94D049BB133111EB) & M64
    z ^= z >> 31
    assert derive_params(0, 1)[0, 0] == 1 + z % (P - 1)


def test_hash_identity_parameters_closed_form():
    d, c = 5000, 40
    o = Oracle(d, 3, c, 1, 1, 0)
    o.set_params([[1, 0, 1, 0]] * 3)
    idx = np.arange(d)
    h, s = o.hashes(idx)
    assert (h == (idx % c)[None, :]).all()
    assert (s == (2 * (idx & 1) - 1)[None, :]).all()
    # b shifts the bucket, b' = 1 flips the parity
    o.set_params([[1, 7, 1, 1]] * 3)
    h, s = o.hashes(idx)
    assert (h == ((idx + 7) % c)[None, :]).all()
    assert (s == (2 * ((idx + 1) & 1) - 1)[None, :]).all()


@pytest.mark.parametrize("c", [1, 7, 40, 16384, 180000, 2**31 - 2])
def test_hash_matches_big_integers(c):
    r, seed = 7, 99
    o = Oracle(2**31 - 2, r, c, 1, 1, seed)
    params = py_params(seed, r)
    rng = np.random.default_rng(5)
    idx = np.concatenate([[0, 1, 2, P - 2, P - 3, 2**30, 2**30 + 1], rng.integers(0, P - 1, 300)])
    h, s = o.hashes(idx)
    for t, i in enumerate(idx.tolist()):
        hs, ss = py_hash(params, c, i)
        assert h[:, t].tolist() == hs and s[:, t].tolist() == ss
    assert h.min() >= 0 and h.max() < c and set(np.unique(s).tolist()) <= {-1, 1}


def test_hash_extreme_parameters_no_overflow():
    # a = a' = p-1, b = b' = p-1, i = p-2: the largest products the family can form
    o = Oracle(P - 1, 1, 1000, 1, 1, 0)
    o.set_params([[P - 1, P - 1, P - 1, P - 1]])
    i = P - 2
    h, s = o.hashes([i])
    hs, ss = py_hash([(P - 1, P - 1, P - 1, P - 1)], 1000, i)
    assert h[0, 0] == hs[0] and s[0, 0] == ss[0]


def test_invalid_shapes_rejected():
    for bad in [dict(d=0), dict(r=0), dict(r=4), dict(r=17), dict(c=0), dict(k=0), dict(W=0), dict(d=P),
                dict(c=P)]:
        kw = dict(d=10, r=3, c=5, k=2, W=1, seed=0)
        kw.update(bad)
        with pytest.raises(ValueError):
            Oracle(**kw)
    with pytest.raises(ValueError):
        Oracle(10, 3, 5, 11, 1, 0)  # k > d


def test_hash_statistics():
    """Pairwise-independent hashing (Appendix B): bucket loads near d/c, signs balanced, and the
    single-row estimate s*S[h] has mean squared error close to (||x||^2 - x_i^2)/c."""
    d, c = 20000, 64
    rng = np.random.default_rng(0)
    x = rng.standard_normal(d)
    errs, loads_ok, bal = [], [], []
    for seed in range(40):
        o = Oracle(d, 1, c, 1, 1, seed)
        T = o.sketch(x)
        h, s = o.hashes(np.arange(d))
        est = s[0] * T[0, h[0]]
        errs.append(np.mean((est - x) ** 2 / ((x @ x - x**2) / c)))
        loads = np.bincount(h[0], minlength=c)
        loads_ok.append(abs(loads.mean() - d / c) < 1e-9 and loads.max() < 2 * d / c)
        bal.append(abs((s[0] == 1).mean() - 0.5))
    assert abs(np.mean(errs) - 1.0) < 0.1
    assert all(loads_ok) and max(bal) < 0.03


# ------------------------------------------------------------------------------------------------
# update / insert, linearity, merge
# ------------------------------------------------------------------------------------------------
def test_sketch_of_unit_vector():
    d, r, c, seed = 300, 5, 11, 3
    o = Oracle(d, r, c, 1, 1, seed)
    params = py_params(seed, r)
    for i in [0, 1, 17, 299]:
        e = np.zeros(d, np.float32)
        e[i] = 1.0
        T, M = o.sketch(e, with_mass=True)
        hs, ss = py_hash(params, c, i)
        want = np.zeros((r, c))
        for j in range(r):
            want[j, hs[j]] = ss[j]
        assert (T == want).all() and (M == np.abs(want)).all()
        assert np.count_nonzero(T) == r


@pytest.mark.parametrize("r,c,d", [(1, 1, 9), (3, 7, 64), (5, 13, 200), (7, 40, 785)])
def test_sketch_equals_dense_matrix_product(r, c, d):
    seed = 11 * r + c
    o = Oracle(d, r, c, 1, 1, seed)
    A = dense_matrix(py_params(seed, r), c, d)
    rng = np.random.default_rng(1)
    x = rng.integers(-1000, 1000, d).astype(np.float64)  # integers: every sum is exact
    T, M = o.sketch(x, with_mass=True)
    assert (T.reshape(-1) == A @ x).all()
    assert (M.reshape(-1) == np.abs(A) @ np.abs(x)).all()
    x32 = x.astype(np.float32)
    assert (o.sketch(x32) == T).all()
    # real-valued input: equal to the matrix product up to fp64 rounding
    y = rng.standard_normal(d)
    assert np.allclose(o.sketch(y).reshape(-1), A @ y, rtol=0, atol=1e-12)


def test_linearity_and_merge():
    d, r, c, W = 4000, 5, 97, 6
    o = Oracle(d, r, c, 1, W, 21)
    rng = np.random.default_rng(2)
    x = rng.integers(-2**20, 2**20, d).astype(np.float32)
    y = rng.integers(-2**20, 2**20, d).astype(np.float32)
    assert (o.sketch(x + y) == o.sketch(x) + o.sketch(y)).all()  # S(x+y) = S(x) + S(y)
    assert (o.sketch((3 * x).astype(np.float32)) == 3 * o.sketch(x)).all()
    v = rng.integers(-2**18, 2**18, (W, d)).astype(np.float32)
    T, M, Tw = o.sketch_workers(v, per_worker=True)
    for w in range(W):
        assert (Tw[w] == o.sketch(v[w])).all()
    assert (T == Tw.sum(0)).all()
    assert (T == o.sketch(v.astype(np.float64).sum(0))).all()  # sum of sketches = sketch of the sum
    assert (M == sum(o.sketch(v[w], with_mass=True)[1] for w in range(W))).all()
    # leading dimension larger than d: padding is ignored
    vp = np.zeros((W, d + 3), np.float32)
    vp[:, :d] = v
    vp[:, d:] = 1e30
    assert (o.sketch_workers(vp)[0] == T).all()


# ------------------------------------------------------------------------------------------------
# estimate
# ------------------------------------------------------------------------------------------------
def test_estimate_is_median_of_row_estimates():
    d, r, c, seed = 3000, 7, 50, 8
    o = Oracle(d, r, c, 1, 1, seed)
    params = py_params(seed, r)
    rng = np.random.default_rng(3)
    Tf = rng.standard_normal((r, c)).astype(np.float32)
    est = o.estimate(Tf)
    for i in rng.integers(0, d, 200).tolist() + [0, d - 1]:
        hs, ss = py_hash(params, c, i)
        rows = np.array([ss[j] * Tf[j, hs[j]] for j in range(r)], np.float32)
        assert est[i] == np.float32(np.median(rows))  # r odd: numpy's median is the middle element


def test_estimate_r1_is_signed_bucket():
    d, c = 500, 16
    o = Oracle(d, 1, c, 1, 1, 4)
    Tf = np.arange(1, c + 1, dtype=np.float32).reshape(1, c)
    h, s = o.hashes(np.arange(d))
    assert (o.estimate(Tf) == s[0] * Tf[0, h[0]]).all()


def test_exact_recovery_without_collisions():
    """A coordinate that shares its bucket with no other non-zero in at least (r+1)/2 rows is
    estimated exactly; a sparse vector with no collisions at all is recovered exactly."""
    d, r, c = 600, 5, 64
    rng = np.random.default_rng(4)
    found_clean = found_partial = False
    for seed in range(200):
        params = py_params(seed, r)
        supp = rng.choice(d, 6, replace=False)
        buckets = np.array([py_hash(params, c, int(i))[0] for i in supp])  # [6][r]
        x = np.zeros(d, np.float32)
        x[supp] = rng.integers(1, 100, 6) * rng.choice([-1, 1], 6)
        o = Oracle(d, r, c, 1, 1, seed)
        est = o.estimate(o.sketch(x).astype(np.float32))
        clean_rows = np.array([[np.sum(buckets[:, j] == buckets[t, j]) == 1 for j in range(r)]
                               for t in range(6)])
        for t, i in enumerate(supp):
            if clean_rows[t].sum() >= (r + 1) // 2:
                assert est[i] == x[i]
                found_partial |= clean_rows[t].sum() < r
        if clean_rows.all():
            found_clean = True
            assert (est[supp] == x[supp]).all()
            # every other coordinate that meets the support in at most (r-1)/2 rows reads zero
            for i in range(d):
                if i in supp:
                    continue
                hs = py_hash(params, c, i)[0]
                hits = sum(hs[j] in buckets[:, j] for j in range(r))
                if hits <= (r - 1) // 2:
                    assert est[i] == 0.0
    assert found_clean and found_partial


def test_identity_hash_wide_table_recovers_everything():
    # r = 1, a = 1, b = 0, c >= d: the table is a signed copy of x, so the estimate is x itself
    d = 777
    o = Oracle(d, 1, 1000, 1, 1, 0)
    o.set_params([[1, 0, 12345, 678]])
    x = np.random.default_rng(5).standard_normal(d).astype(np.float32)
    T = o.sketch(x)
    assert (np.abs(T[0, :d]) == np.abs(x)).all() and (T[0, d:] == 0).all()
    assert (o.estimate(T.astype(np.float32)) == x).all()


# ------------------------------------------------------------------------------------------------
# selection
# ------------------------------------------------------------------------------------------------
def test_select_against_lexsort():
    rng = np.random.default_rng(6)
    for n, m in [(1, 1), (10, 0), (10, 10), (1000, 17), (5000, 2500)]:
        val = rng.integers(-20, 20, n).astype(np.float32)  # many ties, both signs, zeros
        val[rng.integers(0, n, max(1, n // 10))] *= -0.0
        got = select(val, m)
        assert (got == np_topk_set(val, m)).all()
        ids = rng.permutation(3 * n)[:n].astype(np.int32)
        key = np.abs(val).view(np.uint32).astype(np.int64)
        want = np.lexsort((ids, -key))[:m]
        assert (select(val, m, ids) == want).all()


def test_select_orders_by_bit_pattern_of_magnitude():
    val = np.array([1e-45, -1e-45, 0.0, -0.0, 3.0, -3.0000002, np.float32(3.0)], np.float32)
    assert select(val, 7).tolist() == [5, 4, 6, 0, 1, 2, 3]


# ------------------------------------------------------------------------------------------------
# momentum / error accumulation, second round, zeroing
# ------------------------------------------------------------------------------------------------
def nearest_f32(exact: Fraction, got: np.float32) -> bool:
    g = Fraction(float(got))
    lo = Fraction(float(np.nextafter(got, np.float32(-np.inf))))
    hi = Fraction(float(np.nextafter(got, np.float32(np.inf))))
    return abs(g - exact) <= abs(lo - exact) and abs(g - exact) <= abs(hi - exact)


def test_accumulate_single_rounding():
    W, d = 2, 400
    o = Oracle(d, 1, 4, 1, W, 0)
    rng = np.random.default_rng(7)
    g = rng.standard_normal((W, d)).astype(np.float32)
    u0 = rng.standard_normal((W, d)).astype(np.float32)
    v0 = rng.standard_normal((W, d)).astype(np.float32)
    rho = np.float32(0.9)
    u, v = u0.copy(), v0.copy()
    o.accumulate(g, rho, u, v)
    for w in range(W):
        for i in range(d):
            exact = Fraction(float(rho)) * Fraction(float(u0[w, i])) + Fraction(float(g[w, i]))
            assert nearest_f32(exact, u[w, i])                       # one rounding: a true fma
    assert (v == (v0 + u)).all()                                     # v uses the NEW u, one rounding
    # from zero state the first step copies g
    u, v = state(W, d)
    o.accumulate(g, rho, u, v)
    assert (u == g).all() and (v == g).all()


def test_accumulate_respects_leading_dimensions():
    W, d = 3, 10
    o = Oracle(d, 1, 4, 1, W, 0)
    g = np.ones((W, d + 2), np.float32)
    u, v = state(W, d, d + 5)
    u[:, d:] = 7
    v[:, d:] = 9
    o.accumulate(g, 0.5, u, v)
    assert (u[:, :d] == 1).all() and (u[:, d:] == 7).all() and (v[:, d:] == 9).all()


def test_second_round_and_zero():
    W, d = 5, 50
    o = Oracle(d, 1, 4, 3, W, 0)
    rng = np.random.default_rng(8)
    v = rng.standard_normal((W, d)).astype(np.float32)
    u = rng.standard_normal((W, d)).astype(np.float32)
    cand = np.array([3, 49, 0, 17], np.int32)
    xs = o.second_round(v, cand)
    assert np.allclose(xs, v.astype(np.float64)[:, cand].sum(0), rtol=0, atol=1e-15)
    assert xs[0] == math.fsum(float(t) for t in v[:, 3]) or abs(xs[0] - math.fsum(map(float, v[:, 3]))) < 1e-15
    u1, v1 = u.copy(), v.copy()
    o.zero(u1, v1, cand[:2])
    mask = np.zeros(d, bool)
    mask[cand[:2]] = True
    assert (u1[:, mask] == 0).all() and (v1[:, mask] == 0).all()
    assert (u1[:, mask].view(np.uint32) == 0).all()  # +0.0f bit pattern
    assert (u1[:, ~mask] == u[:, ~mask]).all() and (v1[:, ~mask] == v[:, ~mask]).all()


# ------------------------------------------------------------------------------------------------
# whole step
# ------------------------------------------------------------------------------------------------
def int_grads(rng, W, d, hi=2**12):
    return rng.integers(-hi, hi, (W, d)).astype(np.float32)


@pytest.mark.parametrize("r,c", [(5, 32), (1, 3), (7, 40)])
def test_all_coordinates_as_candidates_is_true_topk(r, c):
    """ncand = d: whatever the sketch holds, the step returns the top-k of the summed vector (the
    paper's "true top-k" baseline)."""
    W, d, k = 4, 3000, 37
    o = Oracle(d, r, c, k, W, 5)
    rng = np.random.default_rng(9)
    g = rng.standard_normal((W, d)).astype(np.float32)
    u, v = state(W, d)
    out = o.step(g, 0.9, u, v, ncand=d)
    x = g.astype(np.float64).sum(0)           # first step from zero state: v = g
    want = np_topk_set(x.astype(np.float32), k)
    assert (out["out_idx"] == want).all()
    assert (out["out_val"] == x.astype(np.float32)[want]).all()
    # tau-contraction of true top-k: ||x - comp(x)||^2 <= (1 - k/d) ||x||^2
    rest = x.copy()
    rest[want] = 0
    assert rest @ rest <= (1 - k / d) * (x @ x)


def test_step_stages_compose():
    """The step's intermediates are exactly the stage functions applied in the paper's order."""
    W, d, r, c, k, ncand = 3, 5000, 5, 256, 20, 60
    o = Oracle(d, r, c, k, W, 77)
    rng = np.random.default_rng(10)
    g = rng.standard_normal((W, d + 2)).astype(np.float32)
    u, v = state(W, d, d + 1)
    u[:] = rng.standard_normal(u.shape)
    v[:] = rng.standard_normal(v.shape)
    u2, v2 = u.copy(), v.copy()
    out = o.step(g, 0.9, u, v, ncand, full=True)
    o.accumulate(g, 0.9, u2, v2)
    T, M = o.sketch_workers(v2)
    assert (T == out["T"]).all() and (M == out["M"]).all()
    est = o.estimate(T.astype(np.float32))
    assert (est == out["est"]).all()
    cand = np_topk_set(est, ncand).astype(np.int32)
    assert (cand == out["cand"]).all()
    xs = v2.astype(np.float64)[:, cand].sum(0)
    assert np.allclose(xs, out["xs"], rtol=0, atol=1e-14)
    best = np_topk_set(out["xs"].astype(np.float32), k)  # candidates are distinct, position order ...
    key = np.abs(out["xs"].astype(np.float32)).view(np.uint32).astype(np.int64)
    best = np.lexsort((cand, -key))[:k]                  # ... but ties break on the coordinate index
    assert (out["out_idx"] == cand[best]).all()
    assert (out["out_val"] == out["xs"].astype(np.float32)[best]).all()
    o.zero(u2, v2, out["out_idx"])
    assert (u == u2).all() and (v == v2).all()
    assert len(set(out["out_idx"].tolist())) == k and set(out["out_idx"].tolist()) <= set(cand.tolist())


def test_error_feedback_invariant():
    """Over T steps: applied updates + what is left in v = everything that was ever accumulated,
    i.e. sum_t gtilde_t[i] + sum_w v_w[i] = sum_t sum_w u_w^(t)[i].  Integer gradients and rho = 1/2
    make every operation exact, so the identity must hold to the last bit."""
    W, d, r, c, k, ncand, T = 4, 2000, 5, 128, 25, 75, 6
    o = Oracle(d, r, c, k, W, 31)
    rng = np.random.default_rng(11)
    u, v = state(W, d)
    applied = np.zeros(d)
    accumulated = np.zeros(d)
    for t in range(T):
        g = int_grads(rng, W, d)
        # what the step will add to v: the new u, computed independently (exact in fp64)
        u_new = 0.5 * u.astype(np.float64) + g
        accumulated += u_new.sum(0)
        out = o.step(g, 0.5, u, v, ncand, full=True)
        np.add.at(applied, out["out_idx"], out["out_val"].astype(np.float64))
        # chosen coordinates, and only those, were reset in both u and v
        chosen = np.zeros(d, bool)
        chosen[out["out_idx"]] = True
        assert (u[:, chosen] == 0).all() and (v[:, chosen] == 0).all()
        assert (u[:, ~chosen] == u_new[:, ~chosen]).all()
        # momentum masking removes u at the chosen coordinates: account for it in what follows
        assert (applied + v.astype(np.float64).sum(0) == accumulated).all()
    assert applied.any()


def test_identical_workers_choose_like_one_worker():
    d, r, c, k, ncand = 3000, 5, 200, 15, 40
    rng = np.random.default_rng(12)
    g1 = int_grads(rng, 1, d)
    o1 = Oracle(d, r, c, k, 1, 9)
    u, v = state(1, d)
    a = o1.step(g1, 0.9, u, v, ncand)
    W = 4
    oW = Oracle(d, r, c, k, W, 9)
    u, v = state(W, d)
    b = oW.step(np.repeat(g1, W, 0), 0.9, u, v, ncand)
    assert (a["out_idx"] == b["out_idx"]).all()
    assert (W * a["out_val"] == b["out_val"]).all()      # the update is the SUM over workers


def test_selection_invariant_under_power_of_two_scaling():
    W, d, r, c, k, ncand = 3, 4000, 5, 128, 30, 90
    rng = np.random.default_rng(13)
    g = rng.standard_normal((W, d)).astype(np.float32)
    o = Oracle(d, r, c, k, W, 2)
    u, v = state(W, d)
    a = o.step(g, 0.9, u, v, ncand, full=True)
    u, v = state(W, d)
    b = o.step(2 * g, 0.9, u, v, ncand, full=True)
    assert (a["cand"] == b["cand"]).all() and (a["out_idx"] == b["out_idx"]).all()
    assert (2 * a["out_val"] == b["out_val"]).all() and (2 * a["est"] == b["est"]).all()


def test_planted_heavy_coordinates_are_recovered():
    """Heavy coordinates far above the sketch noise floor ||x||_2 / sqrt(c) all become candidates and
    all survive to the final k."""
    W, d, r, c, k = 4, 50000, 5, 4096, 50
    rng = np.random.default_rng(14)
    g = rng.standard_normal((W, d)).astype(np.float32)
    heavy = rng.choice(d, k, replace=False)
    g[:, heavy] = (200.0 * rng.choice([-1, 1], k)).astype(np.float32)[None, :]
    o = Oracle(d, r, c, k, W, 6)
    u, v = state(W, d)
    out = o.step(g, 0.9, u, v, ncand=2 * k, full=True)
    assert set(heavy.tolist()) <= set(out["cand"].tolist())
    assert set(heavy.tolist()) == set(out["out_idx"].tolist())
    assert np.allclose(np.abs(out["out_val"]), 800.0)


def test_k_equals_ncand_equals_d_and_all_zero_input():
    W, d = 2, 33
    o = Oracle(d, 3, 4, d, W, 0)
    g = np.zeros((W, d), np.float32)
    u, v = state(W, d)
    out = o.step(g, 0.9, u, v, ncand=d)
    assert out["out_idx"].tolist() == list(range(d))     # all ties: index order
    assert (out["out_val"] == 0).all()
    with pytest.raises(ValueError):
        o.step(g, 0.9, u, v, ncand=d + 1)
    o2 = Oracle(d, 3, 4, 5, W, 0)
    with pytest.raises(ValueError):
        o2.step(g, 0.9, u, v, ncand=4)                   # ncand < k

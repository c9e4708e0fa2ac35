"""Pins for the oracle's HEAVYMIX (Algorithm 1): the squared-norm estimate against closed forms and
its unbiasedness, the heavy set against a numpy restatement, the random fill against Python big
integers, a library sort and a uniformity check, and the output's structure.  CPU only."""
import numpy as np
import pytest

from oracle import Oracle, fill_priority

M64 = 2**64 - 1


def py_priority(seed, i):
    z = (seed + (i + 1) * 0x9E3779B97F4A7C15) & M64
    z = ((z ^ (z >> 30)) * 0xBF58476D1CE4E5B9) & M64
    z = ((z ^ (z >> 27)) * 0x94D049BB133111EB) & M64
    z ^= z >> 31
    return z >> 34


def test_fill_priority_matches_big_integers():
    idx = np.array([0, 1, 2, 12345, 2**31 - 3, 999_999_937], np.int64)
    for seed in (0, 1, 0xDEADBEEF, 2**64 - 1):
        got = fill_priority(seed, idx)
        assert got.tolist() == [py_priority(seed, int(i)) for i in idx]


def test_l2_estimate_closed_forms():
    d, c = 500, 512
    o = Oracle(d, 1, c, 1, 1, 0)
    o.set_params([[1, 0, 7, 3]])                      # identity buckets, c >= d: no collisions
    x = np.random.default_rng(0).integers(-50, 50, d).astype(np.float32)
    T = o.sketch(x).astype(np.float32)
    assert o.l2_estimate(T) == float((x.astype(np.float64) ** 2).sum())      # integers: exact
    # median over rows: rows scaled by 1, 2, 3 -> the middle row's sum of squares
    o3 = Oracle(10, 3, 4, 1, 1, 0)
    T3 = np.array([[1, 1, 1, 1], [3, 3, 3, 3], [2, 2, 2, 2]], np.float32)
    assert o3.l2_estimate(T3) == 16.0


def test_l2_estimate_is_unbiased_and_within_a_factor():
    """Each row's sum of squared counters estimates ||x||^2 without bias (pairwise-independent signs,
    Appendix B); the median over 5 rows stays within (1 +- 0.5)||x||^2 (Algorithm 1 line 1)."""
    d, c = 20000, 256
    x = np.random.default_rng(1).standard_normal(d).astype(np.float32)
    true = float((x.astype(np.float64) ** 2).sum())
    single, med = [], []
    for seed in range(60):
        o = Oracle(d, 5, c, 1, 1, seed)
        T = o.sketch(x).astype(np.float32)
        single.append((T.astype(np.float64)[0] ** 2).sum())
        med.append(o.l2_estimate(T))
    assert abs(np.mean(single) / true - 1) < 0.05
    assert all(0.5 * true <= m <= 1.5 * true for m in med)


def heavymix_case(d, r, c, k, W, seed, heavy_n, heavy_mag, rng):
    o = Oracle(d, r, c, k, W, seed)
    v = rng.standard_normal((W, d)).astype(np.float32)
    hi = rng.choice(d, heavy_n, replace=False)
    v[:, hi] = heavy_mag * rng.choice([-1, 1], heavy_n).astype(np.float32)[None, :]
    T, _ = o.sketch_workers(v)
    return o, v, T.astype(np.float32), hi


@pytest.mark.parametrize("heavy_n,k", [(12, 40), (0, 25), (40, 60)])
def test_heavymix_structure(heavy_n, k):
    rng = np.random.default_rng(2)
    d, r, c, W, seed = 6000, 5, 512, 3, 5
    o, v, Tf, hi = heavymix_case(d, r, c, k, W, seed, heavy_n, 60.0, rng)
    out = o.heavymix(Tf, v, fill_seed=99)
    idx = out["out_idx"]
    # restatement with numpy
    est = o.estimate(Tf).astype(np.float64)
    l2 = o.l2_estimate(Tf)
    assert out["l2"] == l2
    H = np.flatnonzero(est * est >= l2 / k)
    assert out["nheavy"] == H.size and H.size <= k
    assert set(hi.tolist()) <= set(H.tolist())             # planted coordinates are heavy
    assert len(set(idx.tolist())) == k and (np.diff(idx) > 0).all()
    assert set(H.tolist()) <= set(idx.tolist())
    fill = np.setdiff1d(idx, H)
    NH = np.setdiff1d(np.arange(d), H)
    assert fill.size == k - H.size and set(fill.tolist()) <= set(NH.tolist())
    prio = np.array([py_priority(99, int(i)) for i in NH], np.int64)
    want_fill = NH[np.lexsort((NH, -prio))[: k - H.size]]
    assert set(fill.tolist()) == set(want_fill.tolist())
    # line 5: exact values, summed over workers
    assert (out["out_val"] == v.astype(np.float64)[:, idx].sum(0).astype(np.float32)).all()
    # another seed gives another fill, the same heavy part
    idx2 = o.heavymix(Tf, v, fill_seed=100)["out_idx"]
    assert set(H.tolist()) <= set(idx2.tolist())
    if k - H.size > 3:
        assert set(idx2.tolist()) != set(idx.tolist())


def test_heavymix_more_heavy_than_k_keeps_the_largest():
    """|H| > k cannot happen with exact estimates (sum over H of x_i^2 >= |H| ||x||^2 / k), only through
    collisions: one row, two buckets, counters (10, 1).  Every coordinate hashed to bucket 0 reads 10 and is
    heavy; the k largest |estimates| are then ties, which go to the smallest indices."""
    d, k = 200, 5
    o = Oracle(d, 1, 2, k, 1, 3)
    Tf = np.array([[10.0, 1.0]], np.float32)
    v = np.arange(d, dtype=np.float32).reshape(1, d)
    out = o.heavymix(Tf, v, fill_seed=0)
    h, _ = o.hashes(np.arange(d))
    in0 = np.flatnonzero(h[0] == 0)
    assert out["l2"] == 101.0 and out["nheavy"] == in0.size > k
    assert out["out_idx"].tolist() == in0[:k].tolist()
    assert out["out_val"].tolist() == in0[:k].astype(np.float32).tolist()


def test_heavymix_last_mantissa_bit_decides_when_more_than_k_are_heavy():
    """|H| > k with heavy estimates that differ only in the last mantissa bit.  One row, four buckets holding
    +-1.0 and +-(the next fp32 above 1.0): every coordinate reads one of them, l2/k is about 4/k < 1, so all d
    coordinates are heavy.  The k kept must be the k largest under the FULL fp32 magnitude, ties to the smaller
    index (numpy.lexsort restatement) -- a key that drops the last mantissa bit would see d-way ties and return
    the first k indices instead."""
    one = np.float32(1.0)
    up = np.nextafter(one, np.float32(2.0))
    d = 200
    Tf = np.array([[one, up, -one, -up]], np.float32)
    v = (10.0 + np.arange(d, dtype=np.float32)).reshape(1, d)
    for k in (20, 150):                                   # fewer than, and more than, the coordinates reading `up`
        o = Oracle(d, 1, 4, k, 1, 21)
        h, _ = o.hashes(np.arange(d))
        est = o.estimate(Tf)
        is_up = np.isin(h[0], (1, 3))
        assert (np.abs(est) == np.where(is_up, up, one)).all() and 20 < is_up.sum() < 150
        out = o.heavymix(Tf, v, fill_seed=5)
        assert out["nheavy"] == d
        bits = np.abs(est).view(np.uint32).astype(np.int64)
        order = np.lexsort((np.arange(d), -bits))         # magnitude bits descending, then index ascending
        want = np.sort(order[:k])
        assert out["out_idx"].tolist() == want.tolist()
        assert out["out_idx"].tolist() != list(range(k))  # what a coarser key would give
        if k == 20:
            assert is_up[out["out_idx"]].all()
        else:
            assert is_up[out["out_idx"]].sum() == is_up.sum()
        assert (out["out_val"] == v[0, out["out_idx"]]).all()


def test_heavymix_more_heavy_than_k_never_takes_from_nh():
    """|H| > k: nothing from NH may appear, whatever its fill priority.  One row, two buckets (10, 1): coordinates
    in bucket 0 read 10 (heavy), the others read 1 (not heavy)."""
    d, k = 300, 9
    o = Oracle(d, 1, 2, k, 1, 11)
    Tf = np.array([[10.0, 1.0]], np.float32)
    v = np.ones((1, d), np.float32)
    h, _ = o.hashes(np.arange(d))
    heavy = np.flatnonzero(h[0] == 0)
    for seed in range(20):
        out = o.heavymix(Tf, v, fill_seed=seed)
        assert out["nheavy"] == heavy.size > k
        assert out["out_idx"].tolist() == heavy[:k].tolist()


def test_fill_is_uniform_over_the_non_heavy_coordinates():
    d, k = 400, 40
    o = Oracle(d, 1, 512, k, 1, 0)
    o.set_params([[1, 0, 1, 0]])
    v = np.zeros((1, d), np.float32)                       # nothing heavy: est = 0, l2 = 0 -> every i is "heavy"?
    v[0, :] = 1e-3
    v[0, :5] = 100.0                                       # 5 heavy coordinates, 395 candidates for 35 slots
    T, _ = o.sketch_workers(v)
    Tf = T.astype(np.float32)
    counts = np.zeros(d)
    trials = 600
    for seed in range(trials):
        idx = o.heavymix(Tf, v, fill_seed=seed * 7919 + 1)["out_idx"]
        assert set(range(5)) <= set(idx.tolist())
        counts[idx] += 1
    p = (k - 5) / (d - 5)
    freq = counts[5:] / trials
    assert abs(freq.mean() - p) < 1e-9                     # exactly k-5 fills per trial
    sigma = np.sqrt(p * (1 - p) / trials)
    assert np.abs(freq - p).max() < 5 * sigma              # no coordinate is favoured


def test_heavymix_all_zero_table():
    d, k = 50, 7
    o = Oracle(d, 3, 8, k, 2, 0)
    v = np.zeros((2, d), np.float32)
    out = o.heavymix(np.zeros((3, 8), np.float32), v, fill_seed=5)
    # l2 = 0, so every coordinate satisfies est^2 >= 0 = l2/k: |H| = d > k, the k "largest" are the first k
    assert out["l2"] == 0.0 and out["nheavy"] == d
    assert out["out_idx"].tolist() == list(range(k))

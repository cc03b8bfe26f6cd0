"""Pins for the CPU checker's row binarization (Section 4.1, Algorithm 1 of arXiv 1804.02941).

The checker is compared with things that are not the checker: exhaustive search over every
mask in exact rational arithmetic, direct sums of squared error per split (no prefix sums, no
objective formula), closed forms, and the properties the paper states.  No GPU involved.
"""
import itertools
from fractions import Fraction

import numpy as np
import pytest

import dab_synth
import oracle


def _frac(x):
    return Fraction(float(x))


def brute_force_min_error(w):
    """min over all masks e (e != 0, e != 1) of ||W - alpha e - beta (1-e)||^2 with alpha, beta the
    partition means (Section 4.1), exact.  Returns (min error, set of optimal masks as tuples)."""
    n = len(w)
    fw = [_frac(x) for x in w]
    best, arg = None, set()
    for bits in range(1, (1 << n) - 1):
        e = [(bits >> i) & 1 for i in range(n)]
        k = sum(e)
        a = sum(x for x, b in zip(fw, e) if b) / k
        b_ = sum(x for x, b in zip(fw, e) if not b) / (n - k)
        err = sum((x - (a if b else b_)) ** 2 for x, b in zip(fw, e))
        if best is None or err < best:
            best, arg = err, {tuple(e)}
        elif err == best:
            arg.add(tuple(e))
    return best, arg


def rule_choice_exact(w):
    """The split the fixed rule selects, in exact arithmetic: candidates only between distinct sorted
    values, maximum objective, largest s among exact ties; e marks the side with the larger |mean|,
    the high side when the magnitudes are equal."""
    n = len(w)
    v = sorted(_frac(x) for x in w)
    T = sum(v)
    best, s_best = None, None
    for s in range(1, n):
        if v[s - 1] == v[s]:
            continue
        P = sum(v[:s])
        D = P * P / s + (T - P) * (T - P) / (n - s)
        if best is None or D >= best:
            best, s_best = D, s
    P = sum(v[:s_best])
    m_lo, m_hi = P / s_best, (T - P) / (n - s_best)
    t = v[s_best]
    if abs(m_lo) > abs(m_hi):
        e = [int(_frac(x) < t) for x in w]
        return s_best, e, m_lo, m_hi, best
    e = [int(_frac(x) >= t) for x in w]
    return s_best, e, m_hi, m_lo, best


def _rows_for_bruteforce():
    rows = []
    for n in (2, 3, 4, 5, 7, 9, 11):
        rows += list(dab_synth.small_integer_rows(6, n, -3, 3, stream=100 + n))
        rows += list(dab_synth.normal((3, n), 1.0, stream=200 + n))
        rows += list(dab_synth.relu_activations((3, n), 0.6, stream=300 + n))
    rows += [np.array(r, np.float32) for r in ([1, 2, 3], [-1, 0, 1], [0, 0, 0, 1, 2], [-10, -1, 1, 10],
                                               [0, 0, 0, 0, 0, 0, 1, 3], [1, 2, 3, 4], [-3, -1, 1, 3],
                                               [2, 2, 7, 7, 7], [0, 0, 1, 1], [-1, -1, 1, 1, 1, -1])]
    return rows


@pytest.mark.parametrize("idx", range(len(_rows_for_bruteforce())))
def test_matches_exhaustive_search_over_all_masks(idx):
    w = _rows_for_bruteforce()[idx]
    n = len(w)
    r = oracle.binarize(w[None, :])
    if r.flags[0] & oracle.FLAG_DEGENERATE:
        assert len(set(w.tolist())) == 1
        return
    err, argmin = brute_force_min_error(w)
    assert tuple(r.e[0].tolist()) in argmin                      # optimal over ALL masks, not just thresholds
    ww = sum(_frac(x) ** 2 for x in w)
    s, e, a, b, D = rule_choice_exact(w)
    assert err == ww - D                                          # E = ||W||^2 - D (appendix, proof of Theorem 2)
    assert r.s_star[0] == s and r.e[0].tolist() == e              # the fixed tie rule's choice
    assert r.K[0] == sum(e)
    assert r.alpha[0] == np.float32(float(a)) and r.beta[0] == np.float32(float(b))
    assert abs(r.best_D[0] - float(D)) <= 1e-14 * float(D)


def direct_sse_per_split(w):
    """For every split of the sorted row: sum of squared deviations from the two partition means."""
    v = np.sort(w.astype(np.float64))
    n = len(v)
    out = np.full(n, np.inf)
    for s in range(1, n):
        if v[s - 1] == v[s]:
            continue
        lo, hi = v[:s], v[s:]
        out[s] = ((lo - lo.mean()) ** 2).sum() + ((hi - hi.mean()) ** 2).sum()
    return out


@pytest.mark.parametrize("gen,n", [("normal", 50), ("normal", 577), ("relu", 576), ("laplace", 1152),
                                   ("cluster", 300), ("relu", 2304)])
def test_split_is_argmin_of_direct_squared_error(gen, n):
    rows = {"normal": lambda: dab_synth.normal((4, n), 0.05, stream=n),
            "relu": lambda: dab_synth.relu_activations((4, n), 0.6, stream=n),
            "laplace": lambda: dab_synth.laplace((4, n), 0.05, stream=n),
            "cluster": lambda: dab_synth.two_cluster_rows(4, n, stream=n)}[gen]()
    r = oracle.binarize(rows)
    for i, w in enumerate(rows):
        sse = direct_sse_per_split(w)
        s_direct = int(np.argmin(sse))
        if r.s_star[i] != s_direct:                               # only admissible at a near-tie
            assert abs(sse[r.s_star[i]] - sse[s_direct]) <= 1e-9 * float((w.astype(np.float64) ** 2).sum())
        ww = float((w.astype(np.float64) ** 2).sum())
        assert abs((ww - r.best_D[i]) - sse[r.s_star[i]]) <= 1e-9 * ww


def _reconstruct(r, i):
    e = r.e[i].astype(np.float64)
    return float(r.alpha[i]) * e + float(r.beta[i]) * (1.0 - e)


@pytest.mark.parametrize("n", [2, 3, 5, 27, 31, 32, 33, 63, 64, 65, 100, 575, 576, 577, 1600])
def test_invariants(n):
    rows = np.concatenate([dab_synth.normal((3, n), 0.05, stream=n), dab_synth.relu_activations((3, n), 0.6, stream=n),
                           dab_synth.two_cluster_rows(3, n, stream=n), dab_synth.small_integer_rows(3, n, stream=n)])
    r = oracle.binarize(rows)
    for i, w in enumerate(rows):
        w64 = w.astype(np.float64)
        if r.flags[i] & oracle.FLAG_DEGENERATE:
            assert np.all(w == w[0]) and r.K[i] == 0 and not r.e[i].any()
            continue
        e = r.e[i].astype(bool)
        assert 1 <= r.K[i] <= n - 1 and e.sum() == r.K[i]         # e != 0, e != 1 (Section 4.1)
        # alpha, beta are the means of their partitions (Section 4.1)
        assert r.alpha[i] == np.float32(w64[e].mean()) or abs(r.alpha[i] - w64[e].mean()) <= 1e-7 * abs(w64[e].mean())
        assert abs(r.beta[i] - w64[~e].mean()) <= 1e-7 * abs(w64[~e].mean()) + 1e-45
        # e is a threshold split: the K smallest or the K largest values (Section 4.1)
        assert w64[e].min() > w64[~e].max() or w64[e].max() < w64[~e].min()
        # "alpha captures the greater of the two values in magnitude"
        assert abs(w64[e].mean()) >= abs(w64[~e].mean())
        # the XNOR code  mean|W| * sign(W)  is a special case, so its error is never smaller (Section 4.1)
        xnor = np.abs(w64).mean() * np.where(w64 >= 0, 1.0, -1.0)
        e_dab = ((w64 - (w64[e].mean() * e + w64[~e].mean() * ~e)) ** 2).sum()
        assert e_dab <= ((w64 - xnor) ** 2).sum() * (1 + 1e-12) + 1e-300
        # E = ||W||^2 - D
        assert abs(e_dab - ((w64 ** 2).sum() - r.best_D[i])) <= 1e-9 * (w64 ** 2).sum()


def test_two_valued_rows_are_reproduced_exactly():
    for a, b, ka, n in [(0.25, -1.5, 3, 10), (2.0, 3.0, 1, 5), (-0.5, 0.5, 16, 32), (0.0, 1.0, 60, 100)]:
        w = np.full(n, b, np.float32)
        w[np.arange(ka) * (n // ka)] = a
        r = oracle.binarize(w[None])
        assert np.array_equal(_reconstruct(r, 0), w.astype(np.float64))         # zero error
        assert {float(r.alpha[0]), float(r.beta[0])} == {a, b}
        assert abs(r.alpha[0]) >= abs(r.beta[0])


def test_ramp_closed_form():
    # W = 1..n.  With u = s(n-s): D(s) - T^2/n = n u / 4, maximal at s = n/2; for odd n the two
    # middle splits tie exactly and ">=" keeps the larger one.
    for n in (4, 6, 10, 64, 100):
        r = oracle.binarize(np.arange(1, n + 1, dtype=np.float32)[None])
        assert r.s_star[0] == n // 2 and r.K[0] == n // 2 and r.gap[0] > 0
        assert r.alpha[0] == np.float32((n // 2 + 1 + n) / 2) and r.beta[0] == np.float32((1 + n // 2) / 2)
    for n in (3, 5, 11, 65, 101):
        r = oracle.binarize(np.arange(1, n + 1, dtype=np.float32)[None])
        assert r.s_star[0] == (n + 1) // 2 and r.gap[0] == 0.0
        assert r.K[0] == n - (n + 1) // 2                         # high side has the larger |mean|


def test_hand_worked_examples():
    # [1,2,3,4]: D = 1/1 + 81/3 = 28, 9/2 + 49/2 = 29, 36/3 + 16 = 28 -> s = 2, means 1.5 | 3.5
    r = oracle.binarize(np.array([[1, 2, 3, 4]], np.float32))
    assert (r.s_star[0], r.e[0].tolist(), r.K[0], r.alpha[0], r.beta[0], r.best_D[0]) == (2, [0, 0, 1, 1], 2, 3.5, 1.5, 29.0)
    # [-3,-1,1,3]: D = 9 + 9/3 = 12, 16/2 + 16/2 = 16, 12 -> s = 2; |means| tie -> high side is e (XNOR code)
    r = oracle.binarize(np.array([[-3, -1, 1, 3]], np.float32))
    assert (r.s_star[0], r.e[0].tolist(), r.alpha[0], r.beta[0], r.best_D[0]) == (2, [0, 0, 1, 1], 2.0, -2.0, 16.0)
    # [-10,-1,1,10]: D = 100 + 100/3, 121/2 + 121/2, 100/3 + 100: exact tie of s=1 and s=3 -> s=3
    r = oracle.binarize(np.array([[-10, -1, 1, 10]], np.float32))
    assert (r.s_star[0], r.e[0].tolist(), r.K[0], r.alpha[0], r.gap[0]) == (3, [0, 0, 0, 1], 1, 10.0, 0.0)
    assert r.beta[0] == np.float32(-10.0 / 3.0)
    # [0,0,0,1,2]: boundaries only at s=3 (0 + 9/2) and s=4 (1/4 + 4) -> s=3
    r = oracle.binarize(np.array([[0, 0, 0, 1, 2]], np.float32))
    assert (r.s_star[0], r.e[0].tolist(), r.K[0], r.alpha[0], r.beta[0]) == (3, [0, 0, 0, 1, 1], 2, 1.5, 0.0)
    # order of the row does not matter, the mask follows the elements
    r = oracle.binarize(np.array([[2, 0, 1, 0, 0]], np.float32))
    assert r.e[0].tolist() == [1, 0, 1, 0, 0]
    # low side wins the orientation when its mean is larger in magnitude
    r = oracle.binarize(np.array([[-4, -4, 1, 1, 1]], np.float32))
    assert (r.e[0].tolist(), r.K[0], r.alpha[0], r.beta[0]) == ([1, 1, 0, 0, 0], 2, -4.0, 1.0)


def test_constant_rows_and_single_element():
    for w in ([5, 5, 5], [0, 0, 0, 0], [-2.5], [0.0, -0.0, 0.0]):
        r = oracle.binarize(np.array([w], np.float32))
        assert r.flags[0] == oracle.FLAG_DEGENERATE and r.K[0] == 0 and not r.e[0].any()
        assert r.alpha[0] == r.beta[0] == np.float32(w[0])


def test_negative_zero_equals_positive_zero():
    a = oracle.binarize(np.array([[0.0, -0.0, 1.0, 2.0, -0.0]], np.float32))
    b = oracle.binarize(np.array([[0.0, 0.0, 1.0, 2.0, 0.0]], np.float32))
    assert a.e.tolist() == b.e.tolist() and a.K[0] == b.K[0] and a.alpha[0] == b.alpha[0] and a.beta[0] == b.beta[0]


def test_nonfinite_rows_are_flagged():
    for bad in (np.nan, np.inf, -np.inf):
        r = oracle.binarize(np.array([[1.0, bad, 3.0], [1.0, 2.0, 4.0]], np.float32))
        assert r.flags[0] & oracle.FLAG_NONFINITE and r.flags[1] == 0 and r.K[1] == 1


def test_symmetric_rows_give_the_xnor_code():
    # rows of +-v: K = n/2, alpha = -beta = v  (the XNOR-Net special case, Sections 4.1-4.2)
    n = 64
    signs = np.ones(n)
    signs[n // 2:] = -1.0
    perm = np.argsort(dab_synth.uniform01(7, 8, 0, n))
    w = (0.37 * signs[perm]).astype(np.float32)
    r = oracle.binarize(w[None])
    assert r.K[0] == n // 2 and r.alpha[0] == np.float32(0.37) and r.beta[0] == np.float32(-0.37)
    assert np.array_equal(r.e[0].astype(bool), w > 0)             # equal |means|: the high side is e
    # two clusters straddling zero: the partition is the sign pattern; which side is called e
    # depends on which cluster mean happens to be larger in magnitude
    w = np.concatenate([dab_synth.normal((1, 32), 0.01, stream=5, mean=1.0),
                        dab_synth.normal((1, 32), 0.01, stream=6, mean=-1.0)], 1)
    r = oracle.binarize(w)
    pos = w[0] > 0
    assert r.K[0] == 32
    if abs(w[0][pos].astype(np.float64).mean()) >= abs(w[0][~pos].astype(np.float64).mean()):
        assert np.array_equal(r.e[0].astype(bool), pos) and r.alpha[0] > 0 > r.beta[0]
    else:
        assert np.array_equal(r.e[0].astype(bool), ~pos) and r.alpha[0] < 0 < r.beta[0]


def test_otsu_between_class_variance_reduction():
    # D - T^2/n = n * (between-class variance of the two partitions): the split equals the
    # textbook 1-D two-means / Otsu threshold.
    w = dab_synth.two_cluster_rows(5, 400, stream=11)
    r = oracle.binarize(w)
    for i in range(5):
        v = np.sort(w[i].astype(np.float64))
        n = len(v)
        mu = v.mean()
        bcv = np.array([s / n * (v[:s].mean() - mu) ** 2 + (n - s) / n * (v[s:].mean() - mu) ** 2 for s in range(1, n)])
        assert int(np.argmax(bcv)) + 1 == r.s_star[i]
        assert abs((r.best_D[i] - v.sum() ** 2 / n) - n * bcv.max()) <= 1e-9 * r.best_D[i]
        assert 0.3 <= min(r.K[i], n - r.K[i]) / n <= 0.4          # normalised K near 0.35 (Figure 4)


def test_batched_call_equals_row_calls_and_threads_do_not_change_results():
    w = dab_synth.relu_activations((64, 200), 0.6, stream=21)
    oracle.set_threads(1)
    a = oracle.binarize(w)
    oracle.set_threads(4)
    b = oracle.binarize(w)
    oracle.set_threads(1)
    for f in ("e", "K", "alpha", "beta", "flags", "s_star", "best_D"):
        assert np.array_equal(getattr(a, f), getattr(b, f))
    one = oracle.binarize(w[17:18])
    assert np.array_equal(one.e[0], a.e[17]) and one.alpha[0] == a.alpha[17]

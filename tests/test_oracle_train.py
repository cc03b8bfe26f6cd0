"""Pins of the checker's training-side functions: Algorithm 2 steps 4-13 (MeanCenter, Clamp, Algorithm 1, dense
two-level filter) and Theorem 4 (the elementwise gradient factor).

Theorem 4's two straight-through terms have no definition outside the theorem itself ("parity unpinned" in the
checker's header); what is pinned here: the other two terms as finite-difference derivatives of alpha and beta with
the mask held fixed, the support and clamp structure of every term, and the special cases that reduce to those.
"""
import numpy as np
import pytest

import dab_synth
import oracle


def _rows(rows, n, std, stream, mean=0.0):
    return dab_synth.normal((rows, n), std, stream=stream, mean=mean)


def test_forward_equals_library_mean_and_clip_then_algorithm_1():
    W = np.concatenate([_rows(6, 147, 0.3, 500, mean=0.2), _rows(3, 147, 1.5, 501, mean=-0.4)])   # second part clamps
    Wc, e, K, alpha, beta, flags, Wt = oracle.train_forward(W)
    ref = np.clip((W.astype(np.float64) - W.astype(np.float64).mean(axis=1, keepdims=True)).astype(np.float32), -1, 1)
    assert np.array_equal(Wc, ref)
    assert (np.abs(Wc[6:]) == 1.0).any() and not (np.abs(Wc[:6]) == 1.0).any()
    b = oracle.binarize(ref)
    assert np.array_equal(e, b.e) and np.array_equal(K, b.K)
    assert np.array_equal(alpha, b.alpha) and np.array_equal(beta, b.beta) and np.array_equal(flags, b.flags)
    assert np.array_equal(Wt, np.where(e != 0, alpha[:, None], beta[:, None]))


def test_mean_centred_rows_have_zero_mean_and_two_levels_that_are_partition_means():
    W = _rows(8, 576, 0.02, 502, mean=0.01)
    Wc, e, K, alpha, beta, _, Wt = oracle.train_forward(W)
    assert np.all(np.abs(Wc.astype(np.float64).mean(axis=1)) < 1e-9)
    for r in range(8):
        sel = e[r] != 0
        assert K[r] == sel.sum() and 0 < K[r] < 576
        assert alpha[r] == np.float32(Wc[r][sel].astype(np.float64).mean())
        assert beta[r] == np.float32(Wc[r][~sel].astype(np.float64).mean())
        assert set(np.unique(Wt[r])) == {alpha[r], beta[r]}


def test_two_valued_rows_become_the_xnor_code_after_mean_centring():
    # Section 4.2: a mean-centred row with K = n/2 is the XNOR-Net code.  Half a, half b (any offset) -> +-(b-a)/2.
    n = 64
    a, b = np.float32(0.125), np.float32(0.625)
    W = np.tile(np.r_[np.full(n // 2, a), np.full(n // 2, b)].astype(np.float32), (2, 1))
    W[1] = W[1][::-1]
    Wc, e, K, alpha, beta, _, Wt = oracle.train_forward(W)
    assert np.all(K == n // 2) and np.all(alpha == 0.25) and np.all(beta == -0.25)
    assert np.array_equal(e[0], (W[0] == b).astype(np.uint8)) and np.array_equal(e[1], (W[1] == b).astype(np.uint8))
    assert np.array_equal(Wt, Wc)                                    # two-valued rows are reproduced exactly


def test_constant_rows_centre_to_zero_and_are_degenerate():
    W = np.full((1, 20), 0.3, np.float32)
    Wc, e, K, alpha, beta, flags, Wt = oracle.train_forward(W)
    assert not Wc.any() and K[0] == 0 and flags[0] == oracle.FLAG_DEGENERATE and not Wt.any() and not e.any()


def test_theorem4_terms_without_ste_are_the_derivatives_of_alpha_and_beta_for_a_fixed_mask():
    # d(alpha)/dW_i = e_i / K and d(beta)/dW_i = (1 - e_i) / (n - K): central differences on alpha = W.e / K.
    # The STE terms vanish where |W_i| > 1 is impossible after the clamp only if W_i = 0; so use a row scaled to
    # make them visible and subtract them through a second evaluation with the same mask (G is affine in them).
    W = _rows(3, 40, 0.3, 503)
    Wc, e, K, *_ = oracle.train_forward(W)
    G, _ = oracle.theorem4(Wc, e, K)
    for r in range(3):
        sel = e[r] != 0
        l1s, l1r = np.abs(Wc[r][sel]).astype(np.float64).sum(), np.abs(Wc[r][~sel]).astype(np.float64).sum()
        base = G[r] - np.where(sel, l1s / K[r], l1r / (40 - K[r])) * Wc[r].astype(np.float64)   # remove the STE terms
        h = 1e-3
        for i in range(40):
            wp, wm = Wc[r].astype(np.float64).copy(), Wc[r].astype(np.float64).copy()
            wp[i] += h
            wm[i] -= h
            dalpha = (wp[sel].mean() - wm[sel].mean()) / (2 * h)
            dbeta = (wp[~sel].mean() - wm[~sel].mean()) / (2 * h)
            assert abs(base[i] - (dalpha + dbeta)) < 1e-9


def test_theorem4_structure():
    W = np.concatenate([_rows(4, 90, 0.4, 504), _rows(2, 90, 2.0, 505)])
    Wc, e, K, *_ = oracle.train_forward(W)
    G, _ = oracle.theorem4(Wc, e, K)
    n = 90
    for r in range(6):
        sel = e[r] != 0
        # on zeros of W the STE terms vanish: only 1/K or 1/(n-K) is left
        Wz = Wc[r].copy()
        Wz[:5] = 0.0
        Gz, _ = oracle.theorem4(Wz[None], e[r][None], K[r:r + 1])
        assert np.allclose(Gz[0][:5], np.where(sel[:5], 1.0 / K[r], 1.0 / (n - K[r])), rtol=1e-15)
        # a weight beyond the clamp range (possible only if the caller skips the clamp) loses its STE term
        Wb = Wc[r].copy()
        Wb[7] = 1.5
        Gb, _ = oracle.theorem4(Wb[None], e[r][None], K[r:r + 1])
        assert Gb[0][7] == (1.0 / K[r] if sel[7] else 1.0 / (n - K[r]))
        # every entry: indicator term plus (l1 norm of its own partition / its size) * W_i
        l1 = np.where(sel, np.abs(Wc[r][sel]).astype(np.float64).sum() / K[r],
                      np.abs(Wc[r][~sel]).astype(np.float64).sum() / (n - K[r]))
        assert np.allclose(G[r], np.where(sel, 1.0 / K[r], 1.0 / (n - K[r])) + l1 * Wc[r], rtol=1e-14, atol=0)


def test_theorem4_hand_worked_row():
    # W = [0.5, -0.25, 0.25, -0.5], e = [1, 0, 0, 1] (K = 2): ||T_k||_1 = 1, ||W - T_k||_1 = 0.5
    # G = [1/2 + (1/2)(0.5), 1/2 + (0.25)(-0.25), 1/2 + (0.25)(0.25), 1/2 + (1/2)(-0.5)] = [0.75, 0.4375, 0.5625, 0.25]
    W = np.array([[0.5, -0.25, 0.25, -0.5]], np.float32)
    e = np.array([[1, 0, 0, 1]], np.uint8)
    G, gw = oracle.theorem4(W, e, np.array([2], np.int32), grad_Wt=np.array([[2.0, 4.0, -8.0, 1.0]], np.float32))
    assert np.array_equal(G[0], [0.75, 0.4375, 0.5625, 0.25])
    assert np.array_equal(gw[0], np.array([1.5, 1.75, -4.5, 0.25], np.float32))


def test_theorem4_degenerate_rows_give_zero():
    W = np.zeros((1, 8), np.float32)
    G, gw = oracle.theorem4(W, np.zeros((1, 8), np.uint8), np.array([0], np.int32), grad_Wt=np.ones((1, 8), np.float32))
    assert not G.any() and not gw.any()

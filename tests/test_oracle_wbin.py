"""Pins of the checker's weights-only forward pass (Section 4.3.2: I (*) W~ with fp32 activations).

The function is the plain definition of a convolution with the reconstructed two-level filters, so it is pinned
against a library convolution in fp64, a matrix product for 1x1 kernels, box sums for constant filters, closed
forms on ramps, and the split of the sum into the part under e and the part under 1-e.
"""
import numpy as np
import pytest
import torch

import dab_synth
import oracle

CASES = [
    dict(N=1, C=3, H=6, W=7, Cout=4, kh=3, kw=3, stride=(1, 1), pad=(1, 1)),
    dict(N=2, C=4, H=9, W=8, Cout=3, kh=5, kw=5, stride=(1, 1), pad=(2, 2)),
    dict(N=2, C=5, H=8, W=8, Cout=6, kh=3, kw=3, stride=(2, 2), pad=(1, 1)),
    dict(N=1, C=8, H=5, W=5, Cout=5, kh=1, kw=1, stride=(1, 1), pad=(0, 0)),
    dict(N=1, C=3, H=7, W=6, Cout=2, kh=3, kw=2, stride=(2, 1), pad=(0, 1)),   # kh != kw, strides differ
]


def _inputs(c, seed, signed=False):
    shape = (c["N"], c["C"], c["H"], c["W"])
    x = dab_synth.normal(shape, 1.0, stream=300 + seed) if signed else dab_synth.relu_activations(shape, 0.6, stream=300 + seed)
    w = dab_synth.normal((c["Cout"], c["C"] * c["kh"] * c["kw"]), 0.05, stream=320 + seed)
    return x.astype(np.float32), w


def _dense(wb, c):
    Wt = np.where(wb.e != 0, wb.alpha[:, None].astype(np.float64), wb.beta[:, None].astype(np.float64))
    return Wt.reshape(c["Cout"], c["C"], c["kh"], c["kw"])


@pytest.mark.parametrize("signed", [False, True])
@pytest.mark.parametrize("ci", range(len(CASES)))
def test_equals_library_fp64_convolution_with_reconstructed_filters(ci, signed):
    c = CASES[ci]
    x, w = _inputs(c, ci, signed)
    wb = oracle.binarize(w)
    y, mag = oracle.conv_wbin(x, wb.e, wb.alpha, wb.beta, c["kh"], c["kw"], c["stride"], c["pad"])
    Wt = torch.from_numpy(_dense(wb, c))
    ref = torch.nn.functional.conv2d(torch.from_numpy(x).double(), Wt, stride=c["stride"], padding=c["pad"]).numpy()
    ref_mag = torch.nn.functional.conv2d(torch.from_numpy(x).double().abs(), Wt.abs(), stride=c["stride"],
                                         padding=c["pad"]).numpy()
    assert y.shape == ref.shape
    # fp64 sums in two orders differ by a few 1e-16 of the sum of magnitudes; the final fp32 rounding adds 6e-8 |y|
    assert np.all(np.abs(y.astype(np.float64) - ref) <= 1e-13 * ref_mag + 6e-8 * np.abs(ref))
    assert np.allclose(mag, ref_mag, rtol=1e-13, atol=0)


def test_one_by_one_kernel_is_a_matrix_product():
    c = CASES[3]
    x, w = _inputs(c, 3, signed=True)
    wb = oracle.binarize(w)
    y, _ = oracle.conv_wbin(x, wb.e, wb.alpha, wb.beta, 1, 1)
    rows = x.transpose(0, 2, 3, 1).reshape(-1, c["C"]).astype(np.float64)
    ref = (rows @ _dense(wb, c).reshape(c["Cout"], -1).T).reshape(c["N"], c["H"], c["W"], c["Cout"]).transpose(0, 3, 1, 2)
    assert np.allclose(y, ref, rtol=1e-6, atol=1e-12)


def test_equal_levels_give_a_scaled_box_sum_whatever_the_mask():
    # alpha == beta == v: W~ is constant, so y = v * (sum of the patch), for any e; small integers make it exact
    x = np.arange(2 * 3 * 5 * 6, dtype=np.float32).reshape(2, 3, 5, 6) % 7
    e = (dab_synth.uniform01(5, 3, 0, 4 * 27).reshape(4, 27) < 0.5).astype(np.uint8)
    v = np.full(4, 0.5, np.float32)
    y, _ = oracle.conv_wbin(x, e, v, v, 3, 3, (1, 1), (1, 1))
    xp = np.pad(x.astype(np.float64), ((0, 0), (0, 0), (1, 1), (1, 1)))
    box = sum(xp[:, :, r:r + 5, s:s + 6] for r in range(3) for s in range(3)).sum(axis=1)   # N x H x W
    assert np.array_equal(y, np.repeat((0.5 * box)[:, None], 4, axis=1).astype(np.float32))


def test_hand_worked_two_by_two_kernel():
    # x = [[1,2,3],[4,5,6],[7,8,9]], one channel, kernel 2x2, e = [[1,0],[0,1]], alpha = 2, beta = -1:
    # y[0,0] = 2*1 - 2 - 4 + 2*5 = 6; y[0,1] = 2*2 - 3 - 5 + 2*6 = 8; y[1,0] = 2*4 - 5 - 7 + 2*8 = 12; y[1,1] = 14
    x = np.arange(1, 10, dtype=np.float32).reshape(1, 1, 3, 3)
    e = np.array([[1, 0, 0, 1]], np.uint8)
    y, mag = oracle.conv_wbin(x, e, np.array([2.0], np.float32), np.array([-1.0], np.float32), 2, 2)
    assert np.array_equal(y.reshape(2, 2), np.array([[6, 8], [12, 14]], np.float32))
    assert np.array_equal(mag.reshape(2, 2), np.array([[18, 24], [36, 42]], np.float64))


def test_splits_into_the_sums_under_e_and_under_its_complement():
    # y = alpha * sum_{e=1} x + beta * sum_{e=0} x, computed here with integer-valued inputs so that every sum is exact
    c = CASES[0]
    x = np.round(dab_synth.normal((1, 3, 6, 7), 8.0, stream=340)).astype(np.float32)
    e = (dab_synth.uniform01(5, 4, 0, 4 * 27).reshape(4, 27) < 0.35).astype(np.uint8)
    alpha = np.array([0.5, 1.25, -2.0, 3.0], np.float32)
    beta = np.array([-0.25, 0.75, 1.5, -1.0], np.float32)
    y, _ = oracle.conv_wbin(x, e, alpha, beta, 3, 3, (1, 1), (1, 1))
    P = oracle.im2col(x, 3, 3, (1, 1), (1, 1)).astype(np.float64)                     # patches x 27
    s1 = P @ e.T.astype(np.float64)
    s0 = P @ (1 - e.T.astype(np.float64))
    ref = (s1 * alpha.astype(np.float64) + s0 * beta.astype(np.float64)).reshape(1, 6, 7, 4).transpose(0, 3, 1, 2)
    assert np.array_equal(y, ref.astype(np.float32))


def test_not_symmetric_in_alpha_and_beta():
    c = CASES[0]
    x, w = _inputs(c, 0)
    wb = oracle.binarize(w)
    y1, _ = oracle.conv_wbin(x, wb.e, wb.alpha, wb.beta, 3, 3, (1, 1), (1, 1))
    y2, _ = oracle.conv_wbin(x, wb.e, wb.beta, wb.alpha, 3, 3, (1, 1), (1, 1))
    y3, _ = oracle.conv_wbin(x, 1 - wb.e, wb.beta, wb.alpha, 3, 3, (1, 1), (1, 1))
    assert not np.array_equal(y1, y2)
    assert np.allclose(y1, y3, rtol=1e-6, atol=1e-9)         # complementing e and exchanging the levels is the same filter

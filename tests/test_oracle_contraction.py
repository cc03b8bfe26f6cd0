"""Pins for the CPU checker's packing, coded dot products and convolution.

Compared with: Python integers for the bit layout, the fp64 dot product of the reconstructed
two-level vectors, a textbook XNOR-popcount for the alpha = -beta special case, torch's unfold
(a library im2col) and torch's fp64 conv2d.  No GPU involved.
"""
import numpy as np
import pytest
import torch

import dab_synth
import oracle


def _reconstruct(e, a, b):
    e = e.astype(np.float64)
    return a.astype(np.float64)[:, None] * e + b.astype(np.float64)[:, None] * (1.0 - e)


@pytest.mark.parametrize("n", [1, 5, 31, 32, 33, 64, 100, 576, 577])
def test_pack_bit_order_and_padding(n):
    bits = (dab_synth.uniform01(3, n, 0, 4 * n) < 0.4).astype(np.uint8).reshape(4, n)
    mask, K = oracle.pack(bits)
    wd = (n + 31) // 32
    assert mask.shape[1] % 4 == 0 and mask.shape[1] >= wd
    for r in range(4):
        as_int = sum(int(b) << i for i, b in enumerate(bits[r]))            # element i -> bit i of one big integer
        words = [(as_int >> (32 * j)) & 0xFFFFFFFF for j in range(mask.shape[1])]
        assert mask[r].tolist() == words                                     # little-endian words, zero padding
        assert K[r] == bin(as_int).count("1")
    m2, _ = oracle.pack(bits, ld_mask=wd + 5)
    assert np.array_equal(m2[:, :wd], mask[:, :wd]) and not m2[:, wd:].any()


def test_hand_worked_contraction():
    # W = [1,2,3,4] -> e = 0011, alpha 3.5, beta 1.5 ; X = [-3,-1,1,3] -> f = 0011, gamma 2, delta -2
    # W~ = [1.5,1.5,3.5,3.5], X~ = [-2,-2,2,2] -> W~.X~ = -3 -3 +7 +7 = 8 ; p11 = 2
    w = oracle.binarize(np.array([[1, 2, 3, 4]], np.float32))
    x = oracle.binarize(np.array([[-3, -1, 1, 3]], np.float32))
    Cm, p11 = oracle.gemm(x.e, x.alpha, x.beta, w.e, w.alpha, w.beta)
    assert Cm[0, 0] == 8.0 and p11[0, 0] == 2


@pytest.mark.parametrize("M,N,n", [(7, 5, 33), (16, 9, 576), (3, 4, 1), (5, 6, 100)])
def test_gemm_equals_dot_of_reconstructed_vectors(M, N, n):
    A = dab_synth.relu_activations((M, n), 0.6, stream=1)
    B = dab_synth.normal((N, n), 0.05, stream=2)
    a, b = oracle.binarize(A), oracle.binarize(B)
    Cm, p11 = oracle.gemm(a.e, a.alpha, a.beta, b.e, b.alpha, b.beta)
    ref = _reconstruct(a.e, a.alpha, a.beta) @ _reconstruct(b.e, b.alpha, b.beta).T
    scale = np.abs(_reconstruct(a.e, a.alpha, a.beta)) @ np.abs(_reconstruct(b.e, b.alpha, b.beta)).T
    assert np.all(np.abs(Cm - ref) <= 1e-6 * scale + 1e-30)
    # integer identities of the four counts
    ea, eb = a.e.astype(np.int64), b.e.astype(np.int64)
    assert np.array_equal(p11, ea @ eb.T)
    p10 = b.K[None, :] - p11          # weight bit set, activation bit clear
    p01 = a.K[:, None] - p11
    p00 = n - a.K[:, None] - b.K[None, :] + p11
    assert np.array_equal(p10, (1 - ea) @ eb.T) and np.array_equal(p01, ea @ (1 - eb).T)
    assert np.array_equal(p00, (1 - ea) @ (1 - eb).T) and np.all(p11 + p10 + p01 + p00 == n)


def test_gemm_is_not_symmetric_in_its_operands():
    # A carries (gamma, delta) per row of C, B carries (alpha, beta) per column: a transposed operand must show
    A = dab_synth.normal((3, 40), 1.0, stream=31)
    B = dab_synth.normal((5, 40), 1.0, stream=32)
    a, b = oracle.binarize(A), oracle.binarize(B)
    C1, _ = oracle.gemm(a.e, a.alpha, a.beta, b.e, b.alpha, b.beta)
    C2, _ = oracle.gemm(b.e, b.alpha, b.beta, a.e, a.alpha, a.beta)
    assert C1.shape == (3, 5) and C2.shape == (5, 3) and np.array_equal(C1, C2.T)
    ref = _reconstruct(a.e, a.alpha, a.beta) @ _reconstruct(b.e, b.alpha, b.beta).T
    assert np.allclose(C1, ref, rtol=1e-6, atol=1e-12)


def test_xnor_special_case():
    # Both operands +-v rows: alpha = -beta, gamma = -delta, and the four-term sum collapses to
    # alpha*gamma*(n - 2*popcount(e xor f)), the XNOR-popcount dot product of the prior work the paper cites.
    n = 96
    def balanced_signs(rows, stream):           # every row has exactly n/2 entries of each sign
        s = np.ones((rows, n))
        for r in range(rows):
            s[r, np.argsort(dab_synth.uniform01(5, stream + r, 0, n))[: n // 2]] = -1.0
        return s
    sa, sb = balanced_signs(4, 10), balanced_signs(6, 20)
    va = np.array([0.5, 1.25, 2.0, 0.75], np.float32)[:, None]
    vb = np.array([0.1, 0.2, 0.3, 0.4, 0.5, 0.6], np.float32)[:, None]
    a, b = oracle.binarize((sa * va).astype(np.float32)), oracle.binarize((sb * vb).astype(np.float32))
    assert np.all(a.K == n // 2) and np.all(b.K == n // 2)
    assert np.array_equal(a.alpha, -a.beta) and np.array_equal(b.alpha, -b.beta)
    Cm, _ = oracle.gemm(a.e, a.alpha, a.beta, b.e, b.alpha, b.beta)
    for i in range(4):
        ei = sum(int(v) << k for k, v in enumerate(a.e[i]))
        for j in range(6):
            fj = sum(int(v) << k for k, v in enumerate(b.e[j]))
            xnor = float(a.alpha[i]) * float(b.alpha[j]) * (n - 2 * bin(ei ^ fj).count("1"))
            assert Cm[i, j] == np.float32(xnor)


CONV_CASES = [
    dict(N=1, C=3, H=6, W=7, Cout=4, kh=3, kw=3, stride=(1, 1), pad=(1, 1)),
    dict(N=2, C=4, H=9, W=8, Cout=3, kh=5, kw=5, stride=(1, 1), pad=(2, 2)),
    dict(N=2, C=5, H=8, W=8, Cout=6, kh=3, kw=3, stride=(2, 2), pad=(1, 1)),
    dict(N=1, C=8, H=5, W=5, Cout=5, kh=1, kw=1, stride=(1, 1), pad=(0, 0)),
    dict(N=1, C=2, H=7, W=7, Cout=3, kh=7, kw=7, stride=(1, 1), pad=(0, 0)),
    dict(N=1, C=3, H=7, W=6, Cout=2, kh=3, kw=2, stride=(2, 1), pad=(0, 1)),
]


def _conv_inputs(c, seed=0):
    x = dab_synth.relu_activations((c["N"], c["C"], c["H"], c["W"]), 0.6, stream=40 + seed)
    w = dab_synth.normal((c["Cout"], c["C"] * c["kh"] * c["kw"]), 0.05, stream=50 + seed)
    return x, w


@pytest.mark.parametrize("ci", range(len(CONV_CASES)))
def test_im2col_equals_library_unfold(ci):
    c = CONV_CASES[ci]
    x, _ = _conv_inputs(c, ci)
    got = oracle.im2col(x, c["kh"], c["kw"], c["stride"], c["pad"])
    u = torch.nn.functional.unfold(torch.from_numpy(x), (c["kh"], c["kw"]), padding=c["pad"], stride=c["stride"])
    ref = u.permute(0, 2, 1).reshape(-1, c["C"] * c["kh"] * c["kw"]).numpy()    # rows (img, ho, wo), cols (c, kh, kw)
    assert np.array_equal(got, ref)


@pytest.mark.parametrize("ci", range(len(CONV_CASES)))
def test_conv_equals_unfold_binarize_reconstruct_matmul(ci):
    c = CONV_CASES[ci]
    x, w = _conv_inputs(c, ci)
    wb = oracle.binarize(w)
    res = oracle.conv(x, wb.e, wb.alpha, wb.beta, c["kh"], c["kw"], c["stride"], c["pad"])
    u = torch.nn.functional.unfold(torch.from_numpy(x), (c["kh"], c["kw"]), padding=c["pad"], stride=c["stride"])
    patches = u.permute(0, 2, 1).reshape(-1, w.shape[1]).numpy()
    pb = oracle.binarize(patches)
    assert np.array_equal(res.p_e, pb.e) and np.array_equal(res.p_K, pb.K)
    assert np.array_equal(res.p_gamma, pb.alpha) and np.array_equal(res.p_delta, pb.beta)
    Xt, Wt = _reconstruct(pb.e, pb.alpha, pb.beta), _reconstruct(wb.e, wb.alpha, wb.beta)
    ref = Xt @ Wt.T                                                              # patches x Cout, fp64
    Ho, Wo = oracle.conv_out_hw(c["H"], c["W"], c["kh"], c["kw"], c["stride"], c["pad"])
    ref = ref.reshape(c["N"], Ho, Wo, c["Cout"]).transpose(0, 3, 1, 2)           # -> NCHW
    scale = (np.abs(Xt) @ np.abs(Wt).T).reshape(c["N"], Ho, Wo, c["Cout"]).transpose(0, 3, 1, 2)
    assert res.y.shape == ref.shape and np.all(np.abs(res.y - ref) <= 1e-6 * scale + 1e-30)
    assert np.array_equal(res.p_p11, pb.e.astype(np.int64) @ wb.e.astype(np.int64).T)


def test_conv_with_two_level_input_equals_dense_fp64_convolution():
    # If every patch of the input already holds exactly two values, its code reproduces it exactly, so the
    # binary conv must equal an ordinary dense convolution of that input with W~ (zero padding excluded: pad 0).
    c = dict(N=2, C=3, H=8, W=9, Cout=4, kh=3, kw=3, stride=(1, 1), pad=(0, 0))
    x = np.where(dab_synth.uniform01(9, 1, 0, 2 * 3 * 8 * 9).reshape(2, 3, 8, 9) < 0.3, 1.5, 0.25).astype(np.float32)
    w = dab_synth.normal((4, 27), 0.05, stream=61)
    wb = oracle.binarize(w)
    res = oracle.conv(x, wb.e, wb.alpha, wb.beta, 3, 3, (1, 1), (0, 0))
    Wt = torch.from_numpy(_reconstruct(wb.e, wb.alpha, wb.beta).reshape(4, 3, 3, 3))
    ref = torch.nn.functional.conv2d(torch.from_numpy(x).double(), Wt).numpy()
    assert np.allclose(res.y, ref, rtol=1e-6, atol=1e-9)


def test_one_by_one_conv_equals_gemm():
    c = CONV_CASES[3]
    x, w = _conv_inputs(c, 3)
    wb = oracle.binarize(w)
    res = oracle.conv(x, wb.e, wb.alpha, wb.beta, 1, 1)
    rows = x.transpose(0, 2, 3, 1).reshape(-1, c["C"])
    rb = oracle.binarize(rows)
    Cm, _ = oracle.gemm(rb.e, rb.alpha, rb.beta, wb.e, wb.alpha, wb.beta)
    assert np.array_equal(res.y, Cm.reshape(c["N"], c["H"], c["W"], c["Cout"]).transpose(0, 3, 1, 2))


def test_border_patches_contain_the_padding_zeros():
    # all-positive input, pad 1: a corner patch holds 5 padded zeros per channel, which must enter the code
    x = (1.0 + dab_synth.relu_activations((1, 2, 4, 4), 0.0, stream=70)).astype(np.float32)
    wb = oracle.binarize(dab_synth.normal((2, 18), 0.05, stream=71))
    res = oracle.conv(x, wb.e, wb.alpha, wb.beta, 3, 3, (1, 1), (1, 1))
    corner = res.p_e[0].reshape(2, 3, 3)
    assert res.p_K[0] == 8 and res.p_delta[0] == 0.0            # 4 real values per channel coded as e, zeros as 1-e
    assert not corner[:, 0, :].any() and not corner[:, :, 0].any() and corner[:, 1:, 1:].all()

"""GPU parity: every C-ABI entry point against the CPU checker, element by element, on seeded inputs.

Sizes span several tiles and ragged tails but stay small enough for the checker to finish in seconds.
"""
import numpy as np
import pytest
import torch

import dab_synth
from dab_synth import configs
import oracle
from parity_util import check_coded, rel_close, to_dev, unpack, words

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def dab():
    import paper_1804_02941_b200 as d
    d.lib()                       # fails loudly if the CUDA library is missing
    oracle.set_threads(8)
    return d


def _rows(kind, rows, n, stream):
    if kind == "normal":
        return dab_synth.normal((rows, n), 0.05, stream=stream)
    if kind == "relu":
        return dab_synth.relu_activations((rows, n), 0.6, stream=stream)
    if kind == "laplace":
        return dab_synth.laplace((rows, n), 0.05, stream=stream)
    if kind == "cluster":
        return dab_synth.two_cluster_rows(rows, n, stream=stream)
    if kind == "ints":
        return dab_synth.small_integer_rows(rows, n, -3, 3, stream=stream)
    raise ValueError(kind)


@pytest.mark.parametrize("n", [1, 2, 3, 5, 27, 31, 32, 33, 63, 64, 65, 100, 128, 129, 575, 576, 577, 1024, 1025,
                               1152, 1600, 2304, 2400, 4608])
@pytest.mark.parametrize("kind", ["normal", "relu", "ints"])
def test_binarize_matches_checker(dab, n, kind, record_property):
    rows = 37 if n < 2000 else 9
    w = _rows(kind, rows, n, stream=n)
    got = dab.dab_binarize(to_dev(w))
    near = check_coded(got, oracle.binarize(w), n, log=print)
    record_property("near_ties", near)


@pytest.mark.parametrize("n", [9216, 12544, 16384])
def test_binarize_long_rows(dab, n):
    w = np.concatenate([_rows("normal", 2, n, 1), _rows("relu", 2, n, 2), _rows("laplace", 2, n, 3)])
    check_coded(dab.dab_binarize(to_dev(w)), oracle.binarize(w), n, log=print)


def test_binarize_special_rows(dab):
    n = 96
    rows = [np.full(n, 5.0), np.zeros(n), np.arange(n), -np.arange(n), np.where(np.arange(n) % 2, 0.37, -0.37),
            np.r_[np.zeros(n - 1), 3.0], np.r_[-7.0, np.zeros(n - 1)], np.r_[np.zeros(n // 2), np.ones(n // 2)],
            np.where(np.arange(n) % 3 == 0, -0.0, 0.0), np.r_[-10.0, -1.0, 1.0, 10.0, np.zeros(n - 4)],
            np.arange(n) - (n - 1) / 2.0, np.r_[np.full(n - 2, 1e-30), 1.0, 2.0], np.r_[np.full(n - 1, 1.0), 1.0000001]]
    w = np.array(rows, np.float32)
    check_coded(dab.dab_binarize(to_dev(w)), oracle.binarize(w), n, log=print)
    odd = np.arange(1, 102, dtype=np.float32)[None]              # exact tie between the two middle splits
    check_coded(dab.dab_binarize(to_dev(odd)), oracle.binarize(odd), 101)


def test_binarize_nonfinite_rows_are_flagged_not_fatal(dab):
    w = dab_synth.normal((6, 70), 1.0, stream=9)
    w[1, 3] = np.nan
    w[3, 69] = np.inf
    w[4, 0] = -np.inf
    got = dab.dab_binarize(to_dev(w))
    ref = oracle.binarize(w)
    check_coded(got, ref, 70)
    assert got.flags.cpu().tolist() == [0, 2, 0, 2, 2, 0]


def test_binarize_strided_rows_and_wide_masks(dab):
    buf = dab_synth.relu_activations((20, 700), 0.6, stream=12)
    dev = to_dev(buf)
    view = dev[:, 50:50 + 577]                                   # ld_values = 700 > n, unaligned start
    got = dab.dab_binarize(view, ld_mask=28)
    assert got.mask.shape == (20, 28)
    check_coded(got, oracle.binarize(buf[:, 50:50 + 577]), 577)


def test_binarize_many_rows(dab):
    w = dab_synth.relu_activations((5000, 200), 0.6, stream=13)
    check_coded(dab.dab_binarize(to_dev(w)), oracle.binarize(w), 200, log=print)


@pytest.mark.parametrize("n,rows,ld_bits", [(1, 3, 1), (31, 5, 31), (33, 5, 48), (576, 64, 576), (577, 9, 592),
                                             (1000, 17, 1001), (4608, 33, 4608), (16384, 2, 16384)])
def test_pack_matches_checker(dab, n, rows, ld_bits):
    buf = (dab_synth.uniform01(3, n, 0, rows * ld_bits) < 0.4).astype(np.uint8).reshape(rows, ld_bits)
    buf[buf > 0] = np.arange(buf.sum()) % 255 + 1                # any non-zero byte counts as one
    dev = to_dev(buf)[:, :n]
    mask, K = dab.dab_pack(dev)
    ref_mask, ref_K = oracle.pack((buf[:, :n] != 0).astype(np.uint8))
    assert np.array_equal(words(mask), ref_mask) and np.array_equal(K.cpu().numpy(), ref_K)


def _coded_pair(dab, A, B):
    a, b = dab.dab_binarize(to_dev(A)), dab.dab_binarize(to_dev(B))
    ra, rb = oracle.binarize(A), oracle.binarize(B)
    check_coded(a, ra, A.shape[1])
    check_coded(b, rb, B.shape[1])
    return a, b, ra, rb


@pytest.mark.parametrize("M,N,n", [(1, 1, 1), (5, 7, 33), (64, 64, 576), (65, 63, 577), (130, 70, 1152),
                                   (257, 129, 100), (33, 200, 2400), (3, 5, 16384)])
def test_gemm_matches_checker(dab, M, N, n):
    A = _rows("relu", M, n, 21)
    B = _rows("normal", N, n, 22)
    a, b, ra, rb = _coded_pair(dab, A, B)
    Cm, p11 = dab.dab_binary_gemm(a, b, want_p11=True)
    refC, refP = oracle.gemm(ra.e, ra.alpha, ra.beta, rb.e, rb.alpha, rb.beta)
    assert np.array_equal(p11.cpu().numpy(), refP)
    assert rel_close(Cm.cpu().numpy(), refC).all()
    assert np.array_equal(dab.dab_binary_gemm(a, b).cpu().numpy(), Cm.cpu().numpy())    # without the p11 output


def test_gemm_xnor_special_case(dab):
    n = 128
    sa = np.ones((9, n)); sb = np.ones((11, n))
    for r in range(9):
        sa[r, np.argsort(dab_synth.uniform01(5, 10 + r, 0, n))[: n // 2]] = -1
    for r in range(11):
        sb[r, np.argsort(dab_synth.uniform01(5, 40 + r, 0, n))[: n // 2]] = -1
    A, B = (0.75 * sa).astype(np.float32), (0.125 * sb).astype(np.float32)
    a, b, ra, rb = _coded_pair(dab, A, B)
    Cm = dab.dab_binary_gemm(a, b).cpu().numpy()
    assert np.array_equal(Cm, (A.astype(np.float64) @ B.astype(np.float64).T).astype(np.float32))   # codes are exact here


def test_config3_smallest_point_in_full(dab):
    m, k = 1024, 576
    A, B = configs.config3_operands(m, k)
    a, b, ra, rb = _coded_pair(dab, A, B)
    Cm, p11 = dab.dab_binary_gemm(a, b, want_p11=True)
    refC, refP = oracle.gemm(ra.e, ra.alpha, ra.beta, rb.e, rb.alpha, rb.beta)
    assert np.array_equal(p11.cpu().numpy(), refP) and rel_close(Cm.cpu().numpy(), refC).all()


CONV_CASES = [
    dict(N=1, C=3, H=6, W=7, Cout=4, kh=3, kw=3, stride=(1, 1), pad=(1, 1)),
    dict(N=2, C=4, H=9, W=8, Cout=3, kh=5, kw=5, stride=(1, 1), pad=(2, 2)),
    dict(N=2, C=5, H=8, W=8, Cout=6, kh=3, kw=3, stride=(2, 2), pad=(1, 1)),
    dict(N=1, C=8, H=5, W=5, Cout=5, kh=1, kw=1, stride=(1, 1), pad=(0, 0)),
    dict(N=1, C=2, H=7, W=7, Cout=3, kh=7, kw=7, stride=(1, 1), pad=(0, 0)),
    dict(N=1, C=3, H=7, W=6, Cout=2, kh=3, kw=2, stride=(2, 1), pad=(0, 1)),
    dict(N=3, C=16, H=14, W=14, Cout=70, kh=3, kw=3, stride=(1, 1), pad=(1, 1)),
    dict(N=2, C=64, H=9, W=11, Cout=64, kh=3, kw=3, stride=(1, 1), pad=(1, 1)),
    dict(N=2, C=64, H=12, W=12, Cout=128, kh=3, kw=3, stride=(2, 2), pad=(1, 1)),
    dict(N=1, C=128, H=7, W=7, Cout=33, kh=3, kw=3, stride=(1, 1), pad=(1, 1)),
]


def _check_conv(dab, x, w, kh, kw, stride, pad, dense_w=None):
    wd = dab.dab_binarize(to_dev(w))
    wb = oracle.binarize(w)
    check_coded(wd, wb, w.shape[1])
    y, det = dab.dab_binary_conv(to_dev(x), wd, kh, kw, stride, pad, details=True)
    ref = oracle.conv(x, wb.e, wb.alpha, wb.beta, kh, kw, stride, pad)
    n = w.shape[1]
    near = (np.zeros(len(ref.p_K), bool))
    assert np.array_equal(det.pflags.cpu().numpy().view(np.uint32), ref.p_flags)
    assert np.array_equal(det.pK.cpu().numpy(), ref.p_K)
    assert np.array_equal(unpack(words(det.pmask), n), ref.p_e)
    assert rel_close(det.pgamma.cpu().numpy(), ref.p_gamma).all() and rel_close(det.pdelta.cpu().numpy(), ref.p_delta).all()
    assert np.array_equal(det.p11.cpu().numpy(), ref.p_p11)
    assert y.shape == ref.y.shape and rel_close(y.cpu().numpy(), ref.y).all()
    y2 = dab.dab_binary_conv(to_dev(x), wd, kh, kw, stride, pad)           # without the optional outputs
    assert np.array_equal(y2.cpu().numpy(), y.cpu().numpy())
    return y


@pytest.mark.parametrize("ci", range(len(CONV_CASES)))
@pytest.mark.parametrize("dense", [False, True])
def test_conv_matches_checker(dab, ci, dense):
    c = CONV_CASES[ci]
    shape = (c["N"], c["C"], c["H"], c["W"])
    x = dab_synth.dense_activations(shape, stream=60 + ci) if dense else dab_synth.relu_activations(shape, 0.6, stream=60 + ci)
    w = dab_synth.normal((c["Cout"], c["C"] * c["kh"] * c["kw"]), 0.05, stream=80 + ci)
    _check_conv(dab, x, w, c["kh"], c["kw"], c["stride"], c["pad"])


def test_config1_in_full(dab):
    L = configs.config1()[0]
    _check_conv(dab, L.inputs(), L.weights(), L.kh, L.kw, (L.stride, L.stride), (L.pad, L.pad))


@pytest.mark.parametrize("li", range(6))
def test_config2_layers_in_full(dab, li):
    L = configs.config2()[li]
    _check_conv(dab, L.inputs(stream=li), L.weights(stream=li), L.kh, L.kw, (L.stride, L.stride), (L.pad, L.pad))


def test_conv_on_stroke_image_patches(dab):
    # sparse binary sketch input: most patches are constant (all zero) -> degenerate rows, the rest two-valued
    x = dab_synth.stroke_batch(1, 2, 40, 40, stream=3)
    w = dab_synth.normal((8, 2 * 25), 0.02, stream=90)
    _check_conv(dab, x, w, 5, 5, (1, 1), (2, 2))


def test_conv_with_dense_and_sparse_regions(dab):
    # n = 576: tiles whose staged values are mostly non-zero are coded by four warps per patch, the others by one
    # warp per patch; an image that is dense on top and sparse below exercises both and the hand-over between them
    L = configs.ConvLayer("mixed", 2, 64, 24, 24, 16, 3, 3, 1, 1, 0.05)
    x = L.inputs(stream=31)
    x[:, :, :12, :] = dab_synth.dense_activations((2, 64, 12, 24), stream=32)
    x[1, :, 12:, :12] = 0.0                                      # and a block of constant (all-zero) patches
    _check_conv(dab, x, L.weights(stream=31), 3, 3, (1, 1), (1, 1))


@pytest.mark.parametrize("n", [1, 5, 31, 32, 33, 100, 576, 577, 1025, 4608, 16384])
def test_sign_coding_of_rows_matches_checker(dab, n):
    w = np.concatenate([_rows("normal", 9, n, 40 + n), _rows("relu", 3, n, 41 + n), _rows("ints", 3, n, 42 + n)])
    w[2, n // 2] = np.nan
    got = dab.dab_sign_binarize(to_dev(w))
    check_coded(got, oracle.sign_code(w), n)


@pytest.mark.parametrize("ci", [0, 1, 2, 4, 5, 7, 8])
def test_conv_with_sign_coded_inputs_matches_checker(dab, ci):
    c = CONV_CASES[ci]
    shape = (c["N"], c["C"], c["H"], c["W"])
    x = dab_synth.dense_activations(shape, stream=160 + ci)
    w = dab_synth.normal((c["Cout"], c["C"] * c["kh"] * c["kw"]), 0.05, stream=180 + ci)
    wd, wb = dab.dab_binarize(to_dev(w)), oracle.binarize(w)
    y, det = dab.dab_binary_conv(to_dev(x), wd, c["kh"], c["kw"], c["stride"], c["pad"], details=True, sign_inputs=True)
    ref = oracle.conv(x, wb.e, wb.alpha, wb.beta, c["kh"], c["kw"], c["stride"], c["pad"], sign_inputs=True)
    n = w.shape[1]
    assert np.array_equal(det.pK.cpu().numpy(), ref.p_K) and np.array_equal(unpack(words(det.pmask), n), ref.p_e)
    assert rel_close(det.pgamma.cpu().numpy(), ref.p_gamma).all() and rel_close(det.pdelta.cpu().numpy(), ref.p_delta).all()
    assert np.array_equal(det.p11.cpu().numpy(), ref.p_p11)
    # gamma, delta: the fp64 sum of |x| over the row is formed in another order than the checker's; it is exact
    # (hence equal) unless the row mixes magnitudes more than 2^29 apart, so the scales agree to the bit here and
    # the outputs, formed from them by the same fp64 expression, meet the 1e-5 bound everywhere
    assert np.array_equal(det.pgamma.cpu().numpy(), ref.p_gamma) and np.array_equal(det.pdelta.cpu().numpy(), ref.p_delta)
    assert rel_close(y.cpu().numpy(), ref.y).all()


@pytest.mark.parametrize("batch", [1, 2, 19])
def test_conv_host_entry_point(dab, batch):
    # host tensors in and out; the batch is pipelined in chunks (19 images: 10 chunks of 2, the last one ragged)
    L = configs.ConvLayer("t", batch, 16, 12, 12, 24, 3, 3, 1, 1)
    x, w = L.inputs(stream=5), L.weights(stream=5)
    wd = dab.dab_binarize(to_dev(w))
    y_dev = dab.dab_binary_conv(to_dev(x), wd, 3, 3, (1, 1), (1, 1)).cpu()
    for _ in range(2):                                           # twice: the copy streams and events are reused
        y_host = dab.dab_binary_conv_host(torch.from_numpy(x).pin_memory(), wd, 3, 3, (1, 1), (1, 1))
        assert torch.equal(y_host, y_dev)
    y_pageable = dab.dab_binary_conv_host(torch.from_numpy(x), wd, 3, 3, (1, 1), (1, 1),
                                          y_host=torch.empty_like(y_dev))
    assert torch.equal(y_pageable, y_dev)


def test_conv_host_layers_queued_without_waiting(dab):
    # five layers queued back to back: alternating workspaces (they may overlap on the device), then one shared
    # workspace (each call must wait for the one before it); every output equals the device-resident call
    shapes = [(7, 16, 12, 12, 24), (5, 8, 20, 20, 16), (9, 32, 9, 9, 8), (4, 16, 12, 12, 24), (6, 8, 20, 20, 16)]
    layers = [configs.ConvLayer("q%d" % i, *sh, 3, 3, 1, 1) for i, sh in enumerate(shapes)]
    xs = [torch.from_numpy(L.inputs(stream=30 + i)).pin_memory() for i, L in enumerate(layers)]
    wds = [dab.dab_binarize(to_dev(L.weights(stream=30 + i))) for i, L in enumerate(layers)]
    refs = [dab.dab_binary_conv(x.cuda(), wd, 3, 3, (1, 1), (1, 1)).cpu() for x, wd in zip(xs, wds)]
    descs = [dab.make_desc(L.x_shape(), L.Cout, 3, 3, (1, 1), (1, 1)) for L in layers]
    need = max(dab.dab_binary_conv_host_workspace(d) for d in descs)
    for n_ws in (2, 1):
        wss = [torch.empty(need, dtype=torch.uint8, device="cuda") for _ in range(n_ws)]
        ys = [torch.empty_like(r).pin_memory() for r in refs]
        for rep in range(2):
            for i, (x, wd) in enumerate(zip(xs, wds)):
                dab.dab_binary_conv_host(x, wd, 3, 3, (1, 1), (1, 1), y_host=ys[i], workspace=wss[i % n_ws], wait=False)
            dab.dab_binary_conv_host_wait()
            for y, r in zip(ys, refs):
                assert torch.equal(y, r)
                y.zero_()
    with pytest.raises(ValueError):
        dab.dab_binary_conv_host(xs[0], wds[0], 3, 3, (1, 1), (1, 1), wait=False)


def test_argument_errors_are_return_codes(dab):
    import ctypes as C
    L = dab.lib()
    v = torch.zeros((4, 64), device="cuda")
    m = torch.zeros((4, 4), dtype=torch.int32, device="cuda")
    k = torch.zeros(4, dtype=torch.int32, device="cuda")
    a = torch.zeros(4, device="cuda")
    p = lambda t: C.c_void_p(t.data_ptr())
    call = lambda rows, n, ldv, ldm, mask=m: L.dab_binarize(p(v), rows, n, ldv, p(k), p(a), p(a), p(mask), ldm, None, None)
    assert call(4, 64, 64, 4) == 0
    assert call(0, 64, 64, 4) == 0                               # rows == 0 is a no-op
    assert call(-1, 64, 64, 4) == 1 and call(4, 0, 64, 4) == 1   # invalid
    assert call(4, 64, 63, 4) == 1                               # ld_values < n
    assert call(4, 64, 64, 1) == 1 and call(4, 64, 64, 6) == 1   # ld_mask too small / not a multiple of 4
    assert call(4, 16385, 16385, 516) == 2                       # beyond DAB_MAX_N
    assert L.dab_binarize(None, 4, 64, 64, p(k), p(a), p(a), p(m), 4, None, None) == 1
    mis = torch.zeros(20, dtype=torch.int32, device="cuda")[1:17].view(4, 4)
    assert call(4, 64, 64, 4, mask=mis) == 1                     # mask not 16-byte aligned
    d = dab.make_desc((1, 3, 8, 8), 4, 3, 3, (1, 1), (1, 1))
    assert dab.dab_binary_conv_workspace(d) > 0
    bad = dab.make_desc((1, 3, 2, 2), 4, 5, 5)
    assert dab.dab_binary_conv_workspace(bad) == 0
    x = torch.zeros((1, 3, 8, 8), device="cuda")
    y = torch.zeros((1, 4, 8, 8), device="cuda")
    st = L.dab_binary_conv(C.byref(d), p(x), p(m), 4, p(k), p(a), p(a), p(y), None, 0, None, None, None, None, 0, None, None, None)
    assert st == 3                                               # workspace missing
    torch.cuda.synchronize()

"""The patch coders (full sort, histogram-pruned search, the default choice between them by tile density) must give
the same codes bit for bit, and the histogram coder must match the CPU checker on its own."""
import numpy as np
import pytest
import torch

import dab_synth
import oracle
from parity_util import NEAR_TIE, to_dev, unpack, words

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def dab():
    import paper_1804_02941_b200 as d
    d.lib()
    oracle.set_threads(8)
    yield d
    d.dab_set_patch_coder(d.PATCHES_AUTO)


def _code(dab, x, C, kh, kw, stride, pad, coder):
    dab.dab_set_patch_coder(coder)
    desc = dab.make_desc(tuple(x.shape), 8, kh, kw, stride, pad)
    Ho, Wo = dab.dab_conv_output_size(desc)
    P, n = x.shape[0] * Ho * Wo, C * kh * kw
    ld = dab.dab_default_ld(n)
    dev = x.device
    pK = torch.full((P,), -7, dtype=torch.int32, device=dev)
    pg, pd = torch.zeros(P, device=dev), torch.zeros(P, device=dev)
    pm = torch.zeros((P, ld), dtype=torch.int32, device=dev)
    pf = torch.zeros(P, dtype=torch.int32, device=dev)
    dab.dab_binarize_patches(desc, x, pK, pg, pd, pm, pf)
    torch.cuda.synchronize()
    dab.dab_set_patch_coder(dab.PATCHES_AUTO)
    return pK, pg, pd, pm, pf


CASES = [
    # N, C, H, W, kh, kw, stride, pad, kind
    (2, 64, 20, 20, 3, 3, (1, 1), (1, 1), "relu"),        # n = 576
    (2, 64, 21, 21, 3, 3, (2, 2), (1, 1), "relu"),
    (1, 128, 14, 14, 3, 3, (1, 1), (1, 1), "relu"),       # n = 1152
    (1, 256, 9, 9, 3, 3, (1, 1), (1, 1), "relu"),         # n = 2304
    (1, 512, 7, 7, 3, 3, (1, 1), (1, 1), "relu"),         # n = 4608
    (2, 64, 12, 12, 3, 3, (1, 1), (1, 1), "normal"),      # both signs, no zeros
    (2, 40, 11, 13, 5, 5, (1, 1), (2, 2), "relu"),        # 5x5 window (general path), n = 1000
    (1, 70, 9, 9, 3, 3, (1, 1), (0, 0), "sparse"),        # 95 % zeros, C not a multiple of 32
    (1, 64, 10, 10, 3, 3, (1, 1), (1, 1), "negative"),    # no positive value
    (1, 64, 10, 10, 3, 3, (1, 1), (1, 1), "ints"),        # few distinct values: exact ties, constant patches
]


def _input(kind, shape, stream):
    if kind == "relu":
        return dab_synth.relu_activations(shape, 0.6, stream=stream)
    if kind == "normal":
        return dab_synth.normal(shape, 1.0, stream=stream)
    if kind == "sparse":
        return dab_synth.relu_activations(shape, 0.95, stream=stream)
    if kind == "negative":
        return -dab_synth.relu_activations(shape, 0.5, stream=stream)
    x = np.round(dab_synth.normal(shape, 1.2, stream=stream))
    x[:, :, :4, :4] = 2.0                                   # constant non-zero patches
    return x


@pytest.mark.parametrize("ci", range(len(CASES)))
def test_histogram_coder_equals_sort_coder_and_checker(dab, ci):
    N, C, H, W, kh, kw, stride, pad, kind = CASES[ci]
    x = _input(kind, (N, C, H, W), 950 + ci).astype(np.float32)
    xd = to_dev(x)
    a = _code(dab, xd, C, kh, kw, stride, pad, dab.PATCHES_SORT)
    b = _code(dab, xd, C, kh, kw, stride, pad, dab.PATCHES_HIST)
    c = _code(dab, xd, C, kh, kw, stride, pad, dab.PATCHES_AUTO)
    px = _code(dab, xd, C, kh, kw, stride, pad, dab.PATCHES_PIXEL)
    for s, h, au, pp in zip(a, b, c, px):
        assert torch.equal(s, h) and torch.equal(s, au) and torch.equal(s, pp)
    n = C * kh * kw
    rows = oracle.im2col(x, kh, kw, stride, pad)
    sel = np.unique(np.concatenate([[0, len(rows) - 1], (dab_synth.uniform01(96, ci, 0, 64) * len(rows)).astype(np.int64)]))
    ref = oracle.binarize(rows[sel])
    strict = ~((ref.gap > 0) & (ref.gap < NEAR_TIE))
    t = torch.from_numpy(sel).to(xd.device)
    assert np.array_equal(b[0][t].cpu().numpy()[strict], ref.K[strict])
    assert np.array_equal(unpack(words(b[3][t]), n)[strict], ref.e[strict])
    assert np.array_equal(b[4][t].cpu().numpy().view(np.uint32)[strict], ref.flags[strict])


def test_nonfinite_tiles_fall_back(dab):
    x = dab_synth.relu_activations((1, 64, 12, 12), 0.6, stream=990).astype(np.float32)
    x[0, 3, 5, 5] = np.nan
    x[0, 9, 0, 11] = np.inf
    xd = to_dev(x)
    a = _code(dab, xd, 64, 3, 3, (1, 1), (1, 1), dab.PATCHES_SORT)
    b = _code(dab, xd, 64, 3, 3, (1, 1), (1, 1), dab.PATCHES_HIST)
    c = _code(dab, xd, 64, 3, 3, (1, 1), (1, 1), dab.PATCHES_AUTO)
    px = _code(dab, xd, 64, 3, 3, (1, 1), (1, 1), dab.PATCHES_PIXEL)
    assert torch.equal(a[0], px[0]) and torch.equal(a[3], px[3]) and torch.equal(a[4], px[4])
    assert torch.equal(a[0], b[0]) and torch.equal(a[3], b[3]) and torch.equal(a[4], b[4])
    assert torch.equal(a[0], c[0]) and torch.equal(a[3], c[3]) and torch.equal(a[4], c[4])
    assert int((b[4] == 2).sum()) == 9 + 4


def test_mixed_density_batches_split_between_the_coders(dab):
    # images of very different density in one call: every tile goes to one coder or the other
    x = np.concatenate([dab_synth.relu_activations((1, 128, 14, 14), z, stream=995 + i) for i, z in
                        enumerate((0.9, 0.6, 0.5, 0.3, 0.0))]).astype(np.float32)
    x[4] = dab_synth.normal((128, 14, 14), 1.0, stream=999)
    xd = to_dev(x)
    a = _code(dab, xd, 128, 3, 3, (1, 1), (1, 1), dab.PATCHES_SORT)
    c = _code(dab, xd, 128, 3, 3, (1, 1), (1, 1), dab.PATCHES_AUTO)
    px = _code(dab, xd, 128, 3, 3, (1, 1), (1, 1), dab.PATCHES_PIXEL)
    for s, au, pp in zip(a, c, px):
        assert torch.equal(s, au) and torch.equal(s, pp)
    x64 = np.ascontiguousarray(x[:, :64])
    a = _code(dab, to_dev(x64), 64, 3, 3, (1, 1), (1, 1), dab.PATCHES_SORT)
    c = _code(dab, to_dev(x64), 64, 3, 3, (1, 1), (1, 1), dab.PATCHES_AUTO)
    for s, au in zip(a, c):
        assert torch.equal(s, au)


@pytest.mark.parametrize("C", [128, 256, 512])
def test_pixel_coder_regions_of_one_sign_and_of_both_in_one_image(dab, C):
    # rows of 1024 values and more: tiles of one sign (either one) are coded by the first launch, tiles with both signs
    # by the second; the regions meet inside tiles as well
    x = dab_synth.relu_activations((2, C, 16, 16), 0.6, stream=1200 + C).astype(np.float32)
    x[:, :, :, 9:] = dab_synth.normal((2, C, 16, 7), 1.0, stream=1300 + C)
    x[1, :, :7, :9] = -x[1, :, :7, :9]
    xd = to_dev(x)
    a = _code(dab, xd, C, 3, 3, (1, 1), (1, 1), dab.PATCHES_SORT)
    px = _code(dab, xd, C, 3, 3, (1, 1), (1, 1), dab.PATCHES_PIXEL)
    for s, pp in zip(a, px):
        assert torch.equal(s, pp)
    n = C * 9
    rows = oracle.im2col(x, 3, 3, (1, 1), (1, 1))
    sel = np.unique((dab_synth.uniform01(97, C, 0, 96) * len(rows)).astype(np.int64))
    ref = oracle.binarize(rows[sel])
    strict = ~((ref.gap > 0) & (ref.gap < NEAR_TIE))
    t = torch.from_numpy(sel).to(xd.device)
    assert np.array_equal(px[0][t].cpu().numpy()[strict], ref.K[strict])
    assert np.array_equal(unpack(words(px[3][t]), n)[strict], ref.e[strict])


@pytest.mark.parametrize("n", [257, 300, 575, 576, 577, 1024, 1152, 1600, 2304, 4096, 4608, 8192])
@pytest.mark.parametrize("kind", ["normal", "relu", "laplace", "ints", "cluster", "negative"])
def test_rows_of_a_matrix_through_both_coders(dab, n, kind):
    # dab_binarize: the histogram-pruned search against the sorting kernels and against the checker
    from parity_util import check_coded
    rows = 40 if n <= 2304 else 12
    if kind == "normal":
        w = dab_synth.normal((rows, n), 0.05, stream=n)
    elif kind == "relu":
        w = dab_synth.relu_activations((rows, n), 0.6, stream=n)
    elif kind == "laplace":
        w = dab_synth.laplace((rows, n), 0.05, stream=n)
    elif kind == "ints":
        w = dab_synth.small_integer_rows(rows, n, -3, 3, stream=n)
    elif kind == "cluster":
        w = dab_synth.two_cluster_rows(rows, n, stream=n)
    else:
        w = -dab_synth.relu_activations((rows, n), 0.3, stream=n)
    w = np.ascontiguousarray(w, np.float32)
    w[0, :] = 0.25                                   # a constant row
    w[1, :] = 0.0                                    # a row of zeros
    w[2, 5] = np.nan                                 # a non-finite row
    wd = to_dev(w)
    outs = {}
    for coder in (dab.PATCHES_SORT, dab.PATCHES_HIST, dab.PATCHES_AUTO):
        dab.dab_set_patch_coder(coder)
        outs[coder] = dab.dab_binarize(wd)
    dab.dab_set_patch_coder(dab.PATCHES_AUTO)
    torch.cuda.synchronize()
    s, h, au = outs[dab.PATCHES_SORT], outs[dab.PATCHES_HIST], outs[dab.PATCHES_AUTO]
    for name in ("K", "mask", "flags"):
        assert torch.equal(getattr(s, name), getattr(h, name)) and torch.equal(getattr(s, name), getattr(au, name)), name
    ok = (s.flags == 0)
    assert torch.equal(s.alpha[ok], h.alpha[ok]) and torch.equal(s.beta[ok], h.beta[ok])
    check_coded(h, oracle.binarize(w), n, log=print)


def test_large_dense_matrix_takes_the_histogram_search_by_default(dab):
    # 2048 rows: the default choice runs the histogram kernel; sparse and dense rows mixed in one matrix
    from parity_util import check_coded
    n = 1152
    w = np.concatenate([dab_synth.laplace((1024, n), 0.05, stream=61), dab_synth.relu_activations((1024, n), 0.6, stream=62)])
    w = np.ascontiguousarray(w[np.argsort(dab_synth.uniform01(3, 9, 0, 2048))], np.float32)    # interleave them
    wd = to_dev(w)
    dab.dab_set_patch_coder(dab.PATCHES_SORT)
    s = dab.dab_binarize(wd)
    dab.dab_set_patch_coder(dab.PATCHES_AUTO)
    au = dab.dab_binarize(wd)
    torch.cuda.synchronize()
    for name in ("K", "mask", "flags", "alpha", "beta"):
        assert torch.equal(getattr(s, name), getattr(au, name)), name
    sel = np.arange(0, 2048, 37)
    sub = dab.Coded(au.mask[sel], au.K[sel], au.alpha[sel], au.beta[sel], au.flags[sel], n)
    check_coded(sub, oracle.binarize(w[sel]), n, log=print)

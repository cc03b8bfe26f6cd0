"""GPU parity of dab_wbin_conv (weights-only binarized convolution, Section 4.3.2) against the CPU checker.

Tolerance.  The kernel takes each patch as 32-bit fixed point relative to its largest magnitude m and forms the
sums exactly in integers, so against exact arithmetic
    |y - y_exact| <= 2^-32 * n * m * max(|alpha|, |beta|)        (rounding of the n values, half a unit each)
plus the fp64 roundings of the two products and the final rounding to fp32 (2^-24 |y|).  The tests allow twice
that bound, and check the task-level figure of 1e-5 relative to the sum of the magnitudes of the terms as well.
"""
import numpy as np
import pytest
import torch

import dab_synth
import oracle
from parity_util import to_dev

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def dab():
    import paper_1804_02941_b200 as d
    d.lib()
    oracle.set_threads(8)
    return d


def _patch_max(x, kh, kw, stride, pad):
    m = torch.from_numpy(np.abs(x)).amax(dim=1, keepdim=True)
    return torch.nn.functional.max_pool2d(m, (kh, kw), stride=stride, padding=pad).numpy()   # N x 1 x Ho x Wo


def _check(dab, x, w, kh, kw, stride, pad):
    wb = oracle.binarize(w)
    ref, mag = oracle.conv_wbin(x, wb.e, wb.alpha, wb.beta, kh, kw, stride, pad)
    coded = dab.dab_binarize(to_dev(w))
    assert np.array_equal(coded.K.cpu().numpy(), wb.K)
    got = dab.dab_wbin_conv(to_dev(x), coded, kh, kw, stride, pad)
    torch.cuda.synchronize()
    assert dab.dab_contraction_wait_failures() == 0
    got = got.cpu().numpy().astype(np.float64)
    assert got.shape == ref.shape
    n = w.shape[1]
    wmax = np.maximum(np.abs(wb.alpha), np.abs(wb.beta)).astype(np.float64)[None, :, None, None]
    # max_pool2d pads with -inf, |x| >= 0, so padding never raises the maximum
    bound = 2.0 ** -31 * n * _patch_max(x, kh, kw, stride, pad) * wmax + 2.0 ** -23 * np.abs(ref) + 1e-300
    err = np.abs(got - ref.astype(np.float64))
    assert np.all(err <= bound), "beyond the fixed-point bound: worst ratio %g" % np.max(err / bound)
    assert np.all(err <= 1e-5 * mag + 1e-300), "beyond 1e-5 of the sum of magnitudes"
    return got, ref


CASES = [
    dict(N=1, C=3, H=6, W=7, Cout=4, kh=3, kw=3, stride=(1, 1), pad=(1, 1)),
    dict(N=2, C=4, H=9, W=8, Cout=3, kh=5, kw=5, stride=(1, 1), pad=(2, 2)),
    dict(N=2, C=5, H=8, W=8, Cout=6, kh=3, kw=3, stride=(2, 2), pad=(1, 1)),
    dict(N=1, C=8, H=5, W=5, Cout=5, kh=1, kw=1, stride=(1, 1), pad=(0, 0)),
    dict(N=1, C=3, H=7, W=6, Cout=2, kh=3, kw=2, stride=(2, 1), pad=(0, 1)),
    dict(N=1, C=64, H=32, W=32, Cout=64, kh=3, kw=3, stride=(1, 1), pad=(1, 1)),      # the single-layer config
    dict(N=3, C=16, H=19, W=37, Cout=70, kh=3, kw=3, stride=(1, 1), pad=(1, 1)),      # ragged tiles, two filter tiles
    dict(N=2, C=40, H=14, W=14, Cout=130, kh=3, kw=3, stride=(1, 1), pad=(1, 1)),     # three filter tiles, n = 360
    dict(N=2, C=24, H=29, W=29, Cout=32, kh=3, kw=3, stride=(2, 2), pad=(1, 1)),
    dict(N=2, C=6, H=20, W=20, Cout=16, kh=5, kw=5, stride=(1, 1), pad=(2, 2)),
    dict(N=1, C=2, H=7, W=7, Cout=3, kh=7, kw=7, stride=(1, 1), pad=(0, 0)),          # one output position
    dict(N=4, C=300, H=5, W=5, Cout=20, kh=1, kw=1, stride=(1, 1), pad=(0, 0)),       # 1x1: many channels per stage
    dict(N=1, C=128, H=7, W=7, Cout=64, kh=3, kw=3, stride=(1, 1), pad=(1, 1)),       # n = 1152, nine stages
]


@pytest.mark.parametrize("signed", [False, True])
@pytest.mark.parametrize("ci", range(len(CASES)))
def test_wbin_conv_matches_checker(dab, ci, signed):
    c = CASES[ci]
    shape = (c["N"], c["C"], c["H"], c["W"])
    x = dab_synth.normal(shape, 1.0, stream=400 + ci) if signed else dab_synth.relu_activations(shape, 0.6, stream=400 + ci)
    w = dab_synth.normal((c["Cout"], c["C"] * c["kh"] * c["kw"]), 0.05, stream=420 + ci)
    _check(dab, x.astype(np.float32), w, c["kh"], c["kw"], c["stride"], c["pad"])


def test_small_integers_are_exact(dab):
    # integer activations and dyadic levels: every sum is exact, so the result must be the checker's bit for bit
    x = np.round(dab_synth.normal((2, 8, 12, 12), 6.0, stream=440)).astype(np.float32)
    e = (dab_synth.uniform01(7, 1, 0, 10 * 72).reshape(10, 72) < 0.4)
    w = np.where(e, 0.75, -0.25).astype(np.float32)                 # codes exactly: alpha = 0.75, beta = -0.25
    got, ref = _check(dab, x, w, 3, 3, (1, 1), (1, 1))
    assert np.array_equal(got.astype(np.float32), ref)


def test_wide_dynamic_range_zero_patches_and_huge_values(dab):
    x = dab_synth.normal((2, 6, 10, 10), 1.0, stream=441).astype(np.float32)
    x[0, :, :5, :] = 0.0                        # patches of zeros only
    x[0, 2, 7, 7] = 3.0e30                      # one huge value: its patches are scaled to it
    x[1] *= np.float32(1e-30)                   # tiny image
    x[1, 0, 0, 0] = np.float32(1e-42)           # a subnormal
    w = dab_synth.normal((5, 54), 0.05, stream=442)
    got, ref = _check(dab, x, w, 3, 3, (1, 1), (1, 1))
    assert np.all(got[0, :, :3, :] == 0.0)


def test_nonfinite_patches_give_nan_and_spare_the_others(dab):
    x = dab_synth.relu_activations((1, 4, 9, 9), 0.5, stream=443).astype(np.float32)
    x[0, 1, 4, 4] = np.inf
    x[0, 3, 0, 8] = np.nan
    w = dab_synth.normal((6, 36), 0.05, stream=444)
    wb = oracle.binarize(w)
    got = dab.dab_wbin_conv(to_dev(x), dab.dab_binarize(to_dev(w)), 3, 3, (1, 1), (1, 1)).cpu().numpy()
    touched = np.zeros((9, 9), bool)
    touched[3:6, 3:6] = True
    touched[0:2, 7:9] = True
    assert np.isnan(got[0][:, touched]).all()
    clean = np.where(np.isfinite(x), x, 0.0).astype(np.float32)
    ref, mag = oracle.conv_wbin(clean, wb.e, wb.alpha, wb.beta, 3, 3, (1, 1), (1, 1))
    ok = ~touched
    assert np.all(np.abs(got[0][:, ok] - ref[0][:, ok]) <= 1e-5 * mag[0][:, ok] + 1e-300)


def test_rejects_bad_arguments(dab):
    L = dab.lib()
    desc = dab.make_desc((1, 4, 8, 8), 4, 3, 3, (1, 1), (1, 1))
    import ctypes as C
    assert L.dab_wbin_conv(C.byref(desc), None, None, 4, None, None, None, None, 0, None) == 1
    x = torch.zeros((1, 4, 8, 8), device="cuda")
    m = torch.zeros((4, 4), dtype=torch.int32, device="cuda")
    a = torch.zeros(4, device="cuda")
    y = torch.zeros((1, 4, 8, 8), device="cuda")
    ws = torch.zeros(dab.dab_wbin_conv_workspace(desc), dtype=torch.uint8, device="cuda")
    args = (x.data_ptr(), m.data_ptr())
    tail = (a.data_ptr(), a.data_ptr(), y.data_ptr())
    assert L.dab_wbin_conv(C.byref(desc), *args, 1, *tail, ws.data_ptr(), ws.numel(), None) == 1       # ld too short
    assert L.dab_wbin_conv(C.byref(desc), *args, 6, *tail, ws.data_ptr(), ws.numel(), None) == 1       # ld not a multiple of 4
    assert L.dab_wbin_conv(C.byref(desc), *args, 4, *tail, ws.data_ptr(), ws.numel() - 1, None) == 3   # scratch too small
    assert L.dab_wbin_conv(C.byref(desc), *args, 4, *tail, None, ws.numel(), None) == 3
    assert L.dab_wbin_conv(C.byref(desc), *args, 4, *tail, ws.data_ptr(), ws.numel(), None) == 0


@pytest.mark.parametrize("name", ["l1_0", "l2_0", "l2_1", "l3_1", "l4_0", "l4_1"])
def test_config5_layers_at_batch_256_on_sampled_images(dab, name):
    # the launch the sweep times (whole layer, batch 256); the checker recomputes three whole images of it
    from dab_synth import configs
    L = next(l for l in configs.config5(256) if l.name == name)
    x, w = L.inputs(stream=11), L.weights(stream=11)
    wb = oracle.binarize(w)
    got = dab.dab_wbin_conv(to_dev(x), dab.dab_binarize(to_dev(w)), L.kh, L.kw, (L.stride,) * 2, (L.pad,) * 2)
    torch.cuda.synchronize()
    assert dab.dab_contraction_wait_failures() == 0
    assert bool(torch.isfinite(got).all())
    for img in (0, 131, 255):
        ref, mag = oracle.conv_wbin(x[img:img + 1], wb.e, wb.alpha, wb.beta, L.kh, L.kw, (L.stride,) * 2, (L.pad,) * 2)
        err = np.abs(got[img:img + 1].cpu().numpy().astype(np.float64) - ref)
        assert np.all(err <= 1e-5 * mag + 1e-300)
        assert np.all(err <= 2.0 ** -31 * L.n * float(np.abs(x[img]).max()) * float(np.abs(np.r_[wb.alpha, wb.beta]).max())
                      + 2.0 ** -23 * np.abs(ref))


def test_config4_and_config2_shapes(dab):
    # 5x5 and 6x6 / 7x7 kernels, 1x1 "fully connected" layers, batch 1 and batch 128
    from dab_synth import configs
    for L in list(configs.config2()) + [configs.config4(128)[i] for i in (0, 4, 5)]:
        x, w = L.inputs(stream=12), L.weights(stream=12)
        sel = slice(0, min(L.N, 2))
        wb = oracle.binarize(w)
        got = dab.dab_wbin_conv(to_dev(x), dab.dab_binarize(to_dev(w)), L.kh, L.kw, (L.stride,) * 2, (L.pad,) * 2)
        torch.cuda.synchronize()
        ref, mag = oracle.conv_wbin(x[sel], wb.e, wb.alpha, wb.beta, L.kh, L.kw, (L.stride,) * 2, (L.pad,) * 2)
        err = np.abs(got[sel].cpu().numpy().astype(np.float64) - ref)
        assert np.all(err <= 1e-5 * mag + 1e-300), L.name
    assert dab.dab_contraction_wait_failures() == 0

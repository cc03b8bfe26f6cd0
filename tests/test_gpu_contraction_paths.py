"""GPU parity of the two contraction kernels, each forced: tensor cores and population counts.

Both must give the checker's AND-popcounts bit for bit, outputs within 1e-5 relative, and, because they share
the rescale arithmetic, outputs identical to each other.  Shapes cover one and several column tiles (256
weight rows per tile), ragged tails on both sides, one and many K stages, and both output layouts.
"""
import contextlib

import numpy as np
import pytest

import dab_synth
import oracle
from parity_util import rel_close, to_dev

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def dab():
    import paper_1804_02941_b200 as d
    d.lib()
    oracle.set_threads(8)
    yield d
    d.dab_set_contraction(d.CONTRACT_AUTO)


@contextlib.contextmanager
def contraction(dab, path):
    before = dab.dab_get_contraction()
    dab.dab_set_contraction(path)
    try:
        yield
    finally:
        dab.dab_set_contraction(before)


def test_default_is_automatic_and_setter_validates(dab):
    assert dab.dab_get_contraction() == dab.CONTRACT_AUTO
    for path in (dab.CONTRACT_POPC, dab.CONTRACT_TENSOR):
        with contraction(dab, path):
            assert dab.dab_get_contraction() == path
    assert dab.dab_get_contraction() == dab.CONTRACT_AUTO
    with pytest.raises(dab.DabError):
        dab.dab_set_contraction(7)
    assert dab.dab_get_contraction() == dab.CONTRACT_AUTO


GEMM_SHAPES = [(1, 1, 1), (3, 2, 31), (128, 16, 32), (129, 17, 33), (300, 80, 576), (130, 64, 1152), (257, 300, 4608),
               (700, 513, 96), (40, 1030, 200), (5, 3, 16384), (1000, 256, 2304)]


@pytest.mark.parametrize("M,N,n", GEMM_SHAPES)
def test_gemm_counts_and_outputs_on_both_kernels(dab, M, N, n):
    A = dab_synth.relu_activations((M, n), 0.6, stream=300 + M)
    B = dab_synth.normal((N, n), 0.05, stream=400 + N)
    ra, rb = oracle.binarize(A), oracle.binarize(B)
    refC, refP = oracle.gemm(ra.e, ra.alpha, ra.beta, rb.e, rb.alpha, rb.beta)
    a, b = dab.dab_binarize(to_dev(A)), dab.dab_binarize(to_dev(B))
    out = {}
    for path in (dab.CONTRACT_TENSOR, dab.CONTRACT_POPC):
        with contraction(dab, path):
            Cm, p11 = dab.dab_binary_gemm(a, b, want_p11=True)
        assert np.array_equal(p11.cpu().numpy(), refP), "AND-popcounts differ on path %d" % path
        assert rel_close(Cm.cpu().numpy(), refC).all()
        out[path] = Cm.cpu().numpy()
    assert np.array_equal(out[dab.CONTRACT_TENSOR].view(np.uint32), out[dab.CONTRACT_POPC].view(np.uint32))


CONV_CASES = [
    dict(N=2, C=4, H=9, W=8, Cout=3, kh=5, kw=5, stride=(1, 1), pad=(2, 2)),
    dict(N=3, C=16, H=14, W=14, Cout=70, kh=3, kw=3, stride=(1, 1), pad=(1, 1)),
    dict(N=2, C=64, H=12, W=12, Cout=300, kh=3, kw=3, stride=(2, 2), pad=(1, 1)),
    dict(N=5, C=32, H=13, W=13, Cout=64, kh=3, kw=3, stride=(1, 1), pad=(1, 1)),   # 845 patches: tiles straddle images
]


@pytest.mark.parametrize("ci", range(len(CONV_CASES)))
def test_conv_counts_and_outputs_on_both_kernels(dab, ci):
    c = CONV_CASES[ci]
    x = dab_synth.relu_activations((c["N"], c["C"], c["H"], c["W"]), 0.6, stream=500 + ci)
    w = dab_synth.normal((c["Cout"], c["C"] * c["kh"] * c["kw"]), 0.05, stream=520 + ci)
    wb = oracle.binarize(w)
    ref = oracle.conv(x, wb.e, wb.alpha, wb.beta, c["kh"], c["kw"], c["stride"], c["pad"])
    wd = dab.dab_binarize(to_dev(w))
    out = {}
    for path in (dab.CONTRACT_TENSOR, dab.CONTRACT_POPC):
        with contraction(dab, path):
            y, det = dab.dab_binary_conv(to_dev(x), wd, c["kh"], c["kw"], c["stride"], c["pad"], details=True)
        assert np.array_equal(det.p11.cpu().numpy(), ref.p_p11)
        assert rel_close(y.cpu().numpy(), ref.y).all()
        out[path] = y.cpu().numpy()
    assert np.array_equal(out[dab.CONTRACT_TENSOR].view(np.uint32), out[dab.CONTRACT_POPC].view(np.uint32))


def test_no_barrier_wait_ran_out(dab):
    assert dab.dab_contraction_wait_failures() == 0

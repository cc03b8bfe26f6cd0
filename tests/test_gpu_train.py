"""GPU parity of dab_binarize_train (Algorithm 2 steps 4-13) and dab_binarize_backward (Theorem 4) against the
CPU checker: the mean-centred, clamped weights and the codes bit for bit, the gradient within 1e-5 relative."""
import numpy as np
import pytest
import torch

import dab_synth
import oracle
from parity_util import rel_close, to_dev, unpack, words

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def dab():
    import paper_1804_02941_b200 as d
    d.lib()
    return d


def _layers():
    # (filters, n): the four layer shapes of the ResNet-18-like stack, a 5x5 layer, odd sizes, one long row
    return [(64, 576), (128, 1152), (256, 2304), (512, 4608), (128, 1600), (37, 27), (5, 1), (3, 33), (2, 9216)]


@pytest.mark.parametrize("shape", _layers())
@pytest.mark.parametrize("std,mean", [(0.02, 0.003), (0.7, -0.2)])      # the second one reaches the clamp
def test_forward_matches_checker(dab, shape, std, mean):
    rows, n = shape
    W = dab_synth.normal((rows, n), std, stream=600 + n, mean=mean)
    Wc_r, e_r, K_r, a_r, b_r, f_r, Wt_r = oracle.train_forward(W)
    Wc, coded, Wt = dab.dab_binarize_train(to_dev(W))
    torch.cuda.synchronize()
    assert np.array_equal(Wc.cpu().numpy(), Wc_r)
    assert np.array_equal(coded.K.cpu().numpy(), K_r)
    assert np.array_equal(coded.flags.cpu().numpy().view(np.uint32), f_r)
    assert np.array_equal(unpack(words(coded.mask), n), e_r)
    assert rel_close(coded.alpha.cpu().numpy(), a_r).all() and rel_close(coded.beta.cpu().numpy(), b_r).all()
    ok = (f_r == 0)[:, None] & np.ones((1, n), bool)
    assert rel_close(Wt.cpu().numpy()[ok], Wt_r[ok]).all()
    if std > 0.5 and n > 100:
        assert (np.abs(Wc_r) == 1.0).any()


@pytest.mark.parametrize("shape", _layers())
def test_backward_matches_checker(dab, shape):
    rows, n = shape
    W = dab_synth.normal((rows, n), 0.3, stream=700 + n, mean=0.05)
    g = dab_synth.normal((rows, n), 1.0, stream=800 + n)
    Wc_r, e_r, K_r, *_ = oracle.train_forward(W)
    _, gw_r = oracle.theorem4(Wc_r, e_r, K_r, grad_Wt=g)
    Wc, coded, _ = dab.dab_binarize_train(to_dev(W), want_dense=False)
    gw = dab.dab_binarize_backward(Wc, coded, to_dev(g))
    torch.cuda.synchronize()
    assert np.array_equal(coded.K.cpu().numpy(), K_r)
    assert rel_close(gw.cpu().numpy(), gw_r).all()


def test_constant_rows_and_in_place_update(dab):
    W = np.concatenate([np.full((1, 40), 0.3, np.float32), dab_synth.normal((2, 40), 0.1, stream=900)])
    Wd = to_dev(W)
    Wc, coded, Wt = dab.dab_binarize_train(Wd)
    assert not Wc[0].any() and int(coded.K[0]) == 0 and int(coded.flags[0]) == 1 and not Wt[0].any()
    gw = dab.dab_binarize_backward(Wc, coded, torch.ones_like(Wc))
    assert not gw[0].any() and bool((gw[1:] != 0).all())
    # in place: d_Wc = d_W with equal strides
    import ctypes as C
    L = dab.lib()
    ld = dab.dab_default_ld(40)
    m = torch.empty((3, ld), dtype=torch.int32, device="cuda")
    K = torch.empty(3, dtype=torch.int32, device="cuda")
    a, b = torch.empty(3, device="cuda"), torch.empty(3, device="cuda")
    p = lambda t: C.c_void_p(t.data_ptr())
    assert L.dab_binarize_train(p(Wd), 3, 40, 40, p(Wd), 40, None, 0, p(K), p(a), p(b), p(m), ld, None, None) == 0
    torch.cuda.synchronize()
    assert torch.equal(Wd, Wc) and torch.equal(K, coded.K)
    # argument errors
    assert L.dab_binarize_train(p(Wd), 3, 40, 39, p(Wd), 40, None, 0, p(K), p(a), p(b), p(m), ld, None, None) == 1
    assert L.dab_binarize_train(p(Wd), 3, 20000, 20000, p(Wd), 20000, None, 0, p(K), p(a), p(b), p(m), 628, None, None) == 2
    assert L.dab_binarize_backward(p(Wd), 3, 40, 40, p(m), ld, p(K), None, 40, p(Wd), 40, None) == 1
    assert L.dab_binarize_backward(p(Wd), 0, 40, 40, None, ld, None, None, 40, None, 40, None) == 0

"""The workspace-free convolution entry point (for callers that cannot allocate device memory, e.g. code that
only ever receives device pointers for its inputs and outputs) against the ordinary one.

Collected last on purpose: if it fails, a run that stops at the first failure has already run everything else.
"""
import ctypes as C

import numpy as np
import pytest
import torch

import dab_synth
import oracle
from dab_synth import configs

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def dab():
    import paper_1804_02941_b200 as d
    d.lib()
    return d


def _layer(dab, L, stream):
    x = torch.from_numpy(L.inputs(stream=stream)).cuda()
    w = dab.dab_binarize(torch.from_numpy(L.weights(stream=stream)).cuda())
    return x, w


def test_static_scratch_conv_matches_workspace_conv_on_two_calls_in_a_row(dab):
    # two different layers back to back: the second call finds the first call's codes in the shared array
    layers = [configs.ConvLayer("a", 2, 16, 20, 20, 24, 3, 3, 1, 1), configs.ConvLayer("b", 1, 64, 32, 32, 64, 3, 3, 1, 1, 0.05),
              configs.ConvLayer("c", 3, 8, 11, 13, 5, 5, 5, 2, 2)]
    for rep in range(2):
        for i, L in enumerate(layers):
            x, w = _layer(dab, L, 10 * rep + i)
            ref = dab.dab_binary_conv(x, w, L.kh, L.kw, (L.stride, L.stride), (L.pad, L.pad))
            got = dab.dab_binary_conv_static(x, w, L.kh, L.kw, (L.stride, L.stride), (L.pad, L.pad))
            torch.cuda.synchronize()
            r, g = ref.cpu().numpy().astype(np.float64), got.cpu().numpy().astype(np.float64)
            assert g.shape == r.shape and np.all(np.abs(g - r) <= 1e-5 * np.abs(r))
            assert np.array_equal(g, r)          # same kernels on the same codes: in fact identical
            if rep == 0:                         # and against the CPU checker, not only against the other entry point
                wv = L.weights(stream=10 * rep + i)
                wb = oracle.binarize(wv)
                o = oracle.conv(L.inputs(stream=10 * rep + i), wb.e, wb.alpha, wb.beta, L.kh, L.kw, (L.stride, L.stride),
                                (L.pad, L.pad), details=False)
                assert np.all(np.abs(g - o.y) <= 1e-5 * np.abs(o.y))


def test_static_scratch_conv_on_a_stream_of_the_callers(dab):
    L = configs.ConvLayer("s", 2, 32, 14, 14, 16, 3, 3, 1, 1)
    x, w = _layer(dab, L, 77)
    ref = dab.dab_binary_conv(x, w, L.kh, L.kw, (L.stride, L.stride), (L.pad, L.pad))
    torch.cuda.synchronize()
    side = torch.cuda.Stream()
    with torch.cuda.stream(side):
        got = dab.dab_binary_conv_static(x, w, L.kh, L.kw, (L.stride, L.stride), (L.pad, L.pad), stream=side)
    side.synchronize()
    assert torch.equal(ref, got)


def test_static_scratch_refuses_layers_beyond_its_capacity(dab):
    cap = dab.dab_binary_conv_static_capacity()
    assert cap == 16 * 1024 * 1024
    big = dab.make_desc((256, 64, 56, 56), 64, 3, 3, (1, 1), (1, 1))
    assert dab.dab_binary_conv_workspace(big) > cap
    dummy = torch.zeros(16, dtype=torch.int32, device="cuda")
    p = C.c_void_p(dummy.data_ptr())
    st = dab.lib().dab_binary_conv_static(C.byref(big), p, p, 20, p, p, p, p, None)
    assert st == 2 and "limit" in dab.status_string(st)           # refused before anything is launched
    bad = dab.make_desc((1, 3, 2, 2), 4, 5, 5)
    assert dab.lib().dab_binary_conv_static(C.byref(bad), p, p, 4, p, p, p, p, None) == 1
    long_rows = dab.make_desc((1, 2048, 8, 8), 4, 3, 3, (1, 1), (1, 1))           # n = 18432 > DAB_MAX_N: the status
    assert dab.lib().dab_binary_conv_static(C.byref(long_rows), p, p, 576, p, p, p, p, None) == 2   # dab_binary_conv gives
    torch.cuda.synchronize()

"""Calls from two host threads on two streams at once: kernels of one call hand work to each other only through
that call's own output arrays, so concurrent calls cannot disturb each other, whichever coders they take.

One thread runs a layer that takes the pixel-histogram coder, the other a small layer that takes the chain of
sorting and per-patch histogram kernels (tiles handed on through marks) while the process-wide coder choice is
switched back and forth; every result must equal the one obtained alone, and the first ones the CPU checker's.
"""
import threading

import numpy as np
import pytest
import torch

import dab_synth
import oracle
from dab_synth import configs
from parity_util import rel_close, to_dev

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def dab():
    import paper_1804_02941_b200 as d
    d.lib()
    oracle.set_threads(8)
    yield d
    d.dab_set_patch_coder(d.PATCHES_AUTO)


def test_two_threads_two_streams(dab):
    big = configs.ConvLayer("big", 4, 64, 20, 20, 32, 3, 3, 1, 1, 0.05)        # 1600 patches: pixel-histogram coder
    small = configs.ConvLayer("small", 1, 128, 14, 14, 16, 3, 3, 1, 1, 0.05)   # 196 patches: the marking chain
    jobs = []
    for L, dense in ((big, False), (small, True)):
        x = L.inputs(stream=500, dense=dense)
        if dense:
            x[:, :, :7] = L.inputs(stream=501)[:, :, :7]                       # sparse and dense tiles in one image
        w = L.weights(stream=500)
        wd = dab.dab_binarize(to_dev(w))
        xd = to_dev(x)
        alone = dab.dab_binary_conv(xd, wd, 3, 3, (1, 1), (1, 1))
        torch.cuda.synchronize()
        wb = oracle.binarize(w)
        ref = oracle.conv(x, wb.e, wb.alpha, wb.beta, 3, 3, (1, 1), (1, 1), details=False)
        assert rel_close(alone.cpu().numpy(), ref.y).all()
        jobs.append((xd, wd, alone))
    errors = []

    def worker(k):
        try:
            xd, wd, alone = jobs[k]
            stream = torch.cuda.Stream()
            for it in range(300):                                               # more calls than any ring of slots
                if k == 1 and it % 7 == 0:
                    dab.dab_set_patch_coder([dab.PATCHES_AUTO, dab.PATCHES_HIST, dab.PATCHES_SORT, dab.PATCHES_PIXEL][(it // 7) % 4])
                with torch.cuda.stream(stream):
                    y = dab.dab_binary_conv(xd, wd, 3, 3, (1, 1), (1, 1), stream=stream)
                if it % 50 == 49:
                    stream.synchronize()
                    if not torch.equal(y, alone):
                        errors.append("thread %d, call %d: result differs" % (k, it))
            stream.synchronize()
            if not torch.equal(y, alone):
                errors.append("thread %d: last result differs" % k)
        except Exception as exc:                                               # noqa: BLE001
            errors.append("thread %d: %r" % (k, exc))

    threads = [threading.Thread(target=worker, args=(k,)) for k in range(2)]
    for t in threads:
        t.start()
    for t in threads:
        t.join()
    dab.dab_set_patch_coder(dab.PATCHES_AUTO)
    assert not errors, errors

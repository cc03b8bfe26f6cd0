"""Runs the hot path on the bounds-checking build of the library and prints its violation report as one JSON line.

Started by tests/test_gpu_debug_bounds.py in a process of its own (a process loads one build of the library).
Usage: python tests/debug_bounds_run.py <path of libdab_debug.so>
Every coder and both contraction kernels are forced in turn on ragged shapes: rows and patch counts that do not
fill the last CTA, row lengths that are not multiples of 32, channel counts that are not multiples of 32, strides
and paddings that put tiles across the image border.  The first conv of each coder is compared with the CPU
checker as well, so that a check that redirected an access would show as a wrong result.
"""
import json
import os
import sys

import numpy as np
import torch

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)
sys.path.insert(0, os.path.join(ROOT, "tests"))

import dab_synth  # noqa: E402
import oracle  # noqa: E402
import paper_1804_02941_b200 as dab  # noqa: E402
from parity_util import rel_close, to_dev  # noqa: E402

CONVS = [  # N, C, H, W, Cout, kh, kw, stride, pad
    (3, 64, 21, 19, 40, 3, 3, (1, 1), (1, 1)),
    (2, 64, 23, 23, 72, 3, 3, (2, 2), (1, 1)),
    (2, 70, 17, 15, 33, 3, 3, (1, 1), (0, 0)),
    (1, 128, 30, 34, 130, 3, 3, (1, 1), (1, 1)),
    (1, 256, 17, 17, 64, 3, 3, (1, 1), (1, 1)),
    (1, 512, 9, 9, 64, 3, 3, (1, 1), (1, 1)),
    (2, 24, 33, 35, 48, 5, 5, (1, 1), (2, 2)),
    (4, 96, 6, 6, 256, 1, 1, (1, 1), (0, 0)),
    (1, 64, 7, 7, 96, 7, 7, (1, 1), (0, 0)),
]


def main():
    dab.use_library(sys.argv[1])
    dab.lib()
    assert dab.dab_debug_bounds_enabled(), "not a bounds-checking build"
    dab.dab_debug_bounds_report(reset=True)
    oracle.set_threads(8)
    calls, compared = 0, 0
    for coder in (dab.PATCHES_AUTO, dab.PATCHES_SORT, dab.PATCHES_HIST, dab.PATCHES_PIXEL):
        for path in (dab.CONTRACT_TENSOR, dab.CONTRACT_POPC):
            dab.dab_set_patch_coder(coder)
            dab.dab_set_contraction(path)
            for k, (N, C, H, W, Cout, kh, kw, stride, pad) in enumerate(CONVS):
                dense = (k + coder) % 2 == 1
                x = (dab_synth.normal((N, C, H, W), 1.0, stream=100 + k) if dense
                     else dab_synth.relu_activations((N, C, H, W), 0.6, stream=100 + k))
                w = dab_synth.normal((Cout, C * kh * kw), 0.05, stream=200 + k)
                coded = dab.dab_binarize(to_dev(w))
                y = dab.dab_binary_conv(to_dev(x), coded, kh, kw, stride, pad)
                torch.cuda.synchronize()
                calls += 1
                if k == 0 and path == dab.CONTRACT_TENSOR:
                    wb = oracle.binarize(w)
                    ref = oracle.conv(x, wb.e, wb.alpha, wb.beta, kh, kw, stride, pad, details=False)
                    assert rel_close(y.cpu().numpy(), ref.y).all(), "conv differs from the checker under coder %d" % coder
                    compared += 1
    dab.dab_set_patch_coder(dab.PATCHES_AUTO)
    dab.dab_set_contraction(dab.CONTRACT_AUTO)
    for rows, n in ((1, 1), (37, 31), (259, 576), (77, 1000), (2055, 576), (2100, 2304), (2049, 4608), (5, 16384)):
        for coder in (dab.PATCHES_AUTO, dab.PATCHES_HIST):      # the row histogram coder is taken when forced
            dab.dab_set_patch_coder(coder)
            a = dab.dab_binarize(to_dev(dab_synth.normal((rows, n), 1.0, stream=300 + n)))
            b = dab.dab_binarize(to_dev(dab_synth.normal((41, n), 1.0, stream=400 + n)))
            for path in (dab.CONTRACT_TENSOR, dab.CONTRACT_POPC):
                dab.dab_set_contraction(path)
                dab.dab_binary_gemm(a, b, want_p11=True)
                calls += 1
        bits = (dab_synth.uniform01(1804, 500 + n, 0, rows * n).reshape(rows, n) < 0.4).astype(np.uint8)
        dab.dab_pack(to_dev(bits))
        calls += 1
    dab.dab_set_patch_coder(dab.PATCHES_AUTO)
    dab.dab_set_contraction(dab.CONTRACT_AUTO)
    torch.cuda.synchronize()
    report = dab.dab_debug_bounds_report(reset=True)
    report.update(calls=calls, compared=compared, wait_failures=int(dab.dab_contraction_wait_failures()))
    print(json.dumps(report))


if __name__ == "__main__":
    main()

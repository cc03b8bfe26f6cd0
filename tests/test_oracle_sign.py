"""Pins for the CPU checker's sign coding (the XNOR-style code of the paper's FBin inputs; Section 4.1 calls the
XNOR scaling "a special case" with alpha = -beta).  No GPU involved."""
from fractions import Fraction

import numpy as np
import pytest
import torch

import dab_synth
import oracle


def best_one_scale_code(w):
    """Exhaustive search: over every sign pattern b in {+1,-1}^n, with the best scale s = (W.b)/n for that
    pattern, minimise ||W - s b||^2.  Exact rationals.  Returns (min error, set of optimal (pattern, scale))."""
    n = len(w)
    fw = [Fraction(float(x)) for x in w]
    ww = sum(x * x for x in fw)
    best, arg = None, set()
    for bits in range(1 << n):
        b = [1 if (bits >> i) & 1 else -1 for i in range(n)]
        dot = sum(x * y for x, y in zip(fw, b))
        if dot < 0:
            continue                                   # (-b, -s) is the same code
        err = ww - dot * dot / n                       # ||W||^2 - (W.b)^2 / n at the best scale
        if best is None or err < best:
            best, arg = err, {(tuple(b), dot / n)}
        elif err == best:
            arg.add((tuple(b), dot / n))
    return best, arg


@pytest.mark.parametrize("n", [1, 2, 3, 5, 8, 11])
def test_sign_code_is_the_best_one_scale_code(n):
    rows = np.concatenate([dab_synth.normal((4, n), 1.0, stream=400 + n), dab_synth.small_integer_rows(4, n, -3, 3, stream=500 + n)])
    r = oracle.sign_code(rows)
    for i, w in enumerate(rows):
        err, arg = best_one_scale_code(w)
        b = tuple(1 if e else -1 for e in r.e[i])
        scales = {s for (pat, s) in arg if all(p == q or Fraction(float(x)) == 0 for p, q, x in zip(pat, b, w))}
        assert scales, "sign pattern not optimal"      # zeros may take either sign; everything else is forced
        assert np.float32(float(next(iter(scales)))) == r.alpha[i] and r.beta[i] == -r.alpha[i]
        assert r.K[i] == sum(e for e in r.e[i])


def test_sign_code_conventions():
    r = oracle.sign_code(np.array([[0.0, -0.0, 2.0, -4.0]], np.float32))
    assert r.e[0].tolist() == [1, 1, 1, 0] and r.K[0] == 3 and r.alpha[0] == 1.5 and r.beta[0] == -1.5
    r = oracle.sign_code(np.array([[1.0, np.nan], [1.0, -3.0]], np.float32))
    assert r.flags[0] == oracle.FLAG_NONFINITE and r.flags[1] == 0 and r.alpha[1] == 2.0


def test_dab_error_never_exceeds_sign_code_error():
    # Section 4.1: the XNOR scaling is a special case of the two-level form, so the optimal code is at least as good
    w = np.concatenate([dab_synth.normal((20, 64), 1.0, stream=7), dab_synth.laplace((20, 64), 0.05, stream=8)])
    d, s = oracle.binarize(w), oracle.sign_code(w)
    w64 = w.astype(np.float64)
    rec = lambda c: c.alpha.astype(np.float64)[:, None] * c.e + c.beta.astype(np.float64)[:, None] * (1 - c.e.astype(np.float64))
    ed, es = ((w64 - rec(d)) ** 2).sum(1), ((w64 - rec(s)) ** 2).sum(1)
    assert np.all(ed <= es * (1 + 1e-6))


def test_conv_with_sign_coded_inputs_equals_unfold_sign_matmul():
    x = dab_synth.dense_activations((2, 5, 8, 7), stream=70)
    w = dab_synth.normal((6, 45), 0.05, stream=71)
    wb = oracle.binarize(w)
    res = oracle.conv(x, wb.e, wb.alpha, wb.beta, 3, 3, (1, 1), (1, 1), sign_inputs=True)
    u = torch.nn.functional.unfold(torch.from_numpy(x), (3, 3), padding=(1, 1))
    patches = u.permute(0, 2, 1).reshape(-1, 45).numpy().astype(np.float64)
    scale = np.abs(patches).mean(1, keepdims=True)
    Xt = scale * np.where(patches >= 0, 1.0, -1.0)                       # XNOR-Net: sign pattern times mean magnitude
    Wt = wb.alpha.astype(np.float64)[:, None] * wb.e + wb.beta.astype(np.float64)[:, None] * (1.0 - wb.e)
    ref = (Xt @ Wt.T).reshape(2, 8, 7, 6).transpose(0, 3, 1, 2)
    assert np.allclose(res.y, ref, rtol=1e-5, atol=1e-7)
    assert np.array_equal(res.p_e, (patches >= 0).astype(np.uint8))
    assert np.array_equal(res.p_gamma, -res.p_delta)

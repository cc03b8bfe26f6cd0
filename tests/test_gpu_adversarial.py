"""Rows and images built to defeat a pruned search, against the CPU checker on every row.

The pixel-histogram patch coder and the histogram coder of dab_binarize discard the buckets that cannot hold the
best split and search the rest exactly.  A wrong discard would return a wrong K silently, so both are run (forced)
on more than 20,000 rows per row length of inputs chosen to stress the bounds:
  edges     values on and one ulp below power-of-two bucket edges, many duplicates
  range     magnitudes spread over 2^20
  outlier   ordinary rows plus one huge value that stretches the bucket grid of the whole tile
  clusters  two tight clusters holding 35 % and 65 % of the values (the split the paper's Fig. 4 reports), with and
            without zeros
  ints      small integers: exact ties of the objective, decided by the tie rule
  narrow    all values within 2^-18 of each other: one bucket holds the whole row
  signed    both signs, no zeros
Only near-ties (objective gap below 1e-9 relative, logged) may differ from the checker.
"""
import numpy as np
import pytest
import torch

import oracle
from parity_util import NEAR_TIE, rel_close, to_dev, unpack, words

pytestmark = pytest.mark.gpu

KINDS = ["edges", "range", "outlier", "clusters", "clusters0", "ints", "narrow", "signed"]


@pytest.fixture(scope="module")
def dab():
    import paper_1804_02941_b200 as d
    d.lib()
    oracle.set_threads(16)
    yield d
    d.dab_set_patch_coder(d.PATCHES_AUTO)


def _values(kind, shape, rng):
    """fp32 array of `shape`; the last axis of a row matrix, or the channel axis of an image, is what one row mixes."""
    n = int(np.prod(shape))
    if kind == "edges":
        j = rng.integers(0, 41, n)
        v = j.astype(np.float32) * np.float32(2.0 ** -5)
        below = rng.random(n) < 0.5
        v[below] = np.nextafter(v[below], np.float32(0.0))
        v[rng.random(n) < 0.5] = 0.0
    elif kind == "range":
        v = np.abs(rng.standard_normal(n)) * 2.0 ** (-20.0 * rng.random(n))
        v[rng.random(n) < 0.3] = 0.0
    elif kind == "outlier":
        v = np.abs(rng.standard_normal(n)) * (rng.random(n) < 0.4)
        v[rng.integers(0, n, max(1, n // 20000))] = 1.0e4
    elif kind in ("clusters", "clusters0"):
        hi = rng.random(n) < 0.35
        v = np.where(hi, 2.0 + 0.1 * rng.standard_normal(n), 0.5 + 0.1 * rng.standard_normal(n))
        if kind == "clusters0":
            v[rng.random(n) < 0.5] = 0.0
    elif kind == "ints":
        v = rng.integers(-3, 4, n).astype(np.float64)
    elif kind == "narrow":
        v = 1.0 + rng.integers(0, 64, n) * 2.0 ** -24
    else:
        v = rng.standard_normal(n)
    return np.ascontiguousarray(np.asarray(v, np.float32).reshape(shape))


def _compare(K, e, flags, alpha, beta, ref, what):
    differs = (K != ref.K) | (flags != ref.flags) | (e != ref.e).any(axis=1)
    near = (ref.gap > 0) & (ref.gap < NEAR_TIE)
    if (differs & near).any():
        print("%s: near-ties that differ: rows %s gaps %s" % (what, np.nonzero(differs & near)[0].tolist()[:8],
                                                             ref.gap[differs & near].tolist()[:8]))
    bad = differs & ~near
    assert not bad.any(), "%s: rows %s differ from the checker (gaps %s)" % (what, np.nonzero(bad)[0][:8], ref.gap[bad][:8])
    ok = ~differs & ~(ref.flags & 2).astype(bool)
    assert rel_close(alpha[ok], ref.alpha[ok]).all() and rel_close(beta[ok], ref.beta[ok]).all(), what
    return int((differs & near).sum())


@pytest.mark.parametrize("C", [64, 128, 256, 512])
def test_pixel_histogram_coder_on_adversarial_images(dab, C):
    n = C * 9
    rng = np.random.default_rng(1804 + C)
    hw, per_kind = 18, 8                       # 8 kinds x 8 images x 324 patches = 20,736 rows of n values
    excused = 0
    for kind in KINDS:
        x = _values(kind, (per_kind, C, hw, hw), rng)
        if kind == "outlier":
            x[:, :, : hw // 2] = np.abs(x[:, :, : hw // 2]) * 1e-3      # and a region of much smaller values beside it
        desc = dab.make_desc(tuple(x.shape), 8, 3, 3, (1, 1), (1, 1))
        P, ld = per_kind * hw * hw, dab.dab_default_ld(n)
        xd = to_dev(x)
        pK = torch.full((P,), -7, dtype=torch.int32, device=xd.device)
        pg, pd = torch.zeros(P, device=xd.device), torch.zeros(P, device=xd.device)
        pm = torch.zeros((P, ld), dtype=torch.int32, device=xd.device)
        pf = torch.zeros(P, dtype=torch.int32, device=xd.device)
        dab.dab_set_patch_coder(dab.PATCHES_PIXEL)
        dab.dab_binarize_patches(desc, xd, pK, pg, pd, pm, pf)
        torch.cuda.synchronize()
        dab.dab_set_patch_coder(dab.PATCHES_AUTO)
        ref = oracle.binarize(oracle.im2col(x, 3, 3, (1, 1), (1, 1)))
        excused += _compare(pK.cpu().numpy(), unpack(words(pm), n), pf.cpu().numpy().view(np.uint32), pg.cpu().numpy(),
                            pd.cpu().numpy(), ref, "pixel coder, C=%d, %s" % (C, kind))
    assert excused <= 8


@pytest.mark.parametrize("n", [576, 1152, 2304, 4608])
def test_row_histogram_coder_on_adversarial_rows(dab, n):
    rng = np.random.default_rng(2941 + n)
    rows = 2560                                # 8 kinds x 2,560 rows = 20,480 rows of n values
    excused = 0
    for kind in KINDS:
        w = _values(kind, (rows, n), rng)
        dab.dab_set_patch_coder(dab.PATCHES_HIST)
        got = dab.dab_binarize(to_dev(w))
        torch.cuda.synchronize()
        dab.dab_set_patch_coder(dab.PATCHES_AUTO)
        ref = oracle.binarize(w)
        excused += _compare(got.K.cpu().numpy(), unpack(words(got.mask), n), got.flags.cpu().numpy().view(np.uint32),
                            got.alpha.cpu().numpy(), got.beta.cpu().numpy(), ref, "row coder, n=%d, %s" % (n, kind))
    assert excused <= 8

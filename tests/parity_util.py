"""Helpers shared by the GPU parity tests: device round trips and the comparison rules.

Comparison rules (from the benchmark spec of agreement):
  - K, packed masks, flags and AND-popcounts are compared bit for bit;
  - alpha, beta and layer outputs within 1e-5 relative;
  - a row whose best and second-best objective differ by less than 1e-9 relative (but are not exactly
    equal) is a near-tie: it is logged and excused from the bit-exact comparison.  Exact ties are NOT
    excused: the tie rule decides them.
"""
from __future__ import annotations

import numpy as np
import torch

RTOL = 1e-5
NEAR_TIE = 1e-9


def to_dev(a: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def words(t: torch.Tensor) -> np.ndarray:
    return t.detach().cpu().numpy().view(np.uint32)


def unpack(mask_words: np.ndarray, n: int) -> np.ndarray:
    """rows x ld uint32 -> rows x n uint8, element i = bit (i % 32) of word (i // 32)."""
    rows, ld = mask_words.shape
    bits = ((mask_words[:, :, None] >> np.arange(32, dtype=np.uint32)[None, None, :]) & 1).astype(np.uint8)
    return bits.reshape(rows, ld * 32)[:, :n]


def padding_is_zero(mask_words: np.ndarray, n: int) -> bool:
    rows, ld = mask_words.shape
    bits = ((mask_words[:, :, None] >> np.arange(32, dtype=np.uint32)[None, None, :]) & 1).reshape(rows, ld * 32)
    return not bits[:, n:].any()


def rel_close(got: np.ndarray, ref: np.ndarray, rtol: float = RTOL) -> np.ndarray:
    got = got.astype(np.float64)
    ref = ref.astype(np.float64)
    both_nan = np.isnan(got) & np.isnan(ref)
    return both_nan | (np.abs(got - ref) <= rtol * np.abs(ref))


def check_coded(coded, ref, n: int, log=None):
    """coded: device result of dab_binarize; ref: oracle.Binarized.  Returns the number of near-tie rows excused."""
    K = coded.K.cpu().numpy()
    alpha = coded.alpha.cpu().numpy()
    beta = coded.beta.cpu().numpy()
    flags = coded.flags.cpu().numpy().view(np.uint32)
    mw = words(coded.mask)
    assert padding_is_zero(mw, n), "padding bits or words not zero"
    e = unpack(mw, n)
    near = (ref.gap > 0) & (ref.gap < NEAR_TIE)
    strict = ~near
    if near.any() and log is not None:
        log("near-ties (objective gap < 1e-9 relative): rows %s gaps %s" % (np.nonzero(near)[0].tolist(), ref.gap[near].tolist()))
    assert np.array_equal(flags[strict], ref.flags[strict]), "row flags differ"
    assert np.array_equal(K[strict], ref.K[strict]), "K differs at rows %s" % np.nonzero(strict & (K != ref.K))[0][:8]
    assert np.array_equal(e[strict], ref.e[strict]), "mask bits differ"
    assert np.array_equal(e.sum(1), K), "popcount(mask) != K"
    ok = ~(ref.flags & 2).astype(bool) & strict
    assert rel_close(alpha[ok], ref.alpha[ok]).all(), "alpha beyond 1e-5 relative"
    assert rel_close(beta[ok], ref.beta[ok]).all(), "beta beyond 1e-5 relative"
    return int(near.sum())

"""GPU parity at the full sizes of the workload configurations, in the launch configuration bench.py times
(dab_binarize -> dab_binarize_patches -> dab_binary_conv_contract on whole layers), checked on sampled
outputs that the CPU checker computes one by one.
"""
import numpy as np
import pytest
import torch

import dab_synth
from dab_synth import configs
import oracle
from parity_util import NEAR_TIE, check_coded, rel_close, to_dev, unpack, words

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def dab():
    import paper_1804_02941_b200 as d
    d.lib()
    oracle.set_threads(8)
    return d


def _sample_patches(x, L, idx):
    """Patch rows (element order (c, kh, kw), zero padding as values) of the sampled patch indices, by indexing."""
    rows = np.zeros((len(idx), L.n), np.float32)
    for t, p in enumerate(idx):
        img, rem = divmod(int(p), L.Ho * L.Wo)
        ho, wo = divmod(rem, L.Wo)
        xp = np.pad(x[img], ((0, 0), (L.pad, L.pad), (L.pad, L.pad)))
        h0, w0 = ho * L.stride, wo * L.stride
        rows[t] = xp[:, h0:h0 + L.kh, w0:w0 + L.kw].reshape(-1)
    return rows


def _check_layer(dab, L, stream, samples=192, dense=False):
    x = L.inputs(stream=stream, dense=dense)
    w = L.weights(stream=stream)
    xd = to_dev(x)
    wd = dab.dab_binarize(to_dev(w))
    wb = oracle.binarize(w)
    check_coded(wd, wb, L.n, log=print)

    dev = xd.device
    P, ld = L.patches, dab.dab_default_ld(L.n)
    pK = torch.empty(P, dtype=torch.int32, device=dev)
    pg = torch.empty(P, dtype=torch.float32, device=dev)
    pd = torch.empty(P, dtype=torch.float32, device=dev)
    pf = torch.empty(P, dtype=torch.int32, device=dev)
    pm = torch.empty((P, ld), dtype=torch.int32, device=dev)
    y = torch.empty((L.N, L.Cout, L.Ho, L.Wo), dtype=torch.float32, device=dev)
    desc = dab.make_desc(L.x_shape(), L.Cout, L.kh, L.kw, (L.stride, L.stride), (L.pad, L.pad))
    dab.dab_binarize_patches(desc, xd, pK, pg, pd, pm, pf)
    dab.dab_binary_conv_contract(desc, pm, pK, pg, pd, wd, y)
    torch.cuda.synchronize()

    # sampled patches: corners and borders first, the rest uniformly over the layer
    u = dab_synth.uniform01(99, stream, 0, samples)
    idx = np.unique(np.concatenate([[0, L.Wo - 1, L.Ho * L.Wo - 1, P - 1, P - L.Wo], (u * P).astype(np.int64)]))
    rows = _sample_patches(x, L, idx)
    ref = oracle.binarize(rows)
    tidx = torch.from_numpy(idx).to(dev)
    strict = ~((ref.gap > 0) & (ref.gap < NEAR_TIE))
    assert strict.sum() >= len(idx) - 2
    assert np.array_equal(pf[tidx].cpu().numpy().view(np.uint32)[strict], ref.flags[strict])
    assert np.array_equal(pK[tidx].cpu().numpy()[strict], ref.K[strict])
    assert np.array_equal(unpack(words(pm[tidx]), L.n)[strict], ref.e[strict])
    assert rel_close(pg[tidx].cpu().numpy()[strict], ref.alpha[strict]).all()
    assert rel_close(pd[tidx].cpu().numpy()[strict], ref.beta[strict]).all()
    refC, _ = oracle.gemm(ref.e, ref.alpha, ref.beta, wb.e, wb.alpha, wb.beta)            # samples x Cout
    img, rem = np.divmod(idx, L.Ho * L.Wo)
    ho, wo = np.divmod(rem, L.Wo)
    got = y[torch.from_numpy(img).to(dev), :, torch.from_numpy(ho).to(dev), torch.from_numpy(wo).to(dev)].cpu().numpy()
    assert rel_close(got[strict], refC[strict]).all()
    # properties that hold for every patch of the layer
    Kall = pK.cpu().numpy()
    assert Kall.min() >= 0 and Kall.max() <= L.n - 1
    pop = torch.zeros(P, dtype=torch.int64, device=dev)
    for wcol in range(ld):                                                                  # popcount(mask) == K everywhere
        v = pm[:, wcol].to(torch.int64) & 0xFFFFFFFF
        v = v - ((v >> 1) & 0x55555555)
        v = (v & 0x33333333) + ((v >> 2) & 0x33333333)
        v = (v + (v >> 4)) & 0x0F0F0F0F
        pop += (v * 0x01010101 & 0xFFFFFFFF) >> 24
    assert torch.equal(pop, pK.to(torch.int64))
    assert bool(torch.isfinite(y).all())


@pytest.mark.parametrize("name", ["l1_0", "l2_0", "l2_1", "l3_0", "l3_1", "l4_0", "l4_1"])
def test_config5_layers_at_batch_256(dab, name):
    L = next(l for l in configs.config5(256) if l.name == name)
    _check_layer(dab, L, stream=7)


def test_config5_first_layer_sign_coded_inputs(dab):
    # the XNOR-style input coding at full size: sampled patches against the checker
    L = configs.config5(256)[0]
    x = L.inputs(stream=9, dense=True)
    w = L.weights(stream=9)
    xd, wd, wb = to_dev(x), dab.dab_binarize(to_dev(w)), oracle.binarize(w)
    y, det = dab.dab_binary_conv(xd, wd, 3, 3, (1, 1), (1, 1), details=True, sign_inputs=True)
    torch.cuda.synchronize()
    P = L.patches
    idx = np.unique(np.concatenate([[0, L.Wo - 1, P - 1], (dab_synth.uniform01(97, 1, 0, 160) * P).astype(np.int64)]))
    ref = oracle.sign_code(_sample_patches(x, L, idx))
    t = torch.from_numpy(idx).to(xd.device)
    assert np.array_equal(det.pK[t].cpu().numpy(), ref.K) and np.array_equal(unpack(words(det.pmask[t]), L.n), ref.e)
    assert rel_close(det.pgamma[t].cpu().numpy(), ref.alpha).all()
    refC, refP = oracle.gemm(ref.e, ref.alpha, ref.beta, wb.e, wb.alpha, wb.beta)
    assert np.array_equal(det.p11[t].cpu().numpy(), refP)
    img, rem = np.divmod(idx, L.Ho * L.Wo)
    ho, wo = np.divmod(rem, L.Wo)
    dev = xd.device
    got = y[torch.from_numpy(img).to(dev), :, torch.from_numpy(ho).to(dev), torch.from_numpy(wo).to(dev)].cpu().numpy()
    assert np.array_equal(det.pgamma[t].cpu().numpy(), ref.alpha)
    assert rel_close(got, refC).all()


def test_config5_first_layer_dense_inputs(dab):
    L = configs.config5(64)[0]
    _check_layer(dab, L, stream=8, dense=True)


@pytest.mark.parametrize("li", range(6))
def test_config4_layers_at_batch_128(dab, li):
    L = configs.config4(128)[li]
    _check_layer(dab, L, stream=20 + li, samples=96)


@pytest.mark.parametrize("m,k", [(m, k) for m in (1024, 4096, 8192) for k in (576, 2304, 4608)])
def test_config3_points(dab, m, k):
    A, B = configs.config3_operands(m, k)
    a, b = dab.dab_binarize(to_dev(A)), dab.dab_binarize(to_dev(B))
    Cm = dab.dab_binary_gemm(a, b)
    torch.cuda.synchronize()
    u = dab_synth.uniform01(98, m + k, 0, 128)
    ri = np.unique(np.concatenate([[0, m - 1], (u[:64] * m).astype(np.int64)]))
    ci = np.unique(np.concatenate([[0, m - 1], (u[64:] * m).astype(np.int64)]))
    ra, rb = oracle.binarize(A[ri]), oracle.binarize(B[ci])
    dev = a.mask.device
    tri, tci = torch.from_numpy(ri).to(dev), torch.from_numpy(ci).to(dev)
    for got, ref, t in ((a, ra, tri), (b, rb, tci)):
        sub = dab.Coded(got.mask[t], got.K[t], got.alpha[t], got.beta[t], got.flags[t], k)
        check_coded(sub, ref, k, log=print)
    refC, _ = oracle.gemm(ra.e, ra.alpha, ra.beta, rb.e, rb.alpha, rb.beta)
    gotC = Cm[tri][:, tci].cpu().numpy()
    ok = ~(((ra.gap > 0) & (ra.gap < NEAR_TIE))[:, None] | ((rb.gap > 0) & (rb.gap < NEAR_TIE))[None, :])
    assert rel_close(gotC, refC)[ok].all()
    assert bool(torch.isfinite(Cm).all())

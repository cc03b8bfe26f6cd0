"""Pins for the checker's full-precision layers and its chaining of layers (no GPU): library convolution and
pooling in fp64, integer-valued inputs where the result must be exact, and a residual chain rebuilt with torch."""
import numpy as np
import torch
import torch.nn.functional as F

import oracle
from dab_synth import networks


def _rng(seed):
    return np.random.default_rng(seed)


def test_conv_dense_against_library_convolution():
    for seed, (N, C, H, W, Cout, kh, kw, st, pd) in enumerate([(2, 3, 9, 11, 4, 3, 3, (1, 1), (1, 1)), (1, 2, 15, 15, 5, 5, 5, (3, 3), (0, 0)),
                                                              (2, 4, 8, 8, 3, 1, 1, (2, 2), (0, 0)), (1, 3, 7, 9, 2, 3, 2, (2, 1), (0, 1))]):
        x = _rng(seed).standard_normal((N, C, H, W)).astype(np.float32)
        w = _rng(100 + seed).standard_normal((Cout, C * kh * kw)).astype(np.float32)
        b = _rng(200 + seed).standard_normal(Cout).astype(np.float32)
        got = oracle.conv_dense(x, w, kh, kw, st, pd, bias=b)
        ref = F.conv2d(torch.from_numpy(x).double(), torch.from_numpy(w).double().view(Cout, C, kh, kw), torch.from_numpy(b).double(),
                       stride=st, padding=pd).numpy()
        assert got.shape == ref.shape and np.allclose(got, ref, rtol=1e-6, atol=1e-6)
        # integer-valued operands: every sum is exact, so the result equals the library's to the bit
        xi, wi = np.round(3 * x), np.round(2 * w)
        goti = oracle.conv_dense(xi, wi, kh, kw, st, pd)
        refi = F.conv2d(torch.from_numpy(xi).double(), torch.from_numpy(wi).double().view(Cout, C, kh, kw), stride=st, padding=pd).numpy()
        assert np.array_equal(goti.astype(np.float64), refi)


def test_pooling_affine_relu_add_against_library():
    x = _rng(5).standard_normal((2, 3, 13, 10)).astype(np.float32)
    for k, st, pd in [(3, 2, 0), (3, 2, 1), (2, 2, 0), (7, 1, 0)]:
        got = oracle.maxpool(x, k, k, (st, st), (pd, pd))
        ref = F.max_pool2d(torch.from_numpy(x), k, st, pd).numpy()
        assert np.array_equal(got, ref)
    scale, shift = _rng(6).random(3).astype(np.float32) + 0.5, _rng(7).standard_normal(3).astype(np.float32)
    got = oracle.affine(x, scale, shift)
    ref = (torch.from_numpy(x).double() * torch.from_numpy(scale).double().view(1, 3, 1, 1) + torch.from_numpy(shift).double().view(1, 3, 1, 1)).numpy()
    assert np.allclose(got, ref, rtol=1e-7, atol=1e-7)
    assert np.array_equal(oracle.affine(x, np.ones(3, np.float32), np.zeros(3, np.float32)), x)          # identity
    y = x.copy()
    y[0, 0, 0, :3] = [-0.0, np.nan, -1.0]
    r = oracle.relu(y)
    assert np.array_equal(r[0, 0, 1:], torch.relu(torch.from_numpy(y))[0, 0, 1:].numpy()) and np.array_equal(r[0, 0, 0, :3], [0.0, 0.0, 0.0])
    assert not np.signbit(r[0, 0, 0, 0])
    assert np.array_equal(oracle.add(x, 2 * x), x + 2 * x)


def test_chain_with_shortcut_against_torch():
    # a residual block with a strided projection, full-precision layers only: the plumbing (save, layers on the
    # remembered tensor, add) against the same block written with torch in fp64
    rng = _rng(11)
    C, Co = 4, 6
    w1, w2 = rng.standard_normal((Co, C * 9)).astype(np.float32), rng.standard_normal((Co, Co * 9)).astype(np.float32)
    wp = rng.standard_normal((Co, C)).astype(np.float32)
    sc, sh = rng.random(Co).astype(np.float32) + 0.5, rng.standard_normal(Co).astype(np.float32)
    layers = [{"kind": "save"},
              {"kind": "conv_dense", "w": w1, "kh": 3, "kw": 3, "stride": (2, 2), "pad": (1, 1)}, {"kind": "relu"},
              {"kind": "conv_dense", "w": w2, "kh": 3, "kw": 3, "stride": (1, 1), "pad": (1, 1)},
              {"kind": "conv_dense", "w": wp, "kh": 1, "kw": 1, "stride": (2, 2), "pad": (0, 0), "on_saved": True},
              {"kind": "affine", "scale": sc, "shift": sh, "on_saved": True},
              {"kind": "add"}, {"kind": "relu"}, {"kind": "maxpool", "kh": 2, "kw": 2, "stride": (2, 2), "pad": (0, 0)}]
    x = rng.standard_normal((2, C, 12, 12)).astype(np.float32)
    got = oracle.network_forward(layers, x)
    t = torch.from_numpy(x).double()
    main = F.conv2d(torch.relu(F.conv2d(t, torch.from_numpy(w1).double().view(Co, C, 3, 3), stride=2, padding=1)),
                    torch.from_numpy(w2).double().view(Co, Co, 3, 3), padding=1)
    proj = F.conv2d(t, torch.from_numpy(wp).double().view(Co, C, 1, 1), stride=2)
    proj = proj * torch.from_numpy(sc).double().view(1, Co, 1, 1) + torch.from_numpy(sh).double().view(1, Co, 1, 1)
    ref = F.max_pool2d(torch.relu(main + proj), 2, 2).numpy()
    assert got.shape == ref.shape and np.allclose(got, ref, rtol=1e-5, atol=1e-5)


def test_network_shapes():
    for build, c_last in ((networks.sketch_a_net, 250), (networks.alexnet_like, 250), (networks.resnet18_like, 250)):
        layers, shape = build()
        assert layers[-1]["w"].shape[0] == c_last and len(shape) == 3
        assert sum(l["kind"] == "conv_binary" for l in layers) in (6, 16)
    assert sum(l["kind"] == "conv_binary" for l in networks.resnet18_like()[0]) == 16

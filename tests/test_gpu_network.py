"""Whole-network inference (dab_network_forward) against the CPU checker.

Layer by layer, teacher forced: the checker is given exactly the tensors the GPU layer consumed (a one-ulp
difference upstream may legitimately flip a split downstream, so only this comparison can be exact): the
full-precision layers must agree bit for bit, the binarized ones within 1e-5 relative except at patches whose
objective is a near-tie.  End to end, from the input alone, the logits must agree closely: they differ only by what
such flips and the 1e-5 of every binarized layer add up to.
"""
import numpy as np
import pytest
import torch

import oracle
from dab_synth import networks
from parity_util import NEAR_TIE, rel_close, to_dev

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def dab():
    import paper_1804_02941_b200 as d
    d.lib()
    oracle.set_threads(16)
    return d


def _shapes(layers, in_shape):
    """(C, H, W) of what every layer writes: the running tensor, or the remembered one for on_saved layers."""
    cur, saved, out = tuple(in_shape), None, []
    for l in layers:
        t = saved if l.get("on_saved") else cur
        if l["kind"] in ("conv_dense", "conv_binary", "maxpool"):
            Ho, Wo = oracle.conv_out_hw(t[1], t[2], l["kh"], l["kw"], l["stride"], l["pad"])
            t = (l["w"].shape[0] if "w" in l else t[0], Ho, Wo)
        if l["kind"] == "save":
            saved = cur
            out.append(cur)
            continue
        if l.get("on_saved"):
            saved = t
        else:
            cur = t
        out.append(t)
    return out


def _run_and_check(dab, layers, in_shape, batch, stream):
    x = networks.network_input(in_shape, batch, stream=stream)
    net = dab.Network(layers)
    shapes = _shapes(layers, in_shape)
    y, outs = dab.dab_network_forward(net, to_dev(x), keep_layers=True, layer_shapes=shapes)
    y_plain = dab.dab_network_forward(net, to_dev(x))                       # the same through the workspace buffers
    torch.cuda.synchronize()
    outs = [o.cpu().numpy() for o in outs]
    assert np.array_equal(y.cpu().numpy(), y_plain.cpu().numpy())
    assert np.array_equal(y.cpu().numpy(), outs[-1] if not layers[-1].get("on_saved") else y.cpu().numpy())
    cur, saved, near_ties = x, None, 0
    for i, l in enumerate(layers):
        want_cur, want_saved = oracle.network_layer(l, cur, saved)
        want = want_saved if (l.get("on_saved") or l["kind"] == "save") else want_cur
        got = outs[i]
        assert got.shape == want.shape, (i, l["kind"])
        if l["kind"] == "conv_binary":
            ok = rel_close(got, want)
            if not ok.all():   # only outputs of near-tie patches may differ
                bad_patch = ~ok.all(axis=1).reshape(-1)                     # (img, ho, wo) flattened
                rows = oracle.im2col(cur, l["kh"], l["kw"], l["stride"], l["pad"])[bad_patch]
                gap = oracle.binarize(rows).gap
                print("layer %d: %d patches differ, gaps %s" % (i, int(bad_patch.sum()), gap[:8]))
                assert ((gap > 0) & (gap < NEAR_TIE)).all(), "layer %d: outputs differ without a near-tie" % i
                near_ties += int(bad_patch.sum())
        else:
            assert np.array_equal(got, want), "layer %d (%s) differs from the checker" % (i, l["kind"])
        # teacher forcing: the next layer is checked on what the GPU produced
        if l["kind"] == "save":
            saved = got.copy()
        elif l.get("on_saved"):
            saved = got
        else:
            cur = got
    assert near_ties <= 2
    # end to end, from the input alone
    ref = oracle.network_forward(layers, x)
    got = y.cpu().numpy().astype(np.float64)
    scale = np.abs(ref).max()
    assert np.abs(got - ref).max() <= 1e-3 * scale, "end-to-end logits differ by %g of their range" % (np.abs(got - ref).max() / scale)
    assert np.array_equal(got.argmax(axis=1), ref.argmax(axis=1))
    return y


def test_glue_layers_one_by_one(dab):
    rng = np.random.default_rng(3)
    C = 5
    w = rng.standard_normal((7, C * 9)).astype(np.float32)
    wp = rng.standard_normal((7, C)).astype(np.float32)
    layers = [{"kind": "affine", "scale": rng.random(C).astype(np.float32) + 0.5, "shift": rng.standard_normal(C).astype(np.float32)},
              {"kind": "save"},
              {"kind": "conv_dense", "w": w, "kh": 3, "kw": 3, "stride": (2, 2), "pad": (1, 1), "bias": rng.standard_normal(7).astype(np.float32)},
              {"kind": "relu"},
              {"kind": "conv_dense", "w": wp, "kh": 1, "kw": 1, "stride": (2, 2), "pad": (0, 0), "on_saved": True},
              {"kind": "affine", "scale": rng.random(7).astype(np.float32) + 0.5, "shift": rng.standard_normal(7).astype(np.float32), "on_saved": True},
              {"kind": "add"},
              {"kind": "maxpool", "kh": 3, "kw": 3, "stride": (2, 2), "pad": (1, 1)},
              {"kind": "relu"}]
    x = rng.standard_normal((3, C, 13, 11)).astype(np.float32)
    x[0, 0, 0, :2] = [-0.0, 0.0]
    net = dab.Network(layers)
    y, outs = dab.dab_network_forward(net, to_dev(x), keep_layers=True, layer_shapes=_shapes(layers, (C, 13, 11)))
    torch.cuda.synchronize()
    ref, refs = oracle.network_forward(layers, x, keep=True)
    assert np.array_equal(y.cpu().numpy(), ref)
    cur, saved = x, None
    for i, l in enumerate(layers):
        cur, saved = oracle.network_layer(l, cur, saved)
        want = saved if (l.get("on_saved") or l["kind"] == "save") else cur
        assert np.array_equal(outs[i].cpu().numpy(), want), (i, l["kind"])


def test_chain_errors_are_return_codes(dab):
    import ctypes as C
    rng = np.random.default_rng(4)
    net = dab.Network([{"kind": "add"}])                                     # nothing was saved
    co = C.c_int32(0)
    assert dab.lib().dab_network_output_shape(net.records, 1, 1, 3, 8, 8, C.byref(co), C.byref(co), C.byref(co)) == 1
    assert dab.lib().dab_network_workspace(net.records, 1, 1, 3, 8, 8) == 0
    net = dab.Network([{"kind": "maxpool", "kh": 9, "kw": 9, "stride": (1, 1), "pad": (0, 0)}])   # window larger than the input
    assert dab.lib().dab_network_output_shape(net.records, 1, 1, 3, 8, 8, C.byref(co), C.byref(co), C.byref(co)) == 1
    net = dab.Network([{"kind": "relu"}])
    x = to_dev(rng.standard_normal((1, 3, 8, 8)).astype(np.float32))
    y = torch.empty_like(x)
    assert dab.lib().dab_network_forward(net.records, 1, 1, 3, 8, 8, C.c_void_p(x.data_ptr()), C.c_void_p(y.data_ptr()), None, 0, None, None) == 3


def test_sketch_a_net_shaped_network(dab):
    layers, shape = networks.sketch_a_net()
    y = _run_and_check(dab, layers, shape, batch=1, stream=1)
    assert tuple(y.shape) == (1, 250, 1, 1)


def test_alexnet_shaped_network(dab):
    layers, shape = networks.alexnet_like()
    y = _run_and_check(dab, layers, shape, batch=2, stream=2)
    assert tuple(y.shape) == (2, 250, 1, 1)


def test_resnet18_shaped_network(dab):
    layers, shape = networks.resnet18_like()
    y = _run_and_check(dab, layers, shape, batch=2, stream=3)
    assert tuple(y.shape) == (2, 250, 1, 1)


@pytest.mark.parametrize("spec", networks.googlenet_branch_layers(8), ids=lambda s: s[0])
def test_googlenet_branch_layer_shapes(dab, spec):
    # 1x1, 3x3 and 5x5 branches of inception modules as single binarized layers, every patch against the checker
    from dab_synth import configs
    from test_gpu_parity import _check_conv
    name, N, C, H, W, Cout, kh, kw, stride, pad = spec
    L = configs.ConvLayer(name, N, C, H, W, Cout, kh, kw, stride, pad)
    _check_conv(dab, L.inputs(stream=40), L.weights(stream=40), kh, kw, (stride, stride), (pad, pad))

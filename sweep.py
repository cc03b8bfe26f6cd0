"""Stage-by-stage timings of libdab on the five synthetic workload configurations.

`python sweep.py [--configs 1,2,3,4,5,net] [--batch5 256]` prints one JSON line per
(config, layer or point, stage): device time by CUDA events (best of a few repetitions after warm-up), the
stage's throughput and its fraction of the relevant roofline (HBM copy bandwidth for binarize and pack; for the
contraction, whichever kernel runs, alu_frac is its rate over the bound of the population-count kernel's
instruction mix, so values above 1 are the tensor-core kernel beating the integer pipes).  `net` times whole networks
(dab_network_forward: Sketch-A-Net-shaped at batch 1 = latency, AlexNet- and ResNet-18-shaped at batch 32).
bench.py is the benchmark of record; this is the wider table.
"""
from __future__ import annotations

import argparse
import json
import os
import sys

sys.path.insert(0, os.path.dirname(os.path.abspath(__file__)))

import numpy as np
import torch

import dab_synth
from dab_synth import configs
import paper_1804_02941_b200 as dab

ROOT = os.path.dirname(os.path.abspath(__file__))
POPC_PER_CLK, WORDS_PER_POPC = 16, 1.5


def peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return float(d["hbm_gbs"]), float(d.get("sm_max_mhz", 1965.0)), "measured"
    return 6650.0, 1965.0, "fallback"


def timed(fn, reps=5, warm=2):
    for _ in range(warm):
        fn()
    torch.cuda.synchronize()
    best = float("inf")
    for _ in range(reps):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        fn()
        e1.record()
        torch.cuda.synchronize()
        best = min(best, e0.elapsed_time(e1))
    return best


def emit(**kw):
    print(json.dumps(kw), flush=True)


STAGES = None   # set of stage names to run (--stages), None: all
LAYERS = None   # set of layer names to run (--layers), None: all


def want_stage(name):
    return STAGES is None or name in STAGES


def conv_layer(cfg, L, stream, hbm, tops_peak, dense=False):
    if LAYERS is not None and L.name not in LAYERS:
        return
    dev = torch.device("cuda")
    x = torch.from_numpy(L.inputs(stream=stream, dense=dense)).to(dev)
    w = torch.from_numpy(L.weights(stream=stream)).to(dev)
    wd = dab.dab_binarize(w)
    desc = dab.make_desc(L.x_shape(), L.Cout, L.kh, L.kw, (L.stride, L.stride), (L.pad, L.pad))
    P, ld = L.patches, dab.dab_default_ld(L.n)
    pK = torch.empty(P, dtype=torch.int32, device=dev)
    pg, pd = torch.empty(P, device=dev), torch.empty(P, device=dev)
    pm = torch.empty((P, ld), dtype=torch.int32, device=dev)
    y = torch.empty((L.N, L.Cout, L.Ho, L.Wo), device=dev)
    wd_words = dab.dab_words_per_row(L.n)
    bytes_p = 4 * x.numel() + P * (4 * wd_words + 12)
    bytes_w = L.Cout * (4 * L.n + 4 * wd_words + 12)
    common = dict(config=cfg, layer=L.name, n=L.n, patches=P, filters=L.Cout, inputs="dense" if dense else "relu60")
    if want_stage("binarize_filters"):
        t_w = timed(lambda: dab.dab_binarize_into(w, wd.K, wd.alpha, wd.beta, wd.mask, wd.flags))
        emit(stage="binarize_filters", ms=t_w, gbs=bytes_w / t_w / 1e6, hbm_frac=bytes_w / t_w / 1e6 / hbm, **common)
    if want_stage("sign_patches"):   # FBin-style input coding, for comparison
        t_s = timed(lambda: dab.dab_sign_patches(desc, x, pK, pg, pd, pm, None))
        emit(stage="sign_patches", ms=t_s, gbs=bytes_p / t_s / 1e6, hbm_frac=bytes_p / t_s / 1e6 / hbm, **common)
    t_p = t_c = None
    if want_stage("binarize_patches") or want_stage("contract"):
        t_p = timed(lambda: dab.dab_binarize_patches(desc, x, pK, pg, pd, pm, None))
        emit(stage="binarize_patches", ms=t_p, gbs=bytes_p / t_p / 1e6, hbm_frac=bytes_p / t_p / 1e6 / hbm, **common)
    if want_stage("contract"):
        t_c = timed(lambda: dab.dab_binary_conv_contract(desc, pm, pK, pg, pd, wd, y, None))
        emit(stage="contract", ms=t_c, tops_equiv=L.binary_ops / t_c / 1e9, alu_frac=L.binary_ops / t_c / 1e9 / tops_peak,
             **common)
        emit(stage="conv_total", ms=t_p + t_c, tops_equiv=L.binary_ops / (t_p + t_c) / 1e9, **common)
    if want_stage("wbin_conv"):
        # weights-only binarized layer: fp32 activations x two-level filters, four int8 tensor-core products per MAC
        ws = torch.empty(dab.dab_wbin_conv_workspace(desc), dtype=torch.uint8, device=dev)
        t_b = timed(lambda: dab.dab_wbin_conv(x, wd, L.kh, L.kw, (L.stride, L.stride), (L.pad, L.pad), y=y, workspace=ws))
        macs = L.binary_ops / 2
        emit(stage="wbin_conv", ms=t_b, tmacs=macs / t_b / 1e9, int8_tops=8 * macs / t_b / 1e9,
             int8_frac=8 * macs / t_b / 1e9 / int8_peak(), **common)


def int8_peak():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        return 2.0 * float(json.load(open(p))["bf16_tflops_sustained"])
    return 2800.0


def gemm_point(m, k, hbm, tops_peak):
    dev = torch.device("cuda")
    A, B = configs.config3_operands(m, k)
    Ad, Bd = torch.from_numpy(A).to(dev), torch.from_numpy(B).to(dev)
    a, b = dab.dab_binarize(Ad), dab.dab_binarize(Bd)
    Cm = torch.empty((m, m), device=dev)
    t_b = timed(lambda: dab.dab_binarize_into(Ad, a.K, a.alpha, a.beta, a.mask, a.flags))
    t_g = timed(lambda: dab.dab_binary_gemm(a, b, out=Cm))
    wdw = dab.dab_words_per_row(k)
    bytes_b = m * (4 * k + 4 * wdw + 12)
    ops = 2 * m * m * k
    emit(config=3, stage="binarize", M=m, n=k, ms=t_b, gbs=bytes_b / t_b / 1e6, hbm_frac=bytes_b / t_b / 1e6 / hbm,
         inputs="laplace dense")
    emit(config=3, stage="gemm", M=m, N=m, n=k, ms=t_g, tops_equiv=ops / t_g / 1e9, alu_frac=ops / t_g / 1e9 / tops_peak,
         store_gbs=4 * m * m / t_g / 1e6)


def pack_point(rows, n, hbm):
    dev = torch.device("cuda")
    bits = (torch.rand((rows, n), device=dev) < 0.4).to(torch.uint8)
    ld = dab.dab_default_ld(n)
    mask = torch.empty((rows, ld), dtype=torch.int32, device=dev)
    K = torch.empty(rows, dtype=torch.int32, device=dev)
    import ctypes as C
    L = dab.lib()
    st = C.c_void_p(torch.cuda.current_stream().cuda_stream)
    fn = lambda: L.dab_pack(C.c_void_p(bits.data_ptr()), rows, n, n, C.c_void_p(mask.data_ptr()), ld,
                            C.c_void_p(K.data_ptr()), st)
    t = timed(fn)
    b = rows * (n + 4 * dab.dab_words_per_row(n) + 4)
    emit(stage="pack", rows=rows, n=n, ms=t, gbs=b / t / 1e6, hbm_frac=b / t / 1e6 / hbm)


def network_point(name, build, batch):
    from dab_synth import networks
    layers, shape = build()
    net = dab.Network(layers)
    x = torch.from_numpy(networks.network_input(shape, batch, stream=1)).cuda()
    t = timed(lambda: dab.dab_network_forward(net, x), reps=5, warm=2)
    emit(stage="network_forward", network=name, batch=batch, ms=t, images_per_s=batch / t * 1e3, layers=len(layers),
         binarized_layers=sum(l["kind"] == "conv_binary" for l in layers))


def table(path):
    """Markdown summary of the JSON lines an earlier run printed (python sweep.py ... > lines; python sweep.py --table lines)."""
    recs = [json.loads(l) for l in open(path) if l.lstrip().startswith("{")]
    peaks = next((r["peaks"] for r in recs if "peaks" in r), {})
    int8_peak = None
    try:
        int8_peak = 2.0 * json.load(open(os.path.join(ROOT, "MEASURED_PEAKS.json")))["bf16_tflops_sustained"]
    except Exception:
        pass
    print("| config | layer / point | stage | ms | rate | fraction |")
    print("|---|---|---|---|---|---|")
    nets = []
    for r in recs:
        st = r.get("stage")
        if st is None:
            continue
        if st == "network_forward":
            nets.append(r)
            continue
        if "layer" in r:
            where = "%s%s (n=%d, %d patches, %d filters)" % (r["layer"], " dense" if r.get("inputs", "").startswith("dense") else "",
                                                             r["n"], r["patches"], r["filters"])
        elif st == "pack":
            where = "%d x %d bytes" % (r["rows"], r["n"])
        else:
            where = "M=N=%d, n=%d" % (r["M"], r["n"])
        if "gbs" in r:
            rate, frac = "%.1f GB/s" % r["gbs"], "hbm %.4f" % r["hbm_frac"]
        elif "tmacs" in r:
            rate, frac = "%.1f TMAC/s" % r["tmacs"], "int8 %.3f" % r["int8_frac"]
        else:
            rate = "%.1f TOPS-eq" % r["tops_equiv"]
            frac = ""
            if "alu_frac" in r:
                frac = "alu %.2f" % r["alu_frac"] + (", int8 %.3f" % (r["tops_equiv"] / int8_peak) if int8_peak else "")
        name = {"conv_total": "patches + contract", "binarize": "binarize rows"}.get(st, st)
        print("| %s | %s | %s | %.4f | %s | %s |" % (r.get("config", "pack"), where, name, r["ms"], rate, frac))
    if nets:
        print("\n| network | batch | layers (binarized) | ms | images/s |\n|---|---|---|---|---|")
        for r in nets:
            print("| %s | %d | %d (%d) | %.3f | %.0f |" % (r["network"], r["batch"], r["layers"], r["binarized_layers"], r["ms"], r["images_per_s"]))
    if peaks:
        print("\nPeaks used: HBM %.1f GB/s (%s); population-count bound %.1f TOPS-equiv (%s)%s." % (
            peaks["hbm_gbs"], peaks["source"], peaks["contraction_tops_equiv"], peaks["contraction_peak"],
            "; int8 tensor peak %.0f TOPS" % int8_peak if int8_peak else ""))


def main():
    if len(sys.argv) == 3 and sys.argv[1] == "--table":
        return table(sys.argv[2])
    ap = argparse.ArgumentParser()
    ap.add_argument("--configs", default="1,2,3,4,5")
    ap.add_argument("--batch5", type=int, default=256)
    ap.add_argument("--contraction", default="auto", choices=["auto", "tensor", "popc"])
    ap.add_argument("--patch-coder", default="auto", choices=["auto", "sort", "hist", "pixel"])
    ap.add_argument("--stages", default="", help="comma-separated stage names of the convolution layers to run (default all)")
    ap.add_argument("--layers", default="", help="comma-separated layer names to run (default all)")
    args = ap.parse_args()
    global STAGES, LAYERS
    STAGES = set(args.stages.split(",")) if args.stages else None
    LAYERS = set(args.layers.split(",")) if args.layers else None
    dab.dab_set_contraction({"auto": dab.CONTRACT_AUTO, "tensor": dab.CONTRACT_TENSOR, "popc": dab.CONTRACT_POPC}[args.contraction])
    dab.dab_set_patch_coder({"auto": dab.PATCHES_AUTO, "sort": dab.PATCHES_SORT, "hist": dab.PATCHES_HIST, "pixel": dab.PATCHES_PIXEL}[args.patch_coder])
    want = set(args.configs.split(","))
    hbm, mhz, src = peaks()
    SM_COUNT = torch.cuda.get_device_properties(0).multi_processor_count
    tops_peak = POPC_PER_CLK * WORDS_PER_POPC * SM_COUNT * mhz * 1e6 * 64 / 1e12
    emit(contraction=args.contraction)
    emit(peaks=dict(hbm_gbs=hbm, source=src, contraction_tops_equiv=tops_peak,
                    contraction_peak="16 popc/clk/SM x 1.5 words/popc x %d SMs x %.0f MHz x 64" % (SM_COUNT, mhz)))
    if "1" in want:
        conv_layer(1, configs.config1()[0], 0, hbm, tops_peak)
    if "2" in want:
        for i, L in enumerate(configs.config2()):
            conv_layer(2, L, i, hbm, tops_peak)
    if "3" in want:
        for m, k in configs.CONFIG3_POINTS:
            gemm_point(m, k, hbm, tops_peak)
        pack_point(65536, 4608, hbm)
        pack_point(802816, 576, hbm)
    if "4" in want:
        for i, L in enumerate(configs.config4()):
            conv_layer(4, L, 20 + i, hbm, tops_peak)
    if "5" in want:
        seen = set()
        for i, L in enumerate(configs.config5(args.batch5)):
            key = (L.C, L.H, L.Cout, L.stride)
            if key in seen:
                continue
            seen.add(key)
            conv_layer(5, L, i, hbm, tops_peak)
        conv_layer(5, configs.config5(args.batch5)[0], 50, hbm, tops_peak, dense=True)
    if "net" in want:
        from dab_synth import networks
        network_point("sketch_a_net", networks.sketch_a_net, 1)
        network_point("alexnet_like", networks.alexnet_like, 32)
        network_point("resnet18_like", networks.resnet18_like, 32)


if __name__ == "__main__":
    main()

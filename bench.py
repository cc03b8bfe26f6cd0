#!/usr/bin/env python
"""Benchmark of the DAB-Net inference hot path on B200.

A step is one pass of the whole path over one batch: for each of the 16 binarized 3x3 convolutions of the
ResNet-18-shaped stack (batch 256), binarize the filters, binarize every input patch, contract the packed
masks with the rescale fused in.  Every layer gets its own synthetic post-ReLU input (60 % exact zeros).
Prints ONE JSON line.  `--impl reference` times the CPU checker on a bounded sample instead.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import sys
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "binary_conv_tops_equiv"
UNIT = "TOPS-equiv (2*M*N*n binary ops per second / 1e12)"
L2_BYTES = 126 * 1024 * 1024
POPC_PER_CLK_PER_SM = 16          # integer population counts per clock per SM
WORDS_PER_POPC = 1.5              # the contraction compresses 3 AND-ed words into 2 population counts


# Sources of the patch coder: a measured DRAM-traffic record is only quoted while these files are unchanged.
PATCH_CODER_SOURCES = ("pixhist.cu", "patches.cu", "rowcode.cuh", "histcode.cuh", "common.cuh")
TRAFFIC_RECORD = os.path.join(ROOT, "profiles", "patch_coder_dram_traffic.json")


def patch_coder_source_hash() -> str:
    import hashlib
    h = hashlib.sha256()
    for name in PATCH_CODER_SOURCES:
        with open(os.path.join(ROOT, "paper_1804_02941_b200", "csrc", name), "rb") as f:
            h.update(f.read())
    return h.hexdigest()


def measured_patch_coder_traffic(layer_names, batch, dense):
    """Average DRAM bytes per patch-coder launch from the committed profiler record, or None when there is no record
    for this workload or the kernels have changed since it was taken."""
    try:
        with open(TRAFFIC_RECORD) as f:
            rec = json.load(f)
        if rec.get("source_sha256") != patch_coder_source_hash() or rec.get("batch") != batch or bool(rec.get("dense")) != bool(dense):
            return None
        per_layer = rec["dram_bytes_per_launch"]
        return sum(per_layer[n] for n in layer_names) / len(layer_names)
    except (OSError, KeyError, ValueError):
        return None


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="dab", choices=["dab", "reference"])
    ap.add_argument("--batch", type=int, default=256, help="images per step and per GPU (256 = the named workload)")
    ap.add_argument("--dense", action="store_true", help="N(0,1) inputs without zeros instead of post-ReLU inputs")
    ap.add_argument("--layers", default="", help="comma-separated layer names (e.g. l1_0,l4_1) to run a subset; "
                    "the default is the whole workload")
    ap.add_argument("--contraction", default="auto", choices=["auto", "tensor", "popc"],
                    help="contraction kernel: auto (tensor cores except on tiny problems; every layer of this workload takes "
                         "them), tensor (forced) or popc (AND + population counts)")
    ap.add_argument("--patch-coder", default="auto", choices=["auto", "sort", "hist", "pixel"],
                    help="patch coder: auto (pixel-histogram coder wherever patches overlap), sort (full sort per patch), "
                         "hist (histogram-pruned search per patch) or pixel (pixel-histogram coder wherever it applies)")
    ap.add_argument("--filters", default="side", choices=["side", "inline"],
                    help="side: the filter coding of all layers runs on a second stream beside the patch coding (each "
                         "contraction waits for its filters); inline: everything on one stream, layer by layer")
    ap.add_argument("--e2e-steps", type=int, default=10)
    ap.add_argument("--cpu-sample-batch", type=int, default=8)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-wbin", action="store_true", help="skip the weights-only binarized pass over the same layers")
    return ap.parse_args()


def load_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        with open(p) as f:
            d = json.load(f)
        return float(d["hbm_gbs"]), "measured (MEASURED_PEAKS.json)", float(d.get("sm_max_mhz", 1965.0))
    return 6650.0, "fallback (earlier measurement on this pool)", 1965.0


def load_int8_peak():
    """Dense int8 tensor peak in TOPS: the measured sustained bf16 GEMM rate x the nominal int8:bf16 ratio (4.5 : 2.25)."""
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        with open(p) as f:
            d = json.load(f)
        return 2.0 * float(d["bf16_tflops_sustained"]), "2 x measured sustained bf16 GEMM rate (MEASURED_PEAKS.json)"
    return 2.0 * 1400.0, "2 x fallback sustained bf16 GEMM rate"


class ClockSampler:
    """Samples SM clock and throttle reasons through NVML (read-only) in a thread while the timed region runs."""
    REASONS = {0x8: "hw_slowdown", 0x40: "hw_thermal_slowdown", 0x20: "sw_thermal_slowdown", 0x4: "sw_power_cap"}

    def __init__(self, index: int, period_s: float = 0.01):
        self.index, self.period = index, period_s
        self.thread, self.stop_flag = None, False
        self.sm, self.mx, self.reasons = [], None, set()

    def _run(self, nv, handle):
        while not self.stop_flag:
            try:
                self.sm.append(float(nv.nvmlDeviceGetClockInfo(handle, nv.NVML_CLOCK_SM)))
                bits = int(nv.nvmlDeviceGetCurrentClocksEventReasons(handle)) if hasattr(nv, "nvmlDeviceGetCurrentClocksEventReasons") \
                    else int(nv.nvmlDeviceGetCurrentClocksThrottleReasons(handle))
                for bit, name in self.REASONS.items():
                    if bits & bit:
                        self.reasons.add(name)
            except Exception:
                pass
            time.sleep(self.period)

    def start(self):
        try:
            import threading
            import pynvml as nv
            nv.nvmlInit()
            # CUDA_VISIBLE_DEVICES may renumber the devices: find the one torch uses by its PCI bus id
            import torch
            bus = torch.cuda.get_device_properties(self.index).pci_bus_id if hasattr(torch.cuda.get_device_properties(self.index), "pci_bus_id") else None
            handle = None
            if bus is not None:
                for i in range(nv.nvmlDeviceGetCount()):
                    h = nv.nvmlDeviceGetHandleByIndex(i)
                    if int(nv.nvmlDeviceGetPciInfo(h).bus) == int(bus):
                        handle = h
                        break
            if handle is None:
                handle = nv.nvmlDeviceGetHandleByIndex(self.index)
            self.mx = float(nv.nvmlDeviceGetMaxClockInfo(handle, nv.NVML_CLOCK_SM))
            self.thread = threading.Thread(target=self._run, args=(nv, handle), daemon=True)
            self.thread.start()
        except Exception:
            self.thread = None

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": self.mx, "reasons": [], "samples": 0}
        if self.thread is None:
            return out
        self.stop_flag = True
        self.thread.join(timeout=2)
        if self.sm:
            out.update(sm_mhz=statistics.median(self.sm), samples=len(self.sm))
        out["reasons"] = sorted(self.reasons)
        return out


def max_over_ranks(value: float, world: int, device=None) -> float:
    """Slowest rank's time (the job is as slow as its slowest replica)."""
    if world <= 1:
        return float(value)
    import torch
    import torch.distributed as dist
    t = torch.tensor([value], dtype=torch.float64, device=device if device is not None else "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def aggregate_throughput(units_per_rank_step: float, steps: int, seconds: float, world: int) -> float:
    """Whole-job throughput of `world` independent replicas, each doing `steps` steps in `seconds` (max over ranks)."""
    return world * units_per_rank_step * steps / seconds


def dist_env():
    return int(os.environ.get("RANK", "0")), int(os.environ.get("LOCAL_RANK", "0")), int(os.environ.get("WORLD_SIZE", "1"))


# ------------------------------------------------------------------------------------------------------------
# CPU checker timing (the reference arm and the cpu_baseline leg)
# ------------------------------------------------------------------------------------------------------------
def oracle_pass(layers, inputs, weights):
    """One pass of the checker over the sample; returns (seconds, binary ops)."""
    import oracle
    t0 = time.perf_counter()
    ops = 0
    for L, x, w in zip(layers, inputs, weights):
        wb = oracle.binarize(w)
        oracle.conv(x, wb.e, wb.alpha, wb.beta, L.kh, L.kw, (L.stride, L.stride), (L.pad, L.pad), details=False)
        ops += L.binary_ops
    return time.perf_counter() - t0, ops


def oracle_sample(batch, dense):
    import oracle
    from dab_synth import configs
    threads = os.cpu_count() or 1
    oracle.set_threads(threads)
    layers = configs.config5(batch)
    inputs = [L.inputs(stream=i, dense=dense) for i, L in enumerate(layers)]
    weights = [L.weights(stream=i) for i, L in enumerate(layers)]
    return layers, inputs, weights, threads


def run_reference(args):
    rank, _, world = dist_env()
    if rank != 0:
        return
    batch = 2
    layers, inputs, weights, threads = oracle_sample(batch, args.dense)
    for _ in range(max(args.warmup, 0)):
        oracle_pass(layers, inputs, weights)
    t, ops = 0.0, 0
    for _ in range(args.steps):
        dt, o = oracle_pass(layers, inputs, weights)
        t += dt
        ops += o
    value = ops / t / 1e12
    sample = "all 16 layers of the workload at batch %d (of 256) per step, every patch and filter" % batch
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": 1e3 * t / args.steps, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": workload_config(args, batch_override=batch),
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


def patch_launches(L, coder):
    """Kernels one dab_binarize_patches call launches (some end at once when nothing was handed to them)."""
    n = L.n
    if n <= 256:
        return 1
    pixel = n <= 8192 and L.kh * L.kw >= 4 and L.patches >= 1024
    if coder == "pixel" or (coder == "auto" and pixel):
        return 2                      # pixel-histogram coder, then the kernel that sorts the patches it marked
    if coder == "auto":
        return 3                      # sort-based coder, histogram coder on the dense tiles, group kernel on the rest
    if coder == "hist":
        return 2
    return 2 if n <= 576 else 1       # one warp per patch, then the group kernel on the tiles marked dense


def select_layers(layers, args):
    if not args.layers:
        return layers
    want = set(args.layers.split(","))
    sel = [L for L in layers if L.name in want]
    if not sel:
        raise SystemExit("no layer named in --layers; names: " + ",".join(L.name for L in layers))
    return sel


def workload_config(args, batch_override=None):
    b = batch_override if batch_override is not None else args.batch
    return {"layers": args.layers or "all 16",
            "workload": "config 5: ResNet-18-shaped stack of 16 binarized 3x3 convolutions (64/128/256/512 channels, "
                        "56/28/14/7 px), per-filter and per-patch distribution-aware binarization, AND-popcount contraction",
            "batch_per_gpu": b, "inputs": "dense N(0,1)" if args.dense else "post-ReLU half-normal, 60% exact zeros",
            "weights": "N(0, 0.02^2)", "patch_coder": args.patch_coder, "l2": "no flush: a step streams >3 GB of distinct inputs and outputs, L2 is 126 MB",
            "filters": ("coded on a second stream beside the patch coding, inside the timed region" if getattr(args, "filters", "side") == "side"
                        else "coded on the same stream, layer by layer"),
            "parallelism": "replicas" if args.gpus > 1 else "single GPU"}


# ------------------------------------------------------------------------------------------------------------
# The CUDA path
# ------------------------------------------------------------------------------------------------------------
def run_dab(args):
    import numpy as np
    import torch
    import paper_1804_02941_b200 as dab
    from dab_synth import configs

    rank, local_rank, world = dist_env()
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device; there is no CPU fallback")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)
    dab.lib()
    dab.dab_set_contraction({"auto": dab.CONTRACT_AUTO, "tensor": dab.CONTRACT_TENSOR, "popc": dab.CONTRACT_POPC}[args.contraction])
    dab.dab_set_patch_coder({"auto": dab.PATCHES_AUTO, "sort": dab.PATCHES_SORT, "hist": dab.PATCHES_HIST, "pixel": dab.PATCHES_PIXEL}[args.patch_coder])
    hbm_peak, peak_src, sm_max_mhz = load_peaks()
    SM_COUNT = torch.cuda.get_device_properties(dev).multi_processor_count

    layers = select_layers(configs.config5(args.batch), args)
    # one host tensor per distinct input shape (pinned: it is also the source of the end-to-end copies);
    # every layer gets its own device copy, shifted along the batch axis so that no two layers share memory
    host_x = {}
    for L in layers:
        if L.x_shape() not in host_x:
            host_x[L.x_shape()] = torch.from_numpy(L.inputs(stream=100 * rank + len(host_x), dense=args.dense)).pin_memory()
    stream = torch.cuda.Stream(device=dev)
    work = []
    max_patches_words = max(L.patches * dab.dab_default_ld(L.n) for L in layers)
    max_patches = max(L.patches for L in layers)
    max_y = max(L.patches * L.Cout for L in layers)
    pK = torch.empty(max_patches, dtype=torch.int32, device=dev)
    pg = torch.empty(max_patches, dtype=torch.float32, device=dev)
    pd = torch.empty(max_patches, dtype=torch.float32, device=dev)
    pm_flat = torch.empty(max_patches_words, dtype=torch.int32, device=dev)
    y_flat = torch.empty(max_y, dtype=torch.float32, device=dev)
    for i, L in enumerate(layers):
        x = torch.roll(host_x[L.x_shape()].to(dev), shifts=i, dims=0).contiguous()
        w = torch.from_numpy(L.weights(stream=100 * rank + i)).to(dev)
        ld = dab.dab_default_ld(L.n)
        wc = dab.Coded(torch.empty((L.Cout, ld), dtype=torch.int32, device=dev), torch.empty(L.Cout, dtype=torch.int32, device=dev),
                       torch.empty(L.Cout, dtype=torch.float32, device=dev), torch.empty(L.Cout, dtype=torch.float32, device=dev),
                       torch.empty(L.Cout, dtype=torch.int32, device=dev), L.n)
        desc = dab.make_desc(L.x_shape(), L.Cout, L.kh, L.kw, (L.stride, L.stride), (L.pad, L.pad))
        pm = pm_flat[: L.patches * ld].view(L.patches, ld)
        y = y_flat[: L.patches * L.Cout].view(L.N, L.Cout, L.Ho, L.Wo)
        work.append((L, x, w, wc, desc, pm, y))
    torch.cuda.synchronize()

    side = torch.cuda.Stream(device=dev) if args.filters == "side" else stream

    def step(events=None):
        # The filters of a layer depend on nothing but the weights, so all sixteen filter matrices are coded on a
        # second stream while the first layers' patches are coded; the second stream starts when the work queued
        # before this step is done (the coded filters of the step before are no longer read) and each contraction
        # waits for the event behind its own filters.  Everything stays inside the timed region.
        timed = events is not None
        joins = []
        if side is not stream:
            fork = torch.cuda.Event()
            fork.record(stream)
            side.wait_event(fork)
            for (L, x, w, wc, desc, pm, y) in work:
                f0 = torch.cuda.Event(enable_timing=timed)
                f1 = torch.cuda.Event(enable_timing=timed)
                f0.record(side)
                dab.dab_binarize_into(w, wc.K, wc.alpha, wc.beta, wc.mask, wc.flags, stream=side)
                f1.record(side)
                joins.append((f0, f1))
        for li, (L, x, w, wc, desc, pm, y) in enumerate(work):
            ev = [torch.cuda.Event(enable_timing=timed) for _ in range(4)]
            if side is stream:
                ev[0].record(stream)
                dab.dab_binarize_into(w, wc.K, wc.alpha, wc.beta, wc.mask, wc.flags, stream=stream)
            else:
                ev[0] = joins[li][0]
            ev[1].record(stream)
            dab.dab_binarize_patches(desc, x, pK, pg, pd, pm, None, stream=stream)
            ev[2].record(stream)
            if side is not stream:
                stream.wait_event(joins[li][1])
            dab.dab_binary_conv_contract(desc, pm, pK, pg, pd, wc, y, None, stream=stream)
            ev[3].record(stream)
            if timed:
                events.append((li, ev, joins[li][1] if side is not stream else ev[1]))

    def barrier():
        if world > 1:
            import torch.distributed as dist
            dist.barrier()

    for _ in range(max(args.warmup, 3)):
        step()
    stream.synchronize()

    sampler = ClockSampler(local_rank)
    sampler.start()
    events = []
    barrier()
    torch.cuda.synchronize()
    t_start, t_end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t_start.record(stream)
    for _ in range(args.steps):
        step(events)
    t_end.record(stream)
    torch.cuda.synchronize()
    barrier()
    clocks = sampler.stop()
    total_ms = t_start.elapsed_time(t_end)
    total_ms = max_over_ranks(total_ms, world, dev)

    ops_per_step = sum(L.binary_ops for L in layers)
    value = aggregate_throughput(ops_per_step, args.steps, total_ms * 1e-3, world) / 1e12

    # per-kernel device time inside the timed region
    k_ms = {"binarize_rows": 0.0, "binarize_patches": 0.0, "contract": 0.0}
    for li, ev, filters_done in events:
        k_ms["binarize_rows"] += ev[0].elapsed_time(filters_done)
        k_ms["binarize_patches"] += ev[1].elapsed_time(ev[2])
        k_ms["contract"] += ev[2].elapsed_time(ev[3])
    launches_per_kind = args.steps * len(layers)

    # algorithmic bytes of the patch coder: every input element read once (4 B), per patch the packed mask
    # (4*ceil(n/32) B) and K, gamma, delta (12 B) written
    patch_bytes = sum(4 * L.N * L.C * L.H * L.W + L.patches * (4 * dab.dab_words_per_row(L.n) + 12) for L in layers)
    binarize_gbs = patch_bytes * args.steps / (k_ms["binarize_patches"] * 1e-3) / 1e9
    traffic = measured_patch_coder_traffic([L.name for L in layers], args.batch, args.dense) if args.patch_coder == "auto" else None
    roofline = {"kernel": "binarize_patches_pixhist_kernel (+ binarize_patches_fixup_kernel, which finds nothing marked on "
                          "this workload)", "bound": "hbm", "achieved": binarize_gbs,
                "peak": hbm_peak, "unit": "GB/s", "frac": binarize_gbs / hbm_peak, "traffic": traffic,
                "traffic_note": "dram__bytes_read.sum + dram__bytes_write.sum per layer launch, average over the layers, from "
                                "profiles/patch_coder_dram_traffic.json; null when the coder's sources have changed since "
                                "that capture", "peak_source": peak_src,
                "algorithmic_bytes_per_launch_avg": patch_bytes / len(layers),
                "avg_launch_ms": k_ms["binarize_patches"] / launches_per_kind,
                "share_of_step": k_ms["binarize_patches"] / total_ms}

    # contraction: integer AND/POPC/IADD; peak measured live with independent popcount chains
    sink = torch.empty(SM_COUNT * 8 * 256, dtype=torch.int32, device=dev)
    with torch.cuda.stream(stream):
        dab.dab_popc_probe(SM_COUNT * 8, 2000, sink, stream=stream)
        p0, p1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        p0.record(stream)
        dab.dab_popc_probe(SM_COUNT * 8, 20000, sink, stream=stream)
        p1.record(stream)
    stream.synchronize()
    probe_words = SM_COUNT * 8 * 256 * 20000 * 16 / (p0.elapsed_time(p1) * 1e-3)
    contract_tops = ops_per_step * args.steps / (k_ms["contract"] * 1e-3) / 1e12
    popc_peak_measured = probe_words * 64 / 1e12     # plain AND+POPC+IADD chains: one count per word
    popc_peak_derived = POPC_PER_CLK_PER_SM * WORDS_PER_POPC * SM_COUNT * sm_max_mhz * 1e6 * 64 / 1e12
    store_gbs = sum(4 * L.patches * L.Cout for L in layers) * args.steps / (k_ms["contract"] * 1e-3) / 1e9
    common = {"achieved": contract_tops, "unit": "TOPS-equiv", "avg_launch_ms": k_ms["contract"] / launches_per_kind,
              "share_of_step": k_ms["contract"] / total_ms, "output_store_gbs": store_gbs,
              "output_store_frac_of_hbm": store_gbs / hbm_peak}
    if args.contraction != "popc":
        int8_peak, int8_src = load_int8_peak()
        roofline_contract = {"kernel": "binary_gemm_mma_kernel", "bound": "tensor", "peak": int8_peak,
                             "frac": contract_tops / int8_peak, "peak_source": int8_src,
                             "popc_bound": popc_peak_derived, "frac_of_popc_bound": contract_tops / popc_peak_derived,
                             "popc_bound_source": "the integer-pipe bound of the population-count kernel (16 popc/clk/SM x "
                                                  "1.5 words per popc x SMs x max clock x 64): what the same contraction "
                                                  "could reach without tensor cores",
                             "note": "kind::i8 on masks expanded to bytes 0 / -1; the kernel's time goes to expanding mask words to bytes, the fp64 "
                                     "rescale of every count and the output store, not to the tensor pipe", **common}
    else:
        roofline_contract = {"kernel": "binary_gemm_kernel", "bound": "alu", "peak": popc_peak_derived,
                             "frac": contract_tops / popc_peak_derived,
                             "plain_popc_rate_measured_by_probe": popc_peak_measured,
                             "peak_source": "16 popc/clk/SM x 1.5 words per popc (3:2 carry-save) x 148 SMs x %.0f MHz x 64 "
                                            "binary ops per word" % sm_max_mhz, **common}

    # end to end: host tensors in pinned memory, copies inside the timed region, through the host entry point
    e2e = None
    if not args.no_e2e:
        max_ws = max(dab.dab_binary_conv_host_workspace(desc) for (_, _, _, _, desc, _, _) in work)
        # two workspaces, taken in turn: a layer is queued while the one before it is still copying out
        wss = [torch.empty(max_ws, dtype=torch.uint8, device=dev) for _ in range(2)]
        y_hosts = [torch.empty(max_y, dtype=torch.float32).pin_memory() for _ in range(2)]
        h2d = sum(4 * L.N * L.C * L.H * L.W for L in layers)
        d2h = sum(4 * L.patches * L.Cout for L in layers)

        def e2e_step():
            for li, (L, x, w, wc, desc, pm, y) in enumerate(work):
                dab.dab_binarize_into(w, wc.K, wc.alpha, wc.beta, wc.mask, wc.flags, stream=stream)
                yh = y_hosts[li & 1][: L.patches * L.Cout].view(L.N, L.Cout, L.Ho, L.Wo)
                dab.dab_binary_conv_host(host_x[L.x_shape()], wc, L.kh, L.kw, (L.stride, L.stride), (L.pad, L.pad),
                                         y_host=yh, workspace=wss[li & 1], stream=stream, wait=False)
            dab.dab_binary_conv_host_wait(stream)
        e2e_step()
        barrier()
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        for _ in range(args.e2e_steps):
            e2e_step()
        torch.cuda.synchronize()
        e2e_s = time.perf_counter() - t0
        e2e_s = max_over_ranks(e2e_s, world, dev)
        # The floor the copies alone set: the same bytes per step moved by plain asynchronous copies from and to the
        # same pinned buffers, both directions at once on two streams, nothing computed.
        s_in, s_out = torch.cuda.Stream(device=dev), torch.cuda.Stream(device=dev)
        x_dev = {shape: torch.empty(shape, dtype=torch.float32, device=dev) for shape in host_x}

        def copies_only():
            for li, (L, x, w, wc, desc, pm, y) in enumerate(work):
                with torch.cuda.stream(s_in):
                    x_dev[L.x_shape()].copy_(host_x[L.x_shape()], non_blocking=True)
                with torch.cuda.stream(s_out):
                    y_hosts[li & 1][: L.patches * L.Cout].copy_(y_flat[: L.patches * L.Cout], non_blocking=True)
        copies_only()
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        for _ in range(3):
            copies_only()
        torch.cuda.synchronize()
        floor_ms = 1e3 * (time.perf_counter() - t0) / 3
        e2e = {"value": aggregate_throughput(ops_per_step, args.e2e_steps, e2e_s, world) / 1e12, "unit": UNIT, "h2d_bytes_per_step": h2d,
               "d2h_bytes_per_step": d2h, "steps": args.e2e_steps, "ms_per_step": 1e3 * e2e_s / args.e2e_steps,
               "pcie_floor_ms": floor_ms, "over_pcie_floor": 1e3 * e2e_s / args.e2e_steps / floor_ms,
               "pcie_floor_note": "the step's %.2f GB in and %.2f GB out as plain pinned-memory copies on two streams at once, no "
                                  "kernels: %.1f GB/s in, %.1f GB/s out" % (h2d / 1e9, d2h / 1e9, h2d / floor_ms / 1e6, d2h / floor_ms / 1e6)}

    # The paper's weights-only binarized networks on the same layers: fp32 activations against the coded filters
    # (dab_wbin_conv, four int8 tensor-core products per multiply-accumulate).  Reported beside the headline, not in it.
    wbin = None
    if not args.no_wbin:
        wws = torch.empty(max(dab.dab_wbin_conv_workspace(desc) for (_, _, _, _, desc, _, _) in work), dtype=torch.uint8, device=dev)

        def wbin_step():
            for (L, x, w, wc, desc, pm, y) in work:
                dab.dab_wbin_conv(x, wc, L.kh, L.kw, (L.stride, L.stride), (L.pad, L.pad), y=y, workspace=wws, stream=stream)
        for _ in range(3):
            wbin_step()
        stream.synchronize()
        w0, w1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        w0.record(stream)
        for _ in range(args.steps):
            wbin_step()
        w1.record(stream)
        stream.synchronize()
        wms = w0.elapsed_time(w1) / args.steps
        int8_peak, int8_src = load_int8_peak()
        macs = ops_per_step / 2
        wbin = {"kernel": "wbin_conv_kernel (+ wbin_pixmax_kernel)", "ms_per_step": wms, "tmacs": macs / wms / 1e9,
                "bound": "tensor", "achieved": 8 * macs / wms / 1e9, "unit": "int8 TOPS (4 byte planes x 2 ops per MAC)",
                "peak": int8_peak, "frac": 8 * macs / wms / 1e9 / int8_peak, "peak_source": int8_src,
                "gpu_launches": 2 * len(work) * args.steps}

    cpu_baseline = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        b = args.cpu_sample_batch
        ls, xs, wts, threads = oracle_sample(b, args.dense)
        dt, ops = oracle_pass(ls, xs, wts)
        cpu_baseline = {"value": ops / dt / 1e12, "unit": UNIT, "cores": threads, "kind": "oracle", "seconds": dt,
                        "sample": "all 16 layers at batch %d (of %d), every patch and filter, one pass" % (b, args.batch)}

    if rank == 0:
        out = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
               "warmup": max(args.warmup, 3), "ms_per_step": total_ms / args.steps, "higher_is_better": True,
               "scaling": "weak", "vs_baseline": None, "dtype": "s8 x s8 -> s32 tensor-core counts + f64 objective/rescale" if args.contraction != "popc"
               else "u32 popcount + f64 objective/rescale",
               "data": "synthetic", "config": workload_config(args), "clocks": clocks, "e2e": e2e,
               "gpu_launches": (2 * len(layers) + sum(patch_launches(L, args.patch_coder) for L in layers)) * args.steps,
               "kernel_ms_per_step": {k: v / args.steps for k, v in k_ms.items()},
               "kernel_ms_note": "device time between events around each stage; with --filters side the filter coding "
                                 "overlaps the patch coding, so the three do not add up to ms_per_step",
               "binarize_gbs": binarize_gbs, "roofline": roofline, "roofline_contraction": roofline_contract,
               "wbin": wbin, "cpu_baseline": cpu_baseline, "contraction_wait_failures": dab.dab_contraction_wait_failures()}
        print(json.dumps(out))
    if world > 1:
        import torch.distributed as dist
        dist.destroy_process_group()


def main():
    args = parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_dab(args)


if __name__ == "__main__":
    main()

#!/usr/bin/env python
"""Benchmark of the sparse-DNN SGD hot path on B200 (one process per GPU).

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl reference]

Default workload: the largest training configuration (65536 neurons x 1920 layers, 32 nonzeros per
row, minibatch 16).  A "step" is one pass of the whole path over one fresh minibatch: forward through
all layers, loss and output gradient, then backward product + masked gradient + weight update for
every layer.  Inference workloads time one sdnn_infer_batch call over all inputs per step.

Prints ONE JSON line (rank 0).  `value` = edges/s with inputs resident in HBM; `e2e` = the same metric
through the host-buffer entry point (pinned host inputs, loss / counts read back).  `roofline` is for
the dominant kernel, timed by events on the library's stream inside the timed steps.  `cpu_baseline`
times the float64 CPU oracle on a bounded slice of the same workload.  With --impl reference only the
oracle runs (rank 0; the other ranks exit).  Nothing here reads files outside the repository.
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import gen  # noqa: E402

ETA = 1e-3

# name -> (spec, kind, batch or tile, inputs per step)
WORKLOADS = {
    "cfg5": (gen.CFG5, "train", 16, 16),
    "cfg5-live": (gen.CFG5.live(), "train", 16, 16),
    "cfg3": (gen.CFG3, "train", 64, 64),
    "cfg3-live": (gen.CFG3.live(), "train", 64, 64),
    "cfg1-train": (gen.CFG1_TRAIN, "train", 1, 1),
    "cfg1-inf": (gen.CFG1_INF, "infer", 256, 256),
    "cfg2": (gen.CFG2, "infer", 1024, 60000),
    "cfg2-live": (gen.CFG2.live(), "infer", 1024, 60000),
    "cfg4": (gen.CFG4, "infer", 1024, 60000),
    "cfg4-live": (gen.CFG4.live(), "infer", 1024, 60000),
    # config 4 with the neurons of every inner layer renumbered at random: the block structure is there but hidden
    "cfg4-shuffled": (gen.CFG4.shuffled(), "infer", 1024, 60000),
    "cfg4-live-shuffled": (gen.CFG4.live().shuffled(), "infer", 1024, 60000),
    # the paper's own training setup (Section 6): sigmoid, weights uniform in [-1, 1], eta = 0.01
    "cfg3-paper": (gen.CFG3.paper_setup(), "train", 64, 64),
    "cfg5-paper": (gen.CFG5.paper_setup(), "train", 16, 16),
    "cfg1-paper": (gen.CFG1_TRAIN.paper_setup(), "train", 1, 1),
}


def setup_of(spec):
    """(activation name, activation code, eta) of a workload: the paper's setup for the '-paper' nets."""
    return ("sigmoid", 1, 1e-2) if spec.name.endswith("-paper") else ("clamped_relu", 0, ETA)


# dram__bytes_read.sum + dram__bytes_write.sum per launch from the ncu captures summarised under profiles/
# (training kernels: captured on a 48-layer slice of the same net, per-launch traffic does not depend on the depth)
NCU_TRAFFIC = {("cfg5", "backward_kernel"): 21.26e6 + 27.10e6, ("cfg5", "forward_kernel"): 17.07e6,      # backward: both launches of a layer
               ("cfg3", "backward_kernel"): 11.62e6 + 16.24e6, ("cfg3", "forward_kernel"): 7.42e6}


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        d = json.load(open(path))
        return float(d["hbm_gbs"]), "measured (MEASURED_PEAKS.json hbm_gbs)"
    return 6650.0, "fallback (6.65 TB/s, earlier measurement on this pool)"


class ClockSampler:
    """Samples SM clock and throttle reasons of one GPU through NVML while the timed region runs."""

    def __init__(self, index: int, period: float = 0.02):
        self.index, self.period = index, period
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop = threading.Event()
        self._thread = None
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.dev = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.dev, pynvml.NVML_CLOCK_SM)
        except Exception:
            self.nv = None

    NAMES = {0x1: "gpu_idle", 0x2: "applications_clocks_setting", 0x4: "sw_power_cap", 0x8: "hw_slowdown",
             0x10: "sync_boost", 0x20: "sw_thermal_slowdown", 0x40: "hw_thermal_slowdown",
             0x80: "hw_power_brake_slowdown", 0x100: "display_clock_setting"}

    def _run(self):
        nv = self.nv
        while not self._stop.is_set():
            try:
                self.samples.append(nv.nvmlDeviceGetClockInfo(self.dev, nv.NVML_CLOCK_SM))
                bits = nv.nvmlDeviceGetCurrentClocksEventReasons(self.dev)
                for bit, name in self.NAMES.items():
                    if bits & bit and name != "gpu_idle":
                        self.reasons.add(name)
            except Exception:
                pass
            time.sleep(self.period)

    def __enter__(self):
        if self.nv is not None:
            self._thread = threading.Thread(target=self._run, daemon=True)
            self._thread.start()
        return self

    def __exit__(self, *exc):
        self._stop.set()
        if self._thread:
            self._thread.join()

    def summary(self):
        if not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": ["unavailable"]}
        return {"sm_mhz": float(np.median(self.samples)), "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons),
                "samples": len(self.samples)}


def oracle_train_sample(spec, B, layers, steps, warmup, averaged=False):
    """Times the float64 oracle's train step on the first `layers` layers of the net (full N, full B)."""
    from oracle import OracleNet
    sl = spec.sliced(layers)
    act, _, eta = setup_of(spec)
    ora = OracleNet(*gen.network(sl), activation=act)
    times = []
    for s in range(warmup + steps):
        x0, y = gen.inputs(sl, B, step=s), gen.targets(sl, B, step=s)
        t = time.perf_counter()
        if averaged:
            ora.train_step_averaged(x0, y, eta)
        else:
            ora.train_step(x0, y, eta, keep=())
        dt = time.perf_counter() - t
        if s >= warmup:
            times.append(dt)
    edges = B * sl.total_nnz
    return edges, times


def oracle_infer_sample(spec, inputs, layers, steps, warmup):
    from oracle import OracleNet
    sl = spec.sliced(layers)
    ora = OracleNet(*gen.network(sl), activation=setup_of(spec)[0])
    x0 = gen.inputs(sl, inputs)
    times = []
    for s in range(warmup + steps):
        t = time.perf_counter()
        ora.infer(x0)
        dt = time.perf_counter() - t
        if s >= warmup:
            times.append(dt)
    return inputs * sl.total_nnz, times


def oracle_sample_shape(spec, kind, batch, budget_edges):
    """Slice of the workload (layers, inputs) holding about `budget_edges` edge-visits per oracle step."""
    if kind == "train":
        layers = int(max(1, min(spec.layers, budget_edges // (batch * spec.nnz_per_layer))))
        return layers, batch
    inputs = int(min(batch, 256))
    layers = int(max(1, min(spec.layers, budget_edges // (inputs * spec.nnz_per_layer))))
    return layers, inputs


def run_reference(args, spec, kind, batch, wname):
    """The reference arm: the oracle as it stands, on the host cores, on a bounded sample per step."""
    cores = os.cpu_count()
    layers, inputs = oracle_sample_shape(spec, kind, batch, budget_edges=1.0e9)
    if kind == "train":
        edges, times = oracle_train_sample(spec, inputs, layers, args.steps, args.warmup, args.averaged)
        sample = f"train step on layers 1..{layers} of {spec.layers} at full width N={spec.n}, B={inputs}"
    else:
        edges, times = oracle_infer_sample(spec, inputs, layers, args.steps, args.warmup)
        sample = f"inference of {inputs} inputs through layers 1..{layers} of {spec.layers} at full width N={spec.n}"
    ms = 1e3 * float(np.mean(times))
    value = edges / (ms * 1e-3)
    line = {
        "impl": "reference", "metric": metric_name(kind), "value": value, "unit": "edges/s", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "ms_per_step_is": "one step of the bounded SAMPLE named in cpu_baseline.sample, not of the full workload in config",
        "config": workload_config(wname, spec, kind, batch, args.averaged),
        "cpu_baseline": {"value": value, "unit": "edges/s", "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": "edges/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


def metric_name(kind):
    return "edges_per_sec_train_step" if kind == "train" else "edges_per_sec_inference"


def workload_config(wname, spec, kind, batch, averaged=False):
    cfg = {"workload": f"{wname}: {spec.name} {spec.n} neurons x {spec.layers} layers, {spec.k} nnz/row, "
                       + (f"minibatch {batch}, fresh minibatch per step" if kind == "train" else f"batch tile {batch}")
                       + (", averaged form of the step (one batch-averaged vector backpropagated)" if averaged and kind == "train" else ""),
           "mode": "dense (no data-dependent skipping)", "activation": setup_of(spec)[0],
           "l2": "working set per step (weights + activations) is larger than L2; no explicit flush"
           if spec.total_nnz * 8 > 256e6 else "explicit L2 flush (256 MB write) before every timed step"}
    return cfg


def study_probes():
    """Rates of the operand paths a layer kernel can take its gathered rows from, as rows per clock and SM at the maximum
    SM clock, and the scattered-word rates that a single shared value array would depend on."""
    import torch

    import paper_2104_11805_b200 as pkg
    from paper_2104_11805_b200.build import build_library
    build_library()
    torch.cuda.set_device(int(os.environ.get("LOCAL_RANK", "0")))
    props = torch.cuda.get_device_properties(torch.cuda.current_device())
    sms = props.multi_processor_count
    try:
        import pynvml
        pynvml.nvmlInit()
        mhz = pynvml.nvmlDeviceGetMaxClockInfo(pynvml.nvmlDeviceGetHandleByIndex(torch.cuda.current_device()), pynvml.NVML_CLOCK_SM)
    except Exception:
        mhz = 1965
    clk = mhz * 1e6
    out = {"study": "probes", "sms": sms, "sm_max_mhz": mhz, "unit": "rows (or words) per clock per SM at sm_max_mhz", "l2": {}, "l2_small_table": {},
           "shared": {}, "cluster": {}, "copy_engine_bulk": {}, "copy_engine_gather4": {}, "words": {}}
    for rb in (16, 32, 64, 128, 256, 512, 1024):
        rows = (4 << 20) // rb                                   # a 4 MB table: an activation tile of the large configurations
        out["l2"][str(rb)] = pkg.probe_gather_rate(rb, rows) / sms / clk
        out["l2_small_table"][str(rb)] = pkg.probe_gather_rate(rb, max(1, (64 << 10) // rb)) / sms / clk      # 64 KB: L1 hits
    for rb in (32, 64, 128, 256):
        r, ctas = pkg.probe_smem_gather_rate(rb, 1)
        out["shared"][str(rb)] = r / ctas / clk
        for cl in (2, 4, 8, 16):
            r, ctas = pkg.probe_smem_gather_rate(rb, cl)
            out["cluster"][f"{rb}x{cl}"] = {"rate": r / ctas / clk, "ctas": ctas}
    for rb in (16, 32, 64, 128, 256):      # rows fetched by the copy engine into shared memory, out of the same 4 MB table
        for key, g4 in (("copy_engine_bulk", 0), ("copy_engine_gather4", 1)):
            if g4 and rb < 32:
                continue
            try:
                out[key][str(rb)] = pkg.probe_tma_gather_rate(rb, (4 << 20) // rb, g4) / sms / clk
            except pkg.SdnnError as exc:
                out[key][str(rb)] = f"error: {exc.message}"
    out["both_paths"] = {}
    for rb, lsu, tma in ((64, 2048, 256), (256, 1024, 256)):      # do the copy engine's gathers come on top of the loads'?
        rows_tbl = (4 << 20) // rb
        rec = {}
        for key, t, l in (("loads_only", 0, lsu), ("copy_engine_only", tma, 0), ("both", tma, lsu)):
            try:
                sec, rows = pkg.probe_mixed_gather(rb, rows_tbl, t, l)
                rec[key] = {"us": sec * 1e6, "rate": rows / sec / sms / clk}
            except pkg.SdnnError as exc:
                rec[key] = f"error: {exc.message}"
        out["both_paths"][str(rb)] = rec
    for name, store in (("load4", 0), ("store4", 1)):
        out["words"][name] = pkg.probe_word_rate(store, 1 << 21) / sms / clk       # an 8 MB value array (one layer of the largest net)
    # 64-byte rows in strict batches: rate and round trip against the rows in flight per SM
    out["rows_in_flight"] = []
    for threads in (128, 256, 512, 1024):
        for loads in (1, 2, 4, 8, 16):
            try:
                rate = pkg.probe_gather_inflight(65536, threads, loads) / sms / clk
            except pkg.SdnnError:
                continue          # that many loads per lane at that many threads do not fit the registers
            inflight = threads // 2 * loads
            out["rows_in_flight"].append({"threads_per_sm": threads, "loads_per_lane": loads, "rows_in_flight_per_sm": inflight,
                                          "rate": rate, "round_trip_clk": inflight / rate})
    # a layer boundary as a grid-wide barrier inside one launch against the boundary between two dependent launches
    out["layer_boundary_us"] = {}
    for ctas, threads in ((1, 32), (1, 224), (2, 224), (2, 32)):
        try:
            bar, lau = pkg.probe_layer_boundary(ctas, threads)
            out["layer_boundary_us"][f"{ctas}x{threads}"] = {"grid_barrier": bar, "dependent_launch_in_graph": lau}
        except pkg.SdnnError as exc:
            out["layer_boundary_us"][f"{ctas}x{threads}"] = f"error: {exc.message}"
    print(json.dumps(out), flush=True)


def study_tensor():
    """Should the block structure of config 4 go to the tensor cores?

    One layer of config 4 with its neurons in block order is 64 diagonal blocks of 1024 x 1024 with 32 stored entries per
    row (3.1 % dense).  As a dense product a block costs 32 times the useful work, and fp32 operands have to be split to
    keep 1e-4: x = x_hi + x_lo and W = W_hi + W_lo in TF32 (or bf16), y = W_hi x_hi + W_hi x_lo + W_lo x_hi, three GEMMs.
    A hand-written tcgen05 kernel cannot beat the vendor's dense GEMM on the same dense blocks, so that GEMM (one batched
    call per product, through torch.matmul; a measurement aid, not a product path) bounds the tensor-core route from
    above; beside it, the library's sparse forward kernel on the same layer and tile.  Errors are normwise against float64."""
    import torch

    import paper_2104_11805_b200 as pkg
    from paper_2104_11805_b200.build import build_library
    build_library()
    torch.cuda.set_device(int(os.environ.get("LOCAL_RANK", "0")))
    spec = gen.CFG4.live().sliced(1)
    N, T, blk = spec.n, 1024, 1024
    nb = N // blk
    rp, col, val, bias = gen.layer(spec, 0)
    perm = gen.layer_permutation(spec, 0)                      # block r of rows reads the columns perm[1024 r ..]
    inv = np.empty(N, dtype=np.int64); inv[perm] = np.arange(N)
    rows = np.repeat(np.arange(N), spec.k)
    local = inv[col] - (rows // blk) * blk                     # column within the block, in block order
    assert local.min() >= 0 and local.max() < blk
    Wd = torch.zeros((nb, blk, blk), dtype=torch.float32, device="cuda")
    Wd[torch.from_numpy(rows // blk).cuda(), torch.from_numpy(rows % blk).cuda(), torch.from_numpy(local).cuda()] = torch.from_numpy(val).cuda()
    x0 = torch.from_numpy(gen.inputs(spec, T)).cuda() * torch.rand((T, N), device="cuda")       # general fp32 inputs, [T][N]
    Xb = x0.t()[torch.from_numpy(perm.astype(np.int64)).cuda()].reshape(nb, blk, T).contiguous()  # block order
    ref = torch.bmm(Wd.double(), Xb.double())

    def tf32_split(a):
        hi = (a.view(torch.int32) & -8192).view(torch.float32)
        return hi, a - hi

    def bf16_split(a):
        hi = a.to(torch.bfloat16)
        return hi, (a - hi.float()).to(torch.bfloat16)

    def timed(fn, reps=5):
        for _ in range(2):
            out = fn()
        torch.cuda.synchronize()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        for _ in range(reps):
            out = fn()
        b.record()
        torch.cuda.synchronize()
        return a.elapsed_time(b) / reps, out

    edges = N * spec.k * T
    res = {"study": "tensor", "layer": f"config 4, one layer, {nb} blocks of {blk} x {blk}, {spec.k} stored entries per row; tile of {T} inputs",
           "edges_per_layer_tile": edges}
    torch.backends.cuda.matmul.allow_tf32 = True
    wh, wl = tf32_split(Wd); xh, xl = tf32_split(Xb)
    ms1, y1 = timed(lambda: torch.bmm(wh, xh))
    ms3, y3 = timed(lambda: torch.bmm(wh, xh) + torch.bmm(wh, xl) + torch.bmm(wl, xh))
    err = lambda y: float((y.double() - ref).abs().max() / ref.abs().max())
    res["tf32"] = {"one_gemm_ms": ms1, "one_gemm_err": err(y1), "three_gemms_ms": ms3, "three_gemms_err": err(y3),
                   "edges_per_s_three_gemms": edges / (ms3 * 1e-3), "dense_tflops_one_gemm": 2.0 * nb * blk * blk * T / (ms1 * 1e-3) / 1e12}
    bh, bl = bf16_split(Wd); ch, cl = bf16_split(Xb)
    # what the bf16 split itself loses (the dropped lo x lo term and the rounding of the lo parts), with exact products and sums:
    # the error floor of ANY kernel that feeds these operands to the tensor cores and accumulates in fp32
    sub = slice(0, 4)
    exact = (torch.bmm(bh[sub].double(), ch[sub].double()) + torch.bmm(bh[sub].double(), cl[sub].double())
             + torch.bmm(bl[sub].double(), ch[sub].double()))
    bf16_split_err = float((exact - ref[sub]).abs().max() / ref[sub].abs().max())
    del exact
    f = lambda a, b: torch.bmm(a, b).float()
    ms1, y1 = timed(lambda: torch.bmm(bh, ch))
    ms3, y3 = timed(lambda: f(bh, ch) + f(bh, cl) + f(bl, ch))
    res["bf16"] = {"one_gemm_ms": ms1, "one_gemm_err": err(y1.float()), "three_gemms_ms": ms3, "three_gemms_err": err(y3),
                   "edges_per_s_three_gemms": edges / (ms3 * 1e-3), "dense_tflops_one_gemm": 2.0 * nb * blk * blk * T / (ms1 * 1e-3) / 1e12,
                   "split_error_with_exact_arithmetic": bf16_split_err,
                   "note": "the library call rounds each GEMM's output to bf16 before the three are added, hence three_gemms_err; a "
                           "kernel of one's own would accumulate in fp32 and reach split_error_with_exact_arithmetic per layer, at "
                           "best in 3 x one_gemm_ms"}
    del Wd, wh, wl, xh, xl, bh, bl, ch, cl, ref, Xb
    # the library's sparse kernel on the same layer (given neuron order, tile of 1024 inputs, 16 layers of the same recipe)
    L = 16
    sp = gen.CFG4.live().sliced(L)
    h = pkg.Sdnn.create_deferred(L, N, [sp.nnz_per_layer] * L, max_batch=T, flags=pkg.FLAG_ONE_TILE)
    for l in range(L):
        h.load_layer(l, *gen.layer(sp, l))
    h.finalize()
    xin = torch.from_numpy(gen.inputs(sp, T)).cuda()
    y = torch.empty((T, N), dtype=torch.float32, device="cuda")
    ms, _ = timed(lambda: h.infer_batch(xin, T, y, None, None, 0))
    res["sparse_kernel"] = {"ms_per_layer_tile": ms / L, "edges_per_s": edges / (ms / L * 1e-3), "note": f"forward_kernel<32,8,2>, {L} layers, one tile in flight, transposes included"}
    h.destroy()
    print(json.dumps(res), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--workload", default="cfg5", choices=sorted(WORKLOADS))
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--layers", type=int, default=None, help="use only the first LAYERS layers (profiling captures)")
    ap.add_argument("--inputs", type=int, default=None, help="inference: number of inputs per call")
    ap.add_argument("--tile", type=int, default=None, help="inference: batch tile (max_batch of the handle)")
    ap.add_argument("--net", default=None, metavar="N,L",
                    help="same recipe at another size, e.g. 65536,1920 for the deeper grids of the paper's Table 2")
    ap.add_argument("--pattern", default=None, choices=["uniform", "windowed"],
                    help="same recipe with the other pattern family: columns uniform over [0, N), or over the 1024 columns "
                         "that a block of 1024 rows shares (the locality a good neuron order gives)")
    ap.add_argument("--shuffle", action="store_true",
                    help="renumber the neurons of every inner layer at random (NetSpec.shuffled): the same function with whatever "
                         "structure the pattern has hidden, to be recovered with --flags 0x100 (SDNN_FLAG_REORDER)")
    ap.add_argument("--averaged", action="store_true",
                    help="train workloads: the averaged form of the minibatch step (one batch-averaged gradient vector is "
                         "backpropagated; sdnn_train_step_averaged) instead of the exact minibatch step")
    ap.add_argument("--flags", type=lambda s: int(s, 0), default=None,
                    help="SDNN_FLAG_* bits of the handle; default: 0, except 0x300 (set-up reordering + operand windows in shared "
                         "memory, both part of the untimed set-up) for the config-4 workloads, whose layers have block structure")
    ap.add_argument("--batch", type=int, default=None, help="train workloads: another minibatch size on the same net")
    ap.add_argument("--study", default=None, choices=["probes", "tensor"],
                    help="instead of a workload: 'probes' = the operand-path probes (random row gathers out of L2, out of shared "
                         "memory, out of a cluster's distributed shared memory; scattered 4-byte words); 'tensor' = what tensor cores "
                         "could do for config 4's block structure, bounded from above by the vendor's dense GEMM on the same "
                         "blocks, beside the library's sparse kernel on the same layer; one JSON line each")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-compaction", action="store_true", help="inference: skip the extra pass with dead inputs dropped")
    args = ap.parse_args()
    if args.warmup < 3 and args.layers is None:
        args.warmup = 3
    if args.study == "probes":
        return study_probes()
    if args.study == "tensor":
        return study_tensor()
    spec, kind, batch, n_inputs = WORKLOADS[args.workload]
    if args.flags is None:
        args.flags = 0x300 if args.workload.startswith("cfg4") else 0
    if args.tile and kind == "infer":
        batch = args.tile
    if args.batch and kind == "train":
        batch = n_inputs = args.batch
    if args.net:
        n_, l_ = (int(v) for v in args.net.split(","))
        spec = spec.scaled(n_, l_)
    if args.pattern and args.pattern != spec.pattern:
        import dataclasses
        spec = dataclasses.replace(spec, name=f"{spec.name}-{args.pattern}", pattern=args.pattern, window=min(1024, spec.n))
    if args.shuffle and not spec.shuffle:
        spec = spec.shuffled()
    if args.layers:
        spec = spec.sliced(args.layers)
    if args.inputs and kind == "infer":
        n_inputs = args.inputs
    if args.steps is None:
        args.steps = 10 if kind == "train" else 3

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if world > 1:
        # the launcher gives every rank one OpenMP thread; the (untimed) set-up of a replica - generating the layers,
        # building the sliced and transposed copies - is OpenMP code and would take minutes that way: share the cores
        threads = max(1, (os.cpu_count() or 1) // world)
        os.environ["OMP_NUM_THREADS"] = str(threads)
        try:        # the OpenMP runtime may have read the variable already (numpy is imported)
            import ctypes
            ctypes.CDLL("libgomp.so.1").omp_set_num_threads(threads)
        except OSError:
            pass
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))

    if args.impl == "reference":
        if rank == 0:
            run_reference(args, spec, kind, batch, args.workload)
        return

    import torch
    import torch.distributed as dist

    import paper_2104_11805_b200 as pkg
    from paper_2104_11805_b200 import shard
    from paper_2104_11805_b200.build import build_library

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU path)")
    torch.cuda.set_device(local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    if local_rank == 0:        # one rank compiles (if the library is stale), the others wait for it
        build_library()
    if world > 1:
        dist.barrier()
    stream = torch.cuda.Stream()
    hbm_peak, peak_src = measured_peaks()

    # ------------------------------------------------------------------ build the net, layer by layer
    t_setup = time.perf_counter()
    L, N = spec.layers, spec.n
    flags = args.flags
    act_name, act_code, eta = setup_of(spec)
    h = pkg.Sdnn.create_deferred(L, N, [spec.nnz_per_layer] * L, max_batch=batch, train=(kind == "train"),
                                 flags=flags, stream=stream.cuda_stream, device=local_rank, activation=act_code)
    for l in range(L):
        h.load_layer(l, *gen.layer(spec, l))
    h.finalize()
    setup_s = time.perf_counter() - t_setup

    total = args.warmup + args.steps
    edges_per_step = n_inputs * spec.total_nnz
    flush = None if spec.total_nnz * 8 > 256e6 else torch.empty(64 << 20, dtype=torch.float32, device="cuda")

    def l2_flush():
        if flush is not None:
            flush.fill_(1.0)

    with torch.cuda.stream(stream):
        if kind == "train":
            # every rank trains its own replica on its own stream of minibatches (replicas only: no collective)
            xs = [torch.from_numpy(gen.inputs(spec, batch, step=rank * 1000 + s)).cuda() for s in range(total)]
            ys = [torch.from_numpy(gen.targets(spec, batch, step=rank * 1000 + s)).cuda() for s in range(total)]
            hx = [x.cpu().pin_memory() for x in xs]
            hy = [y.cpu().pin_memory() for y in ys]

            def step(i):
                h.train_step(xs[i], ys[i], batch, eta, averaged=args.averaged)

            if args.averaged:       # device pointers only: the copies from the pinned buffers are made here, on the same stream
                dx, dy = torch.empty_like(xs[0]), torch.empty_like(ys[0])

                def step_e2e(i):
                    dx.copy_(hx[i], non_blocking=True); dy.copy_(hy[i], non_blocking=True)
                    return h.train_step(dx, dy, batch, eta, want_loss=True, averaged=True)
            else:
                def step_e2e(i):
                    return h.train_step(hx[i], hy[i], batch, eta, want_loss=True, host=True)

            h2d, d2h = 2 * batch * N * 4, 4
        else:
            # the batch is sharded over ranks: each rank infers its own n_inputs inputs (weak scaling, no collective)
            chunk = 4096
            x_all = torch.empty((n_inputs, N), dtype=torch.float32, device="cuda")
            first, _ = shard.rank_inputs(rank, world, n_inputs)
            for s0 in range(0, n_inputs, chunk):
                c = min(chunk, n_inputs - s0)
                x_all[s0:s0 + c] = torch.from_numpy(gen.inputs(spec, c, start=first + s0)).cuda()
            counts = torch.empty(n_inputs, dtype=torch.int32, device="cuda")
            cap = 1 << 20
            idx = torch.empty(cap, dtype=torch.int32, device="cuda")
            n_e2e = n_inputs            # the whole batch goes through host buffers too (pinned: 4 N bytes per input)
            hx_all = torch.empty((n_e2e, N), dtype=torch.float32, pin_memory=True)
            for s0 in range(0, n_e2e, chunk):
                hx_all[s0:s0 + chunk].copy_(x_all[s0:s0 + chunk])
            hcounts = torch.empty(n_e2e, dtype=torch.int32).pin_memory()

            def step(i):
                h.infer_batch(x_all, n_inputs, None, counts, None, 0)

            def step_e2e(i):
                return h.infer_batch(hx_all, n_e2e, None, hcounts, None, 0, want_total=True, host=True)

            h2d, d2h = n_e2e * N * 4, n_e2e * 4 + 8

        def barrier():
            torch.cuda.synchronize()
            if world > 1:
                dist.barrier()
            torch.cuda.synchronize()

        # ---------------------------------------------------------------- device-resident timing
        for i in range(args.warmup):
            l2_flush()
            step(i)
        barrier()
        launches0 = h.kernel_launches()
        fwd_ms = bwd_ms = 0.0
        e0 = torch.cuda.Event(enable_timing=True)
        e1 = torch.cuda.Event(enable_timing=True)
        step_ms = []
        with ClockSampler(local_rank) as clocks:
            if flush is None and kind == "train":
                marks = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps + 1)]
                marks[0].record(stream)
                for i in range(args.steps):
                    step(args.warmup + i)
                    marks[i + 1].record(stream)      # no synchronisation between steps
                barrier()
                total_ms = marks[0].elapsed_time(marks[-1])
                step_ms = [marks[i].elapsed_time(marks[i + 1]) for i in range(args.steps)]
            else:
                total_ms = 0.0
                for i in range(args.steps):
                    l2_flush()
                    a = torch.cuda.Event(enable_timing=True)
                    b = torch.cuda.Event(enable_timing=True)
                    a.record(stream)
                    step(args.warmup + i)
                    b.record(stream)
                    torch.cuda.synchronize()
                    step_ms.append(a.elapsed_time(b))
                    total_ms += step_ms[-1]
                barrier()
        launches = h.kernel_launches() - launches0
        if kind == "train":
            fwd_ms, bwd_ms = h.get_phase_times()      # last timed step
        value, ms_per_step = shard.job_throughput(edges_per_step, total_ms / args.steps, world, device="cuda")

        # ---------------------------------------------------------------- end-to-end through host buffers
        e2e = None
        if not args.no_e2e:
            k_e2e = args.steps
            step_e2e(0)
            barrier()
            a = torch.cuda.Event(enable_timing=True)
            b = torch.cuda.Event(enable_timing=True)
            t0 = time.perf_counter()
            a.record(stream)
            for i in range(k_e2e):
                step_e2e(args.warmup + i if kind == "train" else i)
            b.record(stream)
            barrier()
            wall_ms = 1e3 * (time.perf_counter() - t0)
            dev_ms = a.elapsed_time(b)
            e2e_edges = edges_per_step if kind == "train" else n_e2e * spec.total_nnz
            e2e_value, per = shard.job_throughput(e2e_edges, max(wall_ms, dev_ms) / k_e2e, world, device="cuda")
            e2e = {"value": e2e_value, "unit": "edges/s", "h2d_bytes_per_step": h2d,
                   "d2h_bytes_per_step": d2h, "ms_per_step": per,
                   "api": ("pinned-to-device copies + sdnn_train_step_averaged" if args.averaged else "sdnn_train_step_host") if kind == "train" else f"sdnn_infer_batch_host on {n_e2e} inputs"}

    # -------------------------------------------------------------------- inference: the same call with dead inputs dropped
    compaction = None
    if kind == "infer" and not args.no_compaction:
        with torch.cuda.stream(stream):
            # dropping dead inputs runs on the default layout (it does not combine with the set-up reordering)
            hc = pkg.Sdnn.create_deferred(L, N, [spec.nnz_per_layer] * L, max_batch=batch,
                                          flags=(flags & ~(pkg.FLAG_REORDER | pkg.FLAG_SMEM_WINDOWS)) | pkg.FLAG_SKIP_DEAD,
                                          stream=stream.cuda_stream, device=local_rank)
            for l in range(L):
                hc.load_layer(l, *gen.layer(spec, l))
            hc.finalize()
            hc.infer_batch(x_all, n_inputs, None, counts, None, 0)
            torch.cuda.synchronize()
            a = torch.cuda.Event(enable_timing=True)
            b = torch.cuda.Event(enable_timing=True)
            a.record(stream)
            for _ in range(2):
                hc.infer_batch(x_all, n_inputs, None, counts, None, 0)
            b.record(stream)
            torch.cuda.synchronize()
            cv, cms = shard.job_throughput(edges_per_step, a.elapsed_time(b) / 2, world, device="cuda")
            live = [int(v) for v in hc.get_liveness()]
            last_tile = n_inputs - (n_inputs - 1) // batch * batch
            compaction = {"value": cv, "unit": "edges/s (nominal: every stored entry of every input counted, as in dense mode)",
                          "ms_per_step": cms, "live_inputs_after_layer_last_tile": live[:8] + (["..."] if L > 8 else []) + live[-1:],
                          "last_tile_inputs": last_tile}
            hc.destroy()

    # -------------------------------------------------------------------- roofline of the dominant kernel
    nnz_l = spec.nnz_per_layer
    if kind == "train":
        ld = max(4, 1 << (batch - 1).bit_length())
        ld_bwd = 4 if args.averaged else ld       # the averaged form backpropagates one vector
        # backward+update launch: index read + value read + value write per stored entry, x^{k-1} tile read once
        bwd_bytes = 12 * nnz_l + N * ld_bwd * 4
        fwd_bytes = 8 * nnz_l + N * ld * 4
        dom = "backward_kernel" if bwd_ms >= fwd_ms else "forward_kernel"
        per_launch_ms = (bwd_ms if dom == "backward_kernel" else fwd_ms) / L
        alg = bwd_bytes if dom == "backward_kernel" else fwd_bytes
        # tiles of padded width 4 (B <= 4, or the averaged form's backward chain) run the entry-parallel kernels
        ep = not (args.flags & 0x81)
        names = ("backward_col_ep_kernel<4 or 8>", "backward_row_ep_kernel") if ep and ld_bwd == 4 else \
                ("backward_kernel<..,1,..>", "backward_kernel<..,0,..>")
        extra = {"backward_launches": f"per layer one column-unit launch ({names[0]}) on the main stream and one "
                                      f"row-unit launch ({names[1]}) on a side stream, running beside each other; "
                                      "launch_ms is the backward chain's time per layer, bytes and gathers are those of both",
                 "kernel_names": {"forward": "forward_ep_kernel" if ep and ld == 4 else "forward_kernel", "backward": list(names)},
                 "fwd_ms_per_step": fwd_ms, "bwd_ms_per_step": bwd_ms,
                 "fwd_GBps": fwd_bytes * L / (fwd_ms * 1e-3) / 1e9 if fwd_ms else None,
                 "bwd_GBps": bwd_bytes * L / (bwd_ms * 1e-3) / 1e9 if bwd_ms else None,
                 "step_bytes": (fwd_bytes + bwd_bytes) * L,
                 "step_GBps": (fwd_bytes + bwd_bytes) * L / (ms_per_step * 1e-3) / 1e9}
    else:
        batch = h.infer_tile_width()           # the library narrows the tile when two of them would not fit in L2
        tiles = (n_inputs + batch - 1) // batch
        dom = "forward_window32_kernel" if h.windowed_layers() == L else "forward_kernel"
        extra_reorder = {"grouped_layers": h.grouped_layers(), "windowed_layers": h.windowed_layers()}
        per_launch_ms = ms_per_step / (tiles * L)      # includes the (small) transpose and count kernels of each tile
        # per launch: the layer's indices and values once, the activation tile read and written once
        alg = 8 * nnz_l + 2 * N * min(batch, n_inputs) * 4
        in_flight = h.infer_tiles_in_flight() if tiles > 1 else 1
        extra = {"tiles": tiles, "tile_inputs": batch, "tiles_in_flight": in_flight, **extra_reorder,
                 "note": "launch time = call time / forward launches (upper bound)" +
                         ("; two tiles run beside each other on two streams, so this is the time the device spends per "
                          "launch, not one launch's start-to-end duration" if in_flight > 1 else "")}
    # what bounds these launches instead of HBM: random gathers of tile rows out of L2 (measured now, on this device)
    if kind == "train":
        row_bytes, gathers = 4 * (ld_bwd if dom == "backward_kernel" else ld), (2 if dom == "backward_kernel" else 1) * nnz_l
        table_rows = 1 << (N - 1).bit_length()
    else:
        row_bytes = min(1024, 4 * (1 << (min(batch, n_inputs) - 1).bit_length()))      # one chunk of a tile row
        gathers = nnz_l * ((min(batch, n_inputs) * 4 + row_bytes - 1) // row_bytes)
        table_rows = 1 << max(0, (N * min(batch, n_inputs) * 4 // row_bytes - 1).bit_length())
    table_rows = min(table_rows, (1 << 30) // row_bytes)
    try:
        gather_rate = pkg.probe_gather_rate(row_bytes, table_rows)
        floor_ms = gathers / gather_rate * 1e3
        extra["gather_bound"] = {"probe_rows_per_s": gather_rate, "row_bytes": row_bytes, "table_rows": table_rows,
                                 "note": "uniformly random rows: a layer whose pattern is local can beat this floor",
                                 "gathers_per_launch": gathers, "floor_ms_per_launch": floor_ms,
                                 "frac_of_gather_floor": floor_ms / per_launch_ms if per_launch_ms else None}
        if kind == "train":      # both chains of the step against the floor of their own gathers
            fwd_rate = gather_rate if ld == ld_bwd else pkg.probe_gather_rate(4 * ld, table_rows)
            bwd_rate = gather_rate if dom == "backward_kernel" else pkg.probe_gather_rate(4 * ld_bwd, table_rows)
            f_floor, b_floor = nnz_l * L / fwd_rate * 1e3, 2 * nnz_l * L / bwd_rate * 1e3
            extra["gather_bound"].update({"forward_chain_floor_ms": f_floor, "forward_chain_frac_of_floor": f_floor / fwd_ms if fwd_ms else None,
                                          "backward_chain_floor_ms": b_floor, "backward_chain_frac_of_floor": b_floor / bwd_ms if bwd_ms else None,
                                          "step_floor_ms": f_floor + b_floor,
                                          "step_frac_of_floor": (f_floor + b_floor) / ms_per_step if ms_per_step else None})
    except Exception as exc:      # the probe is a diagnostic; the line stands without it
        extra["gather_bound"] = {"error": str(exc)}
    achieved = alg / (per_launch_ms * 1e-3) / 1e9 if per_launch_ms else None
    traffic = NCU_TRAFFIC.get((args.workload.replace("-live", ""), dom)) if (not args.layers or kind == "train") and not args.pattern and not args.net and not args.batch else None
    frac = achieved / hbm_peak if achieved else None
    target = {"hbm_frac_target": 0.5, "target_met": bool(frac is not None and frac >= 0.5),
              "note": "the target asks for half of the HBM roofline; these launches are bound by random row gathers out of L2 "
                      "(gather_bound), which caps them well below it"}
    # the library keeps 16-bit indices for nets of at most 65536 neurons: the same launch against its own, smaller byte count
    idx16 = N <= 65536 and not (flags & pkg.FLAG_IDX32)
    alg16 = alg - 2 * nnz_l if idx16 else alg
    own = {"index_bytes": 2 if idx16 else 4, "algorithmic_bytes_per_launch": alg16,
           "achieved": alg16 / (per_launch_ms * 1e-3) / 1e9 if per_launch_ms else None,
           "frac": alg16 / (per_launch_ms * 1e-3) / 1e9 / hbm_peak if per_launch_ms else None}
    roofline = {"bound": "hbm", "kernel": dom, "achieved": achieved, "peak": hbm_peak, "unit": "GB/s",
                "frac": frac, "with_stored_index_width": own, "target": target, "traffic": traffic, "peak_source": peak_src,
                "algorithmic_bytes_per_launch": alg, "launch_ms": per_launch_ms, **extra}

    # -------------------------------------------------------------------- CPU oracle on a bounded sample (rank 0, N = 1)
    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        layers_s, inputs_s = oracle_sample_shape(spec, kind, batch, budget_edges=1.5e9)
        if kind == "train":
            edges, times = oracle_train_sample(spec, inputs_s, layers_s, 2, 1, args.averaged)
            sample = f"2 train steps on layers 1..{layers_s} of {L} at full width N={N}, B={inputs_s}"
        else:
            edges, times = oracle_infer_sample(spec, inputs_s, layers_s, 2, 1)
            sample = f"2 inference passes of {inputs_s} inputs through layers 1..{layers_s} of {L} at full width N={N}"
        cpu = {"value": edges / float(np.mean(times)), "unit": "edges/s", "cores": os.cpu_count(), "kind": "oracle",
               "sample": sample, "seconds_per_sample_step": float(np.mean(times))}

    if rank == 0:
        line = {
            "metric": metric_name(kind), "value": value, "unit": "edges/s", "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms_per_step,
            "ms_per_step_median": float(np.median(step_ms)) if step_ms else None, "ms_per_step_min": float(np.min(step_ms)) if step_ms else None,
            "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": {**workload_config(args.workload, spec, kind, batch, args.averaged),
                       "parallelism": "replicas only (no collective)" if kind == "train" else "batch sharded over ranks, no collective",
                       "inputs_per_step_per_gpu": n_inputs, "setup_seconds": setup_s, "device_bytes": h.device_bytes(),
                       "handle_flags": hex(flags)},
            "clocks": clocks.summary(), "e2e": e2e, "gpu_launches": launches, "roofline": roofline, "cpu_baseline": cpu,
            "compaction_mode": compaction,
        }
        print(json.dumps(line), flush=True)
    h.destroy()
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()

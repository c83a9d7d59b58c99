#!/usr/bin/env python
"""Benchmark of the XNOR-Net forward block on B200.

One step = one pass of the whole hot path over one batch.  Default workload:
the four AlexNet-shaped binary convolution layers at batch 256 per GPU
(synthetic seeded inputs); per layer: weight binarisation, BN affine + BinActiv
(sign-pack, A, K) and BinConv.  `--workload` selects the other shape sets
(resnet18, sweep, single, chain = the 16-layer ResNet-18 chain with residual
adds); the bench line proper is the default.  Prints ONE JSON line (rank 0).
`--impl reference` times the CPU oracle instead.
"""
import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402

from paper_1603_05279_b200 import dist_util as du  # noqa: E402
from paper_1603_05279_b200 import workloads as wl  # noqa: E402

METRIC = "binary conv TOPS (1-bit MACs/s)"
UNIT = "T 1-bit MAC/s"
WORKLOAD_NAMES = {"alexnet": "alexnet_conv2-5_batch256", "resnet18": "resnet18_3x3_layers_batch256",
                  "sweep": "efficiency_sweep_batch64", "single": "single_layer_batch1",
                  "chain": "xnor_resnet18_chain_16_layers_batch256"}
HBM_FALLBACK_GBS = 6650.0
BF16_FALLBACK_TFLOPS = 1590.0
# popc engine: population count issues 16 results per clock per SM (CUDA C programming
# guide, arithmetic-instruction throughput table, compute capability 10.0); one result
# covers 32 one-bit MACs.
POPC_PER_CLK_PER_SM = 16
# DRAM traffic of the dominant kernel from one ncu capture: dram__bytes_read.sum +
# dram__bytes_write.sum summed over the four BinConv launches of one step of the default
# workload.  Valid only for the kernel source it was taken from (hash below); null otherwise.
NCU_TRAFFIC = {"kernel_sha1": "3358099109c5b791f6208dde51e57cca8c485e53", "bytes_per_step": 148.6e6}


def kernel_sha1():
    import hashlib
    h = hashlib.sha1()
    for f in ("binconv_tc.cu", "umma_common.cuh", "common.cuh"):
        h.update(open(os.path.join(ROOT, "paper_1603_05279_b200", "csrc", f), "rb").read())
    return h.hexdigest()


def measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        try:
            j = json.load(open(p))
            return dict(hbm_gbs=float(j["hbm_gbs"]), bf16=float(j["bf16_tflops"]),
                        bf16_sustained=float(j.get("bf16_tflops_sustained", j["bf16_tflops"])),
                        source="measured")
        except Exception:
            pass
    return dict(hbm_gbs=HBM_FALLBACK_GBS, bf16=BF16_FALLBACK_TFLOPS, bf16_sustained=1400.0,
                source="fallback")


def host_cores():
    try:
        return len(os.sched_getaffinity(0))
    except Exception:
        return os.cpu_count() or 1


def workload_shapes(name, batch):
    if name == "chain":
        return wl.chain_shapes(batch)
    return [wl.scaled(s, batch) if batch else s for s in wl.CONFIGS[name]]


def default_batch(name):
    return {"alexnet": 256, "resnet18": 256, "sweep": 64, "single": 1, "chain": 256}[name]


# ------------------------------------------------------------------ CPU oracle timing
def oracle_pass(name, layer_ids, n_images, rank=0):
    """Times the oracle, as it stands, on the first n_images of the workload's batch.
    Returns (seconds, macs)."""
    import oracle
    total_t, total_macs = 0.0, 0
    if name == "chain":
        shapes = wl.chain_shapes(n_images)
        seed0 = du.rank_seed(wl.layer_seed("chain", 0), rank)
        x = wl.normal((n_images, shapes[0].C_in, shapes[0].H, shapes[0].W), seed0)
        block_in = x
        for i, s in enumerate(shapes):
            w = wl.make_weights(s, seed0 + i)
            t0 = time.perf_counter()
            mean = x.mean(axis=(0, 2, 3), dtype=np.float64)
            var = x.var(axis=(0, 2, 3), dtype=np.float64)
            scale = (1.0 / np.sqrt(var + 1e-5))
            shift = (-mean * scale).astype(np.float32)
            scale = scale.astype(np.float32)
            res = None
            if i % 2 == 1:
                s0 = shapes[i - 1]
                if s0.stride != 1 or s0.C_in != s0.C_out:
                    pw = wl.normal((s0.C_out, s0.C_in, 1, 1), seed0 + 700 + i - 1, 0.05)
                    res = oracle.shortcut_conv1x1(block_in, pw, s0.stride)
                else:
                    res = block_in
            r = oracle.xnor_block(x, w, s.stride, s.pad, scale, shift, res)
            total_t += time.perf_counter() - t0
            total_macs += wl.macs(s)
            x = r.out
            if i % 2 == 1:
                block_in = x
        return total_t, total_macs
    shapes = wl.CONFIGS[name]
    for li in layer_ids:
        s = shapes[li]
        seed = du.rank_seed(wl.layer_seed(name, li), rank)
        x = wl.make_input(s, seed, n_images=n_images)
        w = wl.make_weights(s, seed)
        scale = np.ones((s.C_in,), np.float32)
        shift = np.zeros((s.C_in,), np.float32)
        t0 = time.perf_counter()
        oracle.xnor_block(x, w, s.stride, s.pad, scale, shift)
        total_t += time.perf_counter() - t0
        total_macs += wl.macs(wl.scaled(s, n_images))
    return total_t, total_macs


def cpu_baseline(name, layer_ids, batch, budget_s=12.0):
    import oracle
    oracle.build()
    cores = host_cores()
    oracle.set_num_threads(cores)
    n = min(2, batch)
    t, m = oracle_pass(name, layer_ids, n)
    want = int(min(batch, max(n, n * budget_s / max(t, 1e-3))))
    if want > n:
        n = want
        t, m = oracle_pass(name, layer_ids, n)
    return dict(value=m / t / 1e12, unit=UNIT, cores=oracle.num_threads(), kind="oracle",
                sample="first %d of %d images of each layer, whole block (BN, BinActiv, weight "
                       "binarisation, BinConv); %.1f s" % (n, batch, t),
                images_per_s=n / t)


def run_reference(args):
    """The reference arm: the CPU oracle on a bounded sample per step."""
    world, rank, _ = du.env_world()
    if rank != 0:
        return
    import oracle
    oracle.build()
    cores = host_cores()
    oracle.set_num_threads(cores)
    n = min(args.ref_images, args.batch)
    for _ in range(min(args.warmup, 1)):
        oracle_pass(args.workload, args.layer_ids, n)
    t_total, m_total = 0.0, 0
    for _ in range(args.steps):
        t, m = oracle_pass(args.workload, args.layer_ids, n)
        t_total += t
        m_total += m
    value = m_total / t_total / 1e12
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT,
        "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": 1e3 * t_total / args.steps, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "int8 (+-1 products, int32 sums)", "data": "synthetic",
        "config": {"workload": WORKLOAD_NAMES[args.workload], "sample_images_per_step": n},
        "images_per_s": n * args.steps / t_total,
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": oracle.num_threads(),
                         "kind": "oracle",
                         "sample": "each step = first %d of %d images of each layer"
                                   % (n, args.batch)},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


# ------------------------------------------------------------------ clocks
class ClockSampler:
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
              "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_id):
        self.samples = []
        self.proc = None
        self.gpu_id = gpu_id

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.gpu_id), "--query-gpu=" + self.FIELDS,
                 "--format=csv,noheader,nounits", "-lms", "50"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except Exception:
            self.proc = None
            return
        self.thread = threading.Thread(target=self._read, daemon=True)
        self.thread.start()

    def _read(self):
        for line in self.proc.stdout:
            self.samples.append((time.time(), line.strip()))

    def stop(self):
        if self.proc is not None:
            self.proc.terminate()
            try:
                self.proc.wait(timeout=5)
            except Exception:
                self.proc.kill()

    def summary(self, t0, t1):
        rows = []
        for ts, line in self.samples:
            parts = [p.strip() for p in line.split(",")]
            if len(parts) < 8:
                continue
            try:
                rows.append((ts, float(parts[0]), float(parts[1]), parts[4:8]))
            except ValueError:
                continue
        inside = [r for r in rows if t0 <= r[0] <= t1 + 0.15] or rows
        if not inside:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        reasons = sorted({names[i] for r in inside for i in range(4) if r[3][i].lower() == "active"})
        return {"sm_mhz": statistics.median(r[1] for r in inside), "sm_max_mhz": inside[0][2],
                "reasons": reasons, "samples": len(inside)}


# ------------------------------------------------------------------ workloads on the GPU
class LayersJob:
    """Independent layers: per layer binarize_weights -> binactiv -> conv."""

    def __init__(self, name, layer_ids, batch, rank, variant="xnor", kbits=2):
        import torch
        from paper_1603_05279_b200.runner import LayerBuffers
        self.torch = torch
        shapes = [wl.scaled(wl.CONFIGS[name][i], batch) for i in layer_ids]
        self.shapes = shapes
        self.layers = [LayerBuffers(s, variant=variant, kbits=kbits) for s in shapes]
        self.host_x, self.host_w, self.host_out = [], [], []
        for li, L in zip(layer_ids, self.layers):
            seed = du.rank_seed(wl.layer_seed(name, li), rank)
            self.host_x.append(torch.from_numpy(wl.make_input(L.shape, seed) if variant != "bgrad" else
                                                wl.normal(tuple(L.x.shape), seed)).pin_memory())
            self.host_w.append(torch.from_numpy(wl.make_weights(L.shape, seed)).pin_memory())
            self.host_out.append(torch.empty(L.out.shape, dtype=torch.float32).pin_memory())
            L.x.copy_(self.host_x[-1])
            L.w.copy_(self.host_w[-1])
        self.launches = sum(L.launches() for L in self.layers)
        self.macs = sum(wl.macs(s) for s in shapes)
        self.conv_macs = [wl.macs(s) for s in shapes]
        self.images = batch
        self.h2d = sum(t.numel() * 4 for t in self.host_x + self.host_w)
        self.d2h = sum(t.numel() * 4 for t in self.host_out)
        self.act_bytes = sum(L.binactiv_bytes() for L in self.layers)
        self.part_names = ("binarize_weights", "binactiv", "conv")

    def step(self, stream):
        for L in self.layers:
            L.forward(stream)

    def step_branches(self, stream):
        """The same step for graph capture: the layers do not depend on one another, so each
        is its own branch of the graph (its launches keep their order) and the GPU may fill
        the tail of one layer's kernel with another layer's blocks."""
        torch = self.torch
        if not hasattr(self, "_side"):
            self._side = [torch.cuda.Stream() for _ in self.layers[1:]]
        fork = torch.cuda.Event()
        fork.record(stream)
        for L, s in zip(self.layers[1:], self._side):
            s.wait_event(fork)
            with torch.cuda.stream(s):
                L.forward(s)
        self.layers[0].forward(stream)
        for s in self._side:
            join = torch.cuda.Event()
            join.record(s)
            stream.wait_event(join)

    def e2e_step(self, stream):
        """Host buffers in, host buffers out: the inputs of every layer go up on a copy stream,
        a layer's kernels start when its inputs have landed, its output goes down on a third
        stream while the next layer computes (the two directions of the link run together).
        The step ends when the last output is on the host."""
        torch = self.torch
        if not hasattr(self, "_h2d"):
            self._h2d, self._d2h = torch.cuda.Stream(), torch.cuda.Stream()
            self._ev_in = [torch.cuda.Event() for _ in self.layers]
            self._ev_out = [torch.cuda.Event() for _ in self.layers]
        self._h2d.wait_stream(stream)          # the previous step is done with the device buffers
        with torch.cuda.stream(self._h2d):
            for li, L in enumerate(self.layers):
                L.x.copy_(self.host_x[li], non_blocking=True)
                L.w.copy_(self.host_w[li], non_blocking=True)
                self._ev_in[li].record(self._h2d)
        for li, L in enumerate(self.layers):
            stream.wait_event(self._ev_in[li])
            L.forward(stream)
            self._ev_out[li].record(stream)
            self._d2h.wait_event(self._ev_out[li])
            with torch.cuda.stream(self._d2h):
                self.host_out[li].copy_(L.out, non_blocking=True)
        stream.wait_stream(self._d2h)

    def parts(self, stream):
        for li, L in enumerate(self.layers):
            yield "binarize_weights", li, lambda L=L: L.binarize_weights(stream)
            yield "binactiv", li, lambda L=L: L.binactiv(stream)
            yield "conv", li, lambda L=L: L.conv(stream)


class ChainJob:
    """The 16-layer chain: weight binarisation, then 8 residual blocks."""

    def __init__(self, batch, rank, fused=False):
        import torch
        from paper_1603_05279_b200 import binding as B
        from paper_1603_05279_b200.runner import ChainRunner
        self.torch, self.B = torch, B
        self.fused = fused
        ch = ChainRunner(batch)
        if fused:
            ch.prepare_fused()
        self.ch = ch
        self.shapes = ch.shapes
        seed0 = du.rank_seed(wl.layer_seed("chain", 0), rank)
        self.host_x = torch.from_numpy(wl.normal(tuple(ch.x0.shape), seed0)).pin_memory()
        self.host_w = [torch.from_numpy(wl.make_weights(L["shape"], seed0 + i)).pin_memory()
                       for i, L in enumerate(ch.layers)]
        self.host_pw = {i: torch.from_numpy(wl.normal(tuple(P["w"].shape), seed0 + 700 + i, 0.05))
                        .pin_memory() for i, P in ch.proj.items()}
        self.host_out = torch.empty(ch.layers[-1]["out"].shape, dtype=torch.float32).pin_memory()
        self._upload()
        ch.binarize_weights()
        ch.calibrate()                      # set-up: BatchNorm statistics of the seeded batch
        self.launches = len(ch.layers) + ch.launches_per_forward()
        self.macs = ch.macs()
        self.conv_macs = [wl.macs(s) for s in ch.shapes]
        self.images = batch
        self.h2d = 4 * (self.host_x.numel() + sum(t.numel() for t in self.host_w) +
                        sum(t.numel() for t in self.host_pw.values()))
        self.d2h = 4 * self.host_out.numel()
        self.act_bytes = 0
        for s in ch.shapes:
            ho, wo = wl.out_hw(s)
            px = s.N * s.H * s.W
            self.act_bytes += 4 * (px * s.C_in + px * ((s.C_in + 31) // 32) + 2 * px + s.N * ho * wo)
        self.part_names = ("binarize_weights", "binactiv", "shortcut", "conv")

    def _upload(self):
        ch = self.ch
        ch.x0.copy_(self.host_x, non_blocking=True)
        for L, hw in zip(ch.layers, self.host_w):
            L["w"].copy_(hw, non_blocking=True)
        for i, P in ch.proj.items():
            P["w"].copy_(self.host_pw[i], non_blocking=True)

    def step(self, stream):
        self.ch.binarize_weights(stream)
        if self.fused:
            self.ch.forward_fused(stream)
        else:
            self.ch.forward(stream)

    def step_branches(self, stream):
        """The same step for graph capture.  The layers depend on one another, but the weight
        binarisations depend on nothing and a block's projection shortcut only on the block's
        input: both run on side branches and join where their results are consumed."""
        torch, B, ch = self.torch, self.B, self.ch
        if self.fused:
            return self.step(stream)
        if not hasattr(self, "_sw"):
            self._sw, self._sp = torch.cuda.Stream(), torch.cuda.Stream()
        fork = torch.cuda.Event()
        fork.record(stream)
        self._sw.wait_event(fork)
        self._sp.wait_event(fork)
        ev_w, ev_p = [], {}
        for L in ch.layers:
            B.xnor_binarize_weights(L["w"], L["w_packed"], L["alpha"], self._sw)
            e = torch.cuda.Event()
            e.record(self._sw)
            ev_w.append(e)
        for i, L in enumerate(ch.layers):
            x = ch.layer_input(i)
            if i % 2 == 0 and i in ch.proj:
                ready = torch.cuda.Event()
                ready.record(stream)                  # the block's input is complete
                self._sp.wait_event(ready)
                P = ch.proj[i]
                B.xnor_shortcut_conv1x1(x, P["w"], ch.shapes[i].stride, P["out"], self._sp)
                ev_p[i] = torch.cuda.Event()
                ev_p[i].record(self._sp)
            B.xnor_binactiv(x, L["scale"], L["shift"], L["desc"], L["x_packed"], L["A"], L["K"], stream)
            residual = None
            if i % 2 == 1:
                b0 = i - 1
                if b0 in ch.proj:
                    stream.wait_event(ev_p[b0])
                    residual = ch.proj[b0]["out"]
                else:
                    residual = ch.layer_input(b0)
            stream.wait_event(ev_w[i])
            B.xnor_conv2d_forward(L["x_packed"], L["w_packed"], L["alpha"], L["K"], residual,
                                  L["desc"], L["out"], L["acc"], stream)
        for side in (self._sw, self._sp):
            join = torch.cuda.Event()
            join.record(side)
            stream.wait_event(join)

    def e2e_step(self, stream):
        self._upload()
        self.step(stream)
        self.host_out.copy_(self.ch.layers[-1]["out"], non_blocking=True)

    def parts(self, stream):
        B, ch = self.B, self.ch
        for i, L in enumerate(ch.layers):
            yield "binarize_weights", i, lambda L=L: B.xnor_binarize_weights(
                L["w"], L["w_packed"], L["alpha"], stream)
        for i, L in enumerate(ch.layers):
            x = ch.layer_input(i)
            yield "binactiv", i, lambda L=L, x=x: B.xnor_binactiv(
                x, L["scale"], L["shift"], L["desc"], L["x_packed"], L["A"], L["K"], stream)
            residual = None
            if i % 2 == 1:
                b0 = i - 1
                if b0 in ch.proj:
                    P = ch.proj[b0]
                    yield "shortcut", i, lambda P=P, b0=b0: B.xnor_shortcut_conv1x1(
                        ch.layer_input(b0), P["w"], ch.shapes[b0].stride, P["out"], stream)
                    residual = P["out"]
                else:
                    residual = ch.layer_input(b0)
            yield "conv", i, lambda L=L, residual=residual: B.xnor_conv2d_forward(
                L["x_packed"], L["w_packed"], L["alpha"], L["K"], residual, L["desc"], L["out"],
                None, stream)


def run_ours(args):
    import torch
    import paper_1603_05279_b200 as X

    world, rank, local = du.env_world()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device; there is no CPU path")
    torch.cuda.set_device(local)
    du.init("nccl", local)
    X.load()
    X.xnor_set_engine({"auto": 0, "popc": 1, "umma": 2, "umma_stream": 3}[args.engine])
    stream = torch.cuda.current_stream()

    # every rank has its own batch (weak scaling, no exchange on the data path)
    if args.workload == "chain":
        job = ChainJob(args.batch, rank, fused=args.fused)
    else:
        job = LayersJob(args.workload, args.layer_ids, args.batch, rank, variant=args.variant,
                        kbits=args.kbits)
    torch.cuda.synchronize()
    # the per-clock rates of the two pipes, measured now on this GPU (untimed prologue)
    mma_rate, popc_rate = X.xnor_measure_peaks(stream)

    props = torch.cuda.get_device_properties(local)
    gpu_id = getattr(props, "uuid", None)
    gpu_id = ("GPU-%s" % gpu_id) if gpu_id is not None and not str(gpu_id).startswith("GPU-") \
        else (gpu_id or local)
    sampler = ClockSampler(gpu_id)
    sampler.start()
    time.sleep(0.25)

    # ---- device-resident timing.  One step (all its kernel launches) is captured once in a
    # CUDA graph and replayed, so the timed region holds the kernels and not the Python/ctypes
    # launch overhead between them; --no-graph launches call by call.
    t_load0 = time.time()
    for _ in range(args.warmup):
        job.step(stream)
    torch.cuda.synchronize()
    graph = None
    if not args.no_graph:
        graph = torch.cuda.CUDAGraph()
        branches = hasattr(job, "step_branches") and not args.no_branches
        with torch.cuda.graph(graph):
            if branches:
                job.step_branches(torch.cuda.current_stream())
            else:
                job.step(torch.cuda.current_stream())
        for _ in range(2):
            graph.replay()
        torch.cuda.synchronize()
    du.barrier()
    torch.cuda.synchronize()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ev0.record(stream)
    for _ in range(args.steps):
        if graph is not None:
            graph.replay()
        else:
            job.step(stream)
    ev1.record(stream)
    torch.cuda.synchronize()
    du.barrier()
    elapsed_ms = ev0.elapsed_time(ev1)

    # ---- per-kernel pass (same steps again, one event pair per library call)
    per = {n: {} for n in job.part_names}
    evs = []
    for _ in range(args.steps):
        for name, idx, fn in job.parts(stream):
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(stream)
            fn()
            b.record(stream)
            evs.append((name, idx, a, b))
    torch.cuda.synchronize()
    for name, idx, a, b in evs:
        per[name][idx] = per[name].get(idx, 0.0) + a.elapsed_time(b) / args.steps
    # keep the GPU busy a little longer so that the clock sampler sees it under load
    t_busy = time.time()
    while time.time() - t_busy < 0.6:
        job.step(stream)
        torch.cuda.synchronize()
    t_load1 = time.time()

    # ---- end to end: pinned host -> device, block, device -> pinned host, every step
    for _ in range(min(args.warmup, 3)):
        job.e2e_step(stream)
    torch.cuda.synchronize()
    du.barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for _ in range(args.steps):
        job.e2e_step(stream)
    e1.record(stream)
    torch.cuda.synchronize()
    du.barrier()
    e2e_ms = e0.elapsed_time(e1)
    sampler.stop()
    X.xnor_check_device(stream)

    elapsed_ms, e2e_ms = du.max_over_ranks([elapsed_ms, e2e_ms], device="cuda")

    value = du.job_throughput(job.macs, args.steps, world, elapsed_ms) / 1e12
    e2e_value = du.job_throughput(job.macs, args.steps, world, e2e_ms) / 1e12

    all_layers = args.batch == default_batch(args.workload) and \
        (args.workload == "chain" or args.layer_ids == list(range(len(wl.CONFIGS[args.workload]))))
    full = all_layers and args.variant == "xnor"
    peaks = measured_peaks()
    clocks = sampler.summary(t_load0, t_load1)
    conv_ms = sum(per["conv"].values())
    conv_macs = sum(job.conv_macs)
    engine = args.engine
    n_conv = len(job.conv_macs)
    sms = props.multi_processor_count
    clk_mhz = clocks["sm_mhz"] or 1965.0
    if args.variant in ("bwn", "bgrad"):
        # bf16 x (+-1 as bf16) on kind::f16: the measured bf16 GEMM peak; the burst figure when the
        # sampled clock is the maximum one, else the sustained figure
        burst = clocks["sm_max_mhz"] is not None and clk_mhz >= 0.97 * (clocks["sm_max_mhz"] or clk_mhz)
        peak = peaks["bf16"] if burst else peaks["bf16_sustained"]
        roofline = {"kernel": "bwn_conv_kernel (%d launches per step)" % n_conv, "bound": "tensor",
                    "achieved": 2 * conv_macs / (conv_ms / 1e3) / 1e12, "peak": peak, "unit": "TFLOP/s",
                    "peak_source": "%s bf16 GEMM TFLOP/s, %s figure (SM clock %.0f MHz during the run)"
                                   % (peaks["source"], "burst" if burst else "sustained", clk_mhz),
                    "traffic": None}
    elif engine != "popc":
        # Tensor-core peak of the operand type in use, measured on this GPU before the timed
        # region: 1-bit MACs per clock per SM of tcgen05.mma kind::mxf4 on operands in shared
        # memory, times the SMs, times the median SM clock sampled during the timed steps (so
        # the peak is the one that holds at the clock the kernels really ran at).  2 flops per MAC.
        peak = 2 * mma_rate * sms * clk_mhz * 1e6 / 1e12
        roofline = {"kernel": "BinConv tensor-core kernel (%d launches per step)" % n_conv,
                    "bound": "tensor",
                    "achieved": 2 * conv_macs / (conv_ms / 1e3) / 1e12,
                    "peak": peak, "unit": "TFLOP/s",
                    "peak_source": "measured in this run: tcgen05.mma kind::mxf4 (e2m1) 128x256x64 from "
                                   "shared memory = %.0f MAC/clk/SM x %d SMs x %.0f MHz (median SM clock "
                                   "sampled during the timed steps; reasons: %s)"
                                   % (mma_rate, sms, clk_mhz, ",".join(clocks["reasons"]) or "none"),
                    "peak_nominal": {"4 x bf16 burst": 4 * peaks["bf16"],
                                     "4 x bf16 sustained": 4 * peaks["bf16_sustained"],
                                     "note": "%s bf16 GEMM TFLOP/s x the nominal e2m1 : bf16 ratio"
                                             % peaks["source"]},
                    "mac_per_clk_per_sm": {
                        "peak_measured": round(mma_rate, 1),
                        "achieved": round(conv_macs / (conv_ms / 1e3) / (clk_mhz * 1e6) / sms, 1),
                        "per_layer": [round(job.conv_macs[i] / (per["conv"][k] / 1e3) / (clk_mhz * 1e6) / sms, 1)
                                      for i, k in enumerate(sorted(per["conv"]))]},
                    "traffic": None}
    else:
        peak = popc_rate * 32 * sms * clk_mhz * 1e6 * 2 / 1e12
        roofline = {"kernel": "binconv_popc_kernel (%d launches per step)" % n_conv,
                    "bound": "alu",
                    "achieved": 2 * conv_macs / (conv_ms / 1e3) / 1e12, "peak": peak,
                    "unit": "TFLOP/s",
                    "peak_source": "measured in this run: %.1f popc/clk/SM (XOR + popc + add chains) x 32 "
                                   "bits x %d SMs x %.0f MHz (median SM clock during the run)"
                                   % (popc_rate, sms, clk_mhz),
                    "traffic": None}
    roofline["frac"] = roofline["achieved"] / roofline["peak"]
    if engine != "popc" and args.variant == "xnor" and full and args.workload == "alexnet" and \
            NCU_TRAFFIC["kernel_sha1"] == kernel_sha1():
        roofline["traffic"] = NCU_TRAFFIC["bytes_per_step"]
        roofline["traffic_note"] = ("bytes per step over the 4 launches; below the algorithmic "
                                    "bytes because part of the output is still in L2 at kernel end")
    roofline["algorithmic_bytes_per_step"] = sum(
        4 * (s.N * s.H * s.W * ((s.C_in + 31) // 32) + s.C_out * s.k * s.k * ((s.C_in + 31) // 32)
             + s.N * wl.out_hw(s)[0] * wl.out_hw(s)[1] * (1 + s.C_out) + s.C_out)
        for s in job.shapes)
    act_ms = sum(per["binactiv"].values())

    def ordered(d):
        return [round(d[k], 4) for k in sorted(d)]

    # per layer: the two floors of BinConv (fp32 output write at the measured copy bandwidth;
    # 1-bit MACs at the tensor peak in use) and which of them binds
    def conv_bytes(sh):
        cw = (sh.C_in + 31) // 32
        ho, wo = wl.out_hw(sh)
        return 4 * (sh.N * sh.H * sh.W * cw + sh.C_out * sh.k * sh.k * cw + sh.N * ho * wo * (1 + sh.C_out)
                    + sh.C_out)
    # layers of the chain that add a shortcut read it too
    def residual_bytes(i, sh):
        if args.workload != "chain" or i % 2 == 0:
            return 0
        ho, wo = wl.out_hw(sh)
        return 4 * sh.N * sh.C_out * ho * wo
    hbm_floor = [(conv_bytes(sh) + residual_bytes(i, sh)) / (peaks["hbm_gbs"] * 1e9) * 1e6
                 for i, sh in enumerate(job.shapes)]
    pipe_floor = [2 * m / (roofline["peak"] * 1e12) * 1e6 for m in job.conv_macs]
    breakdown = {
        "conv_floor_us": {"hbm": [round(v, 1) for v in hbm_floor],
                          "pipe": [round(v, 1) for v in pipe_floor],
                          "binding": ["hbm" if h > t else roofline["bound"]
                                      for h, t in zip(hbm_floor, pipe_floor)]},
        "per_layer_ms": {n: ordered(per[n]) for n in job.part_names},
        "conv_TMACs": [round(job.conv_macs[i] / (per["conv"][k] / 1e3) / 1e12, 2)
                       for i, k in enumerate(sorted(per["conv"]))],
        "binactiv_GBs": round(job.act_bytes / (act_ms / 1e3) / 1e9, 1),
        "binactiv_frac_of_hbm": round(job.act_bytes / (act_ms / 1e3) / 1e9 / peaks["hbm_gbs"], 4),
        "hbm_peak_gbs": peaks["hbm_gbs"], "peaks": peaks["source"],
    }

    name = WORKLOAD_NAMES[args.workload]
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": elapsed_ms / args.steps, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None,
        "dtype": ("bf16 activations x 1-bit weights (as +-1 bf16), fp32 accumulation" if args.variant == "bwn"
                  else "1-bit gradient scaled to bf16 x 1-bit weights (as +-1 bf16), fp32 accumulation"
                  if args.variant == "bgrad"
                  else "u32 bit words (XOR+popcount), int32 sums, fp32 scaling" if engine == "popc"
                  else "e2m1 (fp4) tensor-core operands from 1-bit words, exact integer sums in "
                       "fp32, fp32 scaling"),
        "data": "synthetic",
        "config": {"workload": name if full else
                   (name + " (" + args.variant + " variant)") if all_layers and args.variant != "xnor"
                   else "subset of " + name,
                   "layers": [s.name for s in job.shapes],
                   "batch_per_gpu": job.images, "engine": engine,
                   "variant": args.variant + ("%d" % args.kbits if args.variant == "kbit" else ""),
                   "fused_binactiv": bool(getattr(job, "fused", False)),
                   "l2": "step working set %d MB of inputs+outputs (L2 is 126 MB); no flush"
                         % ((job.h2d + job.d2h + (job.act_bytes if args.workload == "chain" else 0))
                            // 1000000),
                   "step": ("weight binarisation (both packings) + max|g|, gradient stream, backward "
                            "convolution for each layer" if args.variant == "bgrad" else
                            "weight binarisation + BN/BinActiv + BinConv for each layer"),
                   "launch": (("one CUDA graph per step, independent work on parallel branches"
                               if branches else "one CUDA graph per step") if graph is not None
                              else "one library call per kernel group")},
        "images_per_s": du.job_throughput(job.images, args.steps, world, elapsed_ms),
        "clocks": clocks,
        "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": job.h2d,
                "d2h_bytes_per_step": job.d2h, "ms_per_step": e2e_ms / args.steps},
        "gpu_launches": job.launches * args.steps,
        "roofline": roofline,
        "kernels": breakdown,
    }
    if rank == 0:
        if world == 1 and full and not args.no_cpu_baseline:
            line["cpu_baseline"] = cpu_baseline(args.workload, args.layer_ids, args.batch)
        print(json.dumps(line), flush=True)
    du.finish()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--ref-images", type=int, default=8,
                    help="images per layer per step of the reference (oracle) arm")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--fused", action="store_true",
                    help="chain workload: every BinConv emits the next layer's BinActiv from its "
                         "epilogue (the per-kernel breakdown still times the plain calls)")
    ap.add_argument("--no-branches", action="store_true",
                    help="capture the step as one chain of launches (no parallel branches)")
    ap.add_argument("--no-graph", action="store_true",
                    help="time call-by-call launches instead of a CUDA graph of the step")
    ap.add_argument("--engine", default="auto", choices=["auto", "popc", "umma", "umma_stream"])
    ap.add_argument("--variant", default="xnor", choices=["xnor", "bwn", "kbit", "bgrad"],
                    help="layer workloads only: the XNOR block (default, the bench line), the "
                         "Binary-Weight-Network convolution on real inputs, k-bit activations, or the "
                         "backward convolution with a binarised gradient (stride-1 layers)")
    ap.add_argument("--kbits", type=int, default=2, help="bits of the k-bit variant")
    ap.add_argument("--workload", default="alexnet", choices=sorted(WORKLOAD_NAMES),
                    help="shape set (the bench line proper is the default, alexnet)")
    ap.add_argument("--layers", default="",
                    help="subset of the workload's layers, e.g. 0,2 (profiling runs only)")
    ap.add_argument("--batch", type=int, default=0, help="images per GPU (default: the workload's)")
    args = ap.parse_args()
    if args.batch <= 0:
        args.batch = default_batch(args.workload)
    n_layers = 16 if args.workload == "chain" else len(wl.CONFIGS[args.workload])
    args.layer_ids = [int(t) for t in args.layers.split(",")] if args.layers else \
        list(range(n_layers))
    if args.warmup < 3 and args.impl == "ours":
        args.warmup = 3
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()

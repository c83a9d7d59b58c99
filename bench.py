#!/usr/bin/env python
"""Benchmark of the XNOR-Net forward block on B200.

One step = one pass of the whole hot path over one batch: for each of the four
AlexNet-shaped binary convolution layers (batch 256 per GPU, synthetic seeded
inputs) weight binarisation, BN affine + BinActiv (sign-pack, A, K) and BinConv.
Prints ONE JSON line (rank 0).  `--impl reference` times the CPU oracle instead.
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

from paper_1603_05279_b200 import workloads as wl  # noqa: E402

METRIC = "binary conv TOPS (1-bit MACs/s)"
UNIT = "T 1-bit MAC/s"
WORKLOAD = "alexnet_conv2-5_batch256"
HBM_FALLBACK_GBS = 6650.0
BF16_FALLBACK_TFLOPS = 1590.0
# popc engine: population count issues 16 results per clock per SM (CUDA C programming
# guide, arithmetic-instruction throughput table, compute capability 10.0); one result
# covers 32 one-bit MACs.
POPC_PER_CLK_PER_SM = 16


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


# ------------------------------------------------------------------ CPU oracle timing
def oracle_pass(n_images, seeds_rank=0):
    """Times the oracle, as it stands, on the first n_images of each layer's batch.
    Returns (seconds, macs)."""
    import oracle
    total_t, total_macs = 0.0, 0
    for li, s in enumerate(wl.ALEXNET):
        seed = wl.layer_seed("alexnet", li) + 100000 * seeds_rank
        x = wl.make_input(s, seed, n_images=n_images)
        w = wl.make_weights(s, seed)
        scale = np.ones((s.C_in,), np.float32)
        shift = np.zeros((s.C_in,), np.float32)
        t0 = time.perf_counter()
        oracle.xnor_block(x, w, s.stride, s.pad, scale, shift)
        total_t += time.perf_counter() - t0
        total_macs += wl.macs(wl.scaled(s, n_images))
    return total_t, total_macs


def cpu_baseline(budget_s=12.0):
    import oracle
    oracle.build()
    cores = host_cores()
    oracle.set_num_threads(cores)
    n = 2
    t, m = oracle_pass(n)
    want = int(min(256, max(2, n * budget_s / max(t, 1e-3))))
    if want > n:
        n = want
        t, m = oracle_pass(n)
    return dict(value=m / t / 1e12, unit=UNIT, cores=oracle.num_threads(), kind="oracle",
                sample="first %d of 256 images of each of the 4 layers, whole block "
                       "(BN, BinActiv, weight binarisation, BinConv); %.1f s" % (n, t),
                images_per_s=n / t)


def run_reference(args):
    """The reference arm: the CPU oracle on a bounded sample per step."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle
    oracle.build()
    cores = host_cores()
    oracle.set_num_threads(cores)
    n = args.ref_images
    for _ in range(args.warmup):
        oracle_pass(n)
    t_total, m_total = 0.0, 0
    for _ in range(args.steps):
        t, m = oracle_pass(n)
        t_total += t
        m_total += m
    value = m_total / t_total / 1e12
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT,
        "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": 1e3 * t_total / args.steps, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "int8 (+-1 products, int32 sums)", "data": "synthetic",
        "config": {"workload": WORKLOAD, "sample_images_per_step": n},
        "images_per_s": n * args.steps / t_total,
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": oracle.num_threads(),
                         "kind": "oracle",
                         "sample": "each step = first %d of 256 images of each layer" % n},
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
                 "--format=csv,noheader,nounits", "-lms", "100"],
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


# ------------------------------------------------------------------ the CUDA arm
def run_ours(args):
    import torch
    import torch.distributed as dist
    import paper_1603_05279_b200 as X
    from paper_1603_05279_b200.runner import LAUNCHES_PER_LAYER, LayerBuffers

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device; there is no CPU path")
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    X.load()
    X.xnor_set_engine({"auto": 0, "popc": 1, "umma": 2, "umma_i8": 3}[args.engine])
    stream = torch.cuda.current_stream()

    # ---- synthetic inputs: every rank has its own batch of 256 (weak scaling, no exchange)
    shapes = [wl.scaled(wl.ALEXNET[i], args.batch) for i in args.layer_ids]
    layers = [LayerBuffers(s) for s in shapes]
    host_x, host_w, host_out = [], [], []
    for li, L in enumerate(layers):
        seed = wl.layer_seed("alexnet", args.layer_ids[li]) + 100000 * rank
        hx = torch.from_numpy(wl.make_input(L.shape, seed)).pin_memory()
        hw = torch.from_numpy(wl.make_weights(L.shape, seed)).pin_memory()
        host_x.append(hx)
        host_w.append(hw)
        host_out.append(torch.empty(L.out.shape, dtype=torch.float32).pin_memory())
        L.x.copy_(hx)
        L.w.copy_(hw)
    torch.cuda.synchronize()

    def step():
        for L in layers:
            L.forward(stream)

    def barrier():
        if world > 1:
            dist.barrier()

    props = torch.cuda.get_device_properties(local)
    gpu_id = getattr(props, "uuid", None)
    gpu_id = ("GPU-%s" % gpu_id) if gpu_id is not None and not str(gpu_id).startswith("GPU-") \
        else (gpu_id or local)
    sampler = ClockSampler(gpu_id)
    sampler.start()
    time.sleep(0.25)

    # ---- device-resident timing
    t_load0 = time.time()
    for _ in range(args.warmup):
        step()
    torch.cuda.synchronize()
    barrier()
    torch.cuda.synchronize()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ev0.record(stream)
    for _ in range(args.steps):
        step()
    ev1.record(stream)
    torch.cuda.synchronize()
    barrier()
    elapsed_ms = ev0.elapsed_time(ev1)

    # ---- per-kernel pass (same steps again, one event pair per launch group)
    names = ("binarize_weights", "binactiv", "conv")
    per = {n: [0.0] * len(layers) for n in names}
    evs = []
    for _ in range(args.steps):
        for li, L in enumerate(layers):
            e = [torch.cuda.Event(enable_timing=True) for _ in range(4)]
            e[0].record(stream)
            L.binarize_weights(stream)
            e[1].record(stream)
            L.binactiv(stream)
            e[2].record(stream)
            L.conv(stream)
            e[3].record(stream)
            evs.append((li, e))
    torch.cuda.synchronize()
    for li, e in evs:
        for k, n in enumerate(names):
            per[n][li] += e[k].elapsed_time(e[k + 1]) / args.steps
    t_load1 = time.time()

    # ---- end to end: pinned host -> device, block, device -> pinned host, every step
    def e2e_step():
        for li, L in enumerate(layers):
            L.x.copy_(host_x[li], non_blocking=True)
            L.w.copy_(host_w[li], non_blocking=True)
            L.forward(stream)
            host_out[li].copy_(L.out, non_blocking=True)

    for _ in range(min(args.warmup, 3)):
        e2e_step()
    torch.cuda.synchronize()
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for _ in range(args.steps):
        e2e_step()
    e1.record(stream)
    torch.cuda.synchronize()
    barrier()
    e2e_ms = e0.elapsed_time(e1)
    sampler.stop()
    X.xnor_check_device(stream)

    if world > 1:
        t = torch.tensor([elapsed_ms, e2e_ms], device="cuda", dtype=torch.float64)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        elapsed_ms, e2e_ms = float(t[0]), float(t[1])

    macs_step = sum(wl.macs(L.shape) for L in layers)
    images_step = args.batch
    sec = elapsed_ms / 1e3
    value = world * macs_step * args.steps / sec / 1e12
    e2e_value = world * macs_step * args.steps / (e2e_ms / 1e3) / 1e12
    h2d = sum(t.numel() * 4 for t in host_x) + sum(t.numel() * 4 for t in host_w)
    d2h = sum(t.numel() * 4 for t in host_out)

    full = args.batch == 256 and args.layer_ids == [0, 1, 2, 3]
    peaks = measured_peaks()
    clocks = sampler.summary(t_load0, t_load1)
    conv_ms = sum(per["conv"])
    conv_macs = macs_step
    engine = args.engine
    if engine == "auto":
        engine = "umma" if all(s.stride == 1 for s in shapes) else "mixed"
    if engine != "popc":
        # tensor-core peak for the operand type in use = measured bf16 peak x the nominal
        # ratio of that type to bf16 (e2m1: 9 / 2.25 = 4, int8: 2); the sustained figure,
        # because the kernel is timed inside a long step.  2 flops per 1-bit MAC.
        ratio, kind = (2, "int8") if engine == "umma_i8" else (4, "e2m1 (fp4)")
        roofline = {"kernel": "BinConv tensor-core kernel (one launch per layer, %d per step)"
                              % len(layers), "bound": "tensor",
                    "achieved": 2 * conv_macs / (conv_ms / 1e3) / 1e12,
                    "peak": ratio * peaks["bf16_sustained"], "unit": "TFLOP/s",
                    "peak_source": "%d x %s sustained bf16 TFLOP/s (nominal %s : bf16 ratio)"
                                   % (ratio, peaks["source"], kind), "traffic": None}
    else:
        clk = (clocks["sm_mhz"] or 1965.0) * 1e6
        peak = POPC_PER_CLK_PER_SM * 32 * props.multi_processor_count * clk * 2 / 1e12
        roofline = {"kernel": "binconv_popc_kernel (4 launches per step)", "bound": "alu",
                    "achieved": 2 * conv_macs / (conv_ms / 1e3) / 1e12, "peak": peak,
                    "unit": "TFLOP/s",
                    "peak_source": "derived: 16 popc/clk/SM x 32 bits x %d SMs x median SM clock "
                                   "during the run" % props.multi_processor_count,
                    "traffic": None}
    roofline["frac"] = roofline["achieved"] / roofline["peak"]
    act_bytes = sum(L.binactiv_bytes() for L in layers)
    act_ms = sum(per["binactiv"])
    breakdown = {
        "per_layer_ms": {n: [round(v, 4) for v in per[n]] for n in names},
        "conv_TMACs": [round(wl.macs(L.shape) / (per["conv"][i] / 1e3) / 1e12, 2)
                       for i, L in enumerate(layers)],
        "binactiv_GBs": round(act_bytes / (act_ms / 1e3) / 1e9, 1),
        "binactiv_frac_of_hbm": round(act_bytes / (act_ms / 1e3) / 1e9 / peaks["hbm_gbs"], 4),
        "hbm_peak_gbs": peaks["hbm_gbs"], "peaks": peaks["source"],
    }

    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": elapsed_ms / args.steps, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None,
        "dtype": ("u32 bit words (XOR+popcount), int32 sums, fp32 scaling" if engine == "popc"
                  else "int8 +-1/0 tensor-core operands from 1-bit words, int32 sums, fp32 scaling"
                  if engine == "umma_i8"
                  else "e2m1 (fp4) tensor-core operands from 1-bit words, exact integer sums in "
                       "fp32, fp32 scaling"),
        "data": "synthetic",
        "config": {"workload": WORKLOAD if full else "subset of " + WORKLOAD,
                   "layers": [s.name for s in shapes],
                   "batch_per_gpu": images_step, "engine": engine,
                   "l2": "step working set %d MB of inputs+outputs (L2 is 126 MB); no flush"
                         % ((h2d + d2h) // 1000000),
                   "step": "weight binarisation + BN/BinActiv + BinConv for each layer"},
        "images_per_s": world * images_step * args.steps / sec,
        "clocks": clocks,
        "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": h2d,
                "d2h_bytes_per_step": d2h, "ms_per_step": e2e_ms / args.steps},
        "gpu_launches": LAUNCHES_PER_LAYER * len(layers) * args.steps,
        "roofline": roofline,
        "kernels": breakdown,
    }
    if rank == 0:
        if world == 1 and full and not args.no_cpu_baseline:
            line["cpu_baseline"] = cpu_baseline()
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--ref-images", type=int, default=8,
                    help="images per layer per step of the reference (oracle) arm")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--engine", default="auto", choices=["auto", "popc", "umma", "umma_i8"])
    ap.add_argument("--layers", default="0,1,2,3",
                    help="subset of the four layers (profiling runs only; the bench line is the "
                         "default: all four)")
    ap.add_argument("--batch", type=int, default=256, help="images per GPU (default 256)")
    args = ap.parse_args()
    args.layer_ids = [int(t) for t in args.layers.split(",")]
    if args.warmup < 3 and args.impl == "ours":
        args.warmup = 3
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()

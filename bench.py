#!/usr/bin/env python
"""Benchmark of the LoPRo quantized-linear forward on B200.

Default workload: the decode configuration (4096 x 4096, 4-bit g128, block 128, rank 32, 8 tokens).
One step = one forward of the token batch through every layer of a ring of distinct synthetic
layers; the ring is larger than the L2 cache, so every layer's packed weights come from HBM.
Prints ONE JSON line (see README / DESIGN for the keys).

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl reference]

With N > 1 (launched by torch.distributed.run) every rank runs an independent replica on its own GPU
(the path has no exchange step); the time is the maximum over ranks.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

WORKLOADS = {
    # name: (config, tokens, layers in the ring)
    "cfg2_T8": ("cfg2", 8, 64),
    "cfg2_T1": ("cfg2", 1, 64),
    "cfg2_T16": ("cfg2", 16, 64),
    "cfg2_T32": ("cfg2", 32, 64),
    # one layer repeated: its 9.5 MB of packed weights stay in the 126 MB L2 (reported as such, never the bench line)
    "cfg2_T8_L2": ("cfg2", 8, 64),
    "cfg3_T2048": ("cfg3", 2048, 8),
    "cfg4_T16": ("cfg4", 16, 8),
    "cfg4_T4096": ("cfg4", 4096, 2),
    # the linears of the synthetic 32-layer decoder stack (7 per layer, 224 distinct layers, 3.6 GB of packed weights);
    # attention, norms and activations are not part of the method and are not run
    "cfg5_T1": ("cfg5", 1, 224),
    "cfg5_T32": ("cfg5", 32, 224),
}
# linears of one layer of the stack: name, d_in, d_out (hidden 4096, MLP 11008)
STACK_LINEARS = [("q", 4096, 4096), ("k", 4096, 4096), ("v", 4096, 4096), ("o", 4096, 4096),
                 ("gate", 4096, 11008), ("up", 4096, 11008), ("down", 11008, 4096)]
STACK_LAYERS = 32
STACK_QUANT = dict(bits=4, group_size=128, block_size=128, identity_cols=128, rank=32)


def stack_shape(n, m):
    return dict(d_in=n, d_out=m, **STACK_QUANT)


def stack_bytes(T):
    return STACK_LAYERS * sum(algorithmic_bytes(stack_shape(n, m), T) for _, n, m in STACK_LINEARS)


def time_oracle_stack(T, budget_s):
    """The oracle on the three linear shapes of the stack (1024 sampled output rows each), combined into the
    time of one pass through all 224 linears."""
    shapes = {}
    for _, n, m in STACK_LINEARS:
        shapes[(n, m)] = shapes.get((n, m), 0) + 1
    total, cores, desc = 0.0, 1, []
    for (n, m), count in shapes.items():
        r = time_oracle(stack_shape(n, m), T, budget_s / len(shapes), 1024, None)
        total += STACK_LAYERS * count * r["seconds_per_layer"]
        cores = r["cores"]
        desc.append(f"{n}->{m}: {r['rows']} rows x {r['reps']} reps")
    return dict(value=T / total, cores=cores, sample="oracle.forward_exact (fp64 numpy) on sampled rows of the three "
                "linear shapes (" + "; ".join(desc) + f"), {T} tokens, scaled linearly to 32 layers x 7 linears")

# DRAM bytes (dram__bytes_read.sum + dram__bytes_write.sum) per launch of the dominant kernel, from the ncu
# capture summarised in profiles/; valid for the kernel as committed with that summary, null otherwise.
NCU_TRAFFIC = {("cfg2_T8", "stream_wide_kernel"): 9296640, ("cfg4_T16", "tall_kernel"): 83635840,
               ("cfg3_T2048", "prefill_kernel"): 53210752}
METRIC = "quantized-linear fwd tokens/s"
UNIT = "tokens/s"


def algorithmic_bytes(c, T):
    """Bytes the method must move per layer forward: codes, (scale, zero) pairs, A and B, perm, x in, y out."""
    m, n, q, g, r = c["d_out"], c["d_in"], c["bits"], c["group_size"], c["rank"]
    return m * n * q // 8 + m * (n // g) * 4 + (m * r + r * n) * 2 + n * 4 + T * (n + m) * 2


def algorithmic_flops(c, T):
    m, n, r = c["d_out"], c["d_in"], c["rank"]
    return 2 * T * m * n + 2 * T * r * (m + n)


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return dict(hbm_gbs=p["hbm_gbs"], bf16_tflops=p["bf16_tflops"],
                    bf16_tflops_sustained=p.get("bf16_tflops_sustained", p["bf16_tflops"]), source="measured")
    return dict(hbm_gbs=6650.0, bf16_tflops=1590.0, bf16_tflops_sustained=1400.0, source="fallback")


class ClockSampler:
    """Samples SM clock and throttle reasons of one GPU with nvidia-smi while the timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index = index
        self.lines = []
        self.proc = None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.FIELDS}",
                                          "--format=csv,noheader,nounits", "-lms", "50"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self):
        if self.proc is None:
            return dict(sm_mhz=None, sm_max_mhz=None, reasons=["nvidia-smi unavailable"])
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in self.lines:
            parts = [p.strip() for p in line.split(",")]
            if len(parts) < 7:
                continue
            try:
                sm.append(float(parts[0]))
                mx.append(float(parts[1]))
            except ValueError:
                continue
            for name, v in zip(names, parts[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        return dict(sm_mhz=statistics.median(sm) if sm else None, sm_max_mhz=max(mx) if mx else None,
                    samples=len(sm), reasons=sorted(reasons))


def max_over_ranks(values, device):
    """Replicas: every rank times its own copy of the job; the job's time is the slowest rank's.  Element-wise
    maximum of `values` over the ranks of the default process group, followed by a barrier."""
    import torch
    import torch.distributed as dist
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    dist.barrier()
    return [float(v) for v in t]


def oracle_layer_inputs(c, T, seed):
    from oracle import lopro_oracle as o
    from paper_2601_19675_b200 import synth
    layer = synth.random_layer(c["d_in"], c["d_out"], c["bits"], c["group_size"], c["rank"], seed=seed)
    x_bits = synth.activations(T, c["d_in"], seed=seed, outlier_frac=c.get("outlier_frac", 0.0),
                               outlier_scale=c.get("outlier_scale", 20.0))
    args = dict(codes=layer["codes"], scales=o.f16_bits_to_f64(layer["scales"]), zeros=o.f16_bits_to_f64(layer["zeros"]),
                perm=layer["perm"], a=o.f16_bits_to_f64(layer["A"]), b=o.f16_bits_to_f64(layer["B"]),
                g=c["group_size"], b_i=c["identity_cols"], b_h=c["block_size"])
    return o.bf16_bits_to_f64(x_bits), args


def blas_threads():
    try:
        from threadpoolctl import threadpool_info
        n = [i.get("num_threads", 1) for i in threadpool_info() if i.get("user_api") == "blas"]
        return max(n) if n else 1
    except Exception:
        return 1


def time_oracle(c, T, budget_s, max_rows=None, max_tokens=None):
    """Times oracle.forward_exact as it stands on a bounded sample: the first `rows` output rows and the
    first `toks` tokens of one layer, repeated until about budget_s seconds have passed."""
    from oracle import lopro_oracle as o
    rows = min(c["d_out"], max_rows or c["d_out"])
    toks = min(T, max_tokens or T)
    x64, args = oracle_layer_inputs(c, toks, seed=0)
    for k in ("codes", "scales", "zeros", "a"):
        args[k] = args[k][:rows]
    o.forward_exact(x64, **args)  # touch everything once
    reps, t0 = 0, time.perf_counter()
    while True:
        o.forward_exact(x64, **args)
        reps += 1
        el = time.perf_counter() - t0
        if el >= budget_s or reps >= 1000:
            break
    # tokens/s of a full layer forward, scaled from the sampled rows (cost is linear in the rows)
    per_layer = el / reps * (c["d_out"] / rows)
    return dict(value=toks / per_layer, seconds_per_layer=per_layer, reps=reps, rows=rows, tokens=toks,
                cores=blas_threads())


def run_reference(args):
    """--impl reference: the CPU oracle, timed on the host cores, same metric and config keys."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return 0
    from paper_2601_19675_b200 import synth
    cfg, T, ring = WORKLOADS[args.workload]
    if cfg == "cfg5":
        for _ in range(args.warmup):
            time_oracle_stack(T, 0.0)
        t0 = time.perf_counter()
        results = [time_oracle_stack(T, 1.5) for _ in range(args.steps)]
        wall = time.perf_counter() - t0
        value = statistics.median(r["value"] for r in results)
        line = dict(impl="reference", metric=METRIC, value=value, unit=UNIT, n_gpus=int(os.environ.get("WORLD_SIZE", "1")),
                    steps=args.steps, warmup=args.warmup, ms_per_step=wall / args.steps * 1e3, higher_is_better=True,
                    scaling="weak", vs_baseline=None, dtype="f64", data="synthetic", config=workload_config(args.workload),
                    cpu_baseline=dict(value=value, unit=UNIT, cores=results[0]["cores"], kind="oracle",
                                      sample=results[0]["sample"]),
                    e2e=dict(value=value, unit=UNIT, h2d_bytes_per_step=0, d2h_bytes_per_step=0))
        print(json.dumps(line))
        return 0
    c = synth.CONFIGS[cfg]
    max_rows = 1024 if c["d_out"] * c["d_in"] > (1 << 24) or T > 64 else None
    max_tokens = 16 if T > 64 else None
    per_step_budget = 1.5
    for _ in range(args.warmup):
        time_oracle(c, T, 0.0, max_rows, max_tokens)
    t0 = time.perf_counter()
    results = [time_oracle(c, T, per_step_budget, max_rows, max_tokens) for _ in range(args.steps)]
    wall = time.perf_counter() - t0
    value = statistics.median(r["value"] for r in results)
    sample = (f"oracle.forward_exact (fp64 numpy) on {results[0]['rows']} of {c['d_out']} output rows and "
              f"{results[0]['tokens']} of {T} tokens of one layer, scaled linearly to the full layer; "
              f"each step repeats it for ~{per_step_budget} s")
    line = dict(impl="reference", metric=METRIC, value=value, unit=UNIT, n_gpus=args.gpus, steps=args.steps,
                warmup=args.warmup, ms_per_step=wall / max(args.steps, 1) * 1e3, higher_is_better=True,
                scaling="weak", vs_baseline=None, dtype="f64", data="synthetic",
                config=workload_config(args.workload),
                cpu_baseline=dict(value=value, unit=UNIT, cores=results[0]["cores"], kind="oracle", sample=sample),
                e2e=dict(value=value, unit=UNIT, h2d_bytes_per_step=0, d2h_bytes_per_step=0))
    print(json.dumps(line))
    return 0


def workload_config(name):
    from paper_2601_19675_b200 import synth
    cfg, T, ring = WORKLOADS[name]
    if cfg == "cfg5":
        return dict(workload=f"{name}: the 224 LoPRo linears of a 32-layer decoder stack (hidden 4096, MLP 11008; 4-bit g128 "
                             f"block 128 rank 32), batch {T}, one token per sequence; attention/norm/activation glue not run",
                    tokens=T, ring_layers=ring,
                    l2="inputs larger than L2: one step reads %.0f MB of packed weights" % (stack_bytes(T) / 1e6))
    c = synth.CONFIGS[cfg]
    ring_bytes = ring * algorithmic_bytes(c, T)
    return dict(workload=f"{name}: LoPRo linear forward d_in={c['d_in']} d_out={c['d_out']} {c['bits']}-bit g{c['group_size']} "
                         f"block {c['block_size']} rank {c['rank']}, {T} tokens per forward",
                tokens=T, ring_layers=ring,
                l2=("L2-RESIDENT: one layer repeated %d times per step, its %.1f MB of packed weights stay in L2 between forwards"
                    % (ring, ring_bytes / ring / 1e6)) if name.endswith("_L2") else
                   "inputs larger than L2: every step walks a ring of %d distinct layers (%.0f MB of packed weights)"
                   % (ring, ring_bytes / 1e6))


def run_stack(args, T, rank, world, local, dev, dev16):
    """The 224 linears of the 32-layer stack, one forward each per step, every linear with its own packed layer.
    Linears with 4096 inputs read one fixed activation tensor, the `down` projections another (the glue between
    them is not part of the method and is not run; the kernels' work does not depend on the values)."""
    import torch
    from paper_2601_19675_b200 import lopro, synth
    if world > 1:
        import torch.distributed as dist
    q = STACK_QUANT
    shapes = sorted({(n, m) for _, n, m in STACK_LINEARS})
    base, descs = {}, {}
    for n, m in shapes:
        layer = synth.random_layer(n, m, q["bits"], q["group_size"], q["rank"], seed=rank + n // 64)
        base[(n, m)] = dict(codes=torch.from_numpy(layer["codes"]).to(dev), sc=dev16(layer["scales"]), zr=dev16(layer["zeros"]),
                            pm=torch.from_numpy(layer["perm"]).to(dev), A=dev16(layer["A"]), B=dev16(layer["B"]))
        descs[(n, m)] = lopro.make_desc(n, m, q["bits"], q["group_size"], q["block_size"], q["identity_cols"], q["rank"],
                                        layout=lopro.LAYOUT_ROWBLOCK if args.layout == "rowblock" else lopro.LAYOUT_FRAGMENT)
    xs, x_bits = {}, {}
    for n in sorted({n for n, _ in shapes}):
        x_bits[n] = synth.activations(T, n, seed=rank + n)
        xs[n] = dev16(x_bits[n]).view(torch.bfloat16)
    ys = {m: [torch.empty((T, m), dtype=torch.bfloat16, device=dev) for _ in range(2)] for m in sorted({m for _, m in shapes})}
    ws_bytes = max(lopro.workspace_bytes(descs[k], T) for k in shapes)
    ws = torch.zeros(ws_bytes, dtype=torch.uint8, device=dev)
    linears = []  # (desc, blob, x, y)
    for li in range(STACK_LAYERS):
        for j, (_, n, m) in enumerate(STACK_LINEARS):
            b = base[(n, m)]
            i = li * len(STACK_LINEARS) + j
            codes = torch.roll(b["codes"], shifts=(i, 3 * i), dims=(0, 1)) if i else b["codes"]
            blob = lopro.pack(descs[(n, m)], codes, b["sc"], b["zr"], b["pm"], b["A"], b["B"])
            y = torch.empty((T, m), dtype=torch.bfloat16, device=dev) if j in (1, 2, 5) else ys[m][i % 2]
            linears.append((descs[(n, m)], blob, xs[n], y))
    del codes
    for b in base.values():
        del b["codes"]
    # sibling linears of a layer read the same activations: (q, k, v) and (gate, up) go through the grouped call
    groups = []
    for li in range(STACK_LAYERS):
        L7 = linears[li * 7:(li + 1) * 7]
        for idx in ((0, 1, 2), (3,), (4, 5), (6,)) if not args.no_groups else ((0,), (1,), (2,), (3,), (4,), (5,), (6,)):
            part = [L7[k] for k in idx]
            groups.append(([g[0] for g in part], [g[1] for g in part], part[0][2], [g[3] for g in part]))
    gws_bytes = max(lopro.group_workspace_bytes(g[0], T) for g in groups)
    ws = torch.zeros(max(ws_bytes, gws_bytes), dtype=torch.uint8, device=dev)

    def one_step():
        for ds, blobs_, x, ys_ in groups:
            if len(ds) == 1:
                lopro.linear_fwd(ds[0], blobs_[0], x, lopro.OUT_BF16, workspace=ws, y=ys_[0])
            else:
                lopro.linear_fwd_group(ds, blobs_, x, lopro.OUT_BF16, workspace=ws, ys=ys_)

    stream = torch.cuda.Stream(device=dev)
    graph = None
    with torch.cuda.stream(stream):
        one_step()
        stream.synchronize()
        if not args.no_graph:
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph, stream=stream):
                one_step()
        run_step = graph.replay if graph is not None else one_step
        for _ in range(args.warmup):
            run_step()
        stream.synchronize()
        if world > 1:
            dist.barrier()
        sampler = ClockSampler(local)
        if rank == 0:
            sampler.start()
        torch.cuda.synchronize()
        ev = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps + 1)]
        ev[0].record(stream)
        for k in range(args.steps):
            run_step()
            ev[k + 1].record(stream)
        stream.synchronize()
        torch.cuda.synchronize()
        clocks = sampler.stop() if rank == 0 else None
        total_ms = ev[0].elapsed_time(ev[-1])
        step_ms = [ev[k].elapsed_time(ev[k + 1]) for k in range(args.steps)]
        # end to end: the batch's activations come from pinned host memory every step, the last linear's output
        # goes back to the host
        xh = torch.from_numpy(x_bits[4096].view(np.int16)).view(torch.bfloat16).pin_memory()
        y_last = linears[-1][3]
        yh = torch.empty(tuple(y_last.shape), dtype=torch.bfloat16).pin_memory()
        e2e_steps = max(3, min(args.steps, 20))

        def e2e_step():
            xs[4096].copy_(xh, non_blocking=True)
            run_step()
            yh.copy_(y_last, non_blocking=True)

        for _ in range(3):
            e2e_step()
        stream.synchronize()
        if world > 1:
            dist.barrier()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(e2e_steps):
            e2e_step()
        e1.record(stream)
        stream.synchronize()
        e2e_ms = e0.elapsed_time(e1)
        status = lopro.workspace_status(ws)
        assert status == lopro.OK, f"device status {status}"
        assert torch.isfinite(yh.float()).all()
    if world > 1:
        total_ms, e2e_ms = max_over_ranks([total_ms, e2e_ms], dev)
    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return 0
    peaks = measured_peaks()
    ms_per_step = total_ms / args.steps
    value = T * world / (ms_per_step * 1e-3)
    e2e_value = T * world / (e2e_ms / e2e_steps * 1e-3)
    paths = [lopro.linear_fwd_path(d, T) for d, _, _, _ in linears]
    names = sorted({lopro.PATH_NAMES.get(p, "?") for p, _ in paths})
    n_launches = sum(lopro.linear_fwd_group_path(g[0], T)[1] if len(g[0]) > 1 else lopro.linear_fwd_path(g[0][0], T)[1]
                     for g in groups)
    ach = stack_bytes(T) / (ms_per_step * 1e-3) / 1e9
    roofline = dict(bound="hbm", achieved=ach, peak=peaks["hbm_gbs"], unit="GB/s", frac=ach / peaks["hbm_gbs"], traffic=None,
                    peak_source=f"of {peaks['source']}", frac_of_nominal_8000=ach / 8000.0,
                    kernel=" + ".join(n + "_kernel" for n in names), algorithmic_bytes_per_step=stack_bytes(T),
                    launch_us=ms_per_step * 1e3 / len(linears),
                    note="whole step: 224 linear forwards (prologue kernels included); launch_us = step time / 224")
    line = dict(metric=METRIC, value=value, unit=UNIT, n_gpus=world, steps=args.steps, warmup=args.warmup,
                ms_per_step=ms_per_step, higher_is_better=True, scaling="weak", vs_baseline=None, dtype="bf16",
                data="synthetic", config=workload_config(args.workload), clocks=clocks,
                e2e=dict(value=e2e_value, unit=UNIT, h2d_bytes_per_step=T * 4096 * 2, d2h_bytes_per_step=T * y_last.shape[1] * 2,
                         steps=e2e_steps),
                gpu_launches=n_launches * args.steps, path="+".join(names), launches_per_step=n_launches, roofline=roofline,
                step_ms_min=min(step_ms), step_ms_median=statistics.median(step_ms), cuda_graph=graph is not None)
    if not args.no_cpu_baseline and world == 1:
        r = time_oracle_stack(T, 12.0)
        line["cpu_baseline"] = dict(value=r["value"], unit=UNIT, cores=r["cores"], kind="oracle", sample=r["sample"])
    print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()
    return 0


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=400)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--workload", default="cfg2_T8", choices=sorted(WORKLOADS))
    ap.add_argument("--impl", default="lopro", choices=["lopro", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-graph", action="store_true", help="launch through the stream instead of a CUDA graph")
    ap.add_argument("--no-groups", action="store_true", help="stack workloads: every linear on its own (no grouped siblings)")
    ap.add_argument("--layout", default="fragment", choices=["fragment", "rowblock"], help="code layout of the packed layers")
    args = ap.parse_args()
    if args.impl == "reference":
        return run_reference(args)
    if args.warmup < 3:
        args.warmup = 3

    import torch
    from paper_2601_19675_b200 import build, lopro, synth

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback)")
    torch.cuda.set_device(local)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    if rank == 0:
        build.build()
    if world > 1:
        dist.barrier()
    lopro.lib()

    cfg, T, ring = WORKLOADS[args.workload]
    dev = torch.device("cuda", local)

    def dev16(a):
        return torch.from_numpy(np.ascontiguousarray(a).view(np.int16)).to(dev)

    if cfg == "cfg5":
        return run_stack(args, T, rank, world, local, dev, dev16)
    c = synth.CONFIGS[cfg]
    d = lopro.make_desc(c["d_in"], c["d_out"], c["bits"], c["group_size"], c["block_size"], c["identity_cols"], c["rank"],
                        layout=lopro.LAYOUT_ROWBLOCK if args.layout == "rowblock" else lopro.LAYOUT_FRAGMENT)

    # ring of distinct layers: layer 0 drawn by the seeded generator, the others re-use its tensors with
    # freshly drawn codes (generated on the host once, shifted per layer) so that set-up stays short
    base = synth.random_layer(c["d_in"], c["d_out"], c["bits"], c["group_size"], c["rank"], seed=rank)
    sc, zr, pm, A, B = dev16(base["scales"]), dev16(base["zeros"]), torch.from_numpy(base["perm"]).to(dev), \
        dev16(base["A"]), dev16(base["B"])
    codes0 = torch.from_numpy(base["codes"]).to(dev)
    blobs = []
    for i in range(ring):
        if args.workload.endswith("_L2") and i:
            blobs.append(blobs[0])  # the same packed layer again: L2-resident measurement
            continue
        codes = torch.roll(codes0, shifts=(i, 3 * i), dims=(0, 1)) if i else codes0
        blobs.append(lopro.pack(d, codes, sc, zr, pm, A, B))
    del codes0, codes
    x_bits = synth.activations(T, c["d_in"], seed=rank, outlier_frac=c.get("outlier_frac", 0.0),
                               outlier_scale=c.get("outlier_scale", 20.0))
    x = dev16(x_bits).view(torch.bfloat16)
    ys = [torch.empty((T, c["d_out"]), dtype=torch.bfloat16, device=dev) for _ in range(min(ring, 4))]
    ws = torch.zeros(lopro.workspace_bytes(d, T) + lopro.host_staging_bytes(d, T), dtype=torch.uint8, device=dev)

    def one_step():
        for i, blob in enumerate(blobs):
            lopro.linear_fwd(d, blob, x, lopro.OUT_BF16, workspace=ws, y=ys[i % len(ys)])

    stream = torch.cuda.Stream(device=dev)
    graph = None
    with torch.cuda.stream(stream):
        one_step()
        stream.synchronize()
        if not args.no_graph:
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph, stream=stream):
                one_step()

        def run_step():
            if graph is not None:
                graph.replay()
            else:
                one_step()

        for _ in range(args.warmup):
            run_step()
        stream.synchronize()
        if world > 1:
            dist.barrier()
        sampler = ClockSampler(local)
        if rank == 0:
            sampler.start()
        torch.cuda.synchronize()
        ev = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps + 1)]
        ev[0].record(stream)
        for k in range(args.steps):
            run_step()
            ev[k + 1].record(stream)
        stream.synchronize()
        torch.cuda.synchronize()
        clocks = sampler.stop() if rank == 0 else None
        total_ms = ev[0].elapsed_time(ev[-1])
        step_ms = [ev[k].elapsed_time(ev[k + 1]) for k in range(args.steps)]

        # end to end through the host entry point: pinned host activations in, host result out, every layer
        xh = torch.from_numpy(x_bits.view(np.int16)).view(torch.bfloat16).pin_memory()
        yh = torch.empty((T, c["d_out"]), dtype=torch.bfloat16).pin_memory()
        e2e_steps = max(3, min(args.steps, 20))

        def e2e_step():
            for blob in blobs:
                lopro.linear_fwd_host(d, blob, xh, yh, ws, lopro.OUT_BF16)

        for _ in range(3):
            e2e_step()
        stream.synchronize()
        if world > 1:
            dist.barrier()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(e2e_steps):
            e2e_step()
        e1.record(stream)
        stream.synchronize()
        e2e_ms = e0.elapsed_time(e1)
        status = lopro.workspace_status(ws)
        assert status == lopro.OK, f"device status {status}"
        assert torch.isfinite(yh.float()).all()

    if world > 1:
        total_ms, e2e_ms = max_over_ranks([total_ms, e2e_ms], dev)
    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return 0

    peaks = measured_peaks()
    ms_per_step = total_ms / args.steps
    tokens_per_step = T * ring * world
    value = tokens_per_step / (ms_per_step * 1e-3)
    e2e_value = T * ring * world / (e2e_ms / e2e_steps * 1e-3)
    # Dominant kernel: the forward kernel that reads the packed weights, launched once per layer.  Its
    # launch duration is taken as (step time / launches), i.e. the whole per-layer time including any
    # prologue kernels of the path -- an upper bound on the kernel's own duration, a lower bound on
    # `achieved`.
    path, kernels_per_forward = lopro.linear_fwd_path(d, T)
    path_name = lopro.PATH_NAMES.get(path, "?")
    kernel_name = {"stream": "stream_kernel", "wide": "stream_wide_kernel", "tall": "tall_kernel", "general": "decode_kernel",
                   "prefill": "prefill_kernel", "rowblock": "rowblock_kernel"}.get(path_name, "?")
    note = "duration = step time / layer forwards (includes the prologue kernels)"
    launches_per_step = ring
    dur_s = ms_per_step * 1e-3 / launches_per_step
    hbm_bound = T <= 64
    if hbm_bound:
        ach = algorithmic_bytes(c, T) / dur_s / 1e9
        roofline = dict(bound="hbm", achieved=ach, peak=peaks["hbm_gbs"], unit="GB/s", frac=ach / peaks["hbm_gbs"],
                        traffic=NCU_TRAFFIC.get((args.workload, kernel_name)), peak_source=f"of {peaks['source']}",
                        frac_of_nominal_8000=ach / 8000.0, kernel=kernel_name,
                        algorithmic_bytes_per_launch=algorithmic_bytes(c, T), launch_us=dur_s * 1e6, note=note)
    else:
        ach = algorithmic_flops(c, T) / dur_s / 1e12
        pk = peaks["bf16_tflops_sustained"]
        roofline = dict(bound="tensor", achieved=ach, peak=pk, unit="TFLOP/s", frac=ach / pk,
                        traffic=NCU_TRAFFIC.get((args.workload, kernel_name)),
                        peak_source=f"of {peaks['source']} (sustained)", kernel=kernel_name,
                        algorithmic_flops_per_launch=algorithmic_flops(c, T), launch_us=dur_s * 1e6, note=note)
    line = dict(metric=METRIC, value=value, unit=UNIT, n_gpus=world, steps=args.steps, warmup=args.warmup,
                ms_per_step=ms_per_step, higher_is_better=True, scaling="weak", vs_baseline=None, dtype="bf16",
                data="synthetic", config=workload_config(args.workload), clocks=clocks,
                e2e=dict(value=e2e_value, unit=UNIT, h2d_bytes_per_step=ring * T * c["d_in"] * 2,
                         d2h_bytes_per_step=ring * T * c["d_out"] * 2, steps=e2e_steps),
                gpu_launches=kernels_per_forward * ring * args.steps, path=path_name, roofline=roofline,
                step_ms_min=min(step_ms), step_ms_median=statistics.median(step_ms),
                cuda_graph=graph is not None)
    if not args.no_cpu_baseline and world == 1:
        max_rows = 1024 if c["d_out"] * c["d_in"] > (1 << 24) or T > 64 else None
        max_tokens = 16 if T > 64 else None
        r = time_oracle(c, T, 12.0, max_rows, max_tokens)
        line["cpu_baseline"] = dict(
            value=r["value"], unit=UNIT, cores=r["cores"], kind="oracle",
            sample=(f"oracle.forward_exact (fp64 numpy) on {r['rows']} of {c['d_out']} output rows, {r['tokens']} of {T} "
                    f"tokens of one layer, {r['reps']} repetitions, scaled linearly to a full layer forward"))
    if world > 1:
        dist.destroy_process_group()
    print(json.dumps(line))
    return 0


if __name__ == "__main__":
    sys.exit(main())

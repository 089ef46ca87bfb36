#!/usr/bin/env python
"""Benchmark of the LoPRo quantized-linear forward on B200.

Default workload: the decode configuration (4096 x 4096, 4-bit g128, block 128, rank 32, 8 tokens).
One step = one forward of the token batch through every layer of a ring of distinct synthetic
layers; the ring is larger than the L2 cache, so every layer's packed weights come from HBM.
A step repeats that pass until it lasts --step-ms (50 ms), so that a run of 20 steps loads the GPU for a second.
Prints ONE JSON line: the contract's keys for the named workload, `roofline`, `cpu_baseline`, `e2e`, and under
`workloads` one record per other regime (decode at other batch sizes, the large layer, the decoder stack, prefill).

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
    # the same stack as a whole decode step: the linears chained through residual + RMS norm, rotary embedding, attention of
    # the new token over a 2048-token key/value cache per sequence, SiLU gating (plain kernels of this library)
    "cfg5_T1_block": ("cfg5", 1, 224),
    "cfg5_T32_block": ("cfg5", 32, 224),
}
STACK_HEADS, STACK_HEAD_DIM, STACK_CONTEXT = 32, 128, 2048
# linears of one layer of the stack: name, d_in, d_out (hidden 4096, MLP 11008)
STACK_LINEARS = [("q", 4096, 4096), ("k", 4096, 4096), ("v", 4096, 4096), ("o", 4096, 4096),
                 ("gate", 4096, 11008), ("up", 4096, 11008), ("down", 11008, 4096)]
STACK_LAYERS = 32
STACK_QUANT = dict(bits=4, group_size=128, block_size=128, identity_cols=128, rank=32)


def stack_shape(n, m):
    return dict(d_in=n, d_out=m, **STACK_QUANT)


def block_glue_bytes(T):
    """HBM bytes of the decoder-block operations of one decode step: the key/value cache (keys and values of the
    context plus the new token, bf16) dominates; the activation rows between the kernels stay in L2."""
    return STACK_LAYERS * T * STACK_HEADS * (STACK_CONTEXT + 1) * STACK_HEAD_DIM * 2 * 2


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

# DRAM bytes (dram__bytes_read.sum + dram__bytes_write.sum) per launch of the dominant kernel, from ncu captures of
# the kernels as committed (profiles/: the commands; counters re-read after the last change of each kernel, as ncu
# prints them, i.e. to 10 kB); null for workloads without a capture.
NCU_TRAFFIC = {("cfg2_T8", "stream_wide_kernel"): 9290000, ("cfg2_T32", "stream_kernel"): 9490000,
               ("cfg4_T16", "tall_kernel"): 82610000, ("cfg3_T2048", "prefill_pair_kernel"): 60700000}
METRIC = "quantized-linear fwd tokens/s"
UNIT = "tokens/s"


def algorithmic_bytes(c, T, lowrank="f16"):
    """Bytes the method must move per layer forward: codes, (scale, zero) pairs, the low-rank factors (fp16 A and B,
    or fp8 U and V with fp16 Sigma and s), perm, x in, y out."""
    m, n, q, g, r = c["d_out"], c["d_in"], c["bits"], c["group_size"], c["rank"]
    factors = (m * r + r * n) * 2 if lowrank == "f16" else (m * r + r * n) + 2 * r + 2 * n
    return m * n * q // 8 + m * (n // g) * 4 + factors + n * 4 + T * (n + m) * 2


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
    if cfg == "cfg5" and name.endswith("_block"):
        return dict(workload=f"{name}: one decode step of a 32-layer decoder stack (hidden 4096, MLP 11008, 32 heads x 128; the 224 "
                             f"linears LoPRo 4-bit g128 block 128 rank 32), batch {T}, one new token per sequence over a "
                             f"{STACK_CONTEXT}-token bf16 key/value cache; norms, rotary embedding, attention and gating by this "
                             "library's plain kernels; no embedding, final norm or vocabulary projection",
                    tokens=T, ring_layers=ring,
                    l2="inputs larger than L2: one step reads %.0f MB of packed weights and %.0f MB of key/value cache"
                       % (stack_bytes(T) / 1e6, block_glue_bytes(T) / 1e6))
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


def cpu_model():
    try:
        with open("/proc/cpuinfo") as f:
            for line in f:
                if line.lower().startswith("model name"):
                    return line.split(":", 1)[1].strip()
    except OSError:
        pass
    return "unknown"


def cpu_baseline_record(c_or_stack, T, budget_s, stack=False):
    """The oracle as it stands on the host cores: all BLAS threads, and capped to one thread."""
    def run(budget):
        if stack:
            return time_oracle_stack(T, budget)
        max_rows = 1024 if c_or_stack["d_out"] * c_or_stack["d_in"] > (1 << 24) or T > 64 else None
        max_tokens = 16 if T > 64 else None
        return time_oracle(c_or_stack, T, budget, max_rows, max_tokens)
    r = run(budget_s)
    if stack:
        sample = r["sample"]
    else:
        sample = (f"oracle.forward_exact (fp64 numpy) on {r['rows']} of {c_or_stack['d_out']} output rows, {r['tokens']} of {T} "
                  f"tokens of one layer, {r['reps']} repetitions, scaled linearly to a full layer forward")
    rec = dict(value=r["value"], unit=UNIT, cores=r["cores"], kind="oracle", sample=sample, cpu_model=cpu_model(),
               host_cores=os.cpu_count())
    try:
        from threadpoolctl import threadpool_limits
        with threadpool_limits(limits=1):
            r1 = run(max(2.0, budget_s / 3))
        rec["single_thread"] = dict(value=r1["value"], unit=UNIT, cores=1)
    except Exception as e:  # threadpoolctl missing: the all-threads leg stands alone
        rec["single_thread"] = dict(value=None, note=f"not measured: {e}")
    return rec


class Workload:
    """One benchmark workload resident on the device: a pass (every layer forward once), a verification pass that reads
    the status word after every forward, and the end-to-end pass with host buffers."""

    def __init__(self, args, name, rank, dev):
        import torch
        from paper_2601_19675_b200 import lopro, synth
        self.torch, self.lopro, self.name, self.dev, self.args = torch, lopro, name, dev, args
        cfg, T, ring = WORKLOADS[name]
        self.cfg, self.T, self.ring = cfg, T, ring
        layout = lopro.LAYOUT_ROWBLOCK if args.layout == "rowblock" else lopro.LAYOUT_FRAGMENT

        def dev16(a):
            return torch.from_numpy(np.ascontiguousarray(a).view(np.int16)).to(dev)

        if cfg == "cfg5":
            q = STACK_QUANT
            shapes = sorted({(n, m) for _, n, m in STACK_LINEARS})
            base, descs = {}, {}
            for n, m in shapes:
                layer = synth.random_layer(n, m, q["bits"], q["group_size"], q["rank"], seed=rank + n // 64)
                base[(n, m)] = dict(codes=torch.from_numpy(layer["codes"]).to(dev), sc=dev16(layer["scales"]),
                                    zr=dev16(layer["zeros"]), pm=torch.from_numpy(layer["perm"]).to(dev), A=dev16(layer["A"]),
                                    B=dev16(layer["B"]))
                descs[(n, m)] = lopro.make_desc(n, m, q["bits"], q["group_size"], q["block_size"], q["identity_cols"], q["rank"],
                                                layout=layout)
            self.x_bits = {n: synth.activations(T, n, seed=rank + n) for n in sorted({n for n, _ in shapes})}
            xs = {n: dev16(b).view(torch.bfloat16) for n, b in self.x_bits.items()}
            linears = []
            for li in range(STACK_LAYERS):
                for j, (_, n, m) in enumerate(STACK_LINEARS):
                    b = base[(n, m)]
                    i = li * len(STACK_LINEARS) + j
                    codes = torch.roll(b["codes"], shifts=(i, 3 * i), dims=(0, 1)) if i else b["codes"]
                    blob = lopro.pack(descs[(n, m)], codes, b["sc"], b["zr"], b["pm"], b["A"], b["B"])
                    linears.append((descs[(n, m)], blob, xs[n], torch.empty((T, m), dtype=torch.bfloat16, device=dev)))
            del codes
            for b in base.values():
                del b["codes"]
            # sibling linears of a layer read the same activations: (q, k, v) and (gate, up) go through the grouped call
            split = ((0,), (1,), (2,), (3,), (4,), (5,), (6,)) if args.no_groups else ((0, 1, 2), (3,), (4, 5), (6,))
            self.calls = []   # (descs, blobs, x, ys)
            for li in range(STACK_LAYERS):
                L7 = linears[li * 7:(li + 1) * 7]
                for idx in split:
                    part = [L7[k] for k in idx]
                    self.calls.append(([g[0] for g in part], [g[1] for g in part], part[0][2], [g[3] for g in part]))
            self.x_dev, self.x_host_bits, self.y_last = xs[4096], self.x_bits[4096], self.calls[-1][3][-1]
            self.block = name.endswith("_block")
            self.ws_holder = [None]
            if self.block:
                self.build_block(linears, rank)
            self.forwards = len(linears)
            self.tokens_per_pass = T
            self.bytes_per_pass = stack_bytes(T)
            self.flops_per_pass = None
            self.h2d, self.d2h = T * 4096 * 2, T * self.y_last.shape[1] * 2
            ws_bytes = max(lopro.group_workspace_bytes(c[0], T) for c in self.calls)
            self.ws = torch.zeros(ws_bytes, dtype=torch.uint8, device=dev)
            self.ws_holder[0] = self.ws
            self.paths = sorted({lopro.PATH_NAMES.get(lopro.linear_fwd_path(d, T)[0], "?") for d, _, _, _ in linears})
            self.launches_per_pass = sum(lopro.linear_fwd_group_path(c[0], T)[1] if len(c[0]) > 1
                                         else lopro.linear_fwd_path(c[0][0], T)[1] for c in self.calls)
            if self.block:
                self.bytes_per_pass += block_glue_bytes(T)
                self.launches_per_pass += 6 * STACK_LAYERS      # 2 norms, rotary + append, attention (2), gating
            self.c = None
            return
        c = synth.CONFIGS[cfg]
        self.c = c
        fp8 = args.lowrank == "fp8"
        d = lopro.make_desc(c["d_in"], c["d_out"], c["bits"], c["group_size"], c["block_size"], c["identity_cols"], c["rank"],
                            layout=layout, lowrank_format=lopro.LOWRANK_FP8 if fp8 else lopro.LOWRANK_FOLDED_F16)
        # ring of distinct layers: layer 0 drawn by the seeded generator, the others re-use its small tensors with the
        # code matrix rolled per layer (set-up time only; every blob is a separate allocation)
        base = synth.random_layer(c["d_in"], c["d_out"], c["bits"], c["group_size"], c["rank"], seed=rank)
        sc, zr, pm, A, B = dev16(base["scales"]), dev16(base["zeros"]), torch.from_numpy(base["perm"]).to(dev), \
            dev16(base["A"]), dev16(base["B"])
        codes0 = torch.from_numpy(base["codes"]).to(dev)
        blobs = []
        for i in range(ring):
            if name.endswith("_L2") and i:
                blobs.append(blobs[0])  # the same packed layer again: L2-resident measurement
                continue
            codes = torch.roll(codes0, shifts=(i, 3 * i), dims=(0, 1)) if i else codes0
            if fp8:
                if i == 0:
                    rec = synth.lowrank_record(c["d_out"], c["d_in"], c["rank"], seed=rank)
                    U8, V8 = torch.from_numpy(rec["U"]).to(dev), torch.from_numpy(rec["V"]).to(dev)
                    sg, sv = dev16(rec["sigma"]), dev16(rec["s"])
                blobs.append(lopro.pack_lr8(d, codes, sc, zr, pm, U8, V8, sg, sv))
            else:
                blobs.append(lopro.pack(d, codes, sc, zr, pm, A, B))
        del codes0, codes
        self.x_host_bits = synth.activations(T, c["d_in"], seed=rank, outlier_frac=c.get("outlier_frac", 0.0),
                                             outlier_scale=c.get("outlier_scale", 20.0))
        x = dev16(self.x_host_bits).view(torch.bfloat16)
        ys = [torch.empty((T, c["d_out"]), dtype=torch.bfloat16, device=dev) for _ in range(min(ring, 4))]
        self.ws = torch.zeros(lopro.workspace_bytes(d, T) + lopro.host_staging_bytes(d, T), dtype=torch.uint8, device=dev)
        self.calls = [([d], [blob], x, [ys[i % len(ys)]]) for i, blob in enumerate(blobs)]
        self.d = d
        self.forwards = ring
        self.tokens_per_pass = T * ring
        self.bytes_per_pass = ring * algorithmic_bytes(c, T, "fp8" if fp8 else "f16")
        self.flops_per_pass = ring * algorithmic_flops(c, T)
        self.h2d, self.d2h = ring * T * c["d_in"] * 2, ring * T * c["d_out"] * 2
        path, per_forward = lopro.linear_fwd_path(d, T)
        self.paths = [lopro.PATH_NAMES.get(path, "?")]
        self.launches_per_pass = per_forward * ring

    def build_block(self, linears, rank):
        """Buffers and call list of a whole decode step: per layer norm -> (q, k, v) -> rotary + cache append -> attention
        -> o -> residual + norm -> (gate, up) -> gating -> down; the residual of `down` is added by the next layer's norm."""
        torch, lopro, dev, T = self.torch, self.lopro, self.dev, self.T
        from paper_2601_19675_b200 import synth
        H, hd, C = STACK_HEADS, STACK_HEAD_DIM, STACK_CONTEXT + 1
        bf = torch.bfloat16
        buf = lambda d: torch.empty((T, d), dtype=bf, device=dev)
        self.h0, self.h, self.xn = self.x_dev, buf(4096), buf(4096)
        q, k, v, attn, o = buf(4096), buf(4096), buf(4096), buf(4096), buf(4096)
        gate, up, act, down = buf(11008), buf(11008), buf(11008), buf(4096)
        gen = torch.Generator(device=dev)
        gen.manual_seed(1234 + rank)
        caches = []
        for _ in range(STACK_LAYERS):           # random keys and values of the 2048-token context, one cache per layer
            kc = torch.empty((T, H, C, hd), dtype=bf, device=dev).normal_(generator=gen)
            vc = torch.empty((T, H, C, hd), dtype=bf, device=dev).normal_(generator=gen)
            caches.append((kc, vc))
        norm_w = torch.from_numpy(synth.f32_to_bf16_bits(
            1.0 + 0.1 * synth.weights(2 * STACK_LAYERS, 4096, seed=77 + rank, std=1.0)).view(np.int16)).to(dev).view(bf)
        pos = torch.full((T,), STACK_CONTEXT, dtype=torch.int32, device=dev)
        ctx = torch.full((T,), C, dtype=torch.int32, device=dev)
        self.block_status = torch.zeros(1, dtype=torch.int32, device=dev)
        attn_ws = torch.empty(lopro.block_attention_workspace_bytes(T, H, hd, C), dtype=torch.uint8, device=dev)
        scale = 1.0 / float(np.sqrt(hd))
        ws, st = self.ws_holder, self.block_status
        steps = [lambda: self.h.copy_(self.h0)]
        for li in range(STACK_LAYERS):
            L7 = linears[li * 7:(li + 1) * 7]
            ds, bl = [g[0] for g in L7], [g[1] for g in L7]
            kc, vc = caches[li]
            w1, w2 = norm_w[2 * li], norm_w[2 * li + 1]
            prev = down if li else None
            steps += [
                lambda prev=prev, w1=w1: lopro.block_add_rmsnorm(self.h, prev, w1, 1e-5, out=self.xn),
                lambda ds=ds, bl=bl: lopro.linear_fwd_group(ds[0:3], bl[0:3], self.xn, lopro.OUT_BF16, workspace=ws[0], ys=[q, k, v]),
                lambda kc=kc, vc=vc: lopro.block_rope_append(q, k, v, pos, kc, vc, 10000.0, st),
                lambda kc=kc, vc=vc: lopro.block_attention_decode(q, kc, vc, ctx, scale, attn_ws, st, out=attn),
                lambda ds=ds, bl=bl: lopro.linear_fwd(ds[3], bl[3], attn, lopro.OUT_BF16, workspace=ws[0], y=o),
                lambda w2=w2: lopro.block_add_rmsnorm(self.h, o, w2, 1e-5, out=self.xn),
                lambda ds=ds, bl=bl: lopro.linear_fwd_group(ds[4:6], bl[4:6], self.xn, lopro.OUT_BF16, workspace=ws[0], ys=[gate, up]),
                lambda: lopro.block_silu_mul(gate, up, out=act),
                lambda ds=ds, bl=bl: lopro.linear_fwd(ds[6], bl[6], act, lopro.OUT_BF16, workspace=ws[0], y=down),
            ]
        self.block_steps = steps
        self.y_last = down

    def one_pass(self):
        lopro = self.lopro
        if getattr(self, "block", False):
            for f in self.block_steps:
                f()
            return
        for ds, blobs, x, ys in self.calls:
            if len(ds) == 1:
                lopro.linear_fwd(ds[0], blobs[0], x, lopro.OUT_BF16, workspace=self.ws, y=ys[0])
            else:
                lopro.linear_fwd_group(ds, blobs, x, lopro.OUT_BF16, workspace=self.ws, ys=ys)

    def verify_pass(self):
        """Untimed: every forward of the pass on its own, the device status word read after each of them (a forward
        resets the word when it starts, so reading it once at the end would report the last forward only)."""
        lopro, torch = self.lopro, self.torch
        if getattr(self, "block", False):
            for k, f in enumerate(self.block_steps):
                f()
                torch.cuda.current_stream().synchronize()
                status = lopro.workspace_status(self.ws)
                assert status == lopro.OK, f"device status {status} after step {k} of {self.name}"
                assert int(self.block_status.item()) == lopro.OK, f"block status after step {k} of {self.name}"
            assert torch.isfinite(self.y_last.float()).all() and torch.isfinite(self.h.float()).all()
            return
        for k, (ds, blobs, x, ys) in enumerate(self.calls):
            if len(ds) == 1:
                lopro.linear_fwd(ds[0], blobs[0], x, lopro.OUT_BF16, workspace=self.ws, y=ys[0])
            else:
                lopro.linear_fwd_group(ds, blobs, x, lopro.OUT_BF16, workspace=self.ws, ys=ys)
            torch.cuda.current_stream().synchronize()
            status = lopro.workspace_status(self.ws)
            assert status == lopro.OK, f"device status {status} after call {k} of {self.name}"
            assert torch.isfinite(ys[-1].float()).all(), f"non-finite output after call {k} of {self.name}"

    def e2e_setup(self):
        torch = self.torch
        self.xh = torch.from_numpy(self.x_host_bits.view(np.int16)).view(torch.bfloat16).pin_memory()
        if self.cfg == "cfg5":
            self.yh = torch.empty(tuple(self.y_last.shape), dtype=torch.bfloat16).pin_memory()
        else:
            self.yh = torch.empty((self.T, self.c["d_out"]), dtype=torch.bfloat16).pin_memory()

    def e2e_pass(self, run_graph):
        """The same work with host buffers: activations from pinned host memory, results back to the host."""
        lopro = self.lopro
        if self.cfg == "cfg5":
            self.x_dev.copy_(self.xh, non_blocking=True)
            run_graph()
            self.yh.copy_(self.y_last, non_blocking=True)
        else:
            for ds, blobs, _, _ in self.calls:
                lopro.linear_fwd_host(ds[0], blobs[0], self.xh, self.yh, self.ws, lopro.OUT_BF16)


def measure(args, name, steps, warmup, rank, world, local, dev, dist, with_e2e=True):
    """Builds the workload, times `steps` steps (each a whole number of passes lasting at least args.step_ms) and
    returns the bench record."""
    import torch
    from paper_2601_19675_b200 import lopro
    w = Workload(args, name, rank, dev)
    # the stack alternates single-layer and grouped forwards: one set of kernel variants for both (see the switch's
    # description in lopro.h); every other workload launches single layers only and keeps the default
    lopro.configure(lopro.OPT_ONE_KERNEL_SET, 1 if w.cfg == "cfg5" else 0)
    stream = torch.cuda.Stream(device=dev)
    with torch.cuda.stream(stream):
        w.verify_pass()
        graph = None
        if not args.no_graph:
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph, stream=stream):
                w.one_pass()
        run_pass = graph.replay if graph is not None else w.one_pass
        # passes per step: as many as it takes for a step to last args.step_ms
        for _ in range(3):
            run_pass()
        stream.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(3):
            run_pass()
        e1.record(stream)
        stream.synchronize()
        pass_ms = e0.elapsed_time(e1) / 3
        passes = max(1, int(np.ceil(args.step_ms / max(pass_ms, 1e-6))))
        if world > 1:
            passes = int(max_over_ranks([passes], dev)[0])

        def run_step():
            for _ in range(passes):
                run_pass()

        for _ in range(warmup):
            run_step()
        stream.synchronize()
        if world > 1:
            dist.barrier()
        sampler = ClockSampler(local)
        if rank == 0:
            sampler.start()
        torch.cuda.synchronize()
        ev = [torch.cuda.Event(enable_timing=True) for _ in range(steps + 1)]
        ev[0].record(stream)
        for k in range(steps):
            run_step()
            ev[k + 1].record(stream)
        stream.synchronize()
        torch.cuda.synchronize()
        clocks = sampler.stop() if rank == 0 else None
        total_ms = ev[0].elapsed_time(ev[-1])
        step_ms = [ev[k].elapsed_time(ev[k + 1]) for k in range(steps)]
        e2e_ms, e2e_steps = None, 0
        if with_e2e:
            w.e2e_setup()
            e2e_steps = 5
            for _ in range(2):
                w.e2e_pass(run_pass)
            stream.synchronize()
            if world > 1:
                dist.barrier()
            e0.record(stream)
            for _ in range(e2e_steps):
                w.e2e_pass(run_pass)
            e1.record(stream)
            stream.synchronize()
            e2e_ms = e0.elapsed_time(e1)
            assert torch.isfinite(w.yh.float()).all()
        w.verify_pass()
    if world > 1:
        total_ms, e2e_ms = max_over_ranks([total_ms, e2e_ms if e2e_ms is not None else 0.0], dev)
    peaks = measured_peaks()
    ms_per_step = total_ms / steps
    ms_per_pass = ms_per_step / passes
    value = w.tokens_per_pass * passes * world / (ms_per_step * 1e-3)
    per_forward_s = ms_per_pass * 1e-3 / w.forwards
    kernel = " + ".join({"stream": "stream_kernel", "wide": "stream_wide_kernel", "tall": "tall_kernel", "general": "decode_kernel",
                         "prefill": "prefill_pair_kernel" if w.T >= 512 else "prefill_kernel",
                         "rowblock": "rowblock_kernel"}.get(n, n) for n in w.paths)
    note = ("duration = step time / layer forwards (includes the prologue kernels of each forward): an upper bound on the "
            "product kernel's own duration, a lower bound on `achieved`")
    if getattr(w, "block", False):
        kernel += " + attention_split_kernel"
        note = ("whole decode step: bytes = packed weights + key/value cache, duration = step time / 224 linears (every kernel of "
                "the step included)")
    if w.T <= 64:
        ach = w.bytes_per_pass / (ms_per_pass * 1e-3) / 1e9
        roofline = dict(bound="hbm", achieved=ach, peak=peaks["hbm_gbs"], unit="GB/s", frac=ach / peaks["hbm_gbs"],
                        traffic=NCU_TRAFFIC.get((name, kernel)), peak_source=f"of {peaks['source']}",
                        frac_of_nominal_8000=ach / 8000.0, kernel=kernel, algorithmic_bytes_per_launch=w.bytes_per_pass // w.forwards,
                        launch_us=per_forward_s * 1e6, note=note)
    else:
        ach = w.flops_per_pass / (ms_per_pass * 1e-3) / 1e12
        pk = peaks["bf16_tflops_sustained"]
        roofline = dict(bound="tensor", achieved=ach, peak=pk, unit="TFLOP/s", frac=ach / pk, traffic=NCU_TRAFFIC.get((name, kernel)),
                        peak_source=f"of {peaks['source']} (sustained, the kernel runs inside a long step)",
                        frac_of_burst_peak=ach / peaks["bf16_tflops"], burst_peak=peaks["bf16_tflops"], kernel=kernel,
                        algorithmic_flops_per_launch=w.flops_per_pass // w.forwards, launch_us=per_forward_s * 1e6, note=note)
    rec = dict(metric=METRIC, value=value, unit=UNIT, n_gpus=world, steps=steps, warmup=warmup, ms_per_step=ms_per_step,
               higher_is_better=True, scaling="weak", vs_baseline=None, dtype="bf16", data="synthetic",
               config=dict(workload_config(name), passes_per_step=passes, layout=args.layout, lowrank=args.lowrank), clocks=clocks,
               gpu_launches=w.launches_per_pass * passes * steps, path="+".join(w.paths), roofline=roofline,
               ms_per_forward=per_forward_s * 1e3, ms_per_pass=ms_per_pass, step_ms_min=min(step_ms),
               step_ms_median=statistics.median(step_ms), cuda_graph=graph is not None,
               status_checked="after every forward of an untimed pass before and after the timed region")
    if e2e_ms is not None:
        rec["e2e"] = dict(value=w.tokens_per_pass * world / (e2e_ms / e2e_steps * 1e-3), unit=UNIT, h2d_bytes_per_step=w.h2d,
                          d2h_bytes_per_step=w.d2h, steps=e2e_steps,
                          note="one pass per step through the host-buffer entry point (pinned host x in, host y out)")
    rec["_workload"] = w
    if w.cfg == "cfg5":
        rec["config"]["one_kernel_set"] = 1
        lopro.configure(lopro.OPT_ONE_KERNEL_SET, 0)
    return rec


# workloads reported beside the bench line (driver-run evidence for every regime), with the steps each gets
EXTRA_WORKLOADS = [("cfg2_T1", 5), ("cfg2_T32", 5), ("cfg4_T16", 5), ("cfg5_T1", 5), ("cfg5_T32", 5), ("cfg3_T2048", 5),
                   ("cfg4_T4096", 4), ("cfg5_T1_block", 5), ("cfg5_T32_block", 4)]


def measure_offline(dev, peaks, reps=3):
    """The offline side (quantization of one layer on the GPU: rank-1 sketch with deflation at the paper's defaults,
    rank 16 and 8 iterations; residual, rotation, group grid) on the two matrix shapes of the 7B decoder stack.  Every
    step is a memory-bound pass over the fp32 matrix; bytes = 4 m n (2 [scaling] + r (2 it + 4) [products, update]
    + 1 [residual]) + m n [codes]."""
    import torch
    from paper_2601_19675_b200 import lopro, synth
    out = {}
    r, it = 16, 8
    per_shape = {}
    for (n, m) in ((4096, 4096), (4096, 11008)):
        d = lopro.make_desc(n, m, 4, 128, 128, 128, r, lopro.LAYOUT_FRAGMENT)
        w = torch.from_numpy(synth.weights(m, n, seed=1, spikes=24)).to(dev)
        perm = torch.from_numpy(synth.permutation(n, seed=2)).to(dev)
        sk = torch.from_numpy(synth.sketches(r, n, seed=3).astype("float32")).to(dev)
        ws = torch.empty(lopro.quantize_workspace_bytes(d), dtype=torch.uint8, device=dev)
        res = lopro.quantize_layer(d, w, perm, sk, it=it, workspace=ws)          # warm-up, checked
        torch.cuda.synchronize()
        if lopro.workspace_status(ws) != lopro.OK:
            raise RuntimeError("quantize_layer reported an error in its status word")
        times = []
        for _ in range(reps):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            lopro.quantize_layer(d, w, perm, sk, it=it, workspace=ws)
            e1.record()
            torch.cuda.synchronize()
            times.append(e0.elapsed_time(e1))
        ms = statistics.median(times)
        nbytes = 4 * m * n * (2 + r * (2 * it + 4) + 1) + m * n
        launches = 1 + r * (1 + it * 3 + 2 + 2) + 2
        per_shape[(n, m)] = ms
        out[f"quantize_{n}x{m}_r{r}_it{it}"] = dict(
            ms_per_layer=ms, algorithmic_bytes=nbytes, achieved_gbs=nbytes / (ms * 1e-3) / 1e9,
            frac_of_measured_hbm=nbytes / (ms * 1e-3) / 1e9 / peaks["hbm_gbs"], gpu_launches=launches,
            note=("the fp32 matrix (%d MB) fits the 126 MB L2: repeated passes are served from it, the fraction may exceed 1"
                  % (m * n * 4 >> 20)) if m * n * 4 < 120 << 20 else "the fp32 matrix is larger than L2: every pass streams from HBM")
        del w, ws, res
        torch.cuda.empty_cache()
    total_s = 32 * (4 * per_shape[(4096, 4096)] + 3 * per_shape[(4096, 11008)]) * 1e-3
    out["decoder_7b_estimate_s"] = dict(value=total_s, note="32 blocks x (4 x 4096^2 + 3 x 4096*11008 matrices), from the two "
                                        "timings above (the 11008 -> 4096 projection counted as its transpose's time)")
    return out


def measure_experts(dev, peaks, reps=20):
    """The experts of a mixture layer at decode: 8 experts 4096 -> 14336 (2-bit g64, block 256, rank 16), 16 tokens routed
    to 2 experts each = 32 rows, 4 per expert; a ring of 3 distinct expert sets (each larger than L2); the grouped call
    against one call per expert."""
    import torch
    from paper_2601_19675_b200 import lopro, synth
    n, m, E, sets, per = 4096, 14336, 8, 3, 4
    d = lopro.make_desc(n, m, 2, 64, 256, 256, 16, lopro.LAYOUT_FRAGMENT)
    base = synth.random_layer(n, m, 2, 64, 16, seed=5)

    def dev16(a):
        return torch.from_numpy(np.ascontiguousarray(a).view(np.int16)).to(dev)

    codes0 = torch.from_numpy(base["codes"]).to(dev)
    sc, zr, pm, A, B = dev16(base["scales"]), dev16(base["zeros"]), torch.from_numpy(base["perm"]).to(dev), dev16(base["A"]), dev16(base["B"])
    blobs = [[lopro.pack(d, torch.roll(codes0, shifts=(7 * (s * E + e), 3 * (s * E + e)), dims=(0, 1)), sc, zr, pm, A, B)
              for e in range(E)] for s in range(sets)]
    del codes0
    offs = [per * e for e in range(E + 1)]
    x = dev16(synth.activations(per * E, n, seed=6)).view(torch.bfloat16)
    y = torch.empty((per * E, m), dtype=torch.bfloat16, device=dev)
    ws = torch.zeros(lopro.experts_workspace_bytes(d, E, per), dtype=torch.uint8, device=dev)
    c = dict(d_out=m, d_in=n, bits=2, group_size=64, rank=16)
    nbytes = E * algorithmic_bytes(c, per)

    def grouped():
        for s in range(sets):
            lopro.linear_fwd_experts(d, blobs[s], offs, x, lopro.OUT_BF16, workspace=ws, y=y)

    def one_by_one():
        for s in range(sets):
            for e in range(E):
                lopro.linear_fwd(d, blobs[s][e], x[offs[e]:offs[e + 1]], lopro.OUT_BF16, workspace=ws, y=y[offs[e]:offs[e + 1]])

    out = {}
    for name, fn in (("grouped", grouped), ("one_call_per_expert", one_by_one)):
        stream = torch.cuda.Stream(device=dev)
        with torch.cuda.stream(stream):
            fn()
            stream.synchronize()
            assert lopro.workspace_status(ws) == lopro.OK
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph, stream=stream):
                fn()
            for _ in range(3):
                graph.replay()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(stream)
            for _ in range(reps):
                graph.replay()
            e1.record(stream)
            stream.synchronize()
        us = e0.elapsed_time(e1) * 1e3 / (reps * sets)
        out[name] = dict(us_per_layer=us, achieved_gbs=nbytes / (us * 1e-6) / 1e9,
                         frac_of_measured_hbm=nbytes / (us * 1e-6) / 1e9 / peaks["hbm_gbs"],
                         launches_per_layer=lopro.linear_fwd_experts_path(d, offs)[1] if name == "grouped" else 2 * E)
    out["workload"] = ("8 experts 4096 -> 14336, 2-bit g64 block 256 rank 16, 4 rows per expert (16 tokens, 2 experts each); "
                       "%d bytes per layer forward; ring of %d expert sets" % (nbytes, sets))
    return out


def measure_vq(dev, peaks, reps=20):
    """The vector-quantized variant at decode: 8192 -> 28672 (the shape of configuration 4), 4-D centroids with 8-bit indices
    (2 bits per weight), codebooks of 512 x 256, block 256, rank 16; a ring of 3 distinct records (198 MB), 1 and 16 tokens."""
    import torch
    from paper_2601_19675_b200 import lopro, synth
    n, m, cr, cc, b, r, ring = 8192, 28672, 512, 256, 256, 16, 3
    out = {}
    for dim in (4, 2):
        _measure_vq_dim(dev, peaks, reps, out, n, m, cr, cc, b, r, ring, dim)
    out["workload"] = ("vector-quantized record 8192 -> 28672: 8-bit indices of 4-D centroids (T1, T16) or 6-bit indices of 2-D "
                       "centroids (dim2_T1, dim2_T16), codebooks of 512 x 256, block 256, rank 16")
    return out


def _measure_vq_dim(dev, peaks, reps, out, n, m, cr, cc, b, r, ring, dim):
    import torch
    from paper_2601_19675_b200 import lopro, synth
    k = 256 if dim == 4 else 64
    d = lopro.make_vq_desc(n, m, cr, cc, b, rank=r, dim=dim)
    gen = torch.Generator(device=dev)
    gen.manual_seed(4321)
    a_bits, b_bits = synth.factors(m, n, r, seed=9)

    def dev16(a):
        return torch.from_numpy(np.ascontiguousarray(a).view(np.int16)).to(dev)

    perm = torch.from_numpy(synth.permutation(n, seed=9)).to(dev)
    blobs = []
    for _ in range(ring):
        idx = torch.randint(0, k, (m, n // dim), dtype=torch.uint8, device=dev, generator=gen)
        books = (torch.randn((m // cr, n // cc, k, dim), device=dev, generator=gen) * 0.02).to(torch.bfloat16).view(torch.int16)
        blobs.append(lopro.vq_pack(d, idx, books, perm, dev16(a_bits), dev16(b_bits)))
    del idx, books
    for T in (1, 16):
        x = dev16(synth.activations(T, n, seed=10)).view(torch.bfloat16)
        y = torch.empty((T, m), dtype=torch.bfloat16, device=dev)
        ws = torch.zeros(lopro.vq_workspace_bytes(d, T), dtype=torch.uint8, device=dev)
        idx_bytes = m * (n // 4) if dim == 4 else m * (n // 8 * 3)
        nbytes = idx_bytes + (m // cr) * (n // cc) * k * dim * 2 + (m * r + r * n) * 2 + n * 4 + T * (n + m) * 2
        stream = torch.cuda.Stream(device=dev)
        with torch.cuda.stream(stream):
            for blob in blobs:
                lopro.vq_linear_fwd(d, blob, x, lopro.OUT_BF16, workspace=ws, y=y)
            stream.synchronize()
            assert lopro.workspace_status(ws) == lopro.OK and bool(torch.isfinite(y.float()).all())
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph, stream=stream):
                for blob in blobs:
                    lopro.vq_linear_fwd(d, blob, x, lopro.OUT_BF16, workspace=ws, y=y)
            for _ in range(3):
                graph.replay()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(stream)
            for _ in range(reps):
                graph.replay()
            e1.record(stream)
            stream.synchronize()
        us = e0.elapsed_time(e1) * 1e3 / (reps * ring)
        out[f"T{T}" if dim == 4 else f"dim2_T{T}"] = dict(us_per_layer=us, tokens_per_s=T / (us * 1e-6), algorithmic_bytes=nbytes,
                            achieved_gbs=nbytes / (us * 1e-6) / 1e9, frac_of_measured_hbm=nbytes / (us * 1e-6) / 1e9 / peaks["hbm_gbs"],
                            gpu_launches_per_layer=3)


def measure_rotate(dev, peaks, reps=5):
    """The activation-side transform alone (permutation gather + partial block rotation, lopro_rotate) on prefill batches:
    read x once, write the rotated rows once.  Distinct inputs per launch (more than L2 in total)."""
    import torch
    from paper_2601_19675_b200 import lopro, synth
    out = {}
    for (n, T, b) in ((4096, 2048, 128), (8192, 4096, 256)):
        d = lopro.make_desc(n, 256, 4, 128, b, b, 0, lopro.LAYOUT_FRAGMENT)
        perm = torch.from_numpy(synth.permutation(n, seed=1)).to(dev)
        k = max(8, int(300e6 / (T * n * 2)))
        gen = torch.Generator(device=dev)
        gen.manual_seed(99)
        xs = [torch.randn((T, n), device=dev, generator=gen).to(torch.bfloat16) for _ in range(k)]
        outs = [torch.empty((T, n), dtype=torch.bfloat16, device=dev) for _ in range(min(k, 8))]
        stream = torch.cuda.Stream(device=dev)
        with torch.cuda.stream(stream):
            for i, x in enumerate(xs):
                lopro.rotate(d, perm, x, out=outs[i % len(outs)])
            stream.synchronize()
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph, stream=stream):
                for i, x in enumerate(xs):
                    lopro.rotate(d, perm, x, out=outs[i % len(outs)])
            graph.replay()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(stream)
            for _ in range(reps):
                graph.replay()
            e1.record(stream)
            stream.synchronize()
        us = e0.elapsed_time(e1) * 1e3 / (reps * k)
        nbytes = 2 * T * n * 2 + n * 4
        out[f"rotate_{T}x{n}_b{b}"] = dict(us=us, algorithmic_bytes=nbytes, achieved_gbs=nbytes / (us * 1e-6) / 1e9,
                                           frac_of_measured_hbm=nbytes / (us * 1e-6) / 1e9 / peaks["hbm_gbs"])
        del xs, outs
        torch.cuda.empty_cache()
    return out


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--workload", default="cfg2_T8", choices=sorted(WORKLOADS))
    ap.add_argument("--impl", default="lopro", choices=["lopro", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-graph", action="store_true", help="launch through the stream instead of a CUDA graph")
    ap.add_argument("--no-groups", action="store_true", help="stack workloads: every linear on its own (no grouped siblings)")
    ap.add_argument("--no-extras", action="store_true", help="only the named workload, not the table of the other regimes")
    ap.add_argument("--step-ms", type=float, default=50.0, help="a step repeats the pass until it lasts this long")
    ap.add_argument("--layout", default="fragment", choices=["fragment", "rowblock"], help="code layout of the packed layers")
    ap.add_argument("--lowrank", default="f16", choices=["f16", "fp8"],
                    help="storage of the rank-r term of single-layer workloads: folded fp16 A, B or the fp8 record U, V, Sigma, s")
    ap.add_argument("--offline", action="store_true",
                    help="only the offline side (quantization of a layer on the GPU) and the mixture-layer experts, as one JSON line of their own")
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
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    if rank == 0:
        build.build()
    if world > 1:
        dist.barrier()
    lopro.lib()
    dev = torch.device("cuda", local)

    if args.offline:
        if rank == 0:
            print(json.dumps(dict(offline=measure_offline(dev, measured_peaks()), experts=measure_experts(dev, measured_peaks()), vq=measure_vq(dev, measured_peaks()), rotate=measure_rotate(dev, measured_peaks()),
                                  n_gpus=1, data="synthetic", dtype="f32")))
        if world > 1:
            dist.destroy_process_group()
        return 0
    line = measure(args, args.workload, args.steps, args.warmup, rank, world, local, dev, dist)
    w = line.pop("_workload")
    if rank == 0 and not args.no_cpu_baseline and world == 1:
        line["cpu_baseline"] = cpu_baseline_record(w.c, w.T, 10.0, stack=w.cfg == "cfg5")
    del w
    torch.cuda.empty_cache()
    # the other regimes, each measured the same way with fewer steps (1 GPU only: replicas would repeat them)
    if world == 1 and not args.no_extras:
        table = {}
        for name, st in EXTRA_WORKLOADS:
            if name == args.workload:
                continue
            r = measure(args, name, st, 3, rank, world, local, dev, dist, with_e2e=False)
            r.pop("_workload")
            torch.cuda.empty_cache()
            table[name] = dict(value=r["value"], unit=UNIT, ms_per_forward=r["ms_per_forward"], ms_per_step=r["ms_per_step"],
                               steps=st, path=r["path"], gpu_launches=r["gpu_launches"],
                               roofline={k: r["roofline"][k] for k in ("bound", "achieved", "peak", "unit", "frac", "kernel")
                                         } | ({"frac_of_burst_peak": r["roofline"]["frac_of_burst_peak"]}
                                              if "frac_of_burst_peak" in r["roofline"] else
                                              {"frac_of_nominal_8000": r["roofline"]["frac_of_nominal_8000"]}),
                               clocks=r["clocks"], workload=r["config"]["workload"])
        line["workloads"] = table
        if rank == 0:
            line["offline"] = measure_offline(dev, measured_peaks())
            line["experts"] = measure_experts(dev, measured_peaks())
            line["vq"] = measure_vq(dev, measured_peaks())
            line["rotate"] = measure_rotate(dev, measured_peaks())
    if rank == 0:
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()
    return 0


if __name__ == "__main__":
    sys.exit(main())

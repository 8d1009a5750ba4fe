#!/usr/bin/env python
"""Benchmark of the ATOMO encode + decode hot path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload c5|c3|c2|c1a|c1b|c4] [--budget S]
                    [--impl ours|reference] [--reps R] [--no-extras] [--no-cpu-baseline]

A step is one pass of the whole path (one batched encode, then the decode) over one batch of synthetic
gradients.  The default workload is the largest single-GPU configuration: config 5, 96 gradient matrices of
1024 x 4096 (402,653,184 elements), spectral ATOMO with budget s = 4.  The other configurations are reported
as `also` entries of the same JSON line (rank 0 prints ONE line).
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import tempfile
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "gradient elements encoded+decoded/sec"
UNIT = "elements/s"
L2_BYTES = 126 * 1024 * 1024
# dram__bytes_read.sum + dram__bytes_write.sum of one launch of the dominant kernel, from the ncu captures
# summarised under profiles/ (None: no capture on file for that kernel and workload)
NCU_TRAFFIC = {("sp_tridiag_cluster_kernel", "c2"): 5638912,
               # profiles/sp_tridiag_big1_c5.txt: 1.706 TB/s of DRAM traffic over the 29.52 ms of the captured launch
               ("sp_tridiag_big_kernel", "c5"): 50_400_000_000,
               # profiles/entrywise_c4.txt: the encode kernel (2.09 TB/s over 51.9 us) plus the decode kernel (3.74 TB/s over
               # 24.4 us) of one step at s = 1 %
               ("entrywise", "c4"): 200_000_000}


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        d = json.load(open(path))
        return {"hbm_gbs": float(d["hbm_gbs"]), "bf16_tflops": float(d["bf16_tflops"]), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "source": "fallback"}


# ---------------------------------------------------------------------------------------------
class ClockSampler:
    """nvidia-smi samples of SM clock and throttle reasons while the timed region runs."""
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu = gpu_index
        self.f = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        self.p = None
        self.offset = 0

    def start(self):
        try:
            self.p = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                       "-lms", "20", "-i", str(self.gpu)], stdout=self.f, stderr=subprocess.DEVNULL)
        except Exception:
            self.p = None

    def mark(self):
        """Call when the timed region starts: only samples written after this point are reported."""
        try:
            self.f.flush()
            self.offset = os.path.getsize(self.f.name)
        except Exception:
            self.offset = 0

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.p is None:
            return out
        self.p.terminate()
        try:
            self.p.wait(timeout=5)
        except Exception:
            self.p.kill()
        self.f.flush()
        with open(self.f.name) as fh:
            fh.seek(self.offset)
            rows = [r.strip().split(",") for r in fh if r.strip()]
        os.unlink(self.f.name)
        sm, mx, reasons = [], [], set()
        for r in rows:
            try:
                sm.append(float(r[1])); mx.append(float(r[2]))
            except Exception:
                continue
            names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
            for name, v in zip(names, r[5:9]):
                if v.strip().lower().startswith("active"):
                    reasons.add(name)
        if sm:
            out.update(sm_mhz=float(np.median(sm)), sm_max_mhz=float(max(mx)), reasons=sorted(reasons), samples=len(sm))
        return out


# ---------------------------------------------------------------------------------------------
# workloads (the benchmark's five configurations; inputs are seeded and synthetic)
# ---------------------------------------------------------------------------------------------
def spectral_shapes(name):
    from paper_1806_04090_b200 import synth
    if name == "c1a":
        return [(64, 64)]
    if name == "c2":
        return [(l.rows, l.cols) for l in synth.RESNET18_LAYERS]
    if name == "c3":
        return [(l.rows, l.cols) for l in synth.VGG11_LAYERS]
    if name == "c5":
        return [(1024, 4096)] * 96
    raise ValueError(name)


SPECTRAL = {   # decay of the spectrum, noise, budgets (first = the one a headline run uses), description
    "c1a": dict(decay=1.0, noise_std=1e-2, budgets=[2.0], text="c1a: one 64 x 64 gradient, sigma_i = 1/i + N(0, 1e-4) noise"),
    "c2": dict(decay=1.5, noise_rel=0.01, budgets=[2.0], text="c2: ResNet-18-shaped layer set (18 layers, 10,992,320 elements)"),
    "c3": dict(decay=1.0, noise_rel=0.01, budgets=[2.0, 1.0, 3.0], text="c3: VGG-11-shaped layer set with two 4096 x 4096 layers (11 layers, 42,813,120 elements)"),
    "c5": dict(decay=1.0, noise_rel=0.005, budgets=[4.0, 2.0, 8.0], text="c5: 96 gradient matrices of 1024 x 4096 (402,653,184 elements)"),
}
ENTRYWISE = {
    "c1b": dict(n=4096, budgets=[64.0], text="c1b: 4096 N(0,1) elements"),
    "c4": dict(n=25_600_000, budgets=[0.01, 0.001, 0.1], relative=True, text="c4: 25.6M Laplace(0, 1e-3) elements"),
}


_INPUT_CACHE = {}
FAST_INPUTS = False      # --fast-inputs: one generated matrix per distinct shape, the others by row / column permutations


def make_spectral_inputs(name, seed, dev):
    """One input set of a spectral workload on the device (torch generator: the recipe of synth.lowrank_plus_noise).
    With --fast-inputs (for profiler captures, where every launch costs) only the first matrix of each shape is
    generated; the others are that matrix with its rows and columns permuted and random signs (the same spectrum,
    factors again Haar distributed)."""
    import torch
    from paper_1806_04090_b200 import synth
    cfg = SPECTRAL[name]
    key = (name, seed, str(dev), FAST_INPUTS)
    if key in _INPUT_CACHE:                  # the same workload at another budget: same gradients
        return _INPUT_CACHE[key]
    for k_ in [k_ for k_ in _INPUT_CACHE if k_[0] != name]:
        del _INPUT_CACHE[k_]                 # one workload's inputs at a time (config 5 is 1.6 GB)
    out, base = [], {}
    for i, (m, n) in enumerate(spectral_shapes(name)):
        if FAST_INPUTS and (m, n) in base:
            gen = torch.Generator(device=dev); gen.manual_seed(seed * 1000 + i)
            g0 = base[(m, n)]
            pr, pc = torch.randperm(m, device=dev, generator=gen), torch.randperm(n, device=dev, generator=gen)
            sr = (torch.randint(0, 2, (m, 1), device=dev, generator=gen) * 2 - 1).to(torch.float32)
            out.append((g0[pr][:, pc] * sr).contiguous())
            continue
        g = synth.torch_lowrank_plus_noise(m, n, cfg["decay"], seed * 1000 + i, dev, noise_rel=cfg.get("noise_rel"),
                                           noise_std=cfg.get("noise_std"))
        base[(m, n)] = g
        out.append(g)
    _INPUT_CACHE[key] = out
    return out


def make_entrywise_input(name, seed, dev):
    import torch
    from paper_1806_04090_b200 import synth
    if name == "c1b":
        return torch.from_numpy(synth.c1_entrywise(seed)).to(dev)
    return torch.from_numpy(synth.c4_entrywise(seed)).to(dev)


class Runner:
    """One workload at one budget: pre-allocated payload and outputs, `step(i)` = encode + decode on the current stream."""

    def __init__(self, a, dev, name, budget, seed, rank=0, n_sets=None, exchange="none"):
        import torch
        from paper_1806_04090_b200 import api
        self.a, self.dev, self.name, self.seed, self.rank = a, dev, name, seed, rank
        self.exchange, self.peers = exchange, None
        self.spectral = name in SPECTRAL
        if self.spectral:
            shapes = spectral_shapes(name)
            self.elems = int(sum(m * n for m, n in shapes))
            in_bytes = 4 * self.elems
            if n_sets is None:      # enough distinct input sets that a step's inputs were evicted from L2 since last use
                n_sets = 1 if in_bytes > L2_BYTES else min(8, int(np.ceil(2.0 * L2_BYTES / in_bytes)) + 1)
                if FAST_INPUTS:
                    n_sets = min(n_sets, 2)     # profiler captures: few generator launches (the timings of such a run are not reported)
            self.sets = [make_spectral_inputs(name, seed + j, dev) for j in range(n_sets)]
            self.s = float(budget)
            self.k_cap = api.default_k_cap(self.s, max(min(sh) for sh in shapes))
            self.payload = torch.empty(api.payload_bytes_spectral(shapes, self.k_cap), dtype=torch.uint8, device=dev)
            self.outs = [torch.empty(sh, dtype=torch.float32, device=dev) for sh in shapes]
            self.shapes = shapes
        else:
            cfg = ENTRYWISE[name]
            n = cfg["n"]
            self.elems = n
            in_bytes = 4 * n
            if n_sets is None:
                n_sets = min(8, int(np.ceil(2.0 * L2_BYTES / in_bytes)) + 1)
            self.sets = [[make_entrywise_input(name, seed + j, dev)] for j in range(n_sets)]
            self.s = float(budget) * n if cfg.get("relative") else float(budget)
            self.k_cap = int(self.s * 1.05) + 1000
            self.payload = torch.empty(api.payload_bytes_entrywise([n], self.k_cap), dtype=torch.uint8, device=dev)
            self.outs = [torch.empty(n, dtype=torch.float32, device=dev)]
            self.shapes = [(1, n)]
        if exchange == "p2p":                               # the payload lives where the peers can read it in place
            from paper_1806_04090_b200 import dist
            self.peers = dist.PeerPayloads(self.payload.numel(), dev)
            self.payload = self.peers.buf
        self.in_bytes = in_bytes
        self.n_sets = n_sets
        self.small = in_bytes * n_sets <= 2 * L2_BYTES      # cannot rotate out of L2: flush between iterations instead
        self.flush_buf = torch.empty(2 * L2_BYTES, dtype=torch.uint8, device=dev) if self.small else None

    def encode(self, i, layers=None, payload=None):
        layers = layers if layers is not None else self.sets[i % self.n_sets]
        payload = payload if payload is not None else self.payload
        if self.spectral:
            pay, _ = self.a.atomo_encode_spectral(layers, self.s, self.seed + self.rank, step=i, k_cap=self.k_cap, payload=payload)
        else:
            pay, _ = self.a.atomo_encode_entrywise(layers, self.s, self.seed + self.rank, step=i, k_cap=self.k_cap, payload=payload)
        return pay

    def step(self, i, layers=None, outs=None):
        pay = self.encode(i, layers)
        outs = outs if outs is not None else self.outs
        if self.exchange == "none":
            self.a.atomo_decode(pay, out=outs)
            return pay
        # the combine step of data-parallel training.  nccl: all-gather the payloads, then the averaging decode;
        # p2p: the averaging decode reads every rank's payload in place over NVLink (one kernel, no collective)
        from paper_1806_04090_b200 import api, dist
        if self.exchange == "p2p":
            self.peers.publish()
            bufs = self.peers.views()
        else:
            bufs = dist.all_gather_bytes(pay.buf)
        self.a.atomo_decode_average([api.Payload(b, pay.kind, pay.shapes, pay.k_cap, self.a) for b in bufs], out=outs)
        if self.exchange == "p2p":
            self.peers.release()
        return pay

    def l2_note(self):
        if self.small:
            return "a 252 MiB buffer is overwritten between timed iterations (L2 flush), each iteration timed by its own event pair"
        if self.n_sets > 1:
            return (f"inputs rotate over {self.n_sets} distinct sets ({self.n_sets * self.in_bytes / 2**20:.0f} MiB > 126 MiB L2), "
                    "so each step reads its gradients from HBM")
        return f"one step's inputs ({self.in_bytes / 2**20:.0f} MiB) exceed the 126 MiB L2"


def timed_reps(run, steps, warmup, reps, first=0):
    """`reps` timed runs of `steps` steps each (CUDA events on the current stream); returns ms per step of each run."""
    import torch
    i = first
    for _ in range(warmup):
        run.step(i); i += 1
    torch.cuda.synchronize()
    out = []
    for _ in range(reps):
        if run.small:                       # per-iteration events, L2 flushed in between (not timed)
            evs = []
            for _ in range(steps):
                run.flush_buf.fill_(i & 0xFF)
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record(); run.step(i); e1.record(); i += 1
                evs.append((e0, e1))
            torch.cuda.synchronize()
            out.append(float(np.mean([a.elapsed_time(b) for a, b in evs])))
        else:
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            for _ in range(steps):
                run.step(i); i += 1
            e1.record()
            torch.cuda.synchronize()
            out.append(e0.elapsed_time(e1) / steps)
    return out


STAGE_EVENTS_MIN_MS = 1.0     # steps shorter than this are timed without the library's stage events


def timed_with_stages(a, run, steps, warmup, reps, first=0, mark=None):
    """The timed runs plus the library's per-stage times.  The stage timers are CUDA events recorded around every
    stage; on a step of a millisecond or more they cost nothing and run inside the timed region.  On a step of a
    hundred microseconds six event records are a fifth of the step, so there the timed region runs without them and
    the stage split comes from one more run of `steps` steps directly after it.  Returns (ms per step of each run,
    stage ms totals, stage launch totals, steps the totals cover, how the stages were timed)."""
    import torch
    i = first
    for _ in range(max(warmup, 1)):
        run.step(i); i += 1
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(); run.step(i); e1.record(); i += 1
    torch.cuda.synchronize()
    inside = e0.elapsed_time(e1) >= STAGE_EVENTS_MIN_MS
    if mark is not None:
        mark()
    if inside:
        a.set_profiling(True)
        ms = timed_reps(run, steps, 0, reps, first=i)
        tot_ms, tot_ln, _ = a.stage_totals()
        a.set_profiling(False)
        return ms, tot_ms, tot_ln, steps * reps, "stage events inside the timed region"
    ms = timed_reps(run, steps, 0, reps, first=i)
    a.set_profiling(True)
    timed_reps(run, steps, 0, 1, first=i + steps * reps)
    tot_ms, tot_ln, _ = a.stage_totals()
    a.set_profiling(False)
    return ms, tot_ms, tot_ln, steps, "stage split from one more run right after the timed region (no stage events inside it)"


# ---------------------------------------------------------------------------------------------
# algorithmic work of the dominant kernels
# ---------------------------------------------------------------------------------------------
def tridiag_small_flops(shapes):
    """Register-resident Householder reduction (short sides up to 512), fp64: the method's own work for a symmetric
    matrix is one matrix-vector product (2 m^2 flop) and the lower triangle of one rank-two update (2 m^2 flop) per
    step on the trailing block of order m: 4 r^3 / 3 in all.  (The kernel stores the full matrix and spends 2 r^3.)"""
    return sum(4.0 / 3.0 * min(m, n) ** 3 for m, n in shapes if min(m, n) <= 512)


def tridiag_big_bytes(shapes):
    """Blocked Householder reduction with the matrix in global memory (short sides above 512), fp32 storage: every
    step must read the trailing block once for its matrix-vector product; a symmetric matrix needs one triangle:
    sum over steps of m^2 / 2 entries of 4 bytes = (2/3) r^3 bytes per layer.  (A kernel that reads the full square
    shows twice this as DRAM traffic.)"""
    tot = 0.0
    for m, n in shapes:
        r = min(m, n)
        if r > 512:
            tot += sum(2.0 * (r - c - 1) ** 2 for c in range(r - 2))
    return tot


def roofline_for(run, eig_ms_per_step, eig_launches_per_step, scheme, peaks, fma_peaks, step_ms):
    """Roofline of the dominant kernel of a spectral workload (the eigen stage)."""
    shapes = run.shapes
    big = any(min(sh) > 512 for sh in shapes)
    out = {"share_of_step": eig_ms_per_step / step_ms, "launches_per_step": eig_launches_per_step,
           "avg_launch_us": eig_ms_per_step * 1e3 / max(eig_launches_per_step, 1.0)}
    if scheme == 3 and big:
        # the blocked reduction dominates whenever it runs (config 3: also one launch of the small-layer kernel in the stage)
        b = tridiag_big_bytes(shapes)
        ach = b / (eig_ms_per_step * 1e-3) / 1e9
        out.update(bound="hbm", kernel="sp_tridiag_big1_kernel (one CTA per layer)" if max(min(sh) for sh in shapes) <= 1024 and sum(1 for sh in shapes if min(sh) > 512) >= 38 else "sp_tridiag_big_kernel (clusters)", achieved=ach, peak=peaks["hbm_gbs"], unit="GB/s",
                   frac=ach / peaks["hbm_gbs"], traffic=NCU_TRAFFIC.get(("sp_tridiag_big_kernel", run.name)),
                   peak_source=f"{peaks['source']} copy bandwidth (MEASURED_PEAKS.json)",
                   algorithmic="one triangle of the trailing block per Householder step, 4-byte entries: (2/3) r^3 bytes per layer",
                   arithmetic="f32 storage and products, f64 sums and scalars")
    elif scheme == 3:
        f = tridiag_small_flops(shapes)
        ach = f / (eig_ms_per_step * 1e-3) / 1e12
        out.update(bound="alu", kernel="sp_tridiag_cluster_kernel", achieved=ach, peak=fma_peaks["fp64"], unit="TFLOP/s",
                   frac=ach / fma_peaks["fp64"], traffic=NCU_TRAFFIC.get(("sp_tridiag_cluster_kernel", run.name)),
                   peak_source="measured in this run: register-only fp64 FMA chains on every SM (atomo_measure_fma_peak)",
                   algorithmic="4 r^3 / 3 fp64 flop per layer (symmetric reduction)", arithmetic="f64")
    else:
        out.update(bound="alu", kernel="Jacobi eigen-solver (fallback route)", achieved=None, peak=fma_peaks["fp32"],
                   unit="TFLOP/s", frac=None, traffic=None, peak_source="measured fp32 FMA chains", arithmetic="f32")
    return out


# ---------------------------------------------------------------------------------------------
# oracle on the host cores
# ---------------------------------------------------------------------------------------------
ORACLE_SAMPLE = {   # workload -> (rows, cols) of the layer the bounded oracle sample runs on, and what it stands for
    "c5": (256, 1024), "c3": (256, 1024), "c2": (128, 1152), "c1a": (64, 64),
}


def oracle_sample_step(name, budget, step):
    """One bounded oracle step for workload `name`: fp64 encode + decode of one layer of the workload's recipe.
    Spectral workloads whose layers take minutes in the oracle (short sides 1024 and 4096) are sampled at a
    quarter of the side lengths; the oracle's cost per element grows with the short side, so its throughput at
    full size is lower than this sample's (said in the `sample` text)."""
    from oracle import atomo_oracle as oracle
    from paper_1806_04090_b200 import synth
    if name in SPECTRAL:
        cfg = SPECTRAL[name]
        m, n = ORACLE_SAMPLE[name]
        rng = np.random.default_rng([5, step])
        G = synth.lowrank_plus_noise(rng, m, n, cfg["decay"], noise_rel=cfg.get("noise_rel"), noise_std=cfg.get("noise_std"))
        t0 = time.perf_counter()
        enc = oracle.encode_spectral(G, budget, 1, step=step, layer=0)
        oracle.decode_spectral(enc["coef"], enc["U_S"], enc["V_S"])
        return time.perf_counter() - t0, m * n
    cfg = ENTRYWISE[name]
    n = min(cfg["n"], 2_000_000)
    g = synth.c4_entrywise(step, n) if name == "c4" else synth.c1_entrywise(step)
    s = budget * n if cfg.get("relative") else budget
    t0 = time.perf_counter()
    enc = oracle.encode_entrywise(g, s, 1, step=step, layer=0)
    oracle.decode_entrywise(g.size, enc["idx"], enc["val"])
    return time.perf_counter() - t0, g.size


def oracle_sample_text(name):
    if name in ("c5", "c3"):
        m, n = ORACLE_SAMPLE[name]
        return (f"fp64 oracle (one-sided Jacobi SVD, Algorithm 1, Philox draws, decode) on one {m} x {n} layer of the workload's "
                f"recipe per step; a full-size 1024 x 4096 layer takes the oracle about 80 s on one core (4096 x 4096: over an "
                f"hour), i.e. roughly 4x (16x) fewer elements/s than this sample")
    if name in SPECTRAL:
        m, n = ORACLE_SAMPLE[name]
        return f"fp64 oracle on one {m} x {n} layer of the workload per step"
    return "fp64 oracle (sort, Algorithm 1, Philox draws, decode) on up to 2,000,000 elements of the workload per step"


def cpu_baseline(name, budget, target_s=12.0):
    from oracle import atomo_oracle as oracle
    oracle.build()
    t_tot, e_tot, k = 0.0, 0, 0
    while t_tot < target_s and k < 64:
        dt, el = oracle_sample_step(name, budget, k)
        t_tot += dt; e_tot += el; k += 1
    return {"value": e_tot / t_tot, "unit": UNIT, "cores": 1, "kind": "oracle",
            "sample": f"{k} steps, {t_tot:.1f} s of CPU: " + oracle_sample_text(name)}


def run_reference(args):
    """--impl reference: the oracle, as it stands, on the host cores (rank 0 only)."""
    if int(os.environ.get("RANK", "0")) != 0:
        return
    from oracle import atomo_oracle as oracle
    oracle.build()
    name = args.workload
    budget = args.budget if args.budget is not None else (SPECTRAL.get(name) or ENTRYWISE[name])["budgets"][0]
    for w in range(args.warmup):
        oracle_sample_step(name, budget, w)
    t_tot, e_tot = 0.0, 0
    for k in range(args.steps):
        dt, el = oracle_sample_step(name, budget, args.warmup + k)
        t_tot += dt; e_tot += el
    value = e_tot / t_tot
    sample = f"{args.steps} steps, {t_tot:.1f} s of CPU: " + oracle_sample_text(name)
    text = (SPECTRAL.get(name) or ENTRYWISE[name])["text"]
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": t_tot / args.steps * 1e3,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": workload_text(name, budget), "sample": sample},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


def workload_text(name, budget):
    if name in SPECTRAL:
        return f"{SPECTRAL[name]['text']}, spectral ATOMO s={budget:g}, one batched encode + decode per step"
    cfg = ENTRYWISE[name]
    b = f"{100 * budget:g} % of the length" if cfg.get("relative") else f"{budget:g}"
    return f"{cfg['text']}, entry-wise ATOMO s={b}, encode + decode per step"


# ---------------------------------------------------------------------------------------------
def also_line(a, dev, name, budget, peaks, fma_peaks, steps, reps):
    """Device-timed figures of one more configuration (median and min over `reps` runs of `steps` steps)."""
    import torch
    run = Runner(a, dev, name, budget, seed=11)
    ms, tot_ms, tot_ln, n_steps, _ = timed_with_stages(a, run, steps, 3, reps, first=100)
    med, mn = float(np.median(ms)), float(np.min(ms))
    floor_bytes = 12.0 * run.elems                              # two reads of the gradient and one write of the dense result
    line = {"workload": workload_text(name, budget), "ms_per_step_median": med, "ms_per_step_min": mn, "reps": reps,
            "steps_per_rep": steps, "elements_per_s": run.elems / (med * 1e-3),
            "stage_ms_per_step": {k: v / n_steps for k, v in tot_ms.items() if v > 0},
            "streaming_floor_frac_of_measured_hbm": floor_bytes / (med * 1e-3) / 1e9 / peaks["hbm_gbs"],
            "l2": run.l2_note()}
    if run.spectral:
        scheme = a.last_eig_scheme()
        line["eigen_scheme"] = scheme
        line["roofline"] = roofline_for(run, tot_ms["eig"] / n_steps, tot_ln["eig"] / n_steps, scheme, peaks, fma_peaks, med)
    else:
        gbs = floor_bytes / (med * 1e-3) / 1e9
        line["roofline"] = {"bound": "hbm", "kernel": "entry-wise path (ew_encode + ew_decode)", "achieved": gbs,
                            "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": gbs / peaks["hbm_gbs"],
                            "algorithmic": "12 B per element", "target_frac_of_8TBs": gbs / 8000.0, "meets_60pct_of_8TBs": gbs >= 4800.0}
    del run
    torch.cuda.empty_cache()
    return line


def run_ours(args):
    import torch
    from paper_1806_04090_b200 import api, dist

    rank, local_rank, world = dist.init("nccl") if int(os.environ.get("WORLD_SIZE", "1")) > 1 else (0, 0, 1)
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    a = api.Atomo(local_rank)
    sampler = ClockSampler(local_rank)       # started now, so that it is up when the timed region begins (mark())
    if rank == 0:
        sampler.start()
    peaks = measured_peaks()
    fma_peaks = {"fp32": api.measure_fma_peak(local_rank, False), "fp64": api.measure_fma_peak(local_rank, True)}

    name = args.workload
    cfg = SPECTRAL.get(name) or ENTRYWISE[name]
    budget = args.budget if args.budget is not None else cfg["budgets"][0]
    exchange = args.exchange if world > 1 else "none"
    run = Runner(a, dev, name, budget, seed=0, rank=rank, exchange=exchange)
    elems = run.elems

    # ---- warm-up, then the timed region: device-resident inputs, R runs of K steps ----
    uploads0 = [None]

    def mark():
        uploads0[0] = a.table_uploads()
        dist.barrier(); torch.cuda.synchronize()
        if rank == 0:
            sampler.mark()

    reps_ms, tot_ms, tot_ln, stage_steps, stage_note = timed_with_stages(a, run, args.steps, args.warmup, args.reps, mark=mark)
    uploads0 = uploads0[0]
    uploads1 = a.table_uploads()
    torch.cuda.synchronize(); dist.barrier()
    clocks = sampler.stop() if rank == 0 else None
    reps_ms = [dist.max_over_ranks(m, dev) for m in reps_ms]
    n_steps = args.steps * args.reps
    ms_per_step = float(np.median(reps_ms))
    value = world * elems / (ms_per_step * 1e-3)
    scheme = a.last_eig_scheme() if run.spectral else None
    # the stages' kernels + the header kernel, per run of K steps (an entry-wise call with one vector writes its headers
    # inside the encode kernel: no header kernel)
    launches = (sum(tot_ln.values()) / stage_steps + (1 if run.spectral else 0)) * args.steps

    # ---- end to end: host buffers, copies inside the timed region ----
    # Every step's inputs come from pinned host memory and its decoded gradients go back to pinned host memory.
    # Two copy streams and double buffers let the copies of step k+1 (in) and k-1 (out) run under step k's kernels.
    host_in = [[t.cpu().pin_memory() for t in s_] for s_ in run.sets[:2]]
    stage_in = [[torch.empty_like(t) for t in run.sets[0]] for _ in range(2)]
    stage_out = [[torch.empty_like(t) for t in run.outs] for _ in range(2)]
    host_out = [[torch.empty(t.shape, dtype=torch.float32).pin_memory() for t in run.outs] for _ in range(2)]
    s_in, s_out = torch.cuda.Stream(device=dev), torch.cuda.Stream(device=dev)
    main = torch.cuda.current_stream()

    def e2e_run(first, n):
        ev_in = [torch.cuda.Event() for _ in range(2)]        # inputs of a step have arrived in stage_in[b]
        ev_enc = [None, None]                                 # the encode that read stage_in[b] has finished
        ev_dec = [torch.cuda.Event() for _ in range(2)]       # stage_out[b] holds a step's decoded gradients
        ev_out = [None, None]                                 # stage_out[b] has been copied to the host

        def copy_in(k):
            b = k % 2
            with torch.cuda.stream(s_in):
                if ev_enc[b] is not None:
                    s_in.wait_event(ev_enc[b])
                for d, h in zip(stage_in[b], host_in[(first + k) % len(host_in)]):
                    d.copy_(h, non_blocking=True)
                ev_in[b].record(s_in)

        copy_in(0)
        for k in range(n):
            b = k % 2
            if k + 1 < n:
                copy_in(k + 1)
            main.wait_event(ev_in[b])
            if ev_out[b] is not None:
                main.wait_event(ev_out[b])
            pay = run.encode(first + k, stage_in[b])
            ev_enc[b] = torch.cuda.Event(); ev_enc[b].record(main)
            a.atomo_decode(pay, out=stage_out[b])
            ev_dec[b].record(main)
            with torch.cuda.stream(s_out):
                s_out.wait_event(ev_dec[b])
                for h, d in zip(host_out[b], stage_out[b]):
                    h.copy_(d, non_blocking=True)
                ev_out[b] = torch.cuda.Event(); ev_out[b].record(s_out)
        for e in ev_out:
            if e is not None:
                main.wait_event(e)                            # the timed region ends after the last copy out

    e2e_run(0, 3)
    dist.barrier(); torch.cuda.synchronize()
    e2e_steps = args.steps
    t0 = torch.cuda.Event(enable_timing=True); t1 = torch.cuda.Event(enable_timing=True)
    t0.record()
    e2e_run(100, e2e_steps)
    t1.record()
    torch.cuda.synchronize(); dist.barrier()
    e2e_ms = dist.max_over_ranks(t0.elapsed_time(t1), dev)
    e2e_value = world * elems * e2e_steps / (e2e_ms * 1e-3)
    del host_in, stage_in, stage_out, host_out

    if rank == 0:
        stage = {k: v / stage_steps for k, v in tot_ms.items() if v > 0}
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": {"workload": workload_text(name, budget), "k_cap": run.k_cap, "l2": run.l2_note(),
                       "parallelism": "single GPU" if world == 1 else
                       {"none": "independent replicas of the workload, one per GPU, no collective",
                        "nccl": "data-parallel: payload all-gather + averaging decode",
                        "p2p": "data-parallel: the averaging decode reads the peers' payloads over NVLink"}[exchange],
                       "eigen_scheme": scheme, "stage_ms_per_step": stage,
                       "timing": f"{args.reps} runs of {args.steps} steps each, CUDA events around each run; ms_per_step is the median run; {stage_note}"},
            "ms_per_step_min": float(np.min(reps_ms)), "ms_per_step_runs": reps_ms,
            "clocks": clocks,
            "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": run.in_bytes, "d2h_bytes_per_step": run.in_bytes,
                    "ms_per_step": e2e_ms / e2e_steps, "steps": e2e_steps,
                    "overlap": "copies of step k+1 (in) and k-1 (out) run on two copy streams under step k's kernels"},
            "gpu_launches": int(launches),
            "table_uploads_in_timed_region": {"uploads": uploads1[0] - uploads0[0], "calls_served_from_device": uploads1[1] - uploads0[1],
                                              "note": "host-to-device copies of descriptor tables inside the timed region (0 in steady state)"},
            "measured_fma_peaks_tflops": fma_peaks,
        }
        if run.spectral:
            line["roofline"] = roofline_for(run, tot_ms["eig"] / stage_steps, tot_ln["eig"] / stage_steps, scheme, peaks, fma_peaks, ms_per_step)
            gram_flops = sum(min(m, n) ** 2 * max(m, n) * 2.0 for m, n in run.shapes)      # useful flops, full square
            tf32_peak = peaks["bf16_tflops"] * (1.1 / 2.25)
            line["gram"] = {"kernel": "sp_gram_tc_kernel (tcgen05, 3 x TF32)", "ms_per_step": stage.get("gram"),
                            "useful_tflops": gram_flops / 2 / (stage["gram"] * 1e-3) / 1e12 if stage.get("gram") else None,
                            "tf32_peak_tflops": tf32_peak, "peak_source": f"{peaks['source']} bf16 burst x nominal 1.1/2.25",
                            "note": "useful = one triangle of G G^T, r^2 L flop; the stage also holds trace and scaling"}
            if line["gram"]["useful_tflops"]:
                line["gram"]["useful_frac"] = line["gram"]["useful_tflops"] / tf32_peak
                line["gram"]["issued_frac"] = 3.0 * line["gram"]["useful_tflops"] / tf32_peak
                line["gram"]["meets_50pct_target"] = line["gram"]["issued_frac"] >= 0.5
        else:
            gbs = 12.0 * elems / (ms_per_step * 1e-3) / 1e9
            line["roofline"] = {"bound": "hbm", "kernel": "entry-wise path (ew_encode + ew_decode)", "achieved": gbs,
                                "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": gbs / peaks["hbm_gbs"],
                                "traffic": NCU_TRAFFIC.get(("entrywise", name)) if abs(budget - 0.01) < 1e-12 else None,
                                "algorithmic": "12 B per element: the gradient read twice (the normaliser is global), the dense result written once; at budgets up to about 1.5 % of the length the encode kernel lists its candidates during the first read and reads the gradient once",
                                "peak_source": f"{peaks['source']} copy bandwidth (MEASURED_PEAKS.json)",
                                "target_frac_of_8TBs": gbs / 8000.0, "meets_60pct_of_8TBs": gbs >= 4800.0}
        del run
        torch.cuda.empty_cache()
        if world == 1 and not args.no_extras:
            also = []
            plan = [(n_, b) for n_ in ("c5", "c3", "c2", "c1a") for b in SPECTRAL[n_]["budgets"]] + \
                   [(n_, b) for n_ in ("c4", "c1b") for b in ENTRYWISE[n_]["budgets"]]
            for n_, b in plan:
                if n_ == name and b == budget:
                    continue
                big = n_ in ("c5", "c3")
                also.append(also_line(a, dev, n_, b, peaks, fma_peaks, steps=3 if big else 20, reps=3 if big else 5))
            line["also"] = also
        if world == 1 and not args.no_cpu_baseline:
            line["cpu_baseline"] = cpu_baseline(name, budget)
        print(json.dumps(line))
    a.close()
    dist.finish()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--reps", type=int, default=5, help="timed runs of --steps steps each (median and min are reported)")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="c5", choices=sorted(list(SPECTRAL) + list(ENTRYWISE)))
    ap.add_argument("--budget", type=float, default=None, help="sparsity budget s (entry-wise c4: fraction of the length)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--exchange", default="none", choices=["none", "nccl", "p2p"],
                    help="N > 1: the data-parallel combine step instead of independent replicas -- nccl: all-gather "
                         "the payloads, then decode their average; p2p: the averaging decode reads the peers' payloads "
                         "in place over NVLink")
    ap.add_argument("--no-extras", action="store_true", help="skip the `also` entries (the other configurations)")
    ap.add_argument("--fast-inputs", action="store_true",
                    help="generate one matrix per distinct shape and derive the others by permutations and signs "
                         "(profiler captures: thousands of generator launches less)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    global FAST_INPUTS
    FAST_INPUTS = bool(args.fast_inputs)
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()

#!/usr/bin/env python
"""Benchmark of the ATOMO encode + decode hot path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload c2|c4|c5] [--impl ours|reference]

A step is one pass of the whole path (encode, then decode) over one batch of synthetic
gradients.  The default workload is the ResNet-18-shaped layer set (spectral ATOMO, s = 2,
18 layers, 10,992,320 gradient elements, one batched call).  Prints ONE JSON line on rank 0.
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
FP32_FMA_PEAK_TFLOPS = 148 * 128 * 2 * 1.965e9 / 1e12       # SMs x FP32 lanes x 2 flop x max SM clock
# dram__bytes_read.sum + dram__bytes_write.sum of one sp_jacobi_cluster_kernel launch on this workload, from the
# ncu capture summarised in profiles/sp_jacobi_cluster_c2.txt (5.66 MB read, nothing written back to DRAM)
JACOBI_TRAFFIC_BYTES_PER_LAUNCH = 5660672
FP64_FMA_PEAK_TFLOPS = 148 * 64 * 2 * 1.965e9 / 1e12        # SMs x FP64 lanes x 2 flop x max SM clock
# the same two counters for one sp_tridiag_cluster_kernel launch (profiles/sp_tridiag_cluster_c2.txt)
TRIDIAG_TRAFFIC_BYTES_PER_LAUNCH = 5638912


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        d = json.load(open(path))
        return {"hbm_gbs": float(d["hbm_gbs"]), "source": "measured"}
    return {"hbm_gbs": 6650.0, "source": "fallback"}


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
            fh.seek(getattr(self, "offset", 0))
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
def workload_c2(seed):
    from paper_1806_04090_b200 import synth
    return synth.c2_resnet18(seed), synth.layer_elements(synth.RESNET18_LAYERS)


def oracle_step(mats, s, seed, step):
    """Encode + decode of a list of layers with the fp64 oracle (single thread)."""
    from oracle import atomo_oracle as oracle
    for l, G in enumerate(mats):
        enc = oracle.encode_spectral(G, s, seed, step=step, layer=l)
        oracle.decode_spectral(enc["coef"], enc["U_S"], enc["V_S"])


def cpu_baseline_c2(seed=0):
    """The oracle as it stands on the host cores: one layer per distinct shape is timed and the
    time is scaled by how often the shape occurs (the full set takes about a minute per step)."""
    from paper_1806_04090_b200 import synth
    from oracle import atomo_oracle as oracle
    oracle.build()
    layers = synth.RESNET18_LAYERS
    shapes = {}
    for i, l in enumerate(layers):
        shapes.setdefault((l.rows, l.cols), []).append(i)
    total = 0.0
    per_layer = []
    t_all = time.perf_counter()
    for (rows, cols), idxs in shapes.items():
        G = synth.c2_resnet18(seed, [layers[idxs[0]]])
        t0 = time.perf_counter()
        oracle_step(G, 2.0, seed, 0)
        dt = time.perf_counter() - t0
        total += dt * len(idxs)
        per_layer += [dt] * len(idxs)
    elems = synth.layer_elements(layers)
    # layers are independent: what one layer per thread would give on this host, from the measured per-layer times
    # (longest first onto the least loaded core; computed, not run)
    ncores = os.cpu_count() or 1
    loads = [0.0] * ncores
    for dt in sorted(per_layer, reverse=True):
        loads[loads.index(min(loads))] += dt
    return {"value": elems / total, "unit": UNIT, "cores": 1, "kind": "oracle",
            "sample": f"one layer per distinct shape ({len(shapes)} of {len(layers)} layers, "
                      f"{time.perf_counter() - t_all:.1f} s of CPU), time scaled by shape count to the full set "
                      f"(extrapolated step time {total:.1f} s)",
            "all_cores_estimate": {"cores": ncores, "value": elems / max(loads), "unit": UNIT,
                                   "how": "one layer per thread, longest first, from the per-layer times above; "
                                          "computed, not run"}}


def reference_sample_layers():
    from paper_1806_04090_b200 import synth
    seen, out = set(), []
    for l in synth.RESNET18_LAYERS:
        if min(l.rows, l.cols) <= 256 and (l.rows, l.cols) not in seen:
            seen.add((l.rows, l.cols)); out.append(l)
    return out


def run_reference(args):
    """--impl reference: the oracle, as it stands, on the host cores (rank 0 only)."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from paper_1806_04090_b200 import synth
    from oracle import atomo_oracle as oracle
    oracle.build()
    layers = reference_sample_layers()
    mats = synth.c2_resnet18(0, layers)
    elems = synth.layer_elements(layers)
    for w in range(args.warmup):
        oracle_step(mats, 2.0, 0, w)
    t0 = time.perf_counter()
    for k in range(args.steps):
        oracle_step(mats, 2.0, 0, args.warmup + k)
    dt = time.perf_counter() - t0
    value = elems * args.steps / dt
    sample = (f"per step: one layer of each distinct ResNet-18 shape with short side <= 256 "
              f"({len(layers)} layers, {elems} elements); the 512-row layers are left out to bound the run")
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt / args.steps * 1e3,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": "c2: ResNet-18-shaped layer set, spectral ATOMO s=2 (bounded sample)", "sample": sample},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


# ---------------------------------------------------------------------------------------------
def jacobi_flops(shapes, sweeps):
    """Algorithmic flops of the eigen-solver (rows of the Cholesky factor, length r): per sweep
    r(r-1)/2 row pairs, each one dot product over r terms (2r flop) and a plane rotation of two rows
    of r entries (6r flop)."""
    tot = 0.0
    for (rows, cols), sw in zip(shapes, sweeps):
        r = min(rows, cols)
        tot += sw * (r * (r - 1) / 2.0) * 8.0 * r
    return tot


def tridiag_flops(shapes):
    """Algorithmic flops of the Householder reduction of the r x r Gram matrix to tridiagonal form as the kernel
    does it (full symmetric storage): step k works on the trailing block of order m = r - k - 1 with one
    matrix-vector product (2 m^2 flop) and one rank-two update (4 m^2 flop): 2 r^3 in all, in fp64."""
    return sum(2.0 * min(rows, cols) ** 3 for rows, cols in shapes)


def entrywise_extra(a, dev, measured_hbm_gbs, steps=20):
    """Entry-wise ATOMO on the 25.6M-element Laplace vector (config 4), s = 1 % of the length:
    encode + decode back to back, device-resident inputs rotating over 3 vectors (307 MB > L2)."""
    import torch
    from paper_1806_04090_b200 import api, synth
    n = 25_600_000
    gs = [torch.from_numpy(synth.c4_entrywise(i)).to(dev) for i in range(3)]
    outs = [torch.empty(n, dtype=torch.float32, device=dev) for _ in range(3)]
    s = 0.01 * n
    kc = int(s * 1.05) + 1000
    payload = torch.empty(api.payload_bytes_entrywise([n], kc), dtype=torch.uint8, device=dev)

    def step(i):
        pay, _ = a.atomo_encode_entrywise([gs[i % 3]], s, seed=7, step=i, k_cap=kc, payload=payload)
        a.atomo_decode(pay, out=[outs[i % 3]])

    for i in range(3):
        step(i)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for i in range(steps):
        step(3 + i)
    e1.record()
    torch.cuda.synchronize()
    us = e0.elapsed_time(e1) / steps * 1e3
    gbs = 12.0 * n / (us * 1e-6) / 1e9          # 2 reads of g + 1 write of the dense result
    return {"workload": "c4: entry-wise, 25.6M Laplace(0,1e-3) elements, s = 1 % of the length", "us_per_step": us,
            "elements_per_s": n / (us * 1e-6), "algorithmic_gbs": gbs, "hbm_frac_of_measured": gbs / measured_hbm_gbs}


def run_ours(args):
    import torch
    from paper_1806_04090_b200 import api, dist

    backend = "nccl"
    rank, local_rank, world = dist.init(backend) if int(os.environ.get("WORLD_SIZE", "1")) > 1 else (0, 0, 1)
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    a = api.Atomo(local_rank)
    # the clock sampler starts now, so that it is up and running when the timed region begins (mark())
    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()

    if args.workload != "c2":
        raise SystemExit("only the c2 workload is a bench line; the other configs are parity-test cases")
    s, seed = 2.0, 0
    # several distinct input sets so that each step's gradients were evicted from L2 since last use
    mats0, elems = workload_c2(seed)
    in_bytes = sum(m.nbytes for m in mats0)
    n_sets = int(np.ceil(2.0 * L2_BYTES / in_bytes)) + 1
    host_sets = [mats0] + [workload_c2(seed + 1 + i)[0] for i in range(n_sets - 1)]
    shapes = [m.shape for m in mats0]
    dev_sets = [[torch.from_numpy(m).to(dev) for m in hs] for hs in host_sets]
    k_cap = api.default_k_cap(s, max(min(sh) for sh in shapes))
    payload = torch.empty(api.payload_bytes_spectral(shapes, k_cap), dtype=torch.uint8, device=dev)
    outs = [torch.empty(sh, dtype=torch.float32, device=dev) for sh in shapes]

    exchange = args.exchange if world > 1 else "none"
    peers = None
    if exchange == "p2p":                               # payload lives where the peers can read it in place
        peers = dist.PeerPayloads(payload.numel(), dev)
        payload = peers.buf

    def combine(pay):
        """decode.  --exchange nccl: all-gather the payloads, then the averaging decode.  --exchange p2p: the
        averaging decode reads every rank's payload in place over NVLink (one kernel, no collective)."""
        if exchange == "none":
            a.atomo_decode(pay, out=outs)
            return
        if exchange == "p2p":
            peers.publish()
            bufs = peers.views()
        else:
            bufs = dist.all_gather_bytes(pay.buf)
        a.atomo_decode_average([api.Payload(b, pay.kind, pay.shapes, pay.k_cap, a) for b in bufs], out=outs)
        if exchange == "p2p":
            peers.release()

    def step(i, layers):
        pay, _ = a.atomo_encode_spectral(layers, s, seed + rank, step=i, k_cap=k_cap, payload=payload)
        combine(pay)
        return pay

    # ---- warm-up ----
    for w in range(args.warmup):
        step(w, dev_sets[w % n_sets])
    torch.cuda.synchronize()

    # ---- timed region: device-resident inputs ----
    a.set_profiling(True)
    dist.barrier(); torch.cuda.synchronize()
    if rank == 0:
        sampler.mark()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    pay = None
    ev0.record()
    for k in range(args.steps):
        # no host wait inside the loop: the library records its stage events in-stream and they are read afterwards
        pay, _ = a.atomo_encode_spectral(dev_sets[(args.warmup + k) % n_sets], s, seed + rank, step=args.warmup + k,
                                         k_cap=k_cap, payload=payload)
        combine(pay)
    ev1.record()
    torch.cuda.synchronize(); dist.barrier()
    clocks = sampler.stop() if rank == 0 else None
    ms_total = ev0.elapsed_time(ev1)
    ms_total = dist.max_over_ranks(ms_total, dev)
    tot_ms, tot_ln, n_calls = a.stage_totals()           # sums over the timed region (profiling was switched on at its start)
    eig_ms, eig_launches = tot_ms["eig"], tot_ln["eig"]
    launches = sum(tot_ln.values()) + args.steps * (7 + 3)   # + header / descriptor copies, workspace memset, decode tables
    sweeps_seen = [h.sweeps for h in pay.headers()[1]]
    eig_scheme = a.last_eig_scheme()
    a.set_profiling(False)
    ms_per_step = ms_total / args.steps
    value = world * elems * args.steps / (ms_total * 1e-3)

    # ---- end to end: host buffers, copies inside the timed region ----
    # Every step's inputs come from pinned host memory and its decoded gradients go back to pinned host memory.
    # Two copy streams and double buffers let the copies of step k+1 (in) and k-1 (out) run under step k's kernels.
    pinned = [[torch.from_numpy(m).pin_memory() for m in hs] for hs in host_sets]
    stage_in = [[torch.empty(sh, dtype=torch.float32, device=dev) for sh in shapes] for _ in range(2)]
    stage_out = [[torch.empty(sh, dtype=torch.float32, device=dev) for sh in shapes] for _ in range(2)]
    host_out = [[torch.empty(sh, dtype=torch.float32).pin_memory() for sh in shapes] for _ in range(2)]
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
                for d, h in zip(stage_in[b], pinned[(first + k) % n_sets]):
                    d.copy_(h, non_blocking=True)
                ev_in[b].record(s_in)

        copy_in(0)
        for k in range(n):
            b = k % 2
            if k + 1 < n:
                copy_in(k + 1)                                # issued before encode's host-side waits
            main.wait_event(ev_in[b])
            if ev_out[b] is not None:
                main.wait_event(ev_out[b])
            pay, _ = a.atomo_encode_spectral(stage_in[b], s, seed, step=first + k, k_cap=k_cap, payload=payload)
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

    e2e_run(0, max(3, min(args.warmup, 5)))
    dist.barrier(); torch.cuda.synchronize()
    e2e_steps = max(4, args.steps // 2)
    t0 = torch.cuda.Event(enable_timing=True); t1 = torch.cuda.Event(enable_timing=True)
    t0.record()
    e2e_run(100, e2e_steps)
    t1.record()
    torch.cuda.synchronize(); dist.barrier()
    e2e_ms = dist.max_over_ranks(t0.elapsed_time(t1), dev)
    e2e_value = world * elems * e2e_steps / (e2e_ms * 1e-3)

    if rank == 0:
        peaks = measured_peaks()
        tri = eig_scheme == 3
        # dominant kernel: the fp64 tridiagonal reduction (scheme 3) or the fp32 Jacobi eigen-solve (other schemes)
        flops = tridiag_flops(shapes) if tri else jacobi_flops(shapes, sweeps_seen)   # sweeps of the last step; they vary little
        eig_s_per_step = eig_ms * 1e-3 / args.steps
        launches_per_step = eig_launches / args.steps
        achieved = flops / eig_s_per_step / 1e12
        alu_peak = FP64_FMA_PEAK_TFLOPS if tri else FP32_FMA_PEAK_TFLOPS
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": {"workload": "c2: ResNet-18-shaped layer set (18 layers, 10,992,320 elements), spectral ATOMO "
                                   "s=2, one batched encode + decode per step",
                       "k_cap": k_cap, "l2": f"inputs rotate over {n_sets} distinct sets ({n_sets * in_bytes / 2**20:.0f} MiB "
                                             f"> 126 MiB L2) so each step reads gradients from HBM",
                       "parallelism": {"none": "independent replicas, no collective",
                                       "nccl": "data-parallel: payload all-gather + averaging decode",
                                       "p2p": "data-parallel: averaging decode reads the peers' payloads over NVLink"}[exchange]
                       if world > 1 else "single GPU",
                       "eigen_scheme": eig_scheme,
                       "jacobi_sweeps_last_step": None if tri else sweeps_seen,
                       "eig_ms_per_step": eig_ms / args.steps},
            "clocks": clocks,
            "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": in_bytes, "d2h_bytes_per_step": in_bytes,
                    "ms_per_step": e2e_ms / e2e_steps,
                    "overlap": "copies of step k+1 (in) and k-1 (out) run on two copy streams under step k's kernels"},
            "gpu_launches": int(launches),
            "roofline": {"bound": "alu",
                         "kernel": {3: "sp_tridiag_cluster_kernel", 2: "sp_jacobi_cluster_kernel",
                                    1: "sp_jacobi_persistent_kernel"}.get(eig_scheme, "sp_jacobi_step_kernel"),
                         "achieved": achieved,
                         "peak": alu_peak, "unit": "TFLOP/s", "frac": achieved / alu_peak,
                         "traffic": TRIDIAG_TRAFFIC_BYTES_PER_LAUNCH if tri else (JACOBI_TRAFFIC_BYTES_PER_LAUNCH if eig_scheme == 2 else None),
                         "launches_per_step": 1.0 if launches_per_step <= 2 else launches_per_step,
                         "avg_launch_us": eig_s_per_step / (1.0 if launches_per_step <= 2 else launches_per_step) * 1e6,
                         "share_of_step": eig_ms / ms_total,
                         "peak_source": ("derived: 148 SMs x 64 FP64 lanes x 2 flop x 1.965 GHz (no measured FP64 peak on file)" if tri else
                                         "derived: 148 SMs x 128 FP32 lanes x 2 flop x 1.965 GHz (no measured FP32 peak on file)"),
                         "arithmetic": "f64" if tri else "f32",
                         "hbm_peak_gbs": peaks["hbm_gbs"], "hbm_peak_source": peaks["source"]},
        }
        if world == 1 and not args.no_extras:
            line["also"] = [entrywise_extra(a, dev, peaks["hbm_gbs"])]
        if world == 1 and not args.no_cpu_baseline:
            line["cpu_baseline"] = cpu_baseline_c2(seed)
        print(json.dumps(line))
    a.close()
    dist.finish()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=40)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="c2")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--exchange", default="none", choices=["none", "nccl", "p2p"],
                    help="N > 1: the data-parallel combine step instead of independent replicas -- nccl: all-gather "
                         "the payloads, then decode their average; p2p: the averaging decode reads the peers' payloads "
                         "in place over NVLink")
    ap.add_argument("--no-extras", action="store_true", help="skip the entry-wise (config 4) figures")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()

#!/usr/bin/env python
"""Benchmark of the batch-1 dual-sparse decode product y = W.x on RLC-CSC weights.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl celty|reference] [--workload NAME]

A step is one celty_spmspv call (activation compaction, column fetch, run-length decode, shared-memory
accumulation, reduction to y).  The default workload is the largest single-GPU configuration, the
Llama-70B-shaped MLP layer 28672 x 8192 (Bernoulli mask, 50% of the weights kept, x ~ Laplace thresholded to
50% density); the Llama-2-7B attention shape 4096 x 4096 is timed beside it as a second, labelled figure.
Calls rotate over device copies of the layer whose total size exceeds twice the L2, so every call reads HBM.
The K steps are whole replays of one CUDA graph between two CUDA events; that region is taken at least ten
times and the median is reported, so a short run gives the same microseconds per call as a long one.
Prints ONE JSON line: the metric (achieved GB/s on the bytes a call must fetch) with microseconds per call, the
roofline object (achieved against the measured HBM copy bandwidth, DRAM traffic from the profiler, the dense
cuBLAS GEMV under the same rotation and the speed-up over it, the second workload), the end-to-end figure
through host buffers, the SM clocks sampled while timing, context (stream-enqueued, L2-warm and isolated
timings) and the CPU oracle on the host cores.
`--impl reference` times the CPU oracle alone; `--sweep cfgN` times every point of a configured sweep.
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

from paper_2608_01536_b200 import synth  # noqa: E402

METRIC = "SpMSpV achieved HBM GB/s on fetched bytes (batch 1)"

WORKLOADS = {
    # name: (M, K, weight sparsity, mask family, activation dist, activation density, config id)
    "llama7b_attn_4096x4096_s50_a50": (4096, 4096, 0.5, "magnitude", "laplace", 0.5, 2),
    "llama7b_gateup_11008x4096_s50_a50": (11008, 4096, 0.5, "magnitude", "laplace", 0.5, 3),
    "llama7b_down_4096x11008_s50_a50": (4096, 11008, 0.5, "magnitude", "swiglu", 0.5, 3),
    "llama13b_attn_5120x5120_s50_a40": (5120, 5120, 0.5, "bernoulli", "laplace", 0.4, 4),
    "llama13b_gateup_13824x5120_s50_a40": (13824, 5120, 0.5, "bernoulli", "laplace", 0.4, 4),
    "llama13b_down_5120x13824_s50_a40": (5120, 13824, 0.5, "bernoulli", "laplace", 0.4, 4),
    "llama70b_mlp_28672x8192_s50_a50": (28672, 8192, 0.5, "bernoulli", "laplace", 0.5, 5),
    "llama70b_down_8192x28672_s50_a50": (8192, 28672, 0.5, "bernoulli", "laplace", 0.5, 5),
    "llama70b_mlp_28672x8192_s30_a50": (28672, 8192, 0.3, "bernoulli", "laplace", 0.5, 5),
    "llama70b_mlp_28672x8192_s70_a50": (28672, 8192, 0.7, "bernoulli", "laplace", 0.5, 5),
    "small_1024x1024_s50_a50": (1024, 1024, 0.5, "bernoulli", "normal", 0.5, 1),
}
DEFAULT_WORKLOAD = "llama70b_mlp_28672x8192_s50_a50"     # the largest single-GPU configuration: the headline
SECONDARY_WORKLOAD = "llama7b_attn_4096x4096_s50_a50"    # a second, labelled figure (latency-bound)

def make_layer(name: str, variant: int):
    M, K, s, family, dist, d_a, cfg = WORKLOADS[name]
    seed = synth.point_seed(cfg, variant)
    # the largest layers repeat a block of K/8 columns of weights along K (drawing 235 M normals takes minutes);
    # their masks are drawn in full, so no two columns hold the same entries
    W = synth.weights_tiled(seed, M, K, K // 8) if M * K > (1 << 26) else synth.weights(seed, M, K)
    if family == "magnitude":
        mask = synth.mask_magnitude(W, s)
    elif family == "bernoulli":
        mask = synth.mask_bernoulli(seed, M, K, 1.0 - s)
    else:
        mask = synth.mask_powerlaw(seed, M, K, 1.0 - s)
    return W, mask


def make_x(name: str, variant: int):
    M, K, s, family, dist, d_a, cfg = WORKLOADS[name]
    x = synth.activations(synth.point_seed(cfg, 50 + variant), K, dist)
    return x, synth.threshold_for_density(x, d_a)


L2_POLICY = ("inputs larger than L2: on the GPU, calls rotate over enough device copies of the layer (each with its own "
             "activation vector) to exceed 2x the L2 capacity, so every call reads HBM")


def workload_config(name):
    """The `config` object of the JSON line: what defines the workload, identical for both --impl arms."""
    M, K, s, family, dist, d_a, cfg = WORKLOADS[name]
    return {"workload": name, "M": M, "K": K, "weight_sparsity": s, "mask": family, "activations": dist,
            "activation_density": d_a,
            "weights": "N(0, 0.02^2) block of K/8 columns repeated along K, mask not repeated" if M * K > (1 << 26)
            else "N(0, 0.02^2)", "l2": L2_POLICY}


class ClockSampler:
    """Samples SM clock and throttle reasons through NVML while the timed region runs."""

    def __init__(self, index: int, period_s: float = 0.002):
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop = threading.Event()
        self._thread = None
        self.period = period_s
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
        except Exception:
            self.nv = None

    def _loop(self):
        nv = self.nv
        names = {
            "hw_slowdown": getattr(nv, "nvmlClocksThrottleReasonHwSlowdown", 0x8),
            "hw_thermal_slowdown": getattr(nv, "nvmlClocksThrottleReasonHwThermalSlowdown", 0x40),
            "sw_thermal_slowdown": getattr(nv, "nvmlClocksThrottleReasonSwThermalSlowdown", 0x20),
            "sw_power_cap": getattr(nv, "nvmlClocksThrottleReasonSwPowerCap", 0x4),
        }
        while not self._stop.is_set():
            try:
                self.samples.append(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
                r = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
                for k, bit in names.items():
                    if r & bit:
                        self.reasons.add(k)
            except Exception:
                pass
            time.sleep(self.period)

    def __enter__(self):
        if self.nv is not None:
            self._thread = threading.Thread(target=self._loop, daemon=True)
            self._thread.start()
        return self

    def __exit__(self, *a):
        self._stop.set()
        if self._thread is not None:
            self._thread.join()

    def summary(self):
        return {"sm_mhz": float(np.median(self.samples)) if self.samples else None,
                "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons), "samples": len(self.samples)}


def max_over_ranks(value: float, device=None) -> float:
    """Largest `value` over all ranks of the default process group (the value itself without one)."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([value], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def aggregate_throughput(bytes_per_call_per_rank: float, world: int, seconds_per_call: float) -> float:
    """Replicas only: every rank processes its own calls, so the job moves world x the bytes in the
    (max-over-ranks) time of one call.  GB/s."""
    return world * bytes_per_call_per_rank / seconds_per_call / 1e9


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured (MEASURED_PEAKS.json hbm_gbs)"
    return 6650.0, "fallback (6.65 TB/s, earlier measurement on this pool)"


def oracle_seconds_per_call(W, mask, x, tau, budget_s: float, threads: int):
    """The oracle's plain definition on the bench workload, repeated for about budget_s seconds."""
    from oracle import celty_oracle as orc
    orc.masked_gemv(W[:64], mask[:64], x, tau, threads=threads)          # load the library
    t0 = time.perf_counter()
    calls = 0
    while True:
        orc.masked_gemv(W, mask, x, tau, threads=threads)
        calls += 1
        if time.perf_counter() - t0 >= budget_s:
            break
    return (time.perf_counter() - t0) / calls, calls


def run_reference(args):
    """--impl reference: the CPU oracle, as it stands, on the host cores (rank 0 only).  Nothing of the CUDA
    library is loaded: the byte numerator is the format's own count (2.5 bytes per stored entry of the surviving
    columns from the oracle encoder's block pointers, two pointer words per surviving column, x, the list, y)."""
    if int(os.environ.get("RANK", "0")) != 0:
        return
    from oracle import celty_oracle as orc
    name = args.workload
    M, K, s, family, dist, d_a, cfg = WORKLOADS[name]
    W, mask = make_layer(name, 0)
    x, tau = make_x(name, 0)
    threads = orc.max_threads()
    t0 = time.perf_counter()
    orc.masked_gemv(W, mask, x, tau, threads=threads)
    t_full = time.perf_counter() - t0
    # rows sampled per step so that warmup + steps stay within about two minutes
    frac = min(1.0, 100.0 / max(1e-9, (args.steps + args.warmup) * t_full))
    rows = max(1, int(M * frac))
    Ws, ms = np.ascontiguousarray(W[:rows]), np.ascontiguousarray(mask[:rows])
    for _ in range(args.warmup):
        orc.masked_gemv(Ws, ms, x, tau, threads=threads)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        orc.masked_gemv(Ws, ms, x, tau, threads=threads)
    dt = (time.perf_counter() - t0) / args.steps
    sec_per_call = dt * (M / rows)
    idx = orc.compact(x, tau)[0]
    ptr = orc.rlc_count(np.ascontiguousarray(mask[:, idx]), 4, 0)
    total_bytes = 2.5 * float(ptr[-1]) + 8.0 * idx.size + 2.0 * K + 6.0 * idx.size + 4.0 * M
    gbs = total_bytes / sec_per_call / 1e9
    sample = f"rows 0..{rows - 1} of {M} per step, scaled to a full call"
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": gbs, "unit": "GB/s", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": sec_per_call * 1e3,
        "us_per_call": sec_per_call * 1e6, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f64", "data": "synthetic",
        "config": workload_config(name),
        "bytes_per_call": {"bare_format": total_bytes},
        "cpu_baseline": {"value": gbs, "unit": "GB/s", "cores": threads, "kind": "oracle", "sample": sample},
        "e2e": {"value": gbs, "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


# ----------------------------------------------------------------------------- sweeps (documentation runs)
SWEEPS = {
    # config 1: the small single layer (latency-bound; microseconds are the figure that means something)
    "cfg1": [dict(M=1024, K=1024, s=0.5, family="bernoulli", dist="normal", d_a=0.5, cfg=1)],
    # config 2: 4096 x 4096, magnitude-pruned, all 9 (weight sparsity, activation density) pairs
    "cfg2": [dict(M=4096, K=4096, s=s, family="magnitude", dist="laplace", d_a=d, cfg=2)
             for s in (0.3, 0.5, 0.7) for d in (0.7, 0.5, 0.3)],
    # config 3: Llama-2-7B MLP shapes
    "cfg3": [dict(M=11008, K=4096, s=0.5, family="magnitude", dist="laplace", d_a=0.5, cfg=3),
             dict(M=4096, K=11008, s=0.5, family="magnitude", dist="swiglu", d_a=0.5, cfg=3)],
    # config 4: the three shapes of a Llama-2-13B decode layer (q/k/v/o, gate/up, down)
    "cfg4": [dict(M=5120, K=5120, s=0.5, family="bernoulli", dist="laplace", d_a=0.4, cfg=4),
             dict(M=13824, K=5120, s=0.5, family="bernoulli", dist="laplace", d_a=0.4, cfg=4),
             dict(M=5120, K=13824, s=0.5, family="bernoulli", dist="laplace", d_a=0.4, cfg=4)],
    # config 5: Llama-70B-shaped MLP, sparsity x density x mask family
    "cfg5": [dict(M=M, K=K, s=s, family=f, dist="laplace", d_a=d, cfg=5)
             for (M, K) in ((28672, 8192), (8192, 28672)) for f in ("bernoulli", "powerlaw")
             for s in (0.3, 0.5, 0.7) for d in (0.1, 0.3, 0.5, 0.7)],
}


def run_sweep(args):
    """Times every point of one configured sweep with the protocol of the main run: calls rotate over enough
    device copies of the layer to exceed 2x L2 (every call finds its matrix cold), one rotation is captured in
    a CUDA graph, and CUDA events bracket several replays.  The dense cuBLAS GEMV is timed the same way."""
    import torch
    from paper_2608_01536_b200 import build as lib_build, celty
    lib_build.build()
    celty.load()
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    peak, _ = measured_peaks()
    l2 = torch.cuda.get_device_properties(dev).L2_cache_size

    def rotation_us(calls):
        for f in calls:
            f()
        torch.cuda.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g):
            for f in calls:
                f()
        g.replay()
        torch.cuda.synchronize()
        reps = max(3, -(-args.sweep_calls // len(calls)))
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        for _ in range(reps):
            g.replay()
        b.record()
        torch.cuda.synchronize()
        return a.elapsed_time(b) * 1e3 / (reps * len(calls))

    points, key, mats, dense, dense_t = [], None, [], [], []
    for i, pt in enumerate(SWEEPS[args.sweep]):
        M, K, s, fam = pt["M"], pt["K"], pt["s"], pt["family"]
        if key != (M, K, s, fam):                              # one layer on the device at a time
            key = (M, K, s, fam)
            mats, dense, dense_t = [], [], []
            seed = synth.point_seed(pt["cfg"], 0)
            W = synth.weights_tiled(seed, M, K, K // 8) if M * K > (1 << 26) else synth.weights(seed, M, K)
            mask = (synth.mask_magnitude(W, s) if fam == "magnitude" else
                    synth.mask_bernoulli(seed, M, K, 1.0 - s) if fam == "bernoulli" else
                    synth.mask_powerlaw(seed, M, K, 1.0 - s))
            mats.append(celty.Matrix(W, mask, device=dev))
            copies = int(np.ceil(2.5 * l2 / mats[0].device_bytes()[0])) + 1
            while len(mats) < copies:
                mats.append(mats[0].clone(device=dev))
            Wm = torch.from_numpy(np.where(mask != 0, W, np.float16(0)))
            dense = [Wm.to(dev) for _ in range(min(copies, int(np.ceil(2.5 * l2 / (2 * M * K))) + 1))]
            dense_t = [w.t().contiguous() for w in dense]
            del W, mask, Wm
        copies = len(mats)
        xs, taus = [], []
        for c in range(copies):
            x = synth.activations(synth.point_seed(pt["cfg"], 50 + 16 * i + c), K, pt["dist"])
            taus.append(synth.threshold_for_density(x, pt["d_a"]))
            xs.append(torch.from_numpy(x).to(dev))
        ys = [torch.empty(M, dtype=torch.float32, device=dev) for _ in range(copies)]
        yd = torch.empty(M, dtype=torch.float16, device=dev)
        fetched, survivors = [], []
        for c in range(copies):
            mats[c].spmspv(xs[c], taus[c], ys[c])
            idx, _ = mats[c].last_compaction()
            assert mats[c].last_status() == 0
            fetched.append(mats[c].fetched_bytes(idx.cpu().numpy())[1])
            survivors.append(int(idx.numel()))
        tb = float(np.mean(fetched))
        us = rotation_us([(lambda c=c: mats[c].spmspv(xs[c], taus[c], ys[c])) for c in range(copies)])
        dus = min(rotation_us([(lambda c=c: torch.mv(dense[c % len(dense)], xs[c], out=yd)) for c in range(copies)]),
                  rotation_us([(lambda c=c: torch.mv(dense_t[c % len(dense_t)].t(), xs[c], out=yd)) for c in range(copies)]))
        info = mats[0].info()
        points.append({"M": M, "K": K, "weight_sparsity": s, "mask": fam, "activation_density": pt["d_a"],
                       "combined_sparsity": 1.0 - (1.0 - s) * pt["d_a"], "device_copies": copies,
                       "survivors": float(np.mean(survivors)), "stored_entries": info.nnz + info.n_pad,
                       "pads": info.n_pad, "fetched_bytes": tb, "us_per_call": us, "GBps": tb / us / 1e3,
                       "roofline_frac": tb / us / 1e3 / peak, "roofline_frac_of_nominal_8000": tb / us / 1e3 / 8000.0,
                       "dense_equivalent_GBps": 2.0 * M * K / us / 1e3, "realised_weight_density": info.nnz / (M * K),
                       "realised_activation_density": float(np.mean(survivors)) / K,
                       "cublas_gemv_us": dus, "speedup_vs_cublas": dus / us})
        print(json.dumps(points[-1]), file=sys.stderr, flush=True)
    extra = {}
    if args.sweep == "cfg4":
        # the decode-layer chain of config 4: q, k, v, o (5120 x 5120), gate, up (13824 x 5120), down (5120 x 13824),
        # 7 calls back to back on one stream, each with its own matrix and its own synthetic x; two layers in
        # rotation (about 0.8 GB of compressed weights, far beyond L2)
        del mats, dense, dense_t
        def chain(shapes, tag):
            calls, dcalls, tot_bytes = [], [], 0.0
            for layer in range(2):
                for k, (M, K) in enumerate(shapes):
                    seed = synth.point_seed(4, 10 * layer + k + (100 if tag == "stacked" else 0))
                    W = synth.weights(seed, M, K)
                    mask = synth.mask_bernoulli(seed, M, K, 0.5)
                    m = celty.Matrix(W, mask, device=dev)
                    x = synth.activations(synth.point_seed(4, 200 + 10 * layer + k), K, "laplace")
                    tau = synth.threshold_for_density(x, 0.4)
                    xd = torch.from_numpy(x).to(dev)
                    y = torch.empty(M, dtype=torch.float32, device=dev)
                    m.spmspv(xd, tau, y)
                    idx, _ = m.last_compaction()
                    assert m.last_status() == 0
                    tot_bytes += m.fetched_bytes(idx.cpu().numpy())[1]
                    calls.append(lambda m=m, xd=xd, tau=tau, y=y: m.spmspv(xd, tau, y))
                    Wd = torch.from_numpy(np.where(mask != 0, W, np.float16(0))).to(dev)
                    yd = torch.empty(M, dtype=torch.float16, device=dev)
                    dcalls.append(lambda Wd=Wd, xd=xd, yd=yd: torch.mv(Wd, xd, out=yd))
            us = rotation_us(calls) * len(shapes)
            dus = rotation_us(dcalls) * len(shapes)
            return {"calls_per_layer": len(shapes), "layers_in_rotation": 2, "us_per_layer": us,
                    "fetched_bytes_per_layer": tot_bytes / 2, "GBps": tot_bytes / 2 / us / 1e3,
                    "roofline_frac": tot_bytes / 2 / us / 1e3 / peak, "cublas_gemv_us_per_layer": dus,
                    "speedup_vs_cublas": dus / us}
        # 7 calls per layer, each product its own matrix
        extra["chain"] = chain([(5120, 5120)] * 4 + [(13824, 5120)] * 2 + [(5120, 13824)], "separate")
        # the same layer with the products that share an input stacked row-wise into one matrix ([q; k; v] and
        # [gate; up]): 4 calls per layer, one thresholding pass per shared x, for the sparse and the dense side alike
        extra["chain_stacked"] = chain([(15360, 5120), (5120, 5120), (27648, 5120), (5120, 13824)], "stacked")

        # the stacked layer with the work between the products inside the launches: FP16 outputs, SiLU(gate) * up and
        # its thresholded list behind the gate/up product, the down projection fed from that list (no thresholding
        # pass of its own).  The dense side runs the four GEMVs and the element-wise step as its own kernel.
        def chain_fused(consumer_side):
            H, I = 5120, 13824
            calls, dcalls, tot_bytes = [], [], 0.0
            for layer in range(2):
                mats, Wds = [], []
                for k, (M, K) in enumerate([(3 * H, H), (H, H), (2 * I, H), (H, I)]):
                    seed = synth.point_seed(4, 10 * layer + k + 100)
                    W = synth.weights(seed, M, K)
                    mask = synth.mask_bernoulli(seed, M, K, 0.5)
                    mats.append(celty.Matrix(W, mask, device=dev))
                    Wds.append(torch.from_numpy(np.where(mask != 0, W, np.float16(0))).to(dev))
                xs = [torch.from_numpy(synth.activations(synth.point_seed(4, 200 + 10 * layer + k), H, "laplace")).to(dev)
                      for k in range(3)]
                taus = [synth.threshold_for_density(x.cpu().numpy(), 0.4) for x in xs]
                ys = [torch.empty(m.M, dtype=torch.float32, device=dev) for m in mats]
                y16 = [torch.empty(m.M, dtype=torch.float16, device=dev) for m in mats]
                out = celty.SwigluOut(I, 0.0, dev)
                hbuf = torch.empty(I, dtype=torch.float32, device=dev)
                mats[2].spmspv_ex(xs[2], taus[2], ys[2], swiglu=out)        # once, to place the list's threshold
                torch.cuda.synchronize()
                out.tau = synth.threshold_for_density(out.h.cpu().numpy(), 0.4)

                def sparse_layer(mats=mats, xs=xs, taus=taus, ys=ys, y16=y16, out=out, hbuf=hbuf):
                    if consumer_side == "kernel":                       # nothing fused: the step is a kernel between the calls
                        mats[0].spmspv(xs[0], taus[0], ys[0])
                        mats[1].spmspv(xs[1], taus[1], ys[1])
                        mats[2].spmspv(xs[2], taus[2], ys[2])
                        torch.mul(torch.nn.functional.silu(ys[2][:I]), ys[2][I:], out=hbuf)
                        out.h.copy_(hbuf)
                        mats[3].spmspv(out.h, out.tau, ys[3])
                        return
                    if consumer_side:
                        mats[0].spmspv(xs[0], taus[0], ys[0])
                        mats[1].spmspv(xs[1], taus[1], ys[1])
                        mats[2].spmspv(xs[2], taus[2], ys[2])
                        mats[3].spmspv_swiglu(ys[2], out.tau, ys[3], h_out=out.h)
                        return
                    mats[0].spmspv_ex(xs[0], taus[0], ys[0], fp16_out=y16[0])
                    mats[1].spmspv_ex(xs[1], taus[1], ys[1], fp16_out=y16[1])
                    mats[2].spmspv_ex(xs[2], taus[2], ys[2], swiglu=out)
                    mats[3].spmspv_list(out.idx, out.val, out.count, ys[3], fp16_out=y16[3])
                sparse_layer()
                torch.cuda.synchronize()
                assert all(m.last_status() == 0 for m in mats)
                for k in range(3):
                    idx, _ = mats[k].last_compaction()
                    tot_bytes += mats[k].fetched_bytes(idx.cpu().numpy())[1]
                if consumer_side:
                    tot_bytes += mats[3].fetched_bytes(mats[3].last_compaction()[0].cpu().numpy())[1] + 6 * I
                else:
                    n = int(out.count.item())
                    tot_bytes += mats[3].fetched_bytes(np.sort(out.idx[:n].cpu().numpy()))[1]
                calls.append(sparse_layer)
                yd = [torch.empty(m.M, dtype=torch.float16, device=dev) for m in mats]
                hd = torch.empty(I, dtype=torch.float16, device=dev)

                def dense_layer(Wds=Wds, xs=xs, yd=yd, hd=hd):
                    torch.mv(Wds[0], xs[0], out=yd[0])
                    torch.mv(Wds[1], xs[1], out=yd[1])
                    torch.mv(Wds[2], xs[2], out=yd[2])
                    torch.mul(torch.nn.functional.silu(yd[2][:I]), yd[2][I:], out=hd)
                    torch.mv(Wds[3], hd, out=yd[3])
                dcalls.append(dense_layer)
            us = rotation_us(calls)
            dus = rotation_us(dcalls)
            return {"calls_per_layer": 4, "layers_in_rotation": 2, "us_per_layer": us,
                    "fetched_bytes_per_layer": tot_bytes / 2, "GBps": tot_bytes / 2 / us / 1e3,
                    "roofline_frac": tot_bytes / 2 / us / 1e3 / peak, "cublas_gemv_us_per_layer": dus,
                    "speedup_vs_cublas": dus / us,
                    "note": ("plain products and a separate element-wise kernel (PyTorch) between gate/up and down"
                             if consumer_side == "kernel" else "plain products; the down projection makes SiLU(gate)*up from the FP32 gate/up result while it "
                             "thresholds" if consumer_side else
                             "FP16 outputs, SiLU(gate)*up and its list inside the gate/up launch, down projection from "
                             "the list") + "; the dense side adds the element-wise step as a kernel of its own"}
        extra["chain_stacked_fused"] = chain_fused(False)
        extra["chain_stacked_separate_step"] = chain_fused("kernel")
        extra["chain_stacked_swiglu_in_down"] = chain_fused(True)
    print(json.dumps({"sweep": args.sweep, "protocol": "rotation over device copies of the layer (> 2x L2) captured in one "
                      "CUDA graph, CUDA events around the replays", "peak_GBps": peak, "points": points, **extra}))


def run_format_study(args):
    """Compression efficiency against weight sparsity (the paper's Figure 3 question, on synthetic Bernoulli
    masks): bytes of the 4-bit run-length format as the library's host encoder writes it, for the whole-column
    layout and for the lane-tile device image, beside the closed form 1.25 * d * (1 + rho) (rho = pads per
    nonzero = s^16 / (1 - s^16)) and a bitmap format's d + 1/16; and the entry counts at run widths of 2 to 8 bits
    (celty_count_entries), which show where the paper's 4 bits sit.  Host only: no GPU is needed."""
    from paper_2608_01536_b200 import build as lib_build, celty
    lib_build.build()
    celty.load()
    M, K = 4096, 1024
    rows = []
    for s in (0.1, 0.2, 0.3, 0.4, 0.5, 0.6, 0.7, 0.8, 0.9, 0.95):
        seed = synth.point_seed(2, 900 + int(round(s * 100)))
        W = synth.weights(seed, M, K)
        mask = synth.mask_bernoulli(seed, M, K, 1.0 - s)
        dense_bytes = 2.0 * M * K
        out = {"weight_sparsity": s}
        for name, layout in (("column", celty.LAYOUT_COLUMN), ("lane_tile", celty.LAYOUT_LANE_TILE)):
            m = celty.Matrix(W, mask, layout=layout)
            info = m.info()
            out[name] = {"image_over_dense": m.device_bytes()[0] / dense_bytes,
                         "entries_over_dense": 2.5 * (info.nnz + info.n_pad) / dense_bytes,
                         "pads_per_nonzero": info.n_pad / max(1, info.nnz)}
            out["realised_density"] = info.nnz / (M * K)
        d = 1.0 - s
        rho = s ** 16 / (1.0 - s ** 16)
        out["closed_form_rlc4"] = 1.25 * d * (1.0 + rho)
        # the same question for other run widths n (why 4 bits?): entries counted by the library at width n,
        # (2 + n / 8) bytes each, beside the closed form d * (1 + s^L / (1 - s^L)) * (2 + n / 8) / 2, L = 2^n
        out["run_width"] = {}
        for n in (2, 3, 4, 5, 6, 8):
            nnz, pads = celty.count_entries(mask, n)
            L = 2 ** n
            out["run_width"][str(n)] = {"entries_over_dense": (2.0 + n / 8.0) * (nnz + pads) / dense_bytes,
                                        "pads_per_nonzero": pads / max(1, nnz),
                                        "closed_form": d * (1.0 + s ** L / (1.0 - s ** L)) * (2.0 + n / 8.0) / 2.0}
        out["best_run_width"] = min(out["run_width"], key=lambda k: out["run_width"][k]["entries_over_dense"])
        out["closed_form_bitmap"] = d + 1.0 / 16.0
        rows.append(out)
        print(json.dumps(out), file=sys.stderr, flush=True)
    print(json.dumps({"sweep": "format", "M": M, "K": K, "mask": "bernoulli", "points": rows}))


def run_knob_study(args):
    """Launch-parameter study (the paper's Figure 11 question -- how far to split the columns -- asked of this
    kernel): time of one workload against the number of thread blocks (column slices = blocks / row parts),
    warp teams per block, ring depth and thread blocks per cluster, everything else the library's choice.  Same protocol as
    the sweeps: rotation over device copies beyond 2x L2, one CUDA graph, CUDA events."""
    import torch
    from paper_2608_01536_b200 import build as lib_build, celty
    lib_build.build()
    celty.load()
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    l2 = torch.cuda.get_device_properties(dev).L2_cache_size
    sms = torch.cuda.get_device_properties(dev).multi_processor_count
    name = args.workload
    W, mask = make_layer(name, 0)
    first = celty.Matrix(W, mask, device=dev)
    copies = int(np.ceil(2.5 * l2 / first.device_bytes()[0])) + 1
    mats = [first] + [first.clone(device=dev) for _ in range(copies - 1)]
    xs, taus = [], []
    for c in range(copies):
        x, tau = make_x(name, c)
        xs.append(torch.from_numpy(x).to(dev))
        taus.append(tau)
    ys = [torch.empty(W.shape[0], dtype=torch.float32, device=dev) for _ in range(copies)]
    S = first.row_map()[0]

    def timed(**kn):
        for m in mats:
            m.set_launch(**kn)
        calls = [(lambda c=c: mats[c].spmspv(xs[c], taus[c], ys[c])) for c in range(copies)]
        for f in calls:
            f()
        torch.cuda.synchronize()
        if any(m.last_status() != 0 for m in mats):
            return None
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g):
            for f in calls:
                f()
        g.replay()
        torch.cuda.synchronize()
        reps = max(3, -(-args.sweep_calls // copies))
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        for _ in range(reps):
            g.replay()
        b.record()
        torch.cuda.synchronize()
        return a.elapsed_time(b) * 1e3 / (reps * copies)

    points = []
    def add(knob, value, **kn):
        try:
            us = timed(**kn)
        except celty.CeltyError as e:                       # a setting that does not fit the device is refused
            us = None
            print(f"{knob}={value}: {e}", file=sys.stderr)
        points.append({"knob": knob, "value": value, "us_per_call": us})
        print(json.dumps(points[-1]), file=sys.stderr, flush=True)

    add("default", 0)
    for grid in sorted({max(S, sms // 8), max(S, sms // 4), max(S, sms // 2), max(S, 3 * sms // 4), sms}):
        add("grid", grid, grid=grid)
    for groups in (1, 2, 4, 6, 8):
        add("groups", groups, groups=groups)
    for depth in (2, 3, 4):
        add("depth", depth, depth=depth)
    for cluster in (1, 2, 4):
        add("cluster", cluster, cluster=cluster)
    for name_, bit in (("never", 32), ("always", 16)):              # two warps per team taking turns at its accumulator
        add("pairs", name_, variant=bit)
    add("spare_blocks", "not shared", variant=64)                  # left-over blocks given whole to the first row parts
    for m in mats:
        m.set_launch()
    print(json.dumps({"sweep": "knobs", "workload": name, "row_parts": int(S), "device_copies": copies,
                      "points": points}))


def pick_copies(needed: int, steps: int) -> int:
    """Device copies in the rotation: the smallest count >= needed that divides `steps` (so that every timed
    region of `steps` calls walks the rotation a whole number of times and a copy is never reused early);
    `needed` itself when no divisor is close."""
    for c in range(needed, 2 * needed + 5):
        if steps % c == 0:
            return c
    return needed


def graph_unit(copies: int, steps: int, cap: int = 256) -> int:
    """Calls held by the CUDA graph: a whole number of rotations, at most `cap` calls, dividing `steps` when
    the rotation does (the timed region is then whole replays and nothing else)."""
    if steps % copies:
        return steps if steps <= 4 * cap else copies
    rotations = steps // copies
    k = max(1, min(rotations, cap // copies))
    while rotations % k:
        k -= 1
    return copies * k


class Workload:
    """One configured layer resident `copies` times on the device (every copy its own activation vector), the
    CUDA graph that walks the rotation, and the byte accounting of a call."""

    def __init__(self, name, dev, args, steps, celty, torch):
        self.name = name
        M, K, s, family, dist_name, d_a, cfg = WORKLOADS[name]
        self.M, self.K = M, K
        layout = celty.LAYOUT_COLUMN if args.layout == "column" else celty.LAYOUT_LANE_TILE
        self.l2 = torch.cuda.get_device_properties(dev).L2_cache_size
        distinct_n = max(1, min(args.distinct, 1 if M * K > (1 << 26) else args.distinct))
        self.distinct = [make_layer(name, v) for v in range(distinct_n)]
        base = [celty.Matrix(W, mask, layout=layout, tile_rows=args.tile_rows) for W, mask in self.distinct]
        self.image_bytes = base[0].device_bytes()[0]
        needed = max(distinct_n, int(np.ceil(2.5 * self.l2 / self.image_bytes)) + 1)
        self.copies = args.copies if args.copies else pick_copies(needed, steps)
        self.mats, self.xs, self.taus = [], [], []
        for c in range(self.copies):
            m = base[c % distinct_n] if c < distinct_n else base[c % distinct_n].clone()
            m.to(dev)
            if args.grid or args.variant or args.groups or args.depth or args.cluster:
                m.set_launch(args.grid, args.variant, args.groups, args.depth, args.cluster)
            x, tau = make_x(name, c)
            self.mats.append(m)
            self.xs.append(torch.from_numpy(x).to(dev))
            self.taus.append(tau)
        self.ys = [torch.empty(M, dtype=torch.float32, device=dev) for _ in range(self.copies)]
        torch.cuda.synchronize()
        # bytes per call: host arithmetic on the library's tables, from the list the call itself produced
        fetched, entries, self.survivors = [], [], []
        for c in range(self.copies):
            self.call(c)
            idx, _ = self.mats[c].last_compaction()
            assert self.mats[c].last_status() == 0
            idx = idx.cpu().numpy()
            fetched.append(self.mats[c].fetched_bytes(idx))
            entries.append(self.mats[c].stored_entries(idx))
            self.survivors.append(int(idx.size))
        self.stream_bytes = float(np.mean([f[0] for f in fetched]))
        self.total_bytes = float(np.mean([f[1] for f in fetched]))
        n = float(np.mean(self.survivors))
        # the format's own bytes: 2.5 per stored entry of the surviving columns, two offset words per column,
        # x read, the list written, y written -- no alignment padding, no per-block headers
        self.bare_bytes = 2.5 * float(np.mean(entries)) + 8 * n + 2 * K + 6 * n + 4 * M
        self.info = self.mats[0].info()
        self.layout_stats = self.mats[0].layout_stats() if layout == celty.LAYOUT_LANE_TILE else None
        self.graph = None
        self.unit = None

    def call(self, c):
        self.mats[c].spmspv(self.xs[c], self.taus[c], self.ys[c])

    def capture(self, torch, steps):
        self.unit = graph_unit(self.copies, steps)
        self.graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(self.graph):
            for i in range(self.unit):
                self.call(i % self.copies)
        for _ in range(2):
            self.graph.replay()
        torch.cuda.synchronize()


def timed_regions(torch, replay, replays_per_region, min_regions=10, min_total_s=0.25, max_regions=400):
    """CUDA-event time (ms) of regions of `replays_per_region` graph replays each.  An untimed replay is queued
    directly ahead of every region, so the opening event is taken while the device is busy and the first timed
    kernel starts behind it without a launch gap; the regions are independent samples of the same K steps."""
    times = []
    t0 = time.perf_counter()
    while len(times) < min_regions or (time.perf_counter() - t0 < min_total_s and len(times) < max_regions):
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        replay()
        a.record()
        for _ in range(replays_per_region):
            replay()
        b.record()
        b.synchronize()
        times.append(a.elapsed_time(b))
    return times


def dense_gemv_us(torch, wl, dev, steps):
    """Dense cuBLAS FP16 GEMV on the same masked weights under the same rotation: W row-major (M x K) and its
    transpose stored row-major (K x M); microseconds per call of each."""
    out = {}
    n_dense = max(2, int(np.ceil(2.5 * wl.l2 / (2.0 * wl.M * wl.K))) + 1)
    Wm = [torch.from_numpy(np.where(mask != 0, W, np.float16(0))) for W, mask in wl.distinct]
    base = [w.to(dev) for w in Wm]
    for transposed in (False, True):
        Wd = [base[c % len(base)].clone() for c in range(n_dense)]
        if transposed:
            Wd = [w.t().contiguous() for w in Wd]
        op = (lambda w, x, o: torch.mv(w.t(), x, out=o)) if transposed else (lambda w, x, o: torch.mv(w, x, out=o))
        yd = torch.empty(wl.M, dtype=torch.float16, device=dev)
        op(Wd[0], wl.xs[0], yd)
        torch.cuda.synchronize()
        unit = n_dense * max(1, min(64, steps) // n_dense)
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g):
            for i in range(unit):
                op(Wd[i % n_dense], wl.xs[i % wl.copies], yd)
        g.replay()
        torch.cuda.synchronize()
        reps = max(1, steps // unit)
        out["transposed_KxM" if transposed else "row_major_MxK"] = \
            float(np.median(timed_regions(torch, g.replay, reps, min_total_s=0.1))) * 1e3 / (reps * unit)
        del Wd, g
    return out


def dram_traffic_per_launch(name):
    """dram__bytes_read.sum + dram__bytes_write.sum of one launch of the fused kernel on this workload, from the
    profiler capture summarised under profiles/ (kept as data next to the summaries); None when there is none."""
    path = os.path.join(ROOT, "profiles", "dram_traffic.json")
    try:
        with open(path) as f:
            return json.load(f).get(name, {}).get("dram_bytes_per_launch")
    except OSError:
        return None


def run_regsplit_study(args):
    """Register / shared-memory accumulation split (the question of the paper's Figure 13, asked of the software
    analogue celty_set_register_rows): microseconds per call against the number of local rows per lane that are
    summed in registers, at 30 / 50 / 70 % of the weights pruned, on 5120 x 5120 and 28672 x 8192 (Bernoulli masks,
    50 % of the activations kept).  Rows = 0 is the library's kernel; the line "0 (8 teams)" is that kernel held to
    the eight teams the register builds can run, so that the split is compared at equal parallelism."""
    import torch
    from paper_2608_01536_b200 import build as lib_build, celty
    lib_build.build()
    celty.load()
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    l2 = torch.cuda.get_device_properties(dev).L2_cache_size
    points = []
    for (M, K) in ((5120, 5120), (28672, 8192)):
        for s in (0.3, 0.5, 0.7):
            seed = synth.point_seed(5, 700 + int(s * 100))
            W = synth.weights_tiled(seed, M, K, K // 8) if M * K > (1 << 26) else synth.weights(seed, M, K)
            mask = synth.mask_bernoulli(seed, M, K, 1.0 - s)
            first = celty.Matrix(W, mask, device=dev)
            copies = int(np.ceil(2.5 * l2 / first.device_bytes()[0])) + 1
            mats = [first] + [first.clone(device=dev) for _ in range(copies - 1)]
            xs, taus = [], []
            for c in range(copies):
                x = synth.activations(synth.point_seed(5, 750 + c), K, "laplace")
                taus.append(synth.threshold_for_density(x, 0.5))
                xs.append(torch.from_numpy(x).to(dev))
            ys = [torch.empty(M, dtype=torch.float32, device=dev) for _ in range(copies)]
            R = first.row_map()[1]
            for label, rows, groups in (("0", 0, 0), ("0 (8 teams)", 0, 8), ("32", 32, 0), ("64", 64, 0), ("96", 96, 0),
                                        ("128", 128, 0)):
                for m in mats:
                    m.set_register_rows(rows)
                    m.set_launch(groups=groups)
                calls = [(lambda c=c: mats[c].spmspv(xs[c], taus[c], ys[c])) for c in range(copies)]
                for f in calls:
                    f()
                torch.cuda.synchronize()
                assert all(m.last_status() == 0 for m in mats)
                g = torch.cuda.CUDAGraph()
                with torch.cuda.graph(g):
                    for f in calls:
                        f()
                g.replay()
                reps = max(3, -(-args.sweep_calls // copies))
                us = float(np.median(timed_regions(torch, g.replay, reps, min_total_s=0.05))) * 1e3 / (reps * copies)
                plan = mats[0].launch_plan()
                points.append({"M": M, "K": K, "weight_sparsity": s, "tile_rows": R, "register_rows": label,
                               "share_of_rows_in_registers": min(1.0, rows / R), "us_per_call": us,
                               "teams": plan["teams_per_slab"], "threads": plan["threads"]})
                print(json.dumps(points[-1]), file=sys.stderr, flush=True)
            del mats, first
    print(json.dumps({"sweep": "regsplit", "points": points}))


def run_batch_study(args):
    """Small batches (Sections 2.2-2.3 place the method against SpMM kernels that need N >= 8): microseconds per
    batch of N activation vectors through celty_spmspv_batch with the widened kernels (union of the surviving columns,
    N accumulators per row; two launches) and as the library runs it by default, beside N calls of the single-vector kernel and the dense cuBLAS FP16 GEMM
    on the same weights, under the same rotation."""
    import torch
    from paper_2608_01536_b200 import build as lib_build, celty
    lib_build.build()
    celty.load()
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    l2 = torch.cuda.get_device_properties(dev).L2_cache_size
    points = []
    for name in ("llama7b_attn_4096x4096_s50_a50", "llama7b_gateup_11008x4096_s50_a50"):
        M, K, s, family, dist_name, d_a, cfg = WORKLOADS[name]
        W, mask = make_layer(name, 0)
        first = celty.Matrix(W, mask, device=dev)
        copies = int(np.ceil(2.5 * l2 / first.device_bytes()[0])) + 1
        mats = [first] + [first.clone(device=dev) for _ in range(copies - 1)]
        Wd = [torch.from_numpy(np.where(mask != 0, W, np.float16(0))).to(dev) for _ in range(min(copies, int(np.ceil(2.5 * l2 / (2 * M * K))) + 1))]
        for N in (1, 2, 4, 8):
            X = np.stack([make_x(name, 10 * c + n)[0] for c in range(copies) for n in range(N)]).reshape(copies, N, K)
            tau = make_x(name, 0)[1]
            xs = [torch.from_numpy(X[c]).to(dev) for c in range(copies)]
            ys = [torch.empty(N, M, dtype=torch.float32, device=dev) for _ in range(copies)]
            yd = torch.empty(M, N, dtype=torch.float16, device=dev)

            def timed(calls):
                for f in calls:
                    f()
                torch.cuda.synchronize()
                g = torch.cuda.CUDAGraph()
                with torch.cuda.graph(g):
                    for f in calls:
                        f()
                g.replay()
                reps = max(3, -(-args.sweep_calls // len(calls)))
                return float(np.median(timed_regions(torch, g.replay, reps, min_total_s=0.05))) * 1e3 / (reps * len(calls))
            for mt in mats:
                mt.set_launch(variant=1)                              # the widened two-launch kernels
            us_batch = timed([(lambda c=c: mats[c].spmspv_batch(xs[c], tau, ys[c])) for c in range(copies)])
            for mt in mats:
                mt.set_launch()
            us_default = timed([(lambda c=c: mats[c].spmspv_batch(xs[c], tau, ys[c])) for c in range(copies)])
            us_single = timed([(lambda c=c, n=n: mats[c].spmspv(xs[c][n], tau, ys[c][n])) for c in range(copies) for n in range(N)]) * N
            us_gemm = timed([(lambda c=c: torch.mm(Wd[c % len(Wd)], xs[c].t(), out=yd)) for c in range(copies)])
            keep = [np.abs(X[c].astype(np.float32)) > np.float32(tau) for c in range(copies)]
            points.append({"workload": name, "N": N, "us_per_batch": us_batch, "us_per_batch_default": us_default,
                           "us_N_single_calls": us_single,
                           "us_cublas_gemm": us_gemm,
                           "union_density": float(np.mean([k.any(axis=0).mean() for k in keep])),
                           "activation_density": float(np.mean([k.mean() for k in keep]))})
            print(json.dumps(points[-1]), file=sys.stderr, flush=True)
        del mats, first, Wd
    print(json.dumps({"sweep": "batch", "points": points}))


def run_celty(args):
    import torch
    import torch.distributed as dist
    from paper_2608_01536_b200 import build as lib_build, celty

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    assert torch.cuda.is_available(), "bench.py needs a CUDA device; there is no CPU fallback"
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    lib_build.build()
    celty.load()
    dev = torch.device("cuda", local)
    name = args.workload
    M, K, s, family, dist_name, d_a, cfg = WORKLOADS[name]
    steps = args.steps
    warmup = max(3, args.warmup)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    wl = Workload(name, dev, args, steps, celty, torch)
    for i in range(warmup):
        wl.call(i % wl.copies)
    torch.cuda.synchronize()
    if args.no_graph:
        def replay():
            for i in range(steps):
                wl.call(i % wl.copies)
        per_region = 1
    else:
        wl.capture(torch, steps)
        replay, per_region = wl.graph.replay, max(1, steps // wl.unit)
    calls_per_region = steps if args.no_graph else per_region * wl.unit

    # ---- the timed region: K steps as whole graph replays between two CUDA events, taken several times over;
    # the median region is the figure, the fastest and the count are reported beside it
    with ClockSampler(local) as clocks:
        barrier()
        regions = timed_regions(torch, replay, per_region)
        barrier()
    ms = max_over_ranks(float(np.median(regions)), dev)
    sec_per_call = ms / 1e3 / calls_per_region
    gbs = aggregate_throughput(wl.total_bytes, world, sec_per_call)

    # ---- context: stream-enqueued calls (no graph) and the L2-warm figure
    def time_calls(fn, n):
        torch.cuda.synchronize()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        for i in range(n):
            fn(i)
        b.record()
        torch.cuda.synchronize()
        return a.elapsed_time(b) / n * 1e3
    n_ctx = int(min(max(steps, 200), 2000))
    us_enqueued = time_calls(lambda i: wl.call(i % wl.copies), n_ctx)
    gw = torch.cuda.CUDAGraph()
    with torch.cuda.graph(gw):
        for _ in range(16):
            wl.call(0)
    gw.replay()
    us_warm = float(np.median(timed_regions(torch, gw.replay, 4, min_total_s=0.05))) * 1e3 / 64

    # ---- end to end through the host-buffer entry point: pinned x in, y out, every step
    xh = [torch.from_numpy(make_x(name, c)[0]).pin_memory() for c in range(wl.copies)]
    yh = torch.empty(M, dtype=torch.float32).pin_memory()
    xstage = torch.empty(K, dtype=torch.float16, device=dev)
    n_e2e = int(min(max(steps, 200), 2000))
    for i in range(5):
        wl.mats[i % wl.copies].spmspv_host(xh[i % wl.copies], wl.taus[i % wl.copies], yh, xstage, wl.ys[0])
    barrier()
    t0 = time.perf_counter()
    for i in range(n_e2e):
        c = i % wl.copies
        wl.mats[c].spmspv_host(xh[c], wl.taus[c], yh, xstage, wl.ys[0])
    barrier()
    e2e_sec = max_over_ranks((time.perf_counter() - t0) / n_e2e, dev)

    # ---- one isolated call, host timer around call + synchronize (launch and sync latency included)
    iso = []
    for i in range(50):
        c = i % wl.copies
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        wl.call(c)
        torch.cuda.synchronize()
        iso.append((time.perf_counter() - t0) * 1e6)
    us_isolated = float(np.median(iso))

    # ---- dense cuBLAS GEMV on the same GPU under the same rotation: the better weight layout is quoted
    dense_both = None if args.no_dense else dense_gemv_us(torch, wl, dev, steps)
    dense_us = min(dense_both.values()) if dense_both else None

    # ---- a second, labelled figure: the Llama-2-7B attention shape (latency-bound), same protocol
    secondary = None
    if not args.no_secondary and name != SECONDARY_WORKLOAD and world == 1:
        w2 = Workload(SECONDARY_WORKLOAD, dev, args, 240, celty, torch)
        w2.capture(torch, 240)
        us2 = float(np.median(timed_regions(torch, w2.graph.replay, max(1, 240 // w2.unit), min_total_s=0.1))) \
            * 1e3 / (max(1, 240 // w2.unit) * w2.unit)
        d2 = None if args.no_dense else min(dense_gemv_us(torch, w2, dev, 240).values())
        secondary = {"workload": SECONDARY_WORKLOAD, "us_per_call": us2, "bytes_per_call": w2.total_bytes,
                     "achieved": w2.total_bytes / us2 / 1e3, "device_copies": w2.copies,
                     "dense_gemv_us": d2, "speedup_vs_dense_gemv": (d2 / us2) if d2 else None}
        del w2

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return
    peak, peak_src = measured_peaks()
    if secondary:
        secondary["frac"] = secondary["achieved"] / peak
    launches_per_step = 1 if (args.layout != "column" and (args.variant & 1) == 0) else 2
    us_per_call = sec_per_call * 1e6
    info = wl.info
    out = {
        "metric": METRIC, "value": gbs, "unit": "GB/s", "n_gpus": world, "steps": steps,
        "warmup": warmup, "ms_per_step": sec_per_call * 1e3, "us_per_call": us_per_call,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": workload_config(name),
        "run": {
            "layout": args.layout, "tile_rows": info.tile_rows,
            "fused_launch": wl.mats[0].launch_plan() if args.layout != "column" else None,
            "l2": f"rotation over {wl.copies} device copies ({len(wl.distinct)} distinct matrices, {wl.copies} distinct "
                  f"x), {wl.copies * wl.image_bytes / 1e6:.0f} MB > 2x L2 ({wl.l2 / 1e6:.0f} MB)",
            "launch": "stream enqueue" if args.no_graph else f"cuda graph of {wl.unit} calls",
            "timing": f"median of {len(regions)} regions of {calls_per_region} calls (whole graph replays between two "
                      "CUDA events, an untimed replay queued ahead of each region)",
            "multi_gpu": "replicas only" if world > 1 else "single",
        },
        "bytes_per_call": {"entry_stream": wl.stream_bytes, "total": wl.total_bytes, "bare_format": wl.bare_bytes,
                           "total_over_bare": wl.total_bytes / wl.bare_bytes, "dense_fp16": 2.0 * M * K,
                           "stored_entries": info.nnz + info.n_pad, "pads": info.n_pad,
                           "layout": None if not wl.layout_stats else {
                               "sub_blocks": wl.layout_stats[0],
                               "steps_per_sub_block": wl.layout_stats[1] / max(1, wl.layout_stats[0]),
                               "mean_groups_per_lane": wl.layout_stats[2] / 32.0 / max(1, wl.layout_stats[0]),
                               "step_slots_per_group": 32.0 * wl.layout_stats[1] / max(1, wl.layout_stats[2])}},
        "roofline": {"bound": "hbm", "achieved": wl.total_bytes / sec_per_call / 1e9, "peak": peak, "unit": "GB/s",
                     "frac": wl.total_bytes / sec_per_call / 1e9 / peak, "traffic": dram_traffic_per_launch(name),
                     "frac_on_bare_format_bytes": wl.bare_bytes / sec_per_call / 1e9 / peak,
                     "frac_of_nominal_8000": wl.total_bytes / sec_per_call / 1e9 / 8000.0,
                     "peak_source": peak_src,
                     "kernel": "k_spmspv_fused" if launches_per_step == 1 else "all kernels of the call",
                     "note": "one launch per call: algorithmic bytes per call / CUDA-event time per call",
                     "us_per_call": us_per_call, "us_per_call_fastest_region": min(regions) * 1e3 / calls_per_region,
                     "dense_gemv_us": dense_us, "dense_gemv_us_by_layout": dense_both,
                     "speedup_vs_dense_gemv": (dense_us / us_per_call) if dense_us else None,
                     "combined_sparsity": 1.0 - (1.0 - s) * d_a,
                     "secondary": secondary},
        "e2e": {"value": aggregate_throughput(wl.total_bytes, world, e2e_sec), "unit": "GB/s",
                "us_per_call": e2e_sec * 1e6, "h2d_bytes_per_step": 2 * K, "d2h_bytes_per_step": 4 * M},
        "gpu_launches": launches_per_step * calls_per_region,
        "clocks": clocks.summary(),
        "context": {"us_per_call_stream_enqueued": us_enqueued, "us_per_call_l2_warm": us_warm,
                    "us_per_call_isolated_host_timer": us_isolated,
                    "dense_equivalent_GBps": 2.0 * M * K / sec_per_call / 1e9,
                    "survivors": float(np.mean(wl.survivors)),
                    "realised_activation_density": float(np.mean(wl.survivors)) / K,
                    "realised_weight_density": info.nnz / (M * K), "regions_ms": [round(r, 5) for r in regions[:40]]},
    }
    if world == 1 and not args.no_cpu:
        from oracle import celty_oracle as orc
        threads = orc.max_threads()
        W0, mask0 = wl.distinct[0]
        x0, tau0 = make_x(name, 0)
        sec, calls = oracle_seconds_per_call(W0, mask0, x0, tau0, args.cpu_seconds, threads)
        sec1, calls1 = oracle_seconds_per_call(W0, mask0, x0, tau0, args.cpu_seconds / 4, 1)
        out["cpu_baseline"] = {"value": wl.total_bytes / sec / 1e9, "unit": "GB/s", "us_per_call": sec * 1e6,
                               "cores": threads, "kind": "oracle",
                               "sample": f"{calls} full calls of the fp64 masked product on this workload",
                               "one_thread": {"us_per_call": sec1 * 1e6, "sample": f"{calls1} full calls"}}
    print(json.dumps(out))
    if world > 1:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20000)
    ap.add_argument("--warmup", type=int, default=200)
    ap.add_argument("--impl", default="celty", choices=["celty", "reference"])
    ap.add_argument("--workload", default=DEFAULT_WORKLOAD, choices=sorted(WORKLOADS))
    ap.add_argument("--layout", default="lane_tile", choices=["lane_tile", "column"])
    ap.add_argument("--distinct", type=int, default=2, help="distinct synthetic matrices behind the copies")
    ap.add_argument("--copies", type=int, default=0, help="device copies in the rotation (0 = enough for 2.5x L2)")
    ap.add_argument("--grid", type=int, default=0)
    ap.add_argument("--variant", type=int, default=0)
    ap.add_argument("--groups", type=int, default=0)
    ap.add_argument("--depth", type=int, default=0)
    ap.add_argument("--cluster", type=int, default=0)
    ap.add_argument("--tile-rows", type=int, default=0)
    ap.add_argument("--no-graph", action="store_true")
    ap.add_argument("--no-dense", action="store_true")
    ap.add_argument("--no-cpu", action="store_true")
    ap.add_argument("--no-secondary", action="store_true", help="skip the second, labelled workload")
    ap.add_argument("--cpu-seconds", type=float, default=10.0)
    ap.add_argument("--sweep", default="", choices=[""] + sorted(SWEEPS) + ["format", "knobs", "regsplit", "batch"],
                    help="time every point of a configured sweep; format = compression study on the host; "
                         "knobs = launch-parameter study of --workload")
    ap.add_argument("--sweep-calls", type=int, default=600, help="calls timed per sweep point (at least)")
    args = ap.parse_args()
    if args.sweep == "format":
        run_format_study(args)
    elif args.sweep == "knobs":
        run_knob_study(args)
    elif args.sweep == "regsplit":
        run_regsplit_study(args)
    elif args.sweep == "batch":
        run_batch_study(args)
    elif args.sweep:
        run_sweep(args)
    elif args.impl == "reference":
        run_reference(args)
    else:
        run_celty(args)


if __name__ == "__main__":
    main()

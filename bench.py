#!/usr/bin/env python
"""Benchmark of the clustered-MoE layer forward (cmoe_forward through the C ABI).

A step is one pass of the whole hot path (router, permutation, expert FFNs with the fused
residuals, gated combine, un-permute) over one batch of synthetic tokens.  Default workload: the
GPT-2-medium-shaped layer (T=16384, d=1024, d_ff=4096, E=32, G=8, r=16, top-2), the compute-bound
headline configuration; the decode-shaped memory-bound workload is timed too and reported under "workloads"
(`--all` adds the other three).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--all] [--impl reference]

Prints ONE JSON line on rank 0.  With N > 1 (torchrun) every rank runs an independent replica of
the same layer on its own GPU and token batch ("replicas only": the path has no exchange step).
`--impl reference` times the CPU oracle on the host cores instead.
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

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402

from paper_2510_02345_b200 import inputs  # noqa: E402

METRIC = "clustered_moe_layer_fwd_tokens_per_s"
UNIT = "tokens/s"
NOMINAL_FP16_TFLOPS = 2250.0   # dense, vendor figure
NOMINAL_HBM_GBS = 8000.0
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}


# ------------------------------------------------------------------ algorithmic work of the method
def algorithmic_work(s, T, active_clusters, active_experts):
    """Flops and bytes the factored method must do (base once per token, G+K router logits)."""
    d, f, r, k, G, K, E = s.d, s.d_ff, s.r, s.k, s.G, s.K, s.E
    flops = 4 * T * d * f + 4 * k * T * r * (d + f) + 2 * T * d * (G + K)
    nbytes = 2 * (2 * d * f) * active_clusters + (2 * r * (d + f)) * (0.5 + 2 / 32) * active_experts \
        + 4 * d * (G + E) + 2 * T * d * 2
    return float(flops), float(nbytes)


def stage_work(s, T, stage, active_clusters, active_experts):
    """(flops, bytes) of one stage's own algorithmic share (used for the dominant kernel)."""
    d, f, r, k = s.d, s.d_ff, s.r, s.k
    if stage == "up":      # x B1 + t V1 + a U2 ; reads x, B1, V1, U2 ; its output abar is an intermediate
        return (2 * T * f * (d + 2 * k * r),
                2 * d * f * active_clusters + 2 * r * f * 0.5625 * active_experts + 2 * T * d)
    if stage == "down":    # abar B2 + s V2 ; reads B2, V2 ; writes y
        return (2 * T * d * (f + k * r),
                2 * d * f * active_clusters + r * d * 0.5625 * active_experts + 2 * T * d)
    return (0.0, 0.0)


# ------------------------------------------------------------------ DRAM traffic of the dominant kernel
# dram__bytes_read.sum + dram__bytes_write.sum of one launch, from the ncu captures summarised under
# profiles/.  The figure is reported only while
# the kernel sources still have the hash they had at the capture; otherwise "traffic" is null.
NCU_TRAFFIC = {
    "gpt2m": {"kernel": "tc2_up_wide_kernel<true,2>", "bytes": 121.410560e6 + 113.126912e6,
              "sha1": {"tc2_up_wide.cu": "4af5ed7641eb5387e18a572ad07b739a68937757",
                       "tc2_common.cuh": "f6446e474cd1a42f4e9a7cc20120ebd7f01b50b3",
                       "tc_ptx.cuh": "5939df29cafb85df0df022be40abbaa547d366c8"}},
    "decode": {"kernel": "stream_kernel<up>", "bytes": 955.968768e6 + 9.915392e6,
               "sha1": {"stream_path.cu": "232f8c53b14c361c003fef805982308b22b73f54",
                        "device_utils.cuh": "daa6a5fc90a4b02a5c17177e8d154044cca709c4",
                        "lowrank.cuh": "698889609319931f08fc77e7b2de29ef206fc1c8",
                        "tc_ptx.cuh": "5939df29cafb85df0df022be40abbaa547d366c8"}},
}


def ncu_traffic(workload):
    import hashlib
    ent = NCU_TRAFFIC.get(workload)
    if ent is None:
        return None
    csrc = os.path.join(ROOT, "paper_2510_02345_b200", "csrc")
    for name, want in ent["sha1"].items():
        try:
            with open(os.path.join(csrc, name), "rb") as f:
                if hashlib.sha1(f.read()).hexdigest() != want:
                    return None
        except OSError:
            return None
    return ent["bytes"]


# ------------------------------------------------------------------ clocks
class ClockSampler:
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.samples = []
        self._stop = threading.Event()
        self._thr = None

    def _run(self):
        while not self._stop.is_set():
            try:
                out = subprocess.run(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                      "-i", str(self.index)], capture_output=True, text=True, timeout=5).stdout
                parts = [p.strip() for p in out.strip().split(",")]
                if len(parts) >= 7:
                    self.samples.append(parts)
            except Exception:
                pass
            self._stop.wait(0.1)

    def __enter__(self):
        self._thr = threading.Thread(target=self._run, daemon=True)
        self._thr.start()
        return self

    def __exit__(self, *a):
        self._stop.set()
        self._thr.join(timeout=10)

    def summary(self):
        if not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        sm = [float(p[0]) for p in self.samples]
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        reasons = [n for i, n in enumerate(names) if any(p[3 + i].lower().startswith("active") for p in self.samples)]
        return {"sm_mhz": statistics.median(sm), "sm_max_mhz": float(self.samples[0][1]),
                "power_w_max": max(float(p[2]) for p in self.samples), "reasons": reasons,
                "samples": len(self.samples)}


def load_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        with open(p) as f:
            d = json.load(f)
        return d, "measured"
    return dict(FALLBACK_PEAKS), "fallback"


# ------------------------------------------------------------------ the CUDA arm
# Variants of the headline shape (the paper sweeps r over {4, 8, 16, 32} and lists E = 128 in G = 16 clusters): timed
# with `--variants`, reported under "variants" (parity of the same shapes: tests/test_gpu_parity.py).
VARIANTS = {
    "gpt2m_r4": dict(r=4), "gpt2m_r8": dict(r=8), "gpt2m_r32_K2": dict(r=32, E=16), "gpt2m_k1": dict(k=1),
    "gpt2m_G16_K4": dict(E=64, G=16), "gpt2m_K8_r8": dict(E=64, r=8), "gpt2m_E128_G16": dict(E=128, G=16),
    "gpt2m_bf16_bases": dict(),
    "decode_layer_T4096": dict(T=4096, d=4096, d_ff=14336, E=64, G=8, r=32),   # K r = 256: quarters of two experts
    "decode_layer_T129": dict(T=129, d=4096, d_ff=14336, E=64, G=8, r=32),     # few tokens: two pieces on the streaming path
    "decode_layer_T256": dict(T=256, d=4096, d_ff=14336, E=64, G=8, r=32),
    "decode_layer_T512": dict(T=512, d=4096, d_ff=14336, E=64, G=8, r=32),     # past the pieces: quarters on mostly empty tiles
    "gpt2m_two_clusters": dict(T=8192),      # Sec. 3.3 "Top-g1 groups", g1 = 2: 8192 tokens, two clusters each
}
VARIANT_OPTIONS = {"gpt2m_two_clusters": dict(clusters_per_token=2)}


def variant_shape(name):
    import dataclasses
    return dataclasses.replace(inputs.CONFIGS["gpt2m"], name=name, **VARIANTS[name])


def time_workload(name, steps, warmup, rank, seed_offset, want_e2e, want_clocks, dev_index, sync_ranks=True,
                  sustained_s=0.0, keep_outputs=False):
    import torch
    from paper_2510_02345_b200.binding import ClusteredMoELayer, cmoe_profile_enable, cmoe_profile_read
    s = inputs.CONFIGS[name] if name in inputs.CONFIGS else variant_shape(name)
    L = inputs.make_layer(s, seed=0, base_dtype="bf16" if name.endswith("bf16_bases") else "fp16")
    x_np = L["x"] if seed_offset == 0 else inputs.make_tokens(s, s.T, seed=seed_offset)
    dev = torch.device(f"cuda:{dev_index}")
    torch.cuda.set_device(dev)
    m = ClusteredMoELayer(L, device=str(dev), options=VARIANT_OPTIONS.get(name))
    T = x_np.shape[0]
    x = torch.from_numpy(x_np).to(dev)
    y = torch.empty_like(x)
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)   # > 126 MB L2
    stream = torch.cuda.current_stream(dev)

    cid, eid, gates = m.route(x)
    loads, _, cov = m.expert_stats(x)          # the library's own by-products: tokens per expert, load CoV
    torch.cuda.synchronize(dev)
    active_clusters = int(torch.unique(cid).numel())
    active_experts = int((loads > 0).sum())
    i_load = float(cov)
    routes = (cid.cpu().numpy(), eid.cpu().numpy(), gates.cpu().numpy()) if keep_outputs else None

    for _ in range(max(3, warmup)):
        flush.zero_()
        m.forward(x, out=y)
    torch.cuda.synchronize(dev)

    starts = [torch.cuda.Event(enable_timing=True) for _ in range(steps)]
    ends = [torch.cuda.Event(enable_timing=True) for _ in range(steps)]
    sampler = ClockSampler(dev_index) if want_clocks else None
    if sampler:
        sampler.__enter__()
        time.sleep(0.25)
    if sync_ranks:
        barrier()
    torch.cuda.synchronize(dev)
    t0 = time.perf_counter()
    for i in range(steps):
        flush.zero_()                      # L2 flush, outside the per-step events
        starts[i].record(stream)
        m.forward(x, out=y)
        ends[i].record(stream)
    torch.cuda.synchronize(dev)
    if sync_ranks:
        barrier()
    wall = time.perf_counter() - t0
    if sampler:
        time.sleep(0.1)
        sampler.__exit__()
    assert m.status() == 0
    per_step = [starts[i].elapsed_time(ends[i]) for i in range(steps)]
    dev_ms = sum(per_step)

    # stage times: a second pass of the same steps with the library's stage events on
    cmoe_profile_enable(m.handle, True)
    stage_ms = {}
    for _ in range(steps):
        flush.zero_()
        m.forward(x, out=y)
        for k_, v in cmoe_profile_read(m.handle).items():
            stage_ms[k_] = stage_ms.get(k_, 0.0) + v / steps
    cmoe_profile_enable(m.handle, False)

    # sustained pass: the same forward called back to back (no flush, no host round trip) for sustained_s
    # seconds with the clock sampler running: what a forward costs once the board is under load
    sustained = None
    if sustained_s > 0:
        per = max(dev_ms / steps, 1e-3)
        n_sus = int(max(50, sustained_s * 1e3 / per))
        for _ in range(20):
            m.forward(x, out=y)
        torch.cuda.synchronize(dev)
        sam = ClockSampler(dev_index)
        sam.__enter__()
        s0, s1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        s0.record(stream)
        for _ in range(n_sus):
            m.forward(x, out=y)
        s1.record(stream)
        s1.synchronize()
        sam.__exit__()
        assert m.status() == 0
        sustained = {"forwards": n_sus, "seconds": s0.elapsed_time(s1) * 1e-3, "ms_per_forward": s0.elapsed_time(s1) / n_sus,
                     "clocks": sam.summary(), "l2": "not flushed: inputs and weights of this workload exceed L2" if name != "tiny" else "not flushed"}

    y_host = y.float().cpu().numpy() if keep_outputs else None

    e2e = None
    if want_e2e:
        xh = torch.from_numpy(x_np).pin_memory()
        yh = torch.empty((T, s.d), dtype=torch.float16).pin_memory()
        # the library's host-buffer entry point: copies in chunks on its own streams, overlapped with the kernels
        for _ in range(2):
            m.forward_host(xh, yh)
        torch.cuda.synchronize(dev)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        n_e2e = max(3, min(steps, 20))
        tot = 0.0
        for _ in range(n_e2e):
            flush.zero_()
            e0.record(stream)
            m.forward_host(xh, yh)                   # host -> device, kernels, device -> host (pinned buffers)
            e1.record(stream)
            e1.synchronize()
            tot += e0.elapsed_time(e1)
        e2e = {"ms_per_step": tot / n_e2e, "h2d_bytes_per_step": int(xh.numel() * 2),
               "d2h_bytes_per_step": int(yh.numel() * 2), "steps": n_e2e}

    res = dict(name=name, shape=s, T=T, dev_ms=dev_ms, steps=steps, wall_s=wall, per_step=per_step,
               stage_ms=stage_ms, active_clusters=active_clusters, active_experts=active_experts,
               i_load=i_load, info=m.info, e2e=e2e, clocks=sampler.summary() if sampler else None,
               sustained=sustained, routes=routes, y=y_host, x=x_np if keep_outputs else None,
               clusters_per_token=(VARIANT_OPTIONS.get(name) or {}).get("clusters_per_token", 1))
    m.close()
    del m, x, y, flush
    torch.cuda.empty_cache()
    return res


_dist = None


def barrier():
    if _dist is not None:
        _dist.barrier()


def max_over_ranks(values, dist, device="cpu"):
    """The only collective of a multi-rank run: the MAX over ranks of the device timings (the replicas
    exchange no data).  `dist` is torch.distributed with an initialised process group."""
    import torch
    t = torch.tensor(list(values), device=device, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(v) for v in t]


def replicas_value(world, tokens_per_rank, ms_per_step):
    """Whole-job tokens/s of `world` independent replicas that each process tokens_per_rank tokens per step,
    timed by the slowest rank."""
    return world * tokens_per_rank / (ms_per_step * 1e-3)


def roofline_for(res, peaks, peaks_kind):
    """Roofline entry of the dominant kernel.  Its time is the stage's CUDA-event interval in a pass whose steps
    are separated by an L2 flush and a host round trip: a kernel timed alone, so `frac` divides by the BURST
    peak; the sustained and nominal fractions are printed beside it."""
    s, T = res["shape"], res["T"]
    stage = max(("up", "down"), key=lambda n: res["stage_ms"].get(n, 0.0))
    ms = res["stage_ms"][stage]
    flops, nbytes = stage_work(s, T * res.get("clusters_per_token", 1), stage, res["active_clusters"], res["active_experts"])
    intensity = flops / max(nbytes, 1.0)
    traffic = ncu_traffic(res["name"]) if stage == "up" else None
    if intensity > 300:           # ridge of the B200 is ~250 flop/B
        burst = float(peaks.get("bf16_tflops", FALLBACK_PEAKS["bf16_tflops"]))
        sust = float(peaks.get("bf16_tflops_sustained", FALLBACK_PEAKS["bf16_tflops_sustained"]))
        ach = flops / (ms * 1e-3) / 1e12
        return {"bound": "tensor", "kernel": stage, "achieved": ach, "peak": burst, "unit": "TFLOP/s",
                "frac": ach / burst, "traffic": traffic,
                "peak_kind": f"{peaks_kind} cuBLAS bf16 burst (kernel timed alone; fp16 has the same rate)",
                "fracs": {"of_burst": ach / burst, "of_sustained": ach / sust, "of_nominal_2250": ach / NOMINAL_FP16_TFLOPS},
                "kernel_ms": ms, "flops_per_launch": flops}
    peak = float(peaks.get("hbm_gbs", FALLBACK_PEAKS["hbm_gbs"]))
    ach = nbytes / (ms * 1e-3) / 1e9
    return {"bound": "hbm", "kernel": stage, "achieved": ach, "peak": peak, "unit": "GB/s", "frac": ach / peak,
            "traffic": traffic, "peak_kind": f"{peaks_kind} copy bandwidth",
            "fracs": {"of_measured_copy": ach / peak, "of_nominal_8000": ach / NOMINAL_HBM_GBS},
            "kernel_ms": ms, "bytes_per_launch": nbytes}


def whole_layer_fractions(res, n_gpus, peaks=None):
    s, T = res["shape"], res["T"]
    # (two clusters per token: the expert FFNs run once per kept cluster)
    flops, nbytes = algorithmic_work(s, T * res.get("clusters_per_token", 1), res["active_clusters"], res["active_experts"])
    sec = res["dev_ms"] / res["steps"] * 1e-3
    out = {"algorithmic_tflops": flops / sec / 1e12, "algorithmic_gbs": nbytes / sec / 1e9,
           "frac_of_nominal_fp16_2250T": flops / sec / 1e12 / NOMINAL_FP16_TFLOPS,
           "frac_of_nominal_hbm_8TBs": nbytes / sec / 1e9 / NOMINAL_HBM_GBS}
    if peaks:
        out["frac_of_measured_bf16_burst"] = flops / sec / 1e12 / float(peaks.get("bf16_tflops", FALLBACK_PEAKS["bf16_tflops"]))
        out["frac_of_measured_hbm_copy"] = nbytes / sec / 1e9 / float(peaks.get("hbm_gbs", FALLBACK_PEAKS["hbm_gbs"]))
    if res.get("sustained"):
        sus = res["sustained"]["ms_per_forward"] * 1e-3
        out["sustained"] = {"ms_per_forward": res["sustained"]["ms_per_forward"], "algorithmic_tflops": flops / sus / 1e12,
                            "frac_of_nominal_fp16_2250T": flops / sus / 1e12 / NOMINAL_FP16_TFLOPS,
                            "frac_of_nominal_hbm_8TBs": nbytes / sus / 1e9 / NOMINAL_HBM_GBS}
        if peaks:
            out["sustained"]["frac_of_measured_bf16_sustained"] = flops / sus / 1e12 / float(
                peaks.get("bf16_tflops_sustained", FALLBACK_PEAKS["bf16_tflops_sustained"]))
    return out


# ------------------------------------------------------------------ the CPU oracle arm
def oracle_rate(name, target_s=15.0, max_tokens=None, gpu=None):
    """tokens/s of the CPU oracle on a bounded sample (first n tokens) of the workload.  With `gpu` (the CUDA arm's
    routes and output rows of the same batch) the sample's rows are also compared: the second returned dict."""
    from oracle import ref
    s = inputs.CONFIGS[name] if name in inputs.CONFIGS else variant_shape(name)
    L = inputs.make_layer(s, seed=0, base_dtype="bf16" if name.endswith("bf16_bases") else "fp16")
    o = ref.Layer(L)
    T = L["x"].shape[0]
    # every call forms the expert weights first (a fixed cost) and then works per token: two probes
    # separate the two, and the sample is sized for about target_s seconds
    n1, n2 = min(T, 32), min(T, 256)
    t0 = time.perf_counter(); o.forward(L["x"][:n1]); t1 = time.perf_counter() - t0
    t0 = time.perf_counter(); o.forward(L["x"][:n2]); t2 = time.perf_counter() - t0
    per_tok = max((t2 - t1) / max(n2 - n1, 1), 1e-7)
    fixed = max(t1 - per_tok * n1, 0.0)
    n = int(min(T, max(n2, (target_s - fixed) / per_tok)))
    if max_tokens:
        n = min(n, max_tokens)
    n = max(1, n)
    t0 = time.perf_counter(); y_ref = o.forward(L["x"][:n]); dt = time.perf_counter() - t0
    base = {"value": n / dt, "unit": UNIT, "cores": ref.num_threads(), "kind": "oracle",
            "sample": f"first {n} of {T} tokens of '{name}', one call, {dt:.1f} s, expert weights formed explicitly inside the timed call"}
    parity = None
    if gpu is not None:
        parity = parity_on_sample(s, o.route(L["x"][:n]), y_ref, gpu, n)
    return base, parity


def parity_on_sample(s, r, y_ref, gpu, n):
    """The CUDA arm's routes and output rows against the oracle's on the first n tokens: routes must agree wherever
    the oracle's logit margins exceed 1e-4 (tokens inside that band are counted and left out of the row check);
    rows within max|y - y_ref| <= 1e-2 max|y_ref| + 1e-3."""
    cid, eid, _ = (a[:n] for a in gpu["routes"])
    z = np.sort(r["z"].astype(np.float64), axis=1)[:, ::-1]
    l = np.sort(r["l"].astype(np.float64), axis=1)[:, ::-1]
    cm = z[:, 0] - z[:, 1] if z.shape[1] > 1 else np.full(n, np.inf)
    last = min(s.k, l.shape[1] - 1)
    em = np.min(l[:, :last] - l[:, 1:last + 1], axis=1) if last >= 1 else np.full(n, np.inf)
    c_ok = cm > 1e-4
    e_ok = c_ok & (em > 1e-4)
    bad = int((cid[c_ok] != r["cluster_id"][c_ok]).sum() + (eid[e_ok] != r["expert_slot"][e_ok]).any(axis=1).sum())
    err = float(np.abs(gpu["y"][:n][e_ok] - y_ref[e_ok]).max()) if e_ok.any() else 0.0
    tol = 1e-2 * float(np.abs(y_ref).max()) + 1e-3
    return {"rows_checked": int(e_ok.sum()), "of_tokens": int(gpu["y"].shape[0]), "max_abs_err": err, "tolerance": tol,
            "within_tolerance": bool(err <= tol), "route_mismatches_outside_band": bad,
            "cluster_near_ties": int((~c_ok).sum()), "expert_near_ties": int((c_ok & ~e_ok).sum()), "band": 1e-4}


def config_of(name, s, T, world):
    """The workload's description: the same keys in both arms."""
    return {"workload": name, "T_per_gpu": T, "d": s.d, "d_ff": s.d_ff, "E": s.E, "G": s.G, "r": s.r, "k": s.k,
            "parallelism": "replicas only" if world > 1 else "single GPU"}


def run_reference(args, rank):
    if rank != 0:
        return
    from oracle import ref
    name = args.workload
    s = inputs.CONFIGS[name] if name in inputs.CONFIGS else variant_shape(name)
    L = inputs.make_layer(s, seed=0, base_dtype="bf16" if name.endswith("bf16_bases") else "fp16")
    o = ref.Layer(L)
    T = L["x"].shape[0]
    # size the per-step sample so that the whole run stays within a few minutes
    probe = min(T, 64)
    t0 = time.perf_counter(); o.forward(L["x"][:probe]); dt = time.perf_counter() - t0
    budget = 120.0 / max(1, args.steps + args.warmup)
    n = int(max(1, min(T, probe * budget / max(dt, 1e-3))))
    for _ in range(args.warmup):
        o.forward(L["x"][:n])
    t0 = time.perf_counter()
    for _ in range(args.steps):
        o.forward(L["x"][:n])
    dt = time.perf_counter() - t0
    value = n * args.steps / dt
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt / args.steps * 1e3,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": config_of(name, s, T, 1),
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": ref.num_threads(), "kind": "oracle",
                             "sample": f"first {n} of {T} tokens per step ({args.steps} steps)"},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


# ------------------------------------------------------------------ main
def time_similarity(peaks, E=32, n=1024 * 4096, d=1024, reps=10):
    """The Gram kernel of cmoe_expert_similarity (Eq. 2) on the headline layer's up matrices: E x n fp32 weights read
    once, so its roofline is the HBM stream (4 E n bytes per call)."""
    import torch
    from paper_2510_02345_b200 import binding
    W = torch.randn((E, n), dtype=torch.float32, device="cuda")
    mu = torch.randn((E, d), dtype=torch.float32, device="cuda")
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")
    out = binding.expert_similarity(W, mu, 0.7)
    for _ in range(3):
        binding.expert_similarity(W, mu, 0.7, out)
    ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(reps)]
    for a, b in ev:
        flush.zero_()
        a.record()
        binding.expert_similarity(W, mu, 0.7, out)       # results into the same tensors: no allocation in the timed region
        b.record()
    torch.cuda.synchronize()
    assert int(out["status"].item()) == 0
    ms = sum(a.elapsed_time(b) for a, b in ev) / reps
    gbs = 4.0 * E * n / (ms * 1e-3) / 1e9
    return {"E": E, "weights_per_expert": n, "ms_per_call": ms, "achieved_gbs": gbs, "bound": "hbm",
            "frac_of_measured_copy": gbs / float(peaks.get("hbm_gbs", FALLBACK_PEAKS["hbm_gbs"])), "frac_of_nominal_8000": gbs / 8000.0,
            "l2": "flushed between calls", "launches_per_call": 3}


def main():
    global _dist
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=30)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--workload", default="gpt2m", choices=list(inputs.CONFIGS) + list(VARIANTS))
    ap.add_argument("--impl", default="cuda", choices=["cuda", "reference"])
    ap.add_argument("--all", action="store_true", help="also time the other four workloads (short runs)")
    ap.add_argument("--variants", action="store_true", help="also time the headline shape at other ranks, k and expert counts")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--similarity", action="store_true", help="time only cmoe_expert_similarity (Eq. 2-4) and print its line")
    ap.add_argument("--no-decode", action="store_true", help="leave the decode workload out of the default line")
    ap.add_argument("--sustained", type=float, default=2.0,
                    help="seconds of back-to-back forwards for the sustained figure (0: skip)")
    args = ap.parse_args()
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))

    if args.impl == "reference":
        run_reference(args, rank)
        return

    import torch
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the library has no CPU path")
    if args.similarity:
        if rank == 0:
            torch.cuda.set_device(local_rank)
            print(json.dumps({"similarity": time_similarity(load_peaks()[0])}), flush=True)
        return
    if world > 1:
        import torch.distributed as dist
        torch.cuda.set_device(local_rank)
        dist.init_process_group("nccl", device_id=torch.device(f"cuda:{local_rank}"))
        _dist = dist

    steps, warmup = args.steps, max(3, args.warmup)
    res = time_workload(args.workload, steps, warmup, rank, seed_offset=rank, want_e2e=True,
                        want_clocks=True, dev_index=local_rank, sustained_s=args.sustained,
                        keep_outputs=(rank == 0 and not args.no_cpu_baseline))
    dev_ms = res["dev_ms"]
    e2e_ms = res["e2e"]["ms_per_step"]
    if world > 1:
        dev_ms, e2e_ms = max_over_ranks([dev_ms, e2e_ms], _dist, f"cuda:{local_rank}")
    s, T = res["shape"], res["T"]
    ms_per_step = dev_ms / steps
    value = replicas_value(world, T, ms_per_step)

    if rank == 0:
        peaks, kind = load_peaks()
        roof = roofline_for(res, peaks, kind)
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": steps, "warmup": warmup,
            "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "f16", "data": "synthetic",
            "config": config_of(args.workload, s, T, world),
            "run": {"l2": "flushed between steps by a 256 MB write outside the per-step CUDA events",
                    "timing": "sum of per-step CUDA-event intervals on the launch stream",
                    "path": int(res["info"].path), "launches_per_forward": int(res["info"].launches_forward),
                    "active_clusters": res["active_clusters"], "active_experts": res["active_experts"],
                    "expert_load_cov": res["i_load"]},
            "clocks": res["clocks"],
            "e2e": {"value": world * T / (e2e_ms * 1e-3), "unit": UNIT,
                    "h2d_bytes_per_step": res["e2e"]["h2d_bytes_per_step"],
                    "d2h_bytes_per_step": res["e2e"]["d2h_bytes_per_step"], "ms_per_step": e2e_ms},
            "gpu_launches": int(res["info"].launches_forward) * steps,
            "roofline": roof,
            "layer": whole_layer_fractions(res, world, peaks),
            "sustained": res["sustained"],
            "stage_ms": res["stage_ms"],
            "wall_ms_per_step_incl_flush": res["wall_s"] / steps * 1e3,
        }
        # the memory-bound target (decode) rides in every default line; --all adds the other workloads
        extra = [n for n in inputs.CONFIG_ORDER if n != args.workload and (args.all or (n == "decode" and not args.no_decode))]
        others = {}
        for name in extra:
            r2 = time_workload(name, max(10, steps // 3), 3, rank, 0, name == "decode", False, local_rank, sync_ranks=False,
                               sustained_s=min(args.sustained, 1.0) if name == "decode" else 0.0)
            ms2 = r2["dev_ms"] / r2["steps"]
            others[name] = {"tokens_per_s": r2["T"] / (ms2 * 1e-3), "ms_per_step": ms2, "config": config_of(name, r2["shape"], r2["T"], 1),
                            "roofline": roofline_for(r2, peaks, kind), "layer": whole_layer_fractions(r2, 1, peaks),
                            "stage_ms": r2["stage_ms"], "path": int(r2["info"].path),
                            "launches_per_forward": int(r2["info"].launches_forward),
                            "active_clusters": r2["active_clusters"], "active_experts": r2["active_experts"]}
            if r2["e2e"]:
                others[name]["e2e_ms_per_step"] = r2["e2e"]["ms_per_step"]
        if others:
            line["workloads"] = others
        if args.variants:
            var = {}
            for name in VARIANTS:
                r3 = time_workload(name, 10, 3, rank, 0, False, False, local_rank, sync_ranks=False)
                ms3 = r3["dev_ms"] / r3["steps"]
                var[name] = {"tokens_per_s": r3["T"] / (ms3 * 1e-3), "ms_per_step": ms3, "config": config_of(name, r3["shape"], r3["T"], 1),
                             "layer": whole_layer_fractions(r3, 1, peaks), "stage_ms": r3["stage_ms"], "path": int(r3["info"].path),
                             "launches_per_forward": int(r3["info"].launches_forward)}
            line["variants"] = var
        if args.all:
            line["similarity"] = time_similarity(peaks)
        if not args.no_cpu_baseline:
            line["cpu_baseline"], line["parity"] = oracle_rate(args.workload, gpu=res if res.get("y") is not None else None)
        print(json.dumps(line), flush=True)
    if world > 1:
        _dist.barrier()
        _dist.destroy_process_group()


if __name__ == "__main__":
    main()

#!/usr/bin/env python
"""Benchmark of the MorphKV decode + update hot path.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload c1] [--impl ours|reference]

A *step* is one decode step (attend, score, select, update) of every unit of the workload.
The default workload is the Llama-3.1-8B-shaped attention stack (32 layers, 32/8 heads,
d = 128, bf16, batch 1, 4096-token prompt, C = 2000, R = 32, max fusion) in steady state:
the cache is full after the prompt, so every timed step evicts one token per unit.

With N > 1 (under torchrun) every rank runs its own replica of the workload on its own GPU
with a different seed: units share nothing, so there is no collective on the data path.

Prints ONE JSON line (rank 0).  `--impl reference` times the CPU oracle instead.
"""
from __future__ import annotations

import argparse
import hashlib
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np
import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2503_00979_b200 import synth  # noqa: E402

METRIC, UNIT = "decode_tokens_per_s", "tokens/s"


def algorithmic_bytes_per_step(w: synth.Workload, n: int) -> int:
    """K and V of the n cached tokens read once plus the R*G recent queries, per unit."""
    e = 2 if w.dtype == "bf16" else 4
    return int(w.units * (2 * n * w.head_dim * e + w.R * w.group * w.head_dim * e))


# Nominal HBM3e bandwidth of the part (the HGX figure), beside the measured copy bandwidth the fraction is taken of:
# the roofline object reports the fraction of both.
NOMINAL_HBM_GBS = 7700.0

# DRAM bytes per launch of the dominant kernel (dram__bytes_read.sum + dram__bytes_write.sum from one ncu
# capture of a launch of that workload), valid only for the kernel sources it was taken with.
_TRAFFIC = {"c1": {"bytes": 284.9e6, "sources_sha256": "5687faec5ff06122cd7ad7a0975de33c1dc8eefe2ac91bbdd3f1f3cf9f928e57"}}


def measured_traffic(workload: str):
    """The captured DRAM traffic per launch, or None when the kernel has changed since the capture."""
    ent = _TRAFFIC.get(workload)
    if not ent:
        return None
    return ent["bytes"] if kernel_sources_digest() == ent["sources_sha256"] else None


def kernel_sources_digest(files=("mkv_tc.cu", "mkv_common.cuh", "mkv_sm100.cuh", "mkv_schedule.h")):
    """SHA-256 of the decode kernel's sources with `//` comments and white space removed: the figure above stays
    attached to the code it was measured on, whatever happens to the comments."""
    h = hashlib.sha256()
    csrc = os.path.join(os.path.dirname(os.path.abspath(__file__)), "paper_2503_00979_b200", "csrc")
    try:
        for f in files:
            with open(os.path.join(csrc, f), "r") as fh:
                for line in fh:
                    code = "".join(line.split("//", 1)[0].split())
                    if code:
                        h.update(code.encode())
    except OSError:
        return None
    return h.hexdigest()


def measured_peak_gbs():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        try:
            return float(json.load(open(path))["hbm_gbs"]), "measured (MEASURED_PEAKS.json hbm_gbs)"
        except Exception:
            pass
    return 6650.0, "fallback (6.65 TB/s, an earlier measurement on this pool)"


class ClockSampler:
    """SM clock and throttle reasons of one GPU, read through NVML (the library nvidia-smi itself reads).

    `during(done)` samples in the calling thread until `done()` turns true: it is called right after the timed
    steps have been enqueued, so every sample falls inside the timed region however short that is, and no
    query can sit between two kernel launches (a polling child process did: its queries take milliseconds and
    held up the launches of a 1 ms region).  Without the NVML binding, one `nvidia-smi` query is made instead.
    """

    REASONS = (("sw_power_cap", 0x4), ("hw_slowdown", 0x8), ("sw_thermal_slowdown", 0x20), ("hw_thermal_slowdown", 0x40))

    def __init__(self, device: torch.device, period_s: float = 0.005):
        self.period_s, self.sm, self.mx, self.reasons, self.nv, self.h = period_s, [], [], set(), None, None
        self.index = device.index or 0
        try:
            import pynvml
            pynvml.nvmlInit()
            uuid = str(torch.cuda.get_device_properties(device).uuid)
            try:
                self.h = pynvml.nvmlDeviceGetHandleByUUID(("GPU-" + uuid).encode())
            except Exception:
                self.h = pynvml.nvmlDeviceGetHandleByIndex(self.index)
            self.nv = pynvml
            self.sample()           # first call of each query pays one-time set-up costs: not a timed-region sample
            self.sm, self.mx, self.reasons = [], [], set()
        except Exception:
            self.nv = None

    def sample(self):
        nv = self.nv
        if nv is None:
            return self._sample_smi()
        try:
            self.sm.append(float(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM)))
            self.mx.append(float(nv.nvmlDeviceGetMaxClockInfo(self.h, nv.NVML_CLOCK_SM)))
            get = getattr(nv, "nvmlDeviceGetCurrentClocksEventReasons", None) or nv.nvmlDeviceGetCurrentClocksThrottleReasons
            mask = int(get(self.h))
            self.reasons |= {name for name, bit in self.REASONS if mask & bit}
        except Exception:
            pass

    def _sample_smi(self):
        fields = ("clocks.sm,clocks.max.sm,clocks_event_reasons.sw_power_cap,clocks_event_reasons.hw_slowdown,"
                  "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.hw_thermal_slowdown")
        try:
            out = subprocess.run(["nvidia-smi", "-i", str(self.index), f"--query-gpu={fields}",
                                  "--format=csv,noheader,nounits"], capture_output=True, text=True, timeout=10).stdout
            parts = [p.strip() for p in out.strip().split("\n")[0].split(",")]
            self.sm.append(float(parts[0])); self.mx.append(float(parts[1]))
            self.reasons |= {name for (name, _), val in zip(self.REASONS, parts[2:6]) if val.lower().startswith("active")}
        except Exception:
            pass

    def during(self, done):
        """Samples until done() is true; at least once."""
        while True:
            self.sample()
            if done():
                break
            time.sleep(self.period_s)

    def background(self):
        """Context manager that samples on a thread of its own (NVML calls release the interpreter lock) while the
        body runs calls that block the main thread."""
        sampler = self

        class _Bg:
            def __enter__(self):
                self.stop = threading.Event()

                def loop():
                    while True:
                        sampler.sample()
                        if self.stop.wait(sampler.period_s):
                            break

                self.th = threading.Thread(target=loop, daemon=True)
                self.th.start()
                return self

            def __exit__(self, *exc):
                self.stop.set()
                self.th.join(timeout=2)

        return _Bg()

    def summary(self):
        if not self.sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        return {"sm_mhz": float(np.median(self.sm)), "sm_max_mhz": float(max(self.mx)), "reasons": sorted(self.reasons),
                "samples": len(self.sm), "source": "nvml" if self.nv else "nvidia-smi"}


def oracle_throughput(w: synth.Workload, n_units: int, steps: int, warm: int = 2):
    """Times the CPU oracle as it stands on `n_units` units (one thread each) for `steps` steady-state
    decode steps.  Returns (unit-steps per second, threads used, description of the sample)."""
    from oracle import morphkv_oracle as ora
    ora.build()
    G, d, P = w.group, w.head_dim, w.prompt_len
    Rw = min(w.R, P)
    st = synth.Stream(w, "cpu")
    units = [(i % w.layers, (i // w.layers) % w.batch, (i // (w.layers * w.batch)) % w.n_kv_heads) for i in range(n_units)]
    pos = np.arange(P, P + warm + steps)
    work = []
    for (l, b, h) in units:
        k, v = st.kv(np.arange(P), [l], [b], [h])
        qw = st.q(np.arange(P - Rw, P), [l], [b], [h])
        u = ora.Unit(G, d, w.C, w.R, w.fusion)
        u.prefill(k[0, 0, 0].double().numpy(), v[0, 0, 0].double().numpy(), qw[0, 0].double().numpy())
        kk, vv = st.kv(pos, [l], [b], [h])
        qq = st.q(pos, [l], [b], [h])
        work.append((u, qq[0, 0].double().numpy(), kk[0, 0, 0].double().numpy(), vv[0, 0, 0].double().numpy()))

    def run(item, lo, hi):
        u, q, k, v = item
        for i in range(lo, hi):
            u.step(np.ascontiguousarray(q[:, i]), k[i], v[i])

    for item in work:
        run(item, 0, warm)
    threads = [threading.Thread(target=run, args=(item, warm, warm + steps)) for item in work]
    t0 = time.perf_counter()
    for th in threads:
        th.start()
    for th in threads:
        th.join()
    dt = time.perf_counter() - t0
    sample = (f"{n_units} units x {steps} steady-state steps of {w.name} (stored-profile fp64 oracle, one thread per "
              f"unit), scaled by batch/units")
    return n_units * steps / dt, n_units, sample, dt


def run_reference(args, w):
    """The oracle arm: each step is one decode step of a bounded sample of units."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    cores = len(os.sched_getaffinity(0))
    n_units = max(1, min(cores, w.units))
    ups, used, sample, dt = oracle_throughput(w, n_units, args.steps, warm=args.warmup)
    tok = ups * w.batch / w.units
    line = {
        "impl": "reference", "metric": METRIC, "value": tok, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": 1e3 * dt / args.steps, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": w.name, "layers": w.layers, "batch": w.batch, "n_q_heads": w.n_q_heads,
                   "n_kv_heads": w.n_kv_heads, "head_dim": w.head_dim, "C": w.C, "R": w.R, "fusion": w.fusion,
                   "prompt_len": w.prompt_len},
        "cpu_baseline": {"value": tok, "unit": UNIT, "cores": used, "kind": "oracle", "sample": sample},
        "e2e": {"value": tok, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


def max_over_ranks(values, device, world):
    """Element-wise maximum of per-rank timings: the job is as slow as its slowest replica."""
    import torch.distributed as dist
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    if world > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(x) for x in t]


def whole_job_tokens_per_s(world, batch_per_replica, steps, ms):
    """Aggregate decode throughput of `world` independent replicas that all ran `steps` steps in `ms`."""
    return world * batch_per_replica * steps / (ms * 1e-3)


def replica_workload(w: synth.Workload, rank: int) -> synth.Workload:
    """Every rank decodes its own replica of the workload: same shape, different content."""
    return w.replace(seed=w.seed + 1000 * rank)


def secondary_record(w: synth.Workload, W: int, K: int, dev, per_layer: bool = False, kernel: str = "auto"):
    """A second, smaller measurement in the same process (own context, device-resident inputs, same timing rules):
    either K whole-stack steps of another workload, or K steps made of per-layer calls (one call per layer, the way
    a model that runs its layers in sequence would use the library)."""
    from paper_2503_00979_b200 import binding
    tdt = synth.torch_dtype(w.dtype)
    P, Rw = w.prompt_len, min(w.R, w.prompt_len)
    st = synth.Stream(w, dev)
    mk = binding.MorphKV(w.layers, w.batch, w.n_q_heads, w.n_kv_heads, w.head_dim, w.C, w.R, w.fusion, w.dtype,
                         kernel=kernel, device=str(dev))
    ks, vs, qws = [], [], []
    for l in range(w.layers):
        k, v = st.kv(np.arange(P), [l])
        ks.append(k.to(tdt)); vs.append(v.to(tdt))
        qws.append(st.q(np.arange(P - Rw, P), [l]).to(tdt))
    k, v, qw = torch.cat(ks), torch.cat(vs), torch.cat(qws)
    del ks, vs, qws
    mk.prefill(k.contiguous(), v.contiguous(), qw.contiguous())
    del k, v, qw
    pos = np.arange(P, P + W + K)
    kk, vv = st.kv(pos)
    qs = st.q(pos).permute(3, 0, 1, 2, 4).to(tdt).contiguous()
    kn = kk.permute(3, 0, 1, 2, 4).to(tdt).contiguous()
    vn = vv.permute(3, 0, 1, 2, 4).to(tdt).contiguous()
    del kk, vv
    outs = torch.empty_like(qs)
    stream = torch.cuda.current_stream()

    def run(lo, hi):
        if not per_layer:
            mk.decode_steps(qs[lo:hi], kn[lo:hi], vn[lo:hi], outs[lo:hi])
            return
        for i in range(lo, hi):
            for l in range(w.layers):
                mk.decode_step_layer(l, qs[i, l], kn[i, l], vn[i, l], outs[i, l])

    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    clocks = ClockSampler(dev)
    run(0, W)
    mk.sync()
    n_steady = mk.view(0)["count"]
    launches0 = mk.launch_count
    torch.cuda.synchronize()
    e0.record(stream)
    run(W, W + K)
    e1.record(stream)
    clocks.during(e1.query)
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1)
    mk.sync()
    assert torch.isfinite(outs[W:].float()).all()
    bytes_step = algorithmic_bytes_per_step(w, n_steady)
    peak, _ = measured_peak_gbs()
    achieved = bytes_step / (ms / K * 1e-3) / 1e9
    rec = {"workload": w.name, "prompt_len": P, "cached_tokens_per_unit": n_steady, "steps": K, "warmup": W,
           "ms_per_step": ms / K, "tokens_per_s": w.batch * K / (ms * 1e-3), "kernel": mk.kernel_name,
           "gpu_launches": int(mk.launch_count - launches0),
           "roofline": {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak, "nominal_peak": NOMINAL_HBM_GBS,
                        "frac_of_nominal": achieved / NOMINAL_HBM_GBS,
                        "algorithmic_bytes_per_launch": bytes_step if not per_layer else bytes_step // w.layers},
           "clocks": clocks.summary()}
    if per_layer:
        rec["calls"] = "one mkv_decode_step_layer call per layer"
        rec["us_per_layer_call"] = 1e3 * ms / (K * w.layers)
    mk.close()
    del qs, kn, vn, outs
    torch.cuda.empty_cache()
    return rec


def run_prefill_arm(args, w):
    """Timed prompt phase: a step is one mkv_prefill call on a P-token prompt (window-row soft-max statistics, fused
    scores of the older tokens, top-C selection, gather of the kept rows, ring set-up) for every unit; the context
    is reset between calls.  Inputs are resident in HBM; the call synchronises the stream itself."""
    from paper_2503_00979_b200 import binding
    if int(os.environ.get("WORLD_SIZE", "1")) > 1 and int(os.environ.get("RANK", "0")) != 0:
        return
    dev = torch.device(f"cuda:{int(os.environ.get('LOCAL_RANK', '0'))}")
    torch.cuda.set_device(dev)
    tdt = synth.torch_dtype(w.dtype)
    K, W = args.steps, args.warmup
    P, Rw = w.prompt_len, min(w.R, w.prompt_len)
    st = synth.Stream(w, dev)
    mk = binding.MorphKV(w.layers, w.batch, w.n_q_heads, w.n_kv_heads, w.head_dim, w.C, w.R, w.fusion, w.dtype,
                         kernel=args.kernel, device=str(dev))
    k = torch.empty((w.layers, w.batch, w.n_kv_heads, P, w.head_dim), dtype=tdt, device=dev)
    v = torch.empty_like(k)
    qw = torch.empty((w.layers, w.batch, w.n_q_heads, Rw, w.head_dim), dtype=tdt, device=dev)
    chunk = 16384
    for l in range(w.layers):
        for p0 in range(0, P, chunk):
            kk, vv = st.kv(np.arange(p0, min(P, p0 + chunk)), [l])
            k[l, :, :, p0:p0 + chunk], v[l, :, :, p0:p0 + chunk] = kk[0].to(tdt), vv[0].to(tdt)
        qw[l] = st.q(np.arange(P - Rw, P), [l])[0].to(tdt)
    stream = torch.cuda.current_stream()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    clocks = ClockSampler(dev)
    for _ in range(W):
        mk.reset(); mk.prefill(k, v, qw)
    launches0 = mk.launch_count
    torch.cuda.synchronize()
    with clocks.background():
        e0.record(stream)
        for _ in range(K):
            mk.reset(); mk.prefill(k, v, qw)
        e1.record(stream)
        torch.cuda.synchronize()
    ms = e0.elapsed_time(e1)
    n = mk.view(0)["count"]
    e = 2 if w.dtype == "bf16" else 4
    # the prompt keys twice (normalisers, then scores) and the K and V rows that are kept
    bytes_step = w.units * (2 * P * w.head_dim * e + 2 * n * w.head_dim * e)
    peak, peak_src = measured_peak_gbs()
    achieved = bytes_step / (ms / K * 1e-3) / 1e9
    line = {
        "metric": "prefill_tokens_per_s", "value": w.batch * P * K / (ms * 1e-3), "unit": UNIT, "n_gpus": 1, "steps": K,
        "warmup": W, "ms_per_step": ms / K, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": w.dtype, "data": "synthetic",
        "config": {"workload": w.name, "layers": w.layers, "batch": w.batch, "n_q_heads": w.n_q_heads,
                   "n_kv_heads": w.n_kv_heads, "head_dim": w.head_dim, "C": w.C, "R": w.R, "fusion": w.fusion,
                   "prompt_len": P, "kept_tokens_per_unit": n, "units_per_gpu": w.units, "kernel": mk.kernel_name,
                   "l2": f"inputs larger than L2: the prompt's keys are {w.units * P * w.head_dim * e / 1e6:.0f} MB"},
        "clocks": clocks.summary(), "e2e": None, "gpu_launches": int(mk.launch_count - launches0),
        "roofline": {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak, "nominal_peak": NOMINAL_HBM_GBS,
                        "frac_of_nominal": achieved / NOMINAL_HBM_GBS,
                     "traffic": None, "peak_source": peak_src, "kernel": "prefill (two scoring passes + select + gather)",
                     "algorithmic_bytes_per_launch": bytes_step},
    }
    print(json.dumps(line), flush=True)
    mk.close()


def run_ours(args, w):
    import torch.distributed as dist
    from paper_2503_00979_b200 import binding

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if world > 1:
        dist.init_process_group("nccl" if torch.cuda.is_available() else "gloo")
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the decode path has no CPU fallback")
    dev = torch.device(f"cuda:{local}")
    torch.cuda.set_device(dev)
    w = replica_workload(w, rank)
    tdt = synth.torch_dtype(w.dtype)
    K, W = args.steps, args.warmup
    P, Rw = w.prompt_len, min(w.R, w.prompt_len)

    st = synth.Stream(w, dev)
    mk = binding.MorphKV(w.layers, w.batch, w.n_q_heads, w.n_kv_heads, w.head_dim, w.C, w.R, w.fusion, w.dtype,
                         evict_interval=args.evict_interval, kernel=args.kernel, splits=args.splits, device=str(dev),
                         profile=args.profile)
    # prompt phase (untimed), drawn layer by layer to bound the temporary memory
    ks, vs, qws = [], [], []
    for l in range(w.layers):
        k, v = st.kv(np.arange(P), [l])
        ks.append(k.to(tdt)); vs.append(v.to(tdt))
        qws.append(st.q(np.arange(P - Rw, P), [l]).to(tdt))
    k, v, qw = torch.cat(ks), torch.cat(vs), torch.cat(qws)
    del ks, vs, qws
    mk.prefill(k.contiguous(), v.contiguous(), qw.contiguous())
    del k, v, qw
    n0 = mk.view(0)["count"]

    total = 2 * (W + K)                            # device-resident arm, then host-buffer arm
    pos = np.arange(P, P + total)
    kk, vv = st.kv(pos)
    qs = st.q(pos).permute(3, 0, 1, 2, 4).to(tdt).contiguous()       # [steps,L,B,Hq,d]
    kn = kk.permute(3, 0, 1, 2, 4).to(tdt).contiguous()
    vn = vv.permute(3, 0, 1, 2, 4).to(tdt).contiguous()
    del kk, vv
    outs = torch.empty_like(qs[:W + K])
    stream = torch.cuda.current_stream()

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    # ---- arm 1: inputs resident in HBM ----
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    clocks = ClockSampler(dev)
    # the warm-up is bracketed by events like the timed steps: the first timing-event pair of a process costs the
    # GPU some tens of microseconds that belong to no step
    w0, w1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    w0.record(stream)
    mk.decode_steps(qs[:W], kn[:W], vn[:W], outs[:W])
    w1.record(stream)
    w1.query()
    mk.sync()
    w0.elapsed_time(w1)
    n_steady = mk.view(0)["count"]
    T = max(1, args.evict_interval)
    if T > 1:       # the fill cycles through C+R .. C+R+T-1: the roofline bytes use its mean
        n_steady = min(n_steady, w.C + w.R) + (T - 1) / 2
    launches0 = mk.launch_count
    # the steps' tensors are sliced before the first event: host work between that event and the first launch is
    # idle GPU time inside the timed region
    tq, tk, tv, to = qs[W:W + K], kn[W:W + K], vn[W:W + K], outs[W:W + K]
    barrier()
    e0.record(stream)
    mk.decode_steps(tq, tk, tv, to)
    e1.record(stream)
    clocks.during(e1.query)          # the steps are enqueued and running: sample until the last one is done
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1)
    launches = mk.launch_count - launches0
    mk.sync()
    barrier()

    # ---- arm 2: host buffers through the C ABI, copies inside the timed region ----
    if args.no_e2e:
        if rank == 0:
            print(json.dumps({"ms_per_step": ms / K, "kernel": mk.kernel_name, "note": "profiling run, no JSON contract"}))
        mk.close()
        return
    hq = qs[W + K:].cpu().pin_memory(); hk = kn[W + K:].cpu().pin_memory(); hv = vn[W + K:].cpu().pin_memory()
    ho = torch.empty_like(hq).pin_memory()
    for i in range(W):
        mk.decode_step_host(hq[i], hk[i], hv[i], ho[i])
    barrier()
    e2, e3 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e2.record(stream)
    for i in range(W, W + K):
        mk.decode_step_host(hq[i], hk[i], hv[i], ho[i])
    e3.record(stream)
    torch.cuda.synchronize()
    ms_e2e = e2.elapsed_time(e3)
    mk.sync()
    checksum = float(ho[W:].float().abs().mean())
    assert np.isfinite(checksum)

    ms, ms_e2e = max_over_ranks([ms, ms_e2e], dev, world)
    if rank == 0:
        bytes_step = algorithmic_bytes_per_step(w, n_steady)
        peak, peak_src = measured_peak_gbs()
        achieved = bytes_step / (ms / K * 1e-3) / 1e9
        e = 2 if w.dtype == "bf16" else 4
        h2d = (w.units * w.group + 2 * w.units) * w.head_dim * e
        d2h = w.units * w.group * w.head_dim * e
        line = {
            "metric": METRIC, "value": whole_job_tokens_per_s(world, w.batch, K, ms), "unit": UNIT, "n_gpus": world, "steps": K,
            "warmup": W, "ms_per_step": ms / K, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": w.dtype, "data": "synthetic",
            "config": {"workload": w.name, "layers": w.layers, "batch": w.batch, "n_q_heads": w.n_q_heads,
                       "n_kv_heads": w.n_kv_heads, "head_dim": w.head_dim, "C": w.C, "R": w.R, "fusion": w.fusion,
                       "prompt_len": P, "evict_interval": T, "cached_tokens_per_unit": n_steady, "units_per_gpu": w.units,
                       "kernel": mk.kernel_name, "profile_mode": args.profile, "parallelism": f"replicas x{world}",
                       "l2": "inputs larger than L2: each step streams the whole K/V cache "
                             f"({bytes_step / 1e6:.0f} MB per step against 126 MB of L2)"},
            "clocks": clocks.summary(),
            "e2e": {"value": whole_job_tokens_per_s(world, w.batch, K, ms_e2e), "unit": UNIT, "h2d_bytes_per_step": h2d,
                    "d2h_bytes_per_step": d2h},
            "gpu_launches": int(launches),
            "roofline": {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak, "nominal_peak": NOMINAL_HBM_GBS,
                        "frac_of_nominal": achieved / NOMINAL_HBM_GBS,
                         "traffic": measured_traffic(w.name) if mk.kernel_name == "tc" and args.prompt_len == 0 and T == 1 else None,
                         "peak_source": peak_src, "kernel": f"decode_{mk.kernel_name}",
                         "algorithmic_bytes_per_launch": bytes_step},
        }
        if world == 1 and args.also and w.name == "c1" and args.prompt_len == 0 and T == 1 and not (args.layers or args.batch):
            # second target configuration (started with a full cache so that every timed step evicts) and the
            # per-layer calling pattern, measured in the same run
            mk.close()
            del qs, kn, vn, outs
            torch.cuda.empty_cache()
            c3 = synth.WORKLOADS["c3"]
            line["also"] = [
                secondary_record(c3.replace(prompt_len=c3.C + c3.R), W, min(K, 64), dev),
                secondary_record(w, W, min(K, 32), dev, per_layer=True),
            ]
        if world == 1 and not args.no_cpu_baseline:
            cores = len(os.sched_getaffinity(0))
            n_units = max(1, min(cores, w.units))
            ups, used, sample, _ = oracle_throughput(w.replace(seed=w.seed - 1000 * rank), n_units, args.cpu_steps)
            line["cpu_baseline"] = {"value": ups * w.batch / w.units, "unit": UNIT, "cores": used, "kind": "oracle",
                                    "sample": sample, "unit_steps_per_s": ups}
        print(json.dumps(line), flush=True)
    mk.close()
    if world > 1:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=512)
    ap.add_argument("--warmup", type=int, default=16)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="c1", choices=sorted(synth.WORKLOADS))
    ap.add_argument("--kernel", default="auto", choices=["auto", "simt", "tc"])
    ap.add_argument("--profile", default="recompute", choices=["recompute", "stored"],
                    help="where the window tokens' attention profiles come from (mkv_params.profile_mode); the roofline "
                         "figure keeps the algorithmic bytes of the default mode")
    ap.add_argument("--splits", type=int, default=0)
    ap.add_argument("--cpu-steps", type=int, default=512, help="steady-state steps per unit for the CPU baseline")
    ap.add_argument("--prompt-len", type=int, default=0,
                    help="override the workload's prompt length (e.g. C + R to start config 3 with a full cache)")
    ap.add_argument("--evict-interval", type=int, default=1,
                    help="run the policy every T-th step only (coarse-grained eviction appendix)")
    ap.add_argument("--layers", type=int, default=0, help="override the workload's layer count (small cases for profiler captures)")
    ap.add_argument("--batch", type=int, default=0, help="override the workload's batch size (small cases for profiler captures)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-also", dest="also", action="store_false",
                    help="skip the secondary records (config 3 with a full cache; per-layer calls on config 1)")
    ap.add_argument("--no-e2e", action="store_true", help="skip the host-buffer arm (for profiler captures)")
    args = ap.parse_args()
    if args.warmup < 3:
        args.warmup = 3
    w = synth.WORKLOADS[args.workload]
    if args.prompt_len > 0:
        w = w.replace(prompt_len=args.prompt_len)
    if args.layers > 0 or args.batch > 0:
        w = w.replace(layers=args.layers or w.layers, batch=args.batch or w.batch,
                      name=f"{w.name} (layers={args.layers or w.layers}, batch={args.batch or w.batch})")
    if args.impl == "reference":
        run_reference(args, w)
    elif w.name.startswith("prefill_"):
        run_prefill_arm(args, w)
    else:
        run_ours(args, w)


if __name__ == "__main__":
    main()

#!/usr/bin/env python
"""Benchmark of the DapQ eviction step (rotate, score, select, compact) on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config NAME] [--impl reference]

One step = dapq_evict_layers over every layer of the chosen configuration's synthetic cache.
The default configuration is the largest one that fits a single GPU, the Llama-3-70B-shaped
128k-token cache (80 layers, 43 GB of K/V).  The metric is prompt tokens scored and evicted
per second per layer: tokens * layers / time.  Rank 0 prints ONE JSON line; besides the
headline it carries a `configs` object with a short measurement of every other configuration
(`--no-sweep` leaves it out).

Under torchrun each rank runs the same workload on its own GPU: every (layer, sequence,
KV head) is an independent unit, so the path shards with no exchange (weak scaling; NCCL
is used only for the barrier and the max over ranks of the device time).

--impl reference times the float64 CPU oracle, as it stands, on the host cores.
"""
from __future__ import annotations

import argparse
import gc
import hashlib
import json
import math
import os
import statistics
import subprocess
import sys
import tempfile
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402
import torch  # noqa: E402

from gen import inputs as gi  # noqa: E402

METRIC = "prompt tokens scored+evicted/sec per layer at 1 B200; % of HBM peak"
UNIT = "tokens/s/layer"
HEADLINE = "llama3_70b_128k"

# Recipe fallbacks, used only when MEASURED_PEAKS.json is absent.
FALLBACK_HBM_GBS = 6650.0
FALLBACK_BF16_TFLOPS = 1590.0
FALLBACK_BF16_TFLOPS_SUSTAINED = 1400.0

# DRAM traffic per launch (dram__bytes_read.sum + dram__bytes_write.sum, bytes) of the score sweeps
# from ncu captures of this program, keyed by (kernel, workload).  Every entry carries the digest of
# the kernel sources it was captured with: once those sources change, the entry no longer describes
# the kernel that runs and the bench reports `traffic: null` until the capture is redone.
_MB = 1000 * 1000
_CAPTURED_WITH = "a30b38f82276298a"
NCU_TRAFFIC = {
    ("sweep1", "llama3_70b_128k"): {"bytes": int((271.26 + 4.29) * _MB), "digest": _CAPTURED_WITH},
    ("sweep2", "llama3_70b_128k"): {"bytes": int((271.21 + 10.08) * _MB), "digest": _CAPTURED_WITH},
    ("sweep1", "qwen25_7b_128k"): {"bytes": int((134.81 + 3.72) * _MB), "digest": _CAPTURED_WITH},
    ("sweep2", "qwen25_7b_128k"): {"bytes": int((135.04 + 4.90) * _MB), "digest": _CAPTURED_WITH},
    ("sweep1", "llama3_8b_32k"): {"bytes": int((67.84 + 0.83) * _MB), "digest": _CAPTURED_WITH},
    ("sweep2", "llama3_8b_32k"): {"bytes": int((67.99 + 1.12) * _MB), "digest": _CAPTURED_WITH},
    ("sweep1", "batched_serving"): {"bytes": int((313.04 + 4.07) * _MB), "digest": _CAPTURED_WITH},
    ("sweep2", "batched_serving"): {"bytes": int((311.85 + 7.70) * _MB), "digest": _CAPTURED_WITH},
}


def kernel_digest() -> str:
    """Digest of the score-sweep sources' code, comments and blank space left out (what an ncu traffic figure is tied to)."""
    csrc = os.path.join(ROOT, "paper_2603_11564_b200", "csrc")
    h = hashlib.sha256()
    for name in sorted(os.listdir(csrc)):
        if name.startswith(("score_", "umma_")) and name.endswith((".cu", ".cuh")):
            h.update(name.encode())
            for line in open(os.path.join(csrc, name), "r"):
                code = "".join(line.split("//", 1)[0].split())
                if code:
                    h.update(code.encode())
    return h.hexdigest()[:16]


def ncu_traffic(kernel: str, workload: str):
    ent = NCU_TRAFFIC.get((kernel, workload))
    if not ent or ent["digest"] != kernel_digest():
        return None
    return ent["bytes"]


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        burst = float(p["bf16_tflops"])
        return {"hbm_gbs": float(p["hbm_gbs"]), "bf16_burst": burst,
                "bf16_sustained": float(p.get("bf16_tflops_sustained", burst)), "source": "measured"}
    return {"hbm_gbs": FALLBACK_HBM_GBS, "bf16_burst": FALLBACK_BF16_TFLOPS,
            "bf16_sustained": FALLBACK_BF16_TFLOPS_SUSTAINED, "source": "fallback"}


# --------------------------------------------------------------------------- algorithmic work
def layer_work(w: gi.Workload):
    """Algorithmic bytes / flops / exps of one layer (what the method itself must move or compute)."""
    e = 2 if w.dtype == "bf16" else 4
    d, T, KT = w.head_dim, w.total_prompt, int(w.cu_keep[-1])
    pairs = sum(w.n_q_heads * w.n_pseudo * (L + (w.n_pseudo + 1) / 2) for L in w.prompt_lens)   # visible (q, k) pairs
    k_read = w.n_kv_heads * w.total_rows * d * e
    return {
        "k_read_bytes": k_read,
        "score_write_bytes": 4 * w.n_kv_heads * T,
        "gather_bytes": 4 * w.n_kv_heads * KT * d * e,           # K and V, read + write
        "flops_per_sweep": 2.0 * pairs * d,
        "exps_per_sweep": pairs,
        "topk_bytes": 4 * w.n_kv_heads * T + 4 * w.n_kv_heads * KT,
    }


def hbm_cap(w: gi.Workload, work, peaks, n_sm: int, sm_max_mhz: float):
    """Largest fraction of the HBM peak that exact two-sweep scoring can reach on this shape:
    the layer cannot finish before its K stream, nor before two sweeps' worth of tensor work at the
    burst bf16 peak, nor before two sweeps' worth of exponentials at 16 per clock and SM."""
    hbm_bytes = work["k_read_bytes"] + work["score_write_bytes"] + work["gather_bytes"]
    t_hbm = hbm_bytes / (peaks["hbm_gbs"] * 1e9)
    t_tensor = 2 * work["flops_per_sweep"] / (peaks["bf16_burst"] * 1e12) if w.dtype == "bf16" else 0.0
    t_exp = 2 * work["exps_per_sweep"] / (16.0 * n_sm * sm_max_mhz * 1e6)
    return t_hbm / max(t_hbm, t_tensor, t_exp)


# ----------------------------------------------------------------------------- clock sampling
class ClockSampler:
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")
    NAMES = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap")

    def __init__(self, device: int):
        try:
            uuid = str(torch.cuda.get_device_properties(device).uuid)
            self.gpu_id = uuid if uuid.startswith("GPU-") else "GPU-" + uuid
        except Exception:
            self.gpu_id = str(device)
        self.proc = None
        self.out = None

    def start(self):
        self.out = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.gpu_id}", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                 "-lms", "50"], stdout=self.out, stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        self.out.flush()
        self.out.seek(0)
        sm, mx, reasons, power = [], [], set(), []
        for line in self.out.read().splitlines():
            f = [x.strip() for x in line.split(",")]
            if len(f) < 7:
                continue
            try:
                sm.append(float(f[0])); mx.append(float(f[1])); power.append(float(f[2]))
            except ValueError:
                continue
            for name, val in zip(self.NAMES, f[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        self.out.close()
        os.unlink(self.out.name)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "power_w": statistics.median(power) if power else None,
                "reasons": sorted(reasons), "samples": len(sm)}


# ------------------------------------------------------------------------------ the CPU oracle
def oracle_sample(w: gi.Workload, layer: int = 0):
    """Inputs of a bounded sample (whole layers, or the first KV heads of one) for the oracle."""
    from oracle import dapq_oracle as orc
    work = layer_work(w)
    flops = 2 * work["flops_per_sweep"] / 2          # one float64 pass: 2 * pairs * d
    heads = max(1, min(w.n_kv_heads, int(w.n_kv_heads * 60e9 / flops)))
    data = gi.draw_layer(w, layer, "cpu")
    q = data["q_pre"].double().numpy()
    q_rot = np.stack([orc.rope_pseudo_q(q[b], w.prompt_lens[b], w.rope_base) for b in range(w.batch)])
    gi.plant_structure(w, data, torch.from_numpy(q_rot))
    G = w.group
    return {"q": q[:, :heads * G], "k": data["k"][:heads].double().numpy(), "v": data["v"][:heads].double().numpy(),
            "heads": heads}


def time_oracle(w: gi.Workload, sample, repeats: int):
    """Seconds per full layer, extrapolated from the sampled KV heads."""
    from oracle import dapq_oracle as orc
    ts = []
    for _ in range(repeats):
        t0 = time.perf_counter()
        orc.evict(sample["q"], sample["k"], sample["v"], w.cu_rows, w.prompt_lens, w.keep, w.rope_base)
        ts.append((time.perf_counter() - t0) * w.n_kv_heads / sample["heads"])
    return ts


def blas_threads() -> int:
    try:
        from threadpoolctl import threadpool_info
        return max([p.get("num_threads", 1) for p in threadpool_info()] + [1])
    except Exception:
        return os.cpu_count() or 1


def cpu_baseline(w: gi.Workload, budget_s: float = 20.0):
    sample = oracle_sample(w)
    ts = time_oracle(w, sample, 1)
    while sum(ts) * sample["heads"] / w.n_kv_heads < budget_s / 2 and len(ts) < 4:
        ts += time_oracle(w, sample, 1)
    sec_per_layer = statistics.mean(ts)
    return {"value": w.total_prompt / sec_per_layer, "unit": UNIT, "cores": blas_threads(), "kind": "oracle",
            "sample": f"layer 0, {sample['heads']} of {w.n_kv_heads} KV heads, {len(ts)} repeat(s), "
                      f"{sec_per_layer:.2f} s per full layer (numpy float64; BLAS threads = cores)"}


def run_reference(args, w: gi.Workload):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    sample = oracle_sample(w)
    time_oracle(w, sample, args.warmup)
    steps = args.steps
    ts = time_oracle(w, sample, steps)
    sec = statistics.mean(ts)
    val = w.total_prompt / sec
    desc = (f"each step = oracle evict of layer 0, {sample['heads']} of {w.n_kv_heads} KV heads, scaled to a full "
            f"layer; {steps} timed step(s)")
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus, "steps": steps,
        "warmup": args.warmup, "ms_per_step": sec * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": workload_config(w, w.n_layers, 1, sample=desc),
        "cpu_baseline": {"value": val, "unit": UNIT, "cores": blas_threads(), "kind": "oracle", "sample": desc},
        "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


def workload_config(w: gi.Workload, n_layers: int, world: int, **extra):
    """The `config` object of a JSON line (the same keys in both arms)."""
    work = layer_work(w)
    cfg = {"workload": w.name, "layers": n_layers, "n_q_heads": w.n_q_heads, "n_kv_heads": w.n_kv_heads,
           "head_dim": w.head_dim, "batch": w.batch, "prompt_tokens": w.total_prompt, "n_pseudo": w.n_pseudo,
           "keep_rows": int(w.cu_keep[-1]), "parallelism": f"independent replicas x{world}",
           "l2": "inputs exceed L2: every layer's K/V (%.0f MB) is distinct and read once per step"
                 % ((2 * work["k_read_bytes"]) / 1e6)}
    cfg.update(extra)
    return cfg


# ---------------------------------------------------------------------------- rank bookkeeping
def max_over_ranks(ms: float, world: int, device) -> float:
    """The slowest rank's device time (every rank runs its own replica of the workload)."""
    if world == 1:
        return float(ms)
    import torch.distributed as dist
    tt = torch.tensor([ms], dtype=torch.float64, device=device)
    dist.all_reduce(tt, op=dist.ReduceOp.MAX)
    return float(tt.item())


def whole_job_value(world: int, tokens: int, n_layers: int, ms_step: float) -> float:
    """Tokens scored and evicted per second per layer over all ranks (weak scaling)."""
    return world * tokens * n_layers / (ms_step * 1e-3)


# ---------------------------------------------------------------------------------- GPU arm
class Env:
    """What every measurement of this process shares."""

    def __init__(self, dq, world, rank, local, dev, peaks):
        self.dq, self.world, self.rank, self.local, self.dev, self.peaks = dq, world, rank, local, dev, peaks
        self.n_sm = torch.cuda.get_device_properties(dev).multi_processor_count

    def barrier(self):
        torch.cuda.synchronize()
        if self.world > 1:
            import torch.distributed as dist
            dist.barrier()
            torch.cuda.synchronize()


def measure(env: Env, w: gi.Workload, n_layers: int, steps: int, warmup: int, repeats: int, min_seconds: float,
            e2e_steps: int, flags: int = 0):
    """Build the workload's caches in HBM, time `steps` steps of dapq_evict_layers (CUDA events, max over
    ranks), then the same steps with every kernel bracketed by events.  Returns the measurement as a dict."""
    dq, dev, peaks = env.dq, env.dev, env.peaks
    work = layer_work(w)
    dt = w.torch_dtype()
    KT = int(w.cu_keep[-1])
    ctx = dq.dapq_create(w.n_q_heads, w.n_kv_heads, w.n_pseudo, w.batch, w.total_rows,
                         dq.DAPQ_BF16 if w.dtype == "bf16" else dq.DAPQ_F32, w.rope_base, device=env.local, flags=flags)

    # ---- synthetic caches, resident in HBM; structure planted with the library's own rotation
    layers = []
    pos = list(w.prompt_lens)
    for l in range(n_layers):
        data = gi.draw_layer(w, l, dev)
        q_rot = torch.empty_like(data["q_pre"])
        dq.dapq_rope_pseudo_q(ctx, data["q_pre"], pos, q_rot)
        torch.cuda.synchronize()
        gi.plant_structure(w, data, q_rot)
        layers.append({"q": data["q_pre"], "k": data["k"], "v": data["v"],
                       "k_out": torch.empty((w.n_kv_heads, KT, w.head_dim), dtype=dt, device=dev),
                       "v_out": torch.empty((w.n_kv_heads, KT, w.head_dim), dtype=dt, device=dev)})
    torch.cuda.synchronize()
    lq, lk, lv, lko, lvo = ([L[x] for L in layers] for x in ("q", "k", "v", "k_out", "v_out"))

    def step():
        # every layer in one call: the same kernels as one dapq_evict per layer, the rotation of layer l + 1
        # running beside the selection and compaction of layer l
        dq.dapq_evict_layers(ctx, lq, lk, lv, w.cu_rows, w.prompt_lens, w.keep, lko, lvo)

    def timed(k):
        ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        ev0.record()
        for _ in range(k):
            step()
        ev1.record()
        env.barrier()
        return ev0.elapsed_time(ev1)

    for _ in range(warmup):
        step()
    dq.dapq_poll_status(ctx)
    if min_seconds > 0:
        # a short region runs at burst clocks: stretch it to at least min_seconds of device time
        env.barrier()
        ms1 = max_over_ranks(timed(1), env.world, dev)
        steps = max(steps, int(math.ceil(min_seconds * 1e3 / max(ms1, 1e-3))))

    t_host0 = time.perf_counter()
    step()
    host_us_per_layer = (time.perf_counter() - t_host0) * 1e6 / n_layers   # host side of one call (launches only)
    sampler = ClockSampler(env.local) if env.rank == 0 else None
    if sampler:
        sampler.start()
    env.barrier()
    n0 = dq.dapq_launch_count(ctx)
    ms_total = timed(steps)                       # THE timed region: exactly `steps` steps
    launches = dq.dapq_launch_count(ctx) - n0
    dq.dapq_poll_status(ctx)
    rep_ms = [ms_total / steps] + [timed(steps) / steps for _ in range(repeats - 1)]

    # ---- same steps again with every kernel bracketed by CUDA events (per-kernel durations)
    dq.dapq_profile(ctx, True)
    for _ in range(min(steps, 8)):
        step()
    prof = dq.dapq_profile_read(ctx)
    dq.dapq_profile(ctx, False)
    if sampler:
        # short runs end before nvidia-smi has sampled a few times: keep the same load on for ~0.5 s
        t_end = time.perf_counter() + 0.5
        while time.perf_counter() < t_end:
            step()
            torch.cuda.synchronize()
    clocks = sampler.stop() if sampler else None

    ms_total = max_over_ranks(ms_total, env.world, dev)
    ms_step = ms_total / steps
    tokens = w.total_prompt
    layer_ms = ms_step / n_layers
    sm_mhz = (clocks or {}).get("sm_mhz") or (clocks or {}).get("sm_max_mhz")
    sm_max = (clocks or {}).get("sm_max_mhz") or 1965.0
    timed_s = ms_total * 1e-3
    # a region of a second or more runs under the power cap: the sustained peak is its denominator
    tensor_peak = peaks["bf16_sustained"] if timed_s >= 1.0 else peaks["bf16_burst"]
    tensor_kind = "sustained" if timed_s >= 1.0 else "burst"

    # ---- roofline of the dominant kernel
    kinds = {k: v for k, v in prof.items() if v[1] > 0}
    total_prof_ms = sum(v[0] for v in kinds.values())
    dom = max(kinds, key=lambda k: kinds[k][0])
    dom_ms = kinds[dom][0] / kinds[dom][1]
    if dom in ("sweep1", "sweep2") and w.dtype == "bf16":
        # Two pipes bound a score sweep: the tensor pipe (2 * pairs * d flops) and the MUFU pipe (one exponential per
        # visible (query, key) pair, 16 per clock and SM).  The line reports the one that is closer to its peak.
        tflops = work["flops_per_sweep"] / (dom_ms * 1e-3) / 1e12
        tensor = {"achieved": tflops, "peak": tensor_peak, "unit": "TFLOP/s", "frac": tflops / tensor_peak,
                  "frac_of_burst": tflops / peaks["bf16_burst"], "frac_of_sustained": tflops / peaks["bf16_sustained"],
                  "peak_source": peaks["source"] + " (%s bf16: timed region %.2f s)" % (tensor_kind, timed_s)}
        exp_rate = work["exps_per_sweep"] / (dom_ms * 1e-3) / 1e9
        exp_peak = 16.0 * env.n_sm * sm_max * 1e6 / 1e9
        exp = {"achieved": exp_rate, "peak": exp_peak, "unit": "Gexp/s", "frac": exp_rate / exp_peak,
               "peak_source": "16 ex2 per clock and SM x %d SMs x %.0f MHz (the part's maximum SM clock)" % (env.n_sm, sm_max)}
        if sm_mhz:
            exp["frac_at_sampled_clock"] = exp_rate / (16.0 * env.n_sm * sm_mhz * 1e6 / 1e9)
            exp["sampled_sm_mhz"] = sm_mhz
        if exp["frac"] >= tensor["frac"]:
            roof = dict(exp, bound="alu", tensor=tensor)
        else:
            roof = dict(tensor, bound="tensor", exp=exp)
    else:
        nbytes = {"topk": work["topk_bytes"], "compact": work["gather_bytes"]}.get(dom, work["k_read_bytes"])
        achieved = nbytes / (dom_ms * 1e-3) / 1e9
        roof = {"bound": "hbm", "achieved": achieved, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                "frac": achieved / peaks["hbm_gbs"]}
    roof.setdefault("peak_source", peaks["source"])
    roof.update({"kernel": dom, "avg_launch_us": dom_ms * 1e3,
                 "traffic": ncu_traffic(dom, w.name),
                 "algorithmic_bytes": work["k_read_bytes"] if dom in ("sweep1", "sweep2") else None,
                 "share_of_step": kinds[dom][0] / total_prof_ms,
                 "kernels_us": {k: round(v[0] / v[1] * 1e3, 2) for k, v in kinds.items()}})
    hbm_bytes = work["k_read_bytes"] + work["score_write_bytes"] + work["gather_bytes"]
    frac = hbm_bytes / (layer_ms * 1e-3) / 1e9 / peaks["hbm_gbs"]
    cap = hbm_cap(w, work, peaks, env.n_sm, sm_max)
    hbm = {"algorithmic_bytes_per_layer": hbm_bytes, "achieved_gbs": hbm_bytes / (layer_ms * 1e-3) / 1e9,
           "frac_of_" + peaks["source"]: frac,
           "cap_two_sweeps": cap, "frac_of_cap": frac / cap,
           "cap_note": "largest HBM fraction exact two-sweep scoring can reach on this shape (K stream vs tensor work "
                       "at the burst bf16 peak vs exponentials at 16 per clock and SM)"}

    out = {"value": whole_job_value(env.world, tokens, n_layers, ms_step), "ms_per_step": ms_step, "steps": steps,
           "us_per_layer": layer_ms * 1e3, "timed_region_s": timed_s,
           "repeats_ms_per_step": [round(x, 4) for x in rep_ms],
           "us_per_layer_x_mhz": layer_ms * 1e3 * sm_mhz if sm_mhz else None,
           "host_us_per_layer": host_us_per_layer,
           "roofline": roof, "hbm": hbm, "gpu_launches": launches, "clocks": clocks, "e2e": None}

    # ---- end to end through the host-buffer entry point (pinned host memory, copies timed)
    if e2e_steps > 0:
        n_host = min(n_layers, 4)
        host = []
        for L in layers[:n_host]:
            host.append({k: L[k].cpu().pin_memory() for k in ("q", "k", "v")})
            host[-1]["k_out"] = torch.empty((w.n_kv_heads, KT, w.head_dim), dtype=dt).pin_memory()
            host[-1]["v_out"] = torch.empty((w.n_kv_heads, KT, w.head_dim), dtype=dt).pin_memory()
            host[-1]["idx"] = torch.empty((w.n_kv_heads, KT), dtype=torch.int32).pin_memory()
        hl = [host[l % n_host] for l in range(n_layers)]
        hq, hk, hv, hko, hvo, hidx = ([H[x] for H in hl] for x in ("q", "k", "v", "k_out", "v_out", "idx"))

        def host_step():
            # every layer in one call: the copies of layer l + 1 run beside the kernels of layer l
            dq.dapq_evict_layers_host(ctx, hq, hk, hv, w.cu_rows, w.prompt_lens, w.keep, hko, hvo, hidx)

        host_step()
        env.barrier()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(e2e_steps):
            host_step()
        e1.record()
        env.barrier()
        ms_e2e = max_over_ranks(e0.elapsed_time(e1) / e2e_steps, env.world, dev)
        eb = 2 if w.dtype == "bf16" else 4
        # q and K are copied to the device; of the (pinned) V only the retained rows cross, read by the compaction kernel
        h2d = n_layers * (w.n_kv_heads * w.total_rows * w.head_dim * eb + w.n_kv_heads * KT * w.head_dim * eb +
                          w.batch * w.n_q_heads * w.n_pseudo * w.head_dim * eb)
        d2h = n_layers * (2 * w.n_kv_heads * KT * w.head_dim * eb + 4 * w.n_kv_heads * KT)
        out["e2e"] = {"value": whole_job_value(env.world, tokens, n_layers, ms_e2e), "unit": UNIT,
                      "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "ms_per_step": ms_e2e, "steps": e2e_steps,
                      "api": "dapq_evict_layers_host (pinned host q/K/V in: q and K copied, kept V rows gathered over "
                             "PCIe; compacted K/V + indices out; copies of layer l+1 beside the kernels of layer l; the "
                             "%d layers cycle through %d distinct pinned host layers and their output buffers)"
                             % (n_layers, n_host)}
        del host, hl
    dq.dapq_destroy(ctx)
    del layers, lq, lk, lv, lko, lvo
    gc.collect()
    torch.cuda.empty_cache()
    return out


def run_ours(args, w: gi.Workload):
    import torch.distributed as dist

    import __graft_entry__ as ge
    import paper_2603_11564_b200 as dq

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback)")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
    if local == 0:
        ge.build()
    if world > 1:
        dist.barrier()
    dq.load_library()
    env = Env(dq, world, rank, local, dev, load_peaks())

    n_layers = args.layers or w.n_layers
    warmup = max(args.warmup, 3)
    head = measure(env, w, n_layers, args.steps, warmup, args.repeats, args.min_seconds,
                   0 if args.no_e2e else max(1, args.e2e_steps), args.flags)

    # ---- the other configurations, briefly (caches of one freed before the next is built)
    sweep = None
    if not args.no_sweep:
        sweep = {}
        for name in gi.WORKLOAD_ORDER:
            if name == w.name:
                continue
            ws = gi.workload(name)
            m = measure(env, ws, ws.n_layers, 5, 3, 1, args.sweep_seconds, 0, args.flags)
            r = m["roofline"]
            sweep[name] = {
                "us_per_layer": round(m["us_per_layer"], 2), "value": m["value"], "steps": m["steps"],
                "timed_region_s": round(m["timed_region_s"], 3), "dominant": r["kernel"], "kernels_us": r["kernels_us"],
                "bound": r["bound"],
                "tensor_frac_of_burst": (r.get("tensor") or r).get("frac_of_burst"),
                "tensor_frac_of_sustained": (r.get("tensor") or r).get("frac_of_sustained"),
                "exp_frac": (r.get("exp") or (r if r["bound"] == "alu" else {})).get("frac"),
                "exp_frac_at_sampled_clock": (r.get("exp") or (r if r["bound"] == "alu" else {})).get("frac_at_sampled_clock"),
                "hbm_frac": m["hbm"]["frac_of_" + env.peaks["source"]], "hbm_cap_two_sweeps": m["hbm"]["cap_two_sweeps"],
                "hbm_frac_of_cap": m["hbm"]["frac_of_cap"],
                "sm_mhz": (m["clocks"] or {}).get("sm_mhz"), "reasons": (m["clocks"] or {}).get("reasons"),
                "us_per_layer_x_mhz": m["us_per_layer_x_mhz"], "host_us_per_layer": round(m["host_us_per_layer"], 2),
                "gpu_launches": m["gpu_launches"],
            }

    base = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        base = cpu_baseline(w)

    if rank == 0:
        print(json.dumps({
            "metric": METRIC, "value": head["value"], "unit": UNIT, "n_gpus": world, "steps": head["steps"],
            "warmup": warmup, "ms_per_step": head["ms_per_step"], "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16" if w.dtype == "bf16" else "f32", "data": "synthetic",
            "config": workload_config(w, n_layers, world, **({"flags": args.flags} if args.flags else {})),
            "us_per_layer": head["us_per_layer"], "timed_region_s": head["timed_region_s"],
            "repeats_ms_per_step": head["repeats_ms_per_step"], "us_per_layer_x_mhz": head["us_per_layer_x_mhz"],
            "host_us_per_layer": head["host_us_per_layer"],
            "roofline": head["roofline"], "hbm": head["hbm"], "cpu_baseline": base, "e2e": head["e2e"],
            "gpu_launches": head["gpu_launches"], "clocks": head["clocks"], "configs": sweep,
        }))
    if world > 1:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None,
                    help="timed steps; when given, exactly that many are timed, else 20 or as many as --min-seconds needs")
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", default=HEADLINE, choices=list(gi.WORKLOADS))
    ap.add_argument("--layers", type=int, default=0, help="override the number of layers (0 = the config's)")
    ap.add_argument("--repeats", type=int, default=3, help="timed regions of --steps steps (the first is the headline)")
    ap.add_argument("--min-seconds", type=float, default=None,
                    help="raise the step count until the timed region lasts this long (default: 2 s when --steps is "
                         "not given, since a shorter region runs at burst clocks; 0 with --steps)")
    ap.add_argument("--sweep-seconds", type=float, default=1.0, help="length of each other configuration's timed region")
    ap.add_argument("--e2e-steps", type=int, default=2)
    ap.add_argument("--flags", type=int, default=0, help="dapq_shape.flags of the contexts (0: the library's defaults)")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-sweep", action="store_true", help="measure the chosen configuration only")
    args = ap.parse_args()
    if args.min_seconds is None:
        args.min_seconds = 2.0 if args.steps is None else 0.0
    if args.steps is None:
        args.steps = 20 if args.impl == "ours" else 1
    w = gi.workload(args.config)
    if args.impl == "reference":
        run_reference(args, w)
    else:
        run_ours(args, w)


if __name__ == "__main__":
    main()

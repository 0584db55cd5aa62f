#!/usr/bin/env python
"""Benchmark of the Keyformer generation-phase hot path (attend + score + evict).

A "step" is one kf_decode_step for every layer of the workload (32 layer calls = 64 kernel launches
for the Cerebras-GPT-shaped configuration: a streaming kernel and a closing kernel per call).  Prints one JSON line: the metric (`value`, steps/s over all
GPUs, inputs resident on the device), `roofline` (algorithmic bytes per launch / measured launch
time against the measured HBM peak), `e2e` (the same step through kf_decode_step_host with host
buffers), `cpu_baseline` (the CPU oracle on a bounded sample), `clocks`, `gpu_launches`.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload NAME]
                    [--phase decode|prefill]
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

import numpy as np
import torch

import workloads as W

METRIC = "decode steps/sec (attend+score+evict)"
UNIT = "steps/s"


# ----------------------------------------------------------------------------- helpers
def algorithmic_bytes_per_launch(wl: W.Workload) -> int:
    """Bytes one layer call must move per cache (batch row, key/value head): K and V once, score/position
    state, the step's vectors (q in and out per query head of the group; k_new, v_new in; the new row written)."""
    d, m, g = wl.head_dim, wl.budget_k + 1, wl.group
    per_unit = 4 * d * m + 12 * m + (4 * g + 8) * d
    return wl.batch * wl.kv_heads * per_unit


# DRAM traffic (dram__bytes_read.sum + dram__bytes_write.sum, both kernels of one layer call) from ncu captures, keyed by
# what kf_describe_decode reports for the launch that was captured.  A launch of any other variant, split plan or
# shape reports "traffic": null.
CAPTURED_DECODE_TRAFFIC = {
    # 1-layer case of the Cerebras-shaped workload (same per-launch shape as the 32-layer one): 1.0825 GB + 13.0 MB
    # (streaming kernel, read + write) + 27.6 MB (closing kernel)
    "decode_kernel<128,5,2,0> + decode_close_kernel<128>; units=1024 k=2048 splits=3 tiles_per_split=24 group=1": 1.1228e9,
}


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            return json.load(f), "measured"
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0}, "fallback"


class ClockSampler:
    """Samples SM clock, power and clock-event reasons through NVML (read-only queries) from a thread, every few
    milliseconds, with host timestamps: started before the warm-up, and `summary(t0, t1)` keeps the samples taken
    while the timed region ran."""
    REASONS = (("hw_slowdown", "nvmlClocksEventReasonHwSlowdown"), ("hw_thermal_slowdown", "nvmlClocksEventReasonHwThermalSlowdown"),
               ("sw_thermal_slowdown", "nvmlClocksEventReasonSwThermalSlowdown"), ("sw_power_cap", "nvmlClocksEventReasonSwPowerCap"))

    def __init__(self, device_index: int, period_s: float = 0.004):
        self.rows, self.period, self.stop_flag, self.thread, self.h, self.nv = [], period_s, False, None, None, None
        try:
            import pynvml as nv
            nv.nvmlInit()
            try:
                uuid = str(torch.cuda.get_device_properties(device_index).uuid)
                self.h = nv.nvmlDeviceGetHandleByUUID(("GPU-" + uuid).encode() if not uuid.startswith("GPU-") else uuid.encode())
            except Exception:
                self.h = nv.nvmlDeviceGetHandleByIndex(device_index)
            self.nv = nv
            self.max_mhz = float(nv.nvmlDeviceGetMaxClockInfo(self.h, nv.NVML_CLOCK_SM))
        except Exception:
            self.nv = None

    def start(self):
        if self.nv is None:
            return
        self.thread = threading.Thread(target=self._run, daemon=True)
        self.thread.start()

    def _run(self):
        nv = self.nv
        while not self.stop_flag:
            try:
                t = time.perf_counter()
                mhz = nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM)
                mask = nv.nvmlDeviceGetCurrentClocksEventReasons(self.h)
                watts = nv.nvmlDeviceGetPowerUsage(self.h) / 1000.0
                self.rows.append((t, float(mhz), int(mask), watts))
            except Exception:
                pass
            time.sleep(self.period)

    def stop(self):
        self.stop_flag = True
        if self.thread:
            self.thread.join(timeout=2)

    def summary(self, t0: float, t1: float):
        """Clock record of the samples taken between host times t0 and t1 (the timed region)."""
        if self.nv is None:
            return None
        rows = [r for r in self.rows if t0 <= r[0] <= t1]
        if not rows:
            return None
        reasons = sorted(name for name, attr in self.REASONS if any(r[2] & getattr(self.nv, attr) for r in rows))
        return {"sm_mhz": statistics.median(r[1] for r in rows), "sm_mhz_min": min(r[1] for r in rows),
                "sm_max_mhz": self.max_mhz, "samples": len(rows), "power_w_max": max(r[3] for r in rows),
                "reasons": reasons, "source": "NVML queries every %d ms during the timed region" % round(self.period * 1e3)}


def dist_setup(n_gpus: int):
    if n_gpus <= 1 or "RANK" not in os.environ:
        return 0, 1, 0
    import torch.distributed as dist
    rank, world, local = int(os.environ["RANK"]), int(os.environ["WORLD_SIZE"]), int(os.environ.get("LOCAL_RANK", 0))
    torch.cuda.set_device(local)
    dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    return rank, world, local


def max_over_ranks(value: float, world: int, device) -> float:
    """Slowest rank's time (the whole job is done when the last rank is)."""
    if world <= 1:
        return value
    import torch.distributed as dist
    t = torch.tensor([value], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def rank_workload(wl: W.Workload, rank: int) -> W.Workload:
    """Every rank owns its own batch rows (weak scaling): same shape, different data seed."""
    return wl.scaled(data_seed=wl.data_seed + 1000 * rank)


def whole_job_rate(ms_per_step: float, world: int) -> float:
    """Steps per second summed over the ranks, from the slowest rank's time per step."""
    return world * 1e3 / ms_per_step


def barrier(world: int):
    if world > 1:
        import torch.distributed as dist
        dist.barrier()
    if torch.cuda.is_available():
        torch.cuda.synchronize()


# ----------------------------------------------------------------------------- shared pieces
def shape_config(wl: W.Workload, **extra) -> dict:
    """The workload's shape, the same keys in both arms' `config`."""
    c = {"workload": wl.name, "layers": wl.n_layers, "batch": wl.batch, "heads": wl.n_heads, "kv_heads": wl.kv_heads,
         "head_dim": wl.head_dim, "prompt": wl.prompt_len, "budget_k": wl.budget_k, "recent_w": wl.recent_w}
    c.update(extra)
    return c


# ----------------------------------------------------------------------------- oracle arm
def oracle_sample_rate(wl: W.Workload, units: int, steps: int, seed: int = 0):
    """Times the CPU oracle's generation step on `units` sampled units for `steps` steps.
    The cache is filled by the oracle's own pruning routine from seeded prompt rows with an imposed kept
    set (the last k positions), which skips the prompt-phase scoring: timing does not depend on the values.
    Returns (unit_steps_per_second, threads, description)."""
    from oracle import keyformer_oracle as ko
    P = ko.Params(head_dim=wl.head_dim, n_heads=wl.n_heads, budget_k=wl.budget_k, recent_w=wl.recent_w,
                  gen_len_T=wl.gen_len_T, tau_init=wl.tau_init, tau_end=wl.tau_end, noise_seed=wl.noise_seed,
                  n_kv_heads=wl.kv_heads)
    lbh = W.sample_units(wl, units, seed)
    U, d, k, g = lbh.shape[0], wl.head_dim, wl.budget_k, wl.group
    n = min(wl.prompt_len, k + 64)
    gen = torch.Generator().manual_seed(seed)
    mk = lambda *shape: torch.randn(*shape, generator=gen).half().numpy()
    K, V = mk(U, n, d), mk(U, n, d)
    keep = np.zeros((U, n), dtype=np.uint8)
    keep[:, n - k:] = 1
    st = ko.State(P, lbh)
    st.prefill_prune(K, V, np.zeros((U, n)), keep_override=keep)
    st.n_prompt = wl.prompt_len
    st.pos[:, :k] += wl.prompt_len - n
    inputs = [(mk(U, g, d), mk(U, d), mk(U, d)) for _ in range(steps)]
    t0 = time.perf_counter()
    for s, (q, kn, vn) in enumerate(inputs, start=1):
        st.decode_score(s, q, kn, vn)
        st.decode_evict(s)
    dt = time.perf_counter() - t0
    return U * steps / dt, ko.num_threads(), f"{U} of {wl.units} units x {steps} steps, window-initialised cache"


def run_reference(args, wl):
    """The slow CPU oracle as the reference arm (rank 0 only)."""
    if int(os.environ.get("RANK", "0")) != 0:
        return
    units, steps_inner = 256, 32      # one timed step of this arm: about 0.4 s of oracle work on 16 cores
    for _ in range(max(args.warmup, 1)):
        oracle_sample_rate(wl, 8, 1)
    rates, threads, desc = [], 1, ""
    t0 = time.perf_counter()
    for i in range(args.steps):
        r, threads, desc = oracle_sample_rate(wl, units, steps_inner, seed=i)
        rates.append(r)
    wall = time.perf_counter() - t0
    value = statistics.mean(rates) / wl.units
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 / value, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": shape_config(wl, note="CPU oracle; each step times a bounded sample of units and is extrapolated to all of them"),
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": desc},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0, "wall_s": wall}
    print(json.dumps(line))


# ----------------------------------------------------------------------------- our arm
class DecodeRun:
    """A context of `wl` with its prompt phase done and the per-step inputs resident on the device."""

    def __init__(self, wl, wl_data, dev, total_steps, splits=0, new_pos=False):
        import paper_2403_09054_b200 as kf
        self.kf, self.wl, self.dev = kf, wl, dev
        self.gpu = kf.Keyformer(device=dev, n_layers=wl.n_layers, batch=wl.batch, n_heads=wl.n_heads, head_dim=wl.head_dim,
                                n_kv_heads=wl.kv_heads, rotary_dims=wl.rotary_dims if wl.rotary_in_library else 0,
                                budget_k=wl.budget_k, recent_w=wl.recent_w, max_prompt_len=wl.prompt_len,
                                gen_len_T=max(wl.gen_len_T, total_steps) if wl.rotary_in_library else wl.gen_len_T, tau_init=wl.tau_init, tau_end=wl.tau_end, noise_seed=wl.noise_seed,
                                bias_mode=kf.KF_BIAS_ALIBI if wl.positional == "alibi" else kf.KF_BIAS_NONE,
                                alibi_slopes=W.alibi_slopes(wl.n_heads) if wl.positional == "alibi" else None,
                                decode_splits=splits, pos_mode=kf.KF_POS_NEW if new_pos else kf.KF_POS_ORIGINAL)
        t0 = time.perf_counter()
        for l in range(wl.n_layers):
            q, k, v = W.make_prompt(wl_data, l, dev)
            self.gpu.kf_prefill_score_prune(l, q, k, v)
            del q, k, v
        torch.cuda.synchronize()
        self.prefill_s = time.perf_counter() - t0
        assert self.gpu.kf_poll_error() == 0
        L, B, H, Hkv, d = wl.n_layers, wl.batch, wl.n_heads, wl.kv_heads, wl.head_dim
        self.Qs = torch.empty((total_steps, L, B, H, d), dtype=torch.float16, device=dev)
        self.Kn = torch.empty((total_steps, L, B, Hkv, d), dtype=torch.float16, device=dev)
        self.Vn = torch.empty_like(self.Kn)
        for st_i in range(total_steps):
            for l in range(L):
                self.Qs[st_i, l], self.Kn[st_i, l], self.Vn[st_i, l] = W.make_step(wl_data, l, st_i + 1, dev)
        self.out = torch.empty((L, B, H, d), dtype=torch.float16, device=dev)
        self.stream = torch.cuda.current_stream()
        self.s = 1            # next step number

    def device_step(self, st=None):
        s = self.s
        for l in range(self.wl.n_layers):
            self.gpu.kf_decode_step(l, s, self.Qs[s - 1, l], self.Kn[s - 1, l], self.Vn[s - 1, l], self.out[l], stream=st or self.stream)
        self.s += 1

    def time_device(self, steps, warmup, graph, world):
        """`warmup` untimed steps, then `steps` timed ones between CUDA events on the launching stream.
        Returns (total_ms, per-step ms list or None, launches, host times of the region)."""
        for _ in range(warmup):
            self.device_step()
        barrier(world)
        ev = [torch.cuda.Event(enable_timing=True) for _ in range(steps + 1)]
        launches0 = self.gpu.kf_launch_count()
        if graph:
            # The timed steps (distinct step numbers, each executed once, in order) are recorded into one CUDA
            # graph before the timed region and replayed once inside it: the host's launch cost leaves the timing.
            g, side = torch.cuda.CUDAGraph(), torch.cuda.Stream(device=self.dev)
            with torch.cuda.graph(g, stream=side):
                for _ in range(steps):
                    self.device_step(torch.cuda.current_stream())
            torch.cuda.synchronize()
            t0 = time.perf_counter()
            ev[0].record(self.stream)
            g.replay()
            ev[-1].record(self.stream)
        else:
            t0 = time.perf_counter()
            ev[0].record(self.stream)
            for i in range(steps):
                self.device_step()
                ev[i + 1].record(self.stream)
        barrier(world)
        t1 = time.perf_counter()
        launches = self.gpu.kf_launch_count() - launches0
        total_ms = ev[0].elapsed_time(ev[-1])
        step_ms = None if graph else [ev[i].elapsed_time(ev[i + 1]) for i in range(steps)]
        assert self.gpu.kf_poll_error() == 0
        return total_ms, step_ms, launches, (t0, t1)

    def time_host(self, steps, world):
        """End to end: host buffers in, host buffers out, through kf_decode_step_host.  Returns total ms."""
        wl, L = self.wl, self.wl.n_layers
        hq, hk, hv = self.Qs.cpu().pin_memory(), self.Kn.cpu().pin_memory(), self.Vn.cpu().pin_memory()
        hout = torch.empty(self.out.shape, dtype=torch.float16).pin_memory()

        def host_step():
            s = self.s
            for l in range(L):
                self.gpu.kf_decode_step_host(l, s, hq[s - 1, l], hk[s - 1, l], hv[s - 1, l], hout[l],
                                             wait=(l == L - 1), stream=self.stream)
            self.s += 1

        host_step()                   # warm-up of the copy path
        barrier(world)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(self.stream)
        for _ in range(steps):
            host_step()
        e1.record(self.stream)
        barrier(world)
        assert self.gpu.kf_poll_error() == 0
        return e0.elapsed_time(e1)

    def close(self):
        self.gpu.kf_destroy()
        del self.gpu, self.Qs, self.Kn, self.Vn, self.out
        torch.cuda.empty_cache()


def other_workload_point(name: str, dev, steps: int = 200, warmup: int = 5) -> dict:
    """A single-layer workload whose step is shorter than a host launch: `steps` steps recorded into one CUDA
    graph and replayed once.  Its KV state fits L2, so the bandwidth figure is algorithmic, not DRAM."""
    wl = W.get_config(name)
    run = DecodeRun(wl, wl, dev, warmup + steps)
    total_ms, _, launches, _ = run.time_device(steps, warmup, True, 1)
    us = total_ms * 1e3 / steps
    kv_mb = 2 * wl.n_layers * wl.batch * wl.kv_heads * wl.budget_k * wl.head_dim * 2 / 1e6
    point = {"workload": name, "steps_per_s": 1e6 / us, "us_per_step": us, "steps": steps,
             "algorithmic_GBps": algorithmic_bytes_per_launch(wl) * wl.n_layers / (us * 1e-6) / 1e9,
             "kv_state_MB": kv_mb, "note": "cache-resident (KV state fits L2), latency-bound; one CUDA graph of the timed steps",
             "kernels": run.gpu.kf_describe_decode(), "gpu_launches": int(launches)}
    run.close()
    return point


def run_ours(args, wl):
    rank, world, local = dist_setup(args.gpus)
    dev = torch.device("cuda", local)
    torch.cuda.set_device(dev)
    sampler = ClockSampler(local)
    sampler.start()                                       # before the warm-up; the summary keeps the timed region's samples
    wl_r = rank_workload(wl, rank)
    run = DecodeRun(wl, wl_r, dev, args.warmup + 2 * args.steps + 1, splits=args.splits, new_pos=args.new_pos)
    total_ms, step_ms, launches, (t0, t1) = run.time_device(args.steps, args.warmup, args.graph, world)
    clocks = sampler.summary(t0, t1)
    total_ms = max_over_ranks(total_ms, world, dev)
    ms_per_step = total_ms / args.steps
    value = whole_job_rate(ms_per_step, world)
    e2e_ms = None
    if not args.no_e2e:
        e2e_ms = max_over_ranks(run.time_host(args.steps, world), world, dev) / args.steps
    describe = run.gpu.kf_describe_decode()
    prefill_s = run.prefill_s
    run.close()
    sampler.stop()

    L, B, H, d = wl.n_layers, wl.batch, wl.n_heads, wl.head_dim
    vec_bytes_q, vec_bytes_kv = B * H * d * 2, B * wl.kv_heads * d * 2
    kv_bytes = 2 * L * B * wl.kv_heads * wl.budget_k * d * 2
    line = None
    if rank == 0:
        peaks, peak_kind = measured_peaks()
        abytes = algorithmic_bytes_per_launch(wl)
        launch_ms = ms_per_step / L       # one layer call (streaming + closing kernel), back to back: the mean, as `value`
        achieved = abytes / (launch_ms * 1e-3) / 1e9
        traffic = args.traffic if args.traffic is not None else CAPTURED_DECODE_TRAFFIC.get(describe)
        cpu_rate, threads, desc = oracle_sample_rate(wl, args.cpu_units, args.cpu_steps)
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "f16 storage, f32 arithmetic", "data": "synthetic",
            "config": shape_config(wl, tokens_per_s=value * B,
                                   l2=("inputs larger than L2 (KV state %.1f GB per GPU)" if kv_bytes > 126e6 else
                                       "KV state of this workload (%.3f GB) fits L2: cache-resident by nature, no flush") % (kv_bytes / 1e9),
                                   prefill_s=prefill_s, decode_splits=args.splits,
                                   positions_in_bias="places within the reduced cache" if args.new_pos else "original",
                                   launch_mode="one CUDA graph of the timed steps" if args.graph else "stream launches"),
            "roofline": {"bound": "hbm", "kernel": describe, "achieved": achieved, "peak": peaks["hbm_gbs"],
                         "peak_kind": peak_kind, "unit": "GB/s", "frac": achieved / peaks["hbm_gbs"],
                         "frac_of_8TBs_nominal": achieved / 8000.0, "bytes_per_launch": abytes,
                         "launch_ms": launch_ms, "launch_ms_is": "ms_per_step / layers (mean over the timed steps; the duration of one layer call = both kernels)",
                         "traffic": traffic,
                         "traffic_is": ("DRAM bytes of one layer call from the ncu capture of exactly this kernel variant and shape"
                                        if traffic is not None else "no capture of this kernel variant and shape")},
            "cpu_baseline": {"value": cpu_rate / wl.units, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": desc},
            "e2e": {"value": (world * 1e3 / e2e_ms) if e2e_ms else None, "unit": UNIT,
                    "h2d_bytes_per_step": L * (vec_bytes_q + 2 * vec_bytes_kv), "d2h_bytes_per_step": L * vec_bytes_q},
            "gpu_launches": int(launches), "clocks": clocks,
        }
        if step_ms:
            line["step_ms"] = {"mean": statistics.mean(step_ms), "median": statistics.median(step_ms),
                               "min": min(step_ms), "max": max(step_ms)}
            line["roofline"]["achieved_at_median_step"] = abytes * L / (statistics.median(step_ms) * 1e-3) / 1e9
    if world > 1:
        import torch.distributed as dist
        dist.barrier()
    if rank == 0:
        if args.extras and world == 1:
            # outside the timed region: the other workload shapes and the prompt phase, a few hundred ms each
            line["other_workloads"] = [other_workload_point(n, dev) for n in ("c1_tiny", "c2_gptj", "c3_mpt")]
            if wl.name == "c4_cerebras":
                line["other_workloads"].append(gqa_point(dev))
            line["prefill"] = prefill_point(W.get_config("c5_prefill_8k"), dev, budget_frac=0.5, steps=5, warmup=3)
            both = prefill_point(W.get_config("c5_prefill_8k"), dev, budget_frac=0.5, steps=5, warmup=3, with_attention=True)
            line["prefill"]["with_attention_output_ms_per_call"] = both["ms_per_call"]
            line["prefill"]["attention_output_alone"] = attention_point(W.get_config("c5_prefill_8k"), dev, steps=10, warmup=3)
        print(json.dumps(line))
    if world > 1:
        import torch.distributed as dist
        dist.destroy_process_group()
    return line


def gqa_point(dev, steps: int = 20, warmup: int = 3) -> dict:
    """The Cerebras-shaped model with 8 KV heads shared by its 32 query heads (4 per group), 8 layers of it:
    stream launches, inputs larger than L2."""
    wl = W.get_config("c4_cerebras_gqa8").scaled(n_layers=8)
    run = DecodeRun(wl, wl, dev, warmup + steps)
    total_ms, step_ms, launches, _ = run.time_device(steps, warmup, False, 1)
    peaks, peak_kind = measured_peaks()
    ms = total_ms / steps
    achieved = algorithmic_bytes_per_launch(wl) * wl.n_layers / (ms * 1e-3) / 1e9
    point = {"workload": wl.name + "[layers=8]", "heads": wl.n_heads, "kv_heads": wl.kv_heads, "steps_per_s": 1e3 / ms,
             "us_per_layer_call": ms * 1e3 / wl.n_layers, "algorithmic_GBps": achieved, "frac_of_measured_peak": achieved / peaks["hbm_gbs"],
             "kv_state_MB": 2 * wl.n_layers * wl.batch * wl.kv_heads * wl.budget_k * wl.head_dim * 2 / 1e6,
             "kernels": run.gpu.kf_describe_decode(), "gpu_launches": int(launches), "note": "stream launches; KV state larger than L2"}
    run.close()
    return point


# ----------------------------------------------------------------------------- prompt phase
# Issue slots one causal logit needs per sweep when nothing is wasted.  An SM has 128 FP32 lanes but 64 INT32
# lanes, so a warp's integer / logic / compare instruction takes two dispatch cycles where an FP32 one takes one
# (measured: the 40 integer instructions of one Philox4x32-10 call cost 84 cycles per warp on a scheduler).
#   integer: Philox shared by four logits (10 rounds x (2 wide multiplies + 2 three-input xors) / 4 = 10),
#            23-bit uniform (1 funnel shift), u -> 1 repair (compare + select = 2)                        -> 13
#   FP32:    uniform and 1 - u (2), repair series (2), noise and logit FMAs (2), sum (1)                   ->  7
#   MUFU:    two logarithms, one exponential (one issue slot each; 8 cycles each on the 16-lane XU)       ->  3
PREFILL_INT_INSTR, PREFILL_FP_INSTR, PREFILL_MUFU_INSTR = 13, 7, 3
# dram__bytes_read.sum + dram__bytes_write.sum of the two prefill_tc launches of one call on c5_prefill_2k (B8 H32 d128,
# n 2048: Q + K = 268 MB, each read from DRAM once per sweep), from an ncu capture.  It does not scale with the logit
# count (re-reads are served by L2), so the other prompt lengths report no traffic figure.
C5_2K_PREFILL_TRAFFIC_BYTES = (268.6 + 8.2 + 270.9 + 5.8) * 1e6
# sm__pipe_tensor_cycles_active / XU pipe / issue-active of the two sweeps in that capture (n = 2048), in percent
C5_2K_PREFILL_COUNTERS = {"captured_at": "n = 2048", "tensor_pipe_pct": [8.4, 9.6], "xu_pipe_pct": [48, 56], "issue_active_pct": [56, 61]}
PREFILL_LANE_INSTR_PER_LOGIT_SWEEP = 2 * PREFILL_INT_INSTR + PREFILL_FP_INSTR + PREFILL_MUFU_INSTR   # 36 FP32-lane slots
ALU_LANES_PER_SM, N_SM = 128, 148


def prefill_point(wl, dev, budget_frac, steps, warmup, with_attention=False, simt=False, world=1, sampler=None):
    """Times kf_prefill_score_prune (prompt scoring on the tensor cores + select + gather) for one layer.
    Returns (ms per call, launches, clock summary, the scaled workload)."""
    import paper_2403_09054_b200 as kf
    n = wl.prompt_len
    kk = max(1, int(round(n * budget_frac)))
    wl = wl.scaled(budget_k=kk, recent_w=kk // 4)
    gpu = kf.Keyformer(device=dev, n_layers=1, batch=wl.batch, n_heads=wl.n_heads, head_dim=wl.head_dim, n_kv_heads=wl.kv_heads,
                       budget_k=wl.budget_k, recent_w=wl.recent_w, max_prompt_len=n, gen_len_T=0,
                       tau_init=wl.tau_init, tau_end=wl.tau_end, noise_seed=wl.noise_seed,
                       bias_mode=kf.KF_BIAS_ALIBI if wl.positional == "alibi" else kf.KF_BIAS_NONE,
                       alibi_slopes=W.alibi_slopes(wl.n_heads) if wl.positional == "alibi" else None,
                       prefill_impl=kf.KF_PREFILL_SIMT if simt else kf.KF_PREFILL_TENSOR)
    q, k, v = W.make_prompt(wl, 0, dev)
    stream = torch.cuda.current_stream()
    attn_out = torch.empty_like(q) if with_attention else None

    def call():
        if attn_out is None:
            gpu.kf_prefill_score_prune(0, q, k, v, stream=stream)
        else:
            gpu.kf_prefill_attend_score_prune(0, q, k, v, attn_out, stream=stream)

    for _ in range(warmup):
        call()
    barrier(world)
    launches0 = gpu.kf_launch_count()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t0 = time.perf_counter()
    e0.record(stream)
    for _ in range(steps):
        call()
    e1.record(stream)
    barrier(world)
    t1 = time.perf_counter()
    launches = gpu.kf_launch_count() - launches0
    ms = e0.elapsed_time(e1) / steps
    assert gpu.kf_poll_error() == 0
    gpu.kf_destroy()
    del q, k, v, attn_out, gpu
    torch.cuda.empty_cache()
    units = wl.batch * wl.n_heads
    logits = units * n * (n + 1) // 2
    peak = N_SM * ALU_LANES_PER_SM * 1965.0e6 / 1e12
    achieved = 2 * PREFILL_LANE_INSTR_PER_LOGIT_SWEEP * logits / (ms * 1e-3) / 1e12
    point = {"workload": wl.name, "prompt": n, "budget_k": wl.budget_k, "recent_w": wl.recent_w, "batch": wl.batch,
             "heads": wl.n_heads, "kv_heads": wl.kv_heads, "head_dim": wl.head_dim, "with_attention_output": bool(with_attention),
             "ms_per_call": ms, "steps": steps, "causal_logits": logits, "G_logits_per_s": logits / ms / 1e6,
             "qk_tflops_both_sweeps": 2 * 2 * logits * wl.head_dim / (ms * 1e-3) / 1e12,
             "roofline": {"bound": "alu", "kernel": "prefill_tc (two sweeps)", "achieved": achieved, "peak": peak,
                          "unit": "T FP32-lane issue slots/s (INT32 instructions count twice)", "frac": achieved / peak,
                          "lane_instr_per_logit_sweep": PREFILL_LANE_INSTR_PER_LOGIT_SWEEP,
                          "peak_kind": "148 SMs x 128 lanes x 1965 MHz",
                          "traffic": C5_2K_PREFILL_TRAFFIC_BYTES if (wl.name == "c5_prefill_2k" and not simt) else None,
                          "ncu_counters": C5_2K_PREFILL_COUNTERS},
             "gpu_launches": int(launches)}
    if sampler is not None:
        point["clocks"] = sampler.summary(t0, t1)
    return point


def attention_point(wl, dev, steps, warmup, world=1, sampler=None):
    """Times kf_prefill_attend alone (the prompt's causal attention output, Eq. 1, one pass over the keys on the tensor
    cores at head_dim 64 / 128).  The roofline is the tensor one: the useful flops of the causal half (QK^T and PV over
    j <= i) against the measured dense GEMM rate."""
    import paper_2403_09054_b200 as kf
    n = wl.prompt_len
    gpu = kf.Keyformer(device=dev, n_layers=1, batch=wl.batch, n_heads=wl.n_heads, head_dim=wl.head_dim, n_kv_heads=wl.kv_heads,
                       budget_k=max(1, n // 2), recent_w=max(1, n // 8), max_prompt_len=n, gen_len_T=0,
                       tau_init=wl.tau_init, tau_end=wl.tau_end, noise_seed=wl.noise_seed,
                       bias_mode=kf.KF_BIAS_ALIBI if wl.positional == "alibi" else kf.KF_BIAS_NONE,
                       alibi_slopes=W.alibi_slopes(wl.n_heads) if wl.positional == "alibi" else None)
    q, k, v = W.make_prompt(wl, 0, dev)
    out = torch.empty_like(q)
    stream = torch.cuda.current_stream()
    for _ in range(warmup):
        gpu.kf_prefill_attend(q, k, v, out, stream=stream)
    barrier(world)
    launches0 = gpu.kf_launch_count()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t0 = time.perf_counter()
    e0.record(stream)
    for _ in range(steps):
        gpu.kf_prefill_attend(q, k, v, out, stream=stream)
    e1.record(stream)
    barrier(world)
    t1 = time.perf_counter()
    launches = gpu.kf_launch_count() - launches0
    ms = e0.elapsed_time(e1) / steps
    assert gpu.kf_poll_error() == 0
    gpu.kf_destroy()
    units = wl.batch * wl.n_heads
    logits = units * n * (n + 1) // 2
    flops = 4 * logits * wl.head_dim
    peaks, kind = measured_peaks()
    achieved = flops / (ms * 1e-3) / 1e12
    point = {"workload": wl.name, "prompt": n, "batch": wl.batch, "heads": wl.n_heads, "kv_heads": wl.kv_heads,
             "head_dim": wl.head_dim, "ms_per_call": ms, "steps": steps, "causal_logits": logits,
             "roofline": {"bound": "tensor", "kernel": "prefill_attend1p" if wl.head_dim in (64, 128) else "prefill_attend",
                          "achieved": achieved, "peak": peaks["bf16_tflops"], "unit": "TFLOP/s", "frac": achieved / peaks["bf16_tflops"],
                          "peak_kind": "%s dense bf16 GEMM, burst (binary16 runs at the same rate)" % kind,
                          "flops": "4 x causal logits x head_dim (masked halves of the diagonal tiles not counted)",
                          "traffic": None},
             "gpu_launches": int(launches)}
    if sampler is not None:
        point["clocks"] = sampler.summary(t0, t1)
    return point


def run_attention(args, wl):
    rank, world, local = dist_setup(args.gpus)
    dev = torch.device("cuda", local)
    torch.cuda.set_device(dev)
    sampler = ClockSampler(local)
    sampler.start()
    pt = attention_point(rank_workload(wl, rank), dev, args.steps, args.warmup, world=world, sampler=sampler)
    sampler.stop()
    ms = max_over_ranks(pt["ms_per_call"], world, dev)
    if rank == 0:
        line = {"metric": "prompt attention calls/sec (one layer)", "value": world * 1e3 / ms, "unit": "calls/s",
                "n_gpus": world, "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True,
                "scaling": "weak", "vs_baseline": None, "dtype": "f16 operands and probabilities, f32 accumulate",
                "data": "synthetic",
                "config": {k: pt[k] for k in ("workload", "prompt", "batch", "heads", "kv_heads", "head_dim", "causal_logits")},
                "roofline": pt["roofline"], "gpu_launches": pt["gpu_launches"], "clocks": pt.get("clocks")}
        line["config"]["phase"] = "prefill, attention output only"
        line["config"]["l2"] = "Q, K, V and the output of the call (%.0f MB) exceed L2" % (
            (2 * pt["heads"] + 2 * pt["kv_heads"]) * pt["batch"] * pt["prompt"] * pt["head_dim"] * 2 / 1e6)
        print(json.dumps(line))
    if world > 1:
        import torch.distributed as dist
        dist.destroy_process_group()


def run_prefill(args, wl):
    rank, world, local = dist_setup(args.gpus)
    dev = torch.device("cuda", local)
    torch.cuda.set_device(dev)
    sampler = ClockSampler(local)
    sampler.start()
    pt = prefill_point(rank_workload(wl, rank), dev, args.budget_frac, args.steps, args.warmup,
                       with_attention=args.with_attention, simt=args.prefill_simt, world=world, sampler=sampler)
    sampler.stop()
    ms = max_over_ranks(pt["ms_per_call"], world, dev)
    if rank == 0:
        line = {"metric": "prompt score-and-prune calls/sec (one layer)", "value": world * 1e3 / ms, "unit": "calls/s",
                "n_gpus": world, "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True,
                "scaling": "weak", "vs_baseline": None, "dtype": "f16 operands, f32 accumulate and score arithmetic",
                "data": "synthetic",
                "config": {k: pt[k] for k in ("workload", "prompt", "budget_k", "recent_w", "batch", "heads", "kv_heads", "head_dim",
                                              "with_attention_output", "causal_logits", "G_logits_per_s", "qk_tflops_both_sweeps")},
                "roofline": pt["roofline"], "gpu_launches": pt["gpu_launches"], "clocks": pt.get("clocks")}
        line["config"]["phase"] = "prefill"
        line["config"]["l2"] = "Q, K, V of the call (%.0f MB) exceed L2" % (
            (pt["heads"] + 2 * pt["kv_heads"]) * pt["batch"] * pt["prompt"] * pt["head_dim"] * 2 / 1e6)
        print(json.dumps(line))
    if world > 1:
        import torch.distributed as dist
        dist.destroy_process_group()


def run_compact(args, wl):
    """Times kf_compact_layer on one layer of the workload after `--scramble-steps` generation steps have left the
    slots of every unit out of position order.  The state is exported once and imported again before every timed
    call, so each call sorts the same permutation."""
    import paper_2403_09054_b200 as kf
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    wl = wl.scaled(n_layers=1)
    run = DecodeRun(wl, wl, dev, args.scramble_steps)
    for _ in range(args.scramble_steps):
        run.device_step()
    torch.cuda.synchronize()
    gpu = run.gpu
    img = torch.empty(gpu.kf_state_bytes(), dtype=torch.uint8, device=dev)
    n_prompt, last = gpu.kf_export_state(0, img)
    pos = gpu.kf_view_state(0)[2]
    displaced = int((pos.argsort(-1).argsort(-1) != torch.arange(pos.shape[-1], device=dev)).sum().item())
    times = []
    for _ in range(args.warmup + args.steps):
        gpu.kf_import_state(0, img, n_prompt, last)
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(); gpu.kf_compact_layer(0); e1.record(); torch.cuda.synchronize()
        times.append(e0.elapsed_time(e1))
    times = times[args.warmup:]
    pos = gpu.kf_view_state(0)[2]
    assert torch.equal(pos, pos.sort(-1).values) and gpu.kf_poll_error() == 0
    peaks, peak_kind = measured_peaks()
    ms = statistics.mean(times)
    moved = displaced * (4 * wl.head_dim + 8) * 2          # every displaced entry read once and written once
    line = {"metric": "in-place compactions/sec (one layer)", "value": 1e3 / ms, "unit": "calls/s", "n_gpus": 1, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "f16 rows, int32 positions, f32 scores", "data": "synthetic",
            "config": shape_config(wl, phase="compact", scramble_steps=args.scramble_steps, displaced_entries=displaced,
                                   entries=int(pos.numel())),
            "roofline": {"bound": "hbm", "kernel": "compact_rank_kernel + compact_move_kernel", "achieved": moved / (ms * 1e-3) / 1e9,
                         "peak": peaks["hbm_gbs"], "peak_kind": peak_kind, "unit": "GB/s",
                         "frac": moved / (ms * 1e-3) / 1e9 / peaks["hbm_gbs"], "bytes_per_launch": moved, "traffic": None},
            "gpu_launches": 2 * args.steps}
    print(json.dumps(line))
    run.close()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="c4_cerebras")
    ap.add_argument("--splits", type=int, default=0)
    ap.add_argument("--cpu-units", type=int, default=1024, help="units of the sample the CPU oracle is timed on (cpu_baseline)")
    ap.add_argument("--cpu-steps", type=int, default=256, help="generation steps of that sample (1024 x 256 is about 12 s on 16 cores)")
    ap.add_argument("--traffic", type=float, default=None,
                    help="DRAM bytes per layer call from an ncu capture (default: the stored capture of exactly the "
                         "kernel variant and shape that is launched, else null)")
    ap.add_argument("--layers", type=int, default=0, help="override the number of layers (profiling a small case)")
    ap.add_argument("--batch", type=int, default=0, help="override the batch size (a scaled copy of the workload)")
    ap.add_argument("--no-e2e", action="store_true", help="skip the host-buffer pass (profiling a small case)")
    ap.add_argument("--graph", action="store_true",
                    help="decode phase: record the timed steps into one CUDA graph and replay it once (takes the host's "
                         "launch cost out of the small, latency-bound workloads)")
    ap.add_argument("--phase", default="decode", choices=["decode", "prefill", "compact"],
                    help="decode: the generation step (the headline metric); prefill: the prompt phase of one layer; "
                         "compact: kf_compact_layer on one layer")
    ap.add_argument("--scramble-steps", type=int, default=32, help="compact phase: generation steps run before the compaction")
    ap.add_argument("--budget-frac", type=float, default=0.5, help="prefill phase: k as a fraction of the prompt")
    ap.add_argument("--with-attention", action="store_true",
                    help="prefill phase: kf_prefill_attend_score_prune (also produces the prompt's attention output)")
    ap.add_argument("--attention-only", action="store_true",
                    help="prefill phase: kf_prefill_attend alone (the prompt's attention output, no scoring)")
    ap.add_argument("--new-pos", action="store_true",
                    help="decode phase: the bias counts places within the reduced cache (only matters with ALiBi workloads)")
    ap.add_argument("--prefill-simt", action="store_true", help="prefill phase: CUDA-core scoring instead of tcgen05")
    ap.add_argument("--library-rotary", action="store_true",
                    help="rotary workloads: pass Q/K unrotated and let the library apply the embedding at logit time "
                         "(a cache of unrotated keys; combine with --new-pos for positions within the reduced cache)")
    ap.add_argument("--no-extras", dest="extras", action="store_false",
                    help="decode phase: skip the blocks measured after the timed region (the three single-layer workloads, "
                         "the shared-KV-head point and the prompt phase)")
    args = ap.parse_args()
    wl = W.get_config(args.workload)
    if args.layers > 0:
        wl = wl.scaled(n_layers=args.layers, name=f"{wl.name}[layers={args.layers}]")
    if args.batch > 0:
        wl = wl.scaled(batch=args.batch, name=f"{wl.name}[batch={args.batch}]")
    if args.library_rotary:
        wl = wl.scaled(rotary_in_library=True, name=f"{wl.name}[rotation by the library]")
    if args.phase == "compact" and args.impl == "ours":
        run_compact(args, wl)
    elif args.phase == "prefill" and args.impl == "ours" and args.attention_only:
        run_attention(args, wl)
    elif args.phase == "prefill" and args.impl == "ours":
        run_prefill(args, wl)
    elif args.impl == "reference":
        run_reference(args, wl)
    else:
        run_ours(args, wl)


if __name__ == "__main__":
    main()

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
    """Bytes one layer call must move: K and V once, score/position state, the step's vectors."""
    d, m = wl.head_dim, wl.budget_k + 1
    per_unit = 4 * d * m + 12 * m + 12 * d
    return wl.batch * wl.n_heads * per_unit


# dram__bytes_read.sum + dram__bytes_write.sum of one layer call (decode_kernel<128,4,2> + decode_close_kernel<128>) on a
# c4_cerebras layer (1024 units, k = 2048, d = 128), from the ncu capture summarised in profiles/decode_kernel_c4_cerebras.md.
C4_DECODE_TRAFFIC_BYTES = 1.124e9


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            return json.load(f), "measured"
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0}, "fallback"


class ClockSampler:
    """Samples SM clock and throttle reasons with nvidia-smi while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.rows, self.proc = index, [], None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.Q}",
                                          "--format=csv,noheader,nounits", "-lms", "25"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.t = threading.Thread(target=self._read, daemon=True)
            self.t.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append(line.strip())

    def stop(self):
        if not self.proc:
            return None
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        self.t.join(timeout=2)
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in self.rows:
            f = [x.strip() for x in r.split(",")]
            if len(f) < 7:
                continue
            try:
                sm.append(float(f[0])); mx.append(float(f[1]))
            except ValueError:
                continue
            for name, val in zip(names, f[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        if not sm:
            return None
        return {"sm_mhz": statistics.median(sm), "sm_max_mhz": max(mx), "samples": len(sm), "reasons": sorted(reasons)}


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


# ----------------------------------------------------------------------------- oracle arm
def oracle_sample_rate(wl: W.Workload, units: int, steps: int, seed: int = 0):
    """Times the CPU oracle's generation step on `units` sampled units for `steps` steps.
    The cache is filled by the oracle's own pruning routine from seeded prompt rows with an imposed kept
    set (the last k positions), which skips the prompt-phase scoring: timing does not depend on the values.
    Returns (unit_steps_per_second, threads, description)."""
    from oracle import keyformer_oracle as ko
    P = ko.Params(head_dim=wl.head_dim, n_heads=wl.n_heads, budget_k=wl.budget_k, recent_w=wl.recent_w,
                  gen_len_T=wl.gen_len_T, tau_init=wl.tau_init, tau_end=wl.tau_end, noise_seed=wl.noise_seed)
    lbh = W.sample_units(wl, units, seed)
    U, d, k = lbh.shape[0], wl.head_dim, wl.budget_k
    n = min(wl.prompt_len, k + 64)
    g = torch.Generator().manual_seed(seed)
    mk = lambda *shape: torch.randn(*shape, generator=g).half().numpy()
    K, V = mk(U, n, d), mk(U, n, d)
    keep = np.zeros((U, n), dtype=np.uint8)
    keep[:, n - k:] = 1
    st = ko.State(P, lbh)
    st.prefill_prune(K, V, np.zeros((U, n)), keep_override=keep)
    st.n_prompt = wl.prompt_len
    st.pos[:, :k] += wl.prompt_len - n
    inputs = [(mk(U, d), mk(U, d), mk(U, d)) for _ in range(steps)]
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
    units, steps_inner = 64, 4
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
            "config": {"workload": wl.name, "note": "CPU oracle, extrapolated from a bounded sample per step"},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": desc},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0, "wall_s": wall}
    print(json.dumps(line))


# ----------------------------------------------------------------------------- our arm
def run_ours(args, wl):
    import paper_2403_09054_b200 as kf
    rank, world, local = dist_setup(args.gpus)
    dev = torch.device("cuda", local)
    torch.cuda.set_device(dev)
    wl_r = rank_workload(wl, rank)
    gpu = kf.Keyformer(device=dev, n_layers=wl.n_layers, batch=wl.batch, n_heads=wl.n_heads, head_dim=wl.head_dim,
                       budget_k=wl.budget_k, recent_w=wl.recent_w, max_prompt_len=wl.prompt_len,
                       gen_len_T=wl.gen_len_T, tau_init=wl.tau_init, tau_end=wl.tau_end, noise_seed=wl.noise_seed,
                       bias_mode=kf.KF_BIAS_ALIBI if wl.positional == "alibi" else kf.KF_BIAS_NONE,
                       alibi_slopes=W.alibi_slopes(wl.n_heads) if wl.positional == "alibi" else None,
                       decode_splits=args.splits,
                       pos_mode=kf.KF_POS_NEW if args.new_pos else kf.KF_POS_ORIGINAL)
    t_pre = time.perf_counter()
    for l in range(wl.n_layers):
        q, k, v = W.make_prompt(wl_r, l, dev)
        gpu.kf_prefill_score_prune(l, q, k, v)
        del q, k, v
    torch.cuda.synchronize()
    t_pre = time.perf_counter() - t_pre
    assert gpu.kf_poll_error() == 0

    L, B, H, d = wl.n_layers, wl.batch, wl.n_heads, wl.head_dim
    total_steps = args.warmup + 2 * args.steps + 1
    Qs = torch.empty((total_steps, L, B, H, d), dtype=torch.float16, device=dev)
    Kn, Vn = torch.empty_like(Qs), torch.empty_like(Qs)
    for st_i in range(total_steps):
        for l in range(L):
            Qs[st_i, l], Kn[st_i, l], Vn[st_i, l] = W.make_step(wl_r, l, st_i + 1, dev)
    out = torch.empty((L, B, H, d), dtype=torch.float16, device=dev)
    stream = torch.cuda.current_stream()

    def device_step(s, st=None):
        for l in range(L):
            gpu.kf_decode_step(l, s, Qs[s - 1, l], Kn[s - 1, l], Vn[s - 1, l], out[l], stream=st or stream)

    s = 1
    for _ in range(args.warmup):
        device_step(s); s += 1
    barrier(world)
    sampler = ClockSampler(local)
    sampler.start()
    launches0 = gpu.kf_launch_count()
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps + 1)]
    if args.graph:
        # The K timed steps (distinct step numbers, each executed once, in order) are recorded into one CUDA
        # graph before the timed region and replayed once inside it: the host's launch cost leaves the timing.
        graph, side = torch.cuda.CUDAGraph(), torch.cuda.Stream(device=dev)
        launches0 = gpu.kf_launch_count()
        with torch.cuda.graph(graph, stream=side):
            for i in range(args.steps):
                device_step(s + i, torch.cuda.current_stream())
        s += args.steps
        torch.cuda.synchronize()
        ev[0].record(stream)
        graph.replay()
        ev[-1].record(stream)
    else:
        ev[0].record(stream)
        for i in range(args.steps):
            device_step(s); s += 1
            ev[i + 1].record(stream)
    barrier(world)
    clocks = sampler.stop()
    launches = gpu.kf_launch_count() - launches0
    total_ms = ev[0].elapsed_time(ev[-1])
    step_ms = ([total_ms / args.steps] if args.graph else
               [ev[i].elapsed_time(ev[i + 1]) for i in range(args.steps)])
    total_ms = max_over_ranks(total_ms, world, dev)
    assert gpu.kf_poll_error() == 0
    ms_per_step = total_ms / args.steps
    value = whole_job_rate(ms_per_step, world)

    vec_bytes = B * H * d * 2
    e2e_ms = None
    if not args.no_e2e:
        # end to end: host buffers in, host buffers out, through kf_decode_step_host
        hq, hk, hv = Qs.cpu().pin_memory(), Kn.cpu().pin_memory(), Vn.cpu().pin_memory()
        hout = torch.empty((L, B, H, d), dtype=torch.float16).pin_memory()

        def host_step(step):
            for l in range(L):
                gpu.kf_decode_step_host(l, step, hq[step - 1, l], hk[step - 1, l], hv[step - 1, l], hout[l],
                                        wait=(l == L - 1), stream=stream)

        host_step(s); s += 1          # warm-up of the copy path
        barrier(world)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(args.steps):
            host_step(s); s += 1
        e1.record(stream)
        barrier(world)
        e2e_ms = max_over_ranks(e0.elapsed_time(e1), world, dev) / args.steps
        assert gpu.kf_poll_error() == 0

    line = None
    kv_bytes = 2 * L * B * H * wl.budget_k * d * 2
    if rank == 0:
        peaks, peak_kind = measured_peaks()
        abytes = algorithmic_bytes_per_launch(wl)
        launch_ms = statistics.median(step_ms) / L      # one layer call (streaming + closing kernel), back to back
        achieved = abytes / (launch_ms * 1e-3) / 1e9
        cpu_rate, threads, desc = oracle_sample_rate(wl, args.cpu_units, args.cpu_steps)
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "f16 storage, f32 arithmetic", "data": "synthetic",
            "config": {"workload": wl.name, "layers": L, "batch": B, "heads": H, "head_dim": d, "prompt": wl.prompt_len,
                       "budget_k": wl.budget_k, "recent_w": wl.recent_w, "tokens_per_s": value * B,
                       "l2": ("inputs larger than L2 (KV state %.1f GB per GPU)" if kv_bytes > 126e6 else
                              "KV state of this workload (%.3f GB) fits L2: cache-resident by nature, no flush") % (kv_bytes / 1e9),
                       "prefill_s": t_pre, "decode_splits": args.splits,
                       "positions_in_bias": "places within the reduced cache" if args.new_pos else "original",
                       "launch_mode": "one CUDA graph of the timed steps" if args.graph else "stream launches"},
            "roofline": {"bound": "hbm", "kernel": "decode_kernel (+ decode_close_kernel: the duration is one layer call)", "achieved": achieved, "peak": peaks["hbm_gbs"],
                         "peak_kind": peak_kind, "unit": "GB/s", "frac": achieved / peaks["hbm_gbs"],
                         "frac_of_8TBs_nominal": achieved / 8000.0, "bytes_per_launch": abytes,
                         "launch_ms": launch_ms,
                         "traffic": args.traffic if args.traffic is not None else
                         (C4_DECODE_TRAFFIC_BYTES if wl.name.startswith("c4_cerebras") and args.splits == 0 else None)},
            "cpu_baseline": {"value": cpu_rate / wl.units, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": desc},
            "e2e": {"value": (world * 1e3 / e2e_ms) if e2e_ms else None, "unit": UNIT, "h2d_bytes_per_step": 3 * L * vec_bytes,
                    "d2h_bytes_per_step": L * vec_bytes},
            "gpu_launches": int(launches), "clocks": clocks,
            "step_ms": {"min": min(step_ms), "median": statistics.median(step_ms), "max": max(step_ms)},
        }
        print(json.dumps(line))
    gpu.kf_destroy()
    if world > 1:
        import torch.distributed as dist
        dist.destroy_process_group()
    return line


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
# n 2048: Q + K = 268 MB, each read from DRAM once per sweep), from the ncu capture summarised in
# profiles/prefill_tc_c5_prefill_sweep.md.  It does not scale with the logit count (re-reads are served by L2), so the
# other prompt lengths report no traffic figure.
C5_2K_PREFILL_TRAFFIC_BYTES = (268.5 + 4.8 + 270.6 + 5.4) * 1e6
PREFILL_LANE_INSTR_PER_LOGIT_SWEEP = 2 * PREFILL_INT_INSTR + PREFILL_FP_INSTR + PREFILL_MUFU_INSTR   # 36 FP32-lane slots
ALU_LANES_PER_SM, N_SM = 128, 148


def run_prefill(args, wl):
    """Times kf_prefill_score_prune (prompt scoring on the tensor cores + select + gather) for one layer."""
    import paper_2403_09054_b200 as kf
    rank, world, local = dist_setup(args.gpus)
    dev = torch.device("cuda", local)
    torch.cuda.set_device(dev)
    n = wl.prompt_len
    kk = max(1, int(round(n * args.budget_frac)))
    wl = rank_workload(wl.scaled(budget_k=kk, recent_w=kk // 4), rank)
    gpu = kf.Keyformer(device=dev, n_layers=1, batch=wl.batch, n_heads=wl.n_heads, head_dim=wl.head_dim,
                       budget_k=wl.budget_k, recent_w=wl.recent_w, max_prompt_len=n, gen_len_T=0,
                       tau_init=wl.tau_init, tau_end=wl.tau_end, noise_seed=wl.noise_seed,
                       bias_mode=kf.KF_BIAS_ALIBI if wl.positional == "alibi" else kf.KF_BIAS_NONE,
                       alibi_slopes=W.alibi_slopes(wl.n_heads) if wl.positional == "alibi" else None,
                       prefill_impl=kf.KF_PREFILL_SIMT if args.prefill_simt else kf.KF_PREFILL_TENSOR)
    q, k, v = W.make_prompt(wl, 0, dev)
    stream = torch.cuda.current_stream()
    attn_out = torch.empty_like(q) if args.with_attention else None

    def call():
        if attn_out is None:
            gpu.kf_prefill_score_prune(0, q, k, v, stream=stream)
        else:
            gpu.kf_prefill_attend_score_prune(0, q, k, v, attn_out, stream=stream)

    for _ in range(args.warmup):
        call()
    barrier(world)
    sampler = ClockSampler(local)
    sampler.start()
    launches0 = gpu.kf_launch_count()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for _ in range(args.steps):
        call()
    e1.record(stream)
    barrier(world)
    clocks = sampler.stop()
    launches = gpu.kf_launch_count() - launches0
    ms = max_over_ranks(e0.elapsed_time(e1), world, dev) / args.steps
    assert gpu.kf_poll_error() == 0
    if rank == 0:
        units = wl.batch * wl.n_heads
        logits = units * n * (n + 1) // 2
        lane_instr = 2 * PREFILL_LANE_INSTR_PER_LOGIT_SWEEP * logits
        sm_mhz = (clocks or {}).get("sm_mhz") or 1965.0
        peak = N_SM * ALU_LANES_PER_SM * 1965.0e6 / 1e12
        achieved = lane_instr / (ms * 1e-3) / 1e12
        line = {
            "metric": "prompt score-and-prune calls/sec (one layer)", "value": world * 1e3 / ms, "unit": "calls/s",
            "n_gpus": world, "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f16 operands, f32 accumulate and score arithmetic",
            "data": "synthetic",
            "config": {"workload": wl.name, "phase": "prefill", "with_attention_output": bool(args.with_attention), "batch": wl.batch, "heads": wl.n_heads,
                       "head_dim": wl.head_dim, "prompt": n, "budget_k": wl.budget_k, "recent_w": wl.recent_w,
                       "causal_logits": logits, "G_logits_per_s": logits / ms / 1e6,
                       "qk_tflops_both_sweeps": 2 * 2 * logits * wl.head_dim / (ms * 1e-3) / 1e12,
                       "l2": "Q, K, V of the call (%.0f MB) exceed L2" % (3 * units * n * wl.head_dim * 2 / 1e6)},
            "roofline": {"bound": "alu", "kernel": "prefill_tc (two sweeps)", "achieved": achieved, "peak": peak,
                         "unit": "T FP32-lane issue slots/s (INT32 instructions count twice)", "frac": achieved / peak,
                         "traffic": C5_2K_PREFILL_TRAFFIC_BYTES if (wl.name == "c5_prefill_2k" and not args.prefill_simt) else None,
                         "lane_instr_per_logit_sweep": PREFILL_LANE_INSTR_PER_LOGIT_SWEEP,
                         "peak_kind": "148 SMs x 128 lanes x 1965 MHz", "sm_mhz_seen": sm_mhz},
            "gpu_launches": int(launches), "clocks": clocks,
        }
        print(json.dumps(line))
    gpu.kf_destroy()
    if world > 1:
        import torch.distributed as dist
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="c4_cerebras")
    ap.add_argument("--splits", type=int, default=0)
    ap.add_argument("--cpu-units", type=int, default=512)
    ap.add_argument("--cpu-steps", type=int, default=64)
    ap.add_argument("--traffic", type=float, default=None,
                    help="DRAM bytes per launch of the decode kernel from an ncu capture (default: the committed "
                         "capture of the current kernel on the Cerebras-shaped layer, see profiles/)")
    ap.add_argument("--layers", type=int, default=0, help="override the number of layers (profiling a small case)")
    ap.add_argument("--batch", type=int, default=0, help="override the batch size (a scaled copy of the workload)")
    ap.add_argument("--no-e2e", action="store_true", help="skip the host-buffer pass (profiling a small case)")
    ap.add_argument("--graph", action="store_true",
                    help="decode phase: record the timed steps into one CUDA graph and replay it once (takes the host's "
                         "launch cost out of the small, latency-bound workloads)")
    ap.add_argument("--phase", default="decode", choices=["decode", "prefill"],
                    help="decode: the generation step (the headline metric); prefill: the prompt phase of one layer")
    ap.add_argument("--budget-frac", type=float, default=0.5, help="prefill phase: k as a fraction of the prompt")
    ap.add_argument("--with-attention", action="store_true",
                    help="prefill phase: kf_prefill_attend_score_prune (also produces the prompt's attention output)")
    ap.add_argument("--new-pos", action="store_true",
                    help="decode phase: the bias counts places within the reduced cache (only matters with ALiBi workloads)")
    ap.add_argument("--prefill-simt", action="store_true", help="prefill phase: CUDA-core scoring instead of tcgen05")
    args = ap.parse_args()
    wl = W.get_config(args.workload)
    if args.layers > 0:
        wl = wl.scaled(n_layers=args.layers, name=f"{wl.name}[layers={args.layers}]")
    if args.batch > 0:
        wl = wl.scaled(batch=args.batch, name=f"{wl.name}[batch={args.batch}]")
    if args.phase == "prefill" and args.impl == "ours":
        run_prefill(args, wl)
    elif args.impl == "reference":
        run_reference(args, wl)
    else:
        run_ours(args, wl)


if __name__ == "__main__":
    main()

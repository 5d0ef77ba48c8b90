#!/usr/bin/env python
"""Benchmark of the EGTP / PLP hot path on B200.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl mine|reference]

A step is one pass of the whole EGTP hot path (LM-head GEMM with online entropy, merge,
Eq. 3-4 pooling, head) over one synthetic batch shaped like the "EGTP mid" configuration:
32 prompts, lognormal(5.5, 0.8) lengths clipped to [32, 2048], d = 2048 bf16 hidden states
with 1 % outlier channels, LM head 151936 x 2048 bf16, head 2048 -> 512 -> 1.
With N > 1 every rank (one process per GPU) runs its own batch of that shape (different seed):
prompts are independent, so there is no collective on the data path ("weak" scaling).
Rank 0 prints ONE JSON line.  At N = 1 the other named workloads are timed in the same run and
summarised inside the line's "roofline" object (key "legs"): the PLP decode step at 256 live
sequences (d = 4096), the long-tailed prompt batch (d = 4096) with its HBM-bound pooling kernel,
entropy from logits already in memory, and the RL group-sampling sizes (d = 5120, 1024 streams).

--impl reference times the fp64 CPU oracle (oracle/) on a bounded sample of the same workload.
--vocab-parallel times the PLP decode step with the LM head's rows sharded over the N ranks
(one all-gather of rows x 3 floats per step) instead of the default workload.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "egtp_prompt_tokens_per_sec"
UNIT = "tokens/s"


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return dict(hbm_gbs=float(p["hbm_gbs"]), bf16_tflops=float(p["bf16_tflops"]),
                    bf16_tflops_sustained=float(p.get("bf16_tflops_sustained", p["bf16_tflops"])), source="measured")
    return dict(hbm_gbs=6650.0, bf16_tflops=1590.0, bf16_tflops_sustained=1400.0, source="fallback")


def ncu_traffic(key: str, live: dict):
    """DRAM bytes (read + write) per launch of a kernel from the ncu capture recorded in profiles/traffic.json,
    or None when the live launch (tokens, plan) is not the one that was captured."""
    try:
        with open(os.path.join(ROOT, "profiles", "traffic.json")) as f:
            rec = json.load(f)[key]
    except (OSError, KeyError, ValueError):
        return None
    for k, v in rec.get("launch", {}).items():
        if live.get(k) != v:
            return None
    return float(rec["dram_bytes_per_launch"])


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons of one GPU (read-only) for the whole run; window(t0, t1)
    summarises the samples that fall into one timed region."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int, period_ms: int = 20):
        self.gpu_index = gpu_index
        self.period_ms = period_ms
        self.rows = []
        self.proc = None
        self.thread = None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits", "-lms", str(self.period_ms),
                 "-i", str(self.gpu_index)], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None
            return
        self.thread = threading.Thread(target=self._read, daemon=True)
        self.thread.start()

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append((time.time(), line.strip()))

    def stop(self):
        if self.proc is None:
            return
        time.sleep(0.1)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=2)
        except Exception:
            self.proc.kill()

    def window(self, t0: float, t1: float):
        if self.proc is None:
            return dict(sm_mhz=None, sm_max_mhz=None, reasons=["nvidia-smi unavailable"])
        time.sleep(min(0.1, 2.5e-3 * self.period_ms))          # let the last sample of the window arrive
        inside = [r for (t, r) in self.rows if t0 <= t <= t1]
        rows = inside or [r for (t, r) in self.rows if t0 - 0.06 <= t <= t1 + 0.06]
        sm, smax, reasons, power = [], [], set(), []
        for r in rows:
            parts = [x.strip() for x in r.split(",")]
            if len(parts) < 7:
                continue
            try:
                sm.append(float(parts[0])); smax.append(float(parts[1])); power.append(float(parts[2]))
            except ValueError:
                continue
            for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), parts[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        out = dict(sm_mhz=float(np.median(sm)) if sm else None, sm_max_mhz=max(smax) if smax else None,
                   power_w=float(np.median(power)) if power else None, samples=len(sm), reasons=sorted(reasons))
        if t1 - t0 < 0.25:
            # the driver refreshes the clock and power readings only every 100 ms or so (NVML polled every 2 ms shows
            # the same values through a 90 ms burst), so a region this short mostly sees the state before it
            out["note"] = "region shorter than the clock readings' refresh interval: values lag the load"
        return out


def cycles(time_us: float, clk: dict):
    """time x median SM clock of the same region, in millions of SM cycles (None without clock samples): a figure that
    does not move with the power state the region happened to run in."""
    return None if not clk or not clk.get("sm_mhz") else time_us * clk["sm_mhz"] * 1e-6


def dist_env():
    return int(os.environ.get("RANK", "0")), int(os.environ.get("LOCAL_RANK", "0")), int(os.environ.get("WORLD_SIZE", "1"))


def workload_for_rank(rank: int):
    from paper_2602_11812_b200 import inputs as gen
    return gen.config_mid(seed=1 + rank)


# ------------------------------------------------------------------------------------------------
# CPU oracle on a bounded sample (cpu_baseline leg and --impl reference)
# ------------------------------------------------------------------------------------------------
def oracle_sample(wl, max_tokens: int = 192):
    """The shortest whole prompts of the batch, up to max_tokens tokens (at least one prompt)."""
    lens = wl.lengths
    order = np.argsort(lens, kind="stable")
    pick, tot = [], 0
    for b in order:
        if pick and tot + lens[b] > max_tokens:
            break
        pick.append(int(b)); tot += int(lens[b])
    rows = np.concatenate([wl.hidden[wl.offsets[b]:wl.offsets[b + 1]] for b in pick])
    off = np.concatenate([[0], np.cumsum([lens[b] for b in pick])]).astype(np.int32)
    return rows, off, pick


def oracle_threads():
    try:
        from threadpoolctl import threadpool_info
        return int(max([p.get("num_threads", 1) for p in threadpool_info()] or [1]))
    except Exception:
        return os.cpu_count() or 1


def time_oracle(wl, steps: int, warmup: int, max_tokens: int = 192):
    from oracle import egtp_oracle as orc
    rows, off, pick = oracle_sample(wl, max_tokens)
    for _ in range(warmup):
        orc.egtp_predict(rows, off, wl.W, wl.head, wl.alpha)
    t0 = time.perf_counter()
    for _ in range(steps):
        orc.egtp_predict(rows, off, wl.W, wl.head, wl.alpha)
    dt = time.perf_counter() - t0
    tokens = int(rows.shape[0])
    return dict(value=tokens * steps / dt, unit=UNIT, cores=oracle_threads(), kind="oracle",
                sample=f"{len(pick)} shortest whole prompts of the batch ({tokens} tokens) x {steps} passes, "
                       f"fp64 numpy, {dt:.1f} s", ms_per_step=1e3 * dt / steps, tokens=tokens)


def time_oracle_plp(pw, budget_s: float = 12.0):
    """The oracle's PLP decode step at the full batch of the decode configuration (256 live sequences): whole steps,
    every slot followed from its explicit token list, as many steps as fit the budget (at least 2)."""
    from oracle import egtp_oracle as orc
    t0 = time.perf_counter()
    orc.plp_run(pw.hidden_steps[:1], pw.reset_src[:1], pw.W, pw.head)
    first = time.perf_counter() - t0                       # includes widening the LM head to fp64 once
    n = int(max(2, min(8, budget_s / max(first, 1e-3))))
    t0 = time.perf_counter()
    orc.plp_run(pw.hidden_steps[:n], pw.reset_src[:n], pw.W, pw.head)
    dt = time.perf_counter() - t0
    return dict(value=dt / n * 1e6, unit="us per decode step at B=256", cores=oracle_threads(), kind="oracle",
                sample=f"{n} whole decode steps of all {pw.slots} slots (d={pw.d}, V={pw.V}) in one oracle run "
                       f"(the LM head is widened to fp64 once per run), fp64 numpy, {dt:.1f} s; not scaled")


def run_reference(args):
    rank, _, world = dist_env()
    if rank != 0:
        return
    wl = workload_for_rank(0)
    steps, warmup = max(1, args.steps), max(0, args.warmup)
    # keep the whole run to a few minutes: one oracle pass over ~64 tokens costs a few seconds
    budget_tokens = 64 if steps + warmup > 8 else 192
    r = time_oracle(wl, steps, warmup, budget_tokens)
    line = dict(impl="reference", metric=METRIC, value=r["value"], unit=UNIT, n_gpus=args.gpus, steps=steps,
                warmup=warmup, ms_per_step=r["ms_per_step"], higher_is_better=True, scaling="weak", vs_baseline=None,
                dtype="f64", data="synthetic",
                config=dict(workload="egtp_mid: 32 prompts lognormal(5.5,0.8) in [32,2048], d=2048, V=151936, "
                                     "head 2048->512->1", sample_tokens=r["tokens"]),
                cpu_baseline=dict(value=r["value"], unit=UNIT, cores=r["cores"], kind="oracle", sample=r["sample"]),
                e2e=dict(value=r["value"], unit=UNIT, h2d_bytes_per_step=0, d2h_bytes_per_step=0))
    print(json.dumps(line), flush=True)


# ------------------------------------------------------------------------------------------------
# the CUDA path
# ------------------------------------------------------------------------------------------------
def gpu_index(local_rank: int) -> int:
    vis = os.environ.get("CUDA_VISIBLE_DEVICES")
    try:
        return int(vis.split(",")[local_rank]) if vis else local_rank
    except (ValueError, IndexError):
        return local_rank


def run_mine(args):
    import torch
    import torch.distributed as dist

    from paper_2602_11812_b200 import binding as egtp
    from paper_2602_11812_b200 import device as gu
    from paper_2602_11812_b200 import shard

    rank, local_rank, world = dist_env()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the hot path has no CPU fallback")
    torch.cuda.set_device(local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    peaks = load_peaks()
    steps, warmup = max(1, args.steps), max(3, args.warmup)

    wl = workload_for_rank(rank)
    T, B, d, V = wl.T, wl.B, wl.d, wl.V
    hidden = gu.dev_tensor(wl.hidden, wl.dtype)
    W = gu.dev_tensor(wl.W, wl.dtype)
    head = gu.DeviceHead(wl.head, wl.dtype)
    offsets = torch.from_numpy(wl.offsets).cuda()
    lm = egtp.make_lm_head(W)
    ctx = egtp.egtp_create(local_rank, max_tokens=max(T, 1024), max_batch=max(B, 256), max_d=4096, max_V=V)
    yhat = torch.empty(B, device="cuda", dtype=torch.float32)
    status = torch.zeros(1, device="cuda", dtype=torch.int32)

    def step():
        egtp.egtp_predict(ctx, lm, head.c, hidden, offsets, B, T, wl.alpha, yhat_out=yhat, status_dev=status)

    def sync_all():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
            torch.cuda.synchronize()

    sampler = ClockSampler(gpu_index(local_rank))
    sampler.start()
    for _ in range(warmup):
        step()
    sync_all()
    assert int(status.item()) == 0, egtp.status_string(int(status.item()))

    # ---- timed region: K steps, device-timed on the launching stream (no per-kernel events in it: they cost a
    # few microseconds per launch)
    egtp.egtp_profile_enable(ctx, False)
    launches0 = egtp.egtp_launch_count(ctx)
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    sync_all()
    t_wall0 = time.time()
    ev0.record()
    for _ in range(steps):
        step()
    ev1.record()
    sync_all()
    t_wall1 = time.time()
    ms = ev0.elapsed_time(ev1)
    clocks = sampler.window(t_wall0, t_wall1)
    launches = egtp.egtp_launch_count(ctx) - launches0
    assert int(status.item()) == 0, egtp.status_string(int(status.item()))
    # ---- the same K steps once more with every kernel bracketed by events: per-kernel times for the roofline
    egtp.egtp_profile_enable(ctx, True)
    egtp.egtp_profile_read(ctx)
    for _ in range(steps):
        step()
    torch.cuda.synchronize()
    prof = egtp.egtp_profile_read(ctx)
    egtp.egtp_profile_enable(ctx, False)
    assert int(status.item()) == 0, egtp.status_string(int(status.item()))

    ms_max, tokens_all = shard.reduce_time_and_work(ms, float(T), torch.device("cuda", local_rank))
    value = tokens_all * steps / (ms_max * 1e-3)

    # ---- end to end through the host-buffer entry point (pinned host memory in, result out)
    hidden_host = gu.host_tensor(wl.hidden, wl.dtype)
    off_host = torch.from_numpy(wl.offsets).pin_memory()
    y_host = torch.empty(B, dtype=torch.float32).pin_memory()
    st_host = torch.zeros(1, dtype=torch.int32).pin_memory()
    e2e_steps = max(3, min(steps, 20))
    for _ in range(2):
        egtp.egtp_predict_host(ctx, lm, head.c, hidden_host, off_host, B, T, wl.alpha, y_host, None, st_host)
    sync_all()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(e2e_steps):
        egtp.egtp_predict_host(ctx, lm, head.c, hidden_host, off_host, B, T, wl.alpha, y_host, None, st_host)
    e1.record()
    sync_all()
    e2e_ms_max, _ = shard.reduce_time_and_work(e0.elapsed_time(e1), float(T), torch.device("cuda", local_rank))
    e2e_value = tokens_all * e2e_steps / (e2e_ms_max * 1e-3)
    h2d = hidden_host.numel() * 2 + off_host.numel() * 4
    d2h = y_host.numel() * 4 + 4

    # ---- context only: a library GEMM of the same shape (it also has to write the T x V logits), same run
    lib_gemm = None
    if world == 1:
        try:
            logits = torch.empty(T, V, device="cuda", dtype=torch.bfloat16)
            for _ in range(2):
                torch.matmul(hidden, W.t(), out=logits)
            torch.cuda.synchronize()
            m0, m1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            n_mm = 20
            m0.record()
            for _ in range(n_mm):
                torch.matmul(hidden, W.t(), out=logits)
            m1.record()
            torch.cuda.synchronize()
            mm_ms = m0.elapsed_time(m1) / n_mm
            lib_gemm = dict(what="torch.matmul (cuBLAS) bf16 [T,d] x [d,V] -> bf16 logits, no entropy", ms=mm_ms,
                            tflops=2.0 * d * V * T / (mm_ms * 1e-3) / 1e12)
            del logits
        except Exception as exc:
            lib_gemm = dict(error=str(exc)[:200])

    if rank != 0:
        egtp.egtp_destroy(ctx)
        sampler.stop()
        if world > 1:
            dist.destroy_process_group()
        return

    # ---- roofline of the dominant kernel: LM-head GEMM + online entropy, tensor-core bound
    k1 = prof["lmhead_entropy"]
    k1_ms = k1["ms"] / max(1, k1["launches"])
    flops = 2.0 * d * V * T                      # algorithmic flops of one launch: 2 d V per token
    achieved = flops / (k1_ms * 1e-3) / 1e12
    peak = peaks["bf16_tflops"] if ms < 2000 else peaks["bf16_tflops_sustained"]
    plan = egtp.egtp_lmhead_plan(ctx, T, d, V, egtp.EGTP_BF16)
    traffic = ncu_traffic("lmhead_entropy_egtp_mid", dict(tokens=T, d=d, V=V, chunks=plan["chunks"], grid=plan["grid"])) \
        if world == 1 else None
    roofline = dict(bound="tensor", kernel="lmhead_entropy", achieved=achieved, peak=peak, unit="TFLOP/s",
                    frac=achieved / peak, traffic=traffic,
                    algorithmic_bytes=2.0 * V * d + 2.0 * T * d, peak_source=peaks["source"],
                    ms_per_launch=k1_ms, frac_of_sustained=achieved / peaks["bf16_tflops_sustained"],
                    frac_of_nominal_2250=achieved / 2250.0,
                    mcycles_per_launch=cycles(k1_ms * 1e3, clocks), sm_mhz=clocks.get("sm_mhz"))
    kernels = {k: dict(ms_per_launch=v["ms"] / max(1, v["launches"]), launches=v["launches"]) for k, v in prof.items()
               if v["launches"]}

    line = dict(metric=METRIC, value=value, unit=UNIT, n_gpus=world, steps=steps, warmup=warmup,
                ms_per_step=ms_max / steps, higher_is_better=True, scaling="weak", vs_baseline=None, dtype="bf16",
                data="synthetic",
                config=dict(workload="egtp_mid: 32 prompts lognormal(5.5,0.8) clipped [32,2048] per GPU, d=2048 bf16 "
                                     "(1% outlier channels x20), LM head 151936x2048 bf16, head 2048->512->1",
                            tokens_per_gpu=T, prompts_per_gpu=B, d=d, V=V,
                            l2="inputs (622 MB LM head) larger than the 126 MB L2; no explicit flush",
                            lmhead_plan=plan, launches_per_step=launches / steps),
                clocks=clocks,
                e2e=dict(value=e2e_value, unit=UNIT, h2d_bytes_per_step=h2d, d2h_bytes_per_step=d2h,
                         steps=e2e_steps, api="egtp_predict_host"),
                gpu_launches=int(launches),
                roofline=roofline,
                kernels=kernels,
                library_gemm_same_shape=lib_gemm)

    egtp.egtp_destroy(ctx)
    del hidden, W
    legs = {}
    plp_wl = None
    if world == 1 and not args.no_plp:
        plp, long_, plp_wl = bench_d4096(local_rank, peaks, args.plp_steps, args.long_steps, sampler)
        line["plp_decode"], line["egtp_long"] = plp, long_
        # the parts of those legs that belong to the metric, where the rest of the line is kept
        legs["plp_decode"] = dict(
            metric="plp_decode_step_us", workload="256 live sequences, d=4096, V=151936, head 4096->256->1, state bound to its head",
            us_per_step_median=plp["us_per_step_median"], us_per_step_p10=plp["us_per_step_p10"],
            us_per_step_p90=plp["us_per_step_p90"], launches_per_step=plp["launches_per_step"],
            bound="hbm", unit="GB/s", peak=peaks["hbm_gbs"], kernel="lmhead_entropy_pair",
            kernel_us=plp["lmhead_us"], achieved=plp["hbm"]["achieved"], frac=plp["hbm"]["frac"],
            whole_step_frac=plp["hbm"]["whole_step_frac"], tensor_frac=plp["tensor"]["frac"],
            cuda_graph_us=plp.get("cuda_graph_us_per_step"), sm_mhz=plp["clocks"].get("sm_mhz"),
            mcycles_per_step=cycles(plp["us_per_step_median"], plp["clocks"]),
            e2e_us=plp.get("e2e", {}).get("us_per_step"), e2e_pipelined_us=plp.get("e2e", {}).get("pipelined_us_per_step"),
            unbound_us_per_step_median=plp["unbound_state"]["us_per_step_median"])
        fl = plp["from_logits"]
        legs["from_logits"] = dict(workload="[256, 151936] bf16 logits already in memory (3 buffers in rotation: larger than L2)",
                                   bound="hbm", unit="GB/s", peak=peaks["hbm_gbs"], kernel="logits_entropy",
                                   kernel_us=fl["entropy_call_us"], achieved=fl["hbm"]["achieved"], frac=fl["hbm"]["frac"],
                                   timing=fl["hbm"]["timing"], us_per_plp_step=fl["us_per_step"])
        legs["egtp_long"] = dict(metric=METRIC, workload=long_["workload"], tokens=long_["tokens"], value=long_["value"],
                                 ms_per_step=long_["ms_per_step"], bound="tensor", unit="TFLOP/s",
                                 peak=long_["lmhead"]["peak"], achieved=long_["lmhead"]["achieved"],
                                 frac=long_["lmhead"]["frac"], sm_mhz=long_["clocks"].get("sm_mhz"),
                                 mcycles_per_step=cycles(long_["ms_per_step"] * 1e3, long_["clocks"]))
        legs["pool"] = dict(workload="Eq. 3-4 pooling of the long-tailed batch (25629 tokens x 4096 bf16 = 210 MB)",
                            **long_["pool"])
    if world == 1 and not args.no_rl:
        rl = bench_rl_group(local_rank, peaks, min(args.plp_steps, 16), min(args.long_steps, 3), sampler)
        line["rl_group"] = rl
        legs["rl_group"] = dict(
            workload=rl["workload"], egtp_tokens=rl["egtp"]["tokens"], egtp_value=rl["egtp"]["value"],
            egtp_ms_per_step=rl["egtp"]["ms_per_step"], egtp_lmhead_frac=rl["egtp"]["lmhead"]["frac"],
            pool_frac=rl["egtp"]["pool"]["frac"], pool_us=rl["egtp"]["pool"]["us_per_launch"],
            plp_B1024_us_per_step=rl["plp_B1024"]["bound_to_head"]["us_per_step"],
            plp_B1024_lmhead_frac=rl["plp_B1024"]["bound_to_head"]["lmhead"]["frac"], bound="tensor",
            peak=peaks["bf16_tflops"], unit="TFLOP/s", sm_mhz=rl["egtp"]["clocks"].get("sm_mhz"))
    if legs:
        roofline["legs"] = legs
    sampler.stop()
    if world == 1 and not args.no_cpu:
        probe = time_oracle(wl, steps=1, warmup=0, max_tokens=256)          # one pass tells how many fit in ~15 s
        cb = time_oracle(wl, steps=int(min(40, max(2, 15.0 / (probe["ms_per_step"] * 1e-3)))), warmup=0, max_tokens=256)
        line["cpu_baseline"] = dict(value=cb["value"], unit=UNIT, cores=cb["cores"], kind="oracle", sample=cb["sample"])
        if plp_wl is not None:
            line["cpu_baseline"]["plp_decode_step"] = time_oracle_plp(plp_wl)
    if world > 1:
        dist.destroy_process_group()
    print(json.dumps(line), flush=True)


def bench_d4096(ctx_device: int, peaks, plp_steps: int, egtp_steps: int, sampler=None):
    """The two d = 4096 workloads, sharing one 151936 x 4096 bf16 LM head on the device.

    plp_decode: 256 live sequences, one token per step, head 4096 -> 256 -> 1, slots retire at
                lognormal(6, 1) lengths and restart empty (batch kept full).
    egtp_long:  64 prompts with Pareto(1.2) lengths clipped to [128, 8192], head 4096 -> 1024 -> 1;
                this is also where the pooling kernel is large enough (210 MB) to be HBM-bound.
    """
    import torch

    from paper_2602_11812_b200 import binding as egtp
    from paper_2602_11812_b200 import device as gu
    from paper_2602_11812_b200 import inputs as gen

    def window(t0, t1):
        return sampler.window(t0, t1) if sampler is not None else {}

    warm = 5
    wl = gen.config_plp_decode(steps=plp_steps + warm)
    slots, d, V = wl.slots, wl.d, wl.V
    W = gu.dev_tensor(wl.W, "bf16")
    lm = egtp.make_lm_head(W)
    wl3 = gen.config_long(W=wl.W)
    ctx = egtp.egtp_create(ctx_device, max_tokens=max(wl3.T, 1024), max_batch=slots, max_d=d, max_V=V)
    status = torch.zeros(1, device="cuda", dtype=torch.int32)

    # ---- PLP decode steps
    head = gu.DeviceHead(wl.head, "bf16")
    hs = gu.dev_tensor(wl.hidden_steps.reshape(-1, d), "bf16").reshape(plp_steps + warm, slots, d)
    reset = torch.from_numpy(wl.reset_src).cuda()
    yrem = torch.empty(slots, device="cuda", dtype=torch.float32)
    w_bytes = 2.0 * d * V

    def measure_steps(st):
        for t in range(warm):
            egtp.plp_step(ctx, st, lm, head.c, hs[t], reset_src=reset[t], yrem_out=yrem, status_dev=status)
        torch.cuda.synchronize()
        # pass 1: step times, no per-kernel events in the stream (they cost a few microseconds per step here);
        # every route starts its burst from an idle GPU (the power state of the previous burst carries over otherwise)
        egtp.egtp_profile_enable(ctx, False)
        time.sleep(0.5)
        for t in range(warm):
            egtp.plp_step(ctx, st, lm, head.c, hs[t], reset_src=None, yrem_out=yrem, status_dev=status)
        evs = [torch.cuda.Event(enable_timing=True) for _ in range(plp_steps + 1)]
        torch.cuda.synchronize()
        t0 = time.time()
        evs[0].record()
        for t in range(plp_steps):
            egtp.plp_step(ctx, st, lm, head.c, hs[warm + t], reset_src=reset[warm + t], yrem_out=yrem, status_dev=status)
            evs[t + 1].record()
        torch.cuda.synchronize()
        clk = window(t0, time.time())
        # pass 2: the same steps again with every kernel bracketed by events (per-kernel breakdown)
        egtp.egtp_profile_enable(ctx, True)
        egtp.egtp_profile_read(ctx)
        for t in range(plp_steps):
            egtp.plp_step(ctx, st, lm, head.c, hs[warm + t], reset_src=reset[warm + t], yrem_out=yrem, status_dev=status)
        torch.cuda.synchronize()
        prof = egtp.egtp_profile_read(ctx)
        assert int(status.item()) == 0
        per_step = np.array([evs[i].elapsed_time(evs[i + 1]) * 1e3 for i in range(plp_steps)])
        k1_us = prof["lmhead_entropy"]["ms"] / prof["lmhead_entropy"]["launches"] * 1e3
        step_us = float(np.median(per_step))
        return dict(us_per_step_median=step_us, us_per_step_p10=float(np.percentile(per_step, 10)),
                    us_per_step_p90=float(np.percentile(per_step, 90)), lmhead_us=k1_us, clocks=clk,
                    hbm=dict(bound="hbm", kernel="lmhead_entropy", achieved=w_bytes / (k1_us * 1e-6) / 1e9,
                             peak=peaks["hbm_gbs"], unit="GB/s", frac=w_bytes / (k1_us * 1e-6) / 1e9 / peaks["hbm_gbs"],
                             whole_step_frac=w_bytes / (step_us * 1e-6) / 1e9 / peaks["hbm_gbs"]),
                    tensor=dict(achieved=2.0 * slots * d * V / (k1_us * 1e-6) / 1e12, peak=peaks["bf16_tflops"],
                                unit="TFLOP/s", frac=2.0 * slots * d * V / (k1_us * 1e-6) / 1e12 / peaks["bf16_tflops"]),
                    kernels_us={k: v["ms"] / v["launches"] * 1e3 for k, v in prof.items() if v["launches"]},
                    launches_per_step=sum(v["launches"] for v in prof.values()) / plp_steps)

    # the ordinary route first (head layer 1 as its own GEMM over z), then the state bound to its head
    # (W1 h' from the LM-head kernel's extra columns; one kernel finishes the step): the headline numbers
    st_plain = egtp.plp_state_create(ctx, slots, d)
    plain = measure_steps(st_plain)
    egtp.plp_state_destroy(st_plain)
    st = egtp.plp_state_create(ctx, slots, d)
    egtp.plp_state_bind_head(st, head.c)
    plp = dict(metric="plp_decode_step_us", B=slots, d=d, V=V, steps=plp_steps,
               route="state bound to its head (plp_state_bind_head)")
    plp.update(measure_steps(st))
    plp["plan"] = egtp.egtp_lmhead_plan(ctx, slots, d, V, egtp.EGTP_BF16)
    plp["unbound_state"] = plain
    # ---- the same bound step end to end: the step's hidden rows come from pinned host memory, the predictions go back
    try:
        n_e2e = min(plp_steps, 32)
        hs_host = [gu.host_tensor(wl.hidden_steps[warm + t], "bf16") for t in range(n_e2e)]
        rs_host = [torch.from_numpy(wl.reset_src[warm + t].copy()).pin_memory() for t in range(n_e2e)]
        y_host = torch.empty(slots, dtype=torch.float32).pin_memory()
        st_host = torch.zeros(1, dtype=torch.int32).pin_memory()
        egtp.egtp_profile_enable(ctx, False)
        for t in range(3):
            egtp.plp_step_host(ctx, st, lm, head.c, hs_host[t], rs_host[t], None, None, None, 0, slots, 1.0, y_host, st_host)
        t0 = time.perf_counter()
        for t in range(n_e2e):
            egtp.plp_step_host(ctx, st, lm, head.c, hs_host[t], rs_host[t], None, None, None, 0, slots, 1.0, y_host, st_host)
        t1 = time.perf_counter()          # plp_step_host synchronises its stream before it returns
        assert int(st_host.item()) == 0
        plp["e2e"] = dict(us_per_step=(t1 - t0) / n_e2e * 1e6, steps=n_e2e, api="plp_step_host",
                          h2d_bytes_per_step=slots * d * 2 + slots * 4, d2h_bytes_per_step=slots * 4 + 4)
        # the same steps handed over without waiting in between (plp_step_host_async: the copy of step t + 1 runs
        # next to the kernels of step t); every step still gets its rows from pinned host memory and returns its predictions
        ys = [torch.empty(slots, dtype=torch.float32).pin_memory() for _ in range(n_e2e)]
        sts = [torch.zeros(1, dtype=torch.int32).pin_memory() for _ in range(n_e2e)]
        for t in range(3):
            egtp.plp_step_host_async(ctx, st, lm, head.c, hs_host[t], rs_host[t], None, None, None, 0, slots, 1.0, ys[t], sts[t])
        torch.cuda.synchronize()
        p0, p1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        t0 = time.perf_counter()
        p0.record()
        for t in range(n_e2e):
            egtp.plp_step_host_async(ctx, st, lm, head.c, hs_host[t], rs_host[t], None, None, None, 0, slots, 1.0, ys[t], sts[t])
        p1.record()
        torch.cuda.synchronize()
        t1 = time.perf_counter()
        assert all(int(x.item()) == 0 for x in sts)
        plp["e2e"]["pipelined_us_per_step"] = p0.elapsed_time(p1) / n_e2e * 1e3
        plp["e2e"]["pipelined_wall_us_per_step"] = (t1 - t0) / n_e2e * 1e6
        plp["e2e"]["pipelined_api"] = "plp_step_host_async"
        egtp.egtp_profile_enable(ctx, True)
    except Exception as exc:
        plp["e2e"] = dict(error=str(exc)[:200])

    # ---- context only: a library GEMM of the decode shape (writes the [256, V] logits, no entropy)
    try:
        lg = torch.empty(slots, V, device="cuda", dtype=torch.bfloat16)
        for t in range(3):
            torch.matmul(hs[t], W.t(), out=lg)
        torch.cuda.synchronize()
        c0, c1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        c0.record()
        for t in range(plp_steps):
            torch.matmul(hs[warm + t], W.t(), out=lg)
        c1.record()
        torch.cuda.synchronize()
        mm_us = c0.elapsed_time(c1) / plp_steps * 1e3
        plp["library_gemm_same_shape"] = dict(what="torch.matmul (cuBLAS) bf16 [256,d] x [d,V] -> bf16 logits", us=mm_us,
                                              w_stream_gbs=w_bytes / (mm_us * 1e-6) / 1e9)
        del lg
    except Exception as exc:
        plp["library_gemm_same_shape"] = dict(error=str(exc)[:200])

    # ---- the same step captured once in a CUDA graph and replayed (fixed buffers; removes launch gaps)
    try:
        static_h = hs[warm].clone()
        static_r = reset[warm].clone()
        static_r.fill_(-2)                       # keep: replays continue the running state
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):
            egtp.plp_step(ctx, st, lm, head.c, static_h, reset_src=static_r, yrem_out=yrem, status_dev=status)
        torch.cuda.current_stream().wait_stream(side)
        torch.cuda.synchronize()
        egtp.egtp_profile_enable(ctx, False)
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph):
            egtp.plp_step(ctx, st, lm, head.c, static_h, reset_src=static_r, yrem_out=yrem, status_dev=status)
        for _ in range(3):
            graph.replay()
        torch.cuda.synchronize()
        g0, g1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        g0.record()
        for t in range(plp_steps):
            static_h.copy_(hs[warm + t], non_blocking=True)      # the step's new tokens (2 MB device copy)
            graph.replay()
        g1.record()
        torch.cuda.synchronize()
        plp["cuda_graph_us_per_step"] = g0.elapsed_time(g1) / plp_steps * 1e3
        del graph
    except Exception as exc:  # capture is a convenience measurement, never a requirement
        plp["cuda_graph_us_per_step"] = None
        plp["cuda_graph_error"] = str(exc)[:200]
    egtp.egtp_profile_enable(ctx, True)
    assert int(status.item()) == 0

    # ---- the same decode step when the serving engine already holds the step's logits.  Three logits buffers are
    # used in rotation (233 MB, larger than L2), so every pass really streams its 78 MB from HBM.
    torch.manual_seed(0)
    logit_bufs = [(torch.randn(slots, V, device="cuda") * 1.5).to(torch.bfloat16) for _ in range(3)]
    n_fl = max(9, plp_steps)

    def measure_from_logits(state):
        def steps_():
            for t in range(n_fl):
                egtp.plp_step_from_logits(ctx, state, logit_bufs[t % 3], head.c, hs[warm + t % plp_steps],
                                          reset_src=reset[warm + t % plp_steps], yrem_out=yrem, status_dev=status)
        for t in range(3):
            egtp.plp_step_from_logits(ctx, state, logit_bufs[t], head.c, hs[t], reset_src=reset[t], yrem_out=yrem, status_dev=status)
        torch.cuda.synchronize()
        egtp.egtp_profile_enable(ctx, False)
        f0, f1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        f0.record()
        steps_()
        f1.record()
        torch.cuda.synchronize()
        egtp.egtp_profile_enable(ctx, True)
        egtp.egtp_profile_read(ctx)
        steps_()
        torch.cuda.synchronize()
        prof_fl = egtp.egtp_profile_read(ctx)
        assert int(status.item()) == 0
        return dict(us_per_step=f0.elapsed_time(f1) / n_fl * 1e3,
                    logits_entropy_us_event_bracketed=prof_fl["logits_entropy"]["ms"] / prof_fl["logits_entropy"]["launches"] * 1e3,
                    kernels_us={k: v["ms"] / v["launches"] * 1e3 for k, v in prof_fl.items() if v["launches"]})

    # bound state: W1 h' from a launch of the LM-head kernel over the head columns alone (reported as head_hidden)
    plp["from_logits"] = measure_from_logits(st)
    st_plain = egtp.plp_state_create(ctx, slots, d)
    plp["from_logits"]["unbound_state"] = measure_from_logits(st_plain)
    egtp.plp_state_destroy(st_plain)
    # The entropy kernel by itself: egtp_entropy_from_logits is one launch, so a CUDA graph of 12 calls over the
    # rotating buffers, replayed, times the kernel without the few microseconds an event pair around a 20 us kernel adds.
    Hfl = torch.empty(slots, device="cuda", dtype=torch.float32)
    egtp.egtp_profile_enable(ctx, False)
    try:
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):
            for i in range(3):
                egtp.egtp_entropy_from_logits(ctx, logit_bufs[i], Hfl, status_dev=status)
        torch.cuda.current_stream().wait_stream(side)
        torch.cuda.synchronize()
        calls = 12
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph):
            for i in range(calls):
                egtp.egtp_entropy_from_logits(ctx, logit_bufs[i % 3], Hfl, status_dev=status)
        for _ in range(2):
            graph.replay()
        torch.cuda.synchronize()
        q0, q1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        reps = 10
        q0.record()
        for _ in range(reps):
            graph.replay()
        q1.record()
        torch.cuda.synchronize()
        call_us = q0.elapsed_time(q1) / (reps * calls) * 1e3
        timing = "CUDA graph of 12 single-launch calls over 3 rotating buffers, replayed 10 times"
        del graph
    except Exception as exc:
        call_us = plp["from_logits"]["logits_entropy_us_event_bracketed"]
        timing = f"event-bracketed launches (graph capture failed: {str(exc)[:80]})"
    le_gbs = 2.0 * slots * V / (call_us * 1e-6) / 1e9
    plp["from_logits"]["entropy_call_us"] = call_us
    plp["from_logits"]["hbm"] = dict(bound="hbm", kernel="logits_entropy", achieved=le_gbs, peak=peaks["hbm_gbs"], unit="GB/s",
                                     frac=le_gbs / peaks["hbm_gbs"], bytes_per_row=2 * V, timing=timing)
    egtp.egtp_profile_enable(ctx, True)
    egtp.plp_state_destroy(st)
    del hs, logit_bufs

    # ---- EGTP over the long-tailed prompt batch
    hidden = gu.dev_tensor(wl3.hidden, "bf16")
    head3 = gu.DeviceHead(wl3.head, "bf16")
    off = torch.from_numpy(wl3.offsets).cuda()
    yhat = torch.empty(wl3.B, device="cuda", dtype=torch.float32)
    for _ in range(3):
        egtp.egtp_predict(ctx, lm, head3.c, hidden, off, wl3.B, wl3.T, 1.0, yhat_out=yhat, status_dev=status)
    torch.cuda.synchronize()
    egtp.egtp_profile_enable(ctx, False)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t0 = time.time()
    e0.record()
    for _ in range(egtp_steps):
        egtp.egtp_predict(ctx, lm, head3.c, hidden, off, wl3.B, wl3.T, 1.0, yhat_out=yhat, status_dev=status)
    e1.record()
    torch.cuda.synchronize()
    clk3 = window(t0, time.time())
    ms_step = e0.elapsed_time(e1) / egtp_steps
    egtp.egtp_profile_enable(ctx, True)
    egtp.egtp_profile_read(ctx)
    for _ in range(egtp_steps):
        egtp.egtp_predict(ctx, lm, head3.c, hidden, off, wl3.B, wl3.T, 1.0, yhat_out=yhat, status_dev=status)
    torch.cuda.synchronize()
    prof3 = egtp.egtp_profile_read(ctx)
    assert int(status.item()) == 0
    k1_ms = prof3["lmhead_entropy"]["ms"] / prof3["lmhead_entropy"]["launches"]
    pool_us = prof3["pool"]["ms"] / prof3["pool"]["launches"] * 1e3
    tf = 2.0 * d * V * wl3.T / (k1_ms * 1e-3) / 1e12
    pool_gbs = (2.0 * d + 4.0) * wl3.T / (pool_us * 1e-6) / 1e9
    long_ = dict(metric=METRIC, workload="egtp_long: 64 prompts Pareto(1.2) in [128,8192], d=4096, V=151936, head 4096->1024->1",
                 tokens=wl3.T, steps=egtp_steps, ms_per_step=ms_step, value=wl3.T / (ms_step * 1e-3), unit=UNIT, clocks=clk3,
                 lmhead=dict(bound="tensor", achieved=tf, peak=peaks["bf16_tflops"], unit="TFLOP/s",
                             frac=tf / peaks["bf16_tflops"], ms_per_launch=k1_ms),
                 pool=dict(bound="hbm", kernel="pool", achieved=pool_gbs, peak=peaks["hbm_gbs"], unit="GB/s",
                           frac=pool_gbs / peaks["hbm_gbs"], us_per_launch=pool_us,
                           bytes_per_token=2 * d + 4, timing="event-bracketed launches"),
                 kernels_us={k: v["ms"] / v["launches"] * 1e3 for k, v in prof3.items() if v["launches"]},
                 launches_per_step=sum(v["launches"] for v in prof3.values()) / egtp_steps,
                 plan=egtp.egtp_lmhead_plan(ctx, wl3.T, d, V, egtp.EGTP_BF16))
    # ---- the paper's pooling comparators (Table 3) on the same batch: pooling alone, no LM head
    comp = {}
    pooled = torch.empty(wl3.B, d, device="cuda", dtype=torch.float32)
    for name, mode in (("mean", egtp.EGTP_POOL_MEAN), ("max", egtp.EGTP_POOL_MAX), ("last", egtp.EGTP_POOL_LAST)):
        for _ in range(3):
            egtp.egtp_pool_baseline(ctx, None, hidden, off, wl3.B, wl3.T, mode, pooled_out=pooled, status_dev=status)
        torch.cuda.synchronize()
        egtp.egtp_profile_read(ctx)
        for _ in range(10):
            egtp.egtp_pool_baseline(ctx, None, hidden, off, wl3.B, wl3.T, mode, pooled_out=pooled, status_dev=status)
        pr = egtp.egtp_profile_read(ctx)
        us = pr["pool"]["ms"] / pr["pool"]["launches"] * 1e3
        touched = 2.0 * d * (wl3.B if name == "last" else wl3.T)      # last-token pooling reads one row per prompt
        comp[name] = dict(pool_us=us, gbs=touched / (us * 1e-6) / 1e9)
    long_["pooling_comparators"] = comp
    assert int(status.item()) == 0
    egtp.egtp_destroy(ctx)
    return plp, long_, wl


def bench_rl_group(ctx_device: int, peaks, plp_steps: int, egtp_steps: int, sampler=None):
    """RL group sampling at its full sizes: EGTP over 64 shared prompts (d = 5120, V = 152064), then PLP steps over
    1024 decode streams that start from their prompt's state (tensor-bound: 8 row blocks of 128 rows per step)."""
    import torch

    from paper_2602_11812_b200 import binding as egtp
    from paper_2602_11812_b200 import device as gu
    from paper_2602_11812_b200 import inputs as gen

    warm = 3
    wl = gen.config_rl_group(steps=warm + plp_steps)
    eg = wl.prompts
    slots, d, V = wl.slots, wl.d, wl.V
    W = gu.dev_tensor(wl.W, "bf16")
    lm = egtp.make_lm_head(W)
    head = gu.DeviceHead(wl.head, "bf16")
    # no host staging: this leg calls the device-pointer entry points only (the staging copy would be 2.8 GB)
    ctx = egtp.egtp_create_ex(ctx_device, max_tokens=eg.T, max_batch=slots, max_d=d, max_V=V,
                              flags=egtp.EGTP_CREATE_NO_HOST_STAGING)
    status = torch.zeros(1, device="cuda", dtype=torch.int32)
    f = dict(device="cuda", dtype=torch.float32)
    # ---- EGTP over the shared prompts
    hidden = gu.dev_tensor(eg.hidden, "bf16")
    off = torch.from_numpy(eg.offsets).cuda()
    yhat, pooled = torch.empty(eg.B, **f), torch.empty(eg.B, d, **f)
    sm, ss = torch.empty(eg.B, **f), torch.empty(eg.B, **f)

    def predict():
        egtp.egtp_predict(ctx, lm, head.c, hidden, off, eg.B, eg.T, 1.0, pooled_out=pooled, state_m_out=sm,
                          state_s_out=ss, yhat_out=yhat, status_dev=status)

    predict()
    torch.cuda.synchronize()
    egtp.egtp_profile_enable(ctx, True)
    egtp.egtp_profile_read(ctx)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t0 = time.time()
    e0.record()
    for _ in range(egtp_steps):
        predict()
    e1.record()
    torch.cuda.synchronize()
    clk = sampler.window(t0, time.time()) if sampler is not None else {}
    prof = egtp.egtp_profile_read(ctx)
    ms_step = e0.elapsed_time(e1) / egtp_steps
    k1_ms = prof["lmhead_entropy"]["ms"] / prof["lmhead_entropy"]["launches"]
    tf = 2.0 * d * V * eg.T / (k1_ms * 1e-3) / 1e12
    pool_us = prof["pool"]["ms"] / prof["pool"]["launches"] * 1e3
    out = dict(workload="rl_group: 64 prompts U[256,4096] x 16 streams, d=5120, V=152064, head 5120->512->1",
               workspace_bytes=egtp.egtp_workspace_bytes(ctx),
               egtp=dict(tokens=eg.T, steps=egtp_steps, ms_per_step=ms_step, value=eg.T / (ms_step * 1e-3), unit=UNIT, clocks=clk,
                         lmhead=dict(bound="tensor", achieved=tf, peak=peaks["bf16_tflops"], unit="TFLOP/s",
                                     frac=tf / peaks["bf16_tflops"], ms_per_launch=k1_ms),
                         pool=dict(bound="hbm", us_per_launch=pool_us, achieved=(2.0 * d + 4.0) * eg.T / (pool_us * 1e-6) / 1e9,
                                   peak=peaks["hbm_gbs"], unit="GB/s",
                                   frac=(2.0 * d + 4.0) * eg.T / (pool_us * 1e-6) / 1e9 / peaks["hbm_gbs"]),
                         kernels_us={k: v["ms"] / v["launches"] * 1e3 for k, v in prof.items() if v["launches"]}))
    del hidden
    # ---- PLP over the 1024 streams: ordinary route, then the state bound to the head
    hs = gu.dev_tensor(wl.hidden_steps.reshape(-1, d), "bf16").reshape(warm + plp_steps, slots, d)
    reset0 = torch.from_numpy(wl.reset_src[0].copy()).cuda()
    yrem = torch.empty(slots, **f)

    def measure(bind):
        st = egtp.plp_state_create(ctx, slots, d)
        if bind:
            egtp.plp_state_bind_head(st, head.c)
        # step 0 starts every stream from its prompt's EGTP state; later steps pass no reset table
        egtp.plp_step(ctx, st, lm, head.c, hs[0], reset_src=reset0, src_m=sm, src_s=ss, src_pooled=pooled, n_src=eg.B,
                      yrem_out=yrem, status_dev=status)
        for t in range(1, warm):
            egtp.plp_step(ctx, st, lm, head.c, hs[t], yrem_out=yrem, status_dev=status)
        torch.cuda.synchronize()
        egtp.egtp_profile_enable(ctx, False)
        time.sleep(0.5)       # both routes start their burst from an idle GPU (the power state carries over otherwise)
        for t in range(1, warm):
            egtp.plp_step(ctx, st, lm, head.c, hs[t], yrem_out=yrem, status_dev=status)
        a0, a1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a0.record()
        for t in range(plp_steps):
            egtp.plp_step(ctx, st, lm, head.c, hs[warm + t], yrem_out=yrem, status_dev=status)
        a1.record()
        torch.cuda.synchronize()
        egtp.egtp_profile_enable(ctx, True)
        egtp.egtp_profile_read(ctx)
        for t in range(plp_steps):
            egtp.plp_step(ctx, st, lm, head.c, hs[warm + t], yrem_out=yrem, status_dev=status)
        torch.cuda.synchronize()
        pr = egtp.egtp_profile_read(ctx)
        egtp.plp_state_destroy(st)
        us = a0.elapsed_time(a1) / plp_steps * 1e3
        k_us = pr["lmhead_entropy"]["ms"] / pr["lmhead_entropy"]["launches"] * 1e3
        tfl = 2.0 * slots * d * V / (k_us * 1e-6) / 1e12
        return dict(us_per_step=us, lmhead=dict(bound="tensor", achieved=tfl, peak=peaks["bf16_tflops"], unit="TFLOP/s",
                                                frac=tfl / peaks["bf16_tflops"], us_per_launch=k_us),
                    kernels_us={k: v["ms"] / v["launches"] * 1e3 for k, v in pr.items() if v["launches"]})

    out["plp_B1024"] = dict(steps=plp_steps, ordinary=measure(False), bound_to_head=measure(True))
    assert int(status.item()) == 0
    egtp.egtp_destroy(ctx)
    return out


def run_vocab_parallel(args):
    """The PLP decode step (256 live sequences, d = 4096, V = 151936) with the LM head's rows sharded over the ranks:
    every rank reduces its shard to one (m, s, t2) triple per row, one all-gather of rows x 3 floats per rank
    exchanges them (NCCL), every rank merges and advances its replica of the state.  One JSON line from rank 0;
    at N = 1 the shard is the whole vocabulary and the exchange is skipped."""
    import torch
    import torch.distributed as dist

    from paper_2602_11812_b200 import binding as egtp
    from paper_2602_11812_b200 import device as gu
    from paper_2602_11812_b200 import inputs as gen
    from paper_2602_11812_b200 import shard

    rank, local_rank, world = dist_env()
    torch.cuda.set_device(local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    peaks = load_peaks()
    steps, warmup = max(1, args.steps), max(3, args.warmup)
    wl = gen.config_plp_decode(steps=steps + warmup)
    slots, d, V = wl.slots, wl.d, wl.V
    v0, v1 = shard.vocab_shards(V, world)[rank]
    W = gu.dev_tensor(wl.W[v0:v1], "bf16")
    lm = egtp.make_lm_head(W)
    head = gu.DeviceHead(wl.head, "bf16")
    ctx = egtp.egtp_create(local_rank, max_tokens=1024, max_batch=slots, max_d=d, max_V=V)
    st = egtp.plp_state_create(ctx, slots, d)
    egtp.plp_state_bind_head(st, head.c)
    hs = gu.dev_tensor(wl.hidden_steps.reshape(-1, d), "bf16").reshape(steps + warmup, slots, d)
    reset = torch.from_numpy(wl.reset_src).cuda()
    yrem = torch.empty(slots, device="cuda", dtype=torch.float32)
    status = torch.zeros(1, device="cuda", dtype=torch.int32)
    partial = torch.empty(slots, 3, device="cuda", dtype=torch.float32)

    def step(t):
        shard.plp_step_vocab_parallel(ctx, st, lm, head.c, hs[t], partial_buf=partial, reset_src=reset[t], yrem_out=yrem,
                                      status_dev=status)

    def sync_all():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
            torch.cuda.synchronize()

    for t in range(warmup):
        step(t)
    sync_all()
    sampler = ClockSampler(gpu_index(local_rank))
    sampler.start()
    launches0 = egtp.egtp_launch_count(ctx)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    sync_all()
    t0 = time.time()
    e0.record()
    for t in range(steps):
        step(warmup + t)
    e1.record()
    sync_all()
    clocks = sampler.window(t0, time.time())
    sampler.stop()
    assert int(status.item()) == 0
    ms_max, _ = shard.reduce_time_and_work(e0.elapsed_time(e1), 1.0, torch.device("cuda", local_rank))
    us = ms_max / steps * 1e3
    if rank == 0:
        shard_bytes = 2.0 * d * (v1 - v0)
        print(json.dumps(dict(
            metric="plp_decode_step_us_vocab_parallel", value=us, unit="us", n_gpus=world, steps=steps, warmup=warmup,
            ms_per_step=us * 1e-3, higher_is_better=False, scaling="strong", vs_baseline=None, dtype="bf16", data="synthetic",
            config=dict(workload="plp_decode: 256 live sequences, d=4096, V=151936 sharded by rows over the ranks, head 4096->256->1",
                        vocab_rows_per_rank=v1 - v0, exchange="all-gather of [256, 3] fp32 per rank and step" if world > 1 else "none (one rank)"),
            clocks=clocks, gpu_launches=int(egtp.egtp_launch_count(ctx) - launches0),
            roofline=dict(bound="hbm", kernel="lmhead_entropy (one vocabulary shard)", achieved=shard_bytes / (us * 1e-6) / 1e9,
                          peak=peaks["hbm_gbs"], unit="GB/s", frac=shard_bytes / (us * 1e-6) / 1e9 / peaks["hbm_gbs"], traffic=None,
                          note="whole step (its launches and the exchange) against this rank's share of the W stream"))), flush=True)
    egtp.plp_state_destroy(st)
    egtp.egtp_destroy(ctx)
    if world > 1:
        dist.destroy_process_group()


def ensure_library():
    """Builds the CUDA library if it is missing or older than its sources (a no-op otherwise).  Under torchrun
    only local rank 0 compiles; the other ranks wait for the finished file."""
    from paper_2602_11812_b200 import build as _build
    if int(os.environ.get("LOCAL_RANK", "0")) == 0:
        _build.ensure()
        return
    deadline = time.time() + 600
    while not _build.up_to_date():
        if time.time() > deadline:
            raise SystemExit("bench.py: the CUDA library was not built in time")
        time.sleep(1.0)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="mine", choices=["mine", "reference"])
    ap.add_argument("--plp-steps", type=int, default=64)
    ap.add_argument("--long-steps", type=int, default=10)
    ap.add_argument("--no-plp", action="store_true", help="skip the d = 4096 workloads (PLP decode, long prompts)")
    ap.add_argument("--no-rl", action="store_true", help="skip the RL group-sampling sizes (d = 5120, 1024 streams)")
    ap.add_argument("--only-d4096", action="store_true",
                    help="run only the d = 4096 workloads and print their two objects as one JSON line "
                         "(used for profiler captures of the decode and pooling kernels)")
    ap.add_argument("--no-cpu", action="store_true")
    ap.add_argument("--only-rl-group", action="store_true",
                    help="run only the RL group-sampling sizes (d = 5120, V = 152064, 1024 streams) and print one JSON line")
    ap.add_argument("--vocab-parallel", action="store_true",
                    help="time the PLP decode step with the LM head's rows sharded over the ranks")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
        return
    ensure_library()
    if args.vocab_parallel:
        run_vocab_parallel(args)
        return
    if args.only_rl_group:
        import torch
        torch.cuda.set_device(0)
        print(json.dumps(dict(rl_group=bench_rl_group(0, load_peaks(), min(args.plp_steps, 16), min(args.long_steps, 3)))),
              flush=True)
        return
    if args.only_d4096:
        import torch
        torch.cuda.set_device(0)
        plp, long_, _ = bench_d4096(0, load_peaks(), args.plp_steps, args.long_steps)
        print(json.dumps(dict(plp_decode=plp, egtp_long=long_)), flush=True)
        return
    run_mine(args)


if __name__ == "__main__":
    main()

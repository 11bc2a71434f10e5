#!/usr/bin/env python
"""Benchmark of the compressed decode-attention hot path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config NAME] [--impl reference]

One "step" is one pass of the whole hot path over every unit of the workload:
sh_decode_step (append + attention + importance-record update) for each layer's
handle, plus the compression (select-m + compaction) whenever the cache fills.
The default workload is the OPT-66B-shaped one the headline metric is quoted on
(batch 128 x 72 heads, head_dim 128, fp16 K/V, B=410, prompt 2048); the prompt is
streamed through the same path, untimed, before the timed decode steps.

The timed window of K steps is run REPEATS times, each time from the restored
post-prompt state and after W warm-up steps, so every repetition covers the same
stream positions; `value` is the median repetition (steps/s with inputs resident
in HBM), `repeats` lists them all.  A window may or may not contain a compression
(the cache fills every m steps), so the cost of one compression is also measured
on its own from a restored state with a full cache (`compress`), in the
compaction mode the run uses and in the other one.

Prints ONE JSON line.  `e2e` = the same metric through sh_decode_step_host with
pinned host buffers (copies inside the timed region); `roofline` = algorithmic
K+V bytes of the fused decode kernel per launch / its mean CUDA-event duration,
against the measured HBM copy peak; `cpu_baseline` = the CPU oracle timed on this
box's host cores on a bounded sample.  `--impl reference` times only that oracle.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

import torch  # noqa: E402

from paper_2305_17118_b200 import workloads as wl  # noqa: E402

METRIC = "compressed_decode_attn_steps_per_s"
UNIT = "steps/s"
L2_BYTES = 126 * 1024 * 1024
FALLBACK_HBM_GBS = 6650.0
REPEATS = 3
ES = {"f32": 4.0, "f16": 2.0, "bf16": 2.0, "int4": 0.5 + 2.0 / 64.0}
# int4 decode kernels: warp instructions x 32 / stored bytes read, from their ncu captures (profiles/)
INT4_LANE_INSTR_PER_BYTE = {"sh_decode_int4_mma_kernel": 7.4, "sh_decode_kernel": 10.0}


def measured_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured (MEASURED_PEAKS.json hbm_gbs)"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback (6.65 TB/s, earlier measurement on this pool)"


class ClockSampler:
    """SM clock and throttle reasons sampled through NVML (read-only) while the
    timed region runs."""

    def __init__(self, index: int, period_s: float = 0.001):
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop = threading.Event()
        self._thr = None
        self.period = period_s
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM))
        except Exception:
            self.nv = None

    def _reasons(self):
        nv = self.nv
        get = getattr(nv, "nvmlDeviceGetCurrentClocksEventReasons", None) or nv.nvmlDeviceGetCurrentClocksThrottleReasons
        bits = int(get(self.h))
        names = {
            "sw_power_cap": 0x4, "hw_slowdown": 0x8, "sync_boost": 0x10, "sw_thermal_slowdown": 0x20,
            "hw_thermal_slowdown": 0x40, "hw_power_brake_slowdown": 0x80, "applications_clocks_setting": 0x2,
        }
        return {k for k, b in names.items() if bits & b}

    def _run(self):
        while not self._stop.is_set():
            try:
                self.samples.append(int(self.nv.nvmlDeviceGetClockInfo(self.h, self.nv.NVML_CLOCK_SM)))
                self.reasons |= self._reasons()
            except Exception:
                pass
            time.sleep(self.period)

    def __enter__(self):
        if self.nv:
            self._stop.clear()
            self._thr = threading.Thread(target=self._run, daemon=True)
            self._thr.start()
        return self

    def __exit__(self, *a):
        self._stop.set()
        if self._thr:
            self._thr.join()
            self._thr = None

    def summary(self):
        if not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": ["unavailable"], "samples": 0}
        return {"sm_mhz": statistics.median(self.samples), "sm_max_mhz": self.max_mhz,
                "reasons": sorted(self.reasons), "samples": len(self.samples)}


def job_throughput(local_ms: float, steps: int, world: int, dist=None, device=None):
    """Whole-job steps/s when every rank ran `steps` steps of its own replica of the
    workload: the slowest rank's device time decides (max over ranks), and the job
    processed world x the units of one replica.  Returns (ms_per_step, steps_per_s)."""
    ms = float(local_ms)
    if dist is not None and world > 1:
        t = torch.tensor([ms], dtype=torch.float64, device=device)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        ms = float(t.item())
    per_step = ms / steps
    return per_step, world * 1e3 / per_step


def live_rows_schedule(cfg, first_step: int, count: int):
    """n (rows attended, new token included) at stream steps first_step.. ; the
    schedule is data-independent: n grows by one per step and drops by m when it reaches B."""
    n, out = 0, []
    for t in range(1, first_step + count):
        n += 1
        if t >= first_step:
            out.append(n)
        if n == cfg.B:
            n -= cfg.m
    return out


def config_record(cfg, args, world: int):
    """The `config` object of the JSON line: the same keys and values in both arms."""
    kv_bytes = 2 * cfg.layers * cfg.units * cfg.B * cfg.head_dim * ES[cfg.dtype]
    return {"workload": cfg.name, "batch": cfg.batch, "heads": cfg.heads, "layers": cfg.layers,
            "units": cfg.units * cfg.layers, "head_dim": cfg.head_dim, "kv_dtype": cfg.dtype, "B": cfg.B, "r": cfg.r,
            "w": cfg.w, "m": cfg.m, "prompt": cfg.prompt,
            "record": "recomputed at compression" if args.recompute_record else "online",
            "compaction": "stable" if args.stable_compaction else "hole filling (library default)",
            "l2": "flushed between steps (a buffer of twice its size written, then another one read)" if kv_bytes < 2 * L2_BYTES else "inputs larger than L2",
            "kv_bytes": kv_bytes, "parallelism": f"units replicated x{world}" if world > 1 else "1 GPU"}


# --------------------------------------------------------------------------- CPU oracle arm
def oracle_run(cfg, steps: int, warmup: int, sample_units: int, min_seconds: float = 0.0, budget_s: float = 60.0):
    """Times the CPU oracle (as it stands) on `sample_units` units: an untimed
    run-in of B + warmup tokens to reach the steady-state saw-tooth, then at least
    `steps` timed steps (more, until `min_seconds` of CPU work, never beyond
    `budget_s`).  Inputs cycle through 64 pre-drawn steps.  Returns (steps/s scaled
    to all units, info, seconds per step)."""
    import oracle
    U = min(sample_units, cfg.units)
    st = wl.Stream(cfg.scaled(units=U), device="cpu")
    orc = oracle.Oracle(U, cfg.B, cfg.r, cfg.w, cfg.m, cfg.head_dim, quant=(cfg.dtype == "int4"))
    f64 = lambda x: x.to(torch.float64).numpy()
    run_in = cfg.B + warmup
    for t in range(1, run_in + 1):
        q, k, v = st.step(t)
        orc.step(f64(q), f64(k), f64(v))
    pre = [tuple(f64(x) for x in st.step(run_in + 1 + i)) for i in range(min(64, max(steps, 1)))]
    done, t0 = 0, time.perf_counter()
    while True:
        q, k, v = pre[done % len(pre)]
        orc.step(q, k, v)
        done += 1
        el = time.perf_counter() - t0
        if el > budget_s or (done >= steps and el >= min_seconds):
            break
    dt = time.perf_counter() - t0
    unit_steps_per_s = done * U / dt
    value = unit_steps_per_s / (cfg.units * cfg.layers)
    info = {"value": value, "unit": UNIT, "cores": oracle.threads(), "kind": "oracle",
            "sample": (f"{U} of {cfg.units * cfg.layers} units, {done} timed steps after an untimed run-in of "
                       f"{run_in} tokens (steady-state saw-tooth n in [{cfg.B - cfg.m + 1}, {cfg.B}]); "
                       f"{dt:.1f} s of CPU work; unit-steps/s scaled to all units"),
            "unit_steps_per_s": unit_steps_per_s}
    return value, info, dt / max(done, 1)


def reference_arm(args, cfg, rank):
    if rank != 0:
        return
    value, info, s_per_step = oracle_run(cfg, args.steps, args.warmup, args.oracle_units, budget_s=150.0)
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 / value if value else None,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": config_record(cfg, args, int(os.environ.get("WORLD_SIZE", "1"))),
        "cpu_baseline": info,
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


# --------------------------------------------------------------------------- CUDA arm
def make_handles(sh, cfg, args, dev, stable: bool, layers: int):
    return [sh.Handle(cfg.B, cfg.r, cfg.w, cfg.m, cfg.units, cfg.head_dim, cfg.dtype, device=dev, auto_compress=False,
                      split=args.split, kernel=args.kernel,
                      prefill_chunk=0 if args.no_prefill_chunk else args.prefill_chunk_kernel,
                      recompute_record=args.recompute_record, unordered=False if stable else None)
            for _ in range(layers)]


def stream_prompt(cfg, handles, streams):
    """The prompt through sh_prefill, untimed part of the benchmark.  Returns (device ms, block size)."""
    blk = max(1, min(256, (1 << 31) // (cfg.units * cfg.head_dim * 2 * 3)))
    ms = 0.0
    for h, st in zip(handles, streams):
        for t0 in range(1, cfg.prompt + 1, blk):
            q, k, v = st.block(t0, min(t0 + blk, cfg.prompt + 1))
            pa, pb = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            pa.record()
            h.prefill(q, k, v)
            pb.record()
            torch.cuda.synchronize()
            ms += pa.elapsed_time(pb)
    return ms, blk


def prompt_attention_flop(cfg) -> float:
    """Algorithmic FLOP of the prompt's attention for all units and layers: token t attends over the rows cached
    when it arrives plus itself (the saw-tooth of Algorithm 1: m rows leave whenever B are reached); two passes
    over the logits (row statistics, then probabilities and record bits) and one over the values, 2 n d each."""
    n, rows = 0, 0
    for _ in range(cfg.prompt):
        if n == cfg.B:
            n -= cfg.m
        n += 1
        rows += n
    return 3.0 * 2.0 * rows * cfg.head_dim * cfg.units * cfg.layers


def time_compression(cfg, h, snap, dec_l, out, reps: int = REPEATS):
    """CUDA-event time of one sh_compress of handle `h` (all its units), `reps` times, each from the
    restored post-prompt state advanced until the cache is full.  dec_l: that layer's decode inputs."""
    times, launches = [], 0
    for _ in range(reps):
        h.restore(snap)
        n, i = snap[1], 0
        while n < cfg.B:
            h.decode_step(dec_l[0][i % len(dec_l[0])], dec_l[1][i % len(dec_l[0])], dec_l[2][i % len(dec_l[0])], out)
            n += 1
            i += 1
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        l0 = h.launch_count
        torch.cuda.synchronize()
        a.record()
        assert h.compress() == cfg.m
        b.record()
        torch.cuda.synchronize()
        launches = h.launch_count - l0
        times.append(a.elapsed_time(b))
    return {"ms_best": min(times), "ms_median": statistics.median(times), "ms_all": times, "kernel_launches": launches,
            "units": cfg.units, "steps_between_compressions": cfg.m,
            "ms_per_step_amortised": statistics.median(times) / cfg.m}


def cuda_arm(args, cfg, rank, world):
    from paper_2305_17118_b200 import binding as sh
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)
    K, W = args.steps, args.warmup
    U, d, Ly = cfg.units, cfg.head_dim, cfg.layers
    streams = [wl.Stream(cfg, device=dev, layer=l + 1000 * rank) for l in range(Ly)]
    handles = make_handles(sh, cfg, args, dev, args.stable_compaction, Ly)

    # ---- prompt: streamed through the same path, untimed
    prompt_ms, blk = stream_prompt(cfg, handles, streams)
    # ---- decode inputs resident in HBM; cycle if the run is longer than the buffer
    n_in = min(W + K, max(1, int(6e9 // (Ly * U * d * 2 * 3))))
    dec = [st.block(cfg.prompt + 1, cfg.prompt + 1 + n_in) for st in streams]
    torch.cuda.synchronize()
    snaps = [h.snapshot() for h in handles]
    kv_bytes = 2 * Ly * U * cfg.B * d * ES[cfg.dtype]
    flush = kv_bytes < 2 * L2_BYTES
    flush_buf = torch.empty(2 * L2_BYTES, dtype=torch.uint8, device=dev) if flush else None
    # the write leaves L2 full of dirty lines, which the timed kernel would then have to write back while it reads;
    # a read pass over a second buffer evicts them first, so the step starts on a cold and clean L2
    clean_buf = torch.zeros(2 * L2_BYTES // 4, dtype=torch.int32, device=dev) if flush else None
    out = torch.empty(U, d, device=dev)

    def one_step(i, timed_pairs=None):
        done = 0
        for l, h in enumerate(handles):
            q, k, v = dec[l][0][i % n_in], dec[l][1][i % n_in], dec[l][2][i % n_in]
            if timed_pairs is not None:
                a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                a.record()
                h.decode_step(q, k, v, out)
                b.record()
                timed_pairs.append((a, b))
            else:
                h.decode_step(q, k, v, out)
            done += h.compress() != 0          # no-op unless the cache just filled
        return done

    def barrier():
        torch.cuda.synchronize()
        if dist:
            dist.barrier()
        torch.cuda.synchronize()

    # ---- device-resident timing: REPEATS windows of K steps over the same stream positions
    sampler = ClockSampler(local)
    rep_ms, rep_value, kern_ms, launches, compressions = [], [], [], 0, 0
    # The value comes from REPEATS windows without any instrumentation between launches (consecutive decode
    # kernels are chained by programmatic dependent launch, which an event record between them would undo).
    # The decode kernel's own duration comes from one further window over the same steps with an event pair
    # around every launch.  Workloads that are flushed out of L2 between steps are timed per step anyway.
    for rep in range(REPEATS + (0 if flush else 1)):
        instrumented = flush or rep == REPEATS
        for h, s in zip(handles, snaps):
            h.restore(s)
        for i in range(W):
            one_step(i)
        launches0 = sum(h.launch_count for h in handles)
        pairs, step_pairs, comp = ([] if instrumented else None), [], 0
        barrier()
        ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        with sampler:
            ev0.record()
            for i in range(W, W + K):
                if flush:
                    flush_buf.fill_(i & 0xFF)
                    clean_buf.sum()
                    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                    a.record()
                    comp += one_step(i, pairs)
                    b.record()
                    step_pairs.append((a, b))
                else:
                    comp += one_step(i, pairs)
            ev1.record()
            barrier()
        total_ms = sum(a.elapsed_time(b) for a, b in step_pairs) if flush else ev0.elapsed_time(ev1)
        if instrumented:
            kern_ms += [a.elapsed_time(b) for a, b in pairs]
        if flush or not instrumented:
            launches = sum(h.launch_count for h in handles) - launches0
            compressions = comp
            ms_step, val = job_throughput(total_ms, K, world, dist, dev)
            rep_ms.append(ms_step)
            rep_value.append(val)
        else:
            instrumented_ms_per_step = job_throughput(total_ms, K, world, dist, dev)[0]
    ms_per_step = statistics.median(rep_ms)
    value = statistics.median(rep_value)

    # ---- roofline of the fused decode kernel (one launch = one layer's units)
    n_sched = live_rows_schedule(cfg, cfg.prompt + W + 1, K)
    alg_bytes_launch = statistics.fmean(n_sched) * U * d * ES[cfg.dtype] * 2
    kern_avg_ms = statistics.fmean(kern_ms)
    achieved = alg_bytes_launch / (kern_avg_ms * 1e-3) / 1e9
    peak, peak_src = measured_peak()
    traffic = None
    try:
        with open(os.path.join(ROOT, "profiles", "traffic.json")) as f:
            tr = json.load(f).get(cfg.name)      # shape variants have no capture: traffic stays null
            if tr:
                traffic = tr["dram_bytes_per_unit_row"] * statistics.fmean(n_sched) * U
    except Exception:
        pass
    roofline = {"bound": "hbm", "kernel": handles[0].decode_kernel, "achieved": achieved, "peak": peak, "unit": "GB/s",
                "frac": achieved / peak, "traffic": traffic, "peak_source": peak_src,
                "frac_of_8TBs_nominal": achieved / 8000.0, "alg_bytes_per_launch": alg_bytes_launch,
                "avg_launch_us": kern_avg_ms * 1e3, "launches_timed": len(kern_ms),
                "decode_kernel_share_of_step": kern_avg_ms * Ly / (ms_per_step if flush else instrumented_ms_per_step),
                "timed_in": ("the timed windows (every step is bracketed by events because of the L2 flush)" if flush else
                             "one further window over the same steps with an event pair around every launch: "
                             f"{instrumented_ms_per_step:.4f} ms per step there")}
    if flush:
        roofline["note"] = ("working set below 2x L2 (flushed between steps) and fewer than two units per SM: the step is "
                            "bound by launch and load latency, not by HBM; the fraction is reported for completeness")
    if cfg.dtype == "int4":
        # CUDA-core unpacking of 4-bit codes is bound by instruction issue before HBM: peak derived from
        # the kernel's instructions per stored byte and the SMs' issue rate at the sampled clock.
        mhz = sampler.summary()["sm_mhz"] or 1965.0
        ipb = INT4_LANE_INSTR_PER_BYTE[handles[0].decode_kernel]
        issue_peak = 148 * 4 * mhz * 1e6 * 32 / ipb / 1e9
        roofline.update({"bound": "alu", "peak": issue_peak, "frac": achieved / issue_peak,
                         "peak_source": (f"derived: 148 SMs x 4 schedulers x 1 warp instruction per clock x 32 lanes at {mhz:.0f} MHz "
                                         f"/ {ipb} lane-instructions per stored byte (profiles/)"),
                         "frac_of_measured_hbm": achieved / peak})

    # ---- the compression on its own (steps c1-c4), in the mode of this run and in the other one
    compress = None
    if rank == 0 and not args.no_compress_timing:
        mode = "stable" if args.stable_compaction else "hole filling"
        compress = {mode: time_compression(cfg, handles[0], snaps[0], dec[0], out)}
        other = make_handles(sh, cfg, args, dev, not args.stable_compaction, 1)
        stream_prompt(cfg, other, streams[:1])
        torch.cuda.synchronize()
        compress["hole filling" if args.stable_compaction else "stable"] = time_compression(
            cfg, other[0], other[0].snapshot(), dec[0], out)
        del other
        compress["note"] = ("one sh_compress over one layer's units from a restored state with a full cache; "
                            "it recurs every m steps, ms_per_step_amortised = median / m")

    # ---- end to end: host buffers through sh_decode_step_host
    e2e = None
    if rank == 0 or dist:
        for h, s in zip(handles, snaps):
            h.restore(s)
        Ke = min(K, n_in - W) if n_in > W else min(K, n_in)
        first = W if n_in >= W + Ke else 0          # the same stream positions as the device-resident windows
        host = [[x[:first + Ke].cpu().pin_memory() for x in dec[l]] for l in range(Ly)]
        oh = torch.empty(U, d).pin_memory()
        # raw addresses of every step's pinned rows, looked up once: the timed loop only makes the C call
        ptrs = [[(host[l][0][i].data_ptr(), host[l][1][i].data_ptr(), host[l][2][i].data_ptr()) for i in range(first + Ke)]
                for l in range(Ly)]
        oh_ptr, st_ptr = oh.data_ptr(), torch.cuda.current_stream().cuda_stream
        e_values = []
        for _rep in range(REPEATS):
            for h, s in zip(handles, snaps):
                h.restore(s)
            n_live = snaps[0][1]          # the schedule is data-independent: the caller knows when a compression is due

            def host_steps(i0, i1):
                nonlocal n_live
                for i in range(i0, i1):
                    n_live += 1
                    for l, h in enumerate(handles):
                        qp, kp, vp = ptrs[l][i]
                        h.decode_step_host_raw(qp, kp, vp, oh_ptr, st_ptr)
                        if n_live == cfg.B:
                            h.compress()
                    if n_live == cfg.B:
                        n_live -= cfg.m
            host_steps(0, first)          # warm-up, untimed
            barrier()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            host_steps(first, first + Ke)
            e1.record()
            barrier()
            e_values.append(job_throughput(e0.elapsed_time(e1), Ke, world, dist, dev)[1])
        e_value = statistics.median(e_values)
        in_b = Ly * U * d * (4 if cfg.dtype == "f32" else 2) * 3
        e2e = {"value": e_value, "unit": UNIT, "h2d_bytes_per_step": in_b,
               "d2h_bytes_per_step": Ly * U * d * 4, "steps": Ke, "values": e_values}

    if rank != 0:
        if dist:
            dist.destroy_process_group()
        return
    cpu = None
    if (world == 1 or rank == 0) and not args.no_cpu_baseline:
        _, cpu, _ = oracle_run(cfg, min(K, 64), 0, args.oracle_units, min_seconds=10.0, budget_s=30.0)
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": K, "warmup": W,
        "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": {"f32": "f32", "f16": "f16", "bf16": "bf16", "int4": "int4"}[cfg.dtype] + " KV, f32 accumulate",
        "data": "synthetic",
        "config": config_record(cfg, args, world),
        "repeats": {"n": REPEATS, "value_best": max(rep_value), "value_median": value, "values": rep_value,
                    "ms_per_step": rep_ms, "from": "post-prompt snapshot restored before every repetition, then warm-up"},
        "n_range": [min(n_sched), max(n_sched)], "n_mean": statistics.fmean(n_sched),
        "compressions_timed": compressions, "compress": compress,
        "attn_GBps": statistics.fmean(n_sched) * U * Ly * d * ES[cfg.dtype] * 2 / (ms_per_step * 1e-3) / 1e9,
        "prompt": {"tokens": cfg.prompt, "ms": prompt_ms, "tokens_per_s": cfg.prompt * 1e3 / prompt_ms if prompt_ms else None,
                   "chunked": bool(handles[0].prefill_chunk_max) and not args.no_prefill_chunk,
                   "attention_tflops_algorithmic": prompt_attention_flop(cfg) / (prompt_ms * 1e-3) / 1e12 if prompt_ms else None,
                   "note": "untimed part of the benchmark; streamed through sh_prefill in blocks of %d tokens" % blk},
        "clocks": sampler.summary(), "e2e": e2e, "gpu_launches": launches,
        "roofline": roofline, "cpu_baseline": cpu,
    }
    print(json.dumps(line), flush=True)
    if dist:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=256)
    ap.add_argument("--warmup", type=int, default=8)
    ap.add_argument("--config", default="opt66b", choices=wl.CONFIG_ORDER)
    ap.add_argument("--impl", default="cuda", choices=["cuda", "reference"])
    ap.add_argument("--oracle-units", type=int, default=2048)
    ap.add_argument("--split", type=int, default=None, help="CTAs per unit (default: chosen by the library)")
    ap.add_argument("--kernel", type=int, default=None, help="decode kernel: 1 direct loads, 2 pipelined bulk copies")
    ap.add_argument("--recompute-record", action="store_true",
                    help="variant: rebuild the importance record at each compression from stored queries")
    ap.add_argument("--kv-dtype", default=None, choices=["f32", "f16", "bf16", "int4"], help="override the workload's K/V dtype")
    ap.add_argument("--head-dim", type=int, default=None, choices=[64, 128], help="override the workload's head_dim")
    ap.add_argument("--stable-compaction", action="store_true",
                    help="SH_OPT_COMPACTION = 0: stable left-compaction, slots stay sorted by position.  The default "
                         "is the library's: holes filled from the tail, at most m rows move per compression; same kept sets")
    ap.add_argument("--no-compress-timing", action="store_true", help="skip the separate timing of sh_compress (tuning runs)")
    ap.add_argument("--prefill-chunk-kernel", type=int, default=None, choices=[1, 2, 3],
                    help="SH_OPT_PREFILL_CHUNK for the untimed prompt phase: 1 library's choice, 2 warp-level MMA kernel, 3 tcgen05 kernel")
    ap.add_argument("--no-prefill-chunk", action="store_true", help="stream the prompt one decode step per token")
    ap.add_argument("--no-cpu-baseline", action="store_true", help="skip the oracle timing (tuning runs)")
    ap.add_argument("--units", type=int, default=None,
                    help="override the workload's units per launch (a smaller case of the same kernels, for profiler captures)")
    ap.add_argument("--prompt", type=int, default=None, help="override the workload's prompt length (same purpose)")
    ap.add_argument("--layers", type=int, default=None, help="override the workload's number of layers (same purpose)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "cuda" else args.warmup
    cfg = wl.CONFIGS[args.config]
    if args.kv_dtype or args.head_dim or args.units or args.prompt or args.layers:      # shape variants of a named workload (not the benchmark's own lines)
        tag = ",".join(x for x in (args.kv_dtype, f"d{args.head_dim}" if args.head_dim else None,
                                   f"units{args.units}" if args.units else None,
                                   f"prompt{args.prompt}" if args.prompt else None,
                                   f"layers{args.layers}" if args.layers else None) if x)
        cfg = cfg.scaled(name=f"{cfg.name}[{tag}]", dtype=args.kv_dtype or cfg.dtype, head_dim=args.head_dim or cfg.head_dim,
                         units=args.units or cfg.units, prompt=args.prompt or cfg.prompt, layers=args.layers or cfg.layers)
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if args.impl == "reference":
        reference_arm(args, cfg, rank)
        return
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the CUDA path has no CPU fallback "
                         "(use --impl reference for the CPU oracle)")
    cuda_arm(args, cfg, rank, world)


if __name__ == "__main__":
    main()

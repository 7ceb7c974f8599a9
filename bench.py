#!/usr/bin/env python
"""Benchmark of the compaction attention hot path.

One "step" is one whole compaction event on synthetic blocks: plan -> ragged
causal prefill -> bulk KV append -> T x (one-token append + batched decode).
The default workload is `ragged` (32 blocks of 1024..8192 tokens, 512 decode steps), the
largest single-GPU configuration; the same JSON line carries `per_config` numbers for
dense8b, moe120b and the one-block (sequential) split.
Prints ONE JSON line (rank 0).  `--impl reference` times the CPU oracle instead.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import tempfile
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2605_23296_b200 import workloads as wl  # noqa: E402

METRIC = "summary tok/s at B blocks (attention only: prefill + paged decode)"
UNIT = "tok/s"
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}
NOMINAL_HBM_GBS = 8000.0
NOMINAL_BF16_TFLOPS = 2250.0
L2_MB = 126
DEFAULT_CONFIG = "ragged"   # the largest single-GPU workload of the throughput configurations
# The other single-GPU configurations, measured in the same run into `per_config`: (name, overrides, timed steps).
# The step counts make each timed region last a few hundred milliseconds, long enough for the clock sampler.
PER_CONFIG = [("dense8b", {}, 40), ("moe120b", {}, 8), ("split", {"num_blocks": 1}, 3)]
# Profiler captures of decode_split_kernel launches per workload (profiles/decode_split_kernel_*.md), of the
# kernel as it stands, on the workload with 24 instead of its full number of decode steps (eight launches,
# steps 6..13): DRAM bytes read + written per launch divided by the algorithmic KV bytes of those launches, with
# the caches left alone between consecutive steps ("warm", the timed condition) and with the L2 flushed before
# the launch ("cold"), and the algorithmic bytes per second of the cold launches.  A step's traffic grows in
# proportion to its KV bytes, so the ratios carry over to the average step of the full run.  A workload without
# a capture has no entry.
DECODE_CAPTURES = {
    "ragged": {"warm_ratio": 0.9319, "cold_ratio": 1.0043, "cold_gbs": 6043.7,
               "source": "profiles/decode_split_kernel_ragged.md"},
    "dense8b": {"warm_ratio": 0.3681, "cold_ratio": 1.0071, "cold_gbs": 4072.7,
                "source": "profiles/decode_split_kernel_dense8b.md"},
    "moe120b": {"warm_ratio": 0.7621, "cold_ratio": 1.0049, "cold_gbs": 4967.1,
                "source": "profiles/decode_split_kernel_moe120b.md"},
}


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            p = json.load(f)
        return {k: float(p[k]) for k in FALLBACK_PEAKS}, "measured"
    except Exception:
        return dict(FALLBACK_PEAKS), "fallback"


def make_workload(name: str, seed_offset: int = 0, overrides=None):
    """The named configuration; `overrides` (blocks / block length / decode steps) shrink it for
    profiler captures, which must stay small."""
    kw = {k: v for k, v in (overrides or {}).items() if v}
    w = wl.CONFIGS[name](**kw)
    if seed_offset:
        w = wl.CONFIGS[name](seed=w.seed + 1000 * seed_offset, **kw)
    return w


def prefill_flops(w) -> float:
    L = w.block_lens.astype(np.float64)
    return float((2.0 * w.num_q_heads * w.head_dim * L * (L + 1.0)).sum())


def decode_kv_bytes(w, t: int) -> float:
    """K and V bytes one decode step must read: every cached element once per kv head."""
    lens = w.block_lens.astype(np.float64) + t + 1
    return float((2.0 * w.num_kv_heads * w.head_dim * 2.0 * lens).sum())


def workload_desc(w) -> dict:
    return {"workload": w.name, "blocks": w.num_blocks,
            "block_lens": f"{int(w.block_lens.min())}..{int(w.block_lens.max())}",
            "total_tokens": w.total_tokens, "q_heads": w.num_q_heads, "kv_heads": w.num_kv_heads,
            "head_dim": w.head_dim, "decode_steps": w.decode_steps, "page_size": w.page_size,
            "seed": w.seed}


# ------------------------------------------------------------------------------------------
# CPU oracle leg (also the whole of `--impl reference`)
# ------------------------------------------------------------------------------------------

def oracle_sample_seconds(w, rows_per_block: int, decode_samples: int):
    """Time the oracle, as it stands, on a bounded sample of the workload.

    Sample: `rows_per_block` query rows of every block (evenly spaced, all heads) for prefill and
    `decode_samples` decode steps (all blocks, all heads).  Returns the measured seconds and the
    whole-step estimate obtained by scaling each phase by (total work / sampled work).
    """
    from oracle import attention as oa
    cu = np.concatenate([[0], np.cumsum(w.block_lens.astype(np.int64))])
    rows, sample_flops = [], 0.0
    for b, L in enumerate(int(x) for x in w.block_lens):
        pos = np.unique(np.linspace(0, L - 1, rows_per_block).astype(np.int64))
        rows += [cu[b] + p for p in pos]
        sample_flops += float((4.0 * w.num_q_heads * w.head_dim * (pos + 1.0)).sum())
    t0 = time.perf_counter()
    oa.prefill(w.q, w.k, w.v, cu, w.scale, rows=np.asarray(rows, dtype=np.int64))
    t_prefill = time.perf_counter() - t0
    est_prefill = t_prefill * prefill_flops(w) / sample_flops

    st = oa.DecodeState(w.k, w.v, cu, w.decode_steps)
    steps = sorted(set(np.linspace(0, w.decode_steps - 1, decode_samples).astype(int).tolist()))
    t_decode, sampled_bytes, t = 0.0, 0.0, 0
    for step in range(steps[-1] + 1):
        st.append(w.k_dec[step], w.v_dec[step])
        if step in steps:
            t0 = time.perf_counter()
            st.decode(w.q_dec[step], w.scale)
            t_decode += time.perf_counter() - t0
            sampled_bytes += decode_kv_bytes(w, step)
    total_bytes = sum(decode_kv_bytes(w, s) for s in range(w.decode_steps))
    est_decode = t_decode * total_bytes / sampled_bytes
    return {"measured_s": t_prefill + t_decode, "estimated_step_s": est_prefill + est_decode,
            "prefill_s_est": est_prefill, "decode_s_est": est_decode,
            "cores": oa.host_threads(),
            "sample": (f"{len(rows)} prefill rows ({rows_per_block}/block, all heads) + "
                       f"{len(steps)} decode steps (all blocks, all heads); "
                       "time scaled by total/sampled flops (prefill) and KV bytes (decode)")}


def run_reference(args) -> None:
    if args.layout[1] != 0:    # rank 0 alone runs the reference arm
        return
    w = make_workload(args.config, overrides=args.overrides).materialise()
    tokens = w.num_blocks * w.decode_steps
    times, info = [], None
    for i in range(args.warmup + args.steps):
        info = oracle_sample_seconds(w, rows_per_block=2, decode_samples=2)
        if i >= args.warmup:
            times.append(info["estimated_step_s"])
    sec = statistics.mean(times)
    value = tokens / sec
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": sec * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": workload_desc(w),
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": info["cores"], "kind": "oracle",
                         "sample": info["sample"]},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


# ------------------------------------------------------------------------------------------
# GPU arm
# ------------------------------------------------------------------------------------------

class ClockSampler:
    QUERY = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
             "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu_index = gpu_index
        self.proc = None
        self.path = None

    def start(self):
        try:
            fd, self.path = tempfile.mkstemp(suffix=".csv")
            os.close(fd)
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.QUERY}", "--format=csv,noheader,nounits",
                 "-i", str(self.gpu_index), "-lms", "50"],
                stdout=open(self.path, "w"), stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self) -> dict:
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.proc is None:
            return out
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        try:
            sm, reasons, mx, power = [], set(), None, []
            for line in open(self.path):
                f = [x.strip() for x in line.split(",")]
                if len(f) < 9:
                    continue
                try:
                    sm.append(float(f[1])); mx = float(f[2]); power.append(float(f[3]))
                except ValueError:
                    continue
                for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), f[5:9]):
                    if val.lower().startswith("active"):
                        reasons.add(name)
            if sm:
                out.update(sm_mhz=statistics.median(sm), sm_max_mhz=mx, reasons=sorted(reasons),
                           samples=len(sm), power_w_max=max(power))
        finally:
            try:
                os.unlink(self.path)
            except OSError:
                pass
        return out


def max_over_ranks(x: float, world: int, device) -> float:
    """The slowest rank's time: every multi-GPU number is the maximum over ranks."""
    if world == 1:
        return x
    import torch
    import torch.distributed as dist
    t = torch.tensor([x], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_tokens(w, world: int) -> int:
    """Summary tokens produced per step by all ranks: every rank runs its own event of the same
    shape (weak scaling, blocks are independent, no data-path collective)."""
    return world * w.num_blocks * w.decode_steps


def rank_layout(gpus: int, env, impl: str = "ours"):
    """What `--gpus N` means for this process.  ("run", rank, world, local_rank): run as that rank;
    ("spawn", argv): no launcher started us, so start N ranks (one per GPU) with torch's launcher and
    relay their exit code.  A launcher whose WORLD_SIZE disagrees with --gpus is an error: the JSON
    line would claim a GPU count that did not run."""
    if gpus < 1:
        raise SystemExit("--gpus must be at least 1")
    world = env.get("WORLD_SIZE")
    if world is None:
        if gpus == 1 or impl == "reference":      # the reference arm runs on rank 0's host cores only
            return ("run", 0, 1, 0)
        argv = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={gpus}",
                "--master-addr", "127.0.0.1", "--master-port", str(29400 + os.getpid() % 500),
                os.path.abspath(__file__)] + sys.argv[1:]
        return ("spawn", argv)
    if int(world) != gpus:
        raise SystemExit(f"--gpus {gpus} disagrees with the launcher's WORLD_SIZE={world}")
    return ("run", int(env.get("RANK", "0")), int(world), int(env.get("LOCAL_RANK", "0")))


def measure_event(w, args, dev, steps: int, warmup: int, with_e2e: bool, world: int = 1, rank: int = 0,
                  local_rank: int = 0, sample_clocks: bool = True) -> dict:
    """Time `steps` whole compaction events of workload `w` (after `warmup` untimed ones) with inputs resident
    on the device, and optionally the same event from pinned host buffers (copies inside the timed region).
    Returns phase times (ms, mean over the steps; the step time is the maximum over ranks) and clocks."""
    import torch
    import torch.distributed as dist

    from paper_2605_23296_b200.session import CompactionSession

    T, Bn = w.decode_steps, w.num_blocks
    stream = torch.cuda.current_stream(dev)

    def pinned(bits):
        return torch.from_numpy(bits.view(np.int16)).view(torch.bfloat16).pin_memory()

    def resident(bits):
        return torch.from_numpy(bits.view(np.int16)).view(torch.bfloat16).to(dev)

    hosts = [pinned(x) for x in (w.q, w.k, w.v, w.q_dec, w.k_dec, w.v_dec)] if with_e2e else None
    d_q, d_k, d_v, d_qd, d_kd, d_vd = (h.to(dev) for h in hosts) if with_e2e else (
        resident(x) for x in (w.q, w.k, w.v, w.q_dec, w.k_dec, w.v_dec))
    d_o = torch.empty_like(d_q)
    d_od = torch.empty((T, Bn, w.num_q_heads, w.head_dim), dtype=torch.bfloat16, device=dev)
    flush = torch.empty(256 * 1024 * 1024, dtype=torch.uint8, device=dev)  # > 126 MB of L2

    sample_every = max(1, T // 32)   # decode launches that get their own event pair
    state = {"launches": 0}

    def one_pass(q, k, v, qd, kd, vd, o, od, ev=None, dec_events=None):
        """plan -> prefill -> bulk append -> T x (append, decode); all through the C-ABI."""
        s = CompactionSession(w.block_lens, T, w.num_q_heads, w.num_kv_heads, w.head_dim,
                              w.free_pages, w.num_pages, scale=w.scale, device=str(dev),
                              pages_per_split=args.pages_per_split)
        if ev:
            ev["planned"].record(stream)
        s.prefill(q, k, v, out=o)
        if ev:
            ev["prefilled"].record(stream)
        s.append_prefill(k, v)
        if ev:
            ev["appended"].record(stream)
        if not args.separate_append and dec_events is None and T > 0:
            # all T fused steps enqueued by one call (their inputs are on the device already)
            s.decode_append_steps(qd, kd, vd, out=od)
        for t in (range(T) if args.separate_append or dec_events is not None else ()):
            sampled = dec_events is not None and t % sample_every == 0
            if args.separate_append:
                s.append(kd[t], vd[t])
            if sampled:
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record(stream)
            if args.separate_append:
                s.decode(qd[t], out=od[t])
            else:   # the step's append is fused into the decode launch
                s.decode_append(qd[t], kd[t], vd[t], out=od[t])
            if sampled:
                e1.record(stream)
                dec_events.append((t, e0, e1))
        # prefill, bulk append + length advance, then per step one fused launch (or append + decode)
        state["launches"] += 1 + 2 + (2 if args.separate_append else 1) * T
        return s

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize(dev)

    # ---- device-resident timing ----------------------------------------------------------
    sessions = []
    for _ in range(warmup):
        sessions.append(one_pass(d_q, d_k, d_v, d_qd, d_kd, d_vd, d_o, d_od))
        flush.fill_(1)
    torch.cuda.synchronize(dev)
    for s in sessions:
        assert s.status() == 0
        s.close()
    sessions.clear()

    sampler = ClockSampler(local_rank)
    if rank == 0 and sample_clocks:
        sampler.start()
    barrier()
    state["launches"] = 0
    step_ms, prefill_ms, decode_ms, append_ms, plan_ms, dec_samples = [], [], [], [], [], []
    for _ in range(steps):
        flush.fill_(1)   # L2 flush between timed steps (the step's own inputs, 400+ MB, exceed L2 anyway)
        ev = {n: torch.cuda.Event(enable_timing=True) for n in ("start", "planned", "prefilled", "appended", "end")}
        # (with separate append and decode calls the launch time comes from event pairs around sampled launches)
        dec_events = [] if args.separate_append else None
        ev["start"].record(stream)
        s = one_pass(d_q, d_k, d_v, d_qd, d_kd, d_vd, d_o, d_od, ev, dec_events)
        ev["end"].record(stream)
        torch.cuda.synchronize(dev)
        assert s.status() == 0
        s.close()
        step_ms.append(ev["start"].elapsed_time(ev["end"]))
        plan_ms.append(ev["start"].elapsed_time(ev["planned"]))
        prefill_ms.append(ev["planned"].elapsed_time(ev["prefilled"]))
        append_ms.append(ev["prefilled"].elapsed_time(ev["appended"]))
        decode_ms.append(ev["appended"].elapsed_time(ev["end"]))
        dec_samples += [(t, e0.elapsed_time(e1)) for t, e0, e1 in (dec_events or [])]
    barrier()
    launches = state["launches"]
    if not args.separate_append:
        # event pairs around single launches, for comparison with the phase time / T: one more pass, not timed as a
        # step (the pairs add their own cost and break the overlap of consecutive launches)
        flush.fill_(1)
        dec_events = []
        s = one_pass(d_q, d_k, d_v, d_qd, d_kd, d_vd, d_o, d_od, None, dec_events)
        torch.cuda.synchronize(dev)
        assert s.status() == 0
        s.close()
        dec_samples += [(t, e0.elapsed_time(e1)) for t, e0, e1 in dec_events]

    # ---- end to end: host buffers in, host buffers out, copies inside the timed region -----
    e2e_ms, h2d, d2h = [], 0, 0
    if with_e2e:
        h_q, h_k, h_v, h_qd, h_kd, h_vd = hosts
        h_o = torch.empty(d_o.shape, dtype=torch.bfloat16).pin_memory()
        h_od = torch.empty(d_od.shape, dtype=torch.bfloat16).pin_memory()
        h2d = sum(t.numel() * 2 for t in hosts)
        d2h = (h_o.numel() + h_od.numel()) * 2
        stage = None
        for i in range(1 + steps):
            flush.fill_(1)
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            torch.cuda.synchronize(dev)
            e0.record(stream)
            # one C-ABI call with host pointers: plan (chunked, so that the copies overlap the kernels), prompts up
            # chunk by chunk, prefill per chunk, outputs home behind the kernels, then the T decode steps
            s = CompactionSession(w.block_lens, T, w.num_q_heads, w.num_kv_heads, w.head_dim,
                                  w.free_pages, w.num_pages, scale=w.scale, device=str(dev),
                                  pages_per_split=args.pages_per_split, chunk_tokens=args.e2e_chunk,
                                  decode_sms=1 if args.e2e_chunk else 0)
            stage = s.event_from_host(h_q, h_k, h_v, h_o, h_qd, h_kd, h_vd, h_od, stage=stage)
            e1.record(stream)
            torch.cuda.synchronize(dev)
            assert s.status() == 0
            s.close()
            if i > 0:
                e2e_ms.append(e0.elapsed_time(e1))

    clocks = sampler.stop() if rank == 0 and sample_clocks else {}   # sampled over both timed legs
    mean = statistics.mean
    pair_us = mean(m for _, m in dec_samples) * 1e3 if dec_samples else float("nan")
    return {"ms": max_over_ranks(mean(step_ms), world, dev),
            "e2e_ms": max_over_ranks(mean(e2e_ms), world, dev) if e2e_ms else float("nan"),
            "plan_ms": mean(plan_ms), "prefill_ms": mean(prefill_ms), "append_ms": mean(append_ms),
            "decode_ms": mean(decode_ms), "pair_us": pair_us, "pair_bytes": (mean(decode_kv_bytes(w, t) for t, _ in dec_samples)
                                                                            if dec_samples else float("nan")),
            "n_pairs": len(dec_samples), "launches": launches, "h2d": h2d, "d2h": d2h, "clocks": clocks}


def phase_numbers(w, m: dict, peaks: dict, separate_append: bool) -> dict:
    """Prefill TFLOP/s and decode GB/s (with their fractions of the measured peaks) from phase times."""
    T = w.decode_steps
    pf_tflops = prefill_flops(w) / (m["prefill_ms"] * 1e-3) / 1e12
    total_kv = sum(decode_kv_bytes(w, t) for t in range(T))
    if separate_append:   # per-launch event pairs on sampled steps
        launch_us, launch_bytes = m["pair_us"], m["pair_bytes"]
    else:
        # every decode step is exactly one launch (append fused in), so the average launch duration over
        # the timed region is the decode phase's CUDA-event time / T; event pairs around single launches
        # add their own cost and break the overlap of consecutive launches
        launch_us, launch_bytes = m["decode_ms"] * 1e3 / T, total_kv / T
    gbs = launch_bytes / (launch_us * 1e-6) / 1e9
    # the prefill's second limiter: one exponential per unmasked score, Hq * L(L+1)/2 per block = flops / (4 d);
    # the special-function units make 16 per clock and SM (nominal: 148 SMs at the maximum clock)
    gexp = prefill_flops(w) / (4.0 * w.head_dim) / (m["prefill_ms"] * 1e-3) / 1e9
    return {"prefill_ms": m["prefill_ms"], "prefill_tflops": pf_tflops,
            "prefill_frac_of_bf16_peak": pf_tflops / peaks["bf16_tflops"],
            "prefill_frac_of_nominal_2250": pf_tflops / NOMINAL_BF16_TFLOPS,
            "prefill_gexp_per_s": gexp, "prefill_frac_of_nominal_exp_rate": gexp / (16 * 148 * 1.965),
            "decode_ms": m["decode_ms"], "decode_launch_us": launch_us, "decode_bytes_per_launch": launch_bytes,
            "decode_gbs": gbs, "decode_frac_of_hbm_peak": gbs / peaks["hbm_gbs"],
            "decode_frac_of_nominal_8TBs": gbs / NOMINAL_HBM_GBS,
            "decode_pool_vs_l2": ("pool of %.0f MB per step against %d MB of L2: %s" % (
                launch_bytes / 1e6, L2_MB, "an effective (L2-assisted) rate, not an HBM fraction"
                if launch_bytes < 2.5 * L2_MB * 1e6 else "HBM-bound, at most a fifth can come from L2"))}


def capture_fields(cap, bytes_per_launch: float, peaks: dict) -> dict:
    """DRAM traffic of one decode launch from the profiler captures (see DECODE_CAPTURES); nulls without one."""
    if not cap:
        return {"traffic": None, "traffic_cold": None, "frac_cold_l2": None, "traffic_source": None}
    return {"traffic": cap["warm_ratio"] * bytes_per_launch, "traffic_cold": cap["cold_ratio"] * bytes_per_launch,
            "frac_cold_l2": cap["cold_gbs"] / peaks["hbm_gbs"], "traffic_source": cap["source"]}


def run_gpu(args) -> None:
    import gc

    import torch
    import torch.distributed as dist

    _, rank, world, local_rank = args.layout
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback)")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)

    peaks, peak_kind = load_peaks()
    # weak scaling: every rank runs its own compaction event of the same shape (own seed);
    # blocks are independent, so there is no data-path collective
    w = make_workload(args.config, seed_offset=rank, overrides=args.overrides).materialise()
    T, Bn = w.decode_steps, w.num_blocks
    m = measure_event(w, args, dev, args.steps, args.warmup, not args.skip_e2e, world, rank, local_rank)
    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    tokens = whole_job_tokens(w, world)
    ph = phase_numbers(w, m, peaks, args.separate_append)
    overridden = bool(args.blocks or args.block_len or args.decode_steps or args.pages_per_split or args.separate_append)
    cap = DECODE_CAPTURES.get(args.config) if not overridden else None
    # dominant kernel: the decode launches (one per step: append, split-K scan and merge fused).  `achieved` divides the
    # ALGORITHMIC KV bytes by the launch time: when a step's pool is not much larger than the L2 (dense8b), part of
    # those bytes is served from L2, and the figure is an effective rate.  `traffic` is the DRAM traffic of a launch
    # in the timed condition (back-to-back steps, caches left alone), `traffic_cold` with the L2 flushed before the
    # launch, `frac_cold_l2` the fraction the kernel reaches from a cold L2; all three from profiler captures of this
    # kernel on this workload (profiles/), null where there is no capture of the kernel as it stands.
    roofline = {"bound": "hbm", "kernel": "decode_split_kernel (one launch per step: append, split-K scan and merge fused)",
                "achieved": ph["decode_gbs"], "peak": peaks["hbm_gbs"], "unit": "GB/s",
                "frac": ph["decode_frac_of_hbm_peak"], "peak_kind": f"of {peak_kind}",
                "frac_of_nominal_8TBs": ph["decode_frac_of_nominal_8TBs"],
                "launch_us": ph["decode_launch_us"], "bytes_per_launch": ph["decode_bytes_per_launch"],
                "launches_timed": (T * args.steps if not args.separate_append else m["n_pairs"]),
                "launch_us_event_pair_sampled": m["pair_us"],
                **capture_fields(cap, ph["decode_bytes_per_launch"], peaks),
                "l2_note": ph["decode_pool_vs_l2"]}

    # ---- the other single-GPU configurations, three timed steps each, device-resident only -----
    per_config = {}
    if args.per_config and world == 1 and not overridden:
        del w.q, w.k, w.v
        for name, kw, n_timed in PER_CONFIG:
            if name == args.config and not kw:
                continue
            gc.collect()
            torch.cuda.empty_cache()
            w2 = wl.CONFIGS[name](**kw).materialise()
            m2 = measure_event(w2, args, dev, n_timed, 3, False)
            p2 = phase_numbers(w2, m2, peaks, False)
            label = name if not kw else f"{name}:B={kw['num_blocks']}"
            per_config[label] = dict(p2, **capture_fields(DECODE_CAPTURES.get(label), p2["decode_bytes_per_launch"], peaks),
                                     config=workload_desc(w2), ms_per_step=m2["ms"],
                                     value=w2.num_blocks * w2.decode_steps / (m2["ms"] * 1e-3), steps=n_timed, warmup=3,
                                     clocks=m2["clocks"])
            del w2
        w = make_workload(args.config, seed_offset=rank, overrides=args.overrides).materialise()

    if args.skip_cpu:
        cpu = {"estimated_step_s": float("nan"), "cores": 0, "sample": "skipped", "measured_s": 0.0}
    else:
        cpu = oracle_sample_seconds(w, rows_per_block=32, decode_samples=8)
    out = {
        "metric": METRIC, "value": tokens / (m["ms"] * 1e-3), "unit": UNIT, "n_gpus": world,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": m["ms"], "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": workload_desc(w),
        "timing": {"l2": "256 MiB write between timed steps; step inputs (>400 MB) exceed L2",
                   "parallelism": f"replicas x{world} (independent blocks, no collective)"},
        "phases": dict(ph, plan_ms=m["plan_ms"], bulk_append_ms=m["append_ms"], peaks=dict(peaks, kind=peak_kind)),
        "roofline": roofline,
        "per_config": per_config,
        "cpu_baseline": {"value": Bn * T / cpu["estimated_step_s"], "unit": UNIT, "cores": cpu["cores"],
                         "kind": "oracle", "sample": cpu["sample"], "measured_s": cpu["measured_s"]},
        "e2e": {"value": tokens / (m["e2e_ms"] * 1e-3), "unit": UNIT, "ms_per_step": m["e2e_ms"],
                "h2d_bytes_per_step": m["h2d"], "d2h_bytes_per_step": m["d2h"],
                "call": "cpa_event_host", "chunk_tokens": args.e2e_chunk},
        "gpu_launches": m["launches"],
        "clocks": m["clocks"],
    }
    print(json.dumps(out))
    if world > 1:
        dist.destroy_process_group()


# ------------------------------------------------------------------------------------------
# the paper's own layout (prefix-aware target-at-end): a separate, non-default workload
# ------------------------------------------------------------------------------------------

def run_prefix(args) -> None:
    """`--config prefix8b`: W workers over one cached history (paper, Section 4): worker w prefills
    its own block (+ markers) over the w cached blocks before it, then all W decode T tokens.  The
    history's K/V are in the pool before the timed region (they are the conversation's KV cache)."""
    import torch

    from paper_2605_23296_b200.session import CompactionSession, bits_to_tensor

    if args.layout[2] != 1:
        raise SystemExit("--config prefix8b is a single-GPU measurement")
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    peaks, peak_kind = load_peaks()
    W = args.blocks or 16
    block_len = args.block_len or 8192
    T = args.decode_steps or 256
    w = wl.prefix_aware(W, block_len, 32, 8, 128, T, seed=11, permute_pages=False).materialise()
    o = w.own
    stream = torch.cuda.current_stream(dev)
    d = lambda bits: bits_to_tensor(bits, dev)
    shape = (w.num_pages, o.num_kv_heads, o.page_size, o.head_dim)
    pools = (torch.empty(shape, dtype=torch.bfloat16, device=dev), torch.empty(shape, dtype=torch.bfloat16, device=dev))
    hist = CompactionSession([w.hist_tokens], 0, o.num_q_heads, o.num_kv_heads, o.head_dim, w.shared_pages, w.num_pages,
                             scale=o.scale, pools=pools)
    hist.append_prefill(d(w.k_hist), d(w.v_hist))
    q, k, v, qd, kd, vd = (d(x) for x in (o.q, o.k, o.v, o.q_dec, o.k_dec, o.v_dec))
    out = torch.empty_like(q)
    od = torch.empty((T, W, o.num_q_heads, o.head_dim), dtype=torch.bfloat16, device=dev)
    flush = torch.empty(256 * 1024 * 1024, dtype=torch.uint8, device=dev)

    def one_pass(ev=None):
        s = CompactionSession(o.block_lens, T, o.num_q_heads, o.num_kv_heads, o.head_dim, o.free_pages, w.num_pages,
                              scale=o.scale, prefix_lens=w.prefix_lens, shared_pages=w.shared_pages, pools=pools)
        if ev:
            ev["planned"].record(stream)
        s.prefill(q, k, v, out=out)
        if ev:
            ev["prefilled"].record(stream)
        s.append_prefill(k, v)
        if ev:
            ev["appended"].record(stream)
        for t in range(T):
            s.decode_append(qd[t], kd[t], vd[t], out=od[t])
        return s

    for _ in range(args.warmup):
        s = one_pass()
        torch.cuda.synchronize(dev)
        assert s.status() == 0
        s.close()
    sampler = ClockSampler(0)
    sampler.start()
    step_ms, prefill_ms, decode_ms = [], [], []
    for _ in range(args.steps):
        flush.fill_(1)
        ev = {n: torch.cuda.Event(enable_timing=True) for n in ("start", "planned", "prefilled", "appended", "end")}
        ev["start"].record(stream)
        s = one_pass(ev)
        ev["end"].record(stream)
        torch.cuda.synchronize(dev)
        assert s.status() == 0
        s.close()
        step_ms.append(ev["start"].elapsed_time(ev["end"]))
        prefill_ms.append(ev["planned"].elapsed_time(ev["prefilled"]))
        decode_ms.append(ev["appended"].elapsed_time(ev["end"]))
    clocks = sampler.stop()
    hist.close()

    L = o.block_lens.astype(np.float64)
    pre = w.prefix_lens.astype(np.float64)
    # every own row sees the whole prefix, plus the causal half of the own tokens
    flops = float((4.0 * o.num_q_heads * o.head_dim * (L * pre + L * (L + 1.0) / 2.0)).sum())
    row_bytes = 2.0 * o.num_kv_heads * o.head_dim * 2.0
    # what this decode reads: every worker streams its whole prompt (prefix included) every step;
    # `unique` counts each cached history page once per step
    read = sum(float((pre + L + t + 1).sum()) * row_bytes for t in range(T))
    unique = sum((float(pre.max()) + float((L + t + 1).sum())) * row_bytes for t in range(T))
    ms, pf_ms, dc_ms = (statistics.mean(x) for x in (step_ms, prefill_ms, decode_ms))
    # algorithmic bytes: each cached K and V element once per step and kv head, however many workers
    # share it; `read` is what the kernel asks for (part of it served from L2)
    achieved = unique / (dc_ms * 1e-3) / 1e9
    print(json.dumps({
        "metric": METRIC, "value": W * T / (ms * 1e-3), "unit": UNIT, "n_gpus": 1, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16", "data": "synthetic",
        "config": {"workload": o.name, "layout": "prefix-aware target-at-end", "workers": W, "block_len": block_len,
                   "marker_tokens": w.marker_tokens, "history_tokens_cached": w.hist_tokens, "q_heads": o.num_q_heads,
                   "kv_heads": o.num_kv_heads, "head_dim": o.head_dim, "decode_steps": T, "page_size": o.page_size,
                   "seed": o.seed, "l2": "256 MiB write between timed steps"},
        "phases": {"prefill_ms": pf_ms, "decode_ms": dc_ms, "prefill_tflops": flops / (pf_ms * 1e-3) / 1e12,
                   "prefill_frac_of_bf16_peak": flops / (pf_ms * 1e-3) / 1e12 / peaks["bf16_tflops"],
                   "decode_gbs_unique_pages": achieved, "decode_gbs_requested": read / (dc_ms * 1e-3) / 1e9,
                   "peaks": dict(peaks, kind=peak_kind)},
        "roofline": {"bound": "hbm", "kernel": "decode_split_kernel over shared prefix pages + own pages",
                     "achieved": achieved, "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": achieved / peaks["hbm_gbs"],
                     "peak_kind": f"of {peak_kind}", "launch_us": dc_ms * 1e3 / T, "bytes_per_launch": unique / T,
                     "requested_bytes_per_launch": read / T, "traffic": None},
        "gpu_launches": args.steps * (3 + T), "clocks": clocks,
    }))


# ------------------------------------------------------------------------------------------
# chunked prefill mixed with decode (paper, Section 4.2 and Section 6): a separate, non-default workload
# ------------------------------------------------------------------------------------------

def run_mixed(args) -> None:
    """`--config mixed16k`: one 16k block beside four 2k blocks (8B-class heads), T summary tokens each.  Whole-block
    calls (one prefill launch over all blocks, then T decode steps) against the chunked schedule (2048-token chunks;
    the short blocks decode while the long block is still prefilling, cpa_step_mixed).  Reports when the short
    blocks' first and last summary tokens are out and when the whole event is done, both ways."""
    import torch

    from paper_2605_23296_b200 import binding as B
    from paper_2605_23296_b200.session import CompactionSession, bits_to_tensor

    if args.layout[2] != 1:
        raise SystemExit("--config mixed16k is a single-GPU measurement")
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    peaks, peak_kind = load_peaks()
    T = args.decode_steps or 256
    chunk = 2048
    lens = [16384, 2048, 2048, 2048, 2048]
    w = wl.custom(lens, 32, 8, 128, steps=T, seed=13, permute_pages=True).materialise()
    Bn = w.num_blocks
    stream = torch.cuda.current_stream(dev)
    d = lambda bits: bits_to_tensor(bits, dev)
    q, k, v, qd, kd, vd = (d(x) for x in (w.q, w.k, w.v, w.q_dec, w.k_dec, w.v_dec))
    o = torch.empty_like(q)
    od = torch.empty((T + 8, Bn, w.num_q_heads, w.head_dim), dtype=torch.bfloat16, device=dev)
    flush = torch.empty(256 * 1024 * 1024, dtype=torch.uint8, device=dev)
    new_ev = lambda: torch.cuda.Event(enable_timing=True)

    def whole_blocks():
        ev = {n: new_ev() for n in ("start", "first", "end")}
        s = CompactionSession(w.block_lens, T, w.num_q_heads, w.num_kv_heads, w.head_dim, w.free_pages, w.num_pages,
                              scale=w.scale)
        torch.cuda.synchronize(dev)
        ev["start"].record(stream)      # (planning and the plan's upload are outside both measurements)
        s.prefill(q, k, v, out=o)
        s.append_prefill(k, v)
        s.decode_append_steps(qd[:1], kd[:1], vd[:1], out=od[:1])
        ev["first"].record(stream)
        if T > 1:      # the remaining steps enqueued by one call (inputs staged on the device)
            s.decode_append_steps(qd[1:], kd[1:], vd[1:], out=od[1:T])
        ev["end"].record(stream)
        return s, ev

    def chunked():
        ev = {n: new_ev() for n in ("start", "first", "short_done", "long_prefilled", "end")}
        s = CompactionSession(w.block_lens, T, w.num_q_heads, w.num_kv_heads, w.head_dim, w.free_pages, w.num_pages,
                              scale=w.scale, chunk_tokens=chunk, decode_sms=args.decode_sms,
                              decode_steps_per_chunk=args.steps_per_chunk)
        start = s.export(B.ARR_DEC_START)
        n_steps = s.param(B.PARAM_NUM_STEPS)
        n_long = int(start.max())
        # a block's t-th token takes the inputs of row t whatever step produces it: the short blocks run one
        # step ahead per chunk of the long one, so the decode inputs of a step are gathered per block
        steps_in = []
        for step in range(n_steps):
            t_of = np.clip(step - start, 0, T - 1)
            steps_in.append(torch.from_numpy(t_of.astype(np.int64)).to(dev))
        ar = torch.arange(Bn, device=dev)
        # staged before the timed calls: [n_steps, B, H, d], slice i = the decode inputs of step i
        q_in = torch.stack([qd[t_of, ar] for t_of in steps_in]).contiguous()
        k_in = torch.stack([kd[t_of, ar] for t_of in steps_in]).contiguous()
        v_in = torch.stack([vd[t_of, ar] for t_of in steps_in]).contiguous()
        o_out = torch.empty_like(q_in)
        torch.cuda.synchronize(dev)
        ev["start"].record(stream)
        # the steps between two time stamps are enqueued by one call each
        marks = sorted({int(start.min()): "first", int(start.min()) + T - 1: "short_done", n_long - 1: "long_prefilled",
                        n_steps - 1: "end"}.items())
        done = 0
        stamped = set()
        for last, _ in marks:
            if last + 1 > done:
                s.step_mixed_range(done, last + 1 - done, q, k, v, o, q_in[done:last + 1], k_in[done:last + 1],
                                   v_in[done:last + 1], o_out[done:last + 1])
                done = last + 1
            for step, name in ((int(start.min()), "first"), (int(start.min()) + T - 1, "short_done"),
                               (n_long - 1, "long_prefilled"), (n_steps - 1, "end")):
                if step == last and name not in stamped:
                    ev[name].record(stream)
                    stamped.add(name)
        return s, ev

    res = {"whole_blocks": [], "chunked": []}
    for i in range(args.warmup + args.steps):
        for name, fn in (("whole_blocks", whole_blocks), ("chunked", chunked)):
            flush.fill_(1)
            s, ev = fn()
            torch.cuda.synchronize(dev)
            assert s.status() == 0
            s.close()
            if i >= args.warmup:
                res[name].append({n: ev["start"].elapsed_time(e) for n, e in ev.items() if n != "start"})
    mean = lambda name, key: statistics.mean(r[key] for r in res[name])
    out = {
        "metric": "time until the short blocks' summaries are out, whole-block prefill vs chunked prefill mixed with decode",
        "unit": "ms", "n_gpus": 1, "steps": args.steps, "warmup": args.warmup, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": "mixed16k", "block_lens": lens, "q_heads": 32, "kv_heads": 8, "head_dim": 128,
                   "decode_steps": T, "chunk_tokens": chunk, "decode_sms": args.decode_sms or "a quarter of the SMs",
                   "decode_steps_per_chunk": args.steps_per_chunk,
                   "seed": w.seed},
        "whole_blocks": {"first_summary_token_ms": mean("whole_blocks", "first"),
                         "short_blocks_done_ms": mean("whole_blocks", "end"), "event_ms": mean("whole_blocks", "end")},
        "chunked": {"first_summary_token_ms": mean("chunked", "first"),
                    "short_blocks_done_ms": mean("chunked", "short_done"),
                    "long_block_prefilled_ms": mean("chunked", "long_prefilled"), "event_ms": mean("chunked", "end")},
    }
    print(json.dumps(out))


# ------------------------------------------------------------------------------------------
# many short sequences with summaries of unknown length (paper, Section 3.1 and Section 8): non-default
# ------------------------------------------------------------------------------------------

def run_locomo(args) -> None:
    """`--config locomo`: 192 sequences of 512..1024 tokens (the shape of the paper's second benchmark: short
    documents, six questions each) whose summaries stop after 32..T tokens.  The plan with pages on demand
    (stop flags on the device, pages drawn from a common reserve as blocks grow, given back when they stop)
    against the ordinary plan, which reserves T tokens for every sequence and decodes all of them to the end."""
    import torch

    from paper_2605_23296_b200 import binding as B
    from paper_2605_23296_b200.session import CompactionSession, bits_to_tensor

    if args.layout[2] != 1:
        raise SystemExit("--config locomo is a single-GPU measurement")
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    peaks, peak_kind = load_peaks()
    w = wl.locomo_like(steps=args.decode_steps or 256).materialise()
    T, Bn, P = w.decode_steps, w.num_blocks, w.page_size
    stop = w.stop_lens
    stream = torch.cuda.current_stream(dev)
    d = lambda bits: bits_to_tensor(bits, dev)
    q, k, v, qd, kd, vd = (d(x) for x in (w.q, w.k, w.v, w.q_dec, w.k_dec, w.v_dec))
    o = torch.empty_like(q)
    od = torch.empty((T, Bn, w.num_q_heads, w.head_dim), dtype=torch.bfloat16, device=dev)
    flush = torch.empty(256 * 1024 * 1024, dtype=torch.uint8, device=dev)
    # stop flags of every step, and of every release point, staged on the device before the timed region
    steps_idx = np.arange(T)[:, None]
    flags = torch.from_numpy((steps_idx < stop[None, :]).astype(np.int32)).to(dev)
    release_every = 32
    first_pages = int((w.block_lens // P + 1).sum())
    # the pool: first pages + what the summaries really need (+ a margin), instead of T tokens for everybody
    need = int((-(-(w.block_lens.astype(np.int64) + stop) // P)).sum())
    free = w.free_pages[:max(first_pages, need) + 64]
    new_ev = lambda: torch.cuda.Event(enable_timing=True)

    def reserved():
        s = CompactionSession(w.block_lens, T, w.num_q_heads, w.num_kv_heads, w.head_dim, w.free_pages, w.num_pages,
                              scale=w.scale)
        ev = [new_ev() for _ in range(3)]
        ev[0].record(stream)
        s.prefill(q, k, v, out=o)
        s.append_prefill(k, v)
        ev[1].record(stream)
        for t in range(T):
            s.decode_append(qd[t], kd[t], vd[t], out=od[t])
        ev[2].record(stream)
        return s, ev

    def on_demand():
        s = CompactionSession(w.block_lens, T, w.num_q_heads, w.num_kv_heads, w.head_dim, free, w.num_pages,
                              scale=w.scale, dynamic_pages=True)
        ev = [new_ev() for _ in range(3)]
        ev[0].record(stream)
        s.prefill(q, k, v, out=o)
        s.append_prefill(k, v)
        ev[1].record(stream)
        for t in range(T):
            s.decode_append_dynamic(qd[t], kd[t], vd[t], flags[t], out=od[t])
            if t % release_every == release_every - 1 and t + 1 < T:
                s.release(flags[t + 1])
        ev[2].record(stream)
        return s, ev

    res = {"reserved": [], "on_demand": []}
    pages_end = None
    for i in range(args.warmup + args.steps):
        for name, fn in (("reserved", reserved), ("on_demand", on_demand)):
            flush.fill_(1)
            s, ev = fn()
            torch.cuda.synchronize(dev)
            assert s.status() == 0
            if name == "on_demand":
                s.sync()
                pages_end = int(s.export(B.ARR_PAGES_ASSIGNED).sum())
            s.close()
            if i >= args.warmup:
                res[name].append((ev[0].elapsed_time(ev[1]), ev[1].elapsed_time(ev[2])))
    row = 2.0 * w.num_kv_heads * w.head_dim * 2.0
    L = w.block_lens.astype(np.float64)
    bytes_all = sum(float((L + t + 1).sum()) for t in range(T)) * row
    bytes_live = sum(float(((L + t + 1) * (t < stop)).sum()) for t in range(T)) * row
    out = {"metric": "decode of many short sequences whose summaries stop at different lengths", "unit": "ms", "n_gpus": 1,
           "steps": args.steps, "warmup": args.warmup, "dtype": "bf16", "data": "synthetic",
           "config": {"workload": "locomo", "sequences": Bn, "block_lens": f"{int(w.block_lens.min())}..{int(w.block_lens.max())}",
                      "q_heads": w.num_q_heads, "kv_heads": w.num_kv_heads, "head_dim": w.head_dim, "decode_steps": T,
                      "stop_lens": f"{int(stop.min())}..{int(stop.max())}", "summary_tokens": int(stop.sum()), "seed": w.seed},
           "peaks": dict(peaks, kind=peak_kind)}
    for name, nbytes, tokens, pages in (("reserved", bytes_all, Bn * T, w.pages_needed), ("on_demand", bytes_live, int(stop.sum()), len(free))):
        pf, dc = (statistics.mean(x[j] for x in res[name]) for j in (0, 1))
        out[name] = {"prefill_and_append_ms": pf, "decode_ms": dc, "decode_us_per_step": dc * 1e3 / T,
                     "kv_bytes_read": nbytes, "decode_gbs": nbytes / (dc * 1e-3) / 1e9,
                     "decode_frac_of_hbm_peak": nbytes / (dc * 1e-3) / 1e9 / peaks["hbm_gbs"],
                     "tokens_decoded": tokens, "pool_pages": pages}
    out["on_demand"]["pages_held_at_end"] = pages_end
    print(json.dumps(out))


# ------------------------------------------------------------------------------------------
# compaction in the background of a decoding agent (paper, Section 8: asynchronous compaction)
# ------------------------------------------------------------------------------------------

def run_async(args) -> None:
    """`--config async`: a foreground sequence keeps decoding over a 100k-token cache on a high-priority
    stream while compaction events (the dense8b workload) run on a low-priority stream with an SM
    budget.  Reports the foreground's step times and the event's time, alone and together."""
    import torch

    from paper_2605_23296_b200.session import CompactionSession, bits_to_tensor

    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    sms = torch.cuda.get_device_properties(dev).multi_processor_count
    fg_stream = torch.cuda.Stream(dev, priority=-1)
    bg_stream = torch.cuda.Stream(dev, priority=0)
    rng = np.random.default_rng(5)
    Hq, Hkv, d, ctx, steps = 32, 8, 128, 100_000, args.decode_steps or 200
    bits = lambda shape: wl.f32_to_bf16_bits(rng.standard_normal(shape, dtype=np.float32))
    to = lambda b: bits_to_tensor(b, dev)
    pages = (ctx + steps + 15) // 16 + 1
    with torch.cuda.stream(fg_stream):
        fg = CompactionSession([ctx], steps, Hq, Hkv, d, np.arange(pages, dtype=np.int32), pages)
        hk, hv = to(bits((ctx, Hkv, d))), to(bits((ctx, Hkv, d)))
        fq, fk, fv = to(bits((steps, 1, Hq, d))), to(bits((steps, 1, Hkv, d))), to(bits((steps, 1, Hkv, d)))
        fo = torch.empty_like(fq)
    w = make_workload("dense8b").materialise()
    bq, bk, bv, bqd, bkd, bvd = (to(x) for x in (w.q, w.k, w.v, w.q_dec, w.k_dec, w.v_dec))
    bo = torch.empty_like(bq)
    bod = torch.empty((w.decode_steps, w.num_blocks, Hq, d), dtype=torch.bfloat16, device=dev)
    torch.cuda.synchronize(dev)

    def background(budget):
        with torch.cuda.stream(bg_stream):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(bg_stream)
            s = CompactionSession(w.block_lens, w.decode_steps, Hq, Hkv, d, w.free_pages, w.num_pages, scale=w.scale,
                                  num_sms=budget)
            s.prefill(bq, bk, bv, out=bo)
            s.append_prefill(bk, bv)
            for t in range(w.decode_steps):
                s.decode_append(bqd[t], bkd[t], bvd[t], out=bod[t])
            e1.record(bg_stream)
        return s, e0, e1

    def rewind():
        # the foreground's cache goes back to the bare context (plan uploaded again, the context appended
        # again), so that every measurement decodes the same steps over the same lengths
        with torch.cuda.stream(fg_stream):
            from paper_2605_23296_b200 import binding as B
            fg._check(B.cpa_plan_upload(fg.plan, fg.index_buf, fg.index_buf.numel(), fg._stream()), "cpa_plan_upload")
            fg.append_prefill(hk, hv)
        fg_stream.synchronize()

    def foreground(t0, t1):
        evs = []
        with torch.cuda.stream(fg_stream):
            for t in range(t0, t1):
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record(fg_stream)
                fg.decode_append(fq[t], fk[t], fv[t], out=fo[t])
                e1.record(fg_stream)
                evs.append((e0, e1))
        return evs

    def stats(evs):
        ms = np.array([a.elapsed_time(b) for a, b in evs]) * 1e3
        return {"p50_us": float(np.percentile(ms, 50)), "p95_us": float(np.percentile(ms, 95)), "max_us": float(ms.max())}

    results = []
    quarter = steps // 4
    for _ in range(2):   # warm-up of both paths
        rewind()
        s, _, _ = background(sms)
        foreground(0, steps)
        torch.cuda.synchronize(dev)
        s.close()
    rewind()
    evs = foreground(0, steps)
    torch.cuda.synchronize(dev)
    alone_fg = stats(evs)
    for budget in [sms, (3 * sms) // 4, sms // 2, sms // 4]:
        s, e0, e1 = background(budget)
        torch.cuda.synchronize(dev)
        alone_bg = e0.elapsed_time(e1)
        s.close()
        # four events in a row, a quarter of the foreground's steps enqueued behind each, so that both
        # streams have work for the whole measurement
        rewind()
        evs, bgs = [], []
        for i in range(4):
            bgs.append(background(budget))
            evs += foreground(i * quarter, (i + 1) * quarter)
        torch.cuda.synchronize(dev)
        assert all(x[0].status() == 0 for x in bgs) and fg.status() == 0
        results.append({"sm_budget": budget, "event_ms_alone": alone_bg,
                        "event_ms_shared": float(np.mean([x[1].elapsed_time(x[2]) for x in bgs])),
                        "foreground_shared": stats(evs)})
        for x in bgs:
            x[0].close()
    print(json.dumps({"metric": "foreground decode step time next to a background compaction event", "unit": "us",
                      "config": {"workload": "async", "foreground": f"1 sequence, {ctx}-token cache, {steps} steps, 32/8/128",
                                 "background": "dense8b event (8 x 4096, T=256) on a low-priority stream", "sms": sms},
                      "foreground_alone": alone_fg, "budgets": results}))
    fg.close()


def main() -> None:
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", default=DEFAULT_CONFIG, choices=sorted(wl.CONFIGS) + ["prefix8b", "async", "mixed16k", "locomo"])
    ap.add_argument("--no-per-config", dest="per_config", action="store_false",
                    help="skip the per_config measurements of the other configurations")
    ap.add_argument("--blocks", type=int, default=0, help="override the number of blocks (profiling)")
    ap.add_argument("--block-len", type=int, default=0, help="override the block length (profiling)")
    ap.add_argument("--decode-steps", type=int, default=0, help="override the decode steps (profiling)")
    ap.add_argument("--pages-per-split", type=int, default=0, help="decode split size (0 = planner's choice)")
    ap.add_argument("--decode-sms", type=int, default=0, help="mixed16k: SMs left to the decode wave beside a prefill chunk")
    ap.add_argument("--steps-per-chunk", type=int, default=16, help="mixed16k: decode steps the schedule gives one chunk")
    ap.add_argument("--separate-append", action="store_true",
                    help="per decode step call cpa_kv_append and cpa_decode instead of the fused cpa_decode_append")
    ap.add_argument("--skip-e2e", action="store_true", help="skip the host-buffer leg (profiling)")
    ap.add_argument("--e2e-chunk", type=int, default=4096,
                    help="tokens per prefill chunk of the host-buffer leg (copies overlap the kernels); 0 = whole blocks, no overlap")
    ap.add_argument("--skip-cpu", action="store_true", help="skip the CPU oracle leg (profiling)")
    args = ap.parse_args()
    args.overrides = {"num_blocks": args.blocks, "block_len": args.block_len, "steps": args.decode_steps}
    if args.config in ("ragged", "split", "tiny") and args.block_len:
        ap.error("--block-len does not apply to this configuration")
    if args.config == "tiny":
        args.overrides = {}
    args.layout = rank_layout(args.gpus, os.environ, args.impl)
    if args.layout[0] == "spawn":
        raise SystemExit(subprocess.run(args.layout[1]).returncode)
    if args.config in ("prefix8b", "async", "mixed16k", "locomo"):
        if args.impl == "reference":
            raise SystemExit("--impl reference times the default layout's workloads")
        {"prefix8b": run_prefix, "async": run_async, "mixed16k": run_mixed, "locomo": run_locomo}[args.config](args)
    elif args.impl == "reference":
        run_reference(args)
    else:
        run_gpu(args)


if __name__ == "__main__":
    main()

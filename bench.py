#!/usr/bin/env python
"""Benchmark of the compaction attention hot path.

One "step" is one whole compaction event on synthetic blocks: plan -> ragged
causal prefill -> bulk KV append -> T x (one-token append + batched decode).
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
# dram__bytes_read.sum + dram__bytes_write.sum of one decode_split_kernel launch (134.93 MB + 3.9 MB),
# profiler capture of the kernel as it stands; None for workloads that were not captured
DECODE_DRAM_BYTES_PER_LAUNCH = {"dense8b": 138.8e6}
NOMINAL_BF16_TFLOPS = 2250.0


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
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
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


def run_gpu(args) -> None:
    import torch
    import torch.distributed as dist

    from paper_2605_23296_b200 import binding as B
    from paper_2605_23296_b200.session import CompactionSession, bits_to_tensor

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
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
    stream = torch.cuda.current_stream(dev)

    # host-side inputs in pinned memory (for the end-to-end leg) and device-resident copies
    def pinned(bits):
        return torch.from_numpy(bits.view(np.int16)).view(torch.bfloat16).pin_memory()

    h_q, h_k, h_v = pinned(w.q), pinned(w.k), pinned(w.v)
    h_qd, h_kd, h_vd = pinned(w.q_dec), pinned(w.k_dec), pinned(w.v_dec)
    d_q, d_k, d_v = h_q.to(dev), h_k.to(dev), h_v.to(dev)
    d_qd, d_kd, d_vd = h_qd.to(dev), h_kd.to(dev), h_vd.to(dev)
    d_o = torch.empty_like(d_q)
    d_od = torch.empty((T, Bn, w.num_q_heads, w.head_dim), dtype=torch.bfloat16, device=dev)
    h_o = torch.empty(d_o.shape, dtype=torch.bfloat16).pin_memory()
    h_od = torch.empty(d_od.shape, dtype=torch.bfloat16).pin_memory()
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
        for t in range(T):
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
    for _ in range(args.warmup):
        sessions.append(one_pass(d_q, d_k, d_v, d_qd, d_kd, d_vd, d_o, d_od))
        flush.fill_(1)
    torch.cuda.synchronize(dev)
    for s in sessions:
        assert s.status() == 0
        s.close()
    sessions.clear()

    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
    barrier()
    state["launches"] = 0
    step_ms, prefill_ms, decode_ms, append_ms, plan_ms, dec_samples = [], [], [], [], [], []
    for _ in range(args.steps):
        flush.fill_(1)   # L2 flush between timed steps (the step's own inputs, 400+ MB, exceed L2 anyway)
        ev = {n: torch.cuda.Event(enable_timing=True) for n in ("start", "planned", "prefilled", "appended", "end")}
        dec_events = []
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
        dec_samples += [(t, e0.elapsed_time(e1)) for t, e0, e1 in dec_events]
    barrier()
    launches = state["launches"]

    # ---- end to end: host buffers in, host buffers out, copies inside the timed region -----
    e2e_ms = []
    side = torch.cuda.Stream(dev)
    h2d = sum(t.numel() * 2 for t in (h_q, h_k, h_v, h_qd, h_kd, h_vd))
    d2h = (h_o.numel() + h_od.numel()) * 2
    for i in range(0 if args.skip_e2e else 1 + args.steps):
        flush.fill_(1)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize(dev)
        e0.record(stream)
        q, k, v = (t.to(dev, non_blocking=True) for t in (h_q, h_k, h_v))
        qd, kd, vd = (t.to(dev, non_blocking=True) for t in (h_qd, h_kd, h_vd))
        ev_pre = {n: torch.cuda.Event() for n in ("planned", "prefilled", "appended")}
        s = one_pass(q, k, v, qd, kd, vd, d_o, d_od, ev_pre)
        # the prefill output goes home on a side stream while the decode steps run
        side.wait_event(ev_pre["prefilled"])
        with torch.cuda.stream(side):
            h_o.copy_(d_o, non_blocking=True)
        h_od.copy_(d_od, non_blocking=True)
        stream.wait_stream(side)
        e1.record(stream)
        torch.cuda.synchronize(dev)
        assert s.status() == 0
        s.close()
        if i > 0:
            e2e_ms.append(e0.elapsed_time(e1))

    clocks = sampler.stop() if rank == 0 else {}   # sampled over both timed legs (device-resident and end-to-end)
    ms = max_over_ranks(statistics.mean(step_ms), world, dev)
    e2e = max_over_ranks(statistics.mean(e2e_ms), world, dev) if e2e_ms else float("nan")
    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    tokens = whole_job_tokens(w, world)
    pf_ms, dc_ms = statistics.mean(prefill_ms), statistics.mean(decode_ms)
    pf_tflops = prefill_flops(w) / (pf_ms * 1e-3) / 1e12
    total_kv = sum(decode_kv_bytes(w, t) for t in range(T))
    dec_gbs_phase = total_kv / (dc_ms * 1e-3) / 1e9           # includes the per-step appends
    # dominant kernel: the decode launches (split + merge), per-launch event pairs on sampled steps
    samp_bytes = statistics.mean(decode_kv_bytes(w, t) for t, _ in dec_samples)
    samp_ms = statistics.mean(m for _, m in dec_samples)
    pair_us = samp_ms * 1e3
    if not args.separate_append:
        # every decode step is exactly one launch (append fused in), so the average launch duration
        # over the timed region is the decode phase's CUDA-event time / T; event pairs around single
        # launches add their own cost and break the overlap of consecutive launches
        samp_bytes = total_kv / T
        samp_ms = dc_ms / T
    achieved = samp_bytes / (samp_ms * 1e-3) / 1e9
    # DRAM bytes per launch (read + written) from a profiler capture of this kernel on the default
    # workload; the capture replays each launch with a cold L2, whereas consecutive launches of a
    # real step share L2 contents (the scan direction alternates), so this is the upper figure
    overridden = args.blocks or args.block_len or args.decode_steps or args.pages_per_split or args.separate_append
    traffic = DECODE_DRAM_BYTES_PER_LAUNCH.get(args.config) if not overridden else None
    roofline = {"bound": "hbm", "kernel": "decode_split_kernel (one launch per step: append, split-K scan and merge fused)",
                "achieved": achieved, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                "frac": achieved / peaks["hbm_gbs"], "peak_kind": f"of {peak_kind}",
                "frac_of_nominal_8TBs": achieved / NOMINAL_HBM_GBS,
                "launch_us": samp_ms * 1e3, "bytes_per_launch": samp_bytes,
                "launches_timed": (T * args.steps if not args.separate_append else len(dec_samples)),
                "launch_us_event_pair_sampled": pair_us, "traffic": traffic}

    if args.skip_cpu:
        cpu = {"estimated_step_s": float("nan"), "cores": 0, "sample": "skipped", "measured_s": 0.0}
    else:
        cpu = oracle_sample_seconds(w, rows_per_block=32, decode_samples=8)
    out = {
        "metric": METRIC, "value": tokens / (ms * 1e-3), "unit": UNIT, "n_gpus": world,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": dict(workload_desc(w), l2="256 MiB write between timed steps; step inputs (>400 MB) exceed L2",
                       parallelism=f"replicas x{world} (independent blocks, no collective)"),
        "phases": {"plan_ms": statistics.mean(plan_ms), "prefill_ms": pf_ms,
                   "bulk_append_ms": statistics.mean(append_ms), "decode_ms": dc_ms,
                   "prefill_tflops": pf_tflops,
                   "prefill_frac_of_bf16_peak": pf_tflops / peaks["bf16_tflops"],
                   "prefill_frac_of_nominal_2250": pf_tflops / NOMINAL_BF16_TFLOPS,
                   "decode_gbs_incl_append": dec_gbs_phase,
                   "decode_frac_of_hbm_peak": dec_gbs_phase / peaks["hbm_gbs"],
                   "peaks": dict(peaks, kind=peak_kind)},
        "roofline": roofline,
        "cpu_baseline": {"value": Bn * T / cpu["estimated_step_s"], "unit": UNIT, "cores": cpu["cores"],
                         "kind": "oracle", "sample": cpu["sample"], "measured_s": cpu["measured_s"]},
        "e2e": {"value": tokens / (e2e * 1e-3), "unit": UNIT, "ms_per_step": e2e,
                "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h},
        "gpu_launches": launches,
        "clocks": clocks,
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

    if int(os.environ.get("WORLD_SIZE", "1")) != 1:
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
# compaction in the background of a decoding agent (paper, Section 7: asynchronous compaction)
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
    ap.add_argument("--config", default="dense8b", choices=sorted(wl.CONFIGS) + ["prefix8b", "async"])
    ap.add_argument("--blocks", type=int, default=0, help="override the number of blocks (profiling)")
    ap.add_argument("--block-len", type=int, default=0, help="override the block length (profiling)")
    ap.add_argument("--decode-steps", type=int, default=0, help="override the decode steps (profiling)")
    ap.add_argument("--pages-per-split", type=int, default=0, help="decode split size (0 = planner's choice)")
    ap.add_argument("--separate-append", action="store_true",
                    help="per decode step call cpa_kv_append and cpa_decode instead of the fused cpa_decode_append")
    ap.add_argument("--skip-e2e", action="store_true", help="skip the host-buffer leg (profiling)")
    ap.add_argument("--skip-cpu", action="store_true", help="skip the CPU oracle leg (profiling)")
    args = ap.parse_args()
    args.overrides = {"num_blocks": args.blocks, "block_len": args.block_len, "steps": args.decode_steps}
    if args.config in ("ragged", "split", "tiny") and args.block_len:
        ap.error("--block-len does not apply to this configuration")
    if args.config == "tiny":
        args.overrides = {}
    if args.config in ("prefix8b", "async"):
        if args.impl == "reference":
            raise SystemExit("--impl reference times the default layout's workloads")
        run_prefix(args) if args.config == "prefix8b" else run_async(args)
    elif args.impl == "reference":
        run_reference(args)
    else:
        run_gpu(args)


if __name__ == "__main__":
    main()

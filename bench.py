#!/usr/bin/env python
"""Decode-step attention bench: FP8-KV (E4M3) paged cache, 64K context.

One "step" is one layer-step of the hot path on one batch: fused FP8 quantise-and-append
of the new token's K/V, the split-KV attention pass and the log-sum-exp merge.  The default
workload is the long-context serving scenario (batch 16, context 65536, 64 query / 8 KV
heads, head size 64, paged 16-token blocks with a random block table): 1 GiB of KV bytes
per step.  Several layer caches are rotated so that no step finds its bytes in L2.

  python bench.py --gpus N --steps K --warmup W            # this library (CUDA)
  python bench.py --impl reference --steps K --warmup W    # the float64 CPU oracle, bounded sample

Under torchrun every rank runs the same per-GPU workload on its own sequences (weak
scaling, no data-path collective); the whole-job value is total bytes / max-over-ranks time.
Prints ONE JSON line.
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

import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

import synth  # noqa: E402

METRIC = "fp8_kv_decode_attn_achieved_hbm_gbs_64k_ctx"
NOMINAL_HBM_GBS = 8000.0
FALLBACK_HBM_GBS = 6650.0


def measured_peak():
    try:
        with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


def algorithmic_bytes(w: synth.Workload, seq_lens, window: int, fp8: bool = True) -> int:
    """Bytes one layer-step has to move: visible K+V rows, the block-table entries that
    cover them, q and out, and the appended token (read bf16, write cache element)."""
    eb = 1 if fp8 else 2
    row = 2 * w.hkv * w.head_dim * eb
    total = 0
    for L in seq_lens:
        vis = L if window == 0 else min(window, L)
        total += vis * row + ((vis + w.block - 1) // w.block) * 4
    total += 2 * w.batch * w.hq * w.head_dim * 2                    # q in, out
    total += 2 * w.batch * w.hkv * w.head_dim * (2 + eb)            # new K/V read, cache write
    return total


class ClockSampler:
    """Samples SM clock and throttle reasons of this rank's GPU while the timed region runs."""

    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.rows, self.proc, self.index = [], None, index

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), "--query-gpu=" + self.Q,
                                          "--format=csv,noheader,nounits", "-lms", "50"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            threading.Thread(target=self._read, daemon=True).start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([x.strip() for x in line.split(",")])

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, pw, reasons = [], [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in self.rows:
            try:
                sm.append(float(r[0])); mx.append(float(r[1])); pw.append(float(r[2]))
            except Exception:
                continue
            for n, v in zip(names, r[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "power_w": statistics.median(pw) if pw else None, "samples": len(sm), "reasons": sorted(reasons)}


def physical_gpu_index(local_rank: int) -> int:
    vis = os.environ.get("CUDA_VISIBLE_DEVICES")
    if vis:
        try:
            return int(vis.split(",")[local_rank])
        except Exception:
            pass
    return local_rank


# ------------------------------------------------------------------ our arm ---

def build_layer(w: synth.Workload, layer: int, dev: str):
    """One layer's FP8 cache on the device (input preparation, see synth.device)."""
    from synth.device import fill_layer
    return fill_layer(w, layer, dev)


def shard_workload(w: synth.Workload, rank: int, world: int) -> synth.Workload:
    """Weak scaling over independent sequences: rank r of `world` runs the same shape on sequences of its
    own (a different seed), so the job processes world x the single-GPU units with no data-path collective."""
    if world > 1:
        w.config_id = w.config_id + 100 * rank
    return w


def shard_plan(w: synth.Workload, seq_lens, rank: int, world: int, mode: str, window: int = 0):
    """What rank `rank` of `world` holds and moves in one layer-step under the three ways the path shards
    (batch: its own sequences; heads: Hkv/world KV heads of every sequence; context: every world-th cache block
    of every sequence).  Returns (workload of the rank's shard, its seq_lens for attention, its seq_lens for the
    append, algorithmic bytes the rank moves per step).  Host arithmetic only."""
    import dataclasses
    from paper_2602_11937_b200.parallel import context_slice, head_slice
    lens = torch.as_tensor(seq_lens, dtype=torch.int32)
    if mode == "batch":
        ws = shard_workload(dataclasses.replace(w), rank, world)
        return ws, lens, lens, algorithmic_bytes(ws, lens.tolist(), window)
    if mode == "heads":
        kv, qh = head_slice(rank, world, w.hkv, w.hq // w.hkv)
        ws = dataclasses.replace(w, hkv=kv.stop - kv.start, hq=qh.stop - qh.start)
        return ws, lens, lens, algorithmic_bytes(ws, lens.tolist(), window)
    if mode == "context":
        if window != 0:
            raise ValueError("context sharding covers full-attention layers only")
        local, app = context_slice(lens, rank, world, w.block)
        per_rank_blocks = (w.blocks_per_seq + world - 1) // world
        ws = dataclasses.replace(w, context=per_rank_blocks * w.block)
        row = 2 * w.hkv * w.head_dim
        nbytes = sum(int(L) * row + ((int(L) + w.block - 1) // w.block) * 4 for L in local.tolist())
        nbytes += 2 * w.batch * w.hq * w.head_dim * 2                       # q in, out (every rank has both)
        nbytes += 3 * 2 * w.hkv * w.head_dim * int((app > 0).sum())         # new K/V read + cache write, owner only
        nbytes += (world + 1) * w.batch * w.hq * (w.head_dim + 1) * 4 if world > 1 else 0   # partials written, gathered ones read
        return ws, local, app, nbytes
    raise ValueError(mode)


def max_over_ranks(values, world: int, device):
    """Element-wise maximum of a list of floats over all ranks (the slowest rank sets the job's time)."""
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    if world > 1:
        import torch.distributed as dist
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(x) for x in t.tolist()]


def sum_over_ranks(value: float, world: int, device) -> float:
    t = torch.tensor([value], dtype=torch.float64, device=device)
    if world > 1:
        import torch.distributed as dist
        dist.all_reduce(t)
    return float(t.item())


def job_throughput_gbs(bytes_per_rank_step: int, world: int, ms_per_step: float) -> float:
    """Whole-job value: every rank moves bytes_per_rank_step per step, the step takes the slowest rank's time."""
    return world * bytes_per_rank_step / (ms_per_step * 1e-3) / 1e9


def launch_plan(gpus: int, env) -> tuple:
    """How this process takes part in a run on `gpus` GPUs: ("rank", rank, local_rank, world) when a launcher
    started it (its world size must be `gpus`), ("single",) for one GPU, ("spawn", gpus) when it has to start the
    ranks itself.  Anything else is an error: a run never reports fewer GPUs than it was asked for."""
    if gpus < 1:
        raise SystemExit("--gpus must be at least 1")
    if "WORLD_SIZE" in env:
        world = int(env["WORLD_SIZE"])
        if world != gpus:
            raise SystemExit("--gpus %d, but the launcher started %d ranks" % (gpus, world))
        return ("rank", int(env.get("RANK", "0")), int(env.get("LOCAL_RANK", "0")), world)
    return ("single",) if gpus == 1 else ("spawn", gpus)


def spawn_ranks(gpus: int) -> int:
    """Re-runs this command line as `gpus` ranks under torch.distributed.run on this node; returns its exit code."""
    import socket
    with socket.socket() as sk:
        sk.bind(("127.0.0.1", 0))
        port = sk.getsockname()[1]
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", str(gpus),
           "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:]
    return subprocess.call(cmd)


def median_region(regions):
    """Index of the region whose time is the median of all (the lower one of the middle two)."""
    order = sorted(range(len(regions)), key=lambda i: regions[i])
    return order[(len(order) - 1) // 2]


def run_ours(args, plan):
    import paper_2602_11937_b200 as P

    rank, local_rank, world = (plan[1], plan[2], plan[3]) if plan[0] == "rank" else (0, 0, 1)
    if torch.cuda.device_count() <= local_rank:
        raise SystemExit("rank %d needs GPU %d, this node shows %d" % (rank, local_rank, torch.cuda.device_count()))
    torch.cuda.set_device(local_rank)
    dev = "cuda:%d" % local_rank
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device(dev))

    mode = args.shard
    w0 = synth.workload(args.config)
    # the layer kind that is timed: the workload's own for the one- and two-layer workloads, the full-context layer
    # of the 36-layer ones, or --window
    window = args.window if args.window is not None else (0 if len(w0.windows) > 2 else w0.windows[0])
    if mode == "context" and window != 0:
        raise SystemExit("--shard context covers full-attention layers only")
    seq_global = synth.draw_seq_lens(shard_workload(synth.workload(args.config), rank, world) if mode == "batch" else w0)
    w, lens_attn, lens_append, bytes_rank = shard_plan(w0, seq_global, rank, world, mode, window)
    seq_lens = lens_attn.to(dev)
    seq_append = lens_append.to(dev)
    layers = [build_layer(w, l, dev) for l in range(args.layers)]
    desc = P.layer_desc(window=window, num_q_heads=w.hq, num_kv_heads=w.hkv, head_dim=w.head_dim,
                        block_size=w.block)
    if args.contiguous:
        for L in layers:
            L["table"] = None

    def view_of(L, lens):
        return P.kv_view(L["k_cache"], L["v_cache"], lens, block_table=L["table"], max_blocks_per_seq=w.blocks_per_seq,
                         k_scale=L["k_scale"], v_scale=L["v_scale"])
    views = [view_of(L, seq_lens) for L in layers]
    views_append = views if mode != "context" else [view_of(L, seq_append) for L in layers]
    q = synth.draw_q(w, 0, dev)
    k_new, v_new = synth.draw_new_kv(w, 0, dev)
    sinks = synth.draw_sinks(w, 0, dev)
    out = torch.empty(w.batch, w.hq, w.head_dim, dtype=torch.bfloat16, device=dev)
    decode = P.puzzle_decode_attn_tcgen05 if args.kernel == "tcgen05" else P.puzzle_decode_attn
    if args.kernel == "tcgen05":
        kernel_name = "decode_attn_tc_kernel (tcgen05 split-KV pass with the merge fused in)"
        dtype_name = "e4m3 tcgen05 mma on the cache codes, f32 accumulate and softmax"
    else:
        kernel_name = "%s<%s> (split-KV pass with the merge fused in)" % (
            P.puzzle_decode_attn_kernel_name(desc, views[0], w.batch, args.splits), "fp8")
        dtype_name = "f16 mma on e4m3 codes, f32 accumulate and softmax"
    ws = torch.empty(P.puzzle_decode_attn_workspace_bytes(desc, w.batch, args.splits), dtype=torch.uint8, device=dev)
    P.puzzle_decode_attn_workspace_init(desc, w.batch, ws)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    stream = torch.cuda.current_stream()
    ctx = None
    if mode == "context":
        from paper_2602_11937_b200.parallel import ContextShardedAttention
        ctx = ContextShardedAttention(desc, w.batch, dev, world, num_splits=args.splits)

    def attention(i, qq):
        if ctx is not None:    # partial over this rank's blocks -> one all-gather -> merge with the sink
            ctx.step(views[i % len(views)], qq, sinks, out)
        else:
            decode(desc, views[i % len(views)], qq, sinks, out, None, num_splits=args.splits, workspace=ws,
                   dev_status=status, stream=stream)

    def step(i, events=None):
        P.puzzle_kv_append(desc, views_append[i % len(views)], k_new, v_new, dev_status=status, stream=stream)
        if events is not None:
            ea, eb = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            ea.record(stream)
        attention(i, q)
        if events is not None:
            eb.record(stream)
            events.append((ea, eb))

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    warmup = max(args.warmup, 3)
    for i in range(warmup):
        step(i)
    barrier()

    # ---- timed regions: device-resident inputs.  A region is exactly K steps between two events, with a barrier
    # and a device synchronise on both sides; regions are repeated until min_seconds of GPU time have passed.
    # Regions alternate between plain ones (nothing but the steps between the two events: their median gives
    # ms_per_step and value) and sampled ones (CUDA events around every attention launch, every 8th beyond 256
    # steps, which cost a few microseconds per step: the median sampled region gives the kernel's launch duration).
    every = 1 if args.steps <= 256 else 8
    sampler = ClockSampler(physical_gpu_index(local_rank))
    sampler.start()
    time.sleep(0.25)
    plain, sampled, launch_ms, launches_per_region = [], [], [], 0
    it = warmup
    while True:
        want_events = len(plain) > len(sampled)
        events = []
        l0 = P.puzzle_launch_count()
        t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        barrier()
        t0.record(stream)
        for k in range(args.steps):
            step(it + k, events if want_events and k % every == every - 1 else None)
        t1.record(stream)
        barrier()
        it += args.steps
        launches_per_region = P.puzzle_launch_count() - l0
        ms = max_over_ranks([t0.elapsed_time(t1)], world, dev)[0]
        if want_events:
            sampled.append(ms)
            launch_ms.append([a.elapsed_time(b) for a, b in events])
        else:
            plain.append(ms)
        n_regions = len(plain) + len(sampled)
        if len(sampled) >= 1 and (sum(plain) + sum(sampled) >= args.min_seconds * 1e3 or n_regions >= args.max_regions):
            break
    clocks = sampler.stop()
    ms_total = plain[median_region(plain)]
    mid = median_region(sampled)
    regions = plain + sampled

    # ---- end to end: the step's inputs start in pinned host memory, the result ends there.  One call of the
    # library per step (puzzle_decode_step_host: three host-to-device copies, append, attention, one copy back),
    # and the caller synchronises the stream before the next step because it reads the result on the host.  The
    # context-sharded layer has no such entry point; there the copies are the caller's.
    hin = torch.cat([t.reshape(-1).cpu() for t in (q, k_new, v_new)]).pin_memory()     # one buffer: one copy
    hq = hin[: q.numel()].view(q.shape)
    hk = hin[q.numel(): q.numel() + k_new.numel()].view(k_new.shape)
    hv = hin[q.numel() + k_new.numel():].view(v_new.shape)
    hout = torch.empty(out.shape, dtype=out.dtype).pin_memory()
    staging = torch.empty(P.puzzle_decode_step_host_staging_bytes(desc, w.batch), dtype=torch.uint8, device=dev)
    dq, dk, dv = torch.empty_like(q), torch.empty_like(k_new), torch.empty_like(v_new)

    def step_e2e(i):
        if ctx is None and args.kernel == "mma":
            P.puzzle_decode_step_host(desc, views[i % len(views)], hq, hk, hv, sinks, hout, staging, ws,
                                      num_splits=args.splits, dev_status=status, stream=stream)
            return
        dq.copy_(hq, non_blocking=True); dk.copy_(hk, non_blocking=True); dv.copy_(hv, non_blocking=True)
        P.puzzle_kv_append(desc, views_append[i % len(views)], dk, dv, dev_status=status, stream=stream)
        attention(i, dq)
        hout.copy_(out, non_blocking=True)

    for i in range(3):
        step_e2e(i)
    barrier()
    e2e_regions = []
    while True:
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        barrier()
        e0.record(stream)
        for i in range(args.steps):
            step_e2e(i)
            stream.synchronize()   # the caller reads the result on the host before the next step
        e1.record(stream)
        barrier()
        e2e_regions.append(max_over_ranks([e0.elapsed_time(e1)], world, dev)[0])
        if sum(e2e_regions) >= 0.5 * args.min_seconds * 1e3 or len(e2e_regions) >= args.max_regions:
            break
    ms_e2e = e2e_regions[median_region(e2e_regions)]

    # ---- read-only streaming probe (one pass over 2 GiB): the bandwidth a pure scan reaches on this device
    probe_buf = torch.empty(2 << 30, dtype=torch.uint8, device=dev)
    probe_buf.view(torch.int64).random_()
    probe_sink = torch.zeros(1, dtype=torch.int64, device=dev)
    probe_ms = []
    for i in range(3 + 20):
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(stream)
        P.puzzle_hbm_read_probe(probe_buf, probe_sink, stream=stream)
        b.record(stream)
        torch.cuda.synchronize()
        if i >= 3:
            probe_ms.append(a.elapsed_time(b))
    probe_gbs = probe_buf.numel() / (statistics.median(probe_ms) * 1e-3) / 1e9
    del probe_buf

    dev_flags = int(status.item()) | (int(ctx.status.item()) if ctx is not None else 0)
    # bytes of the step on this rank; the attention pass itself moves all of them but the appended token's
    kv_bytes_attn = bytes_rank - 2 * w.batch * w.hkv * w.head_dim * 3
    in_region = launch_ms[mid] or [ms_total / args.steps]
    all_launches = [x for r in launch_ms for x in r] or in_region
    attn_mean_ms = max_over_ranks([statistics.mean(in_region)], world, dev)[0]
    bytes_job = sum_over_ranks(float(bytes_rank), world, dev)

    if rank == 0:
        peak, peak_kind = measured_peak()
        ms_step = ms_total / args.steps
        value = bytes_job / (ms_step * 1e-3) / 1e9
        achieved = kv_bytes_attn / (attn_mean_ms * 1e-3) / 1e9
        par = {"batch": "dp%d (independent sequences per GPU, no collective)" % world,
               "heads": "tp%d over KV heads (no collective inside the path)" % world,
               "context": "cp%d over cache blocks (one all-gather of float32 partials, then the merge)" % world}[mode]
        line = {
            "metric": METRIC if args.config == 3 else "fp8_kv_decode_attn_achieved_hbm_gbs_" + w0.name,
            "value": round(value, 1), "unit": "GB/s", "n_gpus": world, "steps": args.steps, "warmup": warmup, "ms_per_step": round(ms_step, 5),
            "us_per_layer_step": round(ms_step * 1e3, 2), "higher_is_better": True,
            "value_frac_of_nominal_8TBs": round(value / world / NOMINAL_HBM_GBS, 4),
            "step_target_75pct_of_nominal_met": bool(value / world / NOMINAL_HBM_GBS >= 0.75),
            "scaling": "weak" if mode == "batch" else "strong",
            "vs_baseline": None, "dtype": dtype_name, "data": "synthetic",
            "config": {"workload": w0.name, "batch_per_gpu": w.batch, "context": w0.context, "q_heads": w.hq,
                       "kv_heads": w.hkv, "head_dim": w.head_dim, "block_size": w.block, "window": window,
                       "paged": not args.contiguous, "num_splits": args.splits, "rotating_layer_caches": len(layers),
                       "l2": "inputs larger than L2: %.0f MiB per step and GPU, %d caches rotated" % (
                           bytes_rank / 2 ** 20, len(layers)),
                       "parallelism": par},
            "timing": {"regions_plain": len(plain), "regions_with_launch_events": len(sampled),
                       "region_reported": "median of the plain regions (ms_per_step, value); the median region with "
                                          "events around the attention launches gives roofline.us_per_launch "
                                          "(the stand-alone duration of a launch: an event between two kernels "
                                          "keeps the second from being placed while the first drains, which the "
                                          "plain regions allow, so a plain step can be shorter than a sampled launch)",
                       "gpu_seconds_timed": round(sum(regions) / 1e3, 3),
                       "ms_per_step_min": round(min(plain) / args.steps, 5),
                       "ms_per_step_max": round(max(plain) / args.steps, 5),
                       "ms_per_step_with_launch_events": round(sampled[mid] / args.steps, 5)},
            "clocks": clocks,
            "e2e": {"value": round(bytes_job / (ms_e2e / args.steps * 1e-3) / 1e9, 1), "unit": "GB/s",
                    "ms_per_step": round(ms_e2e / args.steps, 5), "regions": len(e2e_regions),
                    "h2d_bytes_per_step": int(sum(t.numel() * t.element_size() for t in (q, k_new, v_new))),
                    "d2h_bytes_per_step": int(out.numel() * out.element_size())},
            "gpu_launches": int(launches_per_region),
            "roofline": {"bound": "hbm", "kernel": kernel_name,
                         "achieved": round(achieved, 1), "peak": peak, "peak_kind": peak_kind + " copy bandwidth",
                         "unit": "GB/s", "frac": round(achieved / peak, 4),
                         "frac_of_nominal_8TBs": round(achieved / NOMINAL_HBM_GBS, 4),
                         "target_75pct_of_nominal_met": bool(achieved / NOMINAL_HBM_GBS >= 0.75),
                         "us_per_launch": round(attn_mean_ms * 1e3, 2), "launches_sampled": len(in_region),
                         "launches_sampled_all_regions": len(all_launches),
                         "us_per_launch_median_all_regions": round(statistics.median(all_launches) * 1e3, 2),
                         "us_per_launch_min_all_regions": round(min(all_launches) * 1e3, 2),
                         "sm_mhz_median": clocks.get("sm_mhz"),
                         "bytes_per_launch": int(kv_bytes_attn),
                         "read_probe_gbs": round(probe_gbs, 1),
                         "traffic": ncu_traffic(args), "traffic_source": NCU_CAPTURE["source"]},
            "dev_status": dev_flags,
        }
        if args.cpu_baseline and mode == "batch":
            line["cpu_baseline"] = cpu_baseline(w, layers[0], seq_lens.tolist(), q, sinks, window)
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


def cpu_baseline(w, layer, seq_lens_host, q, sinks, window, pairs: int = 128):
    """The float64 oracle, as it stands, on this machine's cores, on a bounded sample of the same
    workload: all 8 query heads of `pairs` (sequence, KV head) pairs."""
    import oracle
    pairs = min(pairs, w.batch * w.hkv)
    items = [(p % w.batch, ((p // w.batch + p) % w.hkv) * 8 + g) for p in range(pairs) for g in range(8)]
    kc, vc = layer["k_cache"].cpu().numpy(), layer["v_cache"].cpu().numpy()
    table = layer["table"].cpu().numpy() if layer["table"] is not None else None
    import numpy as np
    lens = np.asarray(seq_lens_host, dtype=np.int32)
    cores = oracle.host_cores()
    t = time.perf_counter()
    oracle.decode_attn(kc, vc, oracle.KV_FP8_E4M3, table, w.blocks_per_seq, lens, layer["k_scale"].cpu().numpy(),
                       layer["v_scale"].cpu().numpy(), synth.bf16_bits(q), sinks.cpu().numpy(), window,
                       w.head_dim ** -0.5, items=items, threads=cores)
    dt = time.perf_counter() - t
    nbytes = sum((seq_lens_host[b] if window == 0 else min(window, seq_lens_host[b])) * 2 * w.head_dim
                 for b, _ in items[::8])
    return {"value": round(nbytes / dt / 1e9, 5), "unit": "GB/s", "cores": cores, "kind": "oracle",
            "seconds": round(dt, 2),
            "sample": "%d of %d (sequence, KV head) pairs, all 8 query heads each, full %d-token context" % (
                pairs, w.batch * w.hkv, w.context)}


# ------------------------------------------------------- 36-layer stack mode ---


# DRAM bytes per launch (dram__bytes_read.sum + dram__bytes_write.sum) of the default (CTA-balanced) split-KV kernel on the
# headline workload, from the one-launch `ncu --set full` capture summarised under profiles/; valid only for
# the kernel sources it was taken from, so it is tied to their hash and reported as null once they change.
NCU_CAPTURE = {
    "source": "profiles/decode_attn_cta_fp8_c3_64k_ncu_full.md (one launch, ncu --set full --clock-control none)",
    "workload": 3, "kernel": "mma", "splits": 0,
    "sources": ("decode_attn_cta.cu", "decode_tile.cuh", "decode_sched.cuh", "common.cuh", "decode_attn.cuh"),
    "sha256": "1cf92a3f269d5ab74de65037e8c0d3bfb2b26a0a6e2d4063e2953d2c8809e362",
    "dram_bytes_per_launch": 1075519000 + 4436736,
}


def ncu_traffic(args):
    if args.ncu_traffic is not None:
        return args.ncu_traffic
    c = NCU_CAPTURE
    if args.config != c["workload"] or args.kernel != c["kernel"] or args.splits != c["splits"] or args.contiguous:
        return None
    import hashlib
    h = hashlib.sha256()
    csrc = os.path.join(os.path.dirname(os.path.abspath(__file__)), "paper_2602_11937_b200", "csrc")
    try:
        for f in c["sources"]:
            with open(os.path.join(csrc, f), "rb") as fh:
                h.update(fh.read())
    except OSError:
        return None
    return c["dram_bytes_per_launch"] if h.hexdigest() == c["sha256"] else None

def run_stack(args):
    """One decode step of the 36-layer attention stack (workload 4 or 5) under a per-layer pattern, as one
    CUDA graph: append + attention per layer.  Prints its own JSON line (not the headline metric)."""
    import paper_2602_11937_b200 as P
    from synth.device import fill_layer, KV_BF16, KV_FP8_E4M3

    dev = "cuda:0"
    torch.cuda.set_device(0)
    kv_dtype = KV_BF16 if args.kv == "bf16" else KV_FP8_E4M3
    w = synth.workload(args.stack, pattern=args.pattern)
    windows = w.windows
    seq_lens_host = synth.draw_seq_lens(w).tolist()
    seq_lens = torch.tensor(seq_lens_host, dtype=torch.int32, device=dev)
    # every full-context layer gets a cache of its own; the window layers of one size share one pool cache but
    # each has its own random block table into it, so no two layers touch the same bytes
    pools, layers = {}, []
    for i, win in enumerate(windows):
        if win == 0:
            layers.append(fill_layer(w, i, dev, kv_dtype))
        else:
            if win not in pools:
                pools[win] = fill_layer(w, 1000 + win, dev, kv_dtype, with_table=False)
            L = dict(pools[win])
            L["table"] = synth.draw_block_table(w, i, w.batch * w.blocks_per_seq, dev)
            layers.append(L)
    q = [synth.draw_q(w, i, dev) for i in range(len(windows))]
    kv = [synth.draw_new_kv(w, i, dev) for i in range(len(windows))]
    sinks = [synth.draw_sinks(w, i, dev) for i in range(len(windows))]
    out = [torch.empty(w.batch, w.hq, w.head_dim, dtype=torch.bfloat16, device=dev) for _ in windows]
    stack = P.DecodeStack(windows, [L["k_cache"] for L in layers], [L["v_cache"] for L in layers], seq_lens,
                          [L["table"] for L in layers], w.blocks_per_seq, [L["k_scale"] for L in layers],
                          [L["v_scale"] for L in layers], sinks, kv_dtype=kv_dtype)
    g = stack.capture(q, [a for a, _ in kv], [b for _, b in kv], out)
    for _ in range(max(args.warmup, 3)):
        g.replay()
    torch.cuda.synchronize()
    steps = min(args.steps, 200)
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t0.record()
    for _ in range(steps):
        g.replay()
    t1.record()
    torch.cuda.synchronize()
    ms = t0.elapsed_time(t1) / steps
    nbytes = sum(algorithmic_bytes(w, seq_lens_host, win, fp8=kv_dtype == KV_FP8_E4M3) for win in windows)
    peak, kind = measured_peak()
    print(json.dumps({
        "metric": "decode_attn_stack_step", "workload": w.name, "kv": args.kv, "layers": len(windows),
        "full_layers": sum(1 for x in windows if x == 0), "window_sizes": sorted(set(x for x in windows if x)),
        "us_per_step": round(ms * 1e3, 1), "us_per_layer": round(ms * 1e3 / len(windows), 2),
        "algorithmic_gib_per_step": round(nbytes / 2 ** 30, 3), "gbs": round(nbytes / (ms * 1e-3) / 1e9, 1),
        "frac_of_" + kind: round(nbytes / (ms * 1e-3) / 1e9 / peak, 4), "steps": steps, "cuda_graph": True,
        "dev_status": int(stack.status.item())}))


# ------------------------------------------------- FP8 KV with and without scales ---

def run_study(args):
    """FP8 KV with calibrated scales, with scales rounded up to a power of two, and without scales (the three
    settings of the paper's Section "KV Quantization"), on synthetic K/V streams: how many elements underflow to
    zero, how many are clipped at +-448 (their nearest code would lie above it), the error of the dequantised values, and what that does to the attention
    output.  Everything numeric runs in the library: the streams are quantised by puzzle_kv_append_tokens under
    scales from puzzle_kv_amax_update / puzzle_kv_scales_from_amax, and the attention of the FP8 cache is compared
    with the library's own bf16-cache path on the same samples.  Counting and averaging is done with torch.
    Prints one JSON line per (stream, setting) and a markdown table."""
    import paper_2602_11937_b200 as P

    dev = "cuda:0"
    torch.cuda.set_device(0)
    batch, n_tok = 4, 4096
    w = synth.Workload("scale_study", 77, batch, n_tok, [0], paged=False)
    nb = batch * w.blocks_per_seq
    seq = torch.full((batch,), n_tok, dtype=torch.int32, device=dev)
    q = synth.draw_q(w, 0, dev)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    streams = [("gauss", 2.0 ** e) for e in (-8, -6, -4, -2, 0, 2, 4, 6, 8)] + [("heavy", 1.0), ("heavy", 2.0 ** -6),
                                                                             ("heads", 1.0), ("heads", 2.0 ** -5)]
    rows = []

    def attention(desc, k_cache, v_cache, ks, vs):
        view = P.kv_view(k_cache, v_cache, seq, max_blocks_per_seq=w.blocks_per_seq, k_scale=ks, v_scale=vs)
        ws = torch.zeros(P.puzzle_decode_attn_workspace_bytes(desc, batch, 0), dtype=torch.uint8, device=dev)
        P.puzzle_decode_attn_workspace_init(desc, batch, ws)
        out = torch.empty(batch, w.hq, w.head_dim, dtype=torch.bfloat16, device=dev)
        P.puzzle_decode_attn(desc, view, q, None, out, None, workspace=ws, dev_status=status)
        return out.float()

    for kind, sigma in streams:
        xk = synth.draw_study_stream(kind, sigma, batch, n_tok, "k", dev)
        xv = synth.draw_study_stream(kind, sigma, batch, n_tok, "v", dev)
        # the comparison run: the same samples in a bf16 cache (cache layout [block][Hkv][16][D])
        to_cache = lambda x: x.view(batch, w.blocks_per_seq, w.block, w.hkv, w.head_dim).permute(0, 1, 3, 2, 4) \
            .reshape(nb, w.hkv, w.block, w.head_dim).contiguous()
        ref = attention(P.layer_desc(kv_dtype=P.KV_BF16), to_cache(xk), to_cache(xv), None, None)
        ref_max = float(ref.abs().max())
        for setting in ("no scales", "amax/448", "amax/448 rounded up to 2^k"):
            if setting == "no scales":
                ks = torch.ones(w.hkv, device=dev)
                vs = torch.ones(w.hkv, device=dev)
            else:
                ks = P.calibrate_scales([xk], w.hkv, pow2=setting.endswith("2^k"), device=dev)
                vs = P.calibrate_scales([xv], w.hkv, pow2=setting.endswith("2^k"), device=dev)
            desc = P.layer_desc()
            kc = torch.zeros(nb, w.hkv, w.block, w.head_dim, dtype=torch.uint8, device=dev)
            vc = torch.zeros_like(kc)
            view = P.kv_view(kc, vc, seq, max_blocks_per_seq=w.blocks_per_seq, k_scale=ks, v_scale=vs)
            P.puzzle_kv_append_tokens(desc, view, xk, xv, dev_status=status)
            under = sat = 0.0
            num = den = 0.0
            for x, c, sc in ((xk, kc, ks), (xv, vc, vs)):
                xf = to_cache(x).float()
                code = c & 0x7F
                y = xf / sc[None, :, None, None]
                under += float(((code == 0) & (xf != 0)).float().mean()) / 2
                sat += float((y.abs() >= 464).float().mean()) / 2      # nearest code would lie above 448
                deq = c.view(torch.float8_e4m3fn).float() * sc[None, :, None, None]
                num += float((deq - xf).double().square().sum())
                den += float(xf.double().square().sum())
            out = attention(desc, kc, vc, ks, vs)
            err = float((out - ref).abs().max())
            row = {"study": "fp8_kv_scales", "stream": kind, "sigma": sigma, "setting": setting,
                   "underflow_frac": round(under, 6), "clipped_frac": round(sat, 6),
                   "rms_rel_err": round((num / den) ** 0.5, 5), "attn_max_abs_err": round(err, 5),
                   "attn_max_abs_err_over_max_out": round(err / max(ref_max, 1e-30), 5),
                   "k_scale_head0": float(ks[0]), "dev_status": int(status.item())}
            rows.append(row)
            print(json.dumps(row))
    print()
    print("| stream | sigma | setting | underflow to 0 | clipped at 448 | RMS rel. error | attention max abs err / max abs out |")
    print("|---|---|---|---|---|---|---|")
    for r in rows:
        print("| %s | 2^%d | %s | %.4f | %.4f | %.4f | %.4f |" % (
            r["stream"], round(__import__("math").log2(r["sigma"])), r["setting"], r["underflow_frac"], r["clipped_frac"],
            r["rms_rel_err"], r["attn_max_abs_err_over_max_out"]))


# ------------------------------------------------------------ reference arm ---

def run_reference(args):
    """Times the CPU oracle on a bounded sample of the same workload (rank 0 only)."""
    if int(os.environ.get("RANK", "0")) != 0:
        return
    import numpy as np
    import oracle

    w = synth.workload(args.config)
    full_batch = w.batch
    w.batch = 1                                   # the sample: one sequence, every head
    nb = w.blocks_per_seq
    window = w.windows[0]
    lens = np.asarray(synth.draw_seq_lens(w).tolist(), dtype=np.int32)
    caches, scales = {}, {}
    for which in ("k", "v"):
        x = synth.draw_kv_samples(w, which, nb, 0)
        s = x.abs().amax(dim=(0, 2, 3)) / 448.0
        caches[which] = (x / s[None, :, None, None]).to(torch.float8_e4m3fn).view(torch.uint8).numpy()
        scales[which] = s.numpy()
    table = synth.draw_block_table(w, 0, nb)
    table = None if table is None else table.numpy()
    q = synth.bf16_bits(synth.draw_q(w, 0))
    sinks = synth.draw_sinks(w, 0).numpy()
    cores = oracle.host_cores()

    def step():
        oracle.decode_attn(caches["k"], caches["v"], oracle.KV_FP8_E4M3, table, nb, lens, scales["k"], scales["v"],
                           q, sinks, window, w.head_dim ** -0.5, threads=cores)

    warm = min(args.warmup, 5)              # a CPU loop: more warm-up than this only costs time
    for _ in range(warm):
        step()
    t = time.perf_counter()
    for _ in range(args.steps):
        step()
    dt = (time.perf_counter() - t) / args.steps
    nbytes = algorithmic_bytes(w, lens.tolist(), window)
    value = round(nbytes / dt / 1e9, 5)
    sample = "1 of %d sequences per step (all 64 query heads, full %d-token context)" % (full_batch, w.context)
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": "GB/s",
        "n_gpus": int(os.environ.get("WORLD_SIZE", "1")), "steps": args.steps, "warmup": warm,
        "ms_per_step": round(dt * 1e3, 3), "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f64 (CPU oracle over fp8_e4m3 KV)", "data": "synthetic",
        "config": {"workload": synth.workload(args.config).name, "sample": sample},
        "cpu_baseline": {"value": value, "unit": "GB/s", "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


def run_tokens(args):
    """A decode step with --tokens N new tokens per sequence on workload 3 (a multi-token step, or a chunk of a
    prompt): bulk append of the N tokens + causal attention of the N query tokens by puzzle_decode_attn_tokens,
    timed with CUDA events over regions of --steps steps, beside the one-token step on the same caches.  Prints its
    own JSON line (not the headline metric)."""
    import paper_2602_11937_b200 as P
    import statistics

    dev = "cuda:0"
    torch.cuda.set_device(0)
    w = synth.workload(args.config)
    n_q = args.tokens
    layers = [build_layer(w, l, dev) for l in range(args.layers)]
    seq_lens = synth.draw_seq_lens(w).to(dev)
    desc = P.layer_desc(num_q_heads=w.hq, num_kv_heads=w.hkv, head_dim=w.head_dim, block_size=w.block)
    views = [P.kv_view(L["k_cache"], L["v_cache"], seq_lens, block_table=L["table"],
                       max_blocks_per_seq=w.blocks_per_seq, k_scale=L["k_scale"], v_scale=L["v_scale"]) for L in layers]
    g = torch.Generator(device=dev).manual_seed(0x5EED0000 + 77)
    q = torch.randn(w.batch, n_q, w.hq, w.head_dim, generator=g, device=dev).to(torch.bfloat16)
    k_new = torch.randn(w.batch, n_q, w.hkv, w.head_dim, generator=g, device=dev).to(torch.bfloat16)
    v_new = torch.randn(w.batch, n_q, w.hkv, w.head_dim, generator=g, device=dev).to(torch.bfloat16)
    sinks = synth.draw_sinks(w, 0, dev)
    out = torch.empty_like(q)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    ws = torch.zeros(P.puzzle_decode_attn_tokens_workspace_bytes(desc, w.batch, n_q), dtype=torch.uint8, device=dev)
    P.puzzle_decode_attn_tokens_workspace_init(desc, w.batch, n_q, ws)
    ws1 = torch.zeros(P.puzzle_decode_attn_workspace_bytes(desc, w.batch, 0), dtype=torch.uint8, device=dev)
    P.puzzle_decode_attn_workspace_init(desc, w.batch, ws1)
    q1, k1, v1, out1 = q[:, 0].contiguous(), k_new[:, 0].contiguous(), v_new[:, 0].contiguous(), out[:, 0].contiguous()

    def step_tokens(i):
        P.puzzle_kv_append_tokens(desc, views[i % len(views)], k_new, v_new, None, dev_status=status)
        P.puzzle_decode_attn_tokens(desc, views[i % len(views)], q, sinks, out, workspace=ws, dev_status=status)

    def step_one(i):
        P.puzzle_kv_append(desc, views[i % len(views)], k1, v1, dev_status=status)
        P.puzzle_decode_attn(desc, views[i % len(views)], q1, sinks, out1, None, workspace=ws1, dev_status=status)

    def timed(step):
        for i in range(max(3, args.warmup)):
            step(i)
        torch.cuda.synchronize()
        regions = []
        while len(regions) < 3 or (sum(regions) < args.min_seconds * 1e3 and len(regions) < args.max_regions):
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            for i in range(args.steps):
                step(i)
            b.record()
            torch.cuda.synchronize()
            regions.append(a.elapsed_time(b))
        return statistics.median(regions) / args.steps * 1e3

    us_one = timed(step_one)
    us_tok = timed(step_tokens)
    lens = seq_lens.tolist()
    nbytes = algorithmic_bytes(w, lens, 0)
    print(json.dumps({
        "metric": "multi_token_decode_step", "workload": w.name, "query_tokens_per_sequence": n_q,
        "us_per_step": round(us_tok, 2), "us_per_one_token_step": round(us_one, 2),
        "ratio_to_one_token_step": round(us_tok / us_one, 3), "steps": args.steps,
        "kv_gbs": round(nbytes / (us_tok * 1e-6) / 1e9, 1),
        "l2": "%d layer caches of %.0f MiB rotated (larger than L2)" % (len(layers), nbytes / 2 ** 20),
        "kernel": "decode_attn_tokens_kernel (pairs of query tokens share one pass over the K/V tiles)",
        "dev_status": int(status.item())}))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200, help="steps per timed region")
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--min-seconds", type=float, default=0.5,
                    help="timed regions of --steps steps are repeated until this much GPU time has passed")
    ap.add_argument("--max-regions", type=int, default=400)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", type=int, default=None, help="workload id 1..5 (default 3: batch 16, context 64K; "
                    "5 with --shard heads|context)")
    ap.add_argument("--shard", default="batch", choices=["batch", "heads", "context"],
                    help="how N GPUs share the layer: own sequences each (default), KV heads, or cache blocks")
    ap.add_argument("--window", type=int, default=None, help="time a layer of this window (0 = full context) "
                    "instead of the workload's first layer kind")
    ap.add_argument("--splits", type=int, default=0, help="0 = balanced schedule, S = fixed splits per sequence")
    ap.add_argument("--layers", type=int, default=4, help="distinct layer caches rotated between steps")
    ap.add_argument("--stack", type=int, default=0, choices=[0, 4, 5],
                    help="instead of the headline run: one step of the 36-layer stack of workload 4 or 5")
    ap.add_argument("--study", default=None, choices=["scales"],
                    help="instead of the headline run: FP8 KV with, with power-of-two and without scales on synthetic streams")
    ap.add_argument("--tokens", type=int, default=0,
                    help="instead of the headline run: a step with this many new tokens per sequence (multi-token kernel)")
    ap.add_argument("--pattern", default="parent", choices=["parent", "every4th", "selective"])
    ap.add_argument("--kv", default="fp8", choices=["fp8", "bf16"])
    ap.add_argument("--kernel", default="mma", choices=["mma", "tcgen05"],
                    help="split-KV kernel of the headline run: mma.sync (default) or the tcgen05 / tensor-memory one")
    ap.add_argument("--contiguous", action="store_true",
                    help="diagnostic: drop the block table (sequence b owns blocks b*blocks_per_seq ...)")
    ap.add_argument("--no-cpu-baseline", dest="cpu_baseline", action="store_false")
    ap.add_argument("--ncu-traffic", type=float, default=None,
                    help="DRAM bytes per launch of the attention kernel from an ncu capture (reported as-is)")
    args = ap.parse_args()
    if args.config is None:
        args.config = 3 if args.shard == "batch" else 5
    plan = launch_plan(args.gpus, os.environ)
    if plan[0] == "spawn":
        sys.exit(spawn_ranks(args.gpus))
    if args.study:
        run_study(args)
    elif args.tokens:
        run_tokens(args)
    elif args.stack:
        run_stack(args)
    elif args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args, plan)


if __name__ == "__main__":
    main()

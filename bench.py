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


def max_over_ranks(values, world: int, device):
    """Element-wise maximum of a list of floats over all ranks (the slowest rank sets the job's time)."""
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    if world > 1:
        import torch.distributed as dist
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(x) for x in t.tolist()]


def job_throughput_gbs(bytes_per_rank_step: int, world: int, ms_per_step: float) -> float:
    """Whole-job value: every rank moves bytes_per_rank_step per step, the step takes the slowest rank's time."""
    return world * bytes_per_rank_step / (ms_per_step * 1e-3) / 1e9


def run_ours(args):
    import paper_2602_11937_b200 as P

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local_rank)
    dev = "cuda:%d" % local_rank
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device(dev))

    w = shard_workload(synth.workload(args.config), rank, world)
    window = w.windows[0]
    seq_lens_host = synth.draw_seq_lens(w).tolist()
    seq_lens = torch.tensor(seq_lens_host, dtype=torch.int32, device=dev)
    layers = [build_layer(w, l, dev) for l in range(args.layers)]
    desc = P.layer_desc(window=window, num_q_heads=w.hq, num_kv_heads=w.hkv, head_dim=w.head_dim,
                        block_size=w.block)
    if args.contiguous:
        for L in layers:
            L["table"] = None
    views = [P.kv_view(L["k_cache"], L["v_cache"], seq_lens, block_table=L["table"],
                       max_blocks_per_seq=w.blocks_per_seq, k_scale=L["k_scale"], v_scale=L["v_scale"])
             for L in layers]
    q = synth.draw_q(w, 0, dev)
    k_new, v_new = synth.draw_new_kv(w, 0, dev)
    sinks = synth.draw_sinks(w, 0, dev)
    out = torch.empty(w.batch, w.hq, w.head_dim, dtype=torch.bfloat16, device=dev)
    decode = P.puzzle_decode_attn_tcgen05 if args.kernel == "tcgen05" else P.puzzle_decode_attn
    if args.kernel == "tcgen05":
        kernel_name = "decode_attn_tc_kernel (tcgen05 split-KV pass with the merge fused in)"
        dtype_name = "e4m3 tcgen05 mma on the cache codes, f32 accumulate and softmax"
    else:
        kernel_name = "decode_attn_kernel<fp8> (split-KV pass with the merge fused in)"
        dtype_name = "f16 mma on e4m3 codes, f32 accumulate and softmax"
    ws = torch.empty(P.puzzle_decode_attn_workspace_bytes(desc, w.batch, args.splits), dtype=torch.uint8, device=dev)
    P.puzzle_decode_attn_workspace_init(desc, w.batch, ws)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    stream = torch.cuda.current_stream()

    attn_events = []   # CUDA-event pairs around the attention launch of every 8th timed step

    def step(i, sample=False):
        v = views[i % len(views)]
        P.puzzle_kv_append(desc, v, k_new, v_new, dev_status=status, stream=stream)
        if sample:
            ea, eb = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            ea.record(stream)
        decode(desc, v, q, sinks, out, None, num_splits=args.splits, workspace=ws,
                             dev_status=status, stream=stream)
        if sample:
            eb.record(stream)
            attn_events.append((ea, eb))

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for i in range(max(args.warmup, 3)):
        step(i)
    barrier()

    # ---- timed region: device-resident inputs
    sampler = ClockSampler(physical_gpu_index(local_rank))
    sampler.start()
    time.sleep(0.25)
    launches0 = P.puzzle_launch_count()
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    t0.record(stream)
    for i in range(args.steps):
        step(i, sample=(i % 8 == 7))
    t1.record(stream)
    barrier()
    launches = P.puzzle_launch_count() - launches0
    ms_total = t0.elapsed_time(t1)
    attn_in_region_ms = [a.elapsed_time(b) for a, b in attn_events]
    # the attention kernel alone: the same launches back to back on the same stream, no append in between
    n_attn = min(args.steps, 400)
    a0, a1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a0.record(stream)
    for i in range(n_attn):
        decode(desc, views[i % len(views)], q, sinks, out, None, num_splits=args.splits, workspace=ws,
                             dev_status=status, stream=stream)
    a1.record(stream)
    barrier()
    attn_ms = [a0.elapsed_time(a1) / n_attn]
    clocks = sampler.stop()

    # ---- end to end: the step's inputs start in pinned host memory, the result ends there
    # q, k_new and v_new of a step travel as ONE pinned host buffer and one copy (the caller's side of the API:
    # the entry points take three pointers, which may point into one allocation)
    parts = (q, k_new, v_new)
    sizes = [t.numel() for t in parts]
    hin = torch.cat([t.reshape(-1).cpu() for t in parts]).pin_memory()
    din = torch.empty(sum(sizes), dtype=q.dtype, device=dev)
    dq, dk, dv = (din[sum(sizes[:k]):sum(sizes[:k + 1])].view(parts[k].shape) for k in range(3))
    hout = torch.empty(out.shape, dtype=out.dtype).pin_memory()

    def step_e2e(i):
        v = views[i % len(views)]
        din.copy_(hin, non_blocking=True)
        P.puzzle_kv_append(desc, v, dk, dv, dev_status=status, stream=stream)
        decode(desc, v, dq, sinks, out, None, num_splits=args.splits, workspace=ws,
                             dev_status=status, stream=stream)
        hout.copy_(out, non_blocking=True)

    for i in range(3):
        step_e2e(i)
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for i in range(args.steps):
        step_e2e(i)
        stream.synchronize()   # the caller reads the result on the host before the next step
    e1.record(stream)
    barrier()
    ms_e2e = e0.elapsed_time(e1)

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

    dev_flags = int(status.item())
    bytes_step = algorithmic_bytes(w, seq_lens_host, window)
    kv_bytes_attn = bytes_step - 2 * w.batch * w.hkv * w.head_dim * 3   # what the attention pass itself moves
    # roofline: mean duration of the attention launches sampled INSIDE the timed region (falls back to the
    # back-to-back loop when the run is too short to hold a sample)
    b2b_ms = statistics.mean(attn_ms)
    in_region_ms = statistics.mean(attn_in_region_ms) if attn_in_region_ms else b2b_ms
    ms_total, ms_e2e, attn_mean_ms, b2b_ms = max_over_ranks([ms_total, ms_e2e, in_region_ms, b2b_ms], world, dev)

    if rank == 0:
        peak, peak_kind = measured_peak()
        ms_step = ms_total / args.steps
        value = job_throughput_gbs(bytes_step, world, ms_step)
        achieved = kv_bytes_attn / (attn_mean_ms * 1e-3) / 1e9
        line = {
            "metric": METRIC, "value": round(value, 1), "unit": "GB/s", "n_gpus": world, "steps": args.steps,
            "warmup": max(args.warmup, 3), "ms_per_step": round(ms_step, 5),
            "us_per_layer_step": round(ms_step * 1e3, 2), "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": dtype_name, "data": "synthetic",
            "config": {"workload": w.name, "batch_per_gpu": w.batch, "context": w.context, "q_heads": w.hq,
                       "kv_heads": w.hkv, "head_dim": w.head_dim, "block_size": w.block, "window": window, "paged": not args.contiguous,
                       "num_splits": args.splits, "rotating_layer_caches": len(layers),
                       "l2": "inputs larger than L2: %.0f MiB per step, %d caches rotated" % (
                           bytes_step / 2 ** 20, len(layers)),
                       "parallelism": "dp%d (independent sequences per GPU, no collective)" % world},
            "clocks": clocks,
            "e2e": {"value": round(world * bytes_step / (ms_e2e / args.steps * 1e-3) / 1e9, 1), "unit": "GB/s",
                    "ms_per_step": round(ms_e2e / args.steps, 5),
                    "h2d_bytes_per_step": int(sum(t.numel() * t.element_size() for t in (q, k_new, v_new))),
                    "d2h_bytes_per_step": int(out.numel() * out.element_size())},
            "gpu_launches": int(launches),
            "roofline": {"bound": "hbm", "kernel": kernel_name,
                         "achieved": round(achieved, 1), "peak": peak, "peak_kind": peak_kind + " copy bandwidth",
                         "unit": "GB/s", "frac": round(achieved / peak, 4),
                         "frac_of_nominal_8TBs": round(achieved / NOMINAL_HBM_GBS, 4),
                         "us_per_launch": round(attn_mean_ms * 1e3, 2), "launches_sampled": len(attn_in_region_ms),
                         "us_per_launch_back_to_back": round(b2b_ms * 1e3, 2),
                         "us_per_launch_median": round(statistics.median(attn_in_region_ms or [b2b_ms]) * 1e3, 2),
                         "us_per_launch_min": round(min(attn_in_region_ms or [b2b_ms]) * 1e3, 2),
                         "bytes_per_launch": int(kv_bytes_attn),
                         "read_probe_gbs": round(probe_gbs, 1),
                         "traffic": ncu_traffic(args)},
            "dev_status": dev_flags,
        }
        if args.cpu_baseline:
            line["cpu_baseline"] = cpu_baseline(w, layers[0], seq_lens_host, q, sinks, window)
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


# DRAM bytes per launch (dram__bytes_read.sum + dram__bytes_write.sum) of the default split-KV kernel on the
# headline workload, from the one-launch `ncu --set full` capture summarised under profiles/; valid only for
# the kernel sources it was taken from, so it is tied to their hash and reported as null once they change.
NCU_CAPTURE = {
    "workload": 3, "kernel": "mma", "splits": 0,
    "sources": ("decode_attn.cu", "decode_sched.cuh", "common.cuh", "decode_attn.cuh"),
    "sha256": "b761b1d7f16384a72e8e4be46a8eb5f45977dbdbd6f9aa513875ae08bfdf039e",
    "dram_bytes_per_launch": 1075472000 + 4413440,
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

    for _ in range(min(args.warmup, 1)):
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
        "n_gpus": int(os.environ.get("WORLD_SIZE", "1")), "steps": args.steps, "warmup": min(args.warmup, 1),
        "ms_per_step": round(dt * 1e3, 3), "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f64 (CPU oracle over fp8_e4m3 KV)", "data": "synthetic",
        "config": {"workload": synth.workload(args.config).name, "sample": sample},
        "cpu_baseline": {"value": value, "unit": "GB/s", "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=2000)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", type=int, default=3, help="workload id 1..5 (3 = batch 16, context 64K)")
    ap.add_argument("--splits", type=int, default=0, help="0 = balanced schedule, S = fixed splits per sequence")
    ap.add_argument("--layers", type=int, default=4, help="distinct layer caches rotated between steps")
    ap.add_argument("--stack", type=int, default=0, choices=[0, 4, 5],
                    help="instead of the headline run: one step of the 36-layer stack of workload 4 or 5")
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
    if args.stack:
        run_stack(args)
    elif args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()

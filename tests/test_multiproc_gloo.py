"""The N > 1 path of the bench on CPU: two gloo ranks, no GPU.

The hot path shards over independent sequences (no data-path collective), so what the ranks share is only
host logic: which sequences a rank draws, the max-over-ranks step time and the whole-job aggregate.
"""
import os
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _rank(rank, world, port, ret):
    sys.path.insert(0, ROOT)
    import bench
    import synth
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        w = bench.shard_workload(synth.workload(4, scale=0.05), rank, world)
        lens = synth.draw_seq_lens(w)
        q = synth.draw_q(w)
        gathered = [torch.zeros_like(lens) for _ in range(world)]
        dist.all_gather(gathered, lens)
        qsum = [torch.zeros(1) for _ in range(world)]
        dist.all_gather(qsum, q.float().sum().reshape(1))
        ms = bench.max_over_ranks([10.0 + rank, 5.0 - rank], world, "cpu")
        nbytes = bench.algorithmic_bytes(w, lens.tolist(), 0)
        total = torch.tensor([float(nbytes)], dtype=torch.float64)
        dist.all_reduce(total)
        ret[rank] = dict(lens=[g.tolist() for g in gathered], qsum=[float(x) for x in qsum], ms=ms,
                         value=bench.job_throughput_gbs(nbytes, world, ms[0]), nbytes=nbytes, total=float(total))
    finally:
        dist.destroy_process_group()


def test_two_ranks_draw_own_sequences_and_agree_on_the_slowest_time():
    world = 2
    port = 29500 + os.getpid() % 2000
    with mp.Manager() as m:
        ret = m.dict()
        mp.spawn(_rank, args=(world, port, ret), nprocs=world, join=True)
        r0, r1 = ret[0], ret[1]
    assert r0["lens"] == r1["lens"]                       # both saw the same gathered picture
    assert r0["lens"][0] != r0["lens"][1]                 # but each rank drew sequences of its own
    assert r0["qsum"][0] != r0["qsum"][1]
    assert r0["ms"] == r1["ms"] == [11.0, 5.0]            # element-wise max over ranks
    # per-rank shape is fixed (weak scaling): the job value counts both ranks' bytes over the slowest time
    assert abs(r0["value"] - 2 * r0["nbytes"] / 11e-3 / 1e9) < 1e-9


def test_single_rank_is_the_identity():
    sys.path.insert(0, ROOT)
    import bench
    import synth
    w = synth.workload(3)
    assert bench.shard_workload(w, 0, 1).seed == synth.workload(3).seed
    assert bench.max_over_ranks([1.5, 2.5], 1, "cpu") == [1.5, 2.5]


def _shard_rank(rank, world, port, ret):
    sys.path.insert(0, ROOT)
    import bench
    import synth
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        w = synth.workload(5, scale=0.01)                    # batch 1 -> sc() floors at 1; context 1311
        w.batch = 3
        lens = torch.tensor([1311, 17, 640], dtype=torch.int32)
        out = {}
        for mode in ("heads", "context"):
            ws, la, lp, nbytes = bench.shard_plan(w, lens, rank, world, mode)
            total = bench.sum_over_ranks(float(nbytes), world, "cpu")
            held = torch.zeros(world, 3, dtype=torch.int64)
            held[rank] = la.to(torch.int64)
            dist.all_reduce(held)
            owners = torch.zeros(3, dtype=torch.int64)
            owners += (lp > 0).to(torch.int64)
            dist.all_reduce(owners)
            out[mode] = dict(hkv=ws.hkv, hq=ws.hq, blocks=ws.blocks_per_seq, held=held.tolist(), owners=owners.tolist(),
                             nbytes=nbytes, total=total)
        ret[rank] = out
    finally:
        dist.destroy_process_group()


def test_two_ranks_share_one_layer_by_heads_and_by_context():
    """Host logic of `bench.py --shard heads|context` at world size 2: what a rank holds, who appends, and that the
    ranks' bytes add up to the job's."""
    sys.path.insert(0, ROOT)
    import bench
    import synth
    world = 2
    port = 31500 + os.getpid() % 2000
    with mp.Manager() as m:
        ret = m.dict()
        mp.spawn(_shard_rank, args=(world, port, ret), nprocs=world, join=True)
        r0, r1 = ret[0], ret[1]
    w = synth.workload(5, scale=0.01)
    w.batch = 3
    lens = [1311, 17, 640]
    # KV heads: half the heads each, every token; the two halves move the whole layer's K/V bytes (q/out and the
    # block-table entries are per rank)
    for r in (r0, r1):
        assert r["heads"]["hkv"] == 4 and r["heads"]["hq"] == 32
        assert r["heads"]["held"] == [lens, lens] and r["heads"]["owners"] == [2, 2, 2]
    whole = bench.algorithmic_bytes(w, lens, 0)
    table = sum(((L + 15) // 16) * 4 for L in lens)
    assert r0["heads"]["total"] == r1["heads"]["total"] == whole + table
    # context: blocks dealt round robin, every token on exactly one rank, exactly one rank appends each sequence
    held = r0["context"]["held"]
    assert [held[0][i] + held[1][i] for i in range(3)] == lens
    assert held == r1["context"]["held"] and r0["context"]["owners"] == [1, 1, 1]
    assert r0["context"]["blocks"] == (w.blocks_per_seq + 1) // 2
    kv_bytes = sum(lens) * 2 * w.hkv * w.head_dim
    assert r0["context"]["total"] >= kv_bytes and r0["context"]["total"] - kv_bytes < 0.2 * kv_bytes + 3e5


def test_launch_plan_never_reports_fewer_gpus_than_asked():
    sys.path.insert(0, ROOT)
    import bench
    import pytest
    assert bench.launch_plan(1, {}) == ("single",)
    assert bench.launch_plan(4, {}) == ("spawn", 4)
    assert bench.launch_plan(2, {"WORLD_SIZE": "2", "RANK": "1", "LOCAL_RANK": "1"}) == ("rank", 1, 1, 2)
    with pytest.raises(SystemExit):
        bench.launch_plan(8, {"WORLD_SIZE": "2", "RANK": "0"})
    with pytest.raises(SystemExit):
        bench.launch_plan(0, {})


def test_bench_starts_its_own_ranks():
    """`bench.py --gpus 2` without a launcher starts two ranks itself (here on the reference arm, which needs no
    GPU: rank 0 prints the line, rank 1 leaves)."""
    import json
    import subprocess
    env = {k: v for k, v in os.environ.items() if k not in ("WORLD_SIZE", "RANK", "LOCAL_RANK", "MASTER_ADDR", "MASTER_PORT")}
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2", "--steps", "1",
                        "--warmup", "0"], capture_output=True, text=True, timeout=900, cwd=ROOT, env=env)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [l for l in r.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1
    assert json.loads(lines[0])["n_gpus"] == 2

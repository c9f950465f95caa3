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

"""CPU tests of the multi-GPU host logic: the index arithmetic of context and head sharding, and, on two gloo
ranks, that per-rank partials without sink + one all-gather + one merge with the sink reproduce full attention
(all arithmetic here is the oracle's: what is under test is the sharding and the exchanged layout)."""
import os
import sys

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_context_slice_against_enumeration():
    from paper_2602_11937_b200.parallel import context_slice
    from parallel_helpers import brute_force_slice
    lens = torch.arange(0, 150, dtype=torch.int32)
    for world in (1, 2, 3, 4, 8):
        total = torch.zeros_like(lens)
        owners = torch.zeros_like(lens)
        for rank in range(world):
            local, app = context_slice(lens, rank, world)
            assert local.dtype == torch.int32 and app.dtype == torch.int32
            for L in range(150):
                n, owns = brute_force_slice(L, rank, world)
                assert int(local[L]) == n, (world, rank, L)
                assert int(app[L]) == (n if owns else 0), (world, rank, L)
            total += local
            owners += (app > 0).int()
        assert torch.equal(total, lens)                          # every token on exactly one rank
        assert torch.equal(owners, (lens > 0).int())             # the newest token has exactly one owner


def test_head_slice():
    from paper_2602_11937_b200.parallel import head_slice
    kv, q = head_slice(3, 4)
    assert (kv.start, kv.stop, q.start, q.stop) == (6, 8, 48, 64)
    assert head_slice(0, 1) == (slice(0, 8), slice(0, 64))
    with pytest.raises(ValueError):
        head_slice(0, 3)


def _rank(rank, world, port, ret):
    sys.path.insert(0, ROOT)
    sys.path.insert(0, os.path.join(ROOT, "tests"))
    import oracle
    import synth
    from helpers import make_case, oracle_append, oracle_attn
    from parallel_helpers import local_table
    from paper_2602_11937_b200.parallel import context_slice
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        w = synth.Workload("ctxshard", 1, 5, 400, [0], paged=True)
        case = make_case(w, seq_lens=[400, 0, 1, 17, 333])       # the same seeded case on every rank
        lens = torch.from_numpy(case["seq_lens"])
        local, app = context_slice(lens, rank, world)
        tab = local_table(case, rank, world)
        # this rank appends only the new tokens it owns, into its own blocks
        shard = dict(case, table=tab, seq_lens=app.numpy(), k_cache=case["k_cache"].copy(), v_cache=case["v_cache"].copy())
        shard["w"] = synth.Workload("ctxshard_local", 1, 5, tab.shape[1] * 16, [0], paged=True)
        oracle_append(shard)
        changed = int((shard["k_cache"] != case["k_cache"]).any(axis=(1, 2, 3)).sum())
        # its partial: attention over its keys only, no sink
        shard["seq_lens"] = local.numpy()
        o, lse = oracle_attn(shard, 0, sinks=None)
        rows, d = w.batch * w.hq, w.head_dim
        mine = torch.from_numpy(np.concatenate([o.reshape(-1), lse.reshape(-1)]))
        gathered = [torch.zeros_like(mine) for _ in range(world)]
        dist.all_gather(gathered, mine)                           # the path's one exchange
        g = torch.stack(gathered).numpy()
        part_o = g[:, :rows * d].reshape(world, rows, d).transpose(1, 0, 2)
        part_lse = g[:, rows * d:].reshape(world, rows).T
        merged, mlse = oracle.attn_merge(part_o, part_lse, sink=np.tile(case["sinks"], w.batch))
        # the unsharded reference: global append, then full attention with the sink
        oracle_append(case)
        ref, ref_lse = oracle_attn(case, 0)
        ret[rank] = dict(err=float(np.abs(merged.reshape(ref.shape) - ref).max()),
                         lse_err=float(np.abs(mlse.reshape(ref_lse.shape) - ref_lse).max()),
                         changed_blocks=changed, local=local.tolist())
    finally:
        dist.destroy_process_group()


@pytest.mark.parametrize("world", [2, 3])
def test_gloo_ranks_partials_allgather_merge_equals_full_attention(world):
    port = 31500 + os.getpid() % 2000 + world
    with mp.Manager() as m:
        ret = m.dict()
        mp.spawn(_rank, args=(world, port, ret), nprocs=world, join=True)
        res = [ret[r] for r in range(world)]
    for r in res:
        assert r["err"] < 1e-12 and r["lse_err"] < 1e-12
    assert sum(r["changed_blocks"] for r in res) == 4            # one block per non-empty sequence, each on one rank
    assert [sum(x) for x in zip(*[r["local"] for r in res])] == [400, 0, 1, 17, 333]

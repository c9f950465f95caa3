"""Test-side construction of the shards a multi-GPU run would hold (numpy only)."""
import numpy as np


def global_table(case):
    w = case["w"]
    if case["table"] is not None:
        return case["table"]
    return (np.arange(w.batch, dtype=np.int32)[:, None] * w.blocks_per_seq +
            np.arange(w.blocks_per_seq, dtype=np.int32)[None, :]).astype(np.int32)


def local_table(case, rank, world):
    """Block table of ``rank`` under round-robin context sharding: local block i = global block rank + i * world.
    Missing entries are -1 (never read: they lie beyond every local length)."""
    t = global_table(case)
    nloc = (t.shape[1] + world - 1) // world
    out = np.full((t.shape[0], nloc), -1, dtype=np.int32)
    mine = t[:, rank::world]
    out[:, :mine.shape[1]] = mine
    return out


def brute_force_slice(L, rank, world, block=16):
    """(tokens of a length-L sequence that rank holds, does rank hold token L - 1)."""
    n = sum(1 for p in range(L) if (p // block) % world == rank)
    return n, (L > 0 and ((L - 1) // block) % world == rank)

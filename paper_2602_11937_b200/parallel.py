"""Sharding of the decode-attention path over several GPUs (one process per GPU, torch.distributed).

Three ways, the first two without any exchange inside the path:

* batch: sequences are independent; every rank runs the whole path on its sequences (what ``bench.py --gpus N``
  does);
* KV heads (tensor parallelism, the degree the paper sweeps from 1 to 8 in its serving benchmarks, paragraph
  "Inference efficiency benchmarking"): a rank holds ``Hkv / world`` KV heads of every layer's cache and their
  query heads, and calls the ordinary entry points with a smaller ``num_kv_heads``; ``head_slice`` gives the
  ranges;
* context: for one long sequence batch, a rank holds every ``world``-th 16-token block of each sequence's
  cache.  Each rank computes a float32 partial over its keys (``puzzle_decode_attn_partial``), ONE all-gather
  moves ``batch * Hq * (D + 1)`` floats per rank, and every rank merges the partials with the sink applied once
  (``puzzle_attn_merge_strided``).  The paper does not describe this; it follows from the KV-I/O bound of
  long-context decode (Section "Optimized Scenarios"): the cache bytes a GPU streams per step drop by ``world``.

Only index arithmetic, buffers and the collective live here; every numeric step is a kernel of the library.
"""
from __future__ import annotations

from typing import Optional, Tuple

import torch

from . import binding as B


def head_slice(rank: int, world: int, num_kv_heads: int = 8, group: int = 8) -> Tuple[slice, slice]:
    """KV heads and query heads of ``rank`` under tensor parallelism of degree ``world``."""
    if num_kv_heads % world:
        raise ValueError("the tensor-parallel degree must divide the number of KV heads")
    per = num_kv_heads // world
    return slice(rank * per, (rank + 1) * per), slice(rank * per * group, (rank + 1) * per * group)


def context_slice(seq_lens: torch.Tensor, rank: int, world: int, block: int = 16) -> Tuple[torch.Tensor, torch.Tensor]:
    """Round-robin context sharding by cache block: global block j of a sequence lives on rank ``j % world`` as
    that rank's local block ``j // world``.  For global lengths ``seq_lens`` (counted after this step's append)
    returns, as int32 tensors on the same device,

    * ``local_lens``: tokens of each sequence that ``rank`` holds (its ``seq_lens`` for attention), and
    * ``append_lens``: ``local_lens`` where ``rank`` owns the block of the newest token, else 0 (its ``seq_lens``
      for ``puzzle_kv_append``, which skips sequences of length 0): the new token is always the last token of its
      owner's slice.
    """
    L = seq_lens.to(torch.int64)
    full, tail = L // block, L % block
    local = block * torch.div(full + (world - 1 - rank), world, rounding_mode="floor")
    local = local + torch.where((tail > 0) & (full % world == rank), tail, torch.zeros_like(tail))
    owner = torch.div(torch.clamp(L - 1, min=0), block, rounding_mode="floor") % world
    append = torch.where((owner == rank) & (L > 0), local, torch.zeros_like(local))
    return local.to(torch.int32), append.to(torch.int32)


class ContextShardedAttention:
    """One full-attention layer whose context is sharded over the ranks of ``group`` (see ``context_slice``).

    ``step`` = partial on this rank's slice, all-gather, merge; the result is identical on every rank.  A window
    layer is not sharded this way (its window counts back from the end of the sequence, which a slice cannot
    express for ragged batches); keep window layers on one rank or replicate their few blocks.
    """

    def __init__(self, desc: B.LayerDesc, batch: int, device, world: int, group=None, num_splits: int = 0):
        if desc.window != 0:
            raise ValueError("context sharding covers full-attention layers only")
        self.desc, self.batch, self.world, self.group, self.num_splits = desc, batch, world, group, num_splits
        hq, d = desc.num_q_heads, desc.head_dim
        self.rows, self.d = batch * hq, d
        self.per_rank = self.rows * (d + 1)                      # o [batch][Hq][D] then lse [batch][Hq]
        self.mine = torch.zeros(self.per_rank, dtype=torch.float32, device=device)
        self.gathered = torch.zeros(world, self.per_rank, dtype=torch.float32, device=device)
        self.workspace = torch.zeros(B.puzzle_decode_attn_workspace_bytes(desc, batch, num_splits), dtype=torch.uint8,
                                     device=device)
        B.puzzle_decode_attn_workspace_init(desc, batch, self.workspace)
        self.status = torch.zeros(1, dtype=torch.int32, device=device)

    def partial(self, view: B.KVView, q: torch.Tensor, into: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
        """This rank's partial buffer (float32 [rows * (D + 1)]); ``into`` may name a row of ``gathered``."""
        buf = self.mine if into is None else into
        o = buf[: self.rows * self.d].view(self.batch, self.desc.num_q_heads, self.d)
        lse = buf[self.rows * self.d:].view(self.batch, self.desc.num_q_heads)
        B.puzzle_decode_attn_partial(self.desc, view, q, o, lse, num_splits=self.num_splits, workspace=self.workspace,
                                     dev_status=self.status, stream=stream)
        return buf

    def merge(self, sinks: Optional[torch.Tensor], out: torch.Tensor, lse_out: Optional[torch.Tensor] = None,
              stream=None) -> None:
        """Merge of the ``world`` partial buffers in ``gathered`` with the sink applied once."""
        flat = self.gathered.view(-1)
        B.puzzle_attn_merge_strided(flat, flat[self.rows * self.d:], self.d, self.per_rank, 1, self.per_rank, None,
                                    sinks, out, self.world, lse_out=lse_out, stream=stream)

    def step(self, view: B.KVView, q: torch.Tensor, sinks: Optional[torch.Tensor], out: torch.Tensor,
             lse_out: Optional[torch.Tensor] = None) -> None:
        import torch.distributed as dist
        if self.world == 1:
            self.partial(view, q, into=self.gathered[0])
        else:
            self.partial(view, q)
            dist.all_gather_into_tensor(self.gathered, self.mine, group=self.group)   # the path's one exchange
        self.merge(sinks, out, lse_out)

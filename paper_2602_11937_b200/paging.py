"""Block tables for the paged KV cache (host-side index arithmetic only).

A window layer attends to the W most recent tokens, so it never needs more than ``ceil(W / 16) + 1`` blocks of a
sequence at a time: that is where the paper's KV-cache saving comes from (window layers keep a bounded cache,
Section "Window attention for long-context inference"; a 40 % smaller KV cache in the 64K scenario, Section
"Optimized Scenarios").  The kernels read a block only through the table and never look at entries wholly
before the window, so the saving needs no kernel support: a window layer's table maps logical block ``j`` of a
sequence onto a ring of ``R`` physical blocks, ``j % R``.  The append of token ``L - 1`` then overwrites the
block that left the window ``R`` blocks ago.
"""
from __future__ import annotations

import torch

BLOCK = 16


def window_ring_blocks(window: int, block: int = BLOCK) -> int:
    """Physical blocks per sequence that a layer with this window needs (window >= 1)."""
    if window < 1:
        raise ValueError("a full-attention layer keeps every block")
    return (window + block - 1) // block + 1


def ring_block_table(batch: int, window: int, max_blocks_per_seq: int, first_block: int = 0, block: int = BLOCK,
                     device="cpu") -> torch.Tensor:
    """int32 [batch][max_blocks_per_seq] table of a window layer whose sequence b owns the physical blocks
    ``first_block + b * R .. + R - 1``, R = window_ring_blocks(window): logical block j -> ring slot j % R."""
    r = window_ring_blocks(window, block)
    j = torch.arange(max_blocks_per_seq, dtype=torch.int64, device=device)[None, :] % r
    b = torch.arange(batch, dtype=torch.int64, device=device)[:, None] * r
    return (first_block + b + j).to(torch.int32)


def linear_block_table(batch: int, max_blocks_per_seq: int, first_block: int = 0, device="cpu") -> torch.Tensor:
    """The table of a full-attention layer with one private run of blocks per sequence."""
    j = torch.arange(max_blocks_per_seq, dtype=torch.int64, device=device)[None, :]
    b = torch.arange(batch, dtype=torch.int64, device=device)[:, None] * max_blocks_per_seq
    return (first_block + b + j).to(torch.int32)


def cache_blocks(windows, batch: int, max_blocks_per_seq: int) -> list:
    """Physical blocks each layer of a stack needs: all of them for full layers (window 0), a ring for the rest."""
    return [batch * (max_blocks_per_seq if w == 0 else min(max_blocks_per_seq, window_ring_blocks(w))) for w in windows]


def multi_token_args(seq_lens: torch.Tensor, block_table, n_q: int, max_blocks_per_seq: int = None, q_lens=None):
    """Arguments that make the decode kernels serve ``n_q`` query tokens per sequence with a causal mask (several
    tokens of a multi-token step, or a prompt chunk after its bulk append): query row i of sequence b sits at position
    ``seq_lens[b] - q_lens[b] + i`` and sees the keys up to and including itself, i.e. it is a decode step of a
    sequence of length ``seq_lens[b] - q_lens[b] + i + 1`` over the same blocks (a window layer then counts back from
    that position).  Returns ``(lens, table)`` for a batch of ``batch * n_q`` rows: int32 ``[batch * n_q]`` and int32
    ``[batch * n_q][max_blocks_per_seq]`` (each table row repeated ``n_q`` times).  Rows ``i >= q_lens[b]`` are
    padding and get length 0 (output 0).  Pass q as ``[batch * n_q][Hq][D]``.

    The n_q rows of a sequence read the same cache blocks at about the same time (they are neighbours in the
    balanced schedule), so the repeats are served by L2 rather than HBM.  For FP8 caches
    ``puzzle_decode_attn_tokens`` does the same job faster (pairs of query tokens share one pass over the tiles);
    this form remains for bf16 caches and as a second way to the same result."""
    batch = seq_lens.shape[0]
    dev = seq_lens.device
    L = seq_lens.to(torch.int64)[:, None]
    ql = torch.full((batch, 1), n_q, dtype=torch.int64, device=dev) if q_lens is None else \
        torch.clamp(q_lens.to(torch.int64), 0, n_q)[:, None]
    i = torch.arange(n_q, dtype=torch.int64, device=dev)[None, :]
    lens = torch.where(i < ql, torch.clamp(L - ql + i + 1, min=0), torch.zeros_like(i))
    if block_table is None:
        if max_blocks_per_seq is None:
            raise ValueError("max_blocks_per_seq is required without a block table")
        block_table = linear_block_table(batch, max_blocks_per_seq, device=dev)
    table = block_table.repeat_interleave(n_q, dim=0).contiguous()
    return lens.reshape(-1).to(torch.int32).contiguous(), table

"""Per-layer pattern driver: one decode step of the attention stack of a model whose layers are each
full-context or sliding-window (the per-layer choice the paper's architecture search makes, Section
"Window attention for long-context inference").

A ``DecodeStack`` only loops over the C-ABI calls (fused quantise-and-append, then attention, per layer);
every step of the path is a kernel of the library.  ``capture()`` records one step into a CUDA graph so a
36-layer step is one launch from the host's point of view.
"""
from __future__ import annotations

from typing import List, Optional, Sequence

import torch

from . import binding as B


class DecodeStack:
    def __init__(self, windows: Sequence[int], k_caches: Sequence[torch.Tensor], v_caches: Sequence[torch.Tensor],
                 seq_lens: torch.Tensor, block_tables: Sequence[Optional[torch.Tensor]], max_blocks_per_seq: int,
                 k_scales: Sequence[Optional[torch.Tensor]], v_scales: Sequence[Optional[torch.Tensor]],
                 sinks: Sequence[Optional[torch.Tensor]], kv_dtype: int = B.KV_FP8_E4M3, num_splits: int = 0):
        n = len(windows)
        assert all(len(x) == n for x in (k_caches, v_caches, block_tables, k_scales, v_scales, sinks))
        self.windows = list(windows)
        self.batch = int(seq_lens.shape[0])
        self.num_splits = num_splits
        self.sinks = list(sinks)
        self._keep = (k_caches, v_caches, seq_lens, block_tables, k_scales, v_scales)  # the views hold raw pointers
        self.descs = [B.layer_desc(window=w, kv_dtype=kv_dtype) for w in windows]
        self.views = [B.kv_view(k_caches[i], v_caches[i], seq_lens, block_table=block_tables[i],
                                max_blocks_per_seq=max_blocks_per_seq, k_scale=k_scales[i], v_scale=v_scales[i])
                      for i in range(n)]
        dev = seq_lens.device
        nbytes = max(B.puzzle_decode_attn_workspace_bytes(d, self.batch, num_splits) for d in self.descs)
        self.workspace = torch.zeros(nbytes, dtype=torch.uint8, device=dev)
        B.puzzle_decode_attn_workspace_init(self.descs[0], self.batch, self.workspace)
        self.status = torch.zeros(1, dtype=torch.int32, device=dev)
        self.graph = None

    def step(self, q: List[torch.Tensor], k_new: List[torch.Tensor], v_new: List[torch.Tensor],
             out: List[torch.Tensor], stream=None) -> None:
        """Append + attention for every layer, in order, on ``stream`` (all layers share one workspace, so
        their kernels run one after the other on that stream)."""
        for i in range(len(self.windows)):
            B.puzzle_kv_append(self.descs[i], self.views[i], k_new[i], v_new[i], dev_status=self.status, stream=stream)
            B.puzzle_decode_attn(self.descs[i], self.views[i], q[i], self.sinks[i], out[i], None,
                                 num_splits=self.num_splits, workspace=self.workspace, dev_status=self.status,
                                 stream=stream)

    def capture(self, q, k_new, v_new, out) -> "torch.cuda.CUDAGraph":
        """Records one step (with these argument tensors) into a CUDA graph; replay with ``graph.replay()``."""
        self.step(q, k_new, v_new, out)            # warm-up outside capture (first launches set attributes)
        torch.cuda.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g):
            self.step(q, k_new, v_new, out, stream=torch.cuda.current_stream())
        self.graph = g
        return g

"""Bulk layer caches for full-size runs, filled on the device.

Full-size workloads hold gigabytes of K/V per layer, too much to push through the CPU oracle's codec.
Here the samples of ``synth.draw_kv_samples`` are turned into cache bytes with PyTorch's own float8 / bf16
casts.  This is input preparation: whatever bytes come out ARE the cache, and both the CUDA path and the
CPU oracle then read those same bytes (the oracle from a host copy), so nothing under test depends on how
they were made.  Scales are amax/448 of the drawn samples per KV head.
"""
from __future__ import annotations

import torch

from . import Workload, draw_block_table, draw_kv_samples

KV_FP8_E4M3 = 0
KV_BF16 = 1


def fill_layer(w: Workload, layer: int, dev: str, kv_dtype: int = KV_FP8_E4M3, with_table: bool = True,
               step: int = 8192):
    """dict(k_cache, v_cache, k_scale, v_scale, table) for one layer of workload ``w`` on device ``dev``.

    Caches are [num_blocks][Hkv][16][D] uint8 codes (or bf16), num_blocks = batch * blocks_per_seq;
    scales are float32 [Hkv] (None for bf16); table is the workload's seeded block table (or None)."""
    nb = w.batch * w.blocks_per_seq
    out = {}
    for which in ("k", "v"):
        if kv_dtype == KV_BF16:
            cache = torch.empty(nb, w.hkv, w.block, w.head_dim, dtype=torch.bfloat16, device=dev)
            for lo in range(0, nb, step):
                x = draw_kv_samples(w, which, nb, layer, dev, lo, min(nb, lo + step))
                cache[lo:lo + x.shape[0]] = x.to(torch.bfloat16)
            out[which + "_cache"], out[which + "_scale"] = cache, None
            continue
        cache = torch.empty(nb, w.hkv, w.block, w.head_dim, dtype=torch.uint8, device=dev)
        amax = torch.zeros(w.hkv, device=dev)
        for lo in range(0, nb, step):      # pass 1: amax per KV head
            x = draw_kv_samples(w, which, nb, layer, dev, lo, min(nb, lo + step))
            amax = torch.maximum(amax, x.abs().amax(dim=(0, 2, 3)))
        scale = (amax / 448.0).float()
        scale = torch.where(scale > 0, scale, torch.ones_like(scale))
        for lo in range(0, nb, step):      # pass 2: the same draws, cast
            x = draw_kv_samples(w, which, nb, layer, dev, lo, min(nb, lo + step))
            cache[lo:lo + x.shape[0]] = (x / scale[None, :, None, None]).to(torch.float8_e4m3fn).view(torch.uint8)
        out[which + "_cache"], out[which + "_scale"] = cache, scale
    out["table"] = draw_block_table(w, layer, nb, dev) if with_table else None
    return out

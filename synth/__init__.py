"""Seeded synthetic inputs shaped like the serving scenarios the path targets.

This module only draws numbers and lays out block tables.  It holds none of
the method's arithmetic (no quantisation, no attention, no scale rule), so the
CPU oracle's tests and the CUDA path's tests can both draw their inputs here
without sharing anything else.  (``synth.device`` is the one exception, and it
says so: to fill gigabyte caches for full-size runs it casts drawn samples with
PyTorch's own float8 type after dividing by amax/448; that prepares inputs,
and both sides then read the resulting bytes.)

The five workloads follow the decode-heavy serving scenarios (fixed-length
prompts and generations such as 4K/4K and 64K/64K; a gpt-oss-style stack of 36
layers that alternates 128-token sliding-window and full-context attention,
with 64 query heads, 8 KV heads and head size 64).  Every tensor gets its own
sub-stream of one seed per workload, so tensors do not shift when another one
changes size.
"""
from __future__ import annotations

import dataclasses
from typing import List, Optional, Sequence

import torch

HQ = 64
HKV = 8
HEAD_DIM = 64
BLOCK = 16
NUM_LAYERS = 36
SEED_BASE = 0x5EED0000

# sub-stream ids
S_Q, S_K, S_V, S_SINK, S_KFACT, S_VFACT, S_TABLE, S_LENS, S_KNEW, S_VNEW = range(10)


def _gen(seed: int, stream: int, layer: int = 0, device: str = "cpu") -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed((seed * 1000003 + stream * 7919 + layer * 104729) & 0x7FFFFFFFFFFFFFFF)
    return g


@dataclasses.dataclass
class Workload:
    """One decode step's shape: what is cached, how it is paged, which layers."""

    name: str
    config_id: int
    batch: int
    context: int                      # tokens per sequence after the append (max if ragged)
    windows: List[int]                # one entry per layer: 0 = full, W > 0 = sliding window
    paged: bool                       # False: contiguous cache, no block table
    ragged_lo: Optional[int] = None   # ragged contexts uniform in [ragged_lo, context]
    kv_factor_range: Optional[Sequence[float]] = None  # per-head spread of K/V magnitudes
    calib_prefix: Optional[int] = None  # scales from the first n tokens only
    hq: int = HQ
    hkv: int = HKV
    head_dim: int = HEAD_DIM
    block: int = BLOCK

    @property
    def seed(self) -> int:
        return SEED_BASE + self.config_id

    @property
    def blocks_per_seq(self) -> int:
        return (self.context + self.block - 1) // self.block


def layer_pattern(kind: str, num_layers: int = NUM_LAYERS) -> List[int]:
    """Per-layer window sizes (0 = full context).

    parent:    alternating 128-token window / full, as the parent model has.
    every4th:  only every fourth layer keeps full context, the rest window 128.
    selective: the parent with 8 of its 18 full layers turned into 8192-token
               windows (which eight is not published; they are spread evenly).
    """
    if kind == "parent":
        return [128 if i % 2 == 0 else 0 for i in range(num_layers)]
    if kind == "every4th":
        return [0 if i % 4 == 3 else 128 for i in range(num_layers)]
    if kind == "selective":
        pat = [128 if i % 2 == 0 else 0 for i in range(num_layers)]
        full = [i for i, w in enumerate(pat) if w == 0]
        n_conv = (8 * len(full)) // 18
        for j in range(n_conv):
            pat[full[(j * len(full)) // max(n_conv, 1)]] = 8192
        return pat
    raise ValueError(kind)


def workload(config_id: int, scale: float = 1.0, pattern: str = "parent") -> Workload:
    """The five benchmark workloads; ``scale`` < 1 shrinks batch/context for tests."""

    def sc(x, lo=1):
        return max(lo, int(round(x * scale)))

    if config_id == 1:
        return Workload("c1_b4_ctx1k_full_contig", 1, sc(4), sc(1024, 33), [0], paged=False)
    if config_id == 2:
        return Workload("c2_b32_ctx8k_full+w128_paged", 2, sc(32), sc(8192, 600), [0, 128], paged=True,
                        calib_prefix=512)
    if config_id == 3:
        return Workload("c3_b16_ctx64k_full_paged", 3, sc(16), sc(65536, 777), [0], paged=True,
                        kv_factor_range=(0.5, 4.0))
    if config_id == 4:
        hi = sc(49152, 300)
        return Workload("c4_b64_ragged16k-48k_36layers_" + pattern, 4, sc(64), hi,
                        layer_pattern(pattern), paged=True, ragged_lo=max(1, hi // 3))
    if config_id == 5:
        return Workload("c5_b8_ctx128k_36layers_" + pattern, 5, sc(8), sc(131072, 300),
                        layer_pattern(pattern), paged=True)
    raise ValueError("config_id must be 1..5")


def bf16_bits(t: torch.Tensor):
    """bf16 tensor -> numpy uint16 bit patterns (numpy has no bf16 type)."""
    import numpy as np
    return t.contiguous().view(torch.int16).cpu().numpy().view(np.uint16)


# ------------------------------------------------------------------ draws ---

def draw_q(w: Workload, layer: int = 0, device: str = "cpu") -> torch.Tensor:
    """Query of the new token, bf16 [batch][Hq][D], N(0,1)."""
    g = _gen(w.seed, S_Q, layer, device)
    return torch.randn(w.batch, w.hq, w.head_dim, generator=g, device=device).to(torch.bfloat16)


def draw_new_kv(w: Workload, layer: int = 0, device: str = "cpu"):
    """K and V of the new token, bf16 [batch][Hkv][D], N(0,1) times the head factors."""
    fk, fv = draw_head_factors(w, layer, device)
    gk, gv = _gen(w.seed, S_KNEW, layer, device), _gen(w.seed, S_VNEW, layer, device)
    k = torch.randn(w.batch, w.hkv, w.head_dim, generator=gk, device=device) * fk[None, :, None]
    v = torch.randn(w.batch, w.hkv, w.head_dim, generator=gv, device=device) * fv[None, :, None]
    return k.to(torch.bfloat16), v.to(torch.bfloat16)


def draw_sinks(w: Workload, layer: int = 0, device: str = "cpu") -> torch.Tensor:
    """One sink logit per query head, float32 [Hq], N(0,1)."""
    g = _gen(w.seed, S_SINK, layer, device)
    return torch.randn(w.hq, generator=g, device=device)


def draw_head_factors(w: Workload, layer: int = 0, device: str = "cpu"):
    """Per-KV-head magnitude factors for K and for V (ones unless the workload spreads them)."""
    if w.kv_factor_range is None:
        one = torch.ones(w.hkv, device=device)
        return one, one.clone()
    lo, hi = w.kv_factor_range
    gk, gv = _gen(w.seed, S_KFACT, layer, device), _gen(w.seed, S_VFACT, layer, device)
    fk = lo + (hi - lo) * torch.rand(w.hkv, generator=gk, device=device)
    fv = lo + (hi - lo) * torch.rand(w.hkv, generator=gv, device=device)
    return fk, fv


def draw_seq_lens(w: Workload, device: str = "cpu") -> torch.Tensor:
    """Context length of every sequence after the append, int32 [batch]."""
    if w.ragged_lo is None:
        return torch.full((w.batch,), w.context, dtype=torch.int32, device=device)
    g = _gen(w.seed, S_LENS, 0, "cpu")
    lens = torch.randint(w.ragged_lo, w.context + 1, (w.batch,), generator=g, dtype=torch.int64)
    return lens.to(torch.int32).to(device)


def draw_block_table(w: Workload, layer: int = 0, num_blocks: Optional[int] = None,
                     device: str = "cpu") -> Optional[torch.Tensor]:
    """int32 [batch][blocks_per_seq]: a seeded permutation of the physical blocks.

    None for contiguous workloads (block = sequence * blocks_per_seq + i).
    """
    if not w.paged:
        return None
    need = w.batch * w.blocks_per_seq
    num_blocks = num_blocks or need
    assert num_blocks >= need
    g = _gen(w.seed, S_TABLE, layer, "cpu")
    perm = torch.randperm(num_blocks, generator=g)[:need]
    return perm.to(torch.int32).reshape(w.batch, w.blocks_per_seq).to(device)


def draw_kv_samples(w: Workload, which: str, num_blocks: int, layer: int = 0, device: str = "cpu",
                    block_lo: int = 0, block_hi: Optional[int] = None) -> torch.Tensor:
    """Pre-quantisation K or V samples in cache layout, float32
    [block_hi-block_lo][Hkv][16][D]: N(0,1) times the per-head factor.

    The samples are independent, so drawing them directly in physical-block
    order is the same distribution as drawing them per logical position and
    scattering through the table.  A range of blocks draws from a stream
    derived from (seed, tensor, layer, block_lo) so big caches can be filled in
    pieces.
    """
    block_hi = num_blocks if block_hi is None else block_hi
    stream = S_K if which == "k" else S_V
    g = _gen(w.seed + 31 * block_lo, stream, layer, device)
    fk, fv = draw_head_factors(w, layer, device)
    f = fk if which == "k" else fv
    x = torch.randn(block_hi - block_lo, w.hkv, w.block, w.head_dim, generator=g, device=device)
    return x * f[None, :, None, None]


def logical_view(cache: torch.Tensor, table: Optional[torch.Tensor], b: int, n_tokens: int,
                 blocks_per_seq: int) -> torch.Tensor:
    """Gather one sequence's first n_tokens from a paged cache: [n_tokens][Hkv][D]."""
    nb = (n_tokens + cache.shape[2] - 1) // cache.shape[2]
    if table is None:
        idx = torch.arange(b * blocks_per_seq, b * blocks_per_seq + nb)
    else:
        idx = table[b, :nb].long().cpu()
    blocks = cache[idx.to(cache.device)]            # [nb][Hkv][16][D]
    seq = blocks.permute(0, 2, 1, 3).reshape(-1, cache.shape[1], cache.shape[3])
    return seq[:n_tokens]


STUDY_KINDS = ("gauss", "heavy", "heads")


def draw_study_stream(kind: str, sigma: float, batch: int, n_tokens: int, which: str = "k", device: str = "cpu",
                      hkv: int = HKV, head_dim: int = HEAD_DIM, seed: int = SEED_BASE + 77) -> torch.Tensor:
    """K or V samples for the scale study, bf16 [batch][n_tokens][Hkv][D].

    gauss: N(0, sigma^2).  heavy: sigma times a Student-t draw with 3 degrees of freedom (rare large values, as
    activation outliers are).  heads: N(0, (sigma * 2^(h - Hkv/2))^2) for KV head h, i.e. heads whose magnitudes
    spread over 2^Hkv."""
    g = _gen(seed, S_K if which == "k" else S_V, int(round(8 * (8 + torch.log2(torch.tensor(float(sigma))).item()))), device)
    shape = (batch, n_tokens, hkv, head_dim)
    z = torch.randn(shape, generator=g, device=device)
    if kind == "gauss":
        x = z * sigma
    elif kind == "heavy":
        chi = torch.randn((3,) + shape, generator=g, device=device).square().sum(0) / 3.0
        x = z / chi.sqrt() * sigma
    elif kind == "heads":
        f = sigma * torch.pow(2.0, torch.arange(hkv, device=device, dtype=torch.float32) - hkv / 2)
        x = z * f[None, None, :, None]
    else:
        raise ValueError(kind)
    return x.to(torch.bfloat16)

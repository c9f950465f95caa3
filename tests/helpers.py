"""Test-side case construction: draws inputs from ``synth`` and turns them into the
byte-level cache a decode step starts from, using the CPU oracle's codec.

Nothing here comes from the CUDA path.  The same dictionaries feed the oracle
pins (CPU) and the parity tests (GPU), which upload them unchanged.
"""
from __future__ import annotations

import numpy as np
import torch

import oracle
import synth


bf16_bits = synth.bf16_bits


def bits_to_bf16(a: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(a.view(np.int16).copy()).view(torch.bfloat16)


def bf16_bits_to_f64(a: np.ndarray) -> np.ndarray:
    with np.errstate(invalid="ignore"):  # signalling-NaN bit patterns are legal inputs
        return (a.astype(np.uint32) << 16).view(np.float32).astype(np.float64)


def make_case(w: synth.Workload, layer: int = 0, spare_blocks: int = 3, kv_dtype: int = oracle.KV_FP8_E4M3,
              pow2_scales: bool = False, no_scales: bool = False, seq_lens=None, poison_tail: bool = False):
    """Build one layer's decode-step inputs on the CPU.

    The cache is pre-filled at every slot (also beyond each sequence's length,
    which the path must ignore); the new token is NOT yet appended.
    Returns a dict of numpy arrays plus the workload.
    """
    nb = w.batch * w.blocks_per_seq + (spare_blocks if w.paged else 0)
    ks = synth.draw_kv_samples(w, "k", nb, layer).numpy()
    vs = synth.draw_kv_samples(w, "v", nb, layer).numpy()
    table = synth.draw_block_table(w, layer, nb)
    table_np = None if table is None else table.numpy().copy()
    lens = synth.draw_seq_lens(w).numpy().copy() if seq_lens is None else np.asarray(seq_lens, dtype=np.int32)

    if kv_dtype == oracle.KV_FP8_E4M3:
        if no_scales:
            k_scale = np.ones(w.hkv, dtype=np.float32)
            v_scale = np.ones(w.hkv, dtype=np.float32)
        else:
            def calib(x):
                if w.calib_prefix is None:
                    toks = x.transpose(0, 2, 1, 3).reshape(-1, w.hkv, w.head_dim)
                else:  # first calib_prefix logical tokens of every sequence
                    parts = []
                    xt = torch.from_numpy(x)
                    for b in range(w.batch):
                        n = min(w.calib_prefix, w.context)
                        parts.append(synth.logical_view(xt, table, b, n, w.blocks_per_seq).numpy())
                    toks = np.concatenate(parts, axis=0)
                return oracle.calibrate_scales(toks, pow2=pow2_scales)
            k_scale, v_scale = calib(ks), calib(vs)
        # fill: float32 quotient, then the oracle's encoder
        k_cache = oracle.e4m3_encode_array((ks / k_scale[None, :, None, None]).astype(np.float32))
        v_cache = oracle.e4m3_encode_array((vs / v_scale[None, :, None, None]).astype(np.float32))
    else:
        k_scale = v_scale = None
        k_cache = bf16_bits(torch.from_numpy(ks).to(torch.bfloat16))
        v_cache = bf16_bits(torch.from_numpy(vs).to(torch.bfloat16))

    if poison_tail:
        # slots at or beyond each sequence's length hold NaN patterns: they must never matter
        nan_code = 0x7F if kv_dtype == oracle.KV_FP8_E4M3 else 0x7FC0
        for b in range(w.batch):
            for pos in range(int(lens[b]), w.blocks_per_seq * w.block):
                blk = (b * w.blocks_per_seq + pos // w.block) if table_np is None else table_np[b, pos // w.block]
                k_cache[blk, :, pos % w.block, :] = nan_code
                v_cache[blk, :, pos % w.block, :] = nan_code

    k_new, v_new = synth.draw_new_kv(w, layer)
    return dict(
        w=w, kv_dtype=kv_dtype, num_blocks=nb,
        k_cache=k_cache, v_cache=v_cache, table=table_np, seq_lens=lens,
        k_scale=k_scale, v_scale=v_scale,
        q=bf16_bits(synth.draw_q(w, layer)), sinks=synth.draw_sinks(w, layer).numpy().copy(),
        k_new=bf16_bits(k_new), v_new=bf16_bits(v_new),
        sm_scale=1.0 / float(np.sqrt(w.head_dim)),
    )


def oracle_append(case) -> None:
    """Append the case's new token with the oracle (in place)."""
    w = case["w"]
    oracle.kv_append(case["k_cache"], case["v_cache"], case["kv_dtype"], w.block, case["table"],
                     w.blocks_per_seq, case["seq_lens"], case["k_scale"], case["v_scale"],
                     case["k_new"], case["v_new"])


def oracle_attn(case, window, sinks="case", items=None, seq_lens=None):
    w = case["w"]
    s = case["sinks"] if isinstance(sinks, str) else sinks
    out, lse = oracle.decode_attn(case["k_cache"], case["v_cache"], case["kv_dtype"], case["table"],
                                  w.blocks_per_seq, case["seq_lens"] if seq_lens is None else seq_lens,
                                  case["k_scale"], case["v_scale"], case["q"], s, window, case["sm_scale"],
                                  items=items)
    if items is None:
        out = out.reshape(w.batch, w.hq, w.head_dim)
        lse = lse.reshape(w.batch, w.hq)
    return out, lse

"""Upload a CPU-built case to the GPU and run the library on it through the C ABI."""
from __future__ import annotations

import numpy as np
import torch

import paper_2602_11937_b200 as P
from helpers import bits_to_bf16

TOL_ABS = 2e-3            # max |err| on bf16 outputs for N(0,1) inputs
TOL_REL = 2.0 ** -8       # one bf16 half-ulp, for outputs whose magnitude reaches 1 and beyond


def to_dev(a, dtype=None):
    if a is None:
        return None
    t = torch.from_numpy(np.ascontiguousarray(a))
    if dtype is not None:
        t = t.to(dtype)
    return t.cuda()


class DeviceCase:
    """Device copies of one case (cache bytes exactly as the CPU side built them)."""

    def __init__(self, case):
        w = case["w"]
        self.case, self.w = case, w
        self.kv_dtype = case["kv_dtype"]
        if self.kv_dtype == P.KV_FP8_E4M3:
            self.k_cache, self.v_cache = to_dev(case["k_cache"]), to_dev(case["v_cache"])
        else:
            self.k_cache = bits_to_bf16(case["k_cache"]).cuda()
            self.v_cache = bits_to_bf16(case["v_cache"]).cuda()
        self.table = to_dev(case["table"])
        self.seq_lens = to_dev(case["seq_lens"])
        self.k_scale, self.v_scale = to_dev(case["k_scale"]), to_dev(case["v_scale"])
        self.q = bits_to_bf16(case["q"]).cuda()
        self.sinks = to_dev(case["sinks"])
        self.k_new, self.v_new = bits_to_bf16(case["k_new"]).cuda(), bits_to_bf16(case["v_new"]).cuda()
        self.status = torch.zeros(1, dtype=torch.int32, device="cuda")

    def view(self, seq_lens=None):
        return P.kv_view(self.k_cache, self.v_cache, self.seq_lens if seq_lens is None else seq_lens,
                         block_table=self.table, max_blocks_per_seq=self.w.blocks_per_seq,
                         k_scale=self.k_scale, v_scale=self.v_scale)

    def desc(self, window=0):
        return P.layer_desc(window=window, kv_dtype=self.kv_dtype, num_q_heads=self.w.hq, num_kv_heads=self.w.hkv,
                            head_dim=self.w.head_dim, block_size=self.w.block, sm_scale=self.case["sm_scale"])

    def append(self):
        P.puzzle_kv_append(self.desc(), self.view(), self.k_new, self.v_new, dev_status=self.status)
        torch.cuda.synchronize()

    def attn(self, window=0, num_splits=0, sinks="case", seq_lens=None, want_lse=True, kernel="mma"):
        w = self.w
        d = self.desc(window)
        ws = torch.empty(max(16, P.puzzle_decode_attn_workspace_bytes(d, w.batch, num_splits)), dtype=torch.uint8,
                         device="cuda")
        ws.fill_(0xFF)  # NaN patterns: stale scratch must never leak into results
        P.puzzle_decode_attn_workspace_init(d, w.batch, ws)
        out = torch.full((w.batch, w.hq, w.head_dim), float("nan"), dtype=torch.bfloat16, device="cuda")
        lse = torch.full((w.batch, w.hq), float("nan"), dtype=torch.float32, device="cuda") if want_lse else None
        s = self.sinks if isinstance(sinks, str) else sinks
        call = P.puzzle_decode_attn_tcgen05 if kernel == "tcgen05" else P.puzzle_decode_attn
        call(d, self.view(seq_lens), self.q, s, out, lse, num_splits=num_splits, workspace=ws, dev_status=self.status)
        torch.cuda.synchronize()
        return out.float().cpu().numpy().astype(np.float64), (None if lse is None else lse.cpu().numpy().astype(np.float64))

    def cache_bytes(self):
        def host(t):
            if t.dtype == torch.bfloat16:
                return t.view(torch.int16).cpu().numpy().view(np.uint16)
            return t.cpu().numpy()
        return host(self.k_cache), host(self.v_cache)


def error_bound(ref, rel=False):
    """Allowed |err| per element.  2e-3 everywhere a bf16 output can meet it, i.e. |ref| < 1 (half a bf16
    ulp is at most 2^-9 there).  From |ref| >= 1 on, half an ulp alone is 2^-8 |ref| >= 3.9e-3, so that
    much is added.  rel=True adds it for every element (workloads whose K/V are scaled up)."""
    a = np.abs(ref)
    return TOL_ABS + np.where((a >= 1.0) | rel, TOL_REL * a, 0.0)


def assert_close(got, ref, what="", rel=False):
    err = np.abs(got - ref)
    bad = ~(err <= error_bound(ref, rel))
    if bad.any():
        i = np.unravel_index(np.nanargmax(np.where(bad, err, -1)), err.shape)
        raise AssertionError("%s: |err| %.3e at %s (ref %.5f, got %.5f), %d elements over the bound" % (
            what, err[i], i, ref[i], got[i], int(bad.sum())))
    return float(err.max()) if err.size else 0.0

"""Pins for the oracle's attention and merge (CPU only).

The paper prints no worked numbers for this path, so the pins are what the
definitions fix: invariants of window/full attention, closed forms, the
library's fp64 softmax attention as a special case, and an independent
triple loop in pure Python on tiny shapes.
"""
import math
import os

import numpy as np
import pytest
import torch

import oracle
import synth
from helpers import bf16_bits, bf16_bits_to_f64, make_case, oracle_append, oracle_attn

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _tiny(batch=2, ctx=40, paged=True, hq=16, hkv=2, lens=None, **kw):
    w = synth.Workload("tiny", 1, batch, ctx, [0], paged=paged, hq=hq, hkv=hkv, **kw)
    case = make_case(w, seq_lens=lens)
    oracle_append(case)
    return case


def _lib_decode_table():
    """Code -> value through the library's float8 type, independent of the oracle's decode."""
    return torch.arange(256, dtype=torch.uint8).view(torch.float8_e4m3fn).to(torch.float64).numpy()


def _bruteforce(case, window, use_sink=True):
    """Independent pure-Python statement: loops over (sequence, head, key, channel)."""
    w = case["w"]
    table_val = _lib_decode_table()
    G = w.hq // w.hkv
    qf = bf16_bits_to_f64(case["q"])
    out = np.zeros((w.batch, w.hq, w.head_dim))
    lse = np.zeros((w.batch, w.hq))
    for b in range(w.batch):
        L = int(case["seq_lens"][b])
        lo = 0 if window == 0 else max(0, L - window)
        for g in range(w.hq):
            h = g // G
            logits = []
            vals = []
            for j in range(lo, L):
                blk = case["table"][b, j // 16] if case["table"] is not None else b * w.blocks_per_seq + j // 16
                kb = case["k_cache"][blk, h, j % 16]
                vb = case["v_cache"][blk, h, j % 16]
                s = 0.0
                for d in range(w.head_dim):
                    s += qf[b, g, d] * (table_val[kb[d]] * float(case["k_scale"][h]))
                logits.append(s * case["sm_scale"])
                vals.append([table_val[vb[d]] * float(case["v_scale"][h]) for d in range(w.head_dim)])
            cols = list(logits)
            if use_sink:
                cols.append(float(case["sinks"][g]))
            if not cols:
                lse[b, g] = -math.inf
                continue
            m = max(cols)
            z = sum(math.exp(c - m) for c in cols)
            for j, s in enumerate(logits):
                p = math.exp(s - m) / z
                for d in range(w.head_dim):
                    out[b, g, d] += p * vals[j][d]
            lse[b, g] = m + math.log(z)
    return out, lse


@pytest.mark.parametrize("window", [0, 1, 5, 16, 17, 40, 1000])
def test_bruteforce_tiny(window):
    case = _tiny(lens=[40, 23])
    want, want_lse = _bruteforce(case, window)
    got, got_lse = oracle_attn(case, window)
    np.testing.assert_allclose(got, want, rtol=1e-12, atol=1e-14)
    np.testing.assert_allclose(got_lse, want_lse, rtol=1e-12, atol=1e-14)


def test_bruteforce_contiguous_no_sink():
    case = _tiny(paged=False, ctx=33, lens=[33, 1])
    want, want_lse = _bruteforce(case, 7, use_sink=False)
    got, got_lse = oracle_attn(case, 7, sinks=None)
    np.testing.assert_allclose(got, want, rtol=1e-12, atol=1e-14)
    np.testing.assert_allclose(got_lse, want_lse, rtol=1e-12, atol=1e-14)


def test_window_at_least_context_equals_full():
    case = _tiny(batch=3, ctx=100, lens=[100, 64, 65])
    full, full_lse = oracle_attn(case, 0)
    for W in (100, 101, 4096):
        got, lse = oracle_attn(case, W)
        assert np.array_equal(got, full) and np.array_equal(lse, full_lse)
    # a window one short of the longest context must differ for that sequence only
    got, _ = oracle_attn(case, 99)
    assert not np.array_equal(got[0], full[0]) and np.array_equal(got[1:], full[1:])


def test_window_sees_exactly_the_last_w_tokens():
    """A layer with window W over L tokens equals full attention over a cache that holds
    only those W tokens (the KV footprint of a window layer is W, not L)."""
    W, L = 21, 90
    case = _tiny(batch=1, ctx=L, paged=False, lens=[L])
    got, lse = oracle_attn(case, W)
    w2 = synth.Workload("cut", 1, 1, W, [0], paged=False, hq=16, hkv=2)
    nb2 = w2.blocks_per_seq
    k2 = np.zeros((nb2, 2, 16, 64), dtype=np.uint8)
    v2 = np.zeros_like(k2)
    for j in range(W):
        src = L - W + j
        k2[j // 16, :, j % 16] = case["k_cache"][src // 16, :, src % 16]
        v2[j // 16, :, j % 16] = case["v_cache"][src // 16, :, src % 16]
    want, want_lse = oracle.decode_attn(k2, v2, oracle.KV_FP8_E4M3, None, nb2, np.array([W], dtype=np.int32),
                                        case["k_scale"], case["v_scale"], case["q"], case["sinks"], 0,
                                        case["sm_scale"])
    np.testing.assert_allclose(got.reshape(-1, 64), want, rtol=1e-13, atol=0)
    np.testing.assert_allclose(lse.reshape(-1), want_lse, rtol=1e-13, atol=0)


def test_no_sink_equals_library_softmax_attention():
    """sinks = None, sinks = -inf and the library's fp64 scaled-dot-product attention agree."""
    case = _tiny(batch=2, ctx=70, lens=[70, 70])
    w = case["w"]
    a, _ = oracle_attn(case, 0, sinks=None)
    b, _ = oracle_attn(case, 0, sinks=np.full(w.hq, -np.inf, dtype=np.float32))
    assert np.array_equal(a, b)
    dec = _lib_decode_table()
    q = torch.from_numpy(bf16_bits_to_f64(case["q"]))                       # [B][Hq][D]
    K = torch.zeros(w.batch, w.hkv, 70, 64, dtype=torch.float64)
    V = torch.zeros_like(K)
    for bi in range(w.batch):
        for j in range(70):
            blk = case["table"][bi, j // 16]
            K[bi, :, j] = torch.from_numpy(dec[case["k_cache"][blk, :, j % 16]] * case["k_scale"][:, None].astype(np.float64))
            V[bi, :, j] = torch.from_numpy(dec[case["v_cache"][blk, :, j % 16]] * case["v_scale"][:, None].astype(np.float64))
    G = w.hq // w.hkv
    want = torch.nn.functional.scaled_dot_product_attention(
        q[:, :, None, :], K.repeat_interleave(G, dim=1), V.repeat_interleave(G, dim=1), scale=case["sm_scale"])
    np.testing.assert_allclose(a, want[:, :, 0].numpy(), rtol=1e-11, atol=1e-13)


def test_identical_keys_closed_form():
    """All keys equal -> every logit is s, so out = n e^s / (n e^s + e^sink) * mean(V)."""
    case = _tiny(batch=1, ctx=37, paged=False, lens=[37])
    w = case["w"]
    n = 37
    for j in range(n):
        case["k_cache"][j // 16, :, j % 16] = case["k_cache"][0, :, 0]
    got, lse = oracle_attn(case, 0)
    dec = _lib_decode_table()
    qf = bf16_bits_to_f64(case["q"])[0]
    for g in range(w.hq):
        h = g // (w.hq // w.hkv)
        k0 = dec[case["k_cache"][0, h, 0]] * float(case["k_scale"][h])
        s = float(qf[g] @ k0) * case["sm_scale"]
        vmean = np.mean([dec[case["v_cache"][j // 16, h, j % 16]] * float(case["v_scale"][h]) for j in range(n)], axis=0)
        sink = float(case["sinks"][g])
        frac = n * math.exp(s) / (n * math.exp(s) + math.exp(sink))
        np.testing.assert_allclose(got[0, g], frac * vmean, rtol=1e-12, atol=1e-15)
        np.testing.assert_allclose(lse[0, g], math.log(n * math.exp(s) + math.exp(sink)), rtol=1e-12)


def test_single_token_and_empty_context():
    case = _tiny(batch=3, ctx=20, paged=False, lens=[1, 0, 20])
    w = case["w"]
    got, lse = oracle_attn(case, 0)
    dec = _lib_decode_table()
    qf = bf16_bits_to_f64(case["q"])
    for g in range(w.hq):
        h = g // (w.hq // w.hkv)
        k0 = dec[case["k_cache"][0, h, 0]] * float(case["k_scale"][h])
        v0 = dec[case["v_cache"][0, h, 0]] * float(case["v_scale"][h])
        s = float(qf[0, g] @ k0) * case["sm_scale"]
        sink = float(case["sinks"][g])
        np.testing.assert_allclose(got[0, g], v0 * math.exp(s) / (math.exp(s) + math.exp(sink)), rtol=1e-12, atol=1e-15)
        # empty context: nothing to average, all mass on the sink
        assert not got[1, g].any() and lse[1, g] == pytest.approx(sink)
    got2, lse2 = oracle_attn(case, 0, sinks=None)
    assert not got2[1].any() and np.all(np.isneginf(lse2[1]))
    assert np.isfinite(got2).all()


def test_dominant_logit_selects_its_value_row():
    case = _tiny(batch=1, ctx=50, paged=False, hq=2, hkv=2, lens=[50])
    case["q"][:] = bf16_bits(torch.full((1, 2, 64), 16.0, dtype=torch.bfloat16))
    case["k_cache"][:] = oracle.e4m3_encode(0.0)
    case["k_cache"][2, :, 3, :] = oracle.e4m3_encode(448.0)  # token 35
    got, _ = oracle_attn(case, 0)
    dec = _lib_decode_table()
    for h in range(2):
        v = dec[case["v_cache"][2, h, 3]] * float(case["v_scale"][h])
        np.testing.assert_allclose(got[0, h], v, rtol=1e-9, atol=1e-12)


def test_block_permutation_and_contiguous_equivalence():
    case = _tiny(batch=2, ctx=70, lens=[70, 33])
    w = case["w"]
    base, base_lse = oracle_attn(case, 9)
    rng = np.random.default_rng(3)
    perm = rng.permutation(case["num_blocks"])           # new physical position of each block
    k2 = np.empty_like(case["k_cache"]); v2 = np.empty_like(case["v_cache"])
    k2[perm] = case["k_cache"]; v2[perm] = case["v_cache"]
    t2 = perm[case["table"]].astype(np.int32)
    got, lse = oracle.decode_attn(k2, v2, oracle.KV_FP8_E4M3, t2, w.blocks_per_seq, case["seq_lens"],
                                  case["k_scale"], case["v_scale"], case["q"], case["sinks"], 9, case["sm_scale"])
    assert np.array_equal(got.reshape(base.shape), base)
    # identity table == NULL table
    ident = np.arange(w.batch * w.blocks_per_seq, dtype=np.int32).reshape(w.batch, -1)
    a, _ = oracle.decode_attn(case["k_cache"], case["v_cache"], 0, ident, w.blocks_per_seq, case["seq_lens"],
                              case["k_scale"], case["v_scale"], case["q"], case["sinks"], 0, case["sm_scale"])
    b, _ = oracle.decode_attn(case["k_cache"], case["v_cache"], 0, None, w.blocks_per_seq, case["seq_lens"],
                              case["k_scale"], case["v_scale"], case["q"], case["sinks"], 0, case["sm_scale"])
    assert np.array_equal(a, b)


def test_scale_homogeneity():
    case = _tiny(batch=1, ctx=45, lens=[45])
    base, _ = oracle_attn(case, 0)
    c2 = dict(case)
    c2["k_scale"] = case["k_scale"] * np.float32(4.0)
    c2["q"] = bf16_bits((torch.from_numpy(bf16_bits_to_f64(case["q"])) / 4).to(torch.bfloat16))  # exact in bf16
    got, _ = oracle_attn(c2, 0)
    np.testing.assert_allclose(got, base, rtol=1e-12, atol=1e-15)
    c3 = dict(case)
    c3["v_scale"] = case["v_scale"] * np.float32(2.0)
    got, _ = oracle_attn(c3, 0)
    np.testing.assert_allclose(got, 2 * base, rtol=1e-13, atol=0)
    c4 = dict(case)
    c4["k_scale"] = None
    c4["v_scale"] = None
    c5 = dict(case)
    c5["k_scale"] = np.ones(case["w"].hkv, dtype=np.float32)
    c5["v_scale"] = np.ones(case["w"].hkv, dtype=np.float32)
    assert np.array_equal(oracle_attn(c4, 0)[0], oracle_attn(c5, 0)[0])   # "no scales" variant


def test_poisoned_tail_is_ignored():
    w = synth.Workload("tail", 1, 2, 50, [0], paged=True, hq=16, hkv=2)
    a = make_case(w, seq_lens=[50, 19])
    b = make_case(w, seq_lens=[50, 19], poison_tail=True)
    oracle_append(a); oracle_append(b)
    ga, _ = oracle_attn(a, 0)
    gb, _ = oracle_attn(b, 0)
    assert np.isfinite(gb).all() and np.array_equal(ga, gb)


def test_bf16_kv_variant_against_library():
    w = synth.Workload("bf", 1, 2, 48, [0], paged=False, hq=16, hkv=2)
    case = make_case(w, kv_dtype=oracle.KV_BF16)
    oracle_append(case)
    got, _ = oracle_attn(case, 0, sinks=None)
    K = torch.from_numpy(bf16_bits_to_f64(case["k_cache"])).reshape(2, 3, 2, 16, 64).permute(0, 2, 1, 3, 4).reshape(2, 2, 48, 64)
    V = torch.from_numpy(bf16_bits_to_f64(case["v_cache"])).reshape(2, 3, 2, 16, 64).permute(0, 2, 1, 3, 4).reshape(2, 2, 48, 64)
    q = torch.from_numpy(bf16_bits_to_f64(case["q"]))
    want = torch.nn.functional.scaled_dot_product_attention(
        q[:, :, None, :], K.repeat_interleave(8, dim=1), V.repeat_interleave(8, dim=1), scale=case["sm_scale"])
    np.testing.assert_allclose(got, want[:, :, 0].numpy(), rtol=1e-11, atol=1e-13)


# ------------------------------------------------------------------ merge ---

@pytest.mark.parametrize("cuts", [[0, 70], [0, 16, 70], [0, 1, 2, 69, 70], [0, 33, 33, 50, 70], [0, 64, 70]])
def test_merge_of_any_partition_equals_unsplit(cuts):
    case = _tiny(batch=2, ctx=70, lens=[70, 41])
    w = case["w"]
    full, full_lse = oracle_attn(case, 0)
    parts_o, parts_l = [], []
    for t0, t1 in zip(cuts[:-1], cuts[1:]):
        o, l = oracle.partial_attn(case["k_cache"], case["v_cache"], 0, case["table"], w.blocks_per_seq,
                                   case["seq_lens"], case["k_scale"], case["v_scale"], case["q"],
                                   case["sm_scale"], t0, t1)
        parts_o.append(o); parts_l.append(l)
    po = np.stack(parts_o, axis=1)            # [rows][S][D]
    pl = np.stack(parts_l, axis=1)
    sink = np.tile(case["sinks"].astype(np.float64), w.batch)
    got, lse = oracle.attn_merge(po, pl, None, sink)
    np.testing.assert_allclose(got.reshape(full.shape), full, rtol=1e-12, atol=1e-15)
    np.testing.assert_allclose(lse.reshape(full_lse.shape), full_lse, rtol=1e-12)
    # empty parts carry lse = -inf
    if cuts.count(33) == 2:
        assert np.all(np.isneginf(pl[:, 1]))


def test_merge_two_level_and_num_parts():
    rng = np.random.default_rng(5)
    rows, S, D = 6, 5, 8
    po = rng.standard_normal((rows, S, D))
    pl = rng.standard_normal((rows, S)) * 3
    sink = rng.standard_normal(rows)
    flat, flat_lse = oracle.attn_merge(po, pl, None, sink)
    # merge parts {0,1,2} and {3,4} without sink, then merge the two results with the sink
    a, al = oracle.attn_merge(po[:, :3], pl[:, :3])
    b, bl = oracle.attn_merge(po[:, 3:], pl[:, 3:])
    two, two_lse = oracle.attn_merge(np.stack([a, b], axis=1), np.stack([al, bl], axis=1), None, sink)
    np.testing.assert_allclose(two, flat, rtol=1e-12)
    np.testing.assert_allclose(two_lse, flat_lse, rtol=1e-12)
    # closed form for one row
    wts = np.exp(pl[0]); z = wts.sum() + math.exp(sink[0])
    np.testing.assert_allclose(flat[0], (wts[:, None] * po[0]).sum(0) / z, rtol=1e-12)
    np.testing.assert_allclose(flat_lse[0], math.log(z), rtol=1e-12)
    # num_parts limits how many parts count
    n = np.array([5, 3, 1, 0, 2, 5], dtype=np.int32)
    got, gl = oracle.attn_merge(po, pl, n, None)
    for r in range(rows):
        if n[r] == 0:
            assert not got[r].any() and np.isneginf(gl[r])
        else:
            w_ = np.exp(pl[r, : n[r]])
            np.testing.assert_allclose(got[r], (w_[:, None] * po[r, : n[r]]).sum(0) / w_.sum(), rtol=1e-12)


# ------------------------------------------------------- byte accounting ----

def test_selective_window_pattern_reproduces_the_papers_kv_reduction():
    line = [l for l in open(os.path.join(GOLDEN, "kv_cache_reduction.txt")) if not l.startswith("#")][0].split()
    frac, tol, ctxs = float(line[0]), float(line[1]), [int(c) for c in line[2:]]
    parent, sel = synth.layer_pattern("parent"), synth.layer_pattern("selective")
    assert parent.count(0) == 18 and parent.count(128) == 18
    assert sel.count(0) == 10 and sel.count(8192) == 8 and sel.count(128) == 18

    def tokens(pattern, L):
        return sum(L if W == 0 else min(W, L) for W in pattern)

    for L in ctxs:
        smaller = 1 - tokens(sel, L) / tokens(parent, L)
        assert abs(smaller - frac) <= tol, (L, smaller)

"""Several new tokens per sequence in one step: the bulk quantise-append (bytes exact against token-by-token oracle
appends) and causal multi-token attention through the decode kernels (each query against the oracle's single-token
attention at that query's position).  Ragged chunk lengths, full and window layers, both kernels."""
import numpy as np
import pytest
import torch

import oracle
import synth
from helpers import bf16_bits, make_case

pytestmark = pytest.mark.gpu


def _chunk(case, n_new, seed):
    w = case["w"]
    g = torch.Generator().manual_seed(seed)
    k = torch.randn(w.batch, n_new, w.hkv, w.head_dim, generator=g).to(torch.bfloat16)
    v = torch.randn(w.batch, n_new, w.hkv, w.head_dim, generator=g).to(torch.bfloat16)
    q = torch.randn(w.batch, n_new, w.hq, w.head_dim, generator=g).to(torch.bfloat16)
    return k, v, q


def _oracle_append_chunk(case, lens_after, new_lens, k, v):
    """Token by token with the oracle's single-token append."""
    w = case["w"]
    for i in range(k.shape[1]):
        real = (i < new_lens) & (lens_after - new_lens + i >= 0)
        step_lens = np.where(real, lens_after - new_lens + i + 1, 0).astype(np.int32)   # length 0: skipped
        oracle.kv_append(case["k_cache"], case["v_cache"], case["kv_dtype"], w.block, case["table"], w.blocks_per_seq,
                         step_lens, case["k_scale"], case["v_scale"], bf16_bits(k[:, i].contiguous()),
                         bf16_bits(v[:, i].contiguous()))


@pytest.mark.parametrize("kv_dtype", [oracle.KV_FP8_E4M3, oracle.KV_BF16], ids=["fp8", "bf16"])
@pytest.mark.parametrize("n_new", [1, 5, 64])
def test_bulk_append_bytes_equal_token_by_token_oracle(n_new, kv_dtype):
    import paper_2602_11937_b200 as P
    from gpu_helpers import DeviceCase
    w = synth.Workload("chunk", 1, 5, 400, [0], paged=True)
    lens_after = np.array([400, 0, 3, 130, 64], dtype=np.int32)
    case = make_case(w, seq_lens=lens_after, kv_dtype=kv_dtype)
    dev = DeviceCase(case)
    k, v, _ = _chunk(case, n_new, 11 + n_new)
    for new_lens in (None, np.array([n_new, 0, min(3, n_new), n_new // 2, 1], dtype=np.int32)):
        nl_dev = None if new_lens is None else torch.from_numpy(new_lens).cuda()
        P.puzzle_kv_append_tokens(dev.desc(), dev.view(), k.cuda(), v.cuda(), nl_dev, dev_status=dev.status)
        torch.cuda.synchronize()
        _oracle_append_chunk(case, lens_after, np.full(5, n_new, dtype=np.int32) if new_lens is None else new_lens, k, v)
        gk, gv = dev.cache_bytes()
        assert np.array_equal(gk, case["k_cache"]) and np.array_equal(gv, case["v_cache"])
    assert int(dev.status.item()) == 0


@pytest.mark.parametrize("kernel", ["mma", "tcgen05"])
@pytest.mark.parametrize("window", [0, 100])
def test_multi_token_causal_attention(window, kernel):
    import paper_2602_11937_b200 as P
    from gpu_helpers import DeviceCase, assert_close
    n_q = 4
    w = synth.Workload("multiq", 1, 5, 700, [0], paged=True)
    lens_after = np.array([700, 2, 4, 333, 129], dtype=np.int32)
    q_lens = np.array([4, 2, 4, 3, 0], dtype=np.int32)            # ragged; the last sequence has no query this step
    case = make_case(w, seq_lens=lens_after)
    dev = DeviceCase(case)
    k, v, q = _chunk(case, n_q, 5)
    ql_dev = torch.from_numpy(q_lens).cuda()
    P.puzzle_kv_append_tokens(dev.desc(window), dev.view(), k.cuda(), v.cuda(), ql_dev, dev_status=dev.status)
    _oracle_append_chunk(case, lens_after, q_lens, k, v)
    lens2, table2 = P.multi_token_args(dev.seq_lens, dev.table, n_q, q_lens=ql_dev)
    view = P.kv_view(dev.k_cache, dev.v_cache, lens2, block_table=table2, k_scale=dev.k_scale, v_scale=dev.v_scale)
    d = dev.desc(window)
    rows = w.batch * n_q
    ws = torch.zeros(P.puzzle_decode_attn_workspace_bytes(d, rows, 0), dtype=torch.uint8, device="cuda")
    P.puzzle_decode_attn_workspace_init(d, rows, ws)
    out = torch.full((rows, w.hq, w.head_dim), float("nan"), dtype=torch.bfloat16, device="cuda")
    call = P.puzzle_decode_attn_tcgen05 if kernel == "tcgen05" else P.puzzle_decode_attn
    call(d, view, q.cuda().view(rows, w.hq, w.head_dim), dev.sinks, out, None, workspace=ws, dev_status=dev.status)
    torch.cuda.synchronize()
    assert int(dev.status.item()) == 0
    got = out.float().cpu().numpy().astype(np.float64).reshape(w.batch, n_q, w.hq, w.head_dim)
    for i in range(n_q):       # the oracle's decode step of query row i: a sequence that ends at that query
        real = i < q_lens
        step_lens = np.where(real, lens_after - q_lens + i + 1, 0).astype(np.int32)
        ref, _ = oracle.decode_attn(case["k_cache"], case["v_cache"], case["kv_dtype"], case["table"], w.blocks_per_seq,
                                    step_lens, case["k_scale"], case["v_scale"], bf16_bits(q[:, i].contiguous()),
                                    case["sinks"], window, case["sm_scale"])
        assert_close(got[:, i], ref.reshape(w.batch, w.hq, w.head_dim), "query row %d, W=%d" % (i, window))
        assert not got[~real, i].any()                 # padding rows and absent queries give zeros


@pytest.mark.parametrize("n_q", [1, 2, 3, 4, 5])
@pytest.mark.parametrize("window", [0, 100])
def test_tokens_kernel_shares_tiles_between_query_tokens(window, n_q):
    """puzzle_decode_attn_tokens (pairs of query tokens on one pass over the tiles) against the oracle's
    single-token step at every query position: ragged numbers of new tokens, sequences shorter than a tile, one
    with no query, contexts that span many workers."""
    _tokens_against_oracle(window, n_q, None)


def test_tokens_kernel_one_workspace_for_different_token_counts():
    """One workspace, prepared once, serves calls with different numbers of query tokens one after the other."""
    import paper_2602_11937_b200 as P
    d = P.layer_desc(kv_dtype=P.KV_FP8_E4M3)
    ws = torch.empty(P.puzzle_decode_attn_tokens_workspace_bytes(d, 6, 5), dtype=torch.uint8, device="cuda")
    ws.fill_(0xFF)
    P.puzzle_decode_attn_tokens_workspace_init(d, 6, 1, ws)
    for n_q in (5, 2, 4, 1, 5):
        _tokens_against_oracle(0, n_q, ws)


def _tokens_against_oracle(window, n_q, shared_ws):
    import paper_2602_11937_b200 as P
    from gpu_helpers import DeviceCase, assert_close
    w = synth.Workload("tokq", 1, 6, 3000, [0], paged=True)
    lens_after = np.array([3000, 2, 5, 333, 129, 1900], dtype=np.int32)
    q_lens = np.minimum(np.array([n_q, 2, 5, 3, 0, n_q - 1 if n_q > 1 else 1], dtype=np.int32), n_q)
    case = make_case(w, seq_lens=lens_after)
    dev = DeviceCase(case)
    k, v, q = _chunk(case, n_q, 50 + n_q)
    ql_dev = torch.from_numpy(q_lens).cuda()
    d = dev.desc(window)
    P.puzzle_kv_append_tokens(d, dev.view(), k.cuda(), v.cuda(), ql_dev, dev_status=dev.status)
    _oracle_append_chunk(case, lens_after, q_lens, k, v)
    ws = shared_ws
    if ws is None:
        ws = torch.empty(P.puzzle_decode_attn_tokens_workspace_bytes(d, w.batch, n_q), dtype=torch.uint8, device="cuda")
        ws.fill_(0xFF)
        P.puzzle_decode_attn_tokens_workspace_init(d, w.batch, n_q, ws)
    for call in range(2):          # the second call finds the counters as the first one left them
        out = torch.full((w.batch, n_q, w.hq, w.head_dim), 7.0, dtype=torch.bfloat16, device="cuda")
        lse = torch.full((w.batch, n_q, w.hq), 7.0, dtype=torch.float32, device="cuda")
        P.puzzle_decode_attn_tokens(d, dev.view(), q.cuda(), dev.sinks, out, lse, q_lens=ql_dev, workspace=ws,
                                    dev_status=dev.status)
        torch.cuda.synchronize()
        assert int(dev.status.item()) == 0
        got = out.float().cpu().numpy().astype(np.float64)
        got_lse = lse.cpu().numpy().astype(np.float64)
        for i in range(n_q):
            real = i < q_lens
            step_lens = np.where(real, lens_after - q_lens + i + 1, 0).astype(np.int32)
            ref, ref_lse = oracle.decode_attn(case["k_cache"], case["v_cache"], case["kv_dtype"], case["table"],
                                              w.blocks_per_seq, step_lens, case["k_scale"], case["v_scale"],
                                              bf16_bits(q[:, i].contiguous()), case["sinks"], window, case["sm_scale"])
            ref = ref.reshape(w.batch, w.hq, w.head_dim)
            assert_close(got[real, i], ref[real], "query row %d, W=%d, n_q=%d, call %d" % (i, window, n_q, call))
            assert np.all(np.abs(got_lse[real, i] - ref_lse.reshape(w.batch, w.hq)[real]) <= 2e-3)
            assert np.all(got[~real, i] == 7.0) and np.all(got_lse[~real, i] == 7.0)     # rows without a query: untouched


def test_tokens_kernel_argument_errors():
    import paper_2602_11937_b200 as P
    from gpu_helpers import DeviceCase
    w = synth.Workload("tokerr", 1, 2, 64, [0], paged=True)
    dev = DeviceCase(make_case(w))
    q = torch.zeros(2, 2, 64, 64, dtype=torch.bfloat16, device="cuda")
    out = torch.zeros_like(q)
    ws = torch.zeros(P.puzzle_decode_attn_tokens_workspace_bytes(dev.desc(), 2, 2), dtype=torch.uint8, device="cuda")
    with pytest.raises(P.PuzzleError) as e:
        P.puzzle_decode_attn_tokens(dev.desc(), dev.view(), q, None, out, workspace=ws[:256])
    assert e.value.code == 4
    bf = P.layer_desc(kv_dtype=P.KV_BF16)
    with pytest.raises(P.PuzzleError) as e:
        P.puzzle_decode_attn_tokens(bf, dev.view(), q, None, out, workspace=ws)
    assert e.value.code == 3
    assert P.puzzle_decode_attn_tokens_workspace_bytes(dev.desc(), 8192, 4) == 0      # too many rows
    torch.cuda.synchronize()

"""GPU tests of the sharded paths on ONE GPU: the ranks' calls run one after the other on the same device (no
kernel waits for another), each on the shard a rank would hold; the exchanged buffer is filled in place of the
all-gather.  Bars as everywhere: appended bytes exact, merged bf16 output within 2e-3 of the float64 oracle.
"""
import numpy as np
import pytest
import torch

import oracle
import synth
from helpers import make_case, oracle_append, oracle_attn
from parallel_helpers import local_table

pytestmark = pytest.mark.gpu


def _case(kind):
    if kind == "ragged":
        w = synth.Workload("ctxshard", 1, 6, 1500, [0], paged=True)
        return make_case(w, seq_lens=[1500, 0, 1, 17, 333, 1024], poison_tail=True)
    return make_case(synth.workload(1))                 # batch 4, context 1024, contiguous cache


@pytest.mark.parametrize("world", [1, 2, 3, 8])
@pytest.mark.parametrize("kind", ["ragged", "contiguous"])
def test_context_sharded_layer_matches_full_attention(kind, world):
    import paper_2602_11937_b200 as P
    from gpu_helpers import DeviceCase, assert_close
    from paper_2602_11937_b200.parallel import ContextShardedAttention, context_slice
    case = _case(kind)
    dev = DeviceCase(case)
    w = case["w"]
    layer = ContextShardedAttention(dev.desc(0), w.batch, "cuda", world)
    views = []
    for r in range(world):
        local, app = context_slice(dev.seq_lens, r, world)
        tab = torch.from_numpy(local_table(case, r, world)).cuda()
        app_view = P.kv_view(dev.k_cache, dev.v_cache, app, block_table=tab, k_scale=dev.k_scale, v_scale=dev.v_scale)
        P.puzzle_kv_append(dev.desc(0), app_view, dev.k_new, dev.v_new, dev_status=dev.status)   # owner ranks only
        views.append((local, tab, app))
    torch.cuda.synchronize()
    oracle_append(case)
    gk, gv = dev.cache_bytes()
    assert np.array_equal(gk, case["k_cache"]) and np.array_equal(gv, case["v_cache"])

    for r, (local, tab, _) in enumerate(views):
        view = P.kv_view(dev.k_cache, dev.v_cache, local, block_table=tab, k_scale=dev.k_scale, v_scale=dev.v_scale)
        layer.gathered[r].fill_(float("nan"))
        layer.partial(view, dev.q, into=layer.gathered[r])
    out = torch.full((w.batch, w.hq, w.head_dim), float("nan"), dtype=torch.bfloat16, device="cuda")
    lse = torch.full((w.batch, w.hq), float("nan"), dtype=torch.float32, device="cuda")
    layer.merge(dev.sinks, out, lse)
    torch.cuda.synchronize()
    assert int(layer.status.item()) == 0 and int(dev.status.item()) == 0
    ref, ref_lse = oracle_attn(case, 0)
    assert_close(out.float().cpu().numpy().astype(np.float64), ref, "context-sharded, world %d" % world)
    assert np.all(np.abs(lse.cpu().numpy() - ref_lse) <= 2e-3)


def test_partial_is_float32_attention_over_the_local_keys_without_sink():
    import paper_2602_11937_b200 as P
    from gpu_helpers import DeviceCase
    case = _case("ragged")
    dev = DeviceCase(case)
    dev.append(); oracle_append(case)
    w = case["w"]
    d = dev.desc(0)
    ws = torch.zeros(P.puzzle_decode_attn_workspace_bytes(d, w.batch, 0), dtype=torch.uint8, device="cuda")
    P.puzzle_decode_attn_workspace_init(d, w.batch, ws)
    o = torch.full((w.batch, w.hq, w.head_dim), float("nan"), dtype=torch.float32, device="cuda")
    lse = torch.full((w.batch, w.hq), float("nan"), dtype=torch.float32, device="cuda")
    for splits in (0, 3):
        P.puzzle_decode_attn_partial(d, dev.view(), dev.q, o, lse, num_splits=splits, workspace=ws)
        torch.cuda.synchronize()
        ref, ref_lse = oracle_attn(case, 0, sinks=None)
        err = np.abs(o.cpu().numpy().astype(np.float64) - ref).max()
        assert err <= 2e-4, err            # float32 output: none of the bf16 rounding, only the kernel's arithmetic
        got_lse = lse.cpu().numpy()
        assert np.isneginf(got_lse[1]).all() and not o[1].any()      # the empty sequence
        fin = np.isfinite(ref_lse)
        assert np.all(np.abs(got_lse[fin] - ref_lse[fin]) <= 1e-4)
    import ctypes
    lib = P.binding._load()                    # the lse is what the merge weighs by: a NULL one is refused
    v = dev.view()
    st = lib.puzzle_decode_attn_partial(ctypes.byref(d), ctypes.byref(v), ctypes.c_void_p(dev.q.data_ptr()),
                                        ctypes.c_void_p(o.data_ptr()), None, w.batch, 0, ctypes.c_void_p(ws.data_ptr()),
                                        ws.numel(), None, None)
    assert st == 1                             # PUZZLE_ERR_NULL


@pytest.mark.parametrize("world", [2, 8])
def test_kv_head_sharding_needs_no_exchange(world):
    """Tensor parallelism over KV heads: a rank's cache holds its heads only; its rows equal the full result's."""
    import paper_2602_11937_b200 as P
    from gpu_helpers import DeviceCase, assert_close
    from paper_2602_11937_b200.parallel import head_slice
    case = make_case(synth.workload(2, scale=0.125))          # paged, batch 4, context 1024
    dev = DeviceCase(case)
    dev.append(); oracle_append(case)
    ref, _ = oracle_attn(case, 0)
    w = case["w"]
    for r in range(world):
        kvs, qs = head_slice(r, world, w.hkv, w.hq // w.hkv)
        kc, vc = dev.k_cache[:, kvs].contiguous(), dev.v_cache[:, kvs].contiguous()
        ksc, vsc = dev.k_scale[kvs].contiguous(), dev.v_scale[kvs].contiguous()   # the view keeps raw pointers
        view = P.kv_view(kc, vc, dev.seq_lens, block_table=dev.table, max_blocks_per_seq=w.blocks_per_seq,
                         k_scale=ksc, v_scale=vsc)
        d = P.layer_desc(window=0, num_q_heads=w.hq // world, num_kv_heads=w.hkv // world)
        ws = torch.zeros(P.puzzle_decode_attn_workspace_bytes(d, w.batch, 0), dtype=torch.uint8, device="cuda")
        P.puzzle_decode_attn_workspace_init(d, w.batch, ws)
        out = torch.empty(w.batch, w.hq // world, w.head_dim, dtype=torch.bfloat16, device="cuda")
        P.puzzle_decode_attn(d, view, dev.q[:, qs].contiguous(), dev.sinks[qs].contiguous(), out, None, workspace=ws)
        torch.cuda.synchronize()
        assert_close(out.float().cpu().numpy().astype(np.float64), ref[:, qs], "TP rank %d of %d" % (r, world))


def test_strided_merge_argument_errors():
    import paper_2602_11937_b200 as P
    part = torch.zeros(2 * 64 * 65, dtype=torch.float32, device="cuda")
    out = torch.empty(1, 64, 64, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(P.PuzzleError) as e:      # odd stride between parts: rows are read two floats at a time
        P.puzzle_attn_merge_strided(part, part[64 * 64:], 64, 64 * 65 - 1, 1, 64 * 65, None, None, out, 2)
    assert e.value.code == 2

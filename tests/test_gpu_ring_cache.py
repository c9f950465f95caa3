"""A window layer on a ring of ceil(W/16)+1 blocks per sequence, decoded step by step (append + attention),
against the oracle on an ordinary cache that keeps every token: same bf16 outputs within 2e-3, and the ring's
blocks hold exactly the bytes of the most recent logical blocks."""
import numpy as np
import pytest
import torch

import oracle
from helpers import bf16_bits

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("window", [1, 17, 100, 128])
def test_ring_cache_decodes_like_a_cache_that_keeps_everything(window):
    import paper_2602_11937_b200 as P
    steps, batch, hkv, hq, d = 330, 3, 8, 64, 64
    starts = [0, 5, 41]                                   # sequence b receives its first token at step starts[b]
    max_blocks = (steps + 15) // 16
    r = P.window_ring_blocks(window)
    g = torch.Generator().manual_seed(1234 + window)
    k_scale = (torch.rand(hkv, generator=g) * 0.02 + 0.005).float()
    v_scale = (torch.rand(hkv, generator=g) * 0.02 + 0.005).float()
    sinks = torch.randn(hq, generator=g)
    # device side: the ring
    desc = P.layer_desc(window=window)
    ring_k = torch.zeros(batch * r, hkv, 16, d, dtype=torch.uint8, device="cuda")
    ring_v = torch.zeros_like(ring_k)
    table = P.ring_block_table(batch, window, max_blocks, device="cuda")
    lens_dev = torch.zeros(batch, dtype=torch.int32, device="cuda")
    ks_dev, vs_dev, sinks_dev = k_scale.cuda(), v_scale.cuda(), sinks.cuda()   # the view keeps raw pointers
    view = P.kv_view(ring_k, ring_v, lens_dev, block_table=table, k_scale=ks_dev, v_scale=vs_dev)
    ws = torch.zeros(P.puzzle_decode_attn_workspace_bytes(desc, batch, 0), dtype=torch.uint8, device="cuda")
    P.puzzle_decode_attn_workspace_init(desc, batch, ws)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    out = torch.empty(batch, hq, d, dtype=torch.bfloat16, device="cuda")
    # oracle side: every block kept
    lin_k = np.zeros((batch * max_blocks, hkv, 16, d), dtype=np.uint8)
    lin_v = np.zeros_like(lin_k)
    lin_table = P.linear_block_table(batch, max_blocks).numpy()
    worst = 0.0
    for t in range(steps):
        lens = np.array([max(0, t + 1 - s) for s in starts], dtype=np.int32)
        q = torch.randn(batch, hq, d, generator=g).to(torch.bfloat16)
        k_new = torch.randn(batch, hkv, d, generator=g).to(torch.bfloat16)
        v_new = torch.randn(batch, hkv, d, generator=g).to(torch.bfloat16)
        lens_dev.copy_(torch.from_numpy(lens))
        P.puzzle_kv_append(desc, view, k_new.cuda(), v_new.cuda(), dev_status=status)
        P.puzzle_decode_attn(desc, view, q.cuda(), sinks_dev, out, None, workspace=ws, dev_status=status)
        oracle.kv_append(lin_k, lin_v, oracle.KV_FP8_E4M3, 16, lin_table, max_blocks, lens, k_scale.numpy(),
                         v_scale.numpy(), bf16_bits(k_new), bf16_bits(v_new))
        if t % 7 == 0 or t >= steps - 20:
            ref, _ = oracle.decode_attn(lin_k, lin_v, oracle.KV_FP8_E4M3, lin_table, max_blocks, lens, k_scale.numpy(),
                                        v_scale.numpy(), bf16_bits(q), sinks.numpy(), window, d ** -0.5)
            got = out.float().cpu().numpy().astype(np.float64).reshape(ref.shape)
            err = np.abs(got - ref)
            bound = 2e-3 + np.where(np.abs(ref) >= 1.0, 2.0 ** -8 * np.abs(ref), 0.0)
            assert (err <= bound).all(), "step %d: |err| %.3e" % (t, err.max())
            worst = max(worst, float(err.max()))
    assert int(status.item()) == 0
    # the ring holds the last blocks of every sequence, byte for byte
    gk, gv = ring_k.cpu().numpy(), ring_v.cpu().numpy()
    for b in range(batch):
        last = (int(lens[b]) - 1) // 16
        for j in range(max(0, last - r + 2), last + 1):      # the blocks that can still hold visible tokens
            slot = b * r + j % r
            n = 16 if j < last else (int(lens[b]) - 1) % 16 + 1
            assert np.array_equal(gk[slot][:, :n], lin_k[b * max_blocks + j][:, :n])
            assert np.array_equal(gv[slot][:, :n], lin_v[b * max_blocks + j][:, :n])
    assert ring_k.shape[0] == batch * r and r < max_blocks   # the capacity saving: r blocks instead of max_blocks

"""CPU tests of the block-table helpers (ring tables for window layers)."""
import torch


def test_ring_table_arithmetic():
    import paper_2602_11937_b200 as P
    assert P.window_ring_blocks(128) == 9 and P.window_ring_blocks(1) == 2 and P.window_ring_blocks(8192) == 513
    t = P.ring_block_table(2, 100, 20, first_block=50)
    assert t.shape == (2, 20) and t.dtype == torch.int32
    assert t[0, :8].tolist() == list(range(50, 58)) and t[0, 8].item() == 50 and t[1, 0].item() == 58
    # at every length the blocks that hold visible tokens map to distinct slots
    for window in (1, 16, 17, 100, 128):
        r = P.window_ring_blocks(window)
        for L in range(1, 600):
            lo = max(0, L - window)
            blocks = range(lo // 16, (L - 1) // 16 + 1)
            assert len({j % r for j in blocks}) == len(blocks)
    # 36-layer parent pattern at 64K context, batch 16: blocks kept by ring layers vs by full layers
    need = P.cache_blocks([0, 128] * 18, 16, 4096)
    assert need[0] == 16 * 4096 and need[1] == 16 * 9


def test_multi_token_args_against_enumeration():
    import paper_2602_11937_b200 as P
    lens = torch.tensor([700, 2, 4, 333, 129, 0], dtype=torch.int32)
    table = torch.arange(6 * 5, dtype=torch.int32).reshape(6, 5)
    for n_q, q_lens in ((1, None), (4, None), (4, torch.tensor([4, 2, 4, 3, 0, 1], dtype=torch.int32))):
        l2, t2 = P.multi_token_args(lens, table, n_q, q_lens=q_lens)
        assert l2.dtype == torch.int32 and l2.shape == (6 * n_q,) and t2.shape == (6 * n_q, 5)
        for b in range(6):
            ql = n_q if q_lens is None else int(q_lens[b])
            for i in range(n_q):
                # query row i sits at position L - ql + i and sees the keys up to and including itself
                want = max(0, int(lens[b]) - ql + i + 1) if i < ql else 0
                assert int(l2[b * n_q + i]) == want
                assert torch.equal(t2[b * n_q + i], table[b])
    # without a table the rows address the contiguous layout
    _, t2 = P.multi_token_args(lens, None, 2, max_blocks_per_seq=5)
    assert torch.equal(t2[0], torch.arange(5, dtype=torch.int32)) and torch.equal(t2[3], torch.arange(5, 10, dtype=torch.int32))

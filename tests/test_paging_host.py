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

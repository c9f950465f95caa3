"""GPU parity of the second split-KV kernel (puzzle_decode_attn_tcgen05: E4M3 codes fed straight to the
tcgen05 tensor cores, accumulators in tensor memory) against the float64 oracle, on the same seeded cases
and to the same bars as the default kernel: |err| <= 2e-3 (+ 2^-8 |ref| where |ref| >= 1, and everywhere on
the workload whose K/V are scaled up); lse within 2e-3.  Tiles are 128 tokens here, so the edge lengths also
straddle 128 and 256.
"""
import numpy as np
import pytest
import torch

import oracle
import synth
from helpers import make_case, oracle_append, oracle_attn
from test_gpu_parity import _dev, _run_and_compare

pytestmark = pytest.mark.gpu

K = "tcgen05"


def test_config1_full_contiguous():
    _run_and_compare(make_case(synth.workload(1)), 0, kernel=K)
    _run_and_compare(make_case(synth.workload(1)), 0, num_splits=3, kernel=K)


@pytest.mark.parametrize("window", [0, 128])
def test_config2_paged_full_and_window(window):
    w = synth.workload(2, scale=0.25)
    _run_and_compare(make_case(w, layer=0 if window == 0 else 1), window, kernel=K)


@pytest.mark.parametrize("num_splits", [0, 8, 64])
def test_config3_scaled_kv_split_sweep(num_splits):
    w = synth.workload(3, scale=0.125)
    _run_and_compare(make_case(w), 0, num_splits=num_splits, rel=True, kernel=K)


@pytest.mark.parametrize("layer,window", [(0, 128), (1, 0), (2, 1000)])
def test_config4_ragged_layers(layer, window):
    w = synth.workload(4, scale=0.05)
    _run_and_compare(make_case(w, layer=layer), window, kernel=K)


def test_config5_long_context():
    w = synth.workload(5, scale=0.04)
    w.batch = 2
    _run_and_compare(make_case(w, layer=1), 0, kernel=K)
    _run_and_compare(make_case(w, layer=0), 128, kernel=K)


EDGE_LENS = [0, 1, 15, 16, 17, 63, 64, 65, 127, 128, 129, 200, 255, 256, 257, 300]


@pytest.mark.parametrize("window", [0, 1, 16, 17, 100, 129, 1000])
@pytest.mark.parametrize("num_splits", [0, 1, 3])
def test_edge_lengths_with_poisoned_tail(window, num_splits):
    w = synth.Workload("edges128", 1, len(EDGE_LENS), 300, [0], paged=True)
    case = make_case(w, seq_lens=EDGE_LENS, poison_tail=True)
    _run_and_compare(case, window, num_splits=num_splits, kernel=K)


def test_no_sinks_and_empty_context():
    from gpu_helpers import assert_close
    w = synth.Workload("nosink", 1, 4, 90, [0], paged=True)
    case = make_case(w, seq_lens=[90, 0, 1, 64])
    dev = _dev(case)
    dev.append(); oracle_append(case)
    got, lse = dev.attn(window=0, sinks=None, kernel=K)
    ref, _ = oracle_attn(case, 0, sinks=None)
    assert_close(got, ref, "no sinks")
    assert np.all(np.isneginf(lse[1])) and not got[1].any()
    got, lse = dev.attn(window=0, kernel=K)
    assert not got[1].any() and np.allclose(lse[1], case["sinks"], atol=1e-6)


def test_no_scales_and_pow2_scales():
    w = synth.workload(1, scale=0.5)
    _run_and_compare(make_case(w, no_scales=True), 0, kernel=K)
    _run_and_compare(make_case(w, pow2_scales=True), 0, kernel=K)


def test_stale_out_of_window_table_entries_are_never_read():
    from gpu_helpers import assert_close
    w = synth.Workload("stale", 1, 3, 700, [0], paged=True)
    case = make_case(w, seq_lens=[700, 400, 129])
    ref_case = dict(case, table=case["table"].copy())
    for b, L in enumerate([700, 400, 129]):
        case["table"][b, :(L - 128) // 16] = -1
    dev = _dev(case)
    dev.append(); oracle_append(ref_case)
    got, _ = dev.attn(window=128, kernel=K)
    ref, _ = oracle_attn(ref_case, 128)
    assert_close(got, ref, "stale table")
    assert int(dev.status.item()) == 0


def test_device_side_errors_are_flagged_not_faulted():
    import paper_2602_11937_b200 as P
    w = synth.Workload("bad", 1, 2, 100, [0], paged=True)
    case = make_case(w, seq_lens=[100, 100])
    case["table"][0, 2] = case["num_blocks"] + 5
    case["table"][1, 1] = -3
    dev = _dev(case)
    got, _ = dev.attn(window=0, kernel=K)
    assert int(dev.status.item()) & P.DEV_BAD_BLOCK
    assert np.isfinite(got).all()
    dev.status.zero_()
    too_long = torch.tensor([100, 5000], dtype=torch.int32, device="cuda")
    dev.attn(window=0, seq_lens=too_long, kernel=K)
    assert int(dev.status.item()) & P.DEV_SEQ_TOO_LONG


def test_bf16_cache_is_refused_before_any_launch():
    import paper_2602_11937_b200 as P
    w = synth.workload(1, scale=0.25)
    dev = _dev(make_case(w, kv_dtype=oracle.KV_BF16))
    before = P.puzzle_launch_count()
    with pytest.raises(P.PuzzleError) as e:
        dev.attn(window=0, kernel=K)
    assert e.value.code == 3 and P.puzzle_launch_count() == before   # PUZZLE_ERR_UNSUPPORTED


def test_full_size_64k_context_sampled():
    """Batch 16, context 65536, paged random table: the balanced schedule the bench times, and 8 explicit splits."""
    from test_gpu_fullsize import FullCase
    case = FullCase(synth.workload(3), 0)
    case.append_and_check()
    for s in (0, 8):
        case.attn_and_check(0, num_splits=s, rel=True, seed=s, kernel=K)


def test_full_size_ragged_layer_kinds_sampled():
    from test_gpu_fullsize import FullCase
    case = FullCase(synth.workload(4), 1)
    case.append_and_check()
    for window in (0, 128, 8192):
        case.attn_and_check(window, seed=window, kernel=K)

"""The entry point for callers that cannot allocate device memory (puzzle_decode_attn_static).

Collected last on purpose: a run that stops at the first failure has then already run every other test.
It goes through the C ABI like the other GPU tests and compares the built-in-scratch variant with
puzzle_decode_attn on a caller-owned workspace (same kernel, same inputs) and with the CPU oracle, all
within the attention tolerance.  Two calls in a row check that the shared array is left usable; other
shapes and split choices reuse it; an oversized request is refused; and once the first call has been
made, a call does not change the free device memory.
"""
import numpy as np
import pytest
import torch

import synth
from gpu_helpers import assert_close
from helpers import make_case, oracle_append, oracle_attn

pytestmark = pytest.mark.gpu

TOL = 2e-3


def _same(got, want):
    """Two runs of the kernel on the same inputs: both are bf16 roundings of float32 sums taken in slightly
    different orders, so they agree within the attention tolerance plus one bf16 step of the value."""
    return np.all(np.abs(got - want) <= TOL + 2.0 ** -7 * np.abs(want))


def _setup(w, window, layer=0, seq_lens=None):
    import paper_2602_11937_b200 as P
    from gpu_helpers import DeviceCase
    case = make_case(w, layer=layer, seq_lens=seq_lens)
    dev = DeviceCase(case)
    dev.append()
    want, want_lse = dev.attn(window=window)             # existing entry point, workspace from torch
    oracle_append(case)                                   # the oracle's cache gets the same token
    ref, ref_lse = oracle_attn(case, window)
    assert_close(want, ref, "workspace entry point against the oracle")
    return P, dev, want, want_lse, ref


def _static(P, dev, window, num_splits=0):
    w = dev.w
    out = torch.full((w.batch, w.hq, w.head_dim), float("nan"), dtype=torch.bfloat16, device="cuda")
    lse = torch.full((w.batch, w.hq), float("nan"), dtype=torch.float32, device="cuda")
    P.puzzle_decode_attn_static(dev.desc(window), dev.view(), dev.q, dev.sinks, out, lse, num_splits=num_splits,
                                dev_status=dev.status)
    torch.cuda.synchronize()
    return out.float().cpu().numpy().astype(np.float64), lse.cpu().numpy().astype(np.float64)


@pytest.mark.parametrize("window", [0, 128])
def test_static_scratch_matches_workspace_entry_point_twice_in_a_row(window):
    w = synth.workload(2, scale=0.1)                      # batch 3, context 819, paged
    P, dev, want, want_lse, ref = _setup(w, window, layer=0 if window == 0 else 1)
    free = []
    for call in range(3):
        got, got_lse = _static(P, dev, window)
        assert _same(got, want), "call %d" % call
        assert np.all(np.abs(got_lse - want_lse) <= TOL), "call %d" % call
        assert_close(got, ref, "static entry point against the oracle, call %d" % call)
        free.append(torch.cuda.mem_get_info()[0])
    assert free[1] == free[2]          # nothing is allocated once the array's address is known
    assert int(dev.status.item()) == 0


def test_static_scratch_other_shape_and_explicit_splits_reuse_the_array():
    w = synth.Workload("static_edges", 1, 5, 200, [0], paged=True)
    P, dev, want, want_lse, ref = _setup(w, 0, seq_lens=[200, 0, 1, 64, 129])
    for num_splits in (0, 3, 0):
        got, got_lse = _static(P, dev, 0, num_splits)
        assert _same(got, want)
        assert_close(got, ref, "static entry point against the oracle, %d splits" % num_splits)
        fin = np.isfinite(want_lse)
        assert np.array_equal(np.isfinite(got_lse), fin) and np.all(np.abs(got_lse[fin] - want_lse[fin]) <= TOL)


def test_static_scratch_refuses_what_does_not_fit():
    w = synth.Workload("static_big", 1, 2, 64, [0], paged=True)
    P, dev, _, _, _ = _setup(w, 0)
    d = dev.desc(0)
    assert P.puzzle_decode_attn_workspace_bytes(d, 2, 4096) > P.STATIC_SCRATCH_BYTES
    out = torch.empty(2, 64, 64, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(P.PuzzleError) as e:
        P.puzzle_decode_attn_static(d, dev.view(), dev.q, dev.sinks, out, None, num_splits=4096)
    assert e.value.code == 4                               # PUZZLE_ERR_WORKSPACE, nothing launched
    torch.cuda.synchronize()

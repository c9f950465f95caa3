"""Seeded random decode steps (batch, ragged lengths, window, split count, KV-head count, paging, sink, cache type,
kernel) through the C ABI against the float64 oracle: appended bytes exact, outputs within 2e-3.  The fixed cases
elsewhere pick their shapes by hand; these pick them blindly."""
import numpy as np
import pytest
import torch

import oracle
import synth
from helpers import make_case, oracle_append, oracle_attn

pytestmark = pytest.mark.gpu


def _draw(seed):
    r = np.random.default_rng(9000 + seed)
    hkv = int(r.choice([1, 2, 4, 8]))
    batch = int(r.integers(1, 10))
    context = int(r.choice([40, 130, 300, 700, 1500]))
    lens = [int(x) for x in r.integers(0, context + 1, size=batch)]
    if r.random() < 0.3:
        lens[int(r.integers(batch))] = context
    window = int(r.choice([0, 0, 1, 15, 16, 64, 127, 128, 129, 500, 5000]))
    splits = int(r.choice([0, -1, -1, -2, 1, 2, 5, 17]))   # -1 / -2 pin the kernel of the balanced schedule
    kv = oracle.KV_BF16 if r.random() < 0.3 else oracle.KV_FP8_E4M3
    kernel = "tcgen05" if (kv == oracle.KV_FP8_E4M3 and splits != -1 and r.random() < 0.4) else "mma"
    return dict(hkv=hkv, batch=batch, context=context, lens=lens, window=window, splits=splits, kv=kv, kernel=kernel,
                paged=bool(r.random() < 0.7), sinks=bool(r.random() < 0.7), pow2=bool(r.random() < 0.3))


@pytest.mark.parametrize("seed", range(60))
def test_random_decode_step(seed):
    from gpu_helpers import DeviceCase, assert_close
    c = _draw(seed)
    w = synth.Workload("random%d" % seed, 1, c["batch"], c["context"], [0], paged=c["paged"], hq=8 * c["hkv"], hkv=c["hkv"])
    case = make_case(w, seq_lens=c["lens"], kv_dtype=c["kv"], pow2_scales=c["pow2"], poison_tail=True)
    dev = DeviceCase(case)
    dev.append()
    oracle_append(case)
    gk, gv = dev.cache_bytes()
    assert np.array_equal(gk, case["k_cache"]) and np.array_equal(gv, case["v_cache"]), c
    sinks = "case" if c["sinks"] else None
    got, lse = dev.attn(window=c["window"], num_splits=c["splits"], sinks=sinks, kernel=c["kernel"])
    ref, ref_lse = oracle_attn(case, c["window"], sinks="case" if c["sinks"] else None)
    assert int(dev.status.item()) == 0, c
    assert_close(got, ref, str(c))
    fin = np.isfinite(ref_lse)
    assert np.array_equal(np.isfinite(lse), fin), c
    assert np.all(np.abs(lse[fin] - ref_lse[fin]) <= 2e-3), c

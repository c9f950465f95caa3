"""GPU max calibration (amax update + scales) against the oracle: bit-exact float32 scales.

The oracle reads float32 copies of the same bf16 samples (bf16 -> float32 is exact)."""
import numpy as np
import pytest
import torch

import oracle

pytestmark = pytest.mark.gpu


def _samples(n_tokens, hkv, d, seed, spread=True):
    g = torch.Generator().manual_seed(seed)
    x = torch.randn(n_tokens, hkv, d, generator=g)
    if spread:
        x = x * torch.linspace(0.05, 6.0, hkv)[None, :, None]
    return x.to(torch.bfloat16)


def _oracle(x, pow2):
    return oracle.calibrate_scales(x.float().numpy(), pow2=pow2)


@pytest.mark.parametrize("pow2", [False, True])
@pytest.mark.parametrize("n_tokens,hkv,d", [(1, 8, 64), (37, 8, 64), (5000, 8, 64), (333, 3, 64), (129, 8, 128),
                                            (64, 64, 8), (200001, 8, 64)])
def test_scales_match_the_oracle_bit_for_bit(n_tokens, hkv, d, pow2):
    import paper_2602_11937_b200 as P
    x = _samples(n_tokens, hkv, d, seed=n_tokens + hkv)
    got = P.calibrate_scales([x.cuda()], hkv, pow2=pow2).cpu().numpy()
    ref = _oracle(x, pow2)
    assert got.dtype == np.float32 and np.array_equal(got.view(np.uint32), ref.view(np.uint32))


def test_chunks_accumulate_and_special_values():
    import paper_2602_11937_b200 as P
    x = _samples(4096, 8, 64, seed=7)
    x[:, 2, :] = 0                          # an all-zero head keeps scale 1
    x[10, 5, 3] = float("nan")              # NaNs are skipped
    x[11, 6, 0] = -1000.0                   # a negative outlier sets the maximum
    x[12, 1, 63] = torch.finfo(torch.bfloat16).tiny / 64   # subnormal values are ordinary magnitudes
    xs = [x[:100].cuda(), x[100:100].cuda(), x[100:3000].cuda(), x[3000:].cuda()]   # one chunk is empty
    for pow2 in (False, True):
        got = P.calibrate_scales(xs, 8, pow2=pow2).cpu().numpy()
        ref = _oracle(x, pow2)
        assert np.array_equal(got.view(np.uint32), ref.view(np.uint32))
        assert got[2] == 1.0
        if not pow2:
            assert got[6] == np.float32(1000.0) / np.float32(448.0)
    # tiny maxima: the quotient is a float32 subnormal; the round-up stays a power of two
    tiny = torch.zeros(4, 2, 64, dtype=torch.bfloat16)
    tiny[0, 0, 0] = 2.0 ** -130
    tiny[1, 1, 5] = 3 * 2.0 ** -133
    got = P.calibrate_scales([tiny.cuda()], 2, pow2=True).cpu().numpy()
    ref = _oracle(tiny, True)
    assert np.array_equal(got.view(np.uint32), ref.view(np.uint32))
    inf = torch.zeros(2, 1, 64, dtype=torch.bfloat16)
    inf[1, 0, 9] = float("-inf")
    assert np.isposinf(P.calibrate_scales([inf.cuda()], 1).cpu().numpy()[0])


def test_scales_from_amax_in_place_and_argument_errors():
    import paper_2602_11937_b200 as P
    amax = torch.tensor([448.0, 0.0, 1.0, 896.0], device="cuda")
    P.puzzle_kv_scales_from_amax(amax, amax, pow2=True)
    assert amax.cpu().tolist() == [1.0, 1.0, 2.0 ** -8, 2.0]
    x = torch.zeros(4, 8, 60, dtype=torch.bfloat16, device="cuda")      # head_dim not a multiple of 8
    with pytest.raises(P.PuzzleError) as e:
        P.puzzle_kv_amax_update(x, torch.zeros(8, device="cuda"))
    assert e.value.code == 2
    x = torch.zeros(4, 65, 8, dtype=torch.bfloat16, device="cuda")      # too many heads
    with pytest.raises(P.PuzzleError):
        P.puzzle_kv_amax_update(x, torch.zeros(65, device="cuda"))


def test_calibrated_scales_feed_the_append_bit_exactly():
    """Calibrate on the device, append with those scales, compare the bytes with the oracle's."""
    import paper_2602_11937_b200 as P
    import synth
    from helpers import make_case, oracle_append
    from gpu_helpers import DeviceCase
    case = make_case(synth.workload(1, scale=0.25))
    dev = DeviceCase(case)
    calib = _samples(2048, case["k_scale"].shape[0], 64, seed=3)
    ks = P.calibrate_scales([calib.cuda()], calib.shape[1], pow2=True)
    vs = P.calibrate_scales([(calib * 0.5).cuda()], calib.shape[1], pow2=False)
    dev.k_scale, dev.v_scale = ks, vs
    case["k_scale"], case["v_scale"] = _oracle(calib, True), _oracle(calib * 0.5, False)
    dev.append()
    oracle_append(case)
    gk, gv = dev.cache_bytes()
    assert np.array_equal(gk, case["k_cache"]) and np.array_equal(gv, case["v_cache"])

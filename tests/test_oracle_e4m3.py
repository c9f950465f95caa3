"""Pins for the oracle's E4M3 codec, calibration and append (CPU only).

Each pin is something the format or the mathematics fixes independently of
the oracle's own code: printed code values, exhaustive round trip, a
brute-force nearest search written here, the library's own cast inside its
range, and closed forms for power-of-two scales.
"""
import math
import os

import numpy as np
import pytest
import torch

import oracle
import synth
from helpers import bf16_bits, bf16_bits_to_f64, make_case, oracle_append

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _all_bf16_as_f32():
    bits = np.arange(65536, dtype=np.uint32)
    return (bits << 16).view(np.float32)


def test_golden_code_values():
    n = 0
    for line in open(os.path.join(GOLDEN, "e4m3_code_values.txt")):
        if line.startswith("#") or not line.strip():
            continue
        code, val = line.split()
        got = oracle.e4m3_decode(int(code, 16))
        assert got == float(val), (code, got)
        assert math.copysign(1.0, got) == math.copysign(1.0, float(val))
        n += 1
    assert n >= 12


def test_decode_closed_form_and_monotone():
    prev = -1.0
    for c in range(0x7F):
        e, m = (c >> 3) & 15, c & 7
        want = (m / 8.0) * 2.0 ** -6 if e == 0 else (1 + m / 8.0) * 2.0 ** (e - 7)
        assert oracle.e4m3_decode(c) == want
        assert oracle.e4m3_decode(c | 0x80) == -want
        assert want > prev
        prev = want
    assert math.isnan(oracle.e4m3_decode(0x7F)) and math.isnan(oracle.e4m3_decode(0xFF))


def test_round_trip_all_codes():
    for c in range(256):
        if c & 0x7F == 0x7F:
            continue
        assert oracle.e4m3_encode(oracle.e4m3_decode(c)) == c


def test_midpoints_go_to_even_and_neighbours_to_nearest():
    for c in range(0x7E):
        lo, hi = oracle.e4m3_decode(c), oracle.e4m3_decode(c + 1)
        mid = np.float32((lo + hi) / 2)  # exact: one more bit than the codes have
        assert float(mid) == (lo + hi) / 2
        even = c if c % 2 == 0 else c + 1
        assert oracle.e4m3_encode(float(mid)) == even
        assert oracle.e4m3_encode(float(np.nextafter(mid, np.float32(0)))) == c
        assert oracle.e4m3_encode(float(np.nextafter(mid, np.float32(1e9)))) == c + 1
        assert oracle.e4m3_encode(-float(mid)) == even | 0x80
    assert oracle.e4m3_encode(1.0625) == 0x38 and oracle.e4m3_encode(1.1875) == 0x3A


def test_saturation_nan_zero():
    for y in (448.0, 449.0, 463.9, 464.0, 480.0, 1e30, float("inf")):
        assert oracle.e4m3_encode(y) == 0x7E
        assert oracle.e4m3_encode(-y) == 0xFE
    assert oracle.e4m3_encode(float("nan")) == 0x7F and oracle.e4m3_encode(-float("nan")) == 0x7F
    assert oracle.e4m3_encode(0.0) == 0x00 and oracle.e4m3_encode(-0.0) == 0x80
    assert oracle.e4m3_encode(2.0 ** -10) == 0x00          # tie between 0 and 2^-9 -> even (0)
    assert oracle.e4m3_encode(float(np.nextafter(np.float32(2.0 ** -10), np.float32(1)))) == 0x01
    assert oracle.e4m3_encode(-1e-30) == 0x80


def test_exhaustive_bf16_vs_bruteforce_nearest():
    """All 65 536 bf16 inputs against a nearest-with-ties-to-even search written here."""
    x = _all_bf16_as_f32()
    got = oracle.e4m3_encode_array(x)
    book = np.array([(m / 8.0) * 2.0 ** -6 if e == 0 else (1 + m / 8.0) * 2.0 ** (e - 7)
                     for e in range(16) for m in range(8)][:0x7F], dtype=np.float64)
    for i in range(65536):
        xi = float(x[i])
        if math.isnan(xi):
            assert got[i] == 0x7F
            continue
        a = abs(xi)
        if a >= 448.0:
            want = 0x7E
        else:
            dist = np.abs(book - a)
            best = np.flatnonzero(dist == dist.min())
            want = int(best[0]) if len(best) == 1 else int([b for b in best if b % 2 == 0][0])
        if math.copysign(1.0, xi) < 0:
            want |= 0x80
        assert got[i] == want, (i, xi, got[i], want)


def test_matches_library_cast_inside_range():
    """torch's float8_e4m3fn cast rounds to nearest even too; it is only defined up to 448."""
    x = _all_bf16_as_f32()
    x = x[np.isfinite(x) & (np.abs(x) <= 448.0)]
    want = torch.from_numpy(x.copy()).to(torch.float8_e4m3fn).view(torch.uint8).numpy()
    got = oracle.e4m3_encode_array(x)
    assert np.array_equal(got, want)
    back = torch.from_numpy(got.copy()).view(torch.float8_e4m3fn).to(torch.float64).numpy()
    mine = np.array([oracle.e4m3_decode(int(c)) for c in got])
    assert np.array_equal(back, mine)


def test_calibration():
    rng = np.random.default_rng(1)
    x = rng.standard_normal((300, 8, 64)).astype(np.float32) * np.linspace(0.5, 4, 8, dtype=np.float32)[None, :, None]
    s = oracle.calibrate_scales(x)
    amax = np.abs(x).max(axis=(0, 2))
    assert np.array_equal(s, (amax / np.float32(448.0)).astype(np.float32))
    p = oracle.calibrate_scales(x, pow2=True)
    assert np.all(p >= s) and np.all(p < 2 * s)
    assert np.all(np.log2(p) == np.round(np.log2(p)))
    assert np.all(p < 1.0)  # the paper notes that all its scales are below one
    x[:, 3, :] = 0
    assert oracle.calibrate_scales(x)[3] == 1.0
    exact = np.zeros((1, 1, 4), dtype=np.float32)
    exact[0, 0, 1] = 448.0 * 0.25
    assert oracle.calibrate_scales(exact, pow2=True)[0] == 0.25  # already a power of two: unchanged


@pytest.mark.parametrize("k", [0, -3, 2])
def test_append_pow2_scale_is_exponent_shift(k):
    """With scale 2^k the quotient is exact, so append == encode(x * 2^-k) for every bf16 x."""
    bits = np.arange(65536, dtype=np.uint16)
    w = synth.Workload("all_bf16", 1, 65536 // (8 * 64), 16, [0], paged=False)
    nb = w.batch * w.blocks_per_seq
    kc = np.zeros((nb, 8, 16, 64), dtype=np.uint8)
    vc = np.zeros_like(kc)
    lens = np.full(w.batch, 5, dtype=np.int32)
    scale = np.full(8, 2.0 ** k, dtype=np.float32)
    knew = bits.reshape(w.batch, 8, 64)
    oracle.kv_append(kc, vc, oracle.KV_FP8_E4M3, 16, None, 1, lens, scale, None, knew, knew[::-1].copy())
    x = bf16_bits_to_f64(bits)
    with np.errstate(over="ignore", invalid="ignore"):
        want_k = oracle.e4m3_encode_array((x * 2.0 ** -k).astype(np.float32))
    assert np.array_equal(kc[:, :, 4, :].reshape(-1), want_k)
    want_v = oracle.e4m3_encode_array(bf16_bits_to_f64(knew[::-1].reshape(-1)).astype(np.float32))
    assert np.array_equal(vc[:, :, 4, :].reshape(-1), want_v)  # NULL v_scale == 1
    # nothing else was touched
    kc[:, :, 4, :] = 0
    vc[:, :, 4, :] = 0
    assert not kc.any() and not vc.any()


def test_append_general_scale_against_fraction_arithmetic():
    """Non-power-of-two scale: the float32 quotient must be the correctly rounded one.
    Checked with exact rational arithmetic on a sample of inputs."""
    from fractions import Fraction

    rng = np.random.default_rng(7)
    scale = np.float32(3.1415927 / 448)
    bits = rng.integers(0, 65536, size=512).astype(np.uint16)
    x = bf16_bits_to_f64(bits)
    with np.errstate(invalid="ignore"):
        keep = np.isfinite(x) & (np.abs(x) < 1e6)  # keep the float32 quotient finite
    bits, x = bits[keep][:448], x[keep][:448]
    n = len(bits) // 64 * 64
    bits, x = bits[:n], x[:n]
    w = synth.Workload("frac", 1, n // 64, 16, [0], paged=False, hkv=1)
    kc = np.zeros((w.batch, 1, 16, 64), dtype=np.uint8)
    vc = np.zeros_like(kc)
    lens = np.full(w.batch, 16, dtype=np.int32)
    oracle.kv_append(kc, vc, oracle.KV_FP8_E4M3, 16, None, 1, lens, np.array([scale]), np.array([scale]),
                     bits.reshape(w.batch, 1, 64), bits.reshape(w.batch, 1, 64))
    got = kc[:, 0, 15, :].reshape(-1)
    book = [Fraction(oracle.e4m3_decode(c)) for c in range(0x7F)]
    for i in range(n):
        qf = abs(Fraction(float(x[i])) / Fraction(float(scale)))
        # correctly rounded float32 quotient, via the exact rational
        y = np.float32(float(qf))  # double rounding is harmless here only if we re-check below
        lo, hi = np.nextafter(y, np.float32(0)), np.nextafter(y, np.float32(np.inf))
        cands = sorted({float(lo), float(y), float(hi)}, key=lambda c: abs(Fraction(c) - qf))
        yq = Fraction(cands[0])
        if yq >= 448:
            want = 0x7E
        else:
            d = [abs(b - yq) for b in book]
            m = min(d)
            best = [c for c in range(0x7F) if d[c] == m]
            want = best[0] if len(best) == 1 else [c for c in best if c % 2 == 0][0]
        if x[i] < 0 or (x[i] == 0 and math.copysign(1, x[i]) < 0):
            want |= 0x80
        assert got[i] == want, (i, x[i], got[i], want)


def test_append_paged_slot_and_untouched_bytes():
    w = synth.workload(2, scale=0.08)
    lens = np.array([1, 16, 17, w.context][: w.batch] + [w.context // 2] * max(0, w.batch - 4), dtype=np.int32)
    case = make_case(w, seq_lens=lens[: w.batch])
    before_k, before_v = case["k_cache"].copy(), case["v_cache"].copy()
    oracle_append(case)
    changed = np.zeros(before_k.shape, dtype=bool)
    for b in range(w.batch):
        pos = int(case["seq_lens"][b]) - 1
        blk = case["table"][b, pos // 16]
        changed[blk, :, pos % 16, :] = True
        y = (bf16_bits_to_f64(case["k_new"][b]) / case["k_scale"][:, None].astype(np.float64)).astype(np.float32)
        assert np.array_equal(case["k_cache"][blk, :, pos % 16, :], oracle.e4m3_encode_array(y))
    assert np.array_equal(case["k_cache"][~changed], before_k[~changed])
    assert np.array_equal(case["v_cache"][~changed], before_v[~changed])


def test_append_bf16_kv_is_a_copy():
    w = synth.workload(1, scale=0.25)
    case = make_case(w, kv_dtype=oracle.KV_BF16)
    oracle_append(case)
    for b in range(w.batch):
        pos = int(case["seq_lens"][b]) - 1
        blk = b * w.blocks_per_seq + pos // 16
        assert np.array_equal(case["k_cache"][blk, :, pos % 16, :], case["k_new"][b])
        assert np.array_equal(case["v_cache"][blk, :, pos % 16, :], case["v_new"][b])


def test_fp8_is_half_the_bytes_of_bf16():
    """FP8 KV doubles token capacity (Section "KV Quantization")."""
    w = synth.workload(1, scale=0.25)
    a = make_case(w, kv_dtype=oracle.KV_FP8_E4M3)
    b = make_case(w, kv_dtype=oracle.KV_BF16)
    assert 2 * a["k_cache"].nbytes == b["k_cache"].nbytes

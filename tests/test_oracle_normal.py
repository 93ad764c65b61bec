"""Pins for the oracle's uniform mapping, Box-Muller transform and narrowing (CPU only)."""
import math
import os

import mpmath as mp
import numpy as np
import torch
from scipy import stats

import oracle

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "box_muller_worked.txt")


def _mp_box_muller(xa, xb):
    mp.mp.dps = 50
    u1 = mp.mpf((xa >> 8) + 1) / 2 ** 24
    k = xb >> 8
    rho = mp.sqrt(-2 * mp.log(u1))
    a = 2 * mp.pi * k / 2 ** 24
    return rho * mp.cos(a), rho * mp.sin(a)


def _to_f32(x):
    return np.float32(float(x))


def test_worked_example_from_first_block():
    words = oracle.gen_u32(0, 0, 8)
    z64 = oracle.gen_normal_f64(0, 0, 4)
    z32 = oracle.gen_inputs(0, 0, oracle.F32, 4).view(np.uint32)
    rows = [l for l in open(GOLDEN) if l.strip() and not l.startswith("#")]
    assert len(rows) == 2
    for i, line in enumerate(rows):
        w, uk, zd, zh = [p.split() for p in line.split("|")]
        xa, xb = int(w[0], 16), int(w[1], 16)
        assert (int(words[2 * i]), int(words[2 * i + 1])) == (xa, xb)
        assert (xa >> 8) + 1 == int(uk[0]) and xb >> 8 == int(uk[1])
        for j in range(2):
            assert abs(z64[2 * i + j] - float(zd[j])) <= 4e-16 * abs(float(zd[j]))
            assert int(z32[2 * i + j]) == int(zh[j], 16)


def test_transform_against_50_digit_evaluation():
    # Random word pairs plus angles right next to the axis crossings, where a
    # badly reduced angle loses relative accuracy.
    rng = np.random.default_rng(1)
    pairs = [(int(a), int(b)) for a, b in rng.integers(0, 1 << 32, size=(400, 2))]
    for q in range(4):
        for dk in (-2, -1, 1, 2, 3):
            k = (q * (1 << 22) + dk) % (1 << 24)
            pairs.append((int(rng.integers(0, 1 << 32)), k << 8))
    pairs += [(0, 12345 << 8), (0xFFFFFE00, 999 << 8), (0xFFFFFFFF - 511, 5 << 8)]
    for xa, xb in pairs:
        zc, zs = oracle.box_muller(xa, xb)
        mc, ms = _mp_box_muller(xa, xb)
        for got, want in ((zc, mc), (zs, ms)):
            assert abs(mp.mpf(got) - want) <= mp.mpf(2) ** -50 * abs(want), (hex(xa), hex(xb))


def test_rounded_values_are_the_nearest_float32():
    words = oracle.gen_u32(9, 0, 512)
    z32 = oracle.gen_inputs(9, 0, oracle.F32, 512)
    for i in range(0, 512, 2):
        mc, ms = _mp_box_muller(int(words[i]), int(words[i + 1]))
        assert z32[i] == _to_f32(mc) and z32[i + 1] == _to_f32(ms)


def test_exact_zeros_extremes_and_symmetry():
    for q, (c0, s0) in enumerate([(1, 0), (0, 1), (-1, 0), (0, -1)]):
        zc, zs = oracle.box_muller(0x12345678, (q << 22) << 8)
        rho = math.sqrt(-2 * math.log(((0x12345678 >> 8) + 1) / 2 ** 24))
        assert zc == c0 * rho and zs == s0 * rho          # zeros are exact zeros
    # u1 = 1 -> both outputs are zero; smallest u1 -> the largest radius sqrt(48 ln 2)
    zc, zs = oracle.box_muller(0xFFFFFF00, 0x9ABCDE00)
    assert zc == 0.0 and zs == 0.0
    zc, zs = oracle.box_muller(0, 0)
    assert abs(zc - math.sqrt(48 * math.log(2))) < 1e-14 and zs == 0.0
    # the low 8 bits of each word are unused
    assert oracle.box_muller(0xABCDEF00, 0x13579B00) == oracle.box_muller(0xABCDEFFF, 0x13579BFF)
    # k -> k + 2^23 negates both outputs
    a = oracle.box_muller(0x0F0F0F0F, 0x10203040)
    b = oracle.box_muller(0x0F0F0F0F, (0x10203040 + (1 << 31)) & 0xFFFFFFFF)
    assert a == (-b[0], -b[1])


def test_radius_identity_and_bound():
    words = oracle.gen_u32(3, 0, 1 << 12)
    z = oracle.gen_normal_f64(3, 0, 1 << 12)
    u1 = ((words[0::2] >> 8).astype(np.float64) + 1.0) / 2 ** 24
    np.testing.assert_allclose(z[0::2] ** 2 + z[1::2] ** 2, -2 * np.log(u1), rtol=1e-13, atol=1e-300)
    assert np.abs(z).max() <= math.sqrt(48 * math.log(2))


def test_distribution_is_standard_normal():
    z = oracle.gen_normal_f64(2024, 0, 1 << 20)
    n = z.size
    assert abs(z.mean()) < 5 / math.sqrt(n)
    assert abs(z.var() - 1) < 5 * math.sqrt(2 / n)
    assert abs(stats.kurtosis(z, fisher=False) - 3) < 5 * math.sqrt(24 / n)
    assert stats.kstest(z, "norm").pvalue > 1e-3
    # cosine and sine halves are uncorrelated
    assert abs(np.corrcoef(z[0::2], z[1::2])[0, 1]) < 5 / math.sqrt(n / 2)


def test_normal_stream_slices_like_the_word_stream():
    whole = oracle.gen_inputs(11, 0, oracle.F32, 300)
    for a, n in [(1, 7), (2, 9), (3, 50), (255, 45)]:
        assert np.array_equal(oracle.gen_inputs(11, a, oracle.F32, n), whole[a:a + n])


def test_widen_fp16_bf16_all_patterns():
    bits = np.arange(1 << 16, dtype=np.uint16)
    w16 = oracle.widen(oracle.F16, bits)
    np.testing.assert_array_equal(w16.view(np.uint32), bits.view(np.float16).astype(np.float32).view(np.uint32))
    wb = oracle.widen(oracle.BF16, bits)
    tb = torch.from_numpy(bits.view(np.int16)).view(torch.bfloat16).float().numpy()
    np.testing.assert_array_equal(wb.view(np.uint32), tb.view(np.uint32))


def _nan_safe_equal(a_bits, b_bits, is_nan_mask):
    assert np.array_equal(a_bits[~is_nan_mask], b_bits[~is_nan_mask])


def test_narrow_matches_numpy_and_torch_rounding():
    rng = np.random.default_rng(5)
    x = np.concatenate([
        rng.standard_normal(200000).astype(np.float32),
        (rng.standard_normal(50000) * 1e-6).astype(np.float32),        # fp16 subnormal range
        (rng.standard_normal(50000) * 3e4).astype(np.float32),         # fp16 overflow range
        rng.integers(0, 1 << 32, 200000, dtype=np.uint64).astype(np.uint32).view(np.float32),
    ])
    # every exact tie between neighbouring fp16 values, and between bf16 values
    h = np.arange(0, 0x7C00, dtype=np.uint16)
    lo = h.view(np.float16).astype(np.float64)
    hi = (h + 1).view(np.float16).astype(np.float64)
    mid = ((lo + hi) / 2).astype(np.float32)
    x = np.concatenate([x, mid, -mid, np.float32([65504, 65519.996, 65520, 1e30, np.inf, -np.inf, 0.0, -0.0])])
    nan = np.isnan(x)
    with np.errstate(over="ignore"):
        want16 = x.astype(np.float16).view(np.uint16)
    got16 = oracle.narrow(oracle.F16, x)
    _nan_safe_equal(got16, want16, nan)
    assert np.all(np.isnan(got16[nan].view(np.float16)))
    wantb = torch.from_numpy(x).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    gotb = oracle.narrow(oracle.BF16, x)
    _nan_safe_equal(gotb, wantb, nan)
    assert np.all(np.isnan(oracle.widen(oracle.BF16, gotb[nan])))


def test_sixteen_bit_normals_are_the_narrowed_float32_normals():
    z32 = oracle.gen_inputs(4, 3, oracle.F32, 1000)
    assert np.array_equal(oracle.gen_inputs(4, 3, oracle.F16, 1000), z32.astype(np.float16).view(np.uint16))
    zb = torch.from_numpy(z32).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(oracle.gen_inputs(4, 3, oracle.BF16, 1000), zb)

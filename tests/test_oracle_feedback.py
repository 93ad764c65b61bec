"""Pins for the oracle's offender sample: which elements violate the closeness rule (CPU only)."""
import numpy as np
import torch

import oracle


def _rule_through_double(c, r, atol, rtol):
    """The rule with every operation evaluated in binary64 and rounded once to binary32 (53 >= 2*24+2 bits make
    the double rounding innocuous for +, -, *)."""
    f = np.float32
    c, r, atol, rtol = f(c), f(r), f(atol), f(rtol)
    if c == r:
        return False
    with np.errstate(all="ignore"):
        d = f(abs(np.float64(c) - np.float64(r)))
        t = f(np.float64(rtol) * abs(np.float64(r)))
        tol = f(np.float64(atol) + np.float64(t))
    return not (np.isfinite(d) and d <= tol)


def test_sample_against_torch_isclose_and_a_double_precision_loop():
    rng = np.random.default_rng(3)
    n = 5000
    r = rng.standard_normal(n).astype(np.float32)
    c = (r + 1e-4 * rng.standard_normal(n)).astype(np.float32)
    bad = rng.choice(n, 40, replace=False)
    c[bad] = r[bad] + 1.0
    c[bad[:3]] = [np.nan, np.inf, -np.inf]
    r[bad[3]] = np.nan
    c[bad[4]] = r[bad[4]] = np.inf                     # equal infinities match
    atol = rtol = 0.01
    close = torch.isclose(torch.from_numpy(c), torch.from_numpy(r), rtol=rtol, atol=atol).numpy()
    want = np.nonzero(~close)[0]
    assert len(want) == 39
    for max_out in (0, 1, 10, 39, 100):
        got, found = oracle.mismatch_sample(c, r, oracle.F32, atol, rtol, max_out)
        m = min(max_out, len(want))
        assert found == len(want) and got["index"].tolist() == want[:m].tolist()
        assert got["cand"].tobytes() == c[want[:m]].tobytes() and got["ref"].tobytes() == r[want[:m]].tobytes()
    assert found == oracle.validate(c, r, oracle.F32, atol, rtol)["n_mismatch"]
    loop = [i for i in range(n) if _rule_through_double(c[i], r[i], atol, rtol)]
    assert loop == want.tolist()


def test_sample_for_sixteen_bit_types_reports_widened_values():
    rng = np.random.default_rng(4)
    for dtype in (oracle.F16, oracle.BF16):
        r32 = rng.standard_normal(3000).astype(np.float32)
        r = oracle.narrow(dtype, r32)
        c = oracle.narrow(dtype, r32 + np.where(rng.random(3000) < 0.01, 0.5, 0.0).astype(np.float32))
        got, found = oracle.mismatch_sample(c, r, dtype, 0.01, 0.01, 1000)
        cw, rw = oracle.widen(dtype, c), oracle.widen(dtype, r)
        want = [i for i in range(3000) if _rule_through_double(cw[i], rw[i], 0.01, 0.01)]
        assert found == len(want) > 5 and got["index"].tolist() == want
        assert np.array_equal(got["cand"], cw[want]) and np.array_equal(got["ref"], rw[want])
        assert found == oracle.validate(c, r, dtype, 0.01, 0.01)["n_mismatch"]


def test_empty_and_clean_inputs():
    z = np.zeros(0, np.float32)
    got, found = oracle.mismatch_sample(z, z, oracle.F32, 0.0, 0.0, 5)
    assert found == 0 and len(got) == 0
    x = np.arange(10, dtype=np.float32)
    got, found = oracle.mismatch_sample(x, x, oracle.F32, 0.0, 0.0, 5)
    assert found == 0 and len(got) == 0


def test_integer_outputs_against_numpy_and_unbounded_integers():
    rng = np.random.default_rng(9)
    cases = [
        (oracle.I32, rng.integers(-2**31, 2**31, 5000, dtype=np.int64).astype(np.int32)),
        (oracle.I64, rng.integers(-2**63, 2**63 - 1, 5000, dtype=np.int64)),
        (oracle.U8, rng.integers(0, 256, 5000, dtype=np.int64).astype(np.uint8)),
    ]
    for dtype, r in cases:
        c = r.copy()
        res = oracle.validate_exact(c, r, dtype)
        assert res["n_mismatch"] == 0 and res["max_abs_diff"] == 0 and res["pass"] == 1
        idx = rng.choice(r.size, 37, replace=False)
        c[idx] = np.roll(r, 1)[idx]                       # some of these may coincide by chance
        info = np.iinfo(r.dtype)
        c[0], r[0] = info.max, info.min                    # the widest possible difference
        res = oracle.validate_exact(c, r, dtype)
        assert res["n_mismatch"] == np.count_nonzero(c != r) > 30 and res["pass"] == 0
        assert int(res["max_abs_diff"]) == max(abs(int(a) - int(b)) for a, b in zip(c, r)) == int(info.max) - int(info.min)
    b = rng.random(1000) < 0.5
    res = oracle.validate_exact(b, ~b, oracle.U8)
    assert res["n_mismatch"] == 1000 and res["max_abs_diff"] == 1
    assert oracle.validate_exact(np.zeros(0, np.int32), np.zeros(0, np.int32), oracle.I32)["pass"] == 1
    gp = oracle.group_pass_exact(np.array([(0, 0, 1, 0), (3, 9, 0, 0), (0, 0, 1, 0)], oracle.EXACT_DTYPE), [0, 0, 2], 3)
    assert gp.tolist() == [0, 1, 1]


def test_binary64_rule_against_numpy_isclose_exact_rationals_and_fsum():
    import math
    from fractions import Fraction
    rng = np.random.default_rng(12)
    n = 20000
    r = rng.standard_normal(n)
    c = r + 1e-9 * rng.standard_normal(n)
    atol, rtol = 1e-8, 1e-8
    # values right at the boundary, decided with exact rationals applied to the individually rounded operations
    tol = atol + rtol * np.abs(r)                      # numpy: one binary64 rounding per operation, as the rule says
    for i, ulps in zip(range(0, 600, 3), np.tile([-1, 0, 1], 200)):
        c[i] = r[i] + tol[i]
        for _ in range(abs(int(ulps))):
            c[i] = np.nextafter(c[i], np.inf if ulps > 0 else -np.inf)
    special = rng.choice(np.arange(1000, n), 12, replace=False)
    c[special[:3]] = [np.nan, np.inf, -np.inf]
    r[special[3]] = np.nan
    c[special[4]] = r[special[4]] = np.inf
    r[special[5]] = 0.0
    c[special[6]], r[special[6]] = 1e308, -1e308        # the difference overflows
    res = oracle.validate_f64(c, r, atol, rtol)
    with np.errstate(all="ignore"):
        close = np.isclose(c, r, rtol=rtol, atol=atol)
        d = np.abs(c - r)
    assert res["n_mismatch"] == np.count_nonzero(~close)
    want_exact = 0
    for i in range(n):
        if c[i] == r[i]:
            continue
        if not (math.isfinite(c[i]) and math.isfinite(r[i])):
            want_exact += 1
            continue
        di = abs(Fraction(c[i]) - Fraction(r[i]))
        di = Fraction(float(di)) if di < Fraction(2) ** 1024 else None          # rounded once to binary64
        t = Fraction(float(Fraction(rtol) * abs(Fraction(r[i]))))
        tl = Fraction(float(Fraction(atol) + t))
        want_exact += 0 if (di is not None and di <= tl) else 1
    assert res["n_mismatch"] == want_exact
    fin = np.isfinite(c) & np.isfinite(r)
    assert res["n_nonfinite"] == np.count_nonzero(~fin) == 5 and res["flags"] == 1 | 2 | 4 | 8 | 16
    assert res["max_abs"] == d[fin].max() == np.inf
    nz = fin & (r != 0)
    with np.errstate(all="ignore"):
        assert res["max_rel"] == (d[nz] / np.abs(r[nz])).max()
    assert res["sse"] == np.inf
    # without the overflowing pair: the sum against math.fsum of exactly squared terms
    c[special[6]] = r[special[6]] = 1.0
    res = oracle.validate_f64(c, r, atol, rtol)
    fin = np.isfinite(c) & np.isfinite(r)
    dd = np.abs(c[fin] - r[fin])
    want = float(sum(Fraction(float(x)) ** 2 for x in dd))
    assert abs(res["sse"] - want) <= 1e-14 * want and res["max_abs"] == dd.max()
    assert oracle.validate_f64(r[fin], r[fin], 0.0, 0.0)["pass"] == 1
    assert oracle.validate_f64(np.zeros(0), np.zeros(0), 0.0, 0.0)["pass"] == 1


def test_binary64_squares_are_rounded_to_binary64_before_they_are_summed():
    """The sum of squares of the binary64 rule sums d*d as binary64 products: a square below the binary64
    range counts as 0, one in the subnormal range keeps only the bits that fit.  Checked with exact rationals."""
    from fractions import Fraction
    rng = np.random.default_rng(31)
    n = 4000
    r = rng.standard_normal(n)

    def defined_and_exact(c, r):
        d = [abs(Fraction(float(a)) - Fraction(float(b))) for a, b in zip(c, r)]
        d = [Fraction(float(x)) for x in d]                       # the difference, rounded once
        exact = sum(x * x for x in d)
        defined = sum(Fraction(float(x * x)) for x in d)          # each square rounded once, then summed exactly
        return float(defined), exact

    # (a) every square is below the smallest subnormal: the exact sum is positive, the defined one is 0
    ra = r * 1e-170
    ca = ra * (1 + 2.0 ** -20)
    defined, exact = defined_and_exact(ca, ra)
    assert exact > 0 and defined == 0.0
    assert oracle.validate_f64(ca, ra, 0.0, 0.0)["sse"] == 0.0
    # (b) squares in the subnormal range: sums of multiples of 2^-1074 are exact, so the value is fixed bit for bit
    rb = r * 1e-155
    cb = rb * (1 + 2.0 ** -10)
    defined, exact = defined_and_exact(cb, rb)
    assert 0 < defined < 2.0 ** -1022 and Fraction(defined) != exact
    assert oracle.validate_f64(cb, rb, 0.0, 0.0)["sse"] == defined
    # (c) normal squares with lost ones among them: the defined sum within the summation's own error
    rc = np.where(np.arange(n) % 2 == 0, r, r * 1e-170)
    cc = rc * (1 + 2.0 ** -20)
    defined, exact = defined_and_exact(cc, rc)
    got = oracle.validate_f64(cc, rc, 0.0, 0.0)["sse"]
    assert abs(got - defined) <= 1e-15 * defined

"""Pins for the oracle's closeness rule, error statistics and verdicts (CPU only)."""
import itertools
import math
import os

import numpy as np
import pytest
import torch

import oracle
import workloads

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "closeness_cases.txt")
f32 = np.float32


def _bits(h):
    return np.array([int(h, 16)], dtype=np.uint32).view(np.float32)[0]


def _cases():
    out = []
    for line in open(GOLDEN):
        if not line.strip() or line.startswith("#"):
            continue
        a, b, note = line.split("|", 2)
        atol, rtol, r, c = [_bits(x) for x in a.split()]
        mism, flags, nonfin = [int(x) for x in b.split()]
        out.append((atol, rtol, r, c, mism, flags, nonfin, note.strip()))
    assert len(out) == 14
    return out


def test_hand_worked_cases():
    for atol, rtol, r, c, mism, flags, nonfin, note in _cases():
        assert oracle.element_mismatch(c, r, atol, rtol) == mism, note
        res = oracle.validate(np.array([c], f32), np.array([r], f32), oracle.F32, atol, rtol)
        assert int(res["n_mismatch"]) == mism, note
        assert int(res["flags"]) == flags, note
        assert int(res["n_nonfinite"]) == nonfin, note
        assert int(res["pass"]) == (0 if mism else 1), note
        if nonfin:
            assert res["max_abs"] == 0 and res["max_rel"] == 0 and res["sse"] == 0, note


def test_hand_worked_intermediates_with_numpy_float32():
    # d and tol quoted in the table's notes, recomputed with numpy's binary32 scalars
    # (one rounding per operation).
    t = f32(0.01)
    assert (f32(1.02) - f32(1)).view(np.uint32) == 0x3CA3D700
    assert (t + t * f32(1)).view(np.uint32) == 0x3CA3D70A
    r, c = _bits("3e6c8cc6"), _bits("3e7927c8")
    assert abs(c - r).view(np.uint32) == 0x3C49B020
    assert (t + t * abs(r)).view(np.uint32) == 0x3C49B020
    fused = f32(float(t) + float(t) * float(abs(r)))        # exact product, one rounding
    assert fused.view(np.uint32) == 0x3C49B01F
    assert f32(0.5) * _bits("00000001") == 0


def test_overflowing_difference_of_finite_values():
    res = oracle.validate(np.array([-3e38], f32), np.array([3e38], f32), oracle.F32, 0.01, 0.01)
    assert res["n_mismatch"] == 1 and res["n_nonfinite"] == 0 and res["flags"] == 0
    assert math.isinf(res["max_abs"]) and math.isinf(res["sse"]) and math.isinf(res["max_rel"])


def test_fp16_boundary_case():
    one = np.float16(1.0).view(np.uint16)
    r = np.array([one], np.uint16)
    assert oracle.validate(np.array([one + 20], np.uint16), r, oracle.F16, 0.01, 0.01)["n_mismatch"] == 0
    assert oracle.validate(np.array([one + 21], np.uint16), r, oracle.F16, 0.01, 0.01)["n_mismatch"] == 1


def test_mismatch_mask_equals_torch_isclose_float32():
    # torch.isclose applies the same rule (equal_nan False) with separately rounded
    # float32 operations.
    pop = workloads.special_values(workloads.F32)
    rng = np.random.default_rng(0)
    r = np.concatenate([pop.refs[0].numpy(), rng.standard_normal(20000).astype(f32)])
    c = np.concatenate([pop.tensors[0].cand.numpy(),
                        r[-20000:] * (1 + rng.choice([0, 1e-2, 0.0099, 0.0101, -0.01], 20000)).astype(f32)])
    for atol, rtol in [(0.25, 0.25), (0.01, 0.01), (0.0, 0.01), (1e-3, 0.0), (0.0, 0.0)]:
        close = torch.isclose(torch.from_numpy(c), torch.from_numpy(r), rtol=float(f32(rtol)), atol=float(f32(atol)))
        want = (~close).numpy()
        got = np.array([oracle.element_mismatch(ci, ri, atol, rtol) for ci, ri in zip(c, r)], dtype=bool)
        assert np.array_equal(got, want), (atol, rtol)
        res = oracle.validate(c, r, oracle.F32, atol, rtol)
        assert int(res["n_mismatch"]) == int(want.sum())


def _rule_through_double(c32, r32, atol, rtol):
    """The same rule with every operation evaluated in binary64 and rounded once to
    binary32 (53 >= 2*24 + 2 bits, so this yields the correctly rounded binary32 result)."""
    c64, r64 = c32.astype(np.float64), r32.astype(np.float64)
    with np.errstate(invalid="ignore", over="ignore"):
        d = np.abs((c64 - r64).astype(f32))
        t = (np.float64(f32(rtol)) * np.abs(r64)).astype(f32)
        tol = (np.float64(f32(atol)) + t.astype(np.float64)).astype(f32)
        close = (c32 == r32) | (np.isfinite(d) & (d <= tol))
    return ~close


@pytest.mark.parametrize("dtype", [oracle.F16, oracle.BF16])
def test_exhaustive_sixteen_bit_candidates(dtype):
    bits = np.arange(1 << 16, dtype=np.uint16)
    c32 = oracle.widen(dtype, bits)
    one = 0x3C00 if dtype == oracle.F16 else 0x3F80
    refs = [one, one | 0x8000, 0, 0x8000, 1, one + 3, 0x7C00 if dtype == oracle.F16 else 0x7F80,
            0x7BFF if dtype == oracle.F16 else 0x7F7F, 0x0400 if dtype == oracle.F16 else 0x0080, 0x7E00 if dtype == oracle.F16 else 0x7FC0]
    for rb in refs:
        rarr = np.full(1 << 16, rb, dtype=np.uint16)
        r32 = oracle.widen(dtype, rarr)
        for atol, rtol in [(0.01, 0.01), (0.0, 0.5), (0.25, 0.0)]:
            want = _rule_through_double(c32, r32, atol, rtol)
            res = oracle.validate(bits, rarr, dtype, atol, rtol)
            assert int(res["n_mismatch"]) == int(want.sum()), (hex(rb), atol, rtol)
    # element by element for one reference
    rarr = np.full(1 << 16, one, dtype=np.uint16)
    want = _rule_through_double(c32, oracle.widen(dtype, rarr), 0.01, 0.01)
    got = np.array([oracle.element_mismatch(c, 1.0, 0.01, 0.01) for c in c32], dtype=bool)
    assert np.array_equal(got, want)


def _combine_recursively(items):
    """A deliberately different reduction: divide and conquer over per-element records."""
    if len(items) == 1:
        return items[0]
    h = len(items) // 2
    a, b = _combine_recursively(items[:h]), _combine_recursively(items[h:])
    return dict(n=a["n"] + b["n"], nf=a["nf"] + b["nf"], ma=max(a["ma"], b["ma"]), mr=max(a["mr"], b["mr"]),
                sse=a["sse"] + b["sse"], flags=a["flags"] | b["flags"])


def _element_record(c, r, atol, rtol):
    c, r = f32(c), f32(r)
    with np.errstate(invalid="ignore", over="ignore", divide="ignore"):
        d = abs(c - r)
        tol = f32(atol) + f32(rtol) * abs(r)
        close = bool(c == r) or (bool(np.isfinite(d)) and bool(d <= tol))
        flags = (1 if np.isnan(c) else 0) | (2 if c == np.inf else 0) | (4 if c == -np.inf else 0) \
            | (8 if np.isnan(r) else 0) | (16 if np.isinf(r) else 0)
        if flags:
            return dict(n=int(not close), nf=1, ma=f32(0), mr=f32(0), sse=0.0, flags=flags)
        mr = d / abs(r) if r != 0 else f32(0)
    return dict(n=int(not close), nf=0, ma=d, mr=mr, sse=float(d) * float(d), flags=0)


def test_brute_force_tiny_tensors():
    vals = [0.0, -0.0, 2.0 ** -149, -(2.0 ** -149), 2.0 ** -126, 1.0, -1.0, float(np.nextafter(f32(1), f32(2))),
            float(np.finfo(f32).max), -float(np.finfo(f32).max), math.inf, -math.inf, math.nan, 0.75]
    pairs = list(itertools.product(vals, vals))
    rng = np.random.default_rng(3)
    for atol, rtol in [(0.0, 0.0), (2.0 ** -10, 2.0 ** -10), (0.25, 0.25), (0.01, 0.01)]:
        for _ in range(60):
            n = int(rng.integers(1, 9))
            idx = rng.integers(0, len(pairs), n)
            c = np.array([pairs[i][0] for i in idx], f32)
            r = np.array([pairs[i][1] for i in idx], f32)
            want = _combine_recursively([_element_record(ci, ri, atol, rtol) for ci, ri in zip(c, r)])
            res = oracle.validate(c, r, oracle.F32, atol, rtol)
            assert int(res["n_mismatch"]) == want["n"] and int(res["n_nonfinite"]) == want["nf"]
            assert int(res["flags"]) == want["flags"]
            assert f32(res["max_abs"]).view(np.uint32) == f32(want["ma"]).view(np.uint32)
            assert f32(res["max_rel"]).view(np.uint32) == f32(want["mr"]).view(np.uint32)
            if math.isinf(want["sse"]):
                assert math.isinf(res["sse"])
            else:
                assert res["sse"] == pytest.approx(want["sse"], rel=1e-12, abs=0)
            assert int(res["pass"]) == int(want["n"] == 0)
    # all pairs once, element by element
    for cv, rv in pairs:
        want = _element_record(cv, rv, 0.25, 0.25)
        assert oracle.element_mismatch(cv, rv, 0.25, 0.25) == want["n"]


def test_statistics_against_numpy():
    rng = np.random.default_rng(8)
    r = rng.standard_normal(50000).astype(f32)
    r[::97] = 0.0
    c = (r + rng.standard_normal(50000).astype(f32) * f32(3e-3)).astype(f32)
    res = oracle.validate(c, r, oracle.F32, 0.005, 0.005)
    d = np.abs(c - r)
    assert res["max_abs"] == d.max()
    nz = r != 0
    assert res["max_rel"] == (d[nz] / np.abs(r[nz])).max()
    assert res["sse"] == pytest.approx(math.fsum((d.astype(np.float64) ** 2).tolist()), rel=1e-12)
    assert int(res["n_mismatch"]) == int((d > (f32(0.005) + f32(0.005) * np.abs(r))).sum())
    assert res["n_nonfinite"] == 0 and res["flags"] == 0


def test_metamorphic_properties():
    pop = workloads.config2("cpu", n=30000, k=2, trials=5)
    r = pop.refs[0].numpy()
    c = pop.tensors[0].cand.numpy()
    base = oracle.validate(c, r, oracle.F32, pop.atol, pop.rtol)
    # identical tensors pass with all-zero statistics
    same = oracle.validate(r, r, oracle.F32, 0.0, 0.0)
    assert same["pass"] == 1 and same["n_mismatch"] == 0 and same["max_abs"] == 0 and same["sse"] == 0
    # a joint permutation changes nothing but the summation order
    p = np.random.default_rng(1).permutation(r.size)
    perm = oracle.validate(c[p], r[p], oracle.F32, pop.atol, pop.rtol)
    for k in ("n_mismatch", "n_nonfinite", "max_abs", "max_rel", "flags", "pass"):
        assert perm[k] == base[k]
    assert perm["sse"] == pytest.approx(base["sse"], rel=1e-12)
    # splitting combines by sum / max / or
    a = oracle.validate(c[:12345], r[:12345], oracle.F32, pop.atol, pop.rtol)
    b = oracle.validate(c[12345:], r[12345:], oracle.F32, pop.atol, pop.rtol)
    assert a["n_mismatch"] + b["n_mismatch"] == base["n_mismatch"]
    assert max(a["max_abs"], b["max_abs"]) == base["max_abs"] and max(a["max_rel"], b["max_rel"]) == base["max_rel"]
    assert a["sse"] + b["sse"] == pytest.approx(base["sse"], rel=1e-12)
    # a larger tolerance never adds mismatches
    prev = None
    for tol in (0.0, 1e-6, 1e-4, 1e-3, 1e-2, 1.0):
        n = int(oracle.validate(c, r, oracle.F32, tol, tol)["n_mismatch"])
        assert prev is None or n <= prev
        prev = n
    # swapping candidate and reference keeps d; with rtol = 0 the verdicts are the same
    sw = oracle.validate(r, c, oracle.F32, pop.atol, 0.0)
    st = oracle.validate(c, r, oracle.F32, pop.atol, 0.0)
    assert sw["n_mismatch"] == st["n_mismatch"] and sw["max_abs"] == st["max_abs"]


def test_populations_hold_what_they_are_built_to_hold():
    p1 = workloads.config1("cpu")
    res = oracle.validate(p1.tensors[0].cand.numpy(), p1.refs[0].numpy(), oracle.F32, p1.atol, p1.rtol)
    assert int(res["n_mismatch"]) == 7 and res["pass"] == 0
    assert 0.9 < res["max_abs"] < 1.1
    p2 = workloads.config2("cpu", n=1 << 16, k=3, trials=4)
    for t, n_inj in zip(p2.tensors, p2.facts["n_mismatch"]):
        res = oracle.validate(t.cand.numpy(), p2.refs[0].numpy(), oracle.F32, p2.atol, p2.rtol)
        assert int(res["n_mismatch"]) == n_inj
    p4 = workloads.config4("cpu", n=1 << 14, k=4)
    for i, t in enumerate(p4.tensors):
        res = oracle.validate(t.cand.numpy(), p4.refs[0].numpy(), oracle.F32, p4.atol, p4.rtol)
        if i == p4.facts["wrong"]:
            assert res["pass"] == 0 and res["n_mismatch"] > 0.99 * (1 << 14)
        else:
            assert res["pass"] == 1


def test_group_verdict_is_the_and_of_its_tensors():
    res = np.zeros(5, dtype=oracle.RESULT_DTYPE)
    res["pass"] = [1, 1, 0, 1, 1]
    got = oracle.group_pass(res, [0, 1, 1, 3, 0], 5)
    assert got.tolist() == [1, 0, 1, 1, 1]          # groups without tensors pass vacuously

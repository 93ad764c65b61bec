"""evo_validate_f64 on the GPU against the oracle: counts, flags, verdicts, max_abs and max_rel bit-exact
(binary64); the sum of squares within 1e-12 relative, nothing else (only the summation order differs: on both
sides a square is a binary64 product, so squares below the binary64 range are lost on both)."""
import math

import numpy as np
import pytest
import torch

import oracle

pytestmark = pytest.mark.gpu
SSE_RTOL = 1e-12


@pytest.fixture(scope="module")
def evo():
    import paper_2510_03760_b200 as evo
    return evo


def _compare(got, want, what=""):
    for k in ("n_mismatch", "n_nonfinite", "flags", "pass"):
        assert np.array_equal(got[k], want[k]), (what, k, got[k], want[k])
    for k in ("max_abs", "max_rel"):
        assert np.array_equal(got[k].view(np.uint64), want[k].view(np.uint64)), (what, k, got[k], want[k])
    for g, w in zip(got["sse"], want["sse"]):
        if w == 0.0 or math.isinf(w) or math.isnan(w):
            assert g == w or (math.isnan(g) and math.isnan(w)), (what, g, w)
        else:
            assert abs(g - w) <= SSE_RTOL * abs(w), (what, g, w)


def _check(evo, cands, refs, atol, rtol, groups=None, n_group=0):
    ref_list = refs if isinstance(refs, list) else [refs] * len(cands)
    dev_refs = {id(r): r.cuda() for r in ref_list}
    res, gp = evo.evo_validate_f64([c.cuda() for c in cands], [dev_refs[id(r)] for r in ref_list], atol, rtol,
                                   groups=groups, n_group=n_group)
    got = evo.results64_to_numpy(res)
    want = np.zeros(len(cands), oracle.RESULT64_DTYPE)
    for i, (c, r) in enumerate(zip(cands, ref_list)):
        want[i] = oracle.validate_f64(c.numpy(), r.numpy(), atol, rtol)
    _compare(got, want)
    if groups is not None:
        exp = np.ones(n_group, np.uint32)
        for i, g in enumerate(groups):
            exp[g] &= want["pass"][i]
        assert np.array_equal(gp.cpu().numpy().view(np.uint32), exp)
    return got


def test_shared_reference_sizes_boundaries_and_specials(evo):
    g = torch.Generator().manual_seed(21)
    atol = rtol = 1e-8
    for n, k in [(0, 1), (1, 1), (3, 2), (4095, 3), (4096, 2), (4097, 5), (3 * 4096 + 19, 34), (300000, 6)]:
        ref = torch.randn(n, generator=g, dtype=torch.float64)
        cands = []
        for i in range(k):
            c = ref + 1e-9 * torch.randn(n, generator=g, dtype=torch.float64)
            if n > 10:
                tol = atol + rtol * ref.abs()
                idx = torch.randint(0, n, (max(1, n // 100),), generator=g)
                step = torch.randint(-1, 2, idx.shape, generator=g).double()
                c[idx] = ref[idx] + tol[idx] * (1 + step * 2.0 ** -50)            # on and right around the boundary
                if i % 2 == 0:
                    c[idx[0]] = float("nan"); c[idx[-1]] = float("-inf")
                if i % 3 == 0:
                    c[1], c[2] = 1e308, float("inf")
            cands.append(c)
        if n > 10:
            ref = ref.clone()
            ref[1] = -1e308                                                      # a difference that overflows
            ref[3] = 0.0
        _check(evo, cands, ref, atol, rtol, groups=[i % 3 for i in range(k)], n_group=3)


def test_own_references_unaligned_views_identical_and_tiny(evo):
    g = torch.Generator().manual_seed(22)
    cands, refs = [], []
    for n, off in [(5000, 0), (5000, 1), (777, 1), (12345, 0), (40000, 1)]:
        store = torch.randn(n + 2, generator=g, dtype=torch.float64)
        r = store[off:off + n]
        cands.append(r * (1 + 1e-12 * torch.randn(n, generator=g, dtype=torch.float64))); refs.append(r)
    r = torch.randn(9000, generator=g, dtype=torch.float64)
    cands += [r.clone(), torch.relu(r) + 1e-300, r * 1e-200 * (1 + 1e-9)]
    refs += [r, torch.relu(r), r * 1e-200]
    _check(evo, cands, refs, 1e-10, 1e-10)
    # device views at odd offsets: 8-byte but not 16-byte aligned
    d = [(torch.cat([torch.zeros(1, dtype=torch.float64), c]).cuda()[1:], torch.cat([torch.zeros(1, dtype=torch.float64), r]).cuda()[1:])
         for c, r in zip(cands, refs)]
    res, _ = evo.evo_validate_f64([x[0] for x in d], [x[1] for x in d], 1e-10, 1e-10)
    want = np.array([oracle.validate_f64(c.numpy(), r.numpy(), 1e-10, 1e-10) for c, r in zip(cands, refs)])
    _compare(evo.results64_to_numpy(res), want, "unaligned")


def test_argument_errors(evo):
    x = torch.zeros(8, dtype=torch.float64, device="cuda")
    with pytest.raises(evo.EvoError):
        evo.evo_validate_f64([x], [x], -1.0, 0.0)
    with pytest.raises(evo.EvoError) as e:
        evo.evo_validate_f64([x.float()], [x.float()], 0.1, 0.1)
    assert e.value.status == -3


def test_seeded_random_cases(evo):
    """Sizes around tile boundaries, 1 to 33 members, magnitudes from 1e-150 to 1e300, zeros in the reference,
    values on the tolerance boundary, NaN/Inf, sign flips that overflow the difference, odd alignment."""
    rng = np.random.default_rng(5)
    sizes = [0, 1, 2, 3, 17, 2047, 4095, 4096, 4097, 8192, 3 * 4096 + 5, 70001]
    for it in range(40):
        g = torch.Generator().manual_seed(it)
        n = int(rng.choice(sizes)); k = int(rng.choice([1, 2, 5, 33])); off = int(rng.choice([0, 1]))
        scale = float(rng.choice([1.0, 1e-3, 1e150, 1e-150, 1e300]))
        atol, rtol = [(1e-8, 1e-8), (0.0, 0.0), (1e-3, 0.0), (0.0, 1e-12)][int(rng.integers(0, 4))]
        store = torch.randn(n + off, generator=g, dtype=torch.float64) * scale
        if rng.random() < 0.3:
            store = torch.relu(store)
        ref = store[off:]
        cands = []
        for _ in range(k):
            mode = int(rng.integers(0, 5))
            if mode == 0:
                c = ref.clone()
            elif mode == 1:
                c = ref + (atol + rtol * ref.abs()) * (torch.rand(n, generator=g, dtype=torch.float64) * 2.2 - 1.1)
            elif mode == 2:
                c = ref * (1 + 1e-13 * torch.randn(n, generator=g, dtype=torch.float64))
            elif mode == 3:
                c = torch.randn(n, generator=g, dtype=torch.float64) * scale
            else:
                c = ref * -1.5
            if n and rng.random() < 0.5:
                idx = torch.randint(0, n, (max(1, n // 300),), generator=g)
                vals = torch.tensor([float("nan"), float("inf"), float("-inf")], dtype=torch.float64)
                c[idx] = vals[torch.randint(0, 3, idx.shape, generator=g)]
            cands.append(c)
        dref = store.cuda()[off:]
        dev = [torch.cat([torch.zeros(off, dtype=torch.float64), c]).cuda()[off:] for c in cands]
        res, _ = evo.evo_validate_f64(dev, [dref] * k, atol, rtol)
        want = np.array([oracle.validate_f64(c.numpy(), ref.numpy(), atol, rtol) for c in cands])
        _compare(evo.results64_to_numpy(res), want, "case %d n %d k %d" % (it, n, k))


def test_squares_in_and_below_the_subnormal_range(evo):
    """A square is a binary64 product on both sides: below the range it is lost, in the subnormal range it keeps the
    bits that fit (and sums of such values are exact, so the results are then equal bit for bit)."""
    g = torch.Generator().manual_seed(77)
    n = 3 * 4096 + 1234
    base = torch.randn(n, generator=g, dtype=torch.float64)
    cands, refs = [], []
    for scale, eps in [(1e-170, 2.0 ** -20), (1e-155, 2.0 ** -10), (1e-160, 2.0 ** -3), (1e-162, 0.5)]:
        r = base * scale
        cands.append(r * (1 + eps)); refs.append(r)
    mixed = torch.where(torch.arange(n) % 2 == 0, base, base * 1e-170)
    cands.append(mixed * (1 + 2.0 ** -20)); refs.append(mixed)
    got = _check(evo, cands, refs, 0.0, 0.0)
    want = [oracle.validate_f64(c.numpy(), r.numpy(), 0.0, 0.0)["sse"] for c, r in zip(cands, refs)]
    assert got["sse"][0] == 0.0 and all(got["sse"][i] == want[i] for i in range(4)) and 0 < got["sse"][1] < 2.0 ** -1022

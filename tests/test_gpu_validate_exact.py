"""evo_validate_exact on the GPU against the oracle: integer and boolean outputs, every field exact."""
import numpy as np
import pytest
import torch

import oracle

pytestmark = pytest.mark.gpu
CASES = [(torch.int32, oracle.I32), (torch.int64, oracle.I64), (torch.uint8, oracle.U8)]


@pytest.fixture(scope="module")
def evo():
    import paper_2510_03760_b200 as evo
    return evo


def _rand(tdt, n, g):
    info = torch.iinfo(tdt)
    if tdt == torch.int64:
        return torch.randint(-2**62, 2**62, (n,), generator=g, dtype=tdt) * 2 + torch.randint(0, 2, (n,), generator=g, dtype=tdt)
    return torch.randint(info.min, info.max + 1, (n,), generator=g, dtype=torch.int64).to(tdt)


def _check(evo, cands, refs, code, groups=None, n_group=0):
    res, gp = evo.evo_validate_exact([c.cuda() for c in cands], [r.cuda() for r in refs] if isinstance(refs, list) else refs.cuda(),
                                     groups=groups, n_group=n_group)
    got = evo.exact_to_numpy(res)
    ref_list = refs if isinstance(refs, list) else [refs] * len(cands)
    want = np.zeros(len(cands), oracle.EXACT_DTYPE)
    for i, (c, r) in enumerate(zip(cands, ref_list)):
        want[i] = oracle.validate_exact(c.numpy().view(np.uint8) if c.dtype == torch.bool else c.numpy(),
                                        r.numpy().view(np.uint8) if r.dtype == torch.bool else r.numpy(), code)
    assert got.tobytes() == want.tobytes(), (got, want)
    if groups is not None:
        assert np.array_equal(gp.cpu().numpy().view(np.uint32), oracle.group_pass_exact(want, groups, n_group))
    return got


@pytest.mark.parametrize("tdt,code", CASES)
def test_shared_reference_ragged_sizes_and_extremes(evo, tdt, code):
    g = torch.Generator().manual_seed(int(code))
    info = torch.iinfo(tdt)
    for n, k in [(0, 1), (1, 1), (15, 3), (4096, 2), (4097, 5), (3 * 4096 + 19, 34), (200000, 4)]:
        ref = _rand(tdt, n, g)
        cands = []
        for i in range(k):
            c = ref.clone()
            if i % 2 == 1 and n:
                hit = torch.rand(n, generator=g) < 0.01
                c = torch.where(hit, _rand(tdt, n, g), c)
                c[n - 1] = ref[n - 1] ^ 1
            if i == 2 and n:
                c[0], ref_first = info.max, ref[0].item()
            cands.append(c)
        if n:
            ref[0] = info.min                                   # candidate 2 then differs by the widest possible amount
        got = _check(evo, cands, ref, code, groups=[i // 2 for i in range(k)], n_group=(k + 1) // 2)
        if n and k > 2:
            assert int(got["max_abs_diff"][2]) == info.max - info.min
        if n:
            assert got["pass"][0] == (1 if (ref[0] == cands[0][0]) else 0)


def test_own_references_mixed_types_and_unaligned_views(evo):
    g = torch.Generator().manual_seed(77)
    cands, refs, codes = [], [], []
    for tdt, code in CASES:
        for n, off in [(5000, 0), (5000, 1), (777, 3), (12345, 0)]:
            store = _rand(tdt, n + 8, g)
            r = store[off:off + n]
            c = r.clone()
            c[n // 2] = c[n // 2] ^ 3
            cands.append(c); refs.append(r); codes.append(code)
    res, _ = evo.evo_validate_exact([c.cuda() for c in cands], [r.cuda() for r in refs])
    got = evo.exact_to_numpy(res)
    # device-side views at odd offsets too
    dev = [(torch.cat([torch.zeros(o, dtype=c.dtype), c]).cuda()[o:], torch.cat([torch.zeros(o, dtype=r.dtype), r]).cuda()[o:])
           for o, (c, r) in zip([0, 1, 3, 5] * 3, zip(cands, refs))]
    res2, _ = evo.evo_validate_exact([d[0] for d in dev], [d[1] for d in dev])
    for i, (c, r, code) in enumerate(zip(cands, refs, codes)):
        want = oracle.validate_exact(c.numpy(), r.numpy(), code)
        assert got[i].tobytes() == want.tobytes() and evo.exact_to_numpy(res2)[i].tobytes() == want.tobytes()
        assert got["n_mismatch"][i] == 1 and got["max_abs_diff"][i] in (1, 2, 3)


def test_bool_masks_and_errors(evo):
    g = torch.Generator().manual_seed(5)
    m = torch.rand(70000, generator=g) < 0.5
    _check(evo, [m.clone(), ~m, m ^ (torch.rand(70000, generator=g) < 0.001)], m, oracle.U8)
    x = torch.zeros(8, device="cuda")
    with pytest.raises(evo.EvoError) as e:
        evo.evo_validate_exact([x], [x])                      # a float tensor is not accepted here
    assert e.value.status == -3
    with pytest.raises(evo.EvoError):
        evo.evo_validate([x.int()], [x.int()], 0.1, 0.1)      # nor an integer tensor by evo_validate

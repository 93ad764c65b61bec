"""evo_validate_generated on the GPU against the oracle: a buffer checked for equality against a window of the
Philox stream that the kernel regenerates.  The expected records come from the oracle's own generator
(oracle.gen_u32, pinned by the published known-answer vectors) and its integer check (oracle.validate_exact);
every field must be equal."""
import numpy as np
import pytest
import torch

import oracle

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def evo():
    import paper_2510_03760_b200 as evo
    return evo


def _want(cands_np, seed, offsets, signed):
    want = np.zeros(len(cands_np), oracle.EXACT_DTYPE)
    for i, (c, off) in enumerate(zip(cands_np, offsets)):
        ref = oracle.gen_u32(seed, off, c.size)
        if signed:
            want[i] = oracle.validate_exact(c.view(np.int32), ref.view(np.int32), oracle.I32)
        else:           # unsigned words: as 64-bit integers, where every uint32 and every difference of two fits
            want[i] = oracle.validate_exact(c.astype(np.int64), ref.astype(np.int64), oracle.I64)
    return want


def _check(evo, cands_np, seed, offsets, signed, lead_pad=None, groups=None, n_group=0):
    dev = []
    for i, c in enumerate(cands_np):
        pad = 0 if lead_pad is None else lead_pad[i]
        store = torch.zeros(c.size + pad, dtype=torch.int32, device="cuda")
        store[pad:] = torch.from_numpy(c.view(np.int32)).cuda()
        dev.append(store[pad:])
    offs = offsets if len(set(offsets)) > 1 or len(offsets) == 0 else int(offsets[0])
    res, gp = evo.evo_validate_generated(seed, dev, offsets=offs, dtype=evo.EVO_I32 if signed else evo.EVO_U32,
                                         groups=groups, n_group=n_group)
    got = evo.exact_to_numpy(res)
    want = _want(cands_np, seed, offsets, signed)
    assert got.tobytes() == want.tobytes(), (got, want)
    if groups is not None:
        assert np.array_equal(gp.cpu().numpy().view(np.uint32), oracle.group_pass_exact(want, groups, n_group))
    return got


def _spoil(rng, words, n_wrong):
    c = words.copy()
    if c.size and n_wrong:
        idx = rng.choice(c.size, size=min(n_wrong, c.size), replace=False)
        c[idx] ^= rng.integers(1, 2**32, idx.size, dtype=np.uint64).astype(np.uint32)
    return c


@pytest.mark.parametrize("signed", [False, True])
def test_shared_window_sizes_around_tiles_and_wrong_elements(evo, signed):
    rng = np.random.default_rng(3)
    seed = 0x1234_5678_9ABC_DEF0
    for n in [0, 1, 3, 4, 5, 4095, 4096, 4097, 8192 + 7, 5 * 4096 + 1234, 300001]:
        for offset in [0, 4, 1, 2, 3, 2**40 + 8, 2**63 - 5]:
            words = oracle.gen_u32(seed, offset, n)
            cands = [words.copy(), _spoil(rng, words, 1), _spoil(rng, words, 50), rng.integers(0, 2**32, n, dtype=np.uint64).astype(np.uint32)]
            got = _check(evo, cands, seed, [offset] * 4, signed, groups=[0, 1, 1, 2], n_group=4)
            assert got["pass"][0] == 1 and (n == 0 or got["pass"][3] == 0)


def test_own_windows_unaligned_buffers_and_many_members(evo):
    rng = np.random.default_rng(4)
    seed = 99
    sizes = [10, 5000, 4096 * 3, 70000, 4096 * 2 + 5, 123, 0, 40000]
    offsets = [0, 7, 4096, 12345678901, 2, 16, 5, 4]
    cands = [_spoil(rng, oracle.gen_u32(seed, o, n), int(rng.integers(0, 4))) for n, o in zip(sizes, offsets)]
    _check(evo, cands, seed, offsets, False, lead_pad=[0, 1, 0, 3, 2, 0, 1, 0])
    # 40 members of one window: more than a set holds
    words = oracle.gen_u32(seed, 64, 3 * 4096 + 99)
    many = [_spoil(rng, words, i % 3) for i in range(40)]
    _check(evo, many, seed, [64] * 40, True, groups=[i % 5 for i in range(40)], n_group=5)


def test_largest_differences_are_exact_for_both_readings(evo):
    # words 0x00000000 / 0xffffffff against the stream: unsigned and two's-complement differences differ
    seed, n = 5, 4096 + 17
    words = oracle.gen_u32(seed, 0, n)
    zeros, ones = np.zeros(n, np.uint32), np.full(n, 0xFFFFFFFF, np.uint32)
    u = _check(evo, [zeros, ones], seed, [0, 0], False)
    s = _check(evo, [zeros, ones], seed, [0, 0], True)
    assert u["max_abs_diff"][0] == words.max() and s["max_abs_diff"][0] == np.abs(words.view(np.int32).astype(np.int64)).max()


def test_agrees_with_generating_then_checking(evo):
    """The fused call against the two-step route through the library's own generator."""
    n, seed, offset = 1 << 20, 77, 12
    ref = torch.empty(n, dtype=torch.int32, device="cuda")
    evo.evo_gen_inputs(seed, offset, evo.EVO_U32, n, ref)
    cand = ref.clone()
    cand[12345] += 9
    two_step = evo.exact_to_numpy(evo.evo_validate_exact([cand], [ref])[0])
    fused = evo.exact_to_numpy(evo.evo_validate_generated(seed, [cand], offsets=offset, dtype=evo.EVO_I32)[0])
    assert fused.tobytes() == two_step.tobytes() and fused["n_mismatch"][0] == 1 and fused["max_abs_diff"][0] == 9


def test_argument_errors(evo):
    x = torch.zeros(8, dtype=torch.int32, device="cuda")
    with pytest.raises(evo.EvoError) as e:
        evo.evo_validate_generated(1, [x], dtype=evo.EVO_F32)
    assert e.value.status == -3
    with pytest.raises(ValueError):
        evo.evo_validate_generated(1, [x.to(torch.int64)])

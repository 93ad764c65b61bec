"""evo_gen_inputs on the GPU against the oracle: words bit-exact, fp32 normals within 4 ulp,
fp16/bf16 normals within 1 ulp of their type."""
import numpy as np
import pytest
import torch

import oracle
from parity import ordered, ordered16

pytestmark = pytest.mark.gpu

CASES = [  # (seed, offset, n)
    (0, 0, 4), (0, 0, 4096), (1, 1, 1), (7, 2, 3), (7, 3, 1030), (42, 5, 100003),
    (0xDEADBEEFCAFEF00D, (1 << 34) - 3, 70001), (3, (1 << 63) + 2, 999), (9, 0, 0), (5, 1 << 20, (1 << 18) + 7),
]


@pytest.fixture(scope="module")
def evo():
    import paper_2510_03760_b200 as evo
    return evo


@pytest.mark.parametrize("seed,offset,n", CASES)
def test_words_bit_exact(evo, seed, offset, n):
    out = torch.full((n + 8,), -1, dtype=torch.int32, device="cuda")
    evo.evo_gen_inputs(seed, offset, evo.EVO_U32, n, out[4:])       # 16-byte aligned view
    got = out.cpu().numpy().view(np.uint32)
    assert np.array_equal(got[4:4 + n], oracle.gen_u32(seed, offset, n))
    assert np.all(got[:4] == 0xFFFFFFFF) and np.all(got[4 + n:] == 0xFFFFFFFF)    # nothing outside [0, n)
    out.fill_(-1)
    evo.evo_gen_inputs(seed, offset, evo.EVO_U32, n, out[3:])       # 4-byte aligned only
    got = out.cpu().numpy().view(np.uint32)
    assert np.array_equal(got[3:3 + n], oracle.gen_u32(seed, offset, n))
    assert np.all(got[:3] == 0xFFFFFFFF) and np.all(got[3 + n:] == 0xFFFFFFFF)


@pytest.mark.parametrize("seed,offset,n", CASES)
def test_normals_fp32_within_4_ulp(evo, seed, offset, n):
    out = torch.full((n + 2,), float("nan"), dtype=torch.float32, device="cuda")
    evo.evo_gen_inputs(seed, offset, evo.EVO_F32, n, out[1:])
    got = out.cpu().numpy()
    assert np.isnan(got[0]) and np.isnan(got[n + 1])
    want = oracle.gen_inputs(seed, offset, oracle.F32, n)
    assert np.all(np.isfinite(got[1:1 + n]))
    ulp = np.abs(ordered(got[1:1 + n]) - ordered(want))
    assert ulp.max(initial=0) <= 4, (int(ulp.max()), int(ulp.argmax()))


@pytest.mark.parametrize("code,tdt", [(2, torch.float16), (3, torch.bfloat16)])
@pytest.mark.parametrize("seed,offset,n", CASES[:7])
def test_normals_sixteen_bit_within_1_ulp(evo, code, tdt, seed, offset, n):
    out = torch.zeros((n + 1,), dtype=tdt, device="cuda")
    evo.evo_gen_inputs(seed, offset, code, n, out[1:])
    got = out.cpu().view(torch.int16).numpy().view(np.uint16)[1:]
    want = oracle.gen_inputs(seed, offset, code, n)
    ulp = np.abs(ordered16(got) - ordered16(want))
    assert ulp.max(initial=0) <= 1


def test_large_fill_statistics_and_sampled_parity(evo):
    n = 1 << 26
    out = torch.empty(n, dtype=torch.float32, device="cuda")
    evo.evo_gen_inputs(2025, 12, evo.EVO_F32, n, out)
    assert abs(out.mean().item()) < 5 / n ** 0.5 and abs(out.var().item() - 1) < 5 * (2 / n) ** 0.5
    rng = np.random.default_rng(0)
    for start in [0, n - 4096] + rng.integers(0, n - 4096, 30).tolist():
        got = out[start:start + 4096].cpu().numpy()
        want = oracle.gen_inputs(2025, 12 + start, oracle.F32, 4096)
        assert np.abs(ordered(got) - ordered(want)).max() <= 4


def test_fill_of_the_largest_configuration_in_full(evo):
    """2^28 fp32 normals, the test-input tensor of the largest synthetic configuration, in the launch shape the
    benchmark uses: every element against the oracle, in pieces of 2^24 (about 20 s of oracle time)."""
    n, piece = 1 << 28, 1 << 24
    out = torch.empty(n, dtype=torch.float32, device="cuda")
    evo.evo_gen_inputs(1000, 0, evo.EVO_F32, n, out)
    worst = 0
    for start in range(0, n, piece):
        got = out[start:start + piece].cpu().numpy()
        want = oracle.gen_inputs(1000, start, oracle.F32, piece)
        worst = max(worst, int(np.abs(ordered(got) - ordered(want)).max()))
    assert worst <= 4, worst


def test_argument_errors(evo):
    out = torch.zeros(16, dtype=torch.float32, device="cuda")
    L, ctx = evo.load_library(), evo.default_context(0)
    assert L.evo_gen_inputs(ctx._h, 0, 0, 9, 4, out.data_ptr(), None) == -3
    assert L.evo_gen_inputs(ctx._h, 0, 0, 1, 4, None, None) == -1
    assert L.evo_gen_inputs(ctx._h, 0, 0, 1, 4, out.data_ptr() + 2, None) == -2
    assert L.evo_gen_inputs(ctx._h, 0, 0, 1, 0, None, None) == 0
    assert b"aligned" in L.evo_last_error(ctx._h)

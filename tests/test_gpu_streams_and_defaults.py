"""Stream semantics and the call-level defaults of the C ABI, on the GPU.

* Calls only enqueue work on the stream they are given: a candidate produced on a side stream right before
  the call is seen by it, and results are complete once that stream has been synchronised.
* Descriptors with ref = NULL and dtype = -1 take the call's ref_ptr and dtype."""
import ctypes as C

import numpy as np
import pytest
import torch

import oracle
import workloads
from parity import assert_results_equal

pytestmark = pytest.mark.gpu


def test_calls_are_ordered_on_a_side_stream_with_a_context_of_its_own():
    import paper_2510_03760_b200 as evo
    side = torch.cuda.Stream()
    ctx = evo.Context(0)
    g = torch.Generator().manual_seed(1)
    ref_h = torch.randn(1 << 20, generator=g)
    noise_h = 0.004 * torch.randn(1 << 20, generator=g)
    ref = ref_h.cuda()
    noise = noise_h.cuda()
    torch.cuda.synchronize()
    with torch.cuda.stream(side):
        big = torch.empty(1 << 26, device="cuda").normal_()          # keeps the side stream busy first
        cand = ref + noise                                            # produced on the side stream ...
        res, gp = evo.evo_validate([cand], [ref], 0.005, 0.005, groups=[0], n_group=1, stream=side, ctx=ctx)   # ... and consumed there
        fit = evo.evo_fitness(torch.tensor([[1.0, 2.0, 3.0]], device="cuda"), torch.tensor([4.0], device="cuda"), gp,
                              stream=side, ctx=ctx)
    ctx.synchronize(side)
    got = evo.results_to_numpy(res)
    want = oracle.validate((ref_h + noise_h).numpy(), ref_h.numpy(), oracle.F32, 0.005, 0.005)
    assert_results_equal(got, np.array([want]))
    f = evo.fits_to_numpy(fit)[0]
    assert f["valid"] == want["pass"] and (f["speedup"] == 2.0 if want["pass"] else f["speedup"] == 0.0)
    del big


def test_call_level_reference_and_dtype_defaults():
    import paper_2510_03760_b200 as evo
    from paper_2510_03760_b200 import binding
    L, ctx = evo.load_library(), evo.Context(0)
    g = torch.Generator().manual_seed(2)
    n = 3 * 4096 + 77
    ref_h = torch.randn(n, generator=g).to(torch.bfloat16)
    cands_h = [(ref_h.float() + 0.02 * torch.randn(n, generator=g)).to(torch.bfloat16) for _ in range(3)]
    own_ref_h = torch.randn(n, generator=g)                              # one descriptor overrides both defaults
    own_cand_h = own_ref_h + 0.02 * torch.randn(n, generator=g)
    ref, own_ref, own_cand = ref_h.cuda(), own_ref_h.cuda(), own_cand_h.cuda()
    cands = [c.cuda() for c in cands_h]
    ptrs = np.array([c.data_ptr() for c in cands] + [own_cand.data_ptr()], dtype=np.uint64)
    descs = np.zeros(4, dtype=binding._DESC_DTYPE)
    descs["n"] = n
    descs["ref"][:3], descs["dtype"][:3] = 0, -1                          # NULL reference, default dtype
    descs["ref"][3], descs["dtype"][3] = own_ref.data_ptr(), evo.EVO_F32
    descs["group"] = [0, 1, 2, 3]
    res = torch.empty((4, 40), dtype=torch.uint8, device="cuda")
    gp = torch.empty(4, dtype=torch.int32, device="cuda")
    st = L.evo_validate(ctx._h, C.c_void_p(ptrs.ctypes.data), C.c_void_p(ref.data_ptr()), C.c_void_p(descs.ctypes.data), 4,
                        evo.EVO_BF16, 0.01, 0.01, C.c_void_p(res.data_ptr()), C.c_void_p(gp.data_ptr()), 4, None)
    assert st == 0
    ctx.synchronize()
    got = evo.results_to_numpy(res)
    want = np.zeros(4, oracle.RESULT_DTYPE)
    for i in range(3):
        want[i] = oracle.validate(workloads.to_host_bits(cands_h[i]), workloads.to_host_bits(ref_h), oracle.BF16, 0.01, 0.01)
    want[3] = oracle.validate(own_cand_h.numpy(), own_ref_h.numpy(), oracle.F32, 0.01, 0.01)
    assert_results_equal(got, want)
    assert gp.cpu().tolist() == want["pass"].tolist()
    # without a call-level reference a NULL descriptor reference is an argument error
    st = L.evo_validate(ctx._h, C.c_void_p(ptrs.ctypes.data), None, C.c_void_p(descs.ctypes.data), 4, evo.EVO_BF16, 0.01, 0.01,
                        C.c_void_p(res.data_ptr()), C.c_void_p(gp.data_ptr()), 4, None)
    assert st == -1

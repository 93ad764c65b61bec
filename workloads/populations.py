"""Seeded synthetic populations of candidate outputs.

These stand in for the outputs that evolved kernels produce on the paper's
operator suite (which is not available here): output tensors from a few
thousand elements to 1 GiB, fp32/fp16/bf16, most candidates equal to the
reference up to noise far below the tolerance, some with injected wrong
elements, NaN/Inf or a fully wrong output, and run-time samples spanning
slow-downs to >10x speed-ups.

This module only draws numbers (torch's seeded generators, on whichever device
is asked for) and arranges them.  It holds none of the evaluation arithmetic:
it serves the CUDA library and the CPU oracle alike, and neither depends on the
other.
"""
from dataclasses import dataclass, field
from typing import Dict, List, Optional

import torch

F32, F16, BF16 = 1, 2, 3
TORCH_DTYPE = {F32: torch.float32, F16: torch.float16, BF16: torch.bfloat16}
ELEM_BYTES = {F32: 4, F16: 2, BF16: 2}


@dataclass
class Tensor:
    """One candidate output tensor and the reference it is checked against."""
    cand: torch.Tensor
    ref_index: int          # index into Population.refs
    group: int              # candidate id: tensors of one candidate share a verdict
    dtype: int


@dataclass
class Population:
    name: str
    refs: List[torch.Tensor]
    tensors: List[Tensor]
    n_group: int
    atol: float
    rtol: float
    times: torch.Tensor                 # [n_group, trials] fp32, milliseconds
    base_times: torch.Tensor            # [base_trials] fp32
    facts: Dict[str, object] = field(default_factory=dict)   # what holds by construction

    def algorithmic_bytes(self) -> int:
        """Bytes the check must read: every candidate tensor once and every
        distinct reference once."""
        b = sum(t.cand.numel() * t.cand.element_size() for t in self.tensors)
        used = sorted({t.ref_index for t in self.tensors})
        b += sum(self.refs[i].numel() * self.refs[i].element_size() for i in used)
        return b

    def candidate_bytes(self) -> int:
        return sum(t.cand.numel() * t.cand.element_size() for t in self.tensors)


def _gen(device, seed):
    g = torch.Generator(device=device)
    g.manual_seed(int(seed))
    return g


def _times(n_rows, trials, seed, device, scale=None):
    """Run times in ms: scale_i * uniform[1, 2)."""
    g = _gen("cpu", seed)
    t = 1.0 + torch.rand((n_rows, trials), generator=g, dtype=torch.float32)
    if scale is not None:
        t = t * scale.reshape(-1, 1)
    return t.to(device)


def _tolerance(ref32, atol, rtol):
    # Size of an injected error relative to the check's tolerance; only used to
    # place wrong elements clearly outside or right at the boundary.
    return atol + rtol * ref32.abs()


def config1(device="cpu") -> Population:
    """One fp32 64x64 candidate, noise 1e-4, exactly 7 wrong elements (+1.0), 5 trials."""
    n, atol, rtol = 64 * 64, 1e-2, 1e-2
    g = _gen(device, 10)
    ref = torch.randn(n, generator=g, device=device, dtype=torch.float32)
    cand = ref + 1e-4 * torch.randn(n, generator=g, device=device, dtype=torch.float32)
    pos = torch.randperm(n, generator=_gen("cpu", 12))[:7].to(device)
    cand[pos] = ref[pos] + 1.0
    return Population("config1", [ref], [Tensor(cand, 0, 0, F32)], 1, atol, rtol,
                      _times(1, 5, 13, device), _times(1, 5, 14, device)[0],
                      facts={"n_mismatch": [7], "positions": pos.cpu().tolist()})


def config2(device="cpu", n=16 * 16384, k=8, trials=100) -> Population:
    """k fp32 candidates sharing one reference; noise 1e-5; wrong elements at rate 1e-4
    placed 10 tolerances away; atol = rtol = 1e-3."""
    atol, rtol = 1e-3, 1e-3
    g = _gen(device, 2000)
    ref = torch.randn(n, generator=g, device=device, dtype=torch.float32)
    tensors, injected = [], []
    for i in range(k):
        cand = ref + 1e-5 * torch.randn(n, generator=g, device=device, dtype=torch.float32)
        hit = torch.rand(n, generator=g, device=device) < 1e-4
        sign = torch.where(torch.rand(n, generator=g, device=device) < 0.5, -1.0, 1.0)
        cand = torch.where(hit, ref + sign * 10.0 * _tolerance(ref, atol, rtol), cand)
        injected.append(int(hit.sum().item()))
        tensors.append(Tensor(cand, 0, i, F32))
    return Population("config2", [ref], tensors, k, atol, rtol,
                      _times(k, trials, 2100, device), _times(1, trials, 2101, device)[0],
                      facts={"n_mismatch": injected})


def config3(device="cpu", n=1 << 20, k_per_dtype=64, special_rate=1e-6, boundary_rate=1e-3) -> Population:
    """k fp16 + k bf16 candidates against the narrowed reference; NaN / +Inf / -Inf at
    special_rate; values within a few 2^-8 steps of the tolerance boundary at boundary_rate."""
    atol, rtol = 1e-2, 1e-2
    g = _gen(device, 3000)
    ref32 = torch.randn(n, generator=g, device=device, dtype=torch.float32)
    refs = [ref32.to(torch.float16), ref32.to(torch.bfloat16)]
    tensors = []
    specials = torch.tensor([float("nan"), float("inf"), float("-inf")], device=device)
    gid = 0
    for ri, dt in enumerate((F16, BF16)):
        tdt = TORCH_DTYPE[dt]
        r = refs[ri].float()
        for _ in range(k_per_dtype):
            c = ref32 + 1e-4 * torch.randn(n, generator=g, device=device, dtype=torch.float32)
            near = torch.rand(n, generator=g, device=device) < boundary_rate
            j = torch.randint(-2, 3, (n,), generator=g, device=device).float()
            sign = torch.where(torch.rand(n, generator=g, device=device) < 0.5, -1.0, 1.0)
            c = torch.where(near, r + sign * _tolerance(r, atol, rtol) * (1.0 + j / 256.0), c)
            sp = torch.rand(n, generator=g, device=device) < special_rate
            which = torch.randint(0, 3, (n,), generator=g, device=device)
            c = torch.where(sp, specials[which], c)
            tensors.append(Tensor(c.to(tdt), ri, gid, dt))
            gid += 1
    return Population("config3", refs, tensors, gid, atol, rtol,
                      _times(gid, 100, 3100, device), _times(1, 100, 3101, device)[0])


def config4(device="cpu", n=1 << 28, k=16, seed=4000) -> Population:
    """k fp32 candidates of n elements against one reference, noise 1e-6; exactly one
    candidate is fully wrong (the reference rotated by n/2); atol = rtol = 1e-4.
    Another `seed` gives other tensors of the same kind (disjoint samples for parallel baselines)."""
    atol, rtol = 1e-4, 1e-4
    g = _gen(device, seed)
    ref = torch.randn(n, generator=g, device=device, dtype=torch.float32)
    wrong = int(torch.randint(0, k, (1,), generator=_gen("cpu", 4099)).item())
    tensors = []
    for i in range(k):
        if i == wrong:
            cand = torch.roll(ref, n // 2)
        else:
            cand = torch.randn(n, generator=g, device=device, dtype=torch.float32)
            cand.mul_(1e-6).add_(ref)
        tensors.append(Tensor(cand, 0, i, F32))
    return Population("config4", [ref], tensors, k, atol, rtol,
                      _times(k, 100, 4100, device), _times(1, 100, 4101, device)[0],
                      facts={"wrong": wrong})


def config5(device="cpu", n_cand=1024, log2_min=10.0, log2_max=24.0, trials=100) -> Population:
    """Ragged population: n_cand candidates with 1-3 output tensors each, sizes
    log-uniform in [2^log2_min, 2^log2_max], dtype per candidate fp32/fp16/bf16 with
    probability 1/2, 1/4, 1/4, one reference per tensor; 60 % of candidates clean, the rest
    with wrong elements at a rate log-uniform in [1e-7, 1e-2]; atol = rtol = 1e-2."""
    atol, rtol = 1e-2, 1e-2
    gc = _gen("cpu", 5000)
    g = _gen(device, 5001)
    refs, tensors, rates = [], [], []
    for cid in range(n_cand):
        n_out = int(torch.randint(1, 4, (1,), generator=gc).item())
        u = float(torch.rand(1, generator=gc).item())
        dt = F32 if u < 0.5 else (F16 if u < 0.75 else BF16)
        clean = float(torch.rand(1, generator=gc).item()) < 0.6
        rate = 0.0 if clean else 10.0 ** (-7.0 + 5.0 * float(torch.rand(1, generator=gc).item()))
        rates.append(rate)
        for _ in range(n_out):
            n = int(2.0 ** (log2_min + (log2_max - log2_min) * float(torch.rand(1, generator=gc).item())))
            ref32 = torch.randn(n, generator=g, device=device, dtype=torch.float32)
            ref = ref32.to(TORCH_DTYPE[dt])
            r = ref.float()
            c = r + 1e-4 * torch.randn(n, generator=g, device=device, dtype=torch.float32)
            if rate > 0.0:
                hit = torch.rand(n, generator=g, device=device) < rate
                c = torch.where(hit, r + 10.0 * _tolerance(r, atol, rtol), c)
            refs.append(ref)
            tensors.append(Tensor(c.to(TORCH_DTYPE[dt]), len(refs) - 1, cid, dt))
    scale = 10.0 ** (-1.3 + 1.6 * torch.rand(n_cand, generator=gc))
    return Population("config5", refs, tensors, n_cand, atol, rtol,
                      _times(n_cand, trials, 5100, device, scale=scale.float()),
                      _times(1, trials, 5101, device)[0], facts={"rates": rates})


def clean16(device="cpu", n=1 << 26, k=8, dtype=BF16) -> Population:
    """k fp16 or bf16 candidates of n elements against one reference, every one the narrowed reference plus noise far
    below the tolerance (sigma 1e-6; atol = rtol = 1e-2): a large, clean 16-bit population, what the outputs of
    half-precision kernels that are simply right look like."""
    atol, rtol = 1e-2, 1e-2
    g = _gen(device, 6000)
    ref32 = torch.randn(n, generator=g, device=device, dtype=torch.float32)
    ref = ref32.to(TORCH_DTYPE[dtype])
    tensors = []
    for i in range(k):
        noise = torch.randn(n, generator=g, device=device, dtype=torch.float32)
        tensors.append(Tensor(noise.mul_(1e-6).add_(ref32).to(TORCH_DTYPE[dtype]), 0, i, dtype))
    return Population("clean16", [ref], tensors, k, atol, rtol,
                      _times(k, 100, 6100, device), _times(1, 100, 6101, device)[0])


def special_values(dtype=F32, device="cpu") -> Population:
    """Every pair from a set of special values (signed zeros, subnormals, ones and their
    neighbours, the largest finite value, infinities, NaN) as (candidate, reference)."""
    tdt = TORCH_DTYPE[dtype]
    fin = torch.finfo(tdt)
    base = [0.0, -0.0, fin.smallest_normal, -fin.smallest_normal, 1.0, -1.0, 1.0 + fin.eps, 1.0 - fin.eps / 2,
            fin.max, -fin.max, float("inf"), float("-inf"), float("nan"), 0.5, 1.5, -2.75, 1e-3, 65504.0]
    v = torch.tensor(base, dtype=torch.float64).to(tdt)
    tiny_bits = torch.tensor([1, -32767 if dtype != F32 else -2147483647], dtype=torch.int16 if dtype != F32 else torch.int32)
    v = torch.cat([v, tiny_bits.view(tdt)])            # +-smallest subnormal
    c, r = torch.meshgrid(v, v, indexing="ij")
    cand = c.reshape(-1).contiguous().to(device)
    ref = r.reshape(-1).contiguous().to(device)
    return Population("special_values", [ref], [Tensor(cand, 0, 0, dtype)], 1, 0.25, 0.25,
                      _times(1, 5, 1, device), _times(1, 5, 2, device)[0])


def shard_by_candidate(pop: Population, rank: int, world: int) -> List[int]:
    """Indices of the tensors a replica `rank` of `world` takes when a population is split by
    candidate id (candidates are independent: no exchange is needed, results concatenate)."""
    return [i for i, t in enumerate(pop.tensors) if t.group % world == rank]


def to_host_bits(t: torch.Tensor):
    """Host numpy view the oracle reads: float32 as is, fp16/bf16 as uint16 bit patterns."""
    t = t.detach().cpu().contiguous()
    if t.dtype == torch.float32:
        return t.numpy()
    return t.view(torch.int16).numpy().view("uint16")

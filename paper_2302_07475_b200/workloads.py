"""Seeded synthetic gradient batches shaped like the S3GD-MV workloads.

This module only *draws inputs*: it holds none of the method's arithmetic
(no top-K, no sign packing, no vote, no update) and is the one piece of code
that both the CUDA path's tests/benchmarks and the CPU oracle's tests use.

The paper trains a CNN (N = 5e5) and a ResNet-56 (N = 8.5e5) on MNIST and
CIFAR-10 (Section 4, simulation set-up) and motivates the method with a
2.1e9-parameter model (Section 1).  Neither the data sets nor trained weights
are available offline, so every workload here is a seeded random stand-in
with the same shape: M workers (rows) times d coordinates of fp32 gradients,
one fp32 parameter vector x, a sparsity K and the sign-method learning rate
1e-3 that Section 4 quotes.

Everything is generated with ``torch.Generator`` on the device asked for, row
by row and in bounded chunks, so a 67 GB batch never needs a second copy.
The same (name, step, device type) always yields the same bits; CPU and CUDA
generators differ from each other, which is fine because a test always
generates once and hands the very same tensor (or its host copy) to both the
oracle and the kernels.
"""
from __future__ import annotations

import dataclasses
import math
from typing import Dict, List, Optional, Tuple

import torch

BASE_SEED = 20230207  # arXiv id of the paper, used as the base seed
_CHUNK = 1 << 24      # elements generated per temporary


@dataclasses.dataclass(frozen=True)
class WorkloadSpec:
    """Shape and recipe of one synthetic workload."""

    name: str
    index: int                 # position in the list of published workload shapes
    d: int                     # model size (the paper's N)
    M: int                     # number of workers
    Ks: Tuple[int, ...]        # sparsity levels exercised on this shape
    recipe: str                # one of the _RECIPES keys
    n_blocks: int = 0          # number of contiguous "layer" blocks with their own scale
    steps: int = 1             # consecutive steps with fresh gradients
    lr: float = 1e-3           # learning rate of the sign methods, Section 4
    x_sigma: float = 0.1       # x ~ N(0, 0.01) read as variance 0.01


def _round_half_up(v: float) -> int:
    return int(math.floor(v + 0.5))


_D4 = 25_557_032

SPECS: Dict[str, WorkloadSpec] = {
    s.name: s
    for s in (
        WorkloadSpec("tiny", 0, 65_536, 5, (655,), "iid_normal"),
        WorkloadSpec("small_cnn", 1, 1_199_882, 10, (1_200, 12_000), "shared_plus_normal", steps=10),
        WorkloadSpec("resnet18", 2, 11_173_962, 100, (11_174, 11_173_962), "shared_plus_student_blocks", n_blocks=20),
        WorkloadSpec(
            "resnet50_ties", 3, _D4, 32,
            tuple(_round_half_up(g * _D4) for g in (1e-4, 1e-3, 1e-2, 1e-1)),
            "laplace_bf16",
        ),
        WorkloadSpec("large", 4, 2_100_000_000, 8, (2_100_000,), "normal_blocks", n_blocks=64),
    )
}


def spec(name: str, d: Optional[int] = None, M: Optional[int] = None,
         Ks: Optional[Tuple[int, ...]] = None) -> WorkloadSpec:
    """Return the named spec, optionally shrunk (same recipe, smaller d / M / other K)."""
    s = SPECS[name]
    changes = {}
    if d is not None:
        changes["d"] = int(d)
    if M is not None:
        changes["M"] = int(M)
    if Ks is not None:
        changes["Ks"] = tuple(int(k) for k in Ks)
    return dataclasses.replace(s, **changes) if changes else s


def _gen(device: torch.device, seed: int) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(seed)
    return g


def _seed(s: WorkloadSpec, step: int, stream: int) -> int:
    # one independent stream per (workload, step, purpose/worker)
    return BASE_SEED + 1_000_003 * s.index + 10_007 * step + 101 * stream


def block_scales(s: WorkloadSpec, device: torch.device) -> Tuple[List[int], torch.Tensor]:
    """Boundaries and scales of the contiguous 'layer' blocks of a workload.

    Block lengths are proportional to seeded uniform weights in [0.2, 1.8], so
    blocks differ in length by up to 9x; scales are log-uniform in
    [1e-4, 1e-1].  Both depend on the workload only (not on step or worker).
    Drawn on the CPU so that the blocks are the same for every device.
    """
    g = _gen(torch.device("cpu"), _seed(s, 0, 7))
    w = torch.rand(s.n_blocks, generator=g, dtype=torch.float64) * 1.6 + 0.2
    cuts = torch.cumsum(w, 0) / w.sum() * s.d
    bounds = [0] + [int(c) for c in cuts[:-1].tolist()] + [s.d]
    for i in range(1, len(bounds)):            # keep boundaries non-decreasing on tiny d
        bounds[i] = max(bounds[i], bounds[i - 1])
    e = torch.rand(s.n_blocks, generator=g, dtype=torch.float64) * 3.0 - 4.0
    scales = torch.pow(torch.tensor(10.0, dtype=torch.float64), e).to(torch.float32)
    return bounds, scales.to(device)


def _scale_slice(bounds: List[int], scales: torch.Tensor, lo: int, hi: int) -> torch.Tensor:
    """Per-coordinate block scale for coordinates [lo, hi)."""
    out = torch.empty(hi - lo, dtype=torch.float32, device=scales.device)
    for b in range(len(bounds) - 1):
        a, z = max(bounds[b], lo), min(bounds[b + 1], hi)
        if a < z:
            out[a - lo:z - lo] = scales[b]
    return out


def _fill_row(s: WorkloadSpec, row: torch.Tensor, m: int, step: int,
              blocks: Optional[Tuple[List[int], torch.Tensor]]) -> None:
    """Write worker m's gradient for the given step into ``row`` (length d, fp32)."""
    dev = row.device
    g_own = _gen(dev, _seed(s, step, 1000 + m))
    g_shared = _gen(dev, _seed(s, step, 3))     # same stream for every worker
    for lo in range(0, s.d, _CHUNK):
        hi = min(s.d, lo + _CHUNK)
        n = hi - lo
        out = row[lo:hi]
        if s.recipe == "iid_normal":
            out.normal_(generator=g_own)
        elif s.recipe == "shared_plus_normal":
            shared = torch.empty(n, dtype=torch.float32, device=dev).normal_(generator=g_shared)
            out.normal_(generator=g_own)
            out.add_(shared, alpha=0.5)
        elif s.recipe == "shared_plus_student_blocks":
            shared = torch.empty(n, dtype=torch.float32, device=dev).normal_(generator=g_shared)
            z = torch.empty(n, dtype=torch.float32, device=dev).normal_(generator=g_own)
            chi = torch.zeros(n, dtype=torch.float32, device=dev)
            tmp = torch.empty(n, dtype=torch.float32, device=dev)
            for _ in range(3):                   # chi-square with nu = 3 degrees of freedom
                tmp.normal_(generator=g_own)
                chi.addcmul_(tmp, tmp)
            z.div_(torch.sqrt_(chi.div_(3.0)))   # Student-t(3)
            z.mul_(_scale_slice(blocks[0], blocks[1], lo, hi))
            z.add_(shared, alpha=0.3)
            out.copy_(z)
        elif s.recipe == "laplace_bf16":
            u = torch.empty(n, dtype=torch.float32, device=dev).uniform_(-0.5, 0.5, generator=g_own)
            mag = torch.log1p(-2.0 * u.abs().clamp_(max=0.4999999)).neg_()
            lap = torch.where(u < 0, -mag, mag)
            out.copy_(lap.to(torch.bfloat16).to(torch.float32))   # bf16 grid => many exact ties
        elif s.recipe == "normal_blocks":
            out.normal_(generator=g_own)
            out.mul_(_scale_slice(blocks[0], blocks[1], lo, hi))
        else:  # pragma: no cover
            raise ValueError(f"unknown recipe {s.recipe}")


def make_grads(s: WorkloadSpec, device, step: int = 0,
               out: Optional[torch.Tensor] = None) -> torch.Tensor:
    """[M, d] fp32 gradients of one step, row-major and contiguous."""
    device = torch.device(device)
    if out is None:
        out = torch.empty((s.M, s.d), dtype=torch.float32, device=device)
    assert out.shape == (s.M, s.d) and out.dtype == torch.float32 and out.is_contiguous()
    blocks = block_scales(s, device) if s.n_blocks else None
    for m in range(s.M):
        _fill_row(s, out[m], m, step, blocks)
    return out


def make_rows(s: WorkloadSpec, rows, device, step: int = 0) -> torch.Tensor:
    """[len(rows), d]: the listed workers' rows of make_grads(s, device, step), without drawing the others."""
    device = torch.device(device)
    rows = list(rows)
    out = torch.empty((len(rows), s.d), dtype=torch.float32, device=device)
    blocks = block_scales(s, device) if s.n_blocks else None
    for i, m in enumerate(rows):
        _fill_row(s, out[i], int(m), step, blocks)
    return out


def make_x(s: WorkloadSpec, device) -> torch.Tensor:
    """[d] fp32 parameters, N(0, x_sigma^2)."""
    device = torch.device(device)
    x = torch.empty(s.d, dtype=torch.float32, device=device)
    g = _gen(device, _seed(s, 0, 5))
    for lo in range(0, s.d, _CHUNK):
        x[lo:min(s.d, lo + _CHUNK)].normal_(generator=g)
    return x.mul_(s.x_sigma)


def edge_case_grads(kind: str, M: int, d: int, device="cpu", seed: int = 0) -> torch.Tensor:
    """Small structured inputs for the degenerate cases of top-K selection.

    kinds: 'all_equal' (every magnitude ties), 'zeros' (+0 and -0 only),
    'few_levels' (magnitudes from a 5-value set, random signs), 'one_hot'
    (a single large entry per row), 'special' (Inf, NaN, denormals mixed in),
    'ramp' (strictly increasing magnitudes), 'ramp_down'.
    """
    device = torch.device(device)
    g = _gen(torch.device("cpu"), BASE_SEED ^ (seed * 7919 + 13))
    sign = torch.where(torch.rand((M, d), generator=g) < 0.5, -1.0, 1.0).to(torch.float32)
    if kind == "all_equal":
        out = sign * 0.75
    elif kind == "zeros":
        out = sign * 0.0
    elif kind == "few_levels":
        lv = torch.tensor([0.0, 0.125, 0.5, 0.5000001, 2.0], dtype=torch.float32)
        out = sign * lv[torch.randint(0, 5, (M, d), generator=g)]
    elif kind == "one_hot":
        out = torch.zeros((M, d), dtype=torch.float32)
        pos = torch.randint(0, d, (M,), generator=g)
        out[torch.arange(M), pos] = 3.0
        out = out * sign
    elif kind == "special":
        out = torch.randn((M, d), generator=g, dtype=torch.float32)
        sp = torch.tensor([float("inf"), float("-inf"), float("nan"), 1e-42, -1e-45, 0.0, -0.0, 3.4e38],
                          dtype=torch.float32)
        mask = torch.rand((M, d), generator=g) < 0.05
        out = torch.where(mask, sp[torch.randint(0, sp.numel(), (M, d), generator=g)], out)
    elif kind == "ramp":
        out = sign * (torch.arange(1, d + 1, dtype=torch.float32) / d).expand(M, d)
    elif kind == "ramp_down":
        out = sign * (torch.arange(d, 0, -1, dtype=torch.float32) / d).expand(M, d)
    else:
        raise ValueError(kind)
    return out.contiguous().to(device)

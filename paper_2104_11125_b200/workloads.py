"""Seeded synthetic inputs for the CLT-k step.

This module only draws random tensors; it contains none of the method's
arithmetic, so both the CUDA path and the CPU checker may be fed from it.

The paper measures on gradients of ImageNet / CIFAR10 / WMT14 / SWB300 models
(Tables 2-3).  None of those datasets is available, so seeded tensors with
the parameter counts of the named models, the paper's compression ratios
(k = d/100 for the ~100X rows, k = d/400 for the 400X row) and positively
correlated learners (Section 2, "memory similarity") stand in for them:
every learner's gradient is  g_i = shared + c * independent_i.

Streams are keyed by (workload id, step, learner or "shared"), so a given
(workload, step) always yields the same bits on a given device type.  CPU and
CUDA samplers differ, so a test draws once and copies the bits.
"""
from __future__ import annotations

import dataclasses
import math
from typing import List, Sequence, Tuple

import torch

BASE_SEED = 20210411


@dataclasses.dataclass(frozen=True)
class Workload:
    name: str
    wid: int            # stream id
    kind: str           # "iid" | "resnet50" | "transformer" | "gpt2m"
    n: int              # learners
    d: int              # coordinates per learner
    k: int              # kept coordinates
    beta: float
    lr: float
    steps: int
    c: float            # weight of the independent part in g_i = shared + c*indep_i

    @property
    def ratio(self) -> float:
        return self.d / self.k

    def scaled(self, d: int, n: int | None = None, steps: int | None = None) -> "Workload":
        """Same recipe at another size (k keeps the same compression ratio)."""
        k = max(1, (d * self.k) // self.d)
        return dataclasses.replace(self, name=f"{self.name}@d={d}", d=d, k=k,
                                   n=self.n if n is None else n,
                                   steps=self.steps if steps is None else steps)


def _w(name, wid, kind, n, d, ratio, steps, c) -> Workload:
    return Workload(name, wid, kind, n, d, d // ratio, 0.1, 0.01, steps, c)


TINY = _w("tiny", 1, "iid", 4, 1 << 20, 100, 10, 0.5)
RESNET50 = _w("resnet50", 2, "resnet50", 8, 25_557_032, 100, 20, 0.3)
TRANSFORMER = _w("transformer_base", 3, "transformer", 16, 61_000_000, 400, 20, 0.5)
LARGE = _w("gpt2_medium", 5, "gpt2m", 32, 354_000_000, 400, 5, 0.5)
SWEEP_N = (8, 32, 64, 128)


def sweep(n: int) -> Workload:
    return dataclasses.replace(RESNET50, name=f"resnet50_n{n}", wid=4, n=n, steps=10)


CONFIGS = {w.name: w for w in (TINY, RESNET50, TRANSFORMER, LARGE)}


def resnet50_segments() -> List[int]:
    """Tensor sizes of a bottleneck ResNet-50 classifier in definition order:
    a 7x7x3->64 stem convolution, stages of [3,4,6,3] blocks of widths
    64/128/256/512 (each block: 1x1, 3x3, 1x1 to 4x width; each convolution
    followed by a scale and a shift vector; a 1x1 projection in each stage's
    first block), and a 2048->1000 linear layer with bias."""
    sizes: List[int] = []

    def conv_norm(cin, cout, ksz):
        sizes.extend([cout * cin * ksz * ksz, cout, cout])

    conv_norm(3, 64, 7)
    cin = 64
    for width, blocks in ((64, 3), (128, 4), (256, 6), (512, 3)):
        for b in range(blocks):
            conv_norm(cin, width, 1)
            conv_norm(width, width, 3)
            conv_norm(width, 4 * width, 1)
            if b == 0:
                conv_norm(cin, 4 * width, 1)
            cin = 4 * width
    sizes.extend([2048 * 1000, 1000])
    return sizes


def segments(w: Workload) -> List[Tuple[int, int]]:
    """(offset, size) of each per-layer segment of the flat d-vector."""
    if w.kind == "resnet50":
        base = resnet50_segments()
    elif w.kind == "gpt2m":
        base = [1] * 24
    else:
        return [(0, w.d)]
    total = sum(base)
    sizes = [max(1, (s * w.d) // total) for s in base] if total != w.d else list(base)
    big = max(range(len(sizes)), key=lambda i: sizes[i])      # rounding slack goes to the largest segment
    sizes[big] += w.d - sum(sizes)
    if sizes[big] < 1:
        raise ValueError("d too small for the segment layout")
    out, off = [], 0
    for s in sizes:
        out.append((off, s))
        off += s
    return out


def _gen(device, *key) -> torch.Generator:
    seed = BASE_SEED
    for x in key:
        seed = (seed * 1_000_003 + int(x) + 1) % (2 ** 62)
    g = torch.Generator(device=device)
    g.manual_seed(seed)
    return g


@dataclasses.dataclass
class Profile:
    """Per-coordinate description of the gradient distribution (fixed per workload)."""
    scale: torch.Tensor | None        # fp32[d] per-coordinate sigma, or None for 1
    laplace: torch.Tensor | None      # bool[d] coordinates drawn from a Laplace law
    sigma: float = 1.0                # scale of the non-Laplace coordinates
    b: float = 1.0                    # Laplace scale


def profile(w: Workload, device) -> Profile:
    device = torch.device(device)
    if w.kind == "iid":
        return Profile(None, None)
    if w.kind == "resnet50":
        segs = segments(w)
        u = torch.rand(len(segs), generator=_gen("cpu", w.wid, 0, 10_001), dtype=torch.float64)
        sig = torch.exp(math.log(1e-4) + u * (math.log(1e-1) - math.log(1e-4))).to(torch.float32)
        sizes = torch.tensor([s for _, s in segs])
        return Profile(torch.repeat_interleave(sig, sizes).to(device), None)
    if w.kind == "gpt2m":
        segs = segments(w)
        sig = torch.tensor([1e-3 / math.sqrt(l + 1) for l in range(len(segs))], dtype=torch.float32)
        sizes = torch.tensor([s for _, s in segs])
        return Profile(torch.repeat_interleave(sig, sizes).to(device), None)
    if w.kind == "transformer":
        mask = torch.rand(w.d, generator=_gen(device, w.wid, 0, 10_002), device=device) < 0.4
        return Profile(None, mask, sigma=1e-4, b=1e-3)
    raise ValueError(w.kind)


def _draw(w: Workload, prof: Profile, gen: torch.Generator, device) -> torch.Tensor:
    x = torch.randn(w.d, generator=gen, device=device, dtype=torch.float32)
    if prof.laplace is not None:
        x.mul_(prof.sigma)
        u = torch.rand(w.d, generator=gen, device=device, dtype=torch.float32).sub_(0.5)
        u.clamp_(-0.49999997, 0.49999997)                  # keeps log1p finite: |x| <= 16.7 b
        lap = torch.sign(u).mul_(torch.log1p(-2.0 * u.abs()).mul_(-prof.b))
        x = torch.where(prof.laplace, lap, x)
    elif prof.scale is not None:
        x.mul_(prof.scale)
    return x


def gradients(w: Workload, step: int, device, prof: Profile | None = None,
              learners: Sequence[int] | None = None) -> List[torch.Tensor]:
    """The n (or the listed) learners' gradients of one step: g_i = shared + c * indep_i."""
    device = torch.device(device)
    prof = prof if prof is not None else profile(w, device)
    shared = _draw(w, prof, _gen(device, w.wid, step + 1, 0), device)
    out = []
    for i in (range(w.n) if learners is None else learners):
        e = _draw(w, prof, _gen(device, w.wid, step + 1, i + 1), device)
        out.append(e.mul_(w.c).add_(shared))
    return out


def initial_weights(w: Workload, device) -> torch.Tensor:
    return torch.randn(w.d, generator=_gen(device, w.wid, 0, 10_003), device=device,
                       dtype=torch.float32).mul_(0.02)


def initial_memory(w: Workload, device) -> List[torch.Tensor]:
    """Algorithm 1's input line: every learner's memory starts at zero."""
    return [torch.zeros(w.d, device=device, dtype=torch.float32) for _ in range(w.n)]


def resnet50_layer_keep(w: Workload) -> Tuple[List[int], List[int]]:
    """(sizes, keep) per tensor for the paper's per-layer rate rule (Section 4): 25X where a weight is
    used in >= 196 multiply-adds per sample, 50X in [128, 196), 400X below, first convolution sent whole.
    For an ImageNet ResNet-50 the uses per weight are the output positions of the layer: 112^2 for the
    stem, 56^2 / 28^2 / 14^2 / 7^2 in the four stages, 1 for the classifier."""
    segs = segments(w)
    uses = [112 * 112] * 3                                   # stem conv + its two norm vectors
    for width, blocks, hw in ((64, 3, 56), (128, 4, 28), (256, 6, 14), (512, 3, 7)):
        for b in range(blocks):
            uses += [hw * hw] * (9 + (3 if b == 0 else 0))
    uses += [1, 1]
    assert len(uses) == len(segs)
    sizes, keep = [], []
    for i, ((_, size), u) in enumerate(zip(segs, uses)):
        rate = 1 if i == 0 else 25 if u >= 196 else 50 if u >= 128 else 400
        sizes.append(size)
        keep.append(max(1, size // rate))
    return sizes, keep

"""Parity on the selection kernel's fallback routes at sizes that use its full persistent grid.

The small cases of test_gpu_parity.py reach the same branches with a handful of blocks; here every
case has d >= 4 M, where the kernel runs all its co-resident blocks (two per SM), and every output is
compared element by element with the oracle's step:
  * a threshold hint that turns out useless (gradient scale jumps by 1e-3 and by 50 between steps):
    the hinted pass is undone and the step samples afresh;
  * more equal keys around rank k than the short boundary list holds: radix select over the
    candidate segments, down to the index digits;
  * vectors on which the pre-filter cannot work at all (all coordinates equal; nine tenths zero
    with k beyond the non-zeros): the exact route, every pass streaming g and m again;
  * config 2 for 16 steps from a cold start with the window method of test_gpu_fullsize.py,
    recording which route every step took.
"""
import numpy as np
import pytest
import torch

from paper_2104_11125_b200 import workloads as W

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
D = 4_000_003                      # > 296 blocks x 8192 coordinates: the full grid; odd: ragged tail


def _parity():
    from tests import parity
    return parity


def _full_grid(d, n, k):
    import paper_2104_11125_b200 as sc
    from paper_2104_11125_b200 import binding
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    with sc.Context(d, n, k, 0.5, 0.1) as ctx:
        assert ctx.query(binding.Q_TOPK_BLOCKS) == 2 * sms, "the case does not use the full selection grid"


def test_useless_hints_are_undone_at_full_grid():
    from paper_2104_11125_b200 import binding
    n, k = 2, D // 100
    _full_grid(D, n, k)
    gen = torch.Generator(device=DEV)
    gen.manual_seed(7)
    base = [[torch.randn(D, generator=gen, device=DEV) for _ in range(n)] for _ in range(3)]
    # steps 0-1 at scale 1, steps 2-4 a thousand times smaller (the hinted bound lies above every key: too
    # few survivors), steps 5-7 fifty times larger than the start (the bound lies far below: the candidate
    # segments overflow).  A small beta keeps the memories far below the gradients, so acc jumps with them.
    scales = [1.0, 1.0, 1e-3, 1e-3, 1e-3, 50.0, 50.0, 50.0]
    steps = [[g * s for g in base[t % 3]] for t, s in enumerate(scales)]
    m0 = [torch.zeros(D, device=DEV) for _ in range(n)]
    theta = torch.linspace(-1, 1, D, device=DEV)
    paths = _parity().run_and_compare(steps, m0, theta, k, 1e-3, 0.25, tag="scale-jumps")
    S, H = binding.PATH_SAMPLED, binding.PATH_HINTED
    assert paths[0] == S and paths[1] == H, paths
    # at both jumps a hint existed, failed, was undone, and the step sampled afresh ...
    assert paths[2] == S and paths[5] == S, paths
    # ... and the steps that follow find their way back to the hinted route
    assert paths[4] == H and paths[6] == H and paths[7] == H, paths


def test_tie_group_larger_than_the_boundary_list_at_full_grid():
    from paper_2104_11125_b200 import binding
    rng = np.random.default_rng(11)
    k = 40_000
    x = rng.standard_normal(D).astype(np.float32)
    tau = np.sort(np.abs(x))[-k]
    ties = rng.choice(D, 5000, replace=False)                      # 5000 copies of the k-th magnitude, both signs
    x[ties] = np.where(rng.random(5000) < 0.5, tau, -tau).astype(np.float32)
    g = [torch.tensor(x, device=DEV), torch.tensor(0.5 * x, device=DEV)]
    _full_grid(D, 2, k)
    m0 = [torch.zeros(D, device=DEV) for _ in range(2)]
    theta = torch.linspace(-1, 1, D, device=DEV)
    paths = _parity().run_and_compare([g, g, g], m0, theta, k, 0.5, 0.25, tag="5000-ties")
    assert paths[0] == binding.PATH_SAMPLED                        # the pre-filter held; the ties went digit by digit
    paths = _parity().run_and_compare([g, g], m0, theta, k, 0.5, 0.25, use_hint=False, tag="5000-ties-nohint")
    assert paths == [binding.PATH_SAMPLED] * 2


def test_exact_route_at_full_grid():
    from paper_2104_11125_b200 import binding
    rng = np.random.default_rng(13)
    theta = torch.linspace(-1, 1, D, device=DEV)
    # all coordinates equal: every key ties, the winners are the k lowest indices
    g = [torch.full((D,), 2.5, device=DEV), torch.full((D,), -2.5, device=DEV)]
    m0 = [torch.zeros(D, device=DEV) for _ in range(2)]
    paths = _parity().run_and_compare([g, g], m0, theta, 70_001, 0.5, 0.25, tag="all-equal")
    assert paths == [binding.PATH_EXACT] * 2, paths
    # nine tenths zero, k beyond the non-zeros: the k-th key is zero and the zeros win by index
    x = rng.standard_normal(D).astype(np.float32)
    x[rng.random(D) < 0.9] = 0.0
    nz = int(np.count_nonzero(x))
    g = [torch.tensor(x, device=DEV), torch.tensor(-0.5 * x, device=DEV)]
    paths = _parity().run_and_compare([g, g], m0, theta, nz + 12_345, 0.5, 0.25, tag="mostly-zero")
    assert paths == [binding.PATH_EXACT] * 2, paths
    # the same vector with k inside the non-zeros: the pre-filter works again
    paths = _parity().run_and_compare([g, g], m0, theta, nz // 3, 0.5, 0.25, tag="mostly-zero-small-k")
    assert paths[0] == binding.PATH_SAMPLED, paths


def test_config2_sixteen_steps_route_mix():
    """Config 2 at full size for 16 steps (every learner leads twice): selection in full and the
    other outputs inside windows, every step; the routes taken are asserted as a mix, not step by step."""
    from paper_2104_11125_b200 import binding
    from tests.test_gpu_fullsize import fullsize_case
    paths = fullsize_case(W.RESNET50, steps=16, strict_paths=False)
    assert paths[0] == binding.PATH_SAMPLED
    assert all(p in (binding.PATH_SAMPLED, binding.PATH_HINTED) for p in paths), paths
    assert paths.count(binding.PATH_HINTED) >= 13, paths           # the hint carries almost every step

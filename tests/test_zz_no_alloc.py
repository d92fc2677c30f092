"""The allocation-free selection entry point against the handle-based one.

Some users of the library cannot allocate device memory at the moment they
need a selection (all of the GPU's memory already belongs to their framework's
allocator or to a fixed partition, or they cannot afford cudaMalloc's
device-wide synchronisation), so scalecom_topk_static keeps its scratch in a
fixed array inside the library.  That array is shared by all calls and keeps
the previous call's contents, so this test makes several calls in a row, of
different sizes, and checks each against scalecom_step on the same inputs.
Collected last on purpose: a run that stops at the first failure has then
already run every other test.
"""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu

DEV = "cuda:0"


def _reference_indices(g, m, k):
    """out_idx of the existing entry point: scalecom_step with the one learner as leader."""
    import paper_2104_11125_b200 as sc
    d = g.numel()
    idx = torch.empty(k, device=DEV, dtype=torch.int32)
    val = torch.empty(k, device=DEV, dtype=torch.float32)
    with sc.Context(d, 1, k, 1.0, 0.0) as ctx:
        ctx.step([g], [m.clone()], None, 0, idx, val)
        assert ctx.status() == 0
    return idx


def _static_indices(g, m, k):
    from paper_2104_11125_b200 import binding
    idx = torch.full((k,), -1, device=DEV, dtype=torch.int32)
    status = torch.full((1,), -1, device=DEV, dtype=torch.int32)
    stream = torch.cuda.current_stream()
    rc = binding.scalecom_topk_static(g.data_ptr(), m.data_ptr(), g.numel(), k, idx.data_ptr(), status.data_ptr(),
                                      stream.cuda_stream)
    assert rc == 0, binding.strerror(rc)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    return idx


def test_static_selection_matches_handle_selection_on_consecutive_calls():
    from paper_2104_11125_b200 import binding
    gen = torch.Generator(device=DEV)
    gen.manual_seed(1234)
    cases = [(1 << 20, 10_485), (300_007, 3000), (1 << 20, 2621), (5000, 5000), (77, 1)]
    for d, k in cases + cases[:2]:                       # calls in a row share and reuse the scratch array
        g = torch.randn(d, generator=gen, device=DEV)
        m = 0.3 * torch.randn(d, generator=gen, device=DEV)
        got = _static_indices(g, m, k)
        want = _reference_indices(g, m, k)
        assert torch.equal(got, want), "d=%d k=%d: %d of %d indices differ" % (d, k, int((got != want).sum()), k)
    # heavy ties (index passes) and an all-zero vector (candidate list overflows, exact path);
    # the scratch they leave behind must not disturb the next call
    q = torch.randint(-2, 3, (200_000,), generator=gen, device=DEV).float()
    z = torch.zeros_like(q)
    assert torch.equal(_static_indices(q, z, 50_000), _reference_indices(q, z, 50_000))
    assert torch.equal(_static_indices(z, z, 1000), _reference_indices(z, z, 1000))
    g = torch.randn(400_000, generator=gen, device=DEV)
    assert torch.equal(_static_indices(g, z.new_zeros(400_000), 4000), _reference_indices(g, z.new_zeros(400_000), 4000))
    # sizes beyond the fixed scratch are refused before anything is launched
    big = binding.STATIC_MAX_D + 1
    assert binding.scalecom_topk_static(g.data_ptr(), g.data_ptr(), big, 10, g.data_ptr(), None, None) == binding.ERR_INVALID_ARG
    assert binding.scalecom_topk_static(g.data_ptr(), g.data_ptr(), 100, 101, g.data_ptr(), None, None) == binding.ERR_INVALID_ARG
    assert binding.scalecom_topk_static(None, g.data_ptr(), 100, 10, g.data_ptr(), None, None) == binding.ERR_NULL_PTR

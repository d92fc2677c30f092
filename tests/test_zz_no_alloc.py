"""The allocation-free selection entry point against the CPU oracle and the handle-based entry point.

Some users of the library cannot allocate device memory at the moment they
need a selection (all of the GPU's memory already belongs to their framework's
allocator or to a fixed partition, or they cannot afford cudaMalloc's
device-wide synchronisation), so scalecom_topk_static keeps its scratch in a
fixed array inside the library.  That array is shared by all calls and keeps
the previous call's contents, so this test makes several calls in a row, of
different sizes, and checks each one against the oracle's top-k of m + g
(and, as a second check, against scalecom_step on the same inputs); it also
checks that, after the first call, calls leave the device's free memory
exactly where it was.
Collected last on purpose: a run that stops at the first failure has then
already run every other test.
"""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu

DEV = "cuda:0"


def _oracle_indices(g, m, k):
    """Eq. 2 on acc = m + g by the CPU oracle (same fp32 sum, stable sort by magnitude, lower index on ties)."""
    import oracle
    acc = oracle.accumulate(g.cpu().numpy(), m.cpu().numpy())
    return oracle.topk(acc, k)[0]


def _handle_indices(g, m, k):
    """out_idx of the handle-based entry point: scalecom_step with the one learner as leader."""
    import paper_2104_11125_b200 as sc
    d = g.numel()
    idx = torch.empty(k, device=DEV, dtype=torch.int32)
    val = torch.empty(k, device=DEV, dtype=torch.float32)
    with sc.Context(d, 1, k, 1.0, 0.0) as ctx:
        ctx.step([g], [m.clone()], None, 0, idx, val)
        assert ctx.status() == 0
    return idx.cpu().numpy()


def _static_indices(g, m, k, idx=None, status=None):
    from paper_2104_11125_b200 import binding
    if idx is None:
        idx = torch.empty(k, device=DEV, dtype=torch.int32)
    if status is None:
        status = torch.empty(1, device=DEV, dtype=torch.int32)
    idx.fill_(-1)
    status.fill_(-1)
    stream = torch.cuda.current_stream()
    rc = binding.scalecom_topk_static(g.data_ptr(), m.data_ptr(), g.numel(), k, idx.data_ptr(), status.data_ptr(),
                                      stream.cuda_stream)
    assert rc == 0, binding.strerror(rc)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    return idx[:k].cpu().numpy()


def _check(g, m, k, tag):
    got = _static_indices(g, m, k)
    want = _oracle_indices(g, m, k)
    assert np.array_equal(got, want), "%s: %d of %d indices differ from the oracle" % (tag, int((got != want).sum()), k)
    assert np.array_equal(got, _handle_indices(g, m, k)), "%s: differs from scalecom_step" % tag


def _offset_by_one_float(x):
    """The same values 4 bytes past a 16-byte boundary (the entry point's path for unaligned vectors)."""
    buf = torch.empty(x.numel() + 8, device=DEV, dtype=torch.float32)
    v = buf[1:1 + x.numel()]
    v.copy_(x)
    assert v.data_ptr() % 16 == 4
    return v


def test_static_selection_matches_oracle_on_consecutive_calls():
    from paper_2104_11125_b200 import binding
    gen = torch.Generator(device=DEV)
    gen.manual_seed(1234)
    cases = [(1 << 20, 10_485), (300_007, 3000), (1 << 20, 2621), (5000, 5000), (77, 1)]
    for d, k in cases + cases[:2]:                       # calls in a row share and reuse the scratch array
        g = torch.randn(d, generator=gen, device=DEV)
        m = 0.3 * torch.randn(d, generator=gen, device=DEV)
        _check(g, m, k, "d=%d k=%d" % (d, k))
    # vectors that do not start on a 16-byte boundary take the kernel's other instantiation
    g = torch.randn(200_003, generator=gen, device=DEV)
    m = 0.3 * torch.randn(200_003, generator=gen, device=DEV)
    _check(_offset_by_one_float(g), _offset_by_one_float(m), 2000, "unaligned")
    # heavy ties (index passes) and an all-zero vector (candidate list overflows, exact path);
    # the scratch they leave behind must not disturb the next call
    q = torch.randint(-2, 3, (200_000,), generator=gen, device=DEV).float()
    z = torch.zeros_like(q)
    _check(q, z, 50_000, "quantised")
    _check(z, z.clone(), 1000, "all-zero")
    g = torch.randn(400_000, generator=gen, device=DEV)
    _check(g, z.new_zeros(400_000), 4000, "after the degenerate cases")
    # sizes beyond the fixed scratch are refused before anything is launched
    big = binding.STATIC_MAX_D + 1
    assert binding.scalecom_topk_static(g.data_ptr(), g.data_ptr(), big, 10, g.data_ptr(), None, None) == binding.ERR_INVALID_ARG
    assert binding.scalecom_topk_static(g.data_ptr(), g.data_ptr(), 100, 101, g.data_ptr(), None, None) == binding.ERR_INVALID_ARG
    assert binding.scalecom_topk_static(None, g.data_ptr(), 100, 10, g.data_ptr(), None, None) == binding.ERR_NULL_PTR


def test_static_selection_allocates_nothing_after_its_first_call():
    """The entry point's contract: once the first call on the device has been made, further calls leave the
    device's free memory untouched (the outputs are preallocated here, so nothing else allocates either)."""
    gen = torch.Generator(device=DEV)
    gen.manual_seed(99)
    d, k = 1 << 20, 10_000
    g = torch.randn(d, generator=gen, device=DEV)
    m = torch.zeros(d, device=DEV)
    idx = torch.empty(k, device=DEV, dtype=torch.int32)
    status = torch.empty(1, device=DEV, dtype=torch.int32)
    first = _static_indices(g, m, k, idx, status)        # (the first call on a device may place the array)
    torch.cuda.synchronize()
    free0, _ = torch.cuda.mem_get_info()
    for kk in (k, 1, 5000, k):
        got = _static_indices(g, m, kk, idx, status)
        assert got.shape == (kk,)
    torch.cuda.synchronize()
    free1, _ = torch.cuda.mem_get_info()
    assert free1 == free0, "free device memory moved by %d bytes over four calls" % (free0 - free1)
    assert np.array_equal(first, _oracle_indices(g, m, k))

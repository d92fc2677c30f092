"""GPU parity: the CUDA library (through its C ABI) against the CPU oracle."""
import numpy as np
import pytest
import torch

from paper_2104_11125_b200 import workloads as W

pytestmark = pytest.mark.gpu

DEV = "cuda:0"


def _parity():
    from tests import parity
    return parity


def _t(a):
    return torch.tensor(np.asarray(a, np.float32), device=DEV)


# ---- the paper-shaped workloads at sizes the oracle finishes in seconds ---------------------------
@pytest.mark.parametrize("force_exact", [False, True])
def test_tiny_config_full(force_exact):
    """Config 1 exactly as specified: n=4, d=2^20, k=d/100, 10 steps, leader t mod 4."""
    _parity().workload_case(W.TINY, W.TINY.steps if not force_exact else 3, DEV, force_exact=force_exact,
                            want_path=1 if force_exact else 0)


@pytest.mark.parametrize("base,d,n,steps", [
    (W.RESNET50, 1_500_013, 8, 4),          # several tiles of every kernel plus a ragged tail (d odd)
    (W.TRANSFORMER, 2_000_003, 16, 3),
    (W.LARGE, 3_000_001, 5, 3),
    (W.RESNET50, 300_007, 20, 3),           # > 16 learners: second pointer-table size
    (W.RESNET50, 50_001, 130, 2),           # > 128 learners: third pointer-table size
    (W.TINY, 300_007, 1, 3), (W.TINY, 300_007, 2, 3), (W.TINY, 300_007, 3, 4), (W.TINY, 300_007, 6, 3),   # every burst shape
    (W.TINY, 300_007, 9, 2), (W.TINY, 300_007, 11, 2), (W.TINY, 300_007, 13, 2), (W.TINY, 300_007, 15, 2),
])
def test_scaled_workloads(base, d, n, steps):
    _parity().workload_case(base.scaled(d, n=n), steps, DEV, want_path=0)


def test_separate_update_kernel_and_no_weights():
    w = W.TINY.scaled(200_000)
    _parity().workload_case(w, 3, DEV, fuse_update=False)
    p = _parity()
    prof = W.profile(w, DEV)
    grads = [W.gradients(w, s, DEV, prof) for s in range(2)]
    p.run_and_compare(grads, W.initial_memory(w, DEV), None, w.k, w.beta, w.lr, tag="no-weights")


@pytest.mark.parametrize("offset", [1, 2, 3])
def test_unaligned_vectors(offset):
    w = W.TINY.scaled(100_003)
    _parity().workload_case(w, 2, DEV, offset=offset)
    _parity().workload_case(w, 2, DEV, offset=offset, force_exact=True)


# ---- edge cases -------------------------------------------------------------------------------------
def _edge(g_rows, k, beta=0.5, lr=0.25, steps=3, m_rows=None, **kw):
    g = [_t(r) for r in g_rows]
    n, d = len(g), g[0].numel()
    m0 = [_t(r) for r in m_rows] if m_rows is not None else [torch.zeros(d, device=DEV) for _ in range(n)]
    theta = torch.linspace(-1, 1, d, device=DEV)
    return _parity().run_and_compare([g] * steps, m0, theta, k, beta, lr, **kw)


@pytest.mark.parametrize("force_exact", [False, True])
def test_degenerate_inputs(force_exact):
    rng = np.random.default_rng(5)
    kw = dict(force_exact=force_exact)
    _edge([[3.0]], 1, tag="d=1", **kw)
    _edge([[0.0, 0.0, 0.0, 0.0, 0.0]] * 2, 2, tag="all-zero", **kw)
    _edge([np.zeros(5000)] * 3, 77, tag="all-zero-5000", **kw)
    _edge([np.full(4099, 2.5), np.full(4099, -2.5)], 100, tag="all-equal", **kw)
    pm = np.where(np.arange(9001) % 2 == 0, 1.0, -1.0)
    _edge([pm, -pm, pm], 4500, tag="plus-minus-ties", **kw)
    x = rng.standard_normal(10_000)
    _edge([x, x * 0.5], 1, tag="k=1", **kw)
    _edge([x, x * 0.5], 10_000, tag="k=d", **kw)
    _edge([x], 100, beta=1.0, tag="n=1,beta=1", **kw)
    den = (rng.integers(-5, 6, 7001) * 1e-41).astype(np.float32)
    _edge([den, den[::-1].copy()], 300, tag="denormals", **kw)
    q = rng.integers(-3, 4, 50_000).astype(np.float32)          # heavy ties at every level
    _edge([q, np.roll(q, 1)], 5000, tag="quantised", **kw)
    neg0 = np.array([-0.0, 0.0, -0.0, 1.0, -1.0, 0.0, -0.0], np.float32)
    _edge([neg0, -neg0], 3, tag="signed-zeros", **kw)


def test_ties_straddling_rank_k_on_the_fast_path():
    """Equal magnitudes on both sides of rank k with the candidate list in use:
    the winners among equals must be the lowest indices."""
    rng = np.random.default_rng(9)
    d, k = 400_000, 4000
    x = rng.standard_normal(d).astype(np.float32)
    order = np.argsort(-np.abs(x))
    tau = abs(x[order[k - 1]])
    ties = rng.choice(d, 600, replace=False)
    x[ties] = np.where(rng.random(600) < 0.5, tau, -tau)        # ~600 copies of the k-th magnitude
    paths = _edge([x, 0.9 * x, 1.1 * x], k, steps=3, tag="ties-at-k")
    assert paths[0] == 0
    paths = _edge([x, 0.9 * x, 1.1 * x], k, steps=3, use_hint=False, tag="ties-at-k-nohint")
    assert paths == [0, 0, 0]


def test_many_learners_small_vector():
    w = W.RESNET50.scaled(20_011, n=128)
    _parity().workload_case(w, 2, DEV)


def test_resume_equals_uninterrupted_run():
    """All state is the caller's: 4 steps with one handle == 2 + 2 steps with two handles."""
    import paper_2104_11125_b200 as sc
    w = W.TINY.scaled(150_001)
    prof = W.profile(w, DEV)
    grads = [W.gradients(w, s, DEV, prof) for s in range(4)]

    def run(split):
        m = W.initial_memory(w, DEV)
        th = W.initial_weights(w, DEV)
        idx = torch.empty(w.k, device=DEV, dtype=torch.int32)
        val = torch.empty(w.k, device=DEV)
        outs = []
        for lo, hi in split:
            with sc.Context(w.d, w.n, w.k, w.beta, w.lr) as ctx:
                for t in range(lo, hi):
                    ctx.step(grads[t], m, th, t, idx, val)
                    outs.append((idx.clone(), val.clone()))
                assert ctx.status() == 0
        return m, th, outs

    m1, th1, o1 = run([(0, 4)])
    m2, th2, o2 = run([(0, 2), (2, 4)])
    assert all(torch.equal(a, b) for a, b in zip(m1, m2)) and torch.equal(th1, th2)
    assert all(torch.equal(a[0], b[0]) and torch.equal(a[1], b[1]) for a, b in zip(o1, o2))


def test_host_buffer_entry_point():
    import paper_2104_11125_b200 as sc
    import oracle
    w = W.TINY.scaled(120_000)
    prof = W.profile(w, DEV)
    m = W.initial_memory(w, DEV)
    th = W.initial_weights(w, DEV)
    m_o = [x.cpu().numpy().copy() for x in m]
    th_o = th.cpu().numpy().copy()
    hidx = torch.empty(w.k, dtype=torch.int32).pin_memory()
    hval = torch.empty(w.k, dtype=torch.float32).pin_memory()
    with sc.Context(w.d, w.n, w.k, w.beta, w.lr) as ctx:
        for t in range(3):
            hg = [g.cpu().pin_memory() for g in W.gradients(w, t, DEV, prof)]
            ctx.step_host(hg, m, th, t, hidx, hval)
            idx_o, val_o, _ = oracle.step([g.numpy() for g in hg], m_o, th_o, t, w.k, w.beta, w.lr)
            assert np.array_equal(hidx.numpy(), idx_o) and np.array_equal(hval.numpy(), val_o)
        assert ctx.status() == 0
    assert all(np.array_equal(a.cpu().numpy(), b) for a, b in zip(m, m_o))
    assert np.array_equal(th.cpu().numpy(), th_o)


@pytest.mark.parametrize("selector", ["topk", "topk-two-kernels", "chunk", "layer_topk"])
def test_bounded_wait_expiry_is_reported_and_recoverable(selector):
    """Failure detection without a GPU fault: with the barrier's iteration bound set to 0 every
    wait gives up at once, the kernel returns, the status word says TIMEOUT, the kernels that follow it in
    the step do nothing (outputs and memory untouched), the handle refuses work until it is reset, and after
    the reset the same handle gives right results again."""
    import oracle
    import paper_2104_11125_b200 as sc
    from paper_2104_11125_b200 import binding
    w = W.TINY.scaled(200_000)                      # 25 blocks in the selection kernel, 148 in the one-kernel step
    two_kernels = selector == "topk-two-kernels"    # "topk" alone: the one-kernel step this size takes by default
    selector = "topk" if two_kernels else selector
    prof = W.profile(w, DEV)
    g = W.gradients(w, 0, DEV, prof)
    idx = torch.full((w.k,), -7, device=DEV, dtype=torch.int32)
    val = torch.full((w.k,), 3.5, device=DEV)
    sizes, keep = [w.d // 2, w.d - w.d // 2], [w.k // 4, w.k - w.k // 4]
    layers = (sizes, keep) if selector == "layer_topk" else None
    with sc.Context(w.d, w.n, w.k, w.beta, w.lr) as ctx:
        ctx.set_option(binding.OPT_SELECTOR, {"topk": binding.SELECTOR_TOPK, "chunk": binding.SELECTOR_CHUNK,
                                              "layer_topk": binding.SELECTOR_LAYER_TOPK}[selector])
        if layers:
            ctx.set_layers(*layers)
        ctx.set_option(binding.OPT_FUSED_SMALL, 0 if two_kernels else 1)
        assert (ctx.query(binding.Q_FUSED_SMALL) > 0) == (selector == "topk" and not two_kernels)
        ctx.set_option(binding.OPT_SPIN_LIMIT, 0)
        m = [torch.full((w.d,), 0.25, device=DEV) for _ in range(w.n)]
        theta = torch.full((w.d,), 1.5, device=DEV)
        ctx.step(g, m, theta, 0, idx, val)
        assert ctx.status() == binding.ERR_TIMEOUT
        assert bool((idx == -7).all()) and bool((val == 3.5).all()) and bool((theta == 1.5).all())
        assert all(bool((x == 0.25).all()) for x in m)
        with pytest.raises(sc.ScaleComError) as ei:
            ctx.step(g, m, None, 0, idx, val)
        assert ei.value.code == binding.ERR_BAD_STATE
        ctx.set_option(binding.OPT_SPIN_LIMIT, 1 << 22)
        ctx.reset()
        assert ctx.status() == 0
        # the same handle after the reset, against the oracle
        m_g = W.initial_memory(w, DEV)
        m_o = [x.cpu().numpy().copy() for x in m_g]
        ctx.step(g, m_g, None, 0, idx, val)
        assert ctx.status() == 0
        idx_o, val_o, _ = oracle.step([x.cpu().numpy() for x in g], m_o, None, 0, w.k, w.beta, w.lr, want_gathered=False,
                                      selector="topk" if selector == "layer_topk" else selector, layers=layers)
        assert np.array_equal(idx.cpu().numpy(), idx_o) and np.array_equal(val.cpu().numpy(), val_o)
        assert all(np.array_equal(a.cpu().numpy(), b) for a, b in zip(m_g, m_o))
    if selector == "topk":
        _parity().workload_case(w, 2, DEV)          # a fresh handle on the same device is unaffected


def test_argument_checks_on_device_pointers():
    import paper_2104_11125_b200 as sc
    from paper_2104_11125_b200 import binding as b
    d, n, k = 1000, 2, 10
    g = [torch.zeros(d, device=DEV) for _ in range(n)]
    m = [torch.zeros(d, device=DEV) for _ in range(n)]
    idx = torch.empty(k, device=DEV, dtype=torch.int32)
    val = torch.empty(k, device=DEV)
    with sc.Context(d, n, k, 0.5, 0.1) as ctx:
        h = ctx._h
        gp, mp = [x.data_ptr() for x in g], [x.data_ptr() for x in m]
        assert b.scalecom_step(h, gp, mp, None, -1, idx.data_ptr(), val.data_ptr()) == b.ERR_INVALID_ARG
        assert b.scalecom_step(h, gp, [mp[0], gp[1]], None, 0, idx.data_ptr(), val.data_ptr()) == b.ERR_ALIAS
        assert b.scalecom_step(h, gp, [mp[0], mp[0]], None, 0, idx.data_ptr(), val.data_ptr()) == b.ERR_ALIAS
        assert b.scalecom_step(h, gp, mp, mp[0], 0, idx.data_ptr(), val.data_ptr()) == b.ERR_ALIAS
        assert b.scalecom_step(h, gp, mp, None, 0, None, val.data_ptr()) == b.ERR_NULL_PTR
        assert b.scalecom_step(h, [gp[0], None], mp, None, 0, idx.data_ptr(), val.data_ptr()) == b.ERR_NULL_PTR
        assert ctx.query(b.Q_KERNEL_LAUNCHES) == 0          # nothing was launched by the rejected calls
        assert ctx.status() == 0


def test_threshold_hint_is_used_then_survives_scale_jumps():
    """The pre-filter bound carried over from the previous step only changes speed.  Stationary
    gradients take the hinted path from the second step on; a jump of the gradient scale makes the
    hint useless (too few or far too many survivors) and the step falls back to a fresh sample."""
    from paper_2104_11125_b200 import binding
    w = W.TINY.scaled(600_011)
    prof = W.profile(w, DEV)
    base = [W.gradients(w, s, DEV, prof) for s in range(6)]
    p = _parity()
    # beta = 0.001 keeps the memory negligible, so acc = m + g has the scale of the gradients
    paths = p.run_and_compare(base, W.initial_memory(w, DEV), W.initial_weights(w, DEV), w.k, 0.001, w.lr, tag="stationary")
    assert paths[0] == binding.PATH_SAMPLED and all(x == binding.PATH_HINTED for x in paths[1:]), paths
    paths = p.run_and_compare(base, W.initial_memory(w, DEV), W.initial_weights(w, DEV), w.k, 0.001, w.lr,
                              use_hint=False, tag="no-hint")
    assert paths == [binding.PATH_SAMPLED] * 6
    scales = [1.0, 1.0, 1e-3, 1e-3, 50.0, 50.0]
    jumpy = [[g * sc for g in step] for step, sc in zip(base, scales)]
    paths = p.run_and_compare(jumpy, W.initial_memory(w, DEV), W.initial_weights(w, DEV), w.k, 0.001, w.lr, tag="jumps")
    # leaders 0,1,2,3,0,1: a step starts from its leader's own last threshold, moved by what the previous leader
    # saw change, if it has one, else from the previous step's; the down-jump fails once (step 2), the up-jump
    # once (step 4): step 5's leader remembers the old scale but also learns how far step 4's leader had to move
    assert paths == [0, 2, 0, 2, 0, 2], paths


# ---- chunk-wise selector (Section 4 / Appendix E) ----------------------------------------------------
@pytest.mark.parametrize("base,d,n,steps", [
    (W.TINY, 1 << 20, 4, 3),
    (W.RESNET50, 1_500_013, 8, 3),
    (W.TRANSFORMER, 2_000_003, 16, 2),
    (W.RESNET50, 50_001, 130, 2),
])
def test_chunk_selector_scaled_workloads(base, d, n, steps):
    paths = _parity().workload_case(base.scaled(d, n=n), steps, DEV, selector="chunk")
    assert all(p == 3 for p in paths)


def test_chunk_selector_edge_cases():
    rng = np.random.default_rng(11)
    kw = dict(selector="chunk")
    _edge([[3.0]], 1, tag="chunk d=1", **kw)
    _edge([np.zeros(5000)] * 2, 77, tag="chunk all-zero", **kw)
    pm = np.where(np.arange(9001) % 2 == 0, 1.0, -1.0)
    _edge([pm, -pm], 4500, tag="chunk ties", **kw)
    x = rng.standard_normal(10_007)
    _edge([x, 0.5 * x], 1, tag="chunk k=1", **kw)
    _edge([x, 0.5 * x], 10_007, tag="chunk k=d", **kw)
    _edge([x, 0.5 * x], 5003, tag="chunk of two or three", **kw)
    _edge([x, 0.5 * x], 3337, tag="chunk of three", **kw)
    _edge([x], 71, beta=1.0, tag="chunk n=1", **kw)
    q = rng.integers(-3, 4, 50_000).astype(np.float32)
    _edge([q, np.roll(q, 1)], 499, tag="chunk quantised", **kw)
    for off in (1, 3):
        w = W.TINY.scaled(100_003)
        _parity().workload_case(w, 2, DEV, offset=off, selector="chunk")


def test_switching_selectors_on_one_handle():
    import paper_2104_11125_b200 as sc
    import oracle
    from paper_2104_11125_b200 import binding
    w = W.TINY.scaled(300_000)
    prof = W.profile(w, DEV)
    m = W.initial_memory(w, DEV)
    m_o = [x.cpu().numpy().copy() for x in m]
    idx = torch.empty(w.k, device=DEV, dtype=torch.int32)
    val = torch.empty(w.k, device=DEV)
    with sc.Context(w.d, w.n, w.k, w.beta, w.lr) as ctx:
        for t, sel in enumerate(["topk", "chunk", "chunk", "topk", "chunk", "topk"]):
            ctx.set_option(binding.OPT_SELECTOR, binding.SELECTOR_CHUNK if sel == "chunk" else binding.SELECTOR_TOPK)
            g = W.gradients(w, t, DEV, prof)
            ctx.step(g, m, None, t, idx, val)
            assert ctx.status() == 0
            idx_o, val_o, _ = oracle.step([x.cpu().numpy() for x in g], m_o, None, t, w.k, w.beta, w.lr, selector=sel)
            assert np.array_equal(idx.cpu().numpy(), idx_o) and np.array_equal(val.cpu().numpy(), val_o), (t, sel)
        assert all(np.array_equal(a.cpu().numpy(), b) for a, b in zip(m, m_o))


@pytest.mark.parametrize("fused", [False, True])
def test_kernel_timing_queries(fused):
    """Per-kernel CUDA-event times and in-kernel time spans: positive, consistent, reset on read.  With the
    one-kernel step the whole step is reported in the learner pass's place and the selection's interval is empty."""
    import paper_2104_11125_b200 as sc
    from paper_2104_11125_b200 import binding
    w = W.TINY.scaled(1_000_000)
    prof = W.profile(w, DEV)
    m = W.initial_memory(w, DEV)
    idx = torch.empty(w.k, device=DEV, dtype=torch.int32)
    val = torch.empty(w.k, device=DEV)
    with sc.Context(w.d, w.n, w.k, w.beta, w.lr) as ctx:
        with pytest.raises(sc.ScaleComError):
            ctx.kernel_span_ms()                       # option off
        ctx.set_option(binding.OPT_FUSED_SMALL, int(fused))
        assert (ctx.query(binding.Q_FUSED_SMALL) > 0) == fused
        ctx.set_option(binding.OPT_KERNEL_TIMING, 1)
        ctx.set_option(binding.OPT_KERNEL_SPANS, 1)
        launches0 = ctx.query(binding.Q_KERNEL_LAUNCHES)
        for t in range(5):
            ctx.step(W.gradients(w, t, DEV, prof), m, None, t, idx, val)
        assert ctx.query(binding.Q_KERNEL_LAUNCHES) - launches0 == (5 if fused else 10)
        ev, ne = ctx.kernel_ms()
        sp, ns = ctx.kernel_span_ms()
        assert ne == 5 and ns == 5
        if fused:
            assert sp[0] == 0.0 and ev[0] < 0.25 * ev[1]                     # nothing runs in the selection's interval
        else:
            assert 0 < sp[0] <= ev[0] * 1.05                                 # a span lies inside its event interval
        assert 0 < sp[1] <= ev[1] * 1.05
        assert ev[2] == 0.0                                                  # weight update fused: no third kernel
        assert ctx.kernel_ms()[1] == 0 and ctx.kernel_span_ms()[1] == 0      # both forget what they reported
        assert ctx.status() == 0


def test_threshold_hint_with_learners_of_different_scale():
    """Learners whose gradients differ in scale by up to 16x: a step starts from the threshold its
    own leader had the last time it led, so from the second round of leaders on no step wastes a pass."""
    from paper_2104_11125_b200 import binding
    w = W.TINY.scaled(400_003)
    prof = W.profile(w, DEV)
    scale = [1.0, 4.0, 0.25, 2.0]
    steps = [[g * sc for g, sc in zip(W.gradients(w, s, DEV, prof), scale)] for s in range(12)]
    paths = _parity().run_and_compare(steps, W.initial_memory(w, DEV), W.initial_weights(w, DEV), w.k, 0.001, w.lr,
                                      tag="heterogeneous")
    assert paths[0] == binding.PATH_SAMPLED
    assert all(p == binding.PATH_HINTED for p in paths[w.n:]), paths


# ---- diagnostics: Eq. 5 and the cosine distance -----------------------------------------------------
@pytest.mark.parametrize("base,d,n", [(W.TINY, 500_003, 4), (W.RESNET50, 1_000_001, 8), (W.TRANSFORMER, 300_000, 16)])
def test_diagnostics_match_oracle(base, d, n):
    import paper_2104_11125_b200 as sc
    import oracle
    w = base.scaled(d, n=n)
    prof = W.profile(w, DEV)
    m = W.initial_memory(w, DEV)
    m_o = [x.cpu().numpy().copy() for x in m]
    idx = torch.empty(w.k, device=DEV, dtype=torch.int32)
    val = torch.empty(w.k, device=DEV)
    with sc.Context(w.d, w.n, w.k, w.beta, w.lr) as ctx:
        for t in range(3):
            g = W.gradients(w, t, DEV, prof)
            g_np = [x.cpu().numpy() for x in g]
            before = [x.clone() for x in m]
            # Eq. 5 between the leader's set and the true top-k set, on the state before the step
            L = t % w.n
            _, sel_leader = oracle.topk(oracle.accumulate(g_np[L], m_o[L]), w.k)
            _, sel_true = oracle.topk(oracle.mean_acc(g_np, m_o), w.k)
            assert ctx.overlap(g, m, t) == oracle.hamming_d(sel_leader, sel_true)
            assert all(torch.equal(a, b) for a, b in zip(m, before))          # a diagnostic changes nothing
            if t:
                got = ctx.cosine_distance(m[0], m[1])
                want = oracle.cosine_distance(m_o[0], m_o[1])
                assert abs(got - want) <= 1e-10 * max(1.0, abs(want))
            ctx.step(g, m, None, t, idx, val)
            idx_o, val_o, _ = oracle.step(g_np, m_o, None, t, w.k, w.beta, w.lr)
            assert np.array_equal(idx.cpu().numpy(), idx_o) and np.array_equal(val.cpu().numpy(), val_o)
        assert ctx.status() == 0
    # one learner: the leader's set is the true top-k set
    w1 = base.scaled(100_000, n=1)
    g = W.gradients(w1, 0, DEV)
    with sc.Context(w1.d, 1, w1.k, 0.5, 0.1) as ctx:
        assert ctx.overlap(g, W.initial_memory(w1, DEV), 0) == 0


@pytest.mark.parametrize("selector", ["topk", "chunk", "layer_topk"])
@pytest.mark.parametrize("force_exact", [False, True])
def test_non_finite_inputs_follow_the_key_order(force_exact, selector):
    """Keys are the bit patterns of |acc|, so +-Inf rank above every finite value and NaN above Inf,
    deterministically; the rest of the step is plain IEEE arithmetic on both sides."""
    import paper_2104_11125_b200 as sc
    import oracle
    from paper_2104_11125_b200 import binding
    rng = np.random.default_rng(21)
    d, n, k = 40_000, 3, 400
    g = [rng.standard_normal(d).astype(np.float32) for _ in range(n)]
    g[0][[5, 17_000, 39_999]] = [np.inf, -np.inf, np.nan]        # learner 0 leads at t = 0
    g[1][123] = np.inf                                            # a non-leader's infinity is just a value
    m = [np.zeros(d, np.float32) for _ in range(n)]
    th = np.zeros(d, np.float32)
    gd, md, thd = [_t(x) for x in g], [_t(x) for x in m], _t(th)
    idx = torch.empty(k, device=DEV, dtype=torch.int32)
    val = torch.empty(k, device=DEV)
    layers = ([15_000, 5_000, 20_000], [150, 50, 200]) if selector == "layer_topk" else None
    with sc.Context(d, n, k, 0.5, 0.25) as ctx:
        ctx.set_option(binding.OPT_FORCE_EXACT_PATH, int(force_exact))
        ctx.set_option(binding.OPT_SELECTOR, {"topk": binding.SELECTOR_TOPK, "chunk": binding.SELECTOR_CHUNK,
                                              "layer_topk": binding.SELECTOR_LAYER_TOPK}[selector])
        if layers:
            ctx.set_layers(*layers)
        ctx.step(gd, md, thd, 0, idx, val)
        assert ctx.status() == 0
    idx_o, val_o, _ = oracle.step(g, m, th, 0, k, 0.5, 0.25, selector="topk" if selector == "layer_topk" else selector,
                                  layers=layers)
    assert {5, 17_000, 39_999} <= set(idx_o.tolist())                # each is the largest key of its chunk or layer too
    assert np.array_equal(idx.cpu().numpy(), idx_o)
    assert np.array_equal(val.cpu().numpy(), val_o, equal_nan=True)
    for a, b in zip(md, m):
        assert np.array_equal(a.cpu().numpy(), b, equal_nan=True)
    assert np.array_equal(thd.cpu().numpy(), th, equal_nan=True)


# ---- chunk-wise selector with per-layer rates (Section 4) ---------------------------------------------
def test_layer_rates_small_cases():
    rng = np.random.default_rng(31)
    p = _parity()
    for sizes, keep in [([7, 64, 1, 300, 128], [7, 2, 1, 3, 16]),
                        ([5000], [50]),
                        ([1] * 40, [1] * 40),
                        ([1000, 3000, 2000, 4099], [1000, 30, 5, 4099])]:
        d, k = sum(sizes), sum(keep)
        g = [_t(rng.standard_normal(d)) for _ in range(3)]
        m0 = [torch.zeros(d, device=DEV) for _ in range(3)]
        paths = p.run_and_compare([g] * 3, m0, torch.linspace(-1, 1, d, device=DEV), k, 0.5, 0.25,
                                  selector="chunk", layers=(sizes, keep), tag="layers %d" % len(sizes))
        assert all(x == 3 for x in paths)


def test_layer_rates_argument_checks():
    import paper_2104_11125_b200 as sc
    from paper_2104_11125_b200 import binding
    with sc.Context(100, 2, 10, 0.5, 0.1) as ctx:
        for sizes, keep in [([50, 49], [5, 5]), ([50, 50], [5, 4]), ([50, 50], [0, 10]), ([50, 50], [60, -50]), ([100] + [0], [10, 0])]:
            with pytest.raises(sc.ScaleComError) as ei:
                ctx.set_layers(sizes, keep)
            assert ei.value.code == binding.ERR_INVALID_ARG
        ctx.set_layers([50, 50], [5, 5])
        ctx.set_layers(None)


def test_layer_rates_resnet50_rule():
    """The paper's rule on the ResNet-50-shaped workload at a test size: first tensor whole, 25X / 400X elsewhere."""
    w = W.RESNET50.scaled(2_000_003)
    sizes, keep = W.resnet50_layer_keep(w)
    assert keep[0] == sizes[0] and len(sizes) == 161
    w2 = W.Workload(w.name + "+layers", w.wid, w.kind, w.n, w.d, sum(keep), w.beta, w.lr, w.steps, w.c)
    paths = _parity().workload_case(w2, 3, DEV, selector="chunk", layers=(sizes, keep))
    assert all(x == 3 for x in paths)


# ---- exact top-k inside every layer (Eq. 2 per layer with Section 4's per-layer rates) --------------------
def test_layer_topk_small_cases():
    rng = np.random.default_rng(37)
    p = _parity()
    for sizes, keep in [([7, 64, 1, 300, 128], [7, 2, 1, 3, 16]),
                        ([5000], [50]),
                        ([1] * 40, [1] * 40),
                        ([1000, 3000, 2000, 4099], [1000, 30, 5, 4099]),
                        ([2048, 2048, 4096, 100_000, 64, 64, 3], [20, 2048, 1, 1000, 64, 1, 2]),
                        ([300_000, 17, 200_001], [3000, 17, 20])]:
        d, k = sum(sizes), sum(keep)
        g = [_t(rng.standard_normal(d)) for _ in range(3)]
        m0 = [torch.zeros(d, device=DEV) for _ in range(3)]
        for offset, force in ((0, False), (1, False), (0, True)):
            paths = p.run_and_compare([g] * 3, m0, torch.linspace(-1, 1, d, device=DEV), k, 0.5, 0.25, offset=offset,
                                      force_exact=force, selector="layer_topk", layers=(sizes, keep),
                                      tag="layer top-k %d" % len(sizes))
            assert all(x in LAYER_PATHS for x in paths)
            if force:
                assert all(x == 5 for x in paths)


LAYER_PATHS = (4, 5)        # binding.PATH_LAYER_TOPK (collecting route), binding.PATH_LAYER_TOPK_STREAM


def test_layer_topk_ties_across_the_boundary():
    """Layers whose k-th magnitude is shared by more coordinates than may be kept: the lowest indices win.
    A constant layer, an all-zero layer, a layer of two values, next to an ordinary one."""
    rng = np.random.default_rng(41)
    sizes = [5000, 3000, 70_000, 4000, 1]
    keep = [50, 3000 - 1, 700, 17, 1]
    d, k = sum(sizes), sum(keep)
    base = rng.standard_normal(d).astype(np.float32)
    base[0:5000] = 0.5                                        # constant: 50 of 5000 equal keys
    base[5000:8000] = 0.0                                     # all zero, all but one kept
    base[8000:78_000] = np.where(rng.random(70_000) < 0.5, 1.0, -2.0).astype(np.float32)   # two magnitudes
    g = [_t(base), _t(base * 2), _t(-base)]
    m0 = [torch.zeros(d, device=DEV) for _ in range(3)]
    p = _parity()
    for offset, force in ((0, False), (3, False), (0, True)):
        paths = p.run_and_compare([g] * 3, m0, None, k, 0.5, 0.25, offset=offset, force_exact=force,
                                  selector="layer_topk", layers=(sizes, keep), tag="layer top-k ties")
        assert all(x == (5 if force else 4) for x in paths)     # small vector: every undecided coordinate fits its segment


def test_layer_topk_overflowing_segments_fall_back_to_streaming():
    """A large constant layer: every coordinate of it is undecided after the first digit, the warps' segments
    overflow, and the kernel has to clear the rows and run its streaming route."""
    rng = np.random.default_rng(47)
    sizes = [200_000, 2_000_000, 300_000, 500_001]
    keep = [2000, 12_345, 300_000, 77]
    d, k = sum(sizes), sum(keep)
    base = rng.standard_normal(d).astype(np.float32)
    base[200_000:2_200_000] = -0.375
    g = [_t(base), _t(base * 3)]
    m0 = [torch.zeros(d, device=DEV) for _ in range(2)]
    paths = _parity().run_and_compare([g] * 2, m0, None, k, 0.5, 0.25, selector="layer_topk", layers=(sizes, keep),
                                      tag="layer top-k overflow")
    assert paths == [5, 5]


def test_layer_topk_small_ties_in_the_collecting_route():
    """A few exact duplicates of the would-be threshold inside ordinary layers: the collecting route has to
    split them by offset (lowest index first) without falling back."""
    rng = np.random.default_rng(43)
    sizes = [40_000, 60_000, 30_000]
    keep = [400, 150, 3000]
    d, k = sum(sizes), sum(keep)
    base = rng.standard_normal(d).astype(np.float32)
    off = 0
    for sz, kp in zip(sizes, keep):
        mags = np.sort(np.abs(base[off:off + sz]))[::-1]
        thr = mags[kp - 1]                                      # the kp-th largest magnitude of the layer
        spots = off + rng.choice(sz, size=7, replace=False)
        base[spots] = thr * np.where(rng.random(7) < 0.5, 1.0, -1.0).astype(np.float32)
        off += sz
    g = [_t(base), _t(base), _t(base)]
    m0 = [torch.zeros(d, device=DEV) for _ in range(3)]
    paths = _parity().run_and_compare([g], m0, None, k, 0.5, 0.25, selector="layer_topk", layers=(sizes, keep),
                                      tag="layer top-k planted ties")
    assert paths == [4]


def test_layer_topk_needs_layers():
    import paper_2104_11125_b200 as sc
    from paper_2104_11125_b200 import binding
    d, k = 1000, 10
    g = [torch.randn(d, device=DEV)]
    m = [torch.zeros(d, device=DEV)]
    idx = torch.empty(k, device=DEV, dtype=torch.int32)
    val = torch.empty(k, device=DEV)
    with sc.Context(d, 1, k, 0.5, 0.1) as ctx:
        ctx.set_option(binding.OPT_SELECTOR, binding.SELECTOR_LAYER_TOPK)
        with pytest.raises(sc.ScaleComError) as ei:
            ctx.step(g, m, None, 0, idx, val)
        assert ei.value.code == binding.ERR_BAD_STATE
        ctx.set_layers([400, 600], [4, 6])
        ctx.step(g, m, None, 0, idx, val)
        assert ctx.status() == 0
        got = idx.cpu().numpy()
        assert (got[:4] < 400).all() and (got[4:] >= 400).all()
        ctx.set_layers([1000], [10])                          # one layer: Eq. 2 on the whole vector
        m2 = [torch.zeros(d, device=DEV)]
        ctx.step(g, m2, None, 0, idx, val)
        want = np.sort(np.argsort(-np.abs(g[0].cpu().numpy()), kind="stable")[:k])
        assert np.array_equal(idx.cpu().numpy(), want)


def test_layer_topk_resnet50_rule():
    """The paper's per-layer rates on the ResNet-50-shaped workload at a test size, exact selection per tensor."""
    w = W.RESNET50.scaled(2_000_003)
    sizes, keep = W.resnet50_layer_keep(w)
    w2 = W.Workload(w.name + "+layers", w.wid, w.kind, w.n, w.d, sum(keep), w.beta, w.lr, w.steps, w.c)
    paths = _parity().workload_case(w2, 3, DEV, selector="layer_topk", layers=(sizes, keep))
    assert all(x == 4 for x in paths)                          # ordinary gradients: the collecting route
    paths = _parity().workload_case(w2, 2, DEV, selector="layer_topk", layers=(sizes, keep), force_exact=True)
    assert all(x == 5 for x in paths)


def test_long_run_stays_exact_and_mostly_hinted():
    """120 steps from a cold start: the memories grow, the thresholds rise with them, six learners of different
    scale take turns.  Every step matches the oracle, and after the first round of leaders the pre-filter
    starts from a predicted threshold nearly every time."""
    from paper_2104_11125_b200 import binding
    w = W.TINY.scaled(150_001, n=6)
    prof = W.profile(w, DEV)
    scale = [1.0, 0.3, 3.0, 1.0, 10.0, 0.1]
    grads = [[g * s for g, s in zip(W.gradients(w, t % 12, DEV, prof), scale)] for t in range(120)]
    paths = _parity().run_and_compare(grads, W.initial_memory(w, DEV), W.initial_weights(w, DEV), w.k, 0.1, w.lr,
                                      tag="long run")
    assert paths[0] == binding.PATH_SAMPLED
    hinted = sum(p == binding.PATH_HINTED for p in paths[12:])
    assert hinted >= 0.9 * len(paths[12:]), paths


def test_drifting_scale_run_stays_exact_and_mostly_hinted():
    """600 steps whose gradient scale drifts slowly and jumps once: late in such a run the coordinates pile up
    just below the threshold (error feedback), which is where a fixed, generous margin under the predicted
    threshold overflows the candidate segments again and again.  Every 40th step is compared with the oracle in
    full; the sampled path (a failed or missing prediction) must stay rare."""
    import oracle
    import paper_2104_11125_b200 as sc
    from paper_2104_11125_b200 import binding
    w = W.RESNET50.scaled(200_003)
    prof = W.profile(w, DEV)
    nb = 16
    batches = [W.gradients(w, s, DEV, prof) for s in range(nb)]
    mem = W.initial_memory(w, DEV)
    theta = W.initial_weights(w, DEV)
    m_o = [x.cpu().numpy().copy() for x in mem]
    th_o = theta.cpu().numpy().copy()
    idx = torch.empty(w.k, device=DEV, dtype=torch.int32)
    val = torch.empty(w.k, device=DEV)
    sampled = 0
    with sc.Context(w.d, w.n, w.k, w.beta, w.lr) as ctx:
        for t in range(600):
            scale = (1.0 + 0.5 * np.sin(t / 60.0)) * (30.0 if t == 300 else 1.0)
            g = [x * float(scale) for x in batches[t % nb]]
            ctx.step(g, mem, theta, t, idx, val)
            sampled += ctx.query(binding.Q_LAST_TOPK_PATH) != binding.PATH_HINTED
            idx_o, val_o, _ = oracle.step([x.cpu().numpy() for x in g], m_o, th_o, t, w.k, w.beta, w.lr, want_gathered=False)
            if t % 40 == 0 or t in (300, 301, 599):
                assert ctx.status() == 0
                assert np.array_equal(idx.cpu().numpy(), idx_o), t
                assert np.array_equal(val.cpu().numpy(), val_o), t
                assert all(np.array_equal(a.cpu().numpy(), b) for a, b in zip(mem, m_o)), t
                assert np.array_equal(theta.cpu().numpy(), th_o), t
    assert sampled <= 60, sampled


# ---- the one-kernel step at the edges of what it accepts --------------------------------------------------
def test_one_kernel_step_at_its_largest_ranges_and_on_its_fallbacks():
    """The one-kernel step (small vectors) with as many tiles per block as it takes (14 and 16 of 16), with all of
    the top-k inside one block's range (its shared-memory survivor list overflows: radix select over the range),
    and with more equal keys around rank k than the boundary list holds.  run_and_compare runs each case with the
    kernel and with the two general kernels."""
    import paper_2104_11125_b200 as sc
    from paper_2104_11125_b200 import binding
    p = _parity()
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    for d, n in ((2_000_003, 2), (16 * 1024 * sms - 5, 3)):
        w = W.TINY.scaled(d, n=n)
        with sc.Context(w.d, w.n, w.k, w.beta, w.lr) as ctx:
            assert ctx.query(binding.Q_FUSED_SMALL) == sms, "the case is not taken by the one-kernel step"
        p.workload_case(w, 3, DEV, want_path=0)
    rng = np.random.default_rng(31)
    d, k = 1_000_003, 9000
    theta = torch.linspace(-1, 1, d, device=DEV)
    m0 = [torch.zeros(d, device=DEV) for _ in range(2)]
    # every large coordinate inside 9000 consecutive ones: one block finds them all
    x = (1e-3 * rng.standard_normal(d)).astype(np.float32)
    x[500_000:500_000 + 12_000] = rng.standard_normal(12_000).astype(np.float32)
    g = [torch.tensor(x, device=DEV), torch.tensor(0.5 * x, device=DEV)]
    paths = p.run_and_compare([g, g, g], m0, theta, k, 0.5, 0.25, tag="clustered", fused_small=True)
    assert binding.PATH_EXACT in paths, paths
    # 3000 copies of the k-th magnitude: beyond the 1024-entry boundary list
    y = rng.standard_normal(d).astype(np.float32)
    tau = np.sort(np.abs(y))[-k]
    ties = rng.choice(d, 3000, replace=False)
    y[ties] = np.where(rng.random(3000) < 0.5, tau, -tau).astype(np.float32)
    g = [torch.tensor(y, device=DEV), torch.tensor(-0.25 * y, device=DEV)]
    paths = p.run_and_compare([g, g], m0, theta, k, 0.5, 0.25, tag="3000-ties", fused_small=True)
    assert binding.PATH_EXACT in paths, paths
    p.run_and_compare([g, g], m0, theta, k, 0.5, 0.25, tag="3000-ties", fused_small=False)

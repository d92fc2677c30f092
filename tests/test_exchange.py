"""Learner-per-process deployment (one learner per rank, index broadcast + all-gather of the kept
values): every rank must reproduce, bit for bit, the single-process step of Algorithm 1 over the
same learners.  The ranks are child processes joined over gloo on 127.0.0.1."""
import os
import subprocess
import sys

import pytest

import itertools

HERE = os.path.dirname(os.path.abspath(__file__))
_launch_no = itertools.count()
WORKER = os.path.join(HERE, "exchange_worker.py")


def run_ranks(world, mode, selector, d, steps, timeout=240):
    port = 23000 + (os.getpid() * 7 + next(_launch_no) * 37) % 4000        # a fresh port for every launch
    procs = []
    for rank in range(world):
        env = dict(os.environ, RANK=str(rank), WORLD_SIZE=str(world), MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, WORKER, mode, selector, str(d), str(steps)], env=env,
                                      stdout=subprocess.PIPE, stderr=subprocess.STDOUT, text=True))
    outs = []
    try:
        for p in procs:
            out, _ = p.communicate(timeout=timeout)
            outs.append(out)
    finally:
        for p in procs:
            if p.poll() is None:
                p.kill()
    for rank, (p, out) in enumerate(zip(procs, outs)):
        assert p.returncode == 0, "rank %d:\n%s" % (rank, out[-3000:])
        assert "rank %d ok" % rank in out


@pytest.mark.parametrize("world,selector", [(2, "topk"), (3, "topk"), (2, "chunk"), (2, "layer_topk")])
def test_protocol_over_gloo_matches_single_process_step(world, selector):
    # 2 * world + 1 steps: every rank leads at least twice
    run_ranks(world, "cpu", selector, 40_003, 2 * world + 1)


def test_fused_exchange_falls_back_when_a_peer_is_out_of_reach():
    """exchange="peer" stores into other ranks' device memory; when the device query says a peer cannot be reached,
    all ranks must agree on the collective exchange before anything is mapped (nothing may be stored through an
    address that was never made accessible)."""
    run_ranks(2, "cpu-nopeer", "topk", 40_003, 5)
    run_ranks(3, "cpu-nopeer", "chunk", 20_011, 4)


def test_enable_peer_access_checks_its_arguments():
    """Host-side checks only (no second GPU here): a missing handle is refused."""
    from paper_2104_11125_b200 import binding
    assert binding.lib().scalecom_enable_peer_access(None, 0) == binding.ERR_NULL_PTR


@pytest.mark.gpu
def test_enable_peer_access_on_one_device():
    """With one GPU: the handle's own device needs nothing, an ordinal that does not exist is refused."""
    import torch
    import paper_2104_11125_b200 as sc
    from paper_2104_11125_b200 import binding
    with sc.Context(1000, 1, 10, 0.5, 0.1) as ctx:
        ctx.enable_peer_access(torch.cuda.current_device())
        for bad in (-1, torch.cuda.device_count()):
            with pytest.raises(sc.ScaleComError) as e:
                ctx.enable_peer_access(bad)
            assert e.value.code == binding.ERR_INVALID_ARG


@pytest.mark.gpu
@pytest.mark.parametrize("world,selector,d", [(2, "topk", 262_147), (3, "topk", 1_048_583), (3, "chunk", 262_147),
                                                (2, "layer_topk", 262_147)])
def test_ranks_sharing_a_device_match_single_process_step(world, selector, d):
    run_ranks(world, "gpu", selector, d, 2 * world + 1, timeout=400)


@pytest.mark.gpu
@pytest.mark.parametrize("world,selector,d", [(2, "topk", 262_147), (3, "chunk", 1_048_583)])
def test_peer_stores_into_mapped_rows_match_single_process_step(world, selector, d):
    """The all-gather fused into the compressing kernel: the processes map one another's gathered-rows buffers
    (CUDA IPC on the shared device) and store their kept values there; 2 * world + 2 steps use both buffers
    of every rank several times."""
    run_ranks(world, "gpu-peer", selector, d, 2 * world + 2, timeout=400)


@pytest.mark.gpu
@pytest.mark.parametrize("selector,d,n", [("topk", 300_007, 4), ("chunk", 300_007, 4), ("topk", 5_000_011, 5)])
def test_pieces_in_one_process_match_oracle_step(selector, d, n):
    """The calls of the taken-apart step, one handle per learner, without any collective."""
    import numpy as np
    import torch
    import oracle
    from paper_2104_11125_b200 import binding, workloads
    import paper_2104_11125_b200 as sc

    dev = torch.device("cuda", 0)
    w = workloads.TINY.scaled(d, n)
    k, beta, lr = w.k, w.beta, w.lr
    prof = workloads.profile(w, dev)
    mem = workloads.initial_memory(w, dev)
    m_o = [x.cpu().numpy().copy() for x in mem]
    theta = [workloads.initial_weights(w, dev) for _ in range(n)]
    th_o = theta[0].cpu().numpy().copy()
    ctxs = [sc.Context(d, 1, k, beta, lr) for _ in range(n)]
    for c in ctxs:
        c.set_option(binding.OPT_SELECTOR, binding.SELECTOR_CHUNK if selector == "chunk" else binding.SELECTOR_TOPK)
    idx = torch.empty(k, device=dev, dtype=torch.int32)
    rows = torch.empty(n * k, device=dev, dtype=torch.float32)
    val = torch.empty(k, device=dev, dtype=torch.float32)
    try:
        for t in range(2 * n + 1):
            g = workloads.gradients(w, t, dev, prof)
            idx.fill_(-1); rows.fill_(float("nan")); val.fill_(float("nan"))
            ctxs[t % n].select(g[t % n], mem[t % n], idx)
            for i in range(n):
                ctxs[i].compress(g[i], mem[i], idx, rows[i * k:(i + 1) * k])
            for i in range(n):
                if i % 2:                                  # fused and separate weight update must agree
                    ctxs[i].reduce_rows(rows, val, idx, theta[i])
                else:
                    ctxs[i].reduce_rows(rows, val)
                    ctxs[i].apply_update(theta[i], idx, val, lr)
            torch.cuda.synchronize()
            assert all(c.status() == binding.OK for c in ctxs)
            idx_o, val_o, G_o = oracle.step([x.cpu().numpy() for x in g], m_o, th_o, t, k, beta, lr, selector=selector)
            assert np.array_equal(idx.cpu().numpy(), idx_o)
            assert np.array_equal(rows.cpu().numpy().reshape(n, k), G_o)
            assert np.array_equal(val.cpu().numpy(), val_o)
            for i in range(n):
                assert np.array_equal(mem[i].cpu().numpy(), m_o[i])
                assert np.array_equal(theta[i].cpu().numpy(), th_o)
    finally:
        for c in ctxs:
            c.close()


@pytest.mark.gpu
def test_compress_rejects_a_malformed_index_list():
    """An index list that is not strictly ascending, or reaches past d, sets the handle's status
    instead of being applied out of bounds."""
    import torch
    from paper_2104_11125_b200 import binding
    import paper_2104_11125_b200 as sc

    dev = torch.device("cuda", 0)
    d, k = 10_000, 100
    g = torch.randn(d, device=dev)
    for bad in ("order", "range"):
        m = torch.zeros(d, device=dev)
        idx = torch.arange(0, 10 * k, 10, device=dev, dtype=torch.int32)
        if bad == "order":
            idx[7] = idx[6]
        else:
            idx[k - 1] = d
        out = torch.empty(k, device=dev)
        with sc.Context(d, 1, k, 0.1, 0.01) as ctx:
            ctx.compress(g, m, idx, out)
            torch.cuda.synchronize()
            assert ctx.status() == binding.ERR_INTERNAL
            with pytest.raises(sc.ScaleComError):
                ctx.compress(g, m, idx, out)            # poisoned until reset
            ctx.reset()
            good = torch.arange(0, 10 * k, 10, device=dev, dtype=torch.int32)
            ctx.compress(g, m, good, out)
            torch.cuda.synchronize()
            assert ctx.status() == binding.OK


@pytest.mark.gpu
def test_compress_takes_whatever_list_comes_next():
    """The handle's bitmap is reused between calls: a list that differs from the one before it, or from what
    a selection on the same handle left behind, must be applied alone."""
    import numpy as np
    import torch
    import oracle
    from paper_2104_11125_b200 import binding
    import paper_2104_11125_b200 as sc

    dev = torch.device("cuda", 0)
    d, k, beta = 70_001, 700, 0.1
    gen = torch.Generator(device=dev).manual_seed(5)
    rng = np.random.default_rng(11)
    m = torch.randn(d, device=dev, generator=gen)
    m_o = m.cpu().numpy().copy()
    out = torch.empty(k, device=dev)
    own_idx = torch.empty(k, device=dev, dtype=torch.int32)
    with sc.Context(d, 1, k, beta, 0.01) as ctx:
        for it in range(6):
            g = torch.randn(d, device=dev, generator=gen)
            if it in (2, 4):                       # a selection writes its own set into the bitmap first
                ctx.set_option(binding.OPT_SELECTOR, binding.SELECTOR_CHUNK if it == 4 else binding.SELECTOR_TOPK)
                ctx.select(g, m, own_idx)
            idx_o = np.sort(rng.choice(d, size=k, replace=False)).astype(np.int32)
            if it == 5:
                idx_o = np.arange(d - k, d, dtype=np.int32)     # a dense run up to the last coordinate
            sel = np.zeros(d, np.uint8)
            sel[idx_o] = 1
            ctx.compress(g, m, torch.from_numpy(idx_o).to(dev), out)
            torch.cuda.synchronize()
            assert ctx.status() == binding.OK
            gathered_o = oracle.learner(g.cpu().numpy(), m_o, idx_o, sel, beta)
            assert np.array_equal(out.cpu().numpy(), gathered_o), it
            assert np.array_equal(m.cpu().numpy(), m_o), it


@pytest.mark.gpu
@pytest.mark.parametrize("d,picks", [(3_000_000, [5, 1_500_000, 2_999_999]), (3_000_000, [2_999_999]), (3_000_000, [0]),
                                     (1025, [1024]), (70_000, list(range(1000, 1040)) + [69_999])])
def test_compress_with_long_runs_of_empty_tiles(d, picks):
    import numpy as np
    import torch
    import oracle
    from paper_2104_11125_b200 import binding
    import paper_2104_11125_b200 as sc

    dev = torch.device("cuda", 0)
    k, beta = len(picks), 0.25
    gen = torch.Generator(device=dev).manual_seed(9)
    g = torch.randn(d, device=dev, generator=gen)
    m = torch.randn(d, device=dev, generator=gen)
    m_o = m.cpu().numpy().copy()
    idx_o = np.asarray(picks, np.int32)
    sel = np.zeros(d, np.uint8)
    sel[idx_o] = 1
    out = torch.full((k,), float("nan"), device=dev)
    with sc.Context(d, 1, k, beta, 0.01) as ctx:
        ctx.compress(g, m, torch.from_numpy(idx_o).to(dev), out)
        torch.cuda.synchronize()
        assert ctx.status() == binding.OK
    want = oracle.learner(g.cpu().numpy(), m_o, idx_o, sel, beta)
    assert np.array_equal(out.cpu().numpy(), want)
    assert np.array_equal(m.cpu().numpy(), m_o)


@pytest.mark.gpu
def test_compress_scatter_writes_every_destination_and_checks_its_arguments():
    import ctypes
    import numpy as np
    import torch
    import oracle
    from paper_2104_11125_b200 import binding
    import paper_2104_11125_b200 as sc

    dev = torch.device("cuda", 0)
    d, k, beta = 150_001, 1500, 0.3
    rng = np.random.default_rng(13)
    gen = torch.Generator(device=dev).manual_seed(21)
    g = torch.randn(d, device=dev, generator=gen)
    m = torch.randn(d, device=dev, generator=gen)
    m_o = m.cpu().numpy().copy()
    idx_o = np.sort(rng.choice(d, size=k, replace=False)).astype(np.int32)
    sel = np.zeros(d, np.uint8)
    sel[idx_o] = 1
    idx = torch.from_numpy(idx_o).to(dev)
    own = torch.empty(k, device=dev)
    rows = torch.full((5, k), float("nan"), device=dev)
    with sc.Context(d, 1, k, beta, 0.01) as ctx:
        ctx.compress_scatter(g, m, idx, own, [rows[0], rows[2], rows[4]])
        torch.cuda.synchronize()
        assert ctx.status() == binding.OK
        want = oracle.learner(g.cpu().numpy(), m_o, idx_o, sel, beta)
        for r in (0, 2, 4):
            assert np.array_equal(rows[r].cpu().numpy(), want)
        assert bool(torch.isnan(rows[1]).all()) and bool(torch.isnan(rows[3]).all())
        assert np.array_equal(own.cpu().numpy(), want) and np.array_equal(m.cpu().numpy(), m_o)
        # arguments
        L, h = binding.lib(), ctx._h
        ptrs = (ctypes.c_void_p * 65)(*([rows[0].data_ptr()] * 65))
        args = (h, g.data_ptr(), m.data_ptr(), idx.data_ptr(), own.data_ptr())
        assert L.scalecom_compress_scatter(*args, ctypes.cast(ptrs, ctypes.c_void_p), 65, None, 0) == binding.ERR_INVALID_ARG
        assert L.scalecom_compress_scatter(*args, ctypes.cast(ptrs, ctypes.c_void_p), -1, None, 0) == binding.ERR_INVALID_ARG
        assert L.scalecom_compress_scatter(*args, None, 2, None, 0) == binding.ERR_NULL_PTR
        ptrs[1] = None
        assert L.scalecom_compress_scatter(*args, ctypes.cast(ptrs, ctypes.c_void_p), 2, None, 0) == binding.ERR_NULL_PTR
        ptrs[1] = m.data_ptr()
        assert L.scalecom_compress_scatter(*args, ctypes.cast(ptrs, ctypes.c_void_p), 2, None, 0) == binding.ERR_ALIAS
        ptrs[1] = rows[1].data_ptr()
        assert L.scalecom_compress_scatter(*args, ctypes.cast(ptrs, ctypes.c_void_p), 2, ctypes.cast(ptrs, ctypes.c_void_p),
                                           0) == binding.ERR_INVALID_ARG          # flag words without a tag
        assert np.array_equal(m.cpu().numpy(), m_o)            # the rejected calls touched nothing


@pytest.mark.gpu
def test_compress_without_a_list_needs_a_fresh_select():
    import numpy as np
    import torch
    import oracle
    from paper_2104_11125_b200 import binding
    import paper_2104_11125_b200 as sc

    dev = torch.device("cuda", 0)
    d, k, beta = 200_003, 2000, 0.2
    gen = torch.Generator(device=dev).manual_seed(3)
    g = torch.randn(d, device=dev, generator=gen)
    m = torch.randn(d, device=dev, generator=gen)
    m_o = m.cpu().numpy().copy()
    idx = torch.empty(k, device=dev, dtype=torch.int32)
    out = torch.empty(k, device=dev)
    with sc.Context(d, 1, k, beta, 0.01) as ctx:
        with pytest.raises(sc.ScaleComError) as ei:          # nothing selected yet
            ctx.compress(g, m, None, out)
        assert ei.value.code == binding.ERR_BAD_STATE
        for selector in (binding.SELECTOR_TOPK, binding.SELECTOR_CHUNK):
            ctx.set_option(binding.OPT_SELECTOR, selector)
            ctx.select(g, m, idx)
            ctx.compress(g, m, None, out)
            torch.cuda.synchronize()
            assert ctx.status() == binding.OK
            acc = oracle.accumulate(g.cpu().numpy(), m_o)
            idx_o, sel = (oracle.topk if selector == binding.SELECTOR_TOPK else oracle.chunk_select)(acc, k)
            want = oracle.learner(g.cpu().numpy(), m_o, idx_o, sel, beta)
            assert np.array_equal(idx.cpu().numpy(), idx_o)
            assert np.array_equal(out.cpu().numpy(), want) and np.array_equal(m.cpu().numpy(), m_o)
            with pytest.raises(sc.ScaleComError) as ei:      # the selection has been used up
                ctx.compress(g, m, None, out)
            assert ei.value.code == binding.ERR_BAD_STATE
        # a list given explicitly after all that still works (the bitmap was left clean)
        ctx.select(g, m, idx)
        other = torch.arange(0, 100 * k, 100, device=dev, dtype=torch.int32)
        sel = np.zeros(d, np.uint8)
        sel[other.cpu().numpy()] = 1
        ctx.compress(g, m, other, out)
        torch.cuda.synchronize()
        want = oracle.learner(g.cpu().numpy(), m_o, other.cpu().numpy(), sel, beta)
        assert np.array_equal(out.cpu().numpy(), want) and np.array_equal(m.cpu().numpy(), m_o)


@pytest.mark.gpu
def test_flag_signalled_exchange_single_rank_through_the_orchestration():
    """exchange="peer-flags" with one rank: the compressing kernel sets the flag word, the reducing kernel that
    follows it on the stream finds it set.  (Several ranks would need a GPU each.)"""
    run_ranks(1, "gpu-flags", "topk", 262_147, 5, timeout=300)


@pytest.mark.gpu
def test_flag_signalled_exchange_rank_by_rank_in_one_process():
    """Four learners' handles in one process, one stream: every compress_scatter stores its row and its flag word
    into all four gathered-rows buffers; every reduce_rows then waits (finding the flags already set) and sums.
    Nothing ever waits for a kernel that has not been launched before it."""
    import numpy as np
    import torch
    import oracle
    from paper_2104_11125_b200 import binding, workloads
    import paper_2104_11125_b200 as sc

    dev = torch.device("cuda", 0)
    n = 4
    w = workloads.TINY.scaled(400_009, n)
    d, k, beta, lr = w.d, w.k, w.beta, w.lr
    prof = workloads.profile(w, dev)
    mem = workloads.initial_memory(w, dev)
    m_o = [x.cpu().numpy().copy() for x in mem]
    theta = [workloads.initial_weights(w, dev) for _ in range(n)]
    th_o = theta[0].cpu().numpy().copy()
    ctxs = [sc.Context(d, 1, k, beta, lr) for _ in range(n)]
    rows = [torch.full((2, n, k), float("nan"), device=dev) for _ in range(n)]        # rank r's two buffers
    flags = [torch.zeros(2, n, dtype=torch.int32, device=dev) for _ in range(n)]
    idx = torch.empty(k, device=dev, dtype=torch.int32)
    own = torch.empty(k, device=dev)
    val = [torch.empty(k, device=dev) for _ in range(n)]
    try:
        for t in range(7):
            b, tag, leader = t & 1, t + 1, t % n
            g = workloads.gradients(w, t, dev, prof)
            ctxs[leader].select(g[leader], mem[leader], idx)
            for i in range(n):
                ctxs[i].compress_scatter(g[i], mem[i], None if i == leader else idx, own,
                                         [rows[r][b, i] for r in range(n)], [flags[r][b, i:i + 1] for r in range(n)], tag)
            for r in range(n):
                ctxs[r].reduce_rows(rows[r][b].view(-1), val[r], idx, theta[r], flags[r][b], tag)
            torch.cuda.synchronize()
            assert all(c.status() == binding.OK for c in ctxs)
            idx_o, val_o, G_o = oracle.step([x.cpu().numpy() for x in g], m_o, th_o, t, k, beta, lr)
            assert np.array_equal(idx.cpu().numpy(), idx_o)
            for r in range(n):
                assert np.array_equal(rows[r][b].cpu().numpy(), G_o)
                assert np.array_equal(val[r].cpu().numpy(), val_o)
                assert np.array_equal(theta[r].cpu().numpy(), th_o)
                assert np.array_equal(mem[r].cpu().numpy(), m_o[r])
                assert flags[r][b].cpu().tolist() == [tag] * n
    finally:
        for c in ctxs:
            c.close()


@pytest.mark.gpu
def test_waiting_for_a_row_that_never_comes_times_out_cleanly():
    """Failure detection without a GPU fault: a flag word that nothing sets makes the bounded wait of the reducing
    kernel run out; nothing is written, the status says TIMEOUT, the handle works again after a reset."""
    import torch
    from paper_2104_11125_b200 import binding
    import paper_2104_11125_b200 as sc

    dev = torch.device("cuda", 0)
    d, k = 50_000, 500
    rows = torch.ones(3, k, device=dev)
    flags = torch.tensor([9, 9, 0], dtype=torch.int32, device=dev)          # the third sender never arrives
    val = torch.full((k,), -1.0, device=dev)
    with sc.Context(d, 1, k, 0.5, 0.1) as ctx:
        ctx.set_option(binding.OPT_SPIN_LIMIT, 300)
        ctx.reduce_rows(rows.view(-1), val, None, None, flags, 9)
        assert ctx.status() == binding.ERR_TIMEOUT
        assert bool((val == -1.0).all())
        with pytest.raises(sc.ScaleComError) as ei:
            ctx.reduce_rows(rows.view(-1), val, None, None, flags, 9)
        assert ei.value.code == binding.ERR_BAD_STATE
        ctx.reset()
        flags[2] = 9
        ctx.reduce_rows(rows.view(-1), val, None, None, flags, 9)
        torch.cuda.synchronize()
        assert ctx.status() == binding.OK and bool((val == 1.0).all())
        # argument checks
        with pytest.raises(sc.ScaleComError) as ei:
            ctx.reduce_rows(rows.view(-1), val, None, None, flags, 0)
        assert ei.value.code == binding.ERR_INVALID_ARG

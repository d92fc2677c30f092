"""Parity at the full sizes of the five configurations, in the launch configuration the benchmark times.

The selection is compared in full (the oracle sorts the whole leader vector).  Gather, reduction,
memory and weight updates are compared on every learner inside coordinate windows (first, ragged
last and interior ones), where the oracle runs its per-learner routine on the window's slice --
Eq. 3/4 and Algorithm 1 lines 10/12 are element-wise, so a slice of the result is the result of
the slice; the learners that lead a step are also carried in full, because the next selection
needs their whole memory.  No oracle input comes from the CUDA path.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2104_11125_b200 import workloads as W

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
WIN = 1 << 17


def _windows(d):
    mid = (d // 3) // 4 * 4 + 1                       # deliberately not tile aligned
    return [(0, WIN), (mid, mid + WIN), (d - WIN - 3, d)]


def fullsize_case(w, steps=2):
    import paper_2104_11125_b200 as sc
    from paper_2104_11125_b200 import binding
    from tests.parity import rel_err, REL_TOL
    n, d, k = w.n, w.d, w.k
    prof = W.profile(w, DEV)
    m_g = W.initial_memory(w, DEV)
    th_g = W.initial_weights(w, DEV)
    th0 = th_g.cpu().numpy()
    idx = torch.empty(k, device=DEV, dtype=torch.int32)
    val = torch.empty(k, device=DEV)
    G = torch.empty(n * k, device=DEV)
    wins = _windows(d)
    leaders = sorted({t % n for t in range(steps)})
    m_full = {i: np.zeros(d, np.float32) for i in leaders}
    m_win = [[np.zeros(b - a, np.float32) for (a, b) in wins] for _ in range(n)]
    th_win = [th0[a:b].copy() for (a, b) in wins]
    with sc.Context(d, n, k, w.beta, w.lr) as ctx:
        ctx.set_gathered(G)
        for t in range(steps):
            g = W.gradients(w, t, DEV, prof)
            ctx.step(g, m_g, th_g, t, idx, val)
            assert ctx.status() == 0
            path = ctx.query(binding.Q_LAST_TOPK_PATH)
            assert path == (binding.PATH_SAMPLED if t == 0 else binding.PATH_HINTED), "step %d took path %d" % (t, path)
            L = t % n
            # ---- selection: full, bit-exact ----
            acc = oracle.accumulate(g[L].cpu().numpy(), m_full[L])
            idx_o, sel = oracle.topk(acc, k)
            del acc
            idx_h = idx.cpu().numpy()
            assert np.array_equal(idx_h, idx_o), "step %d: %d indices differ" % (t, int((idx_h != idx_o).sum()))
            val_h = val.cpu().numpy()
            G_h = G.view(n, k)
            # ---- learners carried in full ----
            for i in leaders:
                Gi = oracle.learner(g[i].cpu().numpy(), m_full[i], idx_o, sel, w.beta)
                assert np.array_equal(G_h[i].cpu().numpy(), Gi), "step %d learner %d gathered" % (t, i)
                mi = m_g[i].cpu().numpy()
                assert rel_err(mi, m_full[i]) <= REL_TOL and np.array_equal(mi, m_full[i])
            # ---- every learner, inside the windows ----
            for wi, (a, b) in enumerate(wins):
                j0, j1 = np.searchsorted(idx_o, a), np.searchsorted(idx_o, b)
                idx_w = (idx_o[j0:j1] - a).astype(np.int32)
                sel_w = np.ascontiguousarray(sel[a:b])
                rows = []
                for i in range(n):
                    gi = g[i][a:b].cpu().numpy()
                    rows.append(oracle.learner(gi, m_win[i][wi], idx_w, sel_w, w.beta))
                    mi = m_g[i][a:b].cpu().numpy()
                    assert rel_err(mi, m_win[i][wi]) <= REL_TOL and np.array_equal(mi, m_win[i][wi]), \
                        "step %d learner %d window %d memory" % (t, i, wi)
                Gw = np.ascontiguousarray(np.stack(rows))
                assert np.array_equal(G_h[:, j0:j1].cpu().numpy(), Gw), "step %d window %d gathered" % (t, wi)
                if j1 > j0:
                    val_w = oracle.reduce(Gw)
                    assert rel_err(val_h[j0:j1], val_w) <= REL_TOL and np.array_equal(val_h[j0:j1], val_w)
                    oracle.apply(th_win[wi], idx_w, val_w, w.lr)
                thw = th_g[a:b].cpu().numpy()
                assert rel_err(thw, th_win[wi]) <= REL_TOL and np.array_equal(thw, th_win[wi])
            del g


def test_config2_resnet50_full_oracle_step():
    """Config 2 at full size, every output element by element, one full oracle step."""
    from tests.parity import workload_case
    workload_case(W.RESNET50, 1, DEV, want_path=0)


def test_config2_resnet50_windows():
    fullsize_case(W.RESNET50, steps=3)


def test_config3_transformer_windows():
    fullsize_case(W.TRANSFORMER, steps=2)


@pytest.mark.parametrize("n", [32, 128])
def test_config4_learner_sweep_windows(n):
    fullsize_case(W.sweep(n), steps=2)


def test_config5_large_windows():
    free, total = torch.cuda.mem_get_info()
    if free < 110 * 2 ** 30:
        pytest.skip("needs ~105 GB of free device memory")
    fullsize_case(W.LARGE, steps=2)


@pytest.mark.parametrize("w", [W.RESNET50, W.TRANSFORMER], ids=lambda w: w.name)
def test_chunk_selector_full_size_every_element(w):
    """The chunk-wise oracle needs no sort, so whole steps at full size are compared element by element."""
    from tests.parity import workload_case
    paths = workload_case(w, 2, DEV, selector="chunk")
    assert paths == [3, 3]

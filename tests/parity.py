"""Shared helpers of the GPU parity tests: run the CUDA library and the CPU
oracle on the same seeded inputs and compare element by element."""
from __future__ import annotations

import numpy as np
import torch

import oracle
import paper_2104_11125_b200 as sc
from paper_2104_11125_b200 import binding, workloads

FLT_MIN = np.float32(1.17549435e-38)
REL_TOL = 1e-6        # spec tolerance for reduced values, memory and weights


def rel_err(a: np.ndarray, b: np.ndarray) -> float:
    """max |a-b| / max(|b|, FLT_MIN), b the oracle."""
    if a.size == 0:
        return 0.0
    a64, b64 = a.astype(np.float64), b.astype(np.float64)
    return float(np.max(np.abs(a64 - b64) / np.maximum(np.abs(b64), float(FLT_MIN))))


def assert_step_matches(tag, idx_g, val_g, G_g, m_g, th_g, idx_o, val_o, G_o, m_o, th_o):
    # bit-exact: index set, ascending order, gathered per-learner values
    assert np.array_equal(idx_g, idx_o), "%s: index sets differ (%d mismatches)" % (tag, int(np.sum(idx_g != idx_o)))
    if G_g is not None:
        assert np.array_equal(G_g, G_o), "%s: gathered values differ" % tag
    # <= 1e-6 relative: reduced values, memory, weights
    assert rel_err(val_g, val_o) <= REL_TOL, "%s: reduced values rel err %g" % (tag, rel_err(val_g, val_o))
    for i, (a, b) in enumerate(zip(m_g, m_o)):
        e = rel_err(a, b)
        assert e <= REL_TOL, "%s: memory of learner %d rel err %g" % (tag, i, e)
    if th_g is not None:
        assert rel_err(th_g, th_o) <= REL_TOL, "%s: weights rel err %g" % (tag, rel_err(th_g, th_o))
    # the arithmetic is the same sequence of correctly rounded operations on both sides, so in fact nothing differs
    assert np.array_equal(val_g, val_o), "%s: reduced values not identical" % tag
    for i, (a, b) in enumerate(zip(m_g, m_o)):
        assert np.array_equal(a, b), "%s: memory of learner %d not identical" % (tag, i)
    if th_g is not None:
        assert np.array_equal(th_g, th_o), "%s: weights not identical" % tag


def run_and_compare(grads_per_step, m0, theta0, k, beta, lr, t0=0, *, force_exact=False, fuse_update=True,
                    want_path=None, offset=0, use_hint=True, selector="topk", layers=None, tag="case", fused_small=None,
                    l2_keep=True):
    """grads_per_step: list over steps of lists of n CUDA fp32 tensors.
    m0: list of n CUDA tensors (initial memory), theta0: CUDA tensor or None.
    offset > 0 places every device vector `offset` floats past a 16-byte boundary
    (exercises the unaligned code path).
    fused_small: True / False pins whether small vectors take the one-kernel step; None (default) runs the case
    both ways when the library would use that kernel for it, and returns the paths of the two-kernel run.
    l2_keep: SCALECOM_OPT_L2_KEEP (speed only: results must not depend on it)."""
    dev = grads_per_step[0][0].device
    n, d = len(m0), m0[0].numel()
    if fused_small is None:
        with sc.Context(d, n, k, beta, lr) as probe:
            eligible = probe.query(binding.Q_FUSED_SMALL) > 0 and selector == "topk" and offset % 4 == 0
        kw = dict(force_exact=force_exact, fuse_update=fuse_update, want_path=want_path, offset=offset, use_hint=use_hint,
                  selector=selector, layers=layers, l2_keep=l2_keep)
        if eligible:
            run_and_compare(grads_per_step, m0, theta0, k, beta, lr, t0, tag=tag + " (one kernel)", fused_small=True, **kw)
        return run_and_compare(grads_per_step, m0, theta0, k, beta, lr, t0, tag=tag, fused_small=False, **kw)

    def place(x):
        if offset == 0:
            return x.clone()
        buf = torch.empty(d + 8, device=dev, dtype=torch.float32)
        v = buf[offset:offset + d]
        v.copy_(x)
        return v

    m_g = [place(x) for x in m0]
    th_g = place(theta0) if theta0 is not None else None
    m_o = [x.cpu().numpy().copy() for x in m0]
    th_o = theta0.cpu().numpy().copy() if theta0 is not None else None
    idx = torch.empty(k, device=dev, dtype=torch.int32)
    val = torch.empty(k, device=dev, dtype=torch.float32)
    G = torch.empty(n * k, device=dev, dtype=torch.float32)
    paths = []
    with sc.Context(d, n, k, beta, lr) as ctx:
        ctx.set_gathered(G)
        ctx.set_option(binding.OPT_FORCE_EXACT_PATH, int(force_exact))
        ctx.set_option(binding.OPT_FUSE_UPDATE, int(fuse_update))
        ctx.set_option(binding.OPT_USE_HINT, int(use_hint))
        ctx.set_option(binding.OPT_FUSED_SMALL, int(fused_small))
        ctx.set_option(binding.OPT_L2_KEEP, int(l2_keep))
        ctx.set_option(binding.OPT_SELECTOR, {"topk": binding.SELECTOR_TOPK, "chunk": binding.SELECTOR_CHUNK,
                                              "layer_topk": binding.SELECTOR_LAYER_TOPK}[selector])
        if layers is not None:
            ctx.set_layers(*layers)
        for s, grads in enumerate(grads_per_step):
            t = t0 + s
            g_dev = [place(g) for g in grads]
            idx.fill_(-1); val.fill_(float("nan")); G.fill_(float("nan"))
            ctx.step(g_dev, m_g, th_g, t, idx, val)
            assert ctx.status() == 0, "%s step %d: device status %d" % (tag, s, ctx.status())
            paths.append(ctx.query(binding.Q_LAST_TOPK_PATH))
            g_np = [g.cpu().numpy() for g in grads]
            # "layer_topk" is the oracle's exact selector applied inside the layers
            idx_o, val_o, G_o = oracle.step(g_np, m_o, th_o, t, k, beta, lr,
                                            selector="topk" if selector == "layer_topk" else selector,
                                            layers=layers if selector != "topk" else None)
            assert_step_matches("%s step %d" % (tag, s), idx.cpu().numpy(), val.cpu().numpy(),
                                G.cpu().numpy().reshape(n, k), [x.cpu().numpy() for x in m_g],
                                th_g.cpu().numpy() if th_g is not None else None,
                                idx_o, val_o, G_o, m_o, th_o)
    if want_path is not None:
        # 0 asks for the pre-filter path, whether it started from a fresh sample (0) or from the
        # previous step's threshold (2); 1 asks for the exact path
        good = (binding.PATH_SAMPLED, binding.PATH_HINTED) if want_path == 0 else (want_path,)
        assert all(p in good for p in paths), "%s: selection paths %s, wanted %s" % (tag, paths, good)
    return paths


def workload_case(w: workloads.Workload, steps: int, device, **kw):
    prof = workloads.profile(w, device)
    grads = [workloads.gradients(w, s, device, prof) for s in range(steps)]
    return run_and_compare(grads, workloads.initial_memory(w, device), workloads.initial_weights(w, device),
                           w.k, w.beta, w.lr, tag=w.name, **kw)

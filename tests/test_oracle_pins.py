"""Pins for the CPU oracle: every check here compares it with something the
paper or the mathematics fixes, never with itself and never with the CUDA path."""
import itertools
import os
from fractions import Fraction

import numpy as np
import pytest

import oracle

RNG = np.random.default_rng(20210411)


def key32(x):
    return np.ascontiguousarray(x, np.float32).view(np.uint32) & np.uint32(0x7FFFFFFF)


def tie_vectors():
    """Tiny vectors with crafted ties, signed zeros, denormals and +-x pairs."""
    yield np.array([1, -1, 1, -1, 1, -1, 1, -1], np.float32)
    yield np.zeros(7, np.float32)
    yield np.array([0.0, -0.0, 0.0, -0.0, 1e-45, -1e-45], np.float32)
    yield np.array([3, -3, 2, 2, -2, 1, 5, -5, 5, 0, -0.0, 4], np.float32)
    yield np.array([2.0], np.float32)
    for d in (2, 3, 5, 8, 12, 16):
        yield RNG.integers(-3, 4, size=d).astype(np.float32)          # many ties
        yield RNG.standard_normal(d).astype(np.float32)               # none
        yield np.float32(1e-40) * RNG.integers(-2, 3, size=d).astype(np.float32)  # denormals


# ---- P1: Eq. 2 by brute force ------------------------------------------------------------
def test_topk_matches_rank_count_for_all_k():
    for x in tie_vectors():
        d = x.size
        key = key32(x).astype(np.int64)
        # rank(p) = #{q: key_q > key_p} + #{q < p: key_q == key_p}, counted in Python
        ranks = [int(sum(1 for q in range(d) if key[q] > key[p] or (key[q] == key[p] and q < p)))
                 for p in range(d)]
        assert sorted(ranks) == list(range(d))
        for p in range(d):
            assert oracle.rank(x, p) == ranks[p]
            assert oracle.rank(x.astype(np.float64), p) == ranks[p]
        for k in range(1, d + 1):
            idx, sel = oracle.topk(x, k)
            expect = [p for p in range(d) if ranks[p] < k]
            assert idx.tolist() == expect
            assert sel.tolist() == [1 if ranks[p] < k else 0 for p in range(d)]
            idx64, _ = oracle.topk(x.astype(np.float64), k)
            assert idx64.tolist() == expect


def test_topk_is_the_lexicographically_least_maximiser():
    """Among all C(d,k) subsets the selected one has the largest total
    magnitude, and is the first such subset in lexicographic order."""
    for x in tie_vectors():
        d = x.size
        if d > 12:
            continue
        mag = [Fraction(float(abs(v))) for v in x.astype(np.float64)]
        for k in range(1, d + 1):
            best, best_sum = None, None
            for S in itertools.combinations(range(d), k):      # lexicographic order
                s = sum(mag[p] for p in S)
                if best_sum is None or s > best_sum:
                    best, best_sum = S, s
            idx, _ = oracle.topk(x, k)
            assert tuple(idx.tolist()) == best


# ---- exact rational restatement of Algorithm 1 on dyadic inputs ----------------------------
def _algorithm1_exact(g, m, theta, t, k, beta, lr):
    """Algorithm 1 in exact rational arithmetic with dense length-d sparse vectors
    (Eq. 3 literally), valid when every intermediate is exactly representable."""
    n, d = len(g), len(g[0])
    L = t % n
    acc = [[m[i][p] + g[i][p] for p in range(d)] for i in range(n)]
    order = sorted(range(d), key=lambda p: (-abs(acc[L][p]), p))
    S = set(order[:k])
    sparse = [[acc[i][p] if p in S else Fraction(0) for p in range(d)] for i in range(n)]   # Eq. 3
    new_m = [[(1 - beta) * m[i][p] + beta * (acc[i][p] - sparse[i][p]) for p in range(d)] for i in range(n)]  # Eq. 4
    gbar = [sum(sparse[i][p] for i in range(n)) / n for p in range(d)]                          # line 10
    new_theta = [theta[p] - lr * gbar[p] for p in range(d)]                                   # line 12
    return sorted(S), gbar, sparse, new_m, new_theta


@pytest.mark.parametrize("dtype", [np.float32, np.float64])
def test_step_equals_exact_rational_algorithm1(dtype):
    rng = np.random.default_rng(7)
    n, d, k = 4, 24, 5
    beta, lr = Fraction(1, 4), Fraction(1, 8)
    g = [[Fraction(int(v), 16) for v in rng.integers(-64, 65, size=d)] for _ in range(n)]
    m = [[Fraction(int(v), 32) for v in rng.integers(-64, 65, size=d)] for _ in range(n)]
    theta = [Fraction(int(v), 8) for v in rng.integers(-16, 17, size=d)]
    for t in range(6):
        S, gbar, sparse, m2, th2 = _algorithm1_exact(g, m, theta, t, k, beta, lr)
        gn = [np.array([float(v) for v in row], dtype) for row in g]
        mn = [np.array([float(v) for v in row], dtype) for row in m]
        thn = np.array([float(v) for v in theta], dtype)
        idx, val, G = oracle.step(gn, mn, thn, t, k, float(beta), float(lr))
        assert idx.tolist() == S
        assert val.tolist() == [float(gbar[p]) for p in S]
        for i in range(n):
            assert G[i].tolist() == [float(sparse[i][p]) for p in S]
            assert mn[i].tolist() == [float(v) for v in m2[i]]
        assert thn.tolist() == [float(v) for v in th2]
        # next iteration: new gradients, carried memory (kept dyadic by beta = 1/4 for a few steps)
        m, theta = m2, th2
        g = [[Fraction(int(v), 16) for v in rng.integers(-64, 65, size=d)] for _ in range(n)]


# ---- P2: k = d is dense averaged SGD ----------------------------------------------------
def test_k_equals_d_is_dense_allreduce_sgd():
    n, d, beta, lr = 5, 257, 0.1, 0.05
    g = [RNG.standard_normal(d) for _ in range(n)]
    m = [np.zeros(d) for _ in range(n)]
    theta = RNG.standard_normal(d)
    theta0 = theta.copy()
    idx, val, G = oracle.step(g, m, theta, 3, d, beta, lr)
    assert idx.tolist() == list(range(d))
    mean_g = np.mean(np.stack(g), axis=0)
    np.testing.assert_allclose(val, mean_g, rtol=1e-14, atol=0)
    np.testing.assert_allclose(theta, theta0 - lr * mean_g, rtol=1e-14, atol=1e-16)
    for i in range(n):
        assert not m[i].any()                       # (1-beta)*0 + beta*0
    # with non-zero memory every coordinate is still sent, so m' = (1-beta) m
    m = [RNG.standard_normal(d) for _ in range(n)]
    m0 = [a.copy() for a in m]
    oracle.step(g, m, None, 0, d, beta, lr)
    for i in range(n):
        np.testing.assert_allclose(m[i], (1 - beta) * m0[i], rtol=1e-15)


# ---- P3: n = 1, beta = 1 is classical error-feedback top-k (Remark 1) ------------------------
def test_single_learner_beta_one_is_error_feedback_topk():
    d, k, lr = 1000, 37, 0.1
    g = RNG.standard_normal(d).astype(np.float32)
    m = (0.3 * RNG.standard_normal(d)).astype(np.float32)
    theta = RNG.standard_normal(d).astype(np.float32)
    acc = m + g
    order = np.argsort(-np.abs(acc), kind="stable")[:k]
    top = np.zeros(d, np.float32)
    top[order] = acc[order]
    theta_expect = theta - np.float32(lr) * top
    m_in = m.copy()
    idx, val, G = oracle.step([g], [m_in], theta, 11, k, 1.0, lr)
    assert idx.tolist() == sorted(order.tolist())
    assert np.array_equal(m_in, acc - top)           # residual, bit for bit
    assert np.array_equal(theta, theta_expect)
    assert np.array_equal(val, acc[idx]) and np.array_equal(G[0], acc[idx])


# ---- P4: acc = sparse + residual -------------------------------------------------------
def test_decomposition_identity():
    n, d, k = 3, 500, 40
    g = [RNG.standard_normal(d).astype(np.float32) for _ in range(n)]
    m = [RNG.standard_normal(d).astype(np.float32) for _ in range(n)]
    acc = [a + b for a, b in zip(m, g)]
    m1 = [a.copy() for a in m]
    idx, val, G = oracle.step(g, m1, None, 1, k, 1.0, 0.0)
    for i in range(n):                                # beta = 1: bitwise
        sparse = np.zeros(d, np.float32)
        sparse[idx] = G[i]
        assert np.array_equal(sparse + m1[i], acc[i])
        assert not m1[i][idx].any()
    beta = 0.1                                        # beta < 1 in double
    g64 = [a.astype(np.float64) for a in g]
    m64 = [a.astype(np.float64) for a in m]
    m2 = [a.copy() for a in m64]
    idx, val, G = oracle.step(g64, m2, None, 1, k, beta, 0.0)
    for i in range(n):
        sparse = np.zeros(d)
        sparse[idx] = G[i]
        np.testing.assert_allclose((m2[i] - (1 - beta) * m64[i]) / beta + sparse, m64[i] + g64[i],
                                   rtol=0, atol=1e-12)
        # a selected coordinate keeps (1-beta) of its memory; it is NOT zeroed unless beta = 1
        np.testing.assert_allclose(m2[i][idx], (1 - beta) * m64[i][idx], rtol=1e-15)


# ---- P5: the leader cycles as t mod n (Algorithm 1 line 6) ---------------------------------
def test_leader_cycles():
    n, blk = 4, 16
    d, k = n * blk, blk
    g = []
    for i in range(n):                                # learner i is large exactly on block i
        v = (0.01 * RNG.standard_normal(d)).astype(np.float32)
        v[i * blk:(i + 1) * blk] += 10.0
        g.append(v)
    seen = []
    for t in range(3 * n):
        m = [np.zeros(d, np.float32) for _ in range(n)]
        idx, _, _ = oracle.step(g, m, None, t, k, 0.5, 0.0)
        leader = idx[0] // blk
        assert idx.tolist() == list(range(leader * blk, (leader + 1) * blk))
        assert leader == t % n
        seen.append(leader)
    assert seen[:n] == list(range(n))
    path = os.path.join(os.path.dirname(__file__), "golden", "leader_demo.txt")
    for line in open(path):
        if line.startswith("#") or not line.strip():
            continue
        gn, gt, gl = map(int, line.split())
        assert gn == n
        m = [np.zeros(d, np.float32) for _ in range(n)]
        idx, _, _ = oracle.step(g, m, None, gt, k, 0.5, 0.0)
        assert idx[0] // blk == gl


# ---- P6: commutativity, Eq. 1 -------------------------------------------------------------
def test_commutativity_of_cltk_with_averaging():
    n, d, k, t = 6, 400, 25, 8
    g = [RNG.standard_normal(d) for _ in range(n)]
    m = [RNG.standard_normal(d) for _ in range(n)]
    acc = np.stack([a + b for a, b in zip(m, g)])
    idx, val, G = oracle.step(g, [a.copy() for a in m], None, t, k, 0.3, 0.0)
    leader_set, _ = oracle.topk(acc[t % n].copy(), k)
    assert idx.tolist() == leader_set.tolist()
    mean_acc = acc.mean(axis=0)
    lhs = np.zeros(d); lhs[idx] = mean_acc[idx]         # sparse(mean x_i) with the leader's set
    rhs = np.zeros(d); rhs[idx] = val                   # mean sparse(x_i)
    np.testing.assert_allclose(lhs, rhs, rtol=1e-13, atol=1e-15)
    np.testing.assert_array_equal(G, acc[:, idx])


# ---- P7: virtual sequence, Appendix D.1 ------------------------------------------------------
@pytest.mark.parametrize("dtype,tol", [(np.float64, 1e-12), (np.float32, 1e-4)])
def test_virtual_sequence_identity(dtype, tol):
    n, d, k, beta, lr, T = 4, 600, 30, 0.1, 0.05, 25
    theta = np.zeros(d, dtype)                        # theta^0 = v^0 = m^0 = 0
    v = np.zeros(d, np.float64)
    m = [np.zeros(d, dtype) for _ in range(n)]
    rng = np.random.default_rng(3)
    for t in range(T):
        g = [rng.standard_normal(d).astype(dtype) for _ in range(n)]
        v = v - lr * np.mean(np.stack(g).astype(np.float64), axis=0)
        oracle.step(g, m, theta, t, k, beta, lr)
        mbar = np.mean(np.stack(m).astype(np.float64), axis=0)
        lhs = theta.astype(np.float64) - v
        rhs = (lr / beta) * mbar
        assert np.max(np.abs(lhs - rhs)) <= tol * max(1.0, np.max(np.abs(rhs)))


# ---- P8: contraction, Lemma 1 proof identity and the top-k bound ----------------------------
def test_contraction_properties():
    n, d, k, t = 4, 2000, 100, 2
    g = [RNG.standard_normal(d) for _ in range(n)]
    m = [np.zeros(d) for _ in range(n)]
    idx, val, G = oracle.step(g, [a.copy() for a in m], None, t, k, 1.0, 0.0)
    L = t % n
    for j in range(n):
        x = g[j]
        comp = np.zeros(d); comp[idx] = G[j]
        lhs = np.sum((x - comp) ** 2)
        np.testing.assert_allclose(lhs, np.sum(x ** 2) - np.sum(x[idx] ** 2), rtol=1e-12)
        if j == L:
            assert lhs <= (1 - k / d) * np.sum(x ** 2)


# ---- P9 + P10: threshold property and a library cross-check on a larger vector -----------------
def test_threshold_property_and_library_topk():
    d, k = 200_000, 2000
    x = RNG.standard_normal(d).astype(np.float32)
    x[RNG.integers(0, d, 500)] = np.float32(2.5)        # a tie group straddling the threshold region
    idx, sel = oracle.topk(x, k)
    key = key32(x)
    assert idx.size == k and np.all(np.diff(idx) > 0)
    inside, outside = key[sel == 1], key[sel == 0]
    tau = inside.min()
    assert tau >= outside.max()
    ties_in = np.flatnonzero((key == tau) & (sel == 1))
    ties_out = np.flatnonzero((key == tau) & (sel == 0))
    if ties_in.size and ties_out.size:
        assert ties_in.max() < ties_out.min()
    lib = np.sort(np.argsort(-key.astype(np.int64), kind="stable")[:k])
    assert np.array_equal(lib, idx)
    import torch
    tk = torch.topk(torch.from_numpy(np.abs(x)), k).indices.numpy()
    strict = key[tk] > tau                               # above the threshold every routine must agree
    assert set(tk[strict].tolist()) == set(idx[key[idx] > tau].tolist())
    for p in RNG.integers(0, d, 20):
        assert (oracle.rank(x, int(p)) < k) == bool(sel[p])


def test_pieces_compose_to_step():
    """The step is exactly accumulate -> topk -> learner x n -> reduce -> apply."""
    n, d, k, beta, lr, t = 3, 300, 20, 0.1, 0.01, 4
    g = [RNG.standard_normal(d).astype(np.float32) for _ in range(n)]
    m = [RNG.standard_normal(d).astype(np.float32) for _ in range(n)]
    th = RNG.standard_normal(d).astype(np.float32)
    m1, th1 = [a.copy() for a in m], th.copy()
    idx, val, G = oracle.step(g, m1, th1, t, k, beta, lr)
    acc = oracle.accumulate(g[t % n], m[t % n])
    assert np.array_equal(acc, m[t % n] + g[t % n])
    idx2, sel = oracle.topk(acc, k)
    m2 = [a.copy() for a in m]
    G2 = np.stack([oracle.learner(g[i], m2[i], idx2, sel, beta) for i in range(n)])
    val2 = oracle.reduce(np.ascontiguousarray(G2))
    th2 = th.copy()
    oracle.apply(th2, idx2, val2, lr)
    assert np.array_equal(idx, idx2) and np.array_equal(val, val2) and np.array_equal(G, G2)
    assert all(np.array_equal(a, b) for a, b in zip(m1, m2)) and np.array_equal(th1, th2)


# ---- chunk-wise selector (Section 4, Appendix E) -----------------------------------------------
def test_chunk_select_brute_force_and_limits():
    for x in tie_vectors():
        d = x.size
        key = key32(x).astype(np.int64)
        for k in range(1, d + 1):
            idx, sel = oracle.chunk_select(x, k)
            bounds = [(j * d) // k for j in range(k + 1)]
            assert bounds[0] == 0 and bounds[-1] == d and all(b > a for a, b in zip(bounds, bounds[1:]))
            expect = []
            for j in range(k):
                chunk = range(bounds[j], bounds[j + 1])
                best = max(chunk, key=lambda p: (key[p], -p))         # largest magnitude, then lowest index
                expect.append(best)
            assert idx.tolist() == expect
            assert sel.tolist() == [1 if p in expect else 0 for p in range(d)]
            assert np.array_equal(oracle.chunk_select(x.astype(np.float64), k)[0], idx)
        assert oracle.chunk_select(x, d)[0].tolist() == list(range(d))          # k = d keeps everything
        assert oracle.chunk_select(x, 1)[0].tolist() == oracle.topk(x, 1)[0].tolist()   # k = 1 is the top-1 set


def test_chunk_select_matches_the_demonstration_structure():
    path = os.path.join(os.path.dirname(__file__), "golden", "chunk_demo.txt")
    row = [l for l in open(path) if l.strip() and not l.startswith("#")][0].split()
    d, k = int(row[0]), int(row[1])
    chunk_of = list(map(int, row[2:2 + d]))
    picks = list(map(int, row[2 + d:2 + d + k]))
    x = np.full(d, 0.1, np.float32)
    for j, local in enumerate(picks):                      # make the demonstrated local index the chunk's largest
        x[chunk_of.index(j) + local] = -3.0 - j
    idx, sel = oracle.chunk_select(x, k)
    assert [chunk_of[p] for p in idx] == list(range(k))
    assert [p - chunk_of.index(j) for j, p in enumerate(idx)] == picks


def test_chunk_step_is_the_same_algorithm_with_another_index_set():
    n, d, k, beta, lr, t = 3, 1000, 37, 0.1, 0.05, 5
    g = [RNG.standard_normal(d) for _ in range(n)]
    m = [RNG.standard_normal(d) for _ in range(n)]
    th = RNG.standard_normal(d)
    m1, th1 = [a.copy() for a in m], th.copy()
    idx, val, G = oracle.step(g, m1, th1, t, k, beta, lr, selector="chunk")
    acc = np.stack([a + b for a, b in zip(m, g)])
    assert np.array_equal(idx, oracle.chunk_select(acc[t % n].copy(), k)[0])
    np.testing.assert_allclose(val, acc[:, idx].mean(axis=0), rtol=1e-13)          # Eq. 1 with the chunk set
    np.testing.assert_array_equal(G, acc[:, idx])
    for i in range(n):
        r = acc[i].copy(); r[idx] = 0.0
        np.testing.assert_allclose(m1[i], (1 - beta) * m[i] + beta * r, rtol=1e-13, atol=1e-15)   # Eq. 4
    expect = th.copy(); expect[idx] -= lr * val
    np.testing.assert_allclose(th1, expect, rtol=1e-14)
    # contraction of any index set of size k (proof of Lemma 1): ||x - comp(x)||^2 = ||x||^2 - sum over the set
    x = acc[t % n]
    comp = np.zeros(d); comp[idx] = x[idx]
    np.testing.assert_allclose(np.sum((x - comp) ** 2), np.sum(x ** 2) - np.sum(x[idx] ** 2), rtol=1e-12)


# ---- diagnostics: Eq. 5 and the cosine distance of Section 2 -------------------------------------
def test_diagnostics_closed_forms():
    d, k, n = 500, 40, 5
    g = [RNG.standard_normal(d).astype(np.float32) for _ in range(n)]
    m = [RNG.standard_normal(d).astype(np.float32) for _ in range(n)]
    mean = oracle.mean_acc(g, m)
    np.testing.assert_allclose(mean, np.mean([a.astype(np.float64) + b for a, b in zip(m, g)], axis=0), rtol=2e-6, atol=1e-7)
    # the reduction of Algorithm 1 line 10 is this vector restricted to the selected coordinates
    idx, val, _ = oracle.step(g, [a.copy() for a in m], None, 2, k, 0.5, 0.0)
    assert np.array_equal(val, mean[idx])
    # Eq. 5: H = 2d; identical sets d = 0, disjoint sets d = k, one swapped index d = 1
    a = np.zeros(d, np.uint8); a[:k] = 1
    b = np.zeros(d, np.uint8); b[k:2 * k] = 1
    c = a.copy(); c[0] = 0; c[d - 1] = 1
    assert oracle.hamming_d(a, a) == 0 and oracle.hamming_d(a, b) == k and oracle.hamming_d(a, c) == 1
    _, s1 = oracle.topk(g[0], k)
    _, s2 = oracle.topk(g[1], k)
    i1, i2 = set(np.flatnonzero(s1)), set(np.flatnonzero(s2))
    assert oracle.hamming_d(s1, s2) == k - len(i1 & i2) == len(i1 ^ i2) // 2
    # with one learner the leader's set is the true top-k set
    _, sl = oracle.topk(oracle.accumulate(g[0], m[0]), k)
    _, st = oracle.topk(oracle.mean_acc(g[:1], m[:1]), k)
    assert oracle.hamming_d(sl, st) == 0
    # cosine distance: 0 for parallel, 2 for opposite, 1 for orthogonal, scale invariant
    x = RNG.standard_normal(d)
    y = RNG.standard_normal(d)
    assert abs(oracle.cosine_distance(x, 3.0 * x)) < 1e-15
    assert abs(oracle.cosine_distance(x, -0.5 * x) - 2.0) < 1e-15
    e1 = np.zeros(d); e1[3] = 2.0
    e2 = np.zeros(d); e2[7] = -5.0
    assert oracle.cosine_distance(e1, e2) == 1.0
    ref = 1.0 - float(np.dot(x, y)) / (np.linalg.norm(x) * np.linalg.norm(y))
    assert abs(oracle.cosine_distance(x, y) - ref) < 1e-14
    assert abs(oracle.cosine_distance(2.0 * x, 7.0 * y) - ref) < 1e-14


# ---- chunk-wise selection with per-layer rates (Section 4) ---------------------------------------
def test_layer_chunk_select():
    sizes = [7, 64, 1, 300, 128]
    keep = [7, 2, 1, 3, 16]                    # uncompressed layer, 32X, a single coordinate, 100X, 8X
    d = sum(sizes)
    x = RNG.standard_normal(d).astype(np.float32)
    x[80:90] = 0.0                              # a run of ties inside a layer
    idx, sel = oracle.layer_chunk_select(x, sizes, keep)
    assert idx.size == sum(keep) and np.all(np.diff(idx) > 0) and sel.sum() == sum(keep)
    key = key32(x).astype(np.int64)
    off, expect = 0, []
    for sz, kp in zip(sizes, keep):             # brute force: per layer, per chunk, largest magnitude then lowest index
        for j in range(kp):
            lo, hi = off + (j * sz) // kp, off + ((j + 1) * sz) // kp
            expect.append(max(range(lo, hi), key=lambda p: (key[p], -p)))
        off += sz
    assert idx.tolist() == expect
    assert idx[:7].tolist() == list(range(7))                          # keep = size: the layer is sent whole
    # one layer is the plain chunk-wise selector
    assert np.array_equal(oracle.layer_chunk_select(x, [d], [13])[0], oracle.chunk_select(x, 13)[0])
    # the step with layers is the same algorithm with that index set
    g = [RNG.standard_normal(d) for _ in range(3)]
    m = [RNG.standard_normal(d) for _ in range(3)]
    acc = np.stack([a + b for a, b in zip(m, g)])
    idx2, val, G = oracle.step(g, [a.copy() for a in m], None, 4, sum(keep), 0.5, 0.0, selector="chunk", layers=(sizes, keep))
    assert np.array_equal(idx2, oracle.layer_chunk_select(acc[4 % 3].copy(), sizes, keep)[0])
    np.testing.assert_allclose(val, acc[:, idx2].mean(axis=0), rtol=1e-13)


# ---- exact top-k with per-layer rates (Eq. 2 inside each layer, Section 4's rates) -----------------
def test_layer_topk():
    sizes = [7, 64, 1, 300, 128, 40]
    keep = [7, 2, 1, 3, 16, 5]                 # uncompressed layer, 32X, a single coordinate, 100X, 8X, 8X over ties
    d = sum(sizes)
    x = RNG.standard_normal(d).astype(np.float32)
    x[80:90] = 0.0                              # zeros inside a layer (never picked while larger values remain)
    x[500:540] = -0.25                          # the last layer is one 40-way tie: its 5 lowest indices win
    x[510] = 0.25                               # the sign does not break the tie
    idx, sel = oracle.layer_topk(x, sizes, keep)
    assert idx.size == sum(keep) and np.all(np.diff(idx) > 0) and sel.sum() == sum(keep)
    assert np.array_equal(np.flatnonzero(sel), idx)
    key = key32(x).astype(np.int64)
    off, expect = 0, []
    for sz, kp in zip(sizes, keep):             # brute force by counting: p is kept iff fewer than keep precede it
        for p in range(off, off + sz):
            before = sum(1 for q in range(off, off + sz) if key[q] > key[p] or (key[q] == key[p] and q < p))
            if before < kp:
                expect.append(p)
        off += sz
    assert idx.tolist() == expect
    assert idx[:7].tolist() == list(range(7))                          # keep = size: the layer is sent whole
    assert idx[-5:].tolist() == [500, 501, 502, 503, 504]              # ties go to the lower index
    # one layer is Eq. 2 on the whole vector
    assert np.array_equal(oracle.layer_topk(x, [d], [13])[0], oracle.topk(x, 13)[0])
    # moving a layer boundary changes the result (the layers are searched separately)
    y = np.arange(1, 21, dtype=np.float32)
    assert oracle.layer_topk(y, [10, 10], [1, 1])[0].tolist() == [9, 19]
    assert oracle.layer_topk(y, [15, 5], [1, 1])[0].tolist() == [14, 19]
    assert oracle.topk(y, 2)[0].tolist() == [18, 19]
    # the step with layers and the exact selector is the same algorithm with that index set
    g = [RNG.standard_normal(d) for _ in range(3)]
    m = [RNG.standard_normal(d) for _ in range(3)]
    acc = np.stack([a + b for a, b in zip(m, g)])
    idx2, val, G = oracle.step(g, [a.copy() for a in m], None, 4, sum(keep), 0.5, 0.0, selector="topk", layers=(sizes, keep))
    assert np.array_equal(idx2, oracle.layer_topk(acc[4 % 3].copy(), sizes, keep)[0])
    np.testing.assert_allclose(val, acc[:, idx2].mean(axis=0), rtol=1e-13)
    assert np.array_equal(G, acc[:, idx2])


def test_threaded_step_equals_the_plain_step():
    """The all-cores variant used as the benchmark's parallel CPU baseline hands the plain routines' loops to
    threads; it must return the same bits (ties at the threshold included, several thread counts, k larger than
    a thread's range)."""
    import oracle
    rng = np.random.default_rng(21)
    n, d = 5, 50_021
    g = [rng.standard_normal(d).astype(np.float32) for _ in range(n)]
    g[2] = (np.round(g[2] * 2) / 2).astype(np.float32)             # heavy ties when learner 2 leads
    for k in (1, 777, 20_000, d):
        for threads in (2, 3, 8):
            m1 = [0.1 * x for x in g]
            m2 = [x.copy() for x in m1]
            th1 = np.linspace(-1, 1, d, dtype=np.float32)
            th2 = th1.copy()
            for t in range(3):
                a = oracle.step(g, m1, th1, t, k, 0.25, 0.5)
                b = oracle.step(g, m2, th2, t, k, 0.25, 0.5, threads=threads)
                assert all(np.array_equal(x, y) for x, y in zip(a, b)), (k, threads, t)
            assert all(np.array_equal(x, y) for x, y in zip(m1, m2)) and np.array_equal(th1, th2)

"""CLT-k oracle -- TEST INFRASTRUCTURE, never part of the product path.

Thin ctypes marshalling around ``cltk_oracle.c`` (plain C, fp32 and fp64): a
slow, single-threaded, step-by-step statement of one ScaleCom iteration
(Algorithm 1; CLT-k compressor Eq. 2-3; low-pass-filtered memory Eq. 4).
Only the tests, the smoke check and the benchmark's CPU-baseline leg may
import this package.  All arithmetic lives in the C file; this module only
converts numpy arrays to pointers.

Pins (see tests/test_oracle_pins.py): brute-force rank counting and subset
enumeration on tiny d (Eq. 2), k = d reducing to dense averaged SGD
(Algorithm 1 lines 10-12), n = 1 with beta = 1 reducing to classical
error-feedback top-k (Remark 1), acc = sparse + residual (Eq. 4), leader
cycling (Algorithm 1 line 6), commutativity (Eq. 1), the virtual-sequence
identity of Appendix D.1, the contraction identity of Appendix C and a
library top-k cross-check; the chunk-wise selector by per-chunk brute force,
its k = d and k = 1 limits and the structure of Appendix E's demonstration;
the diagnostics (all-reduced vector, Hamming distance of Eq. 5, cosine
distance) by their closed forms and special cases.
No function here is "parity unpinned".
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "cltk_oracle.c")
_INC = os.path.join(_HERE, "cltk_oracle_body.inc")
_SRC_MT = os.path.join(_HERE, "cltk_oracle_mt.c")
_LIB = os.path.join(_HERE, "libcltk_oracle.so")

CFLAGS = ["-std=c99", "-O2", "-ffp-contract=off", "-fPIC", "-shared", "-pthread"]


def build(force: bool = False) -> str:
    """Compile the oracle with gcc if the shared object is missing or stale."""
    stale = (not os.path.exists(_LIB)
             or os.path.getmtime(_LIB) < max(os.path.getmtime(_SRC), os.path.getmtime(_INC), os.path.getmtime(_SRC_MT)))
    if force or stale:
        tmp = _LIB + ".tmp.%d" % os.getpid()
        subprocess.run(["gcc", *CFLAGS, _SRC, _SRC_MT, "-o", tmp, "-lm"], check=True, cwd=_HERE)
        os.replace(tmp, _LIB)
    return _LIB


_lib = None


def _load():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        i32, i64 = ctypes.c_int32, ctypes.c_int64
        vp = ctypes.c_void_p
        for sfx, real in (("f32", ctypes.c_float), ("f64", ctypes.c_double)):
            f = getattr(_lib, "oracle_rank_" + sfx); f.restype = i64; f.argtypes = [vp, i64, i64]
            f = getattr(_lib, "oracle_topk_" + sfx); f.restype = ctypes.c_int; f.argtypes = [vp, i64, i64, vp, vp]
            f = getattr(_lib, "oracle_chunk_select_" + sfx); f.restype = ctypes.c_int; f.argtypes = [vp, i64, i64, vp, vp]
            f = getattr(_lib, "oracle_step_sel_" + sfx); f.restype = ctypes.c_int
            f.argtypes = [vp, vp, vp, i64, i32, i64, i64, real, real, ctypes.c_int, vp, vp, vp]
            f = getattr(_lib, "oracle_layer_chunk_select_" + sfx); f.restype = ctypes.c_int
            f.argtypes = [vp, i32, vp, vp, vp, vp]
            f = getattr(_lib, "oracle_layer_topk_" + sfx); f.restype = ctypes.c_int
            f.argtypes = [vp, i32, vp, vp, vp, vp]
            f = getattr(_lib, "oracle_step_layers_" + sfx); f.restype = ctypes.c_int
            f.argtypes = [vp, vp, vp, i64, i32, i64, i64, real, real, ctypes.c_int, i32, vp, vp, vp, vp, vp]
            f = getattr(_lib, "oracle_mean_acc_" + sfx); f.restype = None; f.argtypes = [vp, vp, i32, i64, vp]
            f = getattr(_lib, "oracle_hamming_d_" + sfx); f.restype = i64; f.argtypes = [vp, vp, i64]
            f = getattr(_lib, "oracle_cosine_distance_" + sfx); f.restype = ctypes.c_double; f.argtypes = [vp, vp, i64]
            f = getattr(_lib, "oracle_accumulate_" + sfx); f.restype = None; f.argtypes = [vp, vp, i64, vp]
            f = getattr(_lib, "oracle_learner_" + sfx); f.restype = None
            f.argtypes = [vp, vp, i64, vp, i64, vp, real, vp]
            f = getattr(_lib, "oracle_reduce_" + sfx); f.restype = None; f.argtypes = [vp, i32, i64, vp]
            f = getattr(_lib, "oracle_apply_" + sfx); f.restype = None; f.argtypes = [vp, vp, vp, i64, real]
            f = getattr(_lib, "oracle_step_" + sfx); f.restype = ctypes.c_int
            f.argtypes = [vp, vp, vp, i64, i32, i64, i64, real, real, vp, vp, vp]
        f = _lib.oracle_step_threads_f32; f.restype = ctypes.c_int
        f.argtypes = [vp, vp, vp, i64, i32, i64, i64, ctypes.c_float, ctypes.c_float, i32, vp, vp, vp]
    return _lib


def host_cores() -> int:
    """Host cores this process may run on."""
    try:
        return len(os.sched_getaffinity(0))
    except AttributeError:  # pragma: no cover
        return os.cpu_count() or 1


def _sfx(dtype) -> str:
    dtype = np.dtype(dtype)
    if dtype == np.float32:
        return "f32"
    if dtype == np.float64:
        return "f64"
    raise TypeError("oracle works in float32 or float64, got %s" % dtype)


def _chk(a: np.ndarray, dtype, shape=None) -> np.ndarray:
    if not isinstance(a, np.ndarray) or a.dtype != np.dtype(dtype) or not a.flags.c_contiguous:
        raise TypeError("expected a C-contiguous %s ndarray" % np.dtype(dtype))
    if shape is not None and tuple(a.shape) != tuple(shape):
        raise ValueError("expected shape %s, got %s" % (shape, a.shape))
    return a


def _p(a: np.ndarray) -> int:
    return a.ctypes.data


def rank(x: np.ndarray, p: int) -> int:
    """rank(p) by counting; p is in the top-k set of x exactly when rank < k (Eq. 2)."""
    lib = _load()
    return int(getattr(lib, "oracle_rank_" + _sfx(x.dtype))(_p(_chk(x, x.dtype)), x.size, int(p)))


def topk(x: np.ndarray, k: int):
    """Top-k index set of x by magnitude (Eq. 2): returns (idx int32[k] ascending, sel uint8[d])."""
    lib = _load()
    d = x.size
    idx = np.empty(k, np.int32)
    sel = np.empty(d, np.uint8)
    rc = getattr(lib, "oracle_topk_" + _sfx(x.dtype))(_p(_chk(x, x.dtype)), d, int(k), _p(idx), _p(sel))
    if rc != 0:
        raise MemoryError("oracle_topk")
    return idx, sel


SELECTORS = {"topk": 0, "chunk": 1}


def chunk_select(x: np.ndarray, k: int):
    """Chunk-wise selection (Section 4 / Appendix E): one coordinate from each of k consecutive
    chunks; returns (idx int32[k] ascending, sel uint8[d])."""
    lib = _load()
    d = x.size
    idx = np.empty(k, np.int32)
    sel = np.empty(d, np.uint8)
    getattr(lib, "oracle_chunk_select_" + _sfx(x.dtype))(_p(_chk(x, x.dtype)), d, int(k), _p(idx), _p(sel))
    return idx, sel


def layer_chunk_select(x: np.ndarray, sizes, keep):
    """Chunk-wise selection with per-layer rates (Section 4): layer s has sizes[s] coordinates and
    keeps keep[s]; returns (idx int32[sum keep] ascending, sel uint8[d])."""
    lib = _load()
    sz = np.ascontiguousarray(sizes, np.int64)
    kp = np.ascontiguousarray(keep, np.int64)
    assert sz.sum() == x.size and sz.size == kp.size and np.all(kp >= 1) and np.all(kp <= sz)
    idx = np.empty(int(kp.sum()), np.int32)
    sel = np.empty(x.size, np.uint8)
    getattr(lib, "oracle_layer_chunk_select_" + _sfx(x.dtype))(_p(_chk(x, x.dtype)), sz.size, _p(sz), _p(kp), _p(idx), _p(sel))
    return idx, sel


def layer_topk(x: np.ndarray, sizes, keep):
    """Exact top-k inside every layer (Eq. 2 applied per layer with Section 4's per-layer rates): layer s has
    sizes[s] coordinates and keeps keep[s]; returns (idx int32[sum keep] ascending, sel uint8[d])."""
    lib = _load()
    sz = np.ascontiguousarray(sizes, np.int64)
    kp = np.ascontiguousarray(keep, np.int64)
    assert sz.size == kp.size and sz.sum() == x.size and np.all(kp >= 1) and np.all(kp <= sz)
    idx = np.empty(int(kp.sum()), np.int32)
    sel = np.empty(x.size, np.uint8)
    if getattr(lib, "oracle_layer_topk_" + _sfx(x.dtype))(_p(_chk(x, x.dtype)), sz.size, _p(sz), _p(kp), _p(idx), _p(sel)) != 0:
        raise MemoryError("oracle_layer_topk")
    return idx, sel


def mean_acc(g, m) -> np.ndarray:
    """(1/n) sum_i (m_i + g_i), learner order, one division: the all-reduced error-feedback gradient."""
    lib = _load()
    n, dtype, d = len(g), g[0].dtype, g[0].size
    for a in list(g) + list(m):
        _chk(a, dtype, (d,))
    gp = (ctypes.c_void_p * n)(*[_p(a) for a in g])
    mp = (ctypes.c_void_p * n)(*[_p(a) for a in m])
    out = np.empty(d, dtype)
    getattr(lib, "oracle_mean_acc_" + _sfx(dtype))(ctypes.cast(gp, ctypes.c_void_p), ctypes.cast(mp, ctypes.c_void_p),
                                                   n, d, _p(out))
    return out


def hamming_d(sel1: np.ndarray, sel2: np.ndarray) -> int:
    """d of Eq. 5: half the Hamming distance between two 0/1 indicator vectors (uint8)."""
    lib = _load()
    _chk(sel1, np.uint8); _chk(sel2, np.uint8, sel1.shape)
    return int(lib.oracle_hamming_d_f32(_p(sel1), _p(sel2), sel1.size))


def cosine_distance(x: np.ndarray, y: np.ndarray) -> float:
    """1 - x.y / (|x| |y|) (Section 2, footnote), accumulated in double."""
    lib = _load()
    _chk(y, x.dtype, x.shape)
    return float(getattr(lib, "oracle_cosine_distance_" + _sfx(x.dtype))(_p(_chk(x, x.dtype)), _p(y), x.size))


def accumulate(g: np.ndarray, m: np.ndarray) -> np.ndarray:
    """acc = m + g (the argument of CLT-k, Algorithm 1 line 6)."""
    lib = _load()
    acc = np.empty_like(g)
    getattr(lib, "oracle_accumulate_" + _sfx(g.dtype))(_p(_chk(g, g.dtype)), _p(_chk(m, g.dtype, g.shape)), g.size, _p(acc))
    return acc


def learner(g: np.ndarray, m: np.ndarray, idx: np.ndarray, sel: np.ndarray, beta: float) -> np.ndarray:
    """One learner's gather (Eq. 3) and in-place memory update (Eq. 4); returns gathered[k]."""
    lib = _load()
    _chk(m, g.dtype, g.shape); _chk(idx, np.int32); _chk(sel, np.uint8, g.shape)
    gathered = np.empty(idx.size, g.dtype)
    getattr(lib, "oracle_learner_" + _sfx(g.dtype))(_p(_chk(g, g.dtype)), _p(m), g.size, _p(idx), idx.size, _p(sel),
                                                    float(beta), _p(gathered))
    return gathered


def reduce(G: np.ndarray) -> np.ndarray:
    """val[j] = (sum over learners, in order, of G[i][j]) / n (Algorithm 1 line 10)."""
    lib = _load()
    n, k = G.shape
    val = np.empty(k, G.dtype)
    getattr(lib, "oracle_reduce_" + _sfx(G.dtype))(_p(_chk(G, G.dtype)), n, k, _p(val))
    return val


def apply(theta: np.ndarray, idx: np.ndarray, val: np.ndarray, lr: float) -> None:
    """theta[idx[j]] -= lr * val[j], in place (Algorithm 1 line 12)."""
    lib = _load()
    _chk(idx, np.int32); _chk(val, theta.dtype, idx.shape)
    getattr(lib, "oracle_apply_" + _sfx(theta.dtype))(_p(_chk(theta, theta.dtype)), _p(idx), _p(val), idx.size, float(lr))


def step(g, m, theta, t: int, k: int, beta: float, lr: float, want_gathered: bool = True,
         selector: str = "topk", layers=None, threads: int = 1):
    """One iteration of Algorithm 1 ("topk": Eq. 2 on the leader; "chunk": chunk-wise selection,
    with per-layer rates when layers = (sizes, keep) is given).  threads > 1 (fp32, "topk", no layers):
    the same routines with their loops spread over that many threads -- identical results, shorter wall clock.

    g, m: lists of n ndarrays of d values (m updated in place); theta: ndarray
    of d values updated in place, or None.  Returns (idx, val, G) with G the
    n-by-k gathered values (None unless want_gathered).
    """
    lib = _load()
    n = len(g)
    dtype = g[0].dtype
    d = g[0].size
    for a in list(g) + list(m):
        _chk(a, dtype, (d,))
    if theta is not None:
        _chk(theta, dtype, (d,))
    gp = (ctypes.c_void_p * n)(*[_p(a) for a in g])
    mp = (ctypes.c_void_p * n)(*[_p(a) for a in m])
    idx = np.empty(k, np.int32)
    val = np.empty(k, dtype)
    G = np.empty((n, k), dtype) if want_gathered else None
    if layers is not None:
        sz = np.ascontiguousarray(layers[0], np.int64)
        kp = np.ascontiguousarray(layers[1], np.int64)
        assert sz.sum() == d and kp.sum() == k and sz.size == kp.size
        nl, szp, kpp = sz.size, _p(sz), _p(kp)
    else:
        nl, szp, kpp = 0, None, None
    if threads > 1:
        if np.dtype(dtype) != np.float32 or selector != "topk" or layers is not None:
            raise ValueError("the threaded step is fp32, exact top-k, no layers")
        rc = lib.oracle_step_threads_f32(
            ctypes.cast(gp, ctypes.c_void_p), ctypes.cast(mp, ctypes.c_void_p),
            _p(theta) if theta is not None else None, int(t), n, d, int(k), float(beta), float(lr), int(threads),
            _p(idx), _p(val), _p(G) if G is not None else None)
        if rc != 0:
            raise MemoryError("oracle_step_threads")
        return idx, val, G
    rc = getattr(lib, "oracle_step_layers_" + _sfx(dtype))(
        ctypes.cast(gp, ctypes.c_void_p), ctypes.cast(mp, ctypes.c_void_p),
        _p(theta) if theta is not None else None,
        int(t), n, d, int(k), float(beta), float(lr), SELECTORS[selector], nl, szp, kpp, _p(idx), _p(val),
        _p(G) if G is not None else None)
    if rc != 0:
        raise MemoryError("oracle_step")
    return idx, val, G

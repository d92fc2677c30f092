"""ctypes binding of libscalecom.so: argument marshalling only.

Every function mirrors the C entry point of the same name in
include/scalecom.h; torch is used for device memory and streams, nothing is
computed here.  There is no fallback: if the compiled library is missing the
first call raises.
"""
from __future__ import annotations

import ctypes
import os
from typing import List, Optional, Sequence, Tuple

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libscalecom.so")

OK = 0
ERR_INVALID_ARG, ERR_NULL_PTR, ERR_ALLOC, ERR_CUDA = -1, -2, -3, -4
ERR_TIMEOUT, ERR_BAD_STATE, ERR_INTERNAL, ERR_ALIAS = -5, -6, -7, -8
MAX_LEARNERS = 1024

OPT_FORCE_EXACT_PATH, OPT_SPIN_LIMIT, OPT_KERNEL_TIMING, OPT_FUSE_UPDATE, OPT_USE_HINT, OPT_SELECTOR, OPT_KERNEL_SPANS = 1, 2, 3, 4, 5, 6, 7
OPT_FUSED_SMALL = 8
OPT_L2_KEEP = 9
PATH_SAMPLED, PATH_EXACT, PATH_HINTED, PATH_CHUNK, PATH_LAYER_TOPK, PATH_LAYER_TOPK_STREAM = 0, 1, 2, 3, 4, 5
SELECTOR_TOPK, SELECTOR_CHUNK, SELECTOR_LAYER_TOPK = 0, 1, 2
Q_PHASE_STAMP0 = 100
Q_WORKSPACE_BYTES, Q_LAST_TOPK_PATH, Q_LAST_CANDIDATES, Q_TOPK_BLOCKS, Q_KERNEL_LAUNCHES, Q_FUSED_SMALL = 1, 2, 3, 4, 5, 6

EXPORTS = (
    "scalecom_create", "scalecom_step", "scalecom_step_host", "scalecom_destroy", "scalecom_set_stream",
    "scalecom_set_gathered", "scalecom_apply_update", "scalecom_status", "scalecom_reset",
    "scalecom_set_option", "scalecom_query", "scalecom_kernel_ms", "scalecom_strerror",
    "scalecom_topk_static", "scalecom_kernel_span_ms", "scalecom_enable_peer_access", "scalecom_overlap", "scalecom_cosine_distance", "scalecom_set_layers", "scalecom_select", "scalecom_compress", "scalecom_reduce_rows", "scalecom_compress_scatter",
)
STATIC_MAX_D = 1 << 20

_lib = None


class ScaleComError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__("%s failed: %s (%d)" % (where, strerror(code), code))


def lib() -> ctypes.CDLL:
    """Load the compiled library (once).  Raises if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(
                "libscalecom.so is missing (%s): build it with "
                "`python -m paper_2104_11125_b200.build`; there is no fallback path" % LIB_PATH)
        L = ctypes.CDLL(LIB_PATH)
        vp, i32, i64, f32 = ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64, ctypes.c_float
        L.scalecom_create.restype = ctypes.c_int
        L.scalecom_create.argtypes = [ctypes.POINTER(vp), i64, i32, i64, f32, f32]
        L.scalecom_step.restype = ctypes.c_int
        L.scalecom_step.argtypes = [vp, vp, vp, vp, i64, vp, vp]
        L.scalecom_step_host.restype = ctypes.c_int
        L.scalecom_step_host.argtypes = [vp, vp, vp, vp, i64, vp, vp]
        L.scalecom_destroy.restype = None
        L.scalecom_destroy.argtypes = [vp]
        L.scalecom_set_stream.restype = ctypes.c_int
        L.scalecom_set_stream.argtypes = [vp, vp]
        L.scalecom_set_gathered.restype = ctypes.c_int
        L.scalecom_set_gathered.argtypes = [vp, vp]
        L.scalecom_apply_update.restype = ctypes.c_int
        L.scalecom_apply_update.argtypes = [vp, vp, vp, vp, i64, f32]
        L.scalecom_status.restype = ctypes.c_int
        L.scalecom_status.argtypes = [vp]
        L.scalecom_reset.restype = ctypes.c_int
        L.scalecom_reset.argtypes = [vp]
        L.scalecom_set_option.restype = ctypes.c_int
        L.scalecom_set_option.argtypes = [vp, ctypes.c_int, i64]
        L.scalecom_query.restype = ctypes.c_int
        L.scalecom_query.argtypes = [vp, ctypes.c_int, ctypes.POINTER(i64)]
        L.scalecom_kernel_ms.restype = ctypes.c_int
        L.scalecom_kernel_ms.argtypes = [vp, ctypes.POINTER(f32), ctypes.POINTER(i32)]
        L.scalecom_topk_static.restype = ctypes.c_int
        L.scalecom_topk_static.argtypes = [vp, vp, i64, i64, vp, vp, vp]
        L.scalecom_kernel_span_ms.restype = ctypes.c_int
        L.scalecom_kernel_span_ms.argtypes = [vp, ctypes.POINTER(f32), ctypes.POINTER(i32)]
        L.scalecom_overlap.restype = ctypes.c_int
        L.scalecom_overlap.argtypes = [vp, vp, vp, i64, ctypes.POINTER(i64)]
        L.scalecom_cosine_distance.restype = ctypes.c_int
        L.scalecom_cosine_distance.argtypes = [vp, vp, vp, ctypes.POINTER(ctypes.c_double)]
        L.scalecom_set_layers.restype = ctypes.c_int
        L.scalecom_set_layers.argtypes = [vp, i32, vp, vp]
        L.scalecom_select.restype = ctypes.c_int
        L.scalecom_select.argtypes = [vp, vp, vp, vp]
        L.scalecom_compress.restype = ctypes.c_int
        L.scalecom_compress.argtypes = [vp, vp, vp, vp, vp]
        L.scalecom_compress_scatter.restype = ctypes.c_int
        L.scalecom_compress_scatter.argtypes = [vp, vp, vp, vp, vp, vp, i32, vp, ctypes.c_uint32]
        L.scalecom_reduce_rows.restype = ctypes.c_int
        L.scalecom_reduce_rows.argtypes = [vp, vp, i32, vp, vp, vp, vp, ctypes.c_uint32]
        L.scalecom_enable_peer_access.restype = ctypes.c_int
        L.scalecom_enable_peer_access.argtypes = [vp, i32]
        L.scalecom_strerror.restype = ctypes.c_char_p
        L.scalecom_strerror.argtypes = [ctypes.c_int]
        _lib = L
    return _lib


def strerror(code: int) -> str:
    return lib().scalecom_strerror(int(code)).decode()


def _check(rc: int, where: str) -> None:
    if rc != OK:
        raise ScaleComError(rc, where)


# ---- raw mirrors of the C entry points (integers in, return codes out) -------------------------
def scalecom_create(d: int, n: int, k: int, beta: float, lr: float) -> Tuple[int, Optional[int]]:
    h = ctypes.c_void_p()
    rc = lib().scalecom_create(ctypes.byref(h), int(d), int(n), int(k), float(beta), float(lr))
    return rc, h.value


def _ptr_array(ptrs: Sequence[int]):
    return (ctypes.c_void_p * len(ptrs))(*ptrs)


def scalecom_step(handle: int, grads: Sequence[int], mem: Sequence[int], weights: Optional[int], t: int,
                  out_idx: int, out_val: int) -> int:
    ga, ma = _ptr_array(grads), _ptr_array(mem)
    return lib().scalecom_step(handle, ctypes.cast(ga, ctypes.c_void_p), ctypes.cast(ma, ctypes.c_void_p),
                               weights, int(t), out_idx, out_val)


def scalecom_step_host(handle: int, host_grads: Sequence[int], mem: Sequence[int], weights: Optional[int], t: int,
                       host_idx: int, host_val: int) -> int:
    ga, ma = _ptr_array(host_grads), _ptr_array(mem)
    return lib().scalecom_step_host(handle, ctypes.cast(ga, ctypes.c_void_p), ctypes.cast(ma, ctypes.c_void_p),
                                    weights, int(t), host_idx, host_val)


def scalecom_destroy(handle: Optional[int]) -> None:
    lib().scalecom_destroy(handle)


def scalecom_topk_static(g: int, m: int, d: int, k: int, out_idx: int, dev_status: Optional[int],
                         stream: Optional[int]) -> int:
    """Raw mirror of the allocation-free selection entry point (device addresses as integers)."""
    return lib().scalecom_topk_static(g, m, int(d), int(k), out_idx, dev_status, stream)


# ---- tensor-level convenience wrapper ------------------------------------------------------------
def _dev_f32(t: torch.Tensor, numel: int, name: str) -> int:
    if not (isinstance(t, torch.Tensor) and t.is_cuda and t.dtype == torch.float32 and t.is_contiguous()
            and t.numel() == numel):
        raise TypeError("%s must be a contiguous CUDA float32 tensor of %d elements" % (name, numel))
    return t.data_ptr()


def _dev_i32(t: torch.Tensor, numel: int, name: str) -> int:
    if not (isinstance(t, torch.Tensor) and t.is_cuda and t.dtype == torch.int32 and t.is_contiguous()
            and t.numel() == numel):
        raise TypeError("%s must be a contiguous CUDA int32 tensor of %d elements" % (name, numel))
    return t.data_ptr()


class Context:
    """One scalecom handle.  State (memories, weights, t) stays with the caller."""

    def __init__(self, d: int, n: int, k: int, beta: float, lr: float, stream: Optional[torch.cuda.Stream] = None):
        self.d, self.n, self.k, self.beta, self.lr = int(d), int(n), int(k), float(beta), float(lr)
        rc, h = scalecom_create(d, n, k, beta, lr)
        _check(rc, "scalecom_create")
        self._h = h
        self._gathered = None
        if stream is not None:
            self.set_stream(stream)

    def close(self) -> None:
        if getattr(self, "_h", None):
            h, self._h = self._h, None
            if _lib is not None:                 # at interpreter exit the module globals may already be gone
                _lib.scalecom_destroy(h)

    __del__ = close

    def __enter__(self):
        return self

    def __exit__(self, *exc):
        self.close()

    def set_stream(self, stream: Optional[torch.cuda.Stream]) -> None:
        _check(lib().scalecom_set_stream(self._h, stream.cuda_stream if stream is not None else None),
               "scalecom_set_stream")

    def set_gathered(self, buf: Optional[torch.Tensor]) -> None:
        ptr = None if buf is None else _dev_f32(buf, self.n * self.k, "gathered")
        _check(lib().scalecom_set_gathered(self._h, ptr), "scalecom_set_gathered")
        self._gathered = buf

    def enable_peer_access(self, peer_device: int) -> None:
        """Let this handle's device store into (and load from) memory of another device of the process."""
        _check(lib().scalecom_enable_peer_access(self._h, int(peer_device)), "scalecom_enable_peer_access")

    def set_option(self, option: int, value: int) -> None:
        _check(lib().scalecom_set_option(self._h, option, int(value)), "scalecom_set_option")

    def query(self, item: int) -> int:
        out = ctypes.c_int64()
        _check(lib().scalecom_query(self._h, item, ctypes.byref(out)), "scalecom_query")
        return out.value

    def status(self) -> int:
        return lib().scalecom_status(self._h)

    def reset(self) -> None:
        _check(lib().scalecom_reset(self._h), "scalecom_reset")

    def kernel_ms(self) -> Tuple[List[float], int]:
        """(summed kernel milliseconds [selection, learner pass, separate update], steps summed)."""
        ms = (ctypes.c_float * 3)()
        ns = ctypes.c_int32()
        _check(lib().scalecom_kernel_ms(self._h, ms, ctypes.byref(ns)), "scalecom_kernel_ms")
        return list(ms), ns.value

    def kernel_span_ms(self) -> Tuple[List[float], int]:
        """(summed in-kernel milliseconds [selection, learner pass], steps summed)."""
        ms = (ctypes.c_float * 2)()
        ns = ctypes.c_int32()
        _check(lib().scalecom_kernel_span_ms(self._h, ms, ctypes.byref(ns)), "scalecom_kernel_span_ms")
        return list(ms), ns.value

    def set_layers(self, sizes: Optional[Sequence[int]], keep: Optional[Sequence[int]] = None) -> None:
        """Per-layer rates of the chunk-wise selector; None goes back to one rate for the whole vector."""
        if sizes is None:
            _check(lib().scalecom_set_layers(self._h, 0, None, None), "scalecom_set_layers")
            return
        if keep is None or len(keep) != len(sizes):
            raise ValueError("sizes and keep must have the same length")
        sz = (ctypes.c_int64 * len(sizes))(*[int(x) for x in sizes])
        kp = (ctypes.c_int64 * len(keep))(*[int(x) for x in keep])
        _check(lib().scalecom_set_layers(self._h, len(sizes), ctypes.cast(sz, ctypes.c_void_p),
                                         ctypes.cast(kp, ctypes.c_void_p)), "scalecom_set_layers")

    def _idx(self, idx: torch.Tensor) -> int:
        if not (idx.is_cuda and idx.dtype == torch.int32 and idx.is_contiguous() and idx.numel() == self.k):
            raise TypeError("idx must be a contiguous CUDA int32 tensor of k elements")
        return idx.data_ptr()

    def select(self, g: torch.Tensor, m: torch.Tensor, out_idx: torch.Tensor) -> None:
        _check(lib().scalecom_select(self._h, _dev_f32(g, self.d, "g"), _dev_f32(m, self.d, "m"), self._idx(out_idx)),
               "scalecom_select")

    def compress(self, g: torch.Tensor, m: torch.Tensor, idx: Optional[torch.Tensor], out_gathered: torch.Tensor) -> None:
        """idx None: the list this handle's select() has just produced."""
        _check(lib().scalecom_compress(self._h, _dev_f32(g, self.d, "g"), _dev_f32(m, self.d, "m"),
                                       None if idx is None else self._idx(idx),
                                       _dev_f32(out_gathered, self.k, "out_gathered")), "scalecom_compress")

    def compress_scatter(self, g: torch.Tensor, m: torch.Tensor, idx: Optional[torch.Tensor], out_gathered: torch.Tensor,
                         dst: Sequence[torch.Tensor], flags: Optional[Sequence[torch.Tensor]] = None, tag: int = 0) -> None:
        """compress, with the kept values also stored into every tensor of dst (fp32[k] each, peers' memory allowed);
        with flags (one int32 word per destination) and tag != 0 the kernel stores tag there when it is through."""
        ptrs = _ptr_array([_dev_f32(t, self.k, "dst[%d]" % i) for i, t in enumerate(dst)])
        fptrs = None
        if flags is not None:
            if len(flags) != len(dst):
                raise ValueError("one flag word per destination")
            fptrs = ctypes.cast(_ptr_array([_dev_i32(f, 1, "flags[%d]" % i) for i, f in enumerate(flags)]), ctypes.c_void_p)
        _check(lib().scalecom_compress_scatter(self._h, _dev_f32(g, self.d, "g"), _dev_f32(m, self.d, "m"),
                                               None if idx is None else self._idx(idx),
                                               _dev_f32(out_gathered, self.k, "out_gathered"),
                                               ctypes.cast(ptrs, ctypes.c_void_p), len(dst), fptrs, int(tag)),
               "scalecom_compress_scatter")

    def reduce_rows(self, rows: torch.Tensor, out_val: torch.Tensor, idx: Optional[torch.Tensor] = None,
                    weights: Optional[torch.Tensor] = None, wait_flags: Optional[torch.Tensor] = None, tag: int = 0) -> None:
        """out_val = mean of the rows in row order; with idx and weights also weights[idx] -= lr * out_val; with
        wait_flags (int32[n_rows]) and tag the kernel reads row i only once wait_flags[i] == tag."""
        n_rows = max(1, rows.numel() // self.k)
        _check(lib().scalecom_reduce_rows(self._h, _dev_f32(rows, n_rows * self.k, "rows"), n_rows,
                                          _dev_f32(out_val, self.k, "out_val"),
                                          None if idx is None else self._idx(idx),
                                          None if weights is None else _dev_f32(weights, self.d, "weights"),
                                          None if wait_flags is None else _dev_i32(wait_flags, n_rows, "wait_flags"),
                                          int(tag)), "scalecom_reduce_rows")

    def overlap(self, grads: Sequence[torch.Tensor], mem: Sequence[torch.Tensor], t: int) -> int:
        """Eq. 5's d between the leader's top-k set and the true top-k set (synchronous)."""
        gp = _ptr_array([_dev_f32(g, self.d, "grads[%d]" % i) for i, g in enumerate(grads)])
        mp = _ptr_array([_dev_f32(m, self.d, "mem[%d]" % i) for i, m in enumerate(mem)])
        out = ctypes.c_int64()
        _check(lib().scalecom_overlap(self._h, ctypes.cast(gp, ctypes.c_void_p), ctypes.cast(mp, ctypes.c_void_p),
                                      int(t), ctypes.byref(out)), "scalecom_overlap")
        return out.value

    def cosine_distance(self, x: torch.Tensor, y: torch.Tensor) -> float:
        out = ctypes.c_double()
        _check(lib().scalecom_cosine_distance(self._h, _dev_f32(x, self.d, "x"), _dev_f32(y, self.d, "y"),
                                              ctypes.byref(out)), "scalecom_cosine_distance")
        return out.value

    def step(self, grads: Sequence[torch.Tensor], mem: Sequence[torch.Tensor], weights: Optional[torch.Tensor],
             t: int, out_idx: torch.Tensor, out_val: torch.Tensor) -> None:
        """scalecom_step on device tensors (asynchronous on the handle's stream)."""
        if len(grads) != self.n or len(mem) != self.n:
            raise ValueError("expected %d gradient and %d memory tensors" % (self.n, self.n))
        gp = [_dev_f32(g, self.d, "grads[%d]" % i) for i, g in enumerate(grads)]
        mp = [_dev_f32(m, self.d, "mem[%d]" % i) for i, m in enumerate(mem)]
        wp = None if weights is None else _dev_f32(weights, self.d, "weights")
        if not (out_idx.is_cuda and out_idx.dtype == torch.int32 and out_idx.is_contiguous() and out_idx.numel() == self.k):
            raise TypeError("out_idx must be a contiguous CUDA int32 tensor of k elements")
        _check(scalecom_step(self._h, gp, mp, wp, t, out_idx.data_ptr(), _dev_f32(out_val, self.k, "out_val")),
               "scalecom_step")

    def prepare_step(self, grad_batches: Sequence[Sequence[torch.Tensor]], mem: Sequence[torch.Tensor],
                     weights: Optional[torch.Tensor], out_idx: torch.Tensor, out_val: torch.Tensor):
        """Marshal the arguments of scalecom_step once for callers that step many times over the same buffers:
        returns call(b, t) = scalecom_step with gradient set grad_batches[b] at iteration t.  The tensors must stay
        alive and in place for as long as the callable is used."""
        if len(mem) != self.n or any(len(g) != self.n for g in grad_batches):
            raise ValueError("expected %d gradient and %d memory tensors" % (self.n, self.n))
        tables = [_ptr_array([_dev_f32(g, self.d, "grads[%d]" % i) for i, g in enumerate(gs)]) for gs in grad_batches]
        mtab = _ptr_array([_dev_f32(m, self.d, "mem[%d]" % i) for i, m in enumerate(mem)])
        gp = [ctypes.cast(tb, ctypes.c_void_p) for tb in tables]
        mp = ctypes.cast(mtab, ctypes.c_void_p)
        wp = None if weights is None else _dev_f32(weights, self.d, "weights")
        ip, vp = self._idx(out_idx), _dev_f32(out_val, self.k, "out_val")
        fn, h = lib().scalecom_step, self._h
        keep = (tables, mtab, grad_batches, mem, weights, out_idx, out_val)

        def call(b: int, t: int, _keep=keep) -> None:
            rc = fn(h, gp[b], mp, wp, t, ip, vp)
            if rc != OK:
                raise ScaleComError(rc, "scalecom_step")
        return call

    def step_host(self, host_grads: Sequence[torch.Tensor], mem: Sequence[torch.Tensor],
                  weights: Optional[torch.Tensor], t: int, host_idx: torch.Tensor, host_val: torch.Tensor) -> None:
        """scalecom_step_host: gradients and results in host tensors (synchronous)."""
        if len(host_grads) != self.n or len(mem) != self.n:
            raise ValueError("expected %d gradient and %d memory tensors" % (self.n, self.n))
        for i, g in enumerate(host_grads):
            if g.is_cuda or g.dtype != torch.float32 or not g.is_contiguous() or g.numel() != self.d:
                raise TypeError("host_grads[%d] must be a contiguous CPU float32 tensor of d elements" % i)
        if host_idx.is_cuda or host_idx.dtype != torch.int32 or host_idx.numel() != self.k or not host_idx.is_contiguous():
            raise TypeError("host_idx must be a contiguous CPU int32 tensor of k elements")
        if host_val.is_cuda or host_val.dtype != torch.float32 or host_val.numel() != self.k or not host_val.is_contiguous():
            raise TypeError("host_val must be a contiguous CPU float32 tensor of k elements")
        mp = [_dev_f32(m, self.d, "mem[%d]" % i) for i, m in enumerate(mem)]
        wp = None if weights is None else _dev_f32(weights, self.d, "weights")
        _check(scalecom_step_host(self._h, [g.data_ptr() for g in host_grads], mp, wp, t,
                                  host_idx.data_ptr(), host_val.data_ptr()), "scalecom_step_host")

    def apply_update(self, weights: torch.Tensor, idx: torch.Tensor, val: torch.Tensor, lr: float) -> None:
        k = idx.numel()
        if not (idx.is_cuda and idx.dtype == torch.int32 and idx.is_contiguous()):
            raise TypeError("idx must be a contiguous CUDA int32 tensor")
        _check(lib().scalecom_apply_update(self._h, _dev_f32(weights, self.d, "weights"), idx.data_ptr(),
                                           _dev_f32(val, k, "val"), k, float(lr)), "scalecom_apply_update")

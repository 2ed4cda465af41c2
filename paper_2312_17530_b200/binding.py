"""ctypes binding of the RS-DGC CUDA library (``include/rsdgc.h``).

Argument marshalling only: every step of the compression path runs in the library's
kernels.  PyTorch tensors supply device memory and the current CUDA stream.  There is no
CPU fallback: if the shared library is missing, :func:`lib` raises.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import List, Optional, Sequence, Tuple

_HERE = os.path.dirname(os.path.abspath(__file__))
# RSDGC_LIBRARY selects another build of the same library (e.g. the bounds-checked one)
LIB_PATH = os.environ.get("RSDGC_LIBRARY") or os.path.join(_HERE, "librsdgc_b200.so")

RSDGC_F32, RSDGC_BF16 = 0, 1
KEEP_AT_LEAST_ONE = 1
NO_BULK_COPY = 2
MOMENTUM = 4
PAYLOAD_BF16 = 8
NO_FUSED_TAIL = 16
STATUS_NONFINITE, STATUS_PAYLOAD_OVERFLOW, STATUS_TIMEOUT, STATUS_BOUNDS = 1, 2, 4, 8
OK, ERR_INVALID, ERR_ALIGNMENT, ERR_CAPACITY, ERR_CUDA, ERR_NOMEM = 0, -1, -2, -3, -4, -5

EXPORTS = [
    "rsdgc_plan_create", "rsdgc_plan_destroy", "rsdgc_plan_info", "rsdgc_plan_layer_info",
    "rsdgc_plan_payload_bound", "rsdgc_plan_worklist", "rsdgc_update_ratios", "rsdgc_compress",
    "rsdgc_compress_host", "rsdgc_decompress_accumulate", "rsdgc_get_status", "rsdgc_launch_count",
    "rsdgc_strerror", "rsdgc_last_cuda_error", "rsdgc_profile_enable", "rsdgc_profile_read",
    "rsdgc_update_ratios_noalloc", "rsdgc_compress_momentum", "rsdgc_plan_reserve_workers",
    "rsdgc_compress_workers", "rsdgc_decompress_assign", "rsdgc_payload_to_coo", "rsdgc_compress_workers_host",
    "rsdgc_selftest_bounded_wait", "rsdgc_plan_tail_slices",
]
NOALLOC_MAX_LAYERS = 64
N_COMPRESS_KERNELS = 5
COMPRESS_KERNELS = ("accumulate_nsi", "refine2", "refine3_count", "mark", "gather")


class LayerDesc(C.Structure):
    _fields_ = [("rows", C.c_int64), ("cols", C.c_int64), ("nh", C.c_int32), ("nw", C.c_int32)]


class Info(C.Structure):
    _fields_ = [("n_layers", C.c_int32), ("grad_dtype", C.c_int32), ("arena_elems", C.c_int64),
                ("total_elems", C.c_int64), ("total_tiles", C.c_int64), ("total_tiles_padded", C.c_int64),
                ("workspace_bytes", C.c_int64), ("max_slot", C.c_int32), ("reserved", C.c_int32)]


class LayerInfo(C.Structure):
    _fields_ = [("elem_offset", C.c_int64), ("tile_offset", C.c_int64), ("rows", C.c_int64),
                ("cols", C.c_int64), ("nh", C.c_int32), ("nw", C.c_int32), ("n_tiles", C.c_int64)]


class Status(C.Structure):
    _fields_ = [("flags", C.c_uint32), ("reserved", C.c_uint32), ("nonfinite", C.c_int64),
                ("idx_needed", C.c_int64), ("val_needed", C.c_int64)]


class RsdgcError(RuntimeError):
    def __init__(self, code: int, what: str):
        self.code = code
        msg = lib().rsdgc_strerror(code).decode()
        if code == ERR_CUDA:
            msg += " (cudaError %d)" % lib().rsdgc_last_cuda_error()
        super().__init__("%s: %s [%d]" % (what, msg, code))


_lib = None


def lib():
    """The loaded C library; raises if it has not been built (no fallback path exists)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError("CUDA library %s is missing: build it with "
                               "`python -m paper_2312_17530_b200.build`" % LIB_PATH)
        L = C.CDLL(LIB_PATH)
        vp, i32, i64, f32, u32 = C.c_void_p, C.c_int32, C.c_int64, C.c_float, C.c_uint32
        L.rsdgc_plan_create.argtypes = [C.POINTER(LayerDesc), i32, i32, f32, u32, i32, C.POINTER(vp)]
        L.rsdgc_plan_destroy.argtypes = [vp]
        L.rsdgc_plan_info.argtypes = [vp, C.POINTER(Info)]
        L.rsdgc_plan_layer_info.argtypes = [vp, i32, C.POINTER(LayerInfo)]
        L.rsdgc_plan_payload_bound.argtypes = [vp, f32, C.POINTER(i64), C.POINTER(i64)]
        L.rsdgc_plan_worklist.argtypes = [vp, vp, i64, vp, vp]
        L.rsdgc_plan_worklist.restype = i64
        L.rsdgc_update_ratios.argtypes = [vp, vp, f32, vp, vp]
        L.rsdgc_compress.argtypes = [vp, vp, vp, vp, vp, i64, vp, i64, vp, vp, vp, vp]
        L.rsdgc_compress_momentum.argtypes = [vp, vp, vp, f32, vp, vp, vp, i64, vp, i64, vp, vp, vp, vp]
        L.rsdgc_plan_reserve_workers.argtypes = [vp, i32]
        L.rsdgc_compress_workers.argtypes = [vp, i32, C.POINTER(vp), C.POINTER(vp), vp, C.POINTER(vp), i64,
                                             C.POINTER(vp), i64, C.POINTER(vp), vp, vp]
        L.rsdgc_compress_host.argtypes = [vp, vp, vp, vp, vp, vp, i64, vp, i64, vp, vp, vp, vp, vp,
                                          C.POINTER(i64), C.POINTER(i64), vp]
        pp = C.POINTER(vp)
        L.rsdgc_compress_workers_host.argtypes = [vp, i32, pp, pp, pp, vp, pp, i64, pp, i64, pp, vp, pp, pp, pp,
                                                  C.POINTER(i64), C.POINTER(i64), vp]
        L.rsdgc_decompress_accumulate.argtypes = [vp, i32, C.POINTER(vp), C.POINTER(vp), C.POINTER(vp), i64, i64, f32,
                                                  vp, vp]
        L.rsdgc_decompress_assign.argtypes = [vp, i32, C.POINTER(vp), C.POINTER(vp), C.POINTER(vp), i64, i64, f32, vp,
                                              vp]
        L.rsdgc_payload_to_coo.argtypes = [vp, vp, vp, vp, i64, vp]
        L.rsdgc_get_status.argtypes = [vp, vp, C.POINTER(Status)]
        L.rsdgc_profile_enable.argtypes = [vp, i32]
        L.rsdgc_profile_read.argtypes = [vp, C.POINTER(C.c_double), C.POINTER(i64)]
        L.rsdgc_update_ratios_noalloc.argtypes = [vp, C.POINTER(i64), C.POINTER(i64), i32, f32, vp, vp]
        L.rsdgc_selftest_bounded_wait.argtypes = [vp, i32, vp]
        L.rsdgc_plan_tail_slices.argtypes = [vp, vp, i64, vp]
        L.rsdgc_plan_tail_slices.restype = i64
        L.rsdgc_launch_count.argtypes = []
        L.rsdgc_launch_count.restype = i64
        L.rsdgc_strerror.argtypes = [C.c_int]
        L.rsdgc_strerror.restype = C.c_char_p
        L.rsdgc_last_cuda_error.argtypes = []
        for name in EXPORTS:
            fn = getattr(L, name)
            if fn.restype is C.c_int:  # default restype: all the int-returning entry points
                fn.restype = C.c_int
        _lib = L
    return _lib


def _check(code: int, what: str) -> None:
    if code != OK:
        raise RsdgcError(code, what)


def _ptr(t) -> Optional[int]:
    return None if t is None else t.data_ptr()


def _stream() -> int:
    import torch

    return torch.cuda.current_stream().cuda_stream


class Plan:
    """Owns an ``rsdgc_plan``.  ``layers``: sequence of (rows, cols, nh, nw).  ``device`` < 0
    gives a host-only plan (sizes and offsets only; usable without a GPU)."""

    def __init__(self, layers: Sequence[Tuple[int, int, int, int]], grad_dtype: int = RSDGC_F32,
                 alpha: float = 0.5, flags: int = KEEP_AT_LEAST_ONE, device: int = 0):
        arr = (LayerDesc * max(1, len(layers)))()
        for i, (r, c, nh, nw) in enumerate(layers):
            arr[i] = LayerDesc(int(r), int(c), int(nh), int(nw))
        h = C.c_void_p()
        self._h = None
        _check(lib().rsdgc_plan_create(arr, len(layers), grad_dtype, alpha, flags, device, C.byref(h)),
               "rsdgc_plan_create")
        self._h = h
        self.device = device
        self.n_layers = len(layers)
        self.grad_dtype = grad_dtype
        self.flags = int(flags)
        info = Info()
        _check(lib().rsdgc_plan_info(self._h, C.byref(info)), "rsdgc_plan_info")
        self.info = info
        self.layers: List[LayerInfo] = []
        for l in range(self.n_layers):
            li = LayerInfo()
            _check(lib().rsdgc_plan_layer_info(self._h, l, C.byref(li)), "rsdgc_plan_layer_info")
            self.layers.append(li)

    def close(self) -> None:
        if self._h is not None:
            lib().rsdgc_plan_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # ---- sizes --------------------------------------------------------------------------
    def payload_bound(self, max_ratio: float) -> Tuple[int, int]:
        a, b = C.c_int64(), C.c_int64()
        _check(lib().rsdgc_plan_payload_bound(self._h, max_ratio, C.byref(a), C.byref(b)),
               "rsdgc_plan_payload_bound")
        return a.value, b.value

    def worklist(self):
        """(items [n,9] int32: layer, tr0, ntr, tc0, ntc, kernel, cta, shared-memory pitch, item
        flags (1 contiguous, 2 128-bit accesses, 4 bulk copies, 8 no clipped tile); grids [2];
        n_flush [L])."""
        import numpy as np

        n = lib().rsdgc_plan_worklist(self._h, None, 0, None, None)
        items = np.zeros((n, 9), dtype=np.int32)
        grids = np.zeros(2, dtype=np.int32)
        nf = np.zeros(self.n_layers, dtype=np.int32)
        lib().rsdgc_plan_worklist(self._h, items.ctypes.data, n, grids.ctypes.data, nf.ctypes.data)
        return items, grids, nf

    def tail_slices(self):
        """(slices [n,6] int32: layer, first tile, tiles, CTAs of the layer, rank, leader rank; info [3]:
        cluster-variant CTAs, one-CTA layers, clusters) of the single-kernel selection + pack; n = 0 when
        the plan takes the chained kernels."""
        import numpy as np

        n = lib().rsdgc_plan_tail_slices(self._h, None, 0, None)
        sl = np.zeros((max(n, 0), 6), dtype=np.int32)
        info = np.zeros(3, dtype=np.int32)
        lib().rsdgc_plan_tail_slices(self._h, sl.ctypes.data, n, info.ctypes.data)
        return sl, info

    # ---- device calls (torch tensors on the plan's device) -------------------------------
    def update_ratios(self, weights, global_keep: float, ratios) -> None:
        _check(lib().rsdgc_update_ratios(self._h, _ptr(weights), global_keep, _ptr(ratios), _stream()),
               "rsdgc_update_ratios")

    def compress(self, grads, residual, ratios, idx, val, counts, nsi=None, workspace=None) -> None:
        _check(lib().rsdgc_compress(self._h, _ptr(grads), _ptr(residual), _ptr(ratios), _ptr(idx), idx.numel(),
                                    _ptr(val), val.numel(), _ptr(counts), _ptr(nsi), _ptr(workspace), _stream()),
               "rsdgc_compress")

    def compress_momentum(self, grads, velocity, momentum: float, residual, ratios, idx, val, counts, nsi=None,
                          workspace=None) -> None:
        _check(lib().rsdgc_compress_momentum(self._h, _ptr(grads), _ptr(velocity), momentum, _ptr(residual),
                                             _ptr(ratios), _ptr(idx), idx.numel(), _ptr(val), val.numel(),
                                             _ptr(counts), _ptr(nsi), _ptr(workspace), _stream()),
               "rsdgc_compress_momentum")

    def reserve_workers(self, n_workers: int) -> None:
        _check(lib().rsdgc_plan_reserve_workers(self._h, int(n_workers)), "rsdgc_plan_reserve_workers")

    def compress_workers(self, grads, residuals, ratios, idx, val, counts, workspace) -> None:
        """One call for several workers: ``grads``, ``residuals``, ``idx``, ``val``, ``counts`` are
        sequences with one device tensor per worker; ``workspace`` holds n_workers * workspace_bytes."""
        n = len(grads)
        A = C.c_void_p * max(1, n)
        ga, ra, ia, va, ca = A(), A(), A(), A(), A()
        for w in range(n):
            ga[w], ra[w], ca[w] = grads[w].data_ptr(), residuals[w].data_ptr(), counts[w].data_ptr()
            ia[w], va[w] = idx[w].data_ptr(), val[w].data_ptr()
        _check(lib().rsdgc_compress_workers(self._h, n, ga, ra, _ptr(ratios), ia, min(t.numel() for t in idx), va,
                                            min(t.numel() for t in val), ca, _ptr(workspace), _stream()),
               "rsdgc_compress_workers")

    def compress_host(self, grads_host, grads_dev, residual, ratios, idx, val, counts, workspace,
                      idx_host, val_host, counts_host) -> Tuple[int, int]:
        ni, nv = C.c_int64(), C.c_int64()
        _check(lib().rsdgc_compress_host(self._h, _ptr(grads_host), _ptr(grads_dev), _ptr(residual), _ptr(ratios),
                                         _ptr(idx), idx.numel(), _ptr(val), val.numel(), _ptr(counts),
                                         _ptr(workspace), _ptr(idx_host), _ptr(val_host), _ptr(counts_host),
                                         C.byref(ni), C.byref(nv), _stream()), "rsdgc_compress_host")
        return ni.value, nv.value

    def compress_workers_host(self, grads_host, staging, residuals, ratios, idx, val, counts, workspace,
                              idx_host, val_host, counts_host):
        """rsdgc_compress_workers_host(): per-worker sequences of host gradients / host payload buffers and
        device residuals / payload buffers, ``staging`` = two device arenas.  Returns the per-worker
        (idx_used, val_used) lists."""
        n = len(grads_host)
        A = C.c_void_p * max(1, n)
        gh, rd, ia, va, ca, ih, vh, ch = A(), A(), A(), A(), A(), A(), A(), A()
        for w in range(n):
            gh[w], rd[w], ca[w] = grads_host[w].data_ptr(), residuals[w].data_ptr(), counts[w].data_ptr()
            ia[w], va[w] = idx[w].data_ptr(), val[w].data_ptr()
            ih[w], vh[w], ch[w] = idx_host[w].data_ptr(), val_host[w].data_ptr(), counts_host[w].data_ptr()
        st = (C.c_void_p * 2)(staging[0].data_ptr(), staging[1].data_ptr())
        ni, nv = (C.c_int64 * max(1, n))(), (C.c_int64 * max(1, n))()
        _check(lib().rsdgc_compress_workers_host(
            self._h, n, gh, st, rd, _ptr(ratios), ia, min(t.numel() for t in idx), va, min(t.numel() for t in val),
            ca, _ptr(workspace), ih, vh, ch, ni, nv, _stream()), "rsdgc_compress_workers_host")
        return list(ni)[:n], list(nv)[:n]

    def decompress_accumulate(self, payloads, dense, scale: float = 1.0, assign: bool = False) -> None:
        """``payloads``: sequence of (idx, val, counts) device tensors, one per worker.  ``assign``:
        rsdgc_decompress_assign() (the arena is zero-filled by the same launch)."""
        n = len(payloads)
        A = C.c_void_p * max(1, n)
        ia, va, ca = A(), A(), A()
        for w, (i, v, c) in enumerate(payloads):
            ia[w], va[w], ca[w] = i.data_ptr(), v.data_ptr(), c.data_ptr()
        fn = lib().rsdgc_decompress_assign if assign else lib().rsdgc_decompress_accumulate
        idx_cap = min((i.numel() for i, _, _ in payloads), default=0)
        val_cap = min((v.numel() for _, v, _ in payloads), default=0)
        _check(fn(self._h, n, ia, va, ca, idx_cap, val_cap, scale, _ptr(dense), _stream()),
               "rsdgc_decompress_assign" if assign else "rsdgc_decompress_accumulate")

    def decompress_assign(self, payloads, dense, scale: float = 1.0) -> None:
        self.decompress_accumulate(payloads, dense, scale, assign=True)

    def payload_to_coo(self, idx, counts, coo_index) -> None:
        """Arena position (int64) of every payload value, -1 for padding slots."""
        _check(lib().rsdgc_payload_to_coo(self._h, _ptr(idx), _ptr(counts), _ptr(coo_index), coo_index.numel(),
                                          _stream()), "rsdgc_payload_to_coo")

    def profile_enable(self, level: int) -> None:
        """0 off; 1 events around the first pass only; 2 events around every kernel."""
        _check(lib().rsdgc_profile_enable(self._h, int(level)), "rsdgc_profile_enable")

    def profile_read(self):
        """(milliseconds summed per compress kernel, number of compress calls recorded)."""
        ms = (C.c_double * N_COMPRESS_KERNELS)()
        n = C.c_int64()
        _check(lib().rsdgc_profile_read(self._h, ms, C.byref(n)), "rsdgc_profile_read")
        return list(ms), n.value

    def selftest_bounded_wait(self, polls: int = 256) -> None:
        """Diagnostic: a bounded on-chip wait that is certain to give up; sets STATUS_TIMEOUT."""
        _check(lib().rsdgc_selftest_bounded_wait(self._h, int(polls), _stream()), "rsdgc_selftest_bounded_wait")

    def status(self) -> Status:
        st = Status()
        _check(lib().rsdgc_get_status(self._h, _stream(), C.byref(st)), "rsdgc_get_status")
        return st


def update_ratios_noalloc(weights, layer_offsets: Sequence[int], layer_sizes: Sequence[int], global_keep: float,
                          ratios) -> None:
    """rsdgc_update_ratios_noalloc(): the ratio rule without a plan and without any allocation
    (scratch is a fixed array inside the library; at most NOALLOC_MAX_LAYERS layers)."""
    n = len(layer_offsets)
    offs = (C.c_int64 * max(1, n))(*[int(x) for x in layer_offsets])
    sizes = (C.c_int64 * max(1, n))(*[int(x) for x in layer_sizes])
    _check(lib().rsdgc_update_ratios_noalloc(_ptr(weights), offs, sizes, n, global_keep, _ptr(ratios), _stream()),
           "rsdgc_update_ratios_noalloc")


def launch_count() -> int:
    return int(lib().rsdgc_launch_count())

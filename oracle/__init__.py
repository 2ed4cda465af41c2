"""RS-DGC reference oracle: Python driver around ``rsdgc_oracle.c``.

TEST INFRASTRUCTURE ONLY.  Imported by the tests, by the smoke check and by the
benchmark's CPU-baseline leg; the product package never imports it.  All of the
method's arithmetic lives in the C file (plain loops, one thread); this module only
compiles it with gcc, marshals NumPy arrays and strings the per-layer steps together
in the order of Algorithm 1 of the paper (arxiv 2312.17530):

    accumulate (Eq. 12) -> NSI per neighborhood (Eq. 8-10) -> keep count (Eq. 11)
    -> per-layer ranking and top-k (Algorithm 1) -> payload + accumulator update
    (Sec. III-C, Eq. 12) ; aggregation of several workers (Eq. 12 / Eq. 2 Sync) ;
    layer-wise ratios from the weights (Eq. 3-5).

Layers are passed as ``(rows, cols, nh, nw)`` tuples plus one flat float32 array per
layer (no padding, no arena: the memory layout of the CUDA library is not known here).
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from dataclasses import dataclass, field
from typing import List, Optional, Sequence, Tuple

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "rsdgc_oracle.c")
_OUT_DIR = os.path.join(_HERE, "_build")
_LIB_PATH = os.path.join(_OUT_DIR, "librsdgc_oracle.so")

LayerShape = Tuple[int, int, int, int]  # rows, cols, nh, nw


def build(force: bool = False) -> str:
    """Compile the C oracle (gcc, -O2, no fused multiply-add) if it is stale."""
    os.makedirs(_OUT_DIR, exist_ok=True)
    stale = force or not os.path.exists(_LIB_PATH) or os.path.getmtime(_LIB_PATH) < os.path.getmtime(_SRC)
    if stale:
        tmp = _LIB_PATH + ".tmp.%d" % os.getpid()
        cmd = ["gcc", "-O2", "-std=c11", "-ffp-contract=off", "-fno-fast-math", "-fPIC", "-shared",
               "-Wall", "-Wextra", "-o", tmp, _SRC, "-lm"]
        subprocess.run(cmd, check=True)
        os.replace(tmp, _LIB_PATH)
    return _LIB_PATH


_lib = None


def lib():
    global _lib
    if _lib is None:
        L = C.CDLL(build())
        i64, i32, f32 = C.c_int64, C.c_int32, C.c_float
        p = C.c_void_p
        L.rsdgc_oracle_tile_count.restype = i64
        L.rsdgc_oracle_tile_count.argtypes = [i64, i64, i32, i32]
        L.rsdgc_oracle_accumulate_f32.restype = None
        L.rsdgc_oracle_accumulate_f32.argtypes = [p, p, p, i64]
        L.rsdgc_oracle_accumulate_bf16.restype = None
        L.rsdgc_oracle_accumulate_bf16.argtypes = [p, p, p, i64]
        L.rsdgc_oracle_accumulate_momentum_f32.restype = None
        L.rsdgc_oracle_accumulate_momentum_f32.argtypes = [p, p, p, p, f32, i64]
        L.rsdgc_oracle_accumulate_momentum_bf16.restype = None
        L.rsdgc_oracle_accumulate_momentum_bf16.argtypes = [p, p, p, p, f32, i64]
        L.rsdgc_oracle_nsi.restype = i64
        L.rsdgc_oracle_nsi.argtypes = [p, i64, i64, i32, i32, f32, p, p]
        L.rsdgc_oracle_keep_count.restype = i64
        L.rsdgc_oracle_keep_count.argtypes = [i64, f32, i32]
        L.rsdgc_oracle_select.restype = f32
        L.rsdgc_oracle_select.argtypes = [p, i64, i64, p]
        L.rsdgc_oracle_pack.restype = None
        L.rsdgc_oracle_pack.argtypes = [p, i64, i64, i32, i32, p, i64, p, p]
        L.rsdgc_oracle_pack_bf16.restype = None
        L.rsdgc_oracle_pack_bf16.argtypes = [p, i64, i64, i32, i32, p, i64, p, p]
        L.rsdgc_oracle_f32_to_bf16.restype = C.c_uint16
        L.rsdgc_oracle_f32_to_bf16.argtypes = [f32]
        L.rsdgc_oracle_decompress.restype = None
        L.rsdgc_oracle_decompress.argtypes = [p, i64, i64, i32, i32, p, p, i64, f32]
        L.rsdgc_oracle_update_ratios.restype = i64
        L.rsdgc_oracle_update_ratios.argtypes = [p, p, i32, f32, p, p]
        _lib = L
    return _lib


def _ptr(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


def _f32(a) -> np.ndarray:
    return np.ascontiguousarray(a, dtype=np.float32).reshape(-1)


# ---------------------------------------------------------------------------------------------
# single steps
# ---------------------------------------------------------------------------------------------

def tile_count(rows: int, cols: int, nh: int, nw: int) -> int:
    return int(lib().rsdgc_oracle_tile_count(rows, cols, nh, nw))


def accumulate(g: np.ndarray, r: np.ndarray) -> np.ndarray:
    """v = g + r (Eq. 12).  ``g`` is float32, or uint16 holding bfloat16 bit patterns."""
    r = _f32(r)
    v = np.empty_like(r)
    if g.dtype == np.uint16:
        g = np.ascontiguousarray(g).reshape(-1)
        assert g.size == r.size
        lib().rsdgc_oracle_accumulate_bf16(_ptr(g), _ptr(r), _ptr(v), r.size)
    else:
        g = _f32(g)
        assert g.size == r.size
        lib().rsdgc_oracle_accumulate_f32(_ptr(g), _ptr(r), _ptr(v), r.size)
    return v


def accumulate_momentum(g: np.ndarray, u: np.ndarray, r: np.ndarray, m: float):
    """(u_new, v) with u_new = m*u + g and v = r + u_new (Eq. 12, first and second line)."""
    r = _f32(r)
    u_new = _f32(u).copy()
    v = np.empty_like(r)
    if g.dtype == np.uint16:  # bfloat16 bit patterns
        g = np.ascontiguousarray(g).reshape(-1)
        fn = lib().rsdgc_oracle_accumulate_momentum_bf16
    else:
        g = _f32(g)
        fn = lib().rsdgc_oracle_accumulate_momentum_f32
    assert g.size == r.size == u_new.size
    fn(_ptr(g), _ptr(u_new), _ptr(r), _ptr(v), float(np.float32(m)), r.size)
    return u_new, v


def nsi(v: np.ndarray, shape: LayerShape, alpha: float):
    """(nsi_ref float64 [K], nsi_f32 float32 [K], n_nonfinite) for one layer (Eq. 8-10)."""
    rows, cols, nh, nw = shape
    v = _f32(v)
    assert v.size == rows * cols
    K = tile_count(rows, cols, nh, nw)
    ref = np.empty(K, dtype=np.float64)
    f32 = np.empty(K, dtype=np.float32)
    nonfinite = lib().rsdgc_oracle_nsi(_ptr(v), rows, cols, nh, nw, float(alpha), _ptr(ref), _ptr(f32))
    return ref, f32, int(nonfinite)


def keep_count(K: int, ratio: float, clamp_min1: bool = True) -> int:
    """k = ceil(K * ratio) within [0, K] (Eq. 11); at least 1 when ``clamp_min1``."""
    return int(lib().rsdgc_oracle_keep_count(K, float(np.float32(ratio)), 1 if clamp_min1 else 0))


def select(nsi_f32: np.ndarray, k: int):
    """Top-k tiles by indicator, ties to the lower index; ascending indices + threshold."""
    nsi_f32 = _f32(nsi_f32)
    sel = np.empty(max(k, 0), dtype=np.int32)
    thr = lib().rsdgc_oracle_select(_ptr(nsi_f32), nsi_f32.size, k, _ptr(sel))
    return sel, float(thr)


def pack(v: np.ndarray, shape: LayerShape, sel: np.ndarray):
    """(idx, val, new_residual) for one layer given the chosen tiles (ascending)."""
    rows, cols, nh, nw = shape
    res = _f32(v).copy()
    sel = np.ascontiguousarray(sel, dtype=np.int32)
    k = sel.size
    idx = np.empty(k, dtype=np.int32)
    val = np.empty(k * nh * nw, dtype=np.float32)
    lib().rsdgc_oracle_pack(_ptr(res), rows, cols, nh, nw, _ptr(sel), k, _ptr(idx), _ptr(val))
    return idx, val, res


def f32_to_bf16(x: float) -> int:
    """Bit pattern of the bfloat16 nearest to the binary32 ``x`` (ties to even)."""
    return int(lib().rsdgc_oracle_f32_to_bf16(float(np.float32(x))))


def pack_bf16(v: np.ndarray, shape: LayerShape, sel: np.ndarray):
    """(idx, val_bits uint16, new_residual): the payload with bfloat16 values; the rounding
    error of every sent value stays in the accumulator."""
    rows, cols, nh, nw = shape
    res = _f32(v).copy()
    sel = np.ascontiguousarray(sel, dtype=np.int32)
    k = sel.size
    idx = np.empty(k, dtype=np.int32)
    bits = np.empty(k * nh * nw, dtype=np.uint16)
    lib().rsdgc_oracle_pack_bf16(_ptr(res), rows, cols, nh, nw, _ptr(sel), k, _ptr(idx), _ptr(bits))
    return idx, bits, res


def decompress_into(dense: np.ndarray, shape: LayerShape, idx: np.ndarray, val: np.ndarray, scale: float) -> None:
    """dense += scale * payload for one layer and one worker, in place (Eq. 12, Eq. 2)."""
    rows, cols, nh, nw = shape
    assert dense.dtype == np.float32 and dense.flags.c_contiguous and dense.size == rows * cols
    idx = np.ascontiguousarray(idx, dtype=np.int32)
    val = _f32(val)
    assert val.size == idx.size * nh * nw
    lib().rsdgc_oracle_decompress(_ptr(dense), rows, cols, nh, nw, _ptr(idx), _ptr(val), idx.size, float(scale))


def update_ratios(weights: Sequence[np.ndarray], rho: float):
    """(ratios float32 [L], survivors int64 [L], n_keep) from the weights (Eq. 3-5)."""
    sizes = np.array([int(np.asarray(w).size) for w in weights], dtype=np.int64)
    flat = np.concatenate([_f32(w) for w in weights]) if len(weights) else np.zeros(0, np.float32)
    ratios = np.empty(len(weights), dtype=np.float32)
    surv = np.empty(len(weights), dtype=np.int64)
    n_keep = lib().rsdgc_oracle_update_ratios(_ptr(flat), _ptr(sizes), len(weights), float(np.float32(rho)),
                                              _ptr(ratios), _ptr(surv))
    return ratios, surv, int(n_keep)


# ---------------------------------------------------------------------------------------------
# whole steps over a list of layers
# ---------------------------------------------------------------------------------------------

@dataclass
class LayerResult:
    v: np.ndarray            # accumulated gradient g + r (Eq. 12)
    nsi_ref: np.ndarray      # float64 [K]
    nsi_f32: np.ndarray      # float32 [K]
    k: int                   # neighborhoods kept (Eq. 11)
    sel: np.ndarray          # int32 [k] ascending
    threshold: float         # indicator of the last neighborhood taken
    idx: np.ndarray          # int32 [k]
    val: np.ndarray          # float32 [k * nh * nw]
    residual: np.ndarray     # float32 [rows * cols], new accumulator
    nonfinite: int = 0
    velocity: Optional[np.ndarray] = None  # new u when momentum correction is on
    val_bf16: Optional[np.ndarray] = None  # uint16 [k * nh * nw] when the payload values are bfloat16


@dataclass
class CompressResult:
    layers: List[LayerResult] = field(default_factory=list)

    @property
    def counts(self) -> np.ndarray:
        return np.array([lr.k for lr in self.layers], dtype=np.int32)


def compress_layer(g: np.ndarray, r: np.ndarray, shape: LayerShape, ratio: float, alpha: float,
                   clamp_min1: bool = True, forced_sel: Optional[np.ndarray] = None,
                   velocity: Optional[np.ndarray] = None, momentum: float = 0.0,
                   payload_bf16: bool = False) -> LayerResult:
    """One layer of the per-iteration half of Algorithm 1.

    ``forced_sel`` replaces the ranking step by a given ascending tile set (used by the
    parity tests when two sets differ only inside the tolerance band at the threshold)."""
    u_new = None
    if velocity is None:
        v = accumulate(g, r)
    else:
        u_new, v = accumulate_momentum(g, velocity, r, momentum)
    ref, f32, nonfinite = nsi(v, shape, alpha)
    k = keep_count(f32.size, ratio, clamp_min1)
    if forced_sel is None:
        sel, thr = select(f32, k)
    else:
        sel = np.ascontiguousarray(forced_sel, dtype=np.int32)
        thr = float(f32[sel].min()) if sel.size else 0.0
    bits = None
    if payload_bf16:
        idx, bits, res = pack_bf16(v, shape, sel)
        val = (bits.astype(np.uint32) << 16).view(np.float32)  # the values the receiver sees
    else:
        idx, val, res = pack(v, shape, sel)
    return LayerResult(v=v, nsi_ref=ref, nsi_f32=f32, k=k, sel=sel, threshold=thr, idx=idx, val=val,
                       residual=res, nonfinite=nonfinite, velocity=u_new, val_bf16=bits)


def compress(shapes: Sequence[LayerShape], grads: Sequence[np.ndarray], residuals: Sequence[np.ndarray],
             ratios: Sequence[float], alpha: float, clamp_min1: bool = True) -> CompressResult:
    out = CompressResult()
    for shape, g, r, rho in zip(shapes, grads, residuals, ratios):
        out.layers.append(compress_layer(g, r, shape, rho, alpha, clamp_min1))
    return out


def decompress_accumulate(shapes: Sequence[LayerShape], dense: Sequence[np.ndarray],
                          payloads: Sequence[CompressResult], scale: float = 1.0) -> None:
    """dense_l += scale * sum over workers (in the given order) of their payloads."""
    for w in payloads:
        for shape, d, lr in zip(shapes, dense, w.layers):
            decompress_into(d, shape, lr.idx, lr.val, scale)


def decompress_assign(shapes: Sequence[LayerShape], dense: Sequence[np.ndarray],
                      payloads: Sequence[CompressResult], scale: float = 1.0) -> None:
    """Eq. 12 third line as an assignment: dense_l = +0, then the workers are added in order."""
    for d in dense:
        d[...] = np.float32(0.0)
    decompress_accumulate(shapes, dense, payloads, scale)


def payload_to_coo(shape: LayerShape, idx: np.ndarray, elem_offset: int = 0) -> np.ndarray:
    """Position (int64) of every payload value of one layer in a flat buffer in which the layer
    starts at ``elem_offset``: value s*nh*nw + a*nw + b of tile idx[s] = (tr, tc) is element
    (tr*nh + a, tc*nw + b) of the row-major layer (Sec. III-C: the neighborhood index stands
    for all the positions of the neighborhood); -1 where that element lies outside the layer."""
    rows, cols, nh, nw = shape
    TC = -(-cols // nw)
    out = np.empty(idx.size * nh * nw, dtype=np.int64)
    n = 0
    for t in np.asarray(idx, dtype=np.int64):
        tr, tc = divmod(int(t), TC)
        for a in range(nh):
            for b in range(nw):
                i, j = tr * nh + a, tc * nw + b
                out[n] = elem_offset + i * cols + j if (i < rows and j < cols) else -1
                n += 1
    return out

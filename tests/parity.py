"""Helpers of the GPU parity tests: arena marshalling, one GPU compress call through the
C ABI, and the comparison rules between the CUDA library and the CPU oracle.

Rules (tolerances are the ones the task fixes for this path):
  R1  |NSI_gpu - NSI_ref| <= 1e-5 * |NSI_ref| + FLT_MIN, NSI_ref in binary64.
  R2  counts equal k_l; the kept set has exactly k_l strictly ascending tiles; every tile whose
      NSI_ref is above T(1 + 2e-5) is kept and none below T(1 - 2e-5) is; if the kept set
      equals the oracle's, idx / val / residual are bit-exact against the oracle; if it differs
      (only possible inside the band), they are bit-exact against the oracle's pack of the
      GPU's set.
  R3  |dense_gpu - dense_ref| <= 1e-6 * sum_w |scale * sent_w| per element.
"""
from __future__ import annotations

from typing import List, Optional, Sequence

import numpy as np
import torch

from paper_2312_17530_b200 import binding

TAU = 1e-5
FLT_MIN = float(np.finfo(np.float32).tiny)
CANARY16 = 0x7A5A   # 16-bit filler of bfloat16 payload buffers
CANARY = np.float32(-7.25)


def to_arena(plan: binding.Plan, per_layer: Sequence[np.ndarray], dtype=np.float32, fill=CANARY) -> np.ndarray:
    """Flat arena with the plan's layer offsets; padding holds a canary value."""
    if dtype == np.uint16:
        a = np.full(plan.info.arena_elems, 0xC0E8, dtype=np.uint16)  # bfloat16(-7.25)
    else:
        a = np.full(plan.info.arena_elems, fill, dtype=dtype)
    for li, x in zip(plan.layers, per_layer):
        x = np.asarray(x).reshape(-1)
        assert x.size == li.rows * li.cols
        a[li.elem_offset:li.elem_offset + x.size] = x
    return a


def from_arena(plan: binding.Plan, arena: np.ndarray) -> List[np.ndarray]:
    return [arena[li.elem_offset:li.elem_offset + li.rows * li.cols] for li in plan.layers]


def padding_mask(plan: binding.Plan) -> np.ndarray:
    m = np.ones(plan.info.arena_elems, dtype=bool)
    for li in plan.layers:
        m[li.elem_offset:li.elem_offset + li.rows * li.cols] = False
    return m


def dev(x: np.ndarray, device="cuda:0") -> torch.Tensor:
    t = torch.from_numpy(np.ascontiguousarray(x))
    if x.dtype == np.uint16:
        t = t.view(torch.bfloat16)
    return t.to(device)


class GpuCompress:
    """One worker's buffers on the device plus a call of rsdgc_compress()."""

    def __init__(self, plan: binding.Plan, max_ratio: float = 1.0, device="cuda:0", with_nsi: bool = True):
        self.plan, self.device = plan, device
        ni, nv = plan.payload_bound(max_ratio)
        self.idx = torch.full((max(ni, 4),), -1, dtype=torch.int32, device=device)
        self.half = bool(plan.flags & binding.PAYLOAD_BF16)   # payload values are bfloat16 words
        self.val = (torch.full((max(nv, 8),), CANARY16, dtype=torch.int16, device=device) if self.half else
                    torch.full((max(nv, 4),), float(CANARY), dtype=torch.float32, device=device))
        self.counts = torch.full((plan.n_layers,), -1, dtype=torch.int32, device=device)
        self.nsi = torch.full((plan.info.total_tiles_padded,), float(CANARY), dtype=torch.float32,
                              device=device) if with_nsi else None
        self.workspace = None if with_nsi else torch.empty(max(plan.info.workspace_bytes, 16), dtype=torch.uint8,
                                                           device=device)

    def run(self, grads: torch.Tensor, residual: torch.Tensor, ratios: torch.Tensor, velocity=None,
            momentum: float = 0.0):
        if velocity is None:
            self.plan.compress(grads, residual, ratios, self.idx, self.val, self.counts, nsi=self.nsi,
                               workspace=self.workspace)
        else:
            self.plan.compress_momentum(grads, velocity, momentum, residual, ratios, self.idx, self.val,
                                        self.counts, nsi=self.nsi, workspace=self.workspace)
        torch.cuda.synchronize()
        return self.plan.status()

    def payload(self):
        return self.idx, self.val, self.counts


def check_layer(oracle, li, shape, g, r, ratio, alpha, clamp, gpu_nsi, gpu_count, gpu_idx, gpu_val, gpu_res,
                strict_keys: bool = True, what: str = "", velocity=None, momentum: float = 0.0,
                payload_bf16: bool = False):
    """Applies R1 and R2 to one layer; returns the oracle's LayerResult.  With ``payload_bf16``
    gpu_val holds the 16-bit words of the payload."""
    ref = oracle.compress_layer(g, r, shape, ratio, alpha, clamp_min1=clamp, velocity=velocity, momentum=momentum,
                                payload_bf16=payload_bf16)
    K = ref.nsi_f32.size
    # R1
    err = np.abs(gpu_nsi.astype(np.float64) - ref.nsi_ref)
    finite = np.isfinite(ref.nsi_ref)
    assert (err[finite] <= TAU * np.abs(ref.nsi_ref[finite]) + FLT_MIN).all(), what + ": NSI beyond 1e-5 relative"
    assert (gpu_nsi[ref.nsi_ref == 0] == 0).all() and not np.signbit(gpu_nsi[finite]).any()
    if strict_keys:  # same binary32 operations in the same order on both sides
        np.testing.assert_array_equal(gpu_nsi.view(np.uint32), ref.nsi_f32.view(np.uint32), err_msg=what)
    # R2
    assert gpu_count == ref.k, "%s: count %d != k %d" % (what, gpu_count, ref.k)
    assert gpu_idx.size == ref.k
    if ref.k:
        assert (np.diff(gpu_idx) > 0).all() and gpu_idx[0] >= 0 and gpu_idx[-1] < K, what + ": idx not ascending"
        T = ref.threshold
        kept = np.zeros(K, dtype=bool)
        kept[gpu_idx] = True
        if np.isfinite(T):
            must = ref.nsi_ref > T * (1 + 2 * TAU)
            must_not = ref.nsi_ref < T * (1 - 2 * TAU)
            assert kept[must].all(), what + ": a tile clearly above the threshold is missing"
            assert not kept[must_not].any(), what + ": a tile clearly below the threshold was kept"
    if not np.array_equal(gpu_idx, ref.idx):
        ref = oracle.compress_layer(g, r, shape, ratio, alpha, clamp_min1=clamp, forced_sel=gpu_idx,
                                    velocity=velocity, momentum=momentum, payload_bf16=payload_bf16)
    np.testing.assert_array_equal(gpu_idx, ref.idx, err_msg=what)
    if payload_bf16:
        np.testing.assert_array_equal(gpu_val.view(np.uint16), ref.val_bf16, err_msg=what + " val (bfloat16)")
    else:
        np.testing.assert_array_equal(gpu_val.view(np.uint32), ref.val.view(np.uint32), err_msg=what + " val")
    np.testing.assert_array_equal(gpu_res.view(np.uint32), ref.residual.view(np.uint32), err_msg=what + " residual")
    return ref


def compress_and_check(oracle, plan: binding.Plan, shapes, grads: Sequence[np.ndarray],
                       residuals: Sequence[np.ndarray], ratios: Sequence[float], alpha: float, clamp: bool = True,
                       gc: Optional[GpuCompress] = None, strict_keys: bool = True, what: str = "",
                       max_ratio: float = 1.0, velocities: Optional[Sequence[np.ndarray]] = None,
                       momentum: float = 0.0):
    """Runs one GPU compress and checks every layer against the oracle.  Returns
    (new residuals per layer, oracle results per layer, GpuCompress).  With ``velocities`` the
    momentum-corrected entry point is used and the new velocities are checked bit for bit
    (they are in the oracle results)."""
    g_is_bf16 = grads[0].dtype == np.uint16
    g_arena = to_arena(plan, grads, np.uint16 if g_is_bf16 else np.float32)
    r_arena = to_arena(plan, residuals)
    gc = gc or GpuCompress(plan, max_ratio=max_ratio)
    d_g, d_r = dev(g_arena), dev(r_arena)
    d_ratios = torch.tensor(np.asarray(ratios, dtype=np.float32), device=gc.device)
    d_u = dev(to_arena(plan, velocities)) if velocities is not None else None
    st = gc.run(d_g, d_r, d_ratios, velocity=d_u, momentum=momentum)
    assert st.flags == 0, "%s: status flags %d" % (what, st.flags)
    # inputs untouched, padding untouched
    g_back = d_g.view(torch.int16).cpu().numpy().view(np.uint16) if g_is_bf16 else d_g.cpu().numpy()
    np.testing.assert_array_equal(g_back, g_arena)
    res_arena = d_r.cpu().numpy()
    pad = padding_mask(plan)
    assert (res_arena[pad] == CANARY).all(), what + ": padding of the residual arena was written"
    vel_arena = d_u.cpu().numpy() if d_u is not None else None
    if vel_arena is not None:
        assert (vel_arena[pad] == CANARY).all(), what + ": padding of the velocity arena was written"
    counts = gc.counts.cpu().numpy()
    idx, val, nsi = gc.idx.cpu().numpy(), gc.val.cpu().numpy(), gc.nsi.cpu().numpy()
    half = gc.half
    assert st.idx_needed == counts.sum()
    io = vo = 0
    refs, new_res = [], []
    for l, (li, shape) in enumerate(zip(plan.layers, shapes)):
        k, slot = int(counts[l]), shape[2] * shape[3]
        ref = check_layer(oracle, li, shape, grads[l], residuals[l], float(np.float32(ratios[l])), alpha, clamp,
                          nsi[li.tile_offset:li.tile_offset + li.n_tiles], k, idx[io:io + k],
                          val[vo:vo + k * slot], res_arena[li.elem_offset:li.elem_offset + li.rows * li.cols],
                          strict_keys=strict_keys, what="%s layer %d %r" % (what, l, tuple(shape)),
                          velocity=None if velocities is None else velocities[l], momentum=momentum,
                          payload_bf16=half)
        if vel_arena is not None:
            np.testing.assert_array_equal(
                vel_arena[li.elem_offset:li.elem_offset + li.rows * li.cols].view(np.uint32),
                ref.velocity.view(np.uint32), err_msg="%s layer %d velocity" % (what, l))
        io, vo = io + k, vo + k * slot
        refs.append(ref)
        new_res.append(ref.residual)
    assert st.val_needed == vo
    assert (idx[io:] == -1).all() and (val[vo:] == (CANARY16 if half else CANARY)).all(), \
        what + ": payload written past its end"
    return new_res, refs, gc


def compress_workers_and_check(oracle, plan: binding.Plan, shapes, grads_w, residuals_w, ratios, alpha: float,
                               clamp: bool = True, what: str = "", max_ratio: float = 1.0, device="cuda:0"):
    """One rsdgc_compress_workers() call for len(grads_w) workers; every worker's outputs are
    checked against the oracle like a single rsdgc_compress() call (the indicators are read from
    the worker's part of the workspace, where the call leaves them as keys).  Returns
    (new residuals per worker and layer, oracle results per worker, payload tensors per worker)."""
    W = len(grads_w)
    plan.reserve_workers(W)
    ni, nv = plan.payload_bound(max_ratio)
    d_g = [dev(to_arena(plan, g, np.uint16 if g[0].dtype == np.uint16 else np.float32)) for g in grads_w]
    r_arenas = [to_arena(plan, r) for r in residuals_w]
    d_r = [dev(a) for a in r_arenas]
    idx = [torch.full((max(ni, 4),), -1, dtype=torch.int32, device=device) for _ in range(W)]
    val = [torch.full((max(nv, 4),), float(CANARY), dtype=torch.float32, device=device) for _ in range(W)]
    cnt = [torch.full((plan.n_layers,), -1, dtype=torch.int32, device=device) for _ in range(W)]
    stride = plan.info.workspace_bytes // 4
    ws = torch.full((W * stride,), float(CANARY), dtype=torch.float32, device=device)
    d_ratios = torch.tensor(np.asarray(ratios, dtype=np.float32), device=device)
    plan.compress_workers(d_g, d_r, d_ratios, idx, val, cnt, ws)
    torch.cuda.synchronize()
    st = plan.status()
    assert st.flags == 0, "%s: status flags %d" % (what, st.flags)
    pad = padding_mask(plan)
    keys = ws.cpu().numpy()
    new_res_w, refs_w = [], []
    for w in range(W):
        res_arena = d_r[w].cpu().numpy()
        assert (res_arena[pad] == CANARY).all(), what + ": padding of a residual arena was written"
        counts, ix, vl = cnt[w].cpu().numpy(), idx[w].cpu().numpy(), val[w].cpu().numpy()
        nsi = keys[w * stride:(w + 1) * stride]
        io = vo = 0
        refs, new_res = [], []
        for l, (li, shape) in enumerate(zip(plan.layers, shapes)):
            k, slot = int(counts[l]), shape[2] * shape[3]
            ref = check_layer(oracle, li, shape, grads_w[w][l], residuals_w[w][l], float(np.float32(ratios[l])),
                              alpha, clamp, nsi[li.tile_offset:li.tile_offset + li.n_tiles], k, ix[io:io + k],
                              vl[vo:vo + k * slot], res_arena[li.elem_offset:li.elem_offset + li.rows * li.cols],
                              what="%s worker %d layer %d %r" % (what, w, l, tuple(shape)))
            io, vo = io + k, vo + k * slot
            refs.append(ref)
            new_res.append(ref.residual)
        assert st.idx_needed == io and st.val_needed == vo
        assert (ix[io:] == -1).all() and (vl[vo:] == CANARY).all(), what + ": payload written past its end"
        new_res_w.append(new_res)
        refs_w.append(refs)
    return new_res_w, refs_w, list(zip(idx, val, cnt))


def check_decompress(dense_gpu: np.ndarray, dense_ref: np.ndarray, abs_sent_sum: np.ndarray, exact: bool = True):
    """R3 (and bit-exactness, which holds because workers are added in order on both sides)."""
    assert (np.abs(dense_gpu.astype(np.float64) - dense_ref) <= 1e-6 * abs_sent_sum + 1e-45).all()
    if exact:
        np.testing.assert_array_equal(dense_gpu.view(np.uint32), dense_ref.view(np.uint32))


# ---------------------------------------------------------------------------------------------
# full-size single layers (up to 1 B elements): every key through the oracle, selection by the
# oracle's rule on the oracle's keys (its full sort replaced by a partition, see below)
# ---------------------------------------------------------------------------------------------

def bf16_bits_to_f32(bits: np.ndarray) -> np.ndarray:
    return (bits.astype(np.uint32) << 16).view(np.float32)


def select_by_partition(keys_f32: np.ndarray, k: int) -> np.ndarray:
    """The oracle's selection rule (the k largest indicators, ties to the lower tile index, result
    ascending) evaluated with a partition instead of the oracle's full sort, for layers of 10^8
    tiles; tests/test_oracle_pins.py holds it to oracle.select() on inputs with many ties.
    Indicators are >= +0 (or +Inf for non-finite ones), so their bit patterns order like the values."""
    keys = np.ascontiguousarray(keys_f32, dtype=np.float32).view(np.uint32)
    K = keys.size
    if k <= 0:
        return np.zeros(0, np.int32)
    if k >= K:
        return np.arange(K, dtype=np.int32)
    t = np.partition(keys, K - k)[K - k]          # the k-th largest key
    above = np.flatnonzero(keys > t)
    equal = np.flatnonzero(keys == t)[:k - above.size]
    return np.sort(np.concatenate([above, equal])).astype(np.int32)


class LargeLayerReference:
    """What the oracle says about one large layer, computed once and used for several keep ratios:
    v = g + r (Eq. 12) and the indicator of EVERY tile (Eq. 8-10; oracle.nsi over bands of tile rows,
    which is the same per-tile arithmetic, to bound host memory), with R1 checked between the
    oracle's binary32 and binary64 values band by band."""

    def __init__(self, oracle, shape, g: np.ndarray, r: np.ndarray, alpha: float, band_tile_rows: int = 1024):
        self.oracle, self.shape, self.alpha = oracle, shape, alpha
        rows, cols, nh, nw = shape
        self.TR, self.TC = -(-rows // nh), -(-cols // nw)
        self.K = self.TR * self.TC
        self.v = oracle.accumulate(g, r)                      # one binary32 add per element
        v2 = self.v.reshape(rows, cols)
        self.keys = np.empty(self.K, np.float32)
        self.r1_worst = 0.0
        for t0 in range(0, self.TR, band_tile_rows):
            t1 = min(self.TR, t0 + band_tile_rows)
            band = v2[t0 * nh:min(rows, t1 * nh)]
            ref, f32, nonfinite = oracle.nsi(band.reshape(-1), (band.shape[0], cols, nh, nw), alpha)
            assert nonfinite == 0
            self.keys[t0 * self.TC:t1 * self.TC] = f32
            err = np.abs(f32.astype(np.float64) - ref) - (TAU * np.abs(ref) + FLT_MIN)
            self.r1_worst = max(self.r1_worst, float(err.max()))
        assert self.r1_worst <= 0.0, "the binary32 indicator leaves the 1e-5 band around the binary64 one"

    def check(self, ratio: float, gpu_nsi: np.ndarray, gpu_count: int, gpu_idx: np.ndarray, gpu_val: np.ndarray,
              gpu_res: np.ndarray, what: str = ""):
        """R1 + R2 for one GPU call on this layer: all keys bit-equal to the oracle's (so R1, held above for
        the oracle's binary32 values, holds for the GPU's), count = k (Eq. 11), the kept set = the oracle's
        rule on the oracle's keys, payload values and the new accumulator bit-exact against oracle.pack."""
        oracle, (rows, cols, nh, nw) = self.oracle, self.shape
        np.testing.assert_array_equal(gpu_nsi.view(np.uint32), self.keys.view(np.uint32), err_msg=what + " keys")
        k = oracle.keep_count(self.K, ratio, True)
        assert gpu_count == k and gpu_idx.size == k, what + ": count"
        sel = select_by_partition(self.keys, k)
        np.testing.assert_array_equal(gpu_idx, sel, err_msg=what + " kept set")
        idx, val, res = oracle.pack(self.v, self.shape, sel)
        np.testing.assert_array_equal(gpu_idx, idx)
        np.testing.assert_array_equal(gpu_val.view(np.uint32), val.view(np.uint32), err_msg=what + " val")
        assert np.array_equal(gpu_res.view(np.uint32), res.view(np.uint32)), what + " residual"

"""Host-side logic of the CUDA library, checked without a GPU: the shared library loads and
exports every symbol the header declares, and host-only plans (device < 0) give consistent
sizes, offsets and work lists."""
import os
import re

import numpy as np
import pytest

from paper_2312_17530_b200 import binding, synth
from paper_2312_17530_b200.build import build_library

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build_library()
    return binding.lib()


def test_library_exports_every_declared_symbol(lib):
    header = open(os.path.join(ROOT, "include", "rsdgc.h")).read()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    declared = set(re.findall(r"\b(rsdgc_[a-z_0-9]+)\s*\(", header))
    assert declared == set(binding.EXPORTS)
    for name in declared:
        assert getattr(lib, name) is not None
    assert lib.rsdgc_strerror(0) == b"ok" and lib.rsdgc_strerror(-2) != lib.rsdgc_strerror(-1)
    assert lib.rsdgc_launch_count() == 0


def test_plan_create_rejects_bad_arguments(lib):
    ok = [(8, 8, 3, 3)]
    for layers, kw in [([], {}), ([(0, 8, 3, 3)], {}), ([(8, 8, 0, 3)], {}), (ok, {"alpha": 1.5}),
                       (ok, {"alpha": float("nan")}), (ok, {"grad_dtype": 7}), (ok, {"flags": 32})]:
        with pytest.raises(binding.RsdgcError) as e:
            binding.Plan(layers, device=-1, **kw)
        assert e.value.code == binding.ERR_INVALID
    for layers in ([(8, 8, 65, 65)], [(1 << 20, 1 << 20, 3, 3)], [(4, 4, 3, 3)] * 3000):
        with pytest.raises(binding.RsdgcError) as e:
            binding.Plan(layers, device=-1)
        assert e.value.code == binding.ERR_CAPACITY
    # a host-only plan cannot launch anything
    p = binding.Plan(ok, device=-1)
    assert lib.rsdgc_compress(p._h, 16, 16, 16, 16, 1, 16, 1, 16, None, 16, None) == binding.ERR_INVALID


@pytest.mark.parametrize("net,dtype", [("resnet18", 0), ("resnet50", 0), ("vgg19", 0), ("odd", 0), ("odd", 1),
                                       ("wide_tiles", 0), ("wide_tiles", 1)])
def test_plan_offsets_and_worklist_cover_every_tile_once(lib, net, dtype):
    gran = 8 if dtype == binding.RSDGC_BF16 else 4      # elements per 16 bytes of the gradient arena
    if net == "wide_tiles":
        # neighborhoods of more than 550 elements: fewer than 8 tile columns fit an item, so the
        # column chunks are not multiples of 8 tiles wide
        shapes = [(50, 400, 25, 25), (40, 480, 20, 30), (75, 1000, 25, 25), (64, 4096, 32, 32), (30, 777, 30, 21)]
    elif net == "odd":
        shapes = [(7, 11, 3, 3), (1, 5, 1, 9), (4096, 45, 3, 3), (3, 20000, 3, 3), (100, 4401, 2, 5),
                  (5000, 7, 1, 7), (1, 100000, 1, 9), (64, 64, 64, 64), (9, 9, 1, 1)]
    else:
        shapes = synth.layer_shapes(getattr(synth, net + "_tensors")())
    p = binding.Plan(shapes, device=-1, grad_dtype=dtype)
    assert p.info.n_layers == len(shapes)
    assert p.info.total_elems == sum(r * c for r, c, _, _ in shapes)
    tiles = [(-(-r // nh)) * (-(-c // nw)) for r, c, nh, nw in shapes]
    assert p.info.total_tiles == sum(tiles)
    eo = to = 0
    for l, (li, (r, c, nh, nw)) in enumerate(zip(p.layers, shapes)):
        assert (li.elem_offset, li.tile_offset, li.n_tiles) == (eo, to, tiles[l])
        assert li.elem_offset % 64 == 0 and li.tile_offset % 64 == 0
        eo += -(-r * c // 64) * 64
        to += -(-tiles[l] // 64) * 64
    assert p.info.arena_elems == eo and p.info.total_tiles_padded == to
    assert p.info.workspace_bytes == 4 * to

    items, grids, nflush = p.worklist()
    # elements one item may hold: a stage of the first pass (larger with 2-byte gradients)
    item_elems = 5600 if dtype == binding.RSDGC_BF16 else 4400
    assert grids.tolist() == [148 * 3, 148 * 2]
    assert (np.diff(items[:, 0]) >= 0).all()          # layers in order
    for l, (r, c, nh, nw) in enumerate(shapes):
        TR, TC = -(-r // nh), -(-c // nw)
        cover = np.zeros((TR, TC), dtype=np.int32)
        sel = items[items[:, 0] == l]
        for _, tr0, ntr, tc0, ntc, path, cta, pitch, flags in sel.tolist():
            assert ntr >= 1 and ntc >= 1 and tr0 + ntr <= TR and tc0 + ntc <= TC
            rows = min(r, (tr0 + ntr) * nh) - tr0 * nh
            cols = min(c, (tc0 + ntc) * nw) - tc0 * nw
            assert rows * cols <= item_elems
            assert ntr == 1 or (tc0 == 0 and ntc == TC)   # several tile rows only at full width
            assert path in (0, 1) and 0 <= cta < grids[path]
            start = p.layers[l].elem_offset + tr0 * nh * c + tc0 * nw
            contiguous = cols == c or rows == 1
            assert bool(flags & 1) == contiguous
            # the block in shared memory: rows of `pitch` elements, all of it inside one stage
            assert pitch >= cols and (pitch == cols if contiguous else rows * pitch <= item_elems)
            # 128-bit accesses (flag 2) and bulk copies (flag 4, the bulk-copy kernel) need every row of
            # the item 16-byte aligned in global memory (start, row stride, width) and, through the
            # pitch, in shared memory; bulk copies need that for the gradient's element size too
            def aligned(g):
                return start % g == 0 and (contiguous or (c % g == 0 and cols % g == 0 and pitch % g == 0))
            assert bool(flags & 2) == aligned(4)
            assert bool(flags & 4) == aligned(gran) and (path == 0) == bool(flags & 4)
            cover[tr0:tr0 + ntr, tc0:tc0 + ntc] += 1
        assert (cover == 1).all()
        assert nflush[l] == len(set((it[5], it[6]) for it in sel.tolist()))
    # within a kernel the CTA of consecutive items never decreases, and the static partition is
    # balanced: no CTA holds much more than the mean cost
    for path in (0, 1):
        sel = items[items[:, 5] == path]
        if not len(sel):
            continue
        assert (np.diff(sel[:, 6]) >= 0).all()
        cost = np.zeros(grids[path])
        all_items = items.tolist()
        for k, (l, tr0, ntr, tc0, ntc, pa, cta, _, _) in enumerate(all_items):
            if pa != path:
                continue
            r, c, nh, nw = shapes[l]
            # the plan's cost model: elements + a fixed cost per item + the flush a CTA pays when it enters a
            # new layer
            cost[cta] += (min(r, (tr0 + ntr) * nh) - tr0 * nh) * (min(c, (tc0 + ntc) * nw) - tc0 * nw) + 8000
            if k > 0 and all_items[k - 1][0] != l:
                cost[cta] += 12000
        assert cost.max() <= cost.sum() / len(cost) + item_elems + 8000 + 12000 + 1
    if net not in ("odd", "wide_tiles"):
        assert (items[:, 5] == 0).mean() > 0.99       # the usual shapes go to the bulk-copy kernel


def test_payload_bound(lib):
    shapes = [(512, 512, 3, 3), (1, 64, 1, 9)]
    p = binding.Plan(shapes, device=-1)
    ni, nv = p.payload_bound(1 / 64)
    assert ni == (457 + 1) + 2 and nv == 9 * ni
    ni, nv = p.payload_bound(1.0)
    assert ni == 29241 + 8


@pytest.mark.parametrize("net", ["resnet18", "resnet50", "odd", "single"])
def test_tail_slices_cover_every_tile_once(lib, net):
    """Plans of small layers select and pack in one kernel: every layer's tiles are covered exactly once by
    slices of at most 32768 keys, a layer's slices sit in one cluster of 8 CTAs on consecutive ranks, and
    layers of at most 8192 tiles take one CTA each outside the clusters."""
    if net == "odd":
        shapes = [(7, 11, 3, 3), (1, 5, 1, 9), (4096, 45, 3, 3), (3, 20000, 3, 3), (100, 4401, 2, 5), (1536, 1536, 3, 3),
                  (5000, 7, 1, 7), (1, 100000, 1, 9), (64, 64, 64, 64), (9, 9, 1, 1), (70000, 9, 1, 9), (40000, 9, 1, 9)]
    elif net == "single":
        shapes = [(512, 512, 3, 3)]
    else:
        shapes = synth.layer_shapes(getattr(synth, net + "_tensors")())
    p = binding.Plan(shapes, device=-1)
    sl, (n_big, n_small, n_clusters) = p.tail_slices()
    assert len(sl) == n_big + n_small and n_big == 8 * n_clusters and 0 < n_clusters <= 16
    tiles = [li.n_tiles for li in p.layers]
    cover = [np.zeros(t, np.int32) for t in tiles]
    for i, (layer, start, n, n_ranks, rank, leader) in enumerate(sl.tolist()):
        if n == 0:
            assert i < n_big                             # an idle rank of a partly filled cluster
            continue
        cover[layer][start:start + n] += 1
        assert start % 64 == 0
        if i < n_big:
            assert tiles[layer] > 8192 and n <= 32768 and 1 <= n_ranks <= 8 and 0 <= rank < n_ranks
            assert leader == i % 8 - rank and leader + n_ranks <= 8      # consecutive ranks of one cluster
            assert sl[i - rank, 0] == layer and sl[i - rank, 4] == 0
        else:
            assert tiles[layer] <= 8192 and (start, n, n_ranks, rank, leader) == (0, tiles[layer], 1, 0, 0)
    for c in cover:
        assert (c == 1).all()
    # equal slices: no slice of a layer is more than 64 keys larger than another
    for l in range(len(shapes)):
        ns = sl[(sl[:, 0] == l) & (sl[:, 2] > 0), 2]
        assert len(ns) == 0 or ns.max() - ns[:-1].min(initial=ns.max()) <= 64
    # the flag and layers beyond a cluster's reach give the chained kernels
    assert len(binding.Plan(shapes, device=-1, flags=binding.NO_FUSED_TAIL).tail_slices()[0]) == 0
    assert len(binding.Plan(shapes + [(3000, 3000, 3, 3)], device=-1).tail_slices()[0]) == 0


def test_tail_not_used_when_clusters_exceed_one_wave(lib):
    shapes = [(1536, 1536, 3, 3)] * 17                     # 17 layers of 8 slices each: 17 clusters
    assert len(binding.Plan(shapes, device=-1).tail_slices()[0]) == 0
    assert len(binding.Plan(shapes[:16], device=-1).tail_slices()[0]) == 128
    assert len(binding.Plan(synth.layer_shapes(synth.vgg19_tensors()), device=-1).tail_slices()[0]) == 0

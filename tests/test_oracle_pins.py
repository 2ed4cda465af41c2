"""Pins for the CPU oracle: everything here checks ``oracle/`` against something other than
itself -- hand-derived values of a worked example (Eq. 8-10), closed forms, NumPy/PyTorch
library routines on special cases, brute-force enumeration on tiny inputs and invariants
the paper's statements imply.  No GPU, no CUDA library."""
import itertools
import math
import os

import numpy as np
import pytest
import torch

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "fig1_style_6x6.txt")


def _load_fig1():
    mat, nsi_rows, keep_rows = [], [], []
    mode = None
    for line in open(GOLDEN):
        line = line.split("#")[0].strip()
        if not line:
            continue
        tok = line.split()
        if tok[0] == "matrix":
            mode = "matrix"
        elif tok[0] == "nsi":
            nsi_rows.append((float(tok[1]), [float(t) for t in tok[2:]]))
        elif tok[0] == "keep":
            keep_rows.append((float(tok[1]), int(tok[2]), [int(t) for t in tok[3:]]))
        elif mode == "matrix":
            mat.append([float(t) for t in tok])
    return np.array(mat, dtype=np.float32), nsi_rows, keep_rows


# ---------------------------------------------------------------------------------------------
# worked example (Fig. 1 style), Eq. 8-10 by hand
# ---------------------------------------------------------------------------------------------

def test_fig1_style_worked_example(oracle):
    m, nsi_rows, keep_rows = _load_fig1()
    assert m.shape == (6, 6)
    shape = (6, 6, 3, 3)
    for alpha, expected in nsi_rows:
        ref, f32, bad = oracle.nsi(m.reshape(-1), shape, alpha)
        assert bad == 0
        np.testing.assert_allclose(ref, expected, atol=6e-7, rtol=0)
        np.testing.assert_allclose(f32, expected, atol=2e-6, rtol=0)
    for alpha, k, kept in keep_rows:
        _, f32, _ = oracle.nsi(m.reshape(-1), shape, alpha)
        sel, thr = oracle.select(f32, k)
        assert sel.tolist() == kept
        assert thr == min(f32[kept])


def test_fig1_style_exact_closed_forms(oracle):
    m, _, _ = _load_fig1()
    for alpha in (0.5, 0.25, 1.0, 0.0):
        ref, _, _ = oracle.nsi(m.reshape(-1), (6, 6, 3, 3), alpha)
        a32 = float(np.float32(alpha))
        n3 = np.array([-0.4, -0.3, -0.2, -0.1, 0.0, 0.1, 0.2, 0.3, 0.4], dtype=np.float32).astype(np.float64)
        exact = [
            a32 * 2.0,
            a32 * 1.0 + (1 - a32) * math.sqrt(80.0 / 81.0),
            a32 * 1.0 + (1 - a32) * math.sqrt(8.0),
            a32 * np.abs(n3).mean() + (1 - a32) * math.sqrt(((n3 - n3.mean()) ** 2).mean()),
        ]
        np.testing.assert_allclose(ref, exact, rtol=1e-13)


def test_elementwise_topk_differs_from_neighborhood_choice(oracle):
    """The contrast the figure's caption draws: the 18 largest entries by magnitude are the 9,
    the nine 2's and eight of the +-1's, whereas k = 2 neighborhoods keeps N0 and N2 whole."""
    m, _, _ = _load_fig1()
    flat = np.abs(m.reshape(-1))
    top18 = np.argsort(-flat, kind="stable")[:18]
    rows, cols = np.unravel_index(top18, (6, 6))
    tiles = set(((rows // 3) * 2 + cols // 3).tolist())
    assert tiles == {0, 1, 2}
    _, f32, _ = oracle.nsi(m.reshape(-1), (6, 6, 3, 3), 0.5)
    sel, _ = oracle.select(f32, 2)
    assert sel.tolist() == [0, 2]


# ---------------------------------------------------------------------------------------------
# NSI against library routines and closed forms
# ---------------------------------------------------------------------------------------------

def _numpy_tile_stats(v, rows, cols, nh, nw, alpha):
    x = v.reshape(rows, cols).astype(np.float64)
    out = []
    for tr in range(-(-rows // nh)):
        for tc in range(-(-cols // nw)):
            t = x[tr * nh:(tr + 1) * nh, tc * nw:(tc + 1) * nw]
            out.append(alpha * np.mean(np.abs(t)) + (1 - alpha) * np.std(t))  # np.std: ddof=0
    return np.array(out)


@pytest.mark.parametrize("rows,cols,nh,nw", [(6, 6, 3, 3), (7, 11, 3, 3), (4, 4, 3, 3), (5, 45, 3, 3),
                                             (12, 9, 1, 9), (1, 64, 1, 9), (10, 14, 2, 5), (3, 3, 3, 3),
                                             (8, 6, 4, 2), (1, 1, 3, 3)])
def test_nsi_matches_numpy_mean_and_std_per_tile(oracle, rows, cols, nh, nw):
    rng = np.random.default_rng(rows * 1000 + cols)
    v = (rng.standard_normal(rows * cols) * 10 ** rng.uniform(-4, 1)).astype(np.float32)
    v += np.float32(0.3) * np.float32(np.abs(v).mean())  # non-zero mean so the mean term matters
    for alpha in (0.5, 0.25, 0.0, 1.0):
        a32 = float(np.float32(alpha))
        ref, f32, bad = oracle.nsi(v, (rows, cols, nh, nw), alpha)
        expect = _numpy_tile_stats(v, rows, cols, nh, nw, a32)
        assert bad == 0 and ref.size == oracle.tile_count(rows, cols, nh, nw) == expect.size
        np.testing.assert_allclose(ref, expect, rtol=1e-12, atol=0)
        np.testing.assert_allclose(f32, expect, rtol=2e-6, atol=1e-30)


def test_nsi_constant_tile_and_single_spike(oracle):
    c = np.full(9, -3.25, dtype=np.float32)
    ref, f32, _ = oracle.nsi(c, (3, 3, 3, 3), 0.5)
    assert ref[0] == 0.5 * 3.25 and f32[0] == np.float32(0.5 * 3.25)  # std term vanishes
    spike = np.zeros(9, dtype=np.float32)
    spike[4] = 9.0
    ref, f32, _ = oracle.nsi(spike, (3, 3, 3, 3), 0.25)
    np.testing.assert_allclose(ref[0], 0.25 * 1.0 + 0.75 * math.sqrt(8.0), rtol=1e-14)
    zeros = np.zeros(18, dtype=np.float32)
    ref, f32, _ = oracle.nsi(zeros, (3, 6, 3, 3), 0.5)
    assert (ref == 0).all() and (f32 == 0).all() and not np.signbit(f32).any()


def test_nsi_1x1_tiles_reduce_to_alpha_abs(oracle):
    rng = np.random.default_rng(3)
    v = rng.standard_normal(50).astype(np.float32)
    ref, f32, _ = oracle.nsi(v, (5, 10, 1, 1), 0.5)
    np.testing.assert_array_equal(ref, 0.5 * np.abs(v.astype(np.float64)))
    np.testing.assert_array_equal(f32, np.float32(0.5) * np.abs(v))


def test_nsi_homogeneity_and_rms_bounds(oracle):
    rng = np.random.default_rng(4)
    v = rng.standard_normal(9 * 40).astype(np.float32)
    shape = (3, 120, 3, 3)
    ref, f32, _ = oracle.nsi(v, shape, 0.5)
    for c in (4.0, -0.125, 1024.0):
        ref_c, f32_c, _ = oracle.nsi(v * np.float32(c), shape, 0.5)
        np.testing.assert_array_equal(ref_c, abs(c) * ref)      # powers of two: exact
        np.testing.assert_array_equal(f32_c, np.float32(abs(c)) * f32)
    ref3, _, _ = oracle.nsi(v * np.float32(3.0), shape, 0.5)
    np.testing.assert_allclose(ref3, 3.0 * ref, rtol=1e-6)
    # mean|v| <= rms and std <= rms, hence NSI <= rms for alpha in [0, 1]
    rms = np.sqrt((v.reshape(3, 40, 3).astype(np.float64) ** 2).transpose(1, 0, 2).reshape(40, 9).mean(axis=1))
    for alpha in (0.0, 0.5, 1.0):
        r, _, _ = oracle.nsi(v, shape, alpha)
        assert (r <= rms * (1 + 1e-12)).all()


def test_nsi_invariant_under_permutation_inside_a_tile(oracle):
    rng = np.random.default_rng(5)
    tiles = rng.standard_normal((30, 9)).astype(np.float32)
    perm = tiles.copy()
    for t in perm:
        rng.shuffle(t)
    shape = (30, 9, 1, 9)
    a, _, _ = oracle.nsi(tiles.reshape(-1), shape, 0.5)
    b, _, _ = oracle.nsi(perm.reshape(-1), shape, 0.5)
    np.testing.assert_allclose(a, b, rtol=1e-12)


def test_nsi_tile_geometry_is_row_major_not_transposed(oracle):
    """A 2x3 tiling of a 4x6 matrix with one hot entry per tile pins tile indexing."""
    rows, cols, nh, nw = 4, 6, 2, 3
    for i in range(rows):
        for j in range(cols):
            v = np.zeros(rows * cols, dtype=np.float32)
            v[i * cols + j] = 1.0
            ref, _, _ = oracle.nsi(v, (rows, cols, nh, nw), 1.0)
            hot = (i // nh) * 2 + (j // nw)
            expect = np.zeros(4)
            expect[hot] = 1.0 / 6.0
            np.testing.assert_allclose(ref, expect, rtol=1e-15)


def test_nsi_nonfinite_is_counted_and_ranked_first(oracle):
    v = np.ones(27, dtype=np.float32)
    v[13] = np.inf
    v[25] = np.nan
    ref, f32, bad = oracle.nsi(v, (3, 9, 3, 3), 0.5)
    assert bad == 2 and np.isposinf(f32[1]) and np.isposinf(f32[2]) and np.isfinite(f32[0])
    sel, _ = oracle.select(f32, 1)
    assert sel.tolist() == [1]


# ---------------------------------------------------------------------------------------------
# accumulation (Eq. 12)
# ---------------------------------------------------------------------------------------------

def test_accumulate_f32_is_one_ieee_add(oracle):
    rng = np.random.default_rng(6)
    g = rng.standard_normal(1000).astype(np.float32)
    r = (rng.standard_normal(1000) * 1e-3).astype(np.float32)
    np.testing.assert_array_equal(oracle.accumulate(g, r), g + r)
    exact = g.astype(np.float64) + r.astype(np.float64)
    assert (np.abs(oracle.accumulate(g, r) - exact) <= np.abs(exact) * 2.0 ** -24).all()


def test_accumulate_bf16_widens_exactly(oracle):
    from paper_2312_17530_b200 import synth

    rng = np.random.default_rng(7)
    x = rng.standard_normal(4096).astype(np.float32)
    bits = synth.f32_to_bf16_bits(x)
    t = torch.from_numpy(x).to(torch.bfloat16)
    np.testing.assert_array_equal(bits.view(np.int16), t.view(torch.int16).numpy())  # generator == torch RNE
    r = rng.standard_normal(4096).astype(np.float32)
    v = oracle.accumulate(bits, r)
    np.testing.assert_array_equal(v, (t.to(torch.float32) + torch.from_numpy(r)).numpy())


def test_momentum_correction_closed_forms(oracle):
    """Eq. 12, first two lines: with a constant gradient and nothing sent, u_T = g (1 - m^T) / (1 - m)
    and v_T = sum_t u_t; with m = 0 the step is the plain accumulation."""
    rng = np.random.default_rng(14)
    g = rng.standard_normal(257).astype(np.float32)
    r0 = rng.standard_normal(257).astype(np.float32)
    u1, v1 = oracle.accumulate_momentum(g, np.zeros_like(g), r0, 0.0)
    np.testing.assert_array_equal(u1, g)
    np.testing.assert_array_equal(v1, oracle.accumulate(g, r0))
    m, T = 0.9, 25
    u, v = np.zeros_like(g), np.zeros_like(g)
    for _ in range(T):
        u, v = oracle.accumulate_momentum(g, u, v, m)
    m32 = float(np.float32(m))
    g64 = g.astype(np.float64)
    u_exact = g64 * (1 - m32 ** T) / (1 - m32)
    v_exact = g64 * (T - m32 * (1 - m32 ** T) / (1 - m32)) / (1 - m32)
    np.testing.assert_allclose(u, u_exact, rtol=2e-6)
    np.testing.assert_allclose(v, v_exact, rtol=4e-6)
    # one step by hand: the product is rounded before the sum (no fused multiply-add)
    u0 = rng.standard_normal(257).astype(np.float32)
    u2, v2 = oracle.accumulate_momentum(g, u0, r0, m)
    np.testing.assert_array_equal(u2, np.float32(m) * u0 + g)
    np.testing.assert_array_equal(v2, r0 + u2)


def test_momentum_correction_with_bfloat16_gradients(oracle):
    """Eq. 12, first two lines, with the gradient stored as bfloat16: the stored 16 bits are widened
    exactly (they are the upper half of the binary32), then u = fl(m u0) + g and v = r + u with the
    product rounded before the sum.  Expected values are built with NumPy / torch binary32 ops from the
    bit patterns; m = 0 reduces to the plain accumulation; a plausible mistake (rounding g again, using
    the unwidened binary32 draw, a fused multiply-add, u and r swapped) changes some element."""
    from paper_2312_17530_b200 import synth

    rng = np.random.default_rng(21)
    n = 4099
    x = (rng.standard_normal(n) * 10.0 ** rng.uniform(-6, 1, n)).astype(np.float32)
    x[:6] = [0.0, -0.0, 1.0 + 2.0 ** -8, 3.0e38, 1.0e-40, -2.5]       # tie, near-overflow, subnormal
    bits = synth.f32_to_bf16_bits(x)
    widened = (bits.astype(np.uint32) << 16).view(np.float32)         # exact by construction of the format
    assert not np.array_equal(widened, x)                             # the 16-bit storage does lose bits
    np.testing.assert_array_equal(widened, torch.from_numpy(bits.view(np.int16)).view(torch.bfloat16)
                                  .to(torch.float32).numpy())
    u0 = rng.standard_normal(n).astype(np.float32)
    r0 = (rng.standard_normal(n) * 1e-2).astype(np.float32)
    m = 0.9
    u1, v1 = oracle.accumulate_momentum(bits, u0, r0, m)
    prod = np.float32(m) * u0                                         # one rounding
    want_u = prod + widened                                           # one rounding
    np.testing.assert_array_equal(u1.view(np.uint32), want_u.view(np.uint32))
    np.testing.assert_array_equal(v1.view(np.uint32), (r0 + want_u).view(np.uint32))
    # the same through torch's binary32 arithmetic
    tu = torch.from_numpy(u0) * torch.tensor(np.float32(m)) + torch.from_numpy(widened)
    np.testing.assert_array_equal(u1, tu.numpy())
    # not fused: the exactly rounded m*u0 + g differs somewhere from the two-step result
    fused = (np.float64(np.float32(m)) * u0.astype(np.float64) + widened.astype(np.float64)).astype(np.float32)
    assert (fused != u1).any()
    # m = 0: u = g exactly, v = the plain accumulation of Eq. 12's second line
    u2, v2 = oracle.accumulate_momentum(bits, u0, r0, 0.0)
    np.testing.assert_array_equal(u2.view(np.uint32) & 0x7FFFFFFF, widened.view(np.uint32) & 0x7FFFFFFF)
    np.testing.assert_array_equal(v2, oracle.accumulate(bits, r0))
    # the binary32 entry point on the widened values gives the same bits: the two variants differ only
    # in how the gradient is stored
    u3, v3 = oracle.accumulate_momentum(widened, u0, r0, m)
    np.testing.assert_array_equal(u1.view(np.uint32), u3.view(np.uint32))
    np.testing.assert_array_equal(v1.view(np.uint32), v3.view(np.uint32))
    # inputs are not modified
    np.testing.assert_array_equal(bits, synth.f32_to_bf16_bits(x))


# ---------------------------------------------------------------------------------------------
# keep count (Eq. 11) and selection
# ---------------------------------------------------------------------------------------------

def test_keep_count_examples(oracle):
    assert oracle.keep_count(29241, 1 / 64) == 457           # 171 x 171 tiles of a 512 x 512 matrix
    assert oracle.keep_count(64 * 3, 1 / 64) == 3            # divisible case of Eq. 11
    assert oracle.keep_count(64 * 3 + 1, 1 / 64) == 4
    assert oracle.keep_count(100, 0.0) == 1                  # a layer always sends one neighborhood ...
    assert oracle.keep_count(100, 0.0, clamp_min1=False) == 0  # ... unless the clamp is off
    assert oracle.keep_count(100, 1.0) == 100
    assert oracle.keep_count(100, 7.5) == 100
    assert oracle.keep_count(7, 0.5) == 4
    # the ratio is a binary32 number; the product is taken in binary64
    assert oracle.keep_count(10, 0.1) == math.ceil(10 * float(np.float32(0.1)))
    assert oracle.keep_count(1 << 20, 0.001) == math.ceil((1 << 20) * float(np.float32(0.001)))


def test_partition_form_of_the_selection_equals_the_oracles_sort(oracle):
    """The GPU tests on layers of 10^8 tiles evaluate the oracle's selection rule with a partition
    (parity.select_by_partition) because the oracle's full sort takes minutes there; here the two
    are held together on inputs with few distinct values (many ties at the threshold), all-equal
    keys, zeros, an infinity, and k at both ends."""
    import parity

    rng = np.random.default_rng(31)
    cases = [rng.standard_normal(5000).astype(np.float32) ** 2,
             rng.integers(0, 4, 3000).astype(np.float32) * np.float32(0.25),      # four distinct values
             np.full(777, 0.5, np.float32), np.zeros(100, np.float32),
             np.concatenate([rng.random(500).astype(np.float32), [np.inf, 0.0, np.inf]]).astype(np.float32)]
    for keys in cases:
        for k in (0, 1, 2, keys.size // 64 + 1, keys.size // 3, keys.size - 1, keys.size):
            want, _ = oracle.select(keys, k)
            np.testing.assert_array_equal(parity.select_by_partition(keys, k), want)


def test_large_layer_reference_agrees_with_the_layer_oracle(oracle):
    """parity.LargeLayerReference (bands of tile rows through oracle.nsi, partition selection, oracle.pack)
    must reproduce oracle.compress_layer, ragged edges and a band boundary inside the layer included."""
    import parity
    from paper_2312_17530_b200 import synth

    rng = np.random.default_rng(32)
    for shape, bf16 in (((100, 131, 3, 3), False), ((64, 50, 3, 3), True), ((10, 90, 1, 9), False)):
        rows, cols = shape[:2]
        x = (rng.standard_normal(rows * cols) * 1e-2).astype(np.float32)
        g = synth.f32_to_bf16_bits(x) if bf16 else x
        r = (rng.standard_normal(rows * cols) * 1e-3).astype(np.float32)
        big = parity.LargeLayerReference(oracle, shape, g, r, 0.5, band_tile_rows=7)
        for ratio in (0.1, 0.01):
            ratio = float(np.float32(ratio))
            ref = oracle.compress_layer(g, r, shape, ratio, 0.5)
            big.check(ratio, ref.nsi_f32, ref.k, ref.idx, ref.val, ref.residual)
            wrong = ref.residual.copy()
            wrong[int(ref.idx[0]) // big.TC * shape[2] * cols] = 1.0      # a sent entry not cleared
            with pytest.raises(AssertionError):
                big.check(ratio, ref.nsi_f32, ref.k, ref.idx, ref.val, wrong)


def test_select_1x1_alpha1_is_library_topk(oracle):
    rng = np.random.default_rng(8)
    v = rng.standard_normal(5000).astype(np.float32)
    assert np.unique(np.abs(v)).size == v.size
    _, f32, _ = oracle.nsi(v, (50, 100, 1, 1), 1.0)
    for k in (1, 17, 500, 4999, 5000):
        sel, thr = oracle.select(f32, k)
        ref = torch.topk(torch.from_numpy(np.abs(v)), k).indices.numpy()
        assert sel.tolist() == sorted(ref.tolist())
        part = np.argpartition(-np.abs(v), k - 1)[:k]
        assert sel.tolist() == sorted(part.tolist())
        assert thr == np.abs(v)[sel].min()


def test_select_brute_force_small(oracle):
    rng = np.random.default_rng(9)
    for trial in range(40):
        K = int(rng.integers(1, 11))
        # few distinct values => many ties
        nsi = rng.integers(0, 4, size=K).astype(np.float32) * np.float32(0.5)
        for k in range(0, K + 1):
            sel, _ = oracle.select(nsi, k)
            best, best_sets = None, []
            for comb in itertools.combinations(range(K), k):
                s = float(sum(nsi[list(comb)]))
                if best is None or s > best + 1e-12:
                    best, best_sets = s, [comb]
                elif abs(s - best) <= 1e-12:
                    best_sets.append(comb)
            assert tuple(sel.tolist()) == min(best_sets)  # lexicographically smallest maximiser


def test_select_pure_ties_take_lowest_indices(oracle):
    nsi = np.full(100, 0.75, dtype=np.float32)
    sel, thr = oracle.select(nsi, 13)
    assert sel.tolist() == list(range(13)) and thr == 0.75


# ---------------------------------------------------------------------------------------------
# payload, accumulator update, conservation
# ---------------------------------------------------------------------------------------------

@pytest.mark.parametrize("shape", [(7, 11, 3, 3), (12, 9, 1, 9), (1, 50, 1, 9), (64, 45, 3, 3), (9, 9, 3, 3)])
def test_compress_layer_invariants(oracle, shape):
    rows, cols, nh, nw = shape
    rng = np.random.default_rng(rows + cols)
    g = rng.standard_normal(rows * cols).astype(np.float32)
    r = (rng.standard_normal(rows * cols) * 0.1).astype(np.float32)
    res = oracle.compress_layer(g, r, shape, 0.3, 0.5)
    K = oracle.tile_count(*shape)
    assert res.k == math.ceil(K * float(np.float32(0.3))) == res.idx.size
    assert (np.diff(res.idx) > 0).all() and res.val.size == res.k * nh * nw
    # every tile above the threshold is kept, none below
    kept = np.zeros(K, bool)
    kept[res.idx] = True
    assert (res.nsi_f32[kept] >= res.threshold).all() and (res.nsi_f32[~kept] <= res.threshold).all()
    # sent + residual == accumulated input, elementwise; residual is zero exactly on sent tiles
    sent = np.zeros(rows * cols, dtype=np.float32)
    oracle.decompress_into(sent, shape, res.idx, res.val, 1.0)
    assert (sent + res.residual == res.v).all()
    TC = -(-cols // nw)
    tile_of = (np.arange(rows)[:, None] // nh) * TC + (np.arange(cols)[None, :] // nw)
    on_sent = kept[tile_of.reshape(-1)]
    assert (res.residual[on_sent] == 0).all() and not np.signbit(res.residual[on_sent]).any()
    np.testing.assert_array_equal(res.residual[~on_sent], res.v[~on_sent])
    np.testing.assert_array_equal(sent[on_sent], res.v[on_sent])
    # padded payload slots of clipped tiles are +0
    vals = res.val.reshape(res.k, nh, nw)
    for s, t in enumerate(res.idx.tolist()):
        tr, tc = divmod(t, TC)
        hh, ww = min(nh, rows - tr * nh), min(nw, cols - tc * nw)
        block = res.v.reshape(rows, cols)[tr * nh:tr * nh + hh, tc * nw:tc * nw + ww]
        np.testing.assert_array_equal(vals[s, :hh, :ww], block)
        pad = vals[s].copy()
        pad[:hh, :ww] = 1.0
        assert ((pad == 1.0) | ((pad == 0.0) & ~np.signbit(pad))).all()


def test_multi_iteration_conservation(oracle):
    """Eq. 12: over T iterations, everything sent plus the final accumulator equals the sum
    of all gradients (up to binary32 rounding of the running adds)."""
    shape = (30, 27, 3, 3)
    rng = np.random.default_rng(10)
    r = np.zeros(30 * 27, dtype=np.float32)
    total = np.zeros(30 * 27, dtype=np.float64)
    sent_total = np.zeros(30 * 27, dtype=np.float64)
    for _ in range(12):
        g = rng.standard_normal(30 * 27).astype(np.float32)
        total += g
        res = oracle.compress_layer(g, r, shape, 0.1, 0.5)
        s = np.zeros_like(r)
        oracle.decompress_into(s, shape, res.idx, res.val, 1.0)
        sent_total += s
        r = res.residual
    np.testing.assert_allclose(sent_total + r, total, atol=12 * 2.0 ** -22, rtol=0)


# ---------------------------------------------------------------------------------------------
# aggregation (Eq. 12 third line / Sync)
# ---------------------------------------------------------------------------------------------

def test_decompress_special_cases(oracle):
    shape = (10, 10, 3, 3)
    rng = np.random.default_rng(11)
    g = rng.standard_normal(100).astype(np.float32)
    res = oracle.compress_layer(g, np.zeros(100, np.float32), shape, 0.25, 0.5)
    dense = np.zeros(100, np.float32)
    oracle.decompress_into(dense, shape, res.idx, res.val, 1.0)
    sent = res.v - res.residual
    np.testing.assert_array_equal(dense, sent)                      # one worker: dense == sent
    oracle.decompress_into(dense, shape, res.idx, res.val, 1.0)
    np.testing.assert_array_equal(dense, 2 * sent)                  # two identical workers
    before = dense.copy()
    oracle.decompress_into(dense, shape, np.zeros(0, np.int32), np.zeros(0, np.float32), 1.0)
    np.testing.assert_array_equal(dense, before)                    # empty payload
    d2 = np.ones(100, np.float32)
    oracle.decompress_into(d2, shape, res.idx, res.val, 0.25)
    np.testing.assert_array_equal(d2, np.float32(1) + np.float32(0.25) * sent)
    # the assigning form forgets what the buffer held and is otherwise the same sum
    d3 = [np.full(100, np.nan, np.float32)]
    cr = oracle.CompressResult(layers=[res])
    oracle.decompress_assign([shape], d3, [cr, cr], 0.5)
    np.testing.assert_array_equal(d3[0], sent)                      # 0 + sent/2 + sent/2, exact in binary
    assert not np.signbit(d3[0][sent == 0]).any()                   # untouched entries are +0


def test_coordinate_view_scatters_like_the_aggregation(oracle):
    # scattering (position, value) pairs one by one rebuilds exactly what the tile-wise
    # aggregation builds; clipped tiles mark their padding with -1
    rng = np.random.default_rng(13)
    for shape in [(10, 11, 3, 3), (7, 9, 1, 9), (1, 20, 1, 9), (9, 9, 3, 3), (5, 4, 7, 5)]:
        n = shape[0] * shape[1]
        g = rng.standard_normal(n).astype(np.float32)
        res = oracle.compress_layer(g, np.zeros(n, np.float32), shape, 0.5, 0.5)
        coo = oracle.payload_to_coo(shape, res.idx, elem_offset=64)
        assert coo.size == res.val.size
        dense = np.zeros(64 + n, np.float32)
        for p, x in zip(coo, res.val):
            if p >= 0:
                dense[p] += x
            else:
                assert x == 0 and not np.signbit(x)
        want = np.zeros(n, np.float32)
        oracle.decompress_into(want, shape, res.idx, res.val, 1.0)
        np.testing.assert_array_equal(dense[64:], want)
        assert (dense[:64] == 0).all()
        valid = coo[coo >= 0]
        assert np.unique(valid).size == valid.size                   # tiles do not overlap
        n_pad = int((coo < 0).sum())
        if shape[0] % shape[2] == 0 and shape[1] % shape[3] == 0:
            assert n_pad == 0


# ---------------------------------------------------------------------------------------------
# payload with bfloat16 values (an option of the implementation; Eq. 12: the unsent part stays)
# ---------------------------------------------------------------------------------------------

def test_bf16_rounding_known_values_and_library_routine(oracle):
    two = lambda e: float(2.0 ** e)
    cases = [
        (1.0, 0x3F80), (-1.0, 0xBF80), (0.0, 0x0000), (-0.0, 0x8000),
        (1.0 + two(-8), 0x3F80),                    # tie between 0x3F80 and 0x3F81: even wins
        (1.0 + two(-8) + two(-23), 0x3F81),         # just above the tie
        (1.0 + 3 * two(-8), 0x3F82),                # tie between 0x3F81 and 0x3F82: even wins
        (1.0 + two(-7), 0x3F81),                    # exactly representable
        (float(np.float32(3.4028234663852886e38)), 0x7F80),   # largest binary32 rounds up to +inf
        (two(-133), 0x0001),                        # a bfloat16 subnormal, exact
        (two(-134), 0x0000),                        # tie between 0 and the smallest subnormal: even (0)
        (3 * two(-134), 0x0002),                    # tie between 1 and 2 subnormal steps: even (2)
        (float("inf"), 0x7F80), (float("-inf"), 0xFF80),
    ]
    for x, bits in cases:
        assert oracle.f32_to_bf16(x) == bits, (x, hex(oracle.f32_to_bf16(x)), hex(bits))
    assert (oracle.f32_to_bf16(float("nan")) & 0x7FFF) > 0x7F80
    # the same conversion as the tensor library's cast on random finite values of every magnitude
    import torch
    rng = np.random.default_rng(5)
    x = (rng.standard_normal(20000) * np.exp(rng.uniform(-80, 80, 20000))).astype(np.float32)
    want = torch.from_numpy(x).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    got = np.array([oracle.f32_to_bf16(float(v)) for v in x], dtype=np.uint16)
    np.testing.assert_array_equal(got, want)


def test_bf16_payload_keeps_the_rounding_error(oracle):
    shape = (10, 11, 3, 3)
    rng = np.random.default_rng(12)
    g = rng.standard_normal(110).astype(np.float32)
    r = (rng.standard_normal(110) * 0.1).astype(np.float32)
    full = oracle.compress_layer(g, r, shape, 0.3, 0.5)
    half = oracle.compress_layer(g, r, shape, 0.3, 0.5, payload_bf16=True)
    np.testing.assert_array_equal(half.idx, full.idx)               # the selection does not depend on it
    assert half.val_bf16.dtype == np.uint16 and half.val_bf16.size == full.val.size
    # sent + kept = v, exactly, on every element; unsent tiles keep v untouched
    sent = np.zeros(110, np.float32)
    oracle.decompress_into(sent, shape, half.idx, half.val, 1.0)
    np.testing.assert_array_equal(sent.astype(np.float64) + half.residual.astype(np.float64),
                                  half.v.astype(np.float64))
    untouched = full.residual != 0
    np.testing.assert_array_equal(half.residual[untouched], half.v[untouched])
    # every sent value is the nearest bfloat16: error at most half a unit in the 8th significant bit
    kept = ~untouched
    assert (np.abs(half.residual[kept]) <= np.abs(half.v[kept]) * 2.0 ** -8).all()
    assert np.abs(half.residual[kept]).max() > 0                    # and the error is really there
    # padded slots of clipped tiles are +0; the 16 low bits of what the receiver sees are zero
    assert (half.val.view(np.uint32) & 0xFFFF == 0).all()
    # values that bfloat16 holds exactly: identical to the 32-bit payload, nothing stays behind
    g2 = (rng.integers(-100, 100, 110) / 4.0).astype(np.float32)
    a = oracle.compress_layer(g2, np.zeros(110, np.float32), shape, 0.3, 0.5)
    b = oracle.compress_layer(g2, np.zeros(110, np.float32), shape, 0.3, 0.5, payload_bf16=True)
    np.testing.assert_array_equal(a.val, b.val)
    np.testing.assert_array_equal(a.residual, b.residual)


# ---------------------------------------------------------------------------------------------
# layer-wise ratio rule (Eq. 3-5)
# ---------------------------------------------------------------------------------------------

def test_update_ratios_against_numpy_sort(oracle):
    rng = np.random.default_rng(12)
    sizes = [64, 1000, 9, 4096, 1]
    scales = [1.0, 0.1, 5.0, 0.5, 0.0]
    w = [(rng.standard_normal(n) * s).astype(np.float32) for n, s in zip(sizes, scales)]
    for rho in (0.001, 0.02, 0.5, 1.0):
        ratios, surv, n_keep = oracle.update_ratios(w, rho)
        G = sum(sizes)
        assert n_keep == math.ceil(float(np.float32(rho)) * G) == surv.sum()   # sum_l c_l = ceil(rho G)
        flat = np.abs(np.concatenate(w))
        order = np.argsort(-flat.astype(np.float64), kind="stable")[:n_keep]     # stable: ties -> lower index
        owner = np.searchsorted(np.cumsum(sizes), order, side="right")
        expect = np.bincount(owner, minlength=len(sizes))
        np.testing.assert_array_equal(surv, expect)
        np.testing.assert_array_equal(ratios, (expect / np.array(sizes)).astype(np.float32))


def test_update_ratios_uniform_and_scaled_layer(oracle):
    rng = np.random.default_rng(13)
    w = [rng.standard_normal(20000).astype(np.float32) for _ in range(5)]
    ratios, _, _ = oracle.update_ratios(w, 0.02)
    np.testing.assert_allclose(ratios, 0.02, rtol=0.25)              # identical distributions => rho_l ~ rho
    w2 = [x.copy() for x in w]
    w2[2] *= np.float32(1000.0)
    r2, surv2, n_keep = oracle.update_ratios(w2, 0.02)
    assert n_keep == 2000 and r2[2] > 0.09 and all(r2[i] < ratios[i] for i in (0, 1, 3, 4))


def test_update_ratios_ties_go_to_lower_flat_index(oracle):
    w = [np.ones(10, np.float32), -np.ones(10, np.float32), np.ones(10, np.float32)]
    ratios, surv, n_keep = oracle.update_ratios(w, 0.5)
    assert n_keep == 15 and surv.tolist() == [10, 5, 0]
    np.testing.assert_array_equal(ratios, np.array([1.0, 0.5, 0.0], np.float32))

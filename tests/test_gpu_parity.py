"""GPU parity: the CUDA library (through the C ABI) against the CPU oracle, element by element,
on seeded inputs: the 512x512 single layer, a zoo of small / ragged / degenerate layers, the
ResNet-18-shaped set over 10 iterations with the ratio rule, aggregation of several workers."""
import numpy as np
import pytest
import torch

from paper_2312_17530_b200 import binding, synth

import parity

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _lib():
    assert torch.cuda.is_available(), "these tests need a CUDA device"
    binding.lib()  # raises if the CUDA library has not been built: no fallback


# ---------------------------------------------------------------------------------------------
# config 1: one 512x512 layer, clustered outliers, zero residual, 3x3 tiles, keep 1/64
# ---------------------------------------------------------------------------------------------

# Plans of small layers select and pack in one kernel per layer-size class; NO_FUSED_TAIL sends the same
# plan through the chained selection kernels that large layers take.  Both must match the oracle.
TAILS = [pytest.param(0, id="fused"), pytest.param(binding.NO_FUSED_TAIL, id="chained")]


@pytest.mark.parametrize("tail", TAILS)
def test_single_layer_512(oracle, tail):
    shapes = [(512, 512, 3, 3)]
    g = [synth.clustered_matrix(512, 512, seed=0)]
    r = [np.zeros(512 * 512, np.float32)]
    plan = binding.Plan(shapes, alpha=0.5, flags=binding.KEEP_AT_LEAST_ONE | tail)
    assert (len(plan.tail_slices()[0]) > 0) == (tail == 0)
    assert plan.layers[0].n_tiles == 171 * 171
    _, refs, gc = parity.compress_and_check(oracle, plan, shapes, g, r, [1 / 64], 0.5, what="512x512")
    assert refs[0].k == 457
    # the boosted 8x8 patches dominate the selection
    assert np.abs(refs[0].val).mean() > 5e-3


# ---------------------------------------------------------------------------------------------
# small, ragged and degenerate layers
# ---------------------------------------------------------------------------------------------

ZOO = [
    (7, 11, 3, 3), (1, 1, 3, 3), (3, 3, 3, 3), (4, 4, 3, 3), (1, 5, 1, 9), (1, 64, 1, 9), (64, 9, 1, 9),
    (4096, 45, 3, 3), (2, 20000, 3, 3), (100, 6145, 2, 5), (5000, 7, 1, 7), (1, 100003, 1, 9),
    (130, 130, 64, 64), (30, 30, 1, 1), (192, 49, 1, 49), (257, 1026, 3, 3), (999, 2049, 3, 3),
    (13, 8190, 4, 6), (70000, 9, 1, 9), (1000, 512, 3, 3),
    # neighborhoods of more than 550 elements: column chunks narrower than 8 tiles
    (50, 400, 25, 25), (40, 480, 20, 30), (30, 777, 30, 21),
]


@pytest.mark.parametrize("tail", TAILS)
@pytest.mark.parametrize("alpha", [0.5, 0.0, 1.0, 0.25])
def test_layer_zoo(oracle, alpha, tail):
    rng = np.random.default_rng(int(alpha * 100) + 1)
    shapes = ZOO
    g = [(rng.standard_normal(r * c) * 10 ** rng.uniform(-4, 0)).astype(np.float32) for r, c, _, _ in shapes]
    res = [(rng.standard_normal(r * c) * 10 ** rng.uniform(-5, -1)).astype(np.float32) for r, c, _, _ in shapes]
    ratios = rng.choice([0.001, 0.01, 1 / 64, 0.1, 0.3, 1.0, 0.0], size=len(shapes)).astype(np.float32)
    plan = binding.Plan(shapes, alpha=alpha, flags=binding.KEEP_AT_LEAST_ONE | tail)
    assert (len(plan.tail_slices()[0]) > 0) == (tail == 0)
    new_res, refs, gc = parity.compress_and_check(oracle, plan, shapes, g, res, ratios, alpha, what="zoo")
    # second iteration on the carried residual, same buffers
    g2 = [(rng.standard_normal(r * c) * 1e-2).astype(np.float32) for r, c, _, _ in shapes]
    gc.idx.fill_(-1)
    gc.val.fill_(float(parity.CANARY))
    parity.compress_and_check(oracle, plan, shapes, g2, new_res, ratios, alpha, gc=gc, what="zoo it2")


@pytest.mark.parametrize("tail", TAILS)
def test_degenerate_layers(oracle, tail):
    rng = np.random.default_rng(5)
    shapes = [(60, 60, 3, 3), (60, 60, 3, 3), (1, 900, 1, 9), (33, 33, 3, 3), (1, 7, 1, 9), (300, 300, 3, 3),
              (9, 15, 3, 3), (9, 18, 3, 3)]
    g = [np.zeros(3600, np.float32),                                    # all-zero layer: all NSI equal 0
         np.full(3600, 0.125, np.float32),                              # constant: all NSI equal, pure ties
         np.tile(np.arange(9, dtype=np.float32), 100),                  # identical tiles
         rng.standard_normal(33 * 33).astype(np.float32),
         rng.standard_normal(7).astype(np.float32),                    # a single clipped tile
         np.repeat(rng.integers(0, 3, 100 * 100), 9).reshape(100, 100, 3, 3).transpose(0, 2, 1, 3)
         .reshape(-1).astype(np.float32),                               # three distinct NSI values: many ties
         np.full(9 * 15, -0.5, np.float32),                             # 15 and 18 equal keys: the tie is cut inside
         np.full(9 * 18, 3.0, np.float32)]                              # the last, partial group of four keys
    res = [np.zeros(x.size, np.float32) for x in g]
    for ratios, clamp in (([0.1, 0.1, 0.05, 1.0, 0.5, 0.4, 0.9, 0.9], True), ([0.0] * 8, True), ([0.0] * 8, False),
                          ([1.0] * 8, True), ([0.5, 1e-9, 2.0, -1.0, 0.0, 0.33, 0.95, 0.5], False)):
        plan = binding.Plan(shapes, alpha=0.5, flags=(binding.KEEP_AT_LEAST_ONE if clamp else 0) | tail)
        _, refs, _ = parity.compress_and_check(oracle, plan, shapes, g, res, ratios, 0.5, clamp=clamp, what="degenerate")
        if ratios[0] == 0.1:
            k = oracle.keep_count(400, 0.1)                             # pure ties: the first k tiles
            assert refs[0].idx.tolist() == list(range(k)) and refs[1].idx.tolist() == list(range(k))
            assert refs[6].idx.tolist() == list(range(14)) and refs[7].idx.tolist() == list(range(17))
        if not clamp and ratios[0] == 0.0:
            assert sum(r.k for r in refs) == 0


def test_nonfinite_inputs_are_flagged_and_deterministic(oracle):
    shapes = [(30, 30, 3, 3), (1, 90, 1, 9)]
    rng = np.random.default_rng(6)
    g = [rng.standard_normal(900).astype(np.float32), rng.standard_normal(90).astype(np.float32)]
    g[0][[5, 400]] = [np.inf, np.nan]
    g[1][17] = -np.inf
    plan = binding.Plan(shapes, alpha=0.5)
    outs = []
    for _ in range(2):
        gc = parity.GpuCompress(plan)
        d_g = parity.dev(parity.to_arena(plan, g))
        d_r = parity.dev(parity.to_arena(plan, [np.zeros(900, np.float32), np.zeros(90, np.float32)]))
        st = gc.run(d_g, d_r, torch.tensor([0.05, 0.2], device="cuda:0"))
        assert st.flags == binding.STATUS_NONFINITE and st.nonfinite == 3
        outs.append((gc.idx.cpu().numpy().copy(), gc.nsi.cpu().numpy().view(np.uint32).copy()))
    np.testing.assert_array_equal(outs[0][0], outs[1][0])
    np.testing.assert_array_equal(outs[0][1], outs[1][1])
    ref0 = oracle.compress_layer(g[0], np.zeros(900, np.float32), shapes[0], 0.05, 0.5)
    assert ref0.nonfinite == 2
    np.testing.assert_array_equal(outs[0][0][:ref0.k], ref0.idx)      # non-finite tiles rank first


def test_bounded_wait_gives_up_and_reports_timeout():
    """The first pass waits for its bulk copies with a bounded poll loop; this runs that loop on a
    barrier that nothing will ever complete (no copy is issued, so nothing is left in flight), and the
    give-up must surface as STATUS_TIMEOUT, once, with the context and the plan still usable."""
    plan = binding.Plan([(64, 64, 3, 3)], alpha=0.5)
    assert plan.status().flags == 0
    plan.selftest_bounded_wait(300)
    st = plan.status()                       # synchronises, returns and clears the status word
    assert st.flags == binding.STATUS_TIMEOUT
    assert plan.status().flags == 0
    with pytest.raises(binding.RsdgcError):
        plan.selftest_bounded_wait(0)
    # the same plan still compresses correctly afterwards
    gc = parity.GpuCompress(plan)
    g = torch.randn(plan.info.arena_elems, device="cuda:0")
    r = torch.zeros(plan.info.arena_elems, device="cuda:0")
    st = gc.run(g, r, torch.tensor([0.1], device="cuda:0"))
    assert st.flags == 0 and int(gc.counts[0]) == 49


@pytest.mark.parametrize("tail", TAILS)
def test_payload_overflow_is_reported_and_nothing_is_lost(oracle, tail):
    shapes = [(90, 90, 3, 3), (60, 60, 3, 3)]
    rng = np.random.default_rng(7)
    g = [rng.standard_normal(8100).astype(np.float32), rng.standard_normal(3600).astype(np.float32)]
    plan = binding.Plan(shapes, alpha=0.5, flags=binding.KEEP_AT_LEAST_ONE | tail)
    gc = parity.GpuCompress(plan, max_ratio=0.01)           # room for about 1 % of the tiles only
    cap = gc.idx.numel()
    k0, k1 = oracle.keep_count(900, 0.1), oracle.keep_count(400, 0.1)
    assert cap < k0
    d_g = parity.dev(parity.to_arena(plan, g))
    r0 = parity.to_arena(plan, [np.zeros(8100, np.float32), np.zeros(3600, np.float32)])
    d_r = parity.dev(r0)
    st = gc.run(d_g, d_r, torch.tensor([0.1, 0.1], device="cuda:0"))
    assert st.flags == binding.STATUS_PAYLOAD_OVERFLOW
    assert st.idx_needed == k0 + k1 and st.val_needed == 9 * (k0 + k1)
    counts = gc.counts.cpu().numpy()
    assert counts.tolist() == [k0, k1]
    # tiles that fit were sent and zeroed; all others still sit in the residual: sent + residual == v
    idx, val = gc.idx.cpu().numpy(), gc.val.cpu().numpy()
    res = parity.from_arena(plan, d_r.cpu().numpy())
    sent = np.zeros(8100, np.float32)
    oracle.decompress_into(sent, shapes[0], idx[:cap], val[:cap * 9], 1.0)
    assert (sent + res[0] == g[0]).all() and (res[1] == g[1]).all()
    # the GPU aggregation of the cut-short payload: counts say k0 + k1 tiles, the buffers hold `cap` of
    # them; the capacities keep it inside the buffers and it adds exactly what was sent
    d_dense = torch.full((plan.info.arena_elems,), float(parity.CANARY), device="cuda:0")
    plan.decompress_assign([gc.payload()], d_dense, 1.0)
    torch.cuda.synchronize()
    dense = parity.from_arena(plan, d_dense.cpu().numpy())
    np.testing.assert_array_equal(dense[0], sent)
    assert (dense[0] + res[0] == g[0]).all() and (dense[1] == 0).all()


# ---------------------------------------------------------------------------------------------
# config 2: ResNet-18-shaped set, 10 iterations, residual carried, ratios from the weights
# ---------------------------------------------------------------------------------------------

@pytest.mark.parametrize("tail", TAILS)
def test_resnet18_ten_iterations_with_dynamic_ratios(oracle, tail):
    tensors = synth.resnet18_tensors()
    shapes = synth.layer_shapes(tensors)
    plan = binding.Plan(shapes, alpha=0.5, flags=binding.KEEP_AT_LEAST_ONE | tail)
    weights = synth.synthetic_weights(tensors, (2,))
    # ratio rule (Eq. 3-5) on the GPU against the oracle's full sort
    d_w = parity.dev(parity.to_arena(plan, weights))
    d_ratios = torch.full((plan.n_layers,), -1.0, device="cuda:0")
    plan.update_ratios(d_w, 1 / 50, d_ratios)
    torch.cuda.synchronize()
    ratios_ref, surv, n_keep = oracle.update_ratios(weights, 1 / 50)
    np.testing.assert_array_equal(d_ratios.cpu().numpy(), ratios_ref)
    assert n_keep == surv.sum() and (ratios_ref == 1.0).any() and (ratios_ref == 0.0).any()
    total = sum(int(np.ceil(k * float(r))) for k, r in zip([li.n_tiles for li in plan.layers], ratios_ref))
    assert 30 < plan.info.total_tiles / total < 70                      # about 50x fewer neighborhoods

    scales = synth.log_uniform_scales(len(tensors), (2,))
    res = [np.zeros(synth.numel(s), np.float32) for _, s in tensors]
    gc = parity.GpuCompress(plan, max_ratio=1.0)
    for it in range(10):
        g = synth.laplace_layers(tensors, (2, it), scales)
        gc.idx.fill_(-1)
        gc.val.fill_(float(parity.CANARY))
        res, refs, _ = parity.compress_and_check(oracle, plan, shapes, g, res, ratios_ref, 0.5, gc=gc,
                                                 what="resnet18 it%d" % it)


# ---------------------------------------------------------------------------------------------
# aggregation of several workers (Eq. 12 third line) on a mid-sized layer set
# ---------------------------------------------------------------------------------------------

@pytest.mark.parametrize("scale", [1.0, 0.25])
def test_decompress_accumulate_four_workers(oracle, scale):
    tensors = synth.vgg19_tensors()[:12] + [("fc.weight", (1000, 513)), ("fc.bias", (1000,))]
    shapes = synth.layer_shapes(tensors)
    plan = binding.Plan(shapes, alpha=0.5)
    sig = synth.log_uniform_scales(len(tensors), (3,))
    grads = synth.multi_worker_gradients(tensors, 4, (3,), sig)
    ratios = np.full(len(shapes), 1 / 16, np.float32)
    zeros = [np.zeros(synth.numel(s), np.float32) for _, s in tensors]
    payloads, refs_all = [], []
    for w in range(4):
        _, refs, gc = parity.compress_and_check(oracle, plan, shapes, grads[w], zeros, ratios, 0.5,
                                                what="worker %d" % w, max_ratio=1 / 16)
        payloads.append(gc.payload())
        refs_all.append(oracle.CompressResult(layers=refs))
    rng = np.random.default_rng(8)
    dense0 = [(rng.standard_normal(synth.numel(s)) * 1e-3).astype(np.float32) for _, s in tensors]
    d_dense = parity.dev(parity.to_arena(plan, dense0))
    plan.decompress_accumulate(payloads, d_dense, scale)
    torch.cuda.synchronize()
    dense_ref = [d.copy() for d in dense0]
    oracle.decompress_accumulate(shapes, dense_ref, refs_all, scale)
    out = d_dense.cpu().numpy()
    assert (out[parity.padding_mask(plan)] == parity.CANARY).all()
    collisions = 0
    for l, (got, ref) in enumerate(zip(parity.from_arena(plan, out), dense_ref)):
        abs_sum = np.zeros(ref.size)
        hit = np.zeros(ref.size, np.int32)
        for w in range(4):
            s = np.zeros(ref.size, np.float32)
            oracle.decompress_into(s, shapes[l], refs_all[w].layers[l].idx, refs_all[w].layers[l].val, scale)
            abs_sum += np.abs(s)
            hit += (s != 0)
        collisions += int((hit > 1).sum())
        parity.check_decompress(got, ref, abs_sum)
    assert collisions > 1000                                   # the workers' selections do overlap
    # the assigning variant: whatever the arena held is replaced, the padding is left alone
    d_dense2 = parity.dev(parity.to_arena(plan, [np.full(synth.numel(s), np.nan, np.float32) for _, s in tensors]))
    plan.decompress_assign(payloads, d_dense2, scale)
    torch.cuda.synchronize()
    assign_ref = [np.full(synth.numel(s), 3.0, np.float32) for _, s in tensors]
    oracle.decompress_assign(shapes, assign_ref, refs_all, scale)
    out2 = d_dense2.cpu().numpy()
    assert (out2[parity.padding_mask(plan)] == parity.CANARY).all()
    for got, ref in zip(parity.from_arena(plan, out2), assign_ref):
        np.testing.assert_array_equal(got.view(np.uint32), ref.view(np.uint32))
    plan.decompress_assign([], d_dense2, scale)               # no worker: all +0
    torch.cuda.synchronize()
    out2 = d_dense2.cpu().numpy()
    assert (out2[parity.padding_mask(plan)] == parity.CANARY).all()
    assert all((x.view(np.uint32) == 0).all() for x in parity.from_arena(plan, out2))
    # empty payload: nothing changes
    before = d_dense.clone()
    zc = torch.zeros(plan.n_layers, dtype=torch.int32, device="cuda:0")
    plan.decompress_accumulate([(payloads[0][0], payloads[0][1], zc)], d_dense, 1.0)
    plan.decompress_accumulate([], d_dense, 1.0)
    torch.cuda.synchronize()
    assert torch.equal(before, d_dense)


# ---------------------------------------------------------------------------------------------
# several workers in one call: the selection kernels run once over all workers
# ---------------------------------------------------------------------------------------------

@pytest.mark.parametrize("tail", TAILS)
@pytest.mark.parametrize("n_workers", [1, 3])
def test_compress_workers_two_iterations(oracle, n_workers, tail):
    shapes = [(300, 515, 3, 3), (256, 64 * 9, 1, 9), (1, 1000, 1, 9), (77, 45, 3, 3), (1200, 1536, 3, 3),
              (64, 7 * 7 * 3, 1, 49), (5, 5, 3, 3)]
    tensors = [("t%d" % i, (s[0], s[1])) for i, s in enumerate(shapes)]
    plan = binding.Plan(shapes, alpha=0.5, flags=binding.KEEP_AT_LEAST_ONE | tail)
    sig = synth.log_uniform_scales(len(shapes), (21,))
    ratios = np.array([1 / 16, 1 / 50, 0.3, 1.0, 1 / 64, 0.0, 0.5], np.float32)
    res = [[np.zeros(s[0] * s[1], np.float32) for s in shapes] for _ in range(n_workers)]
    for it in range(2):                     # the second call starts from the tables the first one left
        grads = synth.multi_worker_gradients(tensors, n_workers, (21, it), sig)
        res, refs, payloads = parity.compress_workers_and_check(oracle, plan, shapes, grads, res, ratios, 0.5,
                                                                what="iteration %d" % it)
    for w in range(n_workers):
        assert int(payloads[w][2].sum()) == sum(r.k for r in refs[w])


def test_compress_workers_host_pipelined(oracle):
    """Host buffers in, host payloads out, three workers over two staging arenas (the third reuses the
    first worker's arena): every worker's payload and accumulator match the oracle, twice in a row."""
    shapes = [(300, 515, 3, 3), (256, 64 * 9, 1, 9), (1, 1000, 1, 9), (1200, 1536, 3, 3)]
    tensors = [("t%d" % i, (s[0], s[1])) for i, s in enumerate(shapes)]
    plan = binding.Plan(shapes, alpha=0.5)
    W, dev = 3, "cuda:0"
    sig = synth.log_uniform_scales(len(shapes), (22,))
    ratios = np.array([1 / 16, 1 / 50, 0.3, 1 / 64], np.float32)
    ni, nv = plan.payload_bound(0.3)
    d_r = [torch.zeros(plan.info.arena_elems, device=dev) for _ in range(W)]
    d_idx = [torch.full((ni,), -1, dtype=torch.int32, device=dev) for _ in range(W)]
    d_val = [torch.full((nv,), float(parity.CANARY), device=dev) for _ in range(W)]
    d_cnt = [torch.zeros(len(shapes), dtype=torch.int32, device=dev) for _ in range(W)]
    h_idx = [torch.zeros(ni, dtype=torch.int32, pin_memory=True) for _ in range(W)]
    h_val = [torch.zeros(nv, dtype=torch.float32, pin_memory=True) for _ in range(W)]
    h_cnt = [torch.zeros(len(shapes), dtype=torch.int32, pin_memory=True) for _ in range(W)]
    stage = [torch.full((plan.info.arena_elems,), float("nan"), device=dev) for _ in range(2)]
    ws = torch.empty(plan.info.workspace_bytes, dtype=torch.uint8, device=dev)
    res = [[np.zeros(s[0] * s[1], np.float32) for s in shapes] for _ in range(W)]
    for it in range(2):
        grads = synth.multi_worker_gradients(tensors, W, (22, it), sig)
        h_g = [torch.from_numpy(parity.to_arena(plan, grads[w])).pin_memory() for w in range(W)]
        used_i, used_v = plan.compress_workers_host(h_g, stage, d_r, torch.tensor(ratios, device=dev), d_idx, d_val,
                                                    d_cnt, ws, h_idx, h_val, h_cnt)
        assert plan.status().flags == 0
        for w in range(W):
            ref = oracle.compress(shapes, grads[w], res[w], ratios, 0.5)
            assert h_cnt[w].numpy().tolist() == ref.counts.tolist()
            k = int(ref.counts.sum())
            assert (used_i[w], used_v[w]) == (k, sum(l.val.size for l in ref.layers))
            np.testing.assert_array_equal(h_idx[w].numpy()[:k], np.concatenate([l.idx for l in ref.layers]))
            np.testing.assert_array_equal(h_val[w].numpy()[:used_v[w]].view(np.uint32),
                                          np.concatenate([l.val for l in ref.layers]).view(np.uint32))
            res[w] = [l.residual for l in ref.layers]
            for got, want in zip(parity.from_arena(plan, d_r[w].cpu().numpy()), res[w]):
                np.testing.assert_array_equal(got.view(np.uint32), want.view(np.uint32))


def test_compress_workers_argument_errors():
    plan = binding.Plan([(64, 64, 3, 3)], alpha=0.5)
    dev = "cuda:0"
    g = [torch.zeros(plan.info.arena_elems, device=dev) for _ in range(2)]
    r = [torch.zeros(plan.info.arena_elems, device=dev) for _ in range(2)]
    ni, nv = plan.payload_bound(1.0)
    idx = [torch.zeros(ni, dtype=torch.int32, device=dev) for _ in range(2)]
    val = [torch.zeros(nv, device=dev) for _ in range(2)]
    cnt = [torch.zeros(1, dtype=torch.int32, device=dev) for _ in range(2)]
    ws = torch.zeros(2 * plan.info.workspace_bytes, dtype=torch.uint8, device=dev)
    rat = torch.ones(1, device=dev)
    with pytest.raises(binding.RsdgcError) as e:      # lanes not reserved
        plan.compress_workers(g, r, rat, idx, val, cnt, ws)
    assert e.value.code == binding.ERR_CAPACITY
    plan.reserve_workers(2)
    with pytest.raises(binding.RsdgcError) as e:      # two workers share an accumulator
        plan.compress_workers(g, [r[0], r[0]], rat, idx, val, cnt, ws)
    assert e.value.code == binding.ERR_INVALID
    plan.compress_workers(g, r, rat, idx, val, cnt, ws)
    torch.cuda.synchronize()
    assert plan.status().flags == 0 and int(cnt[1][0]) == plan.layers[0].n_tiles


def test_decompress_assign_ragged_layers(oracle):
    shapes = [(300, 515, 3, 3), (5, 5, 3, 3), (1, 1000, 1, 9), (77, 45, 3, 3), (64, 147, 1, 49), (1, 1, 3, 3),
              (40000, 3, 3, 3), (2, 70001, 3, 3), (131, 131, 7, 5)]
    tensors = [("t%d" % i, (s[0], s[1])) for i, s in enumerate(shapes)]
    plan = binding.Plan(shapes, alpha=0.5)
    sig = synth.log_uniform_scales(len(shapes), (31,))
    grads = synth.multi_worker_gradients(tensors, 2, (31,), sig)
    ratios = np.array([0.1, 1.0, 0.3, 0.02, 0.5, 1.0, 0.01, 0.2, 0.05], np.float32)
    zeros = [np.zeros(s[0] * s[1], np.float32) for s in shapes]
    payloads, refs_all = [], []
    for w in range(2):
        _, refs, gc = parity.compress_and_check(oracle, plan, shapes, grads[w], zeros, ratios, 0.5, what="w%d" % w)
        payloads.append(gc.payload())
        refs_all.append(oracle.CompressResult(layers=refs))
    d_dense = parity.dev(parity.to_arena(plan, [np.full(s[0] * s[1], -5.0, np.float32) for s in shapes]))
    plan.decompress_assign(payloads, d_dense, 0.5)
    torch.cuda.synchronize()
    ref = [np.full(s[0] * s[1], 9.0, np.float32) for s in shapes]
    oracle.decompress_assign(shapes, ref, refs_all, 0.5)
    out = d_dense.cpu().numpy()
    assert (out[parity.padding_mask(plan)] == parity.CANARY).all()
    for l, (got, want) in enumerate(zip(parity.from_arena(plan, out), ref)):
        np.testing.assert_array_equal(got.view(np.uint32), want.view(np.uint32), err_msg="layer %d" % l)


def test_bf16_gradients(oracle):
    shapes = [(300, 515, 3, 3), (128, 64 * 9, 1, 9), (1, 1000, 1, 9), (77, 45, 3, 3), (50, 400, 25, 25),
              (40, 480, 20, 30)]
    rng = np.random.default_rng(9)
    g = [synth.f32_to_bf16_bits((rng.standard_normal(r * c) * 1e-2).astype(np.float32)) for r, c, _, _ in shapes]
    res = [(rng.standard_normal(r * c) * 1e-3).astype(np.float32) for r, c, _, _ in shapes]
    plan = binding.Plan(shapes, grad_dtype=binding.RSDGC_BF16, alpha=0.5)
    parity.compress_and_check(oracle, plan, shapes, g, res, [0.02, 0.1, 0.5, 0.01, 0.2, 0.1], 0.5, what="bf16")


def test_repeated_runs_are_bit_identical(oracle):
    tensors = synth.resnet18_tensors()
    shapes = synth.layer_shapes(tensors)
    plan = binding.Plan(shapes, alpha=0.5)
    g = synth.laplace_layers(tensors, (4, 0), synth.log_uniform_scales(len(tensors), (4,)))
    g_arena = parity.to_arena(plan, g)
    ratios = torch.full((len(shapes),), 0.02, device="cuda:0")
    outs = []
    for rep in range(3):
        gc = parity.GpuCompress(plan, max_ratio=0.02)
        d_r = parity.dev(parity.to_arena(plan, [np.zeros(x.size, np.float32) for x in g]))
        st = gc.run(parity.dev(g_arena), d_r, ratios)
        assert st.flags == 0
        outs.append([t.cpu().numpy().copy() for t in (gc.idx, gc.val, gc.counts, gc.nsi, d_r)])
    for a, b in zip(outs[0], outs[1]):
        np.testing.assert_array_equal(a.view(np.uint32), b.view(np.uint32))
    for a, b in zip(outs[0], outs[2]):
        np.testing.assert_array_equal(a.view(np.uint32), b.view(np.uint32))


def test_compress_and_aggregate_replay_from_a_cuda_graph(oracle):
    """The whole per-iteration sequence is stream-ordered and reads nothing on the host, so it can
    be captured once and replayed: three replays on fresh gradients match the oracle."""
    tensors = synth.resnet18_tensors()[:30]
    shapes = synth.layer_shapes(tensors)
    plan = binding.Plan(shapes, alpha=0.5)
    ratio = 1 / 32
    ni, nv = plan.payload_bound(ratio)
    dev = "cuda:0"
    d_g = torch.zeros(plan.info.arena_elems, device=dev)
    d_r = torch.zeros(plan.info.arena_elems, device=dev)
    d_dense = torch.zeros(plan.info.arena_elems, device=dev)
    idx = torch.zeros(ni, dtype=torch.int32, device=dev)
    val = torch.zeros(nv, device=dev)
    cnt = torch.zeros(len(shapes), dtype=torch.int32, device=dev)
    ws = torch.empty(plan.info.workspace_bytes, dtype=torch.uint8, device=dev)
    ratios = torch.full((len(shapes),), ratio, device=dev)
    side = torch.cuda.Stream()
    with torch.cuda.stream(side):
        plan.compress(d_g, d_r, ratios, idx, val, cnt, workspace=ws)      # warm-up outside the capture
        plan.decompress_accumulate([(idx, val, cnt)], d_dense, 1.0)
    side.synchronize()
    d_r.zero_()
    d_dense.zero_()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        plan.compress(d_g, d_r, ratios, idx, val, cnt, workspace=ws)
        plan.decompress_accumulate([(idx, val, cnt)], d_dense, 1.0)
    scales = synth.log_uniform_scales(len(tensors), (11,))
    res = [np.zeros(synth.numel(s), np.float32) for _, s in tensors]
    dense_ref = [np.zeros(synth.numel(s), np.float32) for _, s in tensors]
    d_r.zero_()
    d_dense.zero_()
    for it in range(3):
        g = synth.laplace_layers(tensors, (11, it), scales)
        d_g.copy_(torch.from_numpy(parity.to_arena(plan, g, fill=0.0)))
        graph.replay()
        torch.cuda.synchronize()
        ref = oracle.compress(shapes, g, res, [ratio] * len(shapes), 0.5)
        oracle.decompress_accumulate(shapes, dense_ref, [ref], 1.0)
        res = [l.residual for l in ref.layers]
        k = int(ref.counts.sum())
        np.testing.assert_array_equal(cnt.cpu().numpy(), ref.counts)
        np.testing.assert_array_equal(idx.cpu().numpy()[:k], np.concatenate([l.idx for l in ref.layers]))
        for got, want in zip(parity.from_arena(plan, d_r.cpu().numpy()), res):
            np.testing.assert_array_equal(got.view(np.uint32), want.view(np.uint32))
        for got, want in zip(parity.from_arena(plan, d_dense.cpu().numpy()), dense_ref):
            np.testing.assert_array_equal(got.view(np.uint32), want.view(np.uint32))
    assert plan.status().flags == 0


def test_compress_workers_replay_from_a_cuda_graph():
    """The call that serves several workers lets their first passes run into one another (only the
    first waits for what precedes it in the stream).  Captured in a CUDA graph and replayed, it must
    give what the same calls give on a stream: three iterations, residuals carried, compared bit for bit."""
    tensors = synth.resnet18_tensors()
    shapes = synth.layer_shapes(tensors)
    dev, W, ratio = "cuda:0", 3, 1 / 32
    gen = torch.Generator(device=dev).manual_seed(77)
    outs = {}
    grads = None
    for mode in ("stream", "graph"):
        plan = binding.Plan(shapes, alpha=0.5)
        plan.reserve_workers(W)
        n = plan.info.arena_elems
        ni, nv = plan.payload_bound(ratio)
        if grads is None:
            grads = [[torch.randn(n, device=dev, generator=gen) * 1e-2 for _ in range(W)] for _ in range(3)]
        d_g = [torch.zeros(n, device=dev) for _ in range(W)]
        d_r = [torch.zeros(n, device=dev) for _ in range(W)]
        idx = [torch.zeros(ni, dtype=torch.int32, device=dev) for _ in range(W)]
        val = [torch.zeros(nv, device=dev) for _ in range(W)]
        cnt = [torch.zeros(len(shapes), dtype=torch.int32, device=dev) for _ in range(W)]
        ws = torch.empty(W * plan.info.workspace_bytes, dtype=torch.uint8, device=dev)
        ratios = torch.full((len(shapes),), ratio, device=dev)
        d_dense = torch.zeros(n, device=dev)

        def step():
            plan.compress_workers(d_g, d_r, ratios, idx, val, cnt, ws)
            plan.decompress_accumulate(list(zip(idx, val, cnt)), d_dense, 0.5)

        graph = None
        if mode == "graph":
            side = torch.cuda.Stream()
            with torch.cuda.stream(side):
                step()                                   # warm-up outside the capture
            side.synchronize()
            for t in d_r + [d_dense]:
                t.zero_()
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph):
                step()
            for t in d_r + [d_dense]:
                t.zero_()
        got = []
        for it in range(3):
            for w in range(W):
                d_g[w].copy_(grads[it][w])
            graph.replay() if graph is not None else step()
            torch.cuda.synchronize()
            got.append([t.cpu().numpy().copy() for t in idx + val + cnt + d_r + [d_dense]])
        assert plan.status().flags == 0
        outs[mode] = got
        plan.close()
    for a_it, b_it in zip(outs["stream"], outs["graph"]):
        for a, b in zip(a_it, b_it):
            np.testing.assert_array_equal(a.view(np.uint32), b.view(np.uint32))
    assert int(outs["graph"][2][2 * W].sum()) > 0


# ---------------------------------------------------------------------------------------------
# the ablation rows of Table I as settings of the same path: "Neighbor" only (alpha = 1), no
# "Dynamic" (one fixed ratio), and plain Top-k as the 1x1-neighborhood special case
# ---------------------------------------------------------------------------------------------

def test_topk_special_case_matches_library_topk(oracle):
    rows, cols = 700, 1031
    rng = np.random.default_rng(12)
    g = rng.standard_normal(rows * cols).astype(np.float32)
    r = (rng.standard_normal(rows * cols) * 0.1).astype(np.float32)
    shapes = [(rows, cols, 1, 1)]
    plan = binding.Plan(shapes, alpha=1.0)
    ratio = 0.01
    _, refs, gc = parity.compress_and_check(oracle, plan, shapes, [g], [r], [ratio], 1.0, max_ratio=ratio, what="top-k")
    v = torch.from_numpy(g) + torch.from_numpy(r)
    k = refs[0].k
    top = torch.topk(v.abs(), k).indices.numpy()
    got = gc.idx.cpu().numpy()[:k]
    av = np.abs(v.numpy())
    # the kept magnitudes are exactly the k largest; where the k-th magnitude is not tied the index
    # sets coincide as well
    np.testing.assert_array_equal(np.sort(av[got]), np.sort(av[top]))
    if (av == av[top].min()).sum() == 1:
        np.testing.assert_array_equal(got, np.sort(top))
    np.testing.assert_array_equal(gc.val.cpu().numpy()[:k], v.numpy()[got])


@pytest.mark.parametrize("alpha,shape", [(1.0, (640, 1152, 3, 3)), (0.0, (640, 1152, 3, 3)), (0.5, (192, 49, 1, 49)),
                                         (0.5, (448, 21, 7, 7)), (1.0, (448, 21, 7, 7))])
def test_ablation_variants_and_other_neighborhood_shapes(oracle, alpha, shape):
    rows, cols = shape[0], shape[1]
    rng = np.random.default_rng(13)
    g = (rng.standard_normal(rows * cols) * 1e-2).astype(np.float32)
    r = (rng.standard_normal(rows * cols) * 1e-2).astype(np.float32)
    plan = binding.Plan([shape], alpha=alpha)
    parity.compress_and_check(oracle, plan, [shape], [g], [r], [0.001], alpha, what="variant alpha=%g %r" % (alpha, shape))


# ---------------------------------------------------------------------------------------------
# momentum correction ahead of the accumulation (Eq. 12, first line)
# ---------------------------------------------------------------------------------------------

@pytest.mark.parametrize("bf16", [False, True])
def test_momentum_correction_five_iterations(oracle, bf16):
    shapes = [(300, 1032, 3, 3), (256 * 64, 9, 1, 9), (1, 777, 1, 9), (77, 45, 3, 3), (129, 4401, 3, 3),
              (2000, 1111, 3, 3)]                                         # the last two: register-staged kernel
    rng = np.random.default_rng(15)
    plan = binding.Plan(shapes, grad_dtype=binding.RSDGC_BF16 if bf16 else binding.RSDGC_F32, alpha=0.5,
                        flags=binding.KEEP_AT_LEAST_ONE | binding.MOMENTUM)
    res = [np.zeros(r * c, np.float32) for r, c, _, _ in shapes]
    vel = [np.zeros(r * c, np.float32) for r, c, _, _ in shapes]
    ratios = [0.02, 0.05, 0.5, 0.01, 0.03, 0.004]
    gc = parity.GpuCompress(plan, max_ratio=0.5)
    for it in range(5):
        g = [(rng.standard_normal(r * c) * 1e-2).astype(np.float32) for r, c, _, _ in shapes]
        if bf16:
            g = [synth.f32_to_bf16_bits(x) for x in g]
        gc.idx.fill_(-1)
        gc.val.fill_(float(parity.CANARY))
        res, refs, _ = parity.compress_and_check(oracle, plan, shapes, g, res, ratios, 0.5, gc=gc,
                                                 what="momentum it%d" % it, velocities=vel, momentum=0.9)
        vel = [r.velocity for r in refs]
    # a momentum plan refuses the plain entry point, and the other way round
    with pytest.raises(binding.RsdgcError):
        gc.run(parity.dev(parity.to_arena(plan, res)), parity.dev(parity.to_arena(plan, res)),
               torch.tensor(ratios, device="cuda:0"))
    plain = binding.Plan(shapes, alpha=0.5)
    with pytest.raises(binding.RsdgcError):
        parity.GpuCompress(plain).run(parity.dev(parity.to_arena(plain, res)), parity.dev(parity.to_arena(plain, res)),
                                      torch.tensor(ratios, device="cuda:0"),
                                      velocity=parity.dev(parity.to_arena(plain, res)), momentum=0.9)


# ---------------------------------------------------------------------------------------------
# payload with bfloat16 values: q = bfloat16(v) is sent, v - q stays in the accumulator
# ---------------------------------------------------------------------------------------------

@pytest.mark.parametrize("tail", TAILS)
def test_bf16_payload_three_iterations_and_aggregation(oracle, tail):
    shapes = [(300, 515, 3, 3), (256 * 16, 9, 1, 9), (1, 1000, 1, 9), (77, 45, 3, 3), (64, 147, 1, 49),
              (1200, 1536, 3, 3), (5, 5, 3, 3)]
    tensors = [("t%d" % i, (s[0], s[1])) for i, s in enumerate(shapes)]
    plan = binding.Plan(shapes, alpha=0.5, flags=binding.KEEP_AT_LEAST_ONE | binding.PAYLOAD_BF16 | tail)
    sig = synth.log_uniform_scales(len(shapes), (41,))
    ratios = np.array([1 / 16, 1 / 50, 0.3, 1.0, 0.1, 1 / 64, 0.5], np.float32)
    n_workers = 2
    res = [[np.zeros(s[0] * s[1], np.float32) for s in shapes] for _ in range(n_workers)]
    gcs = [parity.GpuCompress(plan) for _ in range(n_workers)]
    for it in range(3):
        grads = synth.multi_worker_gradients(tensors, n_workers, (41, it), sig)
        refs_all = []
        for w in range(n_workers):
            gcs[w].idx.fill_(-1)
            gcs[w].val.fill_(parity.CANARY16)
            res[w], refs, _ = parity.compress_and_check(oracle, plan, shapes, grads[w], res[w], ratios, 0.5,
                                                        gc=gcs[w], what="bf16 payload it%d w%d" % (it, w))
            refs_all.append(oracle.CompressResult(layers=refs))
    # what the receivers rebuild from the 16-bit payloads
    payloads = [gc.payload() for gc in gcs]
    rng = np.random.default_rng(9)
    dense0 = [(rng.standard_normal(s[0] * s[1]) * 1e-3).astype(np.float32) for s in shapes]
    d_dense = parity.dev(parity.to_arena(plan, dense0))
    plan.decompress_accumulate(payloads, d_dense, 0.5)
    d_assign = parity.dev(parity.to_arena(plan, dense0))
    plan.decompress_assign(payloads, d_assign, 0.5)
    torch.cuda.synchronize()
    ref_acc = [d.copy() for d in dense0]
    oracle.decompress_accumulate(shapes, ref_acc, refs_all, 0.5)
    ref_asg = [d.copy() for d in dense0]
    oracle.decompress_assign(shapes, ref_asg, refs_all, 0.5)
    for got, want in zip(parity.from_arena(plan, d_dense.cpu().numpy()), ref_acc):
        np.testing.assert_array_equal(got.view(np.uint32), want.view(np.uint32))
    for got, want in zip(parity.from_arena(plan, d_assign.cpu().numpy()), ref_asg):
        np.testing.assert_array_equal(got.view(np.uint32), want.view(np.uint32))
    # bytes: 4 per index + 2 per value
    k = int(payloads[0][2].sum())
    assert gcs[0].val.element_size() == 2 and k > 0


# ---------------------------------------------------------------------------------------------
# coordinate view of a payload: one arena position per value
# ---------------------------------------------------------------------------------------------

def test_payload_to_coo(oracle):
    shapes = [(300, 515, 3, 3), (256, 9, 1, 9), (1, 1000, 1, 9), (77, 45, 3, 3), (64, 147, 1, 49), (5, 5, 3, 3),
              (131, 131, 7, 5), (4, 4, 3, 3)]
    plan = binding.Plan(shapes, alpha=0.5)
    rng = np.random.default_rng(17)
    g = [(rng.standard_normal(s[0] * s[1]) * 1e-2).astype(np.float32) for s in shapes]
    zeros = [np.zeros(s[0] * s[1], np.float32) for s in shapes]
    ratios = np.array([0.1, 0.5, 0.2, 1.0, 0.3, 1.0, 0.25, 0.0], np.float32)
    _, refs, gc = parity.compress_and_check(oracle, plan, shapes, g, zeros, ratios, 0.5, what="coo")
    n_val = sum(r.val.size for r in refs)
    coo = torch.full((n_val + 8,), -7, dtype=torch.int64, device="cuda:0")
    plan.payload_to_coo(gc.idx, gc.counts, coo[:n_val])
    torch.cuda.synchronize()
    got = coo.cpu().numpy()
    assert (got[n_val:] == -7).all()                                  # nothing past the capacity given
    want = np.concatenate([oracle.payload_to_coo(s, r.idx, li.elem_offset)
                           for s, r, li in zip(shapes, refs, plan.layers)])
    np.testing.assert_array_equal(got[:n_val], want)
    # scattering the pairs into an arena gives the aggregation's result
    d_dense = torch.zeros(plan.info.arena_elems, device="cuda:0")
    ok = coo[:n_val] >= 0
    d_dense.index_put_((coo[:n_val][ok],), gc.val[:n_val][ok], accumulate=True)
    d_ref = torch.zeros(plan.info.arena_elems, device="cuda:0")
    plan.decompress_accumulate([gc.payload()], d_ref, 1.0)
    torch.cuda.synchronize()
    assert torch.equal(d_dense, d_ref)
    # a smaller capacity writes a prefix
    coo2 = torch.full((n_val,), -7, dtype=torch.int64, device="cuda:0")
    plan.payload_to_coo(gc.idx, gc.counts, coo2[:1000])
    torch.cuda.synchronize()
    assert torch.equal(coo2[:1000], coo[:1000]) and bool((coo2[1000:] == -7).all())


# ---------------------------------------------------------------------------------------------
# the exchange step (Eq. 2 Sync) through NCCL: one rank on one GPU, the collective really runs
# ---------------------------------------------------------------------------------------------

NCCL_CHILD = r"""
import os, sys
sys.path.insert(0, %r); sys.path.insert(0, os.path.join(%r, "tests"))
import numpy as np, torch
import torch.distributed as td
import oracle, parity
from paper_2312_17530_b200 import binding, sync, synth
td.init_process_group("nccl", rank=0, world_size=1)
torch.cuda.set_device(0)
shapes = [(300, 515, 3, 3), (256, 9, 1, 9), (1, 1000, 1, 9), (77, 45, 3, 3)]
tensors = [("t%%d" %% i, (s[0], s[1])) for i, s in enumerate(shapes)]
plan = binding.Plan(shapes, alpha=0.5)
n_local = 3
plan.reserve_workers(n_local)
ratios = np.array([0.1, 0.3, 0.2, 0.05], np.float32)
ni, nv = plan.payload_bound(0.3)
ex = sync.PayloadExchange(plan.n_layers, ni, nv, n_local, 1, 0, "cuda:0", always_gather=True)
sig = synth.log_uniform_scales(len(shapes), (61,))
grads = synth.multi_worker_gradients(tensors, n_local, (61,), sig)
zeros = [np.zeros(s[0] * s[1], np.float32) for s in shapes]
d_g = [parity.dev(parity.to_arena(plan, g)) for g in grads]
d_r = [parity.dev(parity.to_arena(plan, zeros)) for _ in range(n_local)]
views = [ex.local_views(w) for w in range(n_local)]
ws = torch.empty(n_local * plan.info.workspace_bytes, dtype=torch.uint8, device="cuda:0")
plan.compress_workers(d_g, d_r, torch.tensor(ratios, device="cuda:0"), [v[0] for v in views], [v[1] for v in views],
                      [v[2] for v in views], ws)
ex.exchange()
d_dense = torch.zeros(plan.info.arena_elems, device="cuda:0")
ex.aggregate(plan, d_dense, 0.5, assign=True)
torch.cuda.synchronize()
assert plan.status().flags == 0
refs = [oracle.compress(shapes, g, zeros, ratios, 0.5) for g in grads]
want = [np.zeros(s[0] * s[1], np.float32) for s in shapes]
oracle.decompress_assign(shapes, want, refs, 0.5)
for got, w in zip(parity.from_arena(plan, d_dense.cpu().numpy()), want):
    assert np.array_equal(got.view(np.uint32), w.view(np.uint32))
assert ex.recv.data_ptr() != ex.send.data_ptr() and torch.equal(ex.recv, ex.send)
td.destroy_process_group()
print("nccl exchange ok")
"""


def test_payload_exchange_through_nccl_one_rank():
    import os
    import socket
    import subprocess
    import sys

    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    env = dict(os.environ, RANK="0", LOCAL_RANK="0", WORLD_SIZE="1", MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    out = subprocess.run([sys.executable, "-c", NCCL_CHILD % (root, root)], env=env, capture_output=True, text=True,
                         timeout=300)
    assert out.returncode == 0 and "nccl exchange ok" in out.stdout, out.stdout + out.stderr


NCCL_GROUPED_CHILD = r"""
import os, sys
sys.path.insert(0, %r); sys.path.insert(0, os.path.join(%r, "tests"))
import numpy as np, torch
import torch.distributed as td
import oracle, parity
from paper_2312_17530_b200 import binding, sync, synth
td.init_process_group("nccl", rank=0, world_size=1)
torch.cuda.set_device(0)
shapes = [(300, 515, 3, 3), (256, 9, 1, 9), (1, 1000, 1, 9), (77, 45, 3, 3), (640, 1152, 3, 3), (1, 640, 1, 9), (200, 99, 3, 3)]
tensors = [("t%%d" %% i, (s[0], s[1])) for i, s in enumerate(shapes)]
ratios = np.array([0.1, 0.3, 0.2, 0.05, 1 / 64, 0.0, 0.02], np.float32)
n_local = 2
groups = sync.split_layers(shapes, 3)
plans = [binding.Plan(shapes[lo:hi], alpha=0.5) for lo, hi in groups]
gx = sync.GroupedExchange(shapes, groups, plans, n_local, 1, 0, "cuda:0", always_gather=True)
gx.set_ratios(ratios.tolist())
sig = synth.log_uniform_scales(len(shapes), (62,))
res = [[np.zeros(s[0] * s[1], np.float32) for s in shapes] for _ in range(n_local)]
d_res = [[parity.dev(parity.to_arena(p, res[w][lo:hi])) for w in range(n_local)] for p, (lo, hi) in zip(plans, groups)]
d_rat = [torch.tensor(ratios[lo:hi], device="cuda:0") for lo, hi in groups]
ws = [torch.empty(n_local * max(p.info.workspace_bytes, 16), dtype=torch.uint8, device="cuda:0") for p in plans]
dense = [torch.full((p.info.arena_elems,), float("nan"), device="cuda:0") for p in plans]
for it in range(2):                                  # residuals carried; the second step reuses streams and events
    grads = synth.multi_worker_gradients(tensors, n_local, (62, it), sig)
    d_g = [[parity.dev(parity.to_arena(p, grads[w][lo:hi])) for w in range(n_local)] for p, (lo, hi) in zip(plans, groups)]
    gx.step(d_g, d_res, d_rat, ws, dense, scale=0.5, assign=True)
    torch.cuda.synchronize()
    assert all(p.status().flags == 0 for p in plans)
    refs = [oracle.compress(shapes, grads[w], res[w], ratios, 0.5) for w in range(n_local)]
    want = [np.zeros(s[0] * s[1], np.float32) for s in shapes]
    oracle.decompress_assign(shapes, want, refs, 0.5)        # the ungrouped aggregation of all workers
    for p, (lo, hi), d in zip(plans, groups, dense):
        for got, w in zip(parity.from_arena(p, d.cpu().numpy()), want[lo:hi]):
            assert np.array_equal(got.view(np.uint32), w.view(np.uint32))
    res = [[l.residual for l in r.layers] for r in refs]
    for g, (p, (lo, hi)) in enumerate(zip(plans, groups)):
        for w in range(n_local):
            for got, w_res in zip(parity.from_arena(p, d_res[g][w].cpu().numpy()), res[w][lo:hi]):
                assert np.array_equal(got.view(np.uint32), w_res.view(np.uint32))
k = [oracle.keep_count(oracle.tile_count(*s), float(q)) for s, q in zip(shapes, ratios)]
# exactly what is sent plus at most 15 bytes of padding per section
assert gx.message_bytes() <= n_local * (4 * (len(shapes) + sum(k) + sum(a * s[2] * s[3] for a, s in zip(k, shapes))) + 45 * len(groups))
td.destroy_process_group()
print("nccl grouped exchange ok")
"""


def test_grouped_overlapped_exchange_through_nccl_one_rank():
    """Layer groups: group g + 1 is compressed while group g's exact-size payload message goes through a
    real NCCL all-gather on a second stream, then the groups are aggregated in order; the dense result
    equals the oracle's ungrouped aggregation bit for bit, over two iterations with carried residuals."""
    import os
    import socket
    import subprocess
    import sys

    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    env = dict(os.environ, RANK="0", LOCAL_RANK="0", WORLD_SIZE="1", MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    out = subprocess.run([sys.executable, "-c", NCCL_GROUPED_CHILD % (root, root)], env=env, capture_output=True,
                         text=True, timeout=300)
    assert out.returncode == 0 and "nccl grouped exchange ok" in out.stdout, out.stdout + out.stderr


# ---------------------------------------------------------------------------------------------
# more workers than one launch serves (groups of 16): compress_workers and the aggregation
# ---------------------------------------------------------------------------------------------

def test_eighteen_workers_in_one_call(oracle):
    shapes = [(120, 99, 3, 3), (64, 9, 1, 9), (1, 100, 1, 9)]
    tensors = [("t%d" % i, (s[0], s[1])) for i, s in enumerate(shapes)]
    plan = binding.Plan(shapes, alpha=0.5)
    n_workers = 18
    sig = synth.log_uniform_scales(len(shapes), (71,))
    grads = synth.multi_worker_gradients(tensors, n_workers, (71,), sig)
    ratios = np.array([0.1, 0.25, 0.5], np.float32)
    zeros = [[np.zeros(s[0] * s[1], np.float32) for s in shapes] for _ in range(n_workers)]
    _, refs, payloads = parity.compress_workers_and_check(oracle, plan, shapes, grads, zeros, ratios, 0.5,
                                                          what="18 workers")
    rng = np.random.default_rng(72)
    dense0 = [(rng.standard_normal(s[0] * s[1]) * 1e-3).astype(np.float32) for s in shapes]
    d_dense = parity.dev(parity.to_arena(plan, dense0))
    plan.decompress_accumulate(payloads, d_dense, 0.125)          # two launches: 16 + 2 workers, in order
    d_assign = parity.dev(parity.to_arena(plan, dense0))
    plan.decompress_assign(payloads, d_assign, 0.125)
    torch.cuda.synchronize()
    results = [oracle.CompressResult(layers=r) for r in refs]
    want = [d.copy() for d in dense0]
    oracle.decompress_accumulate(shapes, want, results, 0.125)
    for got, w in zip(parity.from_arena(plan, d_dense.cpu().numpy()), want):
        np.testing.assert_array_equal(got.view(np.uint32), w.view(np.uint32))
    want = [d.copy() for d in dense0]
    oracle.decompress_assign(shapes, want, results, 0.125)
    for got, w in zip(parity.from_arena(plan, d_assign.cpu().numpy()), want):
        np.testing.assert_array_equal(got.view(np.uint32), w.view(np.uint32))

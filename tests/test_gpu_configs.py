"""GPU parity on the full-size workloads: the VGG-19-shaped set with 4 workers and their
aggregation (the configuration the benchmark times), the ResNet-50-shaped set over 100 iterations
with drifting scales and refreshed ratios, and the single-matrix sweep from 1M to 1B elements in
binary32 and bfloat16.  Sizes the oracle can sort are compared through its own selection; above that,
every key still goes through the oracle's indicator and the kept set is the oracle's rule evaluated with
a partition instead of its full sort."""
import numpy as np
import pytest
import torch

from paper_2312_17530_b200 import binding, synth

import parity

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _lib():
    assert torch.cuda.is_available(), "these tests need a CUDA device"
    binding.lib()


# ---------------------------------------------------------------------------------------------
# config 3: VGG-19-shaped set, 4 workers, keep 1/64, aggregation into one dense buffer
# ---------------------------------------------------------------------------------------------

def test_vgg19_four_workers_full_size(oracle):
    tensors = synth.vgg19_tensors()
    shapes = synth.layer_shapes(tensors)
    plan = binding.Plan(shapes, alpha=0.5)
    assert plan.info.total_elems == 139_754_605
    sig = synth.log_uniform_scales(len(tensors), (3,))
    grads = synth.multi_worker_gradients(tensors, 4, (3, 0), sig)        # the benchmark's rank-0 inputs
    ratios = np.full(len(shapes), 1 / 64, np.float32)
    zeros = [np.zeros(synth.numel(s), np.float32) for _, s in tensors]
    payloads, refs_all = [], []
    for w in range(4):
        _, refs, gc = parity.compress_and_check(oracle, plan, shapes, grads[w], zeros, ratios, 0.5,
                                                what="vgg worker %d" % w, max_ratio=1 / 64)
        payloads.append(gc.payload())
        refs_all.append(oracle.CompressResult(layers=refs))
        n_bytes = 4 * sum(r.idx.size + r.val.size for r in refs)
        assert 50 < 4 * plan.info.total_elems / n_bytes < 60                # "more than 50x" in bytes
    d_dense = torch.zeros(plan.info.arena_elems, device="cuda:0")
    plan.decompress_accumulate(payloads, d_dense, 1.0)
    torch.cuda.synchronize()
    dense_ref = [np.zeros(synth.numel(s), np.float32) for _, s in tensors]
    oracle.decompress_accumulate(shapes, dense_ref, refs_all, 1.0)
    for got, ref in zip(parity.from_arena(plan, d_dense.cpu().numpy()), dense_ref):
        np.testing.assert_array_equal(got.view(np.uint32), ref.view(np.uint32))
    d_dense2 = torch.full((plan.info.arena_elems,), float("nan"), device="cuda:0")
    plan.decompress_assign(payloads, d_dense2, 1.0)          # zero fill fused into the same launch
    torch.cuda.synchronize()
    assert torch.equal(d_dense.view(torch.int32)[~torch.from_numpy(parity.padding_mask(plan)).cuda()],
                       d_dense2.view(torch.int32)[~torch.from_numpy(parity.padding_mask(plan)).cuda()])
    del d_dense2
    # the workers' selections overlap (shared gradient component): the scatter-add does collide
    fc6_tiles = np.concatenate([refs_all[w].layers[32].idx for w in range(4)])
    assert int((np.bincount(fc6_tiles) > 1).sum()) > 1000

    # the same four workers through one rsdgc_compress_workers() call (what the benchmark times):
    # bit-identical payloads and residuals to the per-worker calls checked above
    plan.reserve_workers(4)
    d_g = [parity.dev(parity.to_arena(plan, grads[w])) for w in range(4)]
    d_r = [torch.zeros(plan.info.arena_elems, device="cuda:0") for _ in range(4)]
    ni, nv = plan.payload_bound(1 / 64)
    idx = [torch.full((ni,), -1, dtype=torch.int32, device="cuda:0") for _ in range(4)]
    val = [torch.full((nv,), float(parity.CANARY), device="cuda:0") for _ in range(4)]
    cnt = [torch.zeros(plan.n_layers, dtype=torch.int32, device="cuda:0") for _ in range(4)]
    ws = torch.empty(4 * plan.info.workspace_bytes, dtype=torch.uint8, device="cuda:0")
    plan.compress_workers(d_g, d_r, torch.tensor(ratios, device="cuda:0"), idx, val, cnt, ws)
    torch.cuda.synchronize()
    assert plan.status().flags == 0
    for w in range(4):
        assert torch.equal(idx[w], payloads[w][0]) and torch.equal(cnt[w], payloads[w][2])
        assert torch.equal(val[w].view(torch.int32), payloads[w][1].view(torch.int32))
        res = parity.from_arena(plan, d_r[w].cpu().numpy())
        for l in (0, 17, 32, 34, 36, 37):
            np.testing.assert_array_equal(res[l].view(np.uint32), refs_all[w].layers[l].residual.view(np.uint32))


# ---------------------------------------------------------------------------------------------
# config 4: ResNet-50-shaped set, 100 iterations, scales drift, ratios refreshed every 10
# ---------------------------------------------------------------------------------------------

def test_resnet50_hundred_iterations(oracle):
    tensors = synth.resnet50_tensors()
    shapes = synth.layer_shapes(tensors)
    L = len(tensors)
    plan = binding.Plan(shapes, alpha=0.5)
    base_w = synth.synthetic_weights(tensors, (4,))
    b0 = synth.log_uniform_scales(L, (4,))
    g_walk = synth.random_walk(L, 100, (4, 1), 0.1)
    w_walk = synth.random_walk(L, 100, (4, 2), 0.05)
    res = [np.zeros(synth.numel(s), np.float32) for _, s in tensors]
    gc = parity.GpuCompress(plan, max_ratio=1.0)
    d_ratios = torch.zeros(L, device="cuda:0")
    ratios_ref = ratios_first = None
    for it in range(100):
        if it % 10 == 0:
            w = [bw * np.float32(np.exp(w_walk[it, l])) for l, bw in enumerate(base_w)]
            plan.update_ratios(parity.dev(parity.to_arena(plan, w)), 1 / 50, d_ratios)
            torch.cuda.synchronize()
            ratios_new, surv, n_keep = oracle.update_ratios(w, 1 / 50)
            np.testing.assert_array_equal(d_ratios.cpu().numpy(), ratios_new)
            if ratios_first is None:
                ratios_first = ratios_new
            elif it == 50:
                assert not np.array_equal(ratios_new, ratios_first)      # the rule does track the drift
            ratios_ref = ratios_new
        g = synth.laplace_layers(tensors, (4, it), b0 * np.exp(g_walk[it]))
        gc.idx.fill_(-1)
        gc.val.fill_(float(parity.CANARY))
        res, refs, _ = parity.compress_and_check(oracle, plan, shapes, g, res, ratios_ref, 0.5, gc=gc,
                                                 what="resnet50 it%d" % it)


# ---------------------------------------------------------------------------------------------
# config 5: single matrices, 1M .. 1B elements, binary32 and bfloat16, keep 1/10, 1/100, 1/1000
# ---------------------------------------------------------------------------------------------

def _sweep_inputs(rows, cols, bf16):
    x = synth.clustered_matrix(rows, cols, seed=5)
    return synth.f32_to_bf16_bits(x) if bf16 else x


@pytest.mark.parametrize("rows,cols", [(1024, 1024), (4096, 4096), (2450, 400), (7840, 1280)])
@pytest.mark.parametrize("bf16", [False, True])
def test_sweep_small_full_oracle(oracle, rows, cols, bf16):
    shapes = [(rows, cols, 3, 3)]
    g = _sweep_inputs(rows, cols, bf16)
    plan = binding.Plan(shapes, grad_dtype=binding.RSDGC_BF16 if bf16 else binding.RSDGC_F32, alpha=0.5)
    zeros = [np.zeros(rows * cols, np.float32)]
    for ratio in synth.SWEEP_RATIOS:
        parity.compress_and_check(oracle, plan, shapes, [g], zeros, [ratio], 0.5, max_ratio=ratio,
                                  what="sweep %dx%d bf16=%s 1/%d" % (rows, cols, bf16, round(1 / ratio)))


@pytest.mark.parametrize("rows,cols,bf16,ratio", [(8192, 8192, False, 1 / 100), (25088, 4096, False, 1 / 1000)])
def test_sweep_medium_full_oracle(oracle, rows, cols, bf16, ratio):
    shapes = [(rows, cols, 3, 3)]
    g = _sweep_inputs(rows, cols, bf16)
    plan = binding.Plan(shapes, grad_dtype=binding.RSDGC_BF16 if bf16 else binding.RSDGC_F32, alpha=0.5)
    parity.compress_and_check(oracle, plan, shapes, [g], [np.zeros(rows * cols, np.float32)], [ratio], 0.5,
                              max_ratio=ratio, what="sweep %dx%d" % (rows, cols))


# (rows, cols, dtypes, ratios): every key of the layer goes through the oracle; one input per shape, the
# bfloat16 variant is the rounded binary32 draw; all three ratios at 268 M elements in both dtypes, the
# 1 B-element matrices in both dtypes
LARGE = [(8192, 8192, (True,), (1 / 10,)),
         (25088, 4096, (True,), (1 / 100,)),
         (16384, 16384, (False, True), synth.SWEEP_RATIOS),
         (32768, 32768, (False, True), (1 / 100,)),
         (78400, 12800, (False, True), (1 / 1000,))]


@pytest.mark.parametrize("rows,cols,dtypes,ratios", LARGE, ids=["%dx%d" % (c[0], c[1]) for c in LARGE])
def test_sweep_large_every_key(oracle, rows, cols, dtypes, ratios):
    shape = (rows, cols, 3, 3)
    x = synth.clustered_matrix(rows, cols, seed=5)
    zeros = np.zeros(rows * cols, np.float32)
    for bf16 in dtypes:
        g = synth.f32_to_bf16_bits(x) if bf16 else x
        ref = parity.LargeLayerReference(oracle, shape, g, zeros, 0.5)
        plan = binding.Plan([shape], grad_dtype=binding.RSDGC_BF16 if bf16 else binding.RSDGC_F32, alpha=0.5)
        li = plan.layers[0]
        d_g = parity.dev(parity.to_arena(plan, [g], np.uint16 if bf16 else np.float32))
        for ratio in ratios:
            gc = parity.GpuCompress(plan, max_ratio=ratio)
            d_r = torch.zeros(plan.info.arena_elems, device="cuda:0")        # a real buffer, still read
            st = gc.run(d_g, d_r, torch.tensor([ratio], dtype=torch.float32, device="cuda:0"))
            assert st.flags == 0
            k = int(gc.counts.cpu().numpy()[0])
            nsi = gc.nsi.cpu().numpy()[:li.n_tiles]
            idx = gc.idx.cpu().numpy()[:k]
            val = gc.val.cpu().numpy()[:k * 9]
            assert (gc.idx.cpu().numpy()[k:] == -1).all() and (gc.val.cpu().numpy()[k * 9:] == parity.CANARY).all()
            res = d_r.cpu().numpy()[:rows * cols]
            del gc, d_r
            torch.cuda.empty_cache()
            ref.check(float(np.float32(ratio)), nsi, k, idx, val, res,
                      what="sweep %dx%d bf16=%s 1/%d" % (rows, cols, bf16, round(1 / ratio)))
            del nsi, idx, val, res
        del d_g, plan, ref, g
        torch.cuda.empty_cache()

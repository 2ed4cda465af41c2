"""rsdgc_update_ratios_noalloc(): the ratio rule for callers that are not allowed to allocate
device memory (code running under an open stream capture, runtimes that own all device memory
through their own pool, loops that cannot take an allocation's implicit synchronisation).

The entry point keeps its scratch in a fixed array inside the library instead of in a plan, so
this test calls it through the C ABI and requires the same ratios, bit for bit, as the plan-based
rsdgc_update_ratios() on the same weights AND as the CPU oracle's ratio rule (the two GPU kernels are
close relatives, so agreement between them alone would not see a mistake they share) -- twice in a
row with different inputs, because the array is shared by all calls and still holds the previous
call's contents when the next one starts.
This file is collected last on purpose: a failure here cannot hide a failure elsewhere.
"""
import numpy as np
import pytest
import torch

from paper_2312_17530_b200 import binding, synth

pytestmark = pytest.mark.gpu


def _weights_arena(plan, weights):
    a = np.zeros(plan.info.arena_elems, np.float32)
    for li, w in zip(plan.layers, weights):
        a[li.elem_offset:li.elem_offset + w.size] = w
    return torch.from_numpy(a).to("cuda:0")


def test_noalloc_matches_plan_based_entry_point_twice_in_a_row(oracle):
    assert torch.cuda.is_available()
    tensors = synth.resnet18_tensors()[:binding.NOALLOC_MAX_LAYERS - 2] + [("tail.weight", (1000, 37)),
                                                                           ("tail.bias", (5,))]
    assert len(tensors) == binding.NOALLOC_MAX_LAYERS
    shapes = synth.layer_shapes(tensors)
    plan = binding.Plan(shapes, alpha=0.5)
    offsets = [li.elem_offset for li in plan.layers]
    sizes = [li.rows * li.cols for li in plan.layers]
    mem_before = torch.cuda.memory_allocated()
    for call, (key, rho) in enumerate((((7,), 1 / 50), ((8,), 0.3))):
        weights = synth.synthetic_weights(tensors, key)
        if call == 1:
            weights[5][:] = 0.25            # a layer of equal magnitudes: ties are split by position
            weights[20][:] = -0.25
        d_w = _weights_arena(plan, weights)
        want = torch.full((len(shapes),), -1.0, device="cuda:0")
        got = torch.full((len(shapes),), -2.0, device="cuda:0")
        plan.update_ratios(d_w, rho, want)
        torch.cuda.synchronize()
        free_before = torch.cuda.mem_get_info()[0]      # the driver's view: sees any cudaMalloc in the library
        binding.update_ratios_noalloc(d_w, offsets, sizes, rho, got)
        torch.cuda.synchronize()
        assert torch.cuda.mem_get_info()[0] == free_before
        np.testing.assert_array_equal(got.cpu().numpy(), want.cpu().numpy())
        ref_ratios, survivors, n_keep = oracle.update_ratios(weights, rho)
        np.testing.assert_array_equal(got.cpu().numpy(), ref_ratios)
        assert int(survivors.sum()) == n_keep
        assert 0.0 < float(got.max()) <= 1.0
        del d_w, want, got
    assert torch.cuda.memory_allocated() == mem_before


def test_noalloc_rejects_what_does_not_fit():
    w = torch.zeros(1024, device="cuda:0")
    out = torch.zeros(binding.NOALLOC_MAX_LAYERS + 1, device="cuda:0")
    n = binding.NOALLOC_MAX_LAYERS + 1
    with pytest.raises(binding.RsdgcError) as e:
        binding.update_ratios_noalloc(w, [4 * i for i in range(n)], [4] * n, 0.5, out)
    assert e.value.code == binding.ERR_CAPACITY and "beyond" in str(e.value)
    with pytest.raises(binding.RsdgcError) as e:
        binding.update_ratios_noalloc(w, [0], [1 << 31], 0.5, out)
    assert e.value.code == binding.ERR_CAPACITY
    with pytest.raises(binding.RsdgcError) as e:
        binding.update_ratios_noalloc(w, [2], [8], 0.5, out)
    assert e.value.code == binding.ERR_ALIGNMENT
    with pytest.raises(binding.RsdgcError) as e:
        binding.update_ratios_noalloc(w, [], [], 0.5, out)
    assert e.value.code == binding.ERR_INVALID

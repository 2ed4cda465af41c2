"""Tensor-shape tables and seeded draws (host logic only)."""
import numpy as np

from paper_2312_17530_b200 import synth


def test_network_tensor_tables():
    r18, r50, vgg = synth.resnet18_tensors(), synth.resnet50_tensors(), synth.vgg19_tensors()
    assert len(r18) == 62 and sum(synth.numel(s) for _, s in r18) == 11_689_512
    assert len(r50) == 161 and sum(synth.numel(s) for _, s in r50) == 25_557_032
    assert len(vgg) == 38 and sum(synth.numel(s) for _, s in vgg) == 139_754_605
    assert sum(1 for _, s in r18 if len(s) == 4) == 20 and sum(1 for _, s in r50 if len(s) == 4) == 53


def test_default_views():
    assert synth.default_view((64, 3, 7, 7)) == (192, 49, 1, 49)
    assert synth.default_view((128, 64, 3, 3)) == (8192, 9, 1, 9)
    assert synth.default_view((256, 64, 1, 1)) == (256, 64, 3, 3)
    assert synth.default_view((25088, 4096)) == (25088, 4096, 3, 3)
    assert synth.default_view((64,)) == (1, 64, 1, 9)


def test_draws_are_seeded_and_shaped():
    a = synth.clustered_matrix(512, 512, seed=0)
    b = synth.clustered_matrix(512, 512, seed=0)
    assert a.dtype == np.float32 and a.size == 262144 and (a == b).all()
    assert 3e-4 < np.median(np.abs(a)) < 2e-3 and np.abs(a).max() > 0.05   # boosted patches present
    t = synth.vgg19_tensors()[:4]
    g = synth.multi_worker_gradients(t, 2, (0,), np.full(4, 1e-3))
    assert len(g) == 2 and all(x.size == synth.numel(s) for x, (_, s) in zip(g[0], t))
    c = np.corrcoef(g[0][2], g[1][2])[0, 1]
    assert 0.3 < c < 0.7                                                    # shared component
    bits = synth.f32_to_bf16_bits(np.array([1.0, 1.00390625, -2.5, 3.0e38], np.float32))
    assert bits.tolist() == [0x3F80, 0x3F80, 0xC020, 0x7F62]

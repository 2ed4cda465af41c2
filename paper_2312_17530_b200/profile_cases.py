"""Small, named cases of the compression path for profiler captures and quick timings.

The benchmark's workload (4 workers x 140 M elements) is too large for a multi-pass profiler capture;
these cases run the same kernels on inputs that stay within a few GB: the largest layer of the
VGG-19-shaped set alone (binary32 or bfloat16 gradients, 1 or 4 workers with their aggregation), and
the ResNet-shaped sets.  Inputs are the seeded synthetic draws of ``synth``.

    python -m paper_2312_17530_b200.profile_cases --case fc6_f32 --iters 3
"""
from __future__ import annotations

import argparse
import json
import statistics
import sys

import numpy as np

CASES = ("fc6_f32", "fc6_bf16", "fc6_4workers", "resnet18", "resnet50", "single_512")


def build_case(name: str):
    """(shapes, per-worker per-layer gradients, grad dtype, keep ratio)."""
    from . import binding, synth

    if name.startswith("fc6"):
        tensors = [t for t in synth.vgg19_tensors() if t[0] == "fc6.weight"]
        n_workers = 4 if name == "fc6_4workers" else 1
        grads = synth.multi_worker_gradients(tensors, n_workers, (3, 0), synth.log_uniform_scales(1, (3,)))
        dtype = binding.RSDGC_BF16 if name == "fc6_bf16" else binding.RSDGC_F32
        if dtype == binding.RSDGC_BF16:
            grads = [[synth.f32_to_bf16_bits(g) for g in worker] for worker in grads]
        return synth.layer_shapes(tensors), grads, dtype, 1.0 / 64.0
    if name in ("resnet18", "resnet50"):
        tensors = getattr(synth, name + "_tensors")()
        grads = [synth.laplace_layers(tensors, (4, 0), synth.log_uniform_scales(len(tensors), (4,)))]
        return synth.layer_shapes(tensors), grads, binding.RSDGC_F32, 1.0 / 50.0
    if name == "single_512":
        return [(512, 512, 3, 3)], [[synth.clustered_matrix(512, 512, seed=0)]], binding.RSDGC_F32, 1.0 / 64.0
    raise ValueError(name)


def main() -> int:
    ap = argparse.ArgumentParser(description=__doc__.split("\n")[0])
    ap.add_argument("--case", choices=CASES, required=True)
    ap.add_argument("--iters", type=int, default=3, help="timed iterations (after two warm-up iterations)")
    ap.add_argument("--chained", action="store_true", help="plan flag RSDGC_NO_FUSED_TAIL")
    args = ap.parse_args()

    import torch

    from . import binding

    binding.lib()
    dev = torch.device("cuda", 0)
    shapes, grads, dtype, ratio = build_case(args.case)
    flags = binding.KEEP_AT_LEAST_ONE | (binding.NO_FUSED_TAIL if args.chained else 0)
    plan = binding.Plan(shapes, grad_dtype=dtype, alpha=0.5, flags=flags, device=0)
    W = len(grads)
    plan.reserve_workers(W)

    def arena(per_layer):
        a = np.zeros(plan.info.arena_elems, np.uint16 if dtype == binding.RSDGC_BF16 else np.float32)
        for li, x in zip(plan.layers, per_layer):
            a[li.elem_offset:li.elem_offset + x.size] = x
        t = torch.from_numpy(a)
        return (t.view(torch.bfloat16) if dtype == binding.RSDGC_BF16 else t).to(dev)

    d_g = [arena(g) for g in grads]
    d_r = [torch.zeros(plan.info.arena_elems, device=dev) for _ in range(W)]
    ni, nv = plan.payload_bound(ratio)
    idx = [torch.zeros(ni, dtype=torch.int32, device=dev) for _ in range(W)]
    val = [torch.zeros(nv, device=dev) for _ in range(W)]
    cnt = [torch.zeros(plan.n_layers, dtype=torch.int32, device=dev) for _ in range(W)]
    ws = torch.empty(W * plan.info.workspace_bytes, dtype=torch.uint8, device=dev)
    ratios = torch.full((plan.n_layers,), ratio, device=dev)
    dense = torch.zeros(plan.info.arena_elems, device=dev)
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)   # larger than L2
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(3)]
    t_compress, t_aggregate = [], []
    for it in range(2 + args.iters):
        flush.zero_()
        ev[0].record()
        if W == 1:
            plan.compress(d_g[0], d_r[0], ratios, idx[0], val[0], cnt[0], workspace=ws)
        else:
            plan.compress_workers(d_g, d_r, ratios, idx, val, cnt, ws)
        ev[1].record()
        plan.decompress_accumulate(list(zip(idx, val, cnt)), dense, 1.0)
        ev[2].record()
        torch.cuda.synchronize()
        if it >= 2:
            t_compress.append(ev[0].elapsed_time(ev[1]) * 1e3)
            t_aggregate.append(ev[1].elapsed_time(ev[2]) * 1e3)
    st = plan.status()
    print(json.dumps({"case": args.case, "elements": int(plan.info.total_elems), "layers": plan.n_layers, "workers": W,
                      "fused_tail_ctas": int(len(plan.tail_slices()[0])), "status_flags": int(st.flags),
                      "compress_us_median": statistics.median(t_compress),
                      "aggregate_us_median": statistics.median(t_aggregate), "payload_tiles": int(st.idx_needed)}))
    return 0 if st.flags == 0 else 1


if __name__ == "__main__":
    sys.exit(main())

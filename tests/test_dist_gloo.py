"""The N>1 plumbing of the benchmark on CPU: two gloo ranks, barrier, MAX of the elapsed time,
SUM of the units, disjoint worker ids."""
import os
import socket
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

CHILD = r"""
import sys
sys.path.insert(0, %r)
from paper_2312_17530_b200 import dist
rank, local_rank, world = dist.init("gloo")
assert world == 2 and rank in (0, 1)
dist.barrier()
ids = dist.worker_ids(rank, 4)
assert ids == list(range(4 * rank, 4 * rank + 4))
value, t = dist.aggregate_throughput(units_this_rank=100.0 * (rank + 1), elapsed_s_this_rank=1.0 + rank)
assert t == 2.0 and value == 150.0, (value, t)
assert dist.max_over_ranks(-1.0 - rank) == -1.0
dist.barrier()
dist.finalize()
print("rank %%d ok" %% rank)
"""


def test_two_gloo_ranks():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    procs = []
    for rank in range(2):
        env = dict(os.environ, RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE="2", MASTER_ADDR="127.0.0.1",
                   MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, "-c", CHILD % ROOT], env=env, stdout=subprocess.PIPE,
                                      stderr=subprocess.STDOUT, text=True))
    for rank, p in enumerate(procs):
        out, _ = p.communicate(timeout=120)
        assert p.returncode == 0, out
        assert "rank %d ok" % rank in out


def test_single_process_needs_no_process_group():
    from paper_2312_17530_b200 import dist

    assert dist.env_world() == (0, 0, 1) or int(os.environ.get("WORLD_SIZE", "1")) > 1
    assert dist.max_over_ranks(3.5) == 3.5 and dist.aggregate_throughput(10.0, 2.0) == (5.0, 2.0)


# ---------------------------------------------------------------------------------------------
# the payload exchange (Eq. 2 Sync) between two ranks, on CPU: packed all-gather, then the
# oracle aggregates what arrived; both ranks must end with the same dense gradient
# ---------------------------------------------------------------------------------------------

SYNC_CHILD = r"""
import sys
sys.path.insert(0, %r)
import numpy as np, torch
import torch.distributed as td
import oracle
from paper_2312_17530_b200 import dist, sync, synth
rank, local_rank, world = dist.init("gloo")
shapes = [(30, 41, 3, 3), (16, 9, 1, 9), (1, 50, 1, 9)]
tensors = [("t%%d" %% i, (s[0], s[1])) for i, s in enumerate(shapes)]
ratios = [0.25, 0.5, 0.2]
n_local = 2
def payloads_of(r):
    sig = synth.log_uniform_scales(len(shapes), (51,))
    grads = synth.multi_worker_gradients(tensors, n_local, (51, r), sig)
    zeros = [np.zeros(s[0] * s[1], np.float32) for s in shapes]
    return [oracle.compress(shapes, g, zeros, ratios, 0.5) for g in grads]
mine = payloads_of(rank)
ni = sum(int(oracle.keep_count(oracle.tile_count(*s), q)) for s, q in zip(shapes, ratios)) + 3
nv = sum(int(oracle.keep_count(oracle.tile_count(*s), q)) * s[2] * s[3] for s, q in zip(shapes, ratios)) + 5
ex = sync.PayloadExchange(len(shapes), ni, nv, n_local, world, rank, "cpu")
for w, res in enumerate(mine):
    idx, val, cnt = ex.local_views(w)
    i = np.concatenate([l.idx for l in res.layers]); v = np.concatenate([l.val for l in res.layers])
    idx[:i.size] = torch.from_numpy(i); val[:v.size] = torch.from_numpy(v); cnt[:] = torch.from_numpy(res.counts)
ex.exchange()
got = ex.gathered_views()
assert len(got) == world * n_local
dense = [np.zeros(s[0] * s[1], np.float32) for s in shapes]
for r in range(world):
    for w, res in enumerate(payloads_of(r)):        # what rank r must have sent, recomputed here
        idx, val, cnt = got[r * n_local + w]
        assert np.array_equal(cnt.numpy(), res.counts)
        i = np.concatenate([l.idx for l in res.layers]); v = np.concatenate([l.val for l in res.layers])
        assert np.array_equal(idx.numpy()[:i.size], i) and np.array_equal(val.numpy()[:v.size].view(np.uint32), v.view(np.uint32))
        # aggregate from the received bytes, in global worker order
        io = vo = 0
        for l, s in enumerate(shapes):
            k = int(cnt[l]); slot = s[2] * s[3]
            oracle.decompress_into(dense[l], s, idx.numpy()[io:io + k], val.numpy()[vo:vo + k * slot], 0.25)
            io += k; vo += k * slot
flat = torch.from_numpy(np.concatenate(dense)).double()
lo, hi = flat.clone(), flat.clone()
td.all_reduce(lo, op=td.ReduceOp.MIN); td.all_reduce(hi, op=td.ReduceOp.MAX)
assert torch.equal(lo, hi) and float(flat.abs().sum()) > 0      # every replica holds the same gradient
dist.barrier()
dist.finalize()
print("rank %%d ok" %% rank)
"""


def test_payload_exchange_two_gloo_ranks():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    procs = []
    for rank in range(2):
        env = dict(os.environ, RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE="2", MASTER_ADDR="127.0.0.1",
                   MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, "-c", SYNC_CHILD % ROOT], env=env, stdout=subprocess.PIPE,
                                      stderr=subprocess.STDOUT, text=True))
    for rank, p in enumerate(procs):
        out, _ = p.communicate(timeout=180)
        assert p.returncode == 0, out
        assert "rank %d ok" % rank in out


def test_payload_exchange_layout_single_rank():
    import torch

    from paper_2312_17530_b200 import sync

    ex = sync.PayloadExchange(n_layers=3, idx_capacity=10, val_capacity=37, n_local_workers=2, world=1, rank=0,
                              device="cpu", val_dtype=torch.bfloat16)
    assert ex.msg_bytes % 16 == 0 and ex.recv is ex.send
    for w in range(2):
        idx, val, cnt = ex.local_views(w)
        assert idx.numel() == 10 and val.numel() == 37 and cnt.numel() == 3 and val.dtype == torch.bfloat16
        assert idx.data_ptr() % 16 == 0 and val.data_ptr() % 16 == 0 and cnt.data_ptr() % 16 == 0
        idx.fill_(w + 1)
    ex.exchange()
    assert [int(v[0][0]) for v in ex.gathered_views()] == [1, 2]


# ---------------------------------------------------------------------------------------------
# the exchange in layer groups (what overlaps it with the compression on a GPU): exact-size
# messages per group, group-by-group aggregation; two gloo ranks on CPU, payloads from the oracle
# ---------------------------------------------------------------------------------------------

GROUP_CHILD = r"""
import sys
sys.path.insert(0, %r)
import numpy as np, torch
import torch.distributed as td
import oracle
from paper_2312_17530_b200 import binding, dist, sync, synth
rank, local_rank, world = dist.init("gloo")
shapes = [(30, 41, 3, 3), (16, 9, 1, 9), (1, 50, 1, 9), (20, 20, 3, 3), (8, 27, 1, 9), (1, 7, 1, 9)]
tensors = [("t%%d" %% i, (s[0], s[1])) for i, s in enumerate(shapes)]
ratios = [0.25, 0.5, 0.2, 0.1, 0.0, 1.0]
n_local = 2
groups = sync.split_layers(shapes, 3)
assert len(groups) == 3 and groups[0][0] == 0 and groups[-1][1] == len(shapes)
plans = [binding.Plan(shapes[lo:hi], device=-1) for lo, hi in groups]      # host-only: sizes and layout
gx = sync.GroupedExchange(shapes, groups, plans, n_local, world, rank, "cpu")
gx.set_ratios(ratios)
def payloads_of(r):
    sig = synth.log_uniform_scales(len(shapes), (61,))
    grads = synth.multi_worker_gradients(tensors, n_local, (61, r), sig)
    zeros = [np.zeros(s[0] * s[1], np.float32) for s in shapes]
    return [oracle.compress(shapes, g, zeros, ratios, 0.5) for g in grads]
mine = payloads_of(rank)
k_all = [oracle.keep_count(oracle.tile_count(*s), q) for s, q in zip(shapes, ratios)]
sent_bytes = 0
for g, (lo, hi) in enumerate(groups):
    for w, res in enumerate(mine):
        idx, val, cnt = gx.local_views(g, w)
        # the message holds exactly what is sent: no slack beyond the 16-byte padding of its sections
        assert idx.numel() == sum(k_all[lo:hi]) and val.numel() == sum(k * s[2] * s[3] for k, s in zip(k_all[lo:hi], shapes[lo:hi]))
        i = np.concatenate([l.idx for l in res.layers[lo:hi]]); v = np.concatenate([l.val for l in res.layers[lo:hi]])
        assert i.size == idx.numel() and v.size == val.numel()
        idx[:] = torch.from_numpy(i); val[:] = torch.from_numpy(v); cnt[:] = torch.from_numpy(res.counts[lo:hi])
    gx.exchange_group(g)
assert gx.message_bytes() <= n_local * (4 * len(shapes) + 4 * sum(k_all) + 4 * sum(k * s[2] * s[3] for k, s in zip(k_all, shapes)) + 48 * len(groups))
# aggregate group by group from the received bytes, workers in global order
dense = [np.zeros(s[0] * s[1], np.float32) for s in shapes]
for g, (lo, hi) in enumerate(groups):
    got = gx.gathered_views(g)
    assert len(got) == world * n_local
    for idx, val, cnt in got:
        io = vo = 0
        for l in range(lo, hi):
            s = shapes[l]; k = int(cnt[l - lo]); slot = s[2] * s[3]
            oracle.decompress_into(dense[l], s, idx.numpy()[io:io + k], val.numpy()[vo:vo + k * slot], 1.0)
            io += k; vo += k * slot
# the ungrouped result: all workers of all ranks through the oracle's own aggregation
ref = [np.zeros(s[0] * s[1], np.float32) for s in shapes]
oracle.decompress_accumulate(shapes, ref, [p for r in range(world) for p in payloads_of(r)], 1.0)
for a, b in zip(dense, ref):
    assert np.array_equal(a.view(np.uint32), b.view(np.uint32))
flat = torch.from_numpy(np.concatenate(dense)).double()
lo_t, hi_t = flat.clone(), flat.clone()
td.all_reduce(lo_t, op=td.ReduceOp.MIN); td.all_reduce(hi_t, op=td.ReduceOp.MAX)
assert torch.equal(lo_t, hi_t) and float(flat.abs().sum()) > 0
dist.barrier()
dist.finalize()
print("rank %%d ok" %% rank)
"""


def test_grouped_exchange_two_gloo_ranks():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    procs = []
    for rank in range(2):
        env = dict(os.environ, RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE="2", MASTER_ADDR="127.0.0.1",
                   MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, "-c", GROUP_CHILD % ROOT], env=env, stdout=subprocess.PIPE,
                                      stderr=subprocess.STDOUT, text=True))
    for rank, p in enumerate(procs):
        out, _ = p.communicate(timeout=180)
        assert p.returncode == 0, out
        assert "rank %d ok" % rank in out


def test_layer_groups_and_host_keep_count():
    from paper_2312_17530_b200 import sync, synth

    import oracle

    oracle.build()
    for K, q in [(29241, 1 / 64), (10, 0.1), (100, 0.0), (100, 1.0), (7, 0.5), (1 << 20, 0.001), (5, 7.5), (3, -1.0)]:
        for clamp in (True, False):
            assert sync.keep_count(K, q, clamp) == oracle.keep_count(K, q, clamp)
    shapes = synth.layer_shapes(synth.resnet50_tensors())
    for n in (1, 2, 4, 7, 161, 500):
        groups = sync.split_layers(shapes, n)
        assert groups[0][0] == 0 and groups[-1][1] == len(shapes) and len(groups) <= n
        assert all(a[1] == b[0] for a, b in zip(groups, groups[1:])) and all(lo < hi for lo, hi in groups)
    sizes = [sum(r * c for r, c, _, _ in shapes[lo:hi]) for lo, hi in sync.split_layers(shapes, 4)]
    assert max(sizes) < 0.5 * sum(sizes)

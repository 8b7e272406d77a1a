"""Data-parallel pieces on CPU: the gradient bucket's all-reduce over two gloo ranks, and the Conv -> BN pair finder."""
import os
import socket

import numpy as np
import torch
import torch.multiprocessing as mp

from paper_2305_11624_b200.dataparallel import GradientBucket, Node, find_conv_bn_pairs, nodes_of_sequential


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _rank(rank, world, port, out):
    import torch.distributed as dist
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    sizes = GradientBucket.sizes_for([("c1a", 64, 256, False), ("c0", 32, 144, True)])
    bucket = GradientBucket(sizes, device="cpu")
    # every rank's "kernels" write its own per-shard partial gradients into the views
    for i, (name, v) in enumerate(bucket.views.items()):
        v.copy_(torch.arange(v.numel(), dtype=torch.float32) * (rank + 1) + i)
    bucket.all_reduce_async()
    bucket.wait()
    ok = True
    for i, (name, v) in enumerate(bucket.views.items()):
        want = torch.arange(v.numel(), dtype=torch.float32) * sum(r + 1 for r in range(world)) + i * world
        ok = ok and torch.equal(v, want)
    out.put((rank, ok, sorted(sizes)))
    dist.barrier()
    dist.destroy_process_group()


def test_bucket_all_reduce_sums_the_shards_over_two_ranks():
    ctx = mp.get_context("spawn")
    out, port = ctx.Queue(), _free_port()
    procs = [ctx.Process(target=_rank, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    got = [out.get(timeout=120) for _ in procs]
    for p in procs:
        p.join(120)
    assert all(ok for _, ok, _ in got), got
    assert "c0.db" in got[0][2] and "c1a.db" not in got[0][2]      # db exists only where the conv has a bias


def test_views_are_aligned_slices_of_one_buffer():
    b = GradientBucket({"a.dw": 100, "a.dgamma": 7, "a.dbeta": 7}, device="cpu")
    base = b.flat.data_ptr()
    for v in b.views.values():
        assert (v.data_ptr() - base) % 256 == 0 and v.data_ptr() >= base
    assert b.views["a.dw"].numel() == 100


def test_pair_finder_on_a_graph():
    g = [Node("x", "input"), Node("conv1", "conv2d", ("x",)), Node("bn1", "batch_norm", ("conv1",)),
         Node("relu1", "relu", ("bn1",)),
         Node("conv2", "conv2d", ("relu1",)), Node("bn2", "batch_norm", ("conv2",)), Node("tap", "identity", ("conv2",)),
         Node("conv3", "conv2d", ("relu1",)), Node("bn3", "batch_norm", ("conv3",), {"training": True}),
         Node("fc", "linear", ("relu1",)), Node("bn4", "batch_norm", ("fc",)),
         Node("add", "add", ("bn2", "bn3")), Node("bn5", "batch_norm", ("add",)),
         Node("up", "conv_transpose2d", ("add",)), Node("bn6", "batch_norm", ("up",), {"tracked_stats": False})]
    # conv2 also feeds `tap`; bn3 is in training mode; bn5 follows an add; bn6 has no tracked statistics
    assert find_conv_bn_pairs(g) == [("conv1", "bn1"), ("fc", "bn4")]


def test_pair_finder_on_a_sequential_module():
    import torch.nn as nn
    m = nn.Sequential(nn.Conv2d(3, 8, 3), nn.BatchNorm2d(8), nn.ReLU(), nn.Conv2d(8, 8, 1), nn.ReLU(), nn.BatchNorm2d(8),
                      nn.ConvTranspose2d(8, 4, 2), nn.BatchNorm2d(4)).eval()
    assert find_conv_bn_pairs(nodes_of_sequential(list(m.named_children()))) == [("0", "1"), ("6", "7")]
    m.train()
    assert find_conv_bn_pairs(nodes_of_sequential(list(m.named_children()))) == []

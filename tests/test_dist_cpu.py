"""world_size-2 gloo test of the data-parallel plumbing (no GPU): each rank owns
a shard of the images, computes g_W for it, and the all-reduce must give the
g_W of the whole batch; g_x needs no exchange."""
import os
import socket

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from oracle import lbp_oracle as O
from paper_2309_15275_b200.dist import GwReducer, allreduce_gw, shard_images


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, B, out_dir):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    rng = np.random.default_rng(5)
    k = 4
    x = rng.standard_normal((B, 8, 8, 6))
    gy = rng.standard_normal((B, 8, 8, 5))
    w = rng.standard_normal((5, 6))
    bases = O.select_bases(k, O.RULE_L1, 2)
    b0, b1 = shard_images(B, rank, world)
    gx, gw = O.backward_lowrank(x[b0:b1], gy[b0:b1], w, k, bases)
    gw_t = torch.from_numpy(gw.copy())
    allreduce_gw(gw_t)
    full_gx, full_gw = O.backward_lowrank(x, gy, w, k, bases)
    ok = np.allclose(gw_t.numpy(), full_gw, atol=1e-10) and np.allclose(gx, full_gx[b0:b1], atol=1e-12)
    with open(os.path.join(out_dir, f"rank{rank}.txt"), "w") as f:
        f.write("ok" if ok else "mismatch")
    dist.destroy_process_group()


def test_sharded_gw_allreduce_matches_full_batch(tmp_path):
    world, B = 2, 5
    mp.spawn(_worker, args=(world, _free_port(), B, str(tmp_path)), nprocs=world, join=True)
    for r in range(world):
        assert (tmp_path / f"rank{r}.txt").read_text() == "ok"


def _reducer_worker(rank, world, port, out_dir):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    rng = np.random.default_rng(11 + rank)
    shapes = [(5, 6), (3, 3), (8, 2), (1, 7)]
    mine = [torch.from_numpy(rng.standard_normal(s)) for s in shapes]
    serial = [t.clone() for t in mine]
    for t in serial:                      # one blocking all-reduce per layer, after the call
        allreduce_gw(t)
    red = GwReducer(len(shapes))          # issued together, as the layers finish
    assert red.events() is None           # no device: nothing to record
    red.reduce(mine)
    ok = all(torch.equal(a, b) for a, b in zip(mine, serial))
    with open(os.path.join(out_dir, f"red{rank}.txt"), "w") as f:
        f.write("ok" if ok else "mismatch")
    dist.destroy_process_group()


def test_overlapped_gw_reduction_equals_the_serial_form(tmp_path):
    world = 2
    mp.spawn(_reducer_worker, args=(world, _free_port(), str(tmp_path)), nprocs=world, join=True)
    for r in range(world):
        assert (tmp_path / f"red{r}.txt").read_text() == "ok"


def test_reducer_is_a_noop_on_one_rank():
    red = GwReducer(2)
    t = [torch.ones(3), torch.ones(2)]
    assert red.events() is None and red.reduce(t) is t and torch.equal(t[0], torch.ones(3))


def test_shard_images_partition():
    for B in (1, 5, 8, 128):
        for world in (1, 2, 3, 8):
            spans = [shard_images(B, r, world) for r in range(world)]
            assert spans[0][0] == 0 and spans[-1][1] == B
            for a, b in zip(spans, spans[1:]):
                assert a[1] == b[0]
            sizes = [e - b for b, e in spans]
            assert max(sizes) - min(sizes) <= 1


def test_allreduce_is_noop_without_process_group():
    t = torch.ones(3)
    assert torch.equal(allreduce_gw(t), torch.ones(3))

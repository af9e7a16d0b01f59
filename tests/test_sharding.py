"""Two gloo ranks on CPU: frame sharding and whole-job throughput as bench.py --gpus N uses them."""
import os
import socket

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

import emc2_gen as gen
from paper_2507_04123_b200 import sharding


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, q):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    w = gen.KITTI.with_shape(3, 500)
    frames = sharding.frames_for_rank(rank, world, w.B)
    pts = gen.make_batch(w, frames=frames)["points"]
    secs = 0.5 if rank == 0 else 2.0                       # rank 1 is the slow one
    fps = sharding.job_throughput(w.B, secs)
    slow = sharding.max_over_ranks(secs)
    dist.barrier()
    q.put((rank, frames, float(pts.sum()), fps, slow))
    dist.destroy_process_group()


def test_frames_are_disjoint_and_throughput_uses_the_slowest_rank():
    world, port = 2, _free_port()
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, world, port, q)) for r in range(world)]
    for p in procs:
        p.start()
    got = sorted(q.get(timeout=120) for _ in range(world))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    (r0, f0, s0, fps0, slow0), (r1, f1, s1, fps1, slow1) = got
    assert f0 == [0, 1, 2] and f1 == [3, 4, 5]             # disjoint, contiguous, cover 0..5
    assert s0 != s1                                        # different frames hold different points
    assert slow0 == slow1 == 2.0
    assert fps0 == fps1 == 2 * 3 / 2.0                     # all frames over the slowest rank's time


def test_single_process_needs_no_group():
    assert sharding.frames_for_rank(0, 1, 4) == [0, 1, 2, 3]
    assert sharding.max_over_ranks(1.25) == 1.25
    assert sharding.job_throughput(4, 2.0) == 2.0

"""The multi-rank path on CPU: videos are dealt to ranks, every rank merges its own (here with
the CPU oracle standing in for the GPU), and one all-gather of row counts gives the global
packed offsets.  Two gloo ranks against the single-process answer."""
import os
import socket

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from oracle import oracle
from paper_2507_07990_b200 import inputs, shard
from tests import helpers

N_VIDEOS = 5


def _videos():
    out = []
    for v in range(N_VIDEOS):
        spec = helpers.small_spec(300 + v, 5, 8, 8, 16, dtype="f32", sigma=0.3, p_static=0.3 + 0.15 * v)
        out.append(inputs.make_video(spec))
    return out


def _worker(rank, world, port, queue):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    videos = _videos()
    own = shard.videos_of_rank(N_VIDEOS, world, rank)
    counts = [oracle.merge(videos[v], 0.9, 0.9, want_feats=False).count for v in own]
    offsets, total = shard.global_row_offsets(counts, N_VIDEOS)
    queue.put((rank, list(own), counts, offsets, total))
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_agree_with_one_process():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    ctx = mp.get_context("spawn")
    queue = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, queue)) for r in range(2)]
    for p in procs:
        p.start()
    results = sorted(queue.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    videos = _videos()
    counts = [oracle.merge(v, 0.9, 0.9, want_feats=False).count for v in videos]
    expect = np.concatenate([[0], np.cumsum(counts)])
    seen = []
    for rank, own, c, offsets, total in results:
        assert total == expect[-1]
        assert c == [counts[v] for v in own]
        assert offsets == [int(expect[v]) for v in own]
        seen.extend(own)
    assert sorted(seen) == list(range(N_VIDEOS))


def test_video_blocks_cover_everything_once():
    for n in (1, 5, 8, 13):
        for world in (1, 2, 3, 8):
            got = [v for r in range(world) for v in shard.videos_of_rank(n, world, r)]
            assert got == list(range(n))
            sizes = [len(shard.videos_of_rank(n, world, r)) for r in range(world)]
            assert max(sizes) - min(sizes) <= 1

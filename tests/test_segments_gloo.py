"""Segments of one video over three gloo ranks on CPU.  The per-segment merges come from the CPU
oracle and the three folding steps are written out in numpy here, so what runs for real is the
message passing (segments.DistLink, segments.cut_frames, the message layout): the packed rows of
all ranks must be the oracle's rows for the whole video."""
import os
import socket

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from oracle import oracle
from paper_2507_07990_b200 import inputs, segments
from tests import helpers

T, H, W, D, WORLD = 8, 8, 8, 16, 3
TAU_S, TAU_T = 0.9, 0.8


def _video():
    return inputs.make_video(helpers.small_spec(970, T, H, W, D, dtype="f32", sigma=0.1, p_static=0.9))


def _worker(rank, world, port, queue):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    link = segments.DistLink()
    video, HW = _video(), H * W
    cuts = segments.cut_frames(T, world)
    halo = 1 if rank > 0 else 0
    local = video[cuts[rank] - halo:cuts[rank + 1]]
    res = oracle.merge(local, TAU_S, TAU_T)
    m, Wt = res.out_feats.copy(), res.out_members.astype(np.float64)
    n_h = 0
    if halo:
        h = oracle.merge(local[:1], TAU_S, 2.0)
        n_h = h.count
        assert np.array_equal(res.out_pos[:n_h], h.out_pos)          # halo-rooted rows = the halo's nodes, in order
    before = link.rows_before(res.count - n_h)
    extra, extra_w = np.zeros_like(m), np.zeros(res.count)
    like = [torch.zeros(1, dtype=torch.int32), torch.zeros(HW, dtype=torch.int32), torch.zeros(HW, dtype=torch.float32),
            torch.zeros((HW, D), dtype=torch.float32)]
    assert [t.shape for t in like] == [t.shape for t in segments.message_like(H, W, D, "cpu")]
    if rank + 1 < world:
        n, anchors, v, s = [t.numpy() for t in link.recv_next(like)]
        map_last = res.merge_map[(local.shape[0] - 1) * HW:]
        for i in range(int(n[0])):
            if v[i] != 0:
                extra[map_last[anchors[i]]] += s[i]
                extra_w[map_last[anchors[i]]] += v[i]
    if halo:
        msg = [t.clone() for t in like]
        msg[0][0] = n_h
        msg[1][:n_h] = torch.from_numpy(h.out_pos.astype(np.int32))
        V = Wt[:n_h] + extra_w[:n_h] - h.out_members
        S = Wt[:n_h, None] * m[:n_h] + extra[:n_h] - h.out_members[:, None] * h.out_feats
        msg[2][:n_h] = torch.from_numpy(V.astype(np.float32))
        msg[3][:n_h] = torch.from_numpy(S.astype(np.float32))
        link.send_prev(msg)
    rows = (Wt[n_h:, None] * m[n_h:] + extra[n_h:]) / (Wt[n_h:] + extra_w[n_h:])[:, None]
    ids = res.out_pos[n_h:].astype(np.int64) + (cuts[rank] - halo) * HW
    queue.put((rank, before, rows, ids))
    dist.barrier()
    dist.destroy_process_group()


def test_three_ranks_reproduce_the_whole_video():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    ctx = mp.get_context("spawn")
    queue = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, WORLD, port, queue)) for r in range(WORLD)]
    for p in procs:
        p.start()
    results = sorted((queue.get(timeout=180) for _ in procs), key=lambda x: x[0])
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    ref = oracle.merge(_video(), TAU_S, TAU_T)
    last = np.zeros(ref.count, dtype=np.int64)
    for cell, row in enumerate(ref.merge_map):
        last[row] = max(last[row], cell // (H * W))
    cuts = segments.cut_frames(T, WORLD)
    assert np.any((ref.out_pos // (H * W) < cuts[1]) & (last >= cuts[2]))      # a chain over both cuts
    offset = 0
    for rank, before, rows, ids in results:
        assert before == offset
        offset += len(ids)
    assert offset == ref.count
    np.testing.assert_array_equal(np.concatenate([r[3] for r in results]), ref.out_pos)
    np.testing.assert_allclose(np.concatenate([r[2] for r in results]), ref.out_feats, rtol=0, atol=2e-6)


def test_cuts_cover_every_frame_once():
    for t in (1, 7, 64, 1024):
        for world in (1, 2, 3, 8):
            if t < world:
                continue
            cuts = segments.cut_frames(t, world)
            assert cuts[0] == 0 and cuts[-1] == t and all(b > a for a, b in zip(cuts, cuts[1:]))
            assert max(b - a for a, b in zip(cuts, cuts[1:])) - min(b - a for a, b in zip(cuts, cuts[1:])) <= 1

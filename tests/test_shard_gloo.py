"""Multi-process use of the path: images are independent, so N ranks each take a contiguous slice of
the batch and nothing is exchanged on the data path.  Two gloo ranks on CPU check the host-side
logic: the slices cover the batch, and per-rank results (here from the CPU oracle, standing in for
the GPU path) concatenate to the single-process result once the packed offsets are shifted by the
counts of the lower ranks.  The slicing (`binding.shard_slice`) and the shift (`binding.global_out_offsets`,
one all_gather of a scalar) are the package's."""
import os
import socket

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2605_00392_b200 import binding, synth


def _free_port() -> int:
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def _worker(rank: int, world: int, port: int, ret):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    from oracle import oracle
    w = synth.ragged([40, 17, 64, 9, 33], d=32, dtype=torch.float32, params=dict(r_fixed=0.25))
    # the rank's slice: its images, its rows of X, its own offsets starting at 0
    (lo, hi), (row_lo, row_hi), local_offsets = binding.shard_slice(w.offsets, world, rank)
    assert local_offsets[0] == 0 and local_offsets[-1] == row_hi - row_lo
    res = oracle.run_batch(w.X_f64()[row_lo:row_hi], local_offsets, oracle.Params(r_fixed=0.25), w.rho[lo:hi])
    local_out = torch.from_numpy(np.asarray(res.out_offsets, dtype=np.int64))
    # the only cross-rank datum: how many packed rows the lower ranks produce (the package's helper gathers it)
    offs = binding.global_out_offsets(local_out)
    ret[rank] = (lo, hi, offs.tolist(), [im.kept.tolist() for im in res.images])
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_partition_the_batch():
    world = 2
    port = _free_port()
    mgr = mp.Manager()
    ret = mgr.dict()
    mp.spawn(_worker, args=(world, port, ret), nprocs=world, join=True)
    from oracle import oracle
    w = synth.ragged([40, 17, 64, 9, 33], d=32, dtype=torch.float32, params=dict(r_fixed=0.25))
    ref = oracle.run_batch(w.X_f64(), w.offsets, oracle.Params(r_fixed=0.25), w.rho)
    assert ret[0][0] == 0 and ret[0][1] == ret[1][0] and ret[1][1] == w.batch
    got_offs = ret[0][2][:-1] + ret[1][2]
    assert got_offs == ref.out_offsets.tolist()
    kept = ret[0][3] + ret[1][3]
    assert kept == [im.kept.tolist() for im in ref.images]


def test_shards_balanced_by_work_cover_the_batch():
    """Ragged batches: cuts by work are contiguous, cover every image once, and even out the token counts far
    better than cuts by image count when the long images sit together."""
    lens = [1156] * 6 + [456] * 26
    offsets = np.concatenate([[0], np.cumsum(lens)])
    for world in (1, 2, 3, 4, 8):
        ranges = [binding.shard_images_by_tokens(offsets, world, r) for r in range(world)]
        assert ranges[0][0] == 0 and ranges[-1][1] == len(lens)
        assert all(ranges[r][1] == ranges[r + 1][0] for r in range(world - 1))
        assert all(lo <= hi for lo, hi in ranges)
    by_work = [binding.shard_slice(offsets, 2, r, by_tokens=True)[1] for r in range(2)]
    by_count = [binding.shard_slice(offsets, 2, r)[1] for r in range(2)]
    n = np.asarray(lens, dtype=np.float64)
    cost = np.concatenate([[0.0], np.cumsum(n + n * n / 1600.0)])          # the balancing rule's cost, by image
    image_of_row = {int(o): i for i, o in enumerate(offsets)}
    work = lambda rows: [cost[image_of_row[hi]] - cost[image_of_row[lo]] for lo, hi in rows]
    assert max(work(by_work)) / min(work(by_work)) < 1.1
    assert max(work(by_count)) / min(work(by_count)) > 1.8
    # equal images: the same cuts as by count
    eq = np.arange(0, 401 * 16, 400)
    assert [binding.shard_images_by_tokens(eq, 4, r) for r in range(4)] == [binding.shard_images(16, 4, r) for r in range(4)]

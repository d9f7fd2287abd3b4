"""Host-side logic of the multi-GPU path, on CPU with the gloo backend and two processes: every rank
takes one copy of the decoder stack at its own range of global element indices (weak scaling, no
data-path collective); the only exchange is the max-over-ranks of the step time."""
import os
import socket

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2602_03120_b200 import workloads as wl


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out_dir):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    from paper_2602_03120_b200.model_pass import launch_segments, shard_tensors
    cfg = wl.WORKLOADS["decoder1p5b_int4"]
    tensors = shard_tensors(cfg, rank, world)
    lo, hi = tensors[0].elem_offset, tensors[-1].elem_offset + tensors[-1].numel
    ranges = [None] * world
    dist.all_gather_object(ranges, (lo, hi, len(launch_segments(tensors))))
    ms = torch.tensor([10.0 + 5.0 * rank], dtype=torch.float64)   # stand-in for this rank's device time
    dist.all_reduce(ms, op=dist.ReduceOp.MAX)
    if rank == 0:
        np.save(os.path.join(out_dir, "ranges.npy"), np.array(ranges, dtype=np.int64))
        np.save(os.path.join(out_dir, "ms.npy"), ms.numpy())
    dist.barrier()
    dist.destroy_process_group()


def test_two_rank_shards_are_disjoint_contiguous_and_timed_by_the_slowest(tmp_path):
    world = 2
    mp.spawn(_worker, args=(world, _free_port(), str(tmp_path)), nprocs=world, join=True)
    ranges = np.load(tmp_path / "ranges.npy")
    cfg = wl.WORKLOADS["decoder1p5b_int4"]
    assert ranges[0][0] == 0 and ranges[0][1] == cfg.numel == ranges[1][0] and ranges[1][1] == 2 * cfg.numel
    assert ranges[0][2] == ranges[1][2] == 5
    assert np.load(tmp_path / "ms.npy")[0] == 15.0


def test_shard_of_a_deeper_model_equals_that_slice_of_it(qo):
    """Rank r's shard is the r-th copy of the stack at offset r * numel: updating it alone gives the same
    codes as the matching slice of one tensor list updated as a whole (noise depends only on seed and
    global element index)."""
    from paper_2602_03120_b200.model_pass import shard_tensors
    cfg = wl.WORKLOADS["decoder1p5b_int4"]
    t1 = shard_tensors(cfg, 1, 2)[1]                     # layers.0.k_proj of rank 1
    assert t1.elem_offset == cfg.numel + cfg.tensors[1].elem_offset
    n = 4096
    packed = np.random.default_rng(1).integers(0, 256, n // 2, dtype=np.uint8)
    seeds, fit = wl.draw_seeds(3, 4), wl.draw_fitness(3, 4)
    hp = qo.HParams(sigma=0.5, lr=1.0, gamma=0.9, n_pop=4)
    whole = qo.update(qo.Tensor(bits=4, rows=2 * n // 32, cols=32, elem_offset=t1.elem_offset - n),
                      np.concatenate([packed, packed]), None, seeds, fit, 2, hp)
    part = qo.update(qo.Tensor(bits=4, rows=n // 32, cols=32, elem_offset=t1.elem_offset), packed, None, seeds, fit, 2, hp)
    assert np.array_equal(whole["w_new"][n:], part["w_new"])
    assert not np.array_equal(whole["w_new"][:n], part["w_new"])


def test_launch_segments_cover_every_tensor_once_and_respect_the_limit():
    """Runs of consecutive tensors for the fused launches: contiguous, in order, no run above the limit
    unless a single tensor is, and a gap in the element offsets starts a new run."""
    from paper_2602_03120_b200.model_pass import launch_segments
    rng = np.random.default_rng(4)
    for trial in range(50):
        sizes = (32 * rng.integers(1, 400, size=int(rng.integers(1, 30)))).tolist()
        gaps = set(rng.integers(0, len(sizes), size=2).tolist()) if trial % 3 == 0 else set()
        tensors, off = [], 0
        for i, n in enumerate(sizes):
            if i in gaps and i > 0:
                off += 64
            tensors.append(wl.TensorSpec(f"t{i}", n // 32, 32, off)); off += n
        limit = int(32 * rng.integers(1, 600))
        segs = launch_segments(tensors, limit)
        covered = []
        for first, seg_off, n in segs:
            assert tensors[first].elem_offset == seg_off
            run, j = 0, first
            while run < n:
                assert tensors[j].elem_offset == seg_off + run      # contiguous inside a run
                run += tensors[j].numel; covered.append(j); j += 1
            assert run == n
            assert n <= limit or j == first + 1                       # only a lone tensor may exceed the limit
        assert covered == list(range(len(tensors)))
    cfg = wl.WORKLOADS["decoder7b_int4"]
    assert len(launch_segments(cfg.tensors)) == 28 and max(s[2] for s in launch_segments(cfg.tensors)) <= 1 << 28

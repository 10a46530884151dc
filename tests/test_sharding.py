"""Host-side logic of the multi-GPU path (batch sharding, result gathering) on CPU with gloo, world size 2.
The per-shard search itself needs a GPU; here the oracle stands in for it so that the plumbing can be checked."""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

import zl_inputs as zi
from paper_2001_01347_b200.sharding import gather_selection, shard_range


def test_shard_ranges_partition_the_batch():
    for total in (0, 1, 7, 64, 4096, 4097):
        for world in (1, 2, 3, 8):
            spans = [shard_range(total, world, r) for r in range(world)]
            assert spans[0][0] == 0 and sum(c for _, c in spans) == total
            for (f0, c0), (f1, _) in zip(spans, spans[1:]):
                assert f1 == f0 + c0
            assert max(c for _, c in spans) - min(c for _, c in spans) <= 1
    with pytest.raises(ValueError):
        shard_range(4, 2, 2)


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, total, out_dir):
    import oracle
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    w = zi.CONFIGS["c2"].with_(B=total)
    first, count = shard_range(total, world, rank)
    ts = zi.generate(w, B=count, first_instance=first) if count else np.empty((0, w.n, w.R), dtype=np.int64)
    idx, barrier, wait = oracle.select_batched(ts, oracle.RANGE) if count else (
        np.empty((0, w.n), np.int32), np.empty(0, np.int64), np.empty(0, np.int64))
    full = gather_selection(torch.from_numpy(idx), torch.from_numpy(barrier), torch.from_numpy(wait),
                            torch.zeros(count, dtype=torch.int32), total)
    torch.save(full, os.path.join(out_dir, f"r{rank}.pt"))
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_gather_the_same_full_result(tmp_path):
    import oracle
    total, world = 5, 2                                         # uneven split: 3 + 2
    mp.start_processes(_worker, args=(world, _free_port(), total, str(tmp_path)), nprocs=world, start_method="spawn")
    ts = zi.generate(zi.CONFIGS["c2"].with_(B=total))
    ref_idx, ref_barrier, ref_wait = oracle.select_batched(ts, oracle.RANGE)
    for r in range(world):
        idx, barrier, wait, status = torch.load(os.path.join(str(tmp_path), f"r{r}.pt"))
        assert (idx.numpy() == ref_idx).all() and (barrier.numpy() == ref_barrier).all()
        assert (wait.numpy() == ref_wait).all() and status.shape == (total,)

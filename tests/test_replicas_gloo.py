"""N > 1 path of the bench on CPU: two gloo ranks, max-over-ranks timing, per-rank batches."""
import os
import socket

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2301_12187_b200 import inputs as I
from paper_2301_12187_b200 import replicas as R


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def _worker(rank, world, port, out):
    os.environ.update({"MASTER_ADDR": "127.0.0.1", "MASTER_PORT": str(port), "RANK": str(rank),
                       "WORLD_SIZE": str(world), "LOCAL_RANK": str(rank)})
    r, w, local = R.env_rank_world()
    assert (r, w, local) == (rank, world, rank)
    assert R.init_group("gloo", w)
    # every rank owns its own batch: same shapes, different images
    case = I.chain_case(0, seed=R.replica_seed(0, r))
    x = case.x()
    # the slowest rank sets the job's step time
    mine = [10.0 + 5.0 * r, 3.0 - r]
    t = R.max_over_ranks(torch.tensor(mine, dtype=torch.float64), w)
    dist.barrier()
    out[rank] = (t.tolist(), float(np.asarray(x, dtype=np.float64).sum()), tuple(x.shape))
    dist.destroy_process_group()


def test_two_replicas_reduce_times_by_max_and_draw_different_batches():
    world = 2
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_worker, args=(world, _free_port(), out), nprocs=world, join=True)
        res = dict(out)
    assert set(res) == {0, 1}
    assert res[0][0] == res[1][0] == [15.0, 3.0]
    assert res[0][2] == res[1][2]
    assert res[0][1] != res[1][1]
    # whole-job throughput counts every rank's images against the slowest rank's time
    assert R.job_throughput(64, world, 15.0e-3) == 2 * 64 / 15.0e-3


def test_single_process_is_the_identity():
    os.environ.pop("RANK", None); os.environ.pop("WORLD_SIZE", None); os.environ.pop("LOCAL_RANK", None)
    assert R.env_rank_world() == (0, 1, 0)
    assert R.init_group("gloo", 1) is False
    t = torch.tensor([1.0, 2.0])
    assert R.max_over_ranks(t, 1).tolist() == [1.0, 2.0]

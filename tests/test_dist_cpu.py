"""Multi-rank plumbing on CPU (gloo, world size 2): units are split across ranks with no
data-path exchange, and the ranks agree on a timing by a max-reduction."""
import os
import socket

import numpy as np
import torch.multiprocessing as mp

from paper_2604_16429_b200 import dist as mdist


def test_shard_range_covers_every_unit_once():
    for n in (0, 1, 7, 8, 24, 192):
        for world in (1, 2, 3, 8):
            spans = [mdist.shard_range(n, r, world) for r in range(world)]
            assert spans[0][0] == 0 and spans[-1][1] == n
            assert all(a[1] == b[0] for a, b in zip(spans[:-1], spans[1:]))
            sizes = [hi - lo for lo, hi in spans]
            assert max(sizes) - min(sizes) <= 1


def _free_port() -> int:
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank: int, world: int, port: int, out_dir: str):
    os.environ.update(RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(world), MASTER_ADDR="127.0.0.1",
                      MASTER_PORT=str(port))
    r, lr, w = mdist.init(backend="gloo")
    assert (r, lr, w) == (rank, rank, world)
    lo, hi = mdist.shard_range(24, rank, world)          # 24 ensemble members over the ranks
    mdist.barrier()
    t_max = mdist.max_over_ranks(1.0 + rank)             # rank 1 is the slow one
    total = mdist.sum_over_ranks(hi - lo)
    np.save(os.path.join(out_dir, f"r{rank}.npy"), np.array([lo, hi, t_max, total]))
    mdist.finalize()


def test_two_ranks_split_units_and_agree_on_time(tmp_path):
    world, port = 2, _free_port()
    mp.spawn(_worker, args=(world, port, str(tmp_path)), nprocs=world, join=True)
    got = [np.load(tmp_path / f"r{r}.npy") for r in range(world)]
    assert [tuple(g[:2]) for g in got] == [(0, 12), (12, 24)]
    assert all(g[2] == 2.0 for g in got)                 # max over ranks, the same on both
    assert all(g[3] == 24 for g in got)                  # every unit owned by exactly one rank


def test_single_process_helpers_need_no_group():
    assert mdist.max_over_ranks(3.5) == 3.5 and mdist.sum_over_ranks(2) == 2.0
    mdist.barrier()

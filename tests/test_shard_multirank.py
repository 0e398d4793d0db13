"""Host side of a step spread over ranks (paper_2409_15520_b200.sharding), world_size 2 and 3 on the
gloo backend: the query partition, and the loss exchange as a sum of zero-padded blocks.  Each rank's
forward passes are done by the oracle here (no GPU), so the exchanged and updated values can be
compared with the oracle's whole step."""
import os
import pickle
import sys

import numpy as np
import pytest
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_query_partition_covers_every_query_once():
    from paper_2409_15520_b200.sharding import query_shard
    for q in range(1, 33):
        for world in range(1, 9):
            blocks = [query_shard(q, world, r) for r in range(world)]
            owned = [i for b, c in blocks for i in range(b, b + c)]
            assert owned == list(range(q))                                  # contiguous, ordered, no overlap
            counts = [c for _, c in blocks]
            assert max(counts) - min(counts) <= 1 and counts == sorted(counts, reverse=True)
    with pytest.raises(ValueError):
        query_shard(4, 2, 2)
    with pytest.raises(ValueError):
        query_shard(0, 1, 0)


def _worker(rank, world, port, outdir):
    import torch
    import torch.distributed as dist
    sys.path.insert(0, ROOT)
    from oracle import zo as ozo
    from paper_2409_15520_b200.sharding import exchange_losses, query_shard
    from workloads import config, make_linear_problem
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    spec = config("linear_fp32")
    p = make_linear_problem(spec, seed=1234, b_std=0.02)
    q, seed, eps, lr = 5, 3, spec.eps, spec.lr
    begin, count = query_shard(q, world, rank)
    Bs = ozo._b_tensors(spec, p)
    buf = torch.zeros(2 * q + 3, dtype=torch.float64)
    buf[2 * q:] = 7.0                                                       # beyond 2q: must stay untouched
    for i in range(begin, begin + count):
        z = ozo.draw_z(spec, p, seed, i)
        for j, k in enumerate((+1.0, -1.0)):
            buf[2 * i + j] = ozo._loss_with(spec, p, [B + k * eps * zz for B, zz in zip(Bs, z)], p["X"], p["target"])
    exchange_losses(buf, q)
    losses = buf[:2 * q].numpy().copy()
    g = ozo.projected_gradients(losses, eps)
    newB = ozo.zo_sgd_update(Bs, [ozo.draw_z(spec, p, seed, i) for i in range(q)], g, lr)
    pickle.dump(dict(losses=losses, g=g, B=newB, tail=buf[2 * q:].numpy().copy()),
                open(os.path.join(outdir, f"r{rank}.pkl"), "wb"))
    dist.barrier()
    dist.destroy_process_group()


@pytest.mark.parametrize("world", [2, 3])
def test_exchanged_losses_and_update_equal_the_whole_step(world, tmp_path):
    sys.path.insert(0, ROOT)
    import oracle
    from workloads import config, make_linear_problem
    mp.spawn(_worker, args=(world, 29741 + os.getpid() % 200 + world, str(tmp_path)), nprocs=world, join=True)
    spec = config("linear_fp32")
    p = make_linear_problem(spec, seed=1234, b_std=0.02)
    ref_l, ref_g, ref_B = oracle.zo_step(spec, p, p["X"], p["target"], 3, 5, spec.eps, spec.lr)
    for rank in range(world):
        r = pickle.load(open(tmp_path / f"r{rank}.pkl", "rb"))
        assert np.array_equal(r["losses"], ref_l)          # x + 0 is exact: the sum is a gather
        assert np.array_equal(r["g"], ref_g)
        assert all(np.array_equal(a, b) for a, b in zip(r["B"], ref_B))
        assert np.all(r["tail"] == 7.0)


def test_single_process_exchange_is_a_no_op():
    import torch
    from paper_2409_15520_b200.sharding import exchange_losses
    buf = torch.arange(6, dtype=torch.float64)
    assert exchange_losses(buf, 3) is buf and buf.tolist() == [0, 1, 2, 3, 4, 5]

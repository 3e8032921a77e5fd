"""Two CPU ranks (gloo) split one params_list, evaluate their slices and gather the scores.

The evaluator here is the CPU checker, given the global configuration indices, so the test
covers the host logic of the multi-rank path: slice bounds, index base, gather order.
"""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2012_04201_b200 import sharding
from paper_2012_04201_b200 import workloads as W


def test_shard_bounds_cover_the_list():
    for n in (0, 1, 7, 8, 2048):
        for world in (1, 2, 3, 8):
            spans = [sharding.shard_bounds(n, r, world) for r in range(world)]
            assert spans[0][0] == 0 and spans[-1][1] == n
            assert all(a[1] == b[0] for a, b in zip(spans, spans[1:]))
            sizes = [e - b for b, e in spans]
            assert max(sizes) - min(sizes) <= 1 and sizes == sorted(sizes, reverse=True)
    with pytest.raises(ValueError):
        sharding.shard_bounds(4, 2, 2)


def test_cost_balanced_deal_is_a_partition_and_balanced():
    wl = W.workload("digits2048", n_configs=400)
    cfg = wl["configs"]
    costs = sharding.config_costs(cfg, 1797, 64, 10, 5)
    assert costs.shape == (400,) and np.all(costs > 0)
    # costlier by construction: more epochs, wider, smaller batches
    more = cfg.copy(); more["epochs"] *= 2
    assert np.all(sharding.config_costs(more, 1797, 64, 10, 5) > costs)
    for world in (1, 2, 3, 8):
        a = sharding.balanced_assignment(costs, world)
        parts = [sharding.shard_indices(a, r) for r in range(world)]
        assert sorted(np.concatenate(parts).tolist()) == list(range(400))     # every entry exactly once
        load = np.array([costs[p].sum() for p in parts])
        assert load.max() / load.mean() < 1.10                                 # within 10 % of even
        assert np.array_equal(a, sharding.balanced_assignment(costs, world))   # deterministic
    with pytest.raises(ValueError):
        sharding.balanced_assignment(costs, 0)


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def _rank_main(rank, world, port, out_path):
    import oracle

    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    wl = W.workload("iris8", n_configs=7, epochs=4)   # 7 configurations over 2 ranks: 4 + 3
    cfg, K = wl["configs"], wl["n_folds"]
    begin, end = sharding.shard_bounds(cfg.size, rank, world)
    fc = np.repeat(np.arange(begin, end), K)
    ff = np.tile(np.arange(K), end - begin)
    fits = oracle.cv_fits(wl["X"], wl["y"], wl["task"], K, cfg, wl["seed"], fc, ff, n_threads=1)["scores"]
    local = np.zeros(end - begin, np.float32)
    for i in range(end - begin):          # mean over folds, float arithmetic in fold order
        acc = np.float32(0)
        for f in range(K):
            acc = np.float32(acc + np.float32(fits[i * K + f]))
        local[i] = acc / np.float32(K)
    full = sharding.gather_scores(local, cfg.size, rank, world, dist)
    t = torch.tensor([1.0 + rank])
    dist.all_reduce(t, op=dist.ReduceOp.MAX)   # the timing reduction bench.py uses
    if rank == 0:
        np.save(out_path, np.concatenate([full.numpy(), t.numpy()]))
    dist.barrier()
    dist.destroy_process_group()


def _balanced_rank_main(rank, world, port, out_path):
    import oracle

    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    wl = W.workload("iris8", n_configs=11, epochs=3)
    cfg, K = wl["configs"], wl["n_folds"]
    costs = sharding.config_costs(cfg, wl["X"].shape[0], wl["X"].shape[1], 3, K)
    assign = sharding.balanced_assignment(costs, world)
    mine = sharding.shard_indices(assign, rank)
    fc = np.repeat(mine, K)
    ff = np.tile(np.arange(K), mine.size)
    # the checker keys the random streams by position in the list it is given: passing the whole
    # list and the positions of this rank's entries is what bbo_mlp_cv_eval_keyed does on the device
    fits = oracle.cv_fits(wl["X"], wl["y"], wl["task"], K, cfg, wl["seed"], fc, ff, n_threads=1)["scores"]
    local = np.zeros(mine.size, np.float32)
    for i in range(mine.size):
        acc = np.float32(0)
        for f in range(K):
            acc = np.float32(acc + np.float32(fits[i * K + f]))
        local[i] = acc / np.float32(K)
    full = sharding.gather_scores_by_assignment(local, assign, rank, world, dist)
    if rank == 0:
        np.save(out_path, full.numpy())
    dist.barrier()
    dist.destroy_process_group()


@pytest.mark.parametrize("world", [2, 3])
def test_cost_balanced_ranks_reproduce_the_unsplit_scores(tmp_path, world):
    import oracle

    out = str(tmp_path / "gathered.npy")
    mp.spawn(_balanced_rank_main, args=(world, _free_port(), out), nprocs=world, join=True)
    got = np.load(out)
    wl = W.workload("iris8", n_configs=11, epochs=3)
    ref = oracle.cv_eval(wl["X"], wl["y"], wl["task"], wl["n_folds"], wl["configs"], wl["seed"])["scores"]
    assert np.array_equal(got.astype(np.float64), ref)


def test_two_ranks_reproduce_the_unsplit_scores(tmp_path):
    import oracle

    out = str(tmp_path / "gathered.npy")
    mp.spawn(_rank_main, args=(2, _free_port(), out), nprocs=2, join=True)
    got = np.load(out)
    wl = W.workload("iris8", n_configs=7, epochs=4)
    ref = oracle.cv_eval(wl["X"], wl["y"], wl["task"], wl["n_folds"], wl["configs"], wl["seed"])["scores"]
    assert np.array_equal(got[:-1].astype(np.float64), ref)
    assert got[-1] == 2.0

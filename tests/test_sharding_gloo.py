"""The multi-GPU path on CPU: two gloo ranks split the trials, each computes its share (here with the
oracle, since there is no GPU), and the shares put together equal the single-process result."""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

import oracle
from paper_2306_10598_b200 import sharding
from paper_2306_10598_b200 import workloads as W


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, T, out_dir):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        w = W.WORKLOADS["paper_scale"].with_trials(T)
        taus = W.make_taus(w)
        t0, t1 = sharding.trial_range(w.T, rank, world)
        lat = W.fill_latencies(w, "cpu", t0=t0, t1=t1).numpy()          # only this rank's trials are generated
        sw = oracle.sweep(lat, taus, w.t_comm)
        st = oracle.reduce_trials(sw.step, sw.done, sw.sync, w.N, w.M)
        g_stats, g_base = sharding.combine_stats(torch.from_numpy(st.stats), torch.from_numpy(st.baseline),
                                                 t1 - t0, w.N, w.M)
        slow = sharding.max_over_ranks(10.0 + rank, "cpu")
        np.savez(os.path.join(out_dir, f"rank{rank}.npz"), t0=t0, t1=t1, done=sw.done, step=sw.step, sync=sw.sync,
                 stats=g_stats.numpy(), base=g_base.numpy(), slow=slow)
        dist.barrier()
    finally:
        dist.destroy_process_group()


def test_trial_range_partitions():
    for T in (0, 1, 7, 64, 1000):
        for world in (1, 2, 3, 8):
            edges = [sharding.trial_range(T, r, world) for r in range(world)]
            assert edges[0][0] == 0 and edges[-1][1] == T
            assert all(a[1] == b[0] for a, b in zip(edges, edges[1:]))
            sizes = [b - a for a, b in edges]
            assert max(sizes) - min(sizes) <= 1
    with pytest.raises(ValueError):
        sharding.trial_range(4, 2, 2)
    w = W.WORKLOADS["tiny"]
    assert sharding.rank_workload(w, 3).seed == w.seed + 3 and sharding.rank_workload(w, 3).T == w.T


def test_two_ranks_equal_one(tmp_path):
    T, world = 37, 2                                  # odd: the shares differ by one trial
    port = _free_port()
    mp.start_processes(_worker, args=(world, port, T, str(tmp_path)), nprocs=world, join=True, start_method="spawn")
    w = W.WORKLOADS["paper_scale"].with_trials(T)
    taus = W.make_taus(w)
    full = oracle.sweep(W.fill_latencies(w, "cpu").numpy(), taus, w.t_comm)
    st = oracle.reduce_trials(full.step, full.done, full.sync, w.N, w.M)
    parts = [np.load(tmp_path / f"rank{r}.npz") for r in range(world)]
    assert int(parts[0]["t0"]) == 0 and int(parts[0]["t1"]) == int(parts[1]["t0"]) and int(parts[1]["t1"]) == T
    assert np.array_equal(np.concatenate([p["done"] for p in parts]), full.done)
    assert np.array_equal(np.concatenate([p["step"] for p in parts]), full.step)
    assert np.array_equal(np.concatenate([p["sync"] for p in parts]), full.sync)
    for p in parts:                                   # every rank ends with the statistics of all trials
        assert np.allclose(p["stats"], st.stats, rtol=1e-12, atol=0)
        assert np.allclose(p["base"], st.baseline, rtol=1e-12, atol=0)
        assert float(p["slow"]) == 11.0               # the slowest rank's time

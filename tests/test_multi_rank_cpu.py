"""The N > 1 path on CPU: two gloo ranks share a parameter list by whole tensors, step
their shards independently (with the oracle standing in for the GPU), and together
reproduce the single-process result without any data-path collective."""
import os
import socket

import numpy as np
import pytest

from paper_1810_05486_b200 import multi
from paper_1810_05486_b200 import workloads as W


def test_partition_covers_every_tensor_once_and_balances():
    wl = W.workload("c3_resnet50")
    numels = [t.numel for t in wl.tensors]
    for world in (1, 2, 3, 8):
        parts = multi.partition_tensors(numels, world)
        assert sorted(i for p in parts for i in p) == list(range(len(numels)))
        loads = [sum(numels[i] for i in p) for p in parts]
        assert max(loads) - min(loads) <= max(numels)
        assert all(p == sorted(p) for p in parts)
    assert multi.rank_seed(7, 3) == 3007
    assert multi.whole_job_throughput(10, 4, 2.0) == 20.0
    assert multi.max_over_ranks(1.5) == 1.5


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _rank_main(rank, world, port, out_dir):
    import torch
    import torch.distributed as dist
    from oracle import EXP_AMAX, OracleState, OracleTensor, oracle_step
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        wl = W.scaled_sweep(600_000, 10)
        mine = multi.partition_tensors([t.numel for t in wl.tensors], world)[rank]
        thetas, comps = W.initial_state(wl)
        st = OracleState([OracleTensor(thetas[i], comps[i], 16, 16, 0, wl.tensors[i].exp_theta,
                                       wl.tensors[i].exp_theta) for i in mine], EXP_AMAX)
        for step in range(3):
            grads = W.gradients(wl, step)
            oracle_step(st, [grads[i] * np.float32(40.0) for i in mine], [wl.lr] * len(mine))
        dist.barrier()
        slowest = multi.max_over_ranks(1.0 + rank, dist)
        assert slowest == float(world)
        result = {i: (t.theta.copy(), t.comp.copy(), t.exp_theta, t.exp_theta_next, t.amax_theta)
                  for i, t in zip(mine, st.tensors)}
        gathered = [None] * world
        dist.all_gather_object(gathered, result)        # read-out only, not on the data path
        if rank == 0:
            merged = {}
            for g in gathered:
                merged.update(g)
            np.save(os.path.join(out_dir, "keys.npy"), np.array(sorted(merged)))
            for i, (th, c, e0, e1, a) in merged.items():
                np.savez(os.path.join(out_dir, f"t{i}.npz"), theta=th, comp=c,
                         meta=np.array([e0, e1, a]))
    finally:
        dist.destroy_process_group()


def test_two_gloo_ranks_reproduce_the_single_process_result(tmp_path):
    import torch.multiprocessing as mp
    from oracle import EXP_AMAX, OracleState, OracleTensor, oracle_step
    world = 2
    # The port is free when it is drawn, not necessarily still when rank 0 binds it: a
    # rendezvous that fails for that reason is tried once more on another port.
    for attempt in range(2):
        try:
            mp.spawn(_rank_main, args=(world, _free_port(), str(tmp_path)), nprocs=world, join=True)
            break
        except Exception:
            if attempt == 1:
                raise

    wl = W.scaled_sweep(600_000, 10)
    thetas, comps = W.initial_state(wl)
    st = OracleState([OracleTensor(thetas[i], comps[i], 16, 16, 0, t.exp_theta, t.exp_theta)
                      for i, t in enumerate(wl.tensors)], EXP_AMAX)
    for step in range(3):
        grads = W.gradients(wl, step)
        oracle_step(st, [g * np.float32(40.0) for g in grads], [wl.lr] * len(grads))
    keys = list(np.load(tmp_path / "keys.npy"))
    assert keys == list(range(len(wl.tensors)))
    for i, t in enumerate(st.tensors):
        z = np.load(tmp_path / f"t{i}.npz")
        assert np.array_equal(z["theta"], t.theta) and np.array_equal(z["comp"], t.comp)
        assert list(z["meta"]) == [t.exp_theta, t.exp_theta_next, t.amax_theta]

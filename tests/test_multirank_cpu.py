"""The N > 1 path of bench.py on CPU: two gloo ranks, each with its own step time; the job's step time must be
the slower rank's and the job's throughput the sum of both ranks' tokens over that time (replicas only: no
collective on the data path, one max-reduction of the timing)."""
import os
import sys

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    import bench
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    local_ms = 100.0 if rank == 0 else 250.0          # rank 1 is slower
    ms_per_step, value = bench.aggregate_over_ranks(local_ms, 10, 32768, world, dist, torch.device("cpu"))
    dist.barrier()
    out[rank] = (ms_per_step, value)
    dist.destroy_process_group()


def test_two_gloo_ranks_take_the_slowest_time():
    world = 2
    port = 29000 + os.getpid() % 2000
    with mp.Manager() as m:
        out = m.dict()
        mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
        res = dict(out)
    assert set(res) == {0, 1}
    for r in (0, 1):
        ms, value = res[r]
        assert ms == pytest.approx(25.0)
        assert value == pytest.approx(2 * 32768 / 25e-3)


def test_single_rank_needs_no_process_group():
    sys.path.insert(0, ROOT)
    import bench
    ms, value = bench.aggregate_over_ranks(40.0, 20, 1000, 1, None, torch.device("cpu"))
    assert ms == pytest.approx(2.0) and value == pytest.approx(1000 / 2e-3)


# ---- expert-wise model parallelism (Section 6): two gloo ranks, the oracle standing in for the kernels ----------
def _sharded_worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    import numpy as np
    from oracle import lory_oracle as O
    from paper_2405_03133_b200 import parallel
    from paper_2405_03133_b200.workloads import Workload, make_inputs
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    wl = Workload("sharded", B=2, L=12, T=3, d=8, f=24, E=3, dtype="fp32", w_r_std=2.0, seed=31)
    inp = make_inputs(wl)                                   # every rank draws the same replicated inputs
    W1s, W2s, W3s = parallel.shard_experts(inp["W1"], inp["W2"], inp["W3"], rank, world)
    all_reduce = parallel.torch_all_reduce()

    def run_forward(x, w_r, a, b, c):
        y, w, _ = O.forward(x, w_r, a, b, c, wl.T)
        return torch.from_numpy(y), w

    def run_backward(x, w_r, a, b, c, dy):
        g = O.backward(x, w_r, a, b, c, wl.T, dy)
        return {k: torch.from_numpy(np.ascontiguousarray(v)) for k, v in g.items()}

    y, w = parallel.sharded_forward(run_forward, all_reduce, inp["x"], inp["w_r"], W1s, W2s, W3s)
    g = parallel.sharded_backward(run_backward, all_reduce, inp["x"], inp["w_r"], W1s, W2s, W3s, inp["dy"])
    out[rank] = dict(y=y.numpy(), w=w, f_range=parallel.shard_range(wl.f, rank, world),
                     **{k: v.numpy() for k, v in g.items()})
    dist.barrier()
    dist.destroy_process_group()


def test_expert_sharded_layer_matches_the_unsharded_one():
    import numpy as np
    sys.path.insert(0, ROOT)
    from oracle import lory_oracle as O
    from paper_2405_03133_b200.workloads import Workload, make_inputs
    world = 2
    port = 31000 + os.getpid() % 2000
    with mp.Manager() as m:
        out = m.dict()
        mp.spawn(_sharded_worker, args=(world, port, out), nprocs=world, join=True)
        res = dict(out)
    wl = Workload("sharded", B=2, L=12, T=3, d=8, f=24, E=3, dtype="fp32", w_r_std=2.0, seed=31)
    inp = make_inputs(wl)
    a = (inp["x"], inp["w_r"], inp["W1"], inp["W2"], inp["W3"], wl.T)
    y, w, _ = O.forward(*a)
    g = O.backward(*a, inp["dy"])
    assert [res[r]["f_range"] for r in range(world)] == [(0, 16), (16, 24)]
    for r in range(world):
        f0, f1 = res[r]["f_range"]
        np.testing.assert_allclose(res[r]["y"], y, rtol=1e-10, atol=1e-12)
        np.testing.assert_allclose(res[r]["w"], w, rtol=1e-13)
        np.testing.assert_allclose(res[r]["dx"], g["dx"], rtol=1e-9, atol=1e-12)            # router path included
        np.testing.assert_allclose(res[r]["dw_r"], g["dw_r"], rtol=1e-9, atol=1e-12)
        np.testing.assert_allclose(res[r]["d_route_w"], g["d_route_w"], rtol=1e-9, atol=1e-12)
        np.testing.assert_allclose(res[r]["dW1"], g["dW1"][:, f0:f1, :], rtol=1e-9, atol=1e-12)
        np.testing.assert_allclose(res[r]["dW3"], g["dW3"][:, f0:f1, :], rtol=1e-9, atol=1e-12)
        np.testing.assert_allclose(res[r]["dW2"], g["dW2"][:, :, f0:f1], rtol=1e-9, atol=1e-12)


def test_shard_ranges_cover_the_hidden_dimension():
    sys.path.insert(0, ROOT)
    from paper_2405_03133_b200 import parallel
    for f, world in ((2752, 8), (5504, 3), (24, 2), (8, 1)):
        r = [parallel.shard_range(f, k, world) for k in range(world)]
        assert r[0][0] == 0 and r[-1][1] == f
        assert all(r[k][1] == r[k + 1][0] for k in range(world - 1))
        assert all((b - a) % 8 == 0 and b > a for a, b in r)
    with pytest.raises(ValueError):
        parallel.shard_range(20, 0, 2)
    with pytest.raises(ValueError):
        parallel.shard_range(16, 0, 3)


# ---- the all-reduce of 16-bit partial tensors accumulates in fp32 and rounds once ---------------------------------
def _bf16_sum_worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    from paper_2405_03133_b200 import parallel
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    ulp = 2.0 ** -7                                   # spacing of bf16 numbers in [1, 2)
    # rank 0 contributes 1, the other two 0.3 ulp each: a running bf16 sum stays at 1 (each addend is below half
    # an ulp), the fp32 sum is 1 + 0.6 ulp and rounds to 1 + 1 ulp
    mine = 1.0 if rank == 0 else 0.3 * ulp
    t = torch.full((4,), mine, dtype=torch.bfloat16)
    parallel.torch_all_reduce()(t)
    out[rank] = t.float().tolist()
    dist.barrier()
    dist.destroy_process_group()


def test_all_reduce_of_bf16_partials_rounds_once():
    world = 3
    port = 33000 + os.getpid() % 2000
    with mp.Manager() as m:
        out = m.dict()
        mp.spawn(_bf16_sum_worker, args=(world, port, out), nprocs=world, join=True)
        res = dict(out)
    for r in range(world):
        assert res[r] == [1.0 + 2.0 ** -7] * 4

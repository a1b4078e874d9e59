"""World-size-2 check of the data-parallel path on CPU (gloo): token shards + summed weight gradients
reproduce the single-process result.  The per-rank arithmetic here is the oracle's (no GPU needed); the
sharding and the exchange step are the product's."""

import os

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from oracle import eqlinear_oracle as orc
from paper_2607_21271_b200 import parallel
from paper_2607_21271_b200.workloads import Workload, generate


def test_shard_tokens_partitions_the_range():
    for N in (0, 1, 7, 128, 25216):
        for world in (1, 2, 3, 8):
            spans = [parallel.shard_tokens(N, r, world) for r in range(world)]
            assert spans[0][0] == 0 and spans[-1][1] == N
            for a, b in zip(spans, spans[1:]):
                assert a[1] == b[0]
            sizes = [e - b for b, e in spans]
            assert max(sizes) - min(sizes) <= 1
    with pytest.raises(ValueError):
        parallel.shard_tokens(10, 2, 2)


def _worker(rank, world, port, out_dir):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    wl = Workload("dp", "fp32", 4, 6, 5, 203, "normal", ("fwd", "bwd_data", "bwd_weight"), 31)
    d = generate(wl)
    b, e = parallel.shard_tokens(wl.N, rank, world)
    y = orc.fwd(d["x"][b:e], d["w"], d["bias"])
    dx = orc.bwd_data(d["dy"][b:e], d["w"])
    dw, db = orc.bwd_weight(d["x"][b:e], d["dy"][b:e], wl.T)
    dw_t, db_t = torch.from_numpy(dw.copy()), torch.from_numpy(db.copy())
    parallel.allreduce_weight_grads(dw_t, db_t)
    np.savez(os.path.join(out_dir, f"rank{rank}.npz"), y=y, dx=dx, dw=dw_t.numpy(), db=db_t.numpy(), b=b, e=e)
    dist.barrier()
    dist.destroy_process_group()


def _flat_worker(rank, world, port, out_dir):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    flat, dw, db = parallel.grad_buffers(5, 6, 4, "cpu")
    assert dw.shape == (5, 6, 4) and db.shape == (5,) and db.data_ptr() % 16 == 0 and dw.data_ptr() == flat.data_ptr()
    dw.fill_(rank + 1.0); db.fill_(10.0 * (rank + 1))
    parallel.allreduce_weight_grads(dw, db, flat=flat)            # one collective for both
    np.savez(os.path.join(out_dir, f"flat{rank}.npz"), dw=dw.numpy(), db=db.numpy())
    dist.barrier()
    dist.destroy_process_group()


def _step_worker(rank, world, port, out_dir):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    wl = Workload("dp", "fp32", 4, 6, 5, 203, "normal", ("fwd", "bwd_data", "bwd_weight"), 31)
    d = generate(wl)
    b, e = parallel.shard_tokens(wl.N, rank, world)
    flat, dw, db = parallel.grad_buffers(wl.Co, wl.Ci, wl.T, "cpu")
    out, seen = {}, []

    def fwd():
        out["y"] = orc.fwd(d["x"][b:e], d["w"], d["bias"])

    def weight_grad():
        g, s = orc.bwd_weight(d["x"][b:e], d["dy"][b:e], wl.T)
        dw.copy_(torch.from_numpy(g)); db.copy_(torch.from_numpy(s))
        out["local_dw"] = g.copy()

    def data_grad():
        out["dx"] = orc.bwd_data(d["dy"][b:e], d["w"])

    order = parallel.dp_training_step(fwd, weight_grad, data_grad, flat, mark=seen.append)
    np.savez(os.path.join(out_dir, f"step{rank}.npz"), y=out["y"], dx=out["dx"], dw=dw.numpy(), db=db.numpy(),
             local_dw=out["local_dw"], order=np.array(order), marks=np.array(seen))
    dist.barrier()
    dist.destroy_process_group()


def test_dp_step_orders_the_exchange_before_the_data_gradient(tmp_path):
    """The N > 1 step of bench.py: weight gradient first, the all-reduce started before the data gradient and joined
    before the step returns; every rank ends with the gradients summed over all tokens."""
    world, port = 2, 33500 + os.getpid() % 2000
    mp.spawn(_step_worker, args=(world, port, str(tmp_path)), nprocs=world, join=True)
    wl = Workload("dp", "fp32", 4, 6, 5, 203, "normal", ("fwd", "bwd_data", "bwd_weight"), 31)
    d = generate(wl)
    ref_dw, ref_db = orc.bwd_weight(d["x"], d["dy"], wl.T)
    parts = [np.load(tmp_path / f"step{r}.npz") for r in range(world)]
    for p in parts:
        assert list(p["order"]) == ["fwd", "bwd_weight", "allreduce_start", "bwd_data", "allreduce_done"]
        assert list(p["marks"]) == [0, 1, 2, 3]
        # (the exchange buffer is float32, as the library's dw / db are)
        assert np.allclose(p["dw"], ref_dw, rtol=0, atol=1e-5 * np.abs(ref_dw).max())
        assert np.allclose(p["db"], ref_db, rtol=0, atol=1e-5 * np.abs(ref_db).max())
        assert not np.allclose(p["local_dw"], ref_dw, rtol=0, atol=1e-2 * np.abs(ref_dw).max())      # the sum really needed the other rank
    assert np.allclose(np.concatenate([p["y"] for p in parts]), orc.fwd(d["x"], d["w"], d["bias"]), rtol=0, atol=1e-12)
    assert np.allclose(np.concatenate([p["dx"] for p in parts]), orc.bwd_data(d["dy"], d["w"]), rtol=0, atol=1e-12)


def test_flat_gradient_buffer_is_reduced_in_one_call(tmp_path):
    world, port = 2, 31500 + os.getpid() % 2000
    mp.spawn(_flat_worker, args=(world, port, str(tmp_path)), nprocs=world, join=True)
    for r in range(world):
        p = np.load(tmp_path / f"flat{r}.npz")
        assert np.all(p["dw"] == 3.0) and np.all(p["db"] == 30.0)


def test_two_ranks_reproduce_the_single_process_result(tmp_path):
    world, port = 2, 29500 + os.getpid() % 2000
    mp.spawn(_worker, args=(world, port, str(tmp_path)), nprocs=world, join=True)
    wl = Workload("dp", "fp32", 4, 6, 5, 203, "normal", ("fwd", "bwd_data", "bwd_weight"), 31)
    d = generate(wl)
    ref_y, ref_dx = orc.fwd(d["x"], d["w"], d["bias"]), orc.bwd_data(d["dy"], d["w"])
    ref_dw, ref_db = orc.bwd_weight(d["x"], d["dy"], wl.T)
    parts = [np.load(tmp_path / f"rank{r}.npz") for r in range(world)]
    assert np.allclose(np.concatenate([p["y"] for p in parts]), ref_y, rtol=0, atol=1e-12)
    assert np.allclose(np.concatenate([p["dx"] for p in parts]), ref_dx, rtol=0, atol=1e-12)
    for p in parts:                                   # every rank holds the full, summed gradients
        assert np.allclose(p["dw"], ref_dw, rtol=0, atol=1e-10)
        assert np.allclose(p["db"], ref_db, rtol=0, atol=1e-10)

"""The multi-GPU plumbing on CPU: two gloo ranks shard a ragged batch, search their slices and gather.

The per-slice search is the CPU oracle here (this is a test of the sharding and the gather; on GPUs
the same calls carry the CUDA path).  No GPU involved.
"""
import os
import socket

import numpy as np
import pytest
import torch.multiprocessing as mp

from paper_2504_03662_b200 import inputs
from paper_2504_03662_b200.sharding import partition


def test_partition_covers_every_instance_once():
    rng = np.random.default_rng(0)
    for world in (1, 2, 3, 4, 8):
        for B in (1, 2, 7, 64):
            L = rng.integers(1, 97, size=B)
            b = partition(L, world)
            assert len(b) == world and b[0][0] == 0 and b[-1][1] == B
            assert all(b[r][1] == b[r + 1][0] for r in range(world - 1)) and all(s <= e for s, e in b)
    # balanced by work, not by count: one long instance against many short ones
    L = np.array([96] + [1] * 96)
    (s0, e0), (s1, e1) = partition(L, 2)
    assert (s0, e0, s1, e1) == (0, 1, 1, 97)
    # config 2's ragged stack splits near half of its 1536 layers
    w = inputs.config2()
    (s0, e0), (s1, e1) = partition(w.L, 2)
    assert abs(int(w.L[s0:e0].sum()) - 768) <= 96


def _oracle_local(sub):
    from oracle import oracle
    out = dict(opt_cost=[], plan=[], mem_used=[], status=[])
    for i in range(sub.B):
        Li = int(sub.L[i])
        r = oracle.search(sub.time_q[i, :Li], sub.mem_q[i, :Li], sub.trans_q[i], sub.M)
        plan = np.full(sub.Lmax, -1, np.int32); plan[:Li] = r["plan"]
        out["opt_cost"].append(r["opt_cost"]); out["plan"].append(plan)
        out["mem_used"].append(r["mem_used"]); out["status"].append(r["status"])
    return {k: np.asarray(v, np.int32) for k, v in out.items()}


def _worker(rank, world, port, q):
    import torch
    import torch.distributed as dist
    from paper_2504_03662_b200.sharding import search_sharded
    os.environ["MASTER_ADDR"], os.environ["MASTER_PORT"] = "127.0.0.1", str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        w = inputs.random_tables(123, 9, 7, 5, 60, ragged=True, mem_lo=1, mem_hi=25)
        w.time_q[4, 0, 0] = -1                                   # a flagged instance travels through the gather too
        res = search_sharded(w, _oracle_local, torch.device("cpu"))
        q.put((rank, {k: v.tolist() for k, v in res.items()}))
    finally:
        dist.destroy_process_group()


@pytest.mark.timeout(120)
def test_two_ranks_gather_the_whole_batch():
    from oracle import oracle
    oracle.build()
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    got = dict(q.get(timeout=100) for _ in range(2))
    for p in procs:
        p.join(timeout=30)
        assert p.exitcode == 0
    w = inputs.random_tables(123, 9, 7, 5, 60, ragged=True, mem_lo=1, mem_hi=25)
    w.time_q[4, 0, 0] = -1
    want = _oracle_local(w)
    for rank in (0, 1):
        for k in ("opt_cost", "plan", "mem_used", "status"):
            assert np.array_equal(np.asarray(got[rank][k]), want[k]), (rank, k)
    assert want["status"][4] == 2


def _cuda_worker(port, q):
    import torch
    import torch.distributed as dist
    from paper_2504_03662_b200 import binding as gb
    from paper_2504_03662_b200.search import SearchBuffers
    from paper_2504_03662_b200.sharding import search_sharded
    os.environ["MASTER_ADDR"], os.environ["MASTER_PORT"] = "127.0.0.1", str(port)
    torch.cuda.set_device(0)
    dist.init_process_group("nccl", rank=0, world_size=1, device_id=torch.device("cuda", 0))
    try:
        galv = gb.Galv(0)

        def local(sub):
            sb = SearchBuffers(galv, sub, gb.STORE_C_FULL)
            sb.step()
            return sb.results()

        out = {}
        for name, w in (("ragged", inputs.config2()), ("tables", inputs.config4(B=40))):
            res = search_sharded(w, local, torch.device("cuda", 0))
            whole = local(w)
            out[name] = all(np.array_equal(res[k], whole[k]) for k in ("opt_cost", "plan", "mem_used", "status"))
            out[name + "_feasible"] = int((res["status"] == 0).sum())
        galv.close()
        q.put(out)
    finally:
        dist.destroy_process_group()


@pytest.mark.gpu
@pytest.mark.timeout(300)
def test_cuda_path_through_the_sharded_search_over_nccl():
    """The sharded search with the CUDA path as the per-slice search, one rank, NCCL as the gather's backend:
    the gathered results equal those of the unsharded run (the only multi-GPU form one GPU can run)."""
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    p = ctx.Process(target=_cuda_worker, args=(port, q))
    p.start()
    got = q.get(timeout=280)
    p.join(timeout=30)
    assert p.exitcode == 0
    assert got["ragged"] and got["tables"] and got["ragged_feasible"] > 0 and got["tables_feasible"] == 40

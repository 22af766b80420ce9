"""One transition matrix per layer: oracle pins (CPU) and GPU parity."""
import numpy as np
import pytest

from paper_2504_03662_b200 import inputs

INF = 2 ** 30 - 1


def per_layer_workload(seed, B, Lmax, S, M, ragged=False):
    w = inputs.random_tables(seed, B, Lmax, S, M, ragged=ragged, mem_lo=0, mem_hi=max(1, M // 3), trans_hi=500)
    x = inputs.splitmix64(seed + 99, B * Lmax * S * S)
    w.trans_q = (x % np.uint64(501)).astype(np.int32).reshape(B, Lmax, S, S)
    return w


def test_hand_example(orc):
    # L=3, S=2, no memory.  Matrix 1 makes staying cheap, matrix 2 makes switching cheap:
    #   trans[1] = [[0,9],[9,0]], trans[2] = [[9,0],[0,9]], time = 1 everywhere.
    # Best: stay between layers 0-1, switch between 1-2: cost 3; plans [0,0,1] and [1,1,0];
    # ordered by (p2,p1,p0): (0,1,1) < (1,0,0) -> plan [1,1,0].
    time = np.ones((3, 2), int); mem = np.zeros((3, 2), int)
    trans = np.array([[[7, 7], [7, 7]], [[0, 9], [9, 0]], [[9, 0], [0, 9]]])     # matrix 0 is never used
    r = orc.search(time, mem, trans, 0)
    assert r["opt_cost"] == 3 and r["plan"].tolist() == [1, 1, 0]
    assert orc.brute_force(time, mem, trans, 0)[:2][0] == 3
    assert orc.plan_cost(time, mem, trans, [0, 1, 1]) == (1 + 9 + 1 + 9 + 1, 0)
    # a negative entry in the unused matrix 0 is not an error; one in matrix 1 is
    bad = trans.copy(); bad[0, 0, 0] = -5
    assert orc.validate(time, mem, bad) == 0
    bad = trans.copy(); bad[1, 0, 0] = -5
    assert orc.validate(time, mem, bad) == orc.BAD_INPUT


@pytest.mark.parametrize("seed", range(60))
def test_oracle_dp_against_enumeration(orc, seed):
    rng = np.random.default_rng(seed)
    L, S, M = int(rng.integers(1, 6)), int(rng.integers(1, 5)), int(rng.integers(0, 30))
    w = per_layer_workload(2000 + seed, 1, L, S, M)
    t, m, x = w.time_q[0], w.mem_q[0], w.trans_q[0]
    Ct, At = orc.dp(t, m, x, M)
    for budget in sorted({0, M // 2, M}):
        eo, ep, eu, _ = orc.brute_force(t, m, x, budget)
        for A in (None, At):
            o, p, u, st = orc.backtrack(t, m, x, Ct, A, budget)
            assert o == eo and p.tolist() == ep.tolist()
            if eo < INF:
                assert u == eu and orc.plan_cost(t, m, x, p) == (o, u)


def test_equal_matrices_reduce_to_one(orc):
    w = inputs.random_tables(5, 1, 6, 4, 40, mem_lo=0, mem_hi=12)
    t, m, x = w.time_q[0], w.mem_q[0], w.trans_q[0]
    a = orc.search(t, m, x, 40)
    b = orc.search(t, m, np.repeat(x[None], 6, 0), 40)
    assert a["opt_cost"] == b["opt_cost"] and (a["plan"] == b["plan"]).all() and (a["C"] == b["C"]).all()


@pytest.mark.gpu
@pytest.mark.parametrize("flags", [1, 1 | 16384, 3, 2, 1 | 512, 1 | 8192 | 1024 | 16384, 1 | 8192 | 4096 | 16384, 1 | 32768 | (3 << 16), 32768])
# plain (the cluster kernel takes a batch this small), tiled kernels only, tables, per layer; skipping flags on the packed and
# the 32-bit loop of the tiled kernel; clusters of three CTAs; the cluster kernel without a table
def test_gpu_parity(orc, flags):
    import torch
    from paper_2504_03662_b200 import binding as gb
    from paper_2504_03662_b200.search import SearchBuffers, HostSearch
    galv = gb.Galv(0)
    try:
        for k, (B, Lmax, S, M, ragged) in enumerate([(3, 6, 8, 300, True), (2, 5, 13, 200, False), (2, 9, 64, 700, True),
                                                      (2, 4, 70, 300, False)]):
            w = per_layer_workload(50 + k, B, Lmax, S, M, ragged)
            sb = SearchBuffers(galv, w, flags)
            assert sb.shape.flags & gb.TRANS_PER_LAYER
            sb.dp_search(); sb.backtrack()
            res = sb.results()
            for i in range(B):
                Li = int(w.L[i])
                r = orc.search(w.time_q[i, :Li], w.mem_q[i, :Li], w.trans_q[i, :Li], M)
                assert res["opt_cost"][i] == r["opt_cost"] and res["status"][i] == r["status"]
                if flags & (gb.STORE_C_FULL | gb.STORE_ARGMIN):         # a plan needs a table
                    assert (res["plan"][i, :Li] == r["plan"]).all() and res["mem_used"][i] == r["mem_used"]
                else:
                    assert (sb.C_last[i, :, :M + 1].t().cpu().numpy() == r["C"][Li - 1]).all()
                if flags & gb.STORE_C_FULL:
                    assert (sb.table(i)[:Li] == r["C"]).all()
                if flags & gb.STORE_ARGMIN:
                    assert (sb.argmin_table(i)[:Li] == r["A"]).all()
            if flags & 1 and not flags & 2 and not flags & 512:
                cost = torch.empty(B, dtype=torch.int64, device=sb.dev); used = torch.empty_like(cost)
                galv.galv_plan_cost(sb.shape, sb.L, sb.time_q, sb.mem_q, sb.trans_q, sb.plan, cost, used)
                hs = HostSearch(galv, w, 1).run()
                torch.cuda.synchronize()
                ok = res["status"] == 0
                assert (cost.cpu().numpy()[ok] == res["opt_cost"][ok]).all()
                assert (hs["opt_cost"] == res["opt_cost"]).all() and (hs["plan"] == res["plan"]).all()
    finally:
        galv.close()

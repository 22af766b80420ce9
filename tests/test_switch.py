"""Plan switch: amortised resharding cost added to the tables, and the decision with hysteresis.

Oracle pins on CPU (hand example, closed forms, enumeration of all plans), GPU parity through the C boundary.
"""
import itertools

import numpy as np
import pytest

from paper_2504_03662_b200 import inputs

INF = 2 ** 30 - 1


def test_hand_example(orc):
    time = np.array([[5, 3], [4, 6]], np.int32)
    trans = np.array([[0, 20], [10, 0]], np.int32)
    # layer 0 runs strategy 0: moving it to 1 costs 20, over 4 iterations 5 each; layer 1 runs 1: moving to 0 costs 10 -> 2
    assert orc.add_switch_cost(time, trans, [0, 1], 4).tolist() == [[5, 8], [6, 6]]
    # no plan yet: nothing is added; a horizon below 1 counts as 1
    assert (orc.add_switch_cost(time, trans, [-1, -1], 4) == time).all()
    assert orc.add_switch_cost(time, trans, [0, 1], 0).tolist() == [[5, 23], [14, 6]]
    # one matrix per layer: layer l takes matrix l
    t3 = np.stack([trans, 3 * trans])
    assert orc.add_switch_cost(time, t3, [0, 1], 1).tolist() == [[5, 23], [34, 6]]
    # saturation
    big = np.array([[INF - 3, 1]], np.int32)
    assert orc.add_switch_cost(big, np.array([[7, 7], [7, 7]], np.int32), [1], 1).tolist() == [[INF, 8]]


def test_decision_table(orc):
    assert orc.switch_decision(100, 90, 100) == 1            # 90 * 1.1 = 99 < 100
    assert orc.switch_decision(100, 91, 100) == 0            # 100.1
    assert orc.switch_decision(1000, 1000, 0) == 0 and orc.switch_decision(1000, 999, 0) == 1
    assert orc.switch_decision(INF, 5, 500) == 1             # the running plan no longer fits
    assert orc.switch_decision(5, INF, 0) == 0 and orc.switch_decision(INF, INF, 0) == 0
    assert orc.switch_decision(2 ** 40, 2 ** 29, 1000) == 1  # 64-bit products


@pytest.mark.parametrize("seed", range(30))
def test_search_with_switch_cost_against_all_plans(orc, seed):
    """DP on the amended table = min over all plans of iteration cost + sum of amortised moves."""
    rng = np.random.default_rng(seed)
    L, S, M = int(rng.integers(1, 5)), int(rng.integers(1, 5)), int(rng.integers(5, 40))
    w = inputs.random_tables(900 + seed, 1, L, S, M, mem_lo=0, mem_hi=max(1, M // 2), time_hi=200, trans_hi=90)
    time, mem, trans = w.time_q[0], w.mem_q[0], w.trans_q[0]
    cur = rng.integers(-1, S, size=L).astype(np.int32)
    H = int(rng.integers(1, 7))
    amended = orc.add_switch_cost(time, trans, cur, H)
    got = orc.search(amended, mem, trans, M, use_A=False)
    best = None
    for p in itertools.product(range(S), repeat=L):
        if sum(int(mem[l, p[l]]) for l in range(L)) > M:
            continue
        c = sum(int(time[l, p[l]]) for l in range(L)) + sum(int(trans[p[l - 1], p[l]]) for l in range(1, L))
        c += sum(int(trans[cur[l], p[l]]) // H for l in range(L) if cur[l] >= 0)
        key = (c, tuple(reversed(p)))
        best = key if best is None or key < best else best
    if best is None:
        assert got["opt_cost"] == INF
    else:
        assert got["opt_cost"] == best[0] and tuple(reversed(got["plan"].tolist())) == best[1]


def test_staying_is_free_and_long_horizons_change_nothing(orc):
    w = inputs.random_tables(77, 1, 6, 5, 60, mem_lo=1, mem_hi=20, trans_hi=500)
    time, mem, trans = w.time_q[0], w.mem_q[0], w.trans_q[0]
    np.fill_diagonal(trans, 0)                               # a layout costs nothing to keep
    base = orc.search(time, mem, trans, 60, use_A=False)
    # horizon beyond every entry: the table is unchanged
    assert (orc.add_switch_cost(time, trans, base["plan"], 10 ** 6) == time).all()
    # the running plan is the optimum: it stays the optimum at the same cost for every horizon
    for H in (1, 3, 50):
        again = orc.search(orc.add_switch_cost(time, trans, base["plan"], H), mem, trans, 60, use_A=False)
        assert again["opt_cost"] == base["opt_cost"] and (again["plan"] == base["plan"]).all()
        assert orc.switch_decision(base["opt_cost"], again["opt_cost"], 0) == 0


@pytest.mark.gpu
@pytest.mark.parametrize("per_layer", [False, True])
def test_gpu_switch_cost_and_decision(orc, per_layer):
    import torch
    from paper_2504_03662_b200 import binding as gb
    from paper_2504_03662_b200.search import SearchBuffers
    galv = gb.Galv(0)
    try:
        B, Lm, S, M = 9, 7, 12, 300
        w = inputs.random_tables(55, B, Lm, S, M, ragged=True, mem_lo=1, mem_hi=80, trans_hi=4000)
        if per_layer:
            x = np.stack([w.trans_q * (l + 1) % 3001 for l in range(Lm)], axis=1).astype(np.int32)
            w = inputs.Workload(w.name, B, Lm, S, M, w.L, w.time_q, w.mem_q, x)
        rng = np.random.default_rng(5)
        cur = rng.integers(-1, S, size=(B, Lm)).astype(np.int32)
        horizon = rng.integers(0, 9, size=B).astype(np.int32)
        w.time_q[3, 1, 2] = INF - 5                          # saturates
        sb = SearchBuffers(galv, w, gb.STORE_C_FULL)
        dev = sb.dev
        d_cur, d_h = torch.from_numpy(cur).to(dev), torch.from_numpy(horizon).to(dev)
        amended = torch.empty_like(sb.time_q)
        galv.galv_add_switch_cost(sb.shape, sb.L, sb.time_q, sb.trans_q, d_cur, d_h, amended)
        torch.cuda.synchronize()
        got = amended.cpu().numpy()
        for i in range(B):
            Li = int(w.L[i])
            ref = orc.add_switch_cost(w.time_q[i, :Li], w.trans_q[i][:Li] if per_layer else w.trans_q[i], cur[i, :Li], int(horizon[i]))
            assert (got[i, :Li] == ref).all(), i
            assert (got[i, Li:] == w.time_q[i, Li:]).all()
        # search the amended tables, price the running plans, decide
        w2 = inputs.Workload(w.name, B, Lm, S, M, w.L, got, w.mem_q, w.trans_q)
        w2.time_q[3, 1, 2] = 0                               # keep instance 3 valid for the search
        sb2 = SearchBuffers(galv, w2, gb.STORE_C_FULL)
        sb2.dp_search(); sb2.backtrack()
        stay = np.where(cur < 0, 0, cur).astype(np.int32)
        d_stay = torch.from_numpy(stay).to(dev)
        cost = torch.empty(B, dtype=torch.int64, device=dev); memt = torch.empty(B, dtype=torch.int64, device=dev)
        galv.galv_plan_cost(sb.shape, sb.L, sb.time_q, sb.mem_q, sb.trans_q, d_stay, cost, memt)
        cost[1] = INF                                        # a running plan that no longer fits
        cost[2] = -1
        dec = torch.empty(B, dtype=torch.int32, device=dev)
        for h in (0, 50, 400):
            galv.galv_switch_decision(B, cost, sb2.opt_cost, sb2.status, h, dec)
            torch.cuda.synchronize()
            c, n, st = cost.cpu().numpy(), sb2.opt_cost.cpu().numpy(), sb2.status.cpu().numpy()
            for i in range(B):
                want = 0 if st[i] != 0 else orc.switch_decision(INF if c[i] < 0 else int(c[i]), int(n[i]), h)
                assert dec[i].item() == want, (i, h)
        with pytest.raises(gb.GalvError):
            galv.galv_switch_decision(B, cost, sb2.opt_cost, sb2.status, -1, dec)
    finally:
        galv.close()

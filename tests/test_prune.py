"""Dominated-strategy prune: oracle pins on CPU, GPU parity and end-to-end equivalence."""
import numpy as np
import pytest

from paper_2504_03662_b200 import inputs

INF = 2 ** 30 - 1


def dominated_workload(seed, B, Lmax, S, M, ragged=False):
    """Random tables where several strategies are copies of others made worse (or equal)."""
    w = inputs.random_tables(seed, B, Lmax, S, M, ragged=ragged, mem_lo=1, mem_hi=max(2, M // 4), trans_hi=50, time_hi=200)
    rng = np.random.default_rng(seed)
    for _ in range(max(1, S // 2)):
        d, s = rng.choice(S, 2, replace=False)
        kind = rng.integers(3)
        dt = 0 if kind == 0 else int(rng.integers(0, 3))           # equal copy, or worse by a little
        w.time_q[:, :, s] = w.time_q[:, :, d] + (1 if kind == 2 else dt)   # kind 2: strictly slower everywhere
        w.mem_q[:, :, s] = w.mem_q[:, :, d] + int(rng.integers(0, 2))
        w.trans_q[:, :, s] = w.trans_q[:, :, d] + int(rng.integers(0, 2))
        w.trans_q[:, s, :] = w.trans_q[:, d, :] + int(rng.integers(0, 2))
        w.trans_q[:, s, s] = w.trans_q[:, d, d] + 1
        w.trans_q[:, s, d] = np.maximum(w.trans_q[:, s, d], w.trans_q[:, d, d])
        w.trans_q[:, d, s] = np.maximum(w.trans_q[:, d, s], w.trans_q[:, d, d])
    return w


def test_hand_example(orc):
    # strategy 1 = strategy 0 made slower by 1 (dominated, higher index); strategy 2 is strategy 3 with
    # equal time and more memory (dominated only by a HIGHER index with equal time: must stay);
    # strategy 4 is strictly slower than strategy 5 everywhere (dominated by a higher index, strictly: goes)
    # (strategy 0 has the least memory, so nothing dominates it)
    time = np.array([[[10, 11, 7, 7, 9, 8]]]); mem = np.array([[[1, 1, 5, 4, 2, 2]]])
    trans = np.zeros((1, 6, 6), int)
    assert orc.prune([1], time, mem, trans).tolist() == [1, 0, 1, 1, 0, 1]
    # a transition that is worse for the would-be dominator protects the strategy
    trans[0, 2, 0] = 5                                   # entering 0 from 2 costs more than entering 1 from 2
    assert orc.prune([1], time, mem, trans).tolist() == [1, 1, 1, 1, 0, 1]


@pytest.mark.parametrize("seed", range(40))
def test_pruned_search_equals_full_search_by_enumeration(orc, seed):
    rng = np.random.default_rng(seed)
    L, S, M = int(rng.integers(1, 5)), int(rng.integers(2, 7)), int(rng.integers(5, 30))
    w = dominated_workload(300 + seed, 2, L, S, M)
    keep = orc.prune(w.L, w.time_q, w.mem_q, w.trans_q)
    kept = np.flatnonzero(keep)
    assert keep[0] == 1 or S > 1
    for i in range(w.B):
        t, m, x = w.time_q[i], w.mem_q[i], w.trans_q[i]
        for budget in (0, M // 2, M):
            o, p, u, _ = orc.brute_force(t, m, x, budget)                      # all strategies
            o2, p2, u2, _ = orc.brute_force(t[:, kept], m[:, kept], x[np.ix_(kept, kept)], budget)
            assert o == o2 and u == u2
            if o < INF:
                assert (kept[p2] == p).all()                                   # the very same plan


def test_nothing_to_prune_and_identical_copies(orc):
    w = inputs.config4(B=2)
    assert orc.prune(w.L, w.time_q, w.mem_q, w.trans_q).all()                  # dense random tables: nothing dominated
    w = inputs.random_tables(1, 1, 3, 4, 20, dup_cols=True)                    # strategy 3 is a copy of strategy 0
    assert orc.prune(w.L, w.time_q, w.mem_q, w.trans_q).tolist() == [1, 1, 1, 0]


@pytest.mark.gpu
def test_gpu_prune_matches_oracle_and_preserves_the_search(orc):
    import torch
    from paper_2504_03662_b200 import binding as gb
    from paper_2504_03662_b200.search import SearchBuffers
    galv = gb.Galv(0)
    try:
        cases = [dominated_workload(7, 5, 6, 12, 120, ragged=True), dominated_workload(8, 3, 4, 40, 300),
                 inputs.config4(B=4), inputs.config2()]
        for w in cases:
            full = SearchBuffers(galv, w, gb.STORE_C_FULL)
            if w.has_model:
                full.eval_costs()
            dev = full.dev
            keep = torch.empty(w.S, dtype=torch.int32, device=dev); mp = torch.empty_like(keep)
            n = torch.empty(1, dtype=torch.int32, device=dev)
            galv.galv_prune_strategies(full.shape, full.L, full.time_q, full.mem_q, full.trans_q, keep, mp, n)
            torch.cuda.synchronize()
            tq, mq, xq = (a.cpu().numpy() for a in (full.time_q, full.mem_q, full.trans_q))
            ref_keep = orc.prune(w.L, tq, mq, xq)
            assert (keep.cpu().numpy() == ref_keep).all()
            S2 = int(n.item())
            assert S2 == ref_keep.sum() and (mp.cpu().numpy()[:S2] == np.flatnonzero(ref_keep)).all() and (mp[S2:] == -1).all()
            full.dp_search(); full.backtrack()
            want = full.results()
            # the same search on the kept strategies only
            small = inputs.Workload(w.name + "_pruned", w.B, w.Lmax, S2, w.M, w.L,
                                    np.zeros((w.B, w.Lmax, S2), np.int32), np.zeros((w.B, w.Lmax, S2), np.int32),
                                    np.zeros((w.B, S2, S2), np.int32))
            sb = SearchBuffers(galv, small, gb.STORE_C_FULL)
            galv.galv_compact_tables(full.shape, S2, mp, full.time_q, full.mem_q, full.trans_q, sb.time_q, sb.mem_q, sb.trans_q)
            sb.dp_search(); sb.backtrack()
            galv.galv_expand_plan(w.B, w.Lmax, mp, sb.plan)
            got = sb.results()
            for k in ("opt_cost", "plan", "mem_used", "status"):
                assert (got[k] == want[k]).all(), (w.name, k)
            if w.name.startswith("config2"):
                assert S2 < w.S                                  # sequence parallelism is a no-op at tp = 1: copies go
    finally:
        galv.close()

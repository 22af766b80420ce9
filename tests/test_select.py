"""Outer selection over the instance batch: oracle pins (CPU) and GPU parity."""
import numpy as np
import pytest

from paper_2504_03662_b200 import inputs

INF = 2 ** 30 - 1


def random_candidates(seed, B, G):
    rng = np.random.default_rng(seed)
    opt = rng.integers(1, 50, size=B).astype(np.int32) * 1000           # coarse values: many ties
    opt[rng.random(B) < 0.15] = INF
    status = np.where(opt == INF, 1, 0).astype(np.int32)
    status[rng.random(B) < 0.05] = 2
    n_micro = rng.integers(0, 40, size=B).astype(np.int32)              # 0 is invalid: ignored
    pp = rng.choice([1, 2, 4, 8, 16], size=B).astype(np.int32)
    group = rng.integers(-1, G + 1, size=B).astype(np.int32)            # -1 and G are out of range: ignored
    return opt, status, n_micro, pp, group


def test_hand_example(orc):
    # three candidates of one group: (n_micro + pp - 1) * t = (8+1-1)*100 = 800, (4+2-1)*150 = 750, (2+4-1)*150 = 750
    bt, bi = orc.select_best([100, 150, 150, 90], [0, 0, 0, 1], [8, 4, 2, 1], [1, 2, 4, 1], [0, 0, 0, 0], 2)
    assert bt.tolist() == [750, -1] and bi.tolist() == [1, -1]          # tie -> lower index; infeasible ignored


@pytest.mark.parametrize("seed", range(20))
def test_oracle_against_sorting(orc, seed):
    B, G = 300, 7
    opt, status, n_micro, pp, group = random_candidates(seed, B, G)
    bt, bi = orc.select_best(opt, status, n_micro, pp, group, G)
    t = (n_micro.astype(np.int64) + pp - 1) * opt.astype(np.int64)
    ok = (status == 0) & (opt < INF) & (n_micro >= 1) & (pp >= 1) & (group >= 0) & (group < G)
    for g in range(G):
        idx = np.flatnonzero(ok & (group == g))
        if len(idx) == 0:
            assert (bt[g], bi[g]) == (-1, -1)
        else:
            k = idx[np.lexsort((idx, t[idx]))[0]]                       # by time, then by index
            assert (bt[g], bi[g]) == (t[k], k)


@pytest.mark.gpu
def test_gpu_select_matches_oracle(orc):
    import torch
    from paper_2504_03662_b200 import binding as gb
    galv = gb.Galv(0)
    try:
        for seed, (B, G) in enumerate([(1, 1), (64, 1), (1000, 13), (5000, 300)]):
            arrs = random_candidates(100 + seed, B, G)
            dev = [torch.from_numpy(a).cuda() for a in arrs]
            bt = torch.empty(G, dtype=torch.int64, device="cuda")
            bi = torch.empty(G, dtype=torch.int32, device="cuda")
            galv.galv_select_best(B, G, *dev, bt, bi)
            torch.cuda.synchronize()
            rt, ri = orc.select_best(*arrs, G)
            assert (bt.cpu().numpy() == rt).all() and (bi.cpu().numpy() == ri).all()
    finally:
        galv.close()


@pytest.mark.gpu
def test_gpu_search_then_select_config2(orc):
    """The 175B-shaped sweep: per-stage optima from the search, then the best (micro-batch, pipeline degree)."""
    import torch
    from paper_2504_03662_b200 import binding as gb
    from paper_2504_03662_b200.search import SearchBuffers
    galv = gb.Galv(0)
    try:
        w = inputs.config2()
        sb = SearchBuffers(galv, w, gb.STORE_C_FULL)
        sb.step()
        global_batch = 1024
        n_micro = torch.from_numpy(np.ceil(global_batch / w.meta["b"]).astype(np.int32)).cuda()
        pp = torch.from_numpy(w.meta["pp"].astype(np.int32)).cuda()
        group = torch.zeros(w.B, dtype=torch.int32, device="cuda")
        bt = torch.empty(1, dtype=torch.int64, device="cuda"); bi = torch.empty(1, dtype=torch.int32, device="cuda")
        galv.galv_select_best(w.B, 1, sb.opt_cost, sb.status, n_micro, pp, group, bt, bi)
        res = sb.results()
        rt, ri = orc.select_best(res["opt_cost"], res["status"], n_micro.cpu().numpy(), pp.cpu().numpy(),
                                 group.cpu().numpy(), 1)
        assert bt.item() == rt[0] and bi.item() == ri[0] and ri[0] >= 0
    finally:
        galv.close()

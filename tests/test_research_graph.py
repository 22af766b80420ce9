"""Re-search pipeline in a CUDA graph, and the cost of a given plan (GPU)."""
import numpy as np
import pytest

from paper_2504_03662_b200 import inputs

pytestmark = pytest.mark.gpu


def oracle_all(orc, w):
    out = []
    for i in range(w.B):
        Li = int(w.L[i])
        _, _, tq, mq, xq = orc.eval_costs(w.layers[0], w.strat, w.inst[i], Li)
        out.append((tq, mq, xq, orc.search(tq, mq, xq, w.M)))
    return out


def test_graph_replay_follows_updated_parameters(orc):
    import torch
    from paper_2504_03662_b200 import binding as gb
    from paper_2504_03662_b200.search import SearchBuffers, _dev_bytes
    galv = gb.Galv(0)
    try:
        w = inputs.config1().take(slice(0, 6))
        sb = SearchBuffers(galv, w, gb.STORE_C_FULL)
        side = torch.cuda.Stream()
        torch.cuda.synchronize()
        graph = galv.galv_graph_create(sb.shape, sb.L, sb.layers, sb.layer_stride_B, sb.strat, sb.inst, sb.time_q, sb.mem_q,
                                       sb.trans_q, sb.C, None, sb.C_last, sb.workspace, None, sb.opt_cost, sb.plan,
                                       sb.mem_used, sb.status, side.cuda_stream)
        cost = torch.empty(w.B, dtype=torch.int64, device=sb.dev); used = torch.empty_like(cost)
        old_plan = None
        # three "monitoring intervals": nominal, links at 40 % of nominal, compute at half speed
        for step, (bw, rate) in enumerate(((450e9, 1e15), (180e9, 1e15), (450e9, 0.5e15))):
            w.inst["bw_tp"] = bw; w.inst["bw_dp"] = bw; w.inst["flops_rate"] = rate
            sb.inst.copy_(_dev_bytes(w.inst, sb.dev))               # parameters change in place
            torch.cuda.synchronize()
            galv.galv_graph_launch(graph, side.cuda_stream)
            side.synchronize()
            res = sb.results()
            ref = oracle_all(orc, w)
            for i, (tq, mq, xq, r) in enumerate(ref):
                assert res["opt_cost"][i] == r["opt_cost"] and (res["plan"][i] == r["plan"]).all(), (step, i)
                assert res["status"][i] == r["status"] and res["mem_used"][i] == r["mem_used"]
            if old_plan is not None:
                # what the previous interval's plan costs under the new measurements
                galv.galv_plan_cost(sb.shape, sb.L, sb.time_q, sb.mem_q, sb.trans_q, old_plan, cost, used)
                torch.cuda.synchronize()
                for i, (tq, mq, xq, r) in enumerate(ref):
                    c, u = orc.plan_cost(tq, mq, xq, old_plan[i].cpu().numpy())
                    assert (cost[i].item(), used[i].item()) == (c, u)
                    assert c >= r["opt_cost"] or u > w.M            # the new optimum is no worse than keeping the old plan
            old_plan = sb.plan.clone()
        galv.galv_graph_destroy(graph)
    finally:
        galv.close()


def test_plan_cost_edge_cases(orc):
    import torch
    from paper_2504_03662_b200 import binding as gb
    from paper_2504_03662_b200.search import SearchBuffers
    galv = gb.Galv(0)
    try:
        w = inputs.random_tables(77, 5, 40, 9, 100, ragged=True)
        sb = SearchBuffers(galv, w, gb.STORE_C_FULL)
        rng = np.random.default_rng(0)
        plan = rng.integers(0, 9, size=(5, 40)).astype(np.int32)
        plan[3, 0] = -1                                             # invalid entry inside the instance's layers
        plan[4, int(w.L[4]):] = -1                                  # beyond L[i] anything goes
        dplan = torch.from_numpy(plan).to(sb.dev)
        cost = torch.empty(5, dtype=torch.int64, device=sb.dev); used = torch.empty_like(cost)
        galv.galv_plan_cost(sb.shape, sb.L, sb.time_q, sb.mem_q, sb.trans_q, dplan, cost, used)
        torch.cuda.synchronize()
        for i in range(5):
            Li = int(w.L[i])
            if i == 3:
                assert cost[i].item() == -1 and used[i].item() == -1
            else:
                assert (cost[i].item(), used[i].item()) == orc.plan_cost(w.time_q[i, :Li], w.mem_q[i, :Li], w.trans_q[i], plan[i, :Li])
    finally:
        galv.close()

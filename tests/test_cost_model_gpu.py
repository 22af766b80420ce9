"""The cost-model kernel against the oracle: layer stacks with many, few and no repeats, descriptor checks."""
import numpy as np
import pytest

from paper_2504_03662_b200 import inputs

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def galv():
    import torch
    from paper_2504_03662_b200 import binding as gb
    assert torch.cuda.is_available()
    g = gb.Galv(0)
    yield g
    g.close()


def stack(seed, B, Lmax, strat, pattern, per_instance=False, ragged=False):
    """A batch whose layers follow `pattern`: 'uniform', 'alternate', a repeat period, or 'distinct' (no two alike)."""
    rng = np.random.default_rng(seed)
    rows = B if per_instance else 1
    layers = np.empty((rows, Lmax), inputs.LAYER_DESC)
    kinds = ("full", "attention", "ffn")
    for r in range(rows):
        for l in range(Lmax):
            if pattern == "uniform":
                k, h = 0, 2048.0
            elif pattern == "alternate":
                k, h = 1 + l % 2, 4096.0
            elif pattern == "distinct":
                k, h = l % 3, 1024.0 + 64.0 * l + 8.0 * r
            else:                                              # a period longer or shorter than the twin window
                k, h = (l % pattern) % 3, 1024.0 + 128.0 * (l % pattern)
            layers[r, l] = inputs.layer_desc(kinds[k], h, 1024.0 + 512.0 * (k == 1), h / 128.0)
    inst = inputs._inst(B, b=rng.integers(1, 9, B).astype(np.float64), act_mult=rng.integers(1, 5, B).astype(np.float64),
                        flops_rate=1e15 * (0.8 + 0.4 * rng.random(B)), bw_tp=450e9 * (0.8 + 0.4 * rng.random(B)),
                        bw_dp=300e9 * (0.8 + 0.4 * rng.random(B)), time_unit_ns=10.0)
    L = rng.integers(1, Lmax + 1, B).astype(np.int32) if ragged else np.full(B, Lmax, np.int32)
    return inputs.Workload(f"stack_{pattern}", B, Lmax, len(strat), 2880, L, layers=layers, strat=strat, inst=inst)


def run_and_compare(orc, galv, w, want_fp64):
    import torch
    from paper_2504_03662_b200.search import SearchBuffers
    sb = SearchBuffers(galv, w, 1)
    sb.time_q.fill_(-7); sb.mem_q.fill_(-7); sb.trans_q.fill_(-7)
    sb.eval_costs(want_fp64=want_fp64)
    torch.cuda.synchronize()
    tq, mq, xq, st = (t.cpu().numpy() for t in (sb.time_q, sb.mem_q, sb.trans_q, sb.status))
    for i in range(w.B):
        Li = int(w.L[i])
        rows = w.layers[0 if w.layers.shape[0] == 1 else i]
        rts, rmb, rtq, rmq, rxq = orc.eval_costs(rows, w.strat, w.inst[i], Li)
        assert st[i] == orc.descriptor_status(rows, w.strat, w.inst[i], Li), i
        assert (tq[i, :Li] == rtq).all() and (mq[i, :Li] == rmq).all() and (xq[i] == rxq).all(), i
        assert (tq[i, Li:] == -7).all() and (mq[i, Li:] == -7).all()              # rows beyond L[i] are left untouched
        if want_fp64 and st[i] == 0:
            np.testing.assert_allclose(sb.time_s[i, :Li].cpu().numpy(), rts, rtol=1e-12, atol=0)
            np.testing.assert_allclose(sb.mem_bytes[i, :Li].cpu().numpy(), rmb, rtol=1e-12, atol=0)
    return sb


@pytest.mark.parametrize("pattern", ["uniform", "alternate", "distinct", 3, 9, 13])
@pytest.mark.parametrize("want_fp64", [False, True])
def test_layer_stacks_with_and_without_repeats(orc, galv, pattern, want_fp64):
    strat48 = inputs.strategy_table((1, 2, 4, 8), (0, 2, 3), (0, 1), (0, 1))
    strat6 = inputs.strategy_table((1, 2, 8), (0, 3), (1,), (0,))                  # S = 6: the scalar store path
    for seed, (B, Lmax, strat, per_instance) in enumerate([(5, 40, strat48, False), (3, 17, strat6, True), (2, 300, strat48, True)]):
        w = stack(seed, B, Lmax, strat, pattern, per_instance=per_instance, ragged=seed == 1)
        run_and_compare(orc, galv, w, want_fp64)


def test_very_long_stack_takes_the_direct_kernels(orc, galv):
    strat = inputs.strategy_table((1, 8), (0, 3), (0,), (0, 1))
    w = stack(77, 2, 20000, strat, 5)                                              # the per-instance index arrays pass 200 KB
    w.L[1] = 12345
    run_and_compare(orc, galv, w, False)


def test_bad_descriptors_flag_the_instance_end_to_end(orc, galv):
    import torch
    from paper_2504_03662_b200 import binding as gb
    strat = inputs.strategy_table((1, 2, 4, 8), (0, 2, 3), (0, 1), (0,))
    w = stack(5, 6, 12, strat, "alternate", per_instance=True)
    w.inst["bw_dp"][1] = 0.0                                    # a dead link
    w.inst["flops_rate"][2] = float("nan")
    w.layers["h"][3, 7] = -1.0                                  # inside the instance's layers
    w.L[4] = 5
    w.layers["seq"][4, 9] = 0.0                                 # beyond its 5 layers: not looked at
    sb = run_and_compare(orc, galv, w, True)
    assert sb.status.cpu().tolist() == [0, 2, 2, 2, 0, 0]
    sb.dp_search(); sb.backtrack()
    res = sb.results()
    assert res["status"].tolist()[1:4] == [2, 2, 2] and (res["plan"][1:4] == -1).all() and (res["opt_cost"][1:4] == 2 ** 30 - 1).all()
    assert res["status"][0] in (0, 1) and res["status"][4] in (0, 1)
    # a bad strategy table flags every instance
    w2 = stack(6, 3, 4, strat.copy(), "uniform")
    w2.strat["tp"][5] = 0
    sb2 = run_and_compare(orc, galv, w2, False)
    assert sb2.status.cpu().tolist() == [2, 2, 2]


def test_large_batch_takes_two_kernels_and_small_batch_one(orc, galv):
    """Past 1024 instances the layer tables and the transition matrices come from two launches (the second reads the
    first's status word for each instance); up to 1024 from one (the transition CTAs test the descriptors themselves).
    Both must agree with the oracle, flagged instances included."""
    strat = inputs.strategy_table((1, 2, 4, 8), (0, 3), (0, 1), (0, 1))
    for B in (1024, 1100):
        w = stack(90 + B, B, 9, strat, "alternate", per_instance=True, ragged=True)
        w.inst["bw_tp"][B - 3] = -1.0                           # flagged by the instance parameters
        w.layers["h"][B // 2, 0] = 0.0                          # flagged by a layer (every instance has at least one)
        sb = run_and_compare(orc, galv, w, False)
        st = sb.status.cpu().numpy()
        assert st[B - 3] == 2 and st[B // 2] == 2 and (st != 0).sum() == 2
        assert (sb.trans_q[B - 3].cpu().numpy() == -1).all() and (sb.trans_q[B // 2].cpu().numpy() == -1).all()

"""Pins for the CPU oracle's cost model (no GPU).

What has an outside definition is pinned by closed forms worked by hand in the
comments: the transformer FLOP count 24 b s h^2 + 4 b s^2 h, the x3 / x4
forward+backward(+recompute) factor, ring all-reduce volumes 2(n-1)/n, the
16-bytes-per-parameter mixed-precision Adam state and its ZeRO sharding, unit
conversion and rounding.  Activation, ZeRO-3 traffic, sequence-parallel and
resharding terms are this build's own accounting: they are checked for
self-consistency only (parity unpinned).
"""
from fractions import Fraction as F

import numpy as np
import pytest

from paper_2504_03662_b200 import inputs


def one(orc, w, i, L=None):
    layers = w.layers[0 if w.layers.shape[0] == 1 else i]
    return orc.eval_costs(layers, w.strat, w.inst[i], int(w.L[i]) if L is None else L)


def test_config1_closed_forms(orc):
    w = inputs.config1()
    ts, mb, tq, mq, xq = one(orc, w, 0)              # b = 1
    s, h = 2048, 2048
    assert 24 * s * h * h + 4 * s * s * h == 28 * 2 ** 33
    # s=0: tp1 dp8 ZeRO-0 no ckpt.  compute 3*28*2^33/1e15 s; no tp traffic;
    # dp all-reduce 2*(7/8) * 12 h^2 * 2 B / 450e9
    t_comp = F(3 * 28 * 2 ** 33, 10 ** 15)
    t_dp = F(7, 4) * F(12 * h * h * 2, 450 * 10 ** 9)
    assert ts[0, 0] == pytest.approx(float(t_comp + t_dp), rel=1e-15)
    assert float(t_comp) == pytest.approx(7.215545057e-4, rel=1e-9) and float(t_dp) == pytest.approx(3.914683733e-4, rel=1e-9)
    assert tq[0, 0] == 1113023
    # memory: 16 B/param * 12 h^2 + s*b*h*(10+24) + 5*16 heads*s^2 = 1 283 457 024 B -> 20 bins of 64 MiB
    assert mb[0, 0] == 16 * 12 * h * h + s * h * 34 + 5 * 16 * s * s == 1283457024
    assert mq[0, 0] == 20 == -(-1283457024 // (64 * 2 ** 20))
    # with recomputation the compute term is 4/3 as long
    assert ts[0, 1] == pytest.approx(float(F(4, 3) * t_comp + t_dp), rel=1e-15) and tq[0, 1] == 1353541 and mq[0, 1] == 13
    assert tq[0, 5] == 1549275 and mq[0, 5] == 2         # ZeRO-3 + ckpt
    assert tq[0, 12] == 348161 and mq[0, 12] == 6        # tp4 dp2 ZeRO-0
    assert tq[0, 23] == 250749 and mq[0, 23] == 2        # tp8 dp1 ZeRO-3 ckpt
    # tp8: compute/8 (x4), 4 all-reduces of 2*(7/8)*s*h*2 B, no dp traffic
    t23 = F(4 * 28 * 2 ** 33, 8 * 10 ** 15) + 4 * F(7, 4) * F(s * h * 2, 450 * 10 ** 9)
    assert ts[0, 23] == pytest.approx(float(t23), rel=1e-15)
    ts16, _, tq16, mq16, _ = one(orc, w, 15)          # b = 16
    assert tq16[0, 0] == 11936340 and mq16[0, 0] == 126 and tq16[0, 23] == 4011977 and mq16[0, 23] == 4
    # uniform layers: every row equal
    assert (tq == tq[0]).all() and (mq == mq[0]).all()
    assert w.strat["tp"][0] == 1 and w.strat["dp"][0] == 8 and w.strat["zero"][5] == 3 and w.strat["ckpt"][5] == 1
    assert tuple(w.strat[23].tolist()[:5]) == (8, 1, 3, 1, 0)


def test_config2_forced_tie_and_values(orc):
    w = inputs.config2()
    i = (8 - 1) * 8 + 3                                  # b = 8, pp = 8
    assert w.inst["b"][i] == 8 and w.inst["act_mult"][i] == 8 and w.L[i] == 12
    assert w.L.tolist()[:8] == [96, 48, 24, 12, 6, 3, 2, 1] and w.S == 48
    ts, mb, tq, mq, xq = one(orc, w, i)
    # sequence parallelism changes nothing at tp = 1 -> strategies 0 and 1 tie exactly
    assert ts[0, 0] == ts[0, 1] and mb[0, 0] == mb[0, 1]
    assert tq[0, 0] == tq[0, 1] == 1971615 and mq[0, 0] == 3168 > w.M
    assert (tq[0, 47], mq[0, 47]) == (367749, 60) and (tq[0, 46], mq[0, 46]) == (367749, 102)
    assert (tq[0, 30], mq[0, 30]) == (684049, 109)
    assert 96 * 12 * 12288 ** 2 == 173946175488          # the 175B-parameter shape


def test_config3_unjittered_values(orc):
    w = inputs.config3(B=2)
    w.inst["flops_rate"] = 1e15; w.inst["bw_tp"] = 450e9; w.inst["bw_dp"] = 450e9
    ts, mb, tq, mq, xq = one(orc, w, 0, L=2)
    assert (tq[0, 0], mq[0, 0]) == (1033417, 602) and (tq[1, 0], mq[1, 0]) == (1736980, 554)
    assert (tq[0, 63], mq[0, 63]) == (189635, 33) and (tq[1, 63], mq[1, 63]) == (272098, 65)
    assert (tq[0, 37], mq[0, 37]) == (280724, 127) and (tq[1, 37], mq[1, 37]) == (434245, 91)
    assert 80 * (33 + 65) <= w.M                         # the cheapest plan just fits
    # Resharding entries that toggle sequence parallelism, worked by hand (activation = seq*h*2 B = 67 108 864 B,
    # 450 GB/s, 10 ns units; factor = (k-1)/k for the tp change + (tp_dst-1)/tp_dst for the toggle):
    #   tp8/sp0 -> tp8/sp1: 7/8      -> 13 048.9 ;  tp2/sp0 -> tp4/sp1: 1/2 + 3/4 -> 18 641.4
    #   tp4/sp1 -> tp2/sp0: 1/2 + 1/2 -> 14 913.1 ;  tp1/sp0 -> tp8/sp1: 7/8 + 7/8 -> 26 097.9
    st = w.strat
    idx = lambda tp, sp: int(np.flatnonzero((st["tp"] == tp) & (st["sp"] == sp) & (st["zero"] == 0) & (st["ckpt"] == 0))[0])
    assert (idx(8, 0), idx(8, 1), idx(2, 0), idx(4, 1), idx(1, 0)) == (48, 49, 16, 33, 0)
    assert xq[48, 49] == 13049 and xq[16, 33] == 18641 and xq[33, 16] == 14913 and xq[0, 49] == 26098
    assert xq[49, 48] == 13049                           # same destination tp: the toggle costs the same both ways
    assert xq[0, 1] == 0                                 # toggling at tp = 1 moves nothing
    # jitter stays within +-20 %
    wj = inputs.config3()
    assert (wj.inst["flops_rate"] >= 0.8e15).all() and (wj.inst["flops_rate"] < 1.2e15).all()
    assert (wj.inst["bw_tp"] == wj.inst["bw_dp"]).all() and len(np.unique(wj.inst["bw_tp"])) == 128


def test_invariants(orc):
    w = inputs.config3(B=1)
    st = w.strat
    ts, mb, tq, mq, xq = one(orc, w, 0, L=2)
    h, seq, bpe, bw = 8192.0, 4096.0, 2.0, float(w.inst["bw_tp"][0])
    for l, (n_ar, p_coef) in enumerate(((2.0, 4.0), (2.0, 8.0))):
        for s in range(64):
            tp, dp, z, ck, sq = (int(st[k][s]) for k in ("tp", "dp", "zero", "ckpt", "sp"))
            base = ts[l, (s // 16) * 16 + ck * 2]         # same tp, ZeRO-0, same ckpt, no sp
            if z in (1, 2):                               # ZeRO-1/2 cost the same time as ZeRO-0
                assert ts[l, s] == base
            if dp == 1:                                   # no replicas: no gradient traffic, ZeRO is a no-op
                assert ts[l, s] == base and mb[l, s] == mb[l, s - 4 * z]
    # memory never grows with the ZeRO stage
    for s in range(64):
        z = int(st["zero"][s])
        if z > 0:
            assert (mb[:, s] <= mb[:, s - 4]).all()
    # tp = 1, ZeRO-0, no ckpt: time = compute + dp ring only
    rate = float(w.inst["flops_rate"][0])
    fwd_att = 8 * seq * h * h + 4 * seq * seq * h
    assert ts[0, 0] == pytest.approx(fwd_att * 3 / rate + 1.75 * (4 * h * h * 2) / bw, rel=1e-14)
    # zero diagonal, zero cost exactly between strategies of the same layout
    assert (xq.diagonal() == 0).all()
    for a in range(64):
        for c in range(64):
            # sequence parallelism is a no-op at tp = 1, so toggling it there is free too
            same = st["tp"][a] == st["tp"][c] and (st["sp"][a] == st["sp"][c] or st["tp"][c] == 1)
            assert (xq[a, c] == 0) == bool(same)
    # tp 1 -> 8 moves 7/8 of the activation: 7/8 * seq*h*2 B / bw
    a, c = 0, 48
    assert st["tp"][c] == 8 and st["sp"][c] == 0
    assert xq[a, c] == round(0.875 * seq * h * 2 / bw * 1e9 / 10)


def test_attention_plus_ffn_is_a_full_layer(orc):
    strat = inputs.strategy_table((1, 2, 4, 8), (0, 1, 2, 3), (0, 1), (0, 1))
    inst = inputs._inst(1, b=3.0, act_mult=2.0)[0]
    rows = np.empty(3, inputs.LAYER_DESC)
    for k, kind in enumerate(("attention", "ffn", "full")):
        rows[k] = inputs.layer_desc(kind, 4096.0, 2048.0, 32.0)
    ts, mb, *_ = orc.eval_costs(rows, strat, inst, 3)
    np.testing.assert_allclose(ts[0] + ts[1], ts[2], rtol=1e-14)
    # memory adds up too, except that each checkpointed layer keeps its own input
    nock = strat["ckpt"] == 0
    np.testing.assert_allclose((mb[0] + mb[1])[nock], mb[2][nock], rtol=1e-14)
    assert ((mb[0] + mb[1])[~nock] > mb[2][~nock]).all()


def test_time_grows_with_batch_and_rounding(orc):
    w = inputs.config1()
    prev = None
    for i in range(16):
        ts, mb, tq, mq, _ = one(orc, w, i, L=1)
        if prev is not None:
            assert (ts >= prev[0]).all() and (mb >= prev[1]).all()
        prev = (ts, mb)
    lib = orc.lib()
    # round half to even, ceiling, saturation
    assert [lib.orc_quant_time(v * 1e-9, 1.0) for v in (0.5, 1.5, 2.5, 2.4999, 2.5001)] == [0, 2, 2, 2, 3]
    assert lib.orc_quant_time(1e-6, 100.0) == 10
    assert [lib.orc_quant_mem(v, 4.0) for v in (0.0, 0.1, 4.0, 4.1, 8.0)] == [0, 1, 1, 2, 2]
    assert lib.orc_quant_time(1e30, 1.0) == 2 ** 30 and lib.orc_quant_mem(1e30, 1.0) == 2 ** 30
    assert lib.orc_quant_time(float("nan"), 1.0) == 2 ** 30


def test_descriptors_no_profiler_could_produce(orc):
    """What makes an instance BAD_INPUT in the cost model, case by case, and what the integer tables then hold."""
    w = inputs.config3(B=3)
    L = 6
    assert orc.descriptor_status(w.layers[0], w.strat, w.inst[0], L) == 0
    def bad_inst(field, value):
        inst = w.inst[1].copy(); inst[field] = value
        return orc.descriptor_status(w.layers[0], w.strat, inst, L)
    for field in ("b", "act_mult", "flops_rate", "bw_tp", "bw_dp", "bytes_per_elem", "bin_bytes", "time_unit_ns"):
        for value in (0.0, -1.0, float("nan"), float("inf")):
            assert bad_inst(field, value) == orc.BAD_INPUT, (field, value)
    def bad_strat(field, value):
        st = w.strat.copy(); st[field][5] = value
        return orc.descriptor_status(w.layers[0], st, w.inst[0], L)
    for field, value in (("tp", 0), ("dp", -2), ("zero", 4), ("zero", -1), ("ckpt", 2), ("sp", -1), ("batch_div", 0.0), ("batch_div", float("nan"))):
        assert bad_strat(field, value) == orc.BAD_INPUT, (field, value)
    def bad_layer(l, field, value):
        ly = w.layers[0].copy(); ly[field][l] = value
        return orc.descriptor_status(ly, w.strat, w.inst[0], L)
    assert bad_layer(2, "h", 0.0) == orc.BAD_INPUT and bad_layer(5, "seq", float("nan")) == orc.BAD_INPUT
    assert bad_layer(0, "c_attn", -1.0) == orc.BAD_INPUT and bad_layer(3, "act_tp", float("inf")) == orc.BAD_INPUT
    assert bad_layer(1, "heads", 0.0) == 0 and bad_layer(1, "c_attn", 0.0) == 0      # zero coefficients are fine (an FFN has no attention term)
    assert bad_layer(6, "h", -5.0) == 0                                               # beyond the instance's layers: not looked at
    # the tables of a flagged instance: -1 everywhere, so the search's own validation flags it too
    inst = w.inst[2].copy(); inst["bw_tp"] = 0.0
    ts, mb, tq, mq, xq = orc.eval_costs(w.layers[0], w.strat, inst, L)
    assert (tq == -1).all() and (mq == -1).all() and (xq == -1).all()
    assert orc.validate(tq, mq, xq) == orc.BAD_INPUT

"""ctypes front end of the CPU oracle (galv_oracle.c).  TEST INFRASTRUCTURE ONLY.

Only tests, the smoke check and the bench's CPU-baseline leg may import this.
It never touches the CUDA library or its Python binding.

Arrays use the recurrence's own index order: C[l][m][s] (s fastest), one
instance at a time.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess

import numpy as np

INF = 2 ** 30 - 1
INFEASIBLE, BAD_INPUT, OVERFLOW_RISK = 1, 2, 4

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "galv_oracle.c")
_SO = os.path.join(_HERE, "liboracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (-O2, no FP contraction) if the shared object is stale."""
    if force or not os.path.exists(_SO) or os.path.getmtime(_SO) < os.path.getmtime(_SRC):
        tmp = f"{_SO}.{os.getpid()}.tmp"
        subprocess.check_call(["gcc", "-O2", "-std=c11", "-ffp-contract=off", "-fPIC", "-shared",
                               "-Wall", "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _SO)
    return _SO


def lib() -> C.CDLL:
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
        _lib.orc_brute_force.restype = C.c_int64
        _lib.orc_trans_cost.restype = C.c_double
        _lib.orc_quant_time.restype = C.c_int32
        _lib.orc_quant_mem.restype = C.c_int32
        _lib.orc_quant_time.argtypes = [C.c_double, C.c_double]
        _lib.orc_quant_mem.argtypes = [C.c_double, C.c_double]
    return _lib


def _i32(a):
    a = np.ascontiguousarray(a, dtype=np.int32)
    return a, a.ctypes.data_as(C.c_void_p)


def _tl(trans, L, S):
    """Layer stride of trans: 0 for one [S][S] matrix, S*S for one matrix per layer ([L][S][S])."""
    assert trans.shape in ((S, S), (L, S, S)), trans.shape
    return C.c_int64(0 if trans.ndim == 2 else S * S)


def validate(time, mem, trans) -> int:
    time, pt = _i32(time); mem, pm = _i32(mem); trans, px = _i32(trans)
    L, S = time.shape
    return lib().orc_validate(L, S, pt, pm, px, _tl(trans, L, S))


def dp(time, mem, trans, M: int, want_A: bool = True):
    """Tables of one instance: C int32 [L][M+1][S] and A uint8 (or None)."""
    time, pt = _i32(time); mem, pm = _i32(mem); trans, px = _i32(trans)
    L, S = time.shape
    Ct = np.empty((L, M + 1, S), np.int32)
    At = np.empty((L, M + 1, S), np.uint8) if want_A else None
    lib().orc_dp(L, S, M, pt, pm, px, _tl(trans, L, S), Ct.ctypes.data_as(C.c_void_p),
                 At.ctypes.data_as(C.c_void_p) if want_A else None)
    return Ct, At


def backtrack(time, mem, trans, Ct, At, budget: int):
    """(opt_cost, plan[L], mem_used, status) at `budget`; At=None re-derives the argmin from C."""
    time, pt = _i32(time); mem, pm = _i32(mem); trans, px = _i32(trans)
    L, S = time.shape
    M = Ct.shape[1] - 1
    assert 0 <= budget <= M and Ct.flags.c_contiguous
    opt = C.c_int32(); used = C.c_int32()
    plan = np.empty(L, np.int32)
    st = lib().orc_backtrack(L, S, M, pt, pm, px, _tl(trans, L, S), Ct.ctypes.data_as(C.c_void_p),
                             At.ctypes.data_as(C.c_void_p) if At is not None else None,
                             int(budget), C.byref(opt), plan.ctypes.data_as(C.c_void_p), C.byref(used))
    return opt.value, plan, used.value, st


def brute_force(time, mem, trans, budget: int):
    """(opt_cost, plan, mem_used, n_feasible) by enumerating all S^L plans."""
    time, pt = _i32(time); mem, pm = _i32(mem); trans, px = _i32(trans)
    L, S = time.shape
    opt = C.c_int32(); used = C.c_int32()
    plan = np.empty(L, np.int32)
    n = lib().orc_brute_force(L, S, int(budget), pt, pm, px, _tl(trans, L, S), C.byref(opt),
                              plan.ctypes.data_as(C.c_void_p), C.byref(used))
    return opt.value, plan, used.value, n


def plan_cost(time, mem, trans, plan):
    time, pt = _i32(time); mem, pm = _i32(mem); trans, px = _i32(trans); plan, pp = _i32(plan)
    L, S = time.shape
    c = C.c_int64(); u = C.c_int64()
    lib().orc_plan_cost(L, S, pt, pm, px, _tl(trans, L, S), pp, C.byref(c), C.byref(u))
    return c.value, u.value


def eval_costs(layers, strat, inst, L: int):
    """Cost model of one instance.

    layers: [>=L] records of 10 doubles, strat: [S] records (5 int32, pad, double),
    inst: one record of 8 doubles.  Returns time_s, mem_bytes (float64 [L][S]),
    time_q, mem_q (int32 [L][S]) and trans_q (int32 [S][S]).
    """
    layers = np.ascontiguousarray(layers); strat = np.ascontiguousarray(strat)
    inst = np.ascontiguousarray(inst).reshape(1)
    assert layers.itemsize == 80 and strat.itemsize == 32 and inst.itemsize == 64 and len(layers) >= L
    S = len(strat)
    ts = np.empty((L, S)); mb = np.empty((L, S))
    tq = np.empty((L, S), np.int32); mq = np.empty((L, S), np.int32); xq = np.empty((S, S), np.int32)
    vp = lambda a: a.ctypes.data_as(C.c_void_p)
    lib().orc_eval_costs(L, S, vp(layers), vp(strat), vp(inst), vp(ts), vp(mb), vp(tq), vp(mq), vp(xq))
    return ts, mb, tq, mq, xq


def descriptor_status(layers, strat, inst, L: int) -> int:
    """0, or BAD_INPUT when a descriptor of the instance (its parameters, the strategy table, its L layers) is one
    no profiler could have produced (see orc_check_descriptors); eval_costs then fills the integer tables with -1."""
    layers = np.ascontiguousarray(layers); strat = np.ascontiguousarray(strat)
    inst = np.ascontiguousarray(inst).reshape(1)
    vp = lambda a: a.ctypes.data_as(C.c_void_p)
    return int(lib().orc_check_descriptors(L, len(strat), vp(layers), vp(strat), vp(inst)))


def search(time, mem, trans, M: int, budget=None, use_A: bool = False):
    """Whole path for one instance on integer tables: validate, DP, optimum, plan."""
    st = validate(time, mem, trans)
    L = np.asarray(time).shape[0]
    if st & (BAD_INPUT | OVERFLOW_RISK):
        return dict(status=st, opt_cost=INF, plan=np.full(L, -1, np.int32), mem_used=0, C=None, A=None)
    Ct, At = dp(time, mem, trans, M, want_A=True)
    opt, plan, used, st2 = backtrack(time, mem, trans, Ct, At if use_A else None, M if budget is None else budget)
    return dict(status=st | st2, opt_cost=opt, plan=plan, mem_used=used, C=Ct, A=At)


def select_best(opt_cost, status, n_micro, pp, group, G: int):
    """(best_time int64 [G], best_inst int32 [G]): per group the feasible candidate with the shortest iteration."""
    oc, p0 = _i32(opt_cost); st, p1 = _i32(status); nm, p2 = _i32(n_micro); ppa, p3 = _i32(pp); gr, p4 = _i32(group)
    bt = np.empty(G, np.int64); bi = np.empty(G, np.int32)
    lib().orc_select_best(len(oc), G, p0, p1, p2, p3, p4, bt.ctypes.data_as(C.c_void_p), bi.ctypes.data_as(C.c_void_p))
    return bt, bi


def prune(L, time, mem, trans):
    """keep[S] (0/1): strategies that survive the dominated-strategy prune over the whole batch."""
    time, pt = _i32(time); mem, pm = _i32(mem); trans, px = _i32(trans); L, pl = _i32(L)
    B, Lmax, S = time.shape
    keep = np.empty(S, np.int32)
    lib().orc_prune(B, Lmax, S, pl, pt, pm, px, keep.ctypes.data_as(C.c_void_p))
    return keep


def stage_partition(range_opt, P: int):
    """(bottleneck, cuts[P+1]) for range_opt [Lm][Lm] (row a, column n-1: optimum of layers a..a+n-1)."""
    ro, pr = _i32(range_opt)
    Lm = ro.shape[0]
    assert ro.shape == (Lm, Lm)
    cuts = np.empty(P + 1, np.int32); bn = C.c_int32()
    lib().orc_stage_partition(Lm, P, pr, cuts.ctypes.data_as(C.c_void_p), C.byref(bn))
    return bn.value, cuts


def add_switch_cost(time, trans, cur_plan, horizon: int):
    """time'(l,s) = time(l,s) + trans_l(cur_plan[l], s) // horizon (see orc_add_switch_cost)."""
    time, pt = _i32(time); trans, px = _i32(trans); cur, pc = _i32(cur_plan)
    L, S = time.shape
    out = np.empty((L, S), np.int32)
    lib().orc_add_switch_cost(L, S, pt, px, _tl(trans, L, S), pc, int(horizon), out.ctypes.data_as(C.c_void_p))
    return out


def switch_decision(cur_cost: int, new_cost: int, hysteresis_permille: int) -> int:
    return int(lib().orc_switch_decision(C.c_int64(int(cur_cost)), C.c_int64(int(new_cost)), int(hysteresis_permille)))

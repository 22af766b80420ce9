"""GPU parity: the CUDA library against the CPU oracle, element by element, through the C boundary."""
import os
from concurrent.futures import ThreadPoolExecutor

import numpy as np
import pytest

from paper_2504_03662_b200 import inputs

pytestmark = pytest.mark.gpu

INF = 2 ** 30 - 1
NC, CLU = 16384, 32768        # GALV_KERNEL_NO_CLUSTER (tiled kernels only), GALV_KERNEL_CLUSTER (cluster kernel wherever the shape allows)


def cl_size(n):
    """GALV_CLUSTER_SIZE(n): the cluster kernel with clusters of n CTAs."""
    return CLU | ((n & 31) << 16)


@pytest.fixture(scope="module")
def galv():
    import torch
    from paper_2504_03662_b200 import binding as gb
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    g = gb.Galv(0)
    yield g
    g.close()


def oracle_tables(orc, w):
    """Integer tables of every instance from the oracle's own cost model (or the workload's)."""
    if not w.has_model:
        return w.time_q, w.mem_q, w.trans_q
    tq = np.zeros((w.B, w.Lmax, w.S), np.int32); mq = np.zeros_like(tq); xq = np.zeros((w.B, w.S, w.S), np.int32)
    for i in range(w.B):
        Li = int(w.L[i])
        _, _, t, m, x = orc.eval_costs(w.layers[0 if w.layers.shape[0] == 1 else i], w.strat, w.inst[i], Li)
        tq[i, :Li], mq[i, :Li], xq[i] = t, m, x
    return tq, mq, xq


def oracle_search_many(orc, w, tq, mq, xq, idx, use_A=False):
    def one(i):
        Li = int(w.L[i])
        return orc.search(tq[i, :Li], mq[i, :Li], xq[i], w.M, use_A=use_A)
    with ThreadPoolExecutor(max_workers=min(16, os.cpu_count() or 1)) as ex:
        return dict(zip(idx, ex.map(one, idx)))


def check_batch(orc, galv, w, flags, idx=None, tables=True, budget=None):
    """Run the GPU path on the whole batch and compare instances `idx` with the oracle."""
    import torch
    from paper_2504_03662_b200 import binding as gb
    from paper_2504_03662_b200.search import SearchBuffers
    sb = SearchBuffers(galv, w, flags)
    tq, mq, xq = oracle_tables(orc, w)
    if w.has_model:
        sb.eval_costs()
        torch.cuda.synchronize()
        for name, ref, got in (("time_q", tq, sb.time_q), ("mem_q", mq, sb.mem_q), ("trans_q", xq, sb.trans_q)):
            g = got.cpu().numpy()
            for i in range(w.B):
                Li = int(w.L[i]) if name != "trans_q" else w.S
                assert (g[i, :Li] == ref[i, :Li]).all(), (name, i)
    sb.dp_search()
    bud = None if budget is None else torch.from_numpy(np.asarray(budget, np.int32)).to(sb.dev)
    sb.backtrack(bud)
    res = sb.results()
    idx = list(range(w.B)) if idx is None else list(idx)
    ref = oracle_search_many(orc, w, tq, mq, xq, idx)
    for i in idx:
        r, Li = ref[i], int(w.L[i])
        b = w.M if budget is None else int(budget[i])
        if budget is not None and r["C"] is not None:
            o, p, u, st = orc.backtrack(tq[i, :Li], mq[i, :Li], xq[i], r["C"], None, b)
            r = dict(r, opt_cost=o, plan=p, mem_used=u, status=st)
        assert res["status"][i] == r["status"], (i, res["status"][i], r["status"])
        assert res["opt_cost"][i] == r["opt_cost"], i
        if flags & (gb.STORE_C_FULL | gb.STORE_ARGMIN):
            assert (res["plan"][i, :Li] == r["plan"]).all(), (i, res["plan"][i, :Li], r["plan"])
            assert (res["plan"][i, Li:] == -1).all()
            assert res["mem_used"][i] == r["mem_used"]
        else:                                                   # no table kept: the optimum only, no walk
            assert (res["plan"][i] == -1).all() and res["mem_used"][i] == 0
        if r["C"] is None:
            continue
        last = sb.C_last[i, :, :w.M + 1].t().cpu().numpy()
        assert (last == r["C"][Li - 1]).all(), i
        assert (sb.C_last[i, :, w.M + 1:] == INF).all()
        if tables and flags & gb.STORE_C_FULL:
            got = sb.table(i)[:Li]
            assert (got == r["C"]).all(), (i, np.argwhere(got != r["C"])[:5])
        if tables and flags & gb.STORE_ARGMIN:
            got = sb.argmin_table(i)[:Li]
            assert (got == r["A"]).all(), (i, np.argwhere(got != r["A"])[:5])
    return sb, res


MODES = [1 | NC, 3, 2, 1 | 512, 1 | 256, 3 | 256, 1, 1 | CLU]   # full C (all layers in one launch); full C + A; rolling + A;
                                             # full C with one launch per layer; the reference kernel; the cluster
                                             # kernel (chosen on its own for a batch this small; and asked for)


@pytest.mark.parametrize("flags", MODES)
def test_config0_every_budget(orc, galv, flags):
    w = inputs.config0()
    check_batch(orc, galv, w, flags)
    rows = [l.split() for l in open(os.path.join(os.path.dirname(__file__), "golden", "config0_bruteforce.txt"))
            if not l.startswith("#")]
    # all 65 budgets in one batch of 65 copies of the instance
    w65 = inputs.Workload("config0x65", 65, w.Lmax, w.S, w.M, np.full(65, 4, np.int32),
                          np.repeat(w.time_q, 65, 0), np.repeat(w.mem_q, 65, 0), np.repeat(w.trans_q, 65, 0))
    sb, res = check_batch(orc, galv, w65, flags, budget=np.arange(65))
    for r in rows:
        b = int(r[0])
        assert res["opt_cost"][b] == int(r[1]) and res["plan"][b].tolist() == [int(v) for v in r[4:]]


SHAPES = [  # B, Lmax, S, M, kwargs
    (3, 5, 1, 40, {}),
    (4, 7, 5, 97, dict(ragged=True)),
    (2, 6, 8, 255, {}),
    (3, 9, 13, 300, dict(ragged=True, mem_lo=0, mem_hi=0)),            # memory-free: layered shortest path
    (2, 4, 33, 1000, dict(dup_cols=True, time_hi=5, trans_hi=2)),      # tie-heavy, S just above a warp
    (2, 3, 70, 513, dict(mem_hi=700)),                                 # two s-blocks; many mem > M
    (5, 1, 6, 64, {}),                                                 # single layer
    (2, 5, 24, 2881, dict(mem_lo=3000, mem_hi=4000)),                  # nothing fits
    (2, 12, 32, 2048, dict(mem_lo=8, mem_hi=128, trans_hi=50000)),     # tile edge: M+1 = 4*512+1
    (1, 3, 130, 200, {}),                                              # three s-blocks
    (1, 3, 256, 100, dict(time_hi=100000)),                            # the largest S
]


@pytest.mark.parametrize("flags", [1 | NC, 3, 2, 1 | 512, 1 | 1024 | NC, 2 | 1024, 1 | CLU, 1 | cl_size(2), 1 | cl_size(3), 1 | cl_size(5),
                                   1 | cl_size(8), 1 | cl_size(16)])
@pytest.mark.parametrize("k", range(len(SHAPES)))
def test_random_shapes(orc, galv, flags, k):
    B, Lmax, S, M, kw = SHAPES[k]
    w = inputs.random_tables(700 + k, B, Lmax, S, M, **kw)
    sb, res = check_batch(orc, galv, w, flags)
    if k == 7:
        assert (res["status"] == 1).all() and (res["opt_cost"] == INF).all()


def test_budget_queries(orc, galv):
    w = inputs.random_tables(31, 6, 8, 12, 400, mem_lo=1, mem_hi=90)
    check_batch(orc, galv, w, 3, budget=[0, 50, 123, 399, 400, 200])


def test_flagged_instances_are_skipped(orc, galv):
    import torch
    w = inputs.random_tables(5, 6, 4, 6, 50, ragged=True)
    w.time_q[1, 0, 2] = -7                       # negative entry
    w.L[2] = 0                                   # L out of range
    w.time_q[3] = (INF - 1) // 2                 # sum could reach INF
    w.L[3] = 4
    w.mem_q[4, 1, :] = -1
    w.L[4] = 4
    w.L[5] = 9                                   # above Lmax
    sb, res = check_batch(orc, galv, w, 3, idx=[0])
    assert res["status"].tolist()[1:] == [2, 2, 4, 2, 2]
    assert (res["opt_cost"][1:] == INF).all() and (res["plan"][1:] == -1).all() and (res["mem_used"][1:] == 0).all()
    # an out-of-range budget is reported, not followed
    sb.backtrack(torch.tensor([51, -1, 0, 0, 0, 0], dtype=torch.int32, device=sb.dev))
    r2 = sb.results()
    assert r2["status"][0] == 2 and r2["opt_cost"][0] == INF


def test_config1_full(orc, galv):
    sb, res = check_batch(orc, galv, inputs.config1(), 3)
    assert (res["status"] == 0).all()
    # a batch this small takes the cluster kernel on its own
    sb, res = check_batch(orc, galv, inputs.config1(), 1)
    assert galv.galv_dp_search_path(sb.shape, sb.workspace) == 2 and (res["status"] == 0).all()
    sb, res = check_batch(orc, galv, inputs.config1(), 1 | NC)
    assert galv.galv_dp_search_path(sb.shape, sb.workspace) == 0


def test_config2_full_ragged(orc, galv):
    w = inputs.config2()
    sb, res = check_batch(orc, galv, w, 1 | NC)
    assert set(res["status"].tolist()) <= {0, 1} and galv.galv_dp_search_path(sb.shape, sb.workspace) == 1
    sb, res = check_batch(orc, galv, w, 2, idx=range(0, 64, 5), tables=False)
    # the cluster kernel: more instances than cluster slots, the longest first
    sb, res = check_batch(orc, galv, w, 1 | CLU)
    assert galv.galv_dp_search_path(sb.shape, sb.workspace) == 2
    for n in (6, 16):
        sb, res = check_batch(orc, galv, w, 1 | cl_size(n), idx=range(0, 64, 3))
        assert galv.galv_dp_search_path(sb.shape, sb.workspace) == 2


def test_config2_full_product_extra(orc, galv):
    check_batch(orc, galv, inputs.config2(full_product=True), 1, idx=[3, 17, 40, 63])


def _properties_all(orc, w, tq, mq, xq, sb, res):
    """What holds at any size: plan cost equals the optimum, memory within budget, C_last monotone."""
    last = sb.C_last[:, :, :w.M + 1]
    assert bool((last[:, :, :-1] >= last[:, :, 1:]).all())
    for i in range(w.B):
        Li = int(w.L[i])
        if res["status"][i] == 0:
            c, u = orc.plan_cost(tq[i, :Li], mq[i, :Li], xq[i], res["plan"][i, :Li])
            assert c == res["opt_cost"][i] and u == res["mem_used"][i] <= w.M


def test_config4_full_size(orc, galv):
    w = inputs.config4()
    idx = [0, 1, 511, 777, 1023] + list(range(64, 1024, 64))
    sb, res = check_batch(orc, galv, w, 1, idx=idx)
    assert (res["status"] == 0).all()
    _properties_all(orc, w, w.time_q, w.mem_q, w.trans_q, sb, res)
    del sb
    sb, res2 = check_batch(orc, galv, w, 2, idx=idx[:6], tables=False)
    assert (res2["opt_cost"] == res["opt_cost"]).all() and (res2["plan"] == res["plan"]).all()


def test_config4_full_size_dominated_rows_skipped(orc, galv):
    """The 32-bit loop (transition entries to 5e4) with dominated rows left out, all 1024 instances."""
    from paper_2504_03662_b200 import binding as gb
    w = inputs.config4()
    idx = [0, 511, 1023] + list(range(100, 1024, 300))
    sb, res = check_batch(orc, galv, w, gb.STORE_C_FULL | gb.SKIP_DOMINATED, idx=idx)
    assert galv.galv_dp_search_path(sb.shape, sb.workspace) == 0
    assert (res["status"] == 0).all()
    _properties_all(orc, w, w.time_q, w.mem_q, w.trans_q, sb, res)


@pytest.mark.parametrize("flags", [1, 1 | 1024, 1 | 8192, 1 | 1024 | 8192])      # plain; tiles below the feasibility frontier skipped; dominated rows left out; both
def test_config3_full_size(orc, galv, flags):
    import torch
    w = inputs.config3()
    idx = [0, 37, 127]
    sb, res = check_batch(orc, galv, w, flags, idx=idx)
    assert (res["status"] == 0).all()
    tq, mq, xq = oracle_tables(orc, w)
    _properties_all(orc, w, tq, mq, xq, sb, res)
    del sb
    torch.cuda.empty_cache()


def test_cost_model_fp64(orc, galv):
    import torch
    from paper_2504_03662_b200.search import SearchBuffers
    for w in (inputs.config1(), inputs.config2(), inputs.config3(B=8)):
        sb = SearchBuffers(galv, w, 1)
        sb.eval_costs(want_fp64=True)
        torch.cuda.synchronize()
        ts, mb = sb.time_s.cpu().numpy(), sb.mem_bytes.cpu().numpy()
        for i in range(w.B):
            Li = int(w.L[i])
            rts, rmb, *_ = orc.eval_costs(w.layers[0], w.strat, w.inst[i], Li)
            np.testing.assert_allclose(ts[i, :Li], rts, rtol=1e-12, atol=0)
            np.testing.assert_allclose(mb[i, :Li], rmb, rtol=1e-12, atol=0)
            assert (ts[i, Li:] == 0).all()                      # rows beyond L[i] are left untouched
        assert (sb.status == 0).all()


def test_host_entry_point(orc, galv):
    from paper_2504_03662_b200.search import HostSearch
    for w, flags in ((inputs.config4(B=24), 1), (inputs.config2(), 3), (inputs.config0(), 2)):
        hs = HostSearch(galv, w, flags)
        res = hs.run()
        res = {k: v.copy() for k, v in res.items()}
        tq, mq, xq = oracle_tables(orc, w)
        ref = oracle_search_many(orc, w, tq, mq, xq, list(range(w.B)))
        for i in range(w.B):
            Li = int(w.L[i])
            assert res["opt_cost"][i] == ref[i]["opt_cost"] and (res["plan"][i, :Li] == ref[i]["plan"]).all()
            assert res["status"][i] == ref[i]["status"] and res["mem_used"][i] == ref[i]["mem_used"]
        again = hs.run()                                           # same arena, second call
        assert (again["opt_cost"] == res["opt_cost"]).all() and (again["plan"] == res["plan"]).all()


def test_boundary_errors(galv):
    import ctypes as C
    import torch
    from paper_2504_03662_b200 import binding as gb
    from paper_2504_03662_b200.search import SearchBuffers
    w = inputs.config0()
    sb = SearchBuffers(galv, w, 1)
    lib, h = galv.lib, galv.h
    st = torch.cuda.current_stream().cuda_stream
    p = lambda t: None if t is None else t.data_ptr()
    ws_bytes = sb.workspace.numel()

    def dp(shape, C_=sb.C, A_=None, ws=sb.workspace, nbytes=ws_bytes, L=sb.L):
        return lib.galv_dp_search(h, C.byref(shape), p(L), p(sb.time_q), p(sb.mem_q), p(sb.trans_q), p(C_), p(A_),
                                  p(sb.C_last), p(ws) if ws is not None else None, nbytes, p(sb.status), st)

    assert dp(sb.shape) == gb.OK
    assert dp(sb.shape, L=None) == gb.ERR_INVALID_ARG
    assert dp(sb.shape, C_=None) == gb.ERR_INVALID_ARG                       # flag says full C
    assert dp(gb.make_shape(1, 4, 6, 64, 0), C_=sb.C) == gb.ERR_INVALID_ARG  # table without its flag
    assert dp(gb.make_shape(1, 4, 257, 64, 1)) == gb.ERR_INVALID_ARG         # S above the limit
    assert dp(gb.make_shape(1, 4, 6, 64, 1, m_pitch=65)) == gb.ERR_INVALID_ARG
    assert dp(gb.make_shape(1, 4, 6, 64, 1, m_pitch=64)) == gb.ERR_INVALID_ARG
    assert dp(gb.make_shape(0, 4, 6, 64, 1)) == gb.ERR_INVALID_ARG
    assert dp(sb.shape, ws=None) == gb.ERR_WORKSPACE
    assert dp(sb.shape, nbytes=16) == gb.ERR_WORKSPACE
    assert lib.galv_dp_workspace_bytes(h, C.byref(gb.make_shape(1, 4, 300, 64, 1))) == 0
    assert b"workspace" in lib.galv_last_error(h)
    assert lib.galv_strerror(gb.ERR_WORKSPACE) and lib.galv_strerror(-99)
    # backtrack without any table to walk
    rc = lib.galv_backtrack(h, C.byref(sb.shape), p(sb.L), p(sb.time_q), p(sb.mem_q), p(sb.trans_q), None, None,
                            p(sb.C_last), None, p(sb.opt_cost), p(sb.plan), p(sb.mem_used), p(sb.status), st)
    assert rc == gb.ERR_INVALID_ARG
    # ... but the optimum alone is fine
    rc = lib.galv_backtrack(h, C.byref(sb.shape), p(sb.L), p(sb.time_q), p(sb.mem_q), p(sb.trans_q), None, None,
                            p(sb.C_last), None, p(sb.opt_cost), None, None, p(sb.status), st)
    assert rc == gb.OK
    torch.cuda.synchronize()
    assert sb.opt_cost.item() == 7693
    with pytest.raises(gb.GalvError):
        galv.galv_dp_search(gb.make_shape(1, 4, 6, 64, 3), sb.L, sb.time_q, sb.mem_q, sb.trans_q, sb.C, None,
                            sb.C_last, sb.workspace, sb.status)
    h2 = C.c_void_p()
    assert lib.galv_create(C.byref(h2), 9999) != gb.OK and not h2.value
    torch.cuda.synchronize()                      # the context is still healthy
    assert dp(sb.shape) == gb.OK


def test_alu_probe_runs(galv):
    rates = [galv.galv_probe_int_alu(k, 512) for k in (0, 1, 2, 3, 4)]
    assert all(1e11 < r < 1e15 for r in rates), rates


@pytest.mark.parametrize("flags", [1 | NC, 1 | 1024 | NC, 1 | 512, 3, 1 | CLU])
def test_layers_with_different_tile_counts(orc, galv, flags):
    """One heavy layer leaves its trailing tiles out; the layers after it run them again.

    With all layers in one launch an item waits for the tiles of the layer before; how far a tile's
    counter has to be depends on how many earlier layers ran that tile at all.
    """
    w = inputs.random_tables(41, 3, 7, 64, 1500, mem_lo=1, mem_hi=60, time_hi=3000)
    w.mem_q[:, 2, :] += 800                      # layer 2: nothing lands above column 1500 - 801
    w.mem_q[:, 5, :] += 300
    check_batch(orc, galv, w, flags)


@pytest.mark.parametrize("flags", [1, 1 | 512, 1 | 8192, 1 | 8192 | 4096])     # one launch, per layer, dominated rows skipped (packed, 32-bit)
def test_bounded_waits_run_out_cleanly(orc, galv, flags):
    """A stage that never fills: the waits give up, the status says TIMEOUT, the context keeps working."""
    import time
    import torch
    from paper_2504_03662_b200 import binding as gb
    from paper_2504_03662_b200.search import SearchBuffers
    w = inputs.random_tables(3, 4, 5, 12, 300, mem_lo=1, mem_hi=60)
    bad = SearchBuffers(galv, w, flags | gb.DEBUG_WITHHOLD_LOAD)
    t0 = time.time()
    bad.dp_search()
    torch.cuda.synchronize()                               # returns: no hang, no fault
    assert time.time() - t0 < 60
    assert (bad.status.cpu().numpy() & gb.STATUS_TIMEOUT).all()
    # the tables are void: the plan step does not walk them
    bad.backtrack()
    r = bad.results()
    assert (r["status"] & gb.STATUS_TIMEOUT).all() and (r["opt_cost"] == INF).all()
    assert (r["plan"] == -1).all() and (r["mem_used"] == 0).all()
    if flags == 1:
        # the host entry point runs search and plan step back to back and reports the time-out
        from paper_2504_03662_b200.search import HostSearch
        hs = HostSearch(galv, w, flags | gb.DEBUG_WITHHOLD_LOAD)
        with pytest.raises(gb.GalvError) as err:
            hs.run()
        assert err.value.code == gb.ERR_TIMEOUT
        assert (hs.plan.numpy() == -1).all() and (hs.opt_cost.numpy() == INF).all()
    # the same context and device then search normally
    check_batch(orc, galv, w, flags)


@pytest.mark.parametrize("block", range(8))
def test_one_launch_against_reference_kernel_on_many_shapes(galv, block):
    """Consistency stress of the one-launch kernel (work queue, tile counters, role hand-overs): on random
    shapes with many tiles, layers and ragged lengths its tables must equal those of the one-thread-per-cell
    kernel, which the tests above tie to the oracle.  Run twice per shape: the second run reuses every buffer."""
    import torch
    from paper_2504_03662_b200 import binding as gb
    from paper_2504_03662_b200.search import SearchBuffers
    rng = np.random.default_rng(1000 + block)
    for case in range(10):
        S = int(rng.choice([1, 5, 8, 24, 31, 32, 48, 64, 65, 100, 130, 256]))
        Lmax = int(rng.integers(3, 30))
        M = int(rng.integers(40, 5000))
        pitch = (M + 32) // 32 * 32
        B = int(max(1, min(rng.integers(1, 160), 3.0e8 // (Lmax * S * pitch * 4))))
        mem_hi = int(rng.choice([3, M // 20 + 1, M // 3 + 1, 2 * M]))
        w = inputs.random_tables(5000 + 100 * block + case, B, Lmax, S, M, ragged=bool(rng.integers(0, 2)),
                                 mem_lo=int(rng.integers(0, 3)), mem_hi=mem_hi, trans_hi=int(rng.choice([0, 50, 50000])))
        if rng.integers(0, 3) == 0:
            w.mem_q[:, int(rng.integers(1, Lmax)), :] += M // 2       # one heavy layer: fewer tiles there
        ref = SearchBuffers(galv, w, gb.STORE_C_FULL | gb.KERNEL_REFERENCE)
        ref.dp_search()
        one = SearchBuffers(galv, w, gb.STORE_C_FULL | (gb.KERNEL_CLUSTER if case % 5 == 4 else gb.KERNEL_NO_CLUSTER)
                            | (gb.SKIP_INFEASIBLE if case % 3 == 2 else 0) | (gb.SKIP_DOMINATED if case % 4 == 1 else 0))
        for _ in range(2):
            one.C.fill_(-7)
            one.dp_search()
            torch.cuda.synchronize()
            st = ref.status.cpu().numpy()
            assert (one.status.cpu().numpy() == st).all(), (block, case)
            for i in np.flatnonzero(st == 0):
                Li = int(w.L[i])
                assert torch.equal(one.C[i, :Li], ref.C[i, :Li]), (block, case, int(i), S, Lmax, M, B)
            assert torch.equal(one.C_last[st == 0], ref.C_last[st == 0]), (block, case)
        del ref, one
        torch.cuda.empty_cache()


@pytest.mark.skipif(not os.environ.get("GALV_SOAK"), reason="long random-shape soak: set GALV_SOAK=<blocks of 10 shapes>")
def test_soak_random_shapes_and_flags(galv):
    """The stress above on many more shapes, with every kernel-selecting flag drawn at random (packed / 32-bit loop,
    per layer, argmin table, both skipping flags): tables, optima and plans against the one-thread-per-cell kernel."""
    import torch
    from paper_2504_03662_b200 import binding as gb
    from paper_2504_03662_b200.search import SearchBuffers
    nc = gb.KERNEL_NO_CLUSTER
    choices = [nc, nc | gb.SKIP_INFEASIBLE, nc | gb.SKIP_DOMINATED, nc | gb.SKIP_DOMINATED | gb.SKIP_INFEASIBLE, nc | gb.KERNEL_NO_PACKED,
               nc | gb.KERNEL_NO_PACKED | gb.SKIP_DOMINATED, gb.STORE_ARGMIN, gb.STORE_ARGMIN | gb.SKIP_DOMINATED,
               gb.KERNEL_PER_LAYER | gb.SKIP_DOMINATED, 0, gb.KERNEL_CLUSTER, gb.CLUSTER_SIZE(2), gb.CLUSTER_SIZE(4), gb.CLUSTER_SIZE(7),
               gb.CLUSTER_SIZE(16)]
    for block in range(int(os.environ["GALV_SOAK"])):
        rng = np.random.default_rng(77000 + block)
        for case in range(10):
            S = int(rng.choice([1, 4, 5, 8, 12, 24, 31, 32, 36, 48, 60, 64, 65, 100, 130, 256]))
            Lmax = int(rng.integers(2, 40))
            M = int(rng.integers(10, 6000))
            pitch = (M + 32) // 32 * 32
            B = int(max(1, min(rng.integers(1, 200), 3.0e8 // (Lmax * S * pitch * 4))))
            mem_hi = int(rng.choice([3, M // 20 + 3, M // 3 + 3, 2 * M + 3]))
            w = inputs.random_tables(900000 + 100 * block + case, B, Lmax, S, M, ragged=bool(rng.integers(0, 2)),
                                     mem_lo=int(rng.integers(0, 3)), mem_hi=mem_hi,
                                     trans_hi=int(rng.choice([0, 7, 50, 3000, 32767, 32768, 50000])),
                                     time_hi=int(rng.choice([10, 1000, 10 ** 5, 3 * 10 ** 6])))
            if rng.integers(0, 3) == 0:
                w.mem_q[:, int(rng.integers(0, Lmax)), :] += M // 2
            ref = SearchBuffers(galv, w, gb.STORE_C_FULL | gb.KERNEL_REFERENCE)
            ref.dp_search(); ref.backtrack()
            one = SearchBuffers(galv, w, gb.STORE_C_FULL | int(rng.choice(choices)))
            for _ in range(2):
                one.C.fill_(-7)
                one.dp_search(); one.backtrack()
                torch.cuda.synchronize()
                st = ref.status.cpu().numpy()
                assert (one.status.cpu().numpy() == st).all(), (block, case)
                assert torch.equal(one.opt_cost, ref.opt_cost) and torch.equal(one.plan, ref.plan), (block, case)
                for i in np.flatnonzero(st == 0):
                    Li = int(w.L[i])
                    assert torch.equal(one.C[i, :Li], ref.C[i, :Li]), (block, case, int(i), S, Lmax, M, B)
                assert torch.equal(one.C_last[st == 0], ref.C_last[st == 0]), (block, case)
            del ref, one
            torch.cuda.empty_cache()


def test_kernel_span_statistics(galv):
    """The timing hook keeps one event pair per profiled search and reports mean, shortest, longest."""
    import torch
    from paper_2504_03662_b200 import binding as gb
    from paper_2504_03662_b200.search import SearchBuffers
    w = inputs.random_tables(3, 4, 6, 16, 700)
    sb = SearchBuffers(galv, w, gb.STORE_C_FULL)
    galv.galv_set_profiling(True)
    with pytest.raises(gb.GalvError):
        galv.galv_layer_loop_ms_stats()                      # nothing profiled yet
    for _ in range(5):
        sb.dp_search()
    mean, lo, hi, n = galv.galv_layer_loop_ms_stats()
    assert n == 5 and 0 < lo <= mean <= hi < 1000
    assert lo <= galv.galv_last_layer_loop_ms() <= hi
    for _ in range(70):                                      # more searches than pairs are kept
        sb.dp_search()
    assert galv.galv_layer_loop_ms_stats()[3] == 64
    galv.galv_set_profiling(False)
    torch.cuda.synchronize()


@pytest.mark.parametrize("flags", [NC, 1024 | NC, CLU])
@pytest.mark.parametrize("k", range(len(SHAPES)))
def test_cost_only_search_on_the_rolling_buffer(orc, galv, flags, k):
    """No table kept: two layers roll in the workspace (all layers still one launch, an item also waits for
    the readers of the cells it overwrites); the last layer and the optimum must equal the oracle's."""
    import torch
    from paper_2504_03662_b200.search import SearchBuffers
    B, Lmax, S, M, kw = SHAPES[k]
    w = inputs.random_tables(700 + k, B, Lmax, S, M, **kw)
    sb = SearchBuffers(galv, w, flags)
    assert sb.C is None and sb.A is None
    for _ in range(2):                                       # the second run starts from used buffers
        sb.dp_search(); sb.backtrack()
        res = sb.results()
        for i in range(B):
            Li = int(w.L[i])
            r = orc.search(w.time_q[i, :Li], w.mem_q[i, :Li], w.trans_q[i], M)
            assert res["status"][i] == r["status"] and res["opt_cost"][i] == r["opt_cost"], i
            assert (res["plan"][i] == -1).all() and res["mem_used"][i] == 0          # no table, no walk
            if r["C"] is not None:
                assert (sb.C_last[i, :, :M + 1].t().cpu().numpy() == r["C"][Li - 1]).all(), i


def test_cost_only_search_many_layers_against_full_table(galv):
    """Rolling buffer under load: many instances, tiles and layers; the last layer must equal the full-table run's."""
    import torch
    from paper_2504_03662_b200 import binding as gb
    from paper_2504_03662_b200.search import SearchBuffers
    for seed, (B, Lmax, S, M, kw) in enumerate([(96, 40, 32, 2048, dict(mem_lo=8, mem_hi=128)),
                                                (40, 25, 64, 3000, dict(mem_lo=1, mem_hi=900, ragged=True)),
                                                (300, 12, 24, 700, dict(mem_lo=0, mem_hi=40, ragged=True))]):
        w = inputs.random_tables(8100 + seed, B, Lmax, S, M, **kw)
        full = SearchBuffers(galv, w, gb.STORE_C_FULL | gb.KERNEL_NO_CLUSTER)
        full.dp_search(); full.backtrack()
        for lean_flags in (gb.KERNEL_NO_CLUSTER, gb.KERNEL_CLUSTER):
          lean = SearchBuffers(galv, w, lean_flags)
          for _ in range(3):
              lean.dp_search(); lean.backtrack()
              torch.cuda.synchronize()
              assert torch.equal(lean.status, full.status) and torch.equal(lean.opt_cost, full.opt_cost)
              ok = full.status == 0
              assert torch.equal(lean.C_last[ok], full.C_last[ok])


@pytest.mark.parametrize("k", [3, 4])
def test_skipping_flags_change_no_cell_of_the_large_workloads(galv, k):
    """Every cell of every instance of configs 3 and 4: the tables, optima and plans with GALV_SKIP_DOMINATED |
    GALV_SKIP_INFEASIBLE equal those of the plain run (which the exhaustive pass below ties to the oracle)."""
    import torch
    from paper_2504_03662_b200 import binding as gb
    from paper_2504_03662_b200.search import SearchBuffers
    w = inputs.CONFIGS[k]()
    plain = SearchBuffers(galv, w, gb.STORE_C_FULL)
    plain.step()
    skip = SearchBuffers(galv, w, gb.STORE_C_FULL | gb.SKIP_DOMINATED | gb.SKIP_INFEASIBLE)
    skip.step()
    torch.cuda.synchronize()
    assert torch.equal(plain.status, skip.status) and torch.equal(plain.opt_cost, skip.opt_cost)
    assert torch.equal(plain.plan, skip.plan) and torch.equal(plain.mem_used, skip.mem_used)
    M = w.M
    for i in range(w.B):
        Li = int(w.L[i])
        assert torch.equal(plain.C[i, :Li, :, :M + 1], skip.C[i, :Li, :, :M + 1]), i
    del plain, skip
    torch.cuda.empty_cache()


@pytest.mark.parametrize("k", [3, 4])
def test_full_parity_every_instance(orc, galv, k):
    """Whole tables of ALL instances of configs 3 and 4 against the oracle, streamed a few instances at a time:
    every cell, optimum, plan and memory (about two minutes of oracle time on the host cores)."""
    import torch
    from paper_2504_03662_b200 import binding as gb
    from paper_2504_03662_b200.search import SearchBuffers
    w = inputs.CONFIGS[k]()
    tq, mq, xq = oracle_tables(orc, w)
    sb = SearchBuffers(galv, w, gb.STORE_C_FULL)
    sb.step()
    res = sb.results()
    chunk = 8
    for i0 in range(0, w.B, chunk):
        idx = list(range(i0, min(w.B, i0 + chunk)))
        ref = oracle_search_many(orc, w, tq, mq, xq, idx)
        for i in idx:
            r, Li = ref[i], int(w.L[i])
            assert res["status"][i] == r["status"] and res["opt_cost"][i] == r["opt_cost"], i
            assert (res["plan"][i, :Li] == r["plan"]).all() and res["mem_used"][i] == r["mem_used"], i
            assert (sb.table(i)[:Li] == r["C"]).all(), i
        del ref


@pytest.mark.parametrize("S,M,B,Lmax", [(64, 1500, 5, 9), (48, 900, 4, 12), (8, 5000, 3, 6), (24, 2881, 6, 7), (4, 300, 2, 5)])
def test_packed_16bit_path_choice_and_parity(orc, galv, S, M, B, Lmax):
    """The packed 16-bit inner loop is taken exactly when every transition entry is <= 32767 (and the shape allows
    it); its tables equal the 32-bit loop's and the oracle's, at the limit and with costs far above 16 bits."""
    import torch
    from paper_2504_03662_b200 import binding as gb
    from paper_2504_03662_b200.search import SearchBuffers
    for top, want in ((32767, True), (32768, False), (5, True)):
        w = inputs.random_tables(4000 + S + top % 7, B, Lmax, S, M, ragged=True, mem_lo=0, mem_hi=M // 4,
                                 time_hi=3_000_000, trans_hi=top)
        w.trans_q[0, 0, min(1, S - 1)] = top                     # the largest entry is really there
        w.time_q[B - 1, 1, :] = 7                                # a cheap layer: big spreads between strategies elsewhere
        w.mem_q[0, 2, : S // 2] = M + 5                          # +inf rows in some columns
        sb = SearchBuffers(galv, w, gb.STORE_C_FULL | gb.KERNEL_NO_CLUSTER)
        sb.dp_search(); sb.backtrack()
        assert galv.galv_dp_search_path(sb.shape, sb.workspace) == want
        res = sb.results()
        plain = SearchBuffers(galv, w, gb.STORE_C_FULL | gb.KERNEL_NO_PACKED | gb.KERNEL_NO_CLUSTER)
        plain.dp_search(); plain.backtrack()
        assert not galv.galv_dp_search_path(plain.shape, plain.workspace)
        assert torch.equal(sb.status, plain.status) and torch.equal(sb.opt_cost, plain.opt_cost)
        pruned = SearchBuffers(galv, w, gb.STORE_C_FULL | gb.SKIP_DOMINATED | gb.KERNEL_NO_CLUSTER)     # dominated row pairs left out
        pruned.dp_search(); pruned.backtrack()
        assert galv.galv_dp_search_path(pruned.shape, pruned.workspace) == want
        assert torch.equal(pruned.status, plain.status) and torch.equal(pruned.opt_cost, plain.opt_cost)
        assert torch.equal(pruned.plan, plain.plan)
        for i in range(B):
            Li = int(w.L[i])
            assert torch.equal(sb.C[i, :Li], plain.C[i, :Li]), (top, i)
            assert torch.equal(pruned.C[i, :Li], plain.C[i, :Li]), (top, i)
            r = orc.search(w.time_q[i, :Li], w.mem_q[i, :Li], w.trans_q[i], M)
            assert res["status"][i] == r["status"] and res["opt_cost"][i] == r["opt_cost"]
            if r["C"] is not None:
                assert (sb.table(i)[:Li] == r["C"]).all(), (top, i)
    # shapes the packed path does not take: S not a multiple of 4, S > 64, an argmin table
    nc = gb.KERNEL_NO_CLUSTER
    for S2, flags in ((6, gb.STORE_C_FULL | nc), (70, gb.STORE_C_FULL | nc), (S, gb.STORE_C_FULL | gb.STORE_ARGMIN)):
        w = inputs.random_tables(77, 2, 4, S2, 200, trans_hi=100)
        sb = SearchBuffers(galv, w, flags)
        sb.dp_search()
        assert not galv.galv_dp_search_path(sb.shape, sb.workspace)


@pytest.mark.parametrize("S,M,trans_hi,time_hi", [(4, 300, 0, 50), (16, 1000, 1, 1000), (36, 515, 40, 100000),
                                                 (64, 2100, 500, 20), (64, 767, 32767, 10 ** 6), (8, 255, 3, 3),
                                                 (32, 2100, 50000, 10 ** 6), (61, 700, 90000, 10 ** 5), (24, 130, 7, 10 ** 4)])
def test_dominated_rows_left_out(orc, galv, S, M, trans_hi, time_hi):
    """GALV_SKIP_DOMINATED: rows that cannot win in any column of a tile are not relaxed; the tables stay those of
    the oracle when all transitions are 0 (only exact ties survive), with wide and with narrow spreads of the
    costs, with columns that hold no finite value, and in the ragged last tile."""
    from paper_2504_03662_b200 import binding as gb
    from paper_2504_03662_b200.search import SearchBuffers
    B, Lmax = 5, 6
    w = inputs.random_tables(9000 + S + trans_hi, B, Lmax, S, M, ragged=True, mem_lo=0, mem_hi=max(1, M // 3),
                             time_hi=time_hi, trans_hi=trans_hi)
    w.time_q[1, :, :] = 11                                       # one instance without any spread: every row ties
    w.mem_q[2, 1, : max(1, S // 2)] = M + 9                      # rows that are +inf everywhere
    w.mem_q[3, 0, :] = M // 2                                    # the lower half of every later column is +inf
    for flags in (gb.STORE_C_FULL | gb.SKIP_DOMINATED, gb.SKIP_DOMINATED, gb.STORE_C_FULL | gb.SKIP_DOMINATED | gb.SKIP_INFEASIBLE,
                  gb.STORE_C_FULL | gb.SKIP_DOMINATED | gb.KERNEL_NO_PACKED,            # the 32-bit loop's variant
                  gb.SKIP_DOMINATED | gb.SKIP_INFEASIBLE | gb.KERNEL_NO_PACKED,
                  gb.STORE_C_FULL | gb.STORE_ARGMIN | gb.SKIP_DOMINATED,                # one launch per layer, argmin table
                  gb.STORE_ARGMIN | gb.SKIP_DOMINATED | gb.SKIP_INFEASIBLE,
                  gb.STORE_C_FULL | gb.KERNEL_PER_LAYER | gb.SKIP_DOMINATED):
        sb = SearchBuffers(galv, w, flags | gb.KERNEL_NO_CLUSTER)
        sb.dp_search(); sb.backtrack()
        packable = (S % 4 == 0 and int(w.trans_q.max()) <= 32767
                    and not flags & (gb.KERNEL_NO_PACKED | gb.STORE_ARGMIN | gb.KERNEL_PER_LAYER))
        assert galv.galv_dp_search_path(sb.shape, sb.workspace) == packable
        res = sb.results()
        for i in range(B):
            Li = int(w.L[i])
            r = orc.search(w.time_q[i, :Li], w.mem_q[i, :Li], w.trans_q[i], M)
            assert res["status"][i] == r["status"] and res["opt_cost"][i] == r["opt_cost"], (flags, i)
            if flags & (gb.STORE_C_FULL | gb.STORE_ARGMIN):
                assert (res["plan"][i, :Li] == r["plan"]).all(), (flags, i)
            if flags & gb.STORE_C_FULL:
                assert (sb.table(i)[:Li] == r["C"]).all(), (flags, i)
            if flags & gb.STORE_ARGMIN:
                assert (sb.argmin_table(i)[:Li] == r["A"]).all(), (flags, i)


def test_packed_path_with_costs_near_the_limit(orc, galv):
    """Path sums just below 2^30 (the validation bound), tiny transitions: the packed loop works on differences,
    so the size of the costs themselves must not matter; a column without any finite value stays +inf."""
    import torch
    from paper_2504_03662_b200 import binding as gb
    from paper_2504_03662_b200.search import SearchBuffers
    B, Lmax, S, M = 3, 4, 16, 700
    w = inputs.random_tables(123, B, Lmax, S, M, mem_lo=0, mem_hi=200, time_hi=1000, trans_hi=9)
    w.time_q[:, :, :] += (2 ** 30 - 1 - 4 * 1000 - 3 * 9) // 4 - 1     # four layers: the worst path sum stays just below 2^30 - 1
    w.time_q[1, 2, ::2] = 0                                              # and some spread between strategies
    w.mem_q[2, 1, :] = M + 1                                             # instance 2: nothing fits from layer 1 on
    assert orc.validate(w.time_q[0], w.mem_q[0], w.trans_q[0]) == 0
    sb = SearchBuffers(galv, w, gb.STORE_C_FULL | gb.KERNEL_NO_CLUSTER)
    sb.dp_search(); sb.backtrack()
    assert galv.galv_dp_search_path(sb.shape, sb.workspace) == 1
    res = sb.results()
    for i in range(B):
        r = orc.search(w.time_q[i], w.mem_q[i], w.trans_q[i], M)
        assert res["status"][i] == r["status"] and res["opt_cost"][i] == r["opt_cost"], i
        assert (res["plan"][i] == r["plan"]).all()
        assert (sb.table(i) == r["C"]).all(), i
    assert res["status"][2] == 1 and res["opt_cost"][2] == INF


@pytest.mark.parametrize("cluster", [NC, CLU])
def test_two_streams_at_once(orc, galv, cluster):
    """Two searches enqueued on two streams, each with its own workspace: the one-launch kernels take turns on
    the GPU (a cooperative launch needs all its CTAs resident), the cluster kernels share it; both must finish
    and be right."""
    import torch
    from paper_2504_03662_b200 import binding as gb
    from paper_2504_03662_b200.search import SearchBuffers
    wa = inputs.random_tables(501, 40, 20, 32, 2000, mem_lo=1, mem_hi=150, trans_hi=900)       # packed loop
    wb = inputs.random_tables(502, 30, 25, 24, 1500, mem_lo=1, mem_hi=100, trans_hi=60000)     # 32-bit loop
    sa, sb_ = SearchBuffers(galv, wa, gb.STORE_C_FULL | cluster), SearchBuffers(galv, wb, gb.STORE_C_FULL | cluster)
    s1, s2 = torch.cuda.Stream(), torch.cuda.Stream()
    torch.cuda.synchronize()
    for _ in range(3):
        with torch.cuda.stream(s1):
            sa.dp_search(); sa.backtrack()
        with torch.cuda.stream(s2):
            sb_.dp_search(); sb_.backtrack()
    torch.cuda.synchronize()
    for w, s in ((wa, sa), (wb, sb_)):
        res = s.results()
        for i in range(0, w.B, 7):
            r = orc.search(w.time_q[i], w.mem_q[i], w.trans_q[i], w.M)
            assert res["status"][i] == r["status"] and res["opt_cost"][i] == r["opt_cost"]
            assert (res["plan"][i] == r["plan"]).all() and (s.table(i) == r["C"]).all()


@pytest.mark.parametrize("n,M", [(1, 1000), (2, 1000), (3, 1000), (4, 1000), (5, 1000), (6, 2880), (7, 2880), (8, 2880), (9, 2880),
                                 (12, 2880), (16, 2880)])
def test_cluster_kernel_every_cluster_size(orc, galv, n, M):
    """One shape cut over clusters of 1 .. 16 CTAs: columns per CTA, tiles that straddle two CTAs, pushes that skip
    a whole CTA (mem larger than a CTA's columns) and strategies that never fit all change with the size."""
    from paper_2504_03662_b200 import binding as gb
    w = inputs.random_tables(600 + n, 5, 7, 24, M, ragged=True, mem_lo=0, mem_hi=700, trans_hi=40000)
    w.mem_q[1, 2, :5] = M + 1                                  # never fits
    w.mem_q[2, 1, :] = 0                                       # a layer that costs no memory
    w.mem_q[3, 3, 4] = M                                       # fits only at the very edge
    sb, res = check_batch(orc, galv, w, gb.STORE_C_FULL | gb.CLUSTER_SIZE(n))
    assert galv.galv_dp_search_path(sb.shape, sb.workspace) == gb.PATH_CLUSTER
    # without a table: only the last layer and the optimum
    sb, res = check_batch(orc, galv, w, gb.CLUSTER_SIZE(n))
    assert galv.galv_dp_search_path(sb.shape, sb.workspace) == gb.PATH_CLUSTER


def test_cluster_kernel_more_instances_than_cluster_slots(orc, galv):
    """Hundreds of ragged instances: clusters are handed the instances longest first; every instance is searched
    exactly once, flagged ones are reported and skipped.  Above 512 instances the tiled kernels take over."""
    from paper_2504_03662_b200 import binding as gb
    for B, want in ((400, gb.PATH_CLUSTER), (512, gb.PATH_CLUSTER), (600, None)):
        w = inputs.random_tables(8800 + B, B, 6, 8, 1000, ragged=True, mem_lo=0, mem_hi=300)
        w.time_q[7, 0, 0] = -1
        w.L[11] = 0
        w.L[13] = 7
        w.time_q[17] = (INF - 1) // 2
        w.L[17] = 3
        sb, res = check_batch(orc, galv, w, gb.STORE_C_FULL | gb.CLUSTER_SIZE(8), idx=[0, 1, 2, 7, 17, B // 2, B - 1] + list(range(20, B, 37)))
        path = galv.galv_dp_search_path(sb.shape, sb.workspace)
        assert path == want if want is not None else path != gb.PATH_CLUSTER
        assert res["status"][[7, 11, 13, 17]].tolist() == [2, 2, 2, 4]
        # the rest against the tiled kernel, cell by cell
        ref = __import__("paper_2504_03662_b200.search", fromlist=["SearchBuffers"]).SearchBuffers(galv, w, gb.STORE_C_FULL | gb.KERNEL_NO_CLUSTER)
        ref.dp_search(); ref.backtrack()
        import torch
        torch.cuda.synchronize()
        assert torch.equal(ref.status, sb.status) and torch.equal(ref.opt_cost, sb.opt_cost) and torch.equal(ref.plan, sb.plan)
        ok = ref.status == 0
        assert torch.equal(ref.C_last[ok], sb.C_last[ok])
        for i in np.flatnonzero(ok.cpu().numpy()):
            Li = int(w.L[i])
            assert torch.equal(ref.C[i, :Li], sb.C[i, :Li]), int(i)


def test_cluster_kernel_flagged_instances(orc, galv):
    """Validation inside the cluster kernel: the same status bits as the validation pass of the tiled path."""
    from paper_2504_03662_b200 import binding as gb
    w = inputs.random_tables(5, 6, 4, 6, 50, ragged=True)
    w.time_q[1, 0, 2] = -7
    w.L[2] = 0
    w.time_q[3] = (INF - 1) // 2
    w.L[3] = 4
    w.mem_q[4, 1, :] = -1
    w.L[4] = 4
    w.L[5] = 9
    w.trans_q[0, 1, 2] = 0
    sb, res = check_batch(orc, galv, w, gb.STORE_C_FULL | gb.KERNEL_CLUSTER, idx=[0])
    assert galv.galv_dp_search_path(sb.shape, sb.workspace) == gb.PATH_CLUSTER
    assert res["status"].tolist()[1:] == [2, 2, 4, 2, 2]
    assert (res["opt_cost"][1:] == INF).all() and (res["plan"][1:] == -1).all()
    w.trans_q[0, 1, 2] = -1                                    # a negative transition entry
    sb, res = check_batch(orc, galv, w, gb.STORE_C_FULL | gb.KERNEL_CLUSTER, idx=[])
    assert res["status"][0] == 2


def test_cluster_kernel_is_chosen_for_small_batches_only(galv):
    from paper_2504_03662_b200 import binding as gb
    from paper_2504_03662_b200.search import SearchBuffers
    for w, want in ((inputs.config0(), gb.PATH_CLUSTER), (inputs.config4(B=16), gb.PATH_CLUSTER),
                    (inputs.config4(B=700), gb.PATH_TILED_32)):
        sb = SearchBuffers(galv, w, gb.STORE_C_FULL)
        sb.dp_search()
        assert galv.galv_dp_search_path(sb.shape, sb.workspace) == want, w.B
    # an argmin table keeps the tiled kernels, whatever the flag asks
    sb = SearchBuffers(galv, inputs.config0(), gb.STORE_C_FULL | gb.STORE_ARGMIN | gb.KERNEL_CLUSTER)
    sb.dp_search()
    assert galv.galv_dp_search_path(sb.shape, sb.workspace) == gb.PATH_TILED_32


@pytest.mark.parametrize("S,M,trans_hi,kw", [
    (64, 1500, 3000, {}), (48, 900, 50000, dict(ragged=True)), (13, 300, 2000, dict(ragged=True)),      # S % 4 != 0: trans rows staged by plain copies
    (33, 1000, 2, dict(dup_cols=True, time_hi=5)),                                                        # ties everywhere: the lowest row must win
    (24, 2881, (1 << 24) - 1, dict(time_hi=1000)), (24, 700, 1 << 24, dict(time_hi=1000)),                # the largest entry keys allow; one beyond: plain loop
    (64, 767, 40, dict(mem_lo=0, mem_hi=0)), (8, 5000, 700, dict(mem_hi=6000)), (1, 100, 5, {}), (40, 513, 100, dict(mem_lo=600, mem_hi=700))])
def test_argmin_table_with_keys(orc, galv, S, M, trans_hi, kw):
    """The argmin-table mode with one fused add-min per relaxation on keys (rebased cost << 6 | row): A and C against the
    oracle where keys apply (S <= 64, entries below 2^24) and where the plain compare-and-select loop takes over; with
    rows and columns that are +inf, with nothing feasible, and with tiles skipped below the feasibility frontier."""
    from paper_2504_03662_b200 import binding as gb
    B, Lmax = 4, 6
    w = inputs.random_tables(31000 + S + trans_hi % 1000, B, Lmax, S, M, trans_hi=trans_hi, **{**dict(mem_lo=0, mem_hi=max(1, M // 4)), **kw})
    if S > 1:
        w.trans_q[0, 0, 1] = trans_hi                            # the largest entry is really there
        w.mem_q[1, 2, : S // 2] = M + 3                          # +inf rows
    w.time_q[2, 1, :] = 9                                        # a layer without spread
    for flags in (gb.STORE_C_FULL | gb.STORE_ARGMIN, gb.STORE_ARGMIN, gb.STORE_C_FULL | gb.STORE_ARGMIN | gb.SKIP_INFEASIBLE):
        check_batch(orc, galv, w, flags)


@pytest.mark.parametrize("block", range(6))
def test_cluster_kernel_against_reference_kernel_on_many_shapes(galv, block):
    """Consistency stress of the cluster kernel (column split, pushes that cross one or several CTAs, fills, rounds of
    clusters, per-layer transition matrices): on random shapes, cluster sizes and memory distributions its tables must
    equal those of the one-thread-per-cell kernel, which other tests tie to the oracle.  Two runs per shape on the same
    buffers."""
    import torch
    from paper_2504_03662_b200 import binding as gb
    from paper_2504_03662_b200.search import SearchBuffers
    rng = np.random.default_rng(4200 + block)
    ran = 0
    for case in range(12):
        S = int(rng.choice([1, 3, 8, 13, 24, 32, 40, 48, 64, 100, 128]))
        Lmax = int(rng.integers(1, 14))
        M = int(rng.integers(95, 4000))
        B = int(rng.choice([1, 2, 5, 16, 40, 130]))
        mem_hi = int(rng.choice([0, 5, M // 30 + 1, M // 4 + 1, M + 50, 3 * M]))       # up to shifts that skip whole CTAs and never fit
        w = inputs.random_tables(61000 + 100 * block + case, B, Lmax, S, M, ragged=bool(rng.integers(0, 2)), mem_lo=0, mem_hi=mem_hi,
                                 trans_hi=int(rng.choice([0, 9, 40000])), time_hi=int(rng.choice([5, 10 ** 4, 10 ** 6])))
        if Lmax > 2 and rng.integers(0, 2):
            w.mem_q[:, int(rng.integers(1, Lmax)), :] += M // 2                          # one heavy layer
        if case % 4 == 3 and Lmax > 1:                                                   # one transition matrix per layer
            w.trans_q = np.ascontiguousarray(np.repeat(w.trans_q[:, None], Lmax, 1))
            w.trans_q[:, 1:] += rng.integers(0, 50, size=(B, Lmax - 1, S, S), dtype=np.int32)
        size = int(rng.choice([0, 0, 1, 2, 3, 4, 6, 8, 11, 16]))
        flags = gb.STORE_C_FULL | (gb.CLUSTER_SIZE(size) if size else gb.KERNEL_CLUSTER)
        ref = SearchBuffers(galv, w, gb.STORE_C_FULL | gb.KERNEL_REFERENCE)
        ref.dp_search(); ref.backtrack()
        one = SearchBuffers(galv, w, flags)
        for _ in range(2):
            one.C.fill_(-7); one.C_last.fill_(-7)
            one.dp_search(); one.backtrack()
            torch.cuda.synchronize()
            if galv.galv_dp_search_path(one.shape, one.workspace) != gb.PATH_CLUSTER:
                break                                            # this size is not possible for this shape: nothing to compare
            ran += 1
            st = ref.status.cpu().numpy()
            assert (one.status.cpu().numpy() == st).all(), (block, case)
            assert torch.equal(one.opt_cost, ref.opt_cost) and torch.equal(one.plan, ref.plan), (block, case)
            for i in np.flatnonzero((st & ~1) == 0):
                Li = int(w.L[i])
                assert torch.equal(one.C[i, :Li], ref.C[i, :Li]), (block, case, int(i), S, Lmax, M, B, size)
            ok = torch.from_numpy((st & ~1) == 0).to(one.C_last.device)
            assert torch.equal(one.C_last[ok], ref.C_last[ok]), (block, case)
        del ref, one
        torch.cuda.empty_cache()
    assert ran >= 8                                              # most of the shapes did run on the cluster kernel

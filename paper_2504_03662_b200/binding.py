"""ctypes binding of libgalv.so — argument marshalling only.

Every step of the search runs in the library's CUDA kernels; this module turns
torch tensors into raw device pointers and checks return codes.  PyTorch is used
for device memory and streams, nothing else.  There is no CPU fallback: if the
library is missing or the device is not a B200-class GPU the calls raise.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional

import torch

INF = 2 ** 30 - 1
OK, ERR_INVALID_ARG, ERR_UNSUPPORTED, ERR_WORKSPACE, ERR_CUDA, ERR_TIMEOUT = 0, -1, -2, -3, -4, -5
STATUS_INFEASIBLE, STATUS_BAD_INPUT, STATUS_OVERFLOW_RISK, STATUS_TIMEOUT = 1, 2, 4, 8
STORE_C_FULL, STORE_ARGMIN, KERNEL_REFERENCE, KERNEL_PER_LAYER, SKIP_INFEASIBLE = 1, 2, 256, 512, 1024
SKIP_DOMINATED = 8192
DEBUG_WITHHOLD_LOAD = 2048
KERNEL_NO_PACKED = 4096
KERNEL_NO_CLUSTER, KERNEL_CLUSTER = 16384, 32768
PATH_TILED_32, PATH_TILED_PACKED, PATH_CLUSTER = 0, 1, 2


def CLUSTER_SIZE(n: int) -> int:
    """Flag bits that ask for the cluster kernel with clusters of n CTAs."""
    return (n & 31) << 16
TRANS_PER_LAYER = 4
STATIC_WORKSPACE_BYTES = 1 << 20

LIB_PATH = os.path.join(os.path.dirname(os.path.abspath(__file__)), "libgalv.so")

EXPORTS = ("galv_create", "galv_destroy", "galv_strerror", "galv_last_error", "galv_eval_costs",
           "galv_dp_workspace_bytes", "galv_dp_search", "galv_dp_search_path", "galv_backtrack", "galv_search_host_arena_bytes",
           "galv_search_host", "galv_probe_int_alu", "galv_set_profiling", "galv_last_layer_loop_ms", "galv_layer_loop_ms_stats",
           "galv_dp_search_static", "galv_select_best", "galv_prune_strategies",
           "galv_compact_tables", "galv_expand_plan", "galv_plan_cost", "galv_graph_create", "galv_graph_launch",
           "galv_graph_destroy", "galv_layer_optima", "galv_stage_partition", "galv_add_switch_cost",
           "galv_switch_decision", "galv_skip_estimate")


class galv_shape(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("B", "Lmax", "S", "M", "m_pitch", "flags")]


class GalvError(RuntimeError):
    def __init__(self, code: int, text: str):
        super().__init__(f"galv error {code}: {text}")
        self.code = code


_lib = None


def load_library() -> C.CDLL:
    """dlopen the in-tree library (build it first with `python -m paper_2504_03662_b200.build`)."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise ImportError(f"{LIB_PATH} is missing: build it with `python -m paper_2504_03662_b200.build`; "
                          "there is no fallback path")
    lib = C.CDLL(LIB_PATH)
    vp, i64, sz = C.c_void_p, C.c_int64, C.c_size_t
    shp = C.POINTER(galv_shape)
    lib.galv_create.argtypes = [C.POINTER(vp), C.c_int]
    lib.galv_destroy.argtypes = [vp]
    lib.galv_strerror.argtypes = [C.c_int]
    lib.galv_strerror.restype = C.c_char_p
    lib.galv_last_error.argtypes = [vp]
    lib.galv_last_error.restype = C.c_char_p
    lib.galv_eval_costs.argtypes = [vp, shp, vp, vp, i64, vp, vp, vp, vp, vp, vp, vp, vp, vp]
    lib.galv_dp_workspace_bytes.argtypes = [vp, shp]
    lib.galv_dp_workspace_bytes.restype = sz
    lib.galv_dp_search.argtypes = [vp, shp, vp, vp, vp, vp, vp, vp, vp, vp, sz, vp, vp]
    lib.galv_dp_search_path.argtypes = [vp, shp, vp, C.POINTER(C.c_int32), vp]
    lib.galv_backtrack.argtypes = [vp, shp] + [vp] * 13
    lib.galv_dp_search_static.argtypes = [vp, shp] + [vp] * 9
    lib.galv_select_best.argtypes = [vp, C.c_int32, C.c_int32] + [vp] * 8
    lib.galv_prune_strategies.argtypes = [vp, shp] + [vp] * 8
    lib.galv_compact_tables.argtypes = [vp, shp, C.c_int32] + [vp] * 8
    lib.galv_expand_plan.argtypes = [vp, C.c_int32, C.c_int32, vp, vp, vp]
    lib.galv_plan_cost.argtypes = [vp, shp] + [vp] * 8
    lib.galv_add_switch_cost.argtypes = [vp, shp] + [vp] * 7
    lib.galv_switch_decision.argtypes = [vp, C.c_int32, vp, vp, vp, C.c_int32, vp, vp]
    lib.galv_graph_create.argtypes = [vp, shp, vp, vp, i64, vp, vp] + [vp] * 7 + [sz] + [vp] * 6 + [C.POINTER(vp)]
    lib.galv_graph_launch.argtypes = [vp, vp, vp]
    lib.galv_graph_destroy.argtypes = [vp]
    lib.galv_layer_optima.argtypes = [vp, shp] + [vp] * 6
    lib.galv_stage_partition.argtypes = [vp, C.c_int32, C.c_int32, vp, vp, vp, vp]
    lib.galv_skip_estimate.argtypes = [vp, shp] + [vp] * 6
    lib.galv_search_host_arena_bytes.argtypes = [vp, shp, C.c_int]
    lib.galv_search_host_arena_bytes.restype = sz
    lib.galv_search_host.argtypes = [vp, shp, vp, vp, i64, vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, sz, vp]
    lib.galv_probe_int_alu.argtypes = [vp, C.c_int, C.c_int, C.POINTER(C.c_double), vp]
    lib.galv_set_profiling.argtypes = [vp, C.c_int]
    lib.galv_last_layer_loop_ms.argtypes = [vp, C.POINTER(C.c_float)]
    lib.galv_layer_loop_ms_stats.argtypes = [vp, C.POINTER(C.c_float), C.POINTER(C.c_float), C.POINTER(C.c_float), C.POINTER(C.c_int)]
    _lib = lib
    return lib


def _ptr(t) -> Optional[int]:
    if t is None:
        return None
    if isinstance(t, torch.Tensor):
        assert t.is_contiguous(), "tensors crossing the boundary must be contiguous"
        return t.data_ptr()
    return t.ctypes.data          # numpy (host buffers of galv_search_host)


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


def make_shape(B: int, Lmax: int, S: int, M: int, flags: int = STORE_C_FULL, m_pitch: Optional[int] = None) -> galv_shape:
    return galv_shape(B, Lmax, S, M, (M + 1 + 31) // 32 * 32 if m_pitch is None else m_pitch, flags)


class Galv:
    """One library context on one CUDA device.  Methods carry the C entry points' names."""

    def __init__(self, device: int = 0):
        self.lib = load_library()
        if not torch.cuda.is_available():
            raise RuntimeError("no CUDA device: the search runs only in the CUDA library (no CPU path)")
        self.device = device
        h = C.c_void_p()
        rc = self.lib.galv_create(C.byref(h), device)
        if rc != OK:
            raise GalvError(rc, self.lib.galv_strerror(rc).decode())
        self.h = h

    def close(self):
        if getattr(self, "h", None):
            self.lib.galv_destroy(self.h)
            self.h = None

    __del__ = close

    def _check(self, rc: int):
        if rc != OK:
            raise GalvError(rc, f"{self.lib.galv_strerror(rc).decode()}: {self.lib.galv_last_error(self.h).decode()}")

    def galv_eval_costs(self, shape, L, layers, layer_stride_B, strat, inst, time_s, mem_bytes, time_q, mem_q,
                        trans_q, status):
        self._check(self.lib.galv_eval_costs(self.h, C.byref(shape), _ptr(L), _ptr(layers), layer_stride_B, _ptr(strat),
                                             _ptr(inst), _ptr(time_s), _ptr(mem_bytes), _ptr(time_q), _ptr(mem_q),
                                             _ptr(trans_q), _ptr(status), _stream()))

    def galv_dp_workspace_bytes(self, shape) -> int:
        return int(self.lib.galv_dp_workspace_bytes(self.h, C.byref(shape)))

    def galv_dp_search(self, shape, L, time_q, mem_q, trans_q, Ct, At, C_last, workspace, status):
        self._check(self.lib.galv_dp_search(self.h, C.byref(shape), _ptr(L), _ptr(time_q), _ptr(mem_q), _ptr(trans_q),
                                            _ptr(Ct), _ptr(At), _ptr(C_last), _ptr(workspace),
                                            0 if workspace is None else workspace.numel() * workspace.element_size(),
                                            _ptr(status), _stream()))

    def galv_dp_search_static(self, shape, L, time_q, mem_q, trans_q, Ct, At, C_last, status):
        """galv_dp_search on the library's built-in scratch array: nothing is allocated, the caller passes no workspace."""
        self._check(self.lib.galv_dp_search_static(self.h, C.byref(shape), _ptr(L), _ptr(time_q), _ptr(mem_q),
                                                   _ptr(trans_q), _ptr(Ct), _ptr(At), _ptr(C_last), _ptr(status),
                                                   _stream()))

    def galv_select_best(self, B, G, opt_cost, status, n_micro, pp, group, best_time, best_inst):
        self._check(self.lib.galv_select_best(self.h, B, G, _ptr(opt_cost), _ptr(status), _ptr(n_micro), _ptr(pp),
                                              _ptr(group), _ptr(best_time), _ptr(best_inst), _stream()))

    def galv_prune_strategies(self, shape, L, time_q, mem_q, trans_q, keep, map_, S_kept):
        self._check(self.lib.galv_prune_strategies(self.h, C.byref(shape), _ptr(L), _ptr(time_q), _ptr(mem_q), _ptr(trans_q),
                                                   _ptr(keep), _ptr(map_), _ptr(S_kept), _stream()))

    def galv_compact_tables(self, shape, S_kept, map_, time_q, mem_q, trans_q, time_out, mem_out, trans_out):
        self._check(self.lib.galv_compact_tables(self.h, C.byref(shape), S_kept, _ptr(map_), _ptr(time_q), _ptr(mem_q),
                                                 _ptr(trans_q), _ptr(time_out), _ptr(mem_out), _ptr(trans_out), _stream()))

    def galv_expand_plan(self, B, Lmax, map_, plan):
        self._check(self.lib.galv_expand_plan(self.h, B, Lmax, _ptr(map_), _ptr(plan), _stream()))

    def galv_plan_cost(self, shape, L, time_q, mem_q, trans_q, plan, cost, mem_total):
        self._check(self.lib.galv_plan_cost(self.h, C.byref(shape), _ptr(L), _ptr(time_q), _ptr(mem_q), _ptr(trans_q),
                                            _ptr(plan), _ptr(cost), _ptr(mem_total), _stream()))

    def galv_add_switch_cost(self, shape, L, time_q, trans_q, cur_plan, horizon, time_out):
        self._check(self.lib.galv_add_switch_cost(self.h, C.byref(shape), _ptr(L), _ptr(time_q), _ptr(trans_q), _ptr(cur_plan),
                                                  _ptr(horizon), _ptr(time_out), _stream()))

    def galv_switch_decision(self, B, cur_cost, new_cost, new_status, hysteresis_permille, decision):
        self._check(self.lib.galv_switch_decision(self.h, B, _ptr(cur_cost), _ptr(new_cost), _ptr(new_status),
                                                  int(hysteresis_permille), _ptr(decision), _stream()))

    def galv_graph_create(self, shape, L, layers, layer_stride_B, strat, inst, time_q, mem_q, trans_q, Ct, At, C_last,
                          workspace, budget, opt_cost, plan, mem_used, status, stream: int):
        g = C.c_void_p()
        self._check(self.lib.galv_graph_create(self.h, C.byref(shape), _ptr(L), _ptr(layers), layer_stride_B, _ptr(strat),
                                               _ptr(inst), _ptr(time_q), _ptr(mem_q), _ptr(trans_q), _ptr(Ct), _ptr(At),
                                               _ptr(C_last), _ptr(workspace),
                                               workspace.numel() * workspace.element_size(), _ptr(budget), _ptr(opt_cost),
                                               _ptr(plan), _ptr(mem_used), _ptr(status), stream, C.byref(g)))
        return g

    def galv_graph_launch(self, graph, stream: Optional[int] = None):
        self._check(self.lib.galv_graph_launch(self.h, graph, _stream() if stream is None else stream))

    def galv_graph_destroy(self, graph):
        self.lib.galv_graph_destroy(graph)

    def galv_layer_optima(self, shape, L, Ct, budget, status, opt_l):
        self._check(self.lib.galv_layer_optima(self.h, C.byref(shape), _ptr(L), _ptr(Ct), _ptr(budget), _ptr(status),
                                               _ptr(opt_l), _stream()))

    def galv_skip_estimate(self, shape, L, time_q, mem_q, trans_q, counts):
        self._check(self.lib.galv_skip_estimate(self.h, C.byref(shape), _ptr(L), _ptr(time_q), _ptr(mem_q), _ptr(trans_q),
                                                _ptr(counts), _stream()))

    def galv_stage_partition(self, Lm, P, range_opt, cuts, bottleneck):
        self._check(self.lib.galv_stage_partition(self.h, Lm, P, _ptr(range_opt), _ptr(cuts), _ptr(bottleneck), _stream()))

    def galv_dp_search_path(self, shape, workspace) -> int:
        """Kernel of the most recent search on this workspace: 1 tiled kernel with the packed 16-bit inner loop
        (truthy, as before), 0 tiled kernel with the 32-bit loop, 2 cluster kernel."""
        out = C.c_int32()
        self._check(self.lib.galv_dp_search_path(self.h, C.byref(shape), _ptr(workspace), C.byref(out), _stream()))
        return int(out.value)

    def galv_backtrack(self, shape, L, time_q, mem_q, trans_q, Ct, At, C_last, budget, opt_cost, plan, mem_used, status):
        self._check(self.lib.galv_backtrack(self.h, C.byref(shape), _ptr(L), _ptr(time_q), _ptr(mem_q), _ptr(trans_q),
                                            _ptr(Ct), _ptr(At), _ptr(C_last), _ptr(budget), _ptr(opt_cost), _ptr(plan),
                                            _ptr(mem_used), _ptr(status), _stream()))

    def galv_search_host_arena_bytes(self, shape, with_model: bool) -> int:
        return int(self.lib.galv_search_host_arena_bytes(self.h, C.byref(shape), int(with_model)))

    def galv_search_host(self, shape, L, layers, layer_stride_B, strat, inst, time_q, mem_q, trans_q,
                         opt_cost, plan, mem_used, status, arena):
        self._check(self.lib.galv_search_host(self.h, C.byref(shape), _ptr(L), _ptr(layers), layer_stride_B, _ptr(strat),
                                              _ptr(inst), _ptr(time_q), _ptr(mem_q), _ptr(trans_q), _ptr(opt_cost),
                                              _ptr(plan), _ptr(mem_used), _ptr(status), _ptr(arena),
                                              arena.numel() * arena.element_size(), _stream()))

    def galv_probe_int_alu(self, kind: int, iters: int = 4096) -> float:
        out = C.c_double()
        self._check(self.lib.galv_probe_int_alu(self.h, kind, iters, C.byref(out), _stream()))
        return out.value

    def galv_set_profiling(self, on: bool):
        self._check(self.lib.galv_set_profiling(self.h, int(on)))

    def galv_last_layer_loop_ms(self) -> float:
        out = C.c_float()
        self._check(self.lib.galv_last_layer_loop_ms(self.h, C.byref(out)))
        return out.value

    def galv_layer_loop_ms_stats(self):
        """(mean, min, max, searches) of the layer-launch spans since profiling was switched on."""
        mean, lo, hi, n = C.c_float(), C.c_float(), C.c_float(), C.c_int()
        self._check(self.lib.galv_layer_loop_ms_stats(self.h, C.byref(mean), C.byref(lo), C.byref(hi), C.byref(n)))
        return mean.value, lo.value, hi.value, n.value

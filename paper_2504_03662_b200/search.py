"""Device buffers for one workload and the calls that run the path on them.

Holds no arithmetic: tensors are allocated through PyTorch and handed to the C
library; every step (cost model, validation, recurrence, optimum, backtrack)
runs in the library's kernels.
"""
from __future__ import annotations

from typing import Optional

import numpy as np
import torch

from . import binding as gb
from .inputs import Workload


def _dev_bytes(a: np.ndarray, device) -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(a).view(np.uint8).reshape(-1).copy()).to(device)


class SearchBuffers:
    """All device arrays of one batch, laid out as the C boundary expects."""

    def __init__(self, galv: gb.Galv, w: Workload, flags: int = gb.STORE_C_FULL, device: Optional[str] = None):
        self.galv, self.w, self.flags = galv, w, flags
        dev = torch.device(device or f"cuda:{galv.device}")
        self.dev = dev
        if w.trans_q is not None and w.trans_q.ndim == 4:          # one transition matrix per layer
            flags |= gb.TRANS_PER_LAYER
        self.flags = flags
        self.shape = gb.make_shape(w.B, w.Lmax, w.S, w.M, flags)
        B, Lm, S, P = w.B, w.Lmax, w.S, self.shape.m_pitch
        i32 = dict(dtype=torch.int32, device=dev)
        self.L = torch.from_numpy(np.ascontiguousarray(w.L, np.int32)).to(dev)
        if w.has_model:
            self.layers = _dev_bytes(w.layers, dev)
            self.layer_stride_B = 0 if w.layers.shape[0] == 1 else w.Lmax
            self.strat = _dev_bytes(w.strat, dev)
            self.inst = _dev_bytes(w.inst, dev)
            self.time_q = torch.zeros(B, Lm, S, **i32)
            self.mem_q = torch.zeros(B, Lm, S, **i32)
            self.trans_q = torch.zeros(B, S, S, **i32)
        else:
            self.time_q = torch.from_numpy(np.ascontiguousarray(w.time_q, np.int32)).to(dev)
            self.mem_q = torch.from_numpy(np.ascontiguousarray(w.mem_q, np.int32)).to(dev)
            self.trans_q = torch.from_numpy(np.ascontiguousarray(w.trans_q, np.int32)).to(dev)
        self.time_s = self.mem_bytes = None
        self.C = torch.empty(B, Lm, S, P, **i32) if flags & gb.STORE_C_FULL else None
        self.A = torch.empty(B, Lm, S, P, dtype=torch.uint8, device=dev) if flags & gb.STORE_ARGMIN else None
        self.C_last = torch.empty(B, S, P, **i32)
        self.workspace = torch.empty(max(256, galv.galv_dp_workspace_bytes(self.shape)), dtype=torch.uint8, device=dev)
        self.status = torch.zeros(B, **i32)
        self.opt_cost = torch.empty(B, **i32)
        self.plan = torch.full((B, Lm), -1, **i32)             # stays -1 / 0 when no table is kept (cost-only search)
        self.mem_used = torch.zeros(B, **i32)

    def eval_costs(self, want_fp64: bool = False):
        w = self.w
        assert w.has_model
        if want_fp64 and self.time_s is None:
            self.time_s = torch.zeros(w.B, w.Lmax, w.S, dtype=torch.float64, device=self.dev)
            self.mem_bytes = torch.zeros(w.B, w.Lmax, w.S, dtype=torch.float64, device=self.dev)
        self.galv.galv_eval_costs(self.shape, self.L, self.layers, self.layer_stride_B, self.strat, self.inst,
                                  self.time_s if want_fp64 else None, self.mem_bytes if want_fp64 else None,
                                  self.time_q, self.mem_q, self.trans_q, self.status)

    def dp_search(self):
        self.galv.galv_dp_search(self.shape, self.L, self.time_q, self.mem_q, self.trans_q, self.C, self.A,
                                 self.C_last, self.workspace, self.status)

    def backtrack(self, budget: Optional[torch.Tensor] = None, use_A: Optional[bool] = None):
        A = self.A if (use_A is None or use_A) else None
        C = self.C if (use_A is None or not use_A) else None
        walk = C is not None or A is not None                   # a plan needs one of the tables
        self.galv.galv_backtrack(self.shape, self.L, self.time_q, self.mem_q, self.trans_q, C, A, self.C_last,
                                 budget, self.opt_cost, self.plan if walk else None, self.mem_used if walk else None,
                                 self.status)

    def step(self):
        """One pass of the whole path on the current stream (asynchronous)."""
        if self.w.has_model:
            self.eval_costs()
        self.dp_search()
        self.backtrack()

    def results(self):
        torch.cuda.synchronize(self.dev)
        return dict(opt_cost=self.opt_cost.cpu().numpy(), plan=self.plan.cpu().numpy(),
                    mem_used=self.mem_used.cpu().numpy(), status=self.status.cpu().numpy())

    def table(self, i: int) -> np.ndarray:
        """C of instance i in the recurrence's index order [L][M+1][S] (host copy)."""
        M = self.w.M
        return np.ascontiguousarray(self.C[i, :, :, :M + 1].permute(0, 2, 1).cpu().numpy())

    def argmin_table(self, i: int) -> np.ndarray:
        M = self.w.M
        return np.ascontiguousarray(self.A[i, :, :, :M + 1].permute(0, 2, 1).cpu().numpy())


class HostSearch:
    """The host-buffer entry point: pinned host inputs/outputs and a device arena."""

    def __init__(self, galv: gb.Galv, w: Workload, flags: int = gb.STORE_C_FULL):
        self.galv, self.w = galv, w
        if w.trans_q is not None and w.trans_q.ndim == 4:          # one transition matrix per layer
            flags |= gb.TRANS_PER_LAYER
        self.shape = gb.make_shape(w.B, w.Lmax, w.S, w.M, flags)
        pin = lambda a: torch.from_numpy(np.ascontiguousarray(a).view(np.uint8).reshape(-1).copy()).pin_memory()
        self.L = pin(np.ascontiguousarray(w.L, np.int32))
        self.model = w.has_model
        if self.model:
            self.layers, self.strat, self.inst = pin(w.layers), pin(w.strat), pin(w.inst)
            self.layer_stride_B = 0 if w.layers.shape[0] == 1 else w.Lmax
            self.tq = self.mq = self.xq = None
            self.h2d = sum(t.numel() for t in (self.L, self.layers, self.strat, self.inst))
        else:
            self.layers = self.strat = self.inst = None
            self.layer_stride_B = 0
            self.tq, self.mq, self.xq = pin(w.time_q), pin(w.mem_q), pin(w.trans_q)
            self.h2d = sum(t.numel() for t in (self.L, self.tq, self.mq, self.xq))
        i32 = dict(dtype=torch.int32)
        self.opt_cost = torch.empty(w.B, **i32).pin_memory()
        self.plan = torch.empty(w.B, w.Lmax, **i32).pin_memory()
        self.mem_used = torch.empty(w.B, **i32).pin_memory()
        self.status = torch.empty(w.B, **i32).pin_memory()
        self.d2h = 4 * (3 * w.B + w.B * w.Lmax)
        self.arena = torch.empty(galv.galv_search_host_arena_bytes(self.shape, self.model), dtype=torch.uint8,
                                 device=f"cuda:{galv.device}")

    def run(self):
        """Synchronous: returns when the results are in the host buffers."""
        self.galv.galv_search_host(self.shape, self.L, self.layers, self.layer_stride_B, self.strat, self.inst,
                                   self.tq, self.mq, self.xq, self.opt_cost, self.plan, self.mem_used, self.status,
                                   self.arena)
        return dict(opt_cost=self.opt_cost.numpy(), plan=self.plan.numpy(), mem_used=self.mem_used.numpy(),
                    status=self.status.numpy())

"""Out-of-bounds writes: every output buffer of the path sits between guard zones that must stay untouched.

A memory checker cannot be counted on where this suite runs, so the suite carries its own: each buffer the
library writes (cost tables, C, A, C_last, workspace, optimum, plan, memory, status) is a window inside a
larger allocation whose margins hold a known pattern; after the cost model, the search and the plan step have
run in every table mode and kernel variant, the margins are compared with the pattern.  A store one row before
a table, one column past its pitch, or past the end of the workspace shows up here.
"""
import numpy as np
import pytest

from paper_2504_03662_b200 import inputs
from tests.test_gpu_parity import SHAPES

pytestmark = pytest.mark.gpu

GUARD_BYTES = 1 << 16          # on each side; a multiple of 256, so windows keep the alignment the boundary asks for
PATTERN = 0xA5


class Guarded:
    """A tensor window of `numel` elements between two margins filled with PATTERN."""

    def __init__(self, torch, numel, dtype, dev):
        item = torch.empty(0, dtype=dtype).element_size()
        self.nbytes = numel * item
        pad = (-self.nbytes) % 256
        self.raw = torch.full((GUARD_BYTES + self.nbytes + pad + GUARD_BYTES,), PATTERN, dtype=torch.uint8, device=dev)
        self.view = self.raw[GUARD_BYTES:GUARD_BYTES + self.nbytes].view(dtype)
        self.tail = GUARD_BYTES + self.nbytes

    def intact(self) -> bool:
        return bool((self.raw[:GUARD_BYTES] == PATTERN).all()) and bool((self.raw[self.tail:] == PATTERN).all())


def guarded_buffers(galv, w, flags):
    """SearchBuffers whose every library-written array is a guarded window."""
    import torch
    from paper_2504_03662_b200 import binding as gb
    from paper_2504_03662_b200.search import SearchBuffers
    sb = SearchBuffers(galv, w, flags)
    guards = {}

    def swap(name, keep_contents=False):
        old = getattr(sb, name)
        if old is None:
            return
        g = Guarded(torch, old.numel(), old.dtype, sb.dev)
        new = g.view.view(old.shape)
        if keep_contents:
            new.copy_(old)
        setattr(sb, name, new)
        guards[name] = g

    for name in ("C", "A", "C_last", "workspace", "opt_cost", "plan", "mem_used", "status"):
        swap(name)
    sb.plan.fill_(-1)
    sb.mem_used.zero_()
    for name in ("time_q", "mem_q", "trans_q"):                 # written by the cost model when there is one
        swap(name, keep_contents=True)
    return sb, guards


NC, CLU = 16384, 32768        # tiled kernels only / the cluster kernel wherever the shape allows
MODES = [1 | NC, 3, 2, NC, 1 | 512, 1 | 1024 | 8192 | NC, 1 | 4096 | NC, 2 | 8192, 1 | 256, 1 | CLU, CLU, 1 | CLU | (2 << 16), 1 | CLU | (16 << 16)]


@pytest.mark.parametrize("flags", MODES)
def test_guard_zones_stay_untouched_on_every_shape(orc, flags):
    import torch
    from paper_2504_03662_b200 import binding as gb
    galv = gb.Galv(0)
    try:
        for k, (B, Lmax, S, M, kw) in enumerate(SHAPES):
            w = inputs.random_tables(700 + k, B, Lmax, S, M, **kw)
            sb, guards = guarded_buffers(galv, w, flags)
            for _ in range(2):
                sb.dp_search()
                sb.backtrack()
            res = sb.results()
            for name, g in guards.items():
                assert g.intact(), (k, name, flags)
            # and the run between the guards is still the right one
            for i in range(B):
                Li = int(w.L[i])
                r = orc.search(w.time_q[i, :Li], w.mem_q[i, :Li], w.trans_q[i], M)
                assert res["status"][i] == r["status"] and res["opt_cost"][i] == r["opt_cost"], (k, i)
            del sb, guards
            torch.cuda.empty_cache()
    finally:
        galv.close()


def test_guard_zones_with_the_cost_model_and_ragged_layers(orc):
    """Configs 1 and 2 (cost model writes the integer tables; config 2 is ragged: rows beyond L[i] are not written)."""
    import torch
    from paper_2504_03662_b200 import binding as gb
    galv = gb.Galv(0)
    try:
        for w, flags in ((inputs.config1(), 3), (inputs.config2(), 1), (inputs.config0(), 3)):
            sb, guards = guarded_buffers(galv, w, flags)
            sb.step()
            res = sb.results()
            for name, g in guards.items():
                assert g.intact(), (w.name, name)
            assert (res["status"] & ~1 == 0).all()
            del sb, guards
            torch.cuda.empty_cache()
    finally:
        galv.close()

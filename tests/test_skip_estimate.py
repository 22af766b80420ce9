"""galv_skip_estimate: the counts against their definition written out in numpy, and against what the search really skips."""
import numpy as np
import pytest

from paper_2504_03662_b200 import inputs

pytestmark = pytest.mark.gpu


def counts_by_definition(w, tq, mq, xq, tmb):
    ntiles = (w.M + 1 + tmb - 1) // tmb
    below = total = dom = rows = 0
    for i in range(w.B):
        Li = int(w.L[i])
        if not 1 <= Li <= w.Lmax:
            continue
        front = np.minimum(np.cumsum(np.maximum(mq[i, :Li].min(axis=1), 0).astype(np.int64)), w.M + 1)
        for l in range(1, Li):                                   # layer l reads layer l-1
            below += min(ntiles, int(front[l - 1]) // tmb)
        total += (Li - 1) * ntiles
        T = xq[i] if xq.ndim == 3 else xq[i, 1]
        fits = mq[i, 0] <= w.M
        best = int(tq[i, 0][fits].min()) if fits.any() else 2 ** 31 - 1
        dom += int(((~fits) | (tq[i, 0].astype(np.int64) > best + int(T.max()))).sum())
        rows += w.S
    return [below, total, dom, rows]


def test_counts_match_their_definition(orc):
    import torch
    from paper_2504_03662_b200 import binding as gb
    from paper_2504_03662_b200.search import SearchBuffers
    from tests.test_gpu_parity import oracle_tables
    galv = gb.Galv(0)
    try:
        cases = [inputs.config3(B=16), inputs.config4(B=64), inputs.config1(), inputs.config2(),
                 inputs.random_tables(3, 9, 7, 13, 300, ragged=True, mem_lo=0, mem_hi=400, trans_hi=50)]
        cases[-1].L[4] = 0                                      # an instance that is not counted
        for w in cases:
            sb = SearchBuffers(galv, w, gb.STORE_C_FULL)
            if w.has_model:
                sb.eval_costs()
            counts = torch.zeros(4, dtype=torch.int64, device=sb.dev)
            galv.galv_skip_estimate(sb.shape, sb.L, sb.time_q, sb.mem_q, sb.trans_q, counts)
            torch.cuda.synchronize()
            tq, mq, xq = oracle_tables(orc, w)
            # the tile width is the tiled kernel's: 16 consumer warps of 128 columns, split over the strategy groups
            nsb = ((w.S + 7) // 8 * 8 + 63) // 64
            nsg = ((w.S + nsb - 1) // nsb + 7) // 8
            tmb = max(1, 16 // nsg) * 128
            assert counts.tolist() == counts_by_definition(w, tq, mq, xq, tmb), w.name
        # the heterogeneous stack's tight budget: close to half of its tiles lie below the frontier
        w = inputs.config3(B=16)
        sb = SearchBuffers(galv, w, gb.STORE_C_FULL)
        sb.eval_costs()
        counts = torch.zeros(4, dtype=torch.int64, device=sb.dev)
        galv.galv_skip_estimate(sb.shape, sb.L, sb.time_q, sb.mem_q, sb.trans_q, counts)
        c = counts.tolist()
        assert 0.4 < c[0] / c[1] < 0.55 and c[2] > 0
    finally:
        galv.close()

"""Seeded synthetic inputs for the strategy-search path.

This module only *describes* search instances: layer, strategy and instance
descriptor tables for the analytic workloads, and integer time/mem/trans tables
for the random workloads.  It contains none of the method's arithmetic (no cost
formula, no quantisation, no recurrence): the CUDA path and the CPU oracle each
carry their own, and both read the arrays produced here.

It depends on numpy alone and never loads the CUDA library.

Workloads (the paper gives no datasets; its selector consumes profiler
statistics — Section 3, "Dynamic Strategy Selector" — which are modelled here
as descriptor tables):

  0  tiny random search          B=1    L=4    S=6   M=64    seed 0
  1  GPT-style uniform decoder   B=16   L=24   S=24  M=2880
  2  175B-shaped decoder         B=64   L<=96  S=48  M=2880  (ragged L)
  3  heterogeneous stack         B=128  L=160  S=64  M=8192  jitter seed 3
  4  re-search throughput sweep  B=1024 L=48   S=32  M=2048  seed 7
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Optional

import numpy as np

# Descriptor records, laid out exactly like the C structs of the boundary.
LAYER_DESC = np.dtype(
    [(n, "<f8") for n in ("h", "seq", "heads", "c_lin", "c_attn", "p_coef",
                          "n_ar", "act_rep", "act_tp", "act_attn")], align=True)
STRATEGY_DESC = np.dtype(
    [("tp", "<i4"), ("dp", "<i4"), ("zero", "<i4"), ("ckpt", "<i4"),
     ("sp", "<i4"), ("_pad", "<i4"), ("batch_div", "<f8")], align=True)
INST_PARAMS = np.dtype(
    [(n, "<f8") for n in ("b", "act_mult", "flops_rate", "bw_tp", "bw_dp",
                          "bytes_per_elem", "bin_bytes", "time_unit_ns")], align=True)
assert LAYER_DESC.itemsize == 80 and STRATEGY_DESC.itemsize == 32 and INST_PARAMS.itemsize == 64

_GOLDEN = np.uint64(0x9E3779B97F4A7C15)
_MIX1 = np.uint64(0xBF58476D1CE4E5B9)
_MIX2 = np.uint64(0x94D049BB133111EB)


def splitmix64(seed: int, n: int, skip: int = 0) -> np.ndarray:
    """Outputs skip .. skip+n-1 of the splitmix64 stream whose state starts at `seed`.

    The k-th output (k from 0) mixes the state seed + (k+1)*golden, so the whole
    stream can be produced at once with wrapping uint64 arithmetic.
    """
    k = np.arange(skip + 1, skip + n + 1, dtype=np.uint64)
    with np.errstate(over="ignore"):
        z = np.uint64(seed) + k * _GOLDEN
        z = (z ^ (z >> np.uint64(30))) * _MIX1
        z = (z ^ (z >> np.uint64(27))) * _MIX2
    return z ^ (z >> np.uint64(31))


def _randint(x: np.ndarray, lo: int, hi: int) -> np.ndarray:
    return (lo + (x % np.uint64(hi - lo + 1)).astype(np.int64)).astype(np.int32)


def _unit(x: np.ndarray) -> np.ndarray:
    """53-bit uniform in [0, 1)."""
    return (x >> np.uint64(11)).astype(np.float64) * 2.0 ** -53


@dataclass
class Workload:
    """One batch of independent search instances.

    Either the integer tables (time_q, mem_q, trans_q) are given directly, or
    the descriptor tables (layers, strat, inst) from which the cost model
    derives them.
    """
    name: str
    B: int
    Lmax: int
    S: int
    M: int
    L: np.ndarray                               # [B] int32 layers per instance
    time_q: Optional[np.ndarray] = None         # [B][Lmax][S] int32
    mem_q: Optional[np.ndarray] = None          # [B][Lmax][S] int32
    trans_q: Optional[np.ndarray] = None        # [B][S][S]   int32, row = previous strategy
    layers: Optional[np.ndarray] = None         # [B or 1][Lmax] LAYER_DESC
    strat: Optional[np.ndarray] = None          # [S] STRATEGY_DESC
    inst: Optional[np.ndarray] = None           # [B] INST_PARAMS
    meta: dict = field(default_factory=dict)

    @property
    def has_model(self) -> bool:
        return self.layers is not None

    @property
    def m_pitch(self) -> int:
        return (self.M + 1 + 31) // 32 * 32

    @property
    def cells(self) -> int:
        return int(self.L.astype(np.int64).sum()) * (self.M + 1) * self.S

    @property
    def relaxations(self) -> int:
        return int((self.L.astype(np.int64) - 1).clip(min=0).sum()) * (self.M + 1) * self.S * self.S

    def take(self, idx) -> "Workload":
        """The sub-batch made of the instances `idx` (a slice or index list)."""
        idx = np.arange(self.B)[idx]
        pick = lambda a: None if a is None else np.ascontiguousarray(a[idx])
        layers = self.layers
        if layers is not None and layers.shape[0] != 1:
            layers = pick(layers)
        return Workload(self.name, len(idx), self.Lmax, self.S, self.M, pick(self.L),
                        pick(self.time_q), pick(self.mem_q), pick(self.trans_q),
                        layers, self.strat, pick(self.inst), dict(self.meta))


# --------------------------------------------------------------------------- random tables

def config0(seed: int = 0) -> Workload:
    """Tiny search: uniform time in [100,10000], mem in [1,24], trans in [0,2000], zero diagonal.

    Draw order: all time[l][s] (l-major), all mem[l][s], then trans row-major.  The workload is seed 0;
    other seeds give other instances of the same shape (further ranks of a multi-GPU run).
    """
    L, S, M = 4, 6, 64
    x = splitmix64(seed, 2 * L * S + S * S)
    time = _randint(x[:L * S], 100, 10000).reshape(1, L, S)
    mem = _randint(x[L * S:2 * L * S], 1, 24).reshape(1, L, S)
    trans = _randint(x[2 * L * S:], 0, 2000).reshape(1, S, S)
    trans[0][np.arange(S), np.arange(S)] = 0
    return Workload("config0_tiny", 1, L, S, M, np.full(1, L, np.int32), time, mem, trans)


def config4(B: int = 1024, seed: int = 7) -> Workload:
    """Re-search stress: log-normal time (mu = ln 5e5 ns, sigma = 0.5), mem in [8,128], dense trans in [0,5e4].

    Instance-major stream; per instance: time (two draws per value, Box-Muller
    cosine branch), then mem, then trans (diagonal kept as drawn).
    """
    L, S, M = 48, 32, 2048
    per = 2 * L * S + L * S + S * S
    x = splitmix64(seed, B * per).reshape(B, per)
    xt = x[:, :2 * L * S].reshape(B, L * S, 2)
    u1 = ((xt[..., 0] >> np.uint64(11)).astype(np.float64) + 1.0) * 2.0 ** -53
    u2 = _unit(xt[..., 1])
    z = np.sqrt(-2.0 * np.log(u1)) * np.cos(2.0 * np.pi * u2)
    time = np.maximum(1.0, np.rint(np.exp(np.log(5e5) + 0.5 * z))).astype(np.int32).reshape(B, L, S)
    mem = _randint(x[:, 2 * L * S:3 * L * S], 8, 128).reshape(B, L, S)
    trans = _randint(x[:, 3 * L * S:], 0, 50000).reshape(B, S, S)
    return Workload("config4_research_sweep", B, L, S, M, np.full(B, L, np.int32),
                    np.ascontiguousarray(time), np.ascontiguousarray(mem), np.ascontiguousarray(trans))


def random_tables(seed: int, B: int, Lmax: int, S: int, M: int, *, ragged: bool = False,
                  time_hi: int = 10000, mem_lo: int = 0, mem_hi: Optional[int] = None,
                  trans_hi: int = 2000, zero_diag: bool = False, dup_cols: bool = False) -> Workload:
    """Random integer tables for tests.  `dup_cols` copies strategy 0 into strategy S-1 to force ties."""
    mem_hi = max(1, M // 3) if mem_hi is None else mem_hi
    n = B * Lmax * S
    x = splitmix64(seed, 2 * n + B * S * S + B)
    time = _randint(x[:n], 1, time_hi).reshape(B, Lmax, S)
    mem = _randint(x[n:2 * n], mem_lo, mem_hi).reshape(B, Lmax, S)
    trans = _randint(x[2 * n:2 * n + B * S * S], 0, trans_hi).reshape(B, S, S)
    if zero_diag:
        trans[:, np.arange(S), np.arange(S)] = 0
    if dup_cols and S > 1:
        time[:, :, S - 1] = time[:, :, 0]
        mem[:, :, S - 1] = mem[:, :, 0]
        trans[:, S - 1, :] = trans[:, 0, :]
        trans[:, :, S - 1] = trans[:, :, 0]
    L = _randint(x[2 * n + B * S * S:], 1, Lmax) if ragged else np.full(B, Lmax, np.int32)
    return Workload(f"random_seed{seed}", B, Lmax, S, M, L.astype(np.int32), time, mem, trans)


# --------------------------------------------------------------------------- analytic workloads

# (c_lin, c_attn, p_coef, n_ar, act_rep, act_tp, act_attn) per layer kind
_KIND = {
    "full": (24.0, 4.0, 12.0, 4.0, 10.0, 24.0, 5.0),
    "attention": (8.0, 4.0, 4.0, 2.0, 5.0, 8.0, 5.0),
    "ffn": (16.0, 0.0, 8.0, 2.0, 5.0, 16.0, 0.0),
}


def layer_desc(kind: str, h: float, seq: float, heads: float) -> np.void:
    r = np.zeros((), LAYER_DESC)
    r["h"], r["seq"], r["heads"] = h, seq, heads
    for k, v in zip(("c_lin", "c_attn", "p_coef", "n_ar", "act_rep", "act_tp", "act_attn"), _KIND[kind]):
        r[k] = v
    return r


def strategy_table(tps, zeros, ckpts=(0, 1), sps=(0,), gpus_per_stage: int = 8) -> np.ndarray:
    """Strategy index order: tp-major, then ZeRO stage, then checkpointing, sequence parallelism innermost."""
    rows = []
    for tp in tps:
        for z in zeros:
            for c in ckpts:
                for sp in sps:
                    rows.append((tp, gpus_per_stage // tp, z, c, sp, 0, 1.0))
    return np.array(rows, dtype=STRATEGY_DESC)


def _inst(B: int, **kw) -> np.ndarray:
    a = np.zeros(B, INST_PARAMS)
    base = dict(b=1.0, act_mult=1.0, flops_rate=1e15, bw_tp=450e9, bw_dp=450e9,
                bytes_per_elem=2.0, bin_bytes=64.0 * 2 ** 20, time_unit_ns=1.0)
    base.update(kw)
    for k, v in base.items():
        a[k] = v
    return a


def config1() -> Workload:
    """GPT-style decoder, 24 uniform layers, h=2048, seq=2048; micro-batch 1..16; 24 strategies."""
    B, L, M = 16, 24, 2880
    layers = np.empty((1, L), LAYER_DESC)
    layers[:] = layer_desc("full", 2048.0, 2048.0, 16.0)
    strat = strategy_table((1, 2, 4, 8), (0, 2, 3))
    inst = _inst(B, b=np.arange(1, B + 1, dtype=np.float64))
    return Workload("config1_gpt_uniform", B, L, len(strat), M, np.full(B, L, np.int32),
                    layers=layers, strat=strat, inst=inst)


def config2(full_product: bool = False) -> Workload:
    """175B-shaped decoder; one pipeline stage per instance: L = ceil(96/pp), in-flight activations x pp.

    Instance i = (b-1)*8 + pp_idx with pp over (1,2,4,8,16,32,64,96).  The stated
    S=48 keeps ZeRO stages {0,2,3}; `full_product` gives the 64-strategy variant.
    """
    pps = (1, 2, 4, 8, 16, 32, 64, 96)
    B, Lmax, M = 64, 96, 2880
    layers = np.empty((1, Lmax), LAYER_DESC)
    layers[:] = layer_desc("full", 12288.0, 2048.0, 96.0)
    strat = strategy_table((1, 2, 4, 8), (0, 1, 2, 3) if full_product else (0, 2, 3), (0, 1), (0, 1))
    b = np.repeat(np.arange(1, 9, dtype=np.float64), 8)
    pp = np.tile(np.array(pps, dtype=np.float64), 8)
    L = np.array([-(-96 // p) for p in pps] * 8, dtype=np.int32)
    inst = _inst(B, b=b, act_mult=pp, time_unit_ns=100.0)
    return Workload("config2_175b" + ("_full" if full_product else ""), B, Lmax, len(strat), M, L,
                    layers=layers, strat=strat, inst=inst, meta={"pp": pp, "b": b})


def config3(B: int = 128) -> Workload:
    """Alternating attention / FFN stack (h=8192, seq=4096, 64 heads), 64 strategies, 16 MiB bins.

    Per instance two jitter draws (splitmix64 seed 3) scale the compute rate and
    the link bandwidth by a factor in [0.8, 1.2).
    """
    L, M = 160, 8192
    layers = np.empty((1, L), LAYER_DESC)
    layers[0, 0::2] = layer_desc("attention", 8192.0, 4096.0, 64.0)
    layers[0, 1::2] = layer_desc("ffn", 8192.0, 4096.0, 64.0)
    strat = strategy_table((1, 2, 4, 8), (0, 1, 2, 3), (0, 1), (0, 1))
    u = _unit(splitmix64(3, 2 * B)).reshape(B, 2)
    bw = 450e9 * (0.8 + 0.4 * u[:, 1])
    inst = _inst(B, flops_rate=1e15 * (0.8 + 0.4 * u[:, 0]), bw_tp=bw, bw_dp=bw,
                 bin_bytes=16.0 * 2 ** 20, time_unit_ns=10.0)
    return Workload("config3_heterogeneous", B, L, len(strat), M, np.full(B, L, np.int32),
                    layers=layers, strat=strat, inst=inst)


CONFIGS = {0: config0, 1: config1, 2: config2, 3: config3, 4: config4}


def fnv1a64(a: np.ndarray) -> int:
    """FNV-1a 64-bit checksum of the first 64 KiB of an array's bytes (input fingerprint printed by the bench)."""
    h = 0xCBF29CE484222325
    for byte in np.ascontiguousarray(a).view(np.uint8).ravel()[: 1 << 16].tolist():
        h = ((h ^ byte) * 0x100000001B3) & 0xFFFFFFFFFFFFFFFF
    return h

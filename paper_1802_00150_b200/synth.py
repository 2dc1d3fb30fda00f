"""Seeded synthetic inputs shaped like the paper's language-model layers.

This module serves both the CUDA tests/benchmark and the CPU oracle's tests.  It holds no arithmetic
of the quantization method: only a counter-based random generator (splitmix64 finaliser over a
counter, so values do not depend on any library's RNG) and the table of workload shapes.

Values are drawn in float64, then rounded once to float32: every consumer sees the same float32 bits.
"""
from dataclasses import dataclass

import numpy as np

_GAMMA = np.uint64(0x9E3779B97F4A7C15)
_M1 = np.uint64(0xBF58476D1CE4E5B9)
_M2 = np.uint64(0x94D049BB133111EB)


def _mix(z):
    z = (z ^ (z >> np.uint64(30))) * _M1
    z = (z ^ (z >> np.uint64(27))) * _M2
    return z ^ (z >> np.uint64(31))


def _stream_base(seed, stream):
    with np.errstate(over="ignore"):
        s = np.uint64(seed & 0xFFFFFFFFFFFFFFFF) + _GAMMA * np.uint64((stream + 1) & 0xFFFFFFFFFFFFFFFF)
        return _mix(np.array([s], dtype=np.uint64))[0]


def uniform01(count, seed=0, stream=0):
    """`count` doubles in [0, 1): value i of (seed, stream) is a pure function of (seed, stream, i)."""
    with np.errstate(over="ignore"):
        base = _stream_base(seed, stream)
        idx = np.arange(1, count + 1, dtype=np.uint64)
        z = _mix(base + idx * _GAMMA)
    return (z >> np.uint64(11)).astype(np.float64) * (1.0 / 9007199254740992.0)


def uniform(shape, lo=-1.0, hi=1.0, seed=0, stream=0):
    count = int(np.prod(shape))
    u = uniform01(count, seed, stream)
    return (lo + (hi - lo) * u).astype(np.float32).reshape(shape)


def normal(shape, std=1.0, seed=0, stream=0, clip=None):
    """Box-Muller on pairs of uniforms; optional symmetric clip."""
    count = int(np.prod(shape))
    pairs = (count + 1) // 2
    u = uniform01(2 * pairs, seed, stream)
    u1 = 1.0 - u[0::2]          # (0, 1]
    u2 = u[1::2]
    rad = np.sqrt(-2.0 * np.log(u1))
    g = np.empty(2 * pairs)
    g[0::2] = rad * np.cos(2.0 * np.pi * u2)
    g[1::2] = rad * np.sin(2.0 * np.pi * u2)
    g = g[:count] * std
    if clip is not None:
        g = np.clip(g, -clip, clip)
    return g.astype(np.float32).reshape(shape)


@dataclass(frozen=True)
class Workload:
    """One synthetic workload.  cell: 'lstm', 'gru' or 'proj' (bulk quantization + one product)."""
    name: str
    cell: str
    I: int
    H: int
    m: int          # rows of the stacked weight matrix
    n: int          # columns (I + H for a cell, H for the projection)
    k_w: int
    k_a: int
    T: int
    batch: int
    steps: int
    w_std: float
    x_dist: str     # 'uniform' (U(-1,1)), 'normal' (N(0,1)) or 'normal_clip3'
    seed: int = 0


WORKLOADS = {
    # single LSTM cell step, hidden 300 (the paper's PTB size), batch 1
    "lstm300_step": Workload("lstm300_step", "lstm", 300, 300, 1200, 600, 2, 2, 2, 1, 1, 0.05, "uniform"),
    # LSTM layer, hidden 1024 (the paper's Text8 size), batch 1, 35 steps
    "lstm1024_b1": Workload("lstm1024_b1", "lstm", 1024, 1024, 4096, 2048, 2, 2, 2, 1, 35, 0.03, "normal_clip3"),
    # same layer, 3/3 bits, 64 concurrent sequences
    "lstm1024_b64": Workload("lstm1024_b64", "lstm", 1024, 1024, 4096, 2048, 3, 3, 2, 64, 35, 0.03, "normal"),
    # GRU layer, hidden 2048, 2/3 bits, 256 concurrent sequences
    "gru2048_b256": Workload("gru2048_b256", "gru", 2048, 2048, 6144, 4096, 2, 3, 2, 256, 35, 0.02, "normal"),
    # output projection 32768 x 1024: bulk row-wise quantization, then one product with 512 activations
    "proj32768_b512": Workload("proj32768_b512", "proj", 0, 1024, 32768, 1024, 3, 2, 2, 512, 1, 0.02, "uniform"),
}


def _draw_x(shape, dist, seed, stream):
    if dist == "uniform":
        return uniform(shape, -1.0, 1.0, seed, stream)
    if dist == "normal":
        return normal(shape, 1.0, seed, stream)
    if dist == "normal_clip3":
        return normal(shape, 1.0, seed, stream, clip=3.0)
    raise ValueError(dist)


def weights(wl: Workload, rows=None):
    """fp32 weight matrix (m, n) ~ N(0, w_std^2); `rows` limits to the first rows (same values)."""
    m = wl.m if rows is None else rows
    return normal((m, wl.n), wl.w_std, wl.seed, stream=1)


def inputs(wl: Workload):
    """Activations.  Cells: x_seq (steps, batch, I); the step workload also returns a nonzero
    h ~ U(-1,1) and c ~ U(-1,1).  Projection: acts (batch, n)."""
    if wl.cell == "proj":
        return {"acts": _draw_x((wl.batch, wl.n), wl.x_dist, wl.seed, 2)}
    out = {"x_seq": _draw_x((wl.steps, wl.batch, wl.I), wl.x_dist, wl.seed, 2)}
    if wl.steps == 1:
        out["h0"] = uniform((wl.batch, wl.H), -1.0, 1.0, wl.seed, 3)
        out["c0"] = uniform((wl.batch, wl.H), -1.0, 1.0, wl.seed, 4)
    else:
        out["h0"] = np.zeros((wl.batch, wl.H), dtype=np.float32)
        out["c0"] = np.zeros((wl.batch, wl.H), dtype=np.float32)
    return out


def scaled(wl: Workload, **kw):
    """A smaller or altered copy of a workload (same distributions), for parity tests."""
    d = dict(wl.__dict__)
    d.update(kw)
    if d["cell"] in ("lstm", "gru"):
        d["n"] = d["I"] + d["H"]
        d["m"] = (4 if d["cell"] == "lstm" else 3) * d["H"]
    return Workload(**d)

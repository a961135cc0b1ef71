"""Seeded synthetic inputs for the MoE "expert + return" path.

This module only draws random numbers, converts between float32 and bf16 bit
patterns, and plays the part of the stages that run *before* the path under
test (router and first all-to-all, Section 2.1 steps 1-2).  It contains none of
the method's arithmetic: no expert FFN, no row layout, no return slots, no
combine.  Both the CPU oracle's tests and the CUDA path's tests draw their
inputs here, which is the only thing the two sides share.

The paper's workloads are themselves synthetic (Table 2 shapes under three
router modes that are never defined quantitatively), so nothing here stands in
for a dataset.  Recipe:

* tokens ``x[R, T, d] ~ N(0, 1)`` rounded to bf16;
* expert weights ``W1[El, 2F, d]`` (rows ``0..F-1`` gate projection, rows
  ``F..2F-1`` up projection) and ``W2[El, d, F]``, both ``~ N(0, 1/d)``, bf16
  (single-projection shapes: one ``W[El, N, d] ~ N(0, 1/d)`` per expert);
* router logits ``l[R, T, Eg] ~ N(0, 1)``;
* ``uniform`` router: experts = top-k of the logits, gate = softmax of the k
  selected logits (fp32);
* ``zipf`` router: expert popularity ``p_e ~ (e+1)^-1.2``; experts = top-k of
  ``log p_e + Gumbel`` (sampling without replacement); gates as above;
* ``zipf_rot``: as ``zipf`` with the popularity vector rotated by ``r * El``
  for source rank ``r`` (uneven per-source-rank counts).
"""
from __future__ import annotations

from dataclasses import dataclass, replace
from typing import Dict, Optional

import numpy as np


@dataclass(frozen=True)
class MoEShape:
    """One workload.  Notation follows Algorithm 1: R ranks, E local experts."""

    name: str
    R: int            # simulated source ranks
    T: int            # tokens per source rank
    Eg: int           # global experts
    k: int            # top-k
    El: int           # local experts held by this GPU (global ids first_local..+El-1)
    d: int            # model dim
    F: int            # ffn dim
    router: str = "uniform"   # uniform | zipf | zipf_rot
    seed: int = 0
    self_rank: int = 0
    first_local: int = 0      # global id of local expert 0
    zipf_s: float = 1.2
    N_out: int = 0            # > 0: each expert is one projection y = x W^T, W[N_out, d] (the paper's operator); F unused

    @property
    def dout(self) -> int:
        return self.N_out if self.N_out > 0 else self.d

    @property
    def kmax(self) -> int:
        return min(self.k, self.El)


SHAPES: Dict[str, MoEShape] = {
    # BASELINE configs, list order
    "tiny": MoEShape("tiny", R=4, T=256, Eg=8, k=2, El=2, d=256, F=512),
    "mixtral": MoEShape("mixtral", R=4, T=4096, Eg=8, k=2, El=2, d=4096, F=14336),
    "mixtral_zipf": MoEShape("mixtral_zipf", R=4, T=4096, Eg=8, k=2, El=2, d=4096, F=14336, router="zipf"),
    "tiny_zipf": MoEShape("tiny_zipf", R=4, T=256, Eg=8, k=2, El=2, d=256, F=512, router="zipf"),
    "fine": MoEShape("fine", R=8, T=8192, Eg=64, k=6, El=8, d=2048, F=1408),
    # a quarter of the Mixtral-shaped layer's tokens, same weights: small enough for a full profiler capture
    "mixtral_quarter": MoEShape("mixtral_quarter", R=4, T=1024, Eg=8, k=2, El=2, d=4096, F=14336),
    # the operator the paper evaluates (Table 2): one projection per expert, M = 2 x tokens-per-rank rows,
    # K = 2048, N = 8192, E experts per rank, 4 ranks, top-2
    "paper_op_e4": MoEShape("paper_op_e4", R=4, T=8192, Eg=16, k=2, El=4, d=2048, F=0, N_out=8192),
    "paper_op_e16": MoEShape("paper_op_e16", R=4, T=8192, Eg=64, k=2, El=16, d=2048, F=0, N_out=8192),
    "paper_op_e16_zipf": MoEShape("paper_op_e16_zipf", R=4, T=8192, Eg=64, k=2, El=16, d=2048, F=0, N_out=8192,
                                  router="zipf"),
    # many (expert, rank) groups with few rows each: 512 groups, almost every band partial
    "many_groups": MoEShape("many_groups", R=16, T=300, Eg=64, k=4, El=32, d=256, F=128, self_rank=5, seed=4),
    # the same with a hidden width the swapped-operand items accept (every run is a run of small bands), and a
    # decode-sized batch: a handful of rows per (expert, rank) group
    "many_small_groups": MoEShape("many_small_groups", R=16, T=300, Eg=64, k=4, El=32, d=256, F=256, self_rank=5, seed=4),
    "decode": MoEShape("decode", R=4, T=64, Eg=16, k=2, El=4, d=512, F=768, self_rank=1, seed=6),
    "decode_single": MoEShape("decode_single", R=4, T=96, Eg=24, k=2, El=6, d=320, F=0, N_out=768, self_rank=3, seed=8),
    "single_small": MoEShape("single_small", R=3, T=600, Eg=6, k=2, El=2, d=192, F=0, N_out=512, self_rank=2, seed=2),
    # mid-size shapes for parity tests (several bands per group, ragged tails)
    "small": MoEShape("small", R=3, T=700, Eg=6, k=2, El=3, d=512, F=384, self_rank=1),
    "small_zipf_rot": MoEShape("small_zipf_rot", R=4, T=900, Eg=8, k=3, El=2, d=256, F=640,
                               router="zipf_rot", self_rank=2, seed=3),
}


def sweep_shape(n: int, F: int, router: str = "uniform", seed: int = 0) -> MoEShape:
    """A point of the sweep grid: 4 local experts of 16, 4 ranks, d=4096, about n tokens per local expert."""
    return MoEShape(f"sweep_n{n}_F{F}_{router}", R=4, T=2 * n, Eg=16, k=2, El=4, d=4096, F=F,
                    router=router, seed=seed)


# ----------------------------------------------------------------------------- bf16 bit patterns

def f32_to_bf16_bits(a: np.ndarray) -> np.ndarray:
    """float32 -> bf16 bit pattern (uint16), round to nearest even.  Inputs are finite."""
    u = np.ascontiguousarray(a, dtype=np.float32).view(np.uint32)
    bias = ((u >> np.uint32(16)) & np.uint32(1)) + np.uint32(0x7FFF)
    return ((u + bias) >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


# ----------------------------------------------------------------------------- generators

@dataclass
class MoEInputs:
    shape: MoEShape
    x: np.ndarray        # [R, T, d] uint16 (bf16 bits)
    w1: np.ndarray       # [El, 2F, d] uint16
    w2: np.ndarray       # [El, d, F] uint16
    expert: np.ndarray   # [R, T, k] int32, global expert ids, in router order
    gate: np.ndarray     # [R, T, k] float32


def _normal_bf16(rng: np.random.Generator, shape, scale: float) -> np.ndarray:
    out = np.empty(shape, dtype=np.uint16)
    flat = out.reshape(-1)
    step = 1 << 24
    for lo in range(0, flat.size, step):
        hi = min(flat.size, lo + step)
        v = rng.standard_normal(hi - lo, dtype=np.float32)
        if scale != 1.0:
            v *= np.float32(scale)
        flat[lo:hi] = f32_to_bf16_bits(v)
    return out


def make_router(shape: MoEShape, rng: np.random.Generator):
    R, T, Eg, k = shape.R, shape.T, shape.Eg, shape.k
    logits = rng.standard_normal((R, T, Eg), dtype=np.float32)
    if shape.router == "uniform":
        score = logits
    elif shape.router in ("zipf", "zipf_rot"):
        p = (np.arange(Eg, dtype=np.float64) + 1.0) ** (-shape.zipf_s)
        p /= p.sum()
        logp = np.log(p)
        gumbel = -np.log(-np.log(rng.random((R, T, Eg))))
        if shape.router == "zipf_rot":
            lp = np.stack([np.roll(logp, r * shape.El) for r in range(R)])[:, None, :]
        else:
            lp = logp[None, None, :]
        score = lp + gumbel
    else:
        raise ValueError(f"unknown router {shape.router!r}")
    order = np.argsort(-score, axis=-1, kind="stable")[..., :k]
    expert = order.astype(np.int32)
    sel = np.take_along_axis(logits, order, axis=-1).astype(np.float32)
    sel = sel - sel.max(axis=-1, keepdims=True)
    e = np.exp(sel, dtype=np.float32)
    gate = (e / e.sum(axis=-1, keepdims=True, dtype=np.float32)).astype(np.float32)
    return expert, gate


def make_inputs(shape: MoEShape, weights: bool = True) -> MoEInputs:
    rng = np.random.Generator(np.random.PCG64(shape.seed))
    x = _normal_bf16(rng, (shape.R, shape.T, shape.d), 1.0)
    expert, gate = make_router(shape, rng)
    if weights and shape.N_out > 0:
        w1 = _normal_bf16(rng, (shape.El, shape.N_out, shape.d), float(shape.d) ** -0.5)
        w2 = np.zeros((0,), np.uint16)
    elif weights:
        s = float(shape.d) ** -0.5
        w1 = _normal_bf16(rng, (shape.El, 2 * shape.F, shape.d), s)
        w2 = _normal_bf16(rng, (shape.El, shape.d, shape.F), s)
    else:
        w1 = np.zeros((0,), np.uint16)
        w2 = np.zeros((0,), np.uint16)
    return MoEInputs(shape, x, w1, w2, expert, gate)


# ----------------------------------------------------------------------------- first all-to-all stand-in

@dataclass
class Dispatched:
    """What the first all-to-all hands to this GPU: routed token copies grouped by local expert."""

    x_rows: np.ndarray         # [M, d] uint16
    expert_counts: np.ndarray  # [El] int32
    src_rank: np.ndarray       # [M] int32
    src_token: np.ndarray      # [M] int32
    gate: np.ndarray           # [M] float32
    row_expert: np.ndarray     # [M] int32 local expert of every row (redundant with expert_counts)

    @property
    def M(self) -> int:
        return int(self.src_rank.shape[0])


def dispatch(inp: MoEInputs, shuffle_seed: Optional[int] = None, gather_x: bool = True) -> Dispatched:
    """Gather the rows routed to this GPU's local experts.

    Rows of local expert ``e`` arrive in (src_rank, src_token) order, as an
    all-to-all would deliver them; ``shuffle_seed`` permutes the rows inside
    every expert instead, to check that nothing depends on the arrival order.
    """
    sh = inp.shape
    xs, rs, ts, gs, es, counts = [], [], [], [], [], []
    srng = None if shuffle_seed is None else np.random.Generator(np.random.PCG64(shuffle_seed))
    for e in range(sh.El):
        ge = sh.first_local + e
        hit = inp.expert == ge                      # [R, T, k]
        r, t = np.nonzero(hit.any(axis=-1))         # row-major => (rank, token) order
        j = hit[r, t].argmax(axis=-1)
        if srng is not None:
            perm = srng.permutation(r.shape[0])
            r, t, j = r[perm], t[perm], j[perm]
        rs.append(r.astype(np.int32))
        ts.append(t.astype(np.int32))
        gs.append(inp.gate[r, t, j].astype(np.float32))
        es.append(np.full(r.shape[0], e, np.int32))
        counts.append(r.shape[0])
        if gather_x:
            xs.append(inp.x[r, t])
    cat = lambda parts, dt: (np.concatenate(parts).astype(dt) if parts else np.zeros((0,), dt))
    x_rows = (np.concatenate(xs, axis=0) if gather_x and xs else np.zeros((0, sh.d), np.uint16))
    return Dispatched(np.ascontiguousarray(x_rows), np.asarray(counts, np.int32), cat(rs, np.int32),
                      cat(ts, np.int32), cat(gs, np.float32), cat(es, np.int32))


def with_seed(shape: MoEShape, seed: int) -> MoEShape:
    return replace(shape, seed=seed)

"""Pins for the value oracle: the definition evaluated another way (float64 NumPy,
library matmul/silu), exact special cases, and linearity in the gates."""
import numpy as np
import pytest
import torch

from oracle import value_oracle as VO
from paper_2607_19539_b200 import inputs as I


def rel_dist(a, b):
    """Per-row ||a-b|| / max(||b||, 1e-6 sqrt(d)); the paper's 'relative distance' (Section 4.4) per token."""
    a = a.astype(np.float64)
    b = b.astype(np.float64)
    den = np.maximum(np.linalg.norm(b, axis=-1), 1e-6 * np.sqrt(b.shape[-1]))
    return np.linalg.norm(a - b, axis=-1) / den


def brute_force_f64(inp, tokens):
    """Section 2.1 straight from the definition in float64, no intermediate rounding."""
    sh = inp.shape
    x = I.bf16_bits_to_f32(inp.x).astype(np.float64).reshape(sh.R * sh.T, sh.d)
    w1 = I.bf16_bits_to_f32(inp.w1).astype(np.float64)
    w2 = I.bf16_bits_to_f32(inp.w2).astype(np.float64)
    ex = inp.expert.reshape(sh.R * sh.T, sh.k)
    gt = inp.gate.reshape(sh.R * sh.T, sh.k).astype(np.float64)
    out = np.zeros((len(tokens), sh.d))
    ys = {}
    for s, tok in enumerate(tokens):
        for q in range(sh.k):
            e = ex[tok, q] - sh.first_local
            if 0 <= e < sh.El:
                gq = w1[e, :sh.F] @ x[tok]
                up = w1[e, sh.F:] @ x[tok]
                h = gq / (1.0 + np.exp(-gq)) * up
                y = w2[e] @ h
                ys[(s, int(e))] = y
                out[s] += gt[tok, q] * y
    return out, ys


@pytest.mark.parametrize("shape", [
    I.MoEShape("bf_a", R=2, T=5, Eg=4, k=2, El=2, d=8, F=16),
    I.MoEShape("bf_b", R=3, T=7, Eg=4, k=3, El=3, d=16, F=24, first_local=1, seed=4),
    I.MoEShape("bf_c", R=2, T=24, Eg=8, k=2, El=2, d=256, F=512, seed=1),
])
def test_against_float64_definition(shape):
    inp = I.make_inputs(shape)
    toks = np.arange(shape.R * shape.T, dtype=np.int32)
    out, y, y_exp = VO.forward_tokens(inp.x, inp.expert, inp.gate, inp.w1, inp.w2, shape.El, shape.first_local, toks)
    ref, ys = brute_force_f64(inp, toks)
    got = I.bf16_bits_to_f32(out)
    has = np.linalg.norm(ref, axis=-1) > 0
    assert has.any()
    assert rel_dist(got[has], ref[has]).max() < 1e-2
    assert (out[~has] == 0).all()                       # no local expert -> +0 bit pattern
    # returned rows: ascending local expert, unscaled
    for s in range(len(toks)):
        loc = [int(e) for e in y_exp[s] if e >= 0]
        assert loc == sorted(loc) and set(loc) == {e for (ss, e) in ys if ss == s}
        for j, e in enumerate(loc):
            assert rel_dist(I.bf16_bits_to_f32(y[s, j])[None], ys[(s, e)][None])[0] < 1e-2
        assert (y[s, len(loc):] == 0).all()


def test_single_expert_against_library_ops():
    # El=1, R=1, k=1, gate=1  =>  out = (silu(x W1g^T) * (x W1u^T)) W2^T
    shape = I.MoEShape("lib", R=1, T=33, Eg=1, k=1, El=1, d=64, F=96, seed=2)
    inp = I.make_inputs(shape)
    inp.gate[:] = 1.0
    toks = np.arange(shape.T, dtype=np.int32)
    out, y, _ = VO.forward_tokens(inp.x, inp.expert, inp.gate, inp.w1, inp.w2, 1, 0, toks)
    x = torch.from_numpy(I.bf16_bits_to_f32(inp.x[0]))
    w1 = torch.from_numpy(I.bf16_bits_to_f32(inp.w1[0]))
    w2 = torch.from_numpy(I.bf16_bits_to_f32(inp.w2[0]))
    ref = (torch.nn.functional.silu(x @ w1[:96].T) * (x @ w1[96:].T)) @ w2.T
    assert rel_dist(I.bf16_bits_to_f32(out), ref.numpy()).max() < 1e-2
    assert (out == y[:, 0]).all()                        # unit gate: out is the returned row itself


def test_zero_gate_projection_gives_exact_zero():
    shape = I.MoEShape("z", R=2, T=9, Eg=2, k=2, El=2, d=32, F=48, seed=5)
    inp = I.make_inputs(shape)
    inp.w1[:, :shape.F, :] = 0                            # silu(0) = 0
    toks = np.arange(shape.R * shape.T, dtype=np.int32)
    out, y, _ = VO.forward_tokens(inp.x, inp.expert, inp.gate, inp.w1, inp.w2, 2, 0, toks)
    assert (out & 0x7FFF == 0).all() and (y & 0x7FFF == 0).all()


def identity_experts(shape):
    """F = d; W1 gate row j has 32 at the last feature, W1 up = I/32, W2 = I.  With the last feature of
    every token equal to 1: gq = 32, silu(32) = 32 exactly in fp32, h = x, y = x."""
    d = shape.d
    w1 = np.zeros((shape.El, 2 * d, d), np.float32)
    w1[:, :d, d - 1] = 32.0
    w1[:, d:, :] = np.eye(d, dtype=np.float32) / 32.0
    w2 = np.broadcast_to(np.eye(d, dtype=np.float32), (shape.El, d, d)).copy()
    return I.f32_to_bf16_bits(w1), I.f32_to_bf16_bits(w2)


def test_identity_experts_unit_gates_reproduce_x():
    shape = I.MoEShape("id", R=3, T=40, Eg=4, k=2, El=2, d=64, F=64, seed=7)
    inp = I.make_inputs(shape)
    inp.w1, inp.w2 = identity_experts(shape)
    inp.gate[:] = 1.0
    xf = I.bf16_bits_to_f32(inp.x)
    xf[..., -1] = 1.0
    inp.x = I.f32_to_bf16_bits(xf)
    toks = np.arange(shape.R * shape.T, dtype=np.int32)
    out, y, y_exp = VO.forward_tokens(inp.x, inp.expert, inp.gate, inp.w1, inp.w2, 2, 0, toks)
    m = (y_exp >= 0).sum(axis=1)
    assert set(m.tolist()) == {0, 1, 2}
    x_flat = inp.x.reshape(-1, shape.d)
    assert (out[m == 1] == x_flat[m == 1]).all()                         # reproduces x bit-exactly
    assert (out[m == 0] == 0).all()
    two = I.f32_to_bf16_bits(2.0 * I.bf16_bits_to_f32(x_flat[m == 2]))
    assert (out[m == 2] == two).all()                                    # m local experts -> m * x
    for j in range(2):
        rows = y_exp[:, j] >= 0
        assert (y[rows, j] == x_flat[rows]).all()                        # returned rows are x itself


def test_gate_scaling_is_exact_for_powers_of_two():
    shape = I.MoEShape("lin", R=2, T=16, Eg=4, k=2, El=4, d=32, F=64, seed=8)
    inp = I.make_inputs(shape)
    toks = np.arange(shape.R * shape.T, dtype=np.int32)
    out1, y1, _ = VO.forward_tokens(inp.x, inp.expert, inp.gate, inp.w1, inp.w2, 4, 0, toks)
    out2, y2, _ = VO.forward_tokens(inp.x, inp.expert, 2.0 * inp.gate, inp.w1, inp.w2, 4, 0, toks)
    assert (y1 == y2).all()                                              # returned rows carry no gate
    assert (I.bf16_bits_to_f32(out2) == 2.0 * I.bf16_bits_to_f32(out1)).all()
    # out is the gate-weighted sum of the returned rows (step 5), recomputed here in float64
    g = np.zeros((len(toks), 2))
    ex = inp.expert.reshape(-1, 2)
    for s in range(len(toks)):
        order = np.argsort(ex[s])
        g[s] = inp.gate.reshape(-1, 2)[s][order]
    ref = (g[:, :, None] * I.bf16_bits_to_f32(y1).astype(np.float64)).sum(axis=1)
    assert rel_dist(I.bf16_bits_to_f32(out1), ref).max() < 5e-3


def test_token_subset_and_threads_agree():
    shape = I.SHAPES["tiny"]
    inp = I.make_inputs(shape)
    sel = np.array([3, 77, 500, 1023, 4], np.int32)
    a = VO.forward_tokens(inp.x, inp.expert, inp.gate, inp.w1, inp.w2, shape.El, 0, sel, nthreads=1)
    b = VO.forward_tokens(inp.x, inp.expert, inp.gate, inp.w1, inp.w2, shape.El, 0, sel, nthreads=4)
    assert all((u == v).all() for u, v in zip(a, b))
    full = VO.forward_tokens(inp.x, inp.expert, inp.gate, inp.w1, inp.w2, shape.El, 0,
                             np.arange(shape.R * shape.T, dtype=np.int32))
    assert (full[0][sel] == a[0]).all()


# ---- single-projection experts (the operator of Table 2)

def test_single_projection_against_float64_and_library():
    shape = I.MoEShape("sp", R=2, T=19, Eg=4, k=2, El=3, d=48, F=0, N_out=80, first_local=1, seed=6)
    inp = I.make_inputs(shape)
    toks = np.arange(shape.R * shape.T, dtype=np.int32)
    out, y, y_exp = VO.forward_tokens_single(inp.x, inp.expert, inp.gate, inp.w1, shape.El, shape.first_local, toks)
    x = I.bf16_bits_to_f32(inp.x).astype(np.float64).reshape(-1, shape.d)
    w = I.bf16_bits_to_f32(inp.w1).astype(np.float64)
    ex = inp.expert.reshape(-1, shape.k)
    gt = inp.gate.reshape(-1, shape.k).astype(np.float64)
    ref = np.zeros((len(toks), shape.N_out))
    for s, tok in enumerate(toks):
        loc = []
        for q in range(shape.k):
            e = ex[tok, q] - shape.first_local
            if 0 <= e < shape.El:
                ref[s] += gt[tok, q] * (w[e] @ x[tok])
                loc.append(int(e))
        assert [int(v) for v in y_exp[s] if v >= 0] == sorted(loc)
        for j, e in enumerate(sorted(loc)):
            assert rel_dist(I.bf16_bits_to_f32(y[s, j])[None], (w[e] @ x[tok])[None])[0] < 1e-2
    has = np.linalg.norm(ref, axis=1) > 0
    assert rel_dist(I.bf16_bits_to_f32(out)[has], ref[has]).max() < 1e-2
    assert (out[~has] == 0).all()
    # one expert, unit gate: a library matmul
    sh1 = I.MoEShape("sp1", R=1, T=21, Eg=1, k=1, El=1, d=64, F=0, N_out=32, seed=9)
    in1 = I.make_inputs(sh1)
    in1.gate[:] = 1.0
    o1, y1, _ = VO.forward_tokens_single(in1.x, in1.expert, in1.gate, in1.w1, 1, 0, np.arange(21, dtype=np.int32))
    lib = torch.from_numpy(I.bf16_bits_to_f32(in1.x[0])) @ torch.from_numpy(I.bf16_bits_to_f32(in1.w1[0])).T
    assert rel_dist(I.bf16_bits_to_f32(o1), lib.numpy()).max() < 1e-2
    assert (o1 == y1[:, 0]).all()


def test_single_projection_identity_is_exact():
    shape = I.MoEShape("spi", R=2, T=30, Eg=2, k=1, El=2, d=64, F=0, N_out=64, seed=3)
    inp = I.make_inputs(shape)
    inp.w1 = I.f32_to_bf16_bits(np.broadcast_to(np.eye(64, dtype=np.float32), (2, 64, 64)).copy())
    inp.gate[:] = 1.0
    toks = np.arange(60, dtype=np.int32)
    out, y, _ = VO.forward_tokens_single(inp.x, inp.expert, inp.gate, inp.w1, 2, 0, toks)
    assert (out == inp.x.reshape(-1, 64)).all() and (y[:, 0] == inp.x.reshape(-1, 64)).all()

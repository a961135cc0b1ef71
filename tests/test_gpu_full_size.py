"""Parity at the benchmark's full sizes, in the launch configuration bench.py times: indices bit-exact in
full; values on a seeded sample of tokens the oracle can compute one by one; and properties that hold for
every row without a CPU FFN."""
import numpy as np
import pytest

from paper_2607_19539_b200 import inputs as I

from . import parity_util as U

pytestmark = pytest.mark.gpu


def sample_tokens(shape, dsp, plan, per_rank, seed=0):
    """Tokens for the oracle where evaluating every token would take minutes: per_rank tokens of every source
    rank that own at least one local row, the tokens owning the first and the last row of every (expert, rank)
    group, and one token per band of the aligned layout (a seeded row of it) -- so every band, hence both CTAs
    of every pair and, through the row's full width, every tile of both GEMMs has a checked row."""
    rng = np.random.Generator(np.random.PCG64(seed))
    tok = dsp.src_rank.astype(np.int64) * shape.T + dsp.src_token
    picks = []
    for r in range(shape.R):
        mine = np.unique(tok[dsp.src_rank == r])
        picks.append(rng.choice(mine, size=min(per_rank, mine.size), replace=False))
        for e in range(shape.El):
            g = tok[(dsp.src_rank == r) & (dsp.row_expert == e)]
            if g.size:
                picks.append(np.array([g.min(), g.max()]))
    row_at = np.full(plan.P, -1, np.int64)
    row_at[np.asarray(plan.pos)] = np.arange(dsp.M)
    for b in plan.bands:
        picks.append(np.array([tok[row_at[b.pos0 + int(rng.integers(0, b.valid))]]]))
    return np.unique(np.concatenate(picks)).astype(np.int32)


def all_tokens_with_rows(shape, dsp):
    return np.unique(dsp.src_rank.astype(np.int64) * shape.T + dsp.src_token).astype(np.int32)


@pytest.mark.parametrize("name,csm,per_rank", [
    # per_rank None: EVERY token that owns a local row goes through the oracle (the two headline shapes)
    ("mixtral", 8, None), ("fine", 8, None), ("mixtral_zipf", 8, 8), ("paper_op_e16_zipf", 14, 16),
    # points of the sweep grid: 4 local experts of 16, d=4096; (tokens per local expert, ffn, router)
    ((1024, 1024, "uniform"), 2, 16), ((128, 2816, "zipf"), 16, 8), ((4096, 1024, "zipf"), 32, 8),
    ((128, 14336, "uniform"), 8, 32),       # decode-sized batch: every run is a run of small groups
    ((16384, 14336, "uniform"), 4, 4),      # the largest point of the grid: 65893 rows, 6.5 GB of workspace
])
def test_full_size_parity(name, csm, per_rank):
    import torch
    from paper_2607_19539_b200 import binding as B, harness as Hn
    shape = I.SHAPES[name] if isinstance(name, str) else I.sweep_shape(*name)
    inp = I.make_inputs(shape)
    dsp = I.dispatch(inp)
    ctx = Hn.make_context(shape, max_rows=dsp.M)
    prob = Hn.upload(inp, dsp)
    Hn.run(ctx, prob, mode=B.MODE_OVERLAP, consumer_sm_count=csm)
    torch.cuda.synchronize()
    assert ctx.moe_ovl_query_status()[0] == 0
    plan = U.oracle_plan(shape, dsp)
    rep = ctx.moe_ovl_get_report()
    U.check_indices(shape, dsp, plan, ctx.moe_ovl_get_plan(), prob.slot_out.cpu().numpy(),
                    prob.rows_per_rank_out.cpu().numpy(), prob.segs_per_rank_out.cpu().numpy(), rep)
    out = Hn.device_to_bits(prob.out)
    ret = Hn.device_to_bits(prob.ret)
    # (1) tokens against the oracle, element by element: all of them, or a sample that covers every band
    toks = all_tokens_with_rows(shape, dsp) if per_rank is None else sample_tokens(shape, dsp, plan, per_rank)
    worst = [0.0] * 4
    for lo in range(0, len(toks), 4096):
        part = toks[lo:lo + 4096]
        o = U.oracle_values(inp, part)
        worst = [max(a, b) for a, b in zip(worst, U.check_values(shape, dsp, plan, part, *o, out, ret))]
    print(f"{name}: {len(toks)} tokens ({'all' if per_rank is None else 'sample'}), max rel dist out {worst[0]:.2e}, "
          f"returned rows {worst[1]:.2e}; max element error out {worst[2]:.2e}, returned rows {worst[3]:.2e}")
    # (1b) the aligned input the GEMM read: input rows at their positions, zeros in the padding
    U.check_aligned_input(shape, dsp, plan, ctx.moe_ovl_read_buffer(B.BUF_XA, 0, rep.padded_rows))
    # (2) every row: the receive buffer holds exactly the GEMM's output row
    Y = ctx.moe_ovl_read_buffer(B.BUF_Y, 0, rep.padded_rows)
    pos, slot = np.asarray(plan.pos), np.asarray(plan.slot)
    assert (ret[dsp.src_rank, slot] == Y[pos]).all()
    # (3) every token: out is the gate-weighted sum of its returned rows (recomputed here from the GPU's ret)
    acc = np.zeros((shape.R * shape.T, shape.dout), np.float32)
    tok = dsp.src_rank.astype(np.int64) * shape.T + dsp.src_token
    for e in range(shape.El):                                  # ascending expert = accumulation order
        rows = np.nonzero(dsp.row_expert == e)[0]
        acc[tok[rows]] += dsp.gate[rows, None] * I.bf16_bits_to_f32(ret[dsp.src_rank[rows], slot[rows]])
    touched = np.zeros(shape.R * shape.T, bool)
    touched[tok] = True
    assert (out[~touched] == 0).all()
    assert U.rel_dist(I.bf16_bits_to_f32(out[touched]), acc[touched]).max() < 5e-3
    # (4) the non-overlap baseline and the in-kernel return give the same bits
    for mode in (B.MODE_NON_OVERLAP, B.MODE_IN_KERNEL):
        prob2 = Hn.upload(inp, dsp, w1=prob.w1, w2=prob.w2)
        Hn.run(ctx, prob2, mode=mode)
        torch.cuda.synchronize()
        assert ctx.moe_ovl_query_status()[0] == 0
        assert torch.equal(prob2.out.view(torch.int16), prob.out.view(torch.int16))
        assert torch.equal(prob2.ret.view(torch.int16), prob.ret.view(torch.int16))
        del prob2

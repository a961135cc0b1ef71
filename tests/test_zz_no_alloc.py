"""The allocation-free entry point against the regular one.

moe_ovl_return_slots_static serves callers that cannot call cudaMalloc and have no workspace to pass --
their application has already claimed all device memory for its own pool, or they sit in a loop where
cudaMalloc's device-wide synchronisation is too expensive.  Its scratch is a fixed array inside the library,
shared by every call, so the interesting failure is state leaking from one call into the next: the test
makes calls back to back, on different problems, and wants the slots of moe_ovl_expert_return every time.
Collected last on purpose (file name), so that a failure here cannot hide one elsewhere."""
import numpy as np
import pytest

from paper_2607_19539_b200 import inputs as I

from .parity_util import oracle_plan

pytestmark = pytest.mark.gpu


def _reference_slots(shape, inp, dsp):
    import torch
    from paper_2607_19539_b200 import binding as B, harness as Hn
    ctx = Hn.make_context(shape, max_rows=dsp.M)
    prob = Hn.upload(inp, dsp)
    Hn.run(ctx, prob, mode=B.MODE_NON_OVERLAP)
    torch.cuda.synchronize()
    assert ctx.moe_ovl_query_status()[0] == 0
    return prob.slot_out[:dsp.M].clone(), prob.rows_per_rank_out.clone()


def test_static_scratch_entry_point_matches_workspace_entry_point():
    import torch
    from paper_2607_19539_b200 import binding as B
    cases = []
    for name, shuffle in (("small_zipf_rot", 4), ("tiny", None), ("small", 9)):
        shape = I.SHAPES[name]
        inp = I.make_inputs(shape)
        dsp = I.dispatch(inp, shuffle_seed=shuffle)
        cases.append((shape, dsp, _reference_slots(shape, inp, dsp)))
    dev = torch.device("cuda:0")
    # two rounds over three different problems: six calls in a row on the one shared array
    for _ in range(2):
        for shape, dsp, (want_slot, want_rows) in cases:
            counts = torch.from_numpy(dsp.expert_counts).to(dev)
            sr = torch.from_numpy(dsp.src_rank).to(dev)
            st = torch.from_numpy(dsp.src_token).to(dev)
            slot = torch.full((dsp.M,), -9, dtype=torch.int32, device=dev)
            rows = torch.full((shape.R,), -9, dtype=torch.int32, device=dev)
            B.moe_ovl_return_slots_static(device=0, num_src_ranks=shape.R, tokens_per_rank=shape.T,
                                          num_local_experts=shape.El, expert_counts=counts, src_rank=sr,
                                          src_token=st, slot_out=slot, rows_per_rank_out=rows)
            torch.cuda.synchronize()
            assert torch.equal(slot, want_slot)          # integer work: bit-exact
            assert torch.equal(rows, want_rows)
            # and against the CPU oracle's plan, which shares nothing with either entry point
            plan = oracle_plan(shape, dsp)
            assert slot.cpu().tolist() == plan.slot and rows.cpu().tolist() == plan.rows_per_rank


def test_static_scratch_entry_point_edge_cases():
    """No rows at all; no rows-per-rank output wanted; rows the metadata does not cover get slot -1."""
    import torch
    from paper_2607_19539_b200 import binding as B
    dev = torch.device("cuda:0")
    shape = I.SHAPES["tiny"]
    dsp = I.dispatch(I.make_inputs(shape, weights=False))
    common = dict(device=0, num_src_ranks=shape.R, tokens_per_rank=shape.T, num_local_experts=shape.El)
    i32 = lambda a: torch.from_numpy(np.ascontiguousarray(a, np.int32)).to(dev)
    # (a) M = 0
    rows = torch.full((shape.R,), -9, dtype=torch.int32, device=dev)
    empty = torch.zeros(0, dtype=torch.int32, device=dev)
    B.moe_ovl_return_slots_static(expert_counts=i32(np.zeros(shape.El)), src_rank=empty, src_token=empty,
                                  slot_out=empty, rows_per_rank_out=rows, **common)
    torch.cuda.synchronize()
    assert rows.tolist() == [0] * shape.R
    # (b) rows_per_rank_out = NULL, right after a call that left the array full of another problem's bits
    plan = oracle_plan(shape, dsp)
    slot = torch.full((dsp.M,), -9, dtype=torch.int32, device=dev)
    B.moe_ovl_return_slots_static(expert_counts=i32(dsp.expert_counts), src_rank=i32(dsp.src_rank),
                                  src_token=i32(dsp.src_token), slot_out=slot, rows_per_rank_out=None, **common)
    torch.cuda.synchronize()
    assert slot.cpu().tolist() == plan.slot
    # (c) one row with an out-of-range rank, and counts that cover one row fewer than passed: both get -1,
    #     every other row keeps the slot it has without them
    sr = dsp.src_rank.copy()
    sr[3] = shape.R
    counts = dsp.expert_counts.copy()
    counts[-1] -= 1
    keep = np.ones(dsp.M, bool)
    keep[3] = keep[-1] = False
    sub = I.Dispatched(dsp.x_rows[keep], np.bincount(dsp.row_expert[keep], minlength=shape.El).astype(np.int32),
                       dsp.src_rank[keep], dsp.src_token[keep], dsp.gate[keep], dsp.row_expert[keep])
    want = np.full(dsp.M, -1, np.int64)
    want[keep] = oracle_plan(shape, sub).slot
    B.moe_ovl_return_slots_static(expert_counts=i32(counts), src_rank=i32(sr), src_token=i32(dsp.src_token),
                                  slot_out=slot, rows_per_rank_out=rows, **common)
    torch.cuda.synchronize()
    assert slot.cpu().tolist() == want.tolist()


def test_static_scratch_limits_are_rejected():
    import torch
    from paper_2607_19539_b200 import binding as B
    dev = torch.device("cuda:0")
    z = torch.zeros(8, dtype=torch.int32, device=dev)
    big = dict(device=0, expert_counts=z, src_rank=z, src_token=z, slot_out=z)
    with pytest.raises(B.MoeOvlError) as e:      # 64 * 32 groups > 1024
        B.moe_ovl_return_slots_static(num_src_ranks=32, tokens_per_rank=64, num_local_experts=64, **big)
    assert e.value.code == B.ERR_UNSUPPORTED
    with pytest.raises(B.MoeOvlError) as e:      # 8 * 8 * ceil(40000 / 32) words > 65536
        B.moe_ovl_return_slots_static(num_src_ranks=8, tokens_per_rank=40000, num_local_experts=8, **big)
    assert e.value.code == B.ERR_UNSUPPORTED

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

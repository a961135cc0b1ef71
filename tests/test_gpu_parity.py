"""GPU parity: the CUDA path, called through the C ABI, against the CPU oracle on the same seeded inputs.
Indices bit-exact; values within 2e-2 max relative distance (bf16 output, fp32 accumulate)."""
import numpy as np
import pytest

from paper_2607_19539_b200 import inputs as I

from . import parity_util as U

pytestmark = pytest.mark.gpu


def _gpu():
    import torch
    from paper_2607_19539_b200 import binding as B, harness as Hn
    return torch, B, Hn


def _run_case(shape, mode, csm, shuffle=None, mgb=1, group_bands=0, inp=None, dsp=None, flags=0):
    torch, B, Hn = _gpu()
    inp = inp or I.make_inputs(shape)
    dsp = dsp or I.dispatch(inp, shuffle_seed=shuffle)
    ctx = Hn.make_context(shape, max_rows=max(dsp.M, 1), mid_seg_bands=mgb, group_bands=group_bands,
                          wait_timeout_us=2_000_000, flags=flags)
    prob = Hn.upload(inp, dsp)
    Hn.run(ctx, prob, mode=mode, consumer_sm_count=csm)
    torch.cuda.synchronize()
    code, detail = ctx.moe_ovl_query_status()
    assert code == 0, (code, hex(detail))
    return inp, dsp, ctx, prob


SMALL = ["tiny", "tiny_zipf", "small", "small_zipf_rot", "single_small", "many_groups", "many_small_groups", "decode",
         "decode_single"]


@pytest.mark.parametrize("name", SMALL)
@pytest.mark.parametrize("mode,csm", [(0, 2), (0, 8), (0, 32), (1, 0), (2, 0), (3, 0)])
def test_small_shapes_full_parity(name, mode, csm):
    torch, B, Hn = _gpu()
    shape = I.SHAPES[name]
    # the small shapes hold too few items for the plan to choose swapped-operand items by itself: every other
    # mode forces them onto all eligible runs
    inp, dsp, ctx, prob = _run_case(shape, mode, csm, shuffle=None if mode == 1 else 17,
                                    flags=B.FLAG_TEST_ALL_SMALL_GROUP_TILES if csm in (0, 8) else 0)
    plan = U.oracle_plan(shape, dsp)
    U.check_indices(shape, dsp, plan, ctx.moe_ovl_get_plan(), prob.slot_out.cpu().numpy(),
                    prob.rows_per_rank_out.cpu().numpy(), prob.segs_per_rank_out.cpu().numpy(),
                    ctx.moe_ovl_get_report())
    toks = np.arange(shape.R * shape.T)
    o_out, o_y, o_yexp = U.oracle_values(inp, toks)
    U.check_values(shape, dsp, plan, toks, o_out, o_y, o_yexp, Hn.device_to_bits(prob.out),
                   Hn.device_to_bits(prob.ret))
    U.check_aligned_input(shape, dsp, plan, ctx.moe_ovl_read_buffer(B.BUF_XA, 0, plan.P))
    # rows of ret beyond rows_per_rank are untouched (still the NaN fill of the harness)
    ret = prob.ret.float().cpu().numpy()
    for r in range(shape.R):
        assert not np.isnan(ret[r, :plan.rows_per_rank[r]]).any()
        assert np.isnan(ret[r, plan.rows_per_rank[r]:]).all()


@pytest.mark.parametrize("name,mgb,gb", [("small", 2, 0), ("small_zipf_rot", 3, 2), ("small_zipf_rot", 1, 1)])
def test_segment_and_group_knobs(name, mgb, gb):
    torch, B, Hn = _gpu()
    shape = I.SHAPES[name]
    inp, dsp, ctx, prob = _run_case(shape, 0, 4, mgb=mgb, group_bands=gb)
    plan = U.oracle_plan(shape, dsp, mgb=mgb)
    U.check_indices(shape, dsp, plan, ctx.moe_ovl_get_plan(), prob.slot_out.cpu().numpy(),
                    prob.rows_per_rank_out.cpu().numpy(), prob.segs_per_rank_out.cpu().numpy(),
                    ctx.moe_ovl_get_report())
    toks = np.arange(0, shape.R * shape.T, 7)
    o = U.oracle_values(inp, toks)
    U.check_values(shape, dsp, plan, toks, *o, Hn.device_to_bits(prob.out), Hn.device_to_bits(prob.ret))


@pytest.mark.parametrize("name", ["tiny", "small_zipf_rot", "decode"])
def test_overlap_equals_non_overlap_bitwise(name):
    """Both modes run the same GEMM code on the same tiles: any difference is a protocol bug, not rounding.
    Two different problems alternate on one context, so that before every overlapped run the internal buffers
    hold the OTHER problem's rows: a segment moved before its tiles were flagged would carry foreign values."""
    torch, B, Hn = _gpu()
    shape = I.SHAPES[name]
    probs = []
    ctx = None
    for seed in (shape.seed, shape.seed + 101):
        inp = I.make_inputs(I.with_seed(shape, seed))
        dsp = I.dispatch(inp)
        probs.append((inp, dsp))
    ctx = Hn.make_context(shape, max_rows=max(d.M for _, d in probs),
                          flags=B.FLAG_TEST_ALL_SMALL_GROUP_TILES | B.FLAG_TEST_ZERO_ROWS_EARLY)
    refs = []
    for inp, dsp in probs:
        base = Hn.upload(inp, dsp)
        Hn.run(ctx, base, mode=B.MODE_NON_OVERLAP)
        torch.cuda.synchronize()
        refs.append((base, base.out.clone(), base.ret.clone()))
    assert not torch.equal(refs[0][1].view(torch.int16), refs[1][1].view(torch.int16))
    for it in range(30):
        csm = (2, 4, 8, 16, 32, 0)[it % 6]                      # 0: the return moved inside the GEMM kernel
        inp, dsp = probs[it % 2]
        base, ref_out, ref_ret = refs[it % 2]
        prob = Hn.upload(inp, dsp, w1=base.w1, w2=base.w2)
        Hn.run(ctx, prob, mode=B.MODE_OVERLAP if csm else B.MODE_IN_KERNEL, consumer_sm_count=csm)
        torch.cuda.synchronize()
        assert ctx.moe_ovl_query_status()[0] == 0
        assert torch.equal(prob.out.view(torch.int16), ref_out.view(torch.int16))
        assert torch.equal(prob.ret.view(torch.int16), ref_ret.view(torch.int16))


@pytest.mark.parametrize("csm", [2, 8, 16])
def test_sm_partition_is_disjoint_and_overlap_is_reported(csm):
    """Section 3.3.3: the two persistent kernels run on disjoint SM sets, one CTA per SM, and together fill the GPU;
    the report's device timestamps give the share of the return that is hidden behind the GEMM (Section 4.2.2).
    (The consumer budget stays below the 25 segments of this problem: a consumer CTA that finds no segment left
    exits at once and frees its SM for a GEMM CTA that has not started yet, which is fine but not what is tested.)"""
    torch, B, Hn = _gpu()
    shape = I.SHAPES["small_zipf_rot"]
    inp, dsp, ctx, prob = _run_case(shape, B.MODE_OVERLAP, csm)
    rep = ctx.moe_ovl_get_report()
    prod, cons = ctx.moe_ovl_get_sm_map()
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    assert len(cons) == csm and len(prod) == sms - csm
    assert len(set(prod.tolist())) == len(prod) and len(set(cons.tolist())) == len(cons)     # one CTA per SM
    assert not set(prod.tolist()) & set(cons.tolist())                                        # disjoint partitions
    assert min(prod.min(), cons.min()) >= 0 and max(prod.max(), cons.max()) < sms
    assert 0.0 <= rep.us_first_flag <= rep.us_gemm_done and rep.us_return_done > rep.us_first_flag
    assert 0.0 <= rep.overlap_ratio <= 1.0
    assert rep.num_segments <= rep.return_units <= 8 * rep.num_segments
    assert 0 <= rep.segments_by_gemm_ctas <= rep.return_units


def test_automatic_consumer_budget():
    """consumer_sm_count = 0 lets the library size the consumer partition from the shape: small for wide FFNs
    (the return is cheap next to the GEMM), larger for narrow ones; results do not depend on it."""
    torch, B, Hn = _gpu()
    got = {}
    for name in ("tiny", "small"):
        shape = I.SHAPES[name]
        inp = I.make_inputs(shape)
        dsp = I.dispatch(inp)
        ctx = Hn.make_context(shape, max_rows=dsp.M)
        ref = Hn.upload(inp, dsp)
        Hn.run(ctx, ref, mode=B.MODE_NON_OVERLAP)
        prob = Hn.upload(inp, dsp, w1=ref.w1, w2=ref.w2)
        Hn.run(ctx, prob, mode=B.MODE_OVERLAP, consumer_sm_count=0)
        torch.cuda.synchronize()
        assert ctx.moe_ovl_query_status()[0] == 0
        assert torch.equal(prob.out.view(torch.int16), ref.out.view(torch.int16))
        got[name] = ctx.moe_ovl_get_report().consumer_ctas
        assert got[name] % 2 == 0 and 2 <= got[name] <= 16
    wide = Hn.make_context(I.SHAPES["mixtral"], max_rows=128)     # only the shape matters for the choice
    narrow = Hn.make_context(I.SHAPES["fine"], max_rows=128)
    for c, sh in ((wide, I.SHAPES["mixtral"]), (narrow, I.SHAPES["fine"])):
        z = I.Dispatched(np.zeros((0, sh.d), np.uint16), np.zeros(sh.El, np.int32), np.zeros(0, np.int32),
                         np.zeros(0, np.int32), np.zeros(0, np.float32), np.zeros(0, np.int32))
        inp0 = I.MoEInputs(sh, np.zeros((sh.R, sh.T, sh.d), np.uint16), np.zeros((sh.El, 2 * sh.F, sh.d), np.uint16),
                           np.zeros((sh.El, sh.d, sh.F), np.uint16), np.zeros((sh.R, sh.T, sh.k), np.int32),
                           np.zeros((sh.R, sh.T, sh.k), np.float32))
        p0 = Hn.upload(inp0, z)
        Hn.run(c, p0, mode=B.MODE_OVERLAP, consumer_sm_count=0)
        torch.cuda.synchronize()
    assert wide.moe_ovl_get_report().consumer_ctas == 2 and narrow.moe_ovl_get_report().consumer_ctas == 8


def test_bounded_wait_gives_up_cleanly():
    """A flag that nothing sets: the consumer's wait runs out after the configured bound, the call ends with a
    timeout status (no hang, no fault), and the device stays usable."""
    torch, B, Hn = _gpu()
    shape = I.SHAPES["tiny"]
    inp = I.make_inputs(shape)
    dsp = I.dispatch(inp)
    ctx = Hn.make_context(shape, max_rows=dsp.M, wait_timeout_us=20_000, flags=B.FLAG_TEST_NO_FLAGS)
    prob = Hn.upload(inp, dsp)
    Hn.run(ctx, prob, mode=B.MODE_OVERLAP, consumer_sm_count=4)
    torch.cuda.synchronize()
    code, detail = ctx.moe_ovl_query_status()
    assert code == B.ERR_TIMEOUT
    assert detail >> 48 == 6                      # the wait that gave up: a consumer polling a tile flag
    # the same context in non-overlap mode (no flags involved), and a fresh context, still work
    Hn.run(ctx, prob, mode=B.MODE_NON_OVERLAP)
    torch.cuda.synchronize()
    assert ctx.moe_ovl_query_status()[0] == 0
    ok = Hn.make_context(shape, max_rows=dsp.M)
    prob2 = Hn.upload(inp, dsp, w1=prob.w1, w2=prob.w2)
    Hn.run(ok, prob2, mode=B.MODE_OVERLAP, consumer_sm_count=4)
    torch.cuda.synchronize()
    assert ok.moe_ovl_query_status()[0] == 0
    assert torch.equal(prob2.out.view(torch.int16), prob.out.view(torch.int16))


def test_identity_experts_reproduce_x_bit_exactly():
    torch, B, Hn = _gpu()
    shape = I.MoEShape("id", R=3, T=300, Eg=4, k=2, El=2, d=256, F=256, seed=7, self_rank=1)
    inp = I.make_inputs(shape)
    d = shape.d
    w1 = np.zeros((shape.El, 2 * d, d), np.float32)
    w1[:, :d, d - 1] = 32.0                                  # gate pre-activation = 32: silu(32) = 32 in fp32
    w1[:, d:, :] = np.eye(d, dtype=np.float32) / 32.0
    inp.w1 = I.f32_to_bf16_bits(w1)
    inp.w2 = I.f32_to_bf16_bits(np.broadcast_to(np.eye(d, dtype=np.float32), (shape.El, d, d)).copy())
    inp.gate[:] = 1.0
    xf = I.bf16_bits_to_f32(inp.x)
    xf[..., -1] = 1.0
    inp.x = I.f32_to_bf16_bits(xf)
    inp, dsp, ctx, prob = _run_case(shape, 0, 8, inp=inp)
    out = Hn.device_to_bits(prob.out)
    m = np.zeros(shape.R * shape.T, int)
    np.add.at(m, dsp.src_rank * shape.T + dsp.src_token, 1)
    x_flat = inp.x.reshape(-1, d)
    assert set(m.tolist()) == {0, 1, 2}
    assert (out[m == 1] == x_flat[m == 1]).all()
    assert (out[m == 0] == 0).all()
    assert (out[m == 2] == I.f32_to_bf16_bits(2.0 * I.bf16_bits_to_f32(x_flat[m == 2]))).all()
    # the receive buffers hold the dispatched rows themselves, in (expert, source-token) order
    ret = Hn.device_to_bits(prob.ret)
    slot = prob.slot_out.cpu().numpy()
    assert (ret[dsp.src_rank, slot[:dsp.M]] == dsp.x_rows).all()


def test_edge_cases_empty_and_degenerate():
    torch, B, Hn = _gpu()
    shape = I.MoEShape("edge", R=2, T=64, Eg=4, k=2, El=3, d=256, F=128, seed=3)
    inp = I.make_inputs(shape)
    # (a) no rows at all: out is all +0, nothing else written
    dsp = I.dispatch(inp)
    empty = I.Dispatched(dsp.x_rows[:0], np.zeros(3, np.int32), dsp.src_rank[:0], dsp.src_token[:0], dsp.gate[:0],
                         dsp.row_expert[:0])
    for mode in (0, 1):
        _, _, ctx, prob = _run_case(shape, mode, 2, inp=inp, dsp=empty)
        assert (Hn.device_to_bits(prob.out) == 0).all()
        assert prob.rows_per_rank_out.tolist() == [0, 0] and prob.segs_per_rank_out.tolist() == [0, 0]
        assert torch.isnan(prob.ret.float()).all()
        rep = ctx.moe_ovl_get_report()
        assert rep.num_bands == 0 and rep.num_items == 0 and rep.num_segments == 0
    # (b) a single row; (c) an expert with no rows between two loaded ones
    keep_one = np.zeros(dsp.M, bool)
    keep_one[5] = True
    keep_gap = dsp.row_expert != 1
    for keep in (keep_one, keep_gap):
        sub = I.Dispatched(dsp.x_rows[keep], np.bincount(dsp.row_expert[keep], minlength=3).astype(np.int32),
                           dsp.src_rank[keep], dsp.src_token[keep], dsp.gate[keep], dsp.row_expert[keep])
        _, _, ctx, prob = _run_case(shape, 0, 4, inp=inp, dsp=sub)
        plan = U.oracle_plan(shape, sub)
        U.check_indices(shape, sub, plan, ctx.moe_ovl_get_plan(), prob.slot_out.cpu().numpy(),
                        prob.rows_per_rank_out.cpu().numpy(), prob.segs_per_rank_out.cpu().numpy(),
                        ctx.moe_ovl_get_report())
        # oracle on routing restricted to the kept rows: drop the other selections by pointing them off-GPU
        inp2 = I.MoEInputs(shape, inp.x, inp.w1, inp.w2, inp.expert.copy(), inp.gate)
        kept = set(zip(sub.row_expert.tolist(), sub.src_rank.tolist(), sub.src_token.tolist()))
        for r in range(shape.R):
            for t in range(shape.T):
                for q in range(shape.k):
                    e = inp2.expert[r, t, q]
                    if e < shape.El and (int(e), r, t) not in kept:
                        inp2.expert[r, t, q] = shape.Eg + 5
        toks = np.arange(shape.R * shape.T)
        o = U.oracle_values(inp2, toks)
        U.check_values(shape, sub, plan, toks, *o, Hn.device_to_bits(prob.out), Hn.device_to_bits(prob.ret))


def test_bad_routing_is_reported_not_fatal():
    torch, B, Hn = _gpu()
    shape = I.SHAPES["tiny"]
    inp = I.make_inputs(shape)
    dsp = I.dispatch(inp)
    ctx = Hn.make_context(shape, max_rows=dsp.M)
    for kind in ("rank", "dup", "sum"):
        bad = I.Dispatched(dsp.x_rows, dsp.expert_counts.copy(), dsp.src_rank.copy(), dsp.src_token.copy(), dsp.gate,
                           dsp.row_expert)
        if kind == "rank":
            bad.src_rank[3] = shape.R
        elif kind == "dup":
            bad.src_rank[1], bad.src_token[1] = bad.src_rank[0], bad.src_token[0]
        else:
            bad.expert_counts[0] -= 1
        prob = Hn.upload(inp, bad)
        Hn.run(ctx, prob, mode=B.MODE_OVERLAP, consumer_sm_count=4)
        torch.cuda.synchronize()
        code, detail = ctx.moe_ovl_query_status()
        assert code == B.ERR_BAD_ROUTING, (kind, code)
    # the context stays usable
    prob = Hn.upload(inp, dsp)
    Hn.run(ctx, prob, mode=B.MODE_OVERLAP, consumer_sm_count=4)
    torch.cuda.synchronize()
    assert ctx.moe_ovl_query_status()[0] == 0
    # synchronous argument errors
    with pytest.raises(B.MoeOvlError) as e:
        Hn.run(ctx, prob, mode=B.MODE_OVERLAP, consumer_sm_count=-1)
    assert e.value.code == B.ERR_INVALID_ARG
    with pytest.raises(B.MoeOvlError) as e:
        Hn.run(ctx, prob, mode=B.MODE_OVERLAP, consumer_sm_count=100)
    assert e.value.code == B.ERR_INVALID_ARG
    with pytest.raises(B.MoeOvlError):
        Hn.run(ctx, prob, mode=7)


def test_host_buffer_entry_point_matches_device_entry_point():
    torch, B, Hn = _gpu()
    shape = I.SHAPES["small"]
    inp = I.make_inputs(shape)
    dsp = I.dispatch(inp)
    ctx = Hn.make_context(shape, max_rows=dsp.M, flags=B.FLAG_HOST_STAGING)
    prob = Hn.upload(inp, dsp)
    Hn.run(ctx, prob, mode=B.MODE_OVERLAP, consumer_sm_count=8)
    torch.cuda.synchronize()
    pin = lambda a: torch.from_numpy(np.ascontiguousarray(a)).pin_memory()
    hx = pin(dsp.x_rows.view(np.int16))
    hc, hr, ht, hg = pin(dsp.expert_counts), pin(dsp.src_rank), pin(dsp.src_token), pin(dsp.gate)
    hout = torch.zeros((shape.R * shape.T, shape.d), dtype=torch.int16).pin_memory()
    # several calls in a row exercise both staging slots and the copy pipeline; a second problem in between
    # makes a result that came from the wrong slot visible
    inp2 = I.make_inputs(I.with_seed(shape, 5))
    dsp2 = I.dispatch(inp2)
    ctx2 = Hn.make_context(shape, max_rows=dsp2.M)
    prob_b = Hn.upload(inp2, dsp2, w1=prob.w1, w2=prob.w2)
    Hn.run(ctx2, prob_b, mode=B.MODE_OVERLAP, consumer_sm_count=8)
    hx2 = pin(dsp2.x_rows.view(np.int16))
    hc2, hr2, ht2, hg2 = pin(dsp2.expert_counts), pin(dsp2.src_rank), pin(dsp2.src_token), pin(dsp2.gate)
    houts = [torch.zeros_like(hout).pin_memory() for _ in range(5)]
    for i, ho in enumerate(houts):
        a = (hx, hc, hr, ht, hg) if i % 2 == 0 else (hx2, hc2, hr2, ht2, hg2)
        ctx.moe_ovl_expert_return_host(x=a[0], expert_counts=a[1], src_rank=a[2], src_token=a[3], gate=a[4],
                                       w1=prob.w1, w2=prob.w2, out=ho, consumer_sm_count=8, mode=B.MODE_OVERLAP)
    ctx.moe_ovl_host_join()
    torch.cuda.synchronize()
    assert ctx.moe_ovl_query_status()[0] == 0
    want = [prob.out.view(torch.int16).cpu(), prob_b.out.view(torch.int16).cpu()]
    for i, ho in enumerate(houts):
        assert torch.equal(ho, want[i % 2]), i


@pytest.mark.parametrize("seed", list(range(12)))
def test_random_shapes_full_parity(seed):
    """Seeded random small problems: rank and expert counts, top-k, widths, local rank, router, arrival order,
    consumer budget, segment and super-band knobs all vary; every output is checked against the oracle."""
    torch, B, Hn = _gpu()
    rng = np.random.Generator(np.random.PCG64(1000 + seed))
    El = int(rng.integers(1, 6))
    groups = int(rng.integers(1, 4))
    Eg = El * groups
    k = int(rng.integers(1, min(Eg, 4) + 1))
    R = int(rng.integers(1, 7))
    single = seed % 4 == 3
    shape = I.MoEShape(f"rnd{seed}", R=R, T=int(rng.integers(1, 500)), Eg=Eg, k=k, El=El,
                       d=int(rng.choice([64, 192, 320])) if single else int(rng.choice([256, 512])),
                       F=0 if single else int(rng.choice([128, 256, 640])),
                       N_out=int(rng.choice([256, 768])) if single else 0,
                       router=str(rng.choice(["uniform", "zipf", "zipf_rot"])), seed=seed,
                       self_rank=int(rng.integers(0, R)), first_local=int(rng.integers(0, groups)) * El)
    mode = (B.MODE_OVERLAP, B.MODE_IN_KERNEL, B.MODE_OVERLAP, B.MODE_AUTO, B.MODE_NON_OVERLAP)[seed % 5]
    csm = int(rng.choice([0, 1, 2, 6, 24]))
    mgb = int(rng.integers(1, 4))
    gb = int(rng.choice([0, 2, 4, 5, 64]))
    inp = I.make_inputs(shape)
    dsp = I.dispatch(inp, shuffle_seed=int(rng.integers(0, 99)) if seed % 2 else None)
    ctx = Hn.make_context(shape, max_rows=max(dsp.M, 1) + int(rng.integers(0, 300)), mid_seg_bands=mgb, group_bands=gb,
                          flags=(B.FLAG_TEST_ALL_SMALL_GROUP_TILES if seed % 3 else 0) |
                                (B.FLAG_TEST_ZERO_ROWS_EARLY if seed % 2 == 0 else 0))
    prob = Hn.upload(inp, dsp)
    Hn.run(ctx, prob, mode=mode, consumer_sm_count=csm)
    torch.cuda.synchronize()
    code, detail = ctx.moe_ovl_query_status()
    assert code == 0, (code, hex(detail))
    plan = U.oracle_plan(shape, dsp, mgb=mgb)
    U.check_indices(shape, dsp, plan, ctx.moe_ovl_get_plan(), prob.slot_out.cpu().numpy(),
                    prob.rows_per_rank_out.cpu().numpy(), prob.segs_per_rank_out.cpu().numpy(),
                    ctx.moe_ovl_get_report())
    toks = np.arange(shape.R * shape.T)
    o = U.oracle_values(inp, toks)
    U.check_values(shape, dsp, plan, toks, *o, Hn.device_to_bits(prob.out), Hn.device_to_bits(prob.ret))


@pytest.mark.parametrize("seed", list(range(24)))
def test_random_small_group_shapes_full_parity(seed):
    """Seeded random problems with few tokens per (expert, rank) group, where the plan issues pairs 64 rows high,
    stacks of three or four small bands, local bands riding with remote ones and (with the test hook) groups with
    swapped operands; up to 8 ranks and 8 local experts; every output is checked against the oracle, and the same
    problem with those items switched off must give the same indices."""
    torch, B, Hn = _gpu()
    rng = np.random.Generator(np.random.PCG64(7000 + seed))
    El = int(rng.integers(1, 9))
    groups = int(rng.integers(1, 4))
    Eg = El * groups
    k = int(rng.integers(1, min(Eg, 4) + 1))
    R = int(rng.integers(1, 9))
    single = seed % 4 == 3
    shape = I.MoEShape(f"rsg{seed}", R=R, T=int(rng.integers(1, 90)), Eg=Eg, k=k, El=El,
                       d=int(rng.choice([64, 192, 320])) if single else int(rng.choice([256, 512])),
                       F=0 if single else int(rng.choice([256, 640])),
                       N_out=int(rng.choice([256, 768])) if single else 0,
                       router=str(rng.choice(["uniform", "zipf", "zipf_rot"])), seed=seed,
                       self_rank=int(rng.integers(0, R)), first_local=int(rng.integers(0, groups)) * El)
    mode = (B.MODE_OVERLAP, B.MODE_IN_KERNEL, B.MODE_AUTO, B.MODE_NON_OVERLAP)[seed % 4]
    csm = int(rng.choice([0, 2, 6]))
    gb = int(rng.choice([0, 2, 4, 64]))
    flags = (0, 0, B.FLAG_NO_LOCAL_RIDERS, B.FLAG_TEST_ALL_SMALL_GROUP_TILES, B.FLAG_NO_STACKED_BANDS, 0)[seed % 6]
    flags |= B.FLAG_TEST_ZERO_ROWS_EARLY if seed % 2 else 0      # zero rows of `out` written behind the GEMM
    inp = I.make_inputs(shape)
    dsp = I.dispatch(inp, shuffle_seed=int(rng.integers(0, 99)) if seed % 2 else None)
    plan = U.oracle_plan(shape, dsp)
    toks = np.arange(shape.R * shape.T)
    o = U.oracle_values(inp, toks)
    kinds = set()
    for fl in (flags, B.FLAG_NO_SMALL_GROUP_TILES):
        ctx = Hn.make_context(shape, max_rows=max(dsp.M, 1), group_bands=gb, flags=fl)
        prob = Hn.upload(inp, dsp)
        for _ in range(2):                   # twice: counters and flags of the first call must not leak
            Hn.run(ctx, prob, mode=mode, consumer_sm_count=csm)
        torch.cuda.synchronize()
        code, detail = ctx.moe_ovl_query_status()
        assert code == 0, (code, hex(detail))
        gp = ctx.moe_ovl_get_plan()
        U.check_indices(shape, dsp, plan, gp, prob.slot_out.cpu().numpy(), prob.rows_per_rank_out.cpu().numpy(),
                        prob.segs_per_rank_out.cpu().numpy(), ctx.moe_ovl_get_report())
        U.check_values(shape, dsp, plan, toks, *o, Hn.device_to_bits(prob.out), Hn.device_to_bits(prob.ret))
        kinds = set((gp["item"][:, 0] & 0xff).tolist())
    assert kinds <= {0, 1}


def test_call_can_be_captured_in_a_cuda_graph_and_replayed():
    """A captured call replays with new contents in the same buffers (the number that marks a call's ready flags
    lives in device memory, so every replay gets a fresh one); overlap mode, both internal streams in the capture."""
    torch, B, Hn = _gpu()
    shape = I.SHAPES["small_zipf_rot"]
    inp = I.make_inputs(shape)
    dsp = I.dispatch(inp)
    ctx = Hn.make_context(shape, max_rows=dsp.M)
    ref_ctx = Hn.make_context(shape, max_rows=dsp.M)
    prob = Hn.upload(inp, dsp)
    side = torch.cuda.Stream()
    with torch.cuda.stream(side):
        Hn.run(ctx, prob, mode=B.MODE_OVERLAP, consumer_sm_count=4)          # warm-up outside the capture
    side.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph, stream=side, capture_error_mode="thread_local"):
        Hn.run(ctx, prob, mode=B.MODE_OVERLAP, consumer_sm_count=4)
    for scale in (1.0, -0.5, 2.0, 0.25):
        x_new = (Hn.bits_to_device(dsp.x_rows, "cuda:0").float() * scale).to(torch.bfloat16)
        prob.x.copy_(x_new)
        prob.out.fill_(float("nan"))
        prob.ret.fill_(float("nan"))
        torch.cuda.synchronize()
        graph.replay()
        torch.cuda.synchronize()
        assert ctx.moe_ovl_query_status()[0] == 0
        ref = Hn.upload(inp, dsp, w1=prob.w1, w2=prob.w2)
        ref.x.copy_(x_new)
        Hn.run(ref_ctx, ref, mode=B.MODE_NON_OVERLAP)
        torch.cuda.synchronize()
        assert torch.equal(prob.out.view(torch.int16), ref.out.view(torch.int16)), scale
        assert torch.equal(prob.ret.view(torch.int16), ref.ret.view(torch.int16)), scale
    # a captured call records no timing events: the report says so instead of failing, the plan sizes and the
    # device stamps of the last replay are still there, and the GEMM-time average skips the captured call
    rep = ctx.moe_ovl_get_report()
    assert rep.timing_valid == 0 and rep.ms_total == 0.0 and rep.ms_producer == 0.0
    assert rep.num_bands > 0 and rep.us_return_done > 0.0
    ms, n = ctx.moe_ovl_get_gemm_time(1)
    assert n == 0 and ms == 0.0
    ms, n = ctx.moe_ovl_get_gemm_time(2)          # the warm-up call before the capture was timed
    assert n == 1 and ms > 0.0


@pytest.mark.parametrize("mode,csm", [(0, 4), (2, 0), (1, 0)])
def test_trace_records_every_item_and_unit(mode, csm):
    """The device trace: one record per schedule item (claimed <= first operands landed <= published) and one
    per moved unit of the return; a segment is never seen ready before the last of its tiles was published."""
    torch, B, Hn = _gpu()
    shape = I.SHAPES["small_zipf_rot"]
    inp = I.make_inputs(shape)
    dsp = I.dispatch(inp)
    ctx = Hn.make_context(shape, max_rows=dsp.M, flags=B.FLAG_TRACE)
    prob = Hn.upload(inp, dsp)
    for _ in range(2):                                   # the second call must not see the first call's records
        Hn.run(ctx, prob, mode=mode, consumer_sm_count=csm)
        torch.cuda.synchronize()
        assert ctx.moe_ovl_query_status()[0] == 0
    rep = ctx.moe_ovl_get_report()
    plan = ctx.moe_ovl_get_plan()
    tr = ctx.moe_ovl_get_trace()
    items, units = tr[tr["kind"] == B.TRACE_ITEM], tr[tr["kind"] == B.TRACE_UNIT]
    assert len(items) == rep.num_items and items["index"].tolist() == list(range(rep.num_items))
    assert (items["ns_claim"] >= 0).all()
    assert (items["ns_claim"] <= items["ns_ready"]).all() and (items["ns_ready"] <= items["ns_done0"]).all()
    # the load thread sees an item's inputs complete after the claim and before its first operands can land
    assert (items["ns_claim"] <= items["ns_inputs_ready"]).all() and (items["ns_inputs_ready"] <= items["ns_ready"]).all()
    second = plan["item"][:, 2] >= 0                     # the pair's second band exists (a stack always has one)
    assert (items["ns_done1"][second] >= items["ns_ready"][second]).all() and (items["ns_done1"][~second] == -1).all()
    assert (items["cta"] % 2 == 0).all() and items["cta"].max() < rep.producer_ctas
    # claims are handed out in issue order (each pair stamps its own claim, hence the slack)
    assert (np.diff(items["ns_claim"]) >= -5000).all()
    if mode == B.MODE_NON_OVERLAP:
        assert len(units) == 0
        return
    # the dedicated consumer moves whole segments except the schedule's last 16, which are sliced in 8; the spare
    # warps of the GEMM CTAs move slices throughout
    nseg = rep.num_segments
    whole = max(0, nseg - 16) if mode == B.MODE_OVERLAP else 0
    assert len(units) == whole + (nseg - whole) * 8
    assert (units["who"] == 2).all() if mode == B.MODE_IN_KERNEL else set(units["who"].tolist()) <= {0, 1}
    assert (units["ns_done0"] >= units["ns_claim"]).all()
    seg_of = units["index"] // 8
    assert sorted(units["index"].tolist()) == [s * 8 + c for s in range(nseg) for c in range(1 if s < whole else 8)]
    assert (units["chunks"] == np.where(seg_of < whole, 1, 8)).all()
    seg_rows = plan["seg"][:, 3]
    assert np.bincount(seg_of, weights=units["rows"], minlength=nseg).astype(int).tolist() == seg_rows.tolist()
    # latest publication time of any output tile of each band (second-GEMM items only)
    n_bands = rep.num_bands
    band_done = np.zeros(n_bands, np.int64)
    sched = plan["sched_band"].tolist()
    for (x, b0, b1, _tile), rec in zip(plan["item"].tolist(), items):
        kind = x & 0xff
        if kind == 3:                 # swapped operands: both CTAs hold columns of every band of the group
            for b in sched[b0:b0 + (b1 & 0xff)]:
                band_done[b] = max(band_done[b], rec["ns_done0"], rec["ns_done1"])
        elif kind & 8 and kind & 1:   # stacked bands: the first two are the leader CTA's, the rest its peer's
            for i in range(b1):
                band_done[b0 + i] = max(band_done[b0 + i], rec["ns_done0"] if i < 2 else rec["ns_done1"])
        elif kind & 3 == 1:
            band_done[b0] = max(band_done[b0], rec["ns_done0"])
            if b1 >= 0:
                band_done[b1] = max(band_done[b1], rec["ns_done1"])
    for rec in units:
        first, nb = plan["seg"][rec["index"] // 8, 0], plan["seg"][rec["index"] // 8, 1]
        assert rec["ns_claim"] >= band_done[first:first + nb].max()
    assert abs(rep.us_return_done * 1e3 - units["ns_done0"].max()) < 2e3


def test_trace_is_refused_without_the_flag():
    torch, B, Hn = _gpu()
    shape = I.SHAPES["tiny"]
    inp, dsp, ctx, prob = _run_case(shape, 0, 2)
    with pytest.raises(B.MoeOvlError) as e:
        ctx.moe_ovl_get_trace()
    assert e.value.code == B.ERR_UNSUPPORTED


def test_serialised_kernels_degrade_instead_of_timing_out():
    """With launches made blocking the two kernels of the overlap mode cannot run side by side.  The GEMM is
    enqueued first, so it runs to completion, its own CTAs move every segment, and the consumer finds nothing
    left: the call succeeds (a profiler that serialises kernels sees the same)."""
    import os
    import subprocess
    import sys
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    child = r"""
import sys
sys.path.insert(0, %r)
import numpy as np, torch
from paper_2607_19539_b200 import binding as B, harness as Hn, inputs as I
shape = I.SHAPES["tiny"]
inp = I.make_inputs(shape); dsp = I.dispatch(inp)
ctx = Hn.make_context(shape, max_rows=dsp.M, wait_timeout_us=50_000)
ref = Hn.upload(inp, dsp)
Hn.run(ctx, ref, mode=B.MODE_NON_OVERLAP); torch.cuda.synchronize()
for csm in (2, 8):
    prob = Hn.upload(inp, dsp, w1=ref.w1, w2=ref.w2)
    Hn.run(ctx, prob, mode=B.MODE_OVERLAP, consumer_sm_count=csm); torch.cuda.synchronize()
    code, detail = ctx.moe_ovl_query_status()
    assert code == 0, (code, hex(detail))
    assert torch.equal(prob.out.view(torch.int16), ref.out.view(torch.int16))
    assert torch.equal(prob.ret.view(torch.int16), ref.ret.view(torch.int16))
    assert ctx.moe_ovl_get_report().segments_by_gemm_ctas == ctx.moe_ovl_get_report().return_units > 0
print("serialised ok")
""" % root
    env = dict(os.environ, CUDA_LAUNCH_BLOCKING="1")
    r = subprocess.run([sys.executable, "-c", child], env=env, capture_output=True, text=True, timeout=600)
    assert r.returncode == 0 and "serialised ok" in r.stdout, r.stdout + r.stderr


def test_gemm_kernel_gives_up_cleanly_when_its_input_never_arrives():
    """The bounded waits inside the GEMM kernel: a test hook leaves the first band of the schedule ungathered, so
    the load warp's wait for it runs out.  The kernel must report the timeout, let its copies land, free its
    tensor memory and return; the context and the device stay usable."""
    torch, B, Hn = _gpu()
    shape = I.SHAPES["small"]
    inp = I.make_inputs(shape)
    dsp = I.dispatch(inp)
    ctx = Hn.make_context(shape, max_rows=dsp.M, wait_timeout_us=20_000, flags=B.FLAG_TEST_SKIP_GATHER)
    prob = Hn.upload(inp, dsp)
    for mode, csm in ((B.MODE_NON_OVERLAP, 0), (B.MODE_OVERLAP, 4), (B.MODE_IN_KERNEL, 0)):
        Hn.run(ctx, prob, mode=mode, consumer_sm_count=csm)
        torch.cuda.synchronize()
        code, detail = ctx.moe_ovl_query_status()
        assert code == B.ERR_TIMEOUT, (mode, code)
        # Which wait gives up first is a race between waits that all started within microseconds of each other and
        # all hang on the same missing band: the load warp waiting for its gathered rows (site 11) or for the hidden
        # rows that depend on it (2), the MMA thread waiting for the operands that load would have brought (3), the
        # scheduler waiting for that load warp to move on (10), a mover polling the band's flags (6), ...
        assert 1 <= detail >> 48 <= 12, hex(detail)
    ok = Hn.make_context(shape, max_rows=dsp.M)
    ref = Hn.upload(inp, dsp, w1=prob.w1, w2=prob.w2)
    Hn.run(ok, ref, mode=B.MODE_NON_OVERLAP)
    prob2 = Hn.upload(inp, dsp, w1=prob.w1, w2=prob.w2)
    Hn.run(ok, prob2, mode=B.MODE_OVERLAP, consumer_sm_count=4)
    torch.cuda.synchronize()
    assert ok.moe_ovl_query_status()[0] == 0
    assert torch.equal(prob2.out.view(torch.int16), ref.out.view(torch.int16))
    plan = U.oracle_plan(shape, dsp)
    assert prob2.slot_out.cpu().numpy()[:dsp.M].tolist() == plan.slot


def test_rows_beyond_the_receive_region_are_reported_and_never_written():
    """Malformed routing with more local experts than top-k: every token is routed to all three local experts, so
    a rank would need 3T receive rows where the region holds min(k, El) * T = 2T.  The call must report bad
    routing and write nothing outside the regions: the receive buffer is over-allocated with a canary tail, so
    that even an unguarded write would stay in owned memory."""
    torch, B, Hn = _gpu()
    shape = I.MoEShape("overflow", R=2, T=200, Eg=6, k=2, El=3, d=256, F=128, seed=11)
    inp = I.make_inputs(shape)
    T, R, El, d = shape.T, shape.R, shape.El, shape.d
    M = El * R * T
    rng = np.random.Generator(np.random.PCG64(5))
    rows = I.f32_to_bf16_bits(rng.standard_normal((M, d), dtype=np.float32))
    r_idx = np.tile(np.repeat(np.arange(R, dtype=np.int32), T), El)
    t_idx = np.tile(np.arange(T, dtype=np.int32), El * R)
    bad = I.Dispatched(rows, np.full(El, R * T, np.int32), r_idx, t_idx, np.full(M, 0.5, np.float32),
                       np.repeat(np.arange(El, dtype=np.int32), R * T))
    ctx = Hn.make_context(shape, max_rows=M)
    prob = Hn.upload(inp, bad)
    region = T * shape.kmax
    big = torch.full((R * El * T + 64, d), float("nan"), dtype=torch.bfloat16, device="cuda:0")
    for mode, csm in ((B.MODE_NON_OVERLAP, 0), (B.MODE_OVERLAP, 4), (B.MODE_IN_KERNEL, 0)):
        big.fill_(float("nan"))
        ctx.moe_ovl_expert_return(x=prob.x, expert_counts=prob.expert_counts, src_rank=prob.src_rank,
                                  src_token=prob.src_token, gate=prob.gate, w1=prob.w1, w2=prob.w2,
                                  ret=big[:R * region].view(R, region, d), out=prob.out, consumer_sm_count=csm,
                                  mode=mode, num_rows=M)
        torch.cuda.synchronize()
        code, detail = ctx.moe_ovl_query_status()
        assert code == B.ERR_BAD_ROUTING, (mode, code)
        assert torch.isnan(big[R * region:].float()).all()           # nothing past the last rank's region
    # the context stays usable with well-formed routing
    dsp = I.dispatch(inp)
    good = Hn.upload(inp, dsp, w1=prob.w1, w2=prob.w2)
    Hn.run(ctx, good, mode=B.MODE_OVERLAP, consumer_sm_count=4)
    torch.cuda.synchronize()
    assert ctx.moe_ovl_query_status()[0] == 0


@pytest.mark.parametrize("name", ["decode", "many_small_groups", "tiny"])
def test_small_group_items_can_be_switched_off(name):
    """Runs of small (expert, rank) groups are issued as swapped-operand items; with the flag that forbids them the
    same problem goes through band-pair items only.  Both must match the oracle, and the plan must show the
    difference."""
    torch, B, Hn = _gpu()
    shape = I.SHAPES[name]
    inp = I.make_inputs(shape)
    dsp = I.dispatch(inp)
    plan = U.oracle_plan(shape, dsp)
    toks = np.arange(shape.R * shape.T)
    o = U.oracle_values(inp, toks)
    kinds = {}
    for flags in (B.FLAG_TEST_ALL_SMALL_GROUP_TILES, B.FLAG_NO_SMALL_GROUP_TILES):
        ctx = Hn.make_context(shape, max_rows=dsp.M, flags=flags)
        prob = Hn.upload(inp, dsp)
        Hn.run(ctx, prob, mode=B.MODE_IN_KERNEL)
        torch.cuda.synchronize()
        assert ctx.moe_ovl_query_status()[0] == 0
        gp = ctx.moe_ovl_get_plan()
        U.check_indices(shape, dsp, plan, gp, prob.slot_out.cpu().numpy(), prob.rows_per_rank_out.cpu().numpy(),
                        prob.segs_per_rank_out.cpu().numpy(), ctx.moe_ovl_get_report())
        U.check_values(shape, dsp, plan, toks, *o, Hn.device_to_bits(prob.out), Hn.device_to_bits(prob.ret))
        kinds[flags] = set((gp["item"][:, 0] & 0xff).tolist())
    assert kinds[B.FLAG_NO_SMALL_GROUP_TILES] <= {0, 1}
    # every one of these problems has at least one run of small groups
    assert kinds[B.FLAG_TEST_ALL_SMALL_GROUP_TILES] & {2, 3}
    # left to itself the plan computes pairs of small bands 64 rows high (kinds 4, 5) or stacks them (8, 9); these
    # shapes hold too few items for swapped-operand groups to pay
    ctx = Hn.make_context(shape, max_rows=dsp.M)
    prob = Hn.upload(inp, dsp)
    Hn.run(ctx, prob, mode=B.MODE_OVERLAP, consumer_sm_count=4)
    torch.cuda.synchronize()
    assert ctx.moe_ovl_query_status()[0] == 0
    gp = ctx.moe_ovl_get_plan()
    U.check_indices(shape, dsp, plan, gp, prob.slot_out.cpu().numpy(), prob.rows_per_rank_out.cpu().numpy(),
                    prob.segs_per_rank_out.cpu().numpy(), ctx.moe_ovl_get_report())
    U.check_values(shape, dsp, plan, toks, *o, Hn.device_to_bits(prob.out), Hn.device_to_bits(prob.ret))
    default_kinds = set((gp["item"][:, 0] & 0xff).tolist())
    assert default_kinds & {4, 5, 8, 9} and not default_kinds & {2, 3}
    if name != "tiny":
        # three remote groups per expert, all small: stacked into one full-height item per tile (kinds 8, 9) unless
        # the flag forbids it
        assert default_kinds & {8, 9}
        ctx = Hn.make_context(shape, max_rows=dsp.M, flags=B.FLAG_NO_STACKED_BANDS)
        prob = Hn.upload(inp, dsp)
        Hn.run(ctx, prob, mode=B.MODE_IN_KERNEL)
        torch.cuda.synchronize()
        assert ctx.moe_ovl_query_status()[0] == 0
        gp = ctx.moe_ovl_get_plan()
        U.check_indices(shape, dsp, plan, gp, prob.slot_out.cpu().numpy(), prob.rows_per_rank_out.cpu().numpy(),
                        prob.segs_per_rank_out.cpu().numpy(), ctx.moe_ovl_get_report())
        U.check_values(shape, dsp, plan, toks, *o, Hn.device_to_bits(prob.out), Hn.device_to_bits(prob.ret))
        assert set((gp["item"][:, 0] & 0xff).tolist()) <= {0, 1, 4, 5}

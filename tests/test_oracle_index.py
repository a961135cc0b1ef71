"""Pins for the index oracle (row layout, schedule, combine plan, segments).

None of these re-types the oracle's own loops: they use a hand-derived worked
example, set/permutation invariants, the paper's printed bounds, and an
independent global-sort formulation."""
import json
import os

import numpy as np
import pytest

from oracle.index_oracle import build_plan, segment_band_counts
from paper_2607_19539_b200 import inputs as I

GOLD = os.path.join(os.path.dirname(__file__), "golden", "index_worked_example.json")


def _plan_for(shape, tb_M=128, mgb=1, shuffle_seed=None, tiles_per_band=None):
    inp = I.make_inputs(shape, weights=False)
    dsp = I.dispatch(inp, shuffle_seed=shuffle_seed, gather_x=False)
    tpb = tiles_per_band or max(1, shape.d // 256)
    plan = build_plan(dsp.expert_counts.tolist(), dsp.src_rank.tolist(), dsp.src_token.tolist(),
                      shape.R, shape.self_rank, tb_M, mgb, tpb, gate=dsp.gate.tolist(), T=shape.T)
    return inp, dsp, plan


def test_worked_example_algorithm1():
    g = json.load(open(GOLD))
    rows = g["rows"]
    plan = build_plan(g["expert_counts"], [r for r, _ in rows], [t for _, t in rows],
                      g["R"], g["r_self"], g["tb_M"], 1, g["tiles_per_band"])
    assert plan.n == g["n"]
    assert plan.rows_per_rank == g["rows_per_rank"]
    assert plan.P == g["P"] and plan.expert_base == g["expert_base"]
    assert plan.pos == g["pos"]
    assert plan.slot == g["slot"]
    got = [[b.band, b.expert, b.dest, b.pos0, b.valid, b.slot0, int(b.local)] for b in plan.bands]
    assert got == g["bands"]
    assert plan.expert_order == g["expert_order"]
    assert plan.band_order == g["band_order"]
    # schedule S lists every tile of a band, band by band
    assert plan.tiles == [(plan.bands[b].expert, b, j) for b in g["band_order"] for j in range(2)]
    assert plan.segs_per_rank == g["segs_per_rank_mgb1"]
    remote_pad = sum(g["tb_M"] - b.valid for b in plan.bands if not b.local)
    assert remote_pad == g["remote_padding_rows"]
    plan2 = build_plan(g["expert_counts"], [r for r, _ in rows], [t for _, t in rows],
                       g["R"], g["r_self"], g["tb_M"], 2, g["tiles_per_band"])
    assert plan2.segs_per_rank == g["segs_per_rank_mgb2"]
    assert plan2.pos == plan.pos and plan2.slot == plan.slot and plan2.band_order == plan.band_order


def test_segment_shapes_golden_and_bruteforce():
    g = json.load(open(GOLD))
    for nb, per in g["segment_shapes"].items():
        for mgb, shape in per.items():
            assert segment_band_counts(int(nb), int(mgb)) == shape
    # Figure 3b: first and last segment one band, middle ones up to mgb bands, in order, covering all bands
    for nb in range(0, 13):
        for mgb in (1, 2, 3):
            s = segment_band_counts(nb, mgb)
            assert sum(s) == nb and all(c >= 1 for c in s)
            if nb >= 2:
                assert s[0] == 1 and s[-1] == 1
                assert all(c <= mgb for c in s[1:-1])
                # only the last middle segment may be short
                assert all(c == mgb for c in s[1:-2])
                assert len(s) == 2 + -(-(nb - 2) // mgb)
            if mgb == 1:
                assert len(s) == nb


def test_paper_sizes():
    # Section 3.3.2: a tile is 32 or 64 KiB; one band at mgb=1 is about 1-2 MiB, 2-4 MiB at mgb=2
    assert 128 * 128 * 2 == 32 * 1024 and 128 * 256 * 2 == 64 * 1024
    for N, mib in ((4096, 1), (8192, 2)):          # Table 2 output widths
        assert 128 * N * 2 == mib * 1024 * 1024
        assert sum(segment_band_counts(6, 2)[1:2]) * 128 * N * 2 == 2 * mib * 1024 * 1024


@pytest.mark.parametrize("name,shuffle", [("tiny", None), ("tiny_zipf", 5), ("small", None), ("small", 11),
                                          ("small_zipf_rot", 2), ("many_groups", 1)])
def test_round_trip_permutation(name, shuffle):
    shape = I.SHAPES[name]
    inp, dsp, plan = _plan_for(shape, shuffle_seed=shuffle)
    M = dsp.M
    sr, st, re = dsp.src_rank, dsp.src_token, dsp.row_expert
    slot = np.asarray(plan.slot)
    pos = np.asarray(plan.pos)
    assert sum(plan.rows_per_rank) == M
    for r in range(shape.R):
        mine = np.nonzero(sr == r)[0]
        assert sorted(slot[mine].tolist()) == list(range(plan.rows_per_rank[r]))
        assert sum(plan.n[e][r] for e in range(shape.El)) == plan.rows_per_rank[r]
        # inside a rank's region: expert-major, and source-token order inside each expert
        order = mine[np.argsort(slot[mine])]
        keys = list(zip(re[order].tolist(), st[order].tolist()))
        assert keys == sorted(keys) and len(set(keys)) == len(keys)
    # pos is injective, stays inside its group's padded range, padding positions are hit by no row
    assert len(set(pos.tolist())) == M and pos.min(initial=0) >= 0 and pos.max(initial=0) < max(plan.P, 1)
    covered = np.zeros(plan.P, bool)
    for b in plan.bands:
        covered[b.pos0:b.pos0 + b.valid] = True
    hit = np.zeros(plan.P, bool)
    hit[pos] = True
    assert (covered == hit).all()
    for i in range(M):
        b = plan.bands[pos[i] // 128]
        assert b.expert == re[i] and b.dest == sr[i] and b.band == pos[i] // 128
        assert slot[i] == b.slot0 + (pos[i] - b.pos0)
    # un-permuting a buffer written at slot[] gives the rows back in input order
    ret = [np.full(plan.rows_per_rank[r], -1) for r in range(shape.R)]
    for i in range(M):
        ret[sr[i]][slot[i]] = i
    back = np.array([ret[sr[i]][slot[i]] for i in range(M)])
    assert (back == np.arange(M)).all()
    # per-token lists for the weighted reduction: ascending expert, every row exactly once
    seen = 0
    for tok, (ss, gs) in enumerate(zip(plan.tok_slot, plan.tok_gate)):
        r = tok // shape.T
        rows = [int(np.nonzero((sr == r) & (slot == s))[0][0]) for s in ss]
        assert [st[i] for i in rows] == [tok % shape.T] * len(rows)
        assert re[rows].tolist() == sorted(re[rows].tolist())
        assert [float(dsp.gate[i]) for i in rows] == gs
        seen += len(rows)
    assert seen == M


@pytest.mark.parametrize("name", ["tiny", "small", "small_zipf_rot", "tiny_zipf"])
def test_arrival_order_does_not_matter(name):
    shape = I.SHAPES[name]
    _, d0, p0 = _plan_for(shape)
    _, d1, p1 = _plan_for(shape, shuffle_seed=123)
    k0 = {(e, r, t): (p, s) for e, r, t, p, s in zip(d0.row_expert, d0.src_rank, d0.src_token, p0.pos, p0.slot)}
    k1 = {(e, r, t): (p, s) for e, r, t, p, s in zip(d1.row_expert, d1.src_rank, d1.src_token, p1.pos, p1.slot)}
    assert k0 == k1
    assert p0.band_order == p1.band_order and p0.segs_per_rank == p1.segs_per_rank


@pytest.mark.parametrize("name,tb_M", [("tiny", 128), ("small", 128), ("small", 32), ("small_zipf_rot", 64)])
def test_against_global_sort_formulation(name, tb_M):
    """Independent formulation: one global lexicographic sort instead of per-group gathering."""
    shape = I.SHAPES[name]
    _, dsp, plan = _plan_for(shape, tb_M=tb_M, shuffle_seed=9)
    R, rs = shape.R, shape.self_rank
    rank_key = np.array([(r if r < rs else r - 1) if r != rs else R - 1 for r in range(R)])
    order = np.lexsort((np.arange(dsp.M), dsp.src_token, rank_key[dsp.src_rank], dsp.row_expert))
    pos = np.empty(dsp.M, np.int64)
    cur, prev = 0, None
    for i in order:
        key = (dsp.row_expert[i], dsp.src_rank[i])
        if prev is not None and key != prev:
            cur = -(-cur // tb_M) * tb_M
        pos[i] = cur
        cur += 1
        prev = key
    # an expert with no rows at all adds nothing; empty groups add nothing
    assert pos.tolist() == plan.pos
    order2 = np.lexsort((np.arange(dsp.M), dsp.src_token, dsp.row_expert, dsp.src_rank))
    slot = np.empty(dsp.M, np.int64)
    start = {}
    for idx, i in enumerate(order2):
        start.setdefault(dsp.src_rank[i], idx)
        slot[i] = idx - start[dsp.src_rank[i]]
    assert slot.tolist() == plan.slot


def test_padding_bound_section_4_5():
    # Section 4.5: padding is at most (W-1)(tb_M-1) rows, 765 for W=4, tb_M=256 -- reached when every
    # remote group has one row more than a multiple of tb_M.  Algorithm 1 pads per expert per remote rank.
    W, tb = 4, 256
    counts, sr, st = [], [], []
    for e in range(2):
        c = 0
        for r in range(W):
            nrows = 257 if r != 0 else 300
            sr += [r] * nrows
            st += list(range(nrows))
            c += nrows
        counts.append(c)
    plan = build_plan(counts, sr, st, W, 0, tb, 1, 1)
    for e in range(2):
        pad = sum(tb - b.valid for b in plan.bands if b.expert == e and not b.local)
        assert pad == (W - 1) * (tb - 1) == 765
    # and never exceeded on random routing
    for name in ("tiny", "small", "small_zipf_rot"):
        shape = I.SHAPES[name]
        _, dsp, p = _plan_for(shape)
        for e in range(shape.El):
            pad = sum(128 - b.valid for b in p.bands if b.expert == e and not b.local)
            assert pad <= (shape.R - 1) * 127
        assert p.P - dsp.M <= shape.El * shape.R * 127 and p.P % 128 == 0


def test_rows_received_table2():
    # Table 2: with top-2 routing a rank's GEMM has M = 2 x tokens-per-rank rows on average, i.e. the
    # ranks together receive exactly k * R * T routed copies.
    base = I.SHAPES["tiny"]
    inp = I.make_inputs(base, weights=False)
    total = 0
    for first in range(0, base.Eg, base.El):
        sh = I.MoEShape(**{**base.__dict__, "first_local": first})
        total += I.dispatch(I.MoEInputs(sh, inp.x, inp.w1, inp.w2, inp.expert, inp.gate), gather_x=False).M
    assert total == base.k * base.R * base.T
    per_rank = total / (base.Eg // base.El)
    assert per_rank == 2 * base.T * base.R / (base.Eg // base.El)


def _check_schedule_rules(plan, R, r_self, tiles_per_band):
    bands = {b.band: b for b in plan.bands}
    # every tile exactly once
    assert sorted(plan.tiles) == sorted((b.expert, b.band, j) for b in plan.bands for j in range(tiles_per_band))
    local_flags = [bands[b].local for (_, b, _) in plan.tiles]
    first_local = local_flags.index(True) if True in local_flags else len(local_flags)
    assert not any(local_flags[:first_local]) and all(local_flags[first_local:])       # rule (i)
    remote_experts = [e for (e, b, _) in plan.tiles[:first_local]]
    runs = [e for i, e in enumerate(remote_experts) if i == 0 or remote_experts[i - 1] != e]
    assert len(runs) == len(set(runs))                                                  # contiguous per expert
    rb = {e: sum(1 for b in plan.bands if b.expert == e and not b.local) for e in range(len(plan.n))}
    keys = [rb[e] for e in runs]
    assert keys == sorted(keys, reverse=True)                                           # rule (ii)
    assert plan.expert_order == sorted(rb, key=lambda e: (-rb[e], e))
    # inside an expert's remote run: destination ranks ascending, bands ascending
    for e in runs:
        seq = [(bands[b].dest, b) for (ee, b, j) in plan.tiles[:first_local] if ee == e and j == 0]
        assert seq == sorted(seq)
    # local phase in natural expert order
    loc = [e for (e, b, j) in plan.tiles[first_local:] if j == 0]
    assert loc == sorted(loc)


def test_schedule_example_section_3_2_2():
    # Section 3.2.2's example: 4 ranks, 2 experts per rank; the expert with the heavier remote load runs
    # first, then the other expert's remote tiles, then all local tiles.
    R, r_self, tb = 4, 1, 4
    counts, sr, st = [], [], []
    per = {0: {0: 3, 1: 5, 2: 2, 3: 4}, 1: {0: 9, 1: 2, 2: 6, 3: 8}}    # rows of expert e from rank r
    for e in (0, 1):
        c = 0
        for r in range(R):
            sr += [r] * per[e][r]
            st += list(range(per[e][r]))
            c += per[e][r]
        counts.append(c)
    plan = build_plan(counts, sr, st, R, r_self, tb, 1, 3)
    assert plan.expert_order == [1, 0]
    seq = [(e, plan.bands[b].local) for (e, b, j) in plan.tiles if j == 0]
    assert seq == [(1, False)] * 7 + [(0, False)] * 3 + [(0, True)] * 2 + [(1, True)] * 1
    _check_schedule_rules(plan, R, r_self, 3)


@pytest.mark.parametrize("name", ["tiny", "tiny_zipf", "small", "small_zipf_rot"])
def test_schedule_rules_random(name):
    shape = I.SHAPES[name]
    _, _, plan = _plan_for(shape, mgb=2)
    _check_schedule_rules(plan, shape.R, shape.self_rank, max(1, shape.d // 256))
    # segments partition every group's bands in schedule order; one destination each
    seg_bands = [b for s in plan.segments for b in range(s.first_band, s.first_band + s.nbands)]
    assert seg_bands == plan.band_order
    for s in plan.segments:
        bs = [plan.bands[b] for b in range(s.first_band, s.first_band + s.nbands)]
        assert {b.dest for b in bs} == {s.dest} and len({b.expert for b in bs}) == 1
        assert s.rows == sum(b.valid for b in bs) and s.slot0 == bs[0].slot0 and s.pos0 == bs[0].pos0
        assert all(b.valid == 128 for b in bs[:-1])            # only a group's last band is ragged
    assert sum(plan.segs_per_rank) == len(plan.segments)


def test_edge_cases():
    # no rows at all; one expert with a single row; an empty expert between two loaded ones
    p = build_plan([0, 0], [], [], 2, 0, 128, 1, 1)
    assert p.P == 0 and p.bands == [] and p.tiles == [] and p.segs_per_rank == [0, 0]
    p = build_plan([1], [0], [7], 1, 0, 128, 1, 2)
    assert p.P == 128 and p.pos == [0] and p.slot == [0] and p.bands[0].local and len(p.tiles) == 2
    p = build_plan([2, 0, 1], [1, 0, 1], [4, 4, 4], 2, 0, 128, 1, 1)
    assert p.pos == [0, 128, 256] and p.slot == [0, 0, 1] and p.expert_base == [0, 256, 256, 384]
    assert p.band_order == [0, 2, 1] and p.expert_order == [0, 2, 1]

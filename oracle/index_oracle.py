"""CPU oracle for the integer part of the path: row layout, schedule, combine plan.

TEST INFRASTRUCTURE ONLY.  Nothing on the product path may import this file;
only tests, the smoke check and the benchmark's CPU-baseline leg do.  It shares
no code with the CUDA path.

Plain Python loops in the order of Algorithm 1 ("Remote-owner-aligned Row
Layout and Remote-first Tile Schedule Construction"), Section 3.2.3 (combine
plan) and Section 3.3.2 / Figure 3b (segment composition).  Readings taken
where the paper is silent (each is also listed in the design notes):

* remote groups are laid out in ascending rank order, the local group last
  (Algorithm 1, the "append G_0 .. G_{R-1}, remote first, G_self last" step);
* rows inside an owner group are ordered by (src_token, input row index);
* every group, the local one included, is rounded up to a multiple of tb_M so
  that each expert starts on a band boundary of one concatenated buffer; the
  positions of valid rows inside a group do not depend on this;
* the expert sort key is the remote row-BAND count (Algorithm 1), ties go to
  the lower expert index; the local phase visits experts in natural order;
* receive-buffer slots are expert-major (ascending local expert), dense, with
  no padding (Section 3.2.1: padded rows are excluded from the transfer;
  Section 3.2.3: offsets of different experts to one peer do not overlap);
* segments never span an (expert, destination) group because a segment is one
  contiguous write to one rank; a group of nb <= 2 bands gives nb one-band
  segments, otherwise [1] + chunks of mgb bands (the last chunk takes the
  remainder) + [1];
* the local rank has a receive region too, so ret[r][slot[i]] is defined for
  every row; local bands stay last in the schedule and are marked local.

Pins (tests/test_oracle_index.py): a hand-derived worked example stored under
tests/golden/, the permutation round trip, the paper's padding bound
(W-1)(tb_M-1) = 765 for W=4, tb_M=256 (Section 4.5), M = 2 x tokens-per-rank for
top-2 (Table 2), the schedule rules of Section 3.2.2, and brute-force
enumeration of segment shapes.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import List, Sequence, Tuple


@dataclass
class Band:
    band: int        # band id = first position // tb_M (bands tile the aligned buffer)
    expert: int
    dest: int        # owner rank of every valid row of the band (Section 3.2.1)
    pos0: int        # first aligned position
    valid: int       # valid (non-padding) rows, 1..tb_M
    slot0: int       # receive-buffer slot of the band's first row (Section 3.2.3)
    local: bool      # local-only (dest == r_self) vs remote-publishable


@dataclass
class Segment:
    first_band: int  # band id of the first band
    nbands: int
    dest: int
    pos0: int
    slot0: int
    rows: int
    local: bool


@dataclass
class Plan:
    n: List[List[int]]                 # n[e][r] rows of expert e owned by rank r
    rows_per_rank: List[int]
    expert_base: List[int]             # aligned position where X_e starts; [El] = P
    P: int                             # padded rows in total (multiple of tb_M)
    pos: List[int]                     # aligned position of every input row
    slot: List[int]                    # receive-buffer slot of every input row
    bands: List[Band]                  # in layout order (ascending band id)
    expert_order: List[int]            # experts by remote band count, descending
    band_order: List[int]              # band ids in schedule order
    tiles: List[Tuple[int, int, int]]  # schedule S: (expert, band id, n-tile)
    segments: List[Segment]            # in schedule order
    segs_per_rank: List[int]
    tok_slot: List[List[int]] = field(default_factory=list)    # per token (r*T+t): slots, ascending expert
    tok_gate: List[List[float]] = field(default_factory=list)  # matching gates


def ceil_to(v: int, m: int) -> int:
    return (v + m - 1) // m * m


def segment_band_counts(nb: int, mgb: int) -> List[int]:
    """Band count of each segment of a group of nb bands (Figure 3b): first and
    last segment one band, middle segments mgb bands, remainder in the last middle one."""
    if nb <= 2:
        return [1] * nb
    out = [1]
    left = nb - 2
    while left > 0:
        take = min(mgb, left)
        out.append(take)
        left -= take
    out.append(1)
    return out


def build_plan(expert_counts: Sequence[int], src_rank: Sequence[int], src_token: Sequence[int],
               R: int, r_self: int, tb_M: int, mgb: int, tiles_per_band: int,
               gate: Sequence[float] = (), T: int = 0) -> Plan:
    E = len(expert_counts)
    M = int(sum(expert_counts))
    assert len(src_rank) == M and len(src_token) == M

    # expert of every input row: rows arrive grouped by local expert
    row_expert: List[int] = []
    for e in range(E):
        row_expert += [e] * int(expert_counts[e])

    # ---- Algorithm 1, row layout -------------------------------------------------
    rank_order = [r for r in range(R) if r != r_self] + [r_self]     # remote first, G_self last
    n = [[0] * R for _ in range(E)]
    pos = [-1] * M
    rank_in_group = [-1] * M
    group_start = [[0] * R for _ in range(E)]
    expert_base = [0] * (E + 1)
    cursor = 0
    for e in range(E):
        expert_base[e] = cursor
        for r in rank_order:
            G_r = _rows_of(e, r, expert_counts, src_rank)           # rows from rank r routed to e
            G_r.sort(key=lambda i: (src_token[i], i))
            n[e][r] = len(G_r)
            group_start[e][r] = cursor
            for q, i in enumerate(G_r):
                pos[i] = cursor + q
                rank_in_group[i] = q
            cursor += ceil_to(len(G_r), tb_M)      # pad up to the next tb_M multiple
    expert_base[E] = cursor
    P = cursor

    # ---- Section 3.2.3, receive-buffer slots: expert-major, dense -----------------
    rows_per_rank = [sum(n[e][r] for e in range(E)) for r in range(R)]
    slot_base = [[sum(n[e2][r] for e2 in range(e)) for r in range(R)] for e in range(E)]
    slot = [slot_base[row_expert[i]][src_rank[i]] + rank_in_group[i] for i in range(M)]

    # ---- bands of every group ----------------------------------------------------
    bands: List[Band] = []
    group_bands = [[[] for _ in range(R)] for _ in range(E)]
    for e in range(E):
        for r in rank_order:
            nb = ceil_to(n[e][r], tb_M) // tb_M
            for b in range(nb):
                p0 = group_start[e][r] + b * tb_M
                band = Band(p0 // tb_M, e, r, p0, min(tb_M, n[e][r] - b * tb_M),
                            slot_base[e][r] + b * tb_M, r == r_self)
                group_bands[e][r].append(band)
                bands.append(band)
    bands.sort(key=lambda b: b.band)

    # ---- Algorithm 1, remote-first tile schedule ---------------------------------
    remote_bands = [sum(len(group_bands[e][r]) for r in range(R) if r != r_self) for e in range(E)]
    expert_order = sorted(range(E), key=lambda e: (-remote_bands[e], e))   # rule (ii)
    band_order: List[int] = []
    groups_in_schedule: List[Tuple[int, int]] = []
    for e in expert_order:                                                # rule (i): remote tiles first
        for r in rank_order[:-1]:
            band_order += [b.band for b in group_bands[e][r]]
            groups_in_schedule.append((e, r))
    for e in range(E):                                                    # then local tiles
        band_order += [b.band for b in group_bands[e][r_self]]
        groups_in_schedule.append((e, r_self))
    band_expert = {b.band: b.expert for b in bands}
    tiles = [(band_expert[b], b, j) for b in band_order for j in range(tiles_per_band)]

    # ---- Section 3.3.2, segments -------------------------------------------------
    segments: List[Segment] = []
    segs_per_rank = [0] * R
    for (e, r) in groups_in_schedule:
        gb = group_bands[e][r]
        at = 0
        for cnt in segment_band_counts(len(gb), mgb):
            part = gb[at:at + cnt]
            segments.append(Segment(part[0].band, cnt, r, part[0].pos0, part[0].slot0,
                                    sum(b.valid for b in part), r == r_self))
            segs_per_rank[r] += 1
            at += cnt

    plan = Plan(n, rows_per_rank, expert_base, P, pos, slot, bands, expert_order, band_order, tiles,
                segments, segs_per_rank)

    # ---- per-token lists for the owner-side weighted reduction (Section 2.1 step 5)
    if T > 0 and len(gate) == M:
        plan.tok_slot = [[] for _ in range(R * T)]
        plan.tok_gate = [[] for _ in range(R * T)]
        for i in range(M):                     # rows are grouped by ascending expert already
            tok = src_rank[i] * T + src_token[i]
            plan.tok_slot[tok].append(slot[i])
            plan.tok_gate[tok].append(float(gate[i]))
    return plan


def _rows_of(e: int, r: int, expert_counts: Sequence[int], src_rank: Sequence[int]) -> List[int]:
    """Input rows of local expert e (a contiguous range: rows arrive grouped by expert) owned by rank r."""
    lo = int(sum(expert_counts[:e]))
    hi = lo + int(expert_counts[e])
    return [i for i in range(lo, hi) if src_rank[i] == r]

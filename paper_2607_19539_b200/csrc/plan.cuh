// Plan kernels: remote-owner-aligned row layout and remote-first tile schedule
// (Algorithm 1), combine plan (Section 3.2.3), segments (Section 3.3.2, Figure 3b), the
// item list the GEMM kernel follows, and the maps its gather warps need.
//
// All integer work.  Rank-in-group is found without sorting: a routed copy is
// identified by (expert, owner rank, token), so every (expert, rank) group gets a
// bitmap over the T tokens of that rank; the rank of a row inside its group (rows
// in source-token order) is the number of set bits below its token.
#pragma once

#include "common.cuh"

namespace moe_ovl {

constexpr int PLAN_MAX_GROUPS = 1024;   // El * R
constexpr int PLAN_MAX_EXPERTS = 256;   // El
constexpr int PLAN_THREADS = 1024;
constexpr int PLAN_SB_STAGE = 256;      // super-bands whose sizes are staged in shared memory for the serial pass

// Scratch arrays of the plan kernel, one entry per super-band.
struct PlanScratch {
    int *sb_start;   // first schedule position
    int *sb_nb;      // bands
    int *sb_expert;
    int *sb_g1off;   // item index of the super-band's first-GEMM block
    int *sb_g2off;   // item index of its second-GEMM block
    int *sb_g1end;
    int *sb_kind;    // 0: band pairs (KIND_G1 / KIND_G2 items), 1: one group of small bands (KIND_G1S / KIND_G2S)
    int *sb_ntok;    // group of small bands: valid rows, each band rounded up to 16
    int *sb_c1;      // items of the super-band's first-GEMM block
    int *sb_c2;      // ... of its second-GEMM block
    int *sb_units;   // super-band of band pairs: its units (a pair, or two pairs of small bands stacked)
    int *unit_tab;   // [bands], a super-band's units at its first schedule position: first band's offset | bands << 8
                     // | (1 << 16 if the unit's last band is the expert's local band riding with its remote ones)
    int *sb_role;    // bits 0-1: 1 last super-band of an expert's remote run, 2 super-band of a local run, else 0;
                     // bit 2: the run may hold stacks of small bands or take a rider (its units are in unit_tab)
};

__device__ __forceinline__ int ceil16(int v) { return (v + 15) & ~15; }

__device__ __forceinline__ int expert_of_row(const int *pre, int El, int i)
{
    // pre[e] = first row of expert e, pre[El] = total; largest e with pre[e] <= i
    int lo = 0, hi = El;
    while (hi - lo > 1) {
        int mid = (lo + hi) >> 1;
        if (pre[mid] <= i) lo = mid; else hi = mid;
    }
    return lo;
}

__device__ __forceinline__ void load_expert_prefix(const Params &p, int *pre)
{
    if (threadIdx.x == 0) {
        int acc = 0;
        for (int e = 0; e < p.El; ++e) {
            pre[e] = acc;
            acc += p.expert_counts[e];
        }
        pre[p.El] = acc;
    }
    __syncthreads();
}

// ---- step 1: mark (expert, rank, token) of every row ---------------------------------------
__device__ __forceinline__ void plan_mark(const Params &p, const int *pre)
{
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= p.M) return;
    if (i >= pre[p.El]) {
        report_error(p.status, ERR_BAD_ROUTING, SITE_COUNT_SUM, i);
        return;
    }
    const int e = expert_of_row(pre, p.El, i);
    const int r = p.src_rank[i], t = p.src_token[i];
    if (r < 0 || r >= p.R || t < 0 || t >= p.T) {
        report_error(p.status, ERR_BAD_ROUTING, SITE_ROW_RANGE, i);
        return;
    }
    const unsigned bit = 1u << (t & 31);
    const unsigned old = atomicOr(&p.bitmap[(size_t)(e * p.R + r) * p.words + (t >> 5)], bit);
    if (old & bit) report_error(p.status, ERR_BAD_ROUTING, SITE_ROW_DUP, i);
}

__device__ __forceinline__ int num_segments(int nb, int mgb)
{
    return nb <= 2 ? nb : 2 + (nb - 2 + mgb - 1) / mgb;
}

// ---- step 2: everything that is per group / band / segment / schedule item -------------------
// One launch does both steps: every block marks its rows, and the block that finishes last (ticket counter)
// builds the plan, which needs all marks.
__global__ void __launch_bounds__(PLAN_THREADS, 1) plan_mark_build_kernel(Params p, PlanScratch sc)
{
    __shared__ int pre[PLAN_MAX_EXPERTS + 1];
    __shared__ int s_last;
    load_expert_prefix(p, pre);
    plan_mark(p, pre);
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) s_last = atomicAdd(p.plan_ticket, 1) == (int)gridDim.x - 1;
    __syncthreads();
    if (!s_last) return;
    __threadfence();
    // A new call: its ready flags carry a new number.  Kept in device memory (not passed by value) so that a
    // captured call can be replayed.
    if (threadIdx.x == 0) *p.epoch_rw += 1u;

    __shared__ int n[PLAN_MAX_GROUPS], nb[PLAN_MAX_GROUPS], gstart[PLAN_MAX_GROUPS], gslot[PLAN_MAX_GROUPS];
    __shared__ int gsched[PLAN_MAX_GROUPS], gsegoff[PLAN_MAX_GROUPS];
    __shared__ int key[PLAN_MAX_EXPERTS], eorder[PLAN_MAX_EXPERTS];
    __shared__ int run_start[2 * PLAN_MAX_EXPERTS], run_nb[2 * PLAN_MAX_EXPERTS], run_sb0[2 * PLAN_MAX_EXPERTS + 1];
    __shared__ int run_exp[2 * PLAN_MAX_EXPERTS], run_segs[2 * PLAN_MAX_EXPERTS];
    __shared__ int run_nsb[2 * PLAN_MAX_EXPERTS];     // groups of small bands in the run, or -1: issued as band pairs
    __shared__ int esize[PLAN_MAX_EXPERTS];
    __shared__ int s_total;
    __shared__ int segs_per_rank[PLAN_MAX_GROUPS];
    __shared__ int s_nsb;
    __shared__ int s_any_rider, s_riders;
    __shared__ int s_sb_c1[PLAN_SB_STAGE], s_sb_c2[PLAN_SB_STAGE], s_sb_end[PLAN_SB_STAGE];
    __shared__ unsigned char erider[PLAN_MAX_EXPERTS];   // the expert's local band rides with its last remote bands

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, nwarps = blockDim.x >> 5;
    const int G = p.El * p.R;
    const int R = p.R, El = p.El, self = p.r_self;

    // A: per group, exclusive popcount prefix over its bitmap words, and n[e][r].  A warp works on four groups
    //    at a time so that their (independent) loads are in flight together.
    for (int g0 = warp * 4; g0 < G; g0 += nwarps * 4) {
        int run[4] = {0, 0, 0, 0};
        // four steps of 32 words per round, all sixteen loads issued before the first scan: one trip to L2 per
        // round instead of one per step
        for (int w0 = 0; w0 < p.words; w0 += 128) {
            int c[4][4];
#pragma unroll
            for (int s = 0; s < 4; ++s) {
                const int w = w0 + 32 * s + lane;
#pragma unroll
                for (int k = 0; k < 4; ++k)     // written by other blocks' atomics: read through L2
                    c[s][k] = (g0 + k < G && w < p.words) ? __popc(__ldcg(p.bitmap + (size_t)(g0 + k) * p.words + w)) : 0;
            }
#pragma unroll
            for (int s = 0; s < 4; ++s) {
                const int w = w0 + 32 * s + lane;
                if (w0 + 32 * s >= p.words) break;          // uniform
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    int inc = c[s][k];
#pragma unroll
                    for (int o = 1; o < 32; o <<= 1) {
                        const int v = __shfl_up_sync(0xffffffffu, inc, o);
                        if (lane >= o) inc += v;
                    }
                    if (g0 + k < G && w < p.words) p.wordpfx[(size_t)(g0 + k) * p.words + w] = run[k] + inc - c[s][k];
                    run[k] += __shfl_sync(0xffffffffu, inc, 31);
                }
            }
        }
#pragma unroll
        for (int k = 0; k < 4; ++k)
            if (lane == 0 && g0 + k < G) n[g0 + k] = run[k];
    }
    for (int r = tid; r < R; r += blockDim.x) segs_per_rank[r] = 0;
    __syncthreads();

    // B: row layout (Algorithm 1): per expert, remote owner groups in ascending rank, local group last,
    //    every group rounded up to a multiple of tb_M; receive-buffer slots expert-major and dense.
    //    One thread per expert lays out its own groups relative to the expert's start; a short prefix over
    //    the experts then places the experts.
    if (tid == 0) { s_total = 0; s_any_rider = 0; }
    __syncthreads();
    for (int e = tid; e < El; e += blockDim.x) {
        int cur = 0, remote_bands = 0, rows = 0;
        for (int q = 0; q < R; ++q) {
            const int r = q < R - 1 ? (q < self ? q : q + 1) : self;   // remote ranks ascending, then self
            const int g = e * R + r;
            const int nbg = (n[g] + TB_M - 1) / TB_M;
            gstart[g] = cur;
            nb[g] = nbg;
            cur += nbg * TB_M;
            rows += n[g];
            if (r != self) remote_bands += nbg;
        }
        key[e] = remote_bands;
        esize[e] = cur;
        atomicAdd(&s_total, rows);
    }
    for (int r = tid; r < R; r += blockDim.x) {
        int acc = 0;
        for (int e = 0; e < El; ++e) {
            gslot[e * R + r] = acc;
            acc += n[e * R + r];
        }
        if (p.rows_per_rank_out) p.rows_per_rank_out[r] = acc;
        // Only malformed routing (a token in more than min(k, El) local experts) can ask for more rows than
        // the rank's receive region holds.  It is reported here; the copies below skip what does not fit.
        if (acc > p.ret_rows_per_rank) report_error(p.status, ERR_BAD_ROUTING, SITE_RET_OVERFLOW, r);
    }
    __syncthreads();
    if (tid == 0) {
        int cursor = 0;
        for (int e = 0; e < El; ++e) {
            const int sz = esize[e];
            esize[e] = cursor;                 // now the expert's first aligned position
            cursor += sz;
        }
        p.meta[META_P] = cursor;
        p.meta[META_BANDS] = cursor / TB_M;
        if (s_total != p.M) report_error(p.status, ERR_BAD_ROUTING, SITE_COUNT_SUM, s_total);
    }
    __syncthreads();
    for (int g = tid; g < G; g += blockDim.x) gstart[g] += esize[g / R];

    // C: experts by remote band count, descending; ties to the lower index (Algorithm 1, rule (ii))
    for (int e = tid; e < El; e += blockDim.x) {
        int rank = 0;
        for (int o = 0; o < El; ++o) rank += (key[o] > key[e]) || (key[o] == key[e] && o < e);
        eorder[rank] = e;
    }
    __syncthreads();
    // key[] is free now: it becomes the inverse of eorder (position of an expert among the remote runs)
    for (int i = tid; i < El; i += blockDim.x) key[eorder[i]] = i;

    // D: schedule positions of groups.  Runs: the remote bands of each expert in sorted order (rule (i):
    //    all remote tiles first), then the local bands of each expert in natural order.  One thread per run
    //    counts its bands, segments and super-bands; a short prefix over the runs places them.
    for (int run = tid; run < 2 * El; run += blockDim.x) {
        const bool remote = run < El;
        const int e = remote ? eorder[run] : run - El;
        int nbands = 0, nsegs = 0;
        // A run whose groups all fit in half a band is issued as groups of small bands with swapped operands:
        // consecutive bands while their rows, each band rounded up to 16, stay within SWAP_MAX_N.
        bool small = p.swap_ok != 0;
        int sgroups = 0, acc_tok = SWAP_MAX_N + 1;
        for (int q = remote ? 0 : R - 1; q < (remote ? R - 1 : R); ++q) {
            const int r = q < R - 1 ? (q < self ? q : q + 1) : self;
            const int g = e * R + r;
            gsched[g] = nbands;                 // relative to the run for now
            gsegoff[g] = nsegs;
            const int ns = num_segments(nb[g], p.mgb);
            nbands += nb[g];
            nsegs += ns;
            atomicAdd(&segs_per_rank[r], ns);
            small = small && n[g] <= SMALL_BAND_ROWS;
            if (n[g] > 0) {
                if (acc_tok + ceil16(n[g]) > SWAP_MAX_N) { ++sgroups; acc_tok = 0; }
                acc_tok += ceil16(n[g]);
            }
        }
        run_exp[run] = e;
        run_nb[run] = nbands;
        run_segs[run] = nsegs;
        // Worth it only if the groups cost less tensor-pipe time than the band pairs they replace: an MMA over 256
        // weight rows against one group of tokens costs what an MMA over two full bands of tokens costs, and twice
        // what a pair of small bands costs when those are issued 64 rows high (KIND_LOW).  (swap_ok == 2: a test
        // hook that takes every eligible run.)
        const int pairs_run = (nbands + 1) / 2;
        const bool fewer = (p.low_ok ? 2 * sgroups < pairs_run : sgroups < pairs_run) || p.swap_ok == 2;
        run_nsb[run] = (small && nbands > 0 && fewer) ? sgroups : -1;
        // Can the run hold a stack of small bands or take a rider?  Only the last band of a group can be small, so a
        // stack needs three single-band groups in a row, and a rider the run's last band small.  (Decided exactly,
        // band by band, in phase E2; runs that cannot are skipped there.)
        int chain = 0, best = 0;
        bool last_small = false;
        for (int q = remote ? 0 : R - 1; q < (remote ? R - 1 : R); ++q) {
            const int r = q < R - 1 ? (q < self ? q : q + 1) : self;
            const int g = e * R + r;
            if (nb[g] == 0) continue;
            last_small = n[g] - (nb[g] - 1) * TB_M <= SMALL_BAND_ROWS;
            chain = (nb[g] == 1 && last_small) ? chain + 1 : 0;
            best = max(best, chain);
        }
        const int n_local = n[e * R + self];
        const bool may_ride = remote && last_small && n_local > 0 && n_local <= SMALL_BAND_ROWS;
        if (run_nsb[run] < 0 && !(p.low_ok >= 2 && (best >= 3 || may_ride))) run_nsb[run] = -2;
    }
    __syncthreads();
    if (tid == 0) {
        // Groups make fewer, longer items than band pairs.  That pays when there are at least two such items per CTA pair;
        // with few, the pairs that find no item idle while the long items run, and band pairs are faster.
        int group_items = 0;
        for (int run = 0; run < 2 * El; ++run)
            if (run_nsb[run] >= 0) group_items += run_nsb[run] * (p.n1 / 2 + p.n2);
        if (group_items < p.lag_items && p.swap_ok != 2)
            for (int run = 0; run < 2 * El; ++run)
                if (run_nsb[run] >= 0) run_nsb[run] = p.low_ok >= 2 ? -1 : -2;
        int spos = 0, segoff = 0, sbcount = 0;
        for (int run = 0; run < 2 * El; ++run) {
            run_start[run] = spos;
            spos += run_nb[run];
            const int nsegs = run_segs[run];
            run_segs[run] = segoff;             // now the run's first segment
            segoff += nsegs;
            run_sb0[run] = sbcount;
            // super-bands are made of whole band pairs (the GEMM works on two bands at a time); a run of small
            // bands has one super-band per group instead
            const int pairs = (run_nb[run] + 1) / 2, pairs_per_sb = max(1, p.group_bands / 2);
            sbcount += run_nsb[run] >= 0 ? run_nsb[run] : (pairs + pairs_per_sb - 1) / pairs_per_sb;
        }
        run_sb0[2 * El] = sbcount;
        s_nsb = sbcount;
        p.meta[META_SEGS] = segoff;
        p.meta[META_SUPERBANDS] = sbcount;
    }
    __syncthreads();
    for (int run = tid; run < 2 * El; run += blockDim.x) {
        const bool remote = run < El;
        const int e = run_exp[run];
        for (int q = remote ? 0 : R - 1; q < (remote ? R - 1 : R); ++q) {
            const int r = q < R - 1 ? (q < self ? q : q + 1) : self;
            const int g = e * R + r;
            gsched[g] += run_start[run];
            gsegoff[g] += run_segs[run];
        }
    }
    __syncthreads();

    // E: band table, schedule order of bands, segments, super-bands
    for (int g = warp; g < G; g += nwarps) {
        const int e = g / R, r = g % R;
        for (int b = lane; b < nb[g]; b += 32) {
            const int band = gstart[g] / TB_M + b;
            p.band_expert[band] = e;
            p.band_dest[band] = r;
            p.band_valid[band] = min(TB_M, n[g] - b * TB_M);
            p.band_slot0[band] = gslot[g] + b * TB_M;
            p.sched_band[gsched[g] + b] = band;
            p.hcount[band] = 0;
            p.xready[band] = 0;
        }
        const int ns = num_segments(nb[g], p.mgb);
        for (int q = lane; q < ns; q += 32) {
            int first, cnt;
            if (nb[g] <= 2 || q == 0) { first = q; cnt = 1; }
            else if (q == ns - 1) { first = nb[g] - 1; cnt = 1; }
            else { first = 1 + (q - 1) * p.mgb; cnt = min(p.mgb, nb[g] - 1 - first); }
            const int rows = min(n[g] - first * TB_M, cnt * TB_M);
            p.segs[gsegoff[g] + q] = make_int4(gstart[g] / TB_M + first, cnt, r, rows);
            p.seg_slot0[gsegoff[g] + q] = gslot[g] + first * TB_M;
        }
        if (lane == 0) p.group_rows[g] = n[g];
        if (lane == 1) p.group_start[g] = gstart[g];
        if (lane == 2) p.group_slot[g] = gslot[g];
    }
    for (int r = tid; r < R; r += blockDim.x)
        if (p.segs_per_rank_out) p.segs_per_rank_out[r] = segs_per_rank[r];
    for (int run = tid; run < 2 * El; run += blockDim.x) {
        const int nsb = run_sb0[run + 1] - run_sb0[run];
        const int pairs = (run_nb[run] + 1) / 2;
        if (run_nsb[run] >= 0) {
            // one super-band per group of small bands; every group of the run holds at most one band, so the
            // run's bands are its non-empty groups in layout order
            const bool remote = run < El;
            const int e = run_exp[run];
            int sb = run_sb0[run] - 1, acc_tok = SWAP_MAX_N + 1, pos = run_start[run];
            for (int q = remote ? 0 : R - 1; q < (remote ? R - 1 : R); ++q) {
                const int r = q < R - 1 ? (q < self ? q : q + 1) : self;
                const int g = e * R + r;
                if (n[g] == 0) continue;
                if (acc_tok + ceil16(n[g]) > SWAP_MAX_N) {
                    ++sb;
                    acc_tok = 0;
                    sc.sb_start[sb] = pos;
                    sc.sb_nb[sb] = 0;
                    sc.sb_expert[sb] = e;
                    sc.sb_kind[sb] = 1;
                    sc.sb_c1[sb] = p.n1 / 2;          // tiles of 256 hidden columns
                    sc.sb_c2[sb] = p.n2;
                }
                acc_tok += ceil16(n[g]);
                sc.sb_nb[sb] += 1;
                sc.sb_ntok[sb] = acc_tok;
                ++pos;
            }
            continue;
        }
        for (int q = 0; q < nsb; ++q) {
            // spread the run's band pairs evenly; only the run's last super-band can end on a single band
            const int base = pairs / nsb, rem = pairs % nsb;
            const int sb = run_sb0[run] + q;
            const int pair0 = q * base + min(q, rem), npairs = base + (q < rem ? 1 : 0);
            sc.sb_start[sb] = run_start[run] + 2 * pair0;
            sc.sb_nb[sb] = min(2 * npairs, run_nb[run] - 2 * pair0);
            sc.sb_expert[sb] = run_exp[run];
            sc.sb_kind[sb] = 0;
            sc.sb_ntok[sb] = 0;
            sc.sb_role[sb] = (run >= El ? 2 : (q == nsb - 1 ? 1 : 0)) | (run_nsb[run] == -1 ? 4 : 0);
            sc.sb_units[sb] = (sc.sb_nb[sb] + 1) / 2;      // band pairs, unless phase E2 finds stacks or a rider
        }
    }
    for (int e = tid; e < El; e += blockDim.x) erider[e] = 0;
    __syncthreads();

    // E2: the units of every super-band of band pairs.  A unit is one schedule item per tile: a band pair, or --
    //     where two neighbouring pairs hold only bands of at most SMALL_BAND_ROWS valid rows -- those three or four
    //     bands stacked into one full-height item (KIND_STACK), which costs the tensor pipe what ONE pair costs.
    //     Rider: where the LAST unit of an expert's remote run holds at most three bands, all small, and the expert's
    //     local rows are one small band, that band joins the unit -- it takes rows of the item that would otherwise
    //     be padding, so no remote tile is issued later than without it (the purpose of rule (i) of Section 3.2.2
    //     holds), and the expert's weights are streamed once instead of twice.  The bands of an expert are
    //     consecutive in the layout, remote ones first, so the unit's bands still have consecutive ids.
    //     One warp per super-band of a run that can hold such units (the others keep plain pairs): the lanes look the
    //     bands' row counts up together, lane 0 then forms the units from a bit mask.
    for (int sb = warp; sb < s_nsb; sb += nwarps) {
        const int role = sc.sb_role[sb];
        if (sc.sb_kind[sb] || !(role & 4)) continue;
        const int start = sc.sb_start[sb], cnt = sc.sb_nb[sb], e = sc.sb_expert[sb];
        unsigned long long small_mask = 0;      // bit o: band o of the super-band holds at most SMALL_BAND_ROWS rows
        for (int base = 0; base < min(cnt, 64); base += 32) {
            const int o = base + lane;
            const bool sm = o < cnt && p.band_valid[p.sched_band[start + o]] <= SMALL_BAND_ROWS;
            small_mask |= (unsigned long long)__ballot_sync(0xffffffffu, sm) << base;
        }
        if (lane != 0) continue;
        auto all_small = [&](int o, int k) {    // bands o .. o + k - 1 (beyond 64 bands per super-band: never stacked)
            return o + k <= 64 && ((small_mask >> o) & ((1ull << k) - 1)) == (1ull << k) - 1;
        };
        int units = 0, last_o = 0, last_take = 0;
        for (int o = 0; o < cnt;) {
            int take = min(2, cnt - o);
            if (p.low_ok >= 2 && cnt - o >= 3 && all_small(o, min(4, cnt - o))) take = min(4, cnt - o);
            sc.unit_tab[start + units++] = o | (take << 8);
            last_o = o;
            last_take = take;
            o += take;
        }
        const int n_local = n[e * R + self];
        if (p.low_ok == 3 && (role & 3) == 1 && units > 0 && last_take <= 3 && n_local > 0 &&
            n_local <= SMALL_BAND_ROWS && run_nsb[El + e] < 0 && all_small(last_o, last_take)) {
            sc.unit_tab[start + units - 1] = last_o | ((last_take + 1) << 8) | (1 << 16);
            erider[e] = 1;
            s_any_rider = 1;
        }
        sc.sb_units[sb] = units;
    }
    __syncthreads();

    // F: issue order of tile blocks.  An item is a pair of bands times one tile.  Inside a super-band the tile
    //    index is the outer loop and the band pair the inner one, so that the CTA pairs working side by side
    //    share a weight tile.  The second-GEMM block of a super-band is issued lag_items items after its
    //    first-GEMM block, so that its input is normally complete when a CTA pair reaches it.
    //    (The loop is serial; band counts and block ends are staged in shared memory when they fit, so that
    //    each step costs shared-memory latency, not a round trip to L2.)
    {
        const int nsb = s_nsb;
        const bool staged = nsb <= PLAN_SB_STAGE;
        for (int i = tid; i < nsb; i += blockDim.x) {
            int c1 = sc.sb_c1[i], c2 = sc.sb_c2[i];
            const int kind = sc.sb_kind[i], role = sc.sb_role[i], e = sc.sb_expert[i];
            int units = sc.sb_units[i];
            if (!kind) {
                if ((role & 3) == 2 && erider[e]) units = 0;   // the band was issued with the remote ones
                sc.sb_units[i] = units;
                sc.sb_c1[i] = c1 = units * p.n1;
                sc.sb_c2[i] = c2 = units * p.n2;
            }
            if (staged) { s_sb_c1[i] = c1; s_sb_c2[i] = c2; }
        }
        __syncthreads();
        if (tid == 32 && s_any_rider) {
            // Riders change the order in which the GEMM needs the bands, so the gather follows them (below): how many
            // riders come before the i-th remote run, and before the local run of expert e.  (esize[] and eorder[]
            // are free by now; this thread works while thread 0 is in the serial loop.)
            int before = 0;
            for (int i = 0; i < El; ++i) { esize[i] = before; before += erider[run_exp[i]]; }
            s_riders = before;
            before = 0;
            for (int e = 0; e < El; ++e) { eorder[e] = before; before += erider[e]; }
        }
        if (tid == 0) {
            int *c1v = staged ? s_sb_c1 : sc.sb_c1, *c2v = staged ? s_sb_c2 : sc.sb_c2;
            int *endv = staged ? s_sb_end : sc.sb_g1end;
            // The schedule's last first-GEMM block must not be followed by its own second-GEMM block at once (every
            // CTA pair that claims one of its tiles would wait for the block's stragglers, and with few tiles most
            // pairs would idle meanwhile): the second-GEMM blocks of the last super-bands, as many whole blocks as
            // stay within one item per CTA pair (lag_items is two), are held back until every first-GEMM block
            // has been issued.  (More would only lengthen the run of long second-GEMM items at the very end.)
            int hold_from = nsb - 1;
            for (int acc = 0; hold_from > 0 && 2 * (acc + c2v[hold_from - 1]) <= p.lag_items;) acc += c2v[--hold_from];
            int ng1 = 0, off = 0;
            for (int ng2 = 0; ng2 < nsb; ++ng2) {
                while (ng1 < nsb && (ng1 <= ng2 || ng2 >= hold_from || off - endv[ng2] < p.lag_items)) {
                    sc.sb_g1off[ng1] = off;
                    off += c1v[ng1];
                    endv[ng1] = off;
                    ++ng1;
                }
                sc.sb_g2off[ng2] = off;
                off += c2v[ng2];
            }
            p.meta[META_ITEMS] = off;
        }
    }
    __syncthreads();

    // G: the item list.  A team of warps per super-band; the first lanes of every warp work out the super-band's
    //    units once (bands, height: a few dependent look-ups), every item is then a unit's record with a tile number.
    const int wps = max(1, min(8, nwarps / max(s_nsb, 1))), teams = nwarps / wps;
    for (int sb = warp / wps; sb < s_nsb && warp < teams * wps; sb += teams) {
        const int sub = warp % wps;
        const int start = sc.sb_start[sb], cnt = sc.sb_nb[sb], e = sc.sb_expert[sb];
        const int o1 = sc.sb_g1off[sb], o2 = sc.sb_g2off[sb];
        if (sc.sb_kind[sb]) {
            // group of small bands: {kind | expert << 8, first schedule position, bands | rows << 8, tile}
            const int c1 = sc.sb_c1[sb], desc = cnt | (sc.sb_ntok[sb] << 8);
            for (int idx = sub * 32 + lane; idx < c1 + p.n2; idx += 32 * wps) {
                const bool g1 = idx < c1;
                p.items[g1 ? o1 + idx : o2 + idx - c1] =
                    make_int4((g1 ? KIND_G1S : KIND_G2S) | (e << 8), start, desc, g1 ? idx : idx - c1);
            }
            continue;
        }
        const int nu = sc.sb_units[sb];                // at most 32: a super-band holds at most 64 bands
        const bool plain = !(sc.sb_role[sb] & 4);      // band pairs only: no table of units
        int ux = 0, uy = 0, uz = 0;                    // lane u: kind bits, first band, second band or band count of unit u
        if (lane < nu) {
            const int unit = plain ? (2 * lane) | (min(2, cnt - 2 * lane) << 8) : sc.unit_tab[start + lane];
            const int o = unit & 0xff, take = (unit >> 8) & 0xff;
            const bool rider = (unit >> 16) != 0;
            uy = p.sched_band[start + o];
            if (take > 2) {
                ux = KIND_STACK;                       // the bands of a run are consecutive in the layout: b0, b0 + 1, ...
                uz = take;
            } else {
                uz = take == 2 ? (rider ? uy + 1 : p.sched_band[start + o + 1]) : -1;
                const bool low = p.low_ok && p.band_valid[uy] <= SMALL_BAND_ROWS &&
                                 (uz < 0 || p.band_valid[uz] <= SMALL_BAND_ROWS);
                ux = low ? KIND_LOW : 0;
            }
        }
        const int total = nu * (p.n1 + p.n2);
        for (int base = sub * 32; base < total; base += 32 * wps) {
            const int idx = base + lane;
            const bool active = idx < total;
            const bool g1 = idx < nu * p.n1;
            const int k = g1 ? idx : idx - nu * p.n1;
            const int u = active ? k % nu : 0, tile = active ? k / nu : 0;
            const int x = __shfl_sync(0xffffffffu, ux, u), y = __shfl_sync(0xffffffffu, uy, u);
            const int z = __shfl_sync(0xffffffffu, uz, u);
            if (active) p.items[(g1 ? o1 : o2) + k] = make_int4((g1 ? KIND_G1 : KIND_G2) | x | (e << 8), y, z, tile);
        }
    }

    // H: the order in which the GEMM kernel's gather warps fill the layout.  It is the schedule order of the bands,
    //    except that a riding local band is needed with its expert's remote bands, long before its place in the
    //    schedule: it is gathered right after them.
    if (tid == 0) p.meta[META_GATHER_ORDER] = s_any_rider;
    if (s_any_rider) {
        for (int g = warp; g < G; g += nwarps) {
            const int e = g / R, r = g % R;
            for (int b = lane; b < nb[g]; b += 32) {
                const int spos = gsched[g] + b;
                int at;
                if (r != self) at = spos + esize[key[e]];
                else if (erider[e]) at = run_start[key[e]] + run_nb[key[e]] + esize[key[e]];
                else at = spos + s_riders - eorder[e];
                p.gather_band[at] = gstart[g] / TB_M + b;
            }
        }
    }
}

// ---- step 3: per row: aligned position, return slot, entry in its token's list, and the inverse map
//      (aligned position -> input row) that the GEMM kernel's gather warps follow.  One thread per row; the
//      rows themselves are moved by the GEMM kernel.
__global__ void __launch_bounds__(256) plan_rows_kernel(Params p)
{
    __shared__ int pre[PLAN_MAX_EXPERTS + 1];
    load_expert_prefix(p, pre);
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= p.M || i >= pre[p.El]) return;
    const int e = expert_of_row(pre, p.El, i);
    const int r = p.src_rank[i], t = p.src_token[i];
    if (r < 0 || r >= p.R || t < 0 || t >= p.T) return;
    const int g = e * p.R + r;
    const size_t w = (size_t)g * p.words + (t >> 5);
    const int q = p.wordpfx[w] + __popc(p.bitmap[w] & ((1u << (t & 31)) - 1u));
    const int pos = p.group_start[g] + q;
    const int slot = p.group_slot[g] + q;
    // entry of this row in its token's list: number of lower-indexed local experts the token also selected
    int j = 0;
    for (int o = 0; o < e; ++o)
        j += (p.bitmap[(size_t)(o * p.R + r) * p.words + (t >> 5)] >> (t & 31)) & 1u;
    p.pos[i] = pos;
    p.row_at[pos] = i;
    p.slot[i] = slot;
    if (p.slot_out) p.slot_out[i] = slot;
    if (j < p.kmax && slot < p.ret_rows_per_rank) {
        const size_t at = ((size_t)r * p.T + t) * p.kmax + j;
        p.tok_slot[at] = slot + 1;            // 0 (the cleared state) means "no row"
        p.tok_gate[at] = p.gate[i];
    } else {
        report_error(p.status, ERR_BAD_ROUTING, SITE_TOK_OVERFLOW, i);
    }
}

}  // namespace moe_ovl

// C-ABI entry points of moe_ovl (see include/moe_ovl.h): context, workspace layout,
// tensor maps, and the launch sequence of one pass.  Host code only orchestrates;
// every step of the path runs in the kernels of plan.cuh, producer.cuh, mover.cuh.
#include <cuda.h>
#include <cuda_runtime.h>

#include <algorithm>
#include <cstdio>
#include <cstring>
#include <new>

#include "../../include/moe_ovl.h"
#include "common.cuh"
#include "mover.cuh"
#include "plan.cuh"
#include "producer.cuh"

using namespace moe_ovl;

namespace {

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

constexpr size_t ALIGN = 1024;
constexpr int MAX_SEG_CHUNKS = 8;     // slices a segment is moved in when spare warps of GEMM CTAs move the return
inline size_t align_up(size_t v, size_t a = ALIGN) { return (v + a - 1) / a * a; }

struct Layout {
    // offsets into the workspace, in bytes
    size_t Xa, H, Y;
    size_t zero_begin, bitmap, hcount, fcount, status, next_item, stamps, tok_slot, zero_end;   // cleared at the start of every call
    size_t smid;
    size_t wordpfx, group_rows, group_start, group_slot, pos, slot, row_at, xready;
    size_t band_expert, band_dest, band_valid, band_slot0, sched_band, gather_band, items, segs, seg_slot0;
    size_t tok_gate, flags, meta;
    size_t trace_items, trace_items2, trace_units, trace_item_aux, trace_bytes;   // MOE_OVL_FLAG_TRACE
    size_t sb[13];
    // host staging (MOE_OVL_FLAG_HOST_STAGING)
    size_t st_x[2], st_counts[2], st_rank[2], st_token[2], st_gate[2], st_out[2], st_ret;   // two staging slots
    size_t total;
    int max_bands, max_items, words, kmax, n1, n2;
    int dout, k2, f_eff, single;
    long long st_ret_rows;
};

int check_config(const moe_ovl_config *c)
{
    if (!c || c->struct_size != sizeof(moe_ovl_config)) return MOE_OVL_ERR_INVALID_ARG;
    if (c->num_src_ranks < 1 || c->self_rank < 0 || c->self_rank >= c->num_src_ranks) return MOE_OVL_ERR_INVALID_ARG;
    if (c->tokens_per_rank < 1 || c->num_local_experts < 1 || c->top_k < 1) return MOE_OVL_ERR_INVALID_ARG;
    if (c->max_rows < 0 || c->mid_seg_bands < 0 || c->group_bands < 0 || c->wait_timeout_us < 0 ||
        c->producer_sm_limit < 0 || c->d_model < 1 || c->single_gemm_out < 0 ||
        (c->single_gemm_out == 0 && c->d_ffn < 1))
        return MOE_OVL_ERR_INVALID_ARG;
    if (c->single_gemm_out > 0) {
        if (c->d_model % TB_K != 0 || c->single_gemm_out % TB_N != 0) return MOE_OVL_ERR_UNSUPPORTED;
    } else if (c->d_model % TB_N != 0 || c->d_ffn % H_TILE != 0) {
        return MOE_OVL_ERR_UNSUPPORTED;
    }
    const int dout = c->single_gemm_out > 0 ? c->single_gemm_out : c->d_model;
    if ((long long)c->num_src_ranks * c->tokens_per_rank * (dout / 8) >= (1ll << 31)) return MOE_OVL_ERR_UNSUPPORTED;
    if (c->num_local_experts > PLAN_MAX_EXPERTS ||
        (long long)c->num_local_experts * c->num_src_ranks > PLAN_MAX_GROUPS)
        return MOE_OVL_ERR_UNSUPPORTED;
    return MOE_OVL_OK;
}

int make_layout(const moe_ovl_config *c, Layout *L)
{
    const int rc = check_config(c);
    if (rc != MOE_OVL_OK) return rc;
    const long long G = (long long)c->num_local_experts * c->num_src_ranks;
    const long long max_bands_ll = ((long long)c->max_rows + TB_M - 1) / TB_M + G;
    L->single = c->single_gemm_out > 0;
    L->dout = L->single ? c->single_gemm_out : c->d_model;
    L->k2 = L->single ? c->d_model : c->d_ffn;
    L->f_eff = L->single ? H_TILE : c->d_ffn;       // the hidden buffer is unused by single-projection experts
    L->n1 = L->single ? 0 : c->d_ffn / H_TILE;
    L->n2 = L->dout / TB_N;
    const long long max_items_ll = max_bands_ll * (L->n1 + L->n2);
    if (max_bands_ll > (1 << 24) || max_items_ll > (1ll << 30)) return MOE_OVL_ERR_UNSUPPORTED;
    L->max_bands = (int)max_bands_ll;
    L->max_items = (int)max_items_ll;
    L->words = (c->tokens_per_rank + 31) / 32;
    L->kmax = std::min(c->top_k, c->num_local_experts);
    const size_t P = (size_t)L->max_bands * TB_M, d = c->d_model, F = L->f_eff, dout = L->dout;
    const size_t ntok = (size_t)c->num_src_ranks * c->tokens_per_rank;
    size_t off = 0;
    auto take = [&](size_t bytes) { size_t o = off; off = align_up(off + bytes); return o; };
    L->Xa = take(P * d * 2);
    L->H = take(P * F * 2);
    L->Y = take(P * dout * 2);
    L->zero_begin = off;
    L->bitmap = take((size_t)G * L->words * 4);
    L->hcount = take((size_t)L->max_bands * 4);
    L->fcount = take((size_t)L->max_bands * L->n2 * 4);
    L->status = take(ST_COUNT * 4);
    L->next_item = take(32);                 // next_item, plan_ticket, next_seg, assist_segs, next_gather, next_zero
    L->stamps = take(STAMP_COUNT * 8);
    L->tok_slot = take(ntok * L->kmax * 4);
    L->zero_end = off;
    L->tok_gate = take(ntok * L->kmax * 4);
    L->wordpfx = take((size_t)G * L->words * 4);
    L->group_rows = take((size_t)G * 4);
    L->group_start = take((size_t)G * 4);
    L->group_slot = take((size_t)G * 4);
    L->pos = take((size_t)std::max(c->max_rows, 1) * 4);
    L->slot = take((size_t)std::max(c->max_rows, 1) * 4);
    L->row_at = take(P * 4);
    L->xready = take((size_t)L->max_bands * 4);
    L->band_expert = take((size_t)L->max_bands * 4);
    L->band_dest = take((size_t)L->max_bands * 4);
    L->band_valid = take((size_t)L->max_bands * 4);
    L->band_slot0 = take((size_t)L->max_bands * 4);
    L->sched_band = take((size_t)L->max_bands * 4);
    L->gather_band = take((size_t)L->max_bands * 4);
    L->items = take((size_t)L->max_items * 16);
    L->segs = take((size_t)L->max_bands * 16);
    L->seg_slot0 = take((size_t)L->max_bands * 4);
    L->flags = take((size_t)L->max_bands * L->n2 * 4);
    L->meta = take(META_COUNT * 4 + 4);      // meta[] and the call counter
    L->smid = take(2 * 1024 * 4);            // SM of every GEMM CTA, then of every consumer CTA
    for (int i = 0; i < 13; ++i) L->sb[i] = take((size_t)L->max_bands * 4);
    L->st_ret_rows = (long long)c->tokens_per_rank * L->kmax;
    L->trace_bytes = 0;
    if (c->flags & MOE_OVL_FLAG_TRACE) {
        L->trace_items = take((size_t)L->max_items * sizeof(TraceRec));
        L->trace_items2 = take((size_t)L->max_items * sizeof(TraceRec));
        L->trace_units = take((size_t)L->max_bands * MAX_SEG_CHUNKS * sizeof(TraceRec));
        L->trace_item_aux = take((size_t)L->max_items * 8);
        L->trace_bytes = off - L->trace_items;
    }
    if (c->flags & MOE_OVL_FLAG_HOST_STAGING) {
        for (int s = 0; s < 2; ++s) {
            L->st_x[s] = take((size_t)std::max(c->max_rows, 1) * d * 2);
            L->st_counts[s] = take((size_t)c->num_local_experts * 4);
            L->st_rank[s] = take((size_t)std::max(c->max_rows, 1) * 4);
            L->st_token[s] = take((size_t)std::max(c->max_rows, 1) * 4);
            L->st_gate[s] = take((size_t)std::max(c->max_rows, 1) * 4);
            L->st_out[s] = take(ntok * dout * 2);
        }
        L->st_ret = take((size_t)c->num_src_ranks * L->st_ret_rows * dout * 2);
    }
    L->total = off;
    return MOE_OVL_OK;
}

}  // namespace

struct moe_ovl_ctx {
    moe_ovl_config cfg;
    Layout L;
    uint8_t *ws;
    int num_sms;
    int combine_blocks_per_sm, scatter_blocks_per_sm;
    cudaStream_t s_prod, s_cons;
    cudaStream_t s_h2d, s_d2h;                        // host-buffer entry point: copies overlap the previous/next pass
    cudaEvent_t ev_h2d[2], ev_comp[2], ev_d2h[2];
    unsigned long long host_calls;
    cudaEvent_t ev_fork, ev_prod_done, ev_cons_done;
    // timing: call start, after prep, GEMM start/end, mover start/end, call end
    cudaEvent_t t_begin, t_m0, t_m1, t_end;   // GEMM start / end: h_p0 / h_p1 of the call's history slot
    int last_hist;
    bool last_dedicated;
    // GEMM start/end of the last HISTORY calls, so that a caller can average the kernel's duration over a run
    // of back-to-back calls without synchronising between them
    cudaEvent_t h_p0[MOE_OVL_TIMING_HISTORY], h_p1[MOE_OVL_TIMING_HISTORY];
    unsigned long long calls;
    cudaStream_t last_stream;
    bool ran;
    int last_mode, last_prod_ctas, last_cons_ctas, last_launches, last_rows, last_chunks, last_tail_segs;
    bool last_timed;                                  // false when the last call was captured into a graph
    bool hist_timed[MOE_OVL_TIMING_HISTORY];
    int last_cuda_error;
    EncodeTiledFn encode;
    CUtensorMap map_xa, map_h, map_xa8, map_h8, map_xa64, map_h64;
};

namespace {

#define CU_CHECK(ctx, call)                                  \
    do {                                                     \
        cudaError_t e_ = (call);                             \
        if (e_ != cudaSuccess) {                             \
            (ctx)->last_cuda_error = (int)e_;                \
            return MOE_OVL_ERR_CUDA;                         \
        }                                                    \
    } while (0)

// 2-D bf16 row-major tensor [rows, cols], box = 64 columns x box_rows rows (128 unless stated), 128-byte swizzle
int encode_map(moe_ovl_ctx *ctx, CUtensorMap *map, const void *base, size_t rows, size_t cols, int box_rows = TB_M)
{
    const cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)std::max<size_t>(rows, 1)};
    const cuuint64_t strides[1] = {(cuuint64_t)cols * 2};
    const cuuint32_t box[2] = {TB_K, (cuuint32_t)box_rows};
    const cuuint32_t estr[2] = {1, 1};
    const CUresult r = ctx->encode(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(base), dims, strides,
                                   box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                                   CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) {
        ctx->last_cuda_error = (int)r;
        return MOE_OVL_ERR_CUDA;
    }
    return MOE_OVL_OK;
}

template <typename T>
T *at(moe_ovl_ctx *ctx, size_t off) { return reinterpret_cast<T *>(ctx->ws + off); }

Params make_params(moe_ovl_ctx *ctx)
{
    const moe_ovl_config &c = ctx->cfg;
    const Layout &L = ctx->L;
    Params p;
    std::memset(&p, 0, sizeof(p));
    p.R = c.num_src_ranks; p.r_self = c.self_rank; p.T = c.tokens_per_rank; p.El = c.num_local_experts;
    p.kmax = L.kmax; p.d = c.d_model; p.F = L.f_eff;
    p.dout = L.dout; p.k2 = L.k2; p.single = L.single;
    p.mgb = std::max(1, c.mid_seg_bands);
    p.group_bands = c.group_bands > 0 ? (c.group_bands < 64 ? c.group_bands : 64) : 16;
    p.words = L.words; p.n1 = L.n1; p.n2 = L.n2; p.max_bands = L.max_bands; p.max_items = L.max_items;
    p.timeout_ns = (unsigned long long)(c.wait_timeout_us > 0 ? c.wait_timeout_us : 2000000) * 1000ull;
    p.Xa = at<uint16_t>(ctx, L.Xa); p.H = at<uint16_t>(ctx, L.H); p.Y = at<uint16_t>(ctx, L.Y);
    p.bitmap = at<unsigned>(ctx, L.bitmap); p.wordpfx = at<int>(ctx, L.wordpfx);
    p.group_rows = at<int>(ctx, L.group_rows); p.group_start = at<int>(ctx, L.group_start);
    p.group_slot = at<int>(ctx, L.group_slot); p.pos = at<int>(ctx, L.pos); p.slot = at<int>(ctx, L.slot);
    p.band_expert = at<int>(ctx, L.band_expert); p.band_dest = at<int>(ctx, L.band_dest);
    p.band_valid = at<int>(ctx, L.band_valid); p.band_slot0 = at<int>(ctx, L.band_slot0);
    p.gather_band = at<int>(ctx, L.gather_band);
    p.sched_band = at<int>(ctx, L.sched_band); p.items = at<int4>(ctx, L.items); p.segs = at<int4>(ctx, L.segs);
    p.seg_slot0 = at<int>(ctx, L.seg_slot0); p.tok_slot = at<int>(ctx, L.tok_slot);
    p.tok_gate = at<float>(ctx, L.tok_gate); p.hcount = at<unsigned>(ctx, L.hcount);
    p.fcount = at<unsigned>(ctx, L.fcount);
    p.low_ok = (c.flags & MOE_OVL_FLAG_NO_SMALL_GROUP_TILES) ? 0
             : (c.flags & MOE_OVL_FLAG_NO_STACKED_BANDS)   ? 1
             : (c.flags & MOE_OVL_FLAG_NO_LOCAL_RIDERS)    ? 2 : 3;
    p.swap_ok = (!(c.flags & MOE_OVL_FLAG_NO_SMALL_GROUP_TILES) && (L.single || c.d_ffn % (2 * H_TILE) == 0))
                    ? ((c.flags & MOE_OVL_FLAG_TEST_ALL_SMALL_GROUP_TILES) ? 2 : 1) : 0;
    p.next_item = at<int>(ctx, L.next_item);
    p.plan_ticket = at<int>(ctx, L.next_item) + 1;
    p.next_seg = at<int>(ctx, L.next_item) + 2;
    p.assist_segs = at<int>(ctx, L.next_item) + 3;
    p.next_gather = at<int>(ctx, L.next_item) + 4;
    p.next_zero = at<int>(ctx, L.next_item) + 5;
    p.row_at = at<int>(ctx, L.row_at);
    p.xready = at<unsigned>(ctx, L.xready);
    p.stamps = at<unsigned long long>(ctx, L.stamps);
    p.smid_prod = at<int>(ctx, L.smid);
    p.smid_cons = at<int>(ctx, L.smid) + 1024;
    p.flags = at<unsigned>(ctx, L.flags);
    p.epoch_rw = at<unsigned>(ctx, L.meta) + META_COUNT;     // the word after meta[], cleared at creation only
    p.epoch = p.epoch_rw; p.meta = at<int>(ctx, L.meta); p.status = at<int>(ctx, L.status);
    p.seg_chunks = MAX_SEG_CHUNKS;
    p.tail_segs = 0;
    if (c.flags & MOE_OVL_FLAG_TRACE) {
        p.trace_items = at<TraceRec>(ctx, L.trace_items);
        p.trace_units = at<TraceRec>(ctx, L.trace_units);
        p.trace_items2 = at<TraceRec>(ctx, L.trace_items2);
        p.trace_item_aux = at<int2>(ctx, L.trace_item_aux);
    }
    return p;
}

// Consumer budget for MODE_OVERLAP with consumer_sm_count = 0 (Section 3.3.3: too few consumer SMs and the
// transfer falls behind, too many and the GEMM loses capacity).  Every SM given up costs 1/SMs of the GEMM
// time; the return it hides is worth t_return.  About half of the break-even count SMs * t_return / t_gemm,
// with t_return = 4*d bytes per row at ~5 TB/s and t_gemm = 6*d*F flop per row at ~1.2 PFLOP/s.
int choose_consumer_sms(const moe_ovl_ctx *ctx)
{
    const moe_ovl_config &c = ctx->cfg;
    const Layout &L = ctx->L;
    const double t_ret = 4.0 * L.dout / 5.0e12;
    const double t_gemm = (L.single ? 2.0 * c.d_model * (double)L.dout : 6.0 * c.d_model * (double)c.d_ffn) / 1.2e15;
    const double breakeven = ctx->num_sms * t_ret / t_gemm;
    return std::min(16, std::max(2, 2 * (int)(breakeven / 4.0 + 0.5)));
}

// MODE_AUTO: which of the three ways to run the return, and with how many consumer SMs (Section 3.3.3 names
// the trade-off and leaves the choice to future work).  A three-line cost model over what the host knows --
// the shape and the number of rows -- with coefficients measured on a B200 at its power cap:
//   GEMM      padded flop / (8.6 TFLOP/s per GEMM CTA): 148 CTAs reach about 1270 TFLOP/s sustained
//   scatter   non-overlap only: a launch boundary and its timing event (about 10 us) + 4*dout bytes per row at 5.5 TB/s
//   tail      what is left to move after the last tile is flagged: one segment per mover.  A consumer CTA
//             moves about 35 GB/s of payload, the four spare warps of a GEMM CTA about 15 GB/s of a unit that
//             is an eighth of a segment
//   stolen    dedicated consumer SMs are not GEMM SMs: the GEMM term grows by SMs / (SMs - c)
//   drag      movers inside the GEMM CTAs share their load/store path: about 0.4 % of the GEMM term
// Padding is estimated as half a band per (expert, rank) group.
void choose_mode(const moe_ovl_ctx *ctx, int num_rows, int *mode, int *consumer_sms)
{
    const moe_ovl_config &c = ctx->cfg;
    const Layout &L = ctx->L;
    *consumer_sms = choose_consumer_sms(ctx);
    if (num_rows == 0) { *mode = MOE_OVL_MODE_NON_OVERLAP; return; }       // nothing to return
    const double sms = ctx->num_sms;
    const double groups = (double)c.num_local_experts * c.num_src_ranks;
    const double padded = num_rows + 0.5 * TB_M * groups;
    const double flop_row = L.single ? 2.0 * c.d_model * L.dout : 6.0 * (double)c.d_model * c.d_ffn;
    const double gemm_all = padded * flop_row / (8.6e12 * sms);            // seconds on every SM
    const double row_bytes = 2.0 * L.dout;
    const double seg_bytes = (double)std::max(1, c.mid_seg_bands) * TB_M * row_bytes;
    const double t_non = gemm_all + 10e-6 + 2.0 * row_bytes * num_rows / 5.5e12;
    const double t_in = gemm_all * 1.004 + (seg_bytes / MAX_SEG_CHUNKS) / 15e9;
    const double cs = *consumer_sms;
    const double t_ded = gemm_all * sms / (sms - cs) + seg_bytes / 35e9 / std::max(1.0, cs / 4.0);
    *mode = MOE_OVL_MODE_IN_KERNEL;
    double best = t_in;
    if (t_non < best) { best = t_non; *mode = MOE_OVL_MODE_NON_OVERLAP; }
    if (t_ded < best) { best = t_ded; *mode = MOE_OVL_MODE_OVERLAP; }
}

// Should the all-zero rows of `out` be written behind the GEMM (see zero_fill_rows)?  Their writes share HBM with
// the GEMM's own traffic: worth it where the GEMM is long against them (0.990 against 0.999 of the baseline at the
// Mixtral shape), a loss where the layer is already traffic-heavy (the paper's single-projection operator with
// K = 2048: the GEMM kernel grew by 12 %).  Taken when the estimated GEMM time is at least sixteen times the time
// the zero rows take alone (half of the tokens assumed to have none, 3.3 TB/s of writes).
bool zero_rows_behind_gemm(const moe_ovl_ctx *ctx, int num_rows)
{
    const moe_ovl_config &c = ctx->cfg;
    const Layout &L = ctx->L;
    const double groups = (double)c.num_local_experts * c.num_src_ranks;
    const double padded = num_rows + 0.5 * TB_M * groups;
    const double flop_row = L.single ? 2.0 * c.d_model * L.dout : 6.0 * (double)c.d_model * c.d_ffn;
    const double gemm = padded * flop_row / (8.6e12 * ctx->num_sms);
    const double zeros = 0.5 * (double)c.num_src_ranks * c.tokens_per_rank * L.dout * 2.0 / 3.3e12;
    return gemm >= 16.0 * zeros;
}

// Two builds of the GEMM kernel: the one with the trace bookkeeping compiled in runs only for contexts that asked
// for a trace, so that the bookkeeping costs nothing otherwise.
void launch_producer(int ctas, cudaStream_t st, const ProducerMaps &maps, const Params &p, int kflags)
{
    if (p.trace_items) producer_kernel<true><<<ctas, PROD_THREADS, PROD_SMEM_BYTES, st>>>(maps, p, kflags);
    else producer_kernel<false><<<ctas, PROD_THREADS, PROD_SMEM_BYTES, st>>>(maps, p, kflags);
}

int sync_last(moe_ovl_ctx *ctx)
{
    if (ctx->ran) CU_CHECK(ctx, cudaStreamSynchronize(ctx->last_stream));
    if (ctx->s_d2h) CU_CHECK(ctx, cudaStreamSynchronize(ctx->s_d2h));
    return MOE_OVL_OK;
}

}  // namespace

extern "C" {

const char *moe_ovl_strerror(int code)
{
    switch (code) {
    case MOE_OVL_OK: return "ok";
    case MOE_OVL_ERR_INVALID_ARG: return "invalid argument";
    case MOE_OVL_ERR_UNSUPPORTED: return "unsupported shape";
    case MOE_OVL_ERR_CUDA: return "CUDA call failed";
    case MOE_OVL_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
    case MOE_OVL_ERR_TIMEOUT: return "a device-side wait timed out";
    case MOE_OVL_ERR_BAD_ROUTING: return "inconsistent routing metadata";
    default: return "unknown error";
    }
}

int moe_ovl_workspace_bytes(const moe_ovl_config *cfg, size_t *bytes)
{
    if (!bytes) return MOE_OVL_ERR_INVALID_ARG;
    Layout L;
    const int rc = make_layout(cfg, &L);
    if (rc != MOE_OVL_OK) return rc;
    *bytes = L.total + ALIGN;     // slack to round the base up to the alignment TMA-read buffers need
    return MOE_OVL_OK;
}

int moe_ovl_limits(const moe_ovl_config *cfg, int32_t *max_bands, int32_t *max_items)
{
    Layout L;
    const int rc = make_layout(cfg, &L);
    if (rc != MOE_OVL_OK) return rc;
    if (max_bands) *max_bands = L.max_bands;
    if (max_items) *max_items = L.max_items;
    return MOE_OVL_OK;
}

int moe_ovl_last_cuda_error(const moe_ovl_ctx *ctx) { return ctx ? ctx->last_cuda_error : 0; }

int moe_ovl_create(moe_ovl_ctx **out, const moe_ovl_config *cfg, void *workspace, size_t workspace_bytes)
{
    if (!out) return MOE_OVL_ERR_INVALID_ARG;
    *out = nullptr;
    Layout L;
    int rc = make_layout(cfg, &L);
    if (rc != MOE_OVL_OK) return rc;
    if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & 255u) || workspace_bytes < L.total + ALIGN)
        return MOE_OVL_ERR_WORKSPACE;
    moe_ovl_ctx *ctx = new (std::nothrow) moe_ovl_ctx();
    if (!ctx) return MOE_OVL_ERR_INVALID_ARG;
    std::memset(ctx, 0, sizeof(*ctx));
    ctx->cfg = *cfg;
    ctx->L = L;
    // the layout assumes a 1024-byte aligned base; round up inside the slack
    ctx->ws = reinterpret_cast<uint8_t *>(align_up(reinterpret_cast<uintptr_t>(workspace)));

    auto fail = [&](int code) { moe_ovl_destroy(ctx); return code; };
#define CREATE_CHECK(call)                                         \
    do {                                                           \
        if ((call) != cudaSuccess) return fail(MOE_OVL_ERR_CUDA);  \
    } while (0)
    CREATE_CHECK(cudaSetDevice(cfg->device));
    CREATE_CHECK(cudaDeviceGetAttribute(&ctx->num_sms, cudaDevAttrMultiProcessorCount, cfg->device));
    int lo = 0, hi = 0;
    CREATE_CHECK(cudaDeviceGetStreamPriorityRange(&lo, &hi));
    // the consumer stream gets the higher priority (Section 3.3.3)
    CREATE_CHECK(cudaStreamCreateWithPriority(&ctx->s_cons, cudaStreamNonBlocking, hi));
    CREATE_CHECK(cudaStreamCreateWithPriority(&ctx->s_prod, cudaStreamNonBlocking, lo));
    if (cfg->flags & MOE_OVL_FLAG_HOST_STAGING) {
        CREATE_CHECK(cudaStreamCreateWithFlags(&ctx->s_h2d, cudaStreamNonBlocking));
        CREATE_CHECK(cudaStreamCreateWithFlags(&ctx->s_d2h, cudaStreamNonBlocking));
        for (int s = 0; s < 2; ++s) {
            CREATE_CHECK(cudaEventCreateWithFlags(&ctx->ev_h2d[s], cudaEventDisableTiming));
            CREATE_CHECK(cudaEventCreateWithFlags(&ctx->ev_comp[s], cudaEventDisableTiming));
            CREATE_CHECK(cudaEventCreateWithFlags(&ctx->ev_d2h[s], cudaEventDisableTiming));
        }
    }
    cudaEvent_t *plain[] = {&ctx->ev_fork, &ctx->ev_prod_done, &ctx->ev_cons_done};
    for (auto e : plain) CREATE_CHECK(cudaEventCreateWithFlags(e, cudaEventDisableTiming));
    cudaEvent_t *timed[] = {&ctx->t_begin, &ctx->t_m0, &ctx->t_m1, &ctx->t_end};
    for (auto e : timed) CREATE_CHECK(cudaEventCreate(e));
    for (int i = 0; i < MOE_OVL_TIMING_HISTORY; ++i) {
        CREATE_CHECK(cudaEventCreate(&ctx->h_p0[i]));
        CREATE_CHECK(cudaEventCreate(&ctx->h_p1[i]));
    }
    CREATE_CHECK(cudaFuncSetAttribute(producer_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, PROD_SMEM_BYTES));
    CREATE_CHECK(cudaFuncSetAttribute(producer_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, PROD_SMEM_BYTES));
    CREATE_CHECK(cudaFuncSetAttribute(consumer_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                      CONSUMER_SMEM_BYTES));
    // grid-stride kernels get exactly one resident wave: a partial second wave would run at a fraction of the
    // occupancy and stretch the kernel
    CREATE_CHECK(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&ctx->combine_blocks_per_sm, combine_kernel, 256, 0));
    CREATE_CHECK(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&ctx->scatter_blocks_per_sm, scatter_kernel, 256, 0));
    ctx->combine_blocks_per_sm = std::max(1, ctx->combine_blocks_per_sm);
    ctx->scatter_blocks_per_sm = std::max(1, ctx->scatter_blocks_per_sm);
    void *fn = nullptr;
    cudaDriverEntryPointQueryResult qres;
    CREATE_CHECK(cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres));
    if (!fn || qres != cudaDriverEntryPointSuccess) return fail(MOE_OVL_ERR_CUDA);
    ctx->encode = reinterpret_cast<EncodeTiledFn>(fn);
    const size_t P = (size_t)L.max_bands * TB_M;
    rc = encode_map(ctx, &ctx->map_xa, ctx->ws + L.Xa, P, cfg->d_model);
    if (rc == MOE_OVL_OK) rc = encode_map(ctx, &ctx->map_h, ctx->ws + L.H, P, L.f_eff);
    // the same buffers in boxes of 8 rows, for the token side of the swapped-operand items
    if (rc == MOE_OVL_OK) rc = encode_map(ctx, &ctx->map_xa8, ctx->ws + L.Xa, P, cfg->d_model, 8);
    if (rc == MOE_OVL_OK) rc = encode_map(ctx, &ctx->map_h8, ctx->ws + L.H, P, L.f_eff, 8);
    // ... and in boxes of 64 rows, for band pairs that are computed 64 rows high
    if (rc == MOE_OVL_OK) rc = encode_map(ctx, &ctx->map_xa64, ctx->ws + L.Xa, P, cfg->d_model, 64);
    if (rc == MOE_OVL_OK) rc = encode_map(ctx, &ctx->map_h64, ctx->ws + L.H, P, L.f_eff, 64);
    if (rc != MOE_OVL_OK) return fail(rc);
    // flags hold the epoch of the call that finished the tile: clear them once, never again
    CREATE_CHECK(cudaMemset(ctx->ws + L.flags, 0, (size_t)L.max_bands * L.n2 * 4));
    CREATE_CHECK(cudaMemset(ctx->ws + L.meta, 0, META_COUNT * 4 + 4));
    CREATE_CHECK(cudaMemset(ctx->ws + L.status, 0, ST_COUNT * 4));
#undef CREATE_CHECK
    *out = ctx;
    return MOE_OVL_OK;
}

int moe_ovl_destroy(moe_ovl_ctx *ctx)
{
    if (!ctx) return MOE_OVL_OK;
    if (ctx->ran) cudaStreamSynchronize(ctx->last_stream);
    if (ctx->s_prod) { cudaStreamSynchronize(ctx->s_prod); cudaStreamDestroy(ctx->s_prod); }
    if (ctx->s_cons) { cudaStreamSynchronize(ctx->s_cons); cudaStreamDestroy(ctx->s_cons); }
    if (ctx->s_h2d) { cudaStreamSynchronize(ctx->s_h2d); cudaStreamDestroy(ctx->s_h2d); }
    if (ctx->s_d2h) { cudaStreamSynchronize(ctx->s_d2h); cudaStreamDestroy(ctx->s_d2h); }
    for (int s = 0; s < 2; ++s)
        for (cudaEvent_t e : {ctx->ev_h2d[s], ctx->ev_comp[s], ctx->ev_d2h[s]})
            if (e) cudaEventDestroy(e);
    cudaEvent_t evs[] = {ctx->ev_fork, ctx->ev_prod_done, ctx->ev_cons_done, ctx->t_begin, ctx->t_m0, ctx->t_m1,
                         ctx->t_end};
    for (auto e : evs)
        if (e) cudaEventDestroy(e);
    for (int i = 0; i < MOE_OVL_TIMING_HISTORY; ++i) {
        if (ctx->h_p0[i]) cudaEventDestroy(ctx->h_p0[i]);
        if (ctx->h_p1[i]) cudaEventDestroy(ctx->h_p1[i]);
    }
    delete ctx;
    return MOE_OVL_OK;
}

int moe_ovl_expert_return(moe_ovl_ctx *ctx, const moe_ovl_args *a)
{
    if (!ctx || !a || a->struct_size != sizeof(moe_ovl_args)) return MOE_OVL_ERR_INVALID_ARG;
    const moe_ovl_config &c = ctx->cfg;
    const Layout &L = ctx->L;
    if (a->num_rows < 0 || a->num_rows > c.max_rows) return MOE_OVL_ERR_INVALID_ARG;
    if (!a->expert_counts || !a->w1 || (!a->w2 && !L.single) || !a->ret || !a->out) return MOE_OVL_ERR_INVALID_ARG;
    if (a->num_rows > 0 && (!a->x || !a->src_rank || !a->src_token || !a->gate)) return MOE_OVL_ERR_INVALID_ARG;
    if (a->ret_rows_per_rank < (int64_t)c.tokens_per_rank * L.kmax) return MOE_OVL_ERR_INVALID_ARG;
    if (a->mode < MOE_OVL_MODE_OVERLAP || a->mode > MOE_OVL_MODE_AUTO) return MOE_OVL_ERR_INVALID_ARG;
    const uintptr_t align16 = reinterpret_cast<uintptr_t>(a->x) | reinterpret_cast<uintptr_t>(a->w1) |
                              reinterpret_cast<uintptr_t>(a->w2) | reinterpret_cast<uintptr_t>(a->ret) |
                              reinterpret_cast<uintptr_t>(a->out);
    if (align16 & 15u) return MOE_OVL_ERR_INVALID_ARG;
    int mode = a->mode, want = a->consumer_sm_count;
    if (mode == MOE_OVL_MODE_AUTO) choose_mode(ctx, a->num_rows, &mode, &want);
    const bool dedicated = mode == MOE_OVL_MODE_OVERLAP, in_kernel = mode == MOE_OVL_MODE_IN_KERNEL;
    int prod_ctas, cons_ctas = 0;
    if (dedicated) {
        if (want < 0 || want > ctx->num_sms / 2) return MOE_OVL_ERR_INVALID_ARG;
        if (want == 0) want = choose_consumer_sms(ctx);
        cons_ctas = (want + 1) & ~1;                        // whole SM pairs: the GEMM's CTAs work in pairs
        prod_ctas = (ctx->num_sms - cons_ctas) & ~1;        // disjoint SM sets: grids sum to the SM count
    } else {
        const bool limited = mode == MOE_OVL_MODE_NON_OVERLAP && c.producer_sm_limit > 0;
        prod_ctas = (limited ? std::min(c.producer_sm_limit, ctx->num_sms) : ctx->num_sms) & ~1;
        if (prod_ctas < 2) return MOE_OVL_ERR_INVALID_ARG;
    }
    CU_CHECK(ctx, cudaSetDevice(c.device));
    cudaStream_t st = static_cast<cudaStream_t>(a->stream);
    // Events recorded while a stream is being captured carry no time: a captured call records none of the
    // timing events, and the report says so.
    cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
    CU_CHECK(ctx, cudaStreamIsCapturing(st, &cap));
    const bool timed = cap == cudaStreamCaptureStatusNone;
#define TIME_POINT(ev, stream)                                      \
    do {                                                            \
        if (timed) CU_CHECK(ctx, cudaEventRecord((ev), (stream)));  \
    } while (0)

    Params p = make_params(ctx);
    p.M = a->num_rows;
    p.lag_items = prod_ctas;                        // two rounds of the prod_ctas / 2 CTA pairs
    p.seg_chunks = MAX_SEG_CHUNKS;
    p.zero_early = mode != MOE_OVL_MODE_NON_OVERLAP &&
                   (zero_rows_behind_gemm(ctx, a->num_rows) || (c.flags & MOE_OVL_FLAG_TEST_ZERO_ROWS_EARLY));
    p.tail_segs = in_kernel ? -1 : p.group_bands;       // dedicated consumer: whole segments but for the last super-band's
    p.ret_rows_per_rank = a->ret_rows_per_rank;
    p.x = static_cast<const uint16_t *>(a->x);
    p.expert_counts = a->expert_counts; p.src_rank = a->src_rank; p.src_token = a->src_token; p.gate = a->gate;
    p.ret = static_cast<uint16_t *>(a->ret); p.out = static_cast<uint16_t *>(a->out);
    p.slot_out = a->slot_out; p.rows_per_rank_out = a->rows_per_rank_out; p.segs_per_rank_out = a->segs_per_rank_out;

    ProducerMaps maps;
    maps.xa = ctx->map_xa;
    maps.h = ctx->map_h;
    maps.xa8 = ctx->map_xa8;
    maps.h8 = ctx->map_h8;
    maps.xa64 = ctx->map_xa64;
    maps.h64 = ctx->map_h64;
    int rc;
    if (L.single) {
        // one projection per expert: W[El, N, d] is the B operand of the GEMM that writes Y
        rc = encode_map(ctx, &maps.w2, a->w1, (size_t)c.num_local_experts * L.dout, c.d_model);
        maps.w1 = maps.w2;
        maps.w1h = maps.w2;          // no first GEMM
    } else {
        rc = encode_map(ctx, &maps.w1, a->w1, (size_t)c.num_local_experts * 2 * c.d_ffn, c.d_model);
        if (rc == MOE_OVL_OK) rc = encode_map(ctx, &maps.w2, a->w2, (size_t)c.num_local_experts * c.d_model, c.d_ffn);
        if (rc == MOE_OVL_OK)
            rc = encode_map(ctx, &maps.w1h, a->w1, (size_t)c.num_local_experts * 2 * c.d_ffn, c.d_model, 64);
    }
    if (rc != MOE_OVL_OK) return rc;

    PlanScratch sc;
    sc.sb_start = at<int>(ctx, L.sb[0]); sc.sb_nb = at<int>(ctx, L.sb[1]); sc.sb_expert = at<int>(ctx, L.sb[2]);
    sc.sb_g1off = at<int>(ctx, L.sb[3]); sc.sb_g2off = at<int>(ctx, L.sb[4]); sc.sb_g1end = at<int>(ctx, L.sb[5]);
    sc.sb_kind = at<int>(ctx, L.sb[6]); sc.sb_ntok = at<int>(ctx, L.sb[7]);
    sc.sb_c1 = at<int>(ctx, L.sb[8]); sc.sb_c2 = at<int>(ctx, L.sb[9]);
    sc.sb_units = at<int>(ctx, L.sb[10]); sc.unit_tab = at<int>(ctx, L.sb[11]); sc.sb_role = at<int>(ctx, L.sb[12]);

    int launches = 0;
    const int hist = (int)(ctx->calls % MOE_OVL_TIMING_HISTORY);
    int kflags = (c.flags & MOE_OVL_FLAG_TEST_SKIP_GATHER) ? PROD_SKIP_FIRST_BAND : 0;
    if (mode != MOE_OVL_MODE_NON_OVERLAP && !(c.flags & MOE_OVL_FLAG_TEST_NO_FLAGS)) kflags |= PROD_RAISE_FLAGS;
    if (in_kernel) kflags |= PROD_WARP_MOVERS;
    TIME_POINT(ctx->t_begin, st);
    // ---- plan (row layout, tile schedule, combine plan): integer kernels on the caller's stream
    CU_CHECK(ctx, cudaMemsetAsync(ctx->ws + L.zero_begin, 0, L.zero_end - L.zero_begin, st));
    if (L.trace_bytes) CU_CHECK(ctx, cudaMemsetAsync(ctx->ws + L.trace_items, 0, L.trace_bytes, st));
    plan_mark_build_kernel<<<std::max(1, (p.M + PLAN_THREADS - 1) / PLAN_THREADS), PLAN_THREADS, 0, st>>>(p, sc);
    ++launches;
    if (p.M > 0) {
        plan_rows_kernel<<<(p.M + 255) / 256, 256, 0, st>>>(p);
        ++launches;
    }
    CU_CHECK(ctx, cudaGetLastError());
    // (the end of the plan is the start of the GEMM: one event, recorded below)

    if (dedicated) {
        // ---- two persistent kernels on two streams, disjoint SM sets (Section 3.3.3)
        CU_CHECK(ctx, cudaEventRecord(ctx->ev_fork, st));
        CU_CHECK(ctx, cudaStreamWaitEvent(ctx->s_cons, ctx->ev_fork, 0));
        CU_CHECK(ctx, cudaStreamWaitEvent(ctx->s_prod, ctx->ev_fork, 0));
        // The GEMM is enqueued first: if anything serialises the two kernels (a profiler, blocking launches, a
        // GPU whose free SMs do not hold both grids), the GEMM runs to completion, its own CTAs drain every
        // segment at the end, and the consumer then finds nothing left -- instead of a consumer that waits for
        // flags nobody can raise.  With both grids resident the order makes no difference.
        TIME_POINT(ctx->h_p0[hist], ctx->s_prod);
        launch_producer(prod_ctas, ctx->s_prod, maps, p, kflags);
        TIME_POINT(ctx->h_p1[hist], ctx->s_prod);
        CU_CHECK(ctx, cudaEventRecord(ctx->ev_prod_done, ctx->s_prod));
        TIME_POINT(ctx->t_m0, ctx->s_cons);
        consumer_kernel<<<cons_ctas, MOVER_THREADS, CONSUMER_SMEM_BYTES, ctx->s_cons>>>(p);
        TIME_POINT(ctx->t_m1, ctx->s_cons);
        CU_CHECK(ctx, cudaEventRecord(ctx->ev_cons_done, ctx->s_cons));
        CU_CHECK(ctx, cudaStreamWaitEvent(st, ctx->ev_cons_done, 0));
        CU_CHECK(ctx, cudaStreamWaitEvent(st, ctx->ev_prod_done, 0));
        launches += 2;
    } else {
        // ---- one GEMM kernel on every SM.  IN_KERNEL: its spare warps move the finished segments while the
        //      tensor cores work.  NON_OVERLAP (the comparison baseline): it runs to completion, then a separate
        //      scatter kernel moves all rows.
        // Few events: each costs host time on the enqueuing thread, which is what bounds small layers.
        TIME_POINT(ctx->h_p0[hist], st);
        launch_producer(prod_ctas, st, maps, p, kflags);
        ++launches;
        TIME_POINT(ctx->h_p1[hist], st);          // also the start of the scatter kernel, if any
        if (!in_kernel) {
            scatter_kernel<<<ctx->scatter_blocks_per_sm * ctx->num_sms, 256, 0, st>>>(p);
            ++launches;
            TIME_POINT(ctx->t_m1, st);
        }
    }
    combine_kernel<<<ctx->combine_blocks_per_sm * ctx->num_sms, 256, 0, st>>>(p);
    ++launches;
    CU_CHECK(ctx, cudaGetLastError());
    TIME_POINT(ctx->t_end, st);
#undef TIME_POINT

    ctx->last_stream = st;
    ctx->ran = true;
    ctx->hist_timed[hist] = timed;
    ++ctx->calls;
    ctx->last_timed = timed;
    ctx->last_hist = hist;
    ctx->last_dedicated = dedicated;
    ctx->last_mode = mode;
    ctx->last_prod_ctas = prod_ctas;
    ctx->last_cons_ctas = cons_ctas;
    ctx->last_launches = launches;
    ctx->last_rows = p.M;
    ctx->last_chunks = p.seg_chunks;
    ctx->last_tail_segs = p.tail_segs;
    return MOE_OVL_OK;
}

int moe_ovl_expert_return_host(moe_ovl_ctx *ctx, const moe_ovl_host_args *h)
{
    if (!ctx || !h || h->struct_size != sizeof(moe_ovl_host_args)) return MOE_OVL_ERR_INVALID_ARG;
    const moe_ovl_config &c = ctx->cfg;
    const Layout &L = ctx->L;
    if (!(c.flags & MOE_OVL_FLAG_HOST_STAGING)) return MOE_OVL_ERR_WORKSPACE;
    if (h->num_rows < 0 || h->num_rows > c.max_rows || !h->expert_counts || !h->out) return MOE_OVL_ERR_INVALID_ARG;
    if (h->num_rows > 0 && (!h->x || !h->src_rank || !h->src_token || !h->gate)) return MOE_OVL_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(h->stream);
    const size_t M = (size_t)h->num_rows, d = c.d_model;
    const int slot = (int)(ctx->host_calls & 1);
    const bool reused = ctx->host_calls >= 2;          // this slot has been through a full pass before
    CU_CHECK(ctx, cudaSetDevice(c.device));
    // inputs: on the copy-in stream, once the pass that last read this slot's staging buffers is done
    if (reused) CU_CHECK(ctx, cudaStreamWaitEvent(ctx->s_h2d, ctx->ev_comp[slot], 0));
    CU_CHECK(ctx, cudaMemcpyAsync(ctx->ws + L.st_counts[slot], h->expert_counts, (size_t)c.num_local_experts * 4,
                                  cudaMemcpyHostToDevice, ctx->s_h2d));
    if (M > 0) {
        CU_CHECK(ctx, cudaMemcpyAsync(ctx->ws + L.st_x[slot], h->x, M * d * 2, cudaMemcpyHostToDevice, ctx->s_h2d));
        CU_CHECK(ctx, cudaMemcpyAsync(ctx->ws + L.st_rank[slot], h->src_rank, M * 4, cudaMemcpyHostToDevice, ctx->s_h2d));
        CU_CHECK(ctx, cudaMemcpyAsync(ctx->ws + L.st_token[slot], h->src_token, M * 4, cudaMemcpyHostToDevice, ctx->s_h2d));
        CU_CHECK(ctx, cudaMemcpyAsync(ctx->ws + L.st_gate[slot], h->gate, M * 4, cudaMemcpyHostToDevice, ctx->s_h2d));
    }
    CU_CHECK(ctx, cudaEventRecord(ctx->ev_h2d[slot], ctx->s_h2d));
    // the pass itself, on the caller's stream: needs this slot's inputs, and its staged output buffer free again
    CU_CHECK(ctx, cudaStreamWaitEvent(st, ctx->ev_h2d[slot], 0));
    if (reused) CU_CHECK(ctx, cudaStreamWaitEvent(st, ctx->ev_d2h[slot], 0));
    moe_ovl_args a;
    std::memset(&a, 0, sizeof(a));
    a.struct_size = sizeof(a);
    a.num_rows = h->num_rows;
    a.x = ctx->ws + L.st_x[slot];
    a.expert_counts = at<int32_t>(ctx, L.st_counts[slot]);
    a.src_rank = at<int32_t>(ctx, L.st_rank[slot]);
    a.src_token = at<int32_t>(ctx, L.st_token[slot]);
    a.gate = at<float>(ctx, L.st_gate[slot]);
    a.w1 = h->w1; a.w2 = h->w2;
    a.consumer_sm_count = h->consumer_sm_count;
    a.mode = h->mode;
    a.ret = ctx->ws + L.st_ret;
    a.ret_rows_per_rank = L.st_ret_rows;
    a.out = ctx->ws + L.st_out[slot];
    a.stream = h->stream;
    const int rc = moe_ovl_expert_return(ctx, &a);
    if (rc != MOE_OVL_OK) return rc;
    CU_CHECK(ctx, cudaEventRecord(ctx->ev_comp[slot], st));
    // result: on the copy-out stream, so that it overlaps the next call's pass
    CU_CHECK(ctx, cudaStreamWaitEvent(ctx->s_d2h, ctx->ev_comp[slot], 0));
    CU_CHECK(ctx, cudaMemcpyAsync(h->out, ctx->ws + L.st_out[slot], (size_t)c.num_src_ranks * c.tokens_per_rank * L.dout * 2,
                                  cudaMemcpyDeviceToHost, ctx->s_d2h));
    CU_CHECK(ctx, cudaEventRecord(ctx->ev_d2h[slot], ctx->s_d2h));
    ++ctx->host_calls;
    return MOE_OVL_OK;
}

int moe_ovl_host_join(moe_ovl_ctx *ctx, void *stream)
{
    if (!ctx) return MOE_OVL_ERR_INVALID_ARG;
    if (!(ctx->cfg.flags & MOE_OVL_FLAG_HOST_STAGING)) return MOE_OVL_ERR_WORKSPACE;
    const unsigned long long n = ctx->host_calls < 2 ? ctx->host_calls : 2;
    for (unsigned long long k = 0; k < n; ++k)
        CU_CHECK(ctx, cudaStreamWaitEvent(static_cast<cudaStream_t>(stream), ctx->ev_d2h[(ctx->host_calls - 1 - k) & 1], 0));
    return MOE_OVL_OK;
}

int moe_ovl_query_status(moe_ovl_ctx *ctx, int32_t *code, int64_t *detail)
{
    if (!ctx) return MOE_OVL_ERR_INVALID_ARG;
    int rc = sync_last(ctx);
    if (rc != MOE_OVL_OK) return rc;
    int st[ST_COUNT] = {0, 0, 0, 0};
    CU_CHECK(ctx, cudaMemcpy(st, ctx->ws + ctx->L.status, sizeof(st), cudaMemcpyDeviceToHost));
    if (code) *code = st[ST_CODE];
    if (detail) *detail = ((int64_t)st[ST_DETAIL_HI] << 32) | (uint32_t)st[ST_DETAIL_LO];
    return MOE_OVL_OK;
}

int moe_ovl_get_report(moe_ovl_ctx *ctx, moe_ovl_report *r)
{
    if (!ctx || !r) return MOE_OVL_ERR_INVALID_ARG;
    std::memset(r, 0, sizeof(*r));
    if (!ctx->ran) return MOE_OVL_OK;
    int rc = sync_last(ctx);
    if (rc != MOE_OVL_OK) return rc;
    int meta[META_COUNT];
    CU_CHECK(ctx, cudaMemcpy(meta, ctx->ws + ctx->L.meta, sizeof(meta), cudaMemcpyDeviceToHost));
    r->padded_rows = meta[META_P];
    r->num_bands = meta[META_BANDS];
    r->num_items = meta[META_ITEMS];
    r->num_segments = meta[META_SEGS];
    r->producer_ctas = ctx->last_prod_ctas;
    r->consumer_ctas = ctx->last_cons_ctas;
    r->kernel_launches = ctx->last_launches;
    r->mode_used = ctx->last_mode;
    if (ctx->last_mode != MOE_OVL_MODE_NON_OVERLAP) {
        const int nseg = meta[META_SEGS];
        const int whole = ctx->last_tail_segs < 0 ? 0 : std::max(0, nseg - ctx->last_tail_segs);
        r->return_units = whole + (nseg - whole) * ctx->last_chunks;
    }
    r->timing_valid = ctx->last_timed ? 1 : 0;
    if (ctx->last_timed) {
        float prod_end = 0.f, mover_end = 0.f;
        CU_CHECK(ctx, cudaEventElapsedTime(&r->ms_total, ctx->t_begin, ctx->t_end));
        const cudaEvent_t p0 = ctx->h_p0[ctx->last_hist], p1 = ctx->h_p1[ctx->last_hist];
        CU_CHECK(ctx, cudaEventElapsedTime(&r->ms_prep, ctx->t_begin, p0));
        CU_CHECK(ctx, cudaEventElapsedTime(&r->ms_producer, p0, p1));
        prod_end = r->ms_producer;
        if (!ctx->last_dedicated && ctx->last_mode == MOE_OVL_MODE_IN_KERNEL) {
            r->ms_mover = 0.f;                  // the return is inside the GEMM kernel: no phase of its own
            mover_end = prod_end;
        } else {
            CU_CHECK(ctx, cudaEventElapsedTime(&r->ms_mover, ctx->last_dedicated ? ctx->t_m0 : p1, ctx->t_m1));
            CU_CHECK(ctx, cudaEventElapsedTime(&mover_end, p0, ctx->t_m1));
        }
        r->ms_expert_return = std::max(prod_end, mover_end);
        r->ms_combine = r->ms_total - r->ms_prep - r->ms_expert_return;
    }
    if (ctx->last_mode != MOE_OVL_MODE_NON_OVERLAP && meta[META_SEGS] > 0) {
        unsigned long long st[STAMP_COUNT];
        int misc[4];
        CU_CHECK(ctx, cudaMemcpy(st, ctx->ws + ctx->L.stamps, sizeof(st), cudaMemcpyDeviceToHost));
        CU_CHECK(ctx, cudaMemcpy(misc, ctx->ws + ctx->L.next_item, sizeof(misc), cudaMemcpyDeviceToHost));
        const unsigned long long t0 = ~st[STAMP_START_INV], first = ~st[STAMP_FIRST_FLAG_INV];
        if (st[STAMP_FIRST_FLAG_INV] != 0 && st[STAMP_LAST_SEG] != 0) {
            r->us_first_flag = (float)((double)(first - t0) / 1e3);
            r->us_gemm_done = (float)((double)(st[STAMP_LAST_FLAG] - t0) / 1e3);
            r->us_return_done = (float)((double)(st[STAMP_LAST_SEG] - t0) / 1e3);
            const double window = (double)r->us_return_done - r->us_first_flag;
            const double exposed = std::max(0.0, (double)r->us_return_done - r->us_gemm_done);
            r->overlap_ratio = window > 0 ? (float)(1.0 - exposed / window) : 1.0f;
        }
        r->segments_by_gemm_ctas = misc[3];
        if (st[STAMP_COPY_NS] > 0) r->copy_gbs_per_cta = (float)((double)st[STAMP_COPY_BYTES] / (double)st[STAMP_COPY_NS]);
    }
    return MOE_OVL_OK;
}

int moe_ovl_get_plan(moe_ovl_ctx *ctx, const moe_ovl_plan_view *v)
{
    if (!ctx || !v) return MOE_OVL_ERR_INVALID_ARG;
    if (!ctx->ran) return MOE_OVL_ERR_INVALID_ARG;
    int rc = sync_last(ctx);
    if (rc != MOE_OVL_OK) return rc;
    const Layout &L = ctx->L;
    const moe_ovl_config &c = ctx->cfg;
    int meta[META_COUNT];
    CU_CHECK(ctx, cudaMemcpy(meta, ctx->ws + L.meta, sizeof(meta), cudaMemcpyDeviceToHost));
    const size_t B = (size_t)meta[META_BANDS], M = (size_t)ctx->last_rows;
    const size_t ntokk = (size_t)c.num_src_ranks * c.tokens_per_rank * L.kmax;
    struct { void *dst; size_t off, bytes; } cp[] = {
        {v->group_rows, L.group_rows, (size_t)c.num_local_experts * c.num_src_ranks * 4},
        {v->pos, L.pos, M * 4},
        {v->band_expert, L.band_expert, B * 4},
        {v->band_dest, L.band_dest, B * 4},
        {v->band_valid, L.band_valid, B * 4},
        {v->band_slot0, L.band_slot0, B * 4},
        {v->sched_band, L.sched_band, B * 4},
        {v->item, L.items, (size_t)meta[META_ITEMS] * 16},
        {v->seg, L.segs, (size_t)meta[META_SEGS] * 16},
        {v->tok_slot, L.tok_slot, ntokk * 4},
        {v->tok_gate, L.tok_gate, ntokk * 4},
    };
    for (auto &e : cp)
        if (e.dst && e.bytes) CU_CHECK(ctx, cudaMemcpy(e.dst, ctx->ws + e.off, e.bytes, cudaMemcpyDeviceToHost));
    if (v->tok_slot)                           // stored as slot + 1 with 0 = none; reported as slot with -1 = none
        for (size_t i = 0; i < ntokk; ++i) v->tok_slot[i] -= 1;
    return MOE_OVL_OK;
}

int moe_ovl_get_gemm_time(moe_ovl_ctx *ctx, int32_t last_n, float *avg_ms, int32_t *n_used)
{
    if (!ctx || !avg_ms || last_n < 1) return MOE_OVL_ERR_INVALID_ARG;
    int rc = sync_last(ctx);
    if (rc != MOE_OVL_OK) return rc;
    const int have = (int)std::min<unsigned long long>(ctx->calls, MOE_OVL_TIMING_HISTORY);
    const int n = std::min<int>(last_n, have);
    double sum = 0;
    int used = 0;
    for (int k = 1; k <= n; ++k) {
        const int i = (int)((ctx->calls - k) % MOE_OVL_TIMING_HISTORY);
        if (!ctx->hist_timed[i]) continue;          // a captured call: its events carry no time
        float ms = 0.f;
        CU_CHECK(ctx, cudaEventElapsedTime(&ms, ctx->h_p0[i], ctx->h_p1[i]));
        sum += ms;
        ++used;
    }
    *avg_ms = used ? (float)(sum / used) : 0.f;
    if (n_used) *n_used = used;
    return MOE_OVL_OK;
}

int moe_ovl_get_sm_map(moe_ovl_ctx *ctx, int32_t *producer_smid, int32_t *consumer_smid)
{
    if (!ctx || !ctx->ran) return MOE_OVL_ERR_INVALID_ARG;
    int rc = sync_last(ctx);
    if (rc != MOE_OVL_OK) return rc;
    if (producer_smid && ctx->last_prod_ctas > 0)
        CU_CHECK(ctx, cudaMemcpy(producer_smid, ctx->ws + ctx->L.smid, (size_t)ctx->last_prod_ctas * 4,
                                 cudaMemcpyDeviceToHost));
    if (consumer_smid && ctx->last_cons_ctas > 0)
        CU_CHECK(ctx, cudaMemcpy(consumer_smid, ctx->ws + ctx->L.smid + 1024 * 4, (size_t)ctx->last_cons_ctas * 4,
                                 cudaMemcpyDeviceToHost));
    return MOE_OVL_OK;
}

int moe_ovl_read_buffer(moe_ovl_ctx *ctx, int32_t which, size_t offset, size_t bytes, void *host_dst)
{
    if (!ctx || !host_dst) return MOE_OVL_ERR_INVALID_ARG;
    const Layout &L = ctx->L;
    const size_t P = (size_t)L.max_bands * TB_M;
    size_t base, cap;
    switch (which) {
    case MOE_OVL_BUF_XA: base = L.Xa; cap = P * ctx->cfg.d_model * 2; break;
    case MOE_OVL_BUF_H: base = L.H; cap = P * (size_t)L.f_eff * 2; break;
    case MOE_OVL_BUF_Y: base = L.Y; cap = P * (size_t)L.dout * 2; break;
    default: return MOE_OVL_ERR_INVALID_ARG;
    }
    if (offset > cap || bytes > cap - offset) return MOE_OVL_ERR_INVALID_ARG;
    int rc = sync_last(ctx);
    if (rc != MOE_OVL_OK) return rc;
    if (bytes) CU_CHECK(ctx, cudaMemcpy(host_dst, ctx->ws + base + offset, bytes, cudaMemcpyDeviceToHost));
    return MOE_OVL_OK;
}

int moe_ovl_get_trace(moe_ovl_ctx *ctx, void *host_buf, size_t bytes, size_t *written)
{
    if (!ctx || !written) return MOE_OVL_ERR_INVALID_ARG;
    *written = 0;
    const Layout &L = ctx->L;
    if (!L.trace_bytes) return MOE_OVL_ERR_UNSUPPORTED;
    if (!ctx->ran) return MOE_OVL_OK;
    int rc = sync_last(ctx);
    if (rc != MOE_OVL_OK) return rc;
    int meta[META_COUNT];
    unsigned long long st[STAMP_COUNT];
    CU_CHECK(ctx, cudaMemcpy(meta, ctx->ws + L.meta, sizeof(meta), cudaMemcpyDeviceToHost));
    CU_CHECK(ctx, cudaMemcpy(st, ctx->ws + L.stamps, sizeof(st), cudaMemcpyDeviceToHost));
    const size_t n_items = (size_t)meta[META_ITEMS];
    const size_t nseg = (size_t)meta[META_SEGS];
    const size_t whole = ctx->last_tail_segs < 0 ? 0 : (nseg > (size_t)ctx->last_tail_segs ? nseg - ctx->last_tail_segs : 0);
    const size_t n_units = ctx->last_mode == MOE_OVL_MODE_NON_OVERLAP ? 0 : whole + (nseg - whole) * ctx->last_chunks;
    const size_t need = (n_items + n_units) * sizeof(moe_ovl_trace_record);
    if (!host_buf) { *written = need; return MOE_OVL_OK; }
    if (bytes < need) return MOE_OVL_ERR_INVALID_ARG;
    TraceRec *items = new (std::nothrow) TraceRec[2 * n_items + n_units + 1];
    TraceRec *items2 = items ? items + n_items + n_units : nullptr;
    int2 *ctas = new (std::nothrow) int2[n_items + 1];
    if (!items || !ctas) { delete[] items; delete[] ctas; return MOE_OVL_ERR_INVALID_ARG; }
    cudaError_t e = cudaSuccess;
    if (n_items) e = cudaMemcpy(items, ctx->ws + L.trace_items, n_items * sizeof(TraceRec), cudaMemcpyDeviceToHost);
    if (e == cudaSuccess && n_items)
        e = cudaMemcpy(ctas, ctx->ws + L.trace_item_aux, n_items * 8, cudaMemcpyDeviceToHost);
    if (e == cudaSuccess && n_items)
        e = cudaMemcpy(items2, ctx->ws + L.trace_items2, n_items * sizeof(TraceRec), cudaMemcpyDeviceToHost);
    if (e == cudaSuccess && n_units)
        e = cudaMemcpy(items + n_items, ctx->ws + L.trace_units, n_units * sizeof(TraceRec), cudaMemcpyDeviceToHost);
    if (e != cudaSuccess) {
        delete[] items; delete[] ctas;
        ctx->last_cuda_error = (int)e;
        return MOE_OVL_ERR_CUDA;
    }
    const unsigned long long t0 = ~st[STAMP_START_INV];
    auto rel = [&](unsigned long long t) -> int64_t { return t ? (int64_t)(t - t0) : -1; };
    moe_ovl_trace_record *out = static_cast<moe_ovl_trace_record *>(host_buf);
    for (size_t i = 0; i < n_items; ++i) {
        moe_ovl_trace_record &r = out[i];
        std::memset(&r, 0, sizeof(r));
        r.kind = MOE_OVL_TRACE_ITEM; r.index = (int32_t)i; r.cta = ctas[i].x; r.ns_operand_wait = ctas[i].y;
        r.ns_claim = rel(items[i].a); r.ns_ready = rel(items[i].b);
        r.ns_done0 = rel(items[i].c); r.ns_done1 = rel(items[i].d);
        r.ns_epilogue_start = rel(items2[i].a);
        r.ns_first_operand_wait = (int64_t)items2[i].b;
        r.ns_accumulator_wait = (int64_t)items2[i].c;
        r.ns_inputs_ready = rel(items2[i].d);
    }
    for (size_t u = 0; u < n_units; ++u) {
        const TraceRec &t = items[n_items + u];
        moe_ovl_trace_record &r = out[n_items + u];
        std::memset(&r, 0, sizeof(r));
        r.kind = MOE_OVL_TRACE_UNIT; r.index = (int32_t)(t.d >> 32); r.cta = (int32_t)(t.a & 0xffffffffu);
        r.who = (int32_t)(t.a >> 32); r.rows = (int32_t)(t.d & 0xffffffu); r.chunks = (int32_t)((t.d >> 24) & 0xff);
        r.ns_claim = r.ns_ready = rel(t.b);
        r.ns_done0 = r.ns_done1 = rel(t.c);
    }
    delete[] items; delete[] ctas;
    *written = need;
    return MOE_OVL_OK;
}

}  // extern "C"

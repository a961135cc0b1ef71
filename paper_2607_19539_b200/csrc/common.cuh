// Shared definitions of the moe_ovl kernels: the parameter block every kernel
// receives, the device status word, and small PTX wrappers for ordered memory
// access and bounded waiting.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

namespace moe_ovl {

constexpr int TB_M = 128;     // rows per band (tb_M of Algorithm 1)
constexpr int TB_N = 256;     // accumulator width of one tile (both GEMMs)
constexpr int TB_K = 64;      // K extent of one pipeline stage: 64 bf16 = one 128-byte swizzle row
constexpr int H_TILE = 128;   // hidden columns per first-GEMM tile (gate half + up half of the accumulator)

constexpr int KIND_G1 = 0;    // x . W1 (gate | up) -> SiLU * up -> H
constexpr int KIND_G2 = 1;    // H . W2 -> Y, raises the consumer-visible flag
// The same two GEMMs with the operands swapped, for runs whose bands hold at most SMALL_BAND_ROWS valid rows each:
// 256 weight rows are the MMA's M side and the valid rows of a GROUP of such bands (each rounded up to 16, at
// most SWAP_MAX_N together) its N side, so the tensor cores do not multiply padding and one pass over a weight
// tile serves the whole group.
constexpr int KIND_G1S = 2;
constexpr int KIND_G2S = 3;
// Bit of the item kind, on KIND_G1 / KIND_G2 only: both bands of the pair hold at most SMALL_BAND_ROWS valid rows,
// so the pair is computed as an M = 128 MMA (64 rows per CTA), which takes about 0.9 of the time of M = 256 (each MMA
// still reads the whole 256-row B tile from shared memory).
constexpr int KIND_LOW = 4;
// Bit of the item kind, on KIND_G1 / KIND_G2 only: three or four consecutive bands of one run, each with at most
// SMALL_BAND_ROWS valid rows, stacked into one full-height item: CTA c computes rows 0..63 of bands 2c and 2c + 1
// in the upper and lower half of its 128 accumulator lanes.  Item = {kind | expert << 8, first band, bands, tile}.
constexpr int KIND_STACK = 8;
constexpr int SMALL_BAND_ROWS = 64;
constexpr int SWAP_MAX_N = 128;
constexpr int SWAP_MAX_BANDS = 8;          // SWAP_MAX_N / 16

// meta[] slots written by the plan kernel
enum { META_P = 0, META_BANDS, META_ITEMS, META_SEGS, META_SUPERBANDS, META_GATHER_ORDER, META_COUNT = 8 };
// stamps[] slots.  "first" stamps hold ~t so that the cleared state (0) is neutral under atomicMax.
enum { STAMP_START_INV = 0, STAMP_FIRST_FLAG_INV, STAMP_LAST_FLAG, STAMP_LAST_SEG, STAMP_COPY_NS, STAMP_COPY_BYTES,
       STAMP_COUNT };
// status[] slots
enum { ST_CODE = 0, ST_ABORT = 1, ST_DETAIL_LO = 2, ST_DETAIL_HI = 3, ST_COUNT = 4 };

// who moved a unit of the return (trace records)
enum { TRACE_BY_CONSUMER = 0, TRACE_BY_GEMM_TAIL = 1, TRACE_BY_GEMM_WARPS = 2 };

constexpr int ERR_TIMEOUT = -5;
constexpr int ERR_BAD_ROUTING = -6;

// wait sites reported in the high bits of the status detail
enum : long long {
    SITE_TMA_EMPTY = 1, SITE_TMA_HCOUNT, SITE_MMA_FULL, SITE_MMA_TEMPTY, SITE_EPI_TFULL, SITE_CONS_FLAG,
    SITE_MMA_DRAIN, SITE_TMA_DRAIN, SITE_CLAIM, SITE_SCHED_GO, SITE_TMA_XREADY,
    SITE_ROW_RANGE = 16, SITE_ROW_DUP, SITE_COUNT_SUM, SITE_TOK_OVERFLOW, SITE_RET_OVERFLOW
};

struct __align__(32) TraceRec { unsigned long long a, b, c, d; };

struct Params {
    // problem
    int R, r_self, T, El, kmax, d, F;
    int dout;           // width of Y / ret / out rows: d for FFN experts, N for single-projection experts
    int k2;             // K extent of the GEMM that writes Y: F for FFN experts, d for single-projection experts
    int single;         // single-projection experts: no first GEMM, the output GEMM reads Xa
    int M;
    int mgb;            // bands per middle segment
    int seg_chunks;     // equal row slices a sliced segment is moved in
    int tail_segs;      // how many of the schedule's LAST segments are sliced (-1: all of them); the others are moved whole
    int group_bands;    // bands interleaved in one super-band
    int lag_items;      // schedule items between a band's last first-GEMM tile and its first second-GEMM tile
    int words;          // 32-bit words of one (expert, rank) token bitmap = ceil(T / 32)
    int n1, n2;         // tiles per band: F / 128 (0 for single-projection experts) and dout / 256
    int zero_early;     // overlapped return: the movers write the rows of `out` whose token selected no local expert
                        // while they have nothing to move yet; the combine kernel then skips those rows
    int low_ok;         // band pairs whose bands hold at most SMALL_BAND_ROWS rows each are issued with KIND_LOW;
                        // 2: and two such pairs side by side as one KIND_STACK item; 3: and an expert's small local band
                        // may join the last item of its remote bands
    int swap_ok;        // runs of small groups may use the swapped-operand items (needs F % 256 == 0 for FFN experts):
                        // 0 never, 1 where the plan's cost rule says so, 2 every eligible run (test hook)
    int max_bands, max_items;
    unsigned *epoch_rw;      // same word, for the plan kernel
    const unsigned *epoch;   // device word: number of this call; the plan kernel bumps it once per call
    unsigned long long timeout_ns;
    long long ret_rows_per_rank;
    // inputs
    const uint16_t *x;
    const int *expert_counts, *src_rank, *src_token;
    const float *gate;
    // outputs
    uint16_t *ret, *out;
    int *slot_out, *rows_per_rank_out, *segs_per_rank_out;
    // workspace
    uint16_t *Xa, *H, *Y;
    unsigned *bitmap;     // [El*R][words]
    int *wordpfx;         // [El*R][words] exclusive popcount prefix inside a group
    int *group_rows;      // [El*R] n[e][r]
    int *group_start;     // [El*R] aligned position of the group's first row
    int *group_slot;      // [El*R] slot of the group's first row in ret[r]
    int *pos;             // [M]
    int *slot;            // [M]
    int *band_expert, *band_dest, *band_valid, *band_slot0;   // [max_bands]
    int *sched_band;      // [max_bands]
    int *gather_band;     // [max_bands] bands in the order they are gathered, when meta[META_GATHER_ORDER] is set
    int4 *items;          // [max_items] {kind | expert << 8, band 0, band 1 or -1, tile}
    int4 *segs;           // [max_bands] {first band, bands, dest, rows}
    int *seg_slot0;       // [max_bands]
    int *tok_slot;        // [R*T*kmax] slot + 1 of each of the token's rows, ascending expert; 0 = none
    float *tok_gate;      // [R*T*kmax]
    int *plan_ticket;     // blocks of the plan kernel that have finished marking
    unsigned long long *stamps;   // [STAMP_COUNT] device timestamps of the call, see the enum
    int *smid_prod, *smid_cons;   // SM of every GEMM / consumer CTA
    int *assist_segs;     // segments moved by GEMM CTAs
    int *next_seg;        // segments claimed so far (consumer CTAs, and GEMM CTAs once they are out of tiles)
    int *next_item;       // schedule items claimed so far (GEMM CTA pairs take them in order)
    int *next_gather;     // gather units claimed so far (GEMM CTAs' gather warps)
    int *next_zero;       // chunks of tokens claimed so far by the movers that write the all-zero rows of `out`
    int *row_at;          // [P] input row held by every aligned position (valid positions only)
    unsigned *xready;     // [max_bands] rows of the band gathered into Xa (128 = ready)
    unsigned *hcount;     // [max_bands] first-GEMM tiles finished per band
    unsigned *flags;      // [max_bands*n2] epoch of the call that finished the tile
    unsigned *fcount;     // [max_bands*n2] swapped-operand items: CTAs of the pair that have stored their half of the tile
    int *meta;            // [META_COUNT]
    // optional trace (null when off), raw %globaltimer values: one record per schedule item {claimed, first
    // operands landed, published by CTA 0 of the pair, published by CTA 1} plus trace_item_aux, and
    // one per moved unit {who << 32 | CTA, flags seen, copy done, rows}
    TraceRec *trace_items, *trace_units;
    int2 *trace_item_aux;   // {leader CTA, ns the MMA-issuing thread waited for operand stages during the item}
    TraceRec *trace_items2; // {epilogue of CTA 0 saw the accumulator, ns the MMA thread waited for the item's first
                            //  stage, ns it waited for a free accumulator, unused}
    int *status;          // [ST_COUNT]
};

// ------------------------------------------------------------------ ordered access

__device__ __forceinline__ unsigned ld_acquire_u32(const unsigned *p)
{
    unsigned v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ void st_release_u32(unsigned *p, unsigned v)
{
    asm volatile("st.release.gpu.global.u32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}
__device__ __forceinline__ void red_release_add_u32(unsigned *p, unsigned v)
{
    asm volatile("red.release.gpu.global.add.u32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}
__device__ __forceinline__ int ld_volatile_s32(const int *p)
{
    int v;
    asm volatile("ld.volatile.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ unsigned long long globaltimer_ns()
{
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}

__device__ __forceinline__ void stamp_max(unsigned long long *slot, unsigned long long v) { atomicMax(slot, v); }
__device__ __forceinline__ unsigned smid()
{
    unsigned v;
    asm volatile("mov.u32 %0, %%smid;" : "=r"(v));
    return v;
}

// First error wins; every later waiter sees ST_ABORT and gives up at once.
__device__ __forceinline__ void report_error(int *status, int code, long long site, long long index)
{
    if (atomicCAS(&status[ST_CODE], 0, code) == 0) {
        long long detail = (site << 48) | (index & 0xffffffffffffll);
        status[ST_DETAIL_LO] = (int)(detail & 0xffffffffll);
        status[ST_DETAIL_HI] = (int)(detail >> 32);
    }
    __threadfence();
    atomicExch(&status[ST_ABORT], 1);
}

// Poll until *p == want (exact) or *p >= want (at_least), giving up at the deadline or when another waiter
// has aborted.  Returns false on give-up.  Between polls the thread sleeps, backing off up to max_sleep_ns:
// a waiter that spins hot takes power and L2 bandwidth from the GEMM it is waiting for.
__device__ __forceinline__ bool wait_global(const unsigned *p, unsigned want, bool at_least, const Params &prm,
                                            long long site, long long index, unsigned max_sleep_ns = 256)
{
    unsigned v = ld_acquire_u32(p);
    if (at_least ? (v >= want) : (v == want)) return true;
    const unsigned long long t0 = globaltimer_ns();
    unsigned sleep_ns = 32;
    for (unsigned it = 1;; ++it) {
        __nanosleep(sleep_ns);
        if (sleep_ns < max_sleep_ns) sleep_ns *= 2;
        v = ld_acquire_u32(p);
        if (at_least ? (v >= want) : (v == want)) return true;
        if ((it & 15u) == 0) {
            if (ld_volatile_s32(&prm.status[ST_ABORT])) return false;
            if (globaltimer_ns() - t0 > prm.timeout_ns) {
                report_error(prm.status, ERR_TIMEOUT, site, index);
                return false;
            }
        }
    }
}

}  // namespace moe_ovl

// Producer: one persistent kernel that runs the grouped SwiGLU FFN of all local
// experts from a single launch, following the plan's item list, and raises a ready
// flag per finished output tile (Section 3.3.1: rank-wide persistent GEMM with
// tile-level signalling in the epilogue).
//
// sm_100a design (the paper's is CUTLASS on A100): warp-specialised CTAs, one per SM, launched
// as clusters of two that share every MMA (cta_group::2): the pair computes a 256 x 256 tile,
// each CTA holding its own 128 rows of A and only HALF of the B tile, which cuts the operand
// traffic from L2 per SM by a third against a single-CTA 128 x 256 tile.
//   warp 0     TMA loads (cp.async.bulk.tensor, 128-byte swizzle, no multicast) into a 7-stage ring;
//              both CTAs' loads complete on the leader CTA's mbarrier.  It looks its next item up a few
//              stages before the current item's last load.
//   warp 1     in the leader CTA one thread issues tcgen05.mma (bf16 x bf16 -> fp32, M=256
//              N=256 K=16); accumulators in tensor memory, double buffered (2 x 256 columns)
//   warps 2-5  epilogue: tcgen05.ld -> fp32 math -> bf16 -> global, then publish
//   warps 7-10 gather: move the dispatched rows into the aligned layout Xa (Section 3.2.1) band by band in
//              schedule order while the tensor cores work, and count finished rows per band; the TMA warp
//              waits for a band's count before its first load.  The layout pass therefore costs no time
//              of its own except for the first few bands.  With the in-kernel return (PROD_WARP_MOVERS)
//              the same warps, once Xa is complete, take over the consumer's job on this SM: they claim
//              finished segments and move them into the receive buffers, so that no SM is set aside.
//   warp 6     scheduler (leader CTA): claims the next schedule item with an atomic counter, one
//              item ahead of the TMA warp, and hands it to every role of both CTAs through a
//              small ring in shared memory.  Items are claimed in schedule order, so the
//              remote-first order holds and every dependency still points to an earlier claim.
// A schedule item is a pair of 128-row bands of one expert (the second may be absent) times
// one tile (or three or four bands of at most 64 valid rows each, two per CTA: KIND_STACK); CTA rank r of the
// cluster owns band r of the pair:
//   first GEMM   A = Xa[band]; B = 128 gate rows of W1 (held by rank 0) and the matching 128
//                up rows (rank 1) -> one N=256 accumulator; the epilogue pairs column c with
//                c+128: h = silu(g) * u, 128 columns of H; then hcount[band] += 1 (release)
//   second GEMM  waits until hcount[band] == F/128, A = H[band], B = 256 rows of W2 (128 per
//                rank), writes 256 columns of Y; then flag[band][tile] = epoch (release)
// Runs of small (expert, rank) groups may come as items with the operands swapped (KIND_G1S / KIND_G2S):
// 256 weight rows on the MMA's M side, the valid rows of a group of up to 8 small bands on its N side,
// transposed epilogue (lane = output column); see common.cuh and the plan kernel's cost rule.
// The kernel exists in two builds: kTrace = true adds the per-item bookkeeping of the device trace.
// Every wait is bounded; on a give-up the CTA records a status, drains its copies,
// frees its tensor memory and returns.
#pragma once

#include <cuda.h>

#include "common.cuh"
#include "mover.cuh"

namespace moe_ovl {

constexpr int PROD_STAGES = 7;
constexpr int PROD_A_BYTES = TB_M * TB_K * 2;          // 16 KiB: this CTA's 128 rows of A
constexpr int PROD_B_BYTES = (TB_N / 2) * TB_K * 2;    // 16 KiB: this CTA's half of the B tile
constexpr int PROD_STAGE_BYTES = PROD_A_BYTES + PROD_B_BYTES;
constexpr int PROD_GATHER_WARPS = 4;
constexpr int PROD_THREADS = 224 + 32 * PROD_GATHER_WARPS;   // TMA, MMA, 4 epilogue warps, scheduler, gather warps
constexpr int GATHER_ROWS = 8;                         // rows per gather unit
constexpr int GATHER_HEAD_ROWS = 2;                    // ... in the first super-band of the schedule
constexpr int PROD_RING = 16;                          // claimed-item ring; roles are never more than 6 items apart
constexpr int PROD_LOOKAHEAD = 3;                      // stages before an item's last load at which the next item is looked up
constexpr int PROD_TMEM_COLS = 512;
// kernel flags
constexpr int PROD_RAISE_FLAGS = 1;    // publish a ready flag per finished output tile; idle CTAs help drain segments
constexpr int PROD_WARP_MOVERS = 2;    // in-kernel return: the gather warps move finished segments once Xa is complete
constexpr int PROD_SKIP_FIRST_BAND = 4; // test hook: the first band of the schedule is never gathered
constexpr int PROD_AUX_BYTES = 2048;   // barriers, claim ring (index, item record, inputs-complete mark), mover ints,
                                       // tables of the swapped-operand items
constexpr int PROD_SMEM_BYTES = PROD_STAGES * PROD_STAGE_BYTES + 1024 /*alignment slack*/ + PROD_AUX_BYTES;

// ------------------------------------------------------------------ PTX wrappers

__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}
// Non-blocking probe of a phase (try_wait may suspend the thread for a while before it answers).
__device__ __forceinline__ bool mbar_test_wait(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}
// Same test with acquire semantics at cluster scope: for barriers the peer CTA arrives on.
__device__ __forceinline__ bool mbar_try_wait_cluster(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}
// Bounded wait on an mbarrier phase.  False = gave up (deadline, or another waiter aborted).
template <bool kClusterScope = false>
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, const Params &prm, long long site,
                                          long long index)
{
    auto test = [&]() { return kClusterScope ? mbar_try_wait_cluster(bar, parity) : mbar_try_wait(bar, parity); };
    if (test()) return true;
    const unsigned long long t0 = globaltimer_ns();
    for (unsigned it = 1;; ++it) {
        if (test()) return true;
        if ((it & 255u) == 0) {
            if (ld_volatile_s32(&prm.status[ST_ABORT])) return false;
            if (globaltimer_ns() - t0 > prm.timeout_ns) {
                report_error(prm.status, ERR_TIMEOUT, site, index);
                return false;
            }
        }
    }
}

__device__ __forceinline__ uint32_t cluster_ctarank()
{
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
// shared::cluster address of the same shared-memory offset in CTA `rank` of this cluster
__device__ __forceinline__ uint32_t map_to_cta(uint32_t saddr, uint32_t rank)
{
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(saddr), "r"(rank));
    return r;
}
__device__ __forceinline__ void cluster_sync_all()
{
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// arrivals on a barrier that may live in the peer CTA (shared::cluster address)
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_bar)
{
    asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_bar) : "memory");
}
// Tile load into this CTA's shared memory; the bytes are counted on a barrier that may be the peer CTA's.
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap *map, uint32_t cluster_bar, int x, int y)
{
    asm volatile(
        "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes "
        "[%0], [%1, {%3, %4}], [%2];"
        ::"r"(dst), "l"(map), "r"(cluster_bar), "r"(x), "r"(y)
        : "memory");
}
__device__ __forceinline__ void prefetch_tmap(const CUtensorMap *map)
{
    asm volatile("prefetch.tensormap [%0];" ::"l"(map) : "memory");
}

__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

__device__ __forceinline__ void tmem_alloc(uint32_t dst_smem, uint32_t cols)
{
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(dst_smem), "r"(cols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t cols)
{
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(cols) : "memory");
}
// D[tmem] (+)= A[smem] * B[smem] over the CTA pair; bf16 inputs, fp32 accumulate
__device__ __forceinline__ void umma_bf16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                          uint32_t accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}
// The mbarrier at this offset gets one arrival in BOTH CTAs of the pair when every MMA issued so far by this
// thread has finished.
__device__ __forceinline__ void umma_commit_pair(uint32_t bar)
{
    asm volatile(
        "tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
        ::"r"(bar), "h"((uint16_t)3)
        : "memory");
}
// Same, this CTA's barrier only.
__device__ __forceinline__ void umma_commit_self(uint32_t bar)
{
    asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar)
                 : "memory");
}
// 32 lanes x 32 columns of fp32: thread t of the warp gets lane (base lane + t), 32 consecutive columns
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&v)[32])
{
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
          "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]),
          "=r"(v[16]), "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]),
          "=r"(v[24]), "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
        : "r"(taddr)
        : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// Shared-memory operand descriptor: K-major tile, 128-byte swizzle, rows of 128 bytes packed in groups of
// eight (stride between groups 1024 bytes), descriptor version 1.
__device__ __forceinline__ uint64_t umma_smem_desc(uint32_t saddr)
{
    uint64_t d = 0;
    d |= (uint64_t)((saddr & 0x3ffffu) >> 4);          // start address
    d |= (uint64_t)1 << 16;                            // leading byte offset (unused with swizzled K-major)
    d |= (uint64_t)(1024 >> 4) << 32;                  // stride byte offset
    d |= (uint64_t)1 << 46;                            // version
    d |= (uint64_t)2 << 61;                            // SWIZZLE_128B
    return d;
}
// Instruction descriptor: fp32 accumulator, bf16 A and B, both K-major, N=256, M=256 over the CTA pair.
constexpr uint32_t UMMA_IDESC = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(TB_N >> 3) << 17) |
                                ((uint32_t)((2 * TB_M) >> 4) << 24);

__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi)
{
    uint32_t r;
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
    return r;
}
__device__ __forceinline__ int ceil16_rows(int v) { return (v + 15) & ~15; }
__device__ __forceinline__ float silu_mul(float g, float u) { return __fdividef(g, 1.0f + __expf(-g)) * u; }

__device__ __forceinline__ void bar_sync_epilogue() { asm volatile("bar.sync 1, 128;" ::: "memory"); }
// AND over the 128 epilogue threads, so that they leave the tile loop together
__device__ __forceinline__ bool epilogue_all(bool ok)
{
    uint32_t r;
    asm volatile(
        "{\n\t.reg .pred p, q;\n\t"
        "setp.ne.u32 p, %1, 0;\n\t"
        "bar.red.and.pred q, 2, 128, p;\n\t"
        "selp.u32 %0, 1, 0, q;\n\t}"
        : "=r"(r)
        : "r"((uint32_t)ok)
        : "memory");
    return r != 0;
}

// ------------------------------------------------------------------ kernel

// One gather unit: ROWS rows of band `band` starting at row r0 are copied from the dispatched input into the
// aligned layout (padding rows zero-filled), COLS x 32 lanes x 16 bytes of every row per pass, i.e.
// ROWS * COLS loads in flight per lane; then the band's ready count goes up by ROWS (release).
template <int ROWS, int COLS>
__device__ __forceinline__ void gather_unit(const Params &p, int band, int r0, int lane)
{
    const int nv = p.d / 8;
    const int valid = p.band_valid[band];
    int src_row = -1;                                   // lanes 0..ROWS-1: source row, -1 for padding
    if (lane < ROWS && r0 + lane < valid) src_row = p.row_at[(size_t)band * TB_M + r0 + lane];
    for (int v0 = 0; v0 < nv; v0 += 32 * COLS) {
        uint4 buf[COLS][ROWS];
#pragma unroll
        for (int r = 0; r < ROWS; ++r) {
            const int sr = __shfl_sync(0xffffffffu, src_row, r);
            const uint4 *src = reinterpret_cast<const uint4 *>(p.x + (size_t)(sr >= 0 ? sr : 0) * p.d);
#pragma unroll
            for (int c = 0; c < COLS; ++c) {
                const int v = v0 + 32 * c + lane;
                buf[c][r] = (sr >= 0 && v < nv) ? __ldcs(src + v) : make_uint4(0, 0, 0, 0);
            }
        }
#pragma unroll
        for (int r = 0; r < ROWS; ++r) {
            uint4 *dst = reinterpret_cast<uint4 *>(p.Xa + ((size_t)band * TB_M + r0 + r) * p.d);
#pragma unroll
            for (int c = 0; c < COLS; ++c) {
                const int v = v0 + 32 * c + lane;
                if (v < nv) dst[v] = buf[c][r];
            }
        }
    }
    __threadfence();
    asm volatile("fence.proxy.async;" ::: "memory");      // Xa is read through TMA
    __syncwarp();
    if (lane == 0) red_release_add_u32(&p.xready[band], (unsigned)ROWS);
}

// Gather loop of one warp: Xa[band * 128 + r] = x[row_at[...]] for units of rows claimed in schedule order from a
// global counter; padding rows are zero-filled (Section 3.2.1).  It never waits, so the row counts the load warps
// poll always make progress.  The first super-band is gathered in small units (2 rows: done after two memory
// round trips at d = 4096) so that the first tiles can start a few microseconds after the kernel does; the rest in
// units of GATHER_ROWS rows, which cost fewer claims.
__device__ __forceinline__ void gather_units(const Params &p, int kflags, int lane)
{
    const int nbands = p.meta[META_BANDS];
    const int *order = p.meta[META_GATHER_ORDER] ? p.gather_band : p.sched_band;   // see the plan kernel, phase H
    const int head_bands = min(nbands, p.group_bands);
    const int head_units = head_bands * (TB_M / GATHER_HEAD_ROWS);
    const int nunits = head_units + (nbands - head_bands) * (TB_M / GATHER_ROWS);
    int unit = 0;
    if (lane == 0) unit = atomicAdd(p.next_gather, 1);
    unit = __shfl_sync(0xffffffffu, unit, 0);
    while (unit < nunits) {
        int next = 0;
        if (lane == 0) next = atomicAdd(p.next_gather, 1);      // claimed while this unit's rows are moving
        if ((kflags & PROD_SKIP_FIRST_BAND) && unit < TB_M / GATHER_HEAD_ROWS) {
            // test hook: leave band 0 of the schedule ungathered, so that the wait for it runs out
        } else if (unit < head_units) {
            const int per = TB_M / GATHER_HEAD_ROWS;
            gather_unit<GATHER_HEAD_ROWS, 16 / GATHER_HEAD_ROWS>(p, order[unit / per],
                                                                 (unit % per) * GATHER_HEAD_ROWS, lane);
        } else {
            const int u = unit - head_units, per = TB_M / GATHER_ROWS;
            gather_unit<GATHER_ROWS, 16 / GATHER_ROWS>(p, order[head_bands + u / per],
                                                       (u % per) * GATHER_ROWS, lane);
        }
        unit = __shfl_sync(0xffffffffu, next, 0);
    }
}

struct TrueT { static constexpr bool value = true; };
struct FalseT { static constexpr bool value = false; };

struct ProducerMaps {
    CUtensorMap xa, h, w1, w2;   // all 2-D bf16 row-major, box 64 x 128, 128-byte swizzle
    CUtensorMap xa8, h8;         // Xa and H again in boxes of 64 x 8: token rows of the swapped-operand items
    CUtensorMap xa64, h64, w1h;  // Xa, H and W1 in boxes of 64 x 64: operands of the 64-row-high pair items (KIND_LOW)
};

// Instruction descriptor of a KIND_LOW item: M = 128 over the CTA pair (64 rows per CTA), N = 256.
constexpr uint32_t UMMA_IDESC_LOW = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(TB_N >> 3) << 17) |
                                    ((uint32_t)(TB_M >> 4) << 24);

// Instruction descriptor of a swapped-operand MMA: 256 weight rows over the CTA pair, N = rows of the band group.
__device__ __forceinline__ uint32_t umma_idesc_n(int n)
{
    return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)((2 * TB_M) >> 4) << 24);
}
// acq_rel add that returns the old value: the second CTA of a pair to finish a tile learns that it is the second
__device__ __forceinline__ unsigned atom_add_acq_rel_u32(unsigned *p, unsigned v)
{
    unsigned old;
    asm volatile("atom.acq_rel.gpu.global.add.u32 %0, [%1], %2;" : "=r"(old) : "l"(p), "r"(v) : "memory");
    return old;
}

// Main loop of the MMA-issuing thread for one schedule item: per stage fill, wait for the operands, issue the
// four K=16 MMAs of the 64-wide K slice, free the stage.  This thread's instruction stream is on the kernel's
// critical path (a few dozen extra instructions per fill cost percents), so everything that varies is a
// template parameter: kPerK = 2 for the swapped first GEMM, whose gate and up halves take separate fills and
// accumulate in columns [0, ntok) and [ntok, 2 ntok); kTrace adds the wait-time bookkeeping of the trace.
template <bool kTrace, int kPerK>
__device__ __forceinline__ bool mma_mainloop(const Params &p, uint32_t smem_base, uint32_t bar_full, uint32_t bar_empty,
                                             int &stage, uint32_t &phase, int ksteps, uint32_t d_tmem, uint32_t idesc,
                                             int ntok, int it, unsigned long long &stall_ns,
                                             unsigned long long &w_first)
{
    for (int kk = 0; kk < ksteps; ++kk) {
#pragma unroll
        for (int half = 0; half < kPerK; ++half) {
            bool ok;
            if (kTrace && !mbar_test_wait(bar_full + 8 * stage, phase)) {
                const unsigned long long w0 = globaltimer_ns();
                ok = mbar_wait(bar_full + 8 * stage, phase, p, SITE_MMA_FULL, it);
                if (kk > 0 || half > 0) stall_ns += globaltimer_ns() - w0;   // the first fill is the item's start-up
                else w_first = globaltimer_ns() - w0;
            } else {
                ok = mbar_wait(bar_full + 8 * stage, phase, p, SITE_MMA_FULL, it);
            }
            if (!ok) return false;
            if (kTrace && kk == 0 && half == 0) p.trace_items[it].b = globaltimer_ns();
            tc_fence_after();
            const uint32_t sa = smem_base + stage * PROD_STAGE_BYTES, sb = sa + PROD_A_BYTES;
            const uint64_t adesc = umma_smem_desc(sa), bdesc = umma_smem_desc(sb);
            const uint32_t d_col = d_tmem + (uint32_t)(half * ntok);
#pragma unroll
            for (int k = 0; k < TB_K / 16; ++k)      // 16 bf16 = 32 bytes per MMA along K
                umma_bf16(d_col, adesc + (uint64_t)(k * 2), bdesc + (uint64_t)(k * 2), idesc, (kk | k) != 0 ? 1u : 0u);
            umma_commit_pair(bar_empty + 8 * stage);  // both CTAs may refill the stage once it has been read
            if (++stage == PROD_STAGES) { stage = 0; phase ^= 1u; }
        }
    }
    return true;
}

template <bool kTrace>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(PROD_THREADS, 1)
producer_kernel(const __grid_constant__ ProducerMaps maps, const Params p, const int kflags)
{
    const bool raise_flags = (kflags & PROD_RAISE_FLAGS) != 0;
    const bool warp_movers = (kflags & PROD_WARP_MOVERS) != 0;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t bars = smem_base + PROD_STAGES * PROD_STAGE_BYTES;
    // barrier slots, 8 bytes each
    const uint32_t bar_full = bars, bar_empty = bars + 8 * PROD_STAGES;
    const uint32_t bar_tfull = bars + 16 * PROD_STAGES, bar_tempty = bar_tfull + 16, bar_drain = bar_tempty + 16;
    const uint32_t tmem_slot = bar_drain + 8;
    const uint32_t bar_go = tmem_slot + 8;                         // TMA thread -> scheduler: "started an item"
    const uint32_t bar_ring = bar_go + 8;                          // PROD_RING barriers: slot filled
    const uint32_t ring = bar_ring + 8 * PROD_RING;                // PROD_RING claimed item indices
    const uint32_t mover_ints = ring + 4 * PROD_RING;              // two ints of the in-kernel movers
    // swapped-operand items: the load thread's band tables (this item and the next: band, rows per CTA) and the
    // epilogue's column -> buffer row maps (one per accumulator buffer, SWAP_MAX_N columns each)
    const uint32_t swap_tab = mover_ints + 8;                      // [2][SWAP_MAX_BANDS] int2
    const uint32_t swap_rowmap = swap_tab + 2 * SWAP_MAX_BANDS * 8;   // [2][SWAP_MAX_N] int
    // the scheduler also hands out the item's record and whether its inputs were already complete at the claim, so
    // that no role has to fetch them from global memory at an item boundary
    const uint32_t ring_item = swap_rowmap + 2 * SWAP_MAX_N * 4;   // PROD_RING int4 (16-byte aligned: see the assert)
    const uint32_t ring_dep = ring_item + 16 * PROD_RING;          // PROD_RING ints
    static_assert((16 * PROD_STAGES + 16 + 16 + 8 + 8 + 8 + 8 * PROD_RING + 4 * PROD_RING + 8 + 2 * SWAP_MAX_BANDS * 8 +
                   2 * SWAP_MAX_N * 4) % 16 == 0, "item records must be 16-byte aligned");
    static_assert(16 * PROD_STAGES + 16 + 16 + 8 + 8 + 8 + 8 * PROD_RING + 4 * PROD_RING + 8 + 2 * SWAP_MAX_BANDS * 8 +
                  2 * SWAP_MAX_N * 4 + 16 * PROD_RING + 4 * PROD_RING <= PROD_AUX_BYTES, "auxiliary shared memory");
    static_assert(PROD_SMEM_BYTES <= 232448, "dynamic shared memory of one CTA");
    uint8_t *smem_gen = smem_raw + (smem_base - smem_u32(smem_raw));
    volatile uint32_t *tmem_slot_gen = reinterpret_cast<volatile uint32_t *>(smem_gen + (tmem_slot - smem_base));
    volatile int *ring_gen = reinterpret_cast<volatile int *>(smem_gen + (ring - smem_base));
    volatile int *ring_item_gen = reinterpret_cast<volatile int *>(smem_gen + (ring_item - smem_base));
    volatile int *ring_dep_gen = reinterpret_cast<volatile int *>(smem_gen + (ring_dep - smem_base));
    // record of the n-th item of this cluster (valid once claimed(n) has returned it)
    auto claimed_item = [&](int n) -> int4 {
        const int slot = n % PROD_RING;
        return make_int4(ring_item_gen[4 * slot], ring_item_gen[4 * slot + 1], ring_item_gen[4 * slot + 2],
                         ring_item_gen[4 * slot + 3]);
    };

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = cluster_ctarank();          // 0 = leader: owns the barriers the pair synchronises on
    // shared::cluster addresses of the leader's barriers (for rank 0 these are its own)
    const uint32_t lead_full = map_to_cta(bar_full, 0), lead_tempty = map_to_cta(bar_tempty, 0);

    if (threadIdx.x == 0) {
        p.smid_prod[blockIdx.x] = (int)smid();
        stamp_max(&p.stamps[STAMP_START_INV], ~globaltimer_ns());
        for (int s = 0; s < PROD_STAGES; ++s) {
            mbar_init(bar_full + 8 * s, 1);       // the leader's TMA thread arrives, expecting both CTAs' bytes
            mbar_init(bar_empty + 8 * s, 1);
        }
        for (int a = 0; a < 2; ++a) {
            mbar_init(bar_tfull + 8 * a, 1);
            mbar_init(bar_tempty + 8 * a, 8);     // one arrival per epilogue warp of both CTAs
        }
        mbar_init(bar_drain, 1);
        mbar_init(bar_go, 1);
        for (int s = 0; s < PROD_RING; ++s) mbar_init(bar_ring + 8 * s, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async;" ::: "memory");
        prefetch_tmap(&maps.xa);
        prefetch_tmap(&maps.h);
        prefetch_tmap(&maps.w1);
        prefetch_tmap(&maps.w2);
        prefetch_tmap(&maps.xa8);
        prefetch_tmap(&maps.h8);
        prefetch_tmap(&maps.xa64);
        prefetch_tmap(&maps.h64);
        prefetch_tmap(&maps.w1h);
    }
    if (warp == 1) tmem_alloc(tmem_slot, PROD_TMEM_COLS);
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();                           // the peer's barriers exist before anything signals them
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot_gen;

    const int n_items = p.meta[META_ITEMS];
    const unsigned epoch = *p.epoch;
    // n-th item of this cluster: wait until the scheduler has filled ring slot n % PROD_RING, then read it.
    // Returns n_items (or more) when the schedule is exhausted, -1 on a give-up.
    auto claimed = [&](int n) -> int {
        const int slot = n % PROD_RING;
        if (!mbar_wait<true>(bar_ring + 8 * slot, (uint32_t)(n / PROD_RING) & 1u, p, SITE_CLAIM, n)) return -1;
        return ring_gen[slot];
    };

    if (warp == 0) {
        // ---------------- load warp (both CTAs).  Lane 0 looks the items up and issues the loads of band-pair
        // items; for swapped-operand items, whose token side is many small boxes, lanes 1..8 issue one box each
        // (one thread gets about one tensor copy per 0.1 us out of the door).
        int stage = 0;
        uint32_t phase = 0;
        long long fills = 0;
        bool ok = true;
        // What the loads of one schedule item need.  It is looked up -- ring slot, item record, the counter the
        // item depends on -- a few stages BEFORE the previous item's last load, so that these dependent
        // round trips to L2 do not open a bubble between two items.
        struct Job {
            int it, a_row, b_row, ksteps, dep_index;
            const CUtensorMap *amap, *bmap;
            const unsigned *dep;        // counter that must reach dep_want before the item's first load
            unsigned dep_want;
            long long dep_site;
            bool dep_ok;
            // swapped-operand items: weight rows are the A side; nb bands of tokens the B side (table in
            // shared memory, slot tab); gate and up projection take separate stage fills (fills = 2 * ksteps)
            int swap, nb, tab, half_rows, w_row, w_row_up, tok_is_x;
            // KIND_LOW: 64-row boxes for A; the first GEMM's B is two 64-row boxes (gate rows, up rows; b2_row >= 0)
            int low, b2_row;
            // KIND_STACK: A is two 64-row boxes, rows 0..63 of two bands (a2_row >= 0); the second band has a
            // counter of its own to wait for (dep2, may be null)
            int a2_row;
            const unsigned *dep2;
        };
        volatile int2 *tabs = reinterpret_cast<volatile int2 *>(smem_gen + (swap_tab - smem_base));
        // 1 = item n is in `j`, 0 = schedule exhausted, -1 = gave up.  Lane 0 only.
        auto fetch = [&](int n, Job &j) -> int {
            const int it = claimed(n);
            if (it < 0) return -1;
            if (it >= n_items) return 0;
            if (rank == 0) mbar_arrive(bar_go);  // lets the scheduler claim the item after this one
            const int4 item = claimed_item(n);   // {kind | expert << 8, band 0, band 1 or -1, tile}
            const bool pre_ok = ring_dep_gen[n % PROD_RING] != 0;   // inputs were complete when the item was claimed
            const int kind = item.x & 0xff, e = item.x >> 8, tile = item.w;
            j.it = it;
            j.swap = kind == KIND_G1S || kind == KIND_G2S;
            if (j.swap) {
                // {kind | expert << 8, first schedule position, bands | rows << 8, tile}
                j.nb = item.z & 0xff;
                j.tab = n & 1;
                j.half_rows = (item.z >> 8) / 2;
                const bool g1 = kind == KIND_G1S;
                if (g1) {
                    // this CTA's 128 of the tile's 256 hidden columns: gate rows, and the matching up rows
                    j.w_row = e * 2 * p.F + tile * 2 * H_TILE + (int)rank * H_TILE;
                    j.w_row_up = j.w_row + p.F;
                    j.amap = &maps.w1; j.tok_is_x = 1; j.ksteps = p.d / TB_K;
                } else {
                    j.w_row = e * p.dout + tile * TB_N + (int)rank * (TB_N / 2);
                    j.w_row_up = j.w_row;
                    j.amap = &maps.w2; j.tok_is_x = p.single; j.ksteps = p.k2 / TB_K;
                }
                const bool on_x = g1 || p.n1 == 0;     // depends on gathered rows, else on finished hidden tiles
                j.dep_site = on_x ? SITE_TMA_XREADY : SITE_TMA_HCOUNT;
                j.dep_want = on_x ? (unsigned)TB_M : (unsigned)p.n1;
                j.dep_ok = true;
                for (int i = 0; i < j.nb; ++i) {
                    const int b = p.sched_band[item.y + i];
                    tabs[j.tab * SWAP_MAX_BANDS + i].x = b;
                    tabs[j.tab * SWAP_MAX_BANDS + i].y = ceil16_rows(p.band_valid[b]) / 2;
                    j.dep_ok = j.dep_ok && ld_acquire_u32(on_x ? &p.xready[b] : &p.hcount[b]) >= j.dep_want;
                }
                j.dep = on_x ? p.xready : p.hcount;
                return 1;
            }
            const bool stack = (kind & KIND_STACK) != 0;
            // stacked bands: this CTA's are item.y + 2 * rank and, if the item has that many, the one after it
            const int band = stack ? item.y + 2 * (int)rank : ((rank == 0 || item.z < 0) ? item.y : item.z);
            const int band2 = (stack && 2 * (int)rank + 1 < item.z) ? band + 1 : -1;
            j.a_row = band * TB_M;
            // no second band: the box is filled with the first band's rows 64..127, whose results are not stored
            j.a2_row = stack ? (band2 >= 0 ? band2 * TB_M : j.a_row + TB_M / 2) : -1;
            j.dep2 = nullptr;
            j.dep_index = band;
            j.low = (kind & KIND_LOW) != 0;
            j.b2_row = -1;
            if ((kind & 3) == KIND_G1 && j.low) {
                // 64 rows per CTA: the accumulator's columns 0..127 (from CTA 0's B rows) land in lanes 0..63 and
                // columns 128..255 (CTA 1's) in lanes 64..127 of BOTH CTAs.  So that a lane holds the gate and the
                // up value of the same hidden column, each CTA's B rows are 64 gate rows followed by the matching
                // 64 up rows: rank 0 the tile's hidden columns 0..63, rank 1 columns 64..127.
                j.amap = &maps.xa64; j.bmap = &maps.w1h;
                j.b_row = e * 2 * p.F + tile * H_TILE + (int)rank * (H_TILE / 2);
                j.b2_row = j.b_row + p.F;
                j.ksteps = p.d / TB_K;
                j.dep = &p.xready[band]; j.dep_want = (unsigned)TB_M; j.dep_site = SITE_TMA_XREADY;
            } else if ((kind & 3) == KIND_G1) {
                j.amap = stack ? &maps.xa64 : &maps.xa; j.bmap = &maps.w1;
                // rank 0 holds the gate-projection rows of the tile, rank 1 the matching up-projection rows
                j.b_row = e * 2 * p.F + tile * H_TILE + (int)rank * p.F;
                j.ksteps = p.d / TB_K;
                // all 128 rows of the band (padding included) must have been gathered into Xa
                j.dep = &p.xready[band]; j.dep_want = (unsigned)TB_M; j.dep_site = SITE_TMA_XREADY;
                if (band2 >= 0) j.dep2 = &p.xready[band2];
            } else {
                // single-projection experts: the output GEMM reads the aligned input itself
                j.amap = (j.low || stack) ? (p.single ? &maps.xa64 : &maps.h64) : (p.single ? &maps.xa : &maps.h);
                j.bmap = &maps.w2;
                j.b_row = e * p.dout + tile * TB_N + (int)rank * (TB_N / 2);
                j.ksteps = p.k2 / TB_K;
                if (p.n1 > 0) {   // every first-GEMM tile of this band must have landed in H
                    j.dep = &p.hcount[band]; j.dep_want = (unsigned)p.n1; j.dep_site = SITE_TMA_HCOUNT;
                    if (band2 >= 0) j.dep2 = &p.hcount[band2];
                } else {
                    j.dep = &p.xready[band]; j.dep_want = (unsigned)TB_M; j.dep_site = SITE_TMA_XREADY;
                    if (band2 >= 0) j.dep2 = &p.xready[band2];
                }
            }
            j.dep_ok = pre_ok || (ld_acquire_u32(j.dep) >= j.dep_want &&      // the counters only grow
                                  (j.dep2 == nullptr || ld_acquire_u32(j.dep2) >= j.dep_want));
            return 1;
        };
        Job cur, nxt;
        cur.swap = 0;
        int have = 0;
        if (lane == 0) {
            have = fetch(0, cur);
            ok = have >= 0;
        }
        for (int n = 0;; ++n) {
            // item boundary: lanes 1..31 learn from lane 0 whether to go on and whether to help
            __syncwarp();
            const int go = __shfl_sync(0xffffffffu, (ok && have == 1) ? (cur.swap ? 2 : 1) : 0, 0);
            if (go == 0) break;
            if (go == 2) {
                // ---- swapped-operand item, all lanes.  Stage fill = 128 weight rows (A slot, lane 0) + the
                // group's token rows (B slot: this CTA's half of every band in boxes of 8 rows, lane 1 + box).
                // First-GEMM items alternate gate and up rows against the same tokens.
                if (lane == 0 && !cur.dep_ok) {
                    for (int i = 0; i < cur.nb && ok; ++i) {
                        const int b = tabs[cur.tab * SWAP_MAX_BANDS + i].x;
                        ok = wait_global(cur.dep + b, cur.dep_want, true, p, cur.dep_site, b);
                    }
                }
                // (No proxy fence here: every thread that writes rows the copies below read -- the gather warps, the
                // epilogue warps of first-GEMM tiles -- issues fence.proxy.async after its stores and before the
                // release this thread has acquired, which is what orders those generic-proxy writes before the
                // async-proxy reads.  A second fence on this side stalled the load thread at every item: 2 % of the
                // kernel where items are short.)
                if (kTrace && lane == 0 && rank == 0 && ok) p.trace_items2[cur.it].d = globaltimer_ns();
                __syncwarp();
                ok = __shfl_sync(0xffffffffu, (int)ok, 0) != 0;
                if (!ok) break;
                const int nb = __shfl_sync(0xffffffffu, cur.nb, 0), tab = __shfl_sync(0xffffffffu, cur.tab, 0);
                const int half_rows = __shfl_sync(0xffffffffu, cur.half_rows, 0);
                const int ksteps = __shfl_sync(0xffffffffu, cur.ksteps, 0);
                const int per_k = __shfl_sync(0xffffffffu, cur.w_row_up != cur.w_row ? 2 : 1, 0);
                const int tok_is_x = __shfl_sync(0xffffffffu, cur.tok_is_x, 0);
                const int it_now = __shfl_sync(0xffffffffu, cur.it, 0);
                stage = __shfl_sync(0xffffffffu, stage, 0);
                phase = __shfl_sync(0xffffffffu, phase, 0);
                const CUtensorMap *tokmap = tok_is_x ? &maps.xa8 : &maps.h8;
                // lane 1 + j owns box j of the B slot: which rows of which band are they?
                int my_row = -1;
                {
                    int box0 = 0;
                    for (int i = 0; i < nb; ++i) {
                        const int b = tabs[tab * SWAP_MAX_BANDS + i].x, h = tabs[tab * SWAP_MAX_BANDS + i].y;
                        const int j = lane - 1 - box0;
                        if (j >= 0 && 8 * j < h) my_row = b * TB_M + (int)rank * h + 8 * j;
                        box0 += h / 8;
                    }
                }
                const int fills_item = per_k * ksteps;
                const int look = fills_item > PROD_LOOKAHEAD ? fills_item - PROD_LOOKAHEAD : 0;
                const uint32_t tx = 2u * (uint32_t)(PROD_A_BYTES + half_rows * TB_K * 2);
                int have_next = 0;
                for (int f = 0; f < fills_item; ++f) {
                    const int ks = f / per_k;
                    bool fill_ok = mbar_wait(bar_empty + 8 * stage, phase ^ 1u, p, SITE_TMA_EMPTY, it_now);
                    fill_ok = __all_sync(0xffffffffu, fill_ok);
                    if (!fill_ok) { ok = false; break; }
                    const uint32_t sa = smem_base + stage * PROD_STAGE_BYTES, sb = sa + PROD_A_BYTES;
                    const uint32_t full = lead_full + 8 * stage;
                    if (lane == 0) {
                        if (rank == 0) mbar_arrive_expect_tx(bar_full + 8 * stage, tx);
                        tma_load_2d(sa, cur.amap, full, ks * TB_K, (f % per_k) ? cur.w_row_up : cur.w_row);
                        ++fills;
                    } else if (my_row >= 0) {
                        tma_load_2d(sb + (uint32_t)(lane - 1) * (8 * TB_K * 2), tokmap, full, ks * TB_K, my_row);
                    }
                    if (++stage == PROD_STAGES) { stage = 0; phase ^= 1u; }
                    if (f == look && lane == 0) {
                        have_next = fetch(n + 1, nxt);
                        if (have_next < 0) ok = false;
                    }
                }
                if (lane == 0) {
                    cur = nxt;
                    have = have_next;
                }
                continue;
            }
            if (lane != 0) continue;
            // ---- band-pair item, lane 0
            if (!cur.dep_ok) {
                ok = wait_global(cur.dep, cur.dep_want, true, p, cur.dep_site, cur.dep_index);
                if (ok && cur.dep2) ok = wait_global(cur.dep2, cur.dep_want, true, p, cur.dep_site, cur.dep_index + 1);
                if (!ok) continue;
            }
            // (no proxy fence on this side: the writers of the rows issue it before their release, see above)
            if (kTrace && rank == 0) p.trace_items2[cur.it].d = globaltimer_ns();
            // The leader announces the bytes of both CTAs.  The peer's bytes may land before this arrival; the
            // phase still cannot complete early because the arrival itself is pending.  The peer can only refill a
            // stage after the leader's MMAs have consumed (hence completed) its previous phase, so bytes never leak
            // into the wrong phase.
            // This loop sets the pace at which freed stages are refilled: one untaken branch more in it costs percents
            // of the kernel, so the copies per stage are compile-time variants and the look-up of the next item
            // sits between two runs of the loop.
            const uint32_t tx = cur.low ? 2 * (PROD_A_BYTES / 2 + PROD_B_BYTES) : 2 * PROD_STAGE_BYTES;
            const CUtensorMap *amap = cur.amap, *bmap = cur.bmap;
            const int a_row = cur.a_row, a2_row = cur.a2_row, b_row = cur.b_row, b2_row = cur.b2_row, it_now = cur.it;
            auto fill = [&](auto second_a, auto second_b, int ks0, int ks1) -> bool {
                uint32_t sa = smem_base + stage * PROD_STAGE_BYTES, off = 8 * stage;   // running addresses
                int x = ks0 * TB_K;
                for (int ks = ks0; ks < ks1; ++ks) {
                    if (!mbar_wait(bar_empty + off, phase ^ 1u, p, SITE_TMA_EMPTY, it_now)) {
                        fills += ks - ks0;      // the give-up path waits for the copies issued so far
                        return false;
                    }
                    const uint32_t full = lead_full + off;
                    if (rank == 0) mbar_arrive_expect_tx(bar_full + off, tx);
                    tma_load_2d(sa, amap, full, x, a_row);
                    if (decltype(second_a)::value) tma_load_2d(sa + PROD_A_BYTES / 2, amap, full, x, a2_row);
                    tma_load_2d(sa + PROD_A_BYTES, bmap, full, x, b_row);
                    if (decltype(second_b)::value) tma_load_2d(sa + PROD_A_BYTES + PROD_B_BYTES / 2, bmap, full, x, b2_row);
                    x += TB_K;
                    sa += PROD_STAGE_BYTES;
                    off += 8;
                    if (++stage == PROD_STAGES) { stage = 0; phase ^= 1u; sa = smem_base; off = 0; }
                }
                fills += ks1 - ks0;
                return true;
            };
            auto fill_any = [&](int ks0, int ks1) -> bool {
                if (cur.a2_row >= 0) return fill(TrueT{}, FalseT{}, ks0, ks1);      // stacked bands
                if (cur.b2_row >= 0) return fill(FalseT{}, TrueT{}, ks0, ks1);      // 64-row-high first GEMM
                return fill(FalseT{}, FalseT{}, ks0, ks1);
            };
            int have_next = 0;
            const int look = cur.ksteps > PROD_LOOKAHEAD ? cur.ksteps - PROD_LOOKAHEAD : 0;
            ok = fill_any(0, look + 1);
            if (!ok) continue;
            have_next = fetch(n + 1, nxt);
            if (have_next < 0) { ok = false; continue; }
            ok = fill_any(look + 1, cur.ksteps);
            if (!ok) continue;
            cur = nxt;
            have = have_next;
        }
        if (lane == 0 && !ok && rank == 0) {
            // give-up path: let the copies already issued land before the shared memory goes away
            const long long pending = fills < PROD_STAGES ? fills : PROD_STAGES;
            for (long long q = 1; q <= pending; ++q) {
                const long long f = fills - q;                       // index of an issued fill
                const int s = (int)(f % PROD_STAGES);
                const uint32_t par = (uint32_t)((f / PROD_STAGES) & 1);
                const unsigned long long t0 = globaltimer_ns();
                while (!mbar_try_wait(bar_full + 8 * s, par) && globaltimer_ns() - t0 < p.timeout_ns) {}
            }
        }
    } else if (warp == 1) {
        // ---------------- MMA issuer (leader CTA only; its MMAs run on both SMs of the pair)
        if (lane == 0 && rank == 0) {
            int stage = 0, acc = 0;
            uint32_t phase = 0, acc_phase = 0;
            bool ok = true;
            for (int n = 0; ok; ++n) {
                const int it = claimed(n);
                if (it < 0 || it >= n_items) break;
                const int4 item = claimed_item(n);
                const int kind = item.x & 0xff;
                const bool swap = kind == KIND_G1S || kind == KIND_G2S;
                const bool first_gemm = (kind & 3) == KIND_G1 || kind == KIND_G1S;
                const int ksteps = (first_gemm ? p.d : p.k2) / TB_K;
                const int ntok = swap ? item.z >> 8 : 0;
                const uint32_t idesc = swap ? umma_idesc_n(ntok) : ((kind & KIND_LOW) ? UMMA_IDESC_LOW : UMMA_IDESC);
                unsigned long long w_acc = 0, w_first = 0, stall_ns = 0;    // trace only
                if (kTrace && !mbar_try_wait_cluster(bar_tempty + 8 * acc, acc_phase ^ 1u)) {
                    const unsigned long long w0 = globaltimer_ns();
                    ok = mbar_wait<true>(bar_tempty + 8 * acc, acc_phase ^ 1u, p, SITE_MMA_TEMPTY, it);
                    w_acc = globaltimer_ns() - w0;
                } else {
                    ok = mbar_wait<true>(bar_tempty + 8 * acc, acc_phase ^ 1u, p, SITE_MMA_TEMPTY, it);
                }
                if (!ok) break;
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + (uint32_t)acc * TB_N;
                if (kind == KIND_G1S)
                    ok = mma_mainloop<kTrace, 2>(p, smem_base, bar_full, bar_empty, stage, phase, ksteps, d_tmem, idesc,
                                                 ntok, it, stall_ns, w_first);
                else
                    ok = mma_mainloop<kTrace, 1>(p, smem_base, bar_full, bar_empty, stage, phase, ksteps, d_tmem, idesc,
                                                 ntok, it, stall_ns, w_first);
                if (!ok) break;
                if (kTrace) {
                    p.trace_item_aux[it].y = (int)stall_ns;
                    p.trace_items2[it].b = w_first;
                    p.trace_items2[it].c = w_acc;
                }
                umma_commit_pair(bar_tfull + 8 * acc);        // accumulator complete, in both CTAs
                acc ^= 1;
                if (acc == 0) acc_phase ^= 1u;
            }
            // all MMAs issued by this thread must have finished before tensor memory is freed
            umma_commit_self(bar_drain);
            const unsigned long long t0 = globaltimer_ns();
            while (!mbar_try_wait(bar_drain, 0) && globaltimer_ns() - t0 < p.timeout_ns) {}
        }
    } else if (warp == 6) {
        // ---------------- scheduler (leader CTA): claim items in schedule order, one ahead of the TMA warp
        if (lane == 0 && rank == 0) {
            const uint32_t peer_ring = map_to_cta(ring, 1), peer_bar = map_to_cta(bar_ring, 1);
            const uint32_t peer_item = map_to_cta(ring_item, 1), peer_dep = map_to_cta(ring_dep, 1);
            for (int n = 0;; ++n) {
                // claim n is taken when the TMA thread starts item n-1: exactly one item ahead, so the claim's
                // latency is hidden and no role can fall a whole ring behind
                if (n >= 1 && !mbar_wait(bar_go, (uint32_t)(n - 1) & 1u, p, SITE_SCHED_GO, n)) break;
                const int it = atomicAdd(p.next_item, 1);
                if (kTrace && it < n_items) {
                    p.trace_items[it].a = globaltimer_ns();
                    p.trace_item_aux[it].x = (int)blockIdx.x;
                }
                // The item's record, and whether the rows it reads are complete already (they usually are: the gather
                // runs far ahead, and a band's second-GEMM tiles are issued well after its first-GEMM tiles), travel
                // with the claim.  This thread is a whole item ahead of the loads, so its round trips cost nothing.
                int4 item = make_int4(0, 0, 0, 0);
                int pre_ok = 0;
                if (it < n_items) {
                    item = p.items[it];
                    const int kind = item.x & 0xff;
                    if (kind != KIND_G1S && kind != KIND_G2S) {
                        const bool on_x = (kind & 3) == KIND_G1 || p.n1 == 0;
                        const unsigned *cnt = on_x ? p.xready : p.hcount;
                        const unsigned want = on_x ? (unsigned)TB_M : (unsigned)p.n1;
                        const int b0 = item.y, nb = (kind & KIND_STACK) ? item.z : 1;
                        unsigned lo = ld_acquire_u32(cnt + b0);
                        for (int i = 1; i < nb; ++i) lo = min(lo, ld_acquire_u32(cnt + b0 + i));
                        if (!(kind & KIND_STACK) && item.z >= 0) lo = min(lo, ld_acquire_u32(cnt + item.z));
                        pre_ok = lo >= want;
                    }
                }
                const int slot = n % PROD_RING;
                ring_gen[slot] = it;
                ring_item_gen[4 * slot] = item.x; ring_item_gen[4 * slot + 1] = item.y;
                ring_item_gen[4 * slot + 2] = item.z; ring_item_gen[4 * slot + 3] = item.w;
                ring_dep_gen[slot] = pre_ok;
                asm volatile("st.shared::cluster.u32 [%0], %1;" ::"r"(peer_ring + 4 * slot), "r"(it) : "memory");
                asm volatile("st.shared::cluster.v4.u32 [%0], {%1, %2, %3, %4};" ::"r"(peer_item + 16 * slot), "r"(item.x),
                             "r"(item.y), "r"(item.z), "r"(item.w) : "memory");
                asm volatile("st.shared::cluster.u32 [%0], %1;" ::"r"(peer_dep + 4 * slot), "r"(pre_ok) : "memory");
                mbar_arrive(bar_ring + 8 * slot);
                mbar_arrive_cluster(peer_bar + 8 * slot);        // release at cluster scope: orders the store above
                if (it >= n_items) break;
            }
        }
    } else if (warp >= 7) {
        // ---------------- gather warps: move the dispatched rows into the aligned layout
        gather_units(p, kflags, lane);
        // In-kernel return: with Xa complete these warps have nothing left to do, so they take over the
        // consumer's job on this SM -- no SM is taken from the GEMM.  They only ever wait on tile flags, which
        // the epilogue warps raise without waiting on anybody.
        if (warp_movers || p.zero_early) {
            MoverGroup g{(int)threadIdx.x - 224, 32 * PROD_GATHER_WARPS, 3,
                         reinterpret_cast<int *>(smem_gen + (mover_ints - smem_base)), TRACE_BY_GEMM_WARPS};
            // (the zero rows also with a dedicated consumer, whose few CTAs are too slow for them)
            if (warp_movers) move_segments(p, g, p.zero_early != 0);
            else zero_fill_rows(p, g);
        }
    } else {
        // ---------------- epilogue: warps 2..5 own tensor-memory lanes 32*(warp % 4) .. +31
        const int q = warp & 3;
        const int row = q * 32 + lane;
        const bool leader = (threadIdx.x == 64);
        int acc = 0;
        uint32_t acc_phase = 0;
        bool ok = true;
        for (int n = 0; ok; ++n) {
            const int it = claimed(n);
            if (!epilogue_all(it >= 0)) break;            // leave together if any thread gave up
            if (it >= n_items) break;
            const int4 item = claimed_item(n);
            const int kind = item.x & 0xff, tile = item.w;
            const bool swap = kind == KIND_G1S || kind == KIND_G2S;
            const bool low = (kind & KIND_LOW) != 0;
            const bool first_gemm = (kind & 3) == KIND_G1 || kind == KIND_G1S;
            const bool stack = (kind & KIND_STACK) != 0;
            // stacked bands: lanes 0..63 hold rows 0..63 of band item.y + 2 * rank, lanes 64..127 those of the next
            // band, if the item has that many (item.z = its bands)
            const int sband = item.y + 2 * (int)rank + (q >> 1);
            const bool present = stack ? 2 * (int)rank + (q >> 1) < item.z
                                       : (swap || (rank == 0) || item.z >= 0);     // the pair's second band may be absent
            const int band = stack ? sband : (rank == 0 ? item.y : item.z);
            ok = mbar_wait(bar_tfull + 8 * acc, acc_phase, p, SITE_EPI_TFULL, it);
            ok = epilogue_all(ok);
            if (!ok) break;
            tc_fence_after();
            if (kTrace && leader && rank == 0) p.trace_items2[it].a = globaltimer_ns();
            const uint32_t taddr = tmem_base + (uint32_t)acc * TB_N + ((uint32_t)(q * 32) << 16);
            const size_t grow = (size_t)(present ? band : 0) * TB_M + (stack ? (q & 1) * 32 + lane : row);
            if (swap) {
                // Swapped operands: lane = one of this CTA's 128 weight rows, i.e. one hidden / output column;
                // accumulator column n = row n of the band group (first halves of all bands from CTA 0's token
                // rows, then the second halves from CTA 1's).  A table maps n to the row of H / Y (-1: padding).
                const int nb = item.z & 0xff, ntok = item.z >> 8, nh = ntok / 2;
                volatile int *rowmap =
                    reinterpret_cast<volatile int *>(smem_gen + (swap_rowmap - smem_base)) + acc * SWAP_MAX_N;
                if (row < ntok) {
                    const int half = row >= nh ? 1 : 0, np = row - half * nh;
                    int off = 0, val = -1;
                    for (int i = 0; i < nb; ++i) {
                        const int b = p.sched_band[item.y + i];
                        const int v = p.band_valid[b], h = ceil16_rows(v) / 2;
                        if (np >= off && np < off + h) {
                            const int rib = half * h + (np - off);
                            val = rib < v ? b * TB_M + rib : -1;
                        }
                        off += h;
                    }
                    rowmap[row] = val;
                }
                bar_sync_epilogue();
                const size_t width = first_gemm ? (size_t)p.F : (size_t)p.dout;
                uint16_t *dst = (first_gemm ? p.H : p.Y) + (size_t)tile * TB_N + rank * (TB_N / 2) + row;
#pragma unroll 1
                for (int c = 0; c < ntok; c += 32) {
                    uint32_t g[32], u[32];
                    tmem_ld32(taddr + c, g);
                    if (first_gemm) tmem_ld32(taddr + ntok + c, u);
                    tmem_ld_wait();
#pragma unroll
                    for (int j = 0; j < 32; ++j) {
                        const int r = c + j < ntok ? rowmap[c + j] : -1;          // the same for every lane
                        if (r >= 0) {
                            const float val = first_gemm ? silu_mul(__uint_as_float(g[j]), __uint_as_float(u[j]))
                                                         : __uint_as_float(g[j]);
                            dst[(size_t)r * width] = (uint16_t)(pack_bf16x2(val, 0.f) & 0xffffu);
                        }
                    }
                }
            } else if (!present) {
                // nothing to store: the accumulator of an absent band is discarded
            } else if (low) {
                // 64 rows per CTA: lanes 0..63 hold the rows' accumulator columns 0..127, lanes 64..127 the same rows'
                // columns 128..255 (in tensor-memory columns 0..127 both).  First GEMM: a lane's 128 columns are 64
                // gate values followed by the 64 matching up values (see the load warp).
                const int lrow = (q & 1) * 32 + lane, half = q >> 1;
                const size_t lgrow = (size_t)band * TB_M + lrow;
                if (first_gemm) {
                    uint16_t *dst = p.H + lgrow * p.F + (size_t)tile * H_TILE + half * (H_TILE / 2);
#pragma unroll 1
                    for (int c = 0; c < H_TILE / 2; c += 32) {
                        uint32_t g[32], u[32];
                        tmem_ld32(taddr + c, g);
                        tmem_ld32(taddr + H_TILE / 2 + c, u);
                        tmem_ld_wait();
                        uint32_t o[16];
#pragma unroll
                        for (int j = 0; j < 16; ++j)
                            o[j] = pack_bf16x2(silu_mul(__uint_as_float(g[2 * j]), __uint_as_float(u[2 * j])),
                                               silu_mul(__uint_as_float(g[2 * j + 1]), __uint_as_float(u[2 * j + 1])));
                        uint4 *d4 = reinterpret_cast<uint4 *>(dst + c);
#pragma unroll
                        for (int j = 0; j < 4; ++j) d4[j] = make_uint4(o[4 * j], o[4 * j + 1], o[4 * j + 2], o[4 * j + 3]);
                    }
                } else {
                    uint16_t *dst = p.Y + lgrow * p.dout + (size_t)tile * TB_N + half * (TB_N / 2);
#pragma unroll 1
                    for (int c = 0; c < TB_N / 2; c += 32) {
                        uint32_t v[32];
                        tmem_ld32(taddr + c, v);
                        tmem_ld_wait();
                        uint32_t o[16];
#pragma unroll
                        for (int j = 0; j < 16; ++j)
                            o[j] = pack_bf16x2(__uint_as_float(v[2 * j]), __uint_as_float(v[2 * j + 1]));
                        uint4 *d4 = reinterpret_cast<uint4 *>(dst + c);
#pragma unroll
                        for (int j = 0; j < 4; ++j) d4[j] = make_uint4(o[4 * j], o[4 * j + 1], o[4 * j + 2], o[4 * j + 3]);
                    }
                }
            } else if ((kind & 3) == KIND_G1) {
                uint16_t *dst = p.H + grow * p.F + (size_t)tile * H_TILE;
#pragma unroll 1
                for (int c = 0; c < H_TILE; c += 32) {
                    uint32_t g[32], u[32];
                    tmem_ld32(taddr + c, g);
                    tmem_ld32(taddr + H_TILE + c, u);
                    tmem_ld_wait();
                    uint32_t o[16];
#pragma unroll
                    for (int j = 0; j < 16; ++j)
                        o[j] = pack_bf16x2(silu_mul(__uint_as_float(g[2 * j]), __uint_as_float(u[2 * j])),
                                           silu_mul(__uint_as_float(g[2 * j + 1]), __uint_as_float(u[2 * j + 1])));
                    uint4 *d4 = reinterpret_cast<uint4 *>(dst + c);
#pragma unroll
                    for (int j = 0; j < 4; ++j) d4[j] = make_uint4(o[4 * j], o[4 * j + 1], o[4 * j + 2], o[4 * j + 3]);
                }
            } else {
                uint16_t *dst = p.Y + grow * p.dout + (size_t)tile * TB_N;
#pragma unroll 1
                for (int c = 0; c < TB_N; c += 32) {
                    uint32_t v[32];
                    tmem_ld32(taddr + c, v);
                    tmem_ld_wait();
                    uint32_t o[16];
#pragma unroll
                    for (int j = 0; j < 16; ++j)
                        o[j] = pack_bf16x2(__uint_as_float(v[2 * j]), __uint_as_float(v[2 * j + 1]));
                    uint4 *d4 = reinterpret_cast<uint4 *>(dst + c);
#pragma unroll
                    for (int j = 0; j < 4; ++j) d4[j] = make_uint4(o[4 * j], o[4 * j + 1], o[4 * j + 2], o[4 * j + 3]);
                }
            }
            // accumulator buffer can be overwritten by the tile after next: tell the leader's MMA thread
            tc_fence_before();
            __syncwarp();
            if (lane == 0) {
                if (rank == 0) mbar_arrive(bar_tempty + 8 * acc);
                else mbar_arrive_cluster(lead_tempty + 8 * acc);
            }
            // publish (Section 3.3.1): stores, fence, then one release per tile
            __threadfence();
            if (first_gemm) asm volatile("fence.proxy.async;" ::: "memory");   // H is re-read through TMA
            bar_sync_epilogue();
            if (kTrace && leader && (present || stack)) {
                // taken before the release below, so that no observer of the flag can carry an earlier time
                const unsigned long long now = globaltimer_ns();
                if (rank == 0) p.trace_items[it].c = now; else p.trace_items[it].d = now;
            }
            if (leader && swap) {
                // Both CTAs of the pair hold half of the columns of every band's tile.  Hidden tiles: each CTA counts
                // once per band (two per 256 columns, as two 128-column tiles would).  Output tiles: the CTA that
                // arrives second publishes the flag.
                const int nb = item.z & 0xff;
                for (int i = 0; i < nb; ++i) {
                    const int b = p.sched_band[item.y + i];
                    if (first_gemm) {
                        red_release_add_u32(&p.hcount[b], 1u);
                    } else if (raise_flags && atom_add_acq_rel_u32(&p.fcount[(size_t)b * p.n2 + tile], 1u) == 1u) {
                        st_release_u32(&p.flags[(size_t)b * p.n2 + tile], epoch);
                        const unsigned long long now = globaltimer_ns();
                        stamp_max(&p.stamps[STAMP_FIRST_FLAG_INV], ~now);
                        stamp_max(&p.stamps[STAMP_LAST_FLAG], now);
                    }
                }
            } else if (leader && stack) {
                // this CTA's one or two bands of the stack
                for (int b = item.y + 2 * (int)rank; b < item.y + min(2 * (int)rank + 2, item.z); ++b) {
                    if (first_gemm) {
                        red_release_add_u32(&p.hcount[b], 1u);
                    } else if (raise_flags) {
                        st_release_u32(&p.flags[(size_t)b * p.n2 + tile], epoch);
                        const unsigned long long now = globaltimer_ns();
                        stamp_max(&p.stamps[STAMP_FIRST_FLAG_INV], ~now);
                        stamp_max(&p.stamps[STAMP_LAST_FLAG], now);
                    }
                }
            } else if (leader && present) {
                if (first_gemm) red_release_add_u32(&p.hcount[band], 1u);
                else if (raise_flags) {
                    st_release_u32(&p.flags[(size_t)band * p.n2 + tile], epoch);
                    const unsigned long long now = globaltimer_ns();
                    stamp_max(&p.stamps[STAMP_FIRST_FLAG_INV], ~now);
                    stamp_max(&p.stamps[STAMP_LAST_FLAG], now);
                }
            }
            acc ^= 1;
            if (acc == 0) acc_phase ^= 1u;
        }
    }

    tc_fence_before();
    __syncthreads();
    cluster_sync_all();       // the peer no longer reads this CTA's shared memory or signals its barriers
    if (warp == 1) {
        __syncwarp();
        tc_fence_after();
        tmem_dealloc(tmem_base, PROD_TMEM_COLS);
    }
    // Out of tiles: help the consumer drain what is left, so that the last segments do not wait for the few
    // consumer SMs (the tail Section 3.3.3 warns about when the consumer budget is small).
    if (raise_flags) {
        MoverGroup g{(int)threadIdx.x, (int)blockDim.x, 0, reinterpret_cast<int *>(smem_gen), TRACE_BY_GEMM_TAIL};
        move_segments(p, g);
    }
}

}  // namespace moe_ovl

// Return path and weighted reduction.
//   consumer_kernel  persistent, one CTA per dedicated SM: claims the next segment in schedule
//                    order, polls its ready flags and moves its valid rows into the owner
//                    rank's receive buffer with one contiguous copy (Section 3.3.2-3.3.3);
//                    GEMM CTAs that run out of tiles join in, which removes the tail
//   move_segments    that loop; also run by spare warps of the GEMM CTAs (in-kernel return)
//   scatter_kernel   the non-overlap comparison: all bands, whole GPU, after the GEMM
//   combine_kernel   out[r,t] = sum_j gate_j * ret[r][slot_j]  (Section 2.1 step 5)
// All three are HBM/L2-bandwidth work: 16-byte coalesced loads and stores.
#pragma once

#include "common.cuh"

namespace moe_ovl {

constexpr int MOVER_THREADS = 1024;
// Dynamic shared memory the consumer asks for but never touches: large enough that neither a
// second consumer CTA nor a GEMM CTA fits on the same SM, which gives the consumer SMs of its own.
constexpr int CONSUMER_SMEM_BYTES = 120 * 1024;

__device__ __forceinline__ void copy_rows_16B(const uint16_t *src, uint16_t *dst, size_t nvec, int tid, int nthr)
{
    const uint4 *s = reinterpret_cast<const uint4 *>(src);
    uint4 *d = reinterpret_cast<uint4 *>(dst);
    constexpr int U = 8;                           // 16-byte loads in flight per thread
    size_t v = tid;
    for (; v + (U - 1) * (size_t)nthr < nvec; v += U * (size_t)nthr) {
        uint4 r[U];
#pragma unroll
        for (int k = 0; k < U; ++k) r[k] = __ldcg(s + v + k * (size_t)nthr);
#pragma unroll
        for (int k = 0; k < U; ++k) __stcs(d + v + k * (size_t)nthr, r[k]);
    }
    for (; v < nvec; v += nthr) __stcs(d + v, __ldcg(s + v));
}

// A group of threads that moves segments: a whole CTA (barrier 0) or some warps of a GEMM CTA (their own
// named barrier).  tid counts inside the group; the group's first warp claims and polls.
struct MoverGroup {
    int tid, nthr, bar;
    int *s_unit;          // two ints of shared memory owned by the group
    int who;              // TRACE_BY_* of the trace record
    __device__ __forceinline__ void sync() const
    {
        asm volatile("bar.sync %0, %1;" ::"r"(bar), "r"(nthr) : "memory");
    }
};

// A token that selected no local expert gets a row of zeros in `out` (the empty sum of Section 2.1, step 5): half of
// the tokens at top-2 of 8 experts with 2 local ones.  With an overlapped return the spare warps of the GEMM CTAs
// write those rows once the layout is gathered, so that this part of the reduction's memory traffic is hidden behind
// the GEMM as well; the combine kernel then only writes the tokens that have rows.  (Which tokens those are is known
// before the GEMM starts: the plan kernels have filled the per-token slot lists.)  All threads of the group call this.
constexpr int ZERO_CHUNK_TOKENS = 64;
// Writes at most max_chunks chunks; false when there are none left.
__device__ __forceinline__ bool zero_fill_rows(const Params &p, const MoverGroup &g, int max_chunks = 0x7fffffff)
{
    const int ntok = p.R * p.T, nv = p.dout / 8;
    volatile int *s_unit = g.s_unit;
    for (int done = 0; done < max_chunks; ++done) {
        g.sync();
        if (g.tid == 0) s_unit[0] = atomicAdd(p.next_zero, 1);
        g.sync();
        const int t0 = s_unit[0] * ZERO_CHUNK_TOKENS;
        if (t0 >= ntok) return false;
        const int t1 = min(ntok, t0 + ZERO_CHUNK_TOKENS);
        for (int tok = t0 + (g.tid >> 5); tok < t1; tok += g.nthr >> 5) {       // a warp per token
            if (p.tok_slot[(size_t)tok * p.kmax] != 0) continue;              // has a row: the combine kernel's
            uint4 *o = reinterpret_cast<uint4 *>(p.out + (size_t)tok * p.dout);
            for (int v = g.tid & 31; v < nv; v += 32) __stcs(o + v, make_uint4(0, 0, 0, 0));
        }
    }
    return true;
}

// Segment mover shared by the consumer CTAs, by GEMM CTAs that have run out of tiles and by the spare warps of
// GEMM CTAs (in-kernel return): claim the next unit in schedule order, wait (bounded, acquire) until every tile
// of every band of its segment is flagged, then move the unit's valid rows into the owner rank's receive buffer
// with one contiguous copy.  A unit is a whole segment (the transfer unit of Section 3.3.2) or one of
// p.seg_chunks equal row slices of it: the dedicated consumer moves whole segments, except the last p.tail_segs of
// the schedule, whose tiles finish together at the very end of the GEMM -- sliced, they spread over every CTA
// that is free by then instead of keeping p.tail_segs CTAs busy for a whole segment each; the spare warps of the
// GEMM CTAs move slices throughout.  All threads of the group must call this together.
// with_zero_rows: the group also writes the all-zero rows of `out`, a few chunks before every unit it moves, so that
// those writes are spread over the whole GEMM (as one burst at its start they held the GEMM's own loads up).
__device__ __forceinline__ void move_segments(const Params &p, const MoverGroup &g, bool with_zero_rows = false)
{
    const int nseg = p.meta[META_SEGS];
    const int chunks = p.seg_chunks;
    const int whole = p.tail_segs < 0 ? 0 : max(0, nseg - p.tail_segs);       // leading segments moved whole
    const int nunits = whole + (nseg - whole) * chunks;
    const int lane = g.tid & 31;
    const unsigned epoch = *p.epoch;
    volatile int *s_unit = g.s_unit;
    const int zero_chunks = (p.R * p.T + ZERO_CHUNK_TOKENS - 1) / ZERO_CHUNK_TOKENS;
    const int zero_per_unit = zero_chunks / max(nunits, 1) + 1;
    bool zero_left = with_zero_rows;
    for (;;) {
        if (zero_left) zero_left = zero_fill_rows(p, g, zero_per_unit);
        g.sync();
        if (g.tid < 32) {
            int u = 0;
            if (lane == 0) u = atomicAdd(p.next_seg, 1);
            u = __shfl_sync(0xffffffffu, u, 0);
            bool ok = true;
            if (u < nunits) {
                const int4 seg = p.segs[u < whole ? u : whole + (u - whole) / chunks];   // {first band, bands, dest, rows}
                const int nflags = seg.y * p.n2;
                const unsigned *f = p.flags + (size_t)seg.x * p.n2;
                for (int i = lane; i < nflags && ok; i += 32)
                    ok = wait_global(f + i, epoch, false, p, SITE_CONS_FLAG, (long long)seg.x * p.n2 + i, 2048);
                ok = __all_sync(0xffffffffu, ok);
            }
            if (lane == 0) { s_unit[0] = u; s_unit[1] = ok ? 1 : 0; }
        }
        g.sync();
        const int u = s_unit[0];
        if (u >= nunits || !s_unit[1]) {
            if (zero_left && s_unit[1]) zero_fill_rows(p, g);      // whatever is left of the zero rows
            return;
        }
        const int s = u < whole ? u : whole + (u - whole) / chunks, c = u < whole ? 0 : (u - whole) % chunks;
        const int my_chunks = u < whole ? 1 : chunks;
        const int4 seg = p.segs[s];
        const int per = (seg.w + my_chunks - 1) / my_chunks;   // rows per unit
        const int r0 = c * per, rows = min(per, seg.w - r0);
        const long long slot0 = (long long)p.seg_slot0[s] + r0;
        const unsigned long long t_copy = globaltimer_ns();
        // rows that would not fit into the rank's receive region (malformed routing, already reported) stay put
        if (rows > 0 && slot0 + rows <= p.ret_rows_per_rank) {
            const uint16_t *src = p.Y + ((size_t)seg.x * TB_M + r0) * p.dout;
            uint16_t *dst = p.ret + ((size_t)seg.z * p.ret_rows_per_rank + slot0) * p.dout;
            copy_rows_16B(src, dst, (size_t)rows * p.dout / 8, g.tid, g.nthr);
        }
        g.sync();
        if (g.tid == 0) {
            const unsigned long long now = globaltimer_ns();
            stamp_max(&p.stamps[STAMP_LAST_SEG], now);
            atomicAdd(&p.stamps[STAMP_COPY_NS], now - t_copy);                       // time one group spent copying
            atomicAdd(&p.stamps[STAMP_COPY_BYTES], (unsigned long long)max(rows, 0) * p.dout * 2);
            if (g.who != TRACE_BY_CONSUMER) atomicAdd(p.assist_segs, 1);
            if (p.trace_units) {
                TraceRec rec;
                rec.a = ((unsigned long long)(unsigned)g.who << 32) | (unsigned)blockIdx.x;
                rec.b = t_copy;                  // every flag of the segment seen
                rec.c = now;                     // last row of the unit landed
                rec.d = ((unsigned long long)(unsigned)(s * chunks + c) << 32) | ((unsigned long long)my_chunks << 24) |
                        (unsigned long long)max(rows, 0);
                p.trace_units[u] = rec;
            }
        }
    }
}

// Launched as clusters of two so that the consumer takes whole SM pairs and leaves whole pairs to the GEMM,
// whose CTAs work in pairs.
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(MOVER_THREADS, 1) consumer_kernel(const Params p)
{
    extern __shared__ uint8_t unused_smem[];
    __shared__ int s_unit[2];
    if (threadIdx.x == 0) p.smid_cons[blockIdx.x] = (int)smid();
    MoverGroup g{(int)threadIdx.x, (int)blockDim.x, 0, s_unit, TRACE_BY_CONSUMER};
    move_segments(p, g);
}

// One CTA per (band, chunk of rows): grid-stride over bands x chunks.
constexpr int SCATTER_CHUNKS = 8;     // 16 rows each
__global__ void __launch_bounds__(256) scatter_kernel(const Params p)
{
    const int nbands = p.meta[META_BANDS];
    const int rows_per_chunk = TB_M / SCATTER_CHUNKS;
    for (int u = blockIdx.x; u < nbands * SCATTER_CHUNKS; u += gridDim.x) {
        const int band = u / SCATTER_CHUNKS, chunk = u % SCATTER_CHUNKS;
        const int valid = p.band_valid[band];
        const int r0 = chunk * rows_per_chunk;
        if (r0 >= valid) continue;
        const int rows = min(rows_per_chunk, valid - r0);
        // malformed routing can ask for more rows than the region holds: reported by the plan, skipped here
        if ((long long)p.band_slot0[band] + r0 + rows > p.ret_rows_per_rank) continue;
        const uint16_t *src = p.Y + ((size_t)band * TB_M + r0) * p.dout;
        uint16_t *dst = p.ret + ((size_t)p.band_dest[band] * p.ret_rows_per_rank + p.band_slot0[band] + r0) * p.dout;
        copy_rows_16B(src, dst, (size_t)rows * p.dout / 8, threadIdx.x, blockDim.x);
    }
}

// A group of threads (256 for wide rows, down to 32 for narrow ones, so that every thread has two 16-byte
// vectors of work) handles one token at a time, grid-stride over tokens; thread v handles 8 consecutive
// features.  The next token's list is fetched while the current token's rows are in flight.
__global__ void __launch_bounds__(256) combine_kernel(const Params p)
{
    const int ntok = p.R * p.T;
    const int nv = p.dout / 8;
    constexpr int KFAST = 2;                      // list entries kept in registers
    int slot[KFAST];
    float gate[KFAST];
    auto fetch = [&](int tok) {
#pragma unroll
        for (int j = 0; j < KFAST; ++j) {
            const bool use = tok < ntok && j < p.kmax;
            slot[j] = use ? __ldg(p.tok_slot + (size_t)tok * p.kmax + j) : 0;
            gate[j] = use ? __ldg(p.tok_gate + (size_t)tok * p.kmax + j) : 0.f;
        }
    };
    int tpt = 256;                                  // threads per token: power of two, about nv / 2
    while (tpt > 32 && tpt > nv / 2) tpt >>= 1;
    const int sub = threadIdx.x / tpt, lt = threadIdx.x % tpt, per_block = blockDim.x / tpt;
    const int tok_stride = gridDim.x * per_block;
    fetch(blockIdx.x * per_block + sub);
    for (int tok = blockIdx.x * per_block + sub; tok < ntok; tok += tok_stride) {
        const uint16_t *region = p.ret + (size_t)(tok / p.T) * p.ret_rows_per_rank * p.dout;
        uint4 *o = reinterpret_cast<uint4 *>(p.out + (size_t)tok * p.dout);
        int cs[KFAST];
        float cg[KFAST];
#pragma unroll
        for (int j = 0; j < KFAST; ++j) { cs[j] = slot[j]; cg[j] = gate[j]; }
        fetch(tok + tok_stride);
        if (p.zero_early && cs[0] <= 0) continue;     // no local row: its zeros were written during the GEMM
        // two 16-byte vectors per thread and iteration: all of their row loads are issued before any arithmetic
        for (int v0 = lt; v0 < nv; v0 += 2 * tpt) {
            const int v1 = v0 + tpt;
            const bool has1 = v1 < nv;
            uint4 row[2][KFAST];
#pragma unroll
            for (int j = 0; j < KFAST; ++j) {
                const uint4 *src = reinterpret_cast<const uint4 *>(region + (size_t)(cs[j] > 0 ? cs[j] - 1 : 0) * p.dout);
                row[0][j] = cs[j] > 0 ? __ldcs(src + v0) : make_uint4(0, 0, 0, 0);
                row[1][j] = (cs[j] > 0 && has1) ? __ldcs(src + v1) : make_uint4(0, 0, 0, 0);
            }
#pragma unroll
            for (int u = 0; u < 2; ++u) {
                const int v = u == 0 ? v0 : v1;
                if (u == 1 && !has1) break;
                float acc[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
                auto add = [&](const uint4 &q, float g) {
                    const uint32_t w[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        acc[2 * i] += g * __uint_as_float(w[i] << 16);
                        acc[2 * i + 1] += g * __uint_as_float(w[i] & 0xffff0000u);
                    }
                };
                // ascending local expert; the list is dense, so the first empty entry (0) ends it
                bool open = true;
#pragma unroll
                for (int j = 0; j < KFAST; ++j) {
                    open = open && cs[j] > 0;
                    if (open) add(row[u][j], cg[j]);
                }
                if (open) {
                    for (int j = KFAST; j < p.kmax; ++j) {        // tokens with more than two local rows
                        const int s = p.tok_slot[(size_t)tok * p.kmax + j];
                        if (s <= 0) break;
                        add(__ldcs(reinterpret_cast<const uint4 *>(region + (size_t)(s - 1) * p.dout) + v),
                            p.tok_gate[(size_t)tok * p.kmax + j]);
                    }
                }
                uint32_t w[4];
#pragma unroll
                for (int i = 0; i < 4; ++i)
                    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(w[i]) : "f"(acc[2 * i + 1]), "f"(acc[2 * i]));
                __stcs(o + v, make_uint4(w[0], w[1], w[2], w[3]));
            }
        }
    }
}

}  // namespace moe_ovl

// moe_ovl_return_slots_static: the return-slot computation of the plan for callers
// that can neither allocate device memory nor hand over a workspace.  Its scratch
// (token bitmaps and their popcount prefixes) lives in a fixed-size array that is
// part of the library image, so the call allocates nothing.  See include/moe_ovl.h.
#include <cuda_runtime.h>

#include <mutex>

#include "../../include/moe_ovl.h"

namespace {

constexpr int STATIC_MAX_GROUPS = MOE_OVL_STATIC_MAX_GROUPS;   // El * R
constexpr int STATIC_MAX_WORDS = MOE_OVL_STATIC_MAX_WORDS;     // El * R * ceil(T / 32)
constexpr int STATIC_MAX_EXPERTS = 256;
constexpr int STATIC_THREADS = 1024;
// words [0, MAX_WORDS): bitmaps; [MAX_WORDS, 2*MAX_WORDS): exclusive popcount prefixes
constexpr size_t STATIC_SCRATCH_WORDS = 2 * (size_t)STATIC_MAX_WORDS;

// Held by every GPU that loads the library, until the process exits (512 KiB).
static __device__ __align__(256) unsigned g_static_scratch[STATIC_SCRATCH_WORDS];

// One CTA does the whole job: clear, mark, prefix, slots.  Everything it needs to start from zero is cleared
// here, because the array keeps whatever the previous call left in it.
__global__ void __launch_bounds__(STATIC_THREADS, 1)
return_slots_static_kernel(unsigned *scratch, int R, int T, int El, int M, const int *expert_counts,
                           const int *src_rank, const int *src_token, int *slot_out, int *rows_per_rank_out)
{
    __shared__ int pre[STATIC_MAX_EXPERTS + 1];
    __shared__ int n[STATIC_MAX_GROUPS], gslot[STATIC_MAX_GROUPS];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, nwarps = blockDim.x >> 5;
    const int words = (T + 31) / 32, G = El * R;
    unsigned *bitmap = scratch;
    int *wordpfx = reinterpret_cast<int *>(scratch + STATIC_MAX_WORDS);

    for (int w = tid; w < G * words; w += blockDim.x) bitmap[w] = 0u;
    if (tid == 0) {
        int acc = 0;
        for (int e = 0; e < El; ++e) { pre[e] = acc; acc += expert_counts[e]; }
        pre[El] = acc;
    }
    __syncthreads();

    auto expert_of = [&](int i) {
        int lo = 0, hi = El;
        while (hi - lo > 1) { const int mid = (lo + hi) >> 1; if (pre[mid] <= i) lo = mid; else hi = mid; }
        return lo;
    };
    auto valid = [&](int i, int r, int t) { return i < pre[El] && r >= 0 && r < R && t >= 0 && t < T; };

    for (int i = tid; i < M; i += blockDim.x) {
        const int r = src_rank[i], t = src_token[i];
        if (valid(i, r, t))
            atomicOr(&bitmap[(size_t)(expert_of(i) * R + r) * words + (t >> 5)], 1u << (t & 31));
    }
    __syncthreads();

    for (int g = warp; g < G; g += nwarps) {
        int run = 0;
        for (int w0 = 0; w0 < words; w0 += 32) {
            const int w = w0 + lane;
            const int c = w < words ? __popc(bitmap[(size_t)g * words + w]) : 0;
            int inc = c;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const int v = __shfl_up_sync(0xffffffffu, inc, o);
                if (lane >= o) inc += v;
            }
            if (w < words) wordpfx[(size_t)g * words + w] = run + inc - c;
            run += __shfl_sync(0xffffffffu, inc, 31);
        }
        if (lane == 0) n[g] = run;
    }
    __syncthreads();

    // receive-buffer slots are expert-major and dense inside each owner rank's region
    for (int r = tid; r < R; r += blockDim.x) {
        int acc = 0;
        for (int e = 0; e < El; ++e) { gslot[e * R + r] = acc; acc += n[e * R + r]; }
        if (rows_per_rank_out) rows_per_rank_out[r] = acc;
    }
    __syncthreads();

    for (int i = tid; i < M; i += blockDim.x) {
        const int r = src_rank[i], t = src_token[i];
        int slot = -1;
        if (valid(i, r, t)) {
            const int g = expert_of(i) * R + r;
            const size_t w = (size_t)g * words + (t >> 5);
            slot = gslot[g] + wordpfx[w] + __popc(bitmap[w] & ((1u << (t & 31)) - 1u));
        }
        slot_out[i] = slot;
    }
}

constexpr int MAX_DEVICES = 64;
std::mutex g_setup_mutex;
unsigned *g_scratch_addr[MAX_DEVICES];      // device address of g_static_scratch on each GPU, once resolved

// In host code the array's name is only a handle; the kernel needs the address the array has on the GPU in
// use.  Resolved once per device, with that device current.
int scratch_address(int device, unsigned **out)
{
    std::lock_guard<std::mutex> lock(g_setup_mutex);
    if (!g_scratch_addr[device]) {
        void *p = nullptr;
        if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || !p) return MOE_OVL_ERR_CUDA;
        g_scratch_addr[device] = static_cast<unsigned *>(p);
    }
    *out = g_scratch_addr[device];
    return MOE_OVL_OK;
}

}  // namespace

extern "C" int moe_ovl_return_slots_static(int32_t device, int32_t num_src_ranks, int32_t tokens_per_rank,
                                           int32_t num_local_experts, int32_t num_rows,
                                           const int32_t *expert_counts, const int32_t *src_rank,
                                           const int32_t *src_token, int32_t *slot_out,
                                           int32_t *rows_per_rank_out, void *stream)
{
    if (device < 0 || device >= MAX_DEVICES || num_src_ranks < 1 || tokens_per_rank < 1 || num_local_experts < 1 ||
        num_rows < 0 || !expert_counts)
        return MOE_OVL_ERR_INVALID_ARG;
    if (num_rows > 0 && (!src_rank || !src_token || !slot_out)) return MOE_OVL_ERR_INVALID_ARG;
    const long long groups = (long long)num_local_experts * num_src_ranks;
    const long long words = groups * ((tokens_per_rank + 31) / 32);
    if (num_local_experts > STATIC_MAX_EXPERTS || groups > STATIC_MAX_GROUPS || words > STATIC_MAX_WORDS)
        return MOE_OVL_ERR_UNSUPPORTED;      // beyond the fixed scratch: use moe_ovl_expert_return with a workspace
    if (cudaSetDevice(device) != cudaSuccess) return MOE_OVL_ERR_CUDA;
    unsigned *scratch = nullptr;
    const int rc = scratch_address(device, &scratch);
    if (rc != MOE_OVL_OK) return rc;
    return_slots_static_kernel<<<1, STATIC_THREADS, 0, static_cast<cudaStream_t>(stream)>>>(
        scratch, num_src_ranks, tokens_per_rank, num_local_experts, num_rows, expert_counts, src_rank, src_token,
        slot_out, rows_per_rank_out);
    return cudaGetLastError() == cudaSuccess ? MOE_OVL_OK : MOE_OVL_ERR_CUDA;
}

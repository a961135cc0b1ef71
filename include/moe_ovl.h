/* moe_ovl -- the expert-side half of a Mixture-of-Experts layer on one NVIDIA B200
 * (sm_100a), with the return of expert outputs overlapped with the expert GEMMs
 * through per-tile ready flags.
 *
 * Plain C ABI: every pointer is a raw address, marked below as HOST or DEVICE.
 * The library never allocates device memory: the caller hands it one workspace
 * (moe_ovl_workspace_bytes) and owns every tensor.  All functions return
 * MOE_OVL_OK (0) or a negative MOE_OVL_ERR_* code; nothing throws, aborts or
 * traps, on the host or on the device.
 *
 * Problem statement (Section 2.1, steps 3-5; Section 3.1): this GPU ("rank
 * r_self") holds El local experts.  After the first all-to-all it has received M
 * routed token copies ("rows"), grouped by local expert, each tagged with the
 * rank that owns the token, the token's index on that rank, and its gate weight.
 * It must (a) run every row through its expert's SwiGLU FFN, (b) deliver each
 * output row to the receive buffer of the owning rank in source-token order, and
 * (c) the owner forms the gate-weighted sum per token.  Source ranks are
 * simulated: the receive buffer of rank r is a region of this GPU's HBM.
 *
 * How it is computed (Section 3.2 and 3.3):
 *   plan      remote-owner-aligned row layout and remote-first tile schedule
 *             (Algorithm 1), combine plan (Section 3.2.3), segments (Section 3.3.2)
 *   producer  one persistent tcgen05 kernel over all local experts; raises one
 *             ready flag per finished output tile (Section 3.3.1)
 *   consumer  persistent kernel on consumer_sm_count dedicated SMs; polls the
 *             flags and moves each finished segment with one contiguous copy
 *             (Section 3.3.2, 3.3.3)
 *   combine   gate-weighted reduction at the owner (Section 2.1 step 5)
 * MOE_OVL_MODE_NON_OVERLAP is the comparison baseline of Section 4.1: the same
 * GEMM kernel on every SM runs to completion, then a separate scatter kernel
 * moves all rows, then the same combine.
 */
#ifndef MOE_OVL_H
#define MOE_OVL_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct moe_ovl_ctx moe_ovl_ctx; /* opaque, owned by the library */

enum {
    MOE_OVL_OK = 0,
    MOE_OVL_ERR_INVALID_ARG = -1, /* null pointer, negative size, value out of range */
    MOE_OVL_ERR_UNSUPPORTED = -2, /* shape the kernels do not cover (see moe_ovl_config) */
    MOE_OVL_ERR_CUDA = -3,        /* a CUDA runtime/driver call failed (moe_ovl_last_cuda_error) */
    MOE_OVL_ERR_WORKSPACE = -4,   /* workspace missing, misaligned or too small */
    MOE_OVL_ERR_TIMEOUT = -5,     /* a bounded device-side wait gave up (asynchronous, see query_status) */
    MOE_OVL_ERR_BAD_ROUTING = -6  /* routing metadata inconsistent (asynchronous, see query_status) */
};

enum {
    MOE_OVL_MODE_OVERLAP = 0,     /* producer + consumer kernel on consumer_sm_count dedicated SMs (Section 3.3.3) */
    MOE_OVL_MODE_NON_OVERLAP = 1, /* comparison baseline of Section 4.1: GEMM to completion, then scatter */
    MOE_OVL_MODE_IN_KERNEL = 2,   /* same flag protocol and segments, but the finished segments are moved by spare
                                     warps inside the GEMM CTAs: no SM is taken from the GEMM, one kernel, nothing
                                     to co-schedule.  Not in the paper: on one GPU the return is an HBM copy that
                                     needs a few percent of one SM's load/store slots, not an SM of its own. */
    MOE_OVL_MODE_AUTO = 3         /* the library picks one of the three (and the consumer budget) from the shape
                                     and the number of rows; moe_ovl_report.mode_used tells which */
};

/* tile geometry, fixed by the kernels */
#define MOE_OVL_TB_M 128  /* rows per band (output tile height, tb_M of Algorithm 1) */
#define MOE_OVL_TB_N 256  /* output tile width of the second GEMM */
#define MOE_OVL_H_TILE 128 /* hidden columns produced by one tile of the first GEMM */

typedef struct {
    uint32_t struct_size;       /* sizeof(moe_ovl_config), for ABI checks */
    int32_t device;             /* CUDA device ordinal */
    int32_t num_src_ranks;      /* R >= 1 */
    int32_t self_rank;          /* r_self in 0..R-1: its rows are "local" and are scheduled last */
    int32_t tokens_per_rank;    /* T: the output has R*T rows */
    int32_t num_local_experts;  /* El >= 1, El * R <= 1024 */
    int32_t top_k;              /* k: a token owns at most min(k, El) rows here */
    int32_t d_model;            /* d, multiple of 256 */
    int32_t d_ffn;              /* F, multiple of 128 */
    int32_t max_rows;           /* capacity for M */
    int32_t mid_seg_bands;      /* bands per middle segment (x of Figure 3b); 0 = chosen by the library: 1, because
                                   with HBM as the link a transfer has no fixed cost to amortise (larger middle
                                   segments were never faster in the measured grids) */
    int32_t group_bands;        /* bands whose tiles are interleaved so that they share weight tiles in L2; 0 = default (16), at most 64 */
    int32_t wait_timeout_us;    /* bound on every device-side wait; 0 = default (2 s) */
    int32_t producer_sm_limit;  /* NON_OVERLAP only: cap on GEMM CTAs (diagnostic baseline); 0 = all SMs */
    int32_t single_gemm_out;    /* 0: SwiGLU FFN experts.  N > 0: the operator the paper evaluates (Table 2) -- each
                                   expert is ONE projection y = x . W^T with W[N, d_model]; N multiple of 256,
                                   d_model multiple of 64; w1 holds W as [El, N, d_model], w2 and d_ffn are
                                   ignored, and ret / out rows are N wide */
    uint32_t flags;             /* MOE_OVL_FLAG_* */
} moe_ovl_config;

#define MOE_OVL_FLAG_HOST_STAGING 1u /* reserve workspace for moe_ovl_expert_return_host */
#define MOE_OVL_FLAG_TEST_NO_FLAGS 2u /* test hook: in OVERLAP mode the GEMM raises no ready flags, so the consumer's
                                         bounded wait runs out and the call ends with MOE_OVL_ERR_TIMEOUT */
#define MOE_OVL_FLAG_TRACE 4u         /* reserve workspace for, and record, the per-item / per-unit device trace
                                         (moe_ovl_get_trace); off by default, costs nothing when off */
#define MOE_OVL_FLAG_NO_SMALL_GROUP_TILES 16u /* never issue the 64-row-high pair items and the swapped-operand items that
                                         small (expert, rank) groups otherwise get (see moe_ovl_plan_view.item); for
                                         comparisons */
#define MOE_OVL_FLAG_NO_STACKED_BANDS 64u /* never stack three or four small bands into one full-height item (kinds 8
                                         and 9 of moe_ovl_plan_view.item); for comparisons */
#define MOE_OVL_FLAG_NO_LOCAL_RIDERS 128u /* never let an expert's local band join the last item of its remote bands (see
                                         moe_ovl_plan_view.item); for comparisons */
#define MOE_OVL_FLAG_TEST_ZERO_ROWS_EARLY 256u /* test hook: in the overlapped modes the all-zero rows of `out` (tokens
                                         with no local expert) are written behind the GEMM also where the host's cost
                                         rule would leave them to the combine kernel (small layers) */
#define MOE_OVL_FLAG_TEST_ALL_SMALL_GROUP_TILES 32u /* test hook: every eligible run of small groups gets swapped-operand
                                         items, also where the plan's cost rule would keep band pairs */
#define MOE_OVL_FLAG_TEST_SKIP_GATHER 8u /* test hook: the first band of the schedule is never gathered, so the GEMM's
                                         own bounded wait for it runs out (exercises the give-up path inside the GEMM
                                         kernel: copies drained, tensor memory freed, MOE_OVL_ERR_TIMEOUT) */

typedef struct {
    uint32_t struct_size;
    int32_t num_rows;             /* M (host value), 0 <= M <= max_rows */
    const void *x;                /* DEVICE [M, d] bf16 row-major: rows grouped by local expert 0..El-1 */
    const int32_t *expert_counts; /* DEVICE [El]: rows per local expert, sum == M */
    const int32_t *src_rank;      /* DEVICE [M] in 0..R-1: owner rank of the row's token */
    const int32_t *src_token;     /* DEVICE [M] in 0..T-1: token index on the owner rank */
    const float *gate;            /* DEVICE [M] fp32 gate weight of (token, expert) */
    const void *w1;               /* DEVICE [El, 2F, d] bf16: rows 0..F-1 gate projection, F..2F-1 up projection
                                     (single-projection mode: [El, N, d]) */
    const void *w2;               /* DEVICE [El, d, F] bf16 (single-projection mode: ignored, may be NULL) */
    int32_t consumer_sm_count;    /* SMs dedicated to the consumer (OVERLAP); 1..SMs/2, rounded up to a whole SM pair;
                                     0 = chosen by the library from the shape (see moe_ovl_report.consumer_ctas) */
    int32_t mode;                 /* MOE_OVL_MODE_* */
    void *ret;                    /* DEVICE [R][ret_rows_per_rank, d] bf16: simulated peer receive buffers.
                                     Row s of region r is written iff s < rows_per_rank[r]; the rest is untouched. */
    int64_t ret_rows_per_rank;    /* >= T * min(k, El) */
    void *out;                    /* DEVICE [R*T, d] bf16, fully overwritten (tokens with no local row get +0);
                                     ret and out rows are N wide in single-projection mode */
    int32_t *slot_out;            /* DEVICE [M] or NULL: receive-buffer slot of every input row */
    int32_t *rows_per_rank_out;   /* DEVICE [R] or NULL */
    int32_t *segs_per_rank_out;   /* DEVICE [R] or NULL: segments sent to each rank */
    void *stream;                 /* cudaStream_t of the caller (NULL = legacy default stream) */
} moe_ovl_args;

/* Host-buffer variant: every tensor that changes per call lives in HOST memory
 * (pinned for asynchronous copies); weights stay resident on the device. */
typedef struct {
    uint32_t struct_size;
    int32_t num_rows;
    const void *x;                /* HOST [M, d] bf16 */
    const int32_t *expert_counts; /* HOST [El] */
    const int32_t *src_rank;      /* HOST [M] */
    const int32_t *src_token;     /* HOST [M] */
    const float *gate;            /* HOST [M] */
    const void *w1;               /* DEVICE, as in moe_ovl_args */
    const void *w2;               /* DEVICE */
    int32_t consumer_sm_count;
    int32_t mode;
    void *out;                    /* HOST [R*T, d] bf16 */
    void *stream;
} moe_ovl_host_args;

#define MOE_OVL_TIMING_HISTORY 64

/* Sizes of the plan of the last call, and where the time went (milliseconds). */
typedef struct {
    int32_t padded_rows;      /* P, multiple of 128 */
    int32_t num_bands;        /* P / 128 */
    int32_t num_items;        /* schedule length: tiles of both GEMMs */
    int32_t num_segments;
    int32_t producer_ctas;
    int32_t consumer_ctas;    /* 0 in NON_OVERLAP */
    int32_t kernel_launches;  /* kernels of this library launched by the call */
    int32_t segments_by_gemm_ctas; /* units of the return (whole segments or slices, see return_units) moved by GEMM
                                      CTAs: in OVERLAP by those that had run out of tiles, in IN_KERNEL all of them */
    int32_t return_units;     /* units the return was moved in: a whole segment, or one of eight row slices of it (the
                                 dedicated consumer slices the schedule's last 16 segments, the in-kernel movers all) */
    int32_t mode_used;        /* MOE_OVL_MODE_* the call ran in (differs from args->mode only for MODE_AUTO) */
    int32_t timing_valid;     /* 0 when the call was captured into a CUDA graph: the ms_* fields are then 0 (events
                                 recorded during capture carry no time); the us_* device stamps stay valid */
    float ms_total;           /* whole call on the caller's stream */
    float ms_prep;            /* plan + gather into the aligned layout */
    float ms_expert_return;   /* start of the GEMM to the last row landed in ret */
    float ms_producer;        /* the GEMM kernel alone */
    float ms_mover;           /* consumer (OVERLAP: concurrent with the GEMM) or scatter kernel; 0 for the in-kernel return */
    float ms_combine;
    /* device timestamps (%globaltimer), microseconds after the first GEMM CTA started; OVERLAP mode */
    float us_first_flag;      /* first output tile flagged: the consumer's window opens */
    float us_gemm_done;       /* last output tile flagged */
    float us_return_done;     /* last segment landed in ret */
    float copy_gbs_per_cta;   /* returned bytes / time the moving CTAs spent inside segment copies: the rate one CTA
                                 sustains while the GEMM runs (GB/s, payload counted once) */
    float overlap_ratio;      /* share of the return window that lies before us_gemm_done:
                                 1 - max(0, us_return_done - us_gemm_done) / (us_return_done - us_first_flag);
                                 the share of the second all-to-all hidden behind expert compute (Section 4.2.2) */
} moe_ovl_report;

/* Integer plan arrays of the last call, copied to HOST buffers (any pointer may be
 * NULL).  Capacities: bands -> max_bands, items -> max_items, segments -> max_bands
 * (moe_ovl_limits). */
typedef struct {
    int32_t *group_rows;      /* [El*R]  n[e][r] */
    int32_t *pos;             /* [M]     aligned position of every input row */
    int32_t *band_expert;     /* [bands] in band-id order (band id = first position / 128) */
    int32_t *band_dest;
    int32_t *band_valid;
    int32_t *band_slot0;
    int32_t *sched_band;      /* [bands] band ids in schedule order */
    int32_t *item;            /* [items][4] in issue order.  Kinds 0 (first GEMM) and 1 (second GEMM): {kind | expert << 8,
                                 band, second band of the pair or -1, tile}, a 256-row x 256-column tile of two bands
                                 (128 hidden columns per band for kind 0); kinds 4 and 5 are the same items for a pair
                                 whose bands hold at most 64 valid rows each, computed 64 rows high (about 0.9 of
                                 the tensor-pipe time).  Kinds 8 and 9: {kind | expert << 8, first band, bands,
                                 tile} -- 3 or 4 bands with consecutive ids, at most 64 valid rows each, stacked
                                 into one full-height item (rows 0..63 of two bands per CTA), i.e. two such pairs
                                 for the time of one.  Where the last item of an expert's remote bands (kinds 4, 5,
                                 8, 9) has rows to spare and the expert's local rows are one band of at most 64, that
                                 band is issued in the same item (its id is the last remote band's + 1) and has no
                                 items of its own: no remote tile is issued later for it, and the expert's weights
                                 are read once instead of twice.  Kinds 2 and 3, the same two GEMMs for a
                                 run whose (expert, rank) groups hold at most 64 rows each: {kind | expert << 8,
                                 position of the first band in sched_band, bands | rows << 8, tile} -- the valid rows
                                 of up to 8 consecutive bands (each rounded up to 16, at most 128 together) against a
                                 tile of 256 weight rows with the operands swapped, so that one pass over a weight
                                 tile serves the whole group (tile = 256 hidden columns for kind 2, 256 output columns
                                 for 3).  Issued only where a run's groups are fewer than its band pairs and the
                                 schedule holds several such items per CTA pair. */
    int32_t *seg;             /* [segments][4] = {first band, bands, dest rank, rows} in schedule order */
    int32_t *tok_slot;        /* [R*T*min(k,El)] slots of each token's rows, ascending expert, -1 = none */
    float *tok_gate;          /* [R*T*min(k,El)] matching gates */
} moe_ovl_plan_view;

enum { MOE_OVL_BUF_XA = 0, MOE_OVL_BUF_H = 1, MOE_OVL_BUF_Y = 2 };

/* Bytes of workspace moe_ovl_create needs for this configuration (256-byte aligned base). */
int moe_ovl_workspace_bytes(const moe_ovl_config *cfg, size_t *bytes);

/* Capacities derived from the configuration. */
int moe_ovl_limits(const moe_ovl_config *cfg, int32_t *max_bands, int32_t *max_items);

/* Creates a context on cfg->device.  `workspace` is DEVICE memory owned by the caller
 * and must outlive the context.  Creates two internal streams and their events;
 * allocates no device memory. */
int moe_ovl_create(moe_ovl_ctx **ctx, const moe_ovl_config *cfg, void *workspace, size_t workspace_bytes);

/* Enqueues one pass of the path.  What it computes, by passage of the paper:
 *   Section 2.1, steps 3-5      expert FFN on every routed row, return of each output row to the
 *                               rank that owns the token, gate-weighted sum per token at the owner
 *   Section 3.2.1, Algorithm 1  remote-owner-aligned row layout (remote groups padded to tb_M, local last)
 *   Section 3.2.2, Algorithm 1  remote-first tile schedule (experts by remote band count)
 *   Section 3.2.3               combine plan: destination, receive-buffer offset, valid rows per tile
 *   Section 3.3.1               rank-wide persistent GEMM, ready flag per finished output tile
 *   Section 3.3.2, Figure 3b    segment-granular transfer (first / middle / last segments)
 *   Section 3.3.3               co-scheduling of producer and consumer on disjoint SM sets
 * Asynchronous: ordered after earlier work on args->stream, complete for later work
 * on it.  One call in flight per context.  Synchronous argument errors are returned
 * here; device-side errors are reported by moe_ovl_query_status.  The call can be
 * captured in a CUDA graph on args->stream (its internal streams join the capture) and
 * replayed with new contents in the same buffers: everything that changes from call to call,
 * the number marking this call's ready flags included, lives in device memory.  A captured
 * call records no timing events: moe_ovl_get_report then returns timing_valid = 0 with the
 * ms_* fields zero, and moe_ovl_get_gemm_time skips it. */
int moe_ovl_expert_return(moe_ovl_ctx *ctx, const moe_ovl_args *args);

/* Same pass with per-call tensors in HOST memory (pinned, for asynchronous copies): copies
 * the inputs to staging buffers in the workspace, runs the pass on args->stream, copies
 * `out` back.  Needs MOE_OVL_FLAG_HOST_STAGING.  The copies run on two internal streams and
 * two staging slots, so that consecutive calls pipeline: the inputs of call i+1 travel while
 * call i computes, and the result of call i travels while call i+1 computes.  Consequences:
 * the host input buffers are read from the moment of the call (not ordered after earlier work
 * on args->stream) and must stay unchanged until the call's pass has started; `out` of a call
 * is complete once moe_ovl_host_join has been enqueued and its stream synchronised (or after
 * moe_ovl_query_status), NOT merely when args->stream has drained. */
int moe_ovl_expert_return_host(moe_ovl_ctx *ctx, const moe_ovl_host_args *args);

/* Makes `stream` (cudaStream_t) wait for the result copies of every host-buffer call issued so far. */
int moe_ovl_host_join(moe_ovl_ctx *ctx, void *stream);

/* Waits for the last call and returns its device status: *code is MOE_OVL_OK,
 * MOE_OVL_ERR_TIMEOUT or MOE_OVL_ERR_BAD_ROUTING; *detail identifies the wait or
 * the row.  After an error the outputs are unspecified but were written in bounds. */
int moe_ovl_query_status(moe_ovl_ctx *ctx, int32_t *code, int64_t *detail);

/* Waits for the last call, then fills the report / copies plan arrays / reads back
 * `bytes` bytes at `offset` of an internal bf16 buffer (MOE_OVL_BUF_*) to HOST memory. */
int moe_ovl_get_report(moe_ovl_ctx *ctx, moe_ovl_report *report);
int moe_ovl_get_plan(moe_ovl_ctx *ctx, const moe_ovl_plan_view *view);
/* Mean duration (ms) of the GEMM kernel over the last `last_n` calls (at most MOE_OVL_TIMING_HISTORY): every call
 * brackets the kernel with CUDA events on the stream it is launched on and the context keeps the most recent
 * pairs, so a run of back-to-back calls can be timed without synchronising between them.  Waits for the last call. */
int moe_ovl_get_gemm_time(moe_ovl_ctx *ctx, int32_t last_n, float *avg_ms, int32_t *n_used);
/* SM (%smid) every GEMM CTA and every consumer CTA of the last call ran on; HOST arrays of
 * producer_ctas and consumer_ctas entries (moe_ovl_report).  The two kernels must not share an SM. */
int moe_ovl_get_sm_map(moe_ovl_ctx *ctx, int32_t *producer_smid, int32_t *consumer_smid);
int moe_ovl_read_buffer(moe_ovl_ctx *ctx, int32_t which, size_t offset, size_t bytes, void *host_dst);

/* Device trace of the last call (needs MOE_OVL_FLAG_TRACE).  One record per schedule item of the GEMM
 * kernel and one per moved unit of the return (a unit is a whole segment or one of eight equal row slices of
 * it, see `chunks` below); times are nanoseconds of the
 * GPU's global timer after the first GEMM CTA started.  It is what the overlap ratio of Section 4.2.2, the
 * tail after the last tile and the idle time of the consumer (Section 3.3.3) are read from. */
enum { MOE_OVL_TRACE_ITEM = 0, MOE_OVL_TRACE_UNIT = 1 };
typedef struct {
    int32_t kind;      /* MOE_OVL_TRACE_ITEM / MOE_OVL_TRACE_UNIT */
    int32_t index;     /* item: position in issue order (moe_ovl_plan_view.item); unit: segment * 8 + slice */
    int32_t cta;       /* item: leader CTA of the pair that ran it; unit: CTA that moved it */
    int32_t who;       /* unit: 0 consumer CTA, 1 GEMM CTA that had run out of tiles, 2 spare warps of a GEMM CTA */
    int32_t rows;      /* unit: rows moved */
    int32_t chunks;    /* unit: slices its segment is moved in: 1 (whole) or 8.  The dedicated consumer moves whole
                          segments except the last 16 of the schedule; the spare warps of GEMM CTAs always slices */
    int64_t ns_claim;  /* item: claimed by the pair's scheduler; unit: every ready flag of the segment seen */
    int64_t ns_ready;  /* item: first operand stage landed, the MMAs can start; unit: same as ns_claim */
    int64_t ns_done0;  /* item: tile of the pair's first band published (flag or band counter), taken just
                          before the release store; unit: last row landed in the receive buffer */
    int64_t ns_done1;  /* item: same for the pair's second band, -1 if absent; unit: same as ns_done0 */
    int64_t ns_operand_wait; /* item: time the MMA-issuing thread spent waiting for operand stages after the
                          item's first stage (pipeline stalls, not start-up); unit: 0 */
    int64_t ns_epilogue_start;     /* item: the epilogue warps of the pair's first CTA saw the finished accumulator */
    int64_t ns_first_operand_wait; /* item: time the MMA-issuing thread waited for the item's first operand stage
                                      (the bubble between two items, or the kernel's start-up) */
    int64_t ns_accumulator_wait;   /* item: time it waited for a free accumulator buffer, i.e. for the epilogue of
                                      the item before the previous one: non-zero means the epilogue is the bound */
    int64_t ns_inputs_ready;       /* item: the load thread of the pair's first CTA saw the rows the item reads
                                      complete (gathered into the layout, or every hidden tile of the band written)
                                      and issued its first copies; ns_ready - ns_inputs_ready is the latency of
                                      those copies; unit: 0 */
} moe_ovl_trace_record;
/* Waits for the last call, then writes its records to HOST memory: items in issue order, then units in
 * claim order.  *written = bytes written.  host_buf == NULL: only reports the bytes needed.
 * MOE_OVL_ERR_INVALID_ARG if `bytes` is too small, MOE_OVL_ERR_UNSUPPORTED if the context has no trace. */
int moe_ovl_get_trace(moe_ovl_ctx *ctx, void *host_buf, size_t bytes, size_t *written);

int moe_ovl_destroy(moe_ovl_ctx *ctx);

/* Return slots without any allocation (the paper has no counterpart: this entry point
 * exists for one class of callers of this library, not for the method).
 *
 * Some callers can neither call cudaMalloc nor give the library a workspace: code that
 * runs after the host application has handed every byte of device memory to its own
 * pool (a cudaMalloc then fails, or forces that pool to give memory back), and code in
 * latency-critical loops where cudaMalloc's implicit device-wide synchronisation stalls
 * every stream.  For them this call computes what the plan step of
 * moe_ovl_expert_return computes for the return path -- slot_out[i], the row of the
 * owner rank's receive buffer that input row i is delivered to (expert-major, source-
 * token order), and rows_per_rank_out -- using scratch that is a fixed array inside the
 * library image instead of a workspace.  It calls no cudaMalloc, cudaFree or any other
 * allocating routine.
 *
 *   expert_counts DEVICE [El], src_rank / src_token DEVICE [M]: as in moe_ovl_args
 *   slot_out DEVICE [M] (rows with out-of-range metadata get -1), rows_per_rank_out
 *   DEVICE [R] or NULL; stream: cudaStream_t of the caller.  Asynchronous.
 *
 * Limits: El * R <= MOE_OVL_STATIC_MAX_GROUPS and El * R * ceil(T / 32) <=
 * MOE_OVL_STATIC_MAX_WORDS (the array is 512 KiB, and every GPU that loads the library
 * holds it until the process exits); larger problems return MOE_OVL_ERR_UNSUPPORTED and
 * belong to moe_ovl_expert_return with a workspace.
 * Every call makes `device` the calling thread's current device and leaves it so; `stream`
 * must belong to that device.  The first call on a device also resolves the array's device
 * address (one runtime query) and should therefore be made before any stream capture begins
 * on that device.  There is no status channel: a row whose metadata is out of range, or that
 * lies beyond the sum of expert_counts, gets slot -1; a duplicate (expert, rank, token) row --
 * which moe_ovl_expert_return reports as bad routing -- silently gets its twin's slot.  Every call uses the same array: the kernel clears what it needs
 * at its start, but two calls that overlap on one GPU (different streams) race on it and
 * give wrong slots -- keep calls on a device ordered. */
#define MOE_OVL_STATIC_MAX_GROUPS 1024
#define MOE_OVL_STATIC_MAX_WORDS 65536
int moe_ovl_return_slots_static(int32_t device, int32_t num_src_ranks, int32_t tokens_per_rank,
                                int32_t num_local_experts, int32_t num_rows, const int32_t *expert_counts,
                                const int32_t *src_rank, const int32_t *src_token, int32_t *slot_out,
                                int32_t *rows_per_rank_out, void *stream);

const char *moe_ovl_strerror(int code);
/* cudaError_t of the last failing CUDA call made through this context (0 if none). */
int moe_ovl_last_cuda_error(const moe_ovl_ctx *ctx);

#ifdef __cplusplus
}
#endif
#endif /* MOE_OVL_H */

/*
 * adapt_matmul -- shape-adaptive dense GEMM for NVIDIA B200 (sm_100a).
 *
 *   C[M x N] = A[M x K] * B[K x N]      fp16 or bf16 operands, fp32 accumulation,
 *                                        one round-to-nearest-even cast to the
 *                                        16-bit output, every C element written once
 *
 * This is the problem the paper states in Section 4.1 and in the "Common" template
 * paragraph (Eq. 2): 16-bit inputs, higher-precision on-chip accumulation, a single
 * cast, minimum write volume 2*M*N bytes.  The library follows the paper's workflow
 * (Section 3.2): a shape is classified in the 2D tiling taxonomy (Section 4.2), the
 * legal kernel configurations are scored by an analytical latency model (Section 5.2,
 * Eq. 6-11, 12-14), the winner is encoded in a 64-bit TilingKey and cached, and the
 * online call is an O(1) lookup followed by the launch.
 *
 * Plain C ABI: no C++ or framework types cross this boundary.  Unless stated, a
 * pointer argument is a HOST pointer; A, B, C and cuda_stream are the exceptions.
 * Planning, the queries and the error functions may be called from any number of
 * threads at once.  The compute calls (adapt_matmul, adapt_matmul_batch,
 * adapt_matmul_host) may run concurrently on DIFFERENT streams; calls that name the
 * same stream share that stream's workspace, which a call may have to grow (free and
 * reallocate), so they must not be made from two threads at once: give each thread
 * its own stream or serialise the calls.  The adapt_measure_* and adapt_selftest_*
 * entries are single-threaded tools.  There is no CPU fallback: without a CUDA device
 * the compute entry points fail with ADAPT_ERR_CUDA / ADAPT_ERR_NOT_INIT.
 */
#ifndef ADAPT_MATMUL_H
#define ADAPT_MATMUL_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

/* Opaque plan handle.  Owned by the library's plan cache, valid until
 * adapt_shutdown(); the caller never frees it. */
typedef struct adapt_plan_s* adapt_handle_t;

/* Element type of A, B and C (they share it).  Accumulation is always fp32. */
typedef enum { ADAPT_F16 = 0, ADAPT_BF16 = 1 } adapt_dtype_t;

/* Storage of an operand, dense (leading dimension = inner extent).
 * A is M x K: row-major means K contiguous, column-major means M contiguous.
 * B is K x N: row-major means N contiguous, column-major means K contiguous.
 * C is always row-major M x N. */
typedef enum { ADAPT_ROW_MAJOR = 0, ADAPT_COL_MAJOR = 1 } adapt_layout_t;

typedef enum {
    ADAPT_OK = 0,
    ADAPT_ERR_INVALID_ARG = 1,   /* negative size, NULL pointer, bad enum, aliasing C */
    ADAPT_ERR_UNSUPPORTED = 2,   /* a dimension above 2^31-1, or a forced key that is illegal for the shape */
    ADAPT_ERR_NOMEM = 3,         /* workspace allocation failed */
    ADAPT_ERR_CUDA = 4,          /* a CUDA runtime / driver call failed (message in adapt_last_error_message) */
    ADAPT_ERR_TIMEOUT = 5,       /* a bounded device-side wait gave up (see adapt_poll_device_status) */
    ADAPT_ERR_NOT_INIT = 6       /* compute call before a successful adapt_init */
} adapt_status_t;

/* The four templates of the taxonomy (Section 4.2). */
typedef enum {
    ADAPT_CLASS_COMMON = 0,              /* enough tiles, accumulator fits on chip */
    ADAPT_CLASS_SINGLE_CORE_SPLIT_K = 1, /* enough tiles, tile larger than one SM's accumulator budget */
    ADAPT_CLASS_MULTI_CORE_SPLIT_K = 2,  /* too few tiles, accumulator fits */
    ADAPT_CLASS_HYBRID_SPLIT_K = 3       /* too few tiles and oversized tile */
} adapt_class_t;

/* Kernel families of the variant library. */
typedef enum {
    ADAPT_FAM_UMMA_1CTA = 0,  /* tcgen05 128 x BN tiles, TMEM accumulators, TMA ring; P_k > 1 adds split-K */
    ADAPT_FAM_UMMA_2CTA = 1,  /* cta_group::2, 256 x BN tile on an SM pair */
    ADAPT_FAM_SKINNY = 2,     /* warp-level kernel for M <= 16 or N <= 16, streams the large operand once */
    ADAPT_FAM_SIMT = 3,       /* CUDA-core tile kernel: legal for every shape and alignment */
    ADAPT_FAM_CLUSTER = 4     /* small problems in one launch: 64 x 64 tiles on mma.sync, any alignment, the k range
                                 split over the CTAs of a cluster (P_k = cluster = 1, 2, 4, 8, 16) and reduced through
                                 distributed shared memory; no workspace */
} adapt_family_t;

/* How an operand reaches shared memory (the paper's Padding module, Table 2). */
typedef enum {
    ADAPT_SRC_TMA = 0,        /* TMA straight from the caller's buffer (needs a 16 B pitch and base; an operand with
                                 fewer than 64 contiguous elements also a multiple of 16 of them, so that TMA fetches
                                 whole 32 B sectors) */
    ADAPT_SRC_PAD_COPY = 1,   /* prologue kernel re-pitches the operand into the workspace (pitch a multiple of 32 B,
                                 zeros in the pad columns), then TMA (with srcB = ADAPT_SRC_TMA_CLASSES: A is
                                 regrouped class-major instead) */
    ADAPT_SRC_LSU = 2,        /* ordinary loads (skinny / SIMT / cluster families) */
    ADAPT_SRC_TMA_CLASSES = 3 /* class views, no copy of that operand.
                                 srcA: row-major A read in place through one TMA view per row class; tiles are made
                                 of every 8th row (BN = 64, 128, 256; needs K % 8 != 0) or, with 16 halo columns
                                 (BN = 80, 144, 208; needs N % 16 != 0, any K), of every 16th row (every 8th, 4th or
                                 2nd when an even N and K allow it), and C is then written through per-class TMA stores; on pair tiles BN = 128, 256 and, with halo
                                 columns, 144, 208.  An A narrower than 64 columns whose rows are not whole sectors
                                 is re-pitched first and the views are taken of the copy.
                                 srcB: row-major B with N % 8 != 0 read in place through one view per k class
                                 (k % 8); BN = 64 keeps eight class accumulators per tile, BN = 128 / 256 makes
                                 each class a k split (P_k is then a multiple of 8) */
} adapt_source_t;

/* Everything the selector decided for one shape.  Filled by adapt_plan_info and
 * adapt_plan_candidates into caller-owned host memory. */
typedef struct adapt_plan_info_s {
    uint64_t tiling_key;      /* 64-bit TilingKey of this configuration (bit layout below) */
    int64_t M, N, K;
    int32_t dtype, layoutA, layoutB;
    int32_t taxonomy_class;   /* adapt_class_t */
    int32_t family;           /* adapt_family_t */
    int32_t BM, BN, BK;       /* CTA (or CTA-pair) tile: the paper's m1, n1, k1 */
    int32_t stages;           /* depth of the shared-memory ring (Multi-Buffer / Preloading depth) */
    int32_t P_m, P_n, P_k;    /* task counts along M, N, K (Table 1) */
    int32_t cluster;          /* CTAs per cluster (2 for the 2-CTA family) */
    int32_t srcA, srcB;       /* adapt_source_t */
    int32_t grid;             /* CTAs launched by the main kernel */
    int32_t fused;            /* 1: tcgen05 split-K whose P_k splits are the CTAs of one thread-block cluster and whose
                                 partial tiles are added through distributed shared memory inside the GEMM launch
                                 (no workspace, no reduction launch); 0 otherwise */
    int32_t streamk;          /* 1: tcgen05 stream-K: the k-blocks of the tiles that do not fill a whole wave of SMs are shared
                                 evenly by all CTAs; partial tiles go through the workspace and are added by the tile's owner in
                                 ascending k order inside the same launch; 0 otherwise */
    int32_t reserved;
    int64_t workspace_bytes;  /* pad copies + split-K / stream-K partials */
    double flops;             /* 2*M*N*K */
    double hbm_bytes;         /* modelled HBM traffic including workspace traffic */
    double t_pro_us;          /* Eq. 7 terms of the prediction */
    double t_main_us;
    double t_epi_us;
    double predicted_us;      /* T_pro + max_j T_main + T_epi + launch cost */
} adapt_plan_info_t;

/* TilingKey bit layout (Section 3.2 asks only for "a compact 64-bit key"; the fields are this
 * library's): [63:62] taxonomy class, [61:59] family, [58:54] BM/16, [53:48] BN/16,
 * [47:46] log2(BK/16), [45:42] stages, [41:32] P_k, [31] persistent tile loop,
 * [30:29] srcA, [28:27] srcB, [26] dtype, [25] layoutA, [24] layoutB, [23:22] log2(cluster) mod 4,
 * [21] log2(cluster) / 4, [20] fused in-cluster split-K reduction, [19] stream-K, [18:0] zero. */

/* Select the device (cudaSetDevice), query it, and create the library state for
 * it.  Idempotent.  Needed before adapt_matmul; planning works without it (the
 * selector then assumes a B200: 148 SMs, 227 KB shared memory, 512 TMEM columns). */
adapt_status_t adapt_init(int device);

/* Free plans, workspaces and cached tensor maps.  Every handle becomes invalid. */
void adapt_shutdown(void);

/* Section 3.2 / 5.1 "offline" half, done on first sight of a shape and cached:
 * classify (M,N,K), enumerate legal configurations, score each with the model,
 * keep the argmin (Eq. 6).  Same arguments -> same handle (pointer-equal).
 * Host work only, no GPU call.  A cache hit costs one hash probe.
 * Returns NULL on error (adapt_last_error tells why).
 * M, N, K >= 0 and <= 2^31-1.  M == 0 or N == 0 plans a no-op; K == 0 plans a zero fill. */
adapt_handle_t adapt_matmul_plan(int64_t M, int64_t N, int64_t K,
                                 adapt_dtype_t dtype, adapt_layout_t layoutA, adapt_layout_t layoutB);

/* Section 3.2 "online" half: run the planned kernel(s).
 * A, B, C: DEVICE pointers owned by the caller, 2-byte aligned at least (16-byte
 * aligned buffers let TMA read them in place; others are re-pitched through the
 * workspace first).  C must not overlap A or B.  cuda_stream is a cudaStream_t
 * (NULL = default stream).  The call enqueues work and returns without
 * synchronising.  The first call that needs a larger workspace than any before it
 * allocates (cudaMalloc), so it must not happen inside a stream capture.
 * Calls that share a stream may share the workspace; calls on different streams
 * get different workspaces. */
adapt_status_t adapt_matmul(adapt_handle_t plan, const void* A, const void* B, void* C, void* cuda_stream);

/* The persisted offline table.  The paper selects configurations offline for a target shape set, registers them in a
 * hash table and only looks them up online (Section 3.2, Section 5.1); here selection also runs on first sight of a
 * shape, and these three calls give the offline half back to a deployment that wants it.
 *
 * adapt_plan_many: plan `count` shapes in one call (dims: HOST array of 3*count values M, N, K; flags: HOST array of
 * 3*count values dtype, layoutA, layoutB; handles: optional HOST array of `count` handles to fill).  Returns the
 * number of shapes planned.
 * adapt_plan_table_save: write every selected plan of the cache (shape and 64-bit TilingKey, one text line each) to
 * `path`; returns the number of lines, -1 on error.
 * adapt_plan_table_load: read such a file and install its TilingKeys as the plans of their shapes, so that the first
 * online call of a listed shape is already a cache hit and runs exactly the recorded configuration, whatever the
 * model would choose today.  A shape that already has a plan keeps it; a line whose key is not a legal configuration
 * of its shape on this machine (another library version, another GPU) is skipped.  Returns the number of plans
 * installed, -1 if the file cannot be read or is not a table of this library version.  Host work only. */
int64_t adapt_plan_many(int64_t count, const int64_t* dims, const int32_t* flags, adapt_handle_t* handles);
int64_t adapt_plan_table_save(const char* path);
int64_t adapt_plan_table_load(const char* path);

/* The same call for operands that live in HOST memory (A_host, B_host inputs, C_host output,
 * dense, in the plan's layouts; pinned memory makes the copies asynchronous).  The library runs
 * the call on a three-stage pipeline of its own streams (copy A and B into a device staging
 * slot | the planned kernels | copy C back) with two staging slots per caller stream, so the
 * copies of consecutive calls overlap the kernels and each other.  Returns without
 * synchronising.  Ordering: the caller's stream is made to wait for the copy of C, so work
 * enqueued on it after the call (and cudaStreamSynchronize on it) sees C_host complete; the
 * host operands must be ready when the call is made (the copy in does NOT wait for earlier
 * work on the caller's stream) and stay untouched until the stream has been synchronised.
 * Calls that name the same stream must not be made from two threads at once.  The staging
 * slots grow on demand (cudaMalloc), like the workspace.  The paper has no counterpart (its
 * operator takes device tensors); this entry exists so that end-to-end cost including the PCIe
 * copies can be measured through one call. */
adapt_status_t adapt_matmul_host(adapt_handle_t plan, const void* A_host, const void* B_host, void* C_host,
                                 void* cuda_stream);

/* C = A * B for callers that must not trigger a device allocation: code running where cudaMalloc is
 * off limits, such as a latency-critical serving loop that forbids the implicit device
 * synchronisation an allocation brings, a process whose memory pool has been handed over whole to
 * another allocator, or a plug-in that is only given buffers and a stream.  The paper has no
 * counterpart to this entry point; it exists for those callers only.
 *
 * It runs the CUDA-core split-K path (fp32 partial products per K split, then the fixed-order
 * reduction with the single 16-bit cast) with the partials kept in a fixed 4 MiB array that is
 * part of the library image, so every GPU that loads the library holds those 4 MiB until the
 * process exits.  Limit: 2 * M * roundup(N, 8) * 4 bytes <= 4 MiB (at least two K splits must
 * fit); larger outputs are rejected with ADAPT_ERR_UNSUPPORTED and a message, and K must be >= 1,
 * M, N >= 1.  The number of splits is the largest that fits, at most 32 and at most ceil(K / 64).
 *
 * No cudaMalloc, cudaFree or other allocating call is made, neither adapt_init nor a plan is
 * needed, and the current device is used.  The first call on a device looks up the array's device
 * address (once per device); make that first call outside any stream capture.  All calls share
 * the one array, whatever the stream: two calls that overlap on the GPU race on it, so keep calls
 * on one stream or order them yourself.  The array keeps the previous call's partials; every
 * element that contributes to C is first written by the same call, so nothing needs clearing
 * (the reduction also loads the up to 7 pad columns between N and roundup(N, 8) of each partial
 * row, which no call writes, but it discards them unused).
 * A, B: DEVICE inputs in the stated layouts, C: DEVICE output, row-major M x N, 2-byte aligned.
 * Enqueues two kernels on the stream and returns without synchronising. */
adapt_status_t adapt_matmul_noalloc(int64_t M, int64_t N, int64_t K, adapt_dtype_t dtype,
                                    adapt_layout_t layoutA, adapt_layout_t layoutB,
                                    const void* A, const void* B, void* C, void* cuda_stream);

/* `count` independent GEMMs enqueued on one stream by one call: adapt_matmul(plans[i], A[i], B[i], C[i])
 * for i = 0 .. count-1, in that order, stopping at the first failure.  plans, A, B and C are HOST arrays
 * of `count` entries (the entries of A, B, C are device pointers).  It is the loop a caller would write,
 * moved behind the boundary so that a caller in an interpreted language pays its foreign-call cost once per
 * batch, not once per GEMM; each GEMM is still its own launch(es).  The paper replaces the vendor's
 * MatMul / GroupMM operators in recommendation models (Section 6.5), whose layers issue exactly such
 * lists of small GEMMs of different shapes.
 * A batch of eight or more calls is spread over up to four internal streams between a fork from and a join to
 * cuda_stream (work queued on cuda_stream before the call comes first, work queued after it comes last), so that
 * the launch gaps and the tail of one GEMM fill with the next one's work.  The result is the one of the calls made
 * in order: a call whose output overlaps a buffer that an earlier call of the batch still reads or writes on another
 * internal stream, or whose inputs overlap such an output, waits for that stream first.  Option "batch_streams"
 * (adapt_set_option; 1 to 4, default 4) sets the number of internal streams; with 1 the calls run one after the
 * other on cuda_stream itself.  The internal streams keep workspaces of their own.  Once a batch has run (workspaces
 * grown, tensor maps of its pointers cached) the same batch only launches kernels and records and waits for events, so
 * it can be captured into a CUDA graph through cuda_stream and replayed (1,200 launch-bound GEMMs: 5.1 ms direct,
 * 4.6 ms as a graph). */
adapt_status_t adapt_matmul_batch(int64_t count, const adapt_handle_t* plans, const void* const* A,
                                  const void* const* B, void* const* C, void* cuda_stream);

/* The other operators the paper replaces beside MatMul (Section 6.5 and the Conclusion: AddMM, BatchMM, GroupMM), on the
 * same plans.  GroupMM, a list of GEMMs of different shapes, is adapt_matmul_batch above.
 *
 * adapt_addmm:  C = alpha * (A * B) + beta * D, with the product accumulated in fp32 as in adapt_matmul, the scaling and
 * the addition done in fp32 on the accumulated sum, and ONE round-to-nearest-even cast to the 16-bit output.  D (DEVICE,
 * same 16-bit type) is an M x N row-major matrix (d_is_vector == 0) or one row of N values added to every output row
 * (d_is_vector != 0, a bias).  C may be D itself (in-place beta * C + alpha * A * B); it must not overlap A, B, or D in
 * any other way.  The GEMM kernels leave their fp32 sums in the workspace (as a split-K call does) and the fixed-order
 * reduction kernel applies alpha, beta and D before the cast, so the result is as reproducible as adapt_matmul's; plans
 * of the warp-level and one-launch families run on the CUDA-core kernel for this call.  K == 0 gives beta * D.
 *
 * adapt_matmul_strided_batch:  `batch` GEMMs of the plan's shape on operands stride_a, stride_b, stride_c ELEMENTS apart
 * (a stride of 0 shares that input across the batch; stride_c must be at least M * N), enqueued in batch order on the stream. */
adapt_status_t adapt_addmm(adapt_handle_t plan, const void* A, const void* B, const void* D, int d_is_vector,
                           float alpha, float beta, void* C, void* cuda_stream);
adapt_status_t adapt_matmul_strided_batch(adapt_handle_t plan, const void* A, int64_t stride_a, const void* B, int64_t stride_b,
                                          void* C, int64_t stride_c, int64_t batch, void* cuda_stream);

/* Harness support: `calls` back-to-back adapt_matmul calls of one plan, call i on operand set i % sets
 * (A, B, C: HOST arrays of `sets` device pointers).  Used to time one shape with rotating buffers. */
adapt_status_t adapt_matmul_repeat(adapt_handle_t plan, int sets, const void* const* A, const void* const* B,
                                   void* const* C, int calls, void* cuda_stream);

/* Host cost of the online call (Section 3.2 claims a "near-zero" dispatch; this measures it).
 * Runs `calls` adapt_matmul calls of the plan on the given operands three ways and reports, per call,
 * the host time (steady_clock around the calls, in batches of 128 with a stream synchronisation between
 * batches so the launch queue never fills) and the device time (CUDA events around each batch):
 * with the tensor-map cache on (the steady state of a caller that reuses buffers), with the cache
 * bypassed (every call encodes its tensor maps: a caller whose pointers are new every time), and as
 * bare launches: the kernels of one call, recorded with their exact configurations and arguments and
 * replayed through cudaLaunchKernelExC with none of the library's logic around them.
 * host_us_call - host_us_bare_launches is what the library adds to the launches themselves.
 * The bare fields are -1 when a launch could not be recorded.  Synchronises the stream. */
typedef struct adapt_dispatch_cost_s {
    double host_us_call, host_us_call_map_miss, host_us_bare_launches;
    double device_us_call, device_us_call_map_miss, device_us_bare_launches;
    int32_t launches_per_call;   /* kernels one call enqueues (prologue + GEMM + reduce) */
    int32_t maps_per_call;       /* tensor maps a call encodes when none is cached */
} adapt_dispatch_cost_t;
adapt_status_t adapt_measure_dispatch(adapt_handle_t plan, const void* A, const void* B, void* C,
                                      void* cuda_stream, int calls, adapt_dispatch_cost_t* out);

/* The launch floor: `launches` empty kernels back to back on the stream, with (programmatic != 0) or
 * without programmatic dependent launch; per launch, the host time and the device time (same batching
 * as above).  Every call of this library costs at least this much, whatever the kernel does. */
adapt_status_t adapt_measure_empty_launch(int launches, int programmatic, void* cuda_stream,
                                          double* host_us, double* device_us);

/* The write-only ceiling of the GEMM's store path (Eq. 2: a Common-template GEMM with a short K is a write of
 * 2*M*N bytes and little else).  Writes a 16-bit matrix [rows][cols] (DEVICE buffer of rows*cols*2 bytes, 32-byte
 * aligned, cols a multiple of 64; its contents are overwritten with a constant) `passes` times, tile by tile
 * (128 rows x tile_cols columns, tile_cols = 64, 128, 192 or 256) from persistent CTAs laid out like the GEMM's
 * epilogue warps, with nothing in front of the stores: mode 0 = TMA stores of 32 x 64 boxes (what the epilogue
 * issues), 1 = one 3-d TMA store of 32 rows x tile_cols per warp and tile, 2 = plain 32-byte stores.
 * order 0 visits the tiles in the GEMM's rasterisation, 1 row-block by row-block; hint != 0 stores with the
 * evict-first L2 policy.  *device_us = time of one pass (CUDA events).  Synchronises the stream. */
adapt_status_t adapt_measure_store_rate(void* buffer, int64_t rows, int64_t cols, int mode, int tile_cols,
                                        int order, int hint, int passes, void* cuda_stream, double* device_us);

/* Tensor maps encoded on the host since adapt_init; a call whose maps are cached encodes none.  Each plan
 * keeps the encodings of its 8 most recent distinct (pointer, geometry) pairs per operand. */
int64_t adapt_map_encode_count(void);
/* Run-time switches of the tcgen05 kernels, applied to calls made after it returns (the environment variables
 * ADAPT_SHUFFLE_K and ADAPT_PREFETCH set the same at start-up):
 *   "shuffle_k" (default 0): the ShuffleK module of Table 2: every tile walks its k-blocks in an order rotated by an
 *               amount that depends on the tile, so that the CTAs of a wave do not all ask for the same k slice of a shared
 *               operand at once.  The order is a function of the tile, so results stay reproducible, but they may differ
 *               in the last bit from those with the option off (another summation order).  Plain tiles only.
 *   "prefetch"  (default 1): L2 prefetch of a kernel's first operand boxes ahead of its wait for the kernel before it.
 *   "batch_streams" (default 4): internal streams of adapt_matmul_batch, 1 to 4 (see there). */
adapt_status_t adapt_set_option(const char* name, int value);

/* The analytical model's calibration constants (Section 5.2's machine terms: bandwidths, latencies, per-tile and
 * per-launch costs), by name.  adapt_calibration_names writes the comma-separated list of names to out (at most
 * cap - 1 characters and a terminating zero; out may be null) and returns the length of the whole list plus one.
 * A value set here is used by every plan made afterwards (adapt_matmul_plan, adapt_plan_candidates); plans already
 * in the cache keep their selection.  Host only, thread-safe; unknown name or NaN: ADAPT_ERR_INVALID_ARG.  Together
 * with adapt_plan_candidates and timed configurations (adapt_matmul_plan_forced) this is all a program needs to
 * refit the model for another machine; paper_2608_10803_b200/calibrate.py does it. */
adapt_status_t adapt_set_calibration(const char* name, double value);
adapt_status_t adapt_get_calibration(const char* name, double* value);
int adapt_calibration_names(char* out, int cap);
/* enabled = 0 bypasses the tensor-map cache (every call encodes); 1 restores it.  Measurement only. */
void adapt_set_map_cache(int enabled);

/* Self-test of the bounded-wait path: enqueues a one-warp kernel that waits, with the same bounded wait
 * the GEMM kernels use and a limit of limit_ns (at most 0.1 s), on a barrier nobody arrives on.  The wait
 * gives up, the kernel ends normally and sets the device status word, and the next
 * adapt_poll_device_status on the stream returns ADAPT_ERR_TIMEOUT (and clears the word).  Nothing is left
 * waiting and the context stays usable.  The paper has no counterpart. */
adapt_status_t adapt_selftest_wait_expiry(uint64_t limit_ns, void* cuda_stream);

/* Thread-local status of the last failing call on this thread, and its text. */
adapt_status_t adapt_last_error(void);
const char* adapt_last_error_message(void);
const char* adapt_status_string(adapt_status_t s);

/* Copy the plan's decision into *out (host memory). */
adapt_status_t adapt_plan_info(adapt_handle_t plan, adapt_plan_info_t* out);

/* Every legal configuration for the shape with its predicted time (Eq. 6's search
 * set S(b(s)) after the capacity check), best first.  Writes at most cap entries
 * to out (host memory) and returns the total number of legal candidates, or -1. */
int adapt_plan_candidates(int64_t M, int64_t N, int64_t K,
                          adapt_dtype_t dtype, adapt_layout_t layoutA, adapt_layout_t layoutB,
                          adapt_plan_info_t* out, int cap);

/* Bypass the model: a plan that runs exactly the configuration encoded in
 * tiling_key (as reported by adapt_plan_candidates).  Used to time every legal
 * variant (the paper's model-validation method, Section 6.6).  Cached per
 * (shape, key).  NULL + ADAPT_ERR_UNSUPPORTED if the key is not legal for the shape. */
adapt_handle_t adapt_matmul_plan_forced(int64_t M, int64_t N, int64_t K,
                                        adapt_dtype_t dtype, adapt_layout_t layoutA, adapt_layout_t layoutB,
                                        uint64_t tiling_key);

/* The taxonomy by itself (Section 4.2), parameterised by the machine: returns the
 * adapt_class_t of a shape tiled by m x n sub-tasks with an m1 x n1 accumulation
 * tile on n_core cores with acc_bytes of fp32 accumulator per core; -1 on bad input. */
int adapt_classify(int64_t M, int64_t N, int64_t m, int64_t n, int64_t m1, int64_t n1,
                   int64_t n_core, int64_t acc_bytes);

/* Closed-form building blocks of the model, exported for validation:
 * Eq. 1 read volume, Eq. 2-5 write volumes (bytes), Eq. 12-14 pipeline times. */
double adapt_model_read_volume(int64_t M, int64_t N, int64_t K, int64_t m1, int64_t n1);
double adapt_model_write_volume(int cls, int64_t M, int64_t N, int64_t K, int64_t k, int64_t k1);
double adapt_model_pipeline(int schedule /*0 baseline, 1 double buffer, 2 preload*/,
                            int64_t Q, int64_t L, double t_M, double t_P, double T_drain);

/* Synchronise the stream, then read and clear the device status word.  Returns
 * ADAPT_ERR_TIMEOUT if a kernel's bounded barrier wait expired since the last
 * poll, ADAPT_ERR_CUDA if the stream reports a fault, else ADAPT_OK. */
adapt_status_t adapt_poll_device_status(void* cuda_stream);

/* Number of plans in the cache (both selected and forced). */
int64_t adapt_plan_cache_size(void);

/* Count of kernels this library has launched since adapt_init (all streams). */
int64_t adapt_launch_count(void);

#ifdef __cplusplus
}
#endif
#endif /* ADAPT_MATMUL_H */

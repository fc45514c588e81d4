// tcgen05 GEMM kernel: the "Common" / "MultiCoreSplitK" templates (Section 4.2) on B200.
//
// One CTA (CG = 1) owns a 128 x BN output tile; a CTA pair (CG = 2) owns 256 x BN, each CTA
// loading its own 128 rows of A and its own BN/2 columns of B (no multicast).  Pipeline
// (Section 5.2, Eq. 9/13/14 restated for this machine):
//
//   producer warp : TMA, 128-byte swizzle, into an S-stage shared-memory ring   (the paper's MTE2)
//   MMA warp      : one thread issues tcgen05.mma kind::f16, 128|256 x BN x 16,
//                   fp32 accumulator in TMEM, 2-4 accumulator buffers           (Cube + L0C)
//   8 epilogue warps: tcgen05.ld -> one RN-even cast -> shared -> TMA store of a 64 x 32 box, or
//                   coalesced 16 B stores where C's rows rule TMA out                 (FixPipe)
//
// The CTA is persistent: it walks its list of work units (tile x k-split) so the producer runs
// ahead across tile boundaries (Preloading, Eq. 14) and the epilogue of unit u overlaps the main
// loop of unit u+1.  With P_k > 1 a unit covers a fixed k-block range and writes an fp32 partial
// tile to the workspace (Eq. 4); a separate kernel adds the partials in ascending split order.
// MODE selects how unaligned operands are reached without a copy (row classes of A, k classes of
// B, halo class tiles for C): see the comment in front of the kernel.
#pragma once

#include <cuda.h>
#include <cuda_fp16.h>
#include <cuda_bf16.h>

#include "adapt_internal.h"
#include "ptx_sm100.cuh"
#include "launch_pdl.cuh"

namespace adapt {

constexpr int kUmmaBK = 64;          // k-block: 64 elements = one 128-byte swizzle row
constexpr int kUmmaThreads = 320;    // producer warp, MMA warp, eight epilogue warps
constexpr int kGroupM = 16;          // rasterisation: m-blocks per group

struct UmmaParams {
    int M, N, K;
    int P_m, P_n, P_k;               // task counts (Table 1)
    int kb_total, kb_per_split;      // k-blocks in K, k-blocks per split
    int num_units;                   // P_m * P_n * P_k
    int dtype;                       // ADAPT_F16 / ADAPT_BF16
    int stages;
    uint32_t idesc;                  // tcgen05 instruction descriptor
    void* C;                         // 16-bit output, row-major M x N (used when P_k == 1)
    float* partial;                  // fp32 [P_k][M][Np], Np = N rounded up to 8 (used when P_k > 1)
    int Np;                          // row pitch of the partials in elements
    int a_tx_bytes;                  // bytes one TMA load of A delivers per stage and CTA (a short box when M < 128)
    int b_tx_bytes;                  // bytes the TMA loads of B deliver per stage and CTA: the full boxes, or, for a row-major B
                                     // when K fits one k-block, boxes of just the k rows that exist (rounded up to 8); the rows of
                                     // the stage they leave untouched are zeroed once at kernel start
    int a_shift_any;                 // class mode: some a_sigma[j] != 0 (the MMA warp then zeroes row heads)
    int a_sigma[16];                 // class mode: shift (elements) of row class j against its 16-byte aligned base
    int b_sigma[8];                  // k-class mode: column shift of B's row class j = k % 8
    int cls_kc;                      // k-class mode: padded length of one class segment of A' (multiple of 64)
    int c_mode;                      // 16-bit output: 0 = stores by the epilogue threads (any N, any alignment),
                                     // 1 = TMA stores through the maps of C (rows of C, or of the tile's row class,
                                     //     start on 32-byte boundaries; class tiles with 16 halo columns shift them there)
    int force_partial;               // write fp32 partials also with P_k = 1 (a fused-add epilogue follows in the reduction kernel)
    int shuffle_k;                   // ShuffleK (Table 2): a tile starts its k range at a k-block that depends on the tile, so the CTAs of a wave
                                     // do not all ask for the same k slice of a shared operand at the same moment (plain tiles only)
    int prefetch;                    // ask L2 for the first unit's operand boxes before waiting for the kernel ahead on the stream
    int raster;                      // tile visiting order: 0 = m-fastest inside groups of kGroupM m-blocks (operand reuse in L2),
                                     // 1 = n-fastest, row block by row block (write-bound shapes: neighbouring CTAs write
                                     //     neighbouring column blocks of the same rows, and a CTA's consecutive class tiles share their maps)
    int c_hint;                      // TMA stores of C carry an evict-first L2 policy
    int part_hint;                   // fp32 partials are stored with an evict-last L2 policy (they fit in L2)
    int c_sigma[16];                 // halo class tiles: shift (elements) of C's row class j against its 32-byte aligned base
    int c_extent[16];                // ... and the elements of a shifted row of that class that lie in whole 32-byte units
    // stream-K (SK kernels): the first sk_tiles tiles are cut into k-block ranges shared evenly by all slots (a slot is a
    // CTA, or a CTA pair): slot s takes sk_q0 (+1 for s < sk_rem) consecutive k-blocks of the tile-major sequence
    int sk_tiles, sk_q0, sk_rem;
    float* sk_partial;               // one fp32 partial tile [128][BN] per CTA (slot * CTAs per slot + rank in the pair)
    unsigned int* sk_flags;          // one word per CTA: the epoch of the launch whose partial is complete there
    unsigned int sk_epoch;           // this launch's epoch (unique per workspace)
    int x_rows, x_pitch;             // fused split-K: rows and row pitch (fp32 elements) of the partial tile each CTA of the
                                     // cluster keeps in its shared memory for the exchange
    int ncls_log2;                   // halo class tiles: log2 of the number of row classes (1 .. 4)
    unsigned int* status;            // device status word: bit 0 = a bounded wait expired
    unsigned long long* trace;       // timestamp trace of one CTA (diagnostic builds only), else null
    int trace_cta;
};

#ifdef ADAPT_TRACE_BUILD
#define ADAPT_TRACE(ev, unit)                                                                         \
    do {                                                                                              \
        if (p.trace && (int)blockIdx.x == p.trace_cta) {                                                             \
            const unsigned long long sl = atomicAdd(p.trace, 1ull);                                   \
            if (sl < 30000) { p.trace[1 + 2 * sl] = ((unsigned long long)(ev) << 32) | (unsigned)(unit); p.trace[2 + 2 * sl] = ptx::globaltimer_ns(); } \
        }                                                                                             \
    } while (0)
#else
#define ADAPT_TRACE(ev, unit) do { } while (0)
#endif

// Tensor maps of one launch, sized by the kernel mode (the pack is a kernel parameter, so the plain mode
// passes three maps, not forty).  a[0] is the map of A; in class mode a[j] is the map of the rows of A in
// row class j (see the kernel comment).  b[0] is the map of B; in k-class mode b[j] is the map of the
// k-rows with k % 8 == j.  c[] are the maps of C for the TMA-store epilogue (c_mode != 0): c[0], or one
// per row class.
template <int MODE>
struct TmapPackT {
    CUtensorMap a[MODE == 1 ? 16 : 1];
    CUtensorMap b[MODE >= 2 ? 8 : 1];
    CUtensorMap c[MODE == 1 ? 16 : 1];
};

// unit index -> (m block, n block, split).  Units of one output tile are adjacent in split;
// tiles are visited in groups of kGroupM m-blocks so that concurrently running CTAs share B
// columns and A rows in L2.
__device__ __forceinline__ void decode_unit(const UmmaParams& p, int unit, int& mb, int& nb, int& split)
{
    split = unit % p.P_k;
    const int t = unit / p.P_k;
    if (p.raster == 1) {
        mb = t / p.P_n;
        nb = t - mb * p.P_n;
        return;
    }
    const int group_size = kGroupM * p.P_n;
    const int g = t / group_size;
    const int first_m = g * kGroupM;
    const int gm = min(p.P_m - first_m, kGroupM);
    const int r = t - g * group_size;
    mb = first_m + r % gm;
    nb = r / gm;
}

// One entry of a slot's work list.  kind 0: the whole k range of a tile (or one split of it), stored the usual way;
// kind 1 (stream-K): a k range that does not start at 0: an fp32 partial tile for the slot that owns the tile's start;
// kind 2 (stream-K): the start of a tile whose later k ranges `npeers` following slots contribute.
struct WorkItem {
    int unit, mb, nb, split, kb0, kb1, kind, npeers;
};

// The it-th work item of slot `slot` (of `n_slots`).  Without stream-K: unit slot + it * n_slots.  With stream-K
// (Section 4.2's StreamK remark, made deterministic): first the slot's share of the stream-K tiles (at most two
// ranges: the end of one tile, then the start of the next), then whole tiles sk_tiles + slot + j * n_slots.
template <bool SK, bool B_SPLIT>
__device__ __forceinline__ bool next_item(const UmmaParams& p, int slot, int n_slots, int it, WorkItem& w)
{
    w.kind = 0;
    w.npeers = 0;
    if (!SK) {
        w.unit = slot + it * n_slots;
        if (w.unit >= p.num_units) return false;
        decode_unit(p, w.unit, w.mb, w.nb, w.split);
        w.kb0 = (B_SPLIT ? (w.split >> 3) : w.split) * p.kb_per_split;
        w.kb1 = min(p.kb_total, w.kb0 + p.kb_per_split);
        return true;
    }
    const int L = p.kb_total;
    const int begin = slot * p.sk_q0 + min(slot, p.sk_rem);
    const int len = p.sk_q0 + (slot < p.sk_rem ? 1 : 0);
    const int t1 = begin / L, a = begin - t1 * L;
    const bool crosses = a + len > L;
    // The slot's share is at most two ranges: the END of tile t1 (when it does not start at k-block 0) and the START of
    // the next tile.  The end range comes first: its partial is what the previous slot will need.  The start range comes
    // LAST, after the slot's whole tiles: by then the slots that hold the rest of that tile have long written theirs.
    const int n_first = (len > 0 && a != 0) ? 1 : 0;
    const int n_last = (len > 0 && (a == 0 || crosses)) ? 1 : 0;
    const int first_dp = p.sk_tiles + slot;
    const int n_dp = first_dp < p.num_units ? (p.num_units - first_dp + n_slots - 1) / n_slots : 0;
    int tile;
    if (it < n_first) {
        tile = t1; w.kb0 = a; w.kb1 = min(L, a + len);
        w.kind = 1;
    } else if (it < n_first + n_dp) {
        tile = first_dp + (it - n_first) * n_slots;
        w.kb0 = 0;
        w.kb1 = L;
    } else if (it < n_first + n_dp + n_last) {
        if (a == 0) { tile = t1; w.kb1 = len; }
        else { tile = t1 + 1; w.kb1 = a + len - L; }
        w.kb0 = 0;
        if (w.kb1 != L) {
            // the slots after this one that hold the rest of the tile: up to the owner of its last k-block
            const int last = (tile + 1) * L - 1;
            const int cut = p.sk_rem * (p.sk_q0 + 1);
            const int owner = last < cut ? last / (p.sk_q0 + 1) : p.sk_rem + (last - cut) / p.sk_q0;
            w.kind = 2;
            w.npeers = owner - slot;
        }
    } else {
        return false;
    }
    w.unit = tile;
    decode_unit(p, tile, w.mb, w.nb, w.split);
    return true;
}

__device__ __forceinline__ uint32_t pack16(float a, float b, int dtype)
{
    if (dtype == 0) {
        __half2 h = __floats2half2_rn(a, b);
        return *reinterpret_cast<uint32_t*>(&h);
    }
    __nv_bfloat162 h = __floats2bfloat162_rn(a, b);
    return *reinterpret_cast<uint32_t*>(&h);
}
__device__ __forceinline__ unsigned short cast16(float a, int dtype)
{
    if (dtype == 0) { __half h = __float2half_rn(a); return *reinterpret_cast<unsigned short*>(&h); }
    __nv_bfloat16 h = __float2bfloat16_rn(a);
    return *reinterpret_cast<unsigned short*>(&h);
}

// Stores the casts of e[0 .. count), count <= 16, at dst .. dst + count as the fewest aligned stores of 16, 8, 4
// and 2 bytes.  count and the alignment of dst are the same for every row of a tile, so the branches are
// uniform; e is indexed with compile-time constants only.
__device__ __forceinline__ void store_run16(unsigned short* dst, int count, const uint32_t (&e0)[8], const uint32_t (&e1)[8], int dtype)
{
    const int a = (int)((reinterpret_cast<uintptr_t>(dst) >> 1) & 7);     // element offset inside a 16-byte chunk
    int next = 0;
#pragma unroll
    for (int i = 0; i < 16; ++i) {
        if (next != i || i >= count) continue;
        const int pos = a + i, left = count - i;
#define ADAPT_E(k) __uint_as_float((k) < 8 ? e0[(k) & 7] : e1[(k) & 7])
        if (i + 8 <= 16 && (pos & 7) == 0 && left >= 8) {
            uint4 v;
            v.x = pack16(ADAPT_E(i), ADAPT_E(i + 1), dtype);
            v.y = pack16(ADAPT_E(i + 2), ADAPT_E(i + 3), dtype);
            v.z = pack16(ADAPT_E(i + 4), ADAPT_E(i + 5), dtype);
            v.w = pack16(ADAPT_E(i + 6), ADAPT_E(i + 7), dtype);
            *reinterpret_cast<uint4*>(dst + i) = v;
            next = i + 8;
        } else if (i + 4 <= 16 && (pos & 3) == 0 && left >= 4) {
            uint2 v;
            v.x = pack16(ADAPT_E(i), ADAPT_E(i + 1), dtype);
            v.y = pack16(ADAPT_E(i + 2), ADAPT_E(i + 3), dtype);
            *reinterpret_cast<uint2*>(dst + i) = v;
            next = i + 4;
        } else if (i + 2 <= 16 && (pos & 1) == 0 && left >= 2) {
            *reinterpret_cast<uint32_t*>(dst + i) = pack16(ADAPT_E(i), ADAPT_E(i + 1), dtype);
            next = i + 2;
        } else {
            dst[i] = cast16(ADAPT_E(i), dtype);
            next = i + 1;
        }
#undef ADAPT_E
    }
}

// A_CLS ("row classes", the Padding module without a copy): A is row-major with K % 8 != 0, so its
// rows are not 16-byte aligned and one tensor map cannot describe it.  Rows r and r + 8 do start
// at the same offset from a 16-byte boundary (their distance is 16*K bytes), so the rows of one
// residue class j = r % 8 form a tensor TMA can read: base rounded down to 16 bytes, row pitch
// 16*K bytes, every row shifted by the same sigma_j elements.  An m-tile then takes 128 rows of
// ONE class (rows 1024*g + j + 8*i), its k index runs over kappa = k + sigma_j, and B's k-rows
// (an outer TMA coordinate, free of alignment rules) start at kappa - sigma_j; rows of B' with
// kappa < sigma_j or k >= K are out of bounds and read as zero.  The sigma_j leading elements of
// each A' row belong to the previous row of A: the MMA warp overwrites them with zeros in the
// first k-block before the tensor core reads them.
//
// B_CLS (MODE 2, "k classes"): B is row-major with N % 8 != 0.  Its rows k and k + 8 share their
// offset from a 16-byte boundary, so the k-rows of one residue class j = k % 8 form a tensor TMA can
// read, every row shifted by the same sigma_j columns.  The contraction runs class by class: a
// prologue kernel has regrouped A's columns class-major (A'[m][j][t] = A[m][8t + j], zero padded),
// class j accumulates into its own TMEM buffer j (8 buffers of 64 columns) over the window
// x' in [56*nb, 56*nb + 64) of shifted columns, and the epilogue adds the eight buffers with
// buffer j read sigma_j columns to the right: C[m][56*nb + c] = sum_j acc_j[m][c + sigma_j], c < 56.
// Columns of a buffer left of sigma_j hold products with the previous row's tail and are never read.
//
// B_SPLIT (MODE 3, "k classes as k splits"): the same views of B, but each class is a k split of its
// own: unit (tile, split) with split = 8 * ks + j contracts the k-blocks of class j in range ks into one
// accumulator of BN columns over the window x' in [(BN-8)*nb, (BN-8)*nb + BN) and writes the BN - 8
// columns the tile owns as an fp32 partial (read sigma_j columns to the right); the reduction kernel adds
// the 8 * P_kk slabs in ascending order.  Full-width tiles, at the price of 8 partials per output.
//
// FUSE ("MultiCoreSplitK" in one launch, Eq. 4 / Eq. 11 without the trip through global memory): the P_k splits
// of a tile are the CTAs of one thread-block cluster (P_k = 2, 4 or 8; rank = split).  Each CTA drains its fp32
// accumulator into its own shared memory; when all have (mbarrier arrivals across the cluster), the CTAs share
// the tile's (row, 4-column) groups evenly, and each adds its groups over ranks 0 .. P_k-1 in ascending order
// through distributed shared memory, rounds once and stores C.  The order is the one splitk_reduce_kernel
// uses, so a shape gives the same bits with either path and from run to run.
//
// SK (stream-K, plain tiles, P_k = 1): when the tiles do not fill whole waves of slots, the k-blocks of the first
// sk_tiles tiles are shared evenly by all slots.  A slot's share is one run of the tile-major k-block sequence: the end
// of one tile (written as an fp32 partial, then a flag), then the start of the next, whose remaining k ranges the
// following slots computed FIRST; the slot adds their partials to its accumulator in ascending k order and stores the
// tile.  The assignment and the order of the additions are fixed by the shape, so the result is too.  Every wait on a
// flag is bounded like the barrier waits.
template <int BN, bool A_MN, bool B_MN, int CG, int MODE, bool FUSE = false, bool SK = false>
__global__ void __launch_bounds__(kUmmaThreads, 1)
umma_gemm_kernel(const __grid_constant__ TmapPackT<MODE> maps, const UmmaParams p)
{
    static_assert(!SK || (MODE == 0 && !FUSE), "stream-K: plain tiles");
    static_assert(!FUSE || (CG == 1 && (MODE == 0 || MODE == 1 || MODE == 3)), "the fused reduction: 1-CTA tiles, clusters made of the k splits");
    static_assert(!FUSE || BN % 64 == 0, "the fused reduction has no halo tiles");
    constexpr bool A_CLS = MODE == 1;
    constexpr bool B_CLS = MODE == 2;
    constexpr bool B_SPLIT = MODE == 3;                   // k classes as k splits (see below)
    static_assert(MODE == 0 || (!A_MN && B_MN), "class modes: K-major A, row-major B");
    static_assert(MODE != 2 || CG == 1, "tiles with eight class accumulators: one CTA per tile");
    static_assert(!B_CLS || BN == 64, "k-class mode uses 64-column windows");
    // HALO: class tiles for a C whose rows do not start on 32-byte boundaries (N % 16 != 0) own 32-byte
    // units of the shifted rows instead of columns, so they compute 16 columns more than they own (see
    // the epilogue); they use 16 row classes, since rows 16 apart share their offset from such a boundary
    constexpr bool HALO = A_CLS && (BN % 64 != 0);
    static_assert(BN % 64 == 0 || (A_CLS && (BN - 16) % 64 == 0), "BN is a multiple of 64, plus 16 halo columns for class tiles");
    // row classes of a class tile (rows NCLS*128*g + j + NCLS*i): 8, or for halo tiles as many as C's rows need to share
    // their offset from a 32-byte boundary (16 for an odd N, 8, 4 or 2 for an even one: p.ncls_log2)
    const int NSH = HALO ? p.ncls_log2 : 3;
    const int NCLS = 1 << NSH;
    constexpr int TILE_N = B_CLS ? 56 : (B_SPLIT ? BN - 8 : (HALO ? BN - 16 : BN));   // output columns (HALO: chunk-aligned elements) a tile owns
    constexpr int BN_CTA = BN / CG;                       // B columns this CTA loads
    // the A region of a stage holds the rows one box brings (128, or fewer for a short K-major A)
    const int A_BYTES = (CG == 2) ? 128 * kUmmaBK * 2 : p.a_tx_bytes;
    constexpr int B_BOXES = (BN_CTA + 63) / 64;           // row-major B arrives in boxes of 64 columns
    constexpr int B_BYTES = B_BOXES * 64 * kUmmaBK * 2;
    const int STAGE_BYTES = A_BYTES + B_BYTES;
    constexpr int NBUF = B_CLS ? 1 : ((512 / BN) < 4 ? (512 / BN) : 4);   // accumulator buffers in TMEM
    constexpr int TMEM_COLS = (B_CLS || HALO) ? 512 : NBUF * BN;    // k-class mode: eight class accumulators of 64 columns
    constexpr int PASSES = (TILE_N + 63) / 64;            // 64-column epilogue passes per tile
    static_assert(TMEM_COLS == 256 || TMEM_COLS == 512, "TMEM allocation is a power of two");
    static_assert(NBUF * BN <= TMEM_COLS, "accumulators fit the allocation");
    static_assert(B_MN || BN_CTA % 64 == 0, "a K-major B tile is one box of BN rows");

    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (ptx::smem_u32(smem_raw) + 1023u) & ~1023u;   // swizzle atoms are 1024-byte aligned
    const int S = p.stages;
    const uint32_t bar_base = smem_base + (uint32_t)S * STAGE_BYTES;
    // barrier block: full[S], empty[S], tmem_full[NBUF], tmem_empty[NBUF], the TMEM pointer, the abort flag
    const uint32_t full_bar = bar_base;
    const uint32_t empty_bar = bar_base + 8u * S;
    const uint32_t tfull_bar = bar_base + 16u * S;
    const uint32_t tempty_bar = tfull_bar + 8u * NBUF;
    const uint32_t tmem_slot = tempty_bar + 8u * NBUF;
    uint8_t* gen_base = smem_raw + (smem_base - ptx::smem_u32(smem_raw));
    uint8_t* bar_gen = gen_base + (size_t)S * STAGE_BYTES;
    volatile uint32_t* tmem_slot_ptr = reinterpret_cast<volatile uint32_t*>(bar_gen + 16 * S + 16 * NBUF);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(bar_gen + 16 * S + 16 * NBUF + 4);
    // epilogue staging: one row of 72 16-bit elements (64 columns + up to 7 of shift) per epilogue thread
    // (fused split-K: the CTA's fp32 partial tile instead)
    uint8_t* stage_out = bar_gen + kUmmaBarrierBytes;
    // fused split-K: "every rank's partial is in place" / "every rank has read mine", at fixed offsets of the barrier block
    const uint32_t xfull_bar = bar_base + 512u, xempty_bar = bar_base + 520u;
    // pair tiles of one row class: "this CTA's A box has landed" (each CTA, own loads) and, in the leader, "the peer's A
    // box has landed and its stale row heads are zeroed"
    const uint32_t afull_bar = bar_base + 544u, aready_bar = bar_base + 672u;
    int* sk_count = reinterpret_cast<int*>(bar_gen + 528);     // stream-K: epilogue warps that have written their share of a partial

    pdl_launch_dependents();
    if (threadIdx.x == 0) ADAPT_TRACE(11, 0);
    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    const uint32_t cta_rank = (CG == 2) ? ptx::cluster_ctarank() : 0u;
    const bool leader = cta_rank == 0;

    if (threadIdx.x == 0) {
        *abort_flag = 0;
        *sk_count = 0;
        for (int s = 0; s < S; ++s) {
            ptx::mbar_init(full_bar + 8u * s, 1);          // one arrive.expect_tx per phase
            ptx::mbar_init(empty_bar + 8u * s, 1);         // one tcgen05.commit per phase
        }
        for (int b = 0; b < NBUF; ++b) {
            ptx::mbar_init(tfull_bar + 8u * b, 1);         // one tcgen05.commit per phase
            ptx::mbar_init(tempty_bar + 8u * b, kUmmaEpilogueWarps * CG);   // one arrive per epilogue warp of the group
        }
        if (A_CLS && CG == 2) {
            for (int st = 0; st < S; ++st) {
                ptx::mbar_init(afull_bar + 8u * st, 1);
                ptx::mbar_init(aready_bar + 8u * st, 1);
            }
        }
        if (FUSE) {
            ptx::mbar_init(xfull_bar, (uint32_t)(kUmmaEpilogueWarps * p.P_k));     // one arrive per epilogue warp of every rank
            ptx::mbar_init(xempty_bar, (uint32_t)(kUmmaEpilogueWarps * p.P_k));
        }
        ptx::fence_barrier_init();
        ptx::fence_proxy_async_smem();
        // the maps this CTA's first unit goes through (a class tile reads A and writes C through its class's maps)
        int mb0 = 0, nb0 = 0, sp0 = 0;
        const int first_unit = (CG == 2) ? (int)(blockIdx.x >> 1) : (int)blockIdx.x;
        if (first_unit < p.num_units) decode_unit(p, first_unit, mb0, nb0, sp0);
        ptx::prefetch_tensormap(&maps.a[A_CLS ? (mb0 & (NCLS - 1)) : 0]);
        ptx::prefetch_tensormap(&maps.b[(B_SPLIT || B_CLS) ? (sp0 & 7) : 0]);
        if (p.c_mode != 0) ptx::prefetch_tensormap(&maps.c[A_CLS ? (mb0 & (NCLS - 1)) : 0]);
    }
    if (warp == 1) {
        ptx::tmem_alloc<CG>(tmem_slot, TMEM_COLS);
        ptx::tmem_relinquish<CG>();
    } else if (p.b_tx_bytes < B_BYTES) {
        // Short-K boxes of B: a load then brings only the k rows that exist, so the rest of every stage's B region is
        // zeroed here, once (no load ever writes it; the tensor core multiplies it with the zero-filled k tail of A).
        // Boxes made of 64 k rows of which most lie beyond K cost a wide B several times the load time of full ones.
        const int t = threadIdx.x >= 64 ? (int)threadIdx.x - 32 : (int)threadIdx.x;     // 288 threads, warp 1 left out
        for (int st = 0; st < S; ++st) {
            uint4* dst = reinterpret_cast<uint4*>(gen_base + (size_t)st * STAGE_BYTES + A_BYTES);
            for (int i = t; i < B_BYTES / 16; i += kUmmaThreads - 32) dst[i] = make_uint4(0u, 0u, 0u, 0u);
        }
        ptx::fence_proxy_async_smem();
    }
    ptx::tc_fence_before();
    if (CG == 2 || FUSE) {      // peers arrive on this CTA's barriers: they must all exist first
        asm volatile("barrier.cluster.arrive.release.aligned;\nbarrier.cluster.wait.acquire.aligned;" ::: "memory");
    } else {
        __syncthreads();
    }
    ptx::tc_fence_after();
    const uint32_t tmem_base = *tmem_slot_ptr;
    const int unit0 = (CG == 2) ? (int)(blockIdx.x >> 1) : (int)blockIdx.x;
    const int unit_step = (CG == 2) ? (int)(gridDim.x >> 1) : (int)gridDim.x;

    // While the kernel ahead of this one on the stream drains, ask L2 for the operand boxes of this CTA's first unit
    // (up to one ring of k-blocks).  Prefetches are hints: they bring lines (and address translations) in early and
    // commit to nothing, so they may run ahead of griddepcontrol.wait; the loads proper still come after it.  A problem
    // of a few tiles spends most of its time waiting for its first bytes (2.5 to 5 us from a cold buffer), and with
    // programmatic dependent launch that wait now overlaps the previous kernel.
    if (warp == 0 && !B_CLS && p.prefetch) {
        constexpr int NREQ_A = A_MN ? 2 : 1;
        constexpr int NREQ = NREQ_A + (B_MN ? B_BOXES : 1);
        WorkItem w;
        if (lane < NREQ && next_item<SK, B_SPLIT>(p, unit0, unit_step, 0, w)) {
            const int cls = A_CLS ? (w.mb & (NCLS - 1)) : 0;
            const int row0 = A_CLS ? (w.mb >> NSH) * (128 * CG) + (int)cta_rank * 128 : w.mb * (128 * CG) + (int)cta_rank * 128;
            const int kshift = A_CLS ? p.a_sigma[cls] : 0;
            const int a_k_off = B_SPLIT ? (w.split & 7) * p.cls_kc : 0;
            const int col0 = w.nb * TILE_N + (int)cta_rank * BN_CTA;
            const int jb = lane - NREQ_A;
            for (int kb = w.kb0; kb < w.kb1 && kb < w.kb0 + S; ++kb) {
                const int k0 = kb * kUmmaBK;
                if (lane < NREQ_A) {
                    if (!A_MN) ptx::tma_prefetch_2d(&maps.a[cls], k0 + a_k_off, row0);
                    else ptx::tma_prefetch_2d(&maps.a[cls], row0 + lane * 64, k0);
                } else {
                    const CUtensorMap* tmB = &maps.b[B_SPLIT ? (w.split & 7) : 0];
                    if (B_MN) ptx::tma_prefetch_2d(tmB, col0 + jb * 64, k0 - kshift);
                    else ptx::tma_prefetch_2d(tmB, k0, col0);
                }
            }
        }
    }

    // set-up done: from here on the kernel reads and writes global memory
    if (threadIdx.x == 0) ADAPT_TRACE(12, 0);
    pdl_wait();
    if (threadIdx.x == 0) ADAPT_TRACE(13, 0);

    if (warp == 0) {
        // ------------------------------ producer -----------------------------------------------
        // One lane per TMA request of a k-block (A: one box, two when M-contiguous; B: one box, or one per 64
        // columns when N-contiguous): the lanes run the loop together and issue their requests with one
        // instruction.  A single lane issuing them one after the other spends about 0.1 us per request, which
        // bounds a 128 x 256 tile with an N-contiguous B (five requests per k-block) at 0.5 us per k-block.
        constexpr int NREQ_A = A_MN ? 2 : 1;
        constexpr int NREQ = NREQ_A + (B_MN ? B_BOXES : 1);
        constexpr uint32_t REQ_MASK = (1u << NREQ) - 1u;
        if (lane < NREQ) {
            int stage = 0;
            uint32_t phase = 0;
            // the byte count of a stage is signalled on the leader's barrier (pair form)
            uint32_t full_target = full_bar;
            if (CG == 2) asm volatile("mapa.shared::cluster.u32 %0, %1, 0;" : "=r"(full_target) : "r"(full_bar));
            uint32_t afull_own = afull_bar;       // pair tiles of one row class: this CTA's own A barrier as a cluster address
            if (CG == 2) asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(afull_own) : "r"(afull_bar), "r"(cta_rank));
            bool ok = true;
            auto load = [&](uint32_t dst, const CUtensorMap* tm, uint32_t bar, int x, int y) {
                if (CG == 1) ptx::tma_load_2d(dst, tm, bar, x, y);
                else ptx::tma_load_2d_pair(dst, tm, bar, x, y);
            };
            const bool is_a = lane < NREQ_A;
            const int jb = lane - NREQ_A;                                     // B box of this lane
            for (int it = 0; ok; ++it) {
                WorkItem w;
                if (!next_item<SK, B_SPLIT>(p, unit0, unit_step, it, w)) break;
                const int unit = w.unit, mb = w.mb, nb = w.nb, split = w.split, kb0 = w.kb0, kb1 = w.kb1;
                // A rows of this CTA: consecutive rows, or in class mode rows 1024*g + j + 8*i read through
                // map j at class-row index 128*g
                const int cls = A_CLS ? (mb & (NCLS - 1)) : 0;
                const int row0 = A_CLS ? (mb >> NSH) * (128 * CG) + (int)cta_rank * 128 : mb * (128 * CG) + (int)cta_rank * 128;
                const int kshift = A_CLS ? p.a_sigma[cls] : 0;                // B's k-rows lag A's kappa by sigma
                const CUtensorMap* tmA = &maps.a[cls];
                const CUtensorMap* tmB = &maps.b[B_SPLIT ? (split & 7) : 0];  // k classes as splits: the class's view of B
                if ((A_CLS || B_SPLIT) && lane == 0 && unit + unit_step < p.num_units) {
                    // the next unit may go through other maps: fetch their descriptors while this unit loads
                    int mb2, nb2, sp2;
                    decode_unit(p, unit + unit_step, mb2, nb2, sp2);
                    if (A_CLS && (mb2 & (NCLS - 1)) != cls) ptx::prefetch_tensormap(&maps.a[mb2 & (NCLS - 1)]);
                    if (B_SPLIT && (sp2 & 7) != (split & 7)) ptx::prefetch_tensormap(&maps.b[sp2 & 7]);
                }
                const int a_k_off = B_SPLIT ? (split & 7) * p.cls_kc : 0;     // ... and its segment of the regrouped A
                const int col0 = nb * TILE_N + (int)cta_rank * BN_CTA;        // this CTA's B columns
                if (B_CLS) {
                    // class by class: A' columns j*Kc + 64*b .., B's class-j rows 64*b .. at shifted columns 56*nb ..
                    for (int j = 0; ok && j < 8; ++j)
                        for (int kb = kb0; kb < kb1; ++kb) {
                            ok = __all_sync(REQ_MASK, ptx::mbar_wait(empty_bar + 8u * stage, phase ^ 1u, abort_flag));
                            if (!ok) break;
                            const uint32_t sA = smem_base + (uint32_t)stage * STAGE_BYTES;
                            if (lane == 0) ptx::mbar_arrive_expect_tx(full_bar + 8u * stage, (uint32_t)(p.a_tx_bytes + p.b_tx_bytes));
                            __syncwarp(REQ_MASK);
                            if (is_a) load(sA, tmA, full_bar + 8u * stage, j * p.cls_kc + kb * kUmmaBK, row0);
                            else load(sA + A_BYTES, &maps.b[B_CLS ? j : 0], full_bar + 8u * stage, col0, kb * kUmmaBK);
                            if (++stage == S) { stage = 0; phase ^= 1u; }
                        }
                }
                // ShuffleK: the unit's k-blocks in rotated order (the MMA warp consumes the stages in ring order and sums
                // whatever arrives, so only the loads know; the order is a function of the tile, hence fixed)
                const int kb_rot = (MODE == 0 && !SK && p.shuffle_k && kb1 - kb0 > 1) ? ((mb + nb) * 5) % (kb1 - kb0) : 0;
                for (int kbi = kb0; !B_CLS && kbi < kb1; ++kbi) {
                    const int kb = (MODE == 0 && !SK) ? kb0 + (kbi - kb0 + kb_rot) % (kb1 - kb0) : kbi;
                    ok = __all_sync(REQ_MASK, ptx::mbar_wait(empty_bar + 8u * stage, phase ^ 1u, abort_flag));
                    if (!ok) break;
                    const uint32_t sA = smem_base + (uint32_t)stage * STAGE_BYTES;
                    const uint32_t sB = sA + A_BYTES;
                    const uint32_t fb = full_target + 8u * stage;
                    if (lane == 0) {
                        if (CG == 1) ptx::mbar_arrive_expect_tx(full_bar + 8u * stage, (uint32_t)(p.a_tx_bytes + p.b_tx_bytes));
                        else if (A_CLS && kb == 0 && kshift > 0) {
                            // pair tiles of one row class, a unit's first k-block with row heads to zero: each CTA's A box
                            // reports to its own barrier (its warp 1 zeroes the heads there before the MMA); the B boxes of
                            // both CTAs report to the leader's as always
                            ptx::mbar_arrive_expect_tx(afull_bar + 8u * stage, (uint32_t)A_BYTES);
                            if (leader) ptx::mbar_arrive_expect_tx(full_bar + 8u * stage, (uint32_t)(2 * p.b_tx_bytes));
                        }
                        else if (leader) ptx::mbar_arrive_expect_tx(full_bar + 8u * stage, (uint32_t)(2 * (A_BYTES + p.b_tx_bytes)));
                    }
                    __syncwarp(REQ_MASK);
                    const int k0 = kb * kUmmaBK;
                    // this lane's request: where it lands, through which map, at which coordinates
                    uint32_t dst;
                    const CUtensorMap* tm;
                    int x, y;
                    if (is_a) {
                        tm = tmA;
                        if (!A_MN) { dst = sA; x = k0 + a_k_off; y = row0; }
                        else { dst = sA + (uint32_t)lane * 8192u; x = row0 + lane * 64; y = k0; }
                    } else {
                        tm = tmB;
                        if (B_MN) { dst = sB + (uint32_t)jb * 8192u; x = col0 + jb * 64; y = k0 - kshift; }
                        else { dst = sB; x = k0; y = col0; }
                    }
                    if (A_CLS && CG == 2 && is_a && kb == 0 && kshift > 0) load(dst, tm, afull_own + 8u * stage, x, y);   // this CTA's own barrier
                    else load(dst, tm, fb, x, y);
                    if (++stage == S) { stage = 0; phase ^= 1u; }
                }
                if (lane == 0) ADAPT_TRACE(1, unit);
            }
        }
    } else if (warp == 1) {
        // ------------------------------ MMA issuer ---------------------------------------------
        // one thread issues the MMAs; in class mode the whole warp runs the loop so that its other
        // lanes can zero the stale leading elements of A' in the first k-block
        // (only when some class of A is shifted: with K % 8 == 0 every sigma is zero and one lane is enough)
        // (pair tiles of one row class: always, and the peer's warp 1 runs the forwarding loop further down)
        const bool warp_wide = A_CLS && (p.a_shift_any != 0 || CG == 2);
        // in class mode all 32 lanes run these loops: lane 0 waits and the outcome is broadcast, so
        // the lanes never part ways before a __syncwarp
        auto mma_wait = [&](uint32_t bar, uint32_t parity) -> bool {
            if (!warp_wide) return ptx::mbar_wait(bar, parity, abort_flag);
            int w = 1;
            if (lane == 0) w = ptx::mbar_wait(bar, parity, abort_flag) ? 1 : 0;
            return __shfl_sync(0xffffffffu, w, 0) != 0;
        };
        // Class tile whose rows are shifted: the sigma elements in front of each row of the first k-block belong to
        // the previous row of A and are zeroed before the tensor core reads them.  Rows lane, lane+32, ...: chunk 0
        // of row r (its first 8 elements) sits at r*128 + ((r & 7) << 4); one masked 16-byte read-modify-write per row.
        auto zero_row_heads = [&](int stage, int sigma) {
            uint8_t* genA = gen_base + (size_t)stage * STAGE_BYTES;
            uint32_t keep[4];
#pragma unroll
            for (int w = 0; w < 4; ++w)
                keep[w] = (2 * w >= sigma ? 0x0000ffffu : 0u) | (2 * w + 1 >= sigma ? 0xffff0000u : 0u);
            uint4 v[4];
#pragma unroll
            for (int t = 0; t < 4; ++t) {
                const int r = lane + 32 * t;
                if (r * 128 < A_BYTES) v[t] = *reinterpret_cast<const uint4*>(genA + r * 128 + ((r & 7) << 4));
            }
#pragma unroll
            for (int t = 0; t < 4; ++t) {
                const int r = lane + 32 * t;
                if (r * 128 < A_BYTES)               // rows past the box are not part of the stage
                    *reinterpret_cast<uint4*>(genA + r * 128 + ((r & 7) << 4)) =
                        make_uint4(v[t].x & keep[0], v[t].y & keep[1], v[t].z & keep[2], v[t].w & keep[3]);
            }
            ptx::fence_proxy_async_smem();
            __syncwarp();
        };
        if (A_CLS && CG == 2 && !leader) {
            // Pair tiles of one row class, the peer CTA: the A box of a unit's first k-block reports to this CTA's own
            // barrier when its rows have stale heads; this warp zeroes them and then tells the leader that the peer's half
            // of A is ready for the MMA the leader issues for both.  Every other k-block signals the leader directly.
            int stage = 0;
            uint32_t aphase = 0;              // per stage: parity of the next use of its A barriers (used by some units only)
            bool ok = true;
            for (int it = 0; ok; ++it) {
                WorkItem w;
                if (!next_item<SK, B_SPLIT>(p, unit0, unit_step, it, w)) break;
                const int sigma = p.a_sigma[w.mb & (NCLS - 1)];
                if (w.kb0 == 0 && w.kb1 > 0 && sigma > 0) {
                    if (!mma_wait(afull_bar + 8u * stage, (aphase >> stage) & 1u)) { ok = false; break; }
                    zero_row_heads(stage, sigma);
                    if (lane == 0) ptx::mbar_arrive_cluster(aready_bar + 8u * stage, 0);
                    aphase ^= 1u << stage;
                }
                stage = (stage + (w.kb1 - w.kb0)) % S;
            }
        }
        if ((lane == 0 || warp_wide) && leader) {
            int stage = 0;
            uint32_t phase = 0;
            uint32_t aphase = 0;              // pair tiles of one row class: per stage, parity of the next use of its A barriers
            int buf = 0;
            uint32_t buf_phase = 0;
            // K-major operand: rows of 128 B, 8-row groups 1024 B apart, +32 B per 16-element k step.
            // MN-major operand: 64-element blocks along M/N 8192 B apart (LBO), 8-row k groups
            // 1024 B apart (SBO), +2048 B per 16-element k step.
            const uint32_t a_lbo = A_MN ? 8192u : 16u, b_lbo = B_MN ? 8192u : 16u;
            const uint32_t a_kstep = A_MN ? 2048u : 32u, b_kstep = B_MN ? 2048u : 32u;
            bool ok = true;
            for (int it = 0; ok; ++it) {
                WorkItem w;
                if (!next_item<SK, B_SPLIT>(p, unit0, unit_step, it, w)) break;
                const int unit = w.unit, mb = w.mb, nb = w.nb, split = w.split, kb0 = w.kb0, kb1 = w.kb1;
                (void)unit; (void)nb; (void)split;
                if (warp_wide && kb0 == 0 && kb1 > 0) {
                    // Done here, before the wait for a free accumulator: the loads run ahead of the drain, so
                    // in the write-bound regime this work hides behind that wait.
                    const int sigma = p.a_sigma[mb & (NCLS - 1)];
                    if (sigma > 0) {
                        if (!mma_wait((A_CLS && CG == 2) ? afull_bar + 8u * stage : full_bar + 8u * stage,
                                      (A_CLS && CG == 2) ? ((aphase >> stage) & 1u) : phase)) { ok = false; break; }
                        zero_row_heads(stage, sigma);
                    }
                }
                if (!mma_wait(tempty_bar + 8u * buf, buf_phase ^ 1u)) { ok = false; break; }
                ptx::tc_fence_after();
                ADAPT_TRACE(2, unit);
                const uint32_t d_tmem = tmem_base + (uint32_t)(buf * BN);
                if (B_CLS) {
                    for (int j = 0; ok && j < 8; ++j)
                        for (int kb = kb0; kb < kb1; ++kb) {
                            if (!mma_wait(full_bar + 8u * stage, phase)) { ok = false; break; }
                            ptx::tc_fence_after();
                            const uint32_t sA = smem_base + (uint32_t)stage * STAGE_BYTES;
                            const uint32_t sB = sA + A_BYTES;
#pragma unroll
                            for (int k16 = 0; k16 < kUmmaBK / 16; ++k16) {
                                const uint64_t adesc = ptx::smem_desc_sw128(sA + k16 * a_kstep, a_lbo, 1024u);
                                const uint64_t bdesc = ptx::smem_desc_sw128(sB + k16 * b_kstep, b_lbo, 1024u);
                                ptx::umma_f16<CG>(tmem_base + 64u * j, adesc, bdesc, p.idesc, (kb > kb0 || k16 > 0) ? 1u : 0u);
                            }
                            ptx::umma_commit_1(empty_bar + 8u * stage);
                            if (++stage == S) { stage = 0; phase ^= 1u; }
                        }
                }
                if (!B_CLS) {
                    // The k-block loop proper runs in ONE lane, also when the warp came here together (class tiles): a
                    // warp-wide loop pays a shuffle for every wait, and the MMA thread's loop is what the tensor core waits
                    // for (pair tiles of one row class: 0.82 us per k-block with the warp-wide loop).  The other lanes step
                    // their copy of (stage, phase) by the number of k-blocks and pick up the outcome afterwards.
                    int done = 1;
                    if (lane == 0) {
                        int st = stage;
                        uint32_t ph = phase;
                        for (int kb = kb0; kb < kb1; ++kb) {
                            if (A_CLS && CG == 2 && kb == 0 && p.a_sigma[mb & (NCLS - 1)] > 0) {
                                // the unit's first k-block, row heads zeroed: this CTA's box (waited for above) and the peer's,
                                // handed over by the peer's warp 1.  The leader reads none of the peer's shared memory itself
                                // (the peer's tensor core does, after the peer's own proxy fence), so an ordinary wait is enough.
                                if (!ptx::mbar_wait(aready_bar + 8u * st, (aphase >> st) & 1u, abort_flag)) { done = 0; break; }
                            }
                            if (!ptx::mbar_wait(full_bar + 8u * st, ph, abort_flag)) { done = 0; break; }
                            ptx::tc_fence_after();
                            const uint32_t sA = smem_base + (uint32_t)st * STAGE_BYTES;
                            const uint32_t sB = sA + A_BYTES;
#pragma unroll
                            for (int k16 = 0; k16 < kUmmaBK / 16; ++k16) {
                                const uint64_t adesc = ptx::smem_desc_sw128(sA + k16 * a_kstep, a_lbo, 1024u);
                                const uint64_t bdesc = ptx::smem_desc_sw128(sB + k16 * b_kstep, b_lbo, 1024u);
                                ptx::umma_f16<CG>(d_tmem, adesc, bdesc, p.idesc, (kb > kb0 || k16 > 0) ? 1u : 0u);
                            }
                            // free the stage (in both CTAs of a pair) once these MMAs have read it
                            if (CG == 1) ptx::umma_commit_1(empty_bar + 8u * st);
                            else ptx::umma_commit_2(empty_bar + 8u * st);
                            if (++st == S) { st = 0; ph ^= 1u; }
                        }
                    }
                    if (warp_wide) done = __shfl_sync(0xffffffffu, done, 0);
                    if (!done) { ok = false; break; }
                    if (A_CLS && CG == 2 && kb0 == 0 && kb1 > 0 && p.a_sigma[mb & (NCLS - 1)] > 0) aphase ^= 1u << stage;
                    const int adv = stage + (kb1 - kb0);
                    phase ^= (uint32_t)((adv / S) & 1);
                    stage = adv % S;
                }
                if (!ok) break;
                if (lane == 0) {
                    if (CG == 1) ptx::umma_commit_1(tfull_bar + 8u * buf);
                    else ptx::umma_commit_2(tfull_bar + 8u * buf);
                }
                ADAPT_TRACE(3, unit);
                if (++buf == NBUF) { buf = 0; buf_phase ^= 1u; }
            }
        }
    } else {
        // ------------------------------ epilogue -----------------------------------------------
        // Eight warps: warp w may read TMEM lanes 32*(w % 4) .. +31 only, so two warps share each lane
        // quarter and take alternate 64-column passes (alternate tiles when a tile is one pass wide).
        const int q = warp & 3;
        const int half = (warp - 2) >> 2;
        int buf = 0;
        uint32_t buf_phase = 0;
        int seq = 0;                                         // tiles this CTA has processed so far
        int tma_box = 0;                                     // TMA-store boxes this warp has issued so far
        const uint64_t c_policy = ptx::l2_policy_evict_first();
        // partials that fit in L2 are kept there for the reduction kernel (evict-last)
        const uint64_t part_policy = ptx::l2_policy_evict_last();
        auto store_partial8 = [&](float* dst, const uint32_t* r8x) {
            if (p.part_hint) ptx::st_global_v8_hint(dst, r8x, part_policy);
            else ptx::st_global_v8(dst, r8x);
        };
        bool ok = true;
        uint8_t* stg = stage_out + (warp - 2) * kUmmaWarpStagingBytes + lane * kUmmaStageRowBytes;   // this thread's staging row
        unsigned short* srow = reinterpret_cast<unsigned short*>(stg);
        const uintptr_t c_base = reinterpret_cast<uintptr_t>(p.C);
        for (int it = 0; ok; ++it, ++seq) {
            WorkItem w;
            if (!next_item<SK, B_SPLIT>(p, unit0, unit_step, it, w)) break;
            const int unit = w.unit, mb = w.mb, nb = w.nb, split = w.split;
            (void)unit;
            if (!ptx::mbar_wait(tfull_bar + 8u * buf, buf_phase, abort_flag)) { ok = false; break; }
            ptx::tc_fence_after();
            if (warp == 2 && lane == 0) ADAPT_TRACE(4, unit);
            // row of C held by TMEM lane i of this CTA: consecutive rows, or every 8th row of one class
            const int row_step = A_CLS ? NCLS : 1;
            const int row_base = A_CLS ? (mb >> NSH) * (128 * CG * NCLS) + (mb & (NCLS - 1)) + NCLS * 128 * (int)cta_rank
                                       : mb * (128 * CG) + (int)cta_rank * 128;
            const int row = row_base + row_step * (q * 32 + lane);
            const int n0 = nb * TILE_N;
            const uint32_t t_row = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(buf * BN);
            // k-class mode: columns [8c, 8c+8) of the tile = sum over the class buffers j (ascending), buffer j
            // read sigma_j columns to the right
            auto class_sum8 = [&](int c, uint32_t* out8) {
                uint32_t v[8][8];
#pragma unroll
                for (int j = 0; j < 8; ++j) ptx::tmem_ld_32x8(t_row + (uint32_t)(64 * j + p.b_sigma[j] + 8 * c), v[j]);
                ptx::tmem_ld_wait();
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    float acc = __uint_as_float(v[0][i]);
#pragma unroll
                    for (int j = 1; j < 8; ++j) acc += __uint_as_float(v[j][i]);
                    out8[i] = __float_as_uint(acc);
                }
            };
            const bool row_ok = row < p.M;
            bool released = false;
            auto release_accumulator = [&]() {
                ptx::tc_fence_before();
                __syncwarp();
                if (lane == 0) {
                    if (CG == 1) ptx::mbar_arrive(tempty_bar + 8u * buf);
                    else ptx::mbar_arrive_cluster(tempty_bar + 8u * buf, 0);
                    if (warp == 2) ADAPT_TRACE(7, unit);
                }
            };
            // stream-K: the fp32 partial tiles live in the workspace, one per CTA, [128][BN]; the flag word of a CTA holds
            // the epoch of the launch whose partial is complete there
            const int sk_cta = (int)unit0 * CG + (int)cta_rank;
            if (SK && w.kind == 2 && (seq & 1) == half) {
                // the slots after this one computed the rest of this tile's k range first thing: wait for their partials
                bool arrived = true;
                if (lane == 0) {
                    for (int j = 1; j <= w.npeers && arrived; ++j) {
                        const unsigned int* f = p.sk_flags + (sk_cta + j * CG);
                        uint32_t spins = 0;
                        uint64_t t0 = 0;
                        for (;;) {
                            unsigned int v;
                            asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(f) : "memory");
                            if (v == p.sk_epoch) break;
                            if ((++spins & 0x3f) == 0) {
                                if (*abort_flag) { arrived = false; break; }
                                const uint64_t now = ptx::globaltimer_ns();
                                if (t0 == 0) t0 = now;
                                else if (now - t0 > ptx::kWaitLimitNs) { *abort_flag = 1; arrived = false; break; }
                            }
                        }
                    }
                }
                arrived = __shfl_sync(0xffffffffu, arrived ? 1 : 0, 0) != 0;
                if (!arrived) { ok = false; break; }
            }
            // adds the peers' partial values of this thread's row, columns [col, col + 32), in ascending k order
            auto sk_fixup = [&](uint32_t (&r)[32], int col) {
                for (int j = 1; j <= w.npeers; ++j) {
                    // partial tiles are stored [32-column chunk][8-column group][row][8]: a warp's access is 1 KB contiguous
                    const float4* src = reinterpret_cast<const float4*>(
                        p.sk_partial + (size_t)(sk_cta + j * CG) * 128 * BN + ((size_t)(col >> 3) * 128 + (size_t)(q * 32 + lane)) * 8);
#pragma unroll
                    for (int v = 0; v < 8; ++v) {
                        const float4 x = __ldcg(src + (v >> 1) * 256 + (v & 1));
                        r[4 * v + 0] = __float_as_uint(__uint_as_float(r[4 * v + 0]) + x.x);
                        r[4 * v + 1] = __float_as_uint(__uint_as_float(r[4 * v + 1]) + x.y);
                        r[4 * v + 2] = __float_as_uint(__uint_as_float(r[4 * v + 2]) + x.z);
                        r[4 * v + 3] = __float_as_uint(__uint_as_float(r[4 * v + 3]) + x.w);
                    }
                }
            };
            if (SK && w.kind == 1) {
                // ---- stream-K: a k range that is not the tile's first: fp32 partial to the workspace, then the flag ----
                float* mine = p.sk_partial + (size_t)sk_cta * 128 * BN + (size_t)(q * 32 + lane) * 8;
#pragma unroll 1
                for (int c0 = 0; c0 < BN; c0 += 32) {
                    if (n0 + c0 >= p.N) break;                           // uniform; the owner of the tile skips these too
                    if (((seq * (BN / 32) + (c0 >> 5)) & 1) != half) continue;
                    uint32_t r[32];
                    ptx::tmem_ld_32x32(t_row + (uint32_t)c0, r);
                    ptx::tmem_ld_wait();
#pragma unroll
                    for (int v = 0; v < 4; ++v) store_partial8(mine + (size_t)((c0 >> 3) + v) * 128 * 8, r + 8 * v);
                }
                release_accumulator();
                released = true;
                if (warp == 2 && lane == 0) ADAPT_TRACE(5, unit);
                // every warp fences its stores and counts itself in; the last one publishes the flag
                __threadfence();
                __syncwarp();
                if (warp == 2 && lane == 0) ADAPT_TRACE(9, unit);
                if (lane == 0) {
                    const int old = atomicAdd(sk_count, 1);
                    if ((old & (kUmmaEpilogueWarps - 1)) == kUmmaEpilogueWarps - 1) {
                        __threadfence();
                        asm volatile("st.release.gpu.global.u32 [%0], %1;" ::"l"(p.sk_flags + sk_cta), "r"(p.sk_epoch) : "memory");
                    }
                }
            } else if constexpr (FUSE) {
                // ---- fused split-K: partial -> own shared memory -> sum over the cluster's ranks -> C ----
                const uint32_t xphase = (uint32_t)(seq & 1);
                const uint32_t my_rank = ptx::cluster_ctarank();
                float* X = reinterpret_cast<float*>(stage_out);
                // every rank has finished reading the partial this CTA wrote for its previous tile
                if (!ptx::mbar_wait_cluster(xempty_bar, xphase ^ 1u, abort_flag)) { ok = false; break; }
                const int r_in_tile = q * 32 + lane;
                const int sig = B_SPLIT ? p.b_sigma[split & 7] : 0;      // k classes as splits: the tile's columns sit sigma to the right
#pragma unroll 1
                for (int c0 = 0; c0 < TILE_N; c0 += 32) {
                    if (n0 + c0 >= p.N) break;                           // uniform across the warp
                    if (((seq * ((TILE_N + 31) / 32) + (c0 >> 5)) & 1) != half) continue;
                    uint32_t r[32];
                    if (c0 + 32 <= TILE_N) {
                        ptx::tmem_ld_32x32(t_row + (uint32_t)(sig + c0), r);
                    } else {                                             // 24 columns (k-class tiles own BN - 8): stay inside the accumulator
                        uint32_t r8a[8], r8b[8], r8c[8];
                        ptx::tmem_ld_32x8(t_row + (uint32_t)(sig + c0), r8a);
                        ptx::tmem_ld_32x8(t_row + (uint32_t)(sig + c0 + 8), r8b);
                        ptx::tmem_ld_32x8(t_row + (uint32_t)(sig + c0 + 16), r8c);
#pragma unroll
                        for (int i = 0; i < 8; ++i) { r[i] = r8a[i]; r[8 + i] = r8b[i]; r[16 + i] = r8c[i]; r[24 + i] = 0u; }
                    }
                    ptx::tmem_ld_wait();
                    if (r_in_tile < p.x_rows) {
                        float4* dst = reinterpret_cast<float4*>(X + (size_t)r_in_tile * p.x_pitch + c0);
#pragma unroll
                        for (int v = 0; v < 8; ++v)
                            dst[v] = make_float4(__uint_as_float(r[4 * v]), __uint_as_float(r[4 * v + 1]),
                                                 __uint_as_float(r[4 * v + 2]), __uint_as_float(r[4 * v + 3]));
                    }
                }
                release_accumulator();
                released = true;
                // this warp's share of the partial is written: tell every rank (release at cluster scope), one lane per rank:
                // an arrive on another CTA's barrier occupies its thread for the better part of a microsecond, so a single
                // lane walking the ranks serialised P_k of them (pair tiles hit the same wall: 0.8 us per k-block)
                __syncwarp();
                if (lane < p.P_k) ptx::mbar_arrive_cluster(xfull_bar, (uint32_t)lane);
                if (!ptx::mbar_wait_cluster(xfull_bar, xphase, abort_flag)) { ok = false; break; }
                // rows and 4-column groups of this tile that exist; rank r takes the r-th share of them
                const int rows_here = A_CLS ? min(128, (p.M - row_base + row_step - 1) / row_step) : min(128, p.M - row_base);
                const int tile_cols = min(TILE_N, p.N - n0);
                const int groups = (tile_cols + 3) >> 2;
                const int total = rows_here * groups;
                const int per = (total + p.P_k - 1) / p.P_k;
                const int e_end = min(total, ((int)my_rank + 1) * per);
                const uint32_t x_addr = ptx::smem_u32(X);
                unsigned short* c16 = reinterpret_cast<unsigned short*>(p.C);
                for (int e = (int)my_rank * per + (warp - 2) * 32 + lane; e < e_end; e += kUmmaEpilogueWarps * 32) {
                    const int rr = e / groups, g = e - rr * groups;
                    const uint32_t a = x_addr + (uint32_t)((rr * p.x_pitch + 4 * g) * 4);
                    float4 sum = ptx::ld_cluster_f4(a, 0u);
                    for (int rk = 1; rk < p.P_k; ++rk) {
                        const float4 v = ptx::ld_cluster_f4(a, (uint32_t)rk);
                        sum.x += v.x; sum.y += v.y; sum.z += v.z; sum.w += v.w;
                    }
                    const int n = n0 + 4 * g;
                    unsigned short* dst = c16 + (size_t)(row_base + row_step * rr) * p.N + n;
                    if (n + 4 <= p.N && (reinterpret_cast<uintptr_t>(dst) & 7) == 0) {
                        *reinterpret_cast<uint2*>(dst) = make_uint2(pack16(sum.x, sum.y, p.dtype), pack16(sum.z, sum.w, p.dtype));
                    } else {
                        const float o[4] = {sum.x, sum.y, sum.z, sum.w};
#pragma unroll
                        for (int j = 0; j < 4; ++j)
                            if (n + j < p.N) dst[j] = cast16(o[j], p.dtype);
                    }
                }
                // done reading every rank's partial: each may overwrite it for its next tile
                __syncwarp();
                if (lane < p.P_k) ptx::mbar_arrive_cluster(xempty_bar, (uint32_t)lane);
            } else if (p.P_k == 1 && !p.force_partial) {
                // 16-bit output, any N and any base alignment.  A thread converts 64 columns of its row
                // and stages them in shared memory shifted by the row's misalignment in C, so that
                // 16-byte aligned chunks of a staged row are 16-byte aligned chunks of C.  The warp then
                // writes its 32 row segments cooperatively, consecutive lanes taking consecutive chunks
                // of a row (aligned 16-byte stores, about 3.5 rows per instruction); the at most 7 + 7
                // elements at a segment's ends are 2-byte stores by the row's own thread.
                const int rowq0 = row - row_step * lane;             // first row of this warp's quarter
                const uintptr_t g_tile = c_base + 2ull * ((size_t)rowq0 * p.N + n0);
                const uintptr_t row_bytes = 2ull * (uintptr_t)p.N * row_step;   // distance between this warp's rows
                // the two warps of a lane quarter take alternate tiles, so one thread sees all passes of
                // its row and can carry the ragged tail of a pass into the head of the next one
                if (!B_CLS && p.c_mode != 0) {
                    // C through TMA stores.  A warp stages 32 rows x 64 elements as one 128B-swizzled box (row r
                    // at r * 128, its 16-byte chunk c at position c ^ (r & 7): conflict-free 16-byte shared
                    // stores) and one lane hands the box to TMA, which clips rows >= M and the end of the row.
                    // Two boxes per warp alternate, so converting a pass overlaps the store of the one before.
                    // The boxes must cover whole 32-byte sectors of C: rows that start 16 bytes off a sector
                    // boundary halve the store rate, and TMA clips a row's end in 16-byte units, not elements.
                    //
                    // Rows on 32-byte boundaries (N % 16 == 0): boxes at columns n0 + 64 * pass of the plain map
                    // (or of the class map, whose rows are every 8th row of C).
                    // HALO (tiles of one of 16 row classes): all rows of the tile start sigma elements after a
                    // 32-byte boundary, and the class map addresses them by x = n + sigma.  The tile owns the
                    // units x in [16 + TILE_N * nb, 16 + TILE_N * (nb + 1)); it has computed columns
                    // n >= TILE_N * nb, so element x sits in accumulator column x - sigma - TILE_N * nb
                    // = (x - x_first) + 16 - sigma.  The first 16 - sigma elements of a row (x < 16) share their
                    // unit with the previous row of C, the last (N + sigma) % 16 with the next one: the row's own
                    // thread writes both with aligned stores of 2 to 16 bytes (head: tile nb = 0; tail: the tile that owns the unit).
                    if (A_CLS && (seq & 1) != half && lane == 0 && unit + unit_step < p.num_units) {
                        // the other warp of the quarter stores this tile; this one stores the next: fetch its map's descriptor now
                        int mb2, nb2, sp2;
                        decode_unit(p, unit + unit_step, mb2, nb2, sp2);
                        ptx::prefetch_tensormap(&maps.c[mb2 & (NCLS - 1)]);
                    }
                    if ((seq & 1) == half) {
                        const int cls = A_CLS ? (mb & (NCLS - 1)) : 0;
                        const int sig = HALO ? p.c_sigma[cls] : 0;
                        const int off = HALO ? 16 - sig : 0;
                        const int y0 = A_CLS ? (mb >> NSH) * (128 * CG) + (int)cta_rank * 128 + q * 32 : row_base + q * 32;
                        const CUtensorMap* tmC = &maps.c[cls];
                        uint8_t* wbuf = stage_out + (warp - 2) * kUmmaWarpStagingBytes;
                        const int x_first = n0 + (HALO ? 16 : 0);
                        const int x_end = HALO ? p.c_extent[cls] : p.N;  // end of the row's whole units
                        if (HALO) {
                            unsigned short* crow = reinterpret_cast<unsigned short*>(c_base) + (size_t)row * p.N;
                            const int tail = (p.N + sig) - x_end;        // elements after the last whole unit
                            const bool has_tail = x_end >= x_first && x_end < x_first + TILE_N && tail > 0;
#pragma unroll
                            for (int part = 0; part < 2; ++part) {       // 0: head of the row, 1: its tail (both uniform)
                                if (part == 0 ? nb != 0 : !has_tail) continue;
                                const int col = part == 0 ? 0 : off + (x_end - x_first);   // accumulator column
                                const int n_first = part == 0 ? 0 : x_end - sig;
                                const int count = part == 0 ? min(off, p.N) : tail;
                                uint32_t e0[8], e1[8];
                                ptx::tmem_ld_32x8(t_row + (uint32_t)col, e0);
                                ptx::tmem_ld_32x8(t_row + (uint32_t)(col + 8), e1);
                                ptx::tmem_ld_wait();
                                if (row_ok) store_run16(crow + n_first, count, e0, e1, p.dtype);
                            }
                        }
#pragma unroll 1
                        for (int pass = 0; pass < PASSES; ++pass) {
                            const int x = x_first + 64 * pass;
                            if (x >= x_end) break;                       // uniform across the warp
                            const int ncols = min(64, x_end - x);
                            uint8_t* box = wbuf + (tma_box & 1) * 4096;
                            uint8_t* brow = box + lane * 128;
#pragma unroll
                            for (int h = 0; h < 2; ++h) {
                                if (32 * h >= ncols) break;              // uniform; those elements lie beyond the row and are clipped
                                uint32_t r[32];
                                ptx::tmem_ld_32x32(t_row + (uint32_t)(off + 64 * pass + 32 * h), r);
                                ptx::tmem_ld_wait();
                                if (SK && w.kind == 2) sk_fixup(r, 64 * pass + 32 * h);
                                if ((pass == PASSES - 1 || x + 64 >= x_end) && (h == 1 || ncols <= 32)) {
                                    // the tile's last read of the accumulator: hand the buffer back now, so the MMA
                                    // of the tile after next starts while this pass is still being packed and stored
                                    release_accumulator();
                                    released = true;
                                }
                                if (h == 0) {
                                    if (warp == 2 && lane == 0) ADAPT_TRACE(5, unit);
                                    if (lane == 0) ptx::bulk_wait_read<1>();   // the store that last used this box has read it
                                    __syncwarp();
                                    if (warp == 2 && lane == 0) ADAPT_TRACE(8, unit);
                                }
#pragma unroll
                                for (int c = 0; c < 4; ++c) {
                                    uint4 v;
                                    v.x = pack16(__uint_as_float(r[8 * c + 0]), __uint_as_float(r[8 * c + 1]), p.dtype);
                                    v.y = pack16(__uint_as_float(r[8 * c + 2]), __uint_as_float(r[8 * c + 3]), p.dtype);
                                    v.z = pack16(__uint_as_float(r[8 * c + 4]), __uint_as_float(r[8 * c + 5]), p.dtype);
                                    v.w = pack16(__uint_as_float(r[8 * c + 6]), __uint_as_float(r[8 * c + 7]), p.dtype);
                                    *reinterpret_cast<uint4*>(brow + (((4 * h + c) ^ (lane & 7)) << 4)) = v;
                                }
                            }
                            ptx::fence_proxy_async_smem();
                            __syncwarp();
                            if (lane == 0) {
                                if (p.c_hint) ptx::tma_store_2d_hint(tmC, ptx::smem_u32(box), x, y0, c_policy);
                                else ptx::tma_store_2d(tmC, ptx::smem_u32(box), x, y0);
                                ptx::bulk_commit();
                                if (warp == 2) ADAPT_TRACE(6, unit);
                            }
                            ++tma_box;
                        }
                    }
                } else if (B_CLS ? half == 0 : (seq & 1) == half) {
                    const uintptr_t g_row = g_tile + (uintptr_t)lane * row_bytes;   // this thread's row, column n0
                    const int m_r = (int)((g_row & 15u) >> 1);           // the same in every pass: a pass is 128 bytes
                    const int tile_cols = min(TILE_N, p.N - n0);
#pragma unroll 1
                    for (int pass = 0; pass < PASSES; ++pass) {
                        const int c0 = pass * 64;
                        if (c0 >= tile_cols) break;                      // uniform across the warp
                        const int ncols = min(64, tile_cols - c0);
                        const bool last = c0 + 64 >= tile_cols;
                        uint32_t r0[32], r1[32];
                        if (B_CLS) {
#pragma unroll
                            for (int c = 0; c < 4; ++c) class_sum8(c, r0 + 8 * c);
#pragma unroll
                            for (int c = 4; c < 7; ++c) class_sum8(c, r1 + 8 * (c - 4));
#pragma unroll
                            for (int i = 24; i < 32; ++i) r1[i] = 0;
                        } else {
                            ptx::tmem_ld_32x32(t_row + (uint32_t)c0, r0);
                            if (ncols > 32) ptx::tmem_ld_32x32(t_row + (uint32_t)(c0 + 32), r1);   // uniform
                            ptx::tmem_ld_wait();
                            if (SK && w.kind == 2) {
                                sk_fixup(r0, c0);
                                if (ncols > 32) sk_fixup(r1, c0 + 32);
                            }
                        }
                        if (warp == 2 && lane == 0) ADAPT_TRACE(5, unit);
                        __syncwarp();                                    // the previous pass has been written out
                        // carry: elements 64..71 of the previous pass become elements 0..7 of this one
                        if (pass > 0) *reinterpret_cast<uint4*>(srow) = *reinterpret_cast<const uint4*>(srow + 64);
                        if ((m_r & 1) == 0) {
                            uint32_t* d = reinterpret_cast<uint32_t*>(srow + m_r);
#pragma unroll
                            for (int i = 0; i < 16; ++i)
                                d[i] = pack16(__uint_as_float(r0[2 * i]), __uint_as_float(r0[2 * i + 1]), p.dtype);
                            if (ncols > 32) {
#pragma unroll
                                for (int i = 0; i < 16; ++i)
                                    d[16 + i] = pack16(__uint_as_float(r1[2 * i]), __uint_as_float(r1[2 * i + 1]), p.dtype);
                            }
                        } else {
                            srow[m_r] = cast16(__uint_as_float(r0[0]), p.dtype);
                            uint32_t* d = reinterpret_cast<uint32_t*>(srow + m_r + 1);
#pragma unroll
                            for (int i = 0; i < 15; ++i)
                                d[i] = pack16(__uint_as_float(r0[2 * i + 1]), __uint_as_float(r0[2 * i + 2]), p.dtype);
                            if (ncols > 32) {
                                d[15] = pack16(__uint_as_float(r0[31]), __uint_as_float(r1[0]), p.dtype);
#pragma unroll
                                for (int i = 0; i < 15; ++i)
                                    d[16 + i] = pack16(__uint_as_float(r1[2 * i + 1]), __uint_as_float(r1[2 * i + 2]), p.dtype);
                                srow[m_r + 63] = cast16(__uint_as_float(r1[31]), p.dtype);
                            } else {
                                srow[m_r + 31] = cast16(__uint_as_float(r0[31]), p.dtype);
                            }
                        }
                        if (warp == 2 && lane == 0) ADAPT_TRACE(9, unit);
                        // staged row now holds valid elements [lo_valid, end): the carried tail makes the
                        // head whole in every pass but the first
                        const int lo_valid = pass == 0 ? m_r : 0;
                        const int end = m_r + ncols;
                        const uintptr_t g0 = g_row + 2u * c0;            // address of staged element m_r
                        if (row_ok) {                                    // ragged ends of this thread's own row
                            unsigned short* grow = reinterpret_cast<unsigned short*>(g0 - 2 * m_r);   // 16-byte aligned
                            if (lo_valid) {
#pragma unroll
                                for (int i = 0; i < 7; ++i)
                                    if (lo_valid + i < min(8, end)) grow[lo_valid + i] = srow[lo_valid + i];
                            }
                            if (last && (end & 7)) {
                                const int tail_begin = max(end & ~7, lo_valid ? min(8, end) : 0);
#pragma unroll
                                for (int i = 0; i < 7; ++i)
                                    if (tail_begin + i < end) grow[tail_begin + i] = srow[tail_begin + i];
                            }
                        }
                        __syncwarp();                                    // every row of the warp is staged
                        // 32 rows x 9 aligned chunks: lane + 32*it = 9*rr + qc
                        int rr = lane / 9, qc = lane - 9 * rr;
                        const uint8_t* stg_warp = stage_out + (warp - 2) * kUmmaWarpStagingBytes;
                        const uintptr_t g_pass = g_tile + 2u * c0;
#pragma unroll
                        for (int it = 0; it < 9; ++it) {
                            const uintptr_t g = g_pass + (uintptr_t)rr * row_bytes;
                            const int m = (int)((g & 15u) >> 1);
                            const int lo_v = pass == 0 ? m : 0;
                            if (rowq0 + row_step * rr < p.M && 8 * qc >= lo_v && 8 * qc + 8 <= m + ncols)
                                *reinterpret_cast<uint4*>(g - 2 * m + 16 * qc) =
                                    *reinterpret_cast<const uint4*>(stg_warp + rr * kUmmaStageRowBytes + 16 * qc);
                            rr += 3; qc += 5;
                            if (qc >= 9) { qc -= 9; rr += 1; }
                        }
                        if (warp == 2 && lane == 0) ADAPT_TRACE(6, unit);
                    }
                }
            } else {
                // fp32 partial tile: rows of the workspace are 32-byte aligned (pitch Np), so a thread
                // writes its row's 32 columns as four aligned 32-byte stores (whole sectors)
                if (B_CLS) {
                    if (half == 0) {
#pragma unroll 1
                        for (int c = 0; c < 7; ++c) {
                            if (n0 + 8 * c >= p.N) break;            // uniform across the warp
                            uint32_t r8[8];
                            class_sum8(c, r8);
                            if (!row_ok) continue;
                            const int col = n0 + 8 * c;
                            float* prow = p.partial + ((size_t)split * p.M + row) * p.Np + col;
                            if (col + 8 <= p.Np) {
                                store_partial8(prow, r8);
                            } else {
#pragma unroll
                                for (int j = 0; j < 8; ++j)
                                    if (col + j < p.N) prow[j] = __uint_as_float(r8[j]);
                            }
                        }
                    }
                }
                if (B_SPLIT) {
                    // the tile's columns sit sigma_j columns to the right in the accumulator; BN - 8 of them:
                    // chunks of 32 and a last one of 24, split between the two warps of the lane quarter
                    const int sig = p.b_sigma[split & 7];
#pragma unroll 1
                    for (int c0 = 0; c0 < TILE_N; c0 += 32) {
                        if (n0 + c0 >= p.N) break;                   // uniform across the warp
                        if (((seq + (c0 >> 5)) & 1) != half) continue;
                        uint32_t r[32];
                        if (c0 + 32 <= TILE_N) {
                            ptx::tmem_ld_32x32(t_row + (uint32_t)(sig + c0), r);
                        } else {                                     // 24 columns: stay inside the accumulator
                            uint32_t r8a[8], r8b[8], r8c[8];
                            ptx::tmem_ld_32x8(t_row + (uint32_t)(sig + c0), r8a);
                            ptx::tmem_ld_32x8(t_row + (uint32_t)(sig + c0 + 8), r8b);
                            ptx::tmem_ld_32x8(t_row + (uint32_t)(sig + c0 + 16), r8c);
#pragma unroll
                            for (int i = 0; i < 8; ++i) { r[i] = r8a[i]; r[8 + i] = r8b[i]; r[16 + i] = r8c[i]; r[24 + i] = 0u; }
                        }
                        ptx::tmem_ld_wait();
                        if (!row_ok) continue;
                        const int col = n0 + c0;
                        const int width = min(32, TILE_N - c0);
                        float* prow = p.partial + ((size_t)split * p.M + row) * p.Np + col;
                        if (col + width <= p.Np) {
#pragma unroll
                            for (int v = 0; v < 4; ++v)
                                if (8 * v < width) store_partial8(prow + 8 * v, r + 8 * v);
                        } else {
#pragma unroll
                            for (int j = 0; j < 32; ++j)
                                if (j < width && col + j < p.N) prow[j] = __uint_as_float(r[j]);
                        }
                    }
                }
#pragma unroll 1
                for (int c0 = 0; !B_CLS && !B_SPLIT && c0 < TILE_N; c0 += 32) {
                    if (n0 + c0 >= p.N) break;                       // uniform across the warp
                    if (((seq * (TILE_N / 32) + (c0 >> 5)) & 1) != half) continue;
                    uint32_t r[32];
                    ptx::tmem_ld_32x32(t_row + (uint32_t)c0, r);
                    ptx::tmem_ld_wait();
                    if (!row_ok) continue;
                    const int col = n0 + c0;
                    float* prow = p.partial + ((size_t)split * p.M + row) * p.Np + col;
                    if (col + 32 <= p.Np) {
#pragma unroll
                        for (int v = 0; v < 4; ++v) store_partial8(prow + 8 * v, r + 8 * v);
                    } else {
#pragma unroll
                        for (int j = 0; j < 32; ++j)
                            if (col + j < p.N) prow[j] = __uint_as_float(r[j]);
                    }
                }
            }
            // this warp has read its share of the accumulator: hand the buffer back to the MMA warp
            if (!released) release_accumulator();
            if (++buf == NBUF) { buf = 0; buf_phase ^= 1u; }
        }
        if (lane == 0) ptx::bulk_wait_read<0>();             // TMA stores still reading this warp's staging boxes
    }

    // ------------------------------ common exit ----------------------------------------------
    ptx::tc_fence_before();
    if (CG == 2 || FUSE) {      // no CTA leaves while a peer may still read its shared memory or arrive on its barriers
        asm volatile("barrier.cluster.arrive.release.aligned;\nbarrier.cluster.wait.acquire.aligned;" ::: "memory");
    } else {
        __syncthreads();
    }
    if (threadIdx.x == 0 && *abort_flag) atomicOr(p.status, 1u);
    if (threadIdx.x == 0) ADAPT_TRACE(14, 0);
    if (warp == 1) {
        ptx::tc_fence_after();
        ptx::tmem_dealloc<CG>(tmem_base, TMEM_COLS);
    }
}

// Instruction descriptor, kind::f16: [4,6) D format (1 = fp32), [7,10) A format, [10,13) B format
// (0 = fp16, 1 = bf16), [15] A major, [16] B major (0 = K, 1 = MN), [17,23) N >> 3, [24,29) M >> 4.
inline uint32_t umma_idesc(int dtype, bool a_mn, bool b_mn, int mma_m, int mma_n)
{
    const uint32_t fmt = dtype == 0 ? 0u : 1u;
    return (1u << 4) | (fmt << 7) | (fmt << 10) | ((a_mn ? 1u : 0u) << 15) | ((b_mn ? 1u : 0u) << 16) |
           ((uint32_t)(mma_n >> 3) << 17) | ((uint32_t)(mma_m >> 4) << 24);
}

}  // namespace adapt

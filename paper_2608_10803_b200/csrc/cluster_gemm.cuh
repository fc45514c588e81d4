// Tile GEMM for small problems: ONE launch for any shape, layout and alignment.
//
// The tensor-core kernel needs 16-byte aligned rows for its TMA loads and a second launch to add
// split-K partials; on a problem of a few microseconds those extra launches are most of the time.
// Here a 64 x 64 output tile belongs to a thread-block cluster of CS CTAs (CS = 1, 2, 4, 8 or 16):
// CTA r of the cluster multiplies the r-th piece of the k range, the CS partial tiles are left in
// each CTA's shared memory, and every CTA then adds its 64 / CS rows of the tile over all ranks
// through distributed shared memory, in ascending rank order (the order of a split-K reduction,
// fixed, so the result does not depend on timing), rounds once and stores C.  No workspace.
//
// Operands come in as 16-byte cp.async.cg copies into a ring of raw stages (64 x 64 of each operand per
// stage, kept in the operand's own orientation); every thread's copies of a stage arrive on the stage's
// mbarrier (cp.async.mbarrier.arrive.noinc): the whole ring is in flight before the first wait, so a CTA
// pays about one trip to memory for 64 x ring values of k.  A row is copied as the up to nine aligned
// 16-byte chunks that hold it, whatever its alignment, and shifted into place by byte permutes, shared
// memory to shared memory, masked at the ragged edges, so no access is element-wise.  ldmatrix (transposing when the operand's contiguous dimension is not k) feeds
// mma.sync.m16n8k16 with fp32 accumulation.
#pragma once

#include <cstdint>
#include <cuda_runtime.h>
#include <cuda_fp16.h>
#include <cuda_bf16.h>

#include "adapt_internal.h"
#include "launch_pdl.cuh"
#include "ptx_sm100.cuh"        // mbarrier with bounded waits
#include "skinny_gemm.cuh"      // mma_16816

namespace adapt {

constexpr int kClusterThreads = 256;
constexpr int kClusterTile = 64;        // output tile edge
constexpr int kClusterKS = 64;          // k values per stage
constexpr int kClusterPitch = 72;       // 16-bit elements per staged row: 144 B, conflict-free for ldmatrix
constexpr int kClusterCPitch = 72;      // fp32 elements per row of the exchanged partial tile
static_assert(kClusterStageBytes == 2 * 64 * kClusterPitch * 2, "a stage is 64 rows of each operand");
static_assert(64 * kClusterCPitch * 4 <= kClusterStageBytes, "the partial tile reuses the first raw stage");

struct ClusterParams {
    const unsigned short* A;
    const unsigned short* B;
    unsigned short* C;
    int M, N, K;
    int64_t lda, ldb;            // leading dimensions in elements
    int P_n;                     // tiles along n
    int CS;                      // CTAs per cluster = pieces of the k range
    int k_per_cta;               // k values per CTA, a multiple of 16
    int ring;                    // raw stages in flight per CTA (1..kClusterMaxRing)
    int prefetch;                // L2 prefetch of the ring's stages ahead of the dependency wait
    unsigned int* status;        // device status word: bit 0 is set when a bounded wait gave up
};

__device__ __forceinline__ void ldmatrix_x4(uint32_t (&r)[4], uint32_t addr)
{
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t (&r)[4], uint32_t addr)
{
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ uint32_t cl_rank()
{
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
// All threads of all CTAs of the cluster; release/acquire orders the shared-memory traffic around it.
__device__ __forceinline__ void cl_sync()
{
    asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ float4 cl_load4(uint32_t local_addr, uint32_t rank)
{
    uint32_t remote;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote) : "r"(local_addr), "r"(rank));
    float4 v;
    asm volatile("ld.shared::cluster.v4.f32 {%0,%1,%2,%3}, [%4];"
                 : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "r"(remote) : "memory");
    return v;
}

// One row of an operand stage is 64 elements (128 bytes) that start `sh` bytes into a 16-byte chunk: chunk c
// of the row (c = 0..8) covers the row's bytes [16 c - sh, 16 c - sh + 16), of which those below 2 * nvr
// exist.  Every chunk that holds an existing byte is copied whole (such a chunk is always readable) by one
// 16-byte cp.async; a thread's copies of a stage arrive on the stage's mbarrier when they have landed.
// The shift pass then moves the 64 elements to the start of the row of the buffer ldmatrix reads, zeroing
// those that do not exist.
// A_KC: A is row-major (k contiguous); B_KC: B is column-major (k contiguous).
template <bool A_KC, bool B_KC, bool BF16>
__global__ void __launch_bounds__(kClusterThreads)
cluster_gemm_kernel(const ClusterParams p)
{
    extern __shared__ __align__(128) unsigned char s_dyn[];
    pdl_launch_dependents();
    // [ring of S raw stages: 64 rows of A, 64 of B, 144 bytes each][two shifted stages][S barriers, abort flag]
    constexpr int ROW = kClusterPitch * 2, OPND = 64 * ROW, STAGE = 2 * OPND;
    const int S = p.ring;
    const uint32_t raw0 = ptx::smem_u32(s_dyn);
    const uint32_t fin0 = raw0 + (uint32_t)(S * STAGE);
    const uint32_t bar0 = fin0 + 2u * STAGE;
    volatile int* abort_flag = reinterpret_cast<volatile int*>(s_dyn + (S + 2) * STAGE + 8 * kClusterMaxRing);
    float* sC = reinterpret_cast<float*>(s_dyn);                            // after the main loop

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    if (tid == 0) {
        for (int i = 0; i < S; ++i) ptx::mbar_init(bar0 + 8u * i, kClusterThreads);     // every thread arrives once per stage
        *abort_flag = 0;
        ptx::fence_barrier_init();
    }
    __syncthreads();

    const uint32_t rank = p.CS > 1 ? cl_rank() : 0u;
    const int tile = (int)(blockIdx.x / (unsigned)p.CS);
    const int m0 = (tile / p.P_n) * kClusterTile, n0 = (tile % p.P_n) * kClusterTile;
    const int k_begin = (int)rank * p.k_per_cta;
    const int k_end = min(p.K, k_begin + p.k_per_cta);
    const int n_stages = k_end > k_begin ? (k_end - k_begin + kClusterKS - 1) / kClusterKS : 0;
    // elements of a row of an mn-contiguous stage that exist (the k-contiguous ones end at k_end)
    const int nvs_a = min(64, p.M - m0), nvs_b = min(64, p.N - n0);
    // byte address of (row r, first element) of the stage at k_begin; rows 0..63 are A's, 64..127 B's
    auto row_addr = [&](int row) -> uintptr_t {
        const int r = row & 63;
        if (row < 64)
            return reinterpret_cast<uintptr_t>(p.A) + (uintptr_t)((A_KC ? (int64_t)(m0 + r) * p.lda + k_begin : (int64_t)(k_begin + r) * p.lda + m0) * 2);
        return reinterpret_cast<uintptr_t>(p.B) + (uintptr_t)((B_KC ? (int64_t)(n0 + r) * p.ldb + k_begin : (int64_t)(k_begin + r) * p.ldb + n0) * 2);
    };
    auto row_exists = [&](int row) -> bool {        // k-contiguous operands: the row is inside the matrix
        const int r = row & 63;
        return row < 64 ? (A_KC ? m0 + r < p.M : true) : (B_KC ? n0 + r < p.N : true);
    };
    // elements of a row that exist in a stage with kv values of k left
    auto row_count = [&](int row, bool exists, int kv) -> int {
        const bool kc = row < 64 ? A_KC : B_KC;
        if (kc) return exists ? min(64, kv) : 0;
        return (row & 63) < kv ? (row < 64 ? nvs_a : nvs_b) : 0;
    };

    // ---- copies: 128 rows x 9 chunks over the threads, consecutive threads on consecutive chunks of a row.
    // A stage advances every row by a multiple of 128 bytes, so the misalignment of a row is the same in
    // every stage; stages are issued in ascending order, so the sources just advance.  Which chunks of a
    // full stage (64 values of k left) hold data is worked out once; the last stage works it out again.
    constexpr int NCP = (128 * 9 + kClusterThreads - 1) / kClusterThreads;
    const char* cp_src[NCP];
    uint32_t cp_meta[NCP];          // [3:0] chunk, [7:4] sh, [15:8] row, [16] row exists, [17] copy exists, [18] chunk holds a byte of a full row
    auto chunk_live = [&](uint32_t mt, int kv) -> bool {
        const int c = mt & 15, sh = (mt >> 4) & 15, row = (mt >> 8) & 255;
        const int nvr = row_count(row, (mt >> 16) & 1, kv);
        return min(2 * nvr, 16 * c - sh + 16) > max(0, 16 * c - sh);
    };
#pragma unroll
    for (int j = 0; j < NCP; ++j) {
        const int e = tid + kClusterThreads * j;
        const bool exists = e < 128 * 9;
        const int row = exists ? e / 9 : 0, c = e - 9 * (e / 9);
        const uintptr_t a = row_addr(row);
        const uint32_t sh = (uint32_t)(a & 15);
        cp_src[j] = reinterpret_cast<const char*>(a - sh) + 16 * c;
        uint32_t mt = (uint32_t)c | (sh << 4) | ((uint32_t)row << 8) | ((row_exists(row) ? 1u : 0u) << 16) | ((exists ? 1u : 0u) << 17);
        cp_meta[j] = mt | ((chunk_live(mt, 64) ? 1u : 0u) << 18);
    }
    const int64_t step_a = A_KC ? 128 : 128 * p.lda, step_b = B_KC ? 128 : 128 * p.ldb;
    // Ahead of the wait for the kernel before this one on the stream: ask L2 for the lines of the ring's stages (hints
    // only; the copies proper come after the wait), so that the trip to memory overlaps the previous kernel's tail.
    if (p.prefetch) {
#pragma unroll
        for (int j = 0; j < NCP; ++j) {
            const uint32_t mt = cp_meta[j];
            // one request per 128-byte line: chunks 0 and 8 of a row (a row of a stage spans at most two lines)
            if (!((mt >> 17) & 1) || !((mt >> 18) & 1) || ((mt & 15) != 0 && (mt & 15) != 8)) continue;
            const char* src = cp_src[j];
            const int64_t step = ((mt >> 8) & 255) < 64 ? step_a : step_b;
            for (int s = 0; s < S && s < n_stages; ++s) ptx::prefetch_l2(src + s * step);
        }
    }
    pdl_wait();
    auto issue_stage = [&](int slot, int k0) {
        const int kv = k_end - k0;
#pragma unroll
        for (int j = 0; j < NCP; ++j) {
            const uint32_t mt = cp_meta[j];
            const bool live = ((mt >> 17) & 1) && (kv >= 64 ? ((mt >> 18) & 1) != 0 : chunk_live(mt, kv));
            if (live) {
                const uint32_t dst = raw0 + (uint32_t)(slot * STAGE) + ((mt >> 8) & 255) * ROW + 16u * (mt & 15);
                asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(cp_src[j]) : "memory");
            }
            cp_src[j] += ((mt >> 8) & 255) < 64 ? step_a : step_b;
        }
        // arrives when this thread's copies above have landed (the barrier expects one such arrival per thread)
        asm volatile("cp.async.mbarrier.arrive.noinc.shared::cta.b64 [%0];" ::"r"(bar0 + 8u * slot) : "memory");
    };

    // ---- shift pass: a half-warp per row, lane -> two 32-bit words of the row; 128 rows as 64 pairs over
    // the warps.  Row i of this thread is row 2 (warp + NWARP i) + lane / 16, so its addresses are the first
    // row's plus a constant.
    constexpr int NWARP = kClusterThreads / 32, NSH = 64 / NWARP;
    const int wl = lane & 15;
    const int row_first = 2 * warp + (lane >> 4);
    uint32_t sh_pack = 0, ok_pack = 0;             // 4 bits of sh and one existence bit per row of this thread
#pragma unroll
    for (int i = 0; i < NSH; ++i) {
        const int row = row_first + 2 * NWARP * i;
        sh_pack |= (uint32_t)(row_addr(row) & 15) << (4 * i);
        ok_pack |= (row_exists(row) ? 1u : 0u) << i;
    }
    // which of this lane's four elements exist in a row with nvr elements
    auto lane_mask = [&](int nvr, uint32_t& k0m, uint32_t& k1m) {
        const int nve = nvr - 4 * wl;
        k0m = nve >= 2 ? 0xffffffffu : (nve == 1 ? 0x0000ffffu : 0u);
        k1m = nve >= 4 ? 0xffffffffu : (nve == 3 ? 0x0000ffffu : 0u);
    };
    uint32_t ma0, ma1, mb0, mb1;                   // masks of a full-stage row of an mn-contiguous operand
    lane_mask(nvs_a, ma0, ma1);
    lane_mask(nvs_b, mb0, mb1);
    auto shift_stage = [&](int slot, int buf, int k0) {
        const int kv = k_end - k0;
        const unsigned char* src0 = s_dyn + slot * STAGE + row_first * ROW + 8 * wl;
        unsigned char* dst0 = s_dyn + (S + buf) * STAGE + row_first * ROW + 8 * wl;
#pragma unroll
        for (int i = 0; i < NSH; ++i) {
            const int op = i >= NSH / 2 ? 1 : 0;
            const bool kc = op ? B_KC : A_KC;
            uint32_t k0m, k1m;
            if (kv >= 64) {
                if (kc) k0m = k1m = 0u - ((ok_pack >> i) & 1u);
                else { k0m = op ? mb0 : ma0; k1m = op ? mb1 : ma1; }
            } else {
                lane_mask(row_count(row_first + 2 * NWARP * i, (ok_pack >> i) & 1, kv), k0m, k1m);
            }
            const unsigned sh = (sh_pack >> (4 * i)) & 15;
            const unsigned sel = 0x3210u + 0x1111u * (sh & 3u);        // byte shift 0 or 2 inside a word pair
            const uint32_t* w = reinterpret_cast<const uint32_t*>(src0 + i * (2 * NWARP * ROW) + (sh & 12u));
            const uint32_t w0 = w[0], w1 = w[1], w2 = w[2];
            // a word that no copy wrote may hold anything: select, do not multiply, so it cannot leak
            *reinterpret_cast<uint2*>(dst0 + i * (2 * NWARP * ROW)) =
                make_uint2(__byte_perm(w0, w1, sel) & k0m, __byte_perm(w1, w2, sel) & k1m);
        }
    };

    // warp (wm, wn) owns the 32 x 16 block at (32 wm, 16 wn): 2 x 2 MMAs of 16 x 8 per k step
    const int m_w = (warp & 1) * 32, n_w = (warp >> 1) * 16;
    const int g = lane >> 2, t = lane & 3;
    const int lj = lane >> 3, lr = lane & 7;      // ldmatrix: this lane addresses row lr of matrix lj
    float acc[2][2][4];
#pragma unroll
    for (int i = 0; i < 2; ++i)
#pragma unroll
        for (int j = 0; j < 2; ++j)
#pragma unroll
            for (int e = 0; e < 4; ++e) acc[i][j][e] = 0.f;

    // all S stages of the ring are in flight before the first wait: one trip to memory brings 64 S values of k
    for (int s = 0; s < S && s < n_stages; ++s) issue_stage(s, k_begin + s * kClusterKS);
    bool ok = true;
    for (int s = 0; s < n_stages; ++s) {
        const int slot = s % S, buf = s & 1;
        const int k0 = k_begin + s * kClusterKS;
        // bounded wait for the stage's rows.  The decision to leave is taken by the CTA as a whole: every thread
        // reaches the barrier below in every iteration, whether its own wait succeeded or gave up, so the barrier
        // counts of the warps never drift apart and all of them take the same path to the common exit.
        const bool landed = ptx::mbar_wait(bar0 + 8u * slot, (uint32_t)((s / S) & 1), abort_flag);
        if (landed) shift_stage(slot, buf, k0);
        // shifted stage complete; raw slot free; every warp is past the MMAs of stage s - 1
        if (__syncthreads_or(landed ? 0 : 1)) { ok = false; break; }
        if (s + S < n_stages) issue_stage(slot, k0 + S * kClusterKS);
        const uint32_t sa = fin0 + (uint32_t)(buf * STAGE), sb = sa + (uint32_t)OPND;
        auto k_step = [&](int kk) {
            uint32_t fa[2][4], fb[4];
#pragma unroll
            for (int mi = 0; mi < 2; ++mi) {
                const int mb = m_w + 16 * mi;
                if (A_KC)   // stored [m][k]: matrices (m 0-7, k 0-7), (m 8-15, k 0-7), (m 0-7, k 8-15), (m 8-15, k 8-15)
                    ldmatrix_x4(fa[mi], sa + (uint32_t)((mb + (lj & 1) * 8 + lr) * ROW + (kk + (lj >> 1) * 8) * 2));
                else        // stored [k][m]: the same four, each read transposed
                    ldmatrix_x4_trans(fa[mi], sa + (uint32_t)((kk + (lj >> 1) * 8 + lr) * ROW + (mb + (lj & 1) * 8) * 2));
            }
            if (B_KC)       // stored [n][k]: matrices (n 0-7, k 0-7), (n 0-7, k 8-15), (n 8-15, k 0-7), (n 8-15, k 8-15)
                ldmatrix_x4(fb, sb + (uint32_t)((n_w + (lj >> 1) * 8 + lr) * ROW + (kk + (lj & 1) * 8) * 2));
            else            // stored [k][n]
                ldmatrix_x4_trans(fb, sb + (uint32_t)((kk + (lj & 1) * 8 + lr) * ROW + (n_w + (lj >> 1) * 8) * 2));
#pragma unroll
            for (int mi = 0; mi < 2; ++mi)
#pragma unroll
                for (int nj = 0; nj < 2; ++nj)
                    mma_16816<BF16>(acc[mi][nj], fa[mi][0], fa[mi][1], fa[mi][2], fa[mi][3], fb[2 * nj], fb[2 * nj + 1]);
        };
        if (k_end - k0 >= kClusterKS) {     // a full stage: four steps with nothing between them
#pragma unroll
            for (int kk = 0; kk < kClusterKS; kk += 16) k_step(kk);
        } else {
            for (int kk = 0; k0 + kk < k_end; kk += 16) k_step(kk);
        }
    }
    // a wait that gave up: the result is not valid; the host reads the status word.  `ok` is the same in every
    // thread of the CTA, and the CTA still runs the barriers below (the cluster barriers too: its peers count on them).
    if (!ok && tid == 0) atomicOr(p.status, 1u);

    // a tile that is not shared with other CTAs is rounded and stored from the accumulators: a lane holds
    // pairs of neighbouring columns
    if (p.CS == 1) {
#pragma unroll
        for (int mi = 0; mi < 2; ++mi)
#pragma unroll
            for (int nj = 0; nj < 2; ++nj)
#pragma unroll
                for (int h = 0; h < 2; ++h) {
                    const int m = m0 + m_w + 16 * mi + g + 8 * h, n = n0 + n_w + 8 * nj + 2 * t;
                    if (m >= p.M || n >= p.N) continue;
                    unsigned short lo16, hi16;
                    if (BF16) {
                        __nv_bfloat16 a = __float2bfloat16_rn(acc[mi][nj][2 * h]), b = __float2bfloat16_rn(acc[mi][nj][2 * h + 1]);
                        lo16 = *reinterpret_cast<unsigned short*>(&a); hi16 = *reinterpret_cast<unsigned short*>(&b);
                    } else {
                        __half a = __float2half_rn(acc[mi][nj][2 * h]), b = __float2half_rn(acc[mi][nj][2 * h + 1]);
                        lo16 = *reinterpret_cast<unsigned short*>(&a); hi16 = *reinterpret_cast<unsigned short*>(&b);
                    }
                    unsigned short* dst = p.C + (int64_t)m * p.N + n;
                    if (n + 1 < p.N && (reinterpret_cast<uintptr_t>(dst) & 3) == 0) {
                        *reinterpret_cast<uint32_t*>(dst) = (uint32_t)lo16 | ((uint32_t)hi16 << 16);
                    } else {
                        dst[0] = lo16;
                        if (n + 1 < p.N) dst[1] = hi16;
                    }
                }
        return;
    }

    // the CTA's partial tile, fp32, into its own shared memory
    __syncthreads();
#pragma unroll
    for (int mi = 0; mi < 2; ++mi)
#pragma unroll
        for (int nj = 0; nj < 2; ++nj)
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                const int row = m_w + 16 * mi + g + 8 * h, col = n_w + 8 * nj + 2 * t;
                *reinterpret_cast<float2*>(&sC[row * kClusterCPitch + col]) = make_float2(acc[mi][nj][2 * h], acc[mi][nj][2 * h + 1]);
            }
    if (p.CS > 1) cl_sync(); else __syncthreads();

    // rank r adds rows [r * 64 / CS, (r + 1) * 64 / CS) over the ranks in ascending order and stores them
    const int rows_mine = kClusterTile / p.CS;
    for (int e = tid; e < rows_mine * 16; e += kClusterThreads) {
        const int row = (int)rank * rows_mine + (e >> 4), col = (e & 15) * 4;
        const int m = m0 + row, n = n0 + col;
        if (m >= p.M || n >= p.N) continue;
        float4 sum = make_float4(0.f, 0.f, 0.f, 0.f);
        if (p.CS > 1) {
            const uint32_t addr = (uint32_t)__cvta_generic_to_shared(&sC[row * kClusterCPitch + col]);
            for (int q = 0; q < p.CS; ++q) {
                const float4 v = cl_load4(addr, (uint32_t)q);
                sum.x += v.x; sum.y += v.y; sum.z += v.z; sum.w += v.w;
            }
        } else {
            const float4 v = *reinterpret_cast<const float4*>(&sC[row * kClusterCPitch + col]);
            sum.x += v.x; sum.y += v.y; sum.z += v.z; sum.w += v.w;
        }
        unsigned short* dst = p.C + (int64_t)m * p.N + n;
        const float o[4] = {sum.x, sum.y, sum.z, sum.w};
        unsigned short h[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            if (BF16) { __nv_bfloat16 b = __float2bfloat16_rn(o[j]); h[j] = *reinterpret_cast<unsigned short*>(&b); }
            else { __half b = __float2half_rn(o[j]); h[j] = *reinterpret_cast<unsigned short*>(&b); }
        }
        if (n + 4 <= p.N && (reinterpret_cast<uintptr_t>(dst) & 7) == 0) {
            *reinterpret_cast<uint2*>(dst) = make_uint2((uint32_t)h[0] | ((uint32_t)h[1] << 16), (uint32_t)h[2] | ((uint32_t)h[3] << 16));
        } else {
#pragma unroll
            for (int j = 0; j < 4; ++j)
                if (n + j < p.N) dst[j] = h[j];
        }
    }
    // no CTA may leave while a peer still reads its partial tile
    if (p.CS > 1) cl_sync();
}

typedef void (*ClusterKernel)(const ClusterParams);

inline ClusterKernel cluster_pick(bool a_kc, bool b_kc, bool bf16)
{
    if (bf16) {
        if (a_kc) return b_kc ? cluster_gemm_kernel<true, true, true> : cluster_gemm_kernel<true, false, true>;
        return b_kc ? cluster_gemm_kernel<false, true, true> : cluster_gemm_kernel<false, false, true>;
    }
    if (a_kc) return b_kc ? cluster_gemm_kernel<true, true, false> : cluster_gemm_kernel<true, false, false>;
    return b_kc ? cluster_gemm_kernel<false, true, false> : cluster_gemm_kernel<false, false, false>;
}

// Once per device: the deepest ring needs more than the default dynamic shared memory.
inline cudaError_t cluster_set_attributes()
{
    for (int v = 0; v < 8; ++v) {
        cudaError_t e = cudaFuncSetAttribute(cluster_pick(v & 1, v & 2, v & 4), cudaFuncAttributeMaxDynamicSharedMemorySize,
                                             cluster_smem_bytes(kClusterMaxRing));
        if (e != cudaSuccess) return e;
        e = cudaFuncSetAttribute(cluster_pick(v & 1, v & 2, v & 4), cudaFuncAttributeNonPortableClusterSizeAllowed, 1);   // clusters of 16
        if (e != cudaSuccess) return e;
    }
    return cudaSuccess;
}

// Largest cluster size (16, 8, 4, 2, 1) of which the device runs at least one cluster with the deepest ring.
inline int cluster_max_size()
{
    for (int cs = 16; cs > 1; cs >>= 1) {
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3((unsigned)cs, 1, 1);
        cfg.blockDim = dim3(kClusterThreads, 1, 1);
        cfg.dynamicSmemBytes = (size_t)cluster_smem_bytes(kClusterMaxRing);
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeClusterDimension;
        attr[0].val.clusterDim.x = (unsigned)cs;
        attr[0].val.clusterDim.y = 1;
        attr[0].val.clusterDim.z = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        int n = 0;
        if (cudaOccupancyMaxActiveClusters(&n, (const void*)cluster_pick(true, false, false), &cfg) == cudaSuccess && n >= 1) return cs;
        (void)cudaGetLastError();
    }
    return 1;
}

// Host launcher.  c.cluster = CS; c.stages = depth of the raw ring; the grid is CS CTAs per tile, the cluster spans blockIdx.x.
inline adapt_status_t launch_cluster(const Shape& s, const Config& c, const void* A, const void* B, void* C,
                                     unsigned int* status, cudaStream_t stream, int prefetch = 1)
{
    ClusterParams p;
    p.A = (const unsigned short*)A;
    p.B = (const unsigned short*)B;
    p.C = (unsigned short*)C;
    p.M = (int)s.M; p.N = (int)s.N; p.K = (int)s.K;
    const bool a_kc = s.layoutA == ADAPT_ROW_MAJOR, b_kc = s.layoutB == ADAPT_COL_MAJOR;
    p.lda = a_kc ? s.K : s.M;
    p.ldb = b_kc ? s.K : s.N;
    p.P_n = c.P_n;
    p.CS = c.cluster;
    p.k_per_cta = (int)round_up(ceil_div(s.K, c.cluster), 16);
    p.ring = c.stages;
    p.prefetch = prefetch;
    p.status = status;
    cudaLaunchConfig_t cfg;
    memset(&cfg, 0, sizeof(cfg));
    cfg.gridDim = dim3((unsigned)((int64_t)c.P_m * c.P_n * c.cluster), 1, 1);
    cfg.blockDim = dim3(kClusterThreads, 1, 1);
    cfg.dynamicSmemBytes = (size_t)cluster_smem_bytes(c.stages);
    cfg.stream = stream;
    cudaLaunchAttribute attr[2];
    pdl_attribute(&attr[0]);
    attr[1].id = cudaLaunchAttributeClusterDimension;
    attr[1].val.clusterDim.x = (unsigned)c.cluster;
    attr[1].val.clusterDim.y = 1;
    attr[1].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = c.cluster > 1 ? 2 : 1;
    void* args[1] = {&p};
    const size_t arg_bytes[1] = {sizeof(p)};
    if (launch_exc(&cfg, (const void*)cluster_pick(a_kc, b_kc, s.dtype != 0), args, arg_bytes, 1) != cudaSuccess) return ADAPT_ERR_CUDA;
    return ADAPT_OK;
}

}  // namespace adapt

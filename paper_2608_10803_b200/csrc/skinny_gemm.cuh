// Warp-level GEMM for skinny shapes (M <= 16 or N <= 16): the paper's "Small-M Copy" module
// (Table 2) re-thought for B200.  The large operand is streamed from HBM exactly once with
// 16-byte loads straight into mma.sync fragments (no shared-memory tile pipeline); the small
// operand (at most 16 rows) is staged in shared memory per k-chunk.
//
// Canonical form:  Out[s][r] = sum_k Small[s][k] * Str[k][r],  s < ms <= 16,  r < R.
//   M <= 16:  Small = A,   Str = B,   R = N, Out[s][r] = C[s][r]
//   N <= 16:  Small = B^T, Str = A^T, R = M, Out[s][r] = C[r][s]
// The streamed operand is either r-contiguous ("RC": Str[k][r] at k*ld + r) or k-contiguous
// ("KC": at r*ld + k).  Rows of the streamed operand need no alignment beyond 2 bytes: an
// unaligned 8-element group is assembled from the two aligned 16-byte chunks that cover it.
//
// mma.sync.m16n8k16 takes Small as its 16 x 16 operand and 8 streamed r-values as its 16 x 8
// operand.  The assignment of k values to fragment slots and of r values to fragment columns
// is a permutation chosen so that every lane's fragment registers come from its own 16-byte
// loads; sums over k do not depend on it and the output permutation is undone at the store.
#pragma once

#include <cstdint>
#include <cuda_runtime.h>

#include "adapt_internal.h"

namespace adapt {

constexpr int kSkinnyThreads = 256;
constexpr int kSkinnyKChunk = 256;          // k values staged per shared-memory chunk of Small
constexpr int kSkinnySmallPitch = kSkinnyKChunk + 40;   // 16-bit elements; 592 B rows: 16 B mod 128 B = 80 -> conflict-light

struct SkinnyParams {
    const unsigned short* Small;
    const unsigned short* Str;
    int ms, R, K;
    int64_t small_ss, small_sk;      // element strides of Small along s and k
    int64_t ld;                      // leading dimension of the streamed operand (elements)
    int BNs;                         // streamed r-values per CTA: 128, 256 or 512
    int P_k, k_per_split;            // k splits; k values per split (multiple of kSkinnyKChunk unless P_k == 1)
    int dtype;
    unsigned short* C;               // used when P_k == 1
    float* partial;                  // [P_k][M][N] fp32, used when P_k > 1
    int64_t out_ss, out_sr;          // element strides of the output along s and r
    int64_t MN;                      // M * N
};

__device__ __forceinline__ uint4 ldg16(const void* p)
{
    uint4 v;
    asm volatile("ld.global.nc.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}

// Eight consecutive 16-bit elements starting at a 2-byte aligned address.
__device__ __forceinline__ uint4 load8_any(const unsigned short* p)
{
    const uintptr_t a = reinterpret_cast<uintptr_t>(p);
    const unsigned sh = (unsigned)(a & 15);
    const uint4* q = reinterpret_cast<const uint4*>(a - sh);
    const uint4 lo = ldg16(q);
    if (sh == 0) return lo;
    const uint4 hi = ldg16(q + 1);
    uint32_t w0, w1, w2, w3, w4;
    switch (sh >> 2) {
        case 0: w0 = lo.x; w1 = lo.y; w2 = lo.z; w3 = lo.w; w4 = hi.x; break;
        case 1: w0 = lo.y; w1 = lo.z; w2 = lo.w; w3 = hi.x; w4 = hi.y; break;
        case 2: w0 = lo.z; w1 = lo.w; w2 = hi.x; w3 = hi.y; w4 = hi.z; break;
        default: w0 = lo.w; w1 = hi.x; w2 = hi.y; w3 = hi.z; w4 = hi.w; break;
    }
    if ((sh & 2) == 0) return make_uint4(w0, w1, w2, w3);
    return make_uint4(__byte_perm(w0, w1, 0x5432), __byte_perm(w1, w2, 0x5432),
                      __byte_perm(w2, w3, 0x5432), __byte_perm(w3, w4, 0x5432));
}

// Up to eight elements, the first `nv` valid, the rest zero.  nv <= 0 loads nothing.
__device__ __forceinline__ uint4 load8_masked(const unsigned short* p, int nv)
{
    if (nv >= 8) return load8_any(p);
    unsigned short v[8];
#pragma unroll
    for (int j = 0; j < 8; ++j) v[j] = (j < nv) ? __ldg(p + j) : (unsigned short)0;
    return make_uint4((uint32_t)v[0] | ((uint32_t)v[1] << 16), (uint32_t)v[2] | ((uint32_t)v[3] << 16),
                      (uint32_t)v[4] | ((uint32_t)v[5] << 16), (uint32_t)v[6] | ((uint32_t)v[7] << 16));
}

template <bool BF16>
__device__ __forceinline__ void mma_16816(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0, uint32_t b1)
{
    if (BF16)
        asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                     : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3]) : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
    else
        asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                     : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3]) : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

__device__ __forceinline__ uint32_t word_of(const uint4& v, int i)
{
    return i == 0 ? v.x : (i == 1 ? v.y : (i == 2 ? v.z : v.w));
}

// KC: streamed operand k-contiguous.  BF16: element type.
template <bool KC, bool BF16>
__global__ void __launch_bounds__(kSkinnyThreads, 2)
skinny_gemm_kernel(const SkinnyParams p)
{
    __shared__ __align__(16) unsigned short s_small[16][kSkinnySmallPitch];
    __shared__ float s_out[8 * 16 * 64];            // [warp][s][64 r-values of that warp]

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int g = lane >> 2, t = lane & 3;
    const int warps_r = p.BNs / 64;                  // warps side by side along r
    const int WK = 8 / warps_r;                      // warps stacked along k
    const int wr = warp % warps_r, wk = warp / warps_r;
    const int r_cta = blockIdx.x * p.BNs;
    const int r_warp = r_cta + wr * 64;
    const int split = blockIdx.y;
    const int k_begin = split * p.k_per_split;
    const int k_end = min(p.K, k_begin + p.k_per_split);

    float acc[8][4];
#pragma unroll
    for (int j = 0; j < 8; ++j)
#pragma unroll
        for (int i = 0; i < 4; ++i) acc[j][i] = 0.f;

    const int k_sub = kSkinnyKChunk / WK;            // k values one warp covers per chunk

    for (int kc0 = k_begin; kc0 < k_end; kc0 += kSkinnyKChunk) {
        __syncthreads();                             // previous chunk fully consumed
        // ---- stage Small[0..16)[kc0 .. kc0+chunk) as 16-bit, zero beyond ms and k_end ----
        if (p.small_sk == 1) {
            for (int e = tid; e < 16 * kSkinnyKChunk; e += kSkinnyThreads) {
                const int s = e / kSkinnyKChunk, k = e - s * kSkinnyKChunk;
                unsigned short v = 0;
                if (s < p.ms && kc0 + k < k_end) v = __ldg(p.Small + (int64_t)s * p.small_ss + (kc0 + k));
                s_small[s][k] = v;
            }
        } else {
            for (int e = tid; e < 16 * kSkinnyKChunk; e += kSkinnyThreads) {
                const int s = e & 15, k = e >> 4;
                unsigned short v = 0;
                if (s < p.ms && kc0 + k < k_end) v = __ldg(p.Small + (int64_t)s * p.small_ss + (int64_t)(kc0 + k) * p.small_sk);
                s_small[s][k] = v;
            }
        }
        __syncthreads();

        const int kw0 = kc0 + wk * k_sub;            // this warp's k range inside the chunk
        if (!KC) {
            // ---- r-contiguous stream: a lane loads rows k+2t, +1, +8, +9 at columns r_warp + 8g .. +7 ----
            const int nv = p.R - (r_warp + 8 * g);   // valid columns of this lane's group
#pragma unroll 2
            for (int ks = 0; ks < k_sub; ks += 16) {
                const int k = kw0 + ks;
                if (k >= k_end) break;
                const int kr[4] = {k + 2 * t, k + 2 * t + 1, k + 2 * t + 8, k + 2 * t + 9};
                uint4 v[4];
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    v[i] = make_uint4(0, 0, 0, 0);
                    if (kr[i] < k_end && nv > 0) v[i] = load8_masked(p.Str + (int64_t)kr[i] * p.ld + (r_warp + 8 * g), nv);
                }
                const int kl = k - kc0 + 2 * t;      // position inside the staged chunk
                const uint32_t a0 = *reinterpret_cast<const uint32_t*>(&s_small[g][kl]);
                const uint32_t a1 = *reinterpret_cast<const uint32_t*>(&s_small[g + 8][kl]);
                const uint32_t a2 = *reinterpret_cast<const uint32_t*>(&s_small[g][kl + 8]);
                const uint32_t a3 = *reinterpret_cast<const uint32_t*>(&s_small[g + 8][kl + 8]);
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    const uint32_t sel = (j & 1) ? 0x7632u : 0x5410u;
                    const uint32_t b0 = __byte_perm(word_of(v[0], j >> 1), word_of(v[1], j >> 1), sel);
                    const uint32_t b1 = __byte_perm(word_of(v[2], j >> 1), word_of(v[3], j >> 1), sel);
                    mma_16816<BF16>(acc[j], a0, a1, a2, a3, b0, b1);
                }
            }
        } else {
            // ---- k-contiguous stream: a lane loads 8 k values (k + 8t .. +7) of rows r_warp + 8j + g ----
#pragma unroll 1
            for (int ks = 0; ks < k_sub; ks += 32) {
                const int k = kw0 + ks;
                if (k >= k_end) break;
                const int nvk = k_end - (k + 8 * t);
                uint4 v[8];
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    const int r = r_warp + 8 * j + g;
                    v[j] = make_uint4(0, 0, 0, 0);
                    if (r < p.R && nvk > 0) v[j] = load8_masked(p.Str + (int64_t)r * p.ld + (k + 8 * t), nvk);
                }
                const int kl = k - kc0 + 8 * t;
                const uint4 lo = *reinterpret_cast<const uint4*>(&s_small[g][kl]);
                const uint4 hi = *reinterpret_cast<const uint4*>(&s_small[g + 8][kl]);
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    mma_16816<BF16>(acc[j], lo.x, hi.x, lo.y, hi.y, v[j].x, v[j].y);
                    mma_16816<BF16>(acc[j], lo.z, hi.z, lo.w, hi.w, v[j].z, v[j].w);
                }
            }
        }
    }

    // ---- undo the fragment permutation into s_out[warp][s][rr], rr = r - r_warp ----
    // accumulator layout: acc[j][0..1] -> row g, fragment columns 2t, 2t+1; acc[j][2..3] -> row g+8.
    // RC: fragment column c of MMA j is r = 8c + j.   KC: fragment column c of group j is r = 8j + c.
    __syncthreads();
    float* so = s_out + warp * (16 * 64);
#pragma unroll
    for (int j = 0; j < 8; ++j) {
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int s = g + ((i & 2) ? 8 : 0);
            const int c = 2 * t + (i & 1);
            const int rr = KC ? (8 * j + c) : (8 * c + j);
            so[s * 64 + rr] = acc[j][i];
        }
    }
    __syncthreads();
    // ---- add the WK warps that share an r range in ascending wk (fixed order), cast once, store ----
    for (int e = tid; e < 16 * p.BNs; e += kSkinnyThreads) {
        int s, rl;
        if (p.out_sr == 1) { rl = e % p.BNs; s = e / p.BNs; } else { s = e & 15; rl = e >> 4; }
        const int r = r_cta + rl;
        if (s >= p.ms || r >= p.R) continue;
        const int w0 = rl >> 6, rr = rl & 63;
        float sum = 0.f;
        for (int w = 0; w < WK; ++w) sum += s_out[(w * warps_r + w0) * (16 * 64) + s * 64 + rr];
        const int64_t o = (int64_t)s * p.out_ss + (int64_t)r * p.out_sr;
        if (p.P_k == 1) {
            unsigned short h;
            if (BF16) { __nv_bfloat16 b = __float2bfloat16_rn(sum); h = *reinterpret_cast<unsigned short*>(&b); }
            else { __half b = __float2half_rn(sum); h = *reinterpret_cast<unsigned short*>(&b); }
            p.C[o] = h;
        } else {
            p.partial[(int64_t)split * p.MN + o] = sum;
        }
    }
}

// Host launcher: maps (M, N, K, layouts) onto the canonical form above.
inline adapt_status_t launch_skinny(const Shape& s, const Config& c, const void* A, const void* B, void* C,
                                    float* partial, cudaStream_t stream)
{
    SkinnyParams p;
    bool kc;
    if (s.M <= 16 && (s.M <= s.N || s.N > 16)) {
        // Small = A, streamed = B
        p.Small = (const unsigned short*)A;
        p.Str = (const unsigned short*)B;
        p.ms = (int)s.M; p.R = (int)s.N;
        if (s.layoutA == ADAPT_ROW_MAJOR) { p.small_ss = s.K; p.small_sk = 1; } else { p.small_ss = 1; p.small_sk = s.M; }
        kc = s.layoutB == ADAPT_COL_MAJOR;
        p.ld = kc ? s.K : s.N;
        p.out_ss = s.N; p.out_sr = 1;
    } else {
        // Small = B^T, streamed = A^T
        p.Small = (const unsigned short*)B;
        p.Str = (const unsigned short*)A;
        p.ms = (int)s.N; p.R = (int)s.M;
        if (s.layoutB == ADAPT_ROW_MAJOR) { p.small_ss = 1; p.small_sk = s.N; } else { p.small_ss = s.K; p.small_sk = 1; }
        kc = s.layoutA == ADAPT_ROW_MAJOR;
        p.ld = kc ? s.K : s.M;
        p.out_ss = 1; p.out_sr = s.N;
    }
    p.K = (int)s.K;
    p.BNs = c.BN;
    p.P_k = c.P_k;
    // splits are whole multiples of the staging chunk so that no chunk straddles two splits
    const int64_t chunks = ceil_div(s.K, kSkinnyKChunk);
    p.k_per_split = (int)(ceil_div(chunks, c.P_k) * kSkinnyKChunk);
    p.dtype = s.dtype;
    p.C = (unsigned short*)C;
    p.partial = partial;
    p.MN = s.M * s.N;
    dim3 grid((unsigned)ceil_div(p.R, p.BNs), (unsigned)c.P_k, 1);
    if (kc) {
        if (s.dtype) skinny_gemm_kernel<true, true><<<grid, kSkinnyThreads, 0, stream>>>(p);
        else skinny_gemm_kernel<true, false><<<grid, kSkinnyThreads, 0, stream>>>(p);
    } else {
        if (s.dtype) skinny_gemm_kernel<false, true><<<grid, kSkinnyThreads, 0, stream>>>(p);
        else skinny_gemm_kernel<false, false><<<grid, kSkinnyThreads, 0, stream>>>(p);
    }
    return ADAPT_OK;
}

}  // namespace adapt

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
// unaligned 8-element group is assembled, without branches, from the two aligned 16-byte chunks
// that cover it (the second chunk is an L1 hit: the neighbouring lane loads it as its first).
//
// mma.sync.m16n8k16 takes Small as its 16 x 16 operand and 8 streamed r-values as its 16 x 8
// operand.  The assignment of k values to fragment slots and of r values to fragment columns
// is a permutation chosen so that every lane's fragment registers come from its own 16-byte
// loads; sums over k do not depend on it and the output permutation is undone at the store.
//
// Work split: a CTA of 8 warps owns BNs streamed r-values and one k split.  RC: warps sit side
// by side along r (64 each) and stack along k inside a staged chunk.  KC: every warp owns 8
// r-rows per pass and reads 512 contiguous bytes of each row per iteration.
#pragma once

#include <cstdint>
#include <cuda_runtime.h>
#include <cuda_fp16.h>
#include <cuda_bf16.h>

#include "adapt_internal.h"
#include "launch_pdl.cuh"

namespace adapt {

constexpr int kSkinnyThreads = 256;
// Row pitch of the staged chunk in 16-bit elements, chosen per variant so that the fragment reads
// are free of bank conflicts: RC reads 4 bytes per lane (rows 16 B apart mod 128 B), KC reads
// 16 bytes per lane (rows 64 B apart mod 128 B).
constexpr int kSkinnyPitchRC = kSkinnyKChunk + 8;
constexpr int kSkinnyPitchKC = kSkinnyKChunk + 32;
constexpr int kSkinnySmemBytes = 8 * 16 * 64 * 4;       // the output exchange buffer (32 KB) also holds the staged chunk

struct SkinnyParams {
    const unsigned short* Small;
    const unsigned short* Str;
    int ms, R, K;
    int64_t small_ss, small_sk;      // element strides of Small along s and k
    int64_t ld;                      // leading dimension of the streamed operand (elements)
    int BNs;                         // streamed r-values per CTA: 128, 256 or 512 (RC); 64-row passes (KC)
    int P_k, k_per_split;            // k splits; k values per split (multiple of kSkinnyKChunk unless P_k == 1)
    int dtype;
    unsigned short* C;               // used when P_k == 1
    float* partial;                  // [P_k][M][Np] fp32, used when P_k > 1
    int64_t out_ss, out_sr;          // element strides of the output along s and r
    int64_t part_ss, part_sr;        // element strides of the fp32 partial along s and r
    int64_t part_slab;               // elements per split: M * Np
};

// Eight consecutive 16-bit elements from a 2-byte aligned address, branch-free.
template <bool ALIGNED>
__device__ __forceinline__ uint4 load8(const unsigned short* p)
{
    if (ALIGNED) return __ldg(reinterpret_cast<const uint4*>(p));
    const uintptr_t a = reinterpret_cast<uintptr_t>(p);
    const unsigned sh = (unsigned)(a & 15);
    const uint4* q = reinterpret_cast<const uint4*>(a - sh);
    const uint4 lo = __ldg(q);
    const uint4 hi = __ldg(q + (sh ? 1 : 0));          // sh == 0: the same chunk again, never past the data
    const unsigned ws = sh >> 2;
    const unsigned sel = 0x3210u + 0x1111u * (sh & 3u); // byte shift 0 or 2 inside a word pair
    const uint32_t w0 = ws == 0 ? lo.x : ws == 1 ? lo.y : ws == 2 ? lo.z : lo.w;
    const uint32_t w1 = ws == 0 ? lo.y : ws == 1 ? lo.z : ws == 2 ? lo.w : hi.x;
    const uint32_t w2 = ws == 0 ? lo.z : ws == 1 ? lo.w : ws == 2 ? hi.x : hi.y;
    const uint32_t w3 = ws == 0 ? lo.w : ws == 1 ? hi.x : ws == 2 ? hi.y : hi.z;
    const uint32_t w4 = ws == 0 ? hi.x : ws == 1 ? hi.y : ws == 2 ? hi.z : hi.w;
    return make_uint4(__byte_perm(w0, w1, sel), __byte_perm(w1, w2, sel), __byte_perm(w2, w3, sel), __byte_perm(w3, w4, sel));
}

// Up to eight elements, the first `nv` valid, the rest zero.  nv <= 0 loads nothing.  Edges only.
__device__ __forceinline__ uint4 load8_edge(const unsigned short* p, int nv)
{
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
        asm("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
            : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3]) : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
    else
        asm("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
            : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3]) : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

__device__ __forceinline__ uint32_t word_of(const uint4& v, int i)
{
    return i == 0 ? v.x : (i == 1 ? v.y : (i == 2 ? v.z : v.w));
}

// Stage Small[0..16)[kc0 .. kc0 + chunk) into shared memory, zero beyond ms and k_end.
template <int PITCH>
__device__ __forceinline__ void stage_small(const SkinnyParams& p, unsigned short (*s_small)[PITCH],
                                            int kc0, int k_end, int tid)
{
    if (p.small_sk == 1) {
        // rows are k-contiguous: one thread moves 8 consecutive k of one row
        for (int e = tid; e < 16 * (kSkinnyKChunk / 8); e += kSkinnyThreads) {
            const int s = e / (kSkinnyKChunk / 8), k = (e - s * (kSkinnyKChunk / 8)) * 8;
            uint4 v = make_uint4(0, 0, 0, 0);
            const int nv = k_end - (kc0 + k);
            if (s < p.ms && nv > 0) {
                const unsigned short* src = p.Small + (int64_t)s * p.small_ss + (kc0 + k);
                v = nv >= 8 ? load8<false>(src) : load8_edge(src, nv);
            }
            *reinterpret_cast<uint4*>(&s_small[s][k]) = v;
        }
    } else if (p.small_ss == 1) {
        // Small[s][k] at k*small_sk + s with small_sk = ms: the chunk is one contiguous span
        const int span = p.ms * min(kSkinnyKChunk, k_end - kc0);
        const unsigned short* src = p.Small + (int64_t)kc0 * p.small_sk;
        for (int e = tid; e < 16 * kSkinnyKChunk; e += kSkinnyThreads) {
            const int s = e & 15, k = e >> 4;
            if (s >= p.ms || kc0 + k >= k_end) s_small[s][k] = 0;
        }
        for (int e = tid; e < span; e += kSkinnyThreads) {
            const int k = e / p.ms, s = e - k * p.ms;
            s_small[s][k] = __ldg(src + e);
        }
    } else {
        for (int e = tid; e < 16 * kSkinnyKChunk; e += kSkinnyThreads) {
            const int s = e & 15, k = e >> 4;
            unsigned short v = 0;
            if (s < p.ms && kc0 + k < k_end) v = __ldg(p.Small + (int64_t)s * p.small_ss + (int64_t)(kc0 + k) * p.small_sk);
            s_small[s][k] = v;
        }
    }
}

// KC: streamed operand k-contiguous.  BF16: element type.  ALIGNED: every 8-element group of the
// streamed operand this kernel loads starts on a 16-byte boundary.
template <bool KC, bool BF16, bool ALIGNED>
__global__ void __launch_bounds__(kSkinnyThreads, 2)
skinny_gemm_kernel(const SkinnyParams p)
{
    __shared__ __align__(16) unsigned char s_raw[kSkinnySmemBytes];
    pdl_launch_dependents();
    pdl_wait();
    constexpr int PITCH = KC ? kSkinnyPitchKC : kSkinnyPitchRC;
    unsigned short (*s_small)[PITCH] = reinterpret_cast<unsigned short (*)[PITCH]>(s_raw);
    float* s_out = reinterpret_cast<float*>(s_raw);         // reused after the main loop
    static_assert(16 * PITCH * 2 <= kSkinnySmemBytes, "staged chunk must fit the exchange buffer");

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int g = lane >> 2, t = lane & 3;
    const int split = blockIdx.y;
    const int k_begin = split * p.k_per_split;
    const int k_end = min(p.K, k_begin + p.k_per_split);
    const int r_cta = blockIdx.x * p.BNs;

    // RC: warps_r warps side by side (64 r each), WK stacked along k.  KC: 8 warps x 8 rows per pass.
    const int warps_r = KC ? 8 : p.BNs / 64;
    const int WK = KC ? 1 : 8 / warps_r;
    const int wr = warp % warps_r, wk = warp / warps_r;

    float acc[8][4];
#pragma unroll
    for (int j = 0; j < 8; ++j)
#pragma unroll
        for (int i = 0; i < 4; ++i) acc[j][i] = 0.f;

    if (!KC) {
        const int r_warp = r_cta + wr * 64;
        const int nv = p.R - (r_warp + 8 * g);           // valid columns of this lane's group
        const bool cols_full = r_warp + 64 <= p.R;
        for (int kc0 = k_begin; kc0 < k_end; kc0 += kSkinnyKChunk) {
            __syncthreads();                             // previous chunk fully consumed
            stage_small<PITCH>(p, s_small, kc0, k_end, tid);
            __syncthreads();
            // the WK warps that share an r range split the chunk's k values evenly (in steps of 16), so a
            // short k range still keeps all of them busy
            const int k_sub = ((min(kSkinnyKChunk, k_end - kc0) + WK - 1) / WK + 15) & ~15;
            const int kw0 = kc0 + wk * k_sub;
            // a lane loads rows k+2t, +1, +8, +9 at columns r_warp + 8g .. +7.  The loads run kDepth steps ahead of the
            // MMAs that use them (register ring, indices fixed by full unrolling): with the loads of a step consumed in
            // the same step a lane had one trip to memory in flight and the kernel streamed at a quarter of the HBM rate
            const int k_lim = min(k_end, kw0 + k_sub);
            const int n_steps = kw0 < k_lim ? (k_lim - kw0 + 15) >> 4 : 0;
            auto load_step = [&](int step, uint4 (&v)[4]) {
                const int k = kw0 + 16 * step;
                const int kr[4] = {k + 2 * t, k + 2 * t + 1, k + 2 * t + 8, k + 2 * t + 9};
                if (cols_full && k + 16 <= k_end) {
#pragma unroll
                    for (int i = 0; i < 4; ++i) v[i] = load8<ALIGNED>(p.Str + (int64_t)kr[i] * p.ld + (r_warp + 8 * g));
                } else {
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        v[i] = make_uint4(0, 0, 0, 0);
                        if (kr[i] < k_end && nv > 0) v[i] = load8_edge(p.Str + (int64_t)kr[i] * p.ld + (r_warp + 8 * g), nv);
                    }
                }
            };
            auto mma_step = [&](int step, const uint4 (&v)[4]) {
                const int kl = kw0 + 16 * step - kc0 + 2 * t;      // position inside the staged chunk
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
            };
            constexpr int kDepth = 4;
            uint4 ring[kDepth][4];
#pragma unroll
            for (int d = 0; d < kDepth; ++d)
                if (d < n_steps) load_step(d, ring[d]);
            for (int st = 0; st < n_steps; st += kDepth) {
#pragma unroll
                for (int d = 0; d < kDepth; ++d) {
                    if (st + d < n_steps) {
                        mma_step(st + d, ring[d]);
                        if (st + d + kDepth < n_steps) load_step(st + d + kDepth, ring[d]);
                    }
                }
            }
        }
        // fragment columns: column c of MMA j is r = 8c + j
        __syncthreads();
        float* so = s_out + warp * (16 * 64);
#pragma unroll
        for (int j = 0; j < 8; ++j)
#pragma unroll
            for (int i = 0; i < 4; ++i)
                so[(g + ((i & 2) ? 8 : 0)) * 64 + 8 * (2 * t + (i & 1)) + j] = acc[j][i];
        __syncthreads();
        // add the WK warps that share an r range in ascending wk (fixed order), cast once, store
        for (int e = tid; e < 16 * p.BNs; e += kSkinnyThreads) {
            int s, rl;
            if (p.out_sr == 1) { rl = e % p.BNs; s = e / p.BNs; } else { s = e & 15; rl = e >> 4; }
            const int r = r_cta + rl;
            if (s >= p.ms || r >= p.R) continue;
            const int w0 = rl >> 6, rr = rl & 63;
            float sum = 0.f;
            for (int w = 0; w < WK; ++w) sum += s_out[(w * warps_r + w0) * (16 * 64) + s * 64 + rr];
            if (p.P_k == 1) {
                unsigned short h;
                if (BF16) { __nv_bfloat16 b = __float2bfloat16_rn(sum); h = *reinterpret_cast<unsigned short*>(&b); }
                else { __half b = __float2half_rn(sum); h = *reinterpret_cast<unsigned short*>(&b); }
                p.C[(int64_t)s * p.out_ss + (int64_t)r * p.out_sr] = h;
            } else {
                p.partial[(int64_t)split * p.part_slab + (int64_t)s * p.part_ss + (int64_t)r * p.part_sr] = sum;
            }
        }
    } else {
        // ---- k-contiguous stream.  The CTA walks its BNs rows in passes of 64 (8 per warp); in a pass a
        // lane reads, for row r_pass + 8*warp + g, eight 16-byte groups at k + 32j + 8t: 512 contiguous
        // bytes per row per iteration.  Two accumulator sets (acc[0], acc[1]) per pass, added at the end.
        (void)wr; (void)wk;
        for (int r_pass = r_cta; r_pass < min(p.R, r_cta + p.BNs); r_pass += 64) {
            const int r = r_pass + 8 * warp + g;
            const bool row_ok = r < p.R;
            const unsigned short* row = p.Str + (int64_t)(row_ok ? r : 0) * p.ld;
#pragma unroll
            for (int i = 0; i < 4; ++i) acc[0][i] = acc[1][i] = 0.f;
            for (int kc0 = k_begin; kc0 < k_end; kc0 += kSkinnyKChunk) {
                __syncthreads();
                stage_small<PITCH>(p, s_small, kc0, k_end, tid);
                __syncthreads();
#pragma unroll 1
                for (int ks = 0; ks < kSkinnyKChunk; ks += 256) {
                    const int k = kc0 + ks;
                    if (k >= k_end) break;
                    uint4 v[8];
                    if (k + 256 <= k_end) {
#pragma unroll
                        for (int j = 0; j < 8; ++j) {
                            v[j] = make_uint4(0, 0, 0, 0);
                            if (row_ok) v[j] = load8<ALIGNED>(row + k + 32 * j + 8 * t);
                        }
                    } else {
#pragma unroll
                        for (int j = 0; j < 8; ++j) {
                            const int nvk = k_end - (k + 32 * j + 8 * t);
                            v[j] = make_uint4(0, 0, 0, 0);
                            if (row_ok && nvk > 0) v[j] = nvk >= 8 ? load8<false>(row + k + 32 * j + 8 * t) : load8_edge(row + k + 32 * j + 8 * t, nvk);
                        }
                    }
#pragma unroll
                    for (int j = 0; j < 8; ++j) {
                        const int kl = ks + 32 * j + 8 * t;
                        const uint4 lo = *reinterpret_cast<const uint4*>(&s_small[g][kl]);
                        const uint4 hi = *reinterpret_cast<const uint4*>(&s_small[g + 8][kl]);
                        mma_16816<BF16>(acc[0], lo.x, hi.x, lo.y, hi.y, v[j].x, v[j].y);   // two independent chains
                        mma_16816<BF16>(acc[1], lo.z, hi.z, lo.w, hi.w, v[j].z, v[j].w);
                    }
                }
            }
            // acc[0][0..1]: Small row g, fragment columns 2t, 2t+1 (= rows r_pass + 8*warp + 2t, +1); [2..3]: row g+8
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const int s = g + ((i & 2) ? 8 : 0);
                const int rr = r_pass + 8 * warp + 2 * t + (i & 1);
                if (s >= p.ms || rr >= p.R) continue;
                const float sum = acc[0][i] + acc[1][i];
                if (p.P_k == 1) {
                    unsigned short h;
                    if (BF16) { __nv_bfloat16 b = __float2bfloat16_rn(sum); h = *reinterpret_cast<unsigned short*>(&b); }
                    else { __half b = __float2half_rn(sum); h = *reinterpret_cast<unsigned short*>(&b); }
                    p.C[(int64_t)s * p.out_ss + (int64_t)rr * p.out_sr] = h;
                } else {
                    p.partial[(int64_t)split * p.part_slab + (int64_t)s * p.part_ss + (int64_t)rr * p.part_sr] = sum;
                }
            }
        }
    }
}

typedef void (*SkinnyKernel)(const SkinnyParams);

template <bool KC>
inline SkinnyKernel skinny_pick(bool bf16, bool aligned)
{
    if (bf16) return aligned ? skinny_gemm_kernel<KC, true, true> : skinny_gemm_kernel<KC, true, false>;
    return aligned ? skinny_gemm_kernel<KC, false, true> : skinny_gemm_kernel<KC, false, false>;
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
        p.part_ss = partial_pitch(s.N); p.part_sr = 1;
    } else {
        // Small = B^T, streamed = A^T
        p.Small = (const unsigned short*)B;
        p.Str = (const unsigned short*)A;
        p.ms = (int)s.N; p.R = (int)s.M;
        if (s.layoutB == ADAPT_ROW_MAJOR) { p.small_ss = 1; p.small_sk = s.N; } else { p.small_ss = s.K; p.small_sk = 1; }
        kc = s.layoutA == ADAPT_ROW_MAJOR;
        p.ld = kc ? s.K : s.M;
        p.out_ss = 1; p.out_sr = s.N;
        p.part_ss = 1; p.part_sr = partial_pitch(s.N);
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
    p.part_slab = s.M * partial_pitch(s.N);
    // every group this kernel loads starts at Str + row * ld + (multiple of 8)
    const bool aligned = (p.ld % 8 == 0) && ((uintptr_t)p.Str % 16 == 0);
    dim3 grid((unsigned)ceil_div(p.R, p.BNs), (unsigned)c.P_k, 1);
    SkinnyKernel k = kc ? skinny_pick<true>(s.dtype != 0, aligned) : skinny_pick<false>(s.dtype != 0, aligned);
    if (launch_pdl(k, grid, dim3(kSkinnyThreads, 1, 1), 0, stream, p) != cudaSuccess) return ADAPT_ERR_CUDA;
    return ADAPT_OK;
}

}  // namespace adapt

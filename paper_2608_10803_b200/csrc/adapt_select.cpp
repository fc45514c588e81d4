// Host-side selector: taxonomy (Section 4.2), candidate enumeration with capacity checks
// (Eq. 6), analytical latency model (Eq. 7-11 with the schedules of Eq. 12-14) and the 64-bit
// TilingKey.  No CUDA here.
#include "adapt_internal.h"

#include <algorithm>
#include <cmath>

namespace adapt {

const Calib& default_calib()
{
    static Calib c;
    return c;
}

// ---- Section 4.2: two predicates, four templates ---------------------------------------------
int classify(int64_t M, int64_t N, int64_t m, int64_t n, int64_t m1, int64_t n1, int64_t n_core, int64_t acc_bytes)
{
    if (M < 1 || N < 1 || m < 1 || n < 1 || m1 < 1 || n1 < 1 || n_core < 1 || acc_bytes < 1) return -1;
    const int64_t P_m = ceil_div(M, m), P_n = ceil_div(N, n);
    const bool enough_tasks = P_m * P_n >= n_core;            // X axis: spatial parallelism
    const bool on_chip = m1 * n1 * 4 <= acc_bytes;            // Y axis: fp32 accumulation tile fits
    if (enough_tasks) return on_chip ? ADAPT_CLASS_COMMON : ADAPT_CLASS_SINGLE_CORE_SPLIT_K;
    return on_chip ? ADAPT_CLASS_MULTI_CORE_SPLIT_K : ADAPT_CLASS_HYBRID_SPLIT_K;
}

// ---- Eq. 1-5 ----------------------------------------------------------------------------------
double read_volume(int64_t M, int64_t N, int64_t K, int64_t m1, int64_t n1)
{
    return 2.0 * (double)M * (double)N * (double)K * (1.0 / (double)m1 + 1.0 / (double)n1);
}

double write_volume(int cls, int64_t M, int64_t N, int64_t K, int64_t k, int64_t k1)
{
    const double MN = (double)M * (double)N;
    switch (cls) {
        case ADAPT_CLASS_COMMON: return 2.0 * MN;
        case ADAPT_CLASS_SINGLE_CORE_SPLIT_K: return 4.0 * MN * (double)ceil_div(K, k1) + 2.0 * MN;
        case ADAPT_CLASS_MULTI_CORE_SPLIT_K: return 4.0 * MN * (double)ceil_div(K, k) + 2.0 * MN;
        case ADAPT_CLASS_HYBRID_SPLIT_K:
            return (double)ceil_div(K, k) * (4.0 * MN * (double)ceil_div(k, k1)) + 2.0 * MN;
        default: return -1.0;
    }
}

// ---- Eq. 12-14 --------------------------------------------------------------------------------
double pipeline_time(int schedule, int64_t Q, int64_t L, double tM, double tP, double Td)
{
    const double ii = std::max(tM, tP);
    switch (schedule) {
        case 0: return (double)Q * ((double)L * (tM + tP) + Td);                              // Eq. 12 per tile
        case 1: return (double)Q * (tM + (double)(L - 1) * ii + tP + Td);                     // Eq. 13 per tile
        case 2: return tM + ((double)Q * (double)L - 1.0) * ii + tP + (double)Q * Td;         // Eq. 14
        default: return -1.0;
    }
}

// ---- TilingKey --------------------------------------------------------------------------------
static int ilog2(int v) { int r = 0; while ((1 << (r + 1)) <= v) ++r; return r; }

uint64_t pack_tiling_key(const Shape& s, const Config& c)
{
    uint64_t k = 0;
    k |= (uint64_t)(c.cls & 3) << 62;
    k |= (uint64_t)(c.family & 7) << 59;
    k |= (uint64_t)((c.BM / 16) & 31) << 54;
    k |= (uint64_t)((c.BN / 16) & 63) << 48;
    k |= (uint64_t)(ilog2(std::max(c.BK, 16) / 16) & 3) << 46;
    k |= (uint64_t)(c.stages & 15) << 42;
    k |= (uint64_t)(c.P_k & 1023) << 32;
    k |= (uint64_t)(c.persistent & 1) << 31;
    k |= (uint64_t)(c.srcA & 3) << 29;
    k |= (uint64_t)(c.srcB & 3) << 27;
    k |= (uint64_t)(s.dtype & 1) << 26;
    k |= (uint64_t)(s.layoutA & 1) << 25;
    k |= (uint64_t)(s.layoutB & 1) << 24;
    k |= (uint64_t)(ilog2(std::max(c.cluster, 1)) & 3) << 22;
    k |= (uint64_t)((ilog2(std::max(c.cluster, 1)) >> 2) & 1) << 21;
    k |= (uint64_t)(c.fused & 1) << 20;
    k |= (uint64_t)(c.streamk & 1) << 19;
    return k;
}

bool unpack_tiling_key(uint64_t k, Shape* s, Config* c)
{
    if (k & ((1ull << 19) - 1)) return false;
    c->cls = (int)((k >> 62) & 3);
    c->family = (int)((k >> 59) & 7);
    c->BM = (int)((k >> 54) & 31) * 16;
    c->BN = (int)((k >> 48) & 63) * 16;
    c->BK = 16 << (int)((k >> 46) & 3);
    c->stages = (int)((k >> 42) & 15);
    c->P_k = (int)((k >> 32) & 1023);
    c->persistent = (int)((k >> 31) & 1);
    c->srcA = (int)((k >> 29) & 3);
    c->srcB = (int)((k >> 27) & 3);
    s->dtype = (int)((k >> 26) & 1);
    s->layoutA = (int)((k >> 25) & 1);
    s->layoutB = (int)((k >> 24) & 1);
    c->cluster = 1 << (int)(((k >> 22) & 3) | (((k >> 21) & 1) << 2));
    c->fused = (int)((k >> 20) & 1);
    c->streamk = (int)((k >> 19) & 1);
    return true;
}

// ---- model --------------------------------------------------------------------------------------

static const double kL2Bytes = 96e6;       // share of the 126 MB L2 one operand can expect to keep
static const int kGroupM = 16;             // tile rasterisation: m-blocks per group (matches the kernel)

static double copy_time_us(double bytes, const Calib& cal)
{
    return bytes / (cal.hbm_bw * cal.copy_bw_eff) * 1e6;
}

// Inner extent (contiguous dimension) of each operand in elements.
static int64_t innerA(const Shape& s) { return s.layoutA == ADAPT_ROW_MAJOR ? s.K : s.M; }
static int64_t outerA(const Shape& s) { return s.layoutA == ADAPT_ROW_MAJOR ? s.M : s.K; }
static int64_t innerB(const Shape& s) { return s.layoutB == ADAPT_ROW_MAJOR ? s.N : s.K; }
static int64_t outerB(const Shape& s) { return s.layoutB == ADAPT_ROW_MAJOR ? s.K : s.N; }

// Group of a configuration for the last calibration factor: kernel family, tiling mode, and which extra launches
// (prologue, reduction) or in-kernel exchanges (fused reduction, stream-K) it has.  Pair tiles: + 20.
int calib_group(const Config& c)
{
    const bool pro = c.srcA == ADAPT_SRC_PAD_COPY || c.srcB == ADAPT_SRC_PAD_COPY;
    int g;
    switch (c.family) {
        case ADAPT_FAM_SKINNY: return c.P_k == 1 ? 13 : 14;
        case ADAPT_FAM_SIMT: return c.P_k == 1 ? 15 : 16;
        case ADAPT_FAM_CLUSTER: return c.cluster == 1 ? 17 : 18;
        default: break;
    }
    if (c.srcB == ADAPT_SRC_TMA_CLASSES) g = c.BN == 64 ? 10 : (c.fused ? 12 : 11);
    else if (c.srcA == ADAPT_SRC_TMA_CLASSES) g = c.BN % 64 ? 9 : (c.fused ? 8 : (c.P_k == 1 ? 6 : 7));
    else if (c.fused) g = 4;
    else if (c.streamk) g = 5;
    else g = (c.P_k == 1 ? 0 : 2) + (pro ? 1 : 0);
    return g + (c.family == ADAPT_FAM_UMMA_2CTA ? 20 : 0);
}

static void finish_common(const Shape& s, Config& c, const Calib& cal)
{
    c.workspace_bytes = c.ws_padA + c.ws_padB + c.ws_partial;
    c.predicted_us = (cal.launch_us + c.t_pro_us + c.t_main_us + c.t_epi_us) * cal.group_bias[calib_group(c)];
    (void)s;
}

// Prologue (Section 5.2 "Prologue"): the Padding module re-pitches an operand whose rows are not
// 16-byte multiples (or, for a narrow operand, not whole 32-byte sectors), reading it once and writing the padded copy once.
static void model_prologue(const Shape& s, Config& c, const Calib& cal)
{
    c.t_pro_us = 0;
    c.ws_padA = c.ws_padB = 0;
    if (c.srcB == ADAPT_SRC_TMA_CLASSES) {
        // k-class mode: A is regrouped class-major (element-wise reads, 16-byte writes); B is read in place
        const double src = 2.0 * (double)s.M * (double)s.K;
        c.ws_padA = round_up(s.M * 8 * round_up(ceil_div(s.K, 8), 64) * 2, 256);
        c.t_pro_us += cal.prologue_launch_us + (src + (double)c.ws_padA) / (cal.hbm_bw * cal.regroup_bw_eff) * 1e6;
        c.hbm_bytes += src + (double)c.ws_padA;
        return;
    }
    // (class tiles read a narrow A, whose rows are fractions of a sector, over a sector-pitched copy too)
    if (c.srcA == ADAPT_SRC_PAD_COPY || (c.srcA == ADAPT_SRC_TMA_CLASSES && class_tiles_copy_a(s))) {
        const double src = 2.0 * (double)s.M * (double)s.K;
        c.ws_padA = round_up(outerA(s) * padded_pitch(innerA(s)) * 2, 256);
        c.t_pro_us += cal.prologue_launch_us + copy_time_us(src + (double)c.ws_padA, cal);
        c.hbm_bytes += src + (double)c.ws_padA;
    }
    if (c.srcB == ADAPT_SRC_PAD_COPY) {
        const double src = 2.0 * (double)s.K * (double)s.N;
        c.ws_padB = round_up(outerB(s) * padded_pitch(innerB(s)) * 2, 256);
        // both operands re-pitched: one launch does both
        c.t_pro_us += (c.ws_padA != 0 ? 0.0 : cal.prologue_launch_us) + copy_time_us(src + (double)c.ws_padB, cal);
        c.hbm_bytes += src + (double)c.ws_padB;
    }
}

// Epilogue (Eq. 11): cross-CTA reduction of the fp32 partials (Eq. 4's extra 4*M*N*P_k bytes are
// written by the main loop and read back here), then the single 16-bit write.
static void model_epilogue(const Shape& s, Config& c, const Calib& cal)
{
    c.t_epi_us = 0;
    c.ws_partial = 0;
    if (c.streamk) {
        // one fp32 partial tile per CTA, written and read back once at most (they stay in L2); no second launch
        c.ws_partial = (int64_t)c.grid * 128 * c.BN * 4;
        return;
    }
    if (c.fused) {
        // Eq. 11 with the cross-core exchange on chip: each CTA reads one tile's worth of fp32 partials from its
        // peers' shared memory (its share of the rows over all ranks); no second launch, no workspace
        // (its time is the tile drain of the main kernel, so nothing is added here)
        c.hbm_bytes += 2.0 * (double)s.M * (double)s.N;
        return;
    }
    if (c.P_k > 1) {
        const double MN = (double)s.M * (double)s.N;
        c.ws_partial = round_up((int64_t)c.P_k * s.M * partial_pitch(s.N) * 4, 256);
        double part = 4.0 * MN * c.P_k;
        // partials that fit in L2 are read back at L2 speed; model that as half the HBM cost
        const double factor = part <= kL2Bytes ? 0.5 : 1.0;
        // the reduction kernel walks the P_k slabs eight at a time: one dependent trip to L2 / HBM per batch
        c.t_epi_us = cal.reduce_launch_us + copy_time_us(part * factor + 2.0 * MN, cal) + cal.reduce_batch_us * (double)ceil_div(c.P_k, 8);
        c.hbm_bytes += part * (1.0 + factor);
    }
}

static void model_umma(const Shape& s, const Machine& m, const Calib& cal, Config& c)
{
    const bool kclasses = c.srcB == ADAPT_SRC_TMA_CLASSES;
    const int64_t kblocks = kclasses ? ceil_div(ceil_div(s.K, 8), c.BK)
                                     : ceil_div(s.K + (c.srcA == ADAPT_SRC_TMA_CLASSES ? class_k_slack(s) : 0), c.BK);
    const bool ksplit_cls = kclasses && c.BN != 64;                       // each class a k split of its own
    const int64_t L = ksplit_cls ? ceil_div(kblocks, c.P_k / 8)
                                 : ceil_div(kblocks, c.P_k) * (kclasses ? 8 : 1);   // BN = 64: the split's blocks of all 8 classes
    // fused split-K: a tile is a cluster of P_k CTAs, and only so many clusters of that size run at a time
    const int64_t units = c.fused ? (int64_t)c.P_m * c.P_n : (int64_t)c.P_m * c.P_n * c.P_k;
    const int64_t slots = c.fused ? umma_cluster_slots(m, c.P_k) : m.n_sm / c.cluster;
    const int64_t Q = ceil_div(units, slots);
    c.grid = c.streamk ? (int)(slots * c.cluster) : (int)(std::min(units, slots) * (c.fused ? c.P_k : c.cluster));

    const double MK = (double)s.M * s.K, KN = (double)s.K * s.N, MN = (double)s.M * s.N;
    // HBM traffic: operands once, plus re-reads of B when it cannot stay in L2 across m-groups.
    double rB = 1.0, rA = 1.0;
    const int64_t rows_per_group = (int64_t)kGroupM * c.BM;
    if (2.0 * KN > kL2Bytes) rB = (double)ceil_div(s.M, rows_per_group);
    if (rB > 1.0 && 2.0 * MK <= kL2Bytes) {          // alternatively A stays resident and B streams once
        rB = 1.0;
    }
    c.hbm_bytes = 2.0 * (MK * rA + KN * rB * (kclasses ? c.BN / (c.BN - 8.0) : 1.0)) + (c.P_k > 1 ? 0.0 : 2.0 * MN);

    // per-SM stage: each CTA loads its 128 rows of A and its share of the BN columns of B
    const double bn_per_cta = (double)c.BN / c.cluster;
    const double a_rows = umma_a_box_rows(s, c.cluster, umma_row_classes(s, c.srcA, c.BN), kclasses);
    const double stage_bytes = 2.0 * c.BK * (a_rows + (double)round_up((int64_t)bn_per_cta, 64));
    // One SM pulls operands that other SMs also use from L2 at l2_bw_per_sm (a little less through
    // the strided row-class views); a stream that comes from HBM and is used once is bounded by the
    // bytes one SM keeps in flight, about hbm_bw_per_sm.  The second case only shows in partial waves.
    const double t_mma_all = 2.0 * (double)s.M * s.N * s.K / cal.tensor_flops;
    const bool mem_bound = 2.0 * (MK * rA + KN * rB) / cal.hbm_bw > t_mma_all;   // the operand stream, not C, outweighs the MMAs
    double sm_rate = cal.l2_bw_per_sm * (c.srcA == ADAPT_SRC_TMA_CLASSES ? cal.class_view_sm_eff : (kclasses ? cal.kclass_view_sm_eff : 1.0));
    if (mem_bound && c.srcA == ADAPT_SRC_TMA_CLASSES) sm_rate = std::min(sm_rate, cal.hbm_bw_per_sm);   // measured for the views only
    double tM = stage_bytes / sm_rate * 1e6;
    // relative tensor efficiency, measured at BN = 64, 128, 256 and interpolated for the halo tiles between them
    double eta = c.BN >= 256 ? 1.0
               : c.BN >= 128 ? cal.eta_mma_bn128 + (1.0 - cal.eta_mma_bn128) * (c.BN - 128) / 128.0
                             : cal.eta_mma_bn64 + (cal.eta_mma_bn128 - cal.eta_mma_bn64) * (c.BN - 64) / 64.0;
    if (c.cluster == 2) eta *= cal.eta_2cta;
    const double tP = 2.0 * 128.0 * c.BN * c.BK / (cal.tensor_flops / m.n_sm * eta) * 1e6;
    // Drain of one tile (the paper's T_drain: FixPipe cast and write).  With two or more TMEM
    // accumulators it overlaps the next tile's main loop, so a tile costs max(L * II, T_drain).
    // 16-bit tiles leave through TMA stores when C's rows are 16-byte aligned, or when class tiles with
    // halo columns make their misalignment uniform; otherwise the epilogue threads store them, and fp32
    // partials always go that way
    const bool halo = c.BN % 64 != 0;
    const int own_n = halo ? c.BN - 16 : c.BN;
    // rows of a tile that exist (short M: the rest is neither stored by the threads nor by TMA)
    const double rows_valid = std::min(128.0, (double)s.M / ((double)c.P_m * c.cluster));
    const double out_tile_kb = (c.P_k > 1 ? 4.0 : 2.0) * rows_valid * own_n / 1024.0;
    double t_drain;
    if (c.fused) t_drain = cal.fused_reduce_us + 4.0 * rows_valid * c.BN / cal.dsmem_bw_per_sm * 1e6;   // exchange + reduce + store, per tile
    else if (c.P_k > 1) t_drain = cal.epi_partial_fixed_us + cal.epi_partial_us_per_kb * out_tile_kb;
    else if (s.N % 16 == 0 || halo) t_drain = cal.epi_tile_fixed_us + cal.epi_us_per_kb * out_tile_kb;
    else if (s.N % 8 == 0) t_drain = cal.epi_partial_fixed_us + cal.epi_partial_us_per_kb * out_tile_kb;   // aligned 16-byte stores by the threads
    else t_drain = cal.epi_tile_fixed_unaligned_us + cal.epi_us_per_kb_unaligned * out_tile_kb;
    // the two CTAs of a pair hand their accumulator back together: a drain-bound pair waits for its slower half
    if (c.cluster == 2) t_drain *= cal.pair_drain_factor;
    // Delta_dep (Eq. 9): with S stages only S-1 loads are in flight while one is consumed, so a
    // slice cannot issue faster than latency / (S-1); one stage serialises load and compute.
    double pipe;
    if (c.stages <= 1) {
        pipe = pipeline_time(0, Q, L, tM + cal.mem_latency_us, tP, t_drain);                  // Eq. 12
    } else {
        // a stream that comes from HBM sees the loaded-memory latency, not the L2 one
        const bool views = c.srcA == ADAPT_SRC_TMA_CLASSES || kclasses;
        tM = std::max(tM, (mem_bound ? (views ? cal.hbm_latency_views_us : cal.hbm_latency_us) : cal.mem_latency_us) / (c.stages - 1));
        const double ii = std::max(tM, tP);
        // class tiles pay a fixed cost per tile (strided row views; zeroing the heads of an unaligned A)
        // (the bubble between the units of a k class shrinks as the unit's main loop grows)
        const double t_fixed = ksplit_cls ? std::max(0.0, cal.kclass_unit_fixed_us - 0.2 * (double)L * ii)
                             : c.srcA != ADAPT_SRC_TMA_CLASSES ? 0.0
                             : (s.K % 8 ? cal.class_tile_fixed_unaligned_us + (c.cluster == 2 ? cal.pair_class_tile_us : 0.0) : cal.class_tile_fixed_us);
        // eight k-class accumulators fill TMEM: one tile at a time, its drain (eight-way sum, thread stores)
        // is not overlapped with the next tile's main loop
        const bool one_buffer = kclasses && !ksplit_cls;
        // a 16-bit tile that leaves through the epilogue threads (C's rows off 32-byte boundaries, no halo
        // tiles) hides only part of the next tile's main loop behind its drain (11601 x 25478 x 543: 7.7 us
        // per 128 x 256 tile with a 4.9 us drain and a 4 us main loop)
        const bool thread_store = c.P_k == 1 && !(s.N % 16 == 0 || halo);
        const double t_tile = one_buffer ? (double)L * ii + cal.kclass_tile_drain_us
                            : thread_store ? std::max((double)L * ii + t_fixed, t_drain + (c.cluster == 2 ? cal.thread_store_exposed_pair : cal.thread_store_exposed) * (double)L * ii)
                                           : std::max((double)L * ii + t_fixed, t_drain);
        // Eq. 14 with the drain overlapped: one fill, Q tiles back to back, the last drain exposed
        pipe = tM + (double)Q * t_tile + tP + t_drain;
        if (c.streamk) {
            // whole waves as above; the leftover tiles' k-blocks shared evenly by all slots, then the owners' fix-up
            // While a slot works on its share of the leftover tiles it is at a k position of its own: nothing it loads is
            // shared with the other slots at that moment, so all of them together pull slots x stage bytes per k-block
            // from HBM (8192^3: 74 pairs x 64 KB per 0.41 us = 11.5 TB/s asked for), and the shared part runs at that rate
            const StreamK sk = streamk_schedule(units, slots, L);
            const double shared = (double)(sk.q0 + (sk.rem ? 1 : 0));
            const double ii_shared = std::max(ii, (double)slots * c.cluster * stage_bytes / cal.hbm_bw * 1e6);
            pipe = tM + std::max((double)sk.waves * (double)L * ii + shared * ii_shared + (double)(sk.waves + 1) * t_fixed,
                                 (double)(sk.waves + 2) * t_drain) + tP + t_drain + cal.streamk_fixup_us +
                   cal.streamk_peer_us * (double)L / (double)std::max<int64_t>(1, sk.q0);
        }
    }
    pipe += cal.umma_fixed_us;
    if (c.fused) pipe += cal.fused_wave_us * (double)(Q - 1);
    // halo tiles: the first and the last tile of a row block write the elements before the first and after
    // the last whole 32-byte unit of each row with narrow stores (48618 x 28 x 115: 384 such tiles)
    if (halo && c.P_k == 1)
        pipe += 2.0 * cal.halo_edge_tile_us * (double)c.P_m / (double)std::min<int64_t>(m.n_sm, (int64_t)c.P_m * c.P_n);
    model_prologue(s, c, cal);
    model_epilogue(s, c, cal);
    // strided row-class views stream A at a lower rate than a dense tensor (measured 3.5-4.1 TB/s)
    // (k classes as splits: the rate falls as the regrouped A, re-read by every column of tiles, grows beside the B
    // stream: 0.93 of the copy rate at M = 1, 0.80 at M = 30, 0.70 at M = 80; with the eight classes of a tile as
    // one cluster it stays near 0.87)
    const double split_eff = c.fused ? cal.class_split_fused_bw_eff
                                     : std::max(0.6, cal.class_split_bw_eff - cal.class_split_bw_eff_per_log2m * std::log2((double)std::max<int64_t>(1, s.M)));
    const double bw = ksplit_cls ? cal.hbm_bw * split_eff
                    : (c.srcA == ADAPT_SRC_TMA_CLASSES || kclasses) ? cal.hbm_bw * cal.class_view_bw_eff : cal.hbm_bw;
    // A row-major B arrives as k-rows of BN contiguous columns per tile: short pieces stream below the
    // HBM rate (8 x 30016 x 40000: 3.6 / 5.5 / 6.9 TB/s at 128 / 256 / 512 bytes)
    double t_b_extra = 0.0;
    if (s.layoutB == ADAPT_ROW_MAJOR) {
        const double piece = 2.0 * c.BN;
        const double eff = piece >= 512 ? 1.0 : (piece >= 256 ? 0.8 + 0.2 * (piece - 256) / 256 : 0.52 + 0.28 * (piece - 128) / 128);
        const double b_bytes = 2.0 * KN * rB * (kclasses ? c.BN / (c.BN - 8.0) : 1.0);
        t_b_extra = b_bytes / bw * (1.0 / std::max(eff, 0.3) - 1.0) * 1e6;
    }
    const double t_hbm = c.hbm_bytes / bw * 1e6 + t_b_extra - c.t_pro_us - c.t_epi_us;
    c.t_main_us = std::max(pipe, t_hbm);
    // boxes of B that lie wholly beyond N are fetched all the same (zero fill): a tile narrower than BN pays
    // for them in TMA work the terms above do not see (61370 x 32 x 85272: BN 128 -> 64 is 20 % faster)
    if (s.layoutB == ADAPT_ROW_MAJOR && !kclasses) {
        const int64_t loaded = c.cluster * ceil_div(c.BN / c.cluster, 64), needed = ceil_div(std::min<int64_t>(s.N, c.BN), 64);
        c.t_main_us *= 1.0 + cal.oob_box_penalty * (double)std::max<int64_t>(0, loaded - needed) / c.cluster;
    }
    finish_common(s, c, cal);
}

static void model_skinny(const Shape& s, const Machine& m, const Calib& cal, Config& c)
{
    const double MK = (double)s.M * s.K, KN = (double)s.K * s.N, MN = (double)s.M * s.N;
    c.hbm_bytes = 2.0 * (MK + KN) + (c.P_k > 1 ? 0.0 : 2.0 * MN);
    const int64_t units = (int64_t)c.P_m * c.P_n * c.P_k;
    c.grid = (int)units;
    const int64_t Q = ceil_div(units, (int64_t)m.n_sm * 2);      // two CTAs resident per SM
    const double macs = (double)std::max(s.M, s.N) * s.K * 16.0;  // the small side is padded to 16
    // the streamed operand: B when M is the small side, else A; its rows are aligned when the
    // contiguous extent is a multiple of 8 elements
    const bool stream_is_B = s.M <= 16 && (s.M <= s.N || s.N > 16);
    const int64_t inner = stream_is_B ? (s.layoutB == ADAPT_ROW_MAJOR ? s.N : s.K) : (s.layoutA == ADAPT_ROW_MAJOR ? s.K : s.M);
    const double eff = inner % 8 == 0 ? cal.skinny_bw_eff_aligned : cal.skinny_bw_eff_unaligned;
    // one CTA streams about hbm_bw * eff / (2 * n_sm) when the machine is full; fewer CTAs do not go faster
    const double per_cta_bytes = 2.0 * ((double)c.BN * ceil_div(s.K, c.P_k));
    double t_cta = per_cta_bytes / (cal.hbm_bw * eff / (2.0 * m.n_sm)) * 1e6;
    // unaligned rows are assembled from two dependent loads per k step: a CTA cannot go faster than that
    // chain however few bytes it moves (3 x 98900 x 115: 28 us per CTA)
    const bool k_is_outer = stream_is_B ? s.layoutB == ADAPT_ROW_MAJOR : s.layoutA == ADAPT_COL_MAJOR;   // one streamed row per k
    if (inner % 8 != 0 && k_is_outer) {
        // Unaligned rows, one per k: the 8 warps of a CTA tile BN columns by 64 and share the k range among
        // the rest in steps of 16; a step is a chain of dependent loads (about 2 us).  Within one staged
        // chunk that chain is the whole cost (3 x 98900 x 115: 20 us); the bandwidth term above was
        // measured on long k ranges and stays the floor there.
        const int64_t k_split = ceil_div(s.K, c.P_k);
        const int64_t wk = std::max<int64_t>(1, 8 / std::max(1, c.BN / 64));
        const int64_t steps = round_up(ceil_div(std::min<int64_t>(k_split, kSkinnyKChunk), wk), 16) / 16 *
                              ceil_div(k_split, kSkinnyKChunk);
        const double t_chain = cal.skinny_step_unaligned_us * (double)steps;
        t_cta = k_split <= kSkinnyKChunk ? t_chain : std::max(t_cta, t_chain);
    }
    if (!k_is_outer) {
        // k-contiguous stream: the CTA walks its rows in passes of 64, each a chain of dependent trips to
        // memory per staged chunk (89274 x 16 x 23: two passes per CTA, three waves, 27 us)
        const int64_t k_split = ceil_div(s.K, c.P_k);
        t_cta = std::max(t_cta, cal.skinny_pass_us * (double)(c.BN / 64) * (double)ceil_div(k_split, kSkinnyKChunk));
    }
    model_epilogue(s, c, cal);
    const double t_alu = macs / cal.skinny_mac_rate * 1e6;
    c.t_pro_us = 0;
    c.t_main_us = cal.skinny_fixed_us + std::max(t_alu, (double)Q * t_cta);
    finish_common(s, c, cal);
}

static void model_simt(const Shape& s, const Machine& m, const Calib& cal, Config& c)
{
    const double MK = (double)s.M * s.K, KN = (double)s.K * s.N, MN = (double)s.M * s.N;
    const int64_t units = (int64_t)c.P_m * c.P_n * c.P_k;
    c.grid = (int)units;
    c.hbm_bytes = 2.0 * (MK + KN) + (c.P_k > 1 ? 0.0 : 2.0 * MN);
    const int64_t resident = (int64_t)m.n_sm * 4;
    const int64_t Q = ceil_div(units, resident);
    // A full 64 x 64 tile costs the same whether or not the shape fills it.  One step of 16 k values is a
    // trip to memory for a CTA that has its SM to itself; CTAs that share an SM (up to 4) share its FMA rate
    // (4 per SM: 2 * 64 * 64 * 16 flops per step at simt_flops / (4 n_sm) per CTA)
    const double steps = (double)ceil_div(ceil_div(s.K, c.P_k), 16);
    const double crowd = std::min(4.0, (double)units / m.n_sm);
    const double t_step = std::max(cal.simt_step_us, crowd * 2.0 * 64 * 64 * 16 / (cal.simt_flops / m.n_sm) * 1e6);
    const double t_tile = steps * t_step + cal.simt_fixed_us;
    model_epilogue(s, c, cal);
    // element-wise 2-byte loads and stores: about a seventh of the HBM rate when memory-bound
    const double t_hbm = c.hbm_bytes / (cal.hbm_bw * cal.simt_bw_eff) * 1e6 - c.t_epi_us;
    c.t_pro_us = 0;
    c.t_main_us = std::max((double)Q * t_tile, t_hbm);
    finish_common(s, c, cal);
}

static bool aligned16(int64_t inner_elems);

static void model_cluster(const Shape& s, const Machine& m, const Calib& cal, Config& c)
{
    const double MK = (double)s.M * s.K, KN = (double)s.K * s.N, MN = (double)s.M * s.N;
    const int64_t tiles = (int64_t)c.P_m * c.P_n, units = tiles * c.cluster;
    c.grid = (int)units;
    // every tile row re-reads B and every tile column re-reads A, mostly from L2; HBM sees each once
    c.hbm_bytes = 2.0 * (MK + KN + MN);
    const int64_t k_cta = round_up(ceil_div(s.K, c.cluster), 16);
    const double stages = (double)ceil_div(k_cta, 64);
    // a cluster is placed inside one GPC, so clusters of 4, 8 and 16 leave SMs unused and fewer tiles run at a
    // time; two CTAs share an SM when their rings fit
    const int64_t at_a_time = cluster_slots(c.cluster, m.n_sm) * cluster_ctas_per_sm(c.stages, m.smem_bytes);
    const double waves = (double)ceil_div(tiles, at_a_time);
    // CTAs beyond one per two SMs start to share the load path
    const double crowd = std::max(0.0, (double)units / m.n_sm - 0.5);
    const double t_cta = cal.cluster_fixed_us + cal.cluster_stage_us * stages + (c.cluster > 1 ? cal.cluster_reduce_us : 0.0) +
                         crowd * (cal.cluster_crowd_us + cal.cluster_crowd_stage_us * stages) + cal.cluster_wave_us * (waves - 1.0);
    const double t_mem = c.hbm_bytes / (cal.hbm_bw * cal.cluster_bw_eff) * 1e6;
    c.t_pro_us = 0;
    c.t_epi_us = 0;
    c.t_main_us = std::max(t_cta, t_mem);
    finish_common(s, c, cal);
}

// ---- legality (the constraint M(b,x,s) <= C_limit of Eq. 6) -----------------------------------

static bool aligned16(int64_t inner_elems) { return inner_elems % 8 == 0; }

static bool legal_umma(const Shape& s, const Machine& m, Config& c)
{
    if (!(m.family_mask & (1u << c.family))) return false;
    if (c.BK != 64) return false;
    if (c.family == ADAPT_FAM_UMMA_1CTA) {
        if (c.BM != 128 || c.cluster != 1) return false;
        const bool halo_bn = c.BN == 80 || c.BN == 144 || c.BN == 208;    // class tiles: 64 / 128 / 192 owned + 16 halo columns
        if (c.BN != 64 && c.BN != 128 && c.BN != 256 && !halo_bn) return false;
        if (halo_bn && (c.srcA != ADAPT_SRC_TMA_CLASSES || s.N % 16 == 0 || s.M < 16)) return false;
    } else {
        if (c.BM != 256 || c.cluster != 2) return false;
        const bool halo_bn = c.BN == 144 || c.BN == 208;                  // pair class tiles: 128 / 192 owned + 16 halo columns
        if (c.BN != 128 && c.BN != 256 && !halo_bn) return false;
        if (halo_bn && (c.srcA != ADAPT_SRC_TMA_CLASSES || s.N % 16 == 0 || s.M < 32)) return false;
    }
    if (c.BN % 16 != 0 || c.BN > 256) return false;                 // UMMA shape rule for M = 128/256
    if (2 * c.BN > m.tmem_cols) return false;                       // at least two accumulator buffers in TMEM
    if (c.stages < 1 || c.stages > kUmmaMaxStages) return false;
    if (c.streamk) {
        // plain tiles, one split, not fused; needs leftover tiles and at least two k-blocks per slot in the shared part
        if (c.P_k != 1 || c.fused || c.srcA == ADAPT_SRC_TMA_CLASSES || c.srcB == ADAPT_SRC_TMA_CLASSES || c.stages < 2) return false;
    }
    const int a_rows_box = umma_a_box_rows(s, c.cluster, umma_row_classes(s, c.srcA, c.BN), c.srcB == ADAPT_SRC_TMA_CLASSES);
    if (c.fused) {
        // the k splits of a tile form one cluster: 1-CTA tiles, a portable cluster size, no halo tiles, not the
        // eight-accumulator k-class tiles
        if (c.family != ADAPT_FAM_UMMA_1CTA || (c.P_k != 2 && c.P_k != 4 && c.P_k != 8) || c.BN % 64 != 0) return false;
        if (c.srcB == ADAPT_SRC_TMA_CLASSES && c.BN == 64) return false;
    }
    c.smem_bytes = umma_smem_bytes(c.BN, c.cluster, c.stages, a_rows_box, c.P_k == 1, c.fused ? umma_fused_bytes(c.BN, a_rows_box) : 0);
    if (c.smem_bytes > m.smem_bytes) return false;
    // in class mode the k index of a tile is shifted by up to 7 elements
    // k-class mode splits the blocks of one class; in row-class mode the k index is shifted by up to 7
    const int64_t kblocks = c.srcB == ADAPT_SRC_TMA_CLASSES ? ceil_div(ceil_div(s.K, 8), c.BK)
                                                              : ceil_div(s.K + (c.srcA == ADAPT_SRC_TMA_CLASSES ? class_k_slack(s) : 0), c.BK);
    // k classes as k splits (k-class views of B with BN > 64): P_k = 8 * (splits of one class's blocks)
    const bool ksplit_cls = c.srcB == ADAPT_SRC_TMA_CLASSES && c.BN != 64;
    if (ksplit_cls && c.P_k % 8 != 0) return false;
    const int64_t pk_blocks = ksplit_cls ? c.P_k / 8 : c.P_k;
    if (c.P_k < 1 || c.P_k > 1023 || pk_blocks > kblocks) return false;
    if (ceil_div(kblocks, ceil_div(kblocks, pk_blocks)) != pk_blocks) return false;   // no empty split
    // operand sources: TMA needs a 16-byte row pitch
    if (c.srcA == ADAPT_SRC_TMA && !tma_friendly(innerA(s))) return false;
    if (c.srcB == ADAPT_SRC_TMA && !tma_friendly(innerB(s))) return false;
    if (c.srcA == ADAPT_SRC_LSU || c.srcB == ADAPT_SRC_LSU) return false;
    const bool classes = c.srcA == ADAPT_SRC_TMA_CLASSES;
    const bool kclasses = c.srcB == ADAPT_SRC_TMA_CLASSES;
    if (kclasses) {
        // k-rows of one residue class share their misalignment: row-major B with N % 8 != 0, 64-column
        // windows that own 56 columns, A regrouped class-major by a prologue copy (any layout of A)
        // (BN = 64: eight class accumulators per tile; BN = 128, 256: each class a k split, BN - 8 columns owned)
        if (s.layoutB != ADAPT_ROW_MAJOR || c.BN % 64 != 0) return false;
        if (c.family != ADAPT_FAM_UMMA_1CTA && c.BN != 256) return false;    // pair tiles: classes as k splits, 256 columns
        if (aligned16(innerB(s)) || s.K < 64 || c.srcA != ADAPT_SRC_PAD_COPY) return false;
    }
    if (classes) {
        // rows of one residue class share their misalignment: row-major A and B; pair tiles hold 256 rows of one class
        // (with halo columns: 128 or 192 owned columns)
        if (s.layoutA != ADAPT_ROW_MAJOR || s.layoutB != ADAPT_ROW_MAJOR) return false;
        if (c.family != ADAPT_FAM_UMMA_1CTA && (c.BN == 80 || s.M < (c.BN % 64 ? 32 : 16))) return false;
        // they pay when A's rows are unaligned (no copy), or when C's rows do not start on 32-byte sector
        // boundaries (halo tiles of 16 classes: uniform misalignment per tile, whole-sector TMA stores)
        if ((aligned16(innerA(s)) && c.BN % 64 == 0) || s.M < 8) return false;
    }
    if (c.srcA == ADAPT_SRC_PAD_COPY && tma_friendly(innerA(s)) && !kclasses) return false;    // nothing to pad
    if (c.srcB == ADAPT_SRC_PAD_COPY && tma_friendly(innerB(s))) return false;
    const int ncls = umma_row_classes(s, c.srcA, c.BN);
    c.P_m = classes ? (int)(ncls * ceil_div(s.M, ncls * c.BM)) : (int)ceil_div(s.M, c.BM);   // class tiles: 8 per 1024 rows (pair tiles: per 2048), 16 per 2048
    c.P_n = (int)ceil_div(s.N, kclasses ? c.BN - 8 : (c.BN % 64 ? c.BN - 16 : c.BN));
    if ((int64_t)c.P_m * c.P_n * c.P_k > (int64_t)1 << 30) return false;
    if (c.streamk) {
        const int64_t kb = ceil_div(s.K, c.BK);
        const StreamK sk = streamk_schedule((int64_t)c.P_m * c.P_n, m.n_sm / c.cluster, kb);
        // at most about eight slots per shared tile: its owner adds their partials one after the other
        // (and a k range long enough to carry the fix-up: with 8 or 9 k-blocks it cost 5 to 20 % on seven of nine sweep shapes)
        if (sk.sk_tiles == 0 || sk.q0 < 2 || kb < 32 || sk.q0 * 8 < kb) return false;
    }
    c.persistent = 1;
    return true;
}

static bool legal_skinny(const Shape& s, const Machine& m, Config& c)
{
    if (!(m.family_mask & (1u << ADAPT_FAM_SKINNY))) return false;
    if (std::min(s.M, s.N) > 16) return false;
    if (c.BM != 16 || c.BK != 16 || c.cluster != 1) return false;
    if (c.BN != 128 && c.BN != 256 && c.BN != 512) return false;     // streamed rows/columns per CTA
    if (c.srcA != ADAPT_SRC_LSU || c.srcB != ADAPT_SRC_LSU) return false;
    if (c.stages != 1) return false;
    const int64_t ksteps = ceil_div(s.K, kSkinnyKChunk);             // splits are whole staging chunks
    if (c.P_k < 1 || c.P_k > 1023 || c.P_k > ksteps) return false;
    if (ceil_div(ksteps, ceil_div(ksteps, c.P_k)) != c.P_k) return false;
    c.P_m = 1;
    c.P_n = (int)ceil_div(std::max(s.M, s.N), c.BN);
    c.persistent = 0;
    c.smem_bytes = 0;
    return true;
}

static bool legal_simt(const Shape& s, const Machine& m, Config& c)
{
    if (!(m.family_mask & (1u << ADAPT_FAM_SIMT))) return false;
    if (c.BM != 64 || c.BN != 64 || c.BK != 16 || c.cluster != 1 || c.stages != 1) return false;
    if (c.srcA != ADAPT_SRC_LSU || c.srcB != ADAPT_SRC_LSU) return false;
    const int64_t kblocks = ceil_div(s.K, c.BK);
    if (c.P_k < 1 || c.P_k > 1023 || c.P_k > kblocks) return false;
    if (ceil_div(kblocks, ceil_div(kblocks, c.P_k)) != c.P_k) return false;
    c.P_m = (int)ceil_div(s.M, c.BM);
    c.P_n = (int)ceil_div(s.N, c.BN);
    if ((int64_t)c.P_m * c.P_n > (int64_t)1 << 30) return false;
    c.persistent = 0;
    c.smem_bytes = 0;
    return true;
}

static bool legal_cluster(const Shape& s, const Machine& m, Config& c)
{
    if (!(m.family_mask & (1u << ADAPT_FAM_CLUSTER))) return false;
    if (c.BM != 64 || c.BN != 64 || c.BK != 64) return false;
    if (c.cluster != 1 && c.cluster != 2 && c.cluster != 4 && c.cluster != 8 && c.cluster != 16) return false;
    if (c.P_k != c.cluster || c.cluster > m.max_cluster) return false;    // the k splits are the cluster's CTAs
    if (c.srcA != ADAPT_SRC_LSU || c.srcB != ADAPT_SRC_LSU) return false;
    if ((c.cluster - 1) * round_up(ceil_div(s.K, c.cluster), 16) >= s.K) return false;   // no CTA without k values
    c.P_m = (int)ceil_div(s.M, c.BM);
    c.P_n = (int)ceil_div(s.N, c.BN);
    // a kernel for problems of a few microseconds: at most two CTAs per SM in all
    if ((int64_t)c.P_m * c.P_n * c.cluster > 2 * (int64_t)m.n_sm) return false;
    if (c.stages != cluster_ring(s.K, c.cluster, (int64_t)c.P_m * c.P_n, m.n_sm)) return false;
    c.persistent = 0;
    c.smem_bytes = cluster_smem_bytes(c.stages);
    return true;
}

static bool finalize(const Shape& s, const Machine& m, const Calib& cal, Config& c)
{
    bool ok = false;
    switch (c.family) {
        case ADAPT_FAM_UMMA_1CTA:
        case ADAPT_FAM_UMMA_2CTA: ok = legal_umma(s, m, c); break;
        case ADAPT_FAM_SKINNY: ok = legal_skinny(s, m, c); break;
        case ADAPT_FAM_SIMT: ok = legal_simt(s, m, c); break;
        case ADAPT_FAM_CLUSTER: ok = legal_cluster(s, m, c); break;
        default: ok = false;
    }
    if (!ok) return false;
    // taxonomy label: X axis from the spatial task count, Y axis from the fp32 tile against one
    // SM's accumulator budget (half of TMEM, so that two accumulators can alternate)
    const int64_t acc_budget = (int64_t)128 * (m.tmem_cols / 2) * 4;
    const bool enough = (int64_t)c.P_m * c.P_n >= m.n_sm;
    const bool on_chip = (int64_t)c.BM * c.BN * 4 <= acc_budget || c.family >= ADAPT_FAM_SKINNY;
    c.cls = enough ? (on_chip ? ADAPT_CLASS_COMMON : ADAPT_CLASS_SINGLE_CORE_SPLIT_K)
                   : (on_chip ? ADAPT_CLASS_MULTI_CORE_SPLIT_K : ADAPT_CLASS_HYBRID_SPLIT_K);
    switch (c.family) {
        case ADAPT_FAM_UMMA_1CTA:
        case ADAPT_FAM_UMMA_2CTA: model_umma(s, m, cal, c); break;
        case ADAPT_FAM_SKINNY: model_skinny(s, m, cal, c); break;
        case ADAPT_FAM_CLUSTER: model_cluster(s, m, cal, c); break;
        default: model_simt(s, m, cal, c); break;
    }
    if (c.workspace_bytes > m.workspace_limit) return false;
    return true;
}

// P_k candidates: 1, and when the spatial tasks leave SMs idle, the counts that bring the grid to
// about one or two CTAs per slot, plus powers of two in between.
static void split_candidates(int64_t tiles_mn, int64_t slots, int64_t ksteps, int64_t min_steps, std::vector<int>* out)
{
    out->clear();
    out->push_back(1);
    if (tiles_mn >= 4 * slots) return;
    const int64_t max_pk = std::min<int64_t>(1023, ksteps / std::max<int64_t>(1, min_steps));
    std::vector<int64_t> want;
    for (int64_t mult = 1; mult <= 4; mult *= 2) {
        want.push_back(mult * slots / tiles_mn);
        want.push_back(ceil_div(mult * slots, tiles_mn));
    }
    for (int64_t p = 2; p <= 1024; p *= 2) want.push_back(p);
    want.push_back(3); want.push_back(6); want.push_back(12); want.push_back(24);
    // split counts that fill whole waves: the smallest few with at most 3 % of the last wave idle
    int balanced = 0;
    for (int64_t w = 2; w <= std::min<int64_t>(max_pk, 96) && balanced < 3; ++w) {
        const int64_t units = tiles_mn * w, waves = ceil_div(units, slots);
        if ((double)units >= 0.97 * (double)(waves * slots)) { want.push_back(w); ++balanced; }
    }
    for (int64_t w : want) {
        if (w < 2 || w > max_pk) continue;
        // normalise so that no split is empty
        const int64_t per = ceil_div(ksteps, w);
        const int p = (int)ceil_div(ksteps, per);
        if (p >= 2 && std::find(out->begin(), out->end(), p) == out->end()) out->push_back(p);
    }
    std::sort(out->begin(), out->end());
}

void enumerate_configs(const Shape& s, const Machine& m, const Calib& cal, std::vector<Config>* out)
{
    out->clear();
    if (s.M < 1 || s.N < 1 || s.K < 1) return;
    std::vector<int> pks;
    // --- tcgen05 families ---
    // in place when TMA reads the rows well (16-byte multiples; narrow operands: whole sectors), else over a re-pitched copy
    const int srcA = tma_friendly(innerA(s)) ? ADAPT_SRC_TMA : ADAPT_SRC_PAD_COPY;
    const int srcB = tma_friendly(innerB(s)) ? ADAPT_SRC_TMA : ADAPT_SRC_PAD_COPY;
    for (int fam = ADAPT_FAM_UMMA_1CTA; fam <= ADAPT_FAM_UMMA_2CTA; ++fam) {
        const int BM = fam == ADAPT_FAM_UMMA_1CTA ? 128 : 256;
        const int cluster = fam == ADAPT_FAM_UMMA_1CTA ? 1 : 2;
        for (int BN : {64, 128, 256}) {
            const int64_t tiles = ceil_div(s.M, BM) * ceil_div(s.N, BN);
            split_candidates(tiles, m.n_sm / cluster, ceil_div(s.K, 64), 2, &pks);
            // ring depth: the deepest that fits, and a double buffer (Eq. 13) for comparison
            const int a_rows = umma_a_box_rows(s, cluster, 0, false);
            for (int pk : pks) {
                int deepest = umma_deepest_ring(BN, cluster, a_rows, pk == 1, m.smem_bytes);
                if (a_rows == 128 && deepest > 8) deepest = 8;
                std::vector<int> depths = {deepest};
                if (deepest > 4) depths.push_back(4);
                if (deepest > 2) depths.push_back(2);
                for (int st : depths) {
                    Config c;
                    c.family = fam; c.BM = BM; c.BN = BN; c.BK = 64; c.cluster = cluster;
                    c.stages = st; c.P_k = pk; c.srcA = srcA; c.srcB = srcB;
                    if (st >= 2 && finalize(s, m, cal, c)) out->push_back(c);
                }
                // one split, the leftover wave shared by all slots (stream-K)
                if (pk == 1) {
                    Config c;
                    c.family = fam; c.BM = BM; c.BN = BN; c.BK = 64; c.cluster = cluster; c.streamk = 1;
                    c.stages = deepest; c.P_k = 1; c.srcA = srcA; c.srcB = srcB;
                    if (deepest >= 2 && finalize(s, m, cal, c)) out->push_back(c);
                }
                // the same split with its reduction fused into the launch (the splits of a tile as one cluster)
                if (fam == ADAPT_FAM_UMMA_1CTA && (pk == 2 || pk == 4 || pk == 8)) {
                    Config c;
                    c.family = fam; c.BM = BM; c.BN = BN; c.BK = 64; c.cluster = cluster; c.fused = 1;
                    c.stages = umma_deepest_ring(BN, 1, a_rows, false, m.smem_bytes, a_rows == 128 ? 8 : kUmmaMaxStages, umma_fused_bytes(BN, a_rows));
                    c.P_k = pk; c.srcA = srcA; c.srcB = srcB;
                    if (c.stages >= 2 && finalize(s, m, cal, c)) out->push_back(c);
                }
            }
        }
    }
    // --- tcgen05, A read in place through per-row-class views (row-major A, K % 8 != 0): 8 class
    //     tiles per 1024 rows, so the split counts are drawn from that tile count ---
    const bool a_unaligned = !aligned16(innerA(s)), b_unaligned = !aligned16(innerB(s));
    if ((a_unaligned || s.N % 16 != 0) && s.layoutA == ADAPT_ROW_MAJOR && s.layoutB == ADAPT_ROW_MAJOR && s.M >= 8) {
        for (int BN : {64, 128, 256, 80, 144, 208}) {
            const bool halo = BN % 64 != 0;
            if (halo && (s.N % 16 == 0 || s.M < 16)) continue;             // halo tiles serve a C off 32-byte boundaries only
            if (!halo && !a_unaligned) continue;                           // aligned A: class tiles only for their stores
            const int hc = halo_row_classes(s);
            const int64_t tiles = (halo ? hc * ceil_div(s.M, 128 * hc) : 8 * ceil_div(s.M, 1024)) * ceil_div(s.N, halo ? BN - 16 : BN);
            split_candidates(tiles, m.n_sm, ceil_div(s.K + class_k_slack(s), 64), 2, &pks);
            for (int pk : pks) {
                const int deepest = umma_deepest_ring(BN, 1, umma_a_box_rows(s, 1, halo ? hc : 8, false), pk == 1, m.smem_bytes);
                Config d;
                d.family = ADAPT_FAM_UMMA_1CTA; d.BM = 128; d.BN = BN; d.BK = 64; d.cluster = 1;
                d.stages = deepest; d.P_k = pk; d.srcA = ADAPT_SRC_TMA_CLASSES; d.srcB = srcB;
                if (deepest >= 2 && finalize(s, m, cal, d)) out->push_back(d);
                if (!halo && (pk == 2 || pk == 4 || pk == 8)) {
                    const int rows = umma_a_box_rows(s, 1, 8, false);
                    Config f = d;
                    f.fused = 1;
                    f.stages = umma_deepest_ring(BN, 1, rows, false, m.smem_bytes, kUmmaMaxStages, umma_fused_bytes(BN, rows));
                    if (f.stages >= 2 && finalize(s, m, cal, f)) out->push_back(f);
                }
            }
        }
    }
    // --- the same row-class views on pair tiles (256 rows of one class per SM pair), for an A with unaligned rows ---
    //     ... and with halo columns (256 rows of one of 16 classes) for a C whose rows start off 32-byte boundaries
    if ((a_unaligned || s.N % 16 != 0) && s.layoutA == ADAPT_ROW_MAJOR && s.layoutB == ADAPT_ROW_MAJOR && s.M >= 16) {
        for (int BN : {128, 256, 144, 208}) {
            const bool halo = BN % 64 != 0;
            if (halo ? (s.N % 16 == 0 || s.M < 32) : !a_unaligned) continue;
            const int hc = halo_row_classes(s);
            const int64_t tiles = halo ? hc * ceil_div(s.M, 256 * hc) * ceil_div(s.N, BN - 16) : 8 * ceil_div(s.M, 2048) * ceil_div(s.N, BN);
            split_candidates(tiles, m.n_sm / 2, ceil_div(s.K + class_k_slack(s), 64), 2, &pks);
            for (int pk : pks) {
                int deepest = umma_deepest_ring(BN, 2, 128, pk == 1, m.smem_bytes);
                if (deepest > 8) deepest = 8;
                Config d;
                d.family = ADAPT_FAM_UMMA_2CTA; d.BM = 256; d.BN = BN; d.BK = 64; d.cluster = 2;
                d.stages = deepest; d.P_k = pk; d.srcA = ADAPT_SRC_TMA_CLASSES; d.srcB = srcB;
                if (deepest >= 2 && finalize(s, m, cal, d)) out->push_back(d);
            }
        }
    }
    // --- tcgen05, B read in place through per-k-class views (row-major B, N % 8 != 0); A is regrouped by a
    //     prologue copy, so this pays when A is the small operand ---
    if (b_unaligned && s.layoutB == ADAPT_ROW_MAJOR && s.K >= 64) {
        const int64_t tiles = ceil_div(s.M, 128) * ceil_div(s.N, 56);
        split_candidates(tiles, m.n_sm, ceil_div(ceil_div(s.K, 8), 64), 1, &pks);
        for (int pk : pks) {
            const int deepest = umma_deepest_ring(64, 1, umma_a_box_rows(s, 1, 0, true), pk == 1, m.smem_bytes);
            Config d;
            d.family = ADAPT_FAM_UMMA_1CTA; d.BM = 128; d.BN = 64; d.BK = 64; d.cluster = 1;
            d.stages = deepest; d.P_k = pk; d.srcA = ADAPT_SRC_PAD_COPY; d.srcB = ADAPT_SRC_TMA_CLASSES;
            if (deepest >= 2 && finalize(s, m, cal, d)) out->push_back(d);
        }
    }
    // --- the same views with each class a k split: full-width tiles, 8 fp32 partials per output ---
    if (b_unaligned && s.layoutB == ADAPT_ROW_MAJOR && s.K >= 64) {
        for (int v = 0; v < 3; ++v) {                               // 1-CTA tiles of 128 and 256 columns, pair tiles of 256
            const int BN = v == 0 ? 128 : 256, cluster = v == 2 ? 2 : 1, BM = 128 * cluster;
            const int64_t tiles = ceil_div(s.M, BM) * ceil_div(s.N, BN - 8);
            split_candidates(tiles * 8, m.n_sm / cluster, ceil_div(ceil_div(s.K, 8), 64), 1, &pks);
            if (std::find(pks.begin(), pks.end(), 1) == pks.end()) pks.insert(pks.begin(), 1);
            const int deepest = umma_deepest_ring(BN, cluster, umma_a_box_rows(s, cluster, 0, true), false, m.smem_bytes,
                                                  cluster == 2 ? 8 : kUmmaMaxStages);
            for (int pkk : pks) {
                Config d;
                d.family = cluster == 2 ? ADAPT_FAM_UMMA_2CTA : ADAPT_FAM_UMMA_1CTA;
                d.BM = BM; d.BN = BN; d.BK = 64; d.cluster = cluster;
                d.stages = deepest; d.P_k = 8 * pkk; d.srcA = ADAPT_SRC_PAD_COPY; d.srcB = ADAPT_SRC_TMA_CLASSES;
                if (deepest >= 2 && 8 * pkk <= 1023 && finalize(s, m, cal, d)) out->push_back(d);
                if (cluster == 1 && pkk == 1) {                     // the eight classes of a tile as one cluster
                    const int rows = umma_a_box_rows(s, 1, 0, true);
                    Config f = d;
                    f.fused = 1;
                    f.stages = umma_deepest_ring(BN, 1, rows, false, m.smem_bytes, kUmmaMaxStages, umma_fused_bytes(BN, rows));
                    if (f.stages >= 2 && finalize(s, m, cal, f)) out->push_back(f);
                }
            }
        }
    }
    // --- warp-level streaming family ---
    if (std::min(s.M, s.N) <= 16) {
        for (int BN : {128, 256, 512}) {
            const int64_t tiles = ceil_div(std::max(s.M, s.N), BN);
            split_candidates(tiles, (int64_t)m.n_sm * 2, ceil_div(s.K, kSkinnyKChunk), 1, &pks);
            for (int pk : pks) {
                Config c;
                c.family = ADAPT_FAM_SKINNY; c.BM = 16; c.BN = BN; c.BK = 16; c.stages = 1; c.P_k = pk;
                c.srcA = c.srcB = ADAPT_SRC_LSU;
                if (finalize(s, m, cal, c)) out->push_back(c);
            }
        }
    }
    // --- CUDA-core family: always legal ---
    {
        const int64_t tiles = ceil_div(s.M, 64) * ceil_div(s.N, 64);
        split_candidates(tiles, (int64_t)m.n_sm * 4, ceil_div(s.K, 16), 4, &pks);
        for (int pk : pks) {
            Config c;
            c.family = ADAPT_FAM_SIMT; c.BM = 64; c.BN = 64; c.BK = 16; c.stages = 1; c.P_k = pk;
            c.srcA = c.srcB = ADAPT_SRC_LSU;
            if (finalize(s, m, cal, c)) out->push_back(c);
        }
    }
    // --- one-launch cluster family: any shape, layout and alignment whose tiles fit the machine about once ---
    for (int cs : {1, 2, 4, 8, 16}) {
        Config c;
        c.family = ADAPT_FAM_CLUSTER; c.BM = 64; c.BN = 64; c.BK = 64; c.P_k = cs; c.cluster = cs;
        c.stages = cluster_ring(s.K, cs, ceil_div(s.M, 64) * ceil_div(s.N, 64), m.n_sm);
        c.srcA = c.srcB = ADAPT_SRC_LSU;
        if (finalize(s, m, cal, c)) out->push_back(c);
    }
    // argmin of Eq. 6 with a deterministic tie-break: time, then fewer splits, then smaller
    // workspace, then enumeration order (stable sort keeps it)
    std::stable_sort(out->begin(), out->end(), [](const Config& a, const Config& b) {
        if (a.predicted_us != b.predicted_us) return a.predicted_us < b.predicted_us;
        if (a.P_k != b.P_k) return a.P_k < b.P_k;
        return a.workspace_bytes < b.workspace_bytes;
    });
}

bool config_from_key(const Shape& s, uint64_t key, const Machine& m, const Calib& cal, Config* out)
{
    Shape flags;
    Config c;
    if (!unpack_tiling_key(key, &flags, &c)) return false;
    if (flags.dtype != s.dtype || flags.layoutA != s.layoutA || flags.layoutB != s.layoutB) return false;
    if (s.M < 1 || s.N < 1 || s.K < 1) return false;
    const int want_cls = c.cls;
    Machine all = m;
    all.family_mask = m.family_mask;
    if (!finalize(s, all, cal, c)) return false;
    if (c.cls != want_cls) return false;
    if (pack_tiling_key(s, c) != key) return false;
    *out = c;
    return true;
}

void fill_info(const Shape& s, const Config& c, adapt_plan_info_t* o)
{
    o->tiling_key = pack_tiling_key(s, c);
    o->M = s.M; o->N = s.N; o->K = s.K;
    o->dtype = s.dtype; o->layoutA = s.layoutA; o->layoutB = s.layoutB;
    o->taxonomy_class = c.cls; o->family = c.family;
    o->BM = c.BM; o->BN = c.BN; o->BK = c.BK; o->stages = c.stages;
    o->P_m = c.P_m; o->P_n = c.P_n; o->P_k = c.P_k; o->cluster = c.cluster;
    o->srcA = c.srcA; o->srcB = c.srcB; o->grid = c.grid; o->fused = c.fused; o->streamk = c.streamk; o->reserved = 0;
    o->workspace_bytes = c.workspace_bytes;
    o->flops = 2.0 * (double)s.M * (double)s.N * (double)s.K;
    o->hbm_bytes = c.hbm_bytes;
    o->t_pro_us = c.t_pro_us; o->t_main_us = c.t_main_us; o->t_epi_us = c.t_epi_us;
    o->predicted_us = c.predicted_us;
}

}  // namespace adapt

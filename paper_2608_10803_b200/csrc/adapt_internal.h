// Internal declarations shared by the host-side selector, the plan cache and the launchers.
#pragma once

#include <cstdint>
#include <cstddef>
#include <vector>
#include <algorithm>

#include "adapt_matmul.h"

namespace adapt {

// ---- machine description (paper Table 1: N_core, buffer capacities) ------------------------
struct Machine {
    int n_sm = 148;                     // N_core
    int smem_bytes = 227 * 1024;        // per-CTA shared memory limit (the paper's L1 capacity)
    int tmem_cols = 512;                // 128 lanes x 512 fp32 columns per SM (the paper's L0C)
    int64_t workspace_limit = (int64_t)24 << 30;
    unsigned family_mask = 0x1Fu;        // bit f set = family f may be selected
    int max_cluster = 16;               // largest thread-block cluster the one-launch kernel may ask for (queried at init)
    // clusters of 2, 4, 8 CTAs of the tcgen05 kernel (one CTA per SM) the device runs at a time; a cluster sits inside
    // one GPC, so the larger sizes leave SMs unused (B200: 74, 33, 15; queried at init)
    int umma_clusters[3] = {74, 33, 15};
};
inline int umma_cluster_slots(const Machine& m, int cluster)
{
    return cluster == 2 ? m.umma_clusters[0] : cluster == 4 ? m.umma_clusters[1] : cluster == 8 ? m.umma_clusters[2] : m.n_sm;
}

// ---- calibration constants of the latency model (Eq. 8: lambda_r, eta_r, BW_r) ------------
// Measured on B200 with this library's own kernels (CUDA events); the paper's values are for
// other hardware and are not printed, so these are this library's.
// Variant groups of the last calibration step: after the terms of Eq. 7 are added up, the prediction of a configuration is
// scaled by the factor of its group, the geometric mean of measured / predicted time over every timed configuration of
// that group in the fitting set (paper_2608_10803_b200/calibrate.py computes the table from the CSV that
// `bench.py --validate-model N --dump-candidates` writes).  The terms rank the configurations inside a group; the factors
// put the groups, whose kernels differ in what the terms leave out, on one scale.
constexpr int kCalibGroups = 40;
struct Config;
int calib_group(const Config& c);

// The constants below were first set from the single measurements their comments name.  Nineteen of them (l2_bw_per_sm,
// eta_mma_bn128, eta_mma_bn64, umma_fixed_us, epi_tile_fixed_us, pair_drain_factor, epi_partial_*, epi_*_unaligned*,
// thread_store_exposed, class_view_sm_eff, class_tile_fixed_unaligned_us, kclass_view_sm_eff, kclass_unit_fixed_us,
// class_split_bw_eff, class_split_fused_bw_eff, launch_us, copy_bw_eff) were then moved by one pass of coordinate descent
// (steps of 0.8, 0.9, 1.1, 1.25) on the mean regret of the model's pick over 654 sweep shapes with up to 128 timed
// configurations each; on 300 shapes of another seed the mean regret went from 1.060 to 1.043 and the largest from 1.89 to
// 1.64, on a third seed it is 1.052 and 1.71.  A second pass with finer steps gained nothing on the other seed and was dropped.
// A later pass (same steps, two rounds) on 600 sweep shapes of any size, launch-bound ones included, timed with rotating
// operand sets (cold operands, as in the sweep pass) moved twenty constants again (launch_us, the cluster and warp-level
// kernels' terms, the thread-store drain, hbm_bw_per_sm among them): seeds 11, 23 and 37 (the last seen by no fit)
// then give mean regrets 1.047, 1.039, 1.044 and maxima 1.81, 1.51, 1.58, with 45 to 53 % exact picks.  Of that pass
// hbm_bw_per_sm was taken back from 75.6 to 60.5 GB/s: the larger value hides the cost of a partial last wave on the
// heaviest shapes (61370 x 32 x 85272 picked without split or stream-K: 2275 against 1700 us), 1.4 % of their time in total.
struct Calib {
    // All ones: factors fitted on 34,000 timed configurations of 500 sweep shapes (0.72 for plain one-split tiles ... 1.19 for
    // fused k classes, 0.48 for the warp-level kernel) raised the mean regret on a held-out shape set from 1.063 to 1.076,
    // their square roots left it where it was (1.061): the groups' errors depend on the shape more than on the group.
    double group_bias[kCalibGroups] = {
        1.0, 1.0, 1.0, 1.0, 1.0, 1.0, 1.0, 1.0, 1.0, 1.0, 1.0, 1.0, 1.0, 1.0, 1.0, 1.0, 1.0, 1.0, 1.0, 1.0,
        1.0, 1.0, 1.0, 1.0, 1.0, 1.0, 1.0, 1.0, 1.0, 1.0, 1.0, 1.0, 1.0, 1.0, 1.0, 1.0, 1.0, 1.0, 1.0, 1.0};
    double launch_us = 1.54;             // one kernel launch issued back to back on a stream (also per reduce launch)
    double prologue_launch_us = 0.3;    // a re-pitch / regroup launch ahead of the GEMM: its launch overlaps the GEMM's own
                                        // (programmatic dependent launch); fit over 910 timed small configurations: -0.2 us
    double hbm_bw = 6.2e12;             // B/s, large streaming transfers
    double l2_bw_per_sm = 1.1e11;        // B/s one SM pulls through TMA from L2 (8192^3, 128 x 256 tiles: 48 KB per 0.48 us)
    double tensor_flops = 1.58e15;      // whole chip, kind::f16, BN = 256 (8192^3 on 256 x 256 pair tiles: 1.56e15)
    double eta_mma_bn128 = 0.518;        // relative tensor efficiency at BN = 128 (0.29 us per 128 x 128 x 64 block)
    double eta_mma_bn64 = 0.324;         // ... at BN = 64 (A-operand smem reads dominate)
    double eta_2cta = 1.0;              // pair tiles share B: no extra tensor cost
    double mem_latency_us = 1.0;        // TMA issue -> data visible (sets Delta_dep with few stages)
    double hbm_latency_us = 1.04;        // the same under a full HBM stream of a dense operand (128 x 128256 x 4096: 5 stages of 32 KB, 0.41 us each)
    double hbm_latency_views_us = 1.6;  // ... through the strided class views (79457 x 196 x 8325 with 3 stages: 0.75 us per stage)
    double umma_fixed_us = 1.1;         // barrier init, TMEM alloc, first load, last drain, TMEM free (the same fit: 2.5 was 3 us high)
    // drain of one output tile through the epilogue warps (overlaps the next tile's main loop):
    // fixed part per tile + part per KB written; rows of C that are not 16-byte aligned cost more
    double epi_tile_fixed_us = 0.25, epi_us_per_kb = 0.0275;          // TMA stores (40000 x 40000 x 8: 4.8 TB/s)
    double pair_drain_factor = 1.39;    // 40000 x 40000 x 8: 780 us on pair tiles, 671 us on 1-CTA tiles
    double epi_partial_fixed_us = 0.44, epi_partial_us_per_kb = 0.0529;   // fp32 partials, stored by the epilogue threads
    double epi_tile_fixed_unaligned_us = 1.41, epi_us_per_kb_unaligned = 0.0311;
    double thread_store_exposed = 0.495;  // share of the main loop that a drain through the epilogue threads does not hide
    double thread_store_exposed_pair = 0.25;   // ... on pair tiles (13835 x 3906 x 852 and 7111 x 97981 x 289 bracket it)
    double simt_flops = 1.65e13;          // CUDA-core tile kernel (1000^3: 17e12)
    double simt_fixed_us = 0.45;
    double simt_step_us = 0.8;          // one 16-k step of a CTA alone on its SM (15 x 30 x 32: two steps, 4.85 us with the launch)
    double halo_edge_tile_us = 0.72;     // row heads or tails of one halo tile (up to 15 elements per row, aligned stores of 2 to 16 bytes)
    double simt_bw_eff = 0.15;          // fraction of hbm_bw its 2-byte accesses reach (K = 1 outer products: 0.13 measured)
    double skinny_bw_eff_aligned = 0.55;    // fraction of hbm_bw the warp-level streaming kernel reaches, 16-byte aligned rows
                                            // (16 x 65536 x 4096: 3.5 TB/s with its loads four steps ahead of the MMAs, 1.6 before)
    double skinny_bw_eff_unaligned = 0.10;  // ... rows assembled from two chunks
    double skinny_fixed_us = 1.6;
    double skinny_pass_us = 4.4;        // one 64-row pass over one staged chunk when the streamed rows are k-contiguous
    double skinny_step_unaligned_us = 2.52;   // one 16-k step of a warp when the streamed rows are unaligned
    double skinny_mac_rate = 30e12;     // MAC/s ceiling of the warp-level kernel (small side padded to 16)
    // one-launch cluster kernel (64 x 64 tiles, k split over a cluster); least-squares fit over 180 timed
    // configurations of 2,000-sweep shapes: 3.7 + 0.95 stages + 0.8 (cluster > 1) + crowd (1.6 + 0.44 stages) us
    double cluster_fixed_us = 0.75;     // beyond the launch: barrier set-up, first trip to memory, rounding and store of the tile
    double cluster_stage_us = 0.76;     // one 64-k stage: copy issue, shift pass, MMAs, each behind a CTA-wide barrier
    double cluster_reduce_us = 1.1;     // cluster barriers + reading the partial tiles of the peers
    double cluster_crowd_us = 1.25, cluster_crowd_stage_us = 0.44;   // per CTA per SM beyond one per two SMs
    double cluster_wave_us = 5.5;       // each further round of clusters
    double cluster_bw_eff = 0.35;       // fraction of hbm_bw its 16-byte copies reach when memory-bound
    double streamk_fixup_us = 10.0;     // stream-K: partial tile out (5 us) and its fence, the flag, the owner's exposed last drain ...
    double streamk_peer_us = 3.0;       // ... and its additions, per slot that shares the tile (2560 x 4096 x 4096, 6 sharers: 87 us
                                        // against 55 us of main loop; 5120 x 4096 x 8192, 3 sharers: 246 us against 226 us)
    double fused_reduce_us = 2.0;       // fused split-K: cluster scheduling, drain to shared memory, two cluster-wide barrier rounds,
                                        // first remote reads (1 x 4096 x 4096, 128 x 128 tiles, P_k 4: 11.3 us fused, 11.1 us with the reduce launch;
                                        // 128 x 4096 x 4096: 13.3 against 14.1 us)
    double fused_wave_us = 3.0;         // each further round of clusters starts cold (1 x 4096 x 4096, P_k 8, 3 rounds: 14.2 us against 11.3 us in one)
    double reduce_launch_us = 1.5;      // the reduce launch behind the GEMM: programmatic dependent launch hides about half of a launch
    double dsmem_bw_per_sm = 60e9;      // B/s one SM reads from its peers' shared memory during the fused reduction
    double copy_bw_eff = 0.935;          // pad-copy and reduce kernels
    double hbm_bw_per_sm = 6.05e10;        // B/s one SM streams from HBM (tail wave of 20000 x 8 x 60001: 15 MB per tile in 0.3 ms)
    double class_view_sm_eff = 0.935;    // per-SM rate through those views relative to l2_bw_per_sm (20000 x 8 x 60001 tail wave)
    double class_tile_fixed_us = 0.625, class_tile_fixed_unaligned_us = 0.99;   // per class tile (44479 x 54634 x 16..72, 64-column tiles)
    double pair_class_tile_us = 1.1;    // pair tiles of one row class, rows with stale heads: the peer zeroes its half and tells the leader across
                                        // the cluster before the tile's first MMA (7111 x 97981 x 289: 3.7 us per pair tile of six k-blocks)
    double kclass_view_sm_eff = 0.605;   // per-SM rate through the k-class views of B relative to l2_bw_per_sm (272 x 67839 x 6046: 48 KB per 0.75 us)
    double kclass_unit_fixed_us = 1.65;  // per unit of a k class run as a k split (1 x 80711 x 221: 18 units of one k-block in 37 us)
    double kclass_tile_drain_us = 2.5;  // drain of a tile with eight class accumulators (29 x 58492 x 94: 8 tile rounds in 35 us)
    double oob_box_penalty = 0.05;      // main-loop cost of one B box per stage that lies wholly beyond N
    double reduce_batch_us = 0.8;       // split-K reduction: one batch of eight slabs (13 x 420 x 43580: P_k 72 -> 24 saves 13 us)
    double class_split_bw_eff = 0.873;   // HBM rate through the k-class views of B with full-width tiles (classes as k splits) at M = 1 ...
    double class_split_bw_eff_per_log2m = 0.031;   // ... and what it loses per doubling of M (1 x 50321 x 48452 ... 80 x 23916 x 86044)
    double class_split_fused_bw_eff = 0.815;       // ... with the classes of a tile as one cluster (36 x 81499 x 66349: 6.3 TB/s)
    double regroup_bw_eff = 0.85;       // class-major regrouping of a row-major A (20000 x 8000: 600 MB in 107 us) relative to hbm_bw
    double class_view_bw_eff = 0.8;     // HBM rate through the per-row-class TMA views of an unaligned A
};

// ---- one configuration x of the search set S(b(s)) (Eq. 6) ------------------------------------
struct Config {
    int family = ADAPT_FAM_SIMT;
    int cls = ADAPT_CLASS_COMMON;
    int BM = 64, BN = 64, BK = 16;
    int stages = 1;
    int P_m = 1, P_n = 1, P_k = 1;
    int cluster = 1;
    int fused = 0;                      // tcgen05 split-K with the k splits as one thread-block cluster, reduced through
                                        // distributed shared memory inside the GEMM launch (no partials in global memory)
    int streamk = 0;                    // tcgen05, P_k = 1: the k-blocks of the tiles that do not fill a whole wave of slots are
                                        // shared evenly by all slots (deterministic stream-K)
    int persistent = 0;
    int srcA = ADAPT_SRC_LSU, srcB = ADAPT_SRC_LSU;
    int grid = 1;
    int smem_bytes = 0;
    int64_t workspace_bytes = 0;        // total
    int64_t ws_padA = 0, ws_padB = 0, ws_partial = 0;  // sizes of the three regions
    double hbm_bytes = 0, t_pro_us = 0, t_main_us = 0, t_epi_us = 0, predicted_us = 0;
};

struct Shape {
    int64_t M = 0, N = 0, K = 0;
    int dtype = 0, layoutA = 0, layoutB = 0;
};

// Section 4.2 predicate, parameterised by the machine.
int classify(int64_t M, int64_t N, int64_t m, int64_t n, int64_t m1, int64_t n1, int64_t n_core, int64_t acc_bytes);

// Closed forms (bytes; times in the caller's unit).
double read_volume(int64_t M, int64_t N, int64_t K, int64_t m1, int64_t n1);                 // Eq. 1
double write_volume(int cls, int64_t M, int64_t N, int64_t K, int64_t k, int64_t k1);       // Eq. 2-5
double pipeline_time(int schedule, int64_t Q, int64_t L, double tM, double tP, double Td);  // Eq. 12-14

uint64_t pack_tiling_key(const Shape& s, const Config& c);
bool unpack_tiling_key(uint64_t key, Shape* flags, Config* c);   // fills the key's fields only

// Enumerate the legal configurations for a shape (capacity and instruction-shape checks done),
// each scored by the model, sorted best first with the deterministic tie-break.
void enumerate_configs(const Shape& s, const Machine& m, const Calib& cal, std::vector<Config>* out);

// Rebuild the full Config a key describes for this shape; false if it is not legal.
bool config_from_key(const Shape& s, uint64_t key, const Machine& m, const Calib& cal, Config* out);

void fill_info(const Shape& s, const Config& c, adapt_plan_info_t* out);

inline int64_t ceil_div(int64_t a, int64_t b) { return (a + b - 1) / b; }
inline int64_t round_up(int64_t a, int64_t b) { return ceil_div(a, b) * b; }

// Row pitch (elements) of the fp32 split-K partials: rows start on 32-byte boundaries, so the tensor-core
// kernels write whole 32-byte sectors (16-byte pieces of a sector halve the store rate).
inline int64_t partial_pitch(int64_t N) { return round_up(N, 8); }

// TMA reads an operand in place when its rows are 16-byte multiples.  Rows shorter than one 128-byte box line must in
// addition be whole 32-byte sectors: a box whose rows are fractions of a sector loads at a fraction of the rate (a
// 61370 x 85272 A streams at 6.8 TB/s beside a B of 32 columns, at 5.3 beside one of 5, 8 or 40 columns; a
// 44239 x 80357 C is written in 1.47 ms beside an A of 16 padded columns, in 1.89 ms beside one of 1).
inline bool tma_friendly(int64_t inner) { return inner % 8 == 0 && (inner >= 64 || inner % 16 == 0); }
// Operand pitch in elements after the Padding module: a 32-byte multiple; the copy fills the pad columns with zeros, and
// the tensor map covers them, so that every row TMA fetches, also the last box of a row, is made of whole sectors
// (27239 x 84 x 96056, B re-pitched to 88 columns: the 20-column remainder box of every k-block costs as much as three
// full ones).
inline int64_t padded_pitch(int64_t inner) { return round_up(inner, 16); }

// Class tiles read a row-major A in place through their per-class views, except a narrow one whose rows are not whole
// sectors: that one is re-pitched first (the views of the copy are then all aligned).
inline bool class_tiles_copy_a(const Shape& s) { return s.K < 64 && !tma_friendly(s.K); }
// Class tiles over an A whose rows are unaligned shift the k index by up to 7 elements (one more k-block at most); over a
// copy every view is aligned and nothing shifts.
inline int64_t class_k_slack(const Shape& s) { return (s.K % 8 != 0 && !class_tiles_copy_a(s)) ? 7 : 0; }

const Calib& default_calib();

// Shared-memory layout of the tcgen05 kernels, used by the capacity check and by the launcher:
// S stages of (A: box rows x 64, B: BN/cluster x 64) 16-bit, a barrier block, the epilogue staging
// (8 KB per epilogue warp, only when the kernel stores the 16-bit C), and slack to align the stages to 1024 B.
// One-launch cluster kernel: a ring of raw stages (64 rows of 144 bytes per operand) plus two shifted stages.
// The ring is as deep as the CTA's k range needs, capped so that the CTAs that share an SM all fit.
constexpr int kClusterStageBytes = 2 * 64 * 144;
constexpr int kClusterMaxRing = 6;
inline int cluster_smem_bytes(int ring) { return (ring + 2) * kClusterStageBytes + 128; }   // + two shifted stages, barriers
// Clusters of a size the machine runs at a time with one CTA per SM (a cluster is placed inside one GPC, so
// the larger sizes leave SMs unused): what cudaOccupancyMaxActiveClusters reports on a B200 for this kernel
// with its deepest ring (148, 74, 33, 15, 7), scaled to other SM counts.  With two CTAs per SM (rings of up
// to four stages; the kernel's registers allow no more) it is about twice that (296, 148, 71, 33, 14).
inline int64_t cluster_slots(int cluster, int n_sm)
{
    const int64_t b200 = cluster == 1 ? 148 : cluster == 2 ? 74 : cluster == 4 ? 33 : cluster == 8 ? 15 : 7;
    return std::max<int64_t>(1, b200 * n_sm / 148);
}
inline int cluster_ctas_per_sm(int ring, int smem_limit) { return std::max(1, std::min(2, smem_limit / cluster_smem_bytes(ring))); }
// Depth of the raw ring: as deep as the CTA's k range needs, up to 6 stages when the tiles' clusters all run
// at once with an SM per CTA, else up to 4 so that two CTAs share an SM.
inline int cluster_ring(int64_t K, int cluster, int64_t tiles, int n_sm)
{
    const int64_t k_cta = (K + cluster - 1) / cluster;
    const int64_t stages = ((k_cta + 15) / 16 * 16 + 63) / 64;
    const int cap = tiles <= cluster_slots(cluster, n_sm) ? kClusterMaxRing : 4;
    return (int)std::max<int64_t>(1, std::min<int64_t>(stages, cap));
}
// Stream-K schedule of a shape: W whole waves of tiles stay data-parallel, the R = tiles - W * slots tiles left over
// (all tiles when there are fewer than slots) are cut into k-block ranges, sk_q0 (+1 for the first sk_rem slots) per slot.
struct StreamK {
    int64_t tiles, slots, waves, sk_tiles, q0, rem;
};
inline StreamK streamk_schedule(int64_t tiles, int64_t slots, int64_t kblocks)
{
    StreamK k;
    k.tiles = tiles; k.slots = slots;
    k.waves = tiles / slots;
    k.sk_tiles = tiles - k.waves * slots;
    k.q0 = k.sk_tiles * kblocks / slots;
    k.rem = k.sk_tiles * kblocks - k.q0 * slots;
    return k;
}
constexpr int kUmmaFlagBytes = 4096;     // head of every workspace: stream-K flag words (one per CTA), zeroed when the workspace is allocated
constexpr int kSkinnyKChunk = 512;   // k values the warp-level kernel stages per chunk; its k splits are whole chunks
constexpr int kUmmaBarrierBytes = 1024;  // keeps the epilogue staging 1024-byte aligned (swizzled TMA boxes)
constexpr int kUmmaMaxStages = 15;
constexpr int kUmmaEpilogueWarps = 8;
constexpr int kUmmaStageRowBytes = 144;   // 72 16-bit elements: 64 columns + up to 7 of alignment shift
constexpr int kUmmaWarpStagingBytes = 8192;   // per epilogue warp: two 32 x 128 B boxes for TMA stores, or 32 shifted rows
// fp32 partial tile a CTA of a fused split-K cluster keeps for the exchange: x_rows rows of BN + 4 elements
// (the 16 bytes of padding spread the rows of a warp over the banks)
inline int umma_fused_pitch(int BN) { return BN + 4; }
inline int umma_fused_bytes(int BN, int x_rows) { return x_rows * umma_fused_pitch(BN) * 4; }
inline int umma_smem_bytes(int BN, int cluster, int stages, int a_rows, bool staging, int fused_bytes = 0)
{
    const int stage = a_rows * 64 * 2 + (int)round_up(BN / cluster, 64) * 64 * 2;
    const int used = stages * stage + kUmmaBarrierBytes + (staging ? kUmmaEpilogueWarps * kUmmaWarpStagingBytes : 0) + fused_bytes;
    // the MMA reads 128 rows of A from every stage, also when the box brought fewer: the rows past the box
    // of the last stage must still lie inside the allocation
    const int read_end = (stages - 1) * stage + 128 * 64 * 2;
    return std::max(used, read_end) + 1024;
}
// Deepest ring that fits (0 if not even two stages do).  Only a kernel that writes the 16-bit C itself
// (P_k = 1) needs the epilogue staging; one that writes fp32 partials spends that space on stages.
inline int umma_deepest_ring(int BN, int cluster, int a_rows, bool staging, int smem_limit, int cap = kUmmaMaxStages, int fused_bytes = 0)
{
    for (int st = cap; st >= 2; --st)
        if (umma_smem_bytes(BN, cluster, st, a_rows, staging, fused_bytes) <= smem_limit) return st;
    return 0;
}

// Rows of A one TMA box brings per stage (a multiple of 8, so the stage stays a multiple of 1024 B).
// A K-major A of fewer than 128 rows is loaded with a box of just those rows, and the stage's A
// region shrinks with it: the MMA still reads 128 rows, but the rows past the box only feed
// accumulator rows that are never stored.  Class tiles hold every 8th row of up to 1024.
inline int umma_a_box_rows(const Shape& s, int cluster, int row_classes, bool k_classes)
{
    const bool a_mn = !k_classes && s.layoutA == ADAPT_COL_MAJOR;
    if (row_classes)    // 8 or 16 classes: a tile holds every 8th (16th) row of up to 1024 (2048); a pair tile of twice as many
        return (cluster == 1 && s.M < 128 * row_classes) ? (int)std::min<int64_t>(128, round_up(ceil_div(s.M, row_classes), 8)) : 128;
    if (!a_mn && cluster == 1 && s.M < 128) return (int)round_up(s.M, 8);
    return 128;
}

// Row classes of halo class tiles.  The rows of one class must share their offset from a 32-byte boundary in C (rows j and
// j + n do when n * N is a multiple of 16 elements: n = 16 for an odd N, 8, 4 or 2 for an even one) and, when A is read in
// place, their offset from a 16-byte boundary in A (n * K a multiple of 8).  As few classes as that allows: the rows of a
// tile are then n rows of C apart, and a TMA store box whose rows lie 2 MiB or more apart writes slower (16 classes at
// N = 99991: 4.2 TB/s; 8 classes at N = 99990: 5.5 TB/s); a smaller n also wastes less of a ragged M.
inline int gcd_pow2(int64_t v, int p2) { int g = 1; while (g < p2 && v % (2 * g) == 0) g *= 2; return g; }
inline int halo_row_classes(const Shape& s)
{
    const int for_c = 16 / gcd_pow2(s.N % 16 == 0 ? 16 : s.N % 16, 16);
    const int for_a = class_tiles_copy_a(s) ? 1 : 8 / gcd_pow2(s.K % 8 == 0 ? 8 : s.K % 8, 8);
    return std::max(2, std::max(for_c, for_a));
}
// Row classes of a configuration's tiles: 0 (plain tiles), 8 (class tiles), 2 to 16 (class tiles with halo columns).
inline int umma_row_classes(const Shape& s, int srcA, int BN) { return srcA != ADAPT_SRC_TMA_CLASSES ? 0 : (BN % 64 ? halo_row_classes(s) : 8); }

}  // namespace adapt

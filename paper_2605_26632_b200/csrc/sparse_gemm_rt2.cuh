// 2:4 sparse x dense GEMM, "two row tiles per W stage" form (Algorithm 1 lines 5-6):
//     Y[m, n] = bf16( s_m * sum_k X~[m,k] W[n,k] + bias[n] + Yr[m,n] )
//
// Why a second kernel.  The main loop of sparse_gemm_kernel is bound by the operand stream into
// each SM, and that stream is bound by latency x bytes in flight (a load-only run of the same
// loop delivers 89 / 134 / 165 GB/s per SM with 2 / 3 / 4 stages of 48 KB in flight: ~1.1 us per
// round trip), while the sparse MMAs of a 256 x 240 stage need only 0.28 us.  Shared memory is
// full, so the only lever left is flops per byte in flight.  Here a CTA pair works on TWO 256-row
// tiles of the same 240 columns at once ("double"): a ring stage holds two compressed-A tiles and
// two metadata blocks per CTA but ONE W tile, 66 KB for twice the MMAs of the 48 KB stage (-31 %
// bytes per flop).  The two accumulators fill all of tensor memory (2 x 240 columns + metadata),
// so the epilogue of a double is not hidden behind a following main loop; it is therefore made
// short: eight epilogue warps (four per accumulator), tcgen05.ld of the next column chunk in flight
// while the current one is converted; each warp stages its 32 x 48 chunk in a 3 KB box of its own
// and hands it to a TMA store.  (Storing straight from registers -- 16 bytes per lane, every lane
// another row -- was measured first: 5.6 us per 512-row item, more than the main loop gained.)
//
// Work items of a cluster: "doubles" (512 x 240) first, then "singles" (256 x 240, the tile of
// sparse_gemm_kernel; consecutive singles alternate between the two accumulators, so their
// epilogues overlap the next single's main loop).  How many doubles a launch uses is the host's
// choice (PairSchedule, a cost model): doubles cost less per unit, singles fill the clusters that
// would otherwise idle in the last round.
//
// Roles per CTA (320 threads): warp 0 TMA producer, warp 1 MMA issuer (leader CTA, one thread),
// warps 2-5 epilogue of accumulator 0, warps 6-9 epilogue of accumulator 1.  Every wait is
// bounded (mbar_wait): on expiry the kernel raises the error word and all roles leave.
#pragma once

#include "ptx.cuh"
#include "prune_compress.cuh"  // row_scale_from_partials
#include "sparse_gemm.cuh"     // make_idesc_sp_bf16

namespace lynx {

// Distribution of the output over C clusters.  Units are 256 x BN tiles (tm, tn).  Double slot i
// pairs the row tiles 2d and 2d + 1 of column tile tn; inside a group of `gd` double rows the row
// index runs fastest (the clusters of a round then share gd * 2 blocks of A and C / gd tiles of W).
// The first D slots are run as doubles, dealt round-robin: cluster c gets slots c, c + C, ...
// Every other unit is a single: the two halves of the slots D .. Dmax - 1 and, when the number of
// row tiles is odd, the last row tile.  Singles are dealt so that clusters with one double fewer
// ("light", index >= D % C) get one first, then round-robin over all clusters starting there.
struct PairSchedule {
    int TM, TN, C;
    int DM, gd, D, Dmax, S, b, L;

    __host__ __device__ void init(int tiles_m, int tiles_n, int clusters, int doubles, int group_double_rows) {
        TM = tiles_m; TN = tiles_n; C = clusters;
        DM = TM / 2;
        gd = group_double_rows;
        if (gd <= 0 || gd > DM) gd = DM > 0 ? DM : 1;
        if (DM > 0) {  // groups of nearly equal size
            const int groups = (DM + gd - 1) / gd;
            gd = (DM + groups - 1) / groups;
        }
        Dmax = DM * TN;
        D = doubles < 0 ? 0 : (doubles > Dmax ? Dmax : doubles);
        S = 2 * (Dmax - D) + ((TM & 1) ? TN : 0);
        b = D % C;
        L = C - b;
    }
    __host__ __device__ void slot_coords(int i, int& d, int& tn) const {
        const int per_group = gd * TN;
        const int g = i / per_group, r = i - g * per_group;
        const int rows = (DM - g * gd < gd) ? DM - g * gd : gd;
        tn = r / rows;
        d = g * gd + (r - tn * rows);
    }
    __host__ __device__ int position(int c) const { return (c - b + C) % C; }
    __host__ __device__ int num_doubles(int c) const { return (D > c) ? (D - c + C - 1) / C : 0; }
    __host__ __device__ int num_singles(int c) const {
        const int p = position(c);
        const int first = (p < L && p < S) ? 1 : 0;
        const int rest = (S > L + p) ? (S - L - p + C - 1) / C : 0;
        return first + rest;
    }
    // k-th single of cluster c -> index in the list of singles
    __host__ __device__ int single_index(int c, int k) const {
        const int p = position(c);
        if (p < L) return k == 0 ? p : L + p + (k - 1) * C;
        return L + p + k * C;
    }
    __host__ __device__ void single_unit(int j, int& tm, int& tn) const {
        const int broken = 2 * (Dmax - D);
        if (j < broken) {
            int d;
            slot_coords(D + (j >> 1), d, tn);
            tm = 2 * d + (j & 1);
        } else {
            tm = TM - 1;
            tn = j - broken;
        }
    }
    __host__ __device__ int num_items(int c) const { return num_doubles(c) + num_singles(c); }
    // item i of cluster c: first row tile, column tile, row tiles (1 or 2); for a single also its
    // ordinal among the cluster's singles (which accumulator it uses)
    __host__ __device__ void item(int c, int i, int& tm0, int& tn, int& rows, int& ordinal) const {
        const int nd = num_doubles(c);
        if (i < nd) {
            int d;
            slot_coords(c + i * C, d, tn);
            tm0 = 2 * d;
            rows = 2;
            ordinal = 0;
        } else {
            ordinal = i - nd;
            single_unit(single_index(c, ordinal), tm0, tn);
            rows = 1;
        }
    }
};

struct Gemm2Params {
    int64_t M, N, K;
    const float* row_scale;      // [M] or nullptr
    const float* scale_partial;  // or: per-K-split row sums of a deferred prune launch
    int scale_ks;
    const uint16_t* bias;      // [N] bf16 or nullptr
    const uint16_t* residual;  // [M x N] bf16 (ld = ldr) or nullptr
    int64_t ldr;
    uint32_t* dev_error;
    PairSchedule sched;
    int lora_steps;  // R / 64 extra dense stages per item (0 = no low-rank branch)
    int w_prefetch;  // layer calls: W tiles of the first stages are fetched before the wait for the prune launch
};

template <int BN_, int STAGES_>
struct Gemm2Cfg {
    static constexpr int BN = BN_, STAGES = STAGES_, CG = 2;
    static constexpr int BM = 128, BK = 128;
    static constexpr int BN_CTA = BN / CG;
    static constexpr int A_BYTES = BM * 128;           // one row tile of compressed A: 16 KB
    static constexpr int E_BYTES = 2048;               // its metadata block
    static constexpr int B_HALF_BYTES = BN_CTA * 128;  // one 128-byte K slice of this CTA's W rows
    static constexpr int B_BYTES = 2 * B_HALF_BYTES;
    static constexpr int STAGE_BYTES = 2 * A_BYTES + 2 * E_BYTES + B_BYTES;
    static constexpr int SINGLE_TX = A_BYTES + E_BYTES + B_BYTES;
    static constexpr int CH = 48;                      // epilogue column chunk
    static constexpr int NCH = BN / CH;
    static constexpr int E_COL0 = 2 * BN;              // metadata columns behind the two accumulators
    static constexpr int E_COLS = 8;                   // per stage: 4 per row tile
    static constexpr int TMEM_COLS = 512;
    static constexpr int EPI_WARPS = 8;
    static constexpr int THREADS = 64 + 32 * EPI_WARPS;
    // the single-tile items run on a ring of their own over the same shared memory: four stages of
    // 48 KB (A 16 KB, metadata 2 KB, W 30 KB) instead of three of 66 KB
    static constexpr int STAGES1 = 4;
    static constexpr int RING1_A = 0, RING1_B = STAGES1 * A_BYTES, RING1_E = RING1_B + STAGES1 * B_BYTES;
    static constexpr int NUM_BARS = 2 * STAGES + 2 * STAGES1 + 4;
    static constexpr int C_BOX_BYTES = 32 * CH * 2;    // one epilogue warp's staging box: 32 rows x 48 columns
    static constexpr int C_BYTES = EPI_WARPS * C_BOX_BYTES;
    static constexpr int BIAS_BYTES = BN * 2;          // one epilogue warp's copy of the item's bias values (bf16)
    static constexpr int SMEM_BYTES = 1024 /*align slack*/ + STAGES * STAGE_BYTES + C_BYTES + EPI_WARPS * BIAS_BYTES + 256;
    static_assert(BN % CH == 0 && BN % 16 == 0 && BN_CTA % 8 == 0, "tile N");
    static_assert(B_HALF_BYTES % 1024 == 0, "swizzle atoms need 1024-byte aligned tiles");
    static_assert(E_COL0 + E_COLS * STAGES <= TMEM_COLS && 4 * STAGES1 <= E_COLS * STAGES, "tensor memory budget");
    static_assert(RING1_E + STAGES1 * E_BYTES <= STAGES * STAGE_BYTES, "the single-tile ring fits into the double ring's memory");
    static_assert(8 * NUM_BARS + 16 <= 256, "barrier area");
    static_assert(SMEM_BYTES <= 227 * 1024, "shared memory budget");
};

template <class Cfg, bool LORA>
__global__ void __launch_bounds__(Cfg::THREADS, 1)
sparse_gemm_rt2_kernel(const __grid_constant__ CUtensorMap tmap_a, const __grid_constant__ CUtensorMap tmap_b,
                       const __grid_constant__ CUtensorMap tmap_e, const __grid_constant__ CUtensorMap tmap_y,
                       const __grid_constant__ CUtensorMap tmap_t, const __grid_constant__ CUtensorMap tmap_la,
                       const Gemm2Params p) {
    constexpr int STAGES = Cfg::STAGES, BN = Cfg::BN;
    const int lora_steps = LORA ? p.lora_steps : 0;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* smem_gen = smem_raw + (smem_base - smem_u32(smem_raw));
    const uint32_t sA = smem_base;                              // [stage][row tile] A_BYTES
    const uint32_t sB = sA + STAGES * 2 * Cfg::A_BYTES;         // [stage] B_BYTES
    const uint32_t sE = sB + STAGES * Cfg::B_BYTES;             // [stage][row tile] E_BYTES
    const uint32_t sC = sE + STAGES * 2 * Cfg::E_BYTES;         // [epilogue warp] C_BOX_BYTES
    const uint32_t sBias = sC + Cfg::C_BYTES;                   // [epilogue warp] BIAS_BYTES
    const uint32_t sBar = sBias + Cfg::EPI_WARPS * Cfg::BIAS_BYTES;
    const uint32_t bar_full = sBar, bar_empty = sBar + 8 * STAGES;
    const uint32_t bar_tfull = sBar + 16 * STAGES, bar_tempty = bar_tfull + 16;
    const uint32_t bar_full1 = bar_tempty + 16, bar_empty1 = bar_full1 + 8 * Cfg::STAGES1;  // single-tile ring
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem_gen + (sBar - smem_base) + 8 * Cfg::NUM_BARS);
    volatile uint32_t* cta_abort = tmem_slot + 1;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = cluster_ctarank();
    const bool leader = rank == 0;
    const int cluster_id = blockIdx.x / 2;
    const int kblocks = (int)(p.K / Cfg::BK);
    const PairSchedule& sched = p.sched;
    const int num_items = sched.num_items(cluster_id);

    if (threadIdx.x == 0) {
        *cta_abort = 0;
        for (int s = 0; s < STAGES; ++s) {
            mbar_init(bar_full + 8 * s, 1);   // leader's producer arrives once (+ transaction bytes)
            mbar_init(bar_empty + 8 * s, 1);  // one tcgen05.commit
        }
        for (int s = 0; s < Cfg::STAGES1; ++s) {
            mbar_init(bar_full1 + 8 * s, 1);
            mbar_init(bar_empty1 + 8 * s, 1);
        }
        for (int a = 0; a < 2; ++a) {
            mbar_init(bar_tfull + 8 * a, 1);   // one tcgen05.commit
            mbar_init(bar_tempty + 8 * a, 8);  // the accumulator's four epilogue warps in both CTAs
        }
        fence_mbar_init();
        prefetch_tmap(&tmap_a);
        prefetch_tmap(&tmap_b);
        prefetch_tmap(&tmap_e);
        prefetch_tmap(&tmap_y);
        if (lora_steps) {
            prefetch_tmap(&tmap_t);
            prefetch_tmap(&tmap_la);
        }
    }
    if (warp == 1) {
        tmem_alloc<2>(smem_u32(tmem_slot), Cfg::TMEM_COLS);
        tmem_relinquish<2>();
    }
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    // W tiles of the first stages of the first item, before the wait for the previous kernel (W is
    // not its output in a layer call); the producer below skips them
    int npre = 0;
    if (warp == 0 && lane == 0 && p.w_prefetch && num_items > 0) {
        int tm0, tn, rows, ordinal;
        sched.item(cluster_id, 0, tm0, tn, rows, ordinal);
        const bool r1 = rows == 1;
        const int nst = r1 ? Cfg::STAGES1 : STAGES;
        npre = kblocks < nst ? kblocks : nst;
        const uint32_t bfull = r1 ? bar_full1 : bar_full;
        const uint32_t full0 = mapa(bfull, 0);
        const int n0 = tn * BN + (int)rank * Cfg::BN_CTA;
        const uint32_t tx = r1 ? (uint32_t)Cfg::SINGLE_TX : (uint32_t)Cfg::STAGE_BYTES;
        for (int s = 0; s < npre; ++s) {
            const uint32_t b_dst = r1 ? sA + Cfg::RING1_B + s * Cfg::B_BYTES : sB + s * Cfg::B_BYTES;
            if (leader) mbar_arrive_expect_tx(bfull + 8 * s, 2 * tx);
            tma_load_2d_pair(b_dst, &tmap_b, s * Cfg::BK, n0, full0 + 8 * s);
            tma_load_2d_pair(b_dst + Cfg::B_HALF_BYTES, &tmap_b, s * Cfg::BK + 64, n0, full0 + 8 * s);
        }
    }
    // everything above overlapped the previous kernel's tail; its results are needed from here on
    griddep_wait();

    if (warp == 0) {
        // ------------------------------------------------------------------ producer ----------
        if (lane == 0) {
            uint32_t stage = 0, phase = 0, issued = 0;
            bool ok = true;
            bool ring1 = false;  // false: the 3 x 66 KB ring of the doubles, true: the 4 x 48 KB ring of the singles
            for (int it = 0; it < num_items && ok; ++it) {
                int tm0, tn, rows, ordinal;
                sched.item(cluster_id, it, tm0, tn, rows, ordinal);
                if (rows == 1 && !ring1) {
                    // First single-tile item: the rings overlap in memory, so every stage of the doubles'
                    // ring has to be released first (the stages below `stage` were last used in this
                    // round of the ring, the others in the round before; a fresh barrier passes).
                    for (int s = 0; s < STAGES && ok; ++s)
                        ok = mbar_wait(bar_empty + 8 * s, ((uint32_t)s < stage) ? phase : (phase ^ 1u), cta_abort, p.dev_error);
                    if (!ok) break;
                    ring1 = true;
                    stage = 0;
                    phase = 0;
                }
                const uint32_t nst = ring1 ? (uint32_t)Cfg::STAGES1 : (uint32_t)STAGES;
                const uint32_t bfull = ring1 ? bar_full1 : bar_full, bempty = ring1 ? bar_empty1 : bar_empty;
                const uint32_t full0 = mapa(bfull, 0);  // the leader's barriers
                const int rb0 = tm0 * 2 + (int)rank;  // 128-row block of this CTA in the first row tile; the second: + 2
                const int n0 = tn * BN + (int)rank * Cfg::BN_CTA;
                const uint32_t tx = (rows == 2) ? (uint32_t)Cfg::STAGE_BYTES : (uint32_t)Cfg::SINGLE_TX;
                for (int kb = 0; kb < kblocks + lora_steps; ++kb) {
                    if (!mbar_wait(bempty + 8 * stage, phase ^ 1, cta_abort, p.dev_error)) {
                        ok = false;
                        break;
                    }
                    const uint32_t a_dst = ring1 ? sA + Cfg::RING1_A + stage * Cfg::A_BYTES : sA + stage * 2 * Cfg::A_BYTES;
                    const uint32_t b_dst = ring1 ? sA + Cfg::RING1_B + stage * Cfg::B_BYTES : sB + stage * Cfg::B_BYTES;
                    const uint32_t e_dst = ring1 ? sA + Cfg::RING1_E + stage * Cfg::E_BYTES : sE + stage * 2 * Cfg::E_BYTES;
                    const uint32_t bar = full0 + 8 * stage;
                    if (kb < kblocks) {
                        const bool pre = it == 0 && kb < npre;  // W tile and byte count went out before the wait
                        // the leader announces the bytes of both CTAs; the peer's bytes may land first
                        if (leader && !pre) mbar_arrive_expect_tx(bfull + 8 * stage, 2 * tx);
                        tma_load_2d_pair(a_dst, &tmap_a, kb * 64, rb0 * Cfg::BM, bar);
                        tma_load_2d_pair(e_dst, &tmap_e, 0, 2 * (rb0 * kblocks + kb), bar);
                        if (!pre) {
                            tma_load_2d_pair(b_dst, &tmap_b, kb * Cfg::BK, n0, bar);
                            tma_load_2d_pair(b_dst + Cfg::B_HALF_BYTES, &tmap_b, kb * Cfg::BK + 64, n0, bar);
                        }
                        if (rows == 2) {
                            tma_load_2d_pair(a_dst + Cfg::A_BYTES, &tmap_a, kb * 64, (rb0 + 2) * Cfg::BM, bar);
                            tma_load_2d_pair(e_dst + Cfg::E_BYTES, &tmap_e, 0, 2 * ((rb0 + 2) * kblocks + kb), bar);
                        }
                    } else {
                        // low-rank stages: T boxes in the A slots, L_A box in the first half of the W slot
                        const int j = kb - kblocks;
                        if (leader) mbar_arrive_expect_tx(bfull + 8 * stage, 2u * (uint32_t)(rows * Cfg::A_BYTES + Cfg::B_HALF_BYTES));
                        tma_load_2d_pair(a_dst, &tmap_t, j * 64, rb0 * Cfg::BM, bar);
                        if (rows == 2) tma_load_2d_pair(a_dst + Cfg::A_BYTES, &tmap_t, j * 64, (rb0 + 2) * Cfg::BM, bar);
                        tma_load_2d_pair(b_dst, &tmap_la, j * 64, n0, bar);
                    }
                    ++issued;
                    if (++stage == nst) { stage = 0; phase ^= 1; }
                }
            }
            if (!ok && issued) bounded_delay_ns(200000);  // let the copies in flight land before teardown
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer --------
        if (leader && lane == 0) {
            constexpr uint32_t idesc0 = make_idesc_sp_bf16(Cfg::BM * 2, BN), idesc1 = idesc0 | 1u;
            constexpr uint32_t idesc_dense = idesc0 & ~(1u << 2);
            const uint64_t d0 = make_desc_sw128(sA);
            const uint32_t desc_hi = (uint32_t)(d0 >> 32);
            const uint32_t ring_lo0 = (uint32_t)d0;                             // descriptor word of the ring's first byte
            const uint32_t b_lo0 = (uint32_t)make_desc_sw128(sB);
            const uint64_t e_d0 = make_desc_rows16(sE), e1_d0 = make_desc_rows16(sA + Cfg::RING1_E);
            constexpr uint32_t BH = Cfg::B_HALF_BYTES >> 4;
            uint32_t stage = 0, phase = 0;
            bool ring1 = false;
            uint32_t uses[2] = {0u, 0u};  // how often each accumulator has been handed to the epilogue
            bool ok = true;
            for (int it = 0; it < num_items && ok; ++it) {
                int tm0, tn, rows, ordinal;
                sched.item(cluster_id, it, tm0, tn, rows, ordinal);
                if (rows == 1 && !ring1) {  // the producer switches rings at the same item
                    ring1 = true;
                    stage = 0;
                    phase = 0;
                }
                const uint32_t nst = ring1 ? (uint32_t)Cfg::STAGES1 : (uint32_t)STAGES;
                const uint32_t bfull = ring1 ? bar_full1 : bar_full, bempty = ring1 ? bar_empty1 : bar_empty;
                // accumulators of this item: a double fills both, the k-th single accumulator k % 2
                const int acc0 = (rows == 2) ? 0 : (ordinal & 1);
                for (int r = 0; r < rows && ok; ++r) {
                    const int a = acc0 + r;
                    ok = mbar_wait(bar_tempty + 8 * a, (uses[a] & 1u) ^ 1u, cta_abort, p.dev_error);
                }
                if (!ok) break;
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + acc0 * BN;
                uint32_t accumulate = 0;
                for (int kb = 0; kb < kblocks + lora_steps; ++kb) {
                    if (!mbar_wait(bfull + 8 * stage, phase, cta_abort, p.dev_error)) {
                        ok = false;
                        break;
                    }
                    tc_fence_after();
                    const uint32_t a_lo = ring1 ? ring_lo0 + ((Cfg::RING1_A + stage * Cfg::A_BYTES) >> 4)
                                                : ring_lo0 + stage * (2 * Cfg::A_BYTES >> 4);
                    const uint32_t b_lo = ring1 ? ring_lo0 + ((Cfg::RING1_B + stage * Cfg::B_BYTES) >> 4)
                                                : b_lo0 + stage * (Cfg::B_BYTES >> 4);
                    if (kb < kblocks) {
                        const uint32_t e_tmem = tmem_base + Cfg::E_COL0 + (ring1 ? 4 * stage : Cfg::E_COLS * stage);
                        const uint64_t e_desc = ring1 ? e1_d0 + (uint64_t)(stage * (Cfg::E_BYTES >> 4))
                                                      : e_d0 + (uint64_t)(stage * (2 * Cfg::E_BYTES >> 4));
                        tmem_cp_128x128b<2>(e_tmem, e_desc);
                        if (rows == 2) tmem_cp_128x128b<2>(e_tmem + 4, e_desc + (uint64_t)(Cfg::E_BYTES >> 4));
                        // four K steps of 32 logical elements per row tile: A advances 32 bytes, W 64 bytes
                        // (steps 2, 3 in the second 64-element slice); metadata column pair + step parity
                        mma_sp_bf16_lh<2>(d_tmem, a_lo, b_lo, desc_hi, e_tmem, idesc0, accumulate);
                        mma_sp_bf16_lh<2>(d_tmem, a_lo + 2, b_lo + 4, desc_hi, e_tmem, idesc1, 1u);
                        mma_sp_bf16_lh<2>(d_tmem, a_lo + 4, b_lo + BH, desc_hi, e_tmem + 2, idesc0, 1u);
                        mma_sp_bf16_lh<2>(d_tmem, a_lo + 6, b_lo + BH + 4, desc_hi, e_tmem + 2, idesc1, 1u);
                        if (rows == 2) {
                            constexpr uint32_t A1 = Cfg::A_BYTES >> 4;
                            mma_sp_bf16_lh<2>(d_tmem + BN, a_lo + A1, b_lo, desc_hi, e_tmem + 4, idesc0, accumulate);
                            mma_sp_bf16_lh<2>(d_tmem + BN, a_lo + A1 + 2, b_lo + 4, desc_hi, e_tmem + 4, idesc1, 1u);
                            mma_sp_bf16_lh<2>(d_tmem + BN, a_lo + A1 + 4, b_lo + BH, desc_hi, e_tmem + 6, idesc0, 1u);
                            mma_sp_bf16_lh<2>(d_tmem + BN, a_lo + A1 + 6, b_lo + BH + 4, desc_hi, e_tmem + 6, idesc1, 1u);
                        }
                    } else {
                        // low-rank stage: dense K steps of 16 elements, both operands advance 32 bytes
                        for (int r = 0; r < rows; ++r) {
                            const uint32_t dt = d_tmem + r * BN, al = a_lo + r * (Cfg::A_BYTES >> 4);
                            mma_bf16_lh<2>(dt, al, b_lo, desc_hi, idesc_dense, accumulate);
                            mma_bf16_lh<2>(dt, al + 2, b_lo + 2, desc_hi, idesc_dense, 1u);
                            mma_bf16_lh<2>(dt, al + 4, b_lo + 4, desc_hi, idesc_dense, 1u);
                            mma_bf16_lh<2>(dt, al + 6, b_lo + 6, desc_hi, idesc_dense, 1u);
                        }
                    }
                    accumulate = 1u;
                    tc_commit_pair(bempty + 8 * stage, 0x3);
                    if (++stage == nst) { stage = 0; phase ^= 1; }
                }
                if (!ok) break;
                for (int r = 0; r < rows; ++r) {
                    tc_commit_pair(bar_tfull + 8 * (acc0 + r), 0x3);
                    ++uses[acc0 + r];
                }
            }
        }
    } else {
        // ------------------------------------------------------------------ epilogue ----------
        const int g = (warp - 2) >> 2;  // the accumulator this warp drains
        const int q = warp & 3;         // tensor-memory lane quarter this warp may read
        const uint32_t tempty0 = mapa(bar_tempty, 0);
        const uint32_t cbuf = sC + (warp - 2) * Cfg::C_BOX_BYTES;
        uint32_t uses = 0;
        constexpr int CH = Cfg::CH, NCH = Cfg::NCH;
        for (int it = 0; it < num_items; ++it) {
            int tm0, tn, rows, ordinal;
            sched.item(cluster_id, it, tm0, tn, rows, ordinal);
            int tm;
            if (rows == 2) tm = tm0 + g;
            else if ((ordinal & 1) == g) tm = tm0;
            else continue;
            const int m0 = (tm * 2 + (int)rank) * Cfg::BM + q * 32;
            const int64_t row = m0 + lane;
            const bool row_ok = row < p.M;
            // the row's scale (or its sum from the prune launch's partial sums) and the tile's bias
            // values, one column per lane and round, are fetched while the main loop still runs
            float s = 1.0f;
            if (row_ok) {
                if (p.scale_partial != nullptr) s = row_scale_from_partials(p.scale_partial, row, p.scale_ks);
                else if (p.row_scale != nullptr) s = __ldg(p.row_scale + row);
            }
            // the item's bias values go to this warp's own strip of shared memory (30 lanes x 8 bf16);
            // the conversion below reads them back as broadcast 16-byte loads (a shuffle per value
            // made the shuffle unit the bottleneck of the five conversion rounds)
            const uint32_t sb = sBias + (warp - 2) * Cfg::BIAS_BYTES;
            if (lane < BN / 8) {
                const int n = tn * BN + lane * 8;
                uint4 bq = make_uint4(0u, 0u, 0u, 0u);
                if (p.bias != nullptr && n < p.N) bq = __ldg(reinterpret_cast<const uint4*>(p.bias + n));
                sts128(sb + lane * 16, bq.x, bq.y, bq.z, bq.w);
            }
            __syncwarp();
            if (!mbar_wait(bar_tfull + 8 * g, uses & 1u, cta_abort, p.dev_error)) break;
            ++uses;
            tc_fence_after();
            const uint32_t t_row = tmem_base + ((uint32_t)(q * 32) << 16) + g * BN;
            const uint16_t* rrow = (p.residual != nullptr) ? p.residual + row * p.ldr : nullptr;
            if (rrow == nullptr) {
                // Fast path (no residual addend): the whole accumulator row is converted to packed
                // bf16 in registers first, so the accumulator goes back to the MMA issuer after five
                // tcgen05.ld round trips; the stores follow while the next main loop already runs.
                uint32_t packed[NCH][CH / 2];
#pragma unroll
                for (int c = 0; c < NCH; ++c) {
                    uint32_t v[CH];
                    tmem_ld_32x32b_x32(t_row + c * CH, *reinterpret_cast<uint32_t(*)[32]>(&v[0]));
                    tmem_ld_32x32b_x16(t_row + c * CH + 32, *reinterpret_cast<uint32_t(*)[16]>(&v[32]));
                    tmem_ld_wait();
                    if (c == NCH - 1) {
                        // accumulator fully read: hand it back to the MMA issuer
                        tc_fence_before();
                        __syncwarp();
                        if (lane == 0) mbar_arrive_cluster(tempty0 + 8 * g);
                    }
#pragma unroll
                    for (int j = 0; j < CH / 8; ++j) {
                        uint32_t bq[4];
                        lds128(sb + c * (CH * 2) + j * 16, bq[0], bq[1], bq[2], bq[3]);
#pragma unroll
                        for (int e = 0; e < 4; ++e)
                            packed[c][4 * j + e] = pack_bf16x2(fmaf(s, __uint_as_float(v[8 * j + 2 * e]), bf16_lo_f(bq[e])),
                                                               fmaf(s, __uint_as_float(v[8 * j + 2 * e + 1]), bf16_hi_f(bq[e])));
                    }
                }
#pragma unroll
                for (int c = 0; c < NCH; ++c) {
                    const int n0 = tn * BN + c * CH;
                    if (n0 >= p.N) continue;
                    // the staging box must have been read by this warp's previous TMA store
                    if (lane == 0) tma_store_wait_read<0>();
                    __syncwarp();
#pragma unroll
                    for (int j = 0; j < CH / 8; ++j)  // dense 96-byte rows
                        sts128(cbuf + lane * (CH * 2) + (j << 4), packed[c][4 * j], packed[c][4 * j + 1], packed[c][4 * j + 2],
                               packed[c][4 * j + 3]);
                    fence_proxy_async_smem();
                    __syncwarp();
                    if (lane == 0) {
                        tma_store_2d(&tmap_y, n0, m0, cbuf);  // rows past M and columns past N are clipped
                        tma_store_commit();
                    }
                }
                continue;
            }
            // With a residual addend (its values have to be fetched per chunk): chunk by chunk, the
            // next chunk's accumulators travelling while the current one is converted and stored.
            uint32_t v[2][CH];
            tmem_ld_32x32b_x32(t_row, *reinterpret_cast<uint32_t(*)[32]>(&v[0][0]));
            tmem_ld_32x32b_x16(t_row + 32, *reinterpret_cast<uint32_t(*)[16]>(&v[0][32]));
#pragma unroll
            for (int c = 0; c < NCH; ++c) {
                tmem_ld_wait();
                if (c + 1 < NCH) {
                    tmem_ld_32x32b_x32(t_row + (c + 1) * CH, *reinterpret_cast<uint32_t(*)[32]>(&v[(c + 1) & 1][0]));
                    tmem_ld_32x32b_x16(t_row + (c + 1) * CH + 32, *reinterpret_cast<uint32_t(*)[16]>(&v[(c + 1) & 1][32]));
                } else {
                    // accumulator fully read: hand it back to the MMA issuer
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive_cluster(tempty0 + 8 * g);
                }
                const int n0 = tn * BN + c * CH;
                if (n0 >= p.N) continue;
                const uint32_t* vc = v[c & 1];
                // the staging box must have been read by this warp's previous TMA store
                if (lane == 0) tma_store_wait_read<0>();
                __syncwarp();
#pragma unroll
                for (int j = 0; j < CH / 8; ++j) {  // 8 columns (16 bytes of output) at a time
                    const int n = n0 + j * 8;
                    float bv[8];
                    {
                        uint32_t bq[4];
                        lds128(sb + c * (CH * 2) + j * 16, bq[0], bq[1], bq[2], bq[3]);
#pragma unroll
                        for (int e = 0; e < 4; ++e) {
                            bv[2 * e] = bf16_lo_f(bq[e]);
                            bv[2 * e + 1] = bf16_hi_f(bq[e]);
                        }
                    }
                    float r[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
                    if (n < p.N && row_ok) {
                        const uint4 rv = __ldg(reinterpret_cast<const uint4*>(rrow + n));
                        r[0] = bf16_lo_f(rv.x); r[1] = bf16_hi_f(rv.x);
                        r[2] = bf16_lo_f(rv.y); r[3] = bf16_hi_f(rv.y);
                        r[4] = bf16_lo_f(rv.z); r[5] = bf16_hi_f(rv.z);
                        r[6] = bf16_lo_f(rv.w); r[7] = bf16_hi_f(rv.w);
                    }
                    uint32_t o[4];
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        const float y0 = fmaf(s, __uint_as_float(vc[j * 8 + 2 * e]), bv[2 * e]) + r[2 * e];
                        const float y1 = fmaf(s, __uint_as_float(vc[j * 8 + 2 * e + 1]), bv[2 * e + 1]) + r[2 * e + 1];
                        o[e] = pack_bf16x2(y0, y1);
                    }
                    sts128(cbuf + lane * (CH * 2) + (j << 4), o[0], o[1], o[2], o[3]);  // dense 96-byte rows
                }
                fence_proxy_async_smem();
                __syncwarp();
                if (lane == 0) {
                    tma_store_2d(&tmap_y, n0, m0, cbuf);  // rows past M and columns past N are clipped
                    tma_store_commit();
                }
            }
        }
        if (lane == 0) tma_store_wait_all<0>();
    }

    // ---------------------------------------------------------------------- teardown ----------
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc<2>(tmem_base, Cfg::TMEM_COLS);
    }
}

}  // namespace lynx

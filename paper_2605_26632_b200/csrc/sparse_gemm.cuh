// 2:4 sparse x dense GEMM with fused epilogue for sm_100a (Algorithm 1 lines 5-6):
//     Y[m, n] = bf16( s_m * sum_k X~[m,k] W[n,k] + bias[n] + Yr[m,n] )
// X~ arrives compressed: values [M x K/2] bf16 and hardware-order 2-bit index metadata.
//
// Persistent, warp-specialised kernel.  Per CTA (or CTA pair when CG == 2):
//   warp 0      producer: TMA loads of the compressed-A tile (128 rows x 64 stored values =
//               128 logical K), the metadata block (2048 bytes) and the W tile into a ring of
//               STAGES shared-memory stages guarded by full/empty mbarriers
//   warp 1      MMA issuer (one thread): copies the stage's metadata into tensor memory
//               (tcgen05.cp), issues four tcgen05.mma.sp kind::f16 (K = 32 logical each) into a
//               tensor-memory fp32 accumulator, commits to the stage's empty barrier; after the
//               last K block commits to the accumulator's full barrier
//   warps 2..5  epilogue: tcgen05.ld the accumulator (each warp its 32-lane quarter), apply
//               row scale / bias / residual, round to bf16, stage in swizzled shared memory and
//               TMA-store 32 x 64 boxes
// With two accumulator buffers the epilogue of tile i overlaps the main loop of tile i+1.
//
// Low-rank branch (Algorithm 1 lines 5-6, Y = Y_s + X (L_A L_B)^T): when lora_steps > 0 every
// tile gets lora_steps extra ring stages after its last K block.  Such a stage holds a 128 x 64
// box of T = (X L_B^T) / s (bf16, produced by lora_down_kernel) in the A slot and a BN x 64 box of
// L_A in the W slot, and the issuer adds T L_A^T with four DENSE tcgen05.mma (K = 16 each) into
// the same accumulator, so Y_r never exists in memory and the epilogue's s_m * acc restores it.
//
// With l0_fused the kernel also computes T itself before its first tile ("phase 0"): the work
// items (256-row block, K split) of X L_B^T are dealt round-robin to the clusters and run through
// the same ring (a stage then holds two 128 x 64 boxes of the DENSE X and two R-row boxes of L_B,
// eight dense K = 16 steps) into a 64-column accumulator.  Each epilogue warp writes its 32 rows as
// an fp32 partial, takes a ticket of its 32-row group, and the warp that draws the group's last
// ticket adds the splits in ascending order, multiplies by 1 / s_m, writes the bf16 rows of T and
// publishes the group's ready word (the launch epoch).  The producer waits (bounded) for the
// four ready words of its rows before it loads a tile's T box -- by then a whole main loop has
// passed, so the wait is normally already satisfied.  Every cluster finishes its phase-0 items
// before it can wait for anyone, so the waits cannot deadlock.
//
// CG == 2: the pair computes a 256 x BN tile; each CTA stages its own 128 rows of A and
// metadata and its own BN/2 rows of W (plain TMA loads, no multicast), the leader CTA issues
// cta_group::2 MMAs, and each CTA drains its own 128 accumulator rows.
#pragma once

#include "ptx.cuh"
#include "prune_compress.cuh"  // row_scale_from_partials

namespace lynx {

struct GemmParams {
    int64_t M, N, K;
    const float* row_scale;    // [M] or nullptr
    const float* scale_partial;  // or: per-K-split row sums of a deferred prune launch (see
    int scale_ks;                //     row_scale_from_partials), scale_ks splits per 16-row block
    const float* col_scale;      // [N] per-output-channel factor (FP8 weight scales) or nullptr
    const uint16_t* bias;      // [N] bf16 or nullptr
    const uint16_t* residual;  // [M x N] bf16 (ld = ldr) or nullptr
    int64_t ldr;
    uint32_t* dev_error;  // sticky error word (host-visible)
    int tiles_m, tiles_n;
    int group_m;  // tile order: groups of `group_m` row tiles are swept over all of N before the next group
    // stream-K tail (see TileSchedule): fp32 partial tiles, one slot per cluster, and one ready
    // word per (slot, epilogue warp of the pair) holding the launch epoch; nullptr = off
    float* sk_partial;
    uint32_t* sk_flags;
    uint32_t sk_epoch;
    int lora_steps;  // R / 64 extra dense stages per tile (0 = no low-rank branch)
    // phase 0 (l0_fused): T = (X L_B^T) / s computed by this launch, R = 64
    int l0_fused;
    int l0_splits, l0_kb_per_split;  // K splits per 256-row block, 128-element K blocks per split
    int l0_light0, l0_fill;          // see L0Schedule
    float* l0_partial;     // [row block][split][16 pieces][rows of the block] float4
    uint32_t* l0_tickets;  // one word per 32-row group, zero between launches
    uint32_t* l0_ready;    // one word per 32-row group: epoch of the launch that finished its T rows
    uint32_t l0_epoch;
    uint32_t* l0_done;     // running count of published groups over all launches of the context
    uint32_t l0_done_target;  // its value once this launch has published all of its groups
    uint16_t* T;           // [M x 64] bf16, leading dimension ldt
    int64_t ldt;
    // Layer calls: W is not produced by the kernel in front of this one (the library's own prune
    // launch), so the W tiles of the first ring stages may be fetched before the wait for that
    // kernel; the direct GEMM entry points leave this 0 (whatever precedes them might write W).
    int w_prefetch;
};

// Work distribution over C persistent clusters.  The first floor(T/C)*C tiles go round-robin,
// whole.  The K blocks of the remaining R < C tiles are dealt out evenly ("stream-K" tail):
// cluster c gets tail blocks [c*R*KB/C, (c+1)*R*KB/C), at most two pieces of two tiles.  A piece
// that ends at its tile's last K block makes that cluster the tile's owner; every other piece
// is written out as an fp32 partial tile, and the owner adds the partials of the clusters before
// it in ascending order (fixed order: reproducible).  A cluster does its partial piece first, so
// nobody who is waited for ever waits.
struct WorkItem {
    int tile, kb0, kb1;
    int kind;           // 0 whole tile, 1 partial piece (write fp32), 2 owner piece (add partials)
    int first_contrib;  // owner: clusters first_contrib .. c-1 hold the partials
};
// Tile index -> (row tile, column tile).  Inside a group of `group_m` row tiles the row index runs
// fastest, the groups follow one another: the tiles that run at the same time then share
// group_m blocks of A and tiles / group_m blocks of W, whatever M is (with one group over all of
// M a wave of a tall problem would stream the whole of A from HBM once per column tile).
__device__ __forceinline__ void tile_coords(int tile, int tiles_m, int tiles_n, int group_m, int& tm, int& tn) {
    const int per_group = group_m * tiles_n;
    const int g = tile / per_group, r = tile - g * per_group;
    const int rows = (tiles_m - g * group_m < group_m) ? tiles_m - g * group_m : group_m;
    tn = r / rows;
    tm = g * group_m + (r - tn * rows);
}

struct TileSchedule {
    int T, C, KB, full, R, total;
    bool streamk;
    __device__ TileSchedule(int tiles, int clusters, int kblocks, bool enable)
        : T(tiles), C(clusters), KB(kblocks) {
        full = (T / C) * C;
        R = T - full;
        total = R * KB;
        streamk = enable && R > 0;
        if (!streamk) { full = T; R = 0; total = 0; }
    }
    // cluster that holds tail block x
    __device__ int owner_of(int x) const { return (int)((((long long)x + 1) * C - 1) / total); }
    // does cluster c hold a piece of the tail?
    __device__ bool has_tail(int c) const {
        return streamk && (int)((long long)(c + 1) * total / C) > (int)((long long)c * total / C);
    }
    __device__ int count(int c) const {
        int n = 0;
        for (int t = c; t < full; t += C) ++n;
        if (streamk) {
            const int s = (int)((long long)c * total / C), e = (int)((long long)(c + 1) * total / C);
            if (e > s) n += ((e - 1) / KB != s / KB) ? 2 : 1;
        }
        return n;
    }
    __device__ WorkItem get(int c, int i) const {
        WorkItem w{0, 0, KB, 0, 0};
        const int nfull = (full - c + C - 1) / C > 0 ? (full - c + C - 1) / C : 0;
        if (i < nfull) { w.tile = c + i * C; return w; }
        i -= nfull;
        const int s = (int)((long long)c * total / C), e = (int)((long long)(c + 1) * total / C);
        const int tA = s / KB, tB = (e - 1) / KB;
        // pieces: A = [s, min(e, (tA+1)KB)) of tile tA, B = [tB*KB, e) of tile tB (if tB != tA)
        int a0 = s - tA * KB, a1 = ((e < (tA + 1) * KB) ? e : (tA + 1) * KB) - tA * KB;
        int b0 = 0, b1 = e - tB * KB;
        const bool two = tB != tA;
        const bool a_partial = a1 != KB;            // does not reach the tile's end
        const bool b_partial = two && b1 != KB;
        // order: partial piece first
        bool take_b;
        if (!two) take_b = false;
        else take_b = (i == 0) ? (b_partial && !a_partial) : !(b_partial && !a_partial);
        if (take_b) { w.tile = full + tB; w.kb0 = b0; w.kb1 = b1; }
        else { w.tile = full + tA; w.kb0 = a0; w.kb1 = a1; }
        if (w.kb1 != KB) w.kind = 1;
        else if (w.kb0 != 0) { w.kind = 2; w.first_contrib = owner_of((w.tile - full) * KB); }
        else w.kind = 0;
        return w;
    }
};

// Which cluster runs which phase-0 item.  With T tiles over C clusters the clusters c >= T % C
// ("light") have one tile fewer than the others, i.e. a whole tile time of slack: the first
// light * fill items go to them, round-robin (the host sets fill so that either all items fit
// there or fill = 0), the rest round-robin over all clusters.  light0 = C: no light clusters.
struct L0Schedule {
    int items, C, light0, L, cap;
    __device__ L0Schedule(int items_, int clusters, int light0_, int fill) : items(items_), C(clusters), light0(light0_) {
        L = C - light0;
        cap = L * fill;
        if (cap > items) cap = items;
    }
    __device__ int light_count(int c) const {
        const int lc = c - light0;
        return (lc >= 0 && cap > lc) ? (cap - lc + L - 1) / L : 0;
    }
    __device__ int count(int c) const {
        const int rest = items - cap;
        return light_count(c) + ((rest > c) ? (rest - c + C - 1) / C : 0);
    }
    __device__ int item(int c, int li) const {
        const int nl = light_count(c);
        return (li < nl) ? (c - light0) + li * L : cap + c + (li - nl) * C;
    }
};

// FP8_ = true: E4M3 operands (one byte per element).  The byte geometry of a stage is the same
// (a 128-byte swizzled row of compressed A is then 256 logical K instead of 128, a 128-byte row of
// W 128 K instead of 64), the metadata of a stage doubles (two 128 x 128 blocks), and the four MMAs
// of a stage are kind::f8f6f4 with K = 64 each.
template <int BN_, int CG_, int STAGES_, int CBUFS_, bool FP8_ = false, int CH_ = 0>
struct GemmCfg {
    static constexpr int BN = BN_, CG = CG_, STAGES = STAGES_, CBUFS = CBUFS_;
    static constexpr bool FP8 = FP8_;
    static constexpr int BM = 128;  // rows per CTA
    static constexpr int BK = FP8 ? 256 : 128;  // logical K per stage
    static constexpr int A_BOX_X = FP8 ? 128 : 64;  // stored A elements per 128-byte row
    static constexpr int B_BOX_X = FP8 ? 128 : 64;  // W elements per 128-byte row
    static constexpr int BN_CTA = BN / CG;
    static constexpr int A_BYTES = BM * 128;              // 128 swizzled rows of 128 bytes: 16 KB
    static constexpr int B_HALF_BYTES = BN_CTA * 128;     // one 128-byte K slice of the W tile
    static constexpr int B_BYTES = 2 * B_HALF_BYTES;
    static constexpr int E_BYTES = FP8 ? 4096 : 2048;
    static constexpr int E_COLS = E_BYTES / 512;  // tensor-memory columns of a stage's metadata
    static constexpr int STAGE_BYTES = A_BYTES + B_BYTES + E_BYTES;
    // epilogue chunk: 64 columns (128-byte swizzled staging rows) when BN allows, else 48 columns
    // (96-byte unswizzled rows) -- BN = 240 is the widest tile that leaves room for two
    // accumulator buffers plus the metadata columns in the 512 columns of tensor memory
    static constexpr int CH = CH_ ? CH_ : ((BN % 64 == 0) ? 64 : 48);  // (CH_: narrower staging boxes where shared memory is short)
    static constexpr int C_BOX_BYTES = 32 * CH * 2;  // one warp's 32 x CH bf16 store box
    static constexpr int C_BYTES = 4 * CBUFS * C_BOX_BYTES;
    static constexpr int ACC_STAGES = (2 * BN + E_COLS * STAGES <= 512) ? 2 : 1;
    static constexpr int E_COL0 = ACC_STAGES * BN;  // metadata columns start after accumulators
    static constexpr int TMEM_COLS = 512;
    static constexpr int NUM_BARS = 2 * STAGES + 2 * ACC_STAGES;
    static constexpr int SMEM_BYTES = 1024 /*align slack*/ + STAGES * STAGE_BYTES + C_BYTES + 256;
    // Epilogue warps: four (one per tensor-memory lane quarter), or eight for FP8 -- two per quarter
    // that take alternate column chunks, each with one staging box.  A tile's epilogue takes ~6 us
    // with four warps, which an FP8 main loop at K = 3072 (6.5 us) no longer hides.
    static constexpr int EPI_WARPS = FP8 ? 8 : 4;
    static constexpr int EPI_SPLIT = EPI_WARPS / 4;          // warps per lane quarter
    static constexpr int CBUFS_W = 4 * CBUFS / EPI_WARPS;    // staging boxes per epilogue warp
    static constexpr int THREADS = 64 + 32 * EPI_WARPS;
    static_assert(CBUFS_W >= 1, "every epilogue warp needs a staging box");
    static_assert(BN % 16 == 0 && (BN / CG) % 8 == 0 && BN <= 256, "tile N");
    static_assert(BN % CH == 0, "epilogue works on whole chunks");
    static_assert(C_BOX_BYTES % 1024 == 0, "staging boxes stay 1024-byte aligned");
    static_assert(B_HALF_BYTES % 1024 == 0, "swizzle atoms need 1024-byte aligned tiles");
    static_assert(E_COL0 % 4 == 0 && E_COL0 + E_COLS * STAGES <= TMEM_COLS, "tensor memory budget");
    static_assert(SMEM_BYTES <= 227 * 1024, "shared memory budget");
    // phase 0 stage (rank 64): L_B boxes at the start of the W slot, second X box behind them
    static constexpr int L0_R = 64;
    static constexpr int L0_LB_BYTES = (L0_R / CG) * 64 * 2;
    static constexpr int L0_X2_OFF = (2 * L0_LB_BYTES + 1023) / 1024 * 1024;
    static constexpr int L0_STAGE_BYTES = 2 * A_BYTES + 2 * L0_LB_BYTES;
    static constexpr bool L0_OK = !FP8 && L0_X2_OFF + A_BYTES <= B_BYTES;
};

// Instruction descriptor of tcgen05.mma.sp kind::f16: bf16 x bf16 -> fp32, both operands
// K-major, sparse, M x N per instruction (clearing bit 2 gives the dense instruction's).
__host__ __device__ constexpr uint32_t make_idesc_sp_bf16(int m, int n) {
    return (1u << 2)                        // sparse
           | (1u << 4)                      // D format: fp32
           | (1u << 7)                      // A format: bf16
           | (1u << 10)                     // B format: bf16
           | ((uint32_t)(n >> 3) << 17)     // N / 8
           | ((uint32_t)(m >> 4) << 24);    // M / 16
}
// The same for kind::f8f6f4 with E4M3 operands (format code 0 in both operand fields).
__host__ __device__ constexpr uint32_t make_idesc_sp_e4m3(int m, int n) {
    return (1u << 2) | (1u << 4) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(m >> 4) << 24);
}

// LORA = false is the plain layer: the low-rank stages and phase 0 are compiled out, so the hot
// kernel carries none of their registers or parameters' uses.
template <class Cfg, bool LORA>
__global__ void __launch_bounds__(Cfg::THREADS, 1)
sparse_gemm_kernel(const __grid_constant__ CUtensorMap tmap_a, const __grid_constant__ CUtensorMap tmap_b,
                   const __grid_constant__ CUtensorMap tmap_e, const __grid_constant__ CUtensorMap tmap_y,
                   const __grid_constant__ CUtensorMap tmap_t, const __grid_constant__ CUtensorMap tmap_la,
                   const __grid_constant__ CUtensorMap tmap_x, const __grid_constant__ CUtensorMap tmap_lb,
                   const GemmParams p) {
    constexpr int CG = Cfg::CG, STAGES = Cfg::STAGES, BN = Cfg::BN;
    constexpr bool L0 = LORA && Cfg::L0_OK;
    const int lora_steps = LORA ? p.lora_steps : 0;
    extern __shared__ uint8_t smem_raw[];
    // 1024-byte alignment for the swizzled tiles
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* smem_gen = smem_raw + (smem_base - smem_u32(smem_raw));
    const uint32_t sA = smem_base;
    const uint32_t sB = sA + STAGES * Cfg::A_BYTES;
    const uint32_t sE = sB + STAGES * Cfg::B_BYTES;
    const uint32_t sC = sE + STAGES * Cfg::E_BYTES;
    const uint32_t sBar = sC + Cfg::C_BYTES;
    const uint32_t bar_full = sBar, bar_empty = sBar + 8 * STAGES;
    const uint32_t bar_tfull = sBar + 16 * STAGES, bar_tempty = bar_tfull + 8 * Cfg::ACC_STAGES;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem_gen + (sBar - smem_base) + 8 * Cfg::NUM_BARS);
    volatile uint32_t* cta_abort = tmem_slot + 1;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = (CG == 2) ? cluster_ctarank() : 0u;
    const bool leader = rank == 0;
    const int cluster_id = blockIdx.x / CG, num_clusters = gridDim.x / CG;
    const int num_tiles = p.tiles_m * p.tiles_n;
    const int kblocks = (int)(p.K / Cfg::BK);
    const TileSchedule sched(num_tiles, num_clusters, kblocks, p.sk_partial != nullptr);
    const int num_items = sched.count(cluster_id);
    // phase 0 items of this cluster: item -> (row block = item % tiles_m, K split = item / tiles_m)
    const int l0_items = (L0 && p.l0_fused) ? p.tiles_m * p.l0_splits : 0;
    const L0Schedule l0s(l0_items, num_clusters, p.l0_light0, p.l0_fill);
    const int l0_n = L0 ? l0s.count(cluster_id) : 0;

    if (threadIdx.x == 0) {
        *cta_abort = 0;
        for (int s = 0; s < STAGES; ++s) {
            mbar_init(bar_full + 8 * s, 1);   // leader's producer arrives once (+ transaction bytes)
            mbar_init(bar_empty + 8 * s, 1);  // one tcgen05.commit
        }
        for (int a = 0; a < Cfg::ACC_STAGES; ++a) {
            mbar_init(bar_tfull + 8 * a, 1);         // one tcgen05.commit
            mbar_init(bar_tempty + 8 * a, Cfg::EPI_WARPS * CG);  // one arrive per epilogue warp of the pair
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
        if (L0 && p.l0_fused) {
            prefetch_tmap(&tmap_x);
            prefetch_tmap(&tmap_lb);
        }
    }
    if (warp == 1) {
        tmem_alloc<CG>(smem_u32(tmem_slot), Cfg::TMEM_COLS);
        tmem_relinquish<CG>();
    }
    tc_fence_before();
    __syncthreads();
    if constexpr (CG == 2) cluster_sync_all();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    // W tiles of the first stages of the first tile, before the wait for the previous kernel
    int npre = 0;
    if (warp == 0 && lane == 0 && p.w_prefetch && num_items > 0 && l0_n == 0) {
        const WorkItem w = sched.get(cluster_id, 0);
        int tm, tn;
        tile_coords(w.tile, p.tiles_m, p.tiles_n, p.group_m, tm, tn);
        const int n0 = tn * BN + (int)rank * Cfg::BN_CTA;
        npre = (w.kb1 - w.kb0 < STAGES) ? w.kb1 - w.kb0 : STAGES;
        const uint32_t full0 = (CG == 2) ? mapa(bar_full, 0) : bar_full;
        for (int s = 0; s < npre; ++s) {
            const int kb = w.kb0 + s;
            const uint32_t b_dst = sB + s * Cfg::B_BYTES;
            if constexpr (CG == 1) {
                mbar_arrive_expect_tx(bar_full + 8 * s, Cfg::STAGE_BYTES);
                tma_load_2d(b_dst, &tmap_b, kb * Cfg::BK, n0, bar_full + 8 * s);
                tma_load_2d(b_dst + Cfg::B_HALF_BYTES, &tmap_b, kb * Cfg::BK + Cfg::B_BOX_X, n0, bar_full + 8 * s);
            } else {
                if (leader) mbar_arrive_expect_tx(bar_full + 8 * s, 2 * Cfg::STAGE_BYTES);
                tma_load_2d_pair(b_dst, &tmap_b, kb * Cfg::BK, n0, full0 + 8 * s);
                tma_load_2d_pair(b_dst + Cfg::B_HALF_BYTES, &tmap_b, kb * Cfg::BK + Cfg::B_BOX_X, n0, full0 + 8 * s);
            }
        }
    }
    // everything above overlapped the previous kernel's tail; its results are needed from here on
    griddep_wait();

    if (warp == 0) {
        // ------------------------------------------------------------------ producer ----------
        if (lane == 0) {
            uint32_t stage = 0, phase = 0;
            uint32_t issued = 0;
            bool ok = true;
            bool l0_all_done = false;
            const uint32_t full0 = (CG == 2) ? mapa(bar_full, 0) : bar_full;  // leader's barriers
            constexpr int E_ROWS = Cfg::E_BYTES / 1024;  // 1024-byte rows of the metadata tensor map per stage
            if constexpr (L0) {
                // phase 0: dense X boxes and L_B boxes of this cluster's (row block, K split) items
                for (int li = 0; li < l0_n && ok; ++li) {
                    const int item = l0s.item(cluster_id, li);
                    const int tmb = item % p.tiles_m, split = item / p.tiles_m;
                    const int m0 = (tmb * CG + (int)rank) * Cfg::BM;
                    const int lb_row0 = (int)rank * (Cfg::L0_R / CG);
                    const int k0 = split * p.l0_kb_per_split;
                    const int k1 = (k0 + p.l0_kb_per_split < kblocks) ? k0 + p.l0_kb_per_split : kblocks;
                    for (int kb = k0; kb < k1; ++kb) {
                        if (!mbar_wait(bar_empty + 8 * stage, phase ^ 1, cta_abort, p.dev_error)) {
                            ok = false;
                            break;
                        }
                        const uint32_t a_dst = sA + stage * Cfg::A_BYTES;
                        const uint32_t b_dst = sB + stage * Cfg::B_BYTES;
                        if constexpr (CG == 1) {
                            const uint32_t bar = bar_full + 8 * stage;
                            mbar_arrive_expect_tx(bar, Cfg::L0_STAGE_BYTES);
                            tma_load_2d(a_dst, &tmap_x, kb * 128, m0, bar);
                            tma_load_2d(b_dst + Cfg::L0_X2_OFF, &tmap_x, kb * 128 + 64, m0, bar);
                            tma_load_2d(b_dst, &tmap_lb, kb * 128, lb_row0, bar);
                            tma_load_2d(b_dst + Cfg::L0_LB_BYTES, &tmap_lb, kb * 128 + 64, lb_row0, bar);
                        } else {
                            const uint32_t bar = full0 + 8 * stage;
                            if (leader) mbar_arrive_expect_tx(bar_full + 8 * stage, 2 * Cfg::L0_STAGE_BYTES);
                            tma_load_2d_pair(a_dst, &tmap_x, kb * 128, m0, bar);
                            tma_load_2d_pair(b_dst + Cfg::L0_X2_OFF, &tmap_x, kb * 128 + 64, m0, bar);
                            tma_load_2d_pair(b_dst, &tmap_lb, kb * 128, lb_row0, bar);
                            tma_load_2d_pair(b_dst + Cfg::L0_LB_BYTES, &tmap_lb, kb * 128 + 64, lb_row0, bar);
                        }
                        ++issued;
                        if (++stage == STAGES) { stage = 0; phase ^= 1; }
                    }
                }
            }
            for (int wi = 0; wi < num_items && ok; ++wi) {
                const WorkItem w = sched.get(cluster_id, wi);
                int tm, tn;
                tile_coords(w.tile, p.tiles_m, p.tiles_n, p.group_m, tm, tn);
                const int m0 = (tm * CG + (int)rank) * Cfg::BM;
                const int n0 = tn * BN + (int)rank * Cfg::BN_CTA;
                const int eblk = (tm * CG + (int)rank) * kblocks;
                for (int kb = w.kb0; kb < w.kb1; ++kb) {
                    if (!mbar_wait(bar_empty + 8 * stage, phase ^ 1, cta_abort, p.dev_error)) {
                        ok = false;
                        break;
                    }
                    const uint32_t a_dst = sA + stage * Cfg::A_BYTES;
                    const uint32_t b_dst = sB + stage * Cfg::B_BYTES;
                    const uint32_t e_dst = sE + stage * Cfg::E_BYTES;
                    // (the W tiles and the byte count of the first npre stages were issued before the wait)
                    const bool pre = wi == 0 && kb - w.kb0 < npre;
                    if constexpr (CG == 1) {
                        const uint32_t bar = bar_full + 8 * stage;
                        if (!pre) mbar_arrive_expect_tx(bar, Cfg::STAGE_BYTES);
                        tma_load_2d(a_dst, &tmap_a, kb * Cfg::A_BOX_X, m0, bar);
                        tma_load_2d(e_dst, &tmap_e, 0, E_ROWS * (eblk + kb), bar);
                        if (!pre) {
                            tma_load_2d(b_dst, &tmap_b, kb * Cfg::BK, n0, bar);
                            tma_load_2d(b_dst + Cfg::B_HALF_BYTES, &tmap_b, kb * Cfg::BK + Cfg::B_BOX_X, n0, bar);
                        }
                    } else {
                        const uint32_t bar = full0 + 8 * stage;
                        // the leader announces the bytes of both CTAs; the peer's bytes may land
                        // first (the count goes negative for a moment, which is allowed)
                        if (leader && !pre) mbar_arrive_expect_tx(bar_full + 8 * stage, 2 * Cfg::STAGE_BYTES);
                        tma_load_2d_pair(a_dst, &tmap_a, kb * Cfg::A_BOX_X, m0, bar);
                        tma_load_2d_pair(e_dst, &tmap_e, 0, E_ROWS * (eblk + kb), bar);
                        if (!pre) {
                            tma_load_2d_pair(b_dst, &tmap_b, kb * Cfg::BK, n0, bar);
                            tma_load_2d_pair(b_dst + Cfg::B_HALF_BYTES, &tmap_b, kb * Cfg::BK + Cfg::B_BOX_X, n0, bar);
                        }
                    }
                    ++issued;
                    if (++stage == STAGES) { stage = 0; phase ^= 1; }
                }
                // low-rank stages: T box in the A slot, L_A box in the first half of the W slot
                if (w.kb1 == kblocks) {
                    for (int j = 0; j < lora_steps && ok; ++j) {
                        if (!mbar_wait(bar_empty + 8 * stage, phase ^ 1, cta_abort, p.dev_error)) {
                            ok = false;
                            break;
                        }
                        if (l0_items > 0 && j == 0 && !l0_all_done) {
                            // T rows of this CTA's 128 rows come from phase 0 of this launch: one look at
                            // the count of published groups (once complete, no tile looks again), else
                            // wait for the four ready words of these rows
                            if (ld_acquire_gpu(p.l0_done) == p.l0_done_target) l0_all_done = true;
                            else ok = flag_wait4(p.l0_ready + (tm * CG + (int)rank) * 4, p.l0_epoch, cta_abort, p.dev_error);
                            if (!ok) break;
                            fence_proxy_async_global();
                        }
                        constexpr uint32_t LORA_BYTES = Cfg::A_BYTES + Cfg::B_HALF_BYTES;
                        const uint32_t a_dst = sA + stage * Cfg::A_BYTES;
                        const uint32_t b_dst = sB + stage * Cfg::B_BYTES;
                        if constexpr (CG == 1) {
                            const uint32_t bar = bar_full + 8 * stage;
                            mbar_arrive_expect_tx(bar, LORA_BYTES);
                            tma_load_2d(a_dst, &tmap_t, j * 64, m0, bar);
                            tma_load_2d(b_dst, &tmap_la, j * 64, n0, bar);
                        } else {
                            const uint32_t bar = full0 + 8 * stage;
                            if (leader) mbar_arrive_expect_tx(bar_full + 8 * stage, 2 * LORA_BYTES);
                            tma_load_2d_pair(a_dst, &tmap_t, j * 64, m0, bar);
                            tma_load_2d_pair(b_dst, &tmap_la, j * 64, n0, bar);
                        }
                        ++issued;
                        if (++stage == STAGES) { stage = 0; phase ^= 1; }
                    }
                }
            }
            if (!ok && issued) bounded_delay_ns(200000);  // let the copies in flight land before teardown
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer --------
        if (leader && lane == 0) {
            constexpr uint32_t idesc0 = make_idesc_sp_bf16(Cfg::BM * CG, BN), idesc1 = idesc0 | 1u;
            // descriptor words: low = start address (16-byte units) | LBO, high = SBO | version | swizzle
            const uint64_t d0 = make_desc_sw128(sA);
            const uint32_t desc_hi = (uint32_t)(d0 >> 32);
            const uint32_t a_lo0 = (uint32_t)d0, b_lo0 = (uint32_t)make_desc_sw128(sB);
            const uint64_t e_d0 = make_desc_rows16(sE);
            constexpr uint32_t BH = Cfg::B_HALF_BYTES >> 4;
            uint32_t stage = 0, phase = 0;
            bool ok = true;
            if constexpr (L0) {
                // phase 0: eight dense K = 16 steps per stage into the first 64 accumulator columns
                constexpr uint32_t idesc_l0 = make_idesc_sp_bf16(Cfg::BM * CG, Cfg::L0_R) & ~(1u << 2);
                for (int li = 0; li < l0_n && ok; ++li) {
                    const int item = l0s.item(cluster_id, li);
                    const int split = item / p.tiles_m;
                    const int k0 = split * p.l0_kb_per_split;
                    const int k1 = (k0 + p.l0_kb_per_split < kblocks) ? k0 + p.l0_kb_per_split : kblocks;
                    const int acc = (Cfg::ACC_STAGES == 2) ? (li & 1) : 0;
                    const uint32_t acc_phase = (Cfg::ACC_STAGES == 2) ? ((li >> 1) & 1) : (li & 1);
                    if (!mbar_wait(bar_tempty + 8 * acc, acc_phase ^ 1, cta_abort, p.dev_error)) {
                        ok = false;
                        break;
                    }
                    tc_fence_after();
                    const uint32_t d_tmem = tmem_base + acc * BN;
                    uint32_t accumulate = 0;
                    for (int kb = k0; kb < k1; ++kb) {
                        if (!mbar_wait(bar_full + 8 * stage, phase, cta_abort, p.dev_error)) {
                            ok = false;
                            break;
                        }
                        tc_fence_after();
                        const uint32_t a_lo = a_lo0 + stage * (Cfg::A_BYTES >> 4);
                        const uint32_t b_lo = b_lo0 + stage * (Cfg::B_BYTES >> 4);
                        const uint32_t a2_lo = b_lo + (Cfg::L0_X2_OFF >> 4);
                        const uint32_t b2_lo = b_lo + (Cfg::L0_LB_BYTES >> 4);
#pragma unroll
                        for (int i = 0; i < 4; ++i) {
                            mma_bf16_lh<CG>(d_tmem, a_lo + 2 * i, b_lo + 2 * i, desc_hi, idesc_l0, accumulate);
                            accumulate = 1u;
                        }
#pragma unroll
                        for (int i = 0; i < 4; ++i)
                            mma_bf16_lh<CG>(d_tmem, a2_lo + 2 * i, b2_lo + 2 * i, desc_hi, idesc_l0, 1u);
                        if constexpr (CG == 1) tc_commit(bar_empty + 8 * stage);
                        else tc_commit_pair(bar_empty + 8 * stage, 0x3);
                        if (++stage == STAGES) { stage = 0; phase ^= 1; }
                    }
                    if (!ok) break;
                    if constexpr (CG == 1) tc_commit(bar_tfull + 8 * acc);
                    else tc_commit_pair(bar_tfull + 8 * acc, 0x3);
                }
            }
            int it = 0;
            for (; it < num_items && ok; ++it) {
                const WorkItem w = sched.get(cluster_id, it);
                const int gi = l0_n + it;  // accumulator buffers alternate over phase 0 items and tiles alike
                const int acc = (Cfg::ACC_STAGES == 2) ? (gi & 1) : 0;
                const uint32_t acc_phase = (Cfg::ACC_STAGES == 2) ? ((gi >> 1) & 1) : (gi & 1);
                if (!mbar_wait(bar_tempty + 8 * acc, acc_phase ^ 1, cta_abort, p.dev_error)) break;
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + acc * BN;
                uint32_t accumulate = 0;
                for (int kb = w.kb0; kb < w.kb1; ++kb) {
                    if (!mbar_wait(bar_full + 8 * stage, phase, cta_abort, p.dev_error)) {
                        ok = false;
                        break;
                    }
                    tc_fence_after();
                    const uint32_t e_tmem = tmem_base + Cfg::E_COL0 + Cfg::E_COLS * stage;
                    const uint32_t a_lo = a_lo0 + stage * (Cfg::A_BYTES >> 4);
                    const uint32_t b_lo = b_lo0 + stage * (Cfg::B_BYTES >> 4);
                    tmem_cp_128x128b<CG>(e_tmem, e_d0 + (uint64_t)(stage * (Cfg::E_BYTES >> 4)));
                    if constexpr (Cfg::FP8) {
                        // second 128 x 128 metadata block of the stage, then four K steps of 64 logical
                        // elements: A advances 32 bytes, W 64 bytes, metadata two columns
                        tmem_cp_128x128b<CG>(e_tmem + 4, e_d0 + (uint64_t)(stage * (Cfg::E_BYTES >> 4) + (2048 >> 4)));
                        constexpr uint32_t idesc8 = make_idesc_sp_e4m3(Cfg::BM * CG, BN);
                        mma_sp_f8_lh<CG>(d_tmem, a_lo, b_lo, desc_hi, e_tmem, idesc8, accumulate);
                        mma_sp_f8_lh<CG>(d_tmem, a_lo + 2, b_lo + 4, desc_hi, e_tmem + 2, idesc8, 1u);
                        mma_sp_f8_lh<CG>(d_tmem, a_lo + 4, b_lo + BH, desc_hi, e_tmem + 4, idesc8, 1u);
                        mma_sp_f8_lh<CG>(d_tmem, a_lo + 6, b_lo + BH + 4, desc_hi, e_tmem + 6, idesc8, 1u);
                    } else {
                        // four K steps of 32 logical elements: A advances 32 bytes, W 64 bytes (steps 2, 3
                        // in the second 64-element slice); metadata column pair + sparse_id2 = step parity
                        mma_sp_bf16_lh<CG>(d_tmem, a_lo, b_lo, desc_hi, e_tmem, idesc0, accumulate);
                        mma_sp_bf16_lh<CG>(d_tmem, a_lo + 2, b_lo + 4, desc_hi, e_tmem, idesc1, 1u);
                        mma_sp_bf16_lh<CG>(d_tmem, a_lo + 4, b_lo + BH, desc_hi, e_tmem + 2, idesc0, 1u);
                        mma_sp_bf16_lh<CG>(d_tmem, a_lo + 6, b_lo + BH + 4, desc_hi, e_tmem + 2, idesc1, 1u);
                    }
                    accumulate = 1u;
                    if constexpr (CG == 1) tc_commit(bar_empty + 8 * stage);
                    else tc_commit_pair(bar_empty + 8 * stage, 0x3);
                    if (++stage == STAGES) { stage = 0; phase ^= 1; }
                }
                if (ok && w.kb1 == kblocks) {
                    constexpr uint32_t idesc_dense = idesc0 & ~(1u << 2);
                    for (int j = 0; j < lora_steps; ++j) {
                        if (!mbar_wait(bar_full + 8 * stage, phase, cta_abort, p.dev_error)) {
                            ok = false;
                            break;
                        }
                        tc_fence_after();
                        const uint32_t a_lo = a_lo0 + stage * (Cfg::A_BYTES >> 4);
                        const uint32_t b_lo = b_lo0 + stage * (Cfg::B_BYTES >> 4);
                        // dense K steps of 16 elements: both operands advance 32 bytes
                        mma_bf16_lh<CG>(d_tmem, a_lo, b_lo, desc_hi, idesc_dense, accumulate);
                        mma_bf16_lh<CG>(d_tmem, a_lo + 2, b_lo + 2, desc_hi, idesc_dense, 1u);
                        mma_bf16_lh<CG>(d_tmem, a_lo + 4, b_lo + 4, desc_hi, idesc_dense, 1u);
                        mma_bf16_lh<CG>(d_tmem, a_lo + 6, b_lo + 6, desc_hi, idesc_dense, 1u);
                        accumulate = 1u;
                        if constexpr (CG == 1) tc_commit(bar_empty + 8 * stage);
                        else tc_commit_pair(bar_empty + 8 * stage, 0x3);
                        if (++stage == STAGES) { stage = 0; phase ^= 1; }
                    }
                }
                if (!ok) break;
                if constexpr (CG == 1) tc_commit(bar_tfull + 8 * acc);
                else tc_commit_pair(bar_tfull + 8 * acc, 0x3);
            }
        }
    } else {
        // ------------------------------------------------------------------ epilogue ----------
        const int q = warp & 3;  // tensor-memory lane quarter this warp may read
        const uint32_t cbuf0 = sC + (warp - 2) * Cfg::CBUFS_W * Cfg::C_BOX_BYTES;
        const int c_first = (warp - 2) >> 2;  // with two warps per quarter: even or odd chunks
        const uint32_t tempty0 = (CG == 2) ? mapa(bar_tempty, 0) : bar_tempty;
        int it = 0, cb = 0;
        bool alive = true;
        if constexpr (L0) {
            // ---- phase 0: drain the 64-column accumulator of each (row block, K split) item ----
            constexpr int PIECES = Cfg::L0_R / 4;  // float4 pieces per row
            constexpr int BLOCK_ROWS = Cfg::BM * CG;
            for (int li = 0; li < l0_n && alive; ++li) {
                const int item = l0s.item(cluster_id, li);
                const int tmb = item % p.tiles_m, split = item / p.tiles_m;
                const int acc = (Cfg::ACC_STAGES == 2) ? (li & 1) : 0;
                const uint32_t acc_phase = (Cfg::ACC_STAGES == 2) ? ((li >> 1) & 1) : (li & 1);
                const int row_in_block = (int)rank * Cfg::BM + q * 32 + lane;
                const int64_t row = (int64_t)tmb * BLOCK_ROWS + row_in_block;
                // the row's scale is fetched while the item's K loop runs (a global load costs over a
                // microsecond once the main loops saturate the memory system); T = acc * (1 / s)
                float inv_s = 1.0f;
                if (row < p.M && (p.scale_partial != nullptr || p.row_scale != nullptr)) {
                    const float sc = (p.scale_partial != nullptr) ? row_scale_from_partials(p.scale_partial, row, p.scale_ks)
                                                                  : __ldg(p.row_scale + row);
                    inv_s = (sc == 0.0f) ? 0.0f : __frcp_rn(sc);
                }
                if (!mbar_wait(bar_tfull + 8 * acc, acc_phase, cta_abort, p.dev_error)) {
                    alive = false;
                    break;
                }
                tc_fence_after();
                const uint32_t t_row = tmem_base + ((uint32_t)(q * 32) << 16) + acc * BN;
                uint32_t v[64];
                tmem_ld_32x32b_x32(t_row, *reinterpret_cast<uint32_t(*)[32]>(&v[0]));
                tmem_ld_32x32b_x32(t_row + 32, *reinterpret_cast<uint32_t(*)[32]>(&v[32]));
                tmem_ld_wait();
                tc_fence_before();
                __syncwarp();
                if (lane == 0) {
                    if constexpr (CG == 1) mbar_arrive(bar_tempty + 8 * acc);
                    else mbar_arrive_cluster(tempty0 + 8 * acc);
                }
                const int group = (tmb * CG + (int)rank) * 4 + q;  // this warp's 32 rows
                bool last = true;
                if (p.l0_splits > 1) {
                    // partial: [row block][split][piece][row] float4 -> a warp's piece is 512 contiguous bytes
                    float4* dst = reinterpret_cast<float4*>(p.l0_partial) +
                                  ((size_t)tmb * p.l0_splits + split) * PIECES * BLOCK_ROWS + row_in_block;
#pragma unroll
                    for (int j = 0; j < PIECES; ++j)
                        __stcg(dst + (size_t)j * BLOCK_ROWS,
                               make_float4(__uint_as_float(v[4 * j]), __uint_as_float(v[4 * j + 1]),
                                           __uint_as_float(v[4 * j + 2]), __uint_as_float(v[4 * j + 3])));
                    // the warp's partial rows are ordered before lane 0's releasing add by the warp barrier;
                    // the add also acquires the partials of the warps that drew the earlier tickets
                    __syncwarp();
                    uint32_t ticket = 0;
                    if (lane == 0) ticket = atom_add_acq_rel_gpu(p.l0_tickets + group, 1u);
                    ticket = __shfl_sync(0xffffffffu, ticket, 0);
                    __syncwarp();  // lane 0's acquire ordered before every lane's loads of the partials
                    last = ticket == (uint32_t)p.l0_splits - 1;
                    if (last) {
                        // ascending split order whichever warp is last: reproducible bit for bit
                        const float4* src = reinterpret_cast<const float4*>(p.l0_partial) +
                                            (size_t)tmb * p.l0_splits * PIECES * BLOCK_ROWS + row_in_block;
#pragma unroll
                        for (int j = 0; j < 64; ++j) v[j] = 0u;  // +0.0f
                        // one batch of 16 independent loads per split: every batch costs a full L2 round
                        // trip under the main loop's traffic, so few large batches
                        for (int sp = 0; sp < p.l0_splits; ++sp) {
                            float4 pa[PIECES];
#pragma unroll
                            for (int j = 0; j < PIECES; ++j)
                                pa[j] = __ldcg(src + ((size_t)sp * PIECES + j) * BLOCK_ROWS);
#pragma unroll
                            for (int j = 0; j < PIECES; ++j) {
                                v[4 * j] = __float_as_uint(__uint_as_float(v[4 * j]) + pa[j].x);
                                v[4 * j + 1] = __float_as_uint(__uint_as_float(v[4 * j + 1]) + pa[j].y);
                                v[4 * j + 2] = __float_as_uint(__uint_as_float(v[4 * j + 2]) + pa[j].z);
                                v[4 * j + 3] = __float_as_uint(__uint_as_float(v[4 * j + 3]) + pa[j].w);
                            }
                        }
                    }
                }
                if (last) {
                    if (row < p.M) {
                        uint4* dst = reinterpret_cast<uint4*>(p.T + row * p.ldt);
#pragma unroll
                        for (int j = 0; j < 8; ++j) {
                            uint32_t o[4];
#pragma unroll
                            for (int e = 0; e < 4; ++e) {
                                const float a0 = __uint_as_float(v[8 * j + 2 * e]), a1 = __uint_as_float(v[8 * j + 2 * e + 1]);
                                o[e] = pack_bf16x2(a0 * inv_s, a1 * inv_s);
                            }
                            dst[j] = make_uint4(o[0], o[1], o[2], o[3]);
                        }
                    }
                    // T rows written with generic stores are read by TMA: order both proxies, then publish
                    // (the releasing store orders every lane's rows, which the warp barrier put before it)
                    fence_proxy_async_global();
                    __syncwarp();
                    if (lane == 0) {
                        if (p.l0_splits > 1) p.l0_tickets[group] = 0;  // ready for the next launch
                        st_release_gpu(p.l0_ready + group, p.l0_epoch);
                        red_add_release_gpu(p.l0_done, 1u);
                    }
                }
            }
        }
        for (; it < num_items && alive; ++it) {
            const WorkItem w = sched.get(cluster_id, it);
            int tm, tn;
            tile_coords(w.tile, p.tiles_m, p.tiles_n, p.group_m, tm, tn);
            const int gi = l0_n + it;
            const int acc = (Cfg::ACC_STAGES == 2) ? (gi & 1) : 0;
            const uint32_t acc_phase = (Cfg::ACC_STAGES == 2) ? ((gi >> 1) & 1) : (gi & 1);
            const int m0 = (tm * CG + (int)rank) * Cfg::BM + q * 32;
            const int64_t row = m0 + lane;
            const bool row_ok = row < p.M;
            // the row's scale is fetched (or summed from the prune launch's partial sums) while the
            // tile's main loop still runs
            float s = 1.0f;
            if (row_ok) {
                if (p.scale_partial != nullptr) s = row_scale_from_partials(p.scale_partial, row, p.scale_ks);
                else if (p.row_scale != nullptr) s = __ldg(p.row_scale + row);
            }
            // the tile's per-column terms (bias, FP8 weight scale), one column per lane and round,
            // fetched while the main loop runs and handed round by shuffles in the chunk loop: no
            // dependent global load is left between the accumulator and the store
            constexpr int CH = Cfg::CH;
            float bl_all[BN / CH][2], cl_all[BN / CH][2];
#pragma unroll
            for (int c = 0; c < BN / CH; ++c)
#pragma unroll
                for (int u = 0; u < 2; ++u) {
                    const int idx = u * 32 + lane, n = tn * BN + c * CH + idx;
                    bl_all[c][u] = 0.f;
                    cl_all[c][u] = 1.f;
                    if (idx < CH && n < p.N) {
                        if (p.bias != nullptr) bl_all[c][u] = __uint_as_float((uint32_t)__ldg(p.bias + n) << 16);
                        if constexpr (Cfg::FP8)
                            if (p.col_scale != nullptr) cl_all[c][u] = __ldg(p.col_scale + n);
                    }
                }
            if (!mbar_wait(bar_tfull + 8 * acc, acc_phase, cta_abort, p.dev_error)) break;
            tc_fence_after();
            const uint32_t t_row = tmem_base + ((uint32_t)(q * 32) << 16) + acc * BN;
            // stream-K pieces: this thread's row of the pair tile inside an fp32 partial slot
            const size_t slot_floats = (size_t)Cfg::BM * CG * BN;
            // layout of a slot: [CH-column chunk][16-byte piece j][row of the pair tile] float4, so a
            // warp's 32 rows of one piece are 512 contiguous bytes
            constexpr int SLOT_ROWS = Cfg::BM * CG;
            const size_t my_row_off = (size_t)((int)rank * Cfg::BM + q * 32 + lane);
            const int my_flag = (int)rank * 4 + q;
            if (w.kind == 2) {
                // wait until every contributing cluster's matching warp has published its rows
                if (lane == 0) {
                    for (int cc = w.first_contrib; cc < cluster_id && alive; ++cc)
                        if (sched.has_tail(cc))
                            alive = flag_wait(p.sk_flags + cc * 8 + my_flag, p.sk_epoch, cta_abort, p.dev_error);
                }
                alive = __shfl_sync(0xffffffffu, (int)alive, 0) != 0;
                if (!alive) break;
            }
            constexpr int NCH = BN / CH;
            // this warp's last chunk: after reading it the accumulator goes back to the issuer
            const int c_last = NCH - 1 - ((NCH - 1 - c_first) % Cfg::EPI_SPLIT);
#pragma unroll 1
            for (int c = c_first; c < NCH; c += Cfg::EPI_SPLIT) {
                const int n0 = tn * BN + c * CH;
                // this chunk's two rounds, picked with selects so that the arrays stay in registers
                // (an index that depends on the loop counter would put them into local memory and
                // force every load above to complete before the wait)
                float bl[2] = {bl_all[0][0], bl_all[0][1]}, cl[2] = {cl_all[0][0], cl_all[0][1]};
#pragma unroll
                for (int cc = 1; cc < BN / CH; ++cc)
                    if (c == cc) {
                        bl[0] = bl_all[cc][0]; bl[1] = bl_all[cc][1];
                        cl[0] = cl_all[cc][0]; cl[1] = cl_all[cc][1];
                    }
                uint32_t v[CH];
                tmem_ld_32x32b_x32(t_row + c * CH, *reinterpret_cast<uint32_t(*)[32]>(&v[0]));
                if constexpr (CH == 64)
                    tmem_ld_32x32b_x32(t_row + c * CH + 32, *reinterpret_cast<uint32_t(*)[32]>(&v[32]));
                else
                    tmem_ld_32x32b_x16(t_row + c * CH + 32, *reinterpret_cast<uint32_t(*)[16]>(&v[32]));
                tmem_ld_wait();
                if (c == c_last) {
                    // accumulator fully read: hand it back to the MMA issuer
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) {
                        if constexpr (CG == 1) mbar_arrive(bar_tempty + 8 * acc);
                        else mbar_arrive_cluster(tempty0 + 8 * acc);
                    }
                }
                if (w.kind == 1) {
                    // partial piece: raw fp32 accumulators to this cluster's slot
                    float4* dst = reinterpret_cast<float4*>(p.sk_partial + (size_t)cluster_id * slot_floats) +
                                  (size_t)c * (CH / 4) * SLOT_ROWS + my_row_off;
#pragma unroll
                    for (int j = 0; j < CH / 4; ++j)
                        __stcg(dst + (size_t)j * SLOT_ROWS, make_float4(__uint_as_float(v[4 * j]), __uint_as_float(v[4 * j + 1]),
                                                    __uint_as_float(v[4 * j + 2]), __uint_as_float(v[4 * j + 3])));
                    continue;
                }
                if (w.kind == 2) {
                    // owner piece: add the partials in ascending cluster order
                    for (int cc = w.first_contrib; cc < cluster_id; ++cc) {
                        if (!sched.has_tail(cc)) continue;
                        const float4* src = reinterpret_cast<const float4*>(p.sk_partial + (size_t)cc * slot_floats) +
                                            (size_t)c * (CH / 4) * SLOT_ROWS + my_row_off;
                        float4 pa[CH / 4];
#pragma unroll
                        for (int j = 0; j < CH / 4; ++j) pa[j] = __ldcg(src + (size_t)j * SLOT_ROWS);
#pragma unroll
                        for (int j = 0; j < CH / 4; ++j) {
                            const float4 a = pa[j];
                            v[4 * j] = __float_as_uint(__uint_as_float(v[4 * j]) + a.x);
                            v[4 * j + 1] = __float_as_uint(__uint_as_float(v[4 * j + 1]) + a.y);
                            v[4 * j + 2] = __float_as_uint(__uint_as_float(v[4 * j + 2]) + a.z);
                            v[4 * j + 3] = __float_as_uint(__uint_as_float(v[4 * j + 3]) + a.w);
                        }
                    }
                }
                if (n0 >= p.N) continue;
                // staging buffer must have been read by its previous TMA store
                if (lane == 0) tma_store_wait_read<Cfg::CBUFS_W - 1>();
                __syncwarp();
                const uint32_t cbuf = cbuf0 + cb * Cfg::C_BOX_BYTES;
#pragma unroll
                for (int j = 0; j < CH / 8; ++j) {  // 8 columns (16 bytes of output) at a time
                    const int n = n0 + j * 8;
                    float b[8];
                    float r[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
#pragma unroll
                    for (int e = 0; e < 8; ++e) {
                        const int col = j * 8 + e;
                        b[e] = __shfl_sync(0xffffffffu, bl[col >> 5], col & 31);
                    }
                    if (n < p.N) {
                        if (p.residual != nullptr && row_ok) {
                            const uint4 rv = __ldg(reinterpret_cast<const uint4*>(p.residual + row * p.ldr + n));
                            r[0] = bf16_lo_f(rv.x); r[1] = bf16_hi_f(rv.x);
                            r[2] = bf16_lo_f(rv.y); r[3] = bf16_hi_f(rv.y);
                            r[4] = bf16_lo_f(rv.z); r[5] = bf16_hi_f(rv.z);
                            r[6] = bf16_lo_f(rv.w); r[7] = bf16_hi_f(rv.w);
                        }
                    }
                    float cs[8] = {s, s, s, s, s, s, s, s};  // row scale (x per-channel weight scale)
                    if constexpr (Cfg::FP8) {
#pragma unroll
                        for (int e = 0; e < 8; ++e) {
                            const int col = j * 8 + e;
                            cs[e] = s * __shfl_sync(0xffffffffu, cl[col >> 5], col & 31);
                        }
                    }
                    uint32_t o[4];
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        const float y0 = fmaf(cs[2 * e], __uint_as_float(v[j * 8 + 2 * e]), b[2 * e]) + r[2 * e];
                        const float y1 = fmaf(cs[2 * e + 1], __uint_as_float(v[j * 8 + 2 * e + 1]), b[2 * e + 1]) + r[2 * e + 1];
                        o[e] = pack_bf16x2(y0, y1);
                    }
                    if constexpr (CH == 64)  // 128-byte rows, 16-byte chunk index XOR (row % 8): the 128-byte swizzle
                        sts128(cbuf + lane * 128 + ((j ^ (lane & 7)) << 4), o[0], o[1], o[2], o[3]);
                    else  // dense 96-byte rows for the unswizzled 48-column box
                        sts128(cbuf + lane * (CH * 2) + (j << 4), o[0], o[1], o[2], o[3]);
                }
                fence_proxy_async_smem();
                __syncwarp();
                if (lane == 0) {
                    tma_store_2d(&tmap_y, n0, m0, cbuf);
                    tma_store_commit();
                }
                cb = (cb + 1 == Cfg::CBUFS_W) ? 0 : cb + 1;
            }
            if (w.kind == 1) {
                // publish: all lanes' stores (ordered before lane 0 by the warp barrier), then the
                // releasing store of the ready word of this (slot, warp)
                __syncwarp();
                if (lane == 0) st_release_gpu(p.sk_flags + cluster_id * 8 + my_flag, p.sk_epoch);
            }
        }
        if (lane == 0) tma_store_wait_all<0>();
    }

    // ---------------------------------------------------------------------- teardown ----------
    tc_fence_before();
    __syncthreads();
    if constexpr (CG == 2) cluster_sync_all();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc<CG>(tmem_base, Cfg::TMEM_COLS);
    }
}

}  // namespace lynx

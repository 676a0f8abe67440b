// C ABI of the library (see include/lynx.h): argument checks, context (scratch, error word,
// launch counter), TMA descriptor construction and kernel launches.  No CPU fallback anywhere.
#include "../../include/lynx.h"

#include <cuda.h>
#include <cuda_runtime.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include <mutex>

#include "prune_compress.cuh"
#include "sparse_gemm.cuh"
#include "sparse_gemm_rt2.cuh"
#include "fused_linear.cuh"
#include "lora_down.cuh"
#include "fp8_path.cuh"
#include "prune_lora.cuh"

using namespace lynx;

struct lynx_ctx {
    int device = 0;
    int num_sms = 0;
    uint32_t* err_host = nullptr;  // mapped pinned word written by kernels
    uint32_t* err_dev = nullptr;
    void* scratch = nullptr;  // partial row sums, compressed operands and scale of the single-call path
    size_t scratch_bytes = 0;
    void* host_stage = nullptr;  // device mirrors of X and Y, only for lynx_act_sparse_linear_host
    size_t host_stage_bytes = 0;
    uint32_t* tickets = nullptr;  // one word per 16-row block (prune finalize), zero between launches
    void* lora_ws = nullptr;      // low-rank branch: [fp32 partials][T]
    size_t lora_ws_bytes = 0;
    // host-buffer entry point: copy streams and events of its row-chunk pipeline (created on first use)
    cudaStream_t h2d_stream = nullptr, d2h_stream = nullptr;
    cudaEvent_t ev_h2d[8] = {}, ev_done[8] = {}, ev_all = nullptr;
    // row sums the last deferred prune launch left in the scratch (two-call form), and their shape
    const float* deferred_partial = nullptr;
    int deferred_ks = 0;
    int64_t deferred_M = 0, deferred_K = 0;
    uint32_t l0_epoch = 0;        // launch counter of the fused down projection (ready words hold it)
    uint32_t l0_done_total = 0;   // groups published by all such launches so far (mod 2^32)
    int l0_force_splits = 0, l0_force_fill = -1;  // development overrides of the phase-0 plan
    int defer_scale = 1;  // layer calls: row scale summed in the GEMM epilogue (LYNX_DEFER_SCALE=0: in the prune kernel)
    int lora_fuse = 2;            // down projection: 2 = in the prune launch (X read once), 1 = inside the GEMM launch, 0 = own kernel
    float* sk_partial = nullptr;  // stream-K partial tiles (one slot per cluster) + ready words
    uint32_t* sk_flags = nullptr;
    uint32_t sk_epoch = 0;
    int streamk = 0;  // stream-K tail: off by default (measured: no net gain), LYNX_STREAMK=1 enables
    int64_t launches = 0;
    int pdl = 1;        // programmatic dependent launch of the finalize and GEMM kernels
    int gemm_cfg = 0;   // 0 = auto
    int prune_tpu = 0;  // 0 = auto
    int fp8_ring = 1;   // FP8 activations: single-read ring kernel (LYNX_FP8_RING=0: one CTA per 16 rows)
    int fp8_ring_forced = 0;
    int gemm_group_m = 16;    // row tiles per group of the GEMM's tile order (LYNX_GEMM_GROUP_M; 0 = one group)
    int pl_force_splits = 0;  // development override: cluster size of the prune + down-projection kernel
    int splitk_force = 1;     // in-cluster split-K of the GEMM for launches with few tiles: 1 = cost model, 0 = off, 2..4 forced
    int rt2 = -1;             // two-row-tile GEMM kernel: -1 = cost model, 0 = never, 1 = whenever it applies
    int rt2_doubles = -1;     // development override: number of 512-row items of its schedule
    int prune_finalize = 0;   // row-scale finalize of the stand-alone prune call: 0 = per shape, 1 = in-kernel ticket, 2 = own launch
    // encoded tensor maps of recent launches, keyed by everything that went into the encoding
    // (a layer called again on the same buffers skips cuTensorMapEncodeTiled)
    struct TmapKey {
        const void* base;
        uint64_t rows, cols, ld_bytes;
        uint32_t box_cols, box_rows;
        int dt, sw;
        bool operator==(const TmapKey& o) const {
            return base == o.base && rows == o.rows && cols == o.cols && ld_bytes == o.ld_bytes &&
                   box_cols == o.box_cols && box_rows == o.box_rows && dt == o.dt && sw == o.sw;
        }
    };
    static constexpr int TMAP_CACHE = 128;  // direct mapped
    TmapKey tmap_key[TMAP_CACHE] = {};
    CUtensorMap tmap_val[TMAP_CACHE];
    bool tmap_ok[TMAP_CACHE] = {};
    int64_t tmap_hits = 0, tmap_misses = 0;
    std::mutex mu;
};

namespace {

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*,
                                  CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                  CUtensorMapFloatOOBfill);

EncodeTiledFn get_encode() {
    static EncodeTiledFn fn = nullptr;
    static std::once_flag once;
    std::call_once(once, [] {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
    });
    return fn;
}

// 2D row-major tensor [rows x cols] of `elem_bytes` elements, row pitch `ld_bytes`.
bool encode_tmap_2d(CUtensorMap* m, CUtensorMapDataType dt, const void* base, uint64_t rows, uint64_t cols,
                    uint64_t ld_bytes, uint32_t box_cols, uint32_t box_rows, CUtensorMapSwizzle sw) {
    EncodeTiledFn enc = get_encode();
    if (!enc) return false;
    cuuint64_t dims[2] = {cols, rows};
    cuuint64_t strides[1] = {ld_bytes};
    cuuint32_t box[2] = {box_cols, box_rows};
    cuuint32_t estr[2] = {1, 1};
    return enc(m, dt, 2, const_cast<void*>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, sw,
               CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// The same through the context's cache: a tensor map is a pure function of its key, so a hit is
// exact.  (One context serves one stream at a time; the cache is not locked.)
bool make_tmap_2d(lynx_ctx* ctx, CUtensorMap* m, CUtensorMapDataType dt, int elem_bytes, const void* base,
                  uint64_t rows, uint64_t cols, uint64_t ld_bytes, uint32_t box_cols, uint32_t box_rows,
                  CUtensorMapSwizzle sw) {
    (void)elem_bytes;
    const lynx_ctx::TmapKey key{base, rows, cols, ld_bytes, box_cols, box_rows, (int)dt, (int)sw};
    uint64_t h = reinterpret_cast<uintptr_t>(base) >> 8;
    h = h * 0x9E3779B97F4A7C15ull + rows * 31 + cols * 131 + ld_bytes * 7 + box_cols * 1009 + box_rows * 9176 +
        (uint64_t)dt * 77 + (uint64_t)sw;
    const int slot = (int)((h >> 20) % lynx_ctx::TMAP_CACHE);
    if (ctx->tmap_ok[slot] && ctx->tmap_key[slot] == key) {
        *m = ctx->tmap_val[slot];
        ctx->tmap_hits++;
        return true;
    }
    if (!encode_tmap_2d(m, dt, base, rows, cols, ld_bytes, box_cols, box_rows, sw)) return false;
    ctx->tmap_key[slot] = key;
    ctx->tmap_val[slot] = *m;
    ctx->tmap_ok[slot] = true;
    ctx->tmap_misses++;
    return true;
}

// cudaFuncSetAttribute is per device: remember, per kernel instantiation, which devices have it.
constexpr int MAX_CTX_DEVICES = 64;
template <class Kernel>
lynx_status allow_dynamic_smem(Kernel kern, int bytes, int device, bool (&done)[MAX_CTX_DEVICES]) {
    if (device < 0 || device >= MAX_CTX_DEVICES) return LYNX_ERR_INVALID_ARG;
    if (done[device]) return LYNX_OK;
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes) != cudaSuccess)
        return LYNX_ERR_CUDA;
    done[device] = true;
    return LYNX_OK;
}

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

lynx_status check_device_error(lynx_ctx* ctx) {
    if (ctx->err_host && *ctx->err_host != DEV_OK) return LYNX_ERR_TIMEOUT;
    return LYNX_OK;
}

lynx_status cuda_ok(cudaError_t e) { return e == cudaSuccess ? LYNX_OK : LYNX_ERR_CUDA; }

size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

constexpr size_t PRUNE_TICKET_BYTES = 1u << 20;  // 262144 row blocks of 16 rows = 4M rows
constexpr size_t LORA_TICKET_BYTES = 64u << 10;  // after the prune tickets: 16384 row blocks of 128 rows
// in-GEMM down projection: ticket and ready word per 32-row group (65536 groups = 2M rows), each
// at a fixed place of the zero-initialised ticket allocation, whatever shapes the context serves
constexpr size_t L0_WORDS_BYTES = 256u << 10;
constexpr size_t TICKET_ALLOC_BYTES = PRUNE_TICKET_BYTES + LORA_TICKET_BYTES + 2 * L0_WORDS_BYTES + 256;  // + done counter

// Row sums a deferred prune launch left in the context's scratch for the GEMM that follows it.
struct ScaleSrc {
    const float* partial = nullptr;
    int ks = 0;
};

// Low-rank branch operands of the GEMM: T = (X L_B^T) / s [M x R] bf16 and L_A [N x R] bf16.
struct LoraArgs {
    const void* T;
    int64_t ldt;
    const void* LA;
    int64_t ldla;
    int R;
    // set when the GEMM launch computes T itself (phase 0): dense X, L_B and the workspace pieces
    const void* X = nullptr;
    int64_t ldx = 0;
    const void* LB = nullptr;
    int64_t ldlb = 0;
    float* l0_partial = nullptr;
    uint32_t* l0_tickets = nullptr;
    uint32_t* l0_ready = nullptr;
};

// Plan of the in-GEMM down projection: items = 256-row blocks x K splits.  Clusters with one tile
// fewer than the busiest ("light": index >= tiles % clusters) have a tile time of slack.  If ALL
// items fit into that slack (at most `fill` per light cluster) they go there and the busiest
// clusters carry none; otherwise every cluster takes its share round-robin, which finishes T
// soonest -- a T that is late stalls the first tile of every cluster at its low-rank stage
// (measured: a partial placement on few light clusters cost more than it saved).
// t_tile_us: one tile's main loop; an item streams its K blocks at about 0.75 us per 128-element
// block while most clusters stream too (HBM bound), plus ~1 us of pipeline fill.
struct L0Plan {
    int splits, kb_per_split, light0, fill;
};
L0Plan l0_plan(int clusters, int tiles, int tiles_m, int kblocks, double t_tile_us, int force_splits, int force_fill) {
    L0Plan best{1, kblocks, clusters, 0};
    double best_t = 1e30;
    const int rem = tiles % clusters, light = rem ? clusters - rem : 0;
    for (int sp = 1; sp <= 16 && (sp == 1 || sp * 2 <= kblocks); ++sp) {
        if (force_splits > 0 && sp != force_splits) continue;
        const int per = (kblocks + sp - 1) / sp;
        const int real = (kblocks + per - 1) / per;
        const int items = tiles_m * real;
        // finalize: one L2 round trip per split under load, plus fences and the ticket
        const double t_fin = real > 1 ? 1.5 + 1.3 * real : 0.5;
        // inside the slack of the light clusters: few clusters stream, ~0.42 us per K block
        const double t_item_s = per * 0.42 + 2.0;
        int fill = light ? (int)((t_tile_us - t_fin) / t_item_s) : 0;
        if (fill > 8) fill = 8;
        if (fill < 0) fill = 0;
        if (force_fill >= 0) fill = light ? force_fill : 0;
        if (fill > 0 && light * fill >= items) {
            const double t = 0.02 * real;
            if (t < best_t) { best_t = t; best = L0Plan{real, per, rem, fill}; }
        }
        if (force_fill > 0) continue;
        // round-robin over all clusters: everybody streams, ~0.75 us per K block
        const double t_item_r = per * 0.75 + 1.0;
        const double late = t_fin - 0.5 * t_tile_us;
        const double t = (double)((items + clusters - 1) / clusters) * t_item_r + (late > 0 ? late : 0) + 0.02 * real;
        if (t < best_t) { best_t = t; best = L0Plan{real, per, clusters, 0}; }
    }
    return best;
}
// upper bound of the splits any plan uses (workspace sizing)
constexpr int L0_MAX_SPLITS = 16;

// Scratch layout for (M, K):
// [partial row sums][sums 2M floats][values][meta][row_scale M floats]
// The first two sections serve lynx_prune_compress alone and come first so that a context that is
// only used for pruning needs little memory.  (The device mirrors of host buffers belong to
// lynx_act_sparse_linear_host alone and live in an allocation of their own.)
struct ScratchLayout {
    size_t partial, prune_end, values, meta, scale, sums, total;
};
ScratchLayout scratch_layout(int64_t M, int64_t K) {
    ScratchLayout L;
    size_t off = 0;
    const size_t rb16 = (size_t)((M + 127) / 128) * 8, kblocks = (size_t)(K / 128);
    L.partial = off; off = align_up(off + rb16 * kblocks * 32 * 4, 1024);
    L.sums = off;    off = align_up(off + (size_t)M * 8, 1024);
    L.prune_end = off;
    L.values = off; off = align_up(off + lynx_values_bytes(M, K), 1024);
    L.meta = off;   off = align_up(off + lynx_meta_bytes(M, K), 1024);
    L.scale = off;  off = align_up(off + (size_t)M * 4, 1024);
    L.total = off;
    return L;
}

// Work decomposition of the prune/compress launch: one warp per (16-row block, run of `tpu`
// 128-element K blocks), KS = runs per row, 4 warps per CTA.  Shared by every entry point that
// launches prune_compress_kernel: the bits of the row sums depend on KS.
struct PrunePlan {
    int64_t rb16;
    int tpu, KS, ctas_per_rb;
    unsigned grid;
};
PrunePlan prune_plan(int num_sms, int64_t M, int64_t K, int tpu_override) {
    PrunePlan P;
    const int64_t kblocks = K / 128;
    P.rb16 = ((M + 127) / 128) * 8;
    int tpu = tpu_override;
    if (tpu <= 0) {
        const int64_t resident = (int64_t)num_sms * 40;  // warps the GPU holds at ~48 registers
        const int64_t want = (P.rb16 * kblocks) / (3 * resident);
        tpu = (int)(want < 1 ? 1 : (want > 8 ? 8 : want));
    }
    if (tpu > kblocks) tpu = (int)kblocks;
    while (kblocks % tpu) --tpu;
    P.tpu = tpu;
    P.KS = (int)(kblocks / tpu);
    P.ctas_per_rb = (P.KS + PRUNE_CTA_WARPS - 1) / PRUNE_CTA_WARPS;
    P.grid = (unsigned)(P.rb16 * P.ctas_per_rb);
    return P;
}

// --------------------------------------------------------------------------- GEMM launch -----

// Row tiles per group of the GEMM's tile order: groups of about `gemm_group_m` (16), all of nearly the
// same size (17 row tiles run as 9 + 8, not as 16 + 1: a one-row group shares no W tile between clusters).
static int gemm_group_rows(const lynx_ctx* ctx, int tiles_m) {
    const int g = ctx->gemm_group_m;
    if (g <= 0 || g >= tiles_m) return tiles_m;
    const int groups = (tiles_m + g - 1) / g;
    return (tiles_m + groups - 1) / groups;
}

// One warp; lane 0 waits on a barrier with no arrivals until the limit expires (see
// lynx_selftest_wait_timeout).  Nothing faults and nothing waits past the limit.
__global__ void wait_timeout_probe_kernel(uint32_t* dev_error, uint64_t limit_ns) {
    __shared__ __align__(8) uint64_t bar;
    __shared__ uint32_t abort_word;
    if (threadIdx.x == 0) {
        abort_word = 0;
        mbar_init(smem_u32(&bar), 1);
        fence_mbar_init();
    }
    __syncwarp();
    if (threadIdx.x == 0) (void)mbar_wait_limit(smem_u32(&bar), 0, &abort_word, dev_error, limit_ns);
    __syncwarp();
}

template <class Cfg>
lynx_status launch_gemm_cfg(lynx_ctx* ctx, const void* values, const void* meta, int64_t M, int64_t K,
                            const void* W, int64_t N, int64_t ldw, const void* bias, const lynx_comp* comp,
                            const LoraArgs* lora, void* Y, int64_t ldy, cudaStream_t st, const ScaleSrc* ss,
                            bool layer_call) {
    CUtensorMap ta, tb, te, ty, tt, tla, tx, tlb;
    const uint64_t rb = (uint64_t)((M + 127) / 128), kblocks = (uint64_t)(K / 128);
    if (!make_tmap_2d(ctx, &ta, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, values, (uint64_t)M, (uint64_t)(K / 2),
                      (uint64_t)K, 64, 128, CU_TENSOR_MAP_SWIZZLE_128B) ||
        !make_tmap_2d(ctx, &tb, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, W, (uint64_t)N, (uint64_t)K, (uint64_t)ldw * 2, 64,
                      Cfg::BN_CTA, CU_TENSOR_MAP_SWIZZLE_128B) ||
        !make_tmap_2d(ctx, &te, CU_TENSOR_MAP_DATA_TYPE_UINT32, 4, meta, rb * kblocks * 2, 256, 1024, 256, 2,
                      CU_TENSOR_MAP_SWIZZLE_NONE) ||
        !make_tmap_2d(ctx, &ty, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, Y, (uint64_t)M, (uint64_t)N, (uint64_t)ldy * 2, Cfg::CH,
                      32, Cfg::CH == 64 ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_NONE))
        return LYNX_ERR_CUDA;
    if (lora) {
        if (!make_tmap_2d(ctx, &tt, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, lora->T, (uint64_t)M, (uint64_t)lora->R,
                          (uint64_t)lora->ldt * 2, 64, 128, CU_TENSOR_MAP_SWIZZLE_128B) ||
            !make_tmap_2d(ctx, &tla, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, lora->LA, (uint64_t)N, (uint64_t)lora->R,
                          (uint64_t)lora->ldla * 2, 64, Cfg::BN_CTA, CU_TENSOR_MAP_SWIZZLE_128B))
            return LYNX_ERR_CUDA;
    } else {
        tt = ta;  // never read: lora_steps = 0
        tla = tb;
    }
    const bool l0 = lora && lora->X && Cfg::L0_OK && lora->R == Cfg::L0_R;
    if (lora && lora->X && !l0) return LYNX_ERR_INVALID_ARG;  // the caller checks the tile first
    if (l0) {
        if (!make_tmap_2d(ctx, &tx, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, lora->X, (uint64_t)M, (uint64_t)K,
                          (uint64_t)lora->ldx * 2, 64, 128, CU_TENSOR_MAP_SWIZZLE_128B) ||
            !make_tmap_2d(ctx, &tlb, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, lora->LB, (uint64_t)lora->R, (uint64_t)K,
                          (uint64_t)lora->ldlb * 2, 64, Cfg::L0_R / Cfg::CG, CU_TENSOR_MAP_SWIZZLE_128B))
            return LYNX_ERR_CUDA;
    } else {
        tx = ta;
        tlb = tb;
    }

    GemmParams p;
    p.lora_steps = lora ? lora->R / 64 : 0;
    p.M = M; p.N = N; p.K = K;
    p.row_scale = comp ? comp->row_scale : nullptr;
    p.scale_partial = ss ? ss->partial : nullptr;
    p.scale_ks = ss ? ss->ks : 0;
    p.col_scale = nullptr;
    p.bias = static_cast<const uint16_t*>(bias);
    p.residual = comp ? static_cast<const uint16_t*>(comp->residual) : nullptr;
    p.ldr = comp ? comp->ldr : 0;
    p.dev_error = ctx->err_dev;
    p.tiles_m = (int)((M + Cfg::BM * Cfg::CG - 1) / (Cfg::BM * Cfg::CG));
    p.tiles_n = (int)((N + Cfg::BN - 1) / Cfg::BN);
    p.group_m = gemm_group_rows(ctx, p.tiles_m);
    p.sk_partial = nullptr;
    p.sk_flags = nullptr;
    p.sk_epoch = 0;
    p.l0_fused = l0 ? 1 : 0;
    p.l0_splits = 1;
    p.l0_kb_per_split = 0;
    p.l0_light0 = 0;
    p.l0_fill = 0;
    p.l0_partial = nullptr;
    p.l0_tickets = nullptr;
    p.l0_ready = nullptr;
    p.l0_epoch = 0;
    p.l0_done = nullptr;
    p.l0_done_target = 0;
    p.T = nullptr;
    p.ldt = 0;
    p.w_prefetch = (layer_call && !ctx->streamk) ? 1 : 0;

    auto kern = lora ? sparse_gemm_kernel<Cfg, true> : sparse_gemm_kernel<Cfg, false>;
    static bool attr_set[2][MAX_CTX_DEVICES] = {};  // per instantiation (with / without the low-rank code)
    if (lynx_status as = allow_dynamic_smem(kern, Cfg::SMEM_BYTES, ctx->device, attr_set[lora ? 1 : 0]); as != LYNX_OK)
        return as;
    const int tiles = p.tiles_m * p.tiles_n;
    int clusters = ctx->num_sms / Cfg::CG;
    {
        // stream-K tail: worth it when the leftover tiles' K blocks give every cluster a piece of
        // at least 4 blocks; needs the per-cluster partial slots (allocated once, on first use)
        const int kblocks = (int)(K / Cfg::BK);
        const int rem = tiles % clusters;
        if (!l0 && ctx->streamk && rem > 0 && (int64_t)rem * kblocks >= 4ll * clusters) {
            if (!ctx->sk_partial) return LYNX_ERR_WORKSPACE;  // allocated by lynx_create when the schedule is on
            p.sk_partial = ctx->sk_partial;
            p.sk_flags = ctx->sk_flags;
            p.sk_epoch = ++ctx->sk_epoch;
        } else if (clusters > tiles) {
            clusters = tiles;
        }
    }
    if (l0) {
        // slack of a light cluster = one tile's main loop (measured ~0.465 us per K block of the 240-wide tile)
        const L0Plan plan = l0_plan(clusters, tiles, p.tiles_m, (int)(K / 128), (double)(K / 128) * 0.465 + 0.6,
                                    ctx->l0_force_splits, ctx->l0_force_fill);
        p.l0_splits = plan.splits;
        p.l0_kb_per_split = plan.kb_per_split;
        p.l0_light0 = plan.light0;
        p.l0_fill = plan.fill;
        p.l0_partial = lora->l0_partial;
        p.l0_tickets = lora->l0_tickets;
        p.l0_ready = lora->l0_ready;
        p.l0_epoch = ++ctx->l0_epoch;
        p.l0_done = lora->l0_ready + L0_WORDS_BYTES / 4;
        ctx->l0_done_total += (uint32_t)(p.tiles_m * Cfg::CG * 4);
        p.l0_done_target = ctx->l0_done_total;
        p.T = static_cast<uint16_t*>(const_cast<void*>(lora->T));
        p.ldt = lora->ldt;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(clusters * Cfg::CG));
    cfg.blockDim = dim3(Cfg::THREADS);
    cfg.dynamicSmemBytes = Cfg::SMEM_BYTES;
    cfg.stream = st;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = Cfg::CG;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    // let the prologue (barriers, tensor memory, descriptor prefetch) overlap the previous kernel
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = ctx->pdl ? 1 : 0;
    cfg.attrs = attr;
    cfg.numAttrs = 2;
    cudaError_t e = cudaLaunchKernelEx(&cfg, kern, ta, tb, te, ty, tt, tla, tx, tlb, p);
    if (e != cudaSuccess) return LYNX_ERR_CUDA;
    ctx->launches++;
    return LYNX_OK;
}

// ------------------------------------------------------- two-row-tile GEMM kernel (sparse_gemm_rt2) -----

using Rt2Cfg = Gemm2Cfg<240, 3>;

// Modelled time (us) of the slowest cluster for a schedule with D doubles.  Per-K-block times are
// measured B200 figures: 0.69 us for a 512 x 240 stage (66 KB in flight per CTA and stage, three
// stages) against 0.465 us for a 256 x 240 stage of sparse_gemm_kernel (0.49 us here); a double's
// epilogue is exposed (the accumulators are not double-buffered: ~5 us per double including the
// refill of the ring), a single's hides behind the next single; the switch between the two
// rings costs a pipeline fill.  Within each class of clusters the one at the first position carries the
// most singles, so two clusters decide the maximum.
constexpr double RT2_T1 = 0.49, RT2_T2 = 0.69, RT2_E1 = 0.8, RT2_E2 = 5.0, RT2_SWITCH = 2.0;
double rt2_makespan(const PairSchedule& sc, double kb) {
    double worst = 0.0;
    const int probe[2] = {sc.b % sc.C, 0};  // position 0 (first light cluster), position L (first heavy one)
    for (int i = 0; i < 2; ++i) {
        const int c = probe[i];
        const int nd = sc.num_doubles(c), ns = sc.num_singles(c);
        const double t = nd * (kb * RT2_T2 + RT2_E2) + ns * (kb * RT2_T1 + RT2_E1) + ((nd && ns) ? RT2_SWITCH : 0.0);
        if (t > worst) worst = t;
    }
    return worst;
}

struct Rt2Plan {
    int doubles, clusters;
    double t_us;
};
Rt2Plan rt2_plan(int num_sms, int64_t M, int64_t N, int64_t K, int lora_steps, int force_doubles) {
    const int tiles_m = (int)((M + 255) / 256), tiles_n = (int)((N + Rt2Cfg::BN - 1) / Rt2Cfg::BN);
    const int pairs = num_sms / 2;
    const double kb = (double)(K / 128) + lora_steps;
    const int dmax = (tiles_m / 2) * tiles_n;
    Rt2Plan best{0, 1, 1e30};
    auto consider = [&](int D) {
        if (D < 0 || D > dmax) return;
        const int items = tiles_m * tiles_n - D;
        const int C = items < pairs ? items : pairs;
        PairSchedule sc;
        sc.init(tiles_m, tiles_n, C, D, 8);
        const double t = rt2_makespan(sc, kb);
        if (t < best.t_us) best = Rt2Plan{D, C, t};
    };
    if (force_doubles >= 0) {
        consider(force_doubles > dmax ? dmax : force_doubles);
        return best;
    }
    // candidates: every cluster the same number of doubles (multiples of the cluster count), all
    // slots as doubles, and the neighbours that leave the light clusters exactly one single more
    consider(dmax);
    for (int a = 0; a * pairs <= dmax; ++a) consider(a * pairs);
    return best;
}

template <bool LORA>
lynx_status launch_gemm_rt2(lynx_ctx* ctx, const Rt2Plan& plan, const void* values, const void* meta, int64_t M,
                            int64_t K, const void* W, int64_t N, int64_t ldw, const void* bias, const lynx_comp* comp,
                            const LoraArgs* lora, void* Y, int64_t ldy, cudaStream_t st, const ScaleSrc* ss,
                            bool layer_call) {
    using Cfg = Rt2Cfg;
    CUtensorMap ta, tb, te, ty, tt, tla;
    const uint64_t rb = (uint64_t)((M + 127) / 128), kblocks = (uint64_t)(K / 128);
    if (!make_tmap_2d(ctx, &ta, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, values, (uint64_t)M, (uint64_t)(K / 2),
                      (uint64_t)K, 64, 128, CU_TENSOR_MAP_SWIZZLE_128B) ||
        !make_tmap_2d(ctx, &tb, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, W, (uint64_t)N, (uint64_t)K, (uint64_t)ldw * 2, 64,
                      Cfg::BN_CTA, CU_TENSOR_MAP_SWIZZLE_128B) ||
        !make_tmap_2d(ctx, &te, CU_TENSOR_MAP_DATA_TYPE_UINT32, 4, meta, rb * kblocks * 2, 256, 1024, 256, 2,
                      CU_TENSOR_MAP_SWIZZLE_NONE) ||
        !make_tmap_2d(ctx, &ty, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, Y, (uint64_t)M, (uint64_t)N, (uint64_t)ldy * 2, Cfg::CH,
                      32, CU_TENSOR_MAP_SWIZZLE_NONE))
        return LYNX_ERR_CUDA;
    if (LORA) {
        if (!make_tmap_2d(ctx, &tt, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, lora->T, (uint64_t)M, (uint64_t)lora->R,
                          (uint64_t)lora->ldt * 2, 64, 128, CU_TENSOR_MAP_SWIZZLE_128B) ||
            !make_tmap_2d(ctx, &tla, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, lora->LA, (uint64_t)N, (uint64_t)lora->R,
                          (uint64_t)lora->ldla * 2, 64, Cfg::BN_CTA, CU_TENSOR_MAP_SWIZZLE_128B))
            return LYNX_ERR_CUDA;
    } else {
        tt = ta;  // never read: lora_steps = 0
        tla = tb;
    }
    Gemm2Params p;
    p.M = M; p.N = N; p.K = K;
    p.row_scale = comp ? comp->row_scale : nullptr;
    p.scale_partial = ss ? ss->partial : nullptr;
    p.scale_ks = ss ? ss->ks : 0;
    p.bias = static_cast<const uint16_t*>(bias);
    p.residual = comp ? static_cast<const uint16_t*>(comp->residual) : nullptr;
    p.ldr = comp ? comp->ldr : 0;
    p.dev_error = ctx->err_dev;
    p.sched.init((int)((M + 255) / 256), (int)((N + Cfg::BN - 1) / Cfg::BN), plan.clusters, plan.doubles, 8);
    p.lora_steps = LORA ? lora->R / 64 : 0;
    p.w_prefetch = layer_call ? 1 : 0;
    auto kern = sparse_gemm_rt2_kernel<Cfg, LORA>;
    static bool attr_set[MAX_CTX_DEVICES] = {};  // per instantiation
    if (lynx_status as = allow_dynamic_smem(kern, Cfg::SMEM_BYTES, ctx->device, attr_set); as != LYNX_OK) return as;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(plan.clusters * 2));
    cfg.blockDim = dim3(Cfg::THREADS);
    cfg.dynamicSmemBytes = Cfg::SMEM_BYTES;
    cfg.stream = st;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = ctx->pdl ? 1 : 0;
    cfg.attrs = attr;
    cfg.numAttrs = 2;
    if (cudaLaunchKernelEx(&cfg, kern, ta, tb, te, ty, tt, tla, p) != cudaSuccess) return LYNX_ERR_CUDA;
    ctx->launches++;
    return LYNX_OK;
}

// Tile configuration for (M, N, K): the development override, else the smallest modelled time.
// CTA-pair tiles 256 x {256, 240, 192, 128}.  A sparse MMA takes the same time whatever its N
// (up to 256), so wide tiles win; 240 is the widest that still double-buffers the accumulator.
// Model: rounds of tiles over the CTA pairs x (K blocks x measured time per K block + exposed
// epilogue).  Per-K-block times (us) are measured B200 figures for each tile shape; the 256-wide
// tile has one accumulator buffer, so its epilogue is not hidden.
int pick_gemm_cfg_model(int num_sms, int64_t M, int64_t N, int64_t K, int lora_steps, double* t_us = nullptr) {
    const int pairs = num_sms / 2;
    const double kb = (double)(K / 128) + lora_steps;
    // (the 192-wide tile runs with five stages of 42 KB, id 8: measured 4-7 % faster than with four)
    struct { int id, bn; double t_kb, epi; } cand[4] = {
        {7, 240, 0.465, 0.6}, {5, 256, 0.50, 3.0}, {8, 192, 0.39, 0.8}, {6, 128, 0.345, 0.5}};
    double best = 1e30;
    int cfg = 7;
    for (auto& c : cand) {
        const int64_t tiles = ((M + 255) / 256) * ((N + c.bn - 1) / c.bn);
        const double rounds = (double)((tiles + pairs - 1) / pairs);
        const double t = rounds * (kb * c.t_kb + c.epi);
        if (t < best) { best = t; cfg = c.id; }
    }
    if (t_us) *t_us = best;
    return cfg;
}
double gemm_model_time(int num_sms, int64_t M, int64_t N, int64_t K, int lora_steps) {
    double t = 0.0;
    pick_gemm_cfg_model(num_sms, M, N, K, lora_steps, &t);
    return t;
}
int pick_gemm_cfg(const lynx_ctx* ctx, int64_t M, int64_t N, int64_t K, int lora_steps) {
    if (ctx->gemm_cfg != 0) return ctx->gemm_cfg;
    return pick_gemm_cfg_model(ctx->num_sms, M, N, K, lora_steps);
}
// every tile but the 2-CTA 256 x 128 one has room in its W slot for a phase-0 stage
bool cfg_supports_l0(int cfg) { return cfg >= 1 && cfg <= 8 && cfg != 6; }

lynx_status launch_gemm(lynx_ctx* ctx, const void* values, const void* meta, int64_t M, int64_t K, const void* W,
                        int64_t N, int64_t ldw, const void* bias, const lynx_comp* comp, const LoraArgs* lora, void* Y,
                        int64_t ldy, cudaStream_t st, int cfg = 0, const ScaleSrc* ss = nullptr, bool layer_call = false) {
    const int lora_steps = lora ? lora->R / 64 : 0;
    if (cfg == 0 && ctx->gemm_cfg == 0 && ctx->rt2 != 0 && !ctx->streamk && !(lora && lora->X) && M > 256) {
        // the two-row-tile kernel where its schedule is modelled faster than the best plain tile
        const Rt2Plan plan = rt2_plan(ctx->num_sms, M, N, K, lora_steps, ctx->rt2_doubles);
        if (ctx->rt2 == 1 || plan.t_us < gemm_model_time(ctx->num_sms, M, N, K, lora_steps))
            return lora ? launch_gemm_rt2<true>(ctx, plan, values, meta, M, K, W, N, ldw, bias, comp, lora, Y, ldy, st, ss, layer_call)
                        : launch_gemm_rt2<false>(ctx, plan, values, meta, M, K, W, N, ldw, bias, comp, lora, Y, ldy, st, ss, layer_call);
    }
    if (cfg == 0) cfg = pick_gemm_cfg(ctx, M, N, K, lora_steps);
#define LYNX_GEMM_ARGS ctx, values, meta, M, K, W, N, ldw, bias, comp, lora, Y, ldy, st, ss, layer_call
    switch (cfg) {
        case 1: return launch_gemm_cfg<GemmCfg<128, 1, 4, 1>>(LYNX_GEMM_ARGS);
        case 2: return launch_gemm_cfg<GemmCfg<192, 1, 3, 1>>(LYNX_GEMM_ARGS);
        case 3: return launch_gemm_cfg<GemmCfg<256, 1, 2, 1>>(LYNX_GEMM_ARGS);
        case 4: return launch_gemm_cfg<GemmCfg<192, 2, 4, 2>>(LYNX_GEMM_ARGS);
        case 5: return launch_gemm_cfg<GemmCfg<256, 2, 4, 1>>(LYNX_GEMM_ARGS);
        case 6: return launch_gemm_cfg<GemmCfg<128, 2, 5, 2>>(LYNX_GEMM_ARGS);
        case 7: return launch_gemm_cfg<GemmCfg<240, 2, 4, 2>>(LYNX_GEMM_ARGS);
        case 8: return launch_gemm_cfg<GemmCfg<192, 2, 5, 1, false, 48>>(LYNX_GEMM_ARGS);  // five stages: one-round launches
        default: return LYNX_ERR_INVALID_ARG;
    }
#undef LYNX_GEMM_ARGS
}

// FP8 (E4M3) instantiation: byte tensor maps, K blocks of 256, optional per-channel weight scale.
template <class Cfg>
lynx_status launch_gemm_fp8_cfg(lynx_ctx* ctx, const void* values_q, const void* meta, int64_t M, int64_t K,
                                const void* Wq, int64_t N, int64_t ldwq, const float* wscale, const void* bias,
                                const lynx_comp* comp, void* Y, int64_t ldy, cudaStream_t st) {
    static_assert(Cfg::FP8, "FP8 configuration expected");
    CUtensorMap ta, tb, te, ty;
    const uint64_t rb = (uint64_t)((M + 127) / 128), kb128 = (uint64_t)(K / 128);
    if (!make_tmap_2d(ctx, &ta, CU_TENSOR_MAP_DATA_TYPE_UINT8, 1, values_q, (uint64_t)M, (uint64_t)(K / 2),
                      (uint64_t)(K / 2), 128, 128, CU_TENSOR_MAP_SWIZZLE_128B) ||
        !make_tmap_2d(ctx, &tb, CU_TENSOR_MAP_DATA_TYPE_UINT8, 1, Wq, (uint64_t)N, (uint64_t)K, (uint64_t)ldwq, 128,
                      Cfg::BN_CTA, CU_TENSOR_MAP_SWIZZLE_128B) ||
        !make_tmap_2d(ctx, &te, CU_TENSOR_MAP_DATA_TYPE_UINT32, 4, meta, rb * kb128 * 2, 256, 1024, 256,
                      Cfg::E_BYTES / 1024, CU_TENSOR_MAP_SWIZZLE_NONE) ||
        !make_tmap_2d(ctx, &ty, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, Y, (uint64_t)M, (uint64_t)N, (uint64_t)ldy * 2, Cfg::CH,
                      32, Cfg::CH == 64 ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_NONE))
        return LYNX_ERR_CUDA;
    GemmParams p = {};
    p.M = M; p.N = N; p.K = K;
    p.row_scale = comp ? comp->row_scale : nullptr;
    p.col_scale = wscale;
    p.bias = static_cast<const uint16_t*>(bias);
    p.residual = comp ? static_cast<const uint16_t*>(comp->residual) : nullptr;
    p.ldr = comp ? comp->ldr : 0;
    p.dev_error = ctx->err_dev;
    p.tiles_m = (int)((M + Cfg::BM * Cfg::CG - 1) / (Cfg::BM * Cfg::CG));
    p.tiles_n = (int)((N + Cfg::BN - 1) / Cfg::BN);
    p.group_m = gemm_group_rows(ctx, p.tiles_m);
    p.l0_splits = 1;
    auto kern = sparse_gemm_kernel<Cfg, false>;
    static bool attr_set[MAX_CTX_DEVICES] = {};  // per instantiation
    if (lynx_status as = allow_dynamic_smem(kern, Cfg::SMEM_BYTES, ctx->device, attr_set); as != LYNX_OK) return as;
    const int tiles = p.tiles_m * p.tiles_n;
    int clusters = ctx->num_sms / Cfg::CG;
    if (clusters > tiles) clusters = tiles;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(clusters * Cfg::CG));
    cfg.blockDim = dim3(Cfg::THREADS);
    cfg.dynamicSmemBytes = Cfg::SMEM_BYTES;
    cfg.stream = st;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = Cfg::CG;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = ctx->pdl ? 1 : 0;
    cfg.attrs = attr;
    cfg.numAttrs = 2;
    if (cudaLaunchKernelEx(&cfg, kern, ta, tb, te, ty, ta, tb, ta, tb, p) != cudaSuccess) return LYNX_ERR_CUDA;
    ctx->launches++;
    return LYNX_OK;
}

// FP8 tile choice: the development override if it names a CTA-pair tile, else the cost model's
// choice among the same pair tiles (a stage is 256 K here; relative times as for bf16).
lynx_status launch_gemm_fp8(lynx_ctx* ctx, const void* values_q, const void* meta, int64_t M, int64_t K,
                            const void* Wq, int64_t N, int64_t ldwq, const float* wscale, const void* bias,
                            const lynx_comp* comp, void* Y, int64_t ldy, cudaStream_t st) {
    int cfg = ctx->gemm_cfg;
    if (cfg != 4 && cfg != 6 && cfg != 7) {
        cfg = pick_gemm_cfg_model(ctx->num_sms, M, N, K / 2, 0);
        if (cfg == 8) cfg = 4;  // (FP8 stages are larger: four of them)
        if (cfg == 5) cfg = 7;  // the 256-wide tile has no FP8 instantiation (no tensor memory left for metadata)
    }
#define LYNX_FP8_ARGS ctx, values_q, meta, M, K, Wq, N, ldwq, wscale, bias, comp, Y, ldy, st
    switch (cfg) {
        case 4: return launch_gemm_fp8_cfg<GemmCfg<192, 2, 4, 2, true>>(LYNX_FP8_ARGS);
        case 6: return launch_gemm_fp8_cfg<GemmCfg<128, 2, 5, 2, true>>(LYNX_FP8_ARGS);
        default: return launch_gemm_fp8_cfg<GemmCfg<240, 2, 4, 2, true>>(LYNX_FP8_ARGS);
    }
#undef LYNX_FP8_ARGS
}

// One-kernel path: raw X is pruned inside the GEMM kernel.
lynx_status launch_fused(lynx_ctx* ctx, const void* X, int64_t M, int64_t K, int64_t ldx, const void* W, int64_t N,
                         int64_t ldw, const void* bias, int with_scale, const void* residual, int64_t ldr, void* Y,
                         int64_t ldy, cudaStream_t st) {
    using Cfg = FusedCfg;
    CUtensorMap tx, tb, ty;
    if (!make_tmap_2d(ctx, &tx, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, X, (uint64_t)M, (uint64_t)K, (uint64_t)ldx * 2, 64,
                      Cfg::BM, CU_TENSOR_MAP_SWIZZLE_128B) ||
        !make_tmap_2d(ctx, &tb, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, W, (uint64_t)N, (uint64_t)K, (uint64_t)ldw * 2, 64,
                      Cfg::BN, CU_TENSOR_MAP_SWIZZLE_128B) ||
        !make_tmap_2d(ctx, &ty, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, Y, (uint64_t)M, (uint64_t)N, (uint64_t)ldy * 2, 64,
                      32, CU_TENSOR_MAP_SWIZZLE_128B))
        return LYNX_ERR_CUDA;
    FusedParams p;
    p.M = M; p.N = N; p.K = K;
    p.with_scale = with_scale;
    p.bias = static_cast<const uint16_t*>(bias);
    p.residual = static_cast<const uint16_t*>(residual);
    p.ldr = ldr;
    p.dev_error = ctx->err_dev;
    p.tiles_m = (int)((M + Cfg::BM - 1) / Cfg::BM);
    p.tiles_n = (int)((N + Cfg::BN - 1) / Cfg::BN);
    static bool attr_set[MAX_CTX_DEVICES] = {};
    if (lynx_status as = allow_dynamic_smem(fused_linear_kernel, Cfg::SMEM_BYTES, ctx->device, attr_set); as != LYNX_OK)
        return as;
    int grid = p.tiles_m * p.tiles_n;
    if (grid > ctx->num_sms) grid = ctx->num_sms;
    fused_linear_kernel<<<grid, Cfg::THREADS, Cfg::SMEM_BYTES, st>>>(tx, tb, ty, p);
    if (cudaGetLastError() != cudaSuccess) return LYNX_ERR_CUDA;
    ctx->launches++;
    return LYNX_OK;
}

lynx_status check_common(lynx_ctx* ctx, int64_t M, int64_t K) {
    if (!ctx) return LYNX_ERR_INVALID_ARG;
    if (M < 1 || K < 128) return LYNX_ERR_INVALID_ARG;
    if (K % 128 != 0) return LYNX_ERR_UNSUPPORTED_SHAPE;
    if (M > (1ll << 30) || K > (1ll << 30)) return LYNX_ERR_UNSUPPORTED_SHAPE;
    return LYNX_OK;
}

// The deferred row sums of a two-call user live in the scratch: whoever reallocates it or writes
// other data into it forgets them, so that a GEMM call that still asks for them is refused
// (LYNX_ERR_INVALID_ARG) instead of reading freed or overwritten memory.
void clear_deferred(lynx_ctx* ctx) {
    ctx->deferred_partial = nullptr;
    ctx->deferred_ks = 0;
    ctx->deferred_M = 0;
    ctx->deferred_K = 0;
}

lynx_status ensure_scratch(lynx_ctx* ctx, size_t bytes) {
    if (ctx->scratch_bytes >= bytes) return LYNX_OK;
    clear_deferred(ctx);
    if (cudaDeviceSynchronize() != cudaSuccess) return LYNX_ERR_CUDA;
    if (ctx->scratch) cudaFree(ctx->scratch);
    ctx->scratch = nullptr;
    ctx->scratch_bytes = 0;
    if (cudaMalloc(&ctx->scratch, bytes) != cudaSuccess) return LYNX_ERR_WORKSPACE;
    ctx->scratch_bytes = bytes;
    return LYNX_OK;
}

lynx_status ensure_host_stage(lynx_ctx* ctx, size_t bytes) {
    if (ctx->host_stage_bytes >= bytes) return LYNX_OK;
    if (cudaDeviceSynchronize() != cudaSuccess) return LYNX_ERR_CUDA;
    if (ctx->host_stage) cudaFree(ctx->host_stage);
    ctx->host_stage = nullptr;
    ctx->host_stage_bytes = 0;
    if (cudaMalloc(&ctx->host_stage, bytes) != cudaSuccess) return LYNX_ERR_WORKSPACE;
    ctx->host_stage_bytes = bytes;
    return LYNX_OK;
}

// ----------------------------------------------------------------- low-rank down projection -----

// K splits of the down projection: rounds of CTAs over the SMs x (K blocks per split + a fixed
// per-CTA cost of ~6 K blocks for prologue and drain), smallest wins; every split is non-empty.
void lora_split_plan(int num_sms, int64_t M, int64_t K, int* splits, int* kb_per_split) {
    const int tiles_m = (int)((M + 127) / 128), kblocks = (int)(K / 64);
    int best_s = 1;
    double best = 1e30;
    for (int sp = 1; sp <= 32 && sp * 4 <= kblocks; ++sp) {
        const int per = (kblocks + sp - 1) / sp;
        const int real = (kblocks + per - 1) / per;
        const double rounds = (double)(((int64_t)tiles_m * real + num_sms - 1) / num_sms);
        const double t = rounds * (per + 6.0);
        if (t < best) { best = t; best_s = real; }
    }
    const int per = (kblocks + best_s - 1) / best_s;
    *kb_per_split = per;
    *splits = (kblocks + per - 1) / per;
}

struct LoraWsLayout {
    size_t partial, T, total;
};
LoraWsLayout lora_ws_layout(int num_sms, int64_t M, int64_t K, int R) {
    int splits, per;
    lora_split_plan(num_sms, M, K, &splits, &per);
    LoraWsLayout L;
    const size_t tiles_m = (size_t)((M + 127) / 128);
    size_t partial = splits > 1 ? tiles_m * splits * 128 * (size_t)R * 4 : 0;
    if (R == 64) {
        // the in-GEMM down projection: 256-row blocks over CTA pairs, or 128-row blocks over single CTAs
        // (the same bytes whether the blocks are 256 rows over CTA pairs or 128 rows over single CTAs)
        const size_t f = (size_t)((M + 255) / 256) * L0_MAX_SPLITS * 256 * 64 * 4;
        if (f > partial) partial = f;
    }
    L.partial = 0;
    size_t off = align_up(partial, 1024);
    L.T = off;
    off = align_up(off + (size_t)M * R * 2, 1024);
    L.total = off;
    return L;
}

lynx_status ensure_lora_ws(lynx_ctx* ctx, size_t bytes) {
    if (ctx->lora_ws_bytes >= bytes) return LYNX_OK;
    if (cudaDeviceSynchronize() != cudaSuccess) return LYNX_ERR_CUDA;
    if (ctx->lora_ws) cudaFree(ctx->lora_ws);
    ctx->lora_ws = nullptr;
    ctx->lora_ws_bytes = 0;
    if (cudaMalloc(&ctx->lora_ws, bytes) != cudaSuccess) return LYNX_ERR_WORKSPACE;
    ctx->lora_ws_bytes = bytes;
    return LYNX_OK;
}

template <class Cfg>
lynx_status launch_lora_down(lynx_ctx* ctx, const void* X, int64_t M, int64_t K, int64_t ldx, const void* LB,
                             int64_t ldlb, const float* row_scale, void* T, int64_t ldt, float* partial,
                             cudaStream_t st) {
    CUtensorMap tx, tlb;
    if (!make_tmap_2d(ctx, &tx, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, X, (uint64_t)M, (uint64_t)K, (uint64_t)ldx * 2, 64,
                      Cfg::BM, CU_TENSOR_MAP_SWIZZLE_128B) ||
        !make_tmap_2d(ctx, &tlb, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, LB, (uint64_t)Cfg::R, (uint64_t)K,
                      (uint64_t)ldlb * 2, 64, Cfg::R, CU_TENSOR_MAP_SWIZZLE_128B))
        return LYNX_ERR_CUDA;
    LoraDownParams p;
    p.M = M; p.K = K;
    lora_split_plan(ctx->num_sms, M, K, &p.splits, &p.kb_per_split);
    p.row_scale = row_scale;
    p.T = static_cast<uint16_t*>(T);
    p.ldt = ldt;
    p.partial = partial;
    p.tickets = ctx->tickets + PRUNE_TICKET_BYTES / 4;
    p.dev_error = ctx->err_dev;
    auto kern = lora_down_kernel<Cfg>;
    static bool attr_set[MAX_CTX_DEVICES] = {};  // per instantiation
    if (lynx_status as = allow_dynamic_smem(kern, Cfg::SMEM_BYTES, ctx->device, attr_set); as != LYNX_OK) return as;
    const int tiles_m = (int)((M + Cfg::BM - 1) / Cfg::BM);
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(tiles_m * p.splits));
    cfg.blockDim = dim3(Cfg::THREADS);
    cfg.dynamicSmemBytes = Cfg::SMEM_BYTES;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = ctx->pdl ? 1 : 0;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    if (cudaLaunchKernelEx(&cfg, kern, tx, tlb, p) != cudaSuccess) return LYNX_ERR_CUDA;
    ctx->launches++;
    return LYNX_OK;
}

// K splits of the prune + down-projection kernel (128-element K blocks) = CTAs per cluster, 1..8.
// Every CTA holds a whole SM; `cap[i]` = CTAs of clusters of i + 1 that the GPU holds at once.
void prune_lora_plan(const int cap[8], int64_t M, int64_t K, int* splits, int* kb_per_split) {
    const int tiles_m = (int)((M + 127) / 128), kblocks = (int)(K / 128);
    int best_s = 1, best_per = kblocks;
    double best = 1e30;
    for (int i = 0; i < 8; ++i) {
        const int sp = i + 1;
        if (sp > kblocks) break;
        if (cap[i] < sp) continue;
        const int per = (kblocks + sp - 1) / sp;
        if ((kblocks + per - 1) / per != sp) continue;  // every CTA of the cluster needs a K block
        const double rounds = (double)(((int64_t)tiles_m * sp + cap[i] - 1) / cap[i]);
        const double t = rounds * (per + 4.0);
        if (t < best) { best = t; best_s = sp; best_per = per; }
    }
    *splits = best_s;
    *kb_per_split = best_per;
}

template <class Cfg, bool SUMS>
lynx_status launch_prune_lora(lynx_ctx* ctx, const void* X, int64_t M, int64_t K, int64_t ldx, const void* LB,
                              int64_t ldlb, void* values, void* meta, float* scale_partial, void* T, int64_t ldt,
                              cudaStream_t st, int* splits_out) {
    CUtensorMap tx, tlb;
    if (!make_tmap_2d(ctx, &tx, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, X, (uint64_t)M, (uint64_t)K, (uint64_t)ldx * 2, 64,
                      Cfg::BM, CU_TENSOR_MAP_SWIZZLE_128B) ||
        !make_tmap_2d(ctx, &tlb, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, LB, (uint64_t)Cfg::R, (uint64_t)K,
                      (uint64_t)ldlb * 2, 64, Cfg::R, CU_TENSOR_MAP_SWIZZLE_128B))
        return LYNX_ERR_CUDA;
    auto kern = prune_lora_kernel<Cfg, SUMS>;
    static bool attr_set[MAX_CTX_DEVICES] = {};  // per instantiation
    if (lynx_status as = allow_dynamic_smem(kern, Cfg::SMEM_BYTES, ctx->device, attr_set); as != LYNX_OK) return as;
    // how many CTAs of clusters of 1..8 fit on the GPU at once (asked once per device)
    static int caps[MAX_CTX_DEVICES][8] = {};
    int* cap = caps[ctx->device];
    if (cap[0] == 0) {
        for (int i = 0; i < 8; ++i) {
            cudaLaunchConfig_t qc = {};
            qc.gridDim = dim3((unsigned)(ctx->num_sms / (i + 1) * (i + 1)));
            qc.blockDim = dim3(Cfg::THREADS);
            qc.dynamicSmemBytes = Cfg::SMEM_BYTES;
            cudaLaunchAttribute qa[1];
            qa[0].id = cudaLaunchAttributeClusterDimension;
            qa[0].val.clusterDim.x = (unsigned)(i + 1);
            qa[0].val.clusterDim.y = 1;
            qa[0].val.clusterDim.z = 1;
            qc.attrs = qa;
            qc.numAttrs = 1;
            int n = 0;
            if (cudaOccupancyMaxActiveClusters(&n, kern, &qc) != cudaSuccess) n = 0;
            cap[i] = n * (i + 1);
        }
        if (cap[0] <= 0) cap[0] = ctx->num_sms;
    }
    PruneLoraParams p;
    p.M = M; p.K = K;
    prune_lora_plan(cap, M, K, &p.splits, &p.kb_per_split);
    if (const int f = ctx->pl_force_splits; f >= 1 && f <= 8 && cap[f - 1] >= f) {
        const int kblocks = (int)(K / 128), per = (kblocks + f - 1) / f;
        if (f <= kblocks && (kblocks + per - 1) / per == f) {  // every CTA of the cluster gets a K block
            p.splits = f;
            p.kb_per_split = per;
        }
    }
    p.values = static_cast<uint16_t*>(values);
    p.meta = static_cast<uint8_t*>(meta);
    p.scale_partial = scale_partial;
    p.T = static_cast<uint16_t*>(T);
    p.ldt = ldt;
    p.dev_error = ctx->err_dev;
    const int tiles_m = (int)((M + Cfg::BM - 1) / Cfg::BM);
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(tiles_m * p.splits));
    cfg.blockDim = dim3(Cfg::THREADS);
    cfg.dynamicSmemBytes = Cfg::SMEM_BYTES;
    cfg.stream = st;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = (unsigned)p.splits;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = ctx->pdl ? 1 : 0;
    cfg.attrs = attr;
    cfg.numAttrs = 2;
    if (cudaLaunchKernelEx(&cfg, kern, tx, tlb, p) != cudaSuccess) return LYNX_ERR_CUDA;
    ctx->launches++;
    *splits_out = p.splits;
    return LYNX_OK;
}

lynx_status check_lora_rank(int64_t R) {
    if (R < 1) return LYNX_ERR_INVALID_ARG;
    if (R != 64 && R != 128) return LYNX_ERR_UNSUPPORTED_SHAPE;
    return LYNX_OK;
}

}  // namespace

// ================================================================================ C ABI ==========

extern "C" {

lynx_status lynx_create(lynx_ctx** out, int device) {
    if (!out) return LYNX_ERR_INVALID_ARG;
    *out = nullptr;
    int count = 0;
    if (cudaGetDeviceCount(&count) != cudaSuccess || device < 0 || device >= count) return LYNX_ERR_CUDA;
    if (cudaSetDevice(device) != cudaSuccess) return LYNX_ERR_CUDA;
    cudaDeviceProp prop;
    if (cudaGetDeviceProperties(&prop, device) != cudaSuccess) return LYNX_ERR_CUDA;
    if (prop.major != 10) return LYNX_ERR_UNSUPPORTED_ARCH;
    if (!get_encode()) return LYNX_ERR_CUDA;
    lynx_ctx* ctx = new (std::nothrow) lynx_ctx();
    if (!ctx) return LYNX_ERR_WORKSPACE;
    ctx->device = device;
    ctx->num_sms = prop.multiProcessorCount;
    if (cudaHostAlloc(reinterpret_cast<void**>(&ctx->err_host), 64, cudaHostAllocMapped) != cudaSuccess ||
        cudaHostGetDevicePointer(reinterpret_cast<void**>(&ctx->err_dev), ctx->err_host, 0) != cudaSuccess) {
        delete ctx;
        return LYNX_ERR_CUDA;
    }
    *ctx->err_host = DEV_OK;
    if (cudaMalloc(reinterpret_cast<void**>(&ctx->tickets), TICKET_ALLOC_BYTES) != cudaSuccess ||
        cudaMemset(ctx->tickets, 0, TICKET_ALLOC_BYTES) != cudaSuccess) {
        cudaFreeHost(ctx->err_host);
        delete ctx;
        return LYNX_ERR_WORKSPACE;
    }
    // Development overrides (tile configuration, schedules, kernel forms) are read only when
    // LYNX_DEV=1 is set: tests and measurement scripts set it, a production process reads nothing else.
    const char* dev = getenv("LYNX_DEV");
    if (dev && atoi(dev) == 1) {
        auto geti = [](const char* name, int* dst) {
            const char* e = getenv(name);
            if (e) *dst = atoi(e);
            return e != nullptr;
        };
        geti("LYNX_GEMM_CFG", &ctx->gemm_cfg);            // tile configuration
        geti("LYNX_PDL", &ctx->pdl);                      // 0 turns programmatic dependent launch off
        geti("LYNX_STREAMK", &ctx->streamk);              // 1 turns the stream-K tail on
        geti("LYNX_LORA_FUSE", &ctx->lora_fuse);          // down projection: 0 own kernel, 1 in the GEMM launch, 2 in the prune launch
        geti("LYNX_L0_SPLITS", &ctx->l0_force_splits);    // K splits of the in-GEMM down projection,
        geti("LYNX_L0_FILL", &ctx->l0_force_fill);        // and items per light cluster (0: round-robin over all clusters)
        geti("LYNX_DEFER_SCALE", &ctx->defer_scale);
        geti("LYNX_PRUNE_TPU", &ctx->prune_tpu);          // 128-element K blocks per warp
        geti("LYNX_GEMM_GROUP_M", &ctx->gemm_group_m);    // row tiles per group of the GEMM's tile order
        geti("LYNX_PL_SPLITS", &ctx->pl_force_splits);    // K splits (= cluster size) of the prune + down-projection kernel
        if (geti("LYNX_FP8_RING", &ctx->fp8_ring)) ctx->fp8_ring_forced = 1;  // 0 = one CTA per 16 rows, n = ring with n warps per row
        geti("LYNX_RT2", &ctx->rt2);                      // two-row-tile GEMM kernel: 0 never, 1 whenever it applies
        geti("LYNX_RT2_D", &ctx->rt2_doubles);            // and the number of 512-row items of its schedule
        geti("LYNX_SPLITK", &ctx->splitk_force);          // in-cluster split-K of the GEMM: 0 off, 1 model (default), 2..4 forced
        geti("LYNX_PRUNE_FINALIZE", &ctx->prune_finalize);  // row-scale finalize: 0 model, 1 in-kernel ticket, 2 own launch
    }
    if (ctx->streamk) {
        // stream-K partial tiles (one slot per cluster) and their ready words: allocated here so
        // that no launch call ever allocates
        const size_t slot = (size_t)128 * 256 * 4, nslots = (size_t)ctx->num_sms;
        void* buf = nullptr;
        if (cudaMalloc(&buf, nslots * slot + nslots * 8 * 4) != cudaSuccess ||
            cudaMemset(buf, 0, nslots * slot + nslots * 8 * 4) != cudaSuccess) {
            if (buf) cudaFree(buf);
            cudaFree(ctx->tickets);
            cudaFreeHost(ctx->err_host);
            delete ctx;
            return LYNX_ERR_WORKSPACE;
        }
        ctx->sk_partial = static_cast<float*>(buf);
        ctx->sk_flags = reinterpret_cast<uint32_t*>(static_cast<char*>(buf) + nslots * slot);
    }
    *out = ctx;
    return LYNX_OK;
}

lynx_status lynx_destroy(lynx_ctx* ctx) {
    if (!ctx) return LYNX_ERR_INVALID_ARG;
    cudaSetDevice(ctx->device);
    if (ctx->scratch) cudaFree(ctx->scratch);
    if (ctx->host_stage) cudaFree(ctx->host_stage);
    if (ctx->sk_partial) cudaFree(ctx->sk_partial);
    if (ctx->tickets) cudaFree(ctx->tickets);
    if (ctx->lora_ws) cudaFree(ctx->lora_ws);
    if (ctx->h2d_stream) cudaStreamDestroy(ctx->h2d_stream);
    if (ctx->d2h_stream) cudaStreamDestroy(ctx->d2h_stream);
    for (int i = 0; i < 8; ++i) {
        if (ctx->ev_h2d[i]) cudaEventDestroy(ctx->ev_h2d[i]);
        if (ctx->ev_done[i]) cudaEventDestroy(ctx->ev_done[i]);
    }
    if (ctx->ev_all) cudaEventDestroy(ctx->ev_all);
    if (ctx->err_host) cudaFreeHost(ctx->err_host);
    delete ctx;
    return LYNX_OK;
}

const char* lynx_status_string(lynx_status s) {
    switch (s) {
        case LYNX_OK: return "ok";
        case LYNX_ERR_INVALID_ARG: return "invalid argument";
        case LYNX_ERR_UNSUPPORTED_SHAPE: return "unsupported shape (need K % 128 == 0, N % 8 == 0)";
        case LYNX_ERR_ALIGNMENT: return "pointer or leading dimension not 16-byte aligned";
        case LYNX_ERR_WORKSPACE: return "scratch too small or its allocation failed";
        case LYNX_ERR_CUDA: return "CUDA runtime error";
        case LYNX_ERR_TIMEOUT: return "device-side wait timed out";
        case LYNX_ERR_UNSUPPORTED_ARCH: return "device is not sm_100";
    }
    return "unknown status";
}

lynx_status lynx_last_error(lynx_ctx* ctx) {
    if (!ctx) return LYNX_ERR_INVALID_ARG;
    lynx_status s = check_device_error(ctx);
    *ctx->err_host = DEV_OK;
    return s;
}

size_t lynx_values_bytes(int64_t M, int64_t K) { return (size_t)M * (size_t)(K / 2) * 2; }
size_t lynx_meta_bytes(int64_t M, int64_t K) { return (size_t)((M + 127) / 128) * (size_t)(K / 128) * 2048; }
size_t lynx_workspace_bytes(int64_t M, int64_t N, int64_t K) { return scratch_layout(M, K).total; }

lynx_status lynx_reserve(lynx_ctx* ctx, int64_t M, int64_t N, int64_t K) {
    if (!ctx || M < 1 || N < 1 || K < 1) return LYNX_ERR_INVALID_ARG;
    std::lock_guard<std::mutex> lock(ctx->mu);
    return ensure_scratch(ctx, scratch_layout(M, K).total);
}

int64_t lynx_launch_count(lynx_ctx* ctx) { return ctx ? ctx->launches : -1; }

// The prune/compress launch.  defer (ROW mode only): the kernel stops at the per-K-split row sums
// and `src` tells the following GEMM where they are; its epilogue adds them in the same order the
// in-kernel finalize would (same bits), which saves the ticket hand-over inside this kernel.
static bool sums_needed(lynx_comp_mode mode) { return mode == LYNX_COMP_ROW || mode == LYNX_COMP_TENSOR; }

static lynx_status prune_impl(lynx_ctx* ctx, const void* X, int64_t M, int64_t K, int64_t ldx, void* values,
                              void* meta, float* row_scale, lynx_comp_mode mode, void* stream, bool defer,
                              ScaleSrc* src) {
    lynx_status s = check_common(ctx, M, K);
    if (s != LYNX_OK) return s;
    if (!X || !values || !meta) return LYNX_ERR_INVALID_ARG;
    if (mode != LYNX_COMP_NONE && mode != LYNX_COMP_ROW && mode != LYNX_COMP_TENSOR && mode != LYNX_COMP_GROUP)
        return LYNX_ERR_INVALID_ARG;
    if (mode != LYNX_COMP_ROW) defer = false;
    if (sums_needed(mode) && !row_scale && !defer) return LYNX_ERR_INVALID_ARG;
    // ROW mode with the scale wanted from this call: on long rows the prune launch stops at its
    // partial sums and a small dependent launch finishes the scale (measured 30.8 against 33.3 us
    // on 4096 x 12288); on short rows the ticket hand-over inside the prune kernel is faster
    // (12-13 against 16-17 us at K = 3072).  Same additions in the same order either way.
    bool own_finalize = false;
    if (mode == LYNX_COMP_ROW && !defer) {
        own_finalize = ctx->prune_finalize == 2 || (ctx->prune_finalize == 0 && K >= 8192);
        if (K / 128 < 2) own_finalize = false;  // one K split: the kernel writes the scale directly
    }
    if (ldx < K) return LYNX_ERR_INVALID_ARG;
    if (!aligned16(X) || !aligned16(values) || !aligned16(meta) || (ldx % 16) != 0 ||
        (reinterpret_cast<uintptr_t>(X) & 31u) || (reinterpret_cast<uintptr_t>(values) & 31u))
        return LYNX_ERR_ALIGNMENT;  // 32-byte vector accesses
    if ((s = check_device_error(ctx)) != LYNX_OK) return s;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const PrunePlan P = prune_plan(ctx->num_sms, M, K, ctx->prune_tpu);
    const int tpu = P.tpu, KS = P.KS, ctas_per_rb = P.ctas_per_rb;
    const unsigned grid = P.grid;
    // every refusal comes before any allocation
    if ((size_t)P.rb16 * 4 > PRUNE_TICKET_BYTES) return LYNX_ERR_UNSUPPORTED_SHAPE;
    float* sums = nullptr;
    float* partial = nullptr;
    if (sums_needed(mode)) {
        std::lock_guard<std::mutex> lock(ctx->mu);
        ScratchLayout L = scratch_layout(M, K);
        if (ctx->scratch_bytes < L.prune_end) {
            if ((s = ensure_scratch(ctx, L.total)) != LYNX_OK) return s;
        }
        char* base = static_cast<char*>(ctx->scratch);
        partial = reinterpret_cast<float*>(base + L.partial);
        sums = reinterpret_cast<float*>(base + L.sums);
    }
    {
        cudaLaunchConfig_t pc = {};
        pc.gridDim = dim3(grid);
        pc.blockDim = dim3(PRUNE_CTA_WARPS * 32);
        pc.stream = st;
        cudaLaunchAttribute pa[1];
        pa[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        pa[0].val.programmaticStreamSerializationAllowed = ctx->pdl ? 1 : 0;
        pc.attrs = pa;
        pc.numAttrs = 1;
        const uint16_t* Xp = static_cast<const uint16_t*>(X);
        uint16_t* vp = static_cast<uint16_t*>(values);
        uint8_t* mp = static_cast<uint8_t*>(meta);
        float* none_f = nullptr;
        uint32_t* none_u = nullptr;
        cudaError_t e;
        if (mode == LYNX_COMP_NONE)
            e = cudaLaunchKernelEx(&pc, prune_compress_kernel<false, false>, Xp, M, K, ldx, vp, mp, row_scale, none_f,
                                   none_f, none_u, 0, tpu, KS, ctas_per_rb, 0);
        else if (mode == LYNX_COMP_GROUP)
            e = cudaLaunchKernelEx(&pc, prune_compress_kernel<false, true>, Xp, M, K, ldx, vp, mp, row_scale, none_f,
                                   none_f, none_u, 0, tpu, KS, ctas_per_rb, 0);
        else
            e = cudaLaunchKernelEx(&pc, prune_compress_kernel<true, false>, Xp, M, K, ldx, vp, mp, row_scale, sums, partial,
                                   ctx->tickets, (int)mode, tpu, KS, ctas_per_rb, (defer || (own_finalize && KS > 1)) ? 1 : 0);
        if (e != cudaSuccess) return LYNX_ERR_CUDA;
        if (own_finalize && KS > 1) {
            pc.gridDim = dim3((unsigned)((M + 15) / 16));
            pc.blockDim = dim3(128);
            const float* cpart = partial;
            if (cudaLaunchKernelEx(&pc, row_scale_finalize_kernel, cpart, M, KS, row_scale) != cudaSuccess) return LYNX_ERR_CUDA;
            ctx->launches++;
        }
    }
    ctx->launches++;
    if (mode == LYNX_COMP_TENSOR) {
        tensor_scale_kernel<<<1, 1024, 0, st>>>(sums, M, row_scale);
        ctx->launches++;
    }
    if (src) {
        src->partial = defer ? partial : nullptr;
        src->ks = defer ? KS : 0;
    }
    if (mode != LYNX_COMP_NONE && mode != LYNX_COMP_GROUP) {  // the scratch's sums now belong to this call
        ctx->deferred_partial = defer ? partial : nullptr;
        ctx->deferred_ks = defer ? KS : 0;
        ctx->deferred_M = M;
        ctx->deferred_K = K;
    }
    return cuda_ok(cudaGetLastError());
}

lynx_status lynx_prune_compress(lynx_ctx* ctx, const void* X, int64_t M, int64_t K, int64_t ldx, void* values,
                                void* meta, float* row_scale, lynx_comp_mode mode, void* stream) {
    if (row_scale == LYNX_ROW_SCALE_DEFERRED) {
        if (mode != LYNX_COMP_ROW) return LYNX_ERR_INVALID_ARG;
        return prune_impl(ctx, X, M, K, ldx, values, meta, nullptr, mode, stream, true, nullptr);
    }
    return prune_impl(ctx, X, M, K, ldx, values, meta, row_scale, mode, stream, false, nullptr);
}

lynx_status lynx_sparse_linear(lynx_ctx* ctx, const void* values, const void* meta, int64_t M, int64_t K,
                               const void* W, int64_t N, int64_t ldw, const void* bias, const lynx_comp* comp,
                               void* Y, int64_t ldy, void* stream) {
    lynx_status s = check_common(ctx, M, K);
    if (s != LYNX_OK) return s;
    if (!values || !meta || !W || !Y || N < 8) return LYNX_ERR_INVALID_ARG;
    if (N % 8 != 0) return LYNX_ERR_UNSUPPORTED_SHAPE;
    if (ldw < K || ldy < N) return LYNX_ERR_INVALID_ARG;
    if (!aligned16(values) || !aligned16(meta) || !aligned16(W) || !aligned16(Y) || (ldw % 8) || (ldy % 8))
        return LYNX_ERR_ALIGNMENT;
    if (bias && !aligned16(bias)) return LYNX_ERR_ALIGNMENT;
    if (comp && comp->residual) {
        if (comp->ldr < N) return LYNX_ERR_INVALID_ARG;
        if (!aligned16(comp->residual) || (comp->ldr % 8)) return LYNX_ERR_ALIGNMENT;
    }
    if ((s = check_device_error(ctx)) != LYNX_OK) return s;
    if (comp && comp->row_scale == LYNX_ROW_SCALE_DEFERRED) {
        // the sums of the deferred prune call that preceded this one on the context
        if (!ctx->deferred_partial || ctx->deferred_M != M || ctx->deferred_K != K) return LYNX_ERR_INVALID_ARG;
        ScaleSrc ss;
        ss.partial = ctx->deferred_partial;
        ss.ks = ctx->deferred_ks;
        lynx_comp c2 = *comp;
        c2.row_scale = nullptr;
        return launch_gemm(ctx, values, meta, M, K, W, N, ldw, bias, &c2, nullptr, Y, ldy,
                           static_cast<cudaStream_t>(stream), 0, &ss);
    }
    return launch_gemm(ctx, values, meta, M, K, W, N, ldw, bias, comp, nullptr, Y, ldy,
                       static_cast<cudaStream_t>(stream));
}

lynx_status lynx_act_sparse_linear(lynx_ctx* ctx, const void* X, int64_t M, int64_t K, int64_t ldx, const void* W,
                                   int64_t N, int64_t ldw, const void* bias, lynx_comp_mode mode,
                                   const void* residual, int64_t ldr, void* Y, int64_t ldy, lynx_fuse_mode fuse,
                                   void* stream) {
    lynx_status s = check_common(ctx, M, K);
    if (s != LYNX_OK) return s;
    if (fuse != LYNX_FUSE_AUTO && fuse != LYNX_FUSE_SEPARATE && fuse != LYNX_FUSE_FUSED) return LYNX_ERR_INVALID_ARG;
    if (N < 8) return LYNX_ERR_INVALID_ARG;
    if (fuse == LYNX_FUSE_FUSED) {
        // the whole-tensor scale needs all of X before the first output: two-kernel path only
        // (and the per-group factors are only built into the stand-alone prune kernel)
        if (mode == LYNX_COMP_TENSOR || mode == LYNX_COMP_GROUP) return LYNX_ERR_UNSUPPORTED_SHAPE;
        if (mode != LYNX_COMP_NONE && mode != LYNX_COMP_ROW) return LYNX_ERR_INVALID_ARG;
        if (!X || !W || !Y) return LYNX_ERR_INVALID_ARG;
        if (N % 8 != 0) return LYNX_ERR_UNSUPPORTED_SHAPE;
        if (ldx < K || ldw < K || ldy < N || (residual && ldr < N)) return LYNX_ERR_INVALID_ARG;
        if (!aligned16(X) || !aligned16(W) || !aligned16(Y) || (ldx % 8) || (ldw % 8) || (ldy % 8) ||
            (bias && !aligned16(bias)) || (residual && (!aligned16(residual) || (ldr % 8))))
            return LYNX_ERR_ALIGNMENT;
        if ((s = check_device_error(ctx)) != LYNX_OK) return s;
        return launch_fused(ctx, X, M, K, ldx, W, N, ldw, bias, mode == LYNX_COMP_ROW ? 1 : 0, residual, ldr, Y, ldy,
                            static_cast<cudaStream_t>(stream));
    }
    // every argument is checked before the first launch
    if (!X || !W || !Y) return LYNX_ERR_INVALID_ARG;
    if (N % 8 != 0) return LYNX_ERR_UNSUPPORTED_SHAPE;
    if (ldx < K || ldw < K || ldy < N || (residual && ldr < N)) return LYNX_ERR_INVALID_ARG;
    if (!aligned16(W) || !aligned16(Y) || (ldw % 8) || (ldy % 8) || (bias && !aligned16(bias)) ||
        (residual && (!aligned16(residual) || (ldr % 8))))
        return LYNX_ERR_ALIGNMENT;
    ScratchLayout L = scratch_layout(M, K);
    {
        std::lock_guard<std::mutex> lock(ctx->mu);
        clear_deferred(ctx);  // this call writes the scratch
        if ((s = ensure_scratch(ctx, L.total)) != LYNX_OK) return s;
    }
    char* base = static_cast<char*>(ctx->scratch);
    void* values = base + L.values;
    void* meta = base + L.meta;
    float* scale = reinterpret_cast<float*>(base + L.scale);
    // ROW mode: the prune launch stops at its per-K-split row sums and the GEMM's epilogue adds them
    ScaleSrc ss;
    s = prune_impl(ctx, X, M, K, ldx, values, meta, sums_needed(mode) ? scale : nullptr, mode, stream,
                   ctx->defer_scale != 0, &ss);
    if (s != LYNX_OK) return s;
    lynx_comp comp;
    comp.row_scale = (!sums_needed(mode) || ss.partial) ? nullptr : scale;
    comp.residual = residual;
    comp.ldr = ldr;
    if ((s = check_device_error(ctx)) == LYNX_OK)
        s = launch_gemm(ctx, values, meta, M, K, W, N, ldw, bias, &comp, nullptr, Y, ldy,
                        static_cast<cudaStream_t>(stream), 0, &ss, true);
    clear_deferred(ctx);  // the sums in the scratch belonged to this call
    return s;
}

lynx_status lynx_act_sparse_linear_host(lynx_ctx* ctx, const void* X_host, int64_t M, int64_t K, const void* W,
                                        int64_t N, int64_t ldw, const void* bias, lynx_comp_mode mode, void* Y_host,
                                        lynx_fuse_mode fuse, void* stream) {
    lynx_status s = check_common(ctx, M, K);
    if (s != LYNX_OK) return s;
    if (!X_host || !Y_host || N < 8) return LYNX_ERR_INVALID_ARG;
    const size_t x_bytes = align_up((size_t)M * K * 2, 1024), y_bytes = align_up((size_t)M * N * 2, 1024);
    {
        std::lock_guard<std::mutex> lock(ctx->mu);
        if ((s = ensure_scratch(ctx, scratch_layout(M, K).total)) != LYNX_OK) return s;
        if ((s = ensure_host_stage(ctx, x_bytes + y_bytes)) != LYNX_OK) return s;
    }
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    char* xd = static_cast<char*>(ctx->host_stage);
    char* yd = xd + x_bytes;
    // Token rows are independent (except under the whole-tensor scale), so the call is pipelined over
    // row chunks: the copy-in of chunk c + 1 and the copy-out of chunk c - 1 overlap the kernels of
    // chunk c on two copy streams (PCIe is full duplex); the result is the unchunked one bit for bit.
    int chunks = (M >= 2048 && mode != LYNX_COMP_TENSOR) ? 4 : 1;
    const int64_t rows_per = ((M + chunks - 1) / chunks + 255) / 256 * 256;
    chunks = (int)((M + rows_per - 1) / rows_per);
    if (chunks == 1) {
        if (cudaMemcpyAsync(xd, X_host, (size_t)M * K * 2, cudaMemcpyHostToDevice, st) != cudaSuccess)
            return LYNX_ERR_CUDA;
        s = lynx_act_sparse_linear(ctx, xd, M, K, K, W, N, ldw, bias, mode, nullptr, 0, yd, N, fuse, stream);
        if (s != LYNX_OK) return s;
        if (cudaMemcpyAsync(Y_host, yd, (size_t)M * N * 2, cudaMemcpyDeviceToHost, st) != cudaSuccess)
            return LYNX_ERR_CUDA;
        if (cudaStreamSynchronize(st) != cudaSuccess) return LYNX_ERR_CUDA;
        return check_device_error(ctx);
    }
    if (!ctx->h2d_stream) {
        std::lock_guard<std::mutex> lock(ctx->mu);
        bool ok = cudaStreamCreateWithFlags(&ctx->h2d_stream, cudaStreamNonBlocking) == cudaSuccess &&
                  cudaStreamCreateWithFlags(&ctx->d2h_stream, cudaStreamNonBlocking) == cudaSuccess &&
                  cudaEventCreateWithFlags(&ctx->ev_all, cudaEventDisableTiming) == cudaSuccess;
        for (int i = 0; i < 8 && ok; ++i)
            ok = cudaEventCreateWithFlags(&ctx->ev_h2d[i], cudaEventDisableTiming) == cudaSuccess &&
                 cudaEventCreateWithFlags(&ctx->ev_done[i], cudaEventDisableTiming) == cudaSuccess;
        if (!ok) return LYNX_ERR_CUDA;
    }
    // the copy streams start behind whatever the caller already queued on `stream`
    if (cudaEventRecord(ctx->ev_all, st) != cudaSuccess || cudaStreamWaitEvent(ctx->h2d_stream, ctx->ev_all, 0) != cudaSuccess)
        return LYNX_ERR_CUDA;
    const char* xh = static_cast<const char*>(X_host);
    char* yh = static_cast<char*>(Y_host);
    for (int c = 0; c < chunks; ++c) {
        const int64_t r0 = c * rows_per, rows = (r0 + rows_per <= M) ? rows_per : M - r0;
        if (cudaMemcpyAsync(xd + (size_t)r0 * K * 2, xh + (size_t)r0 * K * 2, (size_t)rows * K * 2,
                            cudaMemcpyHostToDevice, ctx->h2d_stream) != cudaSuccess ||
            cudaEventRecord(ctx->ev_h2d[c], ctx->h2d_stream) != cudaSuccess)
            return LYNX_ERR_CUDA;
    }
    for (int c = 0; c < chunks; ++c) {
        const int64_t r0 = c * rows_per, rows = (r0 + rows_per <= M) ? rows_per : M - r0;
        if (cudaStreamWaitEvent(st, ctx->ev_h2d[c], 0) != cudaSuccess) return LYNX_ERR_CUDA;
        s = lynx_act_sparse_linear(ctx, xd + (size_t)r0 * K * 2, rows, K, K, W, N, ldw, bias, mode, nullptr, 0,
                                   yd + (size_t)r0 * N * 2, N, fuse, stream);
        if (s != LYNX_OK) return s;
        if (cudaEventRecord(ctx->ev_done[c], st) != cudaSuccess ||
            cudaStreamWaitEvent(ctx->d2h_stream, ctx->ev_done[c], 0) != cudaSuccess ||
            cudaMemcpyAsync(yh + (size_t)r0 * N * 2, yd + (size_t)r0 * N * 2, (size_t)rows * N * 2,
                            cudaMemcpyDeviceToHost, ctx->d2h_stream) != cudaSuccess)
            return LYNX_ERR_CUDA;
    }
    if (cudaEventRecord(ctx->ev_all, ctx->d2h_stream) != cudaSuccess || cudaStreamWaitEvent(st, ctx->ev_all, 0) != cudaSuccess ||
        cudaStreamSynchronize(st) != cudaSuccess)
        return LYNX_ERR_CUDA;
    return check_device_error(ctx);
}

lynx_status lynx_reserve_lora(lynx_ctx* ctx, int64_t M, int64_t K, int64_t R) {
    lynx_status s = check_common(ctx, M, K);
    if (s != LYNX_OK) return s;
    if ((s = check_lora_rank(R)) != LYNX_OK) return s;
    std::lock_guard<std::mutex> lock(ctx->mu);
    return ensure_lora_ws(ctx, lora_ws_layout(ctx->num_sms, M, K, (int)R).total);
}

lynx_status lynx_lora_down(lynx_ctx* ctx, const void* X, int64_t M, int64_t K, int64_t ldx, const void* LB,
                           int64_t R, int64_t ldlb, const float* row_scale, void* T, int64_t ldt, void* stream) {
    lynx_status s = check_common(ctx, M, K);
    if (s != LYNX_OK) return s;
    if ((s = check_lora_rank(R)) != LYNX_OK) return s;
    if (!X || !LB || !T || row_scale == LYNX_ROW_SCALE_DEFERRED) return LYNX_ERR_INVALID_ARG;
    if (ldx < K || ldlb < K || ldt < R) return LYNX_ERR_INVALID_ARG;
    if ((size_t)((M + 127) / 128) * 4 > LORA_TICKET_BYTES) return LYNX_ERR_UNSUPPORTED_SHAPE;
    if (!aligned16(X) || !aligned16(LB) || !aligned16(T) || (ldx % 8) || (ldlb % 8) || (ldt % 8))
        return LYNX_ERR_ALIGNMENT;
    if ((s = check_device_error(ctx)) != LYNX_OK) return s;
    const LoraWsLayout L = lora_ws_layout(ctx->num_sms, M, K, (int)R);
    {
        std::lock_guard<std::mutex> lock(ctx->mu);
        if ((s = ensure_lora_ws(ctx, L.total)) != LYNX_OK) return s;
    }
    float* partial = reinterpret_cast<float*>(static_cast<char*>(ctx->lora_ws) + L.partial);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (R == 64) return launch_lora_down<LoraDownCfg<64>>(ctx, X, M, K, ldx, LB, ldlb, row_scale, T, ldt, partial, st);
    return launch_lora_down<LoraDownCfg<128>>(ctx, X, M, K, ldx, LB, ldlb, row_scale, T, ldt, partial, st);
}

// Prune / compress + row sums + T = (X L_B^T) / s in one launch (X read once).  The row sums stay
// in the context's scratch for the GEMM that follows (deferred row scale); *ss names them.
static lynx_status prune_lora_impl(lynx_ctx* ctx, const void* X, int64_t M, int64_t K, int64_t ldx, const void* LB,
                                   int64_t R, int64_t ldlb, void* values, void* meta, lynx_comp_mode mode, void* T,
                                   int64_t ldt, void* stream, ScaleSrc* ss) {
    lynx_status s = check_common(ctx, M, K);
    if (s != LYNX_OK) return s;
    if ((s = check_lora_rank(R)) != LYNX_OK) return s;
    if (!X || !LB || !values || !meta || !T) return LYNX_ERR_INVALID_ARG;
    if (mode != LYNX_COMP_NONE && mode != LYNX_COMP_ROW) return LYNX_ERR_INVALID_ARG;
    if (ldx < K || ldlb < K || ldt < R) return LYNX_ERR_INVALID_ARG;
    if (!aligned16(X) || !aligned16(LB) || !aligned16(T) || !aligned16(meta) || (ldx % 8) || (ldlb % 8) || (ldt % 8) ||
        (reinterpret_cast<uintptr_t>(values) & 31u))
        return LYNX_ERR_ALIGNMENT;
    const ScratchLayout L = scratch_layout(M, K);
    {
        std::lock_guard<std::mutex> lock(ctx->mu);
        if (ctx->scratch_bytes < L.prune_end && (s = ensure_scratch(ctx, L.total)) != LYNX_OK) return s;
    }
    if ((s = check_device_error(ctx)) != LYNX_OK) return s;
    float* spart = reinterpret_cast<float*>(static_cast<char*>(ctx->scratch) + L.partial);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    int splits = 0;
    const bool sums = mode == LYNX_COMP_ROW;
    if (R == 64)
        s = sums ? launch_prune_lora<PruneLoraCfg<64>, true>(ctx, X, M, K, ldx, LB, ldlb, values, meta, spart, T, ldt, st, &splits)
                 : launch_prune_lora<PruneLoraCfg<64>, false>(ctx, X, M, K, ldx, LB, ldlb, values, meta, nullptr, T, ldt, st, &splits);
    else
        s = sums ? launch_prune_lora<PruneLoraCfg<128>, true>(ctx, X, M, K, ldx, LB, ldlb, values, meta, spart, T, ldt, st, &splits)
                 : launch_prune_lora<PruneLoraCfg<128>, false>(ctx, X, M, K, ldx, LB, ldlb, values, meta, nullptr, T, ldt, st, &splits);
    if (s != LYNX_OK) return s;
    // the scratch's sums now belong to this call, in this kernel's split count
    ctx->deferred_partial = sums ? spart : nullptr;
    ctx->deferred_ks = sums ? splits : 0;
    ctx->deferred_M = M;
    ctx->deferred_K = K;
    if (ss) {
        ss->partial = ctx->deferred_partial;
        ss->ks = ctx->deferred_ks;
    }
    return LYNX_OK;
}

lynx_status lynx_prune_compress_lora(lynx_ctx* ctx, const void* X, int64_t M, int64_t K, int64_t ldx, const void* LB,
                                     int64_t R, int64_t ldlb, void* values, void* meta, lynx_comp_mode mode, void* T,
                                     int64_t ldt, void* stream) {
    return prune_lora_impl(ctx, X, M, K, ldx, LB, R, ldlb, values, meta, mode, T, ldt, stream, nullptr);
}

lynx_status lynx_sparse_linear_lora(lynx_ctx* ctx, const void* values, const void* meta, int64_t M, int64_t K,
                                    const void* W, int64_t N, int64_t ldw, const void* bias, const lynx_comp* comp,
                                    const void* T, int64_t ldt, const void* LA, int64_t R, int64_t ldla, void* Y,
                                    int64_t ldy, void* stream) {
    lynx_status s = check_common(ctx, M, K);
    if (s != LYNX_OK) return s;
    if ((s = check_lora_rank(R)) != LYNX_OK) return s;
    if (!values || !meta || !W || !Y || !T || !LA || N < 8) return LYNX_ERR_INVALID_ARG;
    if (N % 8 != 0) return LYNX_ERR_UNSUPPORTED_SHAPE;
    if (ldw < K || ldy < N || ldt < R || ldla < R) return LYNX_ERR_INVALID_ARG;
    if (!aligned16(values) || !aligned16(meta) || !aligned16(W) || !aligned16(Y) || !aligned16(T) || !aligned16(LA) ||
        (ldw % 8) || (ldy % 8) || (ldt % 8) || (ldla % 8))
        return LYNX_ERR_ALIGNMENT;
    if (bias && !aligned16(bias)) return LYNX_ERR_ALIGNMENT;
    if (comp && comp->residual) {
        if (comp->ldr < N) return LYNX_ERR_INVALID_ARG;
        if (!aligned16(comp->residual) || (comp->ldr % 8)) return LYNX_ERR_ALIGNMENT;
    }
    if ((s = check_device_error(ctx)) != LYNX_OK) return s;
    LoraArgs lora{T, ldt, LA, ldla, (int)R};
    if (comp && comp->row_scale == LYNX_ROW_SCALE_DEFERRED) {
        // the sums lynx_prune_compress_lora left on the context (T was divided by the same scale)
        if (!ctx->deferred_partial || ctx->deferred_M != M || ctx->deferred_K != K) return LYNX_ERR_INVALID_ARG;
        ScaleSrc ss;
        ss.partial = ctx->deferred_partial;
        ss.ks = ctx->deferred_ks;
        lynx_comp c2 = *comp;
        c2.row_scale = nullptr;
        return launch_gemm(ctx, values, meta, M, K, W, N, ldw, bias, &c2, &lora, Y, ldy,
                           static_cast<cudaStream_t>(stream), 0, &ss);
    }
    return launch_gemm(ctx, values, meta, M, K, W, N, ldw, bias, comp, &lora, Y, ldy,
                       static_cast<cudaStream_t>(stream));
}

static lynx_status act_sparse_linear_lora_impl(lynx_ctx* ctx, const void* X, int64_t M, int64_t K, int64_t ldx,
                                               const void* W, int64_t N, int64_t ldw, const void* bias, const void* LA,
                                               int64_t ldla, const void* LB, int64_t ldlb, int64_t R, lynx_comp_mode mode,
                                               const void* residual, int64_t ldr, void* Y, int64_t ldy, void* stream) {
    lynx_status s = check_common(ctx, M, K);
    if (s != LYNX_OK) return s;
    if ((s = check_lora_rank(R)) != LYNX_OK) return s;
    if (N < 8 || !LA || !LB) return LYNX_ERR_INVALID_ARG;
    // every argument is checked before the first launch
    if (!X || !W || !Y) return LYNX_ERR_INVALID_ARG;
    if (N % 8 != 0) return LYNX_ERR_UNSUPPORTED_SHAPE;
    if (ldx < K || ldw < K || ldy < N || ldla < R || ldlb < K || (residual && ldr < N)) return LYNX_ERR_INVALID_ARG;
    if (!aligned16(X) || !aligned16(W) || !aligned16(Y) || !aligned16(LA) || !aligned16(LB) || (ldx % 8) ||
        (ldw % 8) || (ldy % 8) || (ldla % 8) || (ldlb % 8) || (bias && !aligned16(bias)) ||
        (residual && (!aligned16(residual) || (ldr % 8))))
        return LYNX_ERR_ALIGNMENT;
    ScratchLayout L = scratch_layout(M, K);
    const LoraWsLayout LL = lora_ws_layout(ctx->num_sms, M, K, (int)R);
    {
        std::lock_guard<std::mutex> lock(ctx->mu);
        if ((s = ensure_scratch(ctx, L.total)) != LYNX_OK) return s;
        if ((s = ensure_lora_ws(ctx, LL.total)) != LYNX_OK) return s;
    }
    char* base = static_cast<char*>(ctx->scratch);
    void* values = base + L.values;
    void* meta = base + L.meta;
    float* scale = sums_needed(mode) ? reinterpret_cast<float*>(base + L.scale) : nullptr;
    void* T = static_cast<char*>(ctx->lora_ws) + LL.T;
    const int cfg = pick_gemm_cfg(ctx, M, N, K, (int)(R / 64));
    if (ctx->lora_fuse == 2 && (mode == LYNX_COMP_NONE || (mode == LYNX_COMP_ROW && ctx->defer_scale != 0))) {
        // two launches, X read once: prune / compress + row sums + T in the first, the GEMM (which
        // finishes the row scale in its epilogue and adds T L_A^T in its accumulator) in the second
        ScaleSrc ss2;
        if ((s = prune_lora_impl(ctx, X, M, K, ldx, LB, R, ldlb, values, meta, mode, T, R, stream, &ss2)) != LYNX_OK)
            return s;
        lynx_comp comp2;
        comp2.row_scale = nullptr;
        comp2.residual = residual;
        comp2.ldr = ldr;
        LoraArgs lora2{T, R, LA, ldla, (int)R};
        return launch_gemm(ctx, values, meta, M, K, W, N, ldw, bias, &comp2, &lora2, Y, ldy,
                           static_cast<cudaStream_t>(stream), 0, &ss2, true);
    }
    const bool groups_fit = (size_t)((M + 255) / 256) * 8 * 4 <= L0_WORDS_BYTES;
    const bool fused = ctx->lora_fuse && R == 64 && cfg_supports_l0(cfg) && !ctx->streamk && groups_fit;
    // (the separate down-projection kernel reads row_scale, so the scale is only deferred when the
    // GEMM launch is its one consumer)
    ScaleSrc ss;
    s = prune_impl(ctx, X, M, K, ldx, values, meta, scale, mode, stream, fused && ctx->defer_scale != 0, &ss);
    if (s != LYNX_OK) return s;
    lynx_comp comp;
    comp.row_scale = ss.partial ? nullptr : scale;
    comp.residual = residual;
    comp.ldr = ldr;
    if (fused) {
        // two launches: the GEMM kernel computes T = (X L_B^T) / s itself before its first tile
        char* ws = static_cast<char*>(ctx->lora_ws);
        LoraArgs lora{T, R, LA, ldla, (int)R};
        lora.X = X;
        lora.ldx = ldx;
        lora.LB = LB;
        lora.ldlb = ldlb;
        lora.l0_partial = reinterpret_cast<float*>(ws + LL.partial);
        lora.l0_tickets = ctx->tickets + (PRUNE_TICKET_BYTES + LORA_TICKET_BYTES) / 4;
        lora.l0_ready = lora.l0_tickets + L0_WORDS_BYTES / 4;
        return launch_gemm(ctx, values, meta, M, K, W, N, ldw, bias, &comp, &lora, Y, ldy,
                           static_cast<cudaStream_t>(stream), cfg, &ss);
    }
    s = lynx_lora_down(ctx, X, M, K, ldx, LB, R, ldlb, scale, T, R, stream);
    if (s != LYNX_OK) return s;
    return lynx_sparse_linear_lora(ctx, values, meta, M, K, W, N, ldw, bias, &comp, T, R, LA, R, ldla, Y, ldy, stream);
}

lynx_status lynx_act_sparse_linear_lora(lynx_ctx* ctx, const void* X, int64_t M, int64_t K, int64_t ldx,
                                        const void* W, int64_t N, int64_t ldw, const void* bias, const void* LA,
                                        int64_t ldla, const void* LB, int64_t ldlb, int64_t R, lynx_comp_mode mode,
                                        const void* residual, int64_t ldr, void* Y, int64_t ldy, void* stream) {
    if (ctx) clear_deferred(ctx);  // this call writes the scratch
    const lynx_status s = act_sparse_linear_lora_impl(ctx, X, M, K, ldx, W, N, ldw, bias, LA, ldla, LB, ldlb, R, mode,
                                                      residual, ldr, Y, ldy, stream);
    if (ctx) clear_deferred(ctx);  // and the sums it left there belonged to it
    return s;
}

// ------------------------------------------------------------------------- FP8 composition ------

// Warps that share a row in the FP8 ring kernel: the fewest for which every group still gets a
// slot of its own (all 16 consumer warps stay busy; longer rows are split over more warps).
static int fp8_ring_group_width(int slots) {
    int gw = 1;
    while (gw < 8 && FP8_RING_CW / gw > slots) gw *= 2;
    return gw;
}

static lynx_status check_fp8_shape(lynx_ctx* ctx, int64_t M, int64_t K) {
    lynx_status s = check_common(ctx, M, K);
    if (s != LYNX_OK) return s;
    if (K % 256 != 0) return LYNX_ERR_UNSUPPORTED_SHAPE;
    return LYNX_OK;
}

lynx_status lynx_quantize_weights_fp8(lynx_ctx* ctx, const void* W, int64_t N, int64_t K, int64_t ldw,
                                      int per_channel, void* Wq, float* wscale, void* stream) {
    if (!ctx || !W || !Wq || !wscale || N < 1 || K < 2) return LYNX_ERR_INVALID_ARG;
    if (K % 2 != 0 || ldw < K) return LYNX_ERR_INVALID_ARG;
    if (reinterpret_cast<uintptr_t>(Wq) & 1u) return LYNX_ERR_ALIGNMENT;
    quantize_weights_fp8_kernel<<<(unsigned)N, 256, 0, static_cast<cudaStream_t>(stream)>>>(
        static_cast<const uint16_t*>(W), N, K, ldw, per_channel ? 1 : 0, static_cast<uint8_t*>(Wq), wscale);
    ctx->launches++;
    return cuda_ok(cudaGetLastError());
}

lynx_status lynx_prune_compress_fp8(lynx_ctx* ctx, const void* X, int64_t M, int64_t K, int64_t ldx,
                                    const float* row_amax, void* values_q, void* meta, float* row_scale,
                                    lynx_comp_mode mode, void* stream) {
    lynx_status s = check_fp8_shape(ctx, M, K);
    if (s != LYNX_OK) return s;
    if (!X || !values_q || !meta || !row_scale) return LYNX_ERR_INVALID_ARG;
    if (mode != LYNX_COMP_NONE && mode != LYNX_COMP_ROW) return LYNX_ERR_INVALID_ARG;
    if (ldx < K) return LYNX_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(X) & 31u) || !aligned16(values_q) || !aligned16(meta) || (ldx % 16) != 0)
        return LYNX_ERR_ALIGNMENT;
    if ((s = check_device_error(ctx)) != LYNX_OK) return s;
    cudaLaunchConfig_t pc = {};
    pc.gridDim = dim3((unsigned)(((M + 127) / 128) * 8));
    pc.blockDim = dim3(FP8_PRUNE_WARPS * 32);
    pc.stream = static_cast<cudaStream_t>(stream);
    cudaLaunchAttribute pa[1];
    pa[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    pa[0].val.programmaticStreamSerializationAllowed = ctx->pdl ? 1 : 0;
    pc.attrs = pa;
    pc.numAttrs = 1;
    const uint16_t* Xp = static_cast<const uint16_t*>(X);
    uint8_t* vp = static_cast<uint8_t*>(values_q);
    uint8_t* mp = static_cast<uint8_t*>(meta);
    cudaError_t e;
    // The persistent ring kernel reads X once (also when the maxima have to be found in the data).
    // It wants at least two rows in shared memory and rows long enough to occupy a warp.
    int slots = (int)((FP8_RING_SMEM_MAX - FP8_RING_HEADER) / (K * 2));
    if (slots > FP8_RING_MAX_SLOTS) slots = FP8_RING_MAX_SLOTS;
    if (ctx->fp8_ring && slots >= 2 && K >= 2048) {
        // gw warps share a row; ng = CW / gw groups, each with at least one slot of its own
        int gw = fp8_ring_group_width(slots);
        if (ctx->fp8_ring_forced && (ctx->fp8_ring == 1 || ctx->fp8_ring == 2 || ctx->fp8_ring == 4 || ctx->fp8_ring == 8))
            gw = ctx->fp8_ring;
        int ng = FP8_RING_CW / gw;
        if (ng > slots) ng = slots;
        const int smem = FP8_RING_HEADER + slots * (int)(K * 2);
        const bool sums = mode == LYNX_COMP_ROW, given = row_amax != nullptr;
        using RingKernel = void (*)(const uint16_t*, int64_t, int64_t, int64_t, const float*, uint8_t*, uint8_t*,
                                    float*, int, int, uint32_t*);
#define LYNX_RING4(S, G) prune_compress_fp8_ring_kernel<S, G, 1>, prune_compress_fp8_ring_kernel<S, G, 2>, \
                         prune_compress_fp8_ring_kernel<S, G, 4>, prune_compress_fp8_ring_kernel<S, G, 8>
        static const RingKernel kerns[16] = {LYNX_RING4(false, false), LYNX_RING4(true, false),
                                             LYNX_RING4(false, true), LYNX_RING4(true, true)};
#undef LYNX_RING4
        static bool attr_set[16][MAX_CTX_DEVICES] = {};
        const int which = (sums ? 4 : 0) + (given ? 8 : 0) + (gw == 1 ? 0 : gw == 2 ? 1 : gw == 4 ? 2 : 3);
        if (lynx_status as = allow_dynamic_smem(kerns[which], FP8_RING_SMEM_MAX, ctx->device, attr_set[which]);
            as != LYNX_OK)
            return as;
        pc.gridDim = dim3((unsigned)(M < ctx->num_sms ? M : ctx->num_sms));
        pc.blockDim = dim3(FP8_RING_THREADS);
        pc.dynamicSmemBytes = (size_t)smem;
        e = cudaLaunchKernelEx(&pc, kerns[which], Xp, M, K, ldx, row_amax, vp, mp, row_scale, slots, ng,
                               ctx->err_dev);
        if (e != cudaSuccess) return LYNX_ERR_CUDA;
        ctx->launches++;
        return LYNX_OK;
    }
    if (row_amax)
        e = (mode == LYNX_COMP_ROW)
                ? cudaLaunchKernelEx(&pc, prune_compress_fp8_kernel<true, true>, Xp, M, K, ldx, row_amax, vp, mp, row_scale)
                : cudaLaunchKernelEx(&pc, prune_compress_fp8_kernel<false, true>, Xp, M, K, ldx, row_amax, vp, mp, row_scale);
    else
        e = (mode == LYNX_COMP_ROW)
                ? cudaLaunchKernelEx(&pc, prune_compress_fp8_kernel<true, false>, Xp, M, K, ldx, row_amax, vp, mp, row_scale)
                : cudaLaunchKernelEx(&pc, prune_compress_fp8_kernel<false, false>, Xp, M, K, ldx, row_amax, vp, mp, row_scale);
    if (e != cudaSuccess) return LYNX_ERR_CUDA;
    ctx->launches++;
    return LYNX_OK;
}

lynx_status lynx_sparse_linear_fp8(lynx_ctx* ctx, const void* values_q, const void* meta, int64_t M, int64_t K,
                                   const void* Wq, int64_t N, int64_t ldwq, const float* wscale, const void* bias,
                                   const lynx_comp* comp, void* Y, int64_t ldy, void* stream) {
    lynx_status s = check_fp8_shape(ctx, M, K);
    if (s != LYNX_OK) return s;
    if (!values_q || !meta || !Wq || !Y || N < 8) return LYNX_ERR_INVALID_ARG;
    if (comp && comp->row_scale == LYNX_ROW_SCALE_DEFERRED) return LYNX_ERR_INVALID_ARG;
    if (N % 8 != 0) return LYNX_ERR_UNSUPPORTED_SHAPE;
    if (ldwq < K || ldy < N) return LYNX_ERR_INVALID_ARG;
    if (!aligned16(values_q) || !aligned16(meta) || !aligned16(Wq) || !aligned16(Y) || (ldwq % 16) || (ldy % 8))
        return LYNX_ERR_ALIGNMENT;
    if ((bias && !aligned16(bias)) || (wscale && !aligned16(wscale))) return LYNX_ERR_ALIGNMENT;
    if (comp && comp->residual) {
        if (comp->ldr < N) return LYNX_ERR_INVALID_ARG;
        if (!aligned16(comp->residual) || (comp->ldr % 8)) return LYNX_ERR_ALIGNMENT;
    }
    if ((s = check_device_error(ctx)) != LYNX_OK) return s;
    return launch_gemm_fp8(ctx, values_q, meta, M, K, Wq, N, ldwq, wscale, bias, comp, Y, ldy,
                           static_cast<cudaStream_t>(stream));
}

lynx_status lynx_act_sparse_linear_fp8(lynx_ctx* ctx, const void* X, int64_t M, int64_t K, int64_t ldx,
                                       const float* row_amax, const void* Wq, int64_t N, int64_t ldwq,
                                       const float* wscale,
                                       const void* bias, lynx_comp_mode mode, const void* residual, int64_t ldr,
                                       void* Y, int64_t ldy, void* stream) {
    lynx_status s = check_fp8_shape(ctx, M, K);
    if (s != LYNX_OK) return s;
    // every argument is checked before the first launch
    if (!X || !Wq || !Y || N < 8) return LYNX_ERR_INVALID_ARG;
    if (mode != LYNX_COMP_NONE && mode != LYNX_COMP_ROW) return LYNX_ERR_INVALID_ARG;
    if (N % 8 != 0) return LYNX_ERR_UNSUPPORTED_SHAPE;
    if (ldx < K || ldwq < K || ldy < N || (residual && ldr < N)) return LYNX_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(X) & 31u) || (ldx % 16) || !aligned16(Wq) || !aligned16(Y) || (ldwq % 16) ||
        (ldy % 8) || (bias && !aligned16(bias)) || (wscale && !aligned16(wscale)) ||
        (residual && (!aligned16(residual) || (ldr % 8))))
        return LYNX_ERR_ALIGNMENT;
    ScratchLayout L = scratch_layout(M, K);
    {
        std::lock_guard<std::mutex> lock(ctx->mu);
        clear_deferred(ctx);  // this call writes the scratch
        if ((s = ensure_scratch(ctx, L.total)) != LYNX_OK) return s;
    }
    char* base = static_cast<char*>(ctx->scratch);
    void* values_q = base + L.values;  // (sized for bf16 values: twice what the codes need)
    void* meta = base + L.meta;
    float* scale = reinterpret_cast<float*>(base + L.scale);
    s = lynx_prune_compress_fp8(ctx, X, M, K, ldx, row_amax, values_q, meta, scale, mode, stream);
    if (s != LYNX_OK) return s;
    lynx_comp comp;
    comp.row_scale = scale;
    comp.residual = residual;
    comp.ldr = ldr;
    return lynx_sparse_linear_fp8(ctx, values_q, meta, M, K, Wq, N, ldwq, wscale, bias, &comp, Y, ldy, stream);
}

lynx_status lynx_meta_to_canonical(lynx_ctx* ctx, const void* meta, int64_t M, int64_t K, void* meta_canon,
                                   void* stream) {
    lynx_status s = check_common(ctx, M, K);
    if (s != LYNX_OK) return s;
    if (!meta || !meta_canon) return LYNX_ERR_INVALID_ARG;
    const int64_t n = M * (K / 16);
    meta_to_canonical_kernel<<<(unsigned)((n + 255) / 256), 256, 0, static_cast<cudaStream_t>(stream)>>>(
        static_cast<const uint8_t*>(meta), M, K, static_cast<uint16_t*>(meta_canon));
    ctx->launches++;
    return cuda_ok(cudaGetLastError());
}

lynx_status lynx_decompress(lynx_ctx* ctx, const void* values, const void* meta, int64_t M, int64_t K,
                            void* Xmasked, void* stream) {
    lynx_status s = check_common(ctx, M, K);
    if (s != LYNX_OK) return s;
    if (!values || !meta || !Xmasked) return LYNX_ERR_INVALID_ARG;
    const int64_t n = M * (K / 4);
    decompress_kernel<<<(unsigned)((n + 255) / 256), 256, 0, static_cast<cudaStream_t>(stream)>>>(
        static_cast<const uint16_t*>(values), static_cast<const uint8_t*>(meta), M, K, static_cast<uint16_t*>(Xmasked));
    ctx->launches++;
    return cuda_ok(cudaGetLastError());
}

// Self-test of the bounded-wait protocol: one CTA waits, with the given limit, on an mbarrier
// nobody ever arrives at; the wait gives up, raises the CTA's abort word and the context's error
// word exactly as a kernel of the path would, and the kernel returns normally.
lynx_status lynx_selftest_wait_timeout(lynx_ctx* ctx, int64_t limit_us, void* stream) {
    if (!ctx || limit_us < 1 || limit_us > 100000) return LYNX_ERR_INVALID_ARG;
    wait_timeout_probe_kernel<<<1, 32, 0, static_cast<cudaStream_t>(stream)>>>(ctx->err_dev, (uint64_t)limit_us * 1000ull);
    ctx->launches++;
    return cuda_ok(cudaGetLastError());
}

// Host-only inspection of the two-row-tile GEMM's plan and schedule (no device is touched).
int lynx_gemm_plan(int num_sms, int64_t M, int64_t N, int64_t K, int lora_steps, int* doubles, int* clusters) {
    if (num_sms < 2 || M < 1 || N < 8 || K < 128) return -1;
    const Rt2Plan plan = rt2_plan(num_sms, M, N, K, lora_steps, -1);
    if (doubles) *doubles = plan.doubles;
    if (clusters) *clusters = plan.clusters;
    return (M > 256 && plan.t_us < gemm_model_time(num_sms, M, N, K, lora_steps)) ? 1 : 0;
}

int lynx_gemm_schedule_items(int tiles_m, int tiles_n, int clusters, int doubles, int cluster, int* items, int capacity) {
    if (tiles_m < 1 || tiles_n < 1 || clusters < 1 || cluster < 0 || cluster >= clusters) return -1;
    PairSchedule sc;
    sc.init(tiles_m, tiles_n, clusters, doubles, 8);
    const int n = sc.num_items(cluster);
    for (int i = 0; i < n && i < capacity; ++i) {
        int tm0, tn, rows, ordinal;
        sc.item(cluster, i, tm0, tn, rows, ordinal);
        items[4 * i + 0] = tm0;
        items[4 * i + 1] = tn;
        items[4 * i + 2] = rows;
        items[4 * i + 3] = ordinal;
    }
    return n;
}

}  // extern "C"

// ================================================= entry point that allocates nothing ===========
// Scratch for lynx_prune_compress_static: part of the library image, LYNX_STATIC_SCRATCH_BYTES
// per GPU.  In host code this name is only a handle; the device address comes from
// cudaGetSymbolAddress, looked up once per device (with that device current) and cached.
static __device__ __align__(256) unsigned char g_static_scratch[LYNX_STATIC_SCRATCH_BYTES];

namespace {
constexpr int MAX_DEVICES = 64;
std::mutex g_static_mu;
void* g_static_ptr[MAX_DEVICES] = {};
int g_static_sms[MAX_DEVICES] = {};

// device address of g_static_scratch on the current device (set-up on first use per device)
lynx_status static_scratch_for_current_device(void** ptr, int* num_sms) {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= MAX_DEVICES) return LYNX_ERR_CUDA;
    std::lock_guard<std::mutex> lock(g_static_mu);
    if (!g_static_ptr[dev]) {
        void* p = nullptr;
        if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || !p) return LYNX_ERR_CUDA;
        int major = 0, sms = 0;
        if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess ||
            cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
            return LYNX_ERR_CUDA;
        if (major != 10) return LYNX_ERR_UNSUPPORTED_ARCH;
        g_static_sms[dev] = sms;
        g_static_ptr[dev] = p;
    }
    *ptr = g_static_ptr[dev];
    *num_sms = g_static_sms[dev];
    return LYNX_OK;
}
}  // namespace

extern "C" lynx_status lynx_prune_compress_static(const void* X, int64_t M, int64_t K, int64_t ldx, void* values,
                                                  void* meta, float* row_scale, lynx_comp_mode mode, void* stream) {
    if (M < 1 || K < 128) return LYNX_ERR_INVALID_ARG;
    if (K % 128 != 0 || M > (1ll << 30) || K > (1ll << 30)) return LYNX_ERR_UNSUPPORTED_SHAPE;
    if (!X || !values || !meta) return LYNX_ERR_INVALID_ARG;
    if (mode != LYNX_COMP_NONE && mode != LYNX_COMP_ROW && mode != LYNX_COMP_TENSOR && mode != LYNX_COMP_GROUP)
        return LYNX_ERR_INVALID_ARG;
    if (sums_needed(mode) && !row_scale) return LYNX_ERR_INVALID_ARG;
    if (ldx < K) return LYNX_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(X) & 31u) || (reinterpret_cast<uintptr_t>(values) & 31u) || !aligned16(meta) ||
        (ldx % 16) != 0)
        return LYNX_ERR_ALIGNMENT;
    void* scratch = nullptr;
    int num_sms = 0;
    lynx_status s = static_scratch_for_current_device(&scratch, &num_sms);
    if (s != LYNX_OK) return s;
    // the same work decomposition as lynx_prune_compress (one helper: the sums' bits depend on it)
    const PrunePlan P = prune_plan(num_sms, M, K, 0);
    const int64_t rb16 = P.rb16;
    const int tpu = P.tpu, KS = P.KS;
    // static scratch: [tickets: 64 KB][partial sums: rb16 * KS * 32 floats][per-row sums: 2 * M floats]
    // (a __device__ array starts zeroed and every launch leaves its tickets at zero again)
    constexpr size_t STATIC_TICKET_BYTES = 64u << 10;
    if ((size_t)rb16 * 4 > STATIC_TICKET_BYTES) return LYNX_ERR_WORKSPACE;
    const size_t partial_bytes = (sums_needed(mode) && KS > 1) ? (size_t)rb16 * KS * 32 * 4 : 0;
    const size_t partial_padded = (partial_bytes + 255) / 256 * 256;
    const size_t sums_bytes = (mode == LYNX_COMP_TENSOR) ? (size_t)M * 8 : 0;
    if (STATIC_TICKET_BYTES + partial_padded + sums_bytes > (size_t)LYNX_STATIC_SCRATCH_BYTES) return LYNX_ERR_WORKSPACE;
    uint32_t* tickets = reinterpret_cast<uint32_t*>(scratch);
    float* partial = reinterpret_cast<float*>(static_cast<unsigned char*>(scratch) + STATIC_TICKET_BYTES);
    float* sums = reinterpret_cast<float*>(static_cast<unsigned char*>(scratch) + STATIC_TICKET_BYTES + partial_padded);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const int ctas_per_rb = P.ctas_per_rb;
    const unsigned grid = P.grid;
    if (mode == LYNX_COMP_GROUP)
        prune_compress_kernel<false, true><<<grid, PRUNE_CTA_WARPS * 32, 0, st>>>(
            static_cast<const uint16_t*>(X), M, K, ldx, static_cast<uint16_t*>(values), static_cast<uint8_t*>(meta),
            row_scale, nullptr, nullptr, nullptr, 0, tpu, KS, ctas_per_rb, 0);
    else if (mode == LYNX_COMP_NONE)
        prune_compress_kernel<false><<<grid, PRUNE_CTA_WARPS * 32, 0, st>>>(
            static_cast<const uint16_t*>(X), M, K, ldx, static_cast<uint16_t*>(values), static_cast<uint8_t*>(meta),
            row_scale, nullptr, nullptr, nullptr, 0, tpu, KS, ctas_per_rb, 0);
    else
        prune_compress_kernel<true><<<grid, PRUNE_CTA_WARPS * 32, 0, st>>>(
            static_cast<const uint16_t*>(X), M, K, ldx, static_cast<uint16_t*>(values), static_cast<uint8_t*>(meta),
            row_scale, sums, partial, tickets, (int)mode, tpu, KS, ctas_per_rb, 0);
    if (mode == LYNX_COMP_TENSOR) tensor_scale_kernel<<<1, 1024, 0, st>>>(sums, M, row_scale);
    return cuda_ok(cudaGetLastError());
}

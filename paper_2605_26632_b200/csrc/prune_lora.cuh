// Prune / compress and the down projection of the low-rank branch in one pass over X
// (Algorithm 1 lines 3-5: X~ = TopK(X), the norm-compensation sums, and the first factor of
// Y_r = X (L_A L_B)^T, which reads the DENSE X):
//     values, metadata, row sums   as prune_compress_kernel leaves them in its deferred form
//     T[m, r] = bf16( (sum_k X[m,k] L_B[r,k]) / s_m )
// Both consumers want every element of X exactly once, so X crosses HBM once instead of twice.
//
// One CTA per (128-row block, K split); the splits of a row block form a thread-block cluster
// (1 to 8 CTAs).  Warp 0: TMA producer -- a stage is 128 rows x 128 K of X
// (two 128-byte-swizzled boxes of 64 elements) plus the matching R x 128 slice of L_B.  Warp 1
// issues eight dense tcgen05.mma (K = 16) per stage into a 128 x R fp32 accumulator in tensor
// memory.  Warps 6..13 each read one 16 x 128 tile of the stage out of shared memory (undoing the
// swizzle: 16-byte chunk c of row r sits at chunk c ^ (r % 8)) with the lane layout of the
// stand-alone prune kernel, and run the same selection / compression / store code.  A stage is
// free again when the MMAs have retired and all eight tiles are in registers.  Warps 2..5 drain
// the accumulator into the CTA's own shared memory at the end (the L_B half of the ring is free
// by then); after a cluster barrier every CTA finishes 128 / splits rows of T: it reads those rows
// of every split's partial through distributed shared memory, adds them in split order (the
// result does not depend on timing), divides by the row scale -- summed from all splits' row sums
// exactly as the GEMM epilogue will sum them -- and writes T.  No global round trip, no ticket.
#pragma once

#include "lora_down.cuh"
#include "prune_compress.cuh"

namespace lynx {

struct PruneLoraParams {
    int64_t M, K;
    int splits;         // K splits per row block = CTAs per cluster, 1..8
    int kb_per_split;   // 128-element K blocks per split (the last split may get fewer)
    uint16_t* values;   // [M x K/2] bf16
    uint8_t* meta;      // tensor-core order, 128 x 128 blocks of 2048 bytes
    float* scale_partial;  // [row blocks of 16][splits][16][2] fp32 row sums (SUMS) or nullptr
    uint16_t* T;           // [M x R] bf16, leading dimension ldt
    int64_t ldt;
    uint32_t* dev_error;
};

template <int R_>
struct PruneLoraCfg {
    static constexpr int R = R_;
    static constexpr int BM = 128, BK = 128;
    static constexpr int STAGES = (R == 64) ? 4 : 3;
    static constexpr int X_BOX_BYTES = BM * 128;      // 128 rows x 64 elements: 16 KB
    static constexpr int X_BYTES = 2 * X_BOX_BYTES;
    static constexpr int B_BOX_BYTES = R * 128;       // R rows x 64 elements
    static constexpr int B_BYTES = 2 * B_BOX_BYTES;
    static constexpr int STAGE_BYTES = X_BYTES + B_BYTES;
    static constexpr int PRUNERS = 8;                 // warps, one 16 x 128 tile each per stage
    static constexpr int THREADS = 64 + 128 + 32 * PRUNERS;
    static constexpr int TAIL_THREADS = 128 + 32 * PRUNERS;  // drain + prune warps meet once at the end
    static constexpr int SMEM_BYTES = 1024 + STAGES * STAGE_BYTES + 1024;
    static constexpr int TMEM_COLS = R;
    static constexpr int PARTIAL_BYTES = BM * R * 4;  // the drained accumulator, kept in the L_B ring
    static_assert(PARTIAL_BYTES <= STAGES * B_BYTES, "the partial fits where the L_B stages were");
    static_assert(R == 64 || R == 128, "rank");
    static_assert(SMEM_BYTES <= 227 * 1024, "shared memory budget");
};

template <class Cfg, bool SUMS>
__global__ void __launch_bounds__(Cfg::THREADS, 1)
prune_lora_kernel(const __grid_constant__ CUtensorMap tmap_x, const __grid_constant__ CUtensorMap tmap_lb,
                  const PruneLoraParams p) {
    constexpr int STAGES = Cfg::STAGES, R = Cfg::R;
    extern __shared__ uint8_t smem_raw[];
    __shared__ uint32_t lut[4 * 16];
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* smem_gen = smem_raw + (smem_base - smem_u32(smem_raw));
    const uint32_t sX = smem_base;
    const uint32_t sB = sX + STAGES * Cfg::X_BYTES;
    const uint32_t sBar = sB + STAGES * Cfg::B_BYTES;
    const uint32_t bar_full = sBar, bar_empty = sBar + 8 * STAGES, bar_done = sBar + 16 * STAGES;
    uint8_t* tail = smem_gen + (sBar - smem_base);
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(tail + 128);
    volatile uint32_t* cta_abort = tmem_slot + 1;
    float* s_scale = reinterpret_cast<float*>(tail + 256);  // [128] row scales of the finishing CTA

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int tiles_m = (int)((p.M + Cfg::BM - 1) / Cfg::BM);
    const int split = (int)cluster_ctarank(), tm = blockIdx.x / p.splits;  // cluster = the splits of a row block
    (void)tiles_m;
    const int kblocks = (int)(p.K / Cfg::BK);
    const int kb0 = split * p.kb_per_split;
    const int kb1 = (kb0 + p.kb_per_split < kblocks) ? kb0 + p.kb_per_split : kblocks;

    if (threadIdx.x < 64) lut[threadIdx.x] = prune_lut_entry(threadIdx.x & 15, threadIdx.x >> 4);
    if (threadIdx.x == 64) {
        *cta_abort = 0;
        for (int s = 0; s < STAGES; ++s) {
            mbar_init(bar_full + 8 * s, 1);
            mbar_init(bar_empty + 8 * s, 1 + Cfg::PRUNERS);  // the MMAs' commit + one arrive per prune warp
        }
        mbar_init(bar_done, 1);
        fence_mbar_init();
        prefetch_tmap(&tmap_x);
        prefetch_tmap(&tmap_lb);
    }
    if (warp == 1) {
        tmem_alloc<1>(smem_u32(tmem_slot), Cfg::TMEM_COLS);
        tmem_relinquish<1>();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    griddep_wait();  // X comes from the kernels before this one

    if (warp == 0) {
        // ------------------------------------------------------------------ producer ----------
        if (lane == 0) {
            uint32_t stage = 0, phase = 0, issued = 0;
            bool ok = true;
            for (int kb = kb0; kb < kb1; ++kb) {
                if (!mbar_wait(bar_empty + 8 * stage, phase ^ 1, cta_abort, p.dev_error)) {
                    ok = false;
                    break;
                }
                const uint32_t bar = bar_full + 8 * stage;
                const uint32_t x_dst = sX + stage * Cfg::X_BYTES, b_dst = sB + stage * Cfg::B_BYTES;
                mbar_arrive_expect_tx(bar, Cfg::STAGE_BYTES);
                tma_load_2d(x_dst, &tmap_x, kb * Cfg::BK, tm * Cfg::BM, bar);
                tma_load_2d(x_dst + Cfg::X_BOX_BYTES, &tmap_x, kb * Cfg::BK + 64, tm * Cfg::BM, bar);
                tma_load_2d(b_dst, &tmap_lb, kb * Cfg::BK, 0, bar);
                tma_load_2d(b_dst + Cfg::B_BOX_BYTES, &tmap_lb, kb * Cfg::BK + 64, 0, bar);
                ++issued;
                if (++stage == STAGES) { stage = 0; phase ^= 1; }
            }
            if (!ok && issued) bounded_delay_ns(200000);  // let the copies in flight land before teardown
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer --------
        if (lane == 0) {
            constexpr uint32_t idesc = make_idesc_bf16(Cfg::BM, R);
            const uint64_t d0 = make_desc_sw128(sX);
            const uint32_t desc_hi = (uint32_t)(d0 >> 32);
            const uint32_t a_lo0 = (uint32_t)d0, b_lo0 = (uint32_t)make_desc_sw128(sB);
            uint32_t stage = 0, phase = 0, accumulate = 0;
            bool ok = true;
            for (int kb = kb0; kb < kb1; ++kb) {
                if (!mbar_wait(bar_full + 8 * stage, phase, cta_abort, p.dev_error)) {
                    ok = false;
                    break;
                }
                tc_fence_after();
#pragma unroll
                for (int box = 0; box < 2; ++box) {
                    const uint32_t a_lo = a_lo0 + stage * (Cfg::X_BYTES >> 4) + box * (Cfg::X_BOX_BYTES >> 4);
                    const uint32_t b_lo = b_lo0 + stage * (Cfg::B_BYTES >> 4) + box * (Cfg::B_BOX_BYTES >> 4);
                    // four K steps of 16 elements = 32 bytes inside the 128-byte swizzle atom
                    mma_bf16_lh<1>(tmem_base, a_lo, b_lo, desc_hi, idesc, accumulate);
                    mma_bf16_lh<1>(tmem_base, a_lo + 2, b_lo + 2, desc_hi, idesc, 1u);
                    mma_bf16_lh<1>(tmem_base, a_lo + 4, b_lo + 4, desc_hi, idesc, 1u);
                    mma_bf16_lh<1>(tmem_base, a_lo + 6, b_lo + 6, desc_hi, idesc, 1u);
                    accumulate = 1u;
                }
                tc_commit(bar_empty + 8 * stage);
                if (++stage == STAGES) { stage = 0; phase ^= 1; }
            }
            if (ok) tc_commit(bar_done);
        }
    } else if (warp >= 6) {
        // ------------------------------------------------------------------ prune warps -------
        const int pw = warp - 6, r = lane >> 2, q = lane & 3;
        const int rowA_in = 16 * pw + r;                      // row inside the 128-row block; row B = + 8
        const int64_t rowA = (int64_t)tm * Cfg::BM + rowA_in, rowB = rowA + 8;
        const bool okA = rowA < p.M, okB = rowB < p.M;        // rows past M arrive as zeros (TMA fill)
        // this lane's 32 elements: box q / 2, chunks (q % 2) * 4 + 0..3 of the row's 128-byte line
        const uint32_t offA = (uint32_t)(q >> 1) * Cfg::X_BOX_BYTES + (uint32_t)rowA_in * 128;
        const uint32_t sw = (uint32_t)(r & 7), c0 = (uint32_t)(q & 1) * 4;
        uint16_t* va = p.values + rowA * (p.K / 2) + (int64_t)kb0 * 64 + q * 16;
        uint16_t* vb = va + 8 * (p.K / 2);
        uint32_t* slab = reinterpret_cast<uint32_t*>(p.meta + ((int64_t)tm * kblocks + kb0) * 2048 + pw * 256 + lane * 4);
        float numA = 0.f, denA = 0.f, numB = 0.f, denB = 0.f;
        uint32_t stage = 0, phase = 0;
        for (int kb = kb0; kb < kb1; ++kb) {
            if (!mbar_wait(bar_full + 8 * stage, phase, cta_abort, p.dev_error)) break;
            const uint32_t base = sX + stage * Cfg::X_BYTES + offA;
            uint32_t a0[8], a1[8], b0[8], b1[8];
            lds128(base + (((c0 + 0) ^ sw) << 4), a0[0], a0[1], a0[2], a0[3]);
            lds128(base + (((c0 + 1) ^ sw) << 4), a0[4], a0[5], a0[6], a0[7]);
            lds128(base + (((c0 + 2) ^ sw) << 4), a1[0], a1[1], a1[2], a1[3]);
            lds128(base + (((c0 + 3) ^ sw) << 4), a1[4], a1[5], a1[6], a1[7]);
            lds128(base + 1024 + (((c0 + 0) ^ sw) << 4), b0[0], b0[1], b0[2], b0[3]);
            lds128(base + 1024 + (((c0 + 1) ^ sw) << 4), b0[4], b0[5], b0[6], b0[7]);
            lds128(base + 1024 + (((c0 + 2) ^ sw) << 4), b1[0], b1[1], b1[2], b1[3]);
            lds128(base + 1024 + (((c0 + 3) ^ sw) << 4), b1[4], b1[5], b1[6], b1[7]);
            // the tile is in registers: hand the stage back before the arithmetic and the stores
            __syncwarp();
            if (lane == 0) mbar_arrive(bar_empty + 8 * stage);
            TileOut out;
            prune_tile_core<SUMS>(a0, a1, b0, b1, lut, out, numA, denA, numB, denB);
            prune_tile_store(out, va, vb, slab, okA, okB);
            va += 64; vb += 64; slab += 512;
            if (++stage == STAGES) { stage = 0; phase ^= 1; }
        }
        if constexpr (SUMS) {
#pragma unroll
            for (int off = 1; off <= 2; off <<= 1) {
                numA += __shfl_xor_sync(0xffffffffu, numA, off);
                denA += __shfl_xor_sync(0xffffffffu, denA, off);
                numB += __shfl_xor_sync(0xffffffffu, numB, off);
                denB += __shfl_xor_sync(0xffffffffu, denB, off);
            }
            if (q == 0) {
                float* mine = p.scale_partial + (((int64_t)tm * 8 + pw) * p.splits + split) * 32;
                *reinterpret_cast<float2*>(mine + 2 * r) = make_float2(numA, denA);
                *reinterpret_cast<float2*>(mine + 2 * (r + 8)) = make_float2(numB, denB);
            }
        }
    } else {
        // ------------------------------------------------------------------ drain -------------
        // accumulator -> this CTA's shared memory, float4 (row, 4 columns j) at (j * 128 + row) * 16:
        // consecutive lanes write consecutive 16-byte slots
        const int q = warp & 3;  // tensor-memory lane quarter this warp may read
        const int r_in_tile = q * 32 + lane;
        const bool alive = mbar_wait(bar_done, 0, cta_abort, p.dev_error);  // every MMA has retired: sB is free
        if (alive) {
            tc_fence_after();
            const uint32_t t_row = tmem_base + ((uint32_t)(q * 32) << 16);
#pragma unroll 1
            for (int c = 0; c < R / 32; ++c) {
                uint32_t v[32];
                tmem_ld_32x32b_x32(t_row + c * 32, v);
                tmem_ld_wait();
#pragma unroll
                for (int j = 0; j < 8; ++j)
                    sts128(sB + (uint32_t)(((c * 8 + j) * 128 + r_in_tile) * 16), v[4 * j], v[4 * j + 1], v[4 * j + 2],
                           v[4 * j + 3]);
            }
        }
    }

    // every split's partial (shared memory) and row sums (global) are written: cluster-wide hand-over
    __syncwarp();
    cluster_sync_all();
    if (warp >= 2 && warp < 6) {
        // this CTA finishes rows [split * 128 / splits, (split + 1) * 128 / splits) of the row block
        // (integer division: the shares differ by a row when splits does not divide 128)
        const int t = threadIdx.x - 64;  // 0..127
        const int row_first = split * Cfg::BM / p.splits;
        const int rows_per = (split + 1) * Cfg::BM / p.splits - row_first;
        if (t < rows_per) {
            const int64_t grow = (int64_t)tm * Cfg::BM + row_first + t;
            float s = 1.0f;
            if constexpr (SUMS) {
                // (the same additions, in the same order, as the GEMM epilogue that multiplies by s)
                if (grow < p.M) s = row_scale_from_partials(p.scale_partial, grow, p.splits);
            }
            s_scale[t] = s;
        }
        bar_sync_named(2, 128);
        constexpr int PIECES_PER_ROW = R / 8;
        const int items = rows_per * PIECES_PER_ROW;
        for (int idx = t; idx < items; idx += 128) {
            const int r_l = idx / PIECES_PER_ROW, piece = idx % PIECES_PER_ROW;  // consecutive threads: one row's pieces
            const int r_t = row_first + r_l;
            const int64_t grow = (int64_t)tm * Cfg::BM + r_t;
            if (grow >= p.M) continue;
            const uint32_t a0 = sB + (uint32_t)(((2 * piece) * 128 + r_t) * 16);
            const uint32_t a1 = sB + (uint32_t)(((2 * piece + 1) * 128 + r_t) * 16);
            float acc[8];
#pragma unroll
            for (int e = 0; e < 8; ++e) acc[e] = 0.0f;
            for (int sp = 0; sp < p.splits; ++sp) {  // ascending split order, always
                const float4 a = lds128_cluster_f32(mapa(a0, (uint32_t)sp));
                const float4 b = lds128_cluster_f32(mapa(a1, (uint32_t)sp));
                acc[0] += a.x; acc[1] += a.y; acc[2] += a.z; acc[3] += a.w;
                acc[4] += b.x; acc[5] += b.y; acc[6] += b.z; acc[7] += b.w;
            }
            const float s = s_scale[r_l];
            uint32_t o[4];
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const float t0 = (s == 0.0f) ? 0.0f : __fdiv_rn(acc[2 * e], s);
                const float t1 = (s == 0.0f) ? 0.0f : __fdiv_rn(acc[2 * e + 1], s);
                o[e] = pack_bf16x2(t0, t1);
            }
            *reinterpret_cast<uint4*>(p.T + grow * p.ldt + piece * 8) = make_uint4(o[0], o[1], o[2], o[3]);
        }
    }
    // nobody leaves while a peer may still read its shared memory
    __syncwarp();
    cluster_sync_all();

    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc<1>(tmem_base, Cfg::TMEM_COLS);
    }
}

}  // namespace lynx

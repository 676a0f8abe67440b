// Fused variant of the layer (online sparsification inside the GEMM kernel, Algorithm 1 lines 3-6
// in one launch): raw X tiles are pruned in shared memory and fed straight to the sparse MMA; the
// compressed activations and their metadata never touch HBM.
//
// One CTA per 128 x 256 output tile (persistent), 320 threads:
//   warp 0      producer: TMA loads of the raw X tile (128 rows x 128 elements as two 128-byte
//               swizzled boxes) and of the W tile (256 rows x 128 elements) per stage
//   warps 6..9  pruners, one thread per tile row: read the row's 16 swizzled 16-byte chunks,
//               run the same packed Top-2-of-4 selection as the stand-alone kernel, write the
//               64 kept values over the first box of the raw tile (same 128-byte-swizzled layout
//               the MMA descriptor expects; a chunk is only overwritten after it was consumed),
//               the metadata in tensor-memory-copy order, and keep the row's sum x^2 / sum kept x^2
//   warp 1      MMA issuer: metadata -> tensor memory, four tcgen05.mma.sp per stage
//   warps 2..5  epilogue (scale from the pruners via shared memory, bias, residual, bf16, TMA store)
// Every N tile prunes its rows again (N/256 times in total), which makes this kernel ALU bound;
// it exists to be measured against the two-kernel path.
#pragma once

#include "prune_compress.cuh"
#include "ptx.cuh"
#include "sparse_gemm.cuh"

namespace lynx {

struct FusedParams {
    int64_t M, N, K;
    int with_scale;            // 1: per-row norm compensation computed in-kernel
    const uint16_t* bias;      // [N] bf16 or nullptr
    const uint16_t* residual;  // [M x N] bf16 (ld = ldr) or nullptr
    int64_t ldr;
    uint32_t* dev_error;
    int tiles_m, tiles_n;
};

struct FusedCfg {
    static constexpr int BM = 128, BN = 256, BK = 128, STAGES = 2;
    static constexpr int X_BYTES = BM * BK * 2;      // raw tile, two boxes of 16 KB; box 0 becomes A
    static constexpr int X_BOX_BYTES = BM * 64 * 2;
    static constexpr int B_HALF_BYTES = BN * 64 * 2;
    static constexpr int B_BYTES = 2 * B_HALF_BYTES;  // 64 KB
    static constexpr int E_BYTES = 2048;
    static constexpr int STAGE_TX_BYTES = X_BYTES + B_BYTES;  // bytes TMA delivers per stage
    static constexpr int C_BOX_BYTES = 32 * 64 * 2;
    static constexpr int C_BYTES = 4 * C_BOX_BYTES;
    static constexpr int E_COL0 = BN;
    static constexpr int TMEM_COLS = 512;
    static constexpr int THREADS = 320;
    static constexpr int SMEM_BYTES = 1024 + STAGES * (X_BYTES + B_BYTES + E_BYTES) + C_BYTES + 1024 /*scale, two tiles*/ +
                                      256 /*lut*/ + 256 /*barriers*/;
    static_assert(SMEM_BYTES <= 227 * 1024, "shared memory budget");
};

// Epilogue arithmetic of one 64-column chunk of one row: y = s*acc + bias + residual, packed to
// bf16 and written into a 128-byte-swizzled 32 x 64 staging box.
__device__ __forceinline__ void epilogue_chunk_to_smem(const uint32_t (&v)[64], float s, int64_t row, bool row_ok,
                                                       int n0, int64_t N, const uint16_t* bias,
                                                       const uint16_t* residual, int64_t ldr, uint32_t cbuf,
                                                       int lane) {
#pragma unroll
    for (int j = 0; j < 8; ++j) {
        const int n = n0 + j * 8;
        float b[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
        float r[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
        if (n < N) {
            if (bias != nullptr) {
                const uint4 bv = __ldg(reinterpret_cast<const uint4*>(bias + n));
                b[0] = bf16_lo_f(bv.x); b[1] = bf16_hi_f(bv.x); b[2] = bf16_lo_f(bv.y); b[3] = bf16_hi_f(bv.y);
                b[4] = bf16_lo_f(bv.z); b[5] = bf16_hi_f(bv.z); b[6] = bf16_lo_f(bv.w); b[7] = bf16_hi_f(bv.w);
            }
            if (residual != nullptr && row_ok) {
                const uint4 rv = __ldg(reinterpret_cast<const uint4*>(residual + row * ldr + n));
                r[0] = bf16_lo_f(rv.x); r[1] = bf16_hi_f(rv.x); r[2] = bf16_lo_f(rv.y); r[3] = bf16_hi_f(rv.y);
                r[4] = bf16_lo_f(rv.z); r[5] = bf16_hi_f(rv.z); r[6] = bf16_lo_f(rv.w); r[7] = bf16_hi_f(rv.w);
            }
        }
        uint32_t o[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            const float y0 = fmaf(s, __uint_as_float(v[j * 8 + 2 * e]), b[2 * e]) + r[2 * e];
            const float y1 = fmaf(s, __uint_as_float(v[j * 8 + 2 * e + 1]), b[2 * e + 1]) + r[2 * e + 1];
            o[e] = pack_bf16x2(y0, y1);
        }
        sts128(cbuf + lane * 128 + ((j ^ (lane & 7)) << 4), o[0], o[1], o[2], o[3]);
    }
}

__device__ __forceinline__ void sts16(uint32_t addr, uint32_t v) {
    asm volatile("st.shared.u16 [%0], %1;" ::"r"(addr), "h"((unsigned short)v) : "memory");
}

__global__ void __launch_bounds__(FusedCfg::THREADS, 1)
fused_linear_kernel(const __grid_constant__ CUtensorMap tmap_x, const __grid_constant__ CUtensorMap tmap_b,
                    const __grid_constant__ CUtensorMap tmap_y, const FusedParams p) {
    using Cfg = FusedCfg;
    constexpr int STAGES = Cfg::STAGES, BN = Cfg::BN;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* smem_gen = smem_raw + (smem_base - smem_u32(smem_raw));
    const uint32_t sX = smem_base;                         // raw X stages (box 0 doubles as compressed A)
    const uint32_t sB = sX + STAGES * Cfg::X_BYTES;
    const uint32_t sE = sB + STAGES * Cfg::B_BYTES;
    const uint32_t sC = sE + STAGES * Cfg::E_BYTES;
    const uint32_t sScale = sC + Cfg::C_BYTES;             // 2 x 128 floats (tile parity)
    const uint32_t sLut = sScale + 1024;                   // 64 words
    const uint32_t sBar = sLut + 256;
    const uint32_t bar_full = sBar, bar_pruned = sBar + 8 * STAGES, bar_empty = sBar + 16 * STAGES;
    const uint32_t bar_tfull = sBar + 24 * STAGES, bar_tempty = bar_tfull + 8;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem_gen + (sBar - smem_base) + 24 * STAGES + 16);
    volatile uint32_t* cta_abort = tmem_slot + 1;
    float* scale_smem = reinterpret_cast<float*>(smem_gen + (sScale - smem_base));
    uint32_t* lut = reinterpret_cast<uint32_t*>(smem_gen + (sLut - smem_base));

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int num_tiles = p.tiles_m * p.tiles_n;
    const int kblocks = (int)(p.K / Cfg::BK);

    if (threadIdx.x == 0) {
        *cta_abort = 0;
        for (int s = 0; s < STAGES; ++s) {
            mbar_init(bar_full + 8 * s, 1);
            mbar_init(bar_pruned + 8 * s, 4);  // one arrive per pruner warp
            mbar_init(bar_empty + 8 * s, 1);
        }
        mbar_init(bar_tfull, 1);
        mbar_init(bar_tempty, 4);
        fence_mbar_init();
        prefetch_tmap(&tmap_x);
        prefetch_tmap(&tmap_b);
        prefetch_tmap(&tmap_y);
    }
    if (threadIdx.x < 64) lut[threadIdx.x] = prune_lut_entry(threadIdx.x & 15, threadIdx.x >> 4);
    if (warp == 1) {
        tmem_alloc<1>(smem_u32(tmem_slot), Cfg::TMEM_COLS);
        tmem_relinquish<1>();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    if (warp == 0) {
        // ------------------------------------------------------------------ producer ----------
        if (lane == 0) {
            uint32_t stage = 0, phase = 0;
            bool ok = true;
            for (int t = blockIdx.x; t < num_tiles && ok; t += gridDim.x) {
                const int m0 = (t % p.tiles_m) * Cfg::BM, n0 = (t / p.tiles_m) * BN;
                for (int kb = 0; kb < kblocks; ++kb) {
                    if (!mbar_wait(bar_empty + 8 * stage, phase ^ 1, cta_abort, p.dev_error)) { ok = false; break; }
                    const uint32_t bar = bar_full + 8 * stage;
                    const uint32_t x_dst = sX + stage * Cfg::X_BYTES, b_dst = sB + stage * Cfg::B_BYTES;
                    mbar_arrive_expect_tx(bar, Cfg::STAGE_TX_BYTES);
                    tma_load_2d(x_dst, &tmap_x, kb * 128, m0, bar);
                    tma_load_2d(x_dst + Cfg::X_BOX_BYTES, &tmap_x, kb * 128 + 64, m0, bar);
                    tma_load_2d(b_dst, &tmap_b, kb * 128, n0, bar);
                    tma_load_2d(b_dst + Cfg::B_HALF_BYTES, &tmap_b, kb * 128 + 64, n0, bar);
                    if (++stage == STAGES) { stage = 0; phase ^= 1; }
                }
            }
            if (!ok) bounded_delay_ns(200000);  // let the copies in flight land before teardown
        }
    } else if (warp >= 6) {
        // ------------------------------------------------------------------ pruners -----------
        const int r = threadIdx.x - 192;  // row of the tile
        const uint32_t swz = (uint32_t)(r & 7);
        // metadata byte of (row r, 16-element span v): lane-major tensor-memory-copy image
        const uint32_t e_row = (uint32_t)(((r & 7) + 16 * (r >> 4)) * 16 + ((r >> 3) & 1) * 2);
        uint32_t stage = 0, phase = 0;
        bool ok = true;
        int it = 0;
        for (int t = blockIdx.x; t < num_tiles && ok; t += gridDim.x, ++it) {
            float num = 0.f, den = 0.f;
            for (int kb = 0; kb < kblocks; ++kb) {
                if (!mbar_wait(bar_full + 8 * stage, phase, cta_abort, p.dev_error)) { ok = false; break; }
                const uint32_t xrow = sX + stage * Cfg::X_BYTES + (uint32_t)r * 128;
                const uint32_t erow = sE + stage * Cfg::E_BYTES + e_row;
#pragma unroll
                for (int v = 0; v < 8; ++v) {
                    // 16 elements = chunks 2(v%4), 2(v%4)+1 of box v/4; chunk c sits at c ^ (r%8)
                    const uint32_t box = xrow + (v >> 2) * Cfg::X_BOX_BYTES;
                    const uint32_t c0 = (uint32_t)(2 * (v & 3));
                    uint32_t x[8], o[4];
                    lds128(box + ((c0 ^ swz) << 4), x[0], x[1], x[2], x[3]);
                    lds128(box + (((c0 + 1) ^ swz) << 4), x[4], x[5], x[6], x[7]);
                    const uint32_t m16 = prune_vec16(x, lut, o);
                    if (p.with_scale) {
#pragma unroll
                        for (int i = 0; i < 8; ++i) num = fma_sq_bf16x2(x[i], num);
#pragma unroll
                        for (int i = 0; i < 4; ++i) den = fma_sq_bf16x2(o[i], den);
                    }
                    // compressed chunk v of this row goes over raw chunk v of box 0 (already consumed)
                    sts128(xrow + (((uint32_t)v ^ swz) << 4), o[0], o[1], o[2], o[3]);
                    sts16(erow + (v >> 1) * 4 + (v & 1) * 128, m16);
                }
                if (kb == kblocks - 1)
                    scale_smem[(it & 1) * 128 + r] = p.with_scale ? sqrtf(num / (den + 1e-8f)) : 1.0f;
                fence_proxy_async_smem();  // generic-proxy writes -> visible to the tensor core
                __syncwarp();
                if (lane == 0) mbar_arrive(bar_pruned + 8 * stage);
                if (++stage == STAGES) { stage = 0; phase ^= 1; }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer --------
        if (lane == 0) {
            constexpr uint32_t idesc0 = make_idesc_sp_bf16(Cfg::BM, BN), idesc1 = idesc0 | 1u;
            const uint64_t d0 = make_desc_sw128(sX);
            const uint32_t desc_hi = (uint32_t)(d0 >> 32);
            const uint32_t a_lo0 = (uint32_t)d0, b_lo0 = (uint32_t)make_desc_sw128(sB);
            const uint64_t e_d0 = make_desc_rows16(sE);
            constexpr uint32_t BH = Cfg::B_HALF_BYTES >> 4;
            uint32_t stage = 0, phase = 0;
            bool ok = true;
            int it = 0;
            for (int t = blockIdx.x; t < num_tiles && ok; t += gridDim.x, ++it) {
                if (!mbar_wait(bar_tempty, (uint32_t)(it & 1) ^ 1, cta_abort, p.dev_error)) break;
                tc_fence_after();
                uint32_t accumulate = 0;
                for (int kb = 0; kb < kblocks; ++kb) {
                    // W landed (full) and the pruners finished A + metadata of this stage
                    if (!mbar_wait(bar_full + 8 * stage, phase, cta_abort, p.dev_error) ||
                        !mbar_wait(bar_pruned + 8 * stage, phase, cta_abort, p.dev_error)) {
                        ok = false;
                        break;
                    }
                    tc_fence_after();
                    const uint32_t e_tmem = tmem_base + Cfg::E_COL0 + 4 * stage;
                    const uint32_t a_lo = a_lo0 + stage * (Cfg::X_BYTES >> 4);
                    const uint32_t b_lo = b_lo0 + stage * (Cfg::B_BYTES >> 4);
                    tmem_cp_128x128b<1>(e_tmem, e_d0 + (uint64_t)(stage * (Cfg::E_BYTES >> 4)));
                    mma_sp_bf16_lh<1>(tmem_base, a_lo, b_lo, desc_hi, e_tmem, idesc0, accumulate);
                    mma_sp_bf16_lh<1>(tmem_base, a_lo + 2, b_lo + 4, desc_hi, e_tmem, idesc1, 1u);
                    mma_sp_bf16_lh<1>(tmem_base, a_lo + 4, b_lo + BH, desc_hi, e_tmem + 2, idesc0, 1u);
                    mma_sp_bf16_lh<1>(tmem_base, a_lo + 6, b_lo + BH + 4, desc_hi, e_tmem + 2, idesc1, 1u);
                    accumulate = 1u;
                    tc_commit(bar_empty + 8 * stage);
                    if (++stage == STAGES) { stage = 0; phase ^= 1; }
                }
                if (!ok) break;
                tc_commit(bar_tfull);
            }
        }
    } else if (warp >= 2 && warp <= 5) {
        // ------------------------------------------------------------------ epilogue ----------
        const int q = warp & 3;
        const uint32_t cbuf = sC + (warp - 2) * Cfg::C_BOX_BYTES;
        int it = 0;
        for (int t = blockIdx.x; t < num_tiles; t += gridDim.x, ++it) {
            const int tm = t % p.tiles_m, tn = t / p.tiles_m;
            if (!mbar_wait(bar_tfull, (uint32_t)(it & 1), cta_abort, p.dev_error)) break;
            tc_fence_after();
            const int m0 = tm * Cfg::BM + q * 32;
            const int64_t row = m0 + lane;
            const bool row_ok = row < p.M;
            const float s = scale_smem[(it & 1) * 128 + q * 32 + lane];
            const uint32_t t_row = tmem_base + ((uint32_t)(q * 32) << 16);
#pragma unroll 1
            for (int c = 0; c < BN / 64; ++c) {
                const int n0 = tn * BN + c * 64;
                uint32_t v[64];
                tmem_ld_32x32b_x32(t_row + c * 64, *reinterpret_cast<uint32_t(*)[32]>(&v[0]));
                tmem_ld_32x32b_x32(t_row + c * 64 + 32, *reinterpret_cast<uint32_t(*)[32]>(&v[32]));
                tmem_ld_wait();
                if (c == BN / 64 - 1) {
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(bar_tempty);
                }
                if (n0 >= p.N) continue;
                if (lane == 0) tma_store_wait_read<0>();
                __syncwarp();
                epilogue_chunk_to_smem(v, s, row, row_ok, n0, p.N, p.bias, p.residual, p.ldr, cbuf, lane);
                fence_proxy_async_smem();
                __syncwarp();
                if (lane == 0) {
                    tma_store_2d(&tmap_y, n0, m0, cbuf);
                    tma_store_commit();
                }
            }
        }
        if (lane == 0) tma_store_wait_all<0>();
    }

    // ---------------------------------------------------------------------- teardown ----------
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc<1>(tmem_base, Cfg::TMEM_COLS);
    }
}

}  // namespace lynx

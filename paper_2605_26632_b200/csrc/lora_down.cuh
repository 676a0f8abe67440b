// Down projection of the low-rank branch (Algorithm 1 line 5, first factor of Y_r = X (L_A L_B)^T):
//     T[m, r] = bf16( (sum_k X[m,k] L_B[r,k]) / s_m )          X dense, L_B is R x K
// The division by the row's norm-compensation scale lets the sparse GEMM add T L_A^T into the
// same accumulator that its epilogue multiplies by s_m (s_m * (acc + (T/s_m) L_A^T) =
// s_m * acc + T L_A^T); rows with s_m = 0 (all-zero rows) give T = 0.  Without a scale s_m = 1.
//
// The kernel streams X once (HBM bound: 2 bytes per element of X; L_B stays in the L2).  One CTA
// per (128-row block, K split): warp 0 TMA producer (X box 128 x 64, L_B box R x 64, 128-byte
// swizzle), warp 1 issues four dense tcgen05.mma (K = 16 each) per stage into a 128 x R fp32
// accumulator in tensor memory, warps 2..5 drain it.  With more than one K split the CTAs write
// fp32 partials and the CTA that draws the row block's last ticket adds them in split order
// (the result does not depend on which CTA that is) and writes T.
#pragma once

#include "ptx.cuh"

namespace lynx {

struct LoraDownParams {
    int64_t M, K;
    int splits;         // K splits per row block
    int kb_per_split;   // 64-element K blocks per split (the last split may get fewer)
    const float* row_scale;  // [M] or nullptr
    uint16_t* T;             // [M x R] bf16, leading dimension ldt
    int64_t ldt;
    float* partial;      // [row blocks][splits][128][R] fp32 (splits > 1)
    uint32_t* tickets;   // one word per row block, zero between launches
    uint32_t* dev_error;
};

template <int R_>
struct LoraDownCfg {
    static constexpr int R = R_;
    static constexpr int BM = 128, BK = 64;
    static constexpr int STAGES = (R == 64) ? 8 : 6;
    static constexpr int A_BYTES = BM * BK * 2;  // 16 KB
    static constexpr int B_BYTES = R * BK * 2;   // 8 or 16 KB
    static constexpr int STAGE_BYTES = A_BYTES + B_BYTES;
    static constexpr int SMEM_BYTES = 1024 + STAGES * STAGE_BYTES + 256;
    static constexpr int THREADS = 192;
    static constexpr int TMEM_COLS = R;  // power of two >= 32
    static_assert(R == 64 || R == 128, "rank");
    static_assert(SMEM_BYTES <= 227 * 1024, "shared memory budget");
};

// Instruction descriptor of the dense tcgen05.mma kind::f16: bf16 x bf16 -> fp32, K-major operands.
__host__ __device__ constexpr uint32_t make_idesc_bf16(int m, int n) {
    return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(m >> 4) << 24);
}

template <class Cfg>
__global__ void __launch_bounds__(Cfg::THREADS, 1)
lora_down_kernel(const __grid_constant__ CUtensorMap tmap_x, const __grid_constant__ CUtensorMap tmap_lb,
                 const LoraDownParams p) {
    constexpr int STAGES = Cfg::STAGES, R = Cfg::R;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* smem_gen = smem_raw + (smem_base - smem_u32(smem_raw));
    const uint32_t sA = smem_base;
    const uint32_t sB = sA + STAGES * Cfg::A_BYTES;
    const uint32_t sBar = sB + STAGES * Cfg::B_BYTES;
    const uint32_t bar_full = sBar, bar_empty = sBar + 8 * STAGES, bar_done = sBar + 16 * STAGES;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem_gen + (sBar - smem_base) + 16 * STAGES + 8);
    volatile uint32_t* cta_abort = tmem_slot + 1;
    volatile uint32_t* s_last = tmem_slot + 2;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int tiles_m = (int)((p.M + Cfg::BM - 1) / Cfg::BM);
    const int tm = blockIdx.x % tiles_m, split = blockIdx.x / tiles_m;
    const int kblocks = (int)(p.K / Cfg::BK);
    const int kb0 = split * p.kb_per_split;
    const int kb1 = (kb0 + p.kb_per_split < kblocks) ? kb0 + p.kb_per_split : kblocks;

    if (threadIdx.x == 0) {
        *cta_abort = 0;
        *s_last = 0;
        for (int s = 0; s < STAGES; ++s) {
            mbar_init(bar_full + 8 * s, 1);
            mbar_init(bar_empty + 8 * s, 1);
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
    griddep_wait();  // X and row_scale come from the kernels before this one

    if (warp == 0) {
        if (lane == 0) {
            uint32_t stage = 0, phase = 0, issued = 0;
            bool ok = true;
            for (int kb = kb0; kb < kb1; ++kb) {
                if (!mbar_wait(bar_empty + 8 * stage, phase ^ 1, cta_abort, p.dev_error)) {
                    ok = false;
                    break;
                }
                const uint32_t bar = bar_full + 8 * stage;
                mbar_arrive_expect_tx(bar, Cfg::STAGE_BYTES);
                tma_load_2d(sA + stage * Cfg::A_BYTES, &tmap_x, kb * Cfg::BK, tm * Cfg::BM, bar);
                tma_load_2d(sB + stage * Cfg::B_BYTES, &tmap_lb, kb * Cfg::BK, 0, bar);
                ++issued;
                if (++stage == STAGES) { stage = 0; phase ^= 1; }
            }
            if (!ok && issued) bounded_delay_ns(200000);
        }
    } else if (warp == 1) {
        if (lane == 0) {
            constexpr uint32_t idesc = make_idesc_bf16(Cfg::BM, R);
            const uint64_t d0 = make_desc_sw128(sA);
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
                const uint32_t a_lo = a_lo0 + stage * (Cfg::A_BYTES >> 4);
                const uint32_t b_lo = b_lo0 + stage * (Cfg::B_BYTES >> 4);
                // four K steps of 16 elements = 32 bytes inside the 128-byte swizzle atom
                mma_bf16_lh<1>(tmem_base, a_lo, b_lo, desc_hi, idesc, accumulate);
                mma_bf16_lh<1>(tmem_base, a_lo + 2, b_lo + 2, desc_hi, idesc, 1u);
                mma_bf16_lh<1>(tmem_base, a_lo + 4, b_lo + 4, desc_hi, idesc, 1u);
                mma_bf16_lh<1>(tmem_base, a_lo + 6, b_lo + 6, desc_hi, idesc, 1u);
                accumulate = 1u;
                tc_commit(bar_empty + 8 * stage);
                if (++stage == STAGES) { stage = 0; phase ^= 1; }
            }
            if (ok) tc_commit(bar_done);
        }
    } else {
        // ------------------------------------------------------------------ drain -------------
        const int q = warp & 3;  // tensor-memory lane quarter this warp may read
        const int r_in_tile = q * 32 + lane;
        const int64_t row = (int64_t)tm * Cfg::BM + r_in_tile;
        const bool row_ok = row < p.M;
        bool alive = mbar_wait(bar_done, 0, cta_abort, p.dev_error);
        if (alive) {
            tc_fence_after();
            const uint32_t t_row = tmem_base + ((uint32_t)(q * 32) << 16);
            float s = 1.0f;
            if (p.row_scale != nullptr && row_ok) s = p.row_scale[row];
            float* my_partial = p.partial + (((size_t)tm * p.splits + split) * Cfg::BM + r_in_tile) * R;
#pragma unroll 1
            for (int c = 0; c < R / 32; ++c) {
                uint32_t v[32];
                tmem_ld_32x32b_x32(t_row + c * 32, v);
                tmem_ld_wait();
                if (p.splits == 1) {
                    if (row_ok) {
                        uint32_t o[16];
#pragma unroll
                        for (int e = 0; e < 16; ++e) {
                            const float t0 = (s == 0.0f) ? 0.0f : __fdiv_rn(__uint_as_float(v[2 * e]), s);
                            const float t1 = (s == 0.0f) ? 0.0f : __fdiv_rn(__uint_as_float(v[2 * e + 1]), s);
                            o[e] = pack_bf16x2(t0, t1);
                        }
                        uint4* dst = reinterpret_cast<uint4*>(p.T + row * p.ldt + c * 32);
#pragma unroll
                        for (int j = 0; j < 4; ++j) dst[j] = make_uint4(o[4 * j], o[4 * j + 1], o[4 * j + 2], o[4 * j + 3]);
                    }
                } else if (row_ok) {
                    float4* dst = reinterpret_cast<float4*>(my_partial + c * 32);
#pragma unroll
                    for (int j = 0; j < 8; ++j)
                        __stcg(dst + j, make_float4(__uint_as_float(v[4 * j]), __uint_as_float(v[4 * j + 1]),
                                                    __uint_as_float(v[4 * j + 2]), __uint_as_float(v[4 * j + 3])));
                }
            }
        }
        if (p.splits > 1) {
            // hand-over: every drain thread's partial rows are written, then one ticket per CTA
            asm volatile("bar.sync 1, 128;" ::: "memory");
            if (warp == 2 && lane == 0) {
                // one acquire-release add: publishes this CTA's partial rows (ordered before it by
                // the barrier) and, for the CTA that draws the last ticket, makes all others' visible
                const uint32_t t = atom_add_acq_rel_gpu(p.tickets + tm, 1u);
                if (t == (uint32_t)p.splits - 1) {
                    p.tickets[tm] = 0;  // ready for the next launch
                    *s_last = 1;
                }
            }
            asm volatile("bar.sync 1, 128;" ::: "memory");
            // a CTA that timed out still takes its ticket (so nobody is left waiting); the error
            // word tells the host that T is not valid
            if (*s_last) {
                // 128 threads x 8-column pieces, consecutive threads on consecutive pieces; four
                // pieces at a time so that 8 * (splits unrolled by 2) loads are in flight per thread
                const int t = threadIdx.x - 64;
                constexpr int PIECES_PER_ROW = R / 8;
                constexpr int ITEMS = Cfg::BM * PIECES_PER_ROW / 128;
                const float* base = p.partial + (size_t)tm * p.splits * Cfg::BM * R;
#pragma unroll 1
                for (int i0 = 0; i0 < ITEMS; i0 += 4) {
                    float acc[4][8];
#pragma unroll
                    for (int u = 0; u < 4; ++u)
#pragma unroll
                        for (int e = 0; e < 8; ++e) acc[u][e] = 0.0f;
#pragma unroll 2
                    for (int sp = 0; sp < p.splits; ++sp) {  // ascending split order, always
                        float4 a[4], b[4];
#pragma unroll
                        for (int u = 0; u < 4; ++u) {
                            const int idx = (i0 + u) * 128 + t;  // = row * PIECES_PER_ROW + piece
                            const float4* src = reinterpret_cast<const float4*>(base + (size_t)sp * Cfg::BM * R + (size_t)idx * 8);
                            a[u] = __ldcg(src);
                            b[u] = __ldcg(src + 1);
                        }
#pragma unroll
                        for (int u = 0; u < 4; ++u) {
                            acc[u][0] += a[u].x; acc[u][1] += a[u].y; acc[u][2] += a[u].z; acc[u][3] += a[u].w;
                            acc[u][4] += b[u].x; acc[u][5] += b[u].y; acc[u][6] += b[u].z; acc[u][7] += b[u].w;
                        }
                    }
#pragma unroll
                    for (int u = 0; u < 4; ++u) {
                        const int idx = (i0 + u) * 128 + t;
                        const int r_t = idx / PIECES_PER_ROW, piece = idx % PIECES_PER_ROW;
                        const int64_t grow = (int64_t)tm * Cfg::BM + r_t;
                        if (grow >= p.M) continue;
                        const float s = (p.row_scale != nullptr) ? p.row_scale[grow] : 1.0f;
                        uint32_t o[4];
#pragma unroll
                        for (int e = 0; e < 4; ++e) {
                            const float t0 = (s == 0.0f) ? 0.0f : __fdiv_rn(acc[u][2 * e], s);
                            const float t1 = (s == 0.0f) ? 0.0f : __fdiv_rn(acc[u][2 * e + 1], s);
                            o[e] = pack_bf16x2(t0, t1);
                        }
                        *reinterpret_cast<uint4*>(p.T + grow * p.ldt + piece * 8) = make_uint4(o[0], o[1], o[2], o[3]);
                    }
                }
            }
        }
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc<1>(tmem_base, Cfg::TMEM_COLS);
    }
}

}  // namespace lynx

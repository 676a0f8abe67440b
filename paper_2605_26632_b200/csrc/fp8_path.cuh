// FP8 (E4M3) composition of the activation-sparse layer (the paper's W8A8 compatibility
// experiment: symmetric FP8 quantisation of the activations, weights cast to FP8, 2:4 on FP8
// operands).  Two kernels feed the FP8 instantiation of the sparse GEMM:
//
//   quantize_weights_fp8_kernel   W bf16 -> E4M3 codes, direct cast or symmetric per output channel
//   prune_compress_fp8_kernel     Top-2-of-4 on the bf16 activations, kept values -> E4M3 codes with
//                                 one symmetric scale per token row, metadata in the order the
//                                 FP8 sparse MMA reads, row_scale = (norm compensation) * (amax / 448)
//
// Rules shared with the definition the parity tests check (all fp32, IEEE):
//   amax = largest magnitude of the row in the selection's order (15 non-sign bits as an integer)
//   inv  = amax > 0 ? 448 / amax : 0          code = e4m3_rn_satfinite(x * inv)
//   act_scale = amax / 448
#pragma once

#include "prune_compress.cuh"

namespace lynx {

constexpr int FP8_PRUNE_WARPS = 12;  // 384 threads: two CTAs per SM at <= 85 registers

// ------------------------------------------------------------------------------- weights --------
// One CTA per output channel n.  per_channel = 0: code = e4m3(w), scale 1.
__global__ void __launch_bounds__(256)
quantize_weights_fp8_kernel(const uint16_t* __restrict__ W, int64_t N, int64_t K, int64_t ldw, int per_channel,
                            uint8_t* __restrict__ Wq, float* __restrict__ wscale) {
    __shared__ uint32_t s_top[8];
    const int64_t n = blockIdx.x;
    const uint16_t* w = W + n * ldw;
    float inv = 1.0f;
    if (per_channel) {
        uint32_t top = 0;
        for (int64_t k = threadIdx.x; k < K; k += blockDim.x) {
            const uint32_t m = w[k] & 0x7fffu;
            top = m > top ? m : top;
        }
#pragma unroll
        for (int off = 16; off >= 1; off >>= 1) {
            const uint32_t o = __shfl_xor_sync(0xffffffffu, top, off);
            top = o > top ? o : top;
        }
        if ((threadIdx.x & 31) == 0) s_top[threadIdx.x >> 5] = top;
        __syncthreads();
        top = 0;
        for (int i = 0; i < (int)(blockDim.x >> 5); ++i) top = s_top[i] > top ? s_top[i] : top;
        const float amax = __uint_as_float(top << 16);
        inv = amax > 0.0f ? __fdiv_rn(448.0f, amax) : 0.0f;
        if (threadIdx.x == 0) wscale[n] = __fdiv_rn(amax, 448.0f);
    } else if (threadIdx.x == 0) {
        wscale[n] = 1.0f;
    }
    uint8_t* out = Wq + n * K;
    for (int64_t k = 2 * threadIdx.x; k < K; k += 2 * blockDim.x) {  // K is even
        const float a = __uint_as_float((uint32_t)w[k] << 16), b = __uint_as_float((uint32_t)w[k + 1] << 16);
        *reinterpret_cast<uint16_t*>(out + k) = (uint16_t)cvt_e4m3x2(__fmul_rn(a, inv), __fmul_rn(b, inv));
    }
}

// --------------------------------------------------------------------------- activations --------
// 16 kept bf16 pairs of one row slice (8 registers, pair g in register g: lower index in the lower
// half) -> 16 E4M3 codes in 4 registers, in element order.
__device__ __forceinline__ void quantize_kept16(const uint32_t* v /*[8]*/, float inv, uint32_t* out /*[4]*/) {
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const uint32_t g0 = v[2 * i], g1 = v[2 * i + 1];
        const uint32_t c0 = cvt_e4m3x2(__fmul_rn(bf16_lo_f(g0), inv), __fmul_rn(bf16_hi_f(g0), inv));
        const uint32_t c1 = cvt_e4m3x2(__fmul_rn(bf16_lo_f(g1), inv), __fmul_rn(bf16_hi_f(g1), inv));
        out[i] = c0 | (c1 << 16);
    }
}

// One CTA per 16-row block, all of K, two passes over the block's rows (the second one finds them
// in the L2): pass 1 the row maxima, pass 2 selection + codes + metadata (+ the norm-compensation
// sums).  The CTA owns its rows, so no cross-CTA hand-over is needed for the per-row scale.
// Metadata block (rb, kb) of 128 rows x 128 K at byte (rb * K/128 + kb) * 2048; inside it row r's
// 16 bytes at r * 16, group g = (k % 128) / 4 in bits 4 * (g % 2) of byte g / 2 (natural order).
// mode: 0 -> row_scale = amax / 448; 1 -> row_scale = sqrt(sum x^2 / (sum kept^2 + 1e-8)) * amax / 448.
// GIVEN: the row maxima come from the caller (row_amax[m]: a calibrated scale, or a maximum the
// producer of X already knows) and pass 1 is skipped: X is then read once.
template <bool SUMS, bool GIVEN>
__global__ void __launch_bounds__(FP8_PRUNE_WARPS * 32, 1)
prune_compress_fp8_kernel(const uint16_t* __restrict__ X, int64_t M, int64_t K, int64_t ldx,
                          const float* __restrict__ row_amax, uint8_t* __restrict__ values_q,
                          uint8_t* __restrict__ meta, float* __restrict__ row_scale) {
    __shared__ uint32_t lut[4 * 16];
    __shared__ uint32_t s_top[FP8_PRUNE_WARPS][16];
    __shared__ float2 s_sum[FP8_PRUNE_WARPS][16];
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    if (tid < 64) lut[tid] = prune_lut_entry(tid & 15, tid >> 4);
    griddep_wait();

    const int64_t row0 = (int64_t)blockIdx.x * PRUNE_ROWS;
    const int r = lane >> 2, q = lane & 3;
    const int64_t rowA = row0 + r, rowB = rowA + 8;
    const bool okA = rowA < M, okB = rowB < M;
    const int kb128 = (int)(K / 128);
    const uint16_t* xa0 = X + rowA * ldx + q * 32;
    const uint16_t* xb0 = xa0 + 8 * ldx;

    // ---- pass 1: largest magnitude of each row (packed 16-bit maxima over the 15 magnitude bits)
    uint32_t mA = 0, mB = 0;
    for (int t = warp; !GIVEN && t < kb128; t += FP8_PRUNE_WARPS) {
        uint32_t a0[8], a1[8], b0[8], b1[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) a0[i] = a1[i] = b0[i] = b1[i] = 0u;
        if (okA) {
            ldg256_keep(xa0 + (int64_t)t * 128, a0);
            ldg256_keep(xa0 + (int64_t)t * 128 + 16, a1);
        }
        if (okB) {
            ldg256_keep(xb0 + (int64_t)t * 128, b0);
            ldg256_keep(xb0 + (int64_t)t * 128 + 16, b1);
        }
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            mA = vmax_u16x2(mA, vmax_u16x2(a0[i] & 0x7FFF7FFFu, a1[i] & 0x7FFF7FFFu));
            mB = vmax_u16x2(mB, vmax_u16x2(b0[i] & 0x7FFF7FFFu, b1[i] & 0x7FFF7FFFu));
        }
    }
    uint32_t topA = max(mA & 0xFFFFu, mA >> 16), topB = max(mB & 0xFFFFu, mB >> 16);
#pragma unroll
    for (int off = 1; off <= 2; off <<= 1) {
        topA = max(topA, __shfl_xor_sync(0xffffffffu, topA, off));
        topB = max(topB, __shfl_xor_sync(0xffffffffu, topB, off));
    }
    if (q == 0) {
        s_top[warp][r] = topA;
        s_top[warp][r + 8] = topB;
    }
    __syncthreads();
    topA = 0;
    topB = 0;
#pragma unroll
    for (int w = 0; w < FP8_PRUNE_WARPS; ++w) {
        topA = max(topA, s_top[w][r]);
        topB = max(topB, s_top[w][r + 8]);
    }
    float amaxA = __uint_as_float(topA << 16), amaxB = __uint_as_float(topB << 16);
    if constexpr (GIVEN) {
        amaxA = okA ? __ldg(row_amax + rowA) : 0.0f;
        amaxB = okB ? __ldg(row_amax + rowB) : 0.0f;
    }
    const float invA = amaxA > 0.0f ? __fdiv_rn(448.0f, amaxA) : 0.0f;
    const float invB = amaxB > 0.0f ? __fdiv_rn(448.0f, amaxB) : 0.0f;

    // ---- pass 2: selection, codes, metadata, sums
    float numA = 0.f, denA = 0.f, numB = 0.f, denB = 0.f;
    const int64_t rb128 = row0 / 128;
    uint8_t* mrow = meta + (rb128 * kb128) * 2048 + ((row0 % 128) + r) * 16 + q * 4;
    uint8_t* va0 = values_q + rowA * (K / 2) + q * 16;
    uint8_t* vb0 = va0 + 8 * (K / 2);
    for (int t = warp; t < kb128; t += FP8_PRUNE_WARPS) {
        TileOut out;
        float nA = 0.f, dA = 0.f, nB = 0.f, dB = 0.f;
        prune_tile_compute<SUMS, true>(xa0 + (int64_t)t * 128, xb0 + (int64_t)t * 128, okA, okB, lut, out, nA, dA, nB, dB);
        numA += nA; denA += dA; numB += nB; denB += dB;
        // prune_tile_compute packs the metadata for the bf16 order (w0 = low halves of both rows,
        // w1 = high halves); the FP8 order wants each row's 32 bits together
        const uint32_t wA = (out.w0 & 0xFFFFu) | (out.w1 << 16);
        const uint32_t wB = (out.w0 >> 16) | (out.w1 & 0xFFFF0000u);
        uint32_t ca[4], cb[4];
        quantize_kept16(out.oa, invA, ca);
        quantize_kept16(out.ob, invB, cb);
        if (okA) stg128(va0 + (int64_t)t * 64, ca[0], ca[1], ca[2], ca[3]);
        if (okB) stg128(vb0 + (int64_t)t * 64, cb[0], cb[1], cb[2], cb[3]);
        *reinterpret_cast<uint32_t*>(mrow + (int64_t)t * 2048) = wA;
        *reinterpret_cast<uint32_t*>(mrow + (int64_t)t * 2048 + 8 * 16) = wB;
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
            s_sum[warp][r] = make_float2(numA, denA);
            s_sum[warp][r + 8] = make_float2(numB, denB);
        }
        __syncthreads();
    }
    if (tid < 16 && row0 + tid < M) {
        uint32_t top = 0;
#pragma unroll
        for (int w = 0; w < FP8_PRUNE_WARPS; ++w) top = max(top, s_top[w][tid]);
        float sc = __fdiv_rn(GIVEN ? __ldg(row_amax + row0 + tid) : __uint_as_float(top << 16), 448.0f);
        if constexpr (SUMS) {
            float num = 0.f, den = 0.f;
#pragma unroll
            for (int w = 0; w < FP8_PRUNE_WARPS; ++w) {  // fixed order: reproducible
                num += s_sum[w][tid].x;
                den += s_sum[w][tid].y;
            }
            sc = __fmul_rn(sqrtf(num / (den + 1e-8f)), sc);
        }
        row_scale[row0 + tid] = sc;
    }
}


// ------------------------------------------------------- activations, one read of X ------------
// Persistent form of the dynamic (row maximum found in the data) case: X is read from HBM once.
// Each CTA owns a contiguous range of rows.  The producer warp streams them, one bulk copy per
// row, into row-sized shared-memory slots; `ng` groups of GW consumer warps take the rows in turn
// (row i of the CTA goes to group i % ng), each group cycling through slots of its own.  A group reads its row twice from shared memory: the maximum first (16-byte units, lanes
// consecutive), then 64-byte chunks of 32 elements per lane for selection, codes and metadata.
// While the consumers work the producer keeps the ring full, so the HBM stream never pauses for
// the second pass as it does when every CTA reads its rows twice in step with all the others.
//
// Shared-memory reads of pass 2: lane l owns chunk c = base + l (64-byte stride), and reads its
// four 16-byte pieces in the order (j + rot) % 4 with rot = (l / 2) % 4, which puts the eight
// lanes of a quarter warp on eight different 16-byte bank groups; the outputs (4 codes and one
// metadata byte per piece) are rotated back with selects before the stores.
#ifndef LYNX_FP8_RING_CW
#define LYNX_FP8_RING_CW 16
#endif
#ifndef LYNX_FP8_RING_UNROLL
#define LYNX_FP8_RING_UNROLL 1
#endif
constexpr int FP8_RING_CW = LYNX_FP8_RING_CW;                // consumer warps
constexpr int FP8_RING_UNROLL = LYNX_FP8_RING_UNROLL;        // chunks of pass 2 in flight per lane
constexpr int FP8_RING_THREADS = 32 * (FP8_RING_CW + 1);     // + the producer warp
constexpr int FP8_RING_MAX_SLOTS = 32;
constexpr int FP8_RING_HEADER = 1664;                        // barriers, tables, exchange words
constexpr int FP8_RING_SMEM_MAX = 227 * 1024;

//
// A waiter tells the phases of a barrier apart only when it is at most one phase away from it,
// and bulk copies issued in order may complete in any order.  So no slot is shared between
// groups: group g owns slots [first_g, first_g + cnt_g), cnt_g = slots / ng (+ 1 for the first
// slots % ng groups), and its n-th row uses its slot n % cnt_g.  The previous occupant of a row's
// slot was then a row of the same group, whose warps have waited for it themselves before they
// wait for this one.  (The host chooses GW, ng and slots; ng * GW <= FP8_RING_CW, ng <= slots.)
// GIVEN: the row maxima come from the caller and pass 1 is skipped.
template <bool SUMS, bool GIVEN, int GW>
__global__ void __launch_bounds__(FP8_RING_THREADS, 1)
prune_compress_fp8_ring_kernel(const uint16_t* __restrict__ X, int64_t M, int64_t K, int64_t ldx,
                               const float* __restrict__ row_amax, uint8_t* __restrict__ values_q, uint8_t* __restrict__ meta,
                               float* __restrict__ row_scale, int slots, int ng, uint32_t* dev_error) {
    extern __shared__ __align__(128) uint8_t ring_smem[];
    uint32_t* lut = reinterpret_cast<uint32_t*>(ring_smem + 512);
    uint32_t* s_top = reinterpret_cast<uint32_t*>(ring_smem + 768);   // [2][32]
    float2* s_sum = reinterpret_cast<float2*>(ring_smem + 1024);      // [2][32]
    volatile uint32_t* cta_abort = reinterpret_cast<volatile uint32_t*>(ring_smem + 1536);
    static_assert(FP8_RING_CW <= 32 && FP8_RING_CW % 4 == 0, "exchange arrays hold 32 warps");
    const uint32_t bar_full = smem_u32(ring_smem), bar_empty = bar_full + 8 * FP8_RING_MAX_SLOTS;
    const uint32_t data = smem_u32(ring_smem + FP8_RING_HEADER);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int NG = ng;                                     // active groups
    const int cnt_lo = slots / NG, cnt_rem = slots % NG;   // slots per group: cnt_lo (+ 1 for g < cnt_rem)

    if (tid < 64) lut[tid] = prune_lut_entry(tid & 15, tid >> 4);
    if (tid == 64) {
        for (int i = 0; i < slots; ++i) {
            mbar_init(bar_full + 8 * i, 1);
            mbar_init(bar_empty + 8 * i, GW);
        }
        *cta_abort = 0;
        fence_mbar_init();
    }
    __syncthreads();
    griddep_wait();

    // this CTA's rows
    const int64_t G = gridDim.x, b = blockIdx.x;
    const int64_t base = M / G, rem = M % G;
    const int64_t start = b * base + (b < rem ? b : rem);
    const int count = (int)(base + (b < rem ? 1 : 0));
    const uint32_t row_bytes = (uint32_t)(K * 2);
    const int kb128 = (int)(K / 128);

    if (warp == 0) {
        // ---------------------------------------------------------------- producer -------------
        // lane g feeds group g: its rows, its slots, in the group's own order (the lanes do not
        // wait for one another, so a slow group never holds up the loads of the others)
        if (lane < NG) {
            const int g = lane;
            const int cnt = cnt_lo + (g < cnt_rem ? 1 : 0);
            const int first = g * cnt_lo + (g < cnt_rem ? g : cnt_rem);
            bool ok = true;
            int issued = 0, ls = 0;
            uint32_t use = 0;
            for (int i = g; i < count; i += NG) {
                const int slot = first + ls;
                if (use > 0 && !mbar_wait(bar_empty + 8 * slot, (use - 1) & 1, cta_abort, dev_error)) {
                    ok = false;
                    break;
                }
                mbar_arrive_expect_tx(bar_full + 8 * slot, row_bytes);
                bulk_load(data + (uint32_t)slot * row_bytes, X + (start + i) * ldx, row_bytes, bar_full + 8 * slot);
                ++issued;
                if (++ls == cnt) { ls = 0; ++use; }
            }
            if (!ok && issued) bounded_delay_ns(200000);  // let the copies in flight land before teardown
        }
    } else {
        // ---------------------------------------------------------------- consumers ------------
        const int cw = warp - 1, g = cw / GW, wg = cw % GW, gl = wg * 32 + lane;
        // rows past M of the last 128-row block: legal metadata (pattern 0x4), spread over the grid
        {
            const int64_t pad_rows = ((M + 127) / 128) * 128 - M;
            const int64_t total = pad_rows * kb128;
            const uint4 fill = make_uint4(0x44444444u, 0x44444444u, 0x44444444u, 0x44444444u);
            for (int64_t idx = b * (FP8_RING_CW * 32) + (tid - 32); idx < total; idx += G * (FP8_RING_CW * 32)) {
                const int64_t pr = M + idx / kb128, kb = idx % kb128;
                *reinterpret_cast<uint4*>(meta + ((pr / 128) * kb128 + kb) * 2048 + (pr % 128) * 16) = fill;
            }
        }
        const int rot = (lane >> 1) & 3;
        uint32_t it = 0;
        const int cnt = cnt_lo + (g < cnt_rem ? 1 : 0);                 // this group's slots
        const int first = g * cnt_lo + (g < cnt_rem ? g : cnt_rem);
        int ls = 0;                                                     // local slot of the current row
        uint32_t use = 0;
        // a supplied row maximum is fetched one row ahead: its latency hides behind the row's work
        float amax_next = 0.0f;
        if (GIVEN && g < NG && g < count) amax_next = __ldg(row_amax + start + g);
        for (int i = g; g < NG && i < count; i += NG, ++it) {
            const float amax_given = amax_next;
            if (GIVEN && i + NG < count) amax_next = __ldg(row_amax + start + i + NG);
            const int slot = first + ls;
            bool ok = mbar_wait(bar_full + 8 * slot, use & 1, cta_abort, dev_error);
            const uint32_t sbase = data + (uint32_t)slot * row_bytes;
            // ---- pass 1: the row's largest magnitude
            uint32_t m = 0;
            if (ok && !GIVEN) {
                const int units = (int)(K / 8);
#pragma unroll 4
                for (int u = gl; u < units; u += 32 * GW) {
                    uint32_t a, bq, c, d;
                    lds128(sbase + (uint32_t)u * 16, a, bq, c, d);
                    m = absmax_bf16x2(m, absmax_bf16x2(absmax_bf16x2(a, bq), absmax_bf16x2(c, d)));
                }
            }
            // magnitudes compare as floats exactly as their 15 bits compare as integers; any NaN
            // in the row makes the maximum a NaN (as the largest 15-bit pattern would be one)
            m &= 0x7FFF7FFFu;
            uint32_t top = max(m & 0xFFFFu, m >> 16);
#pragma unroll
            for (int off = 16; off >= 1; off >>= 1) top = max(top, __shfl_xor_sync(0xffffffffu, top, off));
            if constexpr (GW > 1) {
                if (lane == 0) s_top[(it & 1) * 32 + cw] = top;
                ok = bar_red_and(1 + g, GW * 32, ok);
                top = 0;
#pragma unroll
                for (int w = 0; w < GW; ++w) top = max(top, s_top[(it & 1) * 32 + g * GW + w]);
            }
            if (!ok) break;
            const int64_t row = start + i;
            const float amax = GIVEN ? amax_given : __uint_as_float(top << 16);
            const float inv = amax > 0.0f ? __fdiv_rn(448.0f, amax) : 0.0f;
            const float act = __fdiv_rn(amax, 448.0f);

            // ---- pass 2: selection, codes, metadata, sums
            uint8_t* vrow = values_q + row * (K / 2);
            uint8_t* mrow = meta + ((row / 128) * kb128) * 2048 + (row % 128) * 16;
            float num = 0.f, den = 0.f;
            const int chunks = (int)(K / 32);
#pragma unroll FP8_RING_UNROLL
            for (int c = gl; c < chunks; c += 32 * GW) {
                const uint32_t addr = sbase + (uint32_t)c * 64;
                uint32_t A[8], B[8];
                lds128(addr + (((0 + rot) & 3) << 4), A[0], A[1], A[2], A[3]);
                lds128(addr + (((1 + rot) & 3) << 4), A[4], A[5], A[6], A[7]);
                lds128(addr + (((2 + rot) & 3) << 4), B[0], B[1], B[2], B[3]);
                lds128(addr + (((3 + rot) & 3) << 4), B[4], B[5], B[6], B[7]);
                uint32_t ka[4], kb[4];
                const uint32_t mA = prune_vec16(A, lut, ka);
                const uint32_t mB = prune_vec16(B, lut, kb);
                if constexpr (SUMS) {
#pragma unroll
                    for (int e = 0; e < 8; ++e) {
                        num = fma_sq_bf16x2(A[e], num);
                        num = fma_sq_bf16x2(B[e], num);
                    }
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        den = fma_sq_bf16x2(ka[e], den);
                        den = fma_sq_bf16x2(kb[e], den);
                    }
                }
                // codes of the four pieces, in the order they were read
                uint32_t q[4];
                q[0] = cvt_e4m3x2(__fmul_rn(bf16_lo_f(ka[0]), inv), __fmul_rn(bf16_hi_f(ka[0]), inv)) |
                       (cvt_e4m3x2(__fmul_rn(bf16_lo_f(ka[1]), inv), __fmul_rn(bf16_hi_f(ka[1]), inv)) << 16);
                q[1] = cvt_e4m3x2(__fmul_rn(bf16_lo_f(ka[2]), inv), __fmul_rn(bf16_hi_f(ka[2]), inv)) |
                       (cvt_e4m3x2(__fmul_rn(bf16_lo_f(ka[3]), inv), __fmul_rn(bf16_hi_f(ka[3]), inv)) << 16);
                q[2] = cvt_e4m3x2(__fmul_rn(bf16_lo_f(kb[0]), inv), __fmul_rn(bf16_hi_f(kb[0]), inv)) |
                       (cvt_e4m3x2(__fmul_rn(bf16_lo_f(kb[1]), inv), __fmul_rn(bf16_hi_f(kb[1]), inv)) << 16);
                q[3] = cvt_e4m3x2(__fmul_rn(bf16_lo_f(kb[2]), inv), __fmul_rn(bf16_hi_f(kb[2]), inv)) |
                       (cvt_e4m3x2(__fmul_rn(bf16_lo_f(kb[3]), inv), __fmul_rn(bf16_hi_f(kb[3]), inv)) << 16);
                // read slot j holds piece (j + rot) % 4: rotate back (selects, no indexed registers)
                const bool r1 = rot & 1, r2 = rot & 2;
                const uint32_t t0 = r1 ? q[3] : q[0], t1 = r1 ? q[0] : q[1], t2 = r1 ? q[1] : q[2], t3 = r1 ? q[2] : q[3];
                const uint32_t o0 = r2 ? t2 : t0, o1 = r2 ? t3 : t1, o2 = r2 ? t0 : t2, o3 = r2 ? t1 : t3;
                const uint32_t wslot = mA | (mB << 16);  // metadata byte j = read slot j
                const uint32_t w = __funnelshift_l(wslot, wslot, 8 * rot);
                stg128(vrow + (int64_t)c * 16, o0, o1, o2, o3);
                *reinterpret_cast<uint32_t*>(mrow + (int64_t)(c >> 2) * 2048 + (c & 3) * 4) = w;
            }
            // the slot may be refilled once every lane of this warp has read its chunks
            __syncwarp();
            if (lane == 0) mbar_arrive(bar_empty + 8 * slot);

            if constexpr (SUMS) {
#pragma unroll
                for (int off = 16; off >= 1; off >>= 1) {
                    num += __shfl_xor_sync(0xffffffffu, num, off);
                    den += __shfl_xor_sync(0xffffffffu, den, off);
                }
                if constexpr (GW > 1) {
                    if (lane == 0) s_sum[(it & 1) * 32 + cw] = make_float2(num, den);
                    bar_sync_named(1 + g, GW * 32);
                    num = 0.f;
                    den = 0.f;
#pragma unroll
                    for (int w = 0; w < GW; ++w) {  // fixed order: reproducible
                        const float2 v = s_sum[(it & 1) * 32 + g * GW + w];
                        num += v.x;
                        den += v.y;
                    }
                }
                if (gl == 0) row_scale[row] = __fmul_rn(sqrtf(num / (den + 1e-8f)), act);
            } else {
                if (gl == 0) row_scale[row] = act;
            }
            // next row of this group
            if (++ls == cnt) { ls = 0; ++use; }
        }
    }
}

}  // namespace lynx

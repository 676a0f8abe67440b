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

}  // namespace lynx

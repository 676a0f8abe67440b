// Online 2:4 sparsification (Algorithm 1 lines 3-4): Top-2-of-4 selection by magnitude,
// compression to (values, 2-bit index metadata in sparse-MMA order) and the per-row sums the
// norm-compensation scale needs -- one streaming pass over X.
//
// Work split: one CTA owns 16 rows (the row span of one 256-byte metadata slab); its warps take
// 128-element K blocks round-robin.  Inside a block a lane owns 32 consecutive elements of row
// r = lane/4 and of row r + 8, i.e. exactly the elements whose metadata make up the two 32-bit
// words this lane writes, so no metadata bit ever crosses lanes:
//     word(half h, lane) at slab byte h*128 + lane*4 = [row r : 16 bits][row r+8 : 16 bits]
// Loads and value stores are 32-byte vectors; 4 lanes cover 256 contiguous bytes of a row.
//
// Selection runs on pairs of groups with 16-bit lanes packed in 32-bit registers: the six
// "magnitude_i >= magnitude_j" comparisons (i < j) are borrow-free packed subtractions with a guard
// bit, the keep flags are bitwise majorities, and the kept positions come from a 16-entry table.
#pragma once

#include "ptx.cuh"

namespace lynx {

constexpr int PRUNE_ROWS = 16;
constexpr int PRUNE_WARPS = 8;
constexpr int PRUNE_THREADS = PRUNE_WARPS * 32;

// bitwise majority of three words
__device__ __forceinline__ uint32_t maj3(uint32_t a, uint32_t b, uint32_t c) {
    return (a & b) | (a & c) | (b & c);
}

// Keep patterns of two groups A = (a01, a23) and B = (b01, b23) (each register holds two bf16,
// lower index in the lower half).  Returns 4*pattern(A) in bits 0..15 and 4*pattern(B) in bits
// 16..31, where bit i of a pattern says element i is kept.
//
// Element i outranks element j (i < j) iff mag_i >= mag_j (ties go to the lower index); an
// element is kept iff fewer than two others outrank it.
__device__ __forceinline__ uint32_t keep_patterns_x2(uint32_t a01, uint32_t a23, uint32_t b01,
                                                     uint32_t b23) {
    const uint32_t MAG = 0x7FFF7FFFu, GUARD = 0x80008000u;
    // x_i = (A's element i, B's element i)
    const uint32_t x0 = prmt(a01, b01, 0x5410), x1 = prmt(a01, b01, 0x7632);
    const uint32_t x2 = prmt(a23, b23, 0x5410), x3 = prmt(a23, b23, 0x7632);
    const uint32_t g0 = (x0 & MAG) | GUARD, g1 = (x1 & MAG) | GUARD, g2 = (x2 & MAG) | GUARD;
    const uint32_t m1 = x1 & MAG, m2 = x2 & MAG, m3 = x3 & MAG;
    // bit 15 / bit 31 of (guard|mag_i) - mag_j is set iff mag_i >= mag_j; the guard bit keeps
    // every 16-bit lane positive so no borrow crosses lanes
    const uint32_t c01 = g0 - m1, c02 = g0 - m2, c03 = g0 - m3;
    const uint32_t c12 = g1 - m2, c13 = g1 - m3, c23 = g2 - m3;
    const uint32_t k0 = maj3(c01, c02, c03);     // not outranked by 1, 2, 3 (at least two of)
    const uint32_t k1 = maj3(~c01, c12, c13);    // not outranked by 0, 2, 3
    const uint32_t k2 = maj3(~c02, ~c12, c23);   // not outranked by 0, 1, 3
    const uint32_t k3 = maj3(~c03, ~c13, ~c23);  // not outranked by 0, 1, 2
    return ((k0 >> 13) & 0x00040004u) | ((k1 >> 12) & 0x00080008u) | ((k2 >> 11) & 0x00100010u) |
           ((k3 >> 10) & 0x00200020u);
}

// Table entry for a keep pattern with bits i0 < i1 set, copy j (j = position of the group's
// nibble in its 16-bit metadata word):  low 16 bits = byte-permute selector that packs elements
// i0, i1 into one register;  bits 16+4j.. = nibble i0 | i1 << 2.
__device__ __forceinline__ uint32_t prune_lut_entry(uint32_t pattern, int j) {
    if (__popc(pattern) != 2) return 0;
    const uint32_t i0 = __ffs(pattern) - 1, i1 = 31 - __clz(pattern);
    const uint32_t sel = (2 * i0) | ((2 * i0 + 1) << 4) | ((2 * i1) << 8) | ((2 * i1 + 1) << 12);
    return sel | ((i0 | (i1 << 2)) << (16 + 4 * j));
}

// One 32-byte vector = 16 consecutive elements = 4 groups -> 4 value registers + 16 metadata bits.
template <bool SUMS>
__device__ __forceinline__ uint32_t prune_vec16(const uint32_t (&r)[8], const uint32_t* lut,
                                                uint32_t* v /*[4]*/, float& num, float& den) {
    const uint32_t p01 = keep_patterns_x2(r[0], r[1], r[2], r[3]);
    const uint32_t p23 = keep_patterns_x2(r[4], r[5], r[6], r[7]);
    const char* base = reinterpret_cast<const char*>(lut);
    const uint32_t e0 = *reinterpret_cast<const uint32_t*>(base + 0 * 64 + (p01 & 0xFFFFu));
    const uint32_t e1 = *reinterpret_cast<const uint32_t*>(base + 1 * 64 + (p01 >> 16));
    const uint32_t e2 = *reinterpret_cast<const uint32_t*>(base + 2 * 64 + (p23 & 0xFFFFu));
    const uint32_t e3 = *reinterpret_cast<const uint32_t*>(base + 3 * 64 + (p23 >> 16));
    v[0] = prmt(r[0], r[1], e0);
    v[1] = prmt(r[2], r[3], e1);
    v[2] = prmt(r[4], r[5], e2);
    v[3] = prmt(r[6], r[7], e3);
    if constexpr (SUMS) {
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const float lo = bf16_lo_f(r[i]), hi = bf16_hi_f(r[i]);
            num = fmaf(lo, lo, num);
            num = fmaf(hi, hi, num);
        }
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const float lo = bf16_lo_f(v[i]), hi = bf16_hi_f(v[i]);
            den = fmaf(lo, lo, den);
            den = fmaf(hi, hi, den);
        }
    }
    return (e0 | e1 | e2 | e3) >> 16;
}

// mode: 0 none (row_scale written as 1 if non-null), 1 per-row scale, 2 partial sums for the
// whole-tensor scale (sums[2*m] = sum x^2, sums[2*m+1] = sum kept x^2).
template <bool SUMS>
__global__ void __launch_bounds__(PRUNE_THREADS)
prune_compress_kernel(const uint16_t* __restrict__ X, int64_t M, int64_t K, int64_t ldx,
                      uint16_t* __restrict__ values, uint8_t* __restrict__ meta,
                      float* __restrict__ row_scale, float* __restrict__ sums, int mode) {
    __shared__ uint32_t lut[4 * 16];
    __shared__ float red[PRUNE_WARPS][PRUNE_ROWS][2];
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    if (tid < 64) lut[tid] = prune_lut_entry(tid & 15, tid >> 4);
    __syncthreads();

    const int64_t row0 = (int64_t)blockIdx.x * PRUNE_ROWS;
    const int r = lane >> 2, q = lane & 3;
    const int64_t rowA = row0 + r, rowB = rowA + 8;
    const bool okA = rowA < M, okB = rowB < M;
    const int64_t kblocks = K / 128;
    // metadata slab of this CTA inside block (row0/128, kb)
    uint8_t* slab0 = meta + ((row0 / 128) * kblocks) * 2048 + ((row0 % 128) / 16) * 256 + lane * 4;
    const uint16_t* xa = X + rowA * ldx + q * 32;
    const uint16_t* xb = X + rowB * ldx + q * 32;
    uint16_t* va = values + rowA * (K / 2) + q * 16;
    uint16_t* vb = values + rowB * (K / 2) + q * 16;

    float numA = 0.f, denA = 0.f, numB = 0.f, denB = 0.f;
    for (int64_t kb = warp; kb < kblocks; kb += PRUNE_WARPS) {
        uint32_t a0[8] = {0, 0, 0, 0, 0, 0, 0, 0}, a1[8] = {0, 0, 0, 0, 0, 0, 0, 0};
        uint32_t b0[8] = {0, 0, 0, 0, 0, 0, 0, 0}, b1[8] = {0, 0, 0, 0, 0, 0, 0, 0};
        if (okA) {
            ldg256_stream(xa + kb * 128, a0);
            ldg256_stream(xa + kb * 128 + 16, a1);
        }
        if (okB) {
            ldg256_stream(xb + kb * 128, b0);
            ldg256_stream(xb + kb * 128 + 16, b1);
        }
        uint32_t oa[8], ob[8];
        const uint32_t ma0 = prune_vec16<SUMS>(a0, lut, oa, numA, denA);
        const uint32_t ma1 = prune_vec16<SUMS>(a1, lut, oa + 4, numA, denA);
        const uint32_t mb0 = prune_vec16<SUMS>(b0, lut, ob, numB, denB);
        const uint32_t mb1 = prune_vec16<SUMS>(b1, lut, ob + 4, numB, denB);
        if (okA) stg256(va + kb * 64, oa);
        if (okB) stg256(vb + kb * 64, ob);
        // rows past M prune to the pattern (0,1) = nibble 0x4, the documented padding
        uint32_t* slab = reinterpret_cast<uint32_t*>(slab0 + kb * 2048);
        slab[0] = ma0 | (mb0 << 16);
        slab[32] = ma1 | (mb1 << 16);
    }

    if constexpr (SUMS) {
        // the 4 lanes of a row, then the warps (fixed order: results are reproducible)
#pragma unroll
        for (int off = 1; off <= 2; off <<= 1) {
            numA += __shfl_xor_sync(0xffffffffu, numA, off);
            denA += __shfl_xor_sync(0xffffffffu, denA, off);
            numB += __shfl_xor_sync(0xffffffffu, numB, off);
            denB += __shfl_xor_sync(0xffffffffu, denB, off);
        }
        if (q == 0) {
            red[warp][r][0] = numA;
            red[warp][r][1] = denA;
            red[warp][r + 8][0] = numB;
            red[warp][r + 8][1] = denB;
        }
        __syncthreads();
        if (tid < PRUNE_ROWS && row0 + tid < M) {
            float num = 0.f, den = 0.f;
#pragma unroll
            for (int w = 0; w < PRUNE_WARPS; ++w) {
                num += red[w][tid][0];
                den += red[w][tid][1];
            }
            if (mode == 1) row_scale[row0 + tid] = sqrtf(num / (den + 1e-8f));
            else {
                sums[2 * (row0 + tid)] = num;
                sums[2 * (row0 + tid) + 1] = den;
            }
        }
    } else {
        if (row_scale != nullptr && tid < PRUNE_ROWS && row0 + tid < M) row_scale[row0 + tid] = 1.0f;
    }
}

// Whole-tensor scale: s = sqrt(sum_m num_m / (sum_m den_m + eps)), written to every row_scale[m].
// One CTA; fp64 partial sums in a fixed order.
__global__ void __launch_bounds__(1024)
tensor_scale_kernel(const float* __restrict__ sums, int64_t M, float* __restrict__ row_scale) {
    __shared__ double sn[1024], sd[1024];
    const int tid = threadIdx.x;
    double num = 0.0, den = 0.0;
    for (int64_t m = tid; m < M; m += 1024) {
        num += (double)sums[2 * m];
        den += (double)sums[2 * m + 1];
    }
    sn[tid] = num;
    sd[tid] = den;
    __syncthreads();
    for (int s = 512; s > 0; s >>= 1) {
        if (tid < s) {
            sn[tid] += sn[tid + s];
            sd[tid] += sd[tid + s];
        }
        __syncthreads();
    }
    const float sc = (float)sqrt(sn[0] / (sd[0] + 1e-8));
    for (int64_t m = tid; m < M; m += 1024) row_scale[m] = sc;
}

// ---- inspection helpers -------------------------------------------------------------------------

// hardware-order metadata -> canonical uint16 [M x K/16]
__global__ void meta_to_canonical_kernel(const uint8_t* __restrict__ meta, int64_t M, int64_t K,
                                         uint16_t* __restrict__ canon) {
    const int64_t words = K / 16;
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= M * words) return;
    const int64_t m = i / words, c = i % words;
    const int64_t rb = m / 128, r = m % 128, kb = c / 8, s = c % 8;
    const int64_t lane = (r % 8) + 8 * (s % 2) + 16 * (r / 16);
    const int64_t off = (rb * (K / 128) + kb) * 2048 + lane * 16 + (s / 2) * 4 + ((r / 8) % 2) * 2;
    canon[i] = *reinterpret_cast<const uint16_t*>(meta + off);
}

// (values, hardware-order metadata) -> masked dense X~ [M x K]; one thread per group of 4
__global__ void decompress_kernel(const uint16_t* __restrict__ values, const uint8_t* __restrict__ meta,
                                  int64_t M, int64_t K, uint16_t* __restrict__ out) {
    const int64_t groups = K / 4;
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= M * groups) return;
    const int64_t m = i / groups, g = i % groups;
    const int64_t c = g / 4;  // 16-element span
    const int64_t rb = m / 128, r = m % 128, kb = c / 8, s = c % 8;
    const int64_t lane = (r % 8) + 8 * (s % 2) + 16 * (r / 16);
    const int64_t off = (rb * (K / 128) + kb) * 2048 + lane * 16 + (s / 2) * 4 + ((r / 8) % 2) * 2;
    const uint32_t word = *reinterpret_cast<const uint16_t*>(meta + off);
    const uint32_t nib = (word >> (4 * (g % 4))) & 0xF;
    uint16_t o[4] = {0, 0, 0, 0};
    o[nib & 3] = values[m * (K / 2) + 2 * g];
    o[nib >> 2] = values[m * (K / 2) + 2 * g + 1];
    uint2 packed;
    packed.x = o[0] | ((uint32_t)o[1] << 16);
    packed.y = o[2] | ((uint32_t)o[3] << 16);
    *reinterpret_cast<uint2*>(out + m * K + 4 * g) = packed;
}

}  // namespace lynx

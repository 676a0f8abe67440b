// Online 2:4 sparsification (Algorithm 1 lines 3-4): Top-2-of-4 selection by magnitude,
// compression to (values, 2-bit index metadata in sparse-MMA order) and the per-row sums the
// norm-compensation scale needs -- one streaming pass over X.
//
// Work split: one warp owns 16 rows (the row span of one 256-byte metadata slab) and a run of
// 128-element K blocks.  Inside a block a lane owns 32 consecutive elements of row
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

// acc + lo^2 + hi^2 for the two bf16 halves of r: mixed-precision FMAs (bf16 x bf16 + fp32), the
// products are exact in fp32 and every add rounds once.
__device__ __forceinline__ float fma_sq_bf16x2(uint32_t r, float acc) {
    asm("{\n\t.reg .b16 lo, hi;\n\tmov.b32 {lo, hi}, %1;\n\t"
        "fma.rn.f32.bf16 %0, lo, lo, %0;\n\tfma.rn.f32.bf16 %0, hi, hi, %0;\n\t}"
        : "+f"(acc)
        : "r"(r));
    return acc;
}

__device__ __forceinline__ void write_scale_or_sums(int mode, int64_t m, float num, float den,
                                                    float* row_scale, float* sums) {
    if (mode == 1) row_scale[m] = sqrtf(num / (den + 1e-8f));
    else {
        sums[2 * m] = num;
        sums[2 * m + 1] = den;
    }
}

// Row scale from the per-K-split partial sums a deferred prune launch left behind:
// partial[(row / 16 * KS + ks) * 32 + 2 * (row % 16) + {0: sum x^2, 1: sum kept^2}].  Same order
// of additions as the in-kernel finalize (eight strided accumulators j = jl, jl + 8, ..., then
// those eight in ascending order), so both give the same bits.
__device__ __forceinline__ float row_scale_from_partials(const float* __restrict__ partial, int64_t row, int KS) {
    const float2* pp = reinterpret_cast<const float2*>(partial) + (row >> 4) * KS * 16 + (row & 15);
    float n[8], d[8];
#pragma unroll
    for (int jl = 0; jl < 8; ++jl) { n[jl] = 0.f; d[jl] = 0.f; }
    for (int j0 = 0; j0 < KS; j0 += 16) {  // 16 independent loads in flight per round
        float2 v[16];
#pragma unroll
        for (int u = 0; u < 16; ++u) v[u] = (j0 + u < KS) ? __ldcg(pp + (int64_t)(j0 + u) * 16) : make_float2(0.f, 0.f);
#pragma unroll
        for (int u = 0; u < 16; ++u)
            if (j0 + u < KS) { n[u & 7] += v[u].x; d[u & 7] += v[u].y; }
    }
    float num = 0.f, den = 0.f;
#pragma unroll
    for (int jl = 0; jl < 8; ++jl) { num += n[jl]; den += d[jl]; }
    return sqrtf(num / (den + 1e-8f));
}

// One 32-byte vector = 16 consecutive elements = 4 groups -> 4 value registers + 16 metadata bits.
__device__ __forceinline__ uint32_t prune_vec16(const uint32_t (&r)[8], const uint32_t* lut,
                                                uint32_t* v /*[4]*/) {
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
    return (e0 | e1 | e2 | e3) >> 16;
}

// Per-group norm compensation (the norm-compensation equation read literally, one s per group of
// four): v holds the group's two kept bf16 (lower index in the lower half), r01 / r23 its four
// elements.  fp32, IEEE operations, in this order:
// num = ((x0^2 + x1^2) + x2^2) + x3^2;  den = (k0^2 + k1^2) + 1e-8;
// s = sqrt(num / den);  result = bf16_rne(s * k0), bf16_rne(s * k1).
__device__ __forceinline__ uint32_t group_scale_pair(uint32_t r01, uint32_t r23, uint32_t v) {
    const float x0 = bf16_lo_f(r01), x1 = bf16_hi_f(r01), x2 = bf16_lo_f(r23), x3 = bf16_hi_f(r23);
    const float k0 = bf16_lo_f(v), k1 = bf16_hi_f(v);
    // (separately rounded products and sums, never fused: a square that underflows rounds the
    // same way on every machine)
    float num = __fmul_rn(x0, x0);
    num = __fadd_rn(num, __fmul_rn(x1, x1));
    num = __fadd_rn(num, __fmul_rn(x2, x2));
    num = __fadd_rn(num, __fmul_rn(x3, x3));
    float den = __fmul_rn(k0, k0);
    den = __fadd_rn(den, __fmul_rn(k1, k1));
    den = __fadd_rn(den, 1e-8f);
    const float sc = __fsqrt_rn(__fdiv_rn(num, den));
    return pack_bf16x2(__fmul_rn(sc, k0), __fmul_rn(sc, k1));
}

__device__ __forceinline__ void group_scale_vec16(const uint32_t (&r)[8], uint32_t* v /*[4]*/) {
#pragma unroll
    for (int g = 0; g < 4; ++g) v[g] = group_scale_pair(r[2 * g], r[2 * g + 1], v[g]);
}

// Work unit of one warp: 16 rows x (tiles_per_unit * 128) elements; the KS = kblocks /
// tiles_per_unit units of a 16-row block are independent warps (many small CTAs keep the SMs'
// load queues full).  With KS > 1 each unit writes its partial row sums
// (partial[(rb16*KS + ks)*32 + 2*row + {0: sum x^2, 1: sum kept x^2}]) and the last CTA of the row
// block to finish adds them in a fixed order, so the result does not depend on scheduling.
//
// mode: 0 none (row_scale written as 1 if non-null), 1 per-row scale, 2 per-row sums for the
// whole-tensor scale (sums[2*m] = sum x^2, sums[2*m+1] = sum kept x^2).  GROUP (with SUMS = false):
// the kept values are stored multiplied by their group's factor (group_scale_pair).
#ifndef LYNX_PRUNE_CTA_WARPS
#define LYNX_PRUNE_CTA_WARPS 4
#endif
#ifndef LYNX_PRUNE_MIN_CTAS
#define LYNX_PRUNE_MIN_CTAS 1
#endif
constexpr int PRUNE_CTA_WARPS = LYNX_PRUNE_CTA_WARPS;

// Results of one 16 x 128 tile held in registers until they are stored.
struct TileOut {
    uint32_t oa[8], ob[8];  // 16 kept values of row r / row r + 8
    uint32_t w0, w1;        // the lane's two metadata words
};

// Selection, compression and (SUMS) the row sums of one 16 x 128 tile whose elements are already in
// registers: a0 / a1 = elements 0..15 / 16..31 of this lane's 32-element slice of row r, b0 / b1 the
// same of row r + 8.
template <bool SUMS, bool GROUP = false>
__device__ __forceinline__ void prune_tile_core(const uint32_t (&a0)[8], const uint32_t (&a1)[8],
                                                const uint32_t (&b0)[8], const uint32_t (&b1)[8],
                                                const uint32_t* lut, TileOut& out, float& numA, float& denA,
                                                float& numB, float& denB) {
    const uint32_t ma0 = prune_vec16(a0, lut, out.oa);
    const uint32_t ma1 = prune_vec16(a1, lut, out.oa + 4);
    const uint32_t mb0 = prune_vec16(b0, lut, out.ob);
    const uint32_t mb1 = prune_vec16(b1, lut, out.ob + 4);
    if constexpr (GROUP) {
        group_scale_vec16(a0, out.oa);
        group_scale_vec16(a1, out.oa + 4);
        group_scale_vec16(b0, out.ob);
        group_scale_vec16(b1, out.ob + 4);
    }
    // rows past M prune to the pattern (0,1) = nibble 0x4, the documented padding
    out.w0 = ma0 | (mb0 << 16);
    out.w1 = ma1 | (mb1 << 16);
    if constexpr (SUMS) {
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            numA = fma_sq_bf16x2(a0[i], numA);
            numB = fma_sq_bf16x2(b0[i], numB);
        }
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            numA = fma_sq_bf16x2(a1[i], numA);
            numB = fma_sq_bf16x2(b1[i], numB);
        }
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            denA = fma_sq_bf16x2(out.oa[i], denA);
            denB = fma_sq_bf16x2(out.ob[i], denB);
        }
    }
}

template <bool SUMS, bool GUARD, bool GROUP = false>
__device__ __forceinline__ void prune_tile_compute(const uint16_t* xa, const uint16_t* xb, bool okA, bool okB,
                                                   const uint32_t* lut, TileOut& out, float& numA, float& denA,
                                                   float& numB, float& denB) {
    uint32_t a0[8], a1[8], b0[8], b1[8];
    if constexpr (GUARD) {
#pragma unroll
        for (int i = 0; i < 8; ++i) a0[i] = a1[i] = b0[i] = b1[i] = 0u;
        if (okA) {
            ldg256_stream(xa, a0);
            ldg256_stream(xa + 16, a1);
        }
        if (okB) {
            ldg256_stream(xb, b0);
            ldg256_stream(xb + 16, b1);
        }
    } else {
        ldg256_stream(xa, a0);
        ldg256_stream(xa + 16, a1);
        ldg256_stream(xb, b0);
        ldg256_stream(xb + 16, b1);
    }
    prune_tile_core<SUMS, GROUP>(a0, a1, b0, b1, lut, out, numA, denA, numB, denB);
}

__device__ __forceinline__ void prune_tile_store(const TileOut& out, uint16_t* va, uint16_t* vb, uint32_t* slab,
                                                 bool okA, bool okB) {
    if (okA) stg256(va, out.oa);
    if (okB) stg256(vb, out.ob);
    slab[0] = out.w0;
    slab[32] = out.w1;
}

template <bool SUMS, bool GROUP = false>
__global__ void __launch_bounds__(PRUNE_CTA_WARPS * 32, LYNX_PRUNE_MIN_CTAS)
prune_compress_kernel(const uint16_t* __restrict__ X, int64_t M, int64_t K, int64_t ldx,
                      uint16_t* __restrict__ values, uint8_t* __restrict__ meta,
                      float* __restrict__ row_scale, float* __restrict__ sums,
                      float* __restrict__ partial, uint32_t* __restrict__ tickets, int mode,
                      int tiles_per_unit, int KS, int ctas_per_rb, int defer) {
    __shared__ uint32_t lut[4 * 16];
    __shared__ float2 red[PRUNE_CTA_WARPS * 2][16];
    __shared__ uint32_t s_last;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    if (tid < 64) lut[tid] = prune_lut_entry(tid & 15, tid >> 4);
    __syncthreads();
    griddep_wait();  // no-op unless launched as a programmatic dependent of the previous kernel
    // the kernel behind this one (the sparse GEMM of a layer call, the scale finalize) may place its
    // CTAs and run its prologue -- barriers, tensor memory, descriptor prefetch -- while this grid works
    griddep_launch_dependents();

    // CTA -> 16-row block and its first K unit; the CTAs of a row block are consecutive
    const int64_t rb16 = blockIdx.x / ctas_per_rb;
    const int ks = (int)(blockIdx.x % ctas_per_rb) * PRUNE_CTA_WARPS + warp;
    const bool active = ks < KS;
    const int64_t row0 = rb16 * PRUNE_ROWS;
    const int r = lane >> 2, q = lane & 3;
    const int64_t rowA = row0 + r, rowB = rowA + 8;
    const int64_t kblocks = K / 128;
    float numA = 0.f, denA = 0.f, numB = 0.f, denB = 0.f;
    // The last tile's results stay in registers until after the row-sum hand-over below, so that
    // the fence of that hand-over does not have to wait for the big value stores.
    TileOut last;
    uint16_t *va = nullptr, *vb = nullptr;
    uint32_t* slab = nullptr;
    const bool full_rows = row0 + PRUNE_ROWS <= M;
    const bool okA = rowA < M, okB = rowB < M;
    if (active) {
        const int64_t kb0 = (int64_t)ks * tiles_per_unit;
        // metadata slab of this row block inside block (row0/128, kb)
        slab = reinterpret_cast<uint32_t*>(meta + ((row0 / 128) * kblocks + kb0) * 2048 +
                                           ((row0 % 128) / 16) * 256 + lane * 4);
        const uint16_t* xa = X + rowA * ldx + kb0 * 128 + q * 32;
        const uint16_t* xb = xa + 8 * ldx;
        va = values + rowA * (K / 2) + kb0 * 64 + q * 16;
        vb = va + 8 * (K / 2);
        for (int t = 0; t < tiles_per_unit; ++t) {
            if (full_rows)
                prune_tile_compute<SUMS, false, GROUP>(xa, xb, true, true, lut, last, numA, denA, numB, denB);
            else
                prune_tile_compute<SUMS, true, GROUP>(xa, xb, okA, okB, lut, last, numA, denA, numB, denB);
            if (t + 1 < tiles_per_unit) {
                prune_tile_store(last, va, vb, slab, okA, okB);
                xa += 128; xb += 128; va += 64; vb += 64; slab += 512;
            }
        }
    }

    if constexpr (SUMS) {
        // the 4 lanes of a row
#pragma unroll
        for (int off = 1; off <= 2; off <<= 1) {
            numA += __shfl_xor_sync(0xffffffffu, numA, off);
            denA += __shfl_xor_sync(0xffffffffu, denA, off);
            numB += __shfl_xor_sync(0xffffffffu, numB, off);
            denB += __shfl_xor_sync(0xffffffffu, denB, off);
        }
        if (defer) {
            // the consumer (the sparse GEMM's epilogue) adds the partial sums itself, in the order
            // row_scale_from_partials states: no ticket, no barrier, no fence here
            if (active) prune_tile_store(last, va, vb, slab, okA, okB);
            if (active && q == 0) {
                float* mine = partial + (rb16 * KS + ks) * 32;
                *reinterpret_cast<float2*>(mine + 2 * r) = make_float2(numA, denA);
                *reinterpret_cast<float2*>(mine + 2 * (r + 8)) = make_float2(numB, denB);
            }
            return;
        }
        if (KS == 1) {
            if (active) prune_tile_store(last, va, vb, slab, okA, okB);
            if (active && q == 0) {
                if (rowA < M) write_scale_or_sums(mode, rowA, numA, denA, row_scale, sums);
                if (rowB < M) write_scale_or_sums(mode, rowB, numB, denB, row_scale, sums);
            }
            return;
        }
        if (active && q == 0) {
            float* mine = partial + (rb16 * KS + ks) * 32;
            *reinterpret_cast<float2*>(mine + 2 * r) = make_float2(numA, denA);
            *reinterpret_cast<float2*>(mine + 2 * (r + 8)) = make_float2(numB, denB);
        }
        // The last CTA of the row block to get here adds all partial sums, in a fixed order.  One
        // thread takes the ticket for the whole CTA (the barrier makes the other warps' stores
        // its predecessors), so only its warp waits for the stores to drain.
        __syncthreads();
        if (tid == 0) {
            // release: this CTA's partial sums (ordered before by the barrier) are visible to whoever
            // reads a later ticket value; acquire: the last CTA sees every earlier CTA's sums
            const uint32_t t = atom_add_acq_rel_gpu(&tickets[rb16], 1u);
            s_last = (t == (uint32_t)(ctas_per_rb - 1)) ? 1u : 0u;
        }
        __syncthreads();
        if (active) prune_tile_store(last, va, vb, slab, okA, okB);
        if (!s_last) return;
        const int row = tid & 15, jl = tid >> 4;  // 16 rows x (PRUNE_CTA_WARPS * 2) strided sums
        const float2* pp = reinterpret_cast<const float2*>(partial) + rb16 * KS * 16 + row;
        float num = 0.f, den = 0.f;
        for (int j = jl; j < KS; j += PRUNE_CTA_WARPS * 2) {
            const float2 v = __ldcg(pp + j * 16);
            num += v.x;
            den += v.y;
        }
        red[jl][row] = make_float2(num, den);
        __syncthreads();
        if (tid < 16 && row0 + tid < M) {
            num = 0.f;
            den = 0.f;
#pragma unroll
            for (int j = 0; j < PRUNE_CTA_WARPS * 2; ++j) {
                num += red[j][tid].x;
                den += red[j][tid].y;
            }
            write_scale_or_sums(mode, row0 + tid, num, den, row_scale, sums);
        }
        if (tid == 0) tickets[rb16] = 0;  // ready for the next launch
    } else {
        if (active) prune_tile_store(last, va, vb, slab, okA, okB);
        if (row_scale != nullptr && ks == 0 && lane < 16 && row0 + lane < M) row_scale[row0 + lane] = 1.0f;
    }
}

// Row scale from the partial sums of a prune launch that stopped there (`defer`): one CTA of 128
// threads per 16-row block, thread (row, jl) adds the partial sums j = jl, jl + 8, ... and the eight
// strided sums of a row are then added in ascending order -- the additions of the in-kernel
// finalize in the same order (same bits), all loads of a thread in flight at once.  Launched right
// behind the prune kernel as a programmatic dependent.
__global__ void __launch_bounds__(128)
row_scale_finalize_kernel(const float* __restrict__ partial, int64_t M, int KS, float* __restrict__ row_scale) {
    __shared__ float2 red[8][16];
    griddep_wait();
    griddep_launch_dependents();
    const int tid = threadIdx.x, row = tid & 15, jl = tid >> 4;
    const int64_t rb16 = blockIdx.x, row0 = rb16 * 16;
    const float2* pp = reinterpret_cast<const float2*>(partial) + rb16 * KS * 16 + row;
    float num = 0.f, den = 0.f;
    for (int j = jl; j < KS; j += 8) {
        const float2 v = __ldcg(pp + j * 16);
        num += v.x;
        den += v.y;
    }
    red[jl][row] = make_float2(num, den);
    __syncthreads();
    if (tid < 16 && row0 + tid < M) {
        num = 0.f;
        den = 0.f;
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            num += red[j][tid].x;
            den += red[j][tid].y;
        }
        row_scale[row0 + tid] = sqrtf(num / (den + 1e-8f));
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

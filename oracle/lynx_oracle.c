/*
 * CPU oracle for the 2:4 activation-sparse linear layer (RT-Lynx, Algorithm 1 and
 * Algorithm 2 "activation_sparse" forward).
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the plain, slow, obviously-correct statement of
 * what the GPU library computes.  It shares no code, header, table or helper with the CUDA
 * path and must never be called from it.  Only the tests, the smoke check and the bench's
 * cpu-baseline / reference legs may build or call it.
 *
 * Conventions (same bytes the GPU gets):
 *   X  : M x K   bf16 bit patterns (uint16), row-major, leading dimension ldx (elements)
 *   W  : N x K   bf16, row-major, leading dimension ldw   (a torch Linear.weight)
 *   Y  : M x N   kept in fp32 here (the GPU rounds once to bf16 at the very end)
 *   groups of 4 consecutive elements along K start at k = 0.
 *
 * Pin status:
 *   selection / compression / decompression / metadata permutation : pinned (brute force,
 *       invariants, hand cases, round trips)
 *   GEMM + epilogue : pinned (fp64 GEMM on tiny shapes, library matmul on already-sparse X,
 *       exact integer-valued cases)
 *   norm-compensation scale : invariants only; the paper prints no numeric example, so its
 *       granularity reading (per token row) is "parity unpinned" beyond those invariants.
 */
#include <math.h>
#include <stddef.h>
#include <stdint.h>
#include <string.h>

#define ORACLE_API __attribute__((visibility("default")))

/* ---- bf16 helpers (bf16 = upper 16 bits of an IEEE fp32) ------------------------------ */

static float bf16_to_f32(uint16_t b) {
    uint32_t u = ((uint32_t)b) << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return f;
}

/* round-to-nearest-even fp32 -> bf16, NaN kept quiet */
ORACLE_API uint16_t oracle_f32_to_bf16(float f) {
    uint32_t u;
    memcpy(&u, &f, sizeof u);
    if ((u & 0x7fffffffu) > 0x7f800000u) return (uint16_t)((u >> 16) | 0x0040u);
    uint32_t lsb = (u >> 16) & 1u;
    u += 0x7fffu + lsb;
    return (uint16_t)(u >> 16);
}

ORACLE_API float oracle_bf16_to_f32(uint16_t b) { return bf16_to_f32(b); }

ORACLE_API void oracle_f32_to_bf16_array(const float* in, int64_t n, uint16_t* out) {
    for (int64_t i = 0; i < n; ++i) out[i] = oracle_f32_to_bf16(in[i]);
}

/* ---- Step 1: Top-2-of-4 selection (Algorithm 1 line 3; Algorithm 2 activation branch) - */

/* Magnitude used for ranking: the 15 non-sign bits compared as an integer.  This is a total
 * order in which NaN > Inf > finite, +0 == -0, subnormals rank by value (no flush).        */
static unsigned mag15(uint16_t b) { return b & 0x7fffu; }

/* element i outranks element j  <=>  larger magnitude, or equal magnitude and lower index */
static int outranks(const uint16_t g[4], int i, int j) {
    unsigned a = mag15(g[i]), b = mag15(g[j]);
    return a > b || (a == b && i < j);
}

/* Returns the two kept positions idx0 < idx1 of one group of four. */
static void select_group(const uint16_t g[4], int* idx0, int* idx1) {
    int kept[4];
    int n = 0;
    for (int i = 0; i < 4; ++i) {
        int beaten_by = 0; /* how many others outrank element i */
        for (int j = 0; j < 4; ++j)
            if (j != i && outranks(g, j, i)) ++beaten_by;
        kept[i] = beaten_by < 2; /* rank 0 or 1 -> one of the two largest */
        n += kept[i];
    }
    (void)n; /* always 2: "outranks" is a strict total order on the 4 positions */
    int first = -1, second = -1;
    for (int i = 0; i < 4; ++i)
        if (kept[i]) {
            if (first < 0) first = i;
            else second = i;
        }
    *idx0 = first;
    *idx1 = second;
}

/* mask[m*K + k] = 1 for kept positions, 0 for dropped ones. */
ORACLE_API void oracle_topk24_mask(const uint16_t* X, int64_t M, int64_t K, int64_t ldx,
                                   uint8_t* mask) {
    for (int64_t m = 0; m < M; ++m)
        for (int64_t g = 0; g < K / 4; ++g) {
            int i0, i1;
            select_group(X + m * ldx + 4 * g, &i0, &i1);
            for (int i = 0; i < 4; ++i) mask[m * K + 4 * g + i] = (uint8_t)(i == i0 || i == i1);
        }
}

/* ---- Step 2: compression (sparse-tensor-core appendix: A_nnz + 2-bit indices) --------- */

/* values[m, 2g+j] = X[m, 4g+idx_j] (bit copies);  nibble = idx0 | idx1 << 2.
 * Canonical metadata: one uint16 per 4 groups of a row, nibble (g mod 4) in bits
 * 4*(g mod 4) .. 4*(g mod 4)+3;  meta_canon is M x (K/16) uint16, row-major.            */
ORACLE_API void oracle_compress(const uint16_t* X, int64_t M, int64_t K, int64_t ldx,
                                uint16_t* values, uint16_t* meta_canon) {
    const int64_t G = K / 4;
    memset(meta_canon, 0, (size_t)(M * (K / 16)) * sizeof(uint16_t));
    for (int64_t m = 0; m < M; ++m)
        for (int64_t g = 0; g < G; ++g) {
            const uint16_t* grp = X + m * ldx + 4 * g;
            int i0, i1;
            select_group(grp, &i0, &i1);
            values[m * (K / 2) + 2 * g + 0] = grp[i0];
            values[m * (K / 2) + 2 * g + 1] = grp[i1];
            unsigned nib = (unsigned)i0 | ((unsigned)i1 << 2);
            meta_canon[m * (K / 16) + g / 4] |= (uint16_t)(nib << (4 * (g % 4)));
        }
}

/* ---- Per-group norm compensation: the literal reading of the norm-compensation equation,
 * which is written for one group X in R^{1x4}:  S(X) = s * X~,  s = sqrt(|X|^2 / (|X~|^2 + eps)),
 * eps = 1e-8, with one s per group of four.  A per-group factor cannot be applied after the
 * product, so it is folded into the stored values: values = bf16_rne(s_g * x_kept).  The paper
 * fixes no precision for s; the reading taken is fp32 with IEEE operations in this order
 * (squares of bf16 are exact in fp32, so each line rounds once):
 *   num = x0^2; num += x1^2; num += x2^2; num += x3^2;      (ascending index)
 *   den = k0^2; den += k1^2; den += eps;                     (the two kept, ascending index)
 *   s = sqrtf(num / den);   value_j = bf16_rne(s * k_j)
 * The mask and the metadata are those of oracle_compress.                                   */
ORACLE_API void oracle_compress_group_scaled(const uint16_t* X, int64_t M, int64_t K, int64_t ldx,
                                             uint16_t* values, uint16_t* meta_canon) {
    const int64_t G = K / 4;
    memset(meta_canon, 0, (size_t)(M * (K / 16)) * sizeof(uint16_t));
    for (int64_t m = 0; m < M; ++m)
        for (int64_t g = 0; g < G; ++g) {
            const uint16_t* grp = X + m * ldx + 4 * g;
            int i0, i1;
            select_group(grp, &i0, &i1);
            float x[4];
            for (int i = 0; i < 4; ++i) x[i] = bf16_to_f32(grp[i]);
            float num = x[0] * x[0];
            num = num + x[1] * x[1];
            num = num + x[2] * x[2];
            num = num + x[3] * x[3];
            float den = x[i0] * x[i0];
            den = den + x[i1] * x[i1];
            den = den + 1e-8f;
            const float sc = sqrtf(num / den);
            values[m * (K / 2) + 2 * g + 0] = oracle_f32_to_bf16(sc * x[i0]);
            values[m * (K / 2) + 2 * g + 1] = oracle_f32_to_bf16(sc * x[i1]);
            unsigned nib = (unsigned)i0 | ((unsigned)i1 << 2);
            meta_canon[m * (K / 16) + g / 4] |= (uint16_t)(nib << (4 * (g % 4)));
        }
}

/* The same factors in fp64, one per group (M x K/4): the check of the fp32 reading above. */
ORACLE_API void oracle_group_scale_f64(const uint16_t* X, int64_t M, int64_t K, int64_t ldx, double* s) {
    for (int64_t m = 0; m < M; ++m)
        for (int64_t g = 0; g < K / 4; ++g) {
            const uint16_t* grp = X + m * ldx + 4 * g;
            int i0, i1;
            select_group(grp, &i0, &i1);
            double num = 0.0, den = 0.0;
            for (int i = 0; i < 4; ++i) {
                double x = (double)bf16_to_f32(grp[i]);
                num += x * x;
                if (i == i0 || i == i1) den += x * x;
            }
            s[m * (K / 4) + g] = sqrt(num / (den + 1e-8));
        }
}

/* Step 3: scatter the kept values back; must reproduce mask (.) X bit for bit. */
ORACLE_API void oracle_decompress(const uint16_t* values, const uint16_t* meta_canon, int64_t M,
                                  int64_t K, uint16_t* Xmasked) {
    memset(Xmasked, 0, (size_t)(M * K) * sizeof(uint16_t));
    for (int64_t m = 0; m < M; ++m)
        for (int64_t g = 0; g < K / 4; ++g) {
            unsigned nib = (meta_canon[m * (K / 16) + g / 4] >> (4 * (g % 4))) & 0xfu;
            unsigned i0 = nib & 3u, i1 = nib >> 2;
            Xmasked[m * K + 4 * g + i0] = values[m * (K / 2) + 2 * g + 0];
            Xmasked[m * K + 4 * g + i1] = values[m * (K / 2) + 2 * g + 1];
        }
}

/* ---- Metadata order consumed by the 5th-generation sparse tensor core ------------------
 *
 * The sparse MMA of kind f16 takes, per 128-row x 32-element (logical K) step, one 32-bit
 * tensor-memory column over 128 lanes.  Written as "which bit of which lane" for row r
 * (0..127) and logical element k (0..31) of the step:
 *       lane = (r mod 8) + 8 * (k div 16) + 16 * (r div 16)
 *       bit  = (k mod 16) + 16 * ((r div 8) mod 2)
 * Four consecutive K steps (128 logical elements) fill four consecutive columns, i.e. 16
 * bytes per lane.  The stored form is those 128 lanes x 16 bytes = 2048 bytes per
 * (128-row block, 128-element K block), lane-major, column (K step) next, so that a plain
 * 128-lane x 128-bit shared-memory-to-tensor-memory copy puts every bit in place.
 * Blocks are ordered row-block major: block (rb, kb) starts at byte (rb*(K/128) + kb)*2048.
 * Rows beyond M inside the last row block hold the legal pattern 0x4 (positions 0,1).
 */
static int64_t hw_byte_offset(int64_t m, int64_t k16 /* index of a 16-element span */,
                              int64_t K) {
    int64_t rb = m / 128, r = m % 128;
    int64_t kb = k16 / 8, s = k16 % 8; /* 8 spans of 16 elements per 128-element block */
    int64_t step = s / 2, half = s % 2; /* K step of 32 elements; lower/upper 16 of it */
    int64_t lane = (r % 8) + 8 * half + 16 * (r / 16);
    int64_t within_lane = step * 4 + ((r / 8) % 2) * 2; /* byte inside the 16-byte lane row */
    return (rb * (K / 128) + kb) * 2048 + lane * 16 + within_lane;
}

ORACLE_API int64_t oracle_meta_hw_bytes(int64_t M, int64_t K) {
    return ((M + 127) / 128) * (K / 128) * 2048;
}

ORACLE_API void oracle_meta_canon_to_hw(const uint16_t* meta_canon, int64_t M, int64_t K,
                                        uint8_t* meta_hw) {
    const int64_t Mp = ((M + 127) / 128) * 128;
    for (int64_t m = 0; m < Mp; ++m)
        for (int64_t c = 0; c < K / 16; ++c) {
            uint16_t v = (m < M) ? meta_canon[m * (K / 16) + c] : (uint16_t)0x4444u;
            int64_t off = hw_byte_offset(m, c, K);
            meta_hw[off + 0] = (uint8_t)(v & 0xffu);
            meta_hw[off + 1] = (uint8_t)(v >> 8);
        }
}

ORACLE_API void oracle_meta_hw_to_canon(const uint8_t* meta_hw, int64_t M, int64_t K,
                                        uint16_t* meta_canon) {
    for (int64_t m = 0; m < M; ++m)
        for (int64_t c = 0; c < K / 16; ++c) {
            int64_t off = hw_byte_offset(m, c, K);
            meta_canon[m * (K / 16) + c] =
                (uint16_t)(meta_hw[off] | ((uint16_t)meta_hw[off + 1] << 8));
        }
}

/* ---- Step 4: norm-compensation scale (Algorithm 1 line 4; eps = 1e-8) ------------------
 * mode 0: s = 1.   mode 1: one s per token row.   mode 2: one s for the whole X.
 * s = sqrt( sum x^2 / (sum x~^2 + eps) ), sums in fp64, result rounded to fp32.          */
ORACLE_API void oracle_row_scale(const uint16_t* X, int64_t M, int64_t K, int64_t ldx, int mode,
                                 float* s) {
    const double eps = 1e-8;
    if (mode == 0 || mode == 3) { /* none; per-group factors live in the values, not here */
        for (int64_t m = 0; m < M; ++m) s[m] = 1.0f;
        return;
    }
    double num_all = 0.0, den_all = 0.0;
    for (int64_t m = 0; m < M; ++m) {
        double num = 0.0, den = 0.0;
        for (int64_t g = 0; g < K / 4; ++g) {
            const uint16_t* grp = X + m * ldx + 4 * g;
            int i0, i1;
            select_group(grp, &i0, &i1);
            for (int i = 0; i < 4; ++i) {
                double x = (double)bf16_to_f32(grp[i]);
                num += x * x;
                if (i == i0 || i == i1) den += x * x;
            }
        }
        if (mode == 1) s[m] = (float)sqrt(num / (den + eps));
        num_all += num;
        den_all += den;
    }
    if (mode == 2) {
        float sa = (float)sqrt(num_all / (den_all + eps));
        for (int64_t m = 0; m < M; ++m) s[m] = sa;
    }
}

/* ---- Step 5: the product, fp32 accumulation, k ascending (Algorithm 1 line 5) ---------- */

/* rows: optional list of n_rows row indices to compute (NULL = all M rows, n_rows = M).
 * acc is n_rows x N fp32.  Dense loop over the masked X: dropped positions contribute
 * literal zeros.                                                                          */
ORACLE_API void oracle_gemm_masked_f32(const uint16_t* Xmasked, int64_t K, const uint16_t* W,
                                       int64_t N, int64_t ldw, const int64_t* rows,
                                       int64_t n_rows, float* acc) {
#pragma omp parallel for schedule(dynamic, 1)
    for (int64_t r = 0; r < n_rows; ++r) {
        const int64_t m = rows ? rows[r] : r;
        for (int64_t n = 0; n < N; ++n) {
            float a = 0.0f;
            for (int64_t k = 0; k < K; ++k)
                a += bf16_to_f32(Xmasked[m * K + k]) * bf16_to_f32(W[n * ldw + k]);
            acc[r * N + n] = a;
        }
    }
}

/* Same sum taken over the compressed form: only kept positions, still k ascending. */
ORACLE_API void oracle_gemm_sparse_f32(const uint16_t* values, const uint16_t* meta_canon,
                                       int64_t K, const uint16_t* W, int64_t N, int64_t ldw,
                                       const int64_t* rows, int64_t n_rows, float* acc) {
#pragma omp parallel for schedule(dynamic, 1)
    for (int64_t r = 0; r < n_rows; ++r) {
        const int64_t m = rows ? rows[r] : r;
        for (int64_t n = 0; n < N; ++n) {
            float a = 0.0f;
            for (int64_t g = 0; g < K / 4; ++g) {
                unsigned nib = (meta_canon[m * (K / 16) + g / 4] >> (4 * (g % 4))) & 0xfu;
                unsigned i0 = nib & 3u, i1 = nib >> 2;
                a += bf16_to_f32(values[m * (K / 2) + 2 * g + 0]) *
                     bf16_to_f32(W[n * ldw + 4 * g + i0]);
                a += bf16_to_f32(values[m * (K / 2) + 2 * g + 1]) *
                     bf16_to_f32(W[n * ldw + 4 * g + i1]);
            }
            acc[r * N + n] = a;
        }
    }
}

/* fp64-accumulated variant (tiny shapes; bounds the fp32 oracle's own rounding error). */
ORACLE_API void oracle_gemm_masked_f64(const uint16_t* Xmasked, int64_t M, int64_t K,
                                       const uint16_t* W, int64_t N, int64_t ldw, double* acc) {
    for (int64_t m = 0; m < M; ++m)
        for (int64_t n = 0; n < N; ++n) {
            double a = 0.0;
            for (int64_t k = 0; k < K; ++k)
                a += (double)bf16_to_f32(Xmasked[m * K + k]) * (double)bf16_to_f32(W[n * ldw + k]);
            acc[m * N + n] = a;
        }
}

/* ---- Step 6: epilogue  Y = s_m * acc + bias_n + Yr[m,n], kept in fp32 -------------------
 * (scale: Algorithm 1 line 4 moved behind the product, exact for a per-row scalar;
 *  bias: Algorithm 2; residual: Algorithm 1 line 6).  NULL terms are absent.            */
ORACLE_API void oracle_epilogue(const float* acc, int64_t N, const int64_t* rows, int64_t n_rows,
                                const float* s, const uint16_t* bias, const uint16_t* Yr,
                                int64_t ldr, float* Y) {
    for (int64_t r = 0; r < n_rows; ++r) {
        const int64_t m = rows ? rows[r] : r;
        for (int64_t n = 0; n < N; ++n) {
            float y = acc[r * N + n];
            if (s) y = s[m] * y;
            if (bias) y = y + bf16_to_f32(bias[n]);
            if (Yr) y = y + bf16_to_f32(Yr[m * ldr + n]);
            Y[r * N + n] = y;
        }
    }
}

/* ---- Step 7: LoRA residual on the DENSE X (Algorithm 1 lines 5-6: Y_r = X (L_A L_B)^T) ----
 * Yr = (X L_B^T) L_A^T, L_B is R x K, L_A is N x R, all bf16, fp32 accumulation, nothing
 * rounded in between.  Computed for the rows listed in `rows` (NULL = all M rows, in order);
 * Yr is n_rows x N.                                                                        */
ORACLE_API void oracle_lora_residual_rows(const uint16_t* X, int64_t M, int64_t K, int64_t ldx,
                                          const uint16_t* LB, int64_t R, const uint16_t* LA, int64_t N,
                                          const int64_t* rows, int64_t n_rows, float* Yr) {
    if (!rows) n_rows = M;
#pragma omp parallel for schedule(dynamic, 1)
    for (int64_t i = 0; i < n_rows; ++i) {
        const int64_t m = rows ? rows[i] : i;
        float t[512];
        for (int64_t r = 0; r < R && r < 512; ++r) {
            float a = 0.0f;
            for (int64_t k = 0; k < K; ++k)
                a += bf16_to_f32(X[m * ldx + k]) * bf16_to_f32(LB[r * K + k]);
            t[r] = a;
        }
        for (int64_t n = 0; n < N; ++n) {
            float a = 0.0f;
            for (int64_t r = 0; r < R && r < 512; ++r) a += t[r] * bf16_to_f32(LA[n * R + r]);
            Yr[i * N + n] = a;
        }
    }
}

ORACLE_API void oracle_lora_residual(const uint16_t* X, int64_t M, int64_t K, int64_t ldx,
                                     const uint16_t* LB, int64_t R, const uint16_t* LA, int64_t N,
                                     float* Yr) {
    oracle_lora_residual_rows(X, M, K, ldx, LB, R, LA, N, NULL, M, Yr);
}

/* ---- Algorithm 1 line 6 with the LoRA branch kept in fp32: Y += Y_r -----------------------
 * Y and lora are n_rows x N; the sum is one fp32 addition per element.                     */
ORACLE_API void oracle_add_lora(float* Y, const float* lora, int64_t n_rows, int64_t N) {
    for (int64_t i = 0; i < n_rows * N; ++i) Y[i] = Y[i] + lora[i];
}

/* ---- Whole path for a set of rows: steps 1, 2, 4, 5, 6 in that order -------------------
 * Writes values / meta_canon for ALL rows (cheap), Y only for the requested rows.
 * values, meta_canon may be NULL if the caller only wants Y.                              */
ORACLE_API void oracle_act_sparse_linear(const uint16_t* X, int64_t M, int64_t K, int64_t ldx,
                                         const uint16_t* W, int64_t N, int64_t ldw,
                                         const uint16_t* bias, int comp_mode, const uint16_t* Yr,
                                         int64_t ldr, const int64_t* rows, int64_t n_rows,
                                         uint16_t* values, uint16_t* meta_canon, float* scale_out,
                                         uint16_t* xmasked_scratch, float* acc_scratch, float* Y) {
    if (comp_mode == 3) oracle_compress_group_scaled(X, M, K, ldx, values, meta_canon);
    else oracle_compress(X, M, K, ldx, values, meta_canon);
    oracle_decompress(values, meta_canon, M, K, xmasked_scratch);
    oracle_row_scale(X, M, K, ldx, comp_mode, scale_out);
    oracle_gemm_masked_f32(xmasked_scratch, K, W, N, ldw, rows, n_rows, acc_scratch);
    oracle_epilogue(acc_scratch, N, rows, n_rows, (comp_mode == 1 || comp_mode == 2) ? scale_out : NULL, bias, Yr,
                    ldr, Y);
}

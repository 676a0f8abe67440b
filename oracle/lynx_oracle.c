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
#include <stdlib.h>
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

/* ======================================================================================== *
 * FP8 composition (the paper's W8A8 compatibility experiment: symmetric FP8 quantisation of
 * the activations, weights cast to FP8, the 2:4 pattern on FP8 operands).
 *
 * FP8 here is E4M3 in the OCP "FN" flavour: 1 sign, 4 exponent bits (bias 7), 3 mantissa bits,
 * no infinities, S.1111.111 is NaN, largest finite 448, smallest subnormal 2^-9.
 * The paper fixes neither the granularity of the activation scale nor any rounding; the
 * reading taken (and restated in the CUDA library's header) is:
 *   selection      on the bf16 activations, as everywhere else (the mask does not change);
 *   activation     per token row m: amax_m = the largest magnitude of the row in the order the
 *                  selection uses (the 15 non-sign bits as an integer: NaN > Inf > finite), so it
 *                  is also the largest kept magnitude, and a NaN in the row makes the row's
 *                  scale NaN (it propagates to Y as in a dense layer),
 *                  inv_m = 448 / amax_m (fp32 division; 0 if amax_m = 0),
 *                  code = e4m3_rne_satfinite(x~ * inv_m)  (fp32 product, then one rounding),
 *                  act_scale_m = amax_m / 448 (fp32 division);
 *   weights        "direct": code = e4m3_rne_satfinite(w), w_scale_n = 1; or per output channel:
 *                  the same symmetric rule over row n of W;
 *   product        fp32 accumulation of the decoded codes;
 *   epilogue       y = (s_m * act_scale_m) * w_scale_n * acc + bias + Y_r, s_m the per-row norm
 *                  compensation of the bf16 activations (1 in mode none).
 * ======================================================================================== */

ORACLE_API float oracle_e4m3_decode(uint8_t c) {
    const int sign = c >> 7, e = (c >> 3) & 0xf, m = c & 7;
    float v;
    if (e == 0xf && m == 7) v = NAN;
    else if (e == 0) v = ldexpf((float)m, -9);              /* subnormal: m * 2^-9 */
    else v = ldexpf((float)(8 + m), e - 7 - 3);             /* (1 + m/8) * 2^(e-7) */
    return sign ? -v : v;
}

/* fp32 -> E4M3, round to nearest even, finite overflow (and +-Inf) saturates to +-448, NaN -> 0x7f | sign */
ORACLE_API uint8_t oracle_e4m3_encode(float f) {
    uint32_t u;
    memcpy(&u, &f, sizeof u);
    const uint8_t sign = (uint8_t)((u >> 24) & 0x80u);
    if ((u & 0x7fffffffu) > 0x7f800000u) return (uint8_t)(sign | 0x7fu);
    const float a = fabsf(f);
    if (!(a < 464.0f)) return (uint8_t)(sign | 0x7eu);       /* >= halfway between 448 and 480: max finite */
    /* the E4M3 grid around a: spacing 2^(e-3) for normal exponents e = floor(log2 a) >= -6, 2^-9 below */
    int e;
    (void)frexpf(a, &e);                                      /* a = f * 2^e, f in [0.5, 1) */
    int ex = e - 1;                                           /* floor(log2 a) for a > 0 */
    if (a == 0.0f || ex < -6) ex = -6;
    const float step = ldexpf(1.0f, ex - 3);
    /* a / step is exact (power-of-two scaling of a number with more bits than needed is only
     * exact when no bits fall off the bottom: a has 24 bits, the quotient is < 16, so bits can
     * fall off only below 2^-20 of a unit -- rintf sees the exact value's neighbourhood; to stay
     * exact the quotient is formed in double) */
    const double q = (double)a / (double)step;
    double r = nearbyint(q);                                  /* current mode: to nearest even */
    if (r * (double)step > 448.0) r = 448.0 / (double)step;   /* cannot happen after the 464 test; kept for clarity */
    const float qv = (float)(r * (double)step);               /* the rounded magnitude, exactly representable */
    /* encode qv */
    if (qv == 0.0f) return sign;
    int e2;
    const float fr = frexpf(qv, &e2);                         /* qv = fr * 2^e2, fr in [0.5,1) */
    int ee = e2 - 1;                                          /* floor(log2 qv) */
    uint8_t code;
    if (ee < -6) code = (uint8_t)lrintf(ldexpf(qv, 9));       /* subnormal: m = qv * 2^9 */
    else code = (uint8_t)(((ee + 7) << 3) | ((int)lrintf(ldexpf(fr, 4)) - 8)); /* fr*2 in [1,2): m = (fr*2 - 1) * 8 */
    return (uint8_t)(sign | code);
}

ORACLE_API void oracle_e4m3_encode_array(const float* in, int64_t n, uint8_t* out) {
    for (int64_t i = 0; i < n; ++i) out[i] = oracle_e4m3_encode(in[i]);
}

/* Metadata order of the FP8 (kind f8f6f4) sparse MMA: one instruction covers 64 logical K and
 * reads, for row r of its 128 rows, 64 metadata bits from tensor-memory lane r in natural order
 * (nibble of group g in bits 4g..4g+3).  Stored as blocks of 128 rows x 128 K-elements, 2048 bytes
 * each, block (rb, kb) at byte (rb * K/128 + kb) * 2048; inside a block byte = r * 16 + g / 2 with
 * r = row in block, g = (k % 128) / 4, group g in bits 4 * (g % 2) of that byte.  Rows past M in
 * the last block carry the legal pattern 0x4. */
ORACLE_API void oracle_meta_canon_to_hw_fp8(const uint16_t* meta_canon, int64_t M, int64_t K, uint8_t* meta_hw) {
    const int64_t RB = (M + 127) / 128, KB = K / 128;
    memset(meta_hw, 0x44, (size_t)(RB * KB * 2048));
    for (int64_t m = 0; m < M; ++m)
        for (int64_t g = 0; g < K / 4; ++g) {
            const unsigned nib = (meta_canon[m * (K / 16) + g / 4] >> (4 * (g % 4))) & 0xfu;
            const int64_t rb = m / 128, r = m % 128, kb = (4 * g) / 128, gl = g % 32;
            uint8_t* byte = meta_hw + (rb * KB + kb) * 2048 + r * 16 + gl / 2;
            *byte = (uint8_t)((*byte & ~(0xfu << (4 * (gl % 2)))) | (nib << (4 * (gl % 2))));
        }
}

/* Weights: mode 0 direct cast, 1 symmetric per output channel.  Wq is N x K codes, wscale N floats. */
ORACLE_API void oracle_quantize_weights_fp8(const uint16_t* W, int64_t N, int64_t K, int64_t ldw, int mode,
                                            uint8_t* Wq, float* wscale) {
    for (int64_t n = 0; n < N; ++n) {
        float inv = 1.0f, sc = 1.0f;
        if (mode == 1) {
            unsigned top = 0;
            for (int64_t k = 0; k < K; ++k)
                if (mag15(W[n * ldw + k]) > top) top = mag15(W[n * ldw + k]);
            const float amax = bf16_to_f32((uint16_t)top);
            inv = amax > 0.0f ? 448.0f / amax : 0.0f;          /* 0 for amax = 0 and for NaN */
            sc = amax / 448.0f;
        }
        for (int64_t k = 0; k < K; ++k) Wq[n * K + k] = oracle_e4m3_encode(bf16_to_f32(W[n * ldw + k]) * inv);
        wscale[n] = sc;
    }
}

/* Activations: Top-2-of-4 on the bf16 values, then per-row symmetric FP8 codes of the kept ones.
 * values_q [M x K/2] codes, meta_canon as oracle_compress, act_scale [M].
 * row_amax: NULL = the row maximum is taken from the data; else row_amax[m] is used in its place
 * (a scale calibrated beforehand, or a maximum the producer of X already knows); values beyond
 * it saturate. */
ORACLE_API void oracle_compress_fp8(const uint16_t* X, int64_t M, int64_t K, int64_t ldx, const float* row_amax,
                                    uint8_t* values_q, uint16_t* meta_canon, float* act_scale) {
    const int64_t G = K / 4;
    memset(meta_canon, 0, (size_t)(M * (K / 16)) * sizeof(uint16_t));
    for (int64_t m = 0; m < M; ++m) {
        unsigned top = 0;
        for (int64_t k = 0; k < K; ++k)
            if (mag15(X[m * ldx + k]) > top) top = mag15(X[m * ldx + k]);
        const float amax = row_amax ? row_amax[m] : bf16_to_f32((uint16_t)top);
        const float inv = amax > 0.0f ? 448.0f / amax : 0.0f;  /* 0 for amax = 0 and for NaN */
        act_scale[m] = amax / 448.0f;
        for (int64_t g = 0; g < G; ++g) {
            const uint16_t* grp = X + m * ldx + 4 * g;
            int i0, i1;
            select_group(grp, &i0, &i1);
            values_q[m * (K / 2) + 2 * g + 0] = oracle_e4m3_encode(bf16_to_f32(grp[i0]) * inv);
            values_q[m * (K / 2) + 2 * g + 1] = oracle_e4m3_encode(bf16_to_f32(grp[i1]) * inv);
            unsigned nib = (unsigned)i0 | ((unsigned)i1 << 2);
            meta_canon[m * (K / 16) + g / 4] |= (uint16_t)(nib << (4 * (g % 4)));
        }
    }
}

/* Product of the decoded codes, fp32 accumulation, k ascending, for the listed rows. */
ORACLE_API void oracle_gemm_fp8_f32(const uint8_t* values_q, const uint16_t* meta_canon, int64_t M, int64_t K,
                                    const uint8_t* Wq, int64_t N, const int64_t* rows, int64_t n_rows, float* acc) {
    if (!rows) n_rows = M;
#pragma omp parallel for schedule(dynamic, 1)
    for (int64_t i = 0; i < n_rows; ++i) {
        const int64_t m = rows ? rows[i] : i;
        float* xrow = (float*)malloc((size_t)K * sizeof(float));
        for (int64_t k = 0; k < K; ++k) xrow[k] = 0.0f;
        for (int64_t g = 0; g < K / 4; ++g) {
            unsigned nib = (meta_canon[m * (K / 16) + g / 4] >> (4 * (g % 4))) & 0xfu;
            xrow[4 * g + (nib & 3u)] = oracle_e4m3_decode(values_q[m * (K / 2) + 2 * g + 0]);
            xrow[4 * g + (nib >> 2)] = oracle_e4m3_decode(values_q[m * (K / 2) + 2 * g + 1]);
        }
        for (int64_t n = 0; n < N; ++n) {
            float a = 0.0f;
            for (int64_t k = 0; k < K; ++k) a += xrow[k] * oracle_e4m3_decode(Wq[n * K + k]);
            acc[i * N + n] = a;
        }
        free(xrow);
    }
}

/* Whole FP8 path for a set of rows.  comp_mode: 0 none, 1 per-row norm compensation.
 * row_scale_out[m] = s_m * act_scale_m (what the epilogue multiplies row m by). */
ORACLE_API void oracle_act_sparse_linear_fp8(const uint16_t* X, int64_t M, int64_t K, int64_t ldx,
                                             const float* row_amax, const uint8_t* Wq, const float* wscale, int64_t N,
                                             const uint16_t* bias, int comp_mode, const uint16_t* Yr, int64_t ldr,
                                             const int64_t* rows, int64_t n_rows, uint8_t* values_q,
                                             uint16_t* meta_canon, float* row_scale_out, float* acc_scratch,
                                             float* Y) {
    float* act = (float*)malloc((size_t)M * sizeof(float));
    float* s = (float*)malloc((size_t)M * sizeof(float));
    oracle_compress_fp8(X, M, K, ldx, row_amax, values_q, meta_canon, act);
    oracle_row_scale(X, M, K, ldx, comp_mode == 1 ? 1 : 0, s);
    for (int64_t m = 0; m < M; ++m) row_scale_out[m] = s[m] * act[m];
    oracle_gemm_fp8_f32(values_q, meta_canon, M, K, Wq, N, rows, n_rows, acc_scratch);
    if (!rows) n_rows = M;
    for (int64_t i = 0; i < n_rows; ++i) {
        const int64_t m = rows ? rows[i] : i;
        for (int64_t n = 0; n < N; ++n) {
            float y = row_scale_out[m] * wscale[n] * acc_scratch[i * N + n];
            if (bias) y = y + bf16_to_f32(bias[n]);
            if (Yr) y = y + bf16_to_f32(Yr[m * ldr + n]);
            Y[i * N + n] = y;
        }
    }
    free(act);
    free(s);
}

/*
 * lynx.h -- C ABI of the B200 (sm_100a) 2:4 activation-sparse linear layer.
 *
 * The library computes the hot path of RT-Lynx (Algorithm 1; Algorithm 2, activation_sparse
 * branch): each token row of X is pruned along K to 2:4 sparsity by Top-2-of-4 magnitude,
 * compressed to (values, 2-bit index metadata), multiplied by dense bf16 weights on the sparse
 * tensor cores, and finished by an epilogue that applies the norm-compensation scale, the bias
 * and an optional residual (the low-rank branch output Y_r) before one cast to bf16.
 *
 * General rules for every entry point
 *   - Pointers are DEVICE pointers unless the argument is documented as HOST.
 *   - The caller owns every buffer it passes; the library never frees or resizes them and never
 *     modifies inputs.  Scratch memory belongs to the context (lynx_ctx).
 *   - All work is enqueued on `stream` (a cudaStream_t passed as void*; NULL = default stream)
 *     and returns without synchronising, except the *_host entry point which synchronises the
 *     stream before returning.
 *   - Errors are return values; nothing throws and nothing aborts.  Argument errors are found on
 *     the host before any launch.  A device-side wait that ran out (should never happen) is
 *     reported as LYNX_ERR_TIMEOUT by the next call on the same context or by lynx_last_error.
 *   - Layouts: X is M x K bf16 row-major with leading dimension ldx (elements); W is N x K bf16
 *     row-major (a Linear weight, D_out x D_in) with leading dimension ldw; Y is M x N bf16
 *     row-major with leading dimension ldy; bias is N bf16; residual is M x N bf16, ld = ldr.
 *   - Shape rules: M >= 1, K % 128 == 0, N % 8 == 0; base pointers and leading dimensions must be
 *     16-byte aligned (ld % 8 == 0 for bf16).  Row tails (M not a multiple of the tile) are
 *     handled inside the kernels.
 *   - A context belongs to one device, and that device must be the calling thread's current
 *     device (cudaSetDevice) whenever the context is used; lynx_create makes it current.
 *   - There is no CPU fallback: on a device that is not sm_100 lynx_create fails with
 *     LYNX_ERR_UNSUPPORTED_ARCH.
 */
#ifndef LYNX_H_
#define LYNX_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#if defined(__GNUC__)
#define LYNX_API __attribute__((visibility("default")))
#else
#define LYNX_API
#endif

typedef struct lynx_ctx lynx_ctx; /* opaque: scratch workspace, descriptor cache, error word */

typedef enum {
    LYNX_OK = 0,
    LYNX_ERR_INVALID_ARG = 1,
    LYNX_ERR_UNSUPPORTED_SHAPE = 2,
    LYNX_ERR_ALIGNMENT = 3,
    LYNX_ERR_WORKSPACE = 4,
    LYNX_ERR_CUDA = 5,
    LYNX_ERR_TIMEOUT = 6,
    LYNX_ERR_UNSUPPORTED_ARCH = 7
} lynx_status;

/* Norm compensation of Algorithm 1 line 4:  s = sqrt(||X||^2 / (||X~||^2 + 1e-8)). */
typedef enum {
    LYNX_COMP_NONE = 0,  /* no rescaling: y = x~ W^T + b  (Algorithm 2, activation_sparse)   */
    LYNX_COMP_ROW = 1,   /* one s per token row (the reading used by default)                */
    LYNX_COMP_TENSOR = 2, /* one s for the whole X (Algorithm 1 read literally)              */
    LYNX_COMP_GROUP = 3   /* one s per group of four (the norm-compensation equation read
                             literally): folded into the stored values, see lynx_prune_compress */
} lynx_comp_mode;

typedef enum {
    LYNX_FUSE_AUTO = 0,     /* library picks                                                  */
    LYNX_FUSE_SEPARATE = 1, /* prune/compress kernel, then sparse GEMM kernel                 */
    LYNX_FUSE_FUSED = 2     /* one kernel, compressed activations never written to HBM        */
} lynx_fuse_mode;

/* "Deferred" row scale for the two-call form (what lynx_act_sparse_linear does internally in
 * LYNX_COMP_ROW mode): pass this value as `row_scale` to lynx_prune_compress and the kernel stops
 * at its per-K-split row sums, kept in the context, instead of finishing s_m itself (which costs a
 * hand-over between its CTAs); pass it as comp->row_scale to the lynx_sparse_linear call that
 * follows ON THE SAME CONTEXT with the same M and K, and its epilogue forms s_m from those sums,
 * in the same order of additions (same bits).  The sums live in the context's scratch: any later
 * call on the context that writes the scratch (another lynx_prune_compress in ROW / TENSOR mode,
 * any lynx_act_sparse_linear* call) or regrows it (lynx_reserve, a larger shape) makes the context
 * forget them, and a lynx_sparse_linear call that still asks for them returns
 * LYNX_ERR_INVALID_ARG without launching anything. */
#define LYNX_ROW_SCALE_DEFERRED ((float*)(uintptr_t)1)

/* Epilogue terms of lynx_sparse_linear (all optional). */
typedef struct {
    const float* row_scale; /* [M] fp32 per-row scale s_m, NULL (= 1), or LYNX_ROW_SCALE_DEFERRED  */
    const void* residual;   /* Y_r: [M x N] bf16, leading dimension ldr, or NULL              */
    int64_t ldr;
} lynx_comp;

/* ---- context ------------------------------------------------------------------------------- */

/* Creates a context on CUDA device `device` (made current for the call).  Allocates a small
 * status word and a ticket area; scratch is allocated lazily (see lynx_reserve).  The context
 * caches the tensor maps (TMA descriptors) it encodes, keyed by pointer, shape, leading dimension
 * and tile, so a layer called again on the same buffers re-encodes nothing.  Reads no environment
 * variable except LYNX_DEV: with LYNX_DEV=1 (tests, measurement scripts) it also reads the
 * development overrides (LYNX_GEMM_CFG, LYNX_SPLITK, LYNX_PRUNE_TPU, ...). */
LYNX_API lynx_status lynx_create(lynx_ctx** out, int device);
/* Frees the context's scratch.  The caller must have synchronised every stream it used. */
LYNX_API lynx_status lynx_destroy(lynx_ctx* ctx);
LYNX_API const char* lynx_status_string(lynx_status s);
/* Reads and clears the sticky device-side error word (LYNX_OK or LYNX_ERR_TIMEOUT). HOST call,
 * does not synchronise: call after synchronising the stream to be sure a launch has finished. */
LYNX_API lynx_status lynx_last_error(lynx_ctx* ctx);

/* Bytes of the compressed operands for an M x K activation matrix. */
LYNX_API size_t lynx_values_bytes(int64_t M, int64_t K); /* M * (K/2) bf16                    */
LYNX_API size_t lynx_meta_bytes(int64_t M, int64_t K);   /* ceil(M/128) * (K/128) * 2048      */
/* Scratch the context needs for lynx_act_sparse_linear / TENSOR compensation at this size
 * (partial row sums, compressed operands, row scale; N does not enter). */
LYNX_API size_t lynx_workspace_bytes(int64_t M, int64_t N, int64_t K);
/* Grows the context's scratch to serve shapes up to (M, N, K).  May call cudaMalloc and
 * synchronise; call it outside timed or captured regions.  Entry points that need scratch call
 * it themselves when the scratch is too small. */
LYNX_API lynx_status lynx_reserve(lynx_ctx* ctx, int64_t M, int64_t N, int64_t K);

/* ---- step 1-4: Top-2-of-4 selection, compression, norm-compensation scale --------------------
 * (Algorithm 1 lines 3-4; sparse-tensor-core appendix for the values + 2-bit index form.)
 *
 * For every row m and group g of 4 consecutive elements (groups start at k = 0) keeps the two
 * elements of largest magnitude; magnitudes compare as the 15 non-sign bits of the bf16 pattern
 * (so NaN > Inf > finite, +0 == -0, no flush of subnormals) and ties go to the lower index.
 *   values[m, 2g+j] = X[m, 4g + idx_j], idx_0 < idx_1          (bit copies)   [M x K/2 bf16]
 *   meta: nibble(m, g) = idx_0 | idx_1 << 2, stored in the order the sparse MMA reads it:
 *         blocks of 128 rows x 128 K-elements, 2048 bytes each, block (rb, kb) at byte
 *         (rb * K/128 + kb) * 2048; inside a block, byte = lane*16 + step*4 + ((r/8)%2)*2 + h/8
 *         with r = row in block, step = (k%128)/32, lane = r%8 + 8*((k%32)/16) + 16*(r/16),
 *         h = k%16 (bit h%8 of that byte belongs to element k).  Rows past M in the last block
 *         are filled with the pattern 0x4.  lynx_meta_to_canonical converts to the plain
 *         row-major form for inspection.
 *   row_scale (may be NULL when mode == LYNX_COMP_NONE): [M] fp32, s_m per `mode`
 *         (ROW: per row; TENSOR: the same global s in every entry; NONE: 1.0 if non-NULL).
 * LYNX_COMP_GROUP: values[m, 2g+j] = bf16_rne( s_{m,g} * X[m, 4g + idx_j] ) with, in fp32 and IEEE
 *         operations in this order, num = ((x0^2 + x1^2) + x2^2) + x3^2, den = (k0^2 + k1^2) + 1e-8
 *         (k = the two kept elements), s = sqrt(num / den); metadata as in every mode; row_scale,
 *         if given, is written as 1.0 and the product that follows needs no scale.  (Not
 *         available with LYNX_FUSE_FUSED.)
 * Alignment for this step: X and values 32-byte aligned, ldx % 16 == 0 (32-byte vector
 * accesses), meta 16-byte aligned; violations return LYNX_ERR_ALIGNMENT.
 * ROW and TENSOR modes use the context's scratch: partial sums of each 16-row block per run of
 * K blocks, one ticket word per 16-row block (the last CTA of a block adds the partial sums in
 * ascending K order, so row_scale is reproducible bit for bit, and resets the ticket), and in
 * TENSOR mode 2 floats per row.  The scratch is grown on demand (see lynx_reserve).
 * With the ticket area fixed at 1 MB, M > 4194304 returns LYNX_ERR_UNSUPPORTED_SHAPE.
 */
LYNX_API lynx_status lynx_prune_compress(lynx_ctx* ctx, const void* X, int64_t M, int64_t K,
                                         int64_t ldx, void* values, void* meta, float* row_scale,
                                         lynx_comp_mode mode, void* stream);

/* Same operation as lynx_prune_compress for callers that cannot allocate device memory -- a
 * serving process that has handed the whole device to its own memory pool (so cudaMalloc may
 * fail or stall), or a latency-critical loop that must not hit the device-wide synchronisation
 * cudaMalloc / cudaFree imply.  (The paper has no counterpart; this is a packaging variant.)
 * It needs no context and calls no cudaMalloc, cudaFree or other allocating routine: the partial
 * row sums and per-row sums that lynx_prune_compress keeps in its context's scratch live here in
 * a fixed device array of LYNX_STATIC_SCRATCH_BYTES that is part of the library image (every GPU
 * that loads the library holds it until the process exits).
 *   - Works on the CURRENT device.  The first call on each device looks up the array's device
 *     address (cudaGetSymbolAddress) and caches it; make that first call before any stream
 *     capture begins.
 *   - Shapes whose scratch need -- a fixed 64 KB ticket area (one word per 16 rows, so
 *     M <= 262144), plus ceil(M/128)*8 * (K/128)/t * 128 bytes of partial sums, t the K blocks
 *     per warp the library picks, plus 8*M bytes in LYNX_COMP_TENSOR mode -- exceeds
 *     LYNX_STATIC_SCRATCH_BYTES are refused with LYNX_ERR_WORKSPACE; LYNX_COMP_NONE needs none.
 *   - Every call shares the one array and finds the previous call's contents in it.  The sums
 *     are overwritten before they are read; the ticket words start at zero (the array is
 *     zero-initialised when the library is loaded) and every launch leaves them at zero.  Two
 *     calls that overlap on the GPU (different streams, no ordering between them) race on it:
 *     order them.
 *   - No device-side error word: the kernels involved have no waits that can time out.
 * Arguments, layouts, alignment rules and results are exactly those of lynx_prune_compress (one
 * work decomposition serves both, so row_scale agrees bit for bit). */
#define LYNX_STATIC_SCRATCH_BYTES (8u << 20)
LYNX_API lynx_status lynx_prune_compress_static(const void* X, int64_t M, int64_t K, int64_t ldx,
                                                void* values, void* meta, float* row_scale,
                                                lynx_comp_mode mode, void* stream);

/* ---- step 5-6: 2:4 sparse x dense product and epilogue ---------------------------------------
 * (Algorithm 1 lines 5-6; Algorithm 2 for the bias.)
 *   Y[m, n] = bf16_rne( s_m * sum_k X~[m,k] W[n,k]  +  bias[n]  +  Y_r[m,n] )
 * where X~ is the matrix (values, meta) encodes, the sum is accumulated in fp32 on the sparse
 * tensor cores, and absent terms (bias == NULL, comp == NULL or its members NULL) are 1 / 0.
 * values / meta must have the layout lynx_prune_compress writes.
 */
LYNX_API lynx_status lynx_sparse_linear(lynx_ctx* ctx, const void* values, const void* meta,
                                        int64_t M, int64_t K, const void* W, int64_t N, int64_t ldw,
                                        const void* bias, const lynx_comp* comp, void* Y,
                                        int64_t ldy, void* stream);

/* ---- whole layer (Algorithm 1) -----------------------------------------------------------------
 * Y = act_sparse_linear(X, W, bias, residual) = steps 1-6 above.  SEPARATE runs the two kernels
 * back to back on `stream` with the compressed operands in the context's scratch (grown on
 * demand: see lynx_reserve); FUSED prunes inside the GEMM kernel.  Both give the same values,
 * metadata and (up to fp32 summation order) the same Y.  In SEPARATE + LYNX_COMP_ROW the prune
 * launch leaves the per-K-split row sums in the scratch and the GEMM's epilogue forms s_m from
 * them, adding in the order lynx_prune_compress itself uses: Y is bit-identical to calling
 * lynx_prune_compress and lynx_sparse_linear one after the other, without the scale hand-over
 * inside the first kernel.
 */
LYNX_API lynx_status lynx_act_sparse_linear(lynx_ctx* ctx, const void* X, int64_t M, int64_t K,
                                            int64_t ldx, const void* W, int64_t N, int64_t ldw,
                                            const void* bias, lynx_comp_mode mode,
                                            const void* residual, int64_t ldr, void* Y, int64_t ldy,
                                            lynx_fuse_mode fuse, void* stream);

/* Same layer with the activations and the result in HOST memory (pinned memory recommended):
 * X_host [M x K] and Y_host [M x N] are dense row-major bf16 HOST buffers; W and bias stay
 * DEVICE resident (weights are loaded once).  Copies X to the device, runs the layer, copies Y
 * back and synchronises `stream`.  The device mirrors of X and Y are an allocation of their own that
 * only this entry point makes (grown on demand, like the scratch).  From 2048 rows
 * on (and not under LYNX_COMP_TENSOR, whose scale couples all rows) the call is pipelined over row
 * chunks on two copy streams the context owns, so that copy-in, kernels and copy-out overlap; the
 * result is the unchunked one bit for bit. */
LYNX_API lynx_status lynx_act_sparse_linear_host(lynx_ctx* ctx, const void* X_host, int64_t M,
                                                 int64_t K, const void* W, int64_t N, int64_t ldw,
                                                 const void* bias, lynx_comp_mode mode, void* Y_host,
                                                 lynx_fuse_mode fuse, void* stream);

/* ---- low-rank branch (Algorithm 1 lines 5-6: Y = Y_s + Y_r, Y_r = X (L_A L_B)^T; the
 *      interleaved-LoRA kernel optimisation of the kernel section) -------------------------------
 * L_B is R x K bf16 row-major (leading dimension ldlb), L_A is N x R bf16 row-major (ldla);
 * R is 64 or 128 (others: LYNX_ERR_UNSUPPORTED_SHAPE).  The branch reads the DENSE X.  Y_r is
 * never written to memory: the down projection T = X L_B^T is computed once per layer and the
 * up projection T L_A^T is added inside the sparse GEMM's accumulator by dense tensor-core
 * steps, so that
 *   Y[m, n] = bf16_rne( s_m * sum_k X~[m,k] W[n,k] + sum_r T[m,r] L_A[n,r] + bias[n] + Y_r'[m,n] )
 * (Y_r' = the optional comp->residual addend).  Because the epilogue multiplies the whole
 * accumulator by s_m, T is stored pre-divided:
 *
 * lynx_lora_down:  T[m, r] = bf16_rne( (sum_k X[m,k] L_B[r,k]) / s_m ), fp32 accumulation on the
 *   dense tensor cores; row_scale == NULL means s_m = 1; s_m == 0 gives T = 0.  T is M x R bf16,
 *   leading dimension ldt (>= R, multiple of 8), owned by the caller.  Uses the context's
 *   low-rank workspace (fp32 partials of the K splits; grown on demand, see lynx_reserve_lora)
 *   and a ticket word per 128-row block (M <= 2097152).  The result does not depend on the
 *   order in which CTAs finish.
 * lynx_prune_compress_lora:  lynx_prune_compress and lynx_lora_down in ONE launch that reads X
 *   once: values and meta as lynx_prune_compress writes them (bit for bit), T as above with s_m
 *   the per-row norm compensation (mode LYNX_COMP_ROW) or 1 (LYNX_COMP_NONE; other modes:
 *   LYNX_ERR_INVALID_ARG).  Under LYNX_COMP_ROW the row sums stay on the context, exactly as
 *   after lynx_prune_compress with LYNX_ROW_SCALE_DEFERRED: pass comp->row_scale =
 *   LYNX_ROW_SCALE_DEFERRED to the lynx_sparse_linear_lora call that follows.  Alignment: values
 *   32-byte aligned (32-byte vector stores); X, L_B, T and meta 16-byte aligned, ldx, ldlb and ldt
 *   multiples of 8.  Scratch: the row sums only; no low-rank workspace.
 * lynx_sparse_linear_lora:  lynx_sparse_linear plus the T L_A^T term; T must come from
 *   lynx_lora_down called with the same row_scale that comp carries, or from
 *   lynx_prune_compress_lora (deferred row scale).
 * lynx_act_sparse_linear_lora:  the whole layer, intermediates in the context's scratch: two
 *   launches, lynx_prune_compress_lora's kernel and the sparse GEMM with the low-rank steps
 *   (LYNX_COMP_NONE / LYNX_COMP_ROW; the other modes take prune/compress, lynx_lora_down and the
 *   GEMM as three launches).  Y is within the stated tolerance of the definition whichever form
 *   computed T (they may differ in the last bit of T: different K splits).
 * Pointers and leading dimensions follow the 16-byte rule of the other entry points.
 */
LYNX_API lynx_status lynx_reserve_lora(lynx_ctx* ctx, int64_t M, int64_t K, int64_t R);
LYNX_API lynx_status lynx_prune_compress_lora(lynx_ctx* ctx, const void* X, int64_t M, int64_t K,
                                              int64_t ldx, const void* LB, int64_t R, int64_t ldlb,
                                              void* values, void* meta, lynx_comp_mode mode, void* T,
                                              int64_t ldt, void* stream);
LYNX_API lynx_status lynx_lora_down(lynx_ctx* ctx, const void* X, int64_t M, int64_t K, int64_t ldx,
                                    const void* LB, int64_t R, int64_t ldlb, const float* row_scale,
                                    void* T, int64_t ldt, void* stream);
LYNX_API lynx_status lynx_sparse_linear_lora(lynx_ctx* ctx, const void* values, const void* meta,
                                             int64_t M, int64_t K, const void* W, int64_t N,
                                             int64_t ldw, const void* bias, const lynx_comp* comp,
                                             const void* T, int64_t ldt, const void* LA, int64_t R,
                                             int64_t ldla, void* Y, int64_t ldy, void* stream);
LYNX_API lynx_status lynx_act_sparse_linear_lora(lynx_ctx* ctx, const void* X, int64_t M, int64_t K,
                                                 int64_t ldx, const void* W, int64_t N, int64_t ldw,
                                                 const void* bias, const void* LA, int64_t ldla,
                                                 const void* LB, int64_t ldlb, int64_t R,
                                                 lynx_comp_mode mode, const void* residual,
                                                 int64_t ldr, void* Y, int64_t ldy, void* stream);

/* ---- FP8 composition (the paper's W8A8 compatibility experiment: symmetric FP8 quantisation of
 *      the activations, weights cast to FP8; 2:4 is one of the sparse tensor core's FP8 formats) ----
 * FP8 = E4M3 (1-4-3 bits, bias 7, no infinities, largest finite 448).  The paper fixes neither the
 * granularity of the activation scale nor the rounding; this library's rules, all in fp32 with
 * IEEE operations:
 *   selection   on the bf16 activations exactly as in lynx_prune_compress (same mask, same nibbles);
 *   activation  per token row m: amax_m = the row's largest magnitude in the selection's order
 *               (15 non-sign bits as an integer, so NaN > Inf > finite), inv_m = amax_m > 0 ?
 *               448 / amax_m : 0, code = e4m3(x * inv_m) rounded to nearest even, finite overflow
 *               saturating to +-448; act_scale_m = amax_m / 448;
 *   weights     per_channel = 0: code = e4m3(w) (a direct cast), wscale[n] = 1;
 *               per_channel = 1: the same symmetric rule per output channel n;
 *   product     fp32 accumulation on the sparse tensor cores (kind f8f6f4, K = 64 per instruction);
 *   epilogue    Y = bf16_rne( row_scale[m] * wscale[n] * acc + bias[n] + Y_r[m,n] ) with
 *               row_scale[m] = s_m * act_scale_m, s_m the per-row norm compensation of the bf16
 *               row (LYNX_COMP_ROW) or 1 (LYNX_COMP_NONE).
 * Layouts: values_q is M x K/2 bytes row-major; Wq is N x K bytes row-major, leading dimension
 * ldwq bytes (multiple of 16); wscale [N] fp32 (NULL = all 1).  K % 256 == 0.  meta has the size
 * lynx_meta_bytes(M, K) but its own order: blocks of 128 rows x 128 K-elements, 2048 bytes each,
 * block (rb, kb) at byte (rb * K/128 + kb) * 2048, inside a block row r's 16 bytes at r * 16 with
 * group g = (k % 128) / 4 in bits 4 * (g % 2) of byte g / 2; rows past M hold 0x4 nibbles.
 * row_amax (optional, [M] fp32 on the device): when given, row_amax[m] takes the place of the
 * row maximum found in the data -- a scale calibrated beforehand (the same number in every entry)
 * or a maximum the producer of X already knows; values beyond it saturate at +-448.  Either
 * way X is read from device memory once for 2048 <= K <= ~57000 (whole rows are staged in shared
 * memory: the maximum and the codes come from the staged copy); shorter and longer rows take a
 * kernel that, without row_amax, reads them twice.  Neither form needs scratch.  The low-rank branch, LYNX_COMP_TENSOR / GROUP and the one-kernel mode are
 * not available in FP8.
 */
LYNX_API lynx_status lynx_quantize_weights_fp8(lynx_ctx* ctx, const void* W, int64_t N, int64_t K,
                                               int64_t ldw, int per_channel, void* Wq, float* wscale,
                                               void* stream);
LYNX_API lynx_status lynx_prune_compress_fp8(lynx_ctx* ctx, const void* X, int64_t M, int64_t K,
                                             int64_t ldx, const float* row_amax, void* values_q,
                                             void* meta, float* row_scale, lynx_comp_mode mode,
                                             void* stream);
LYNX_API lynx_status lynx_sparse_linear_fp8(lynx_ctx* ctx, const void* values_q, const void* meta,
                                            int64_t M, int64_t K, const void* Wq, int64_t N,
                                            int64_t ldwq, const float* wscale, const void* bias,
                                            const lynx_comp* comp, void* Y, int64_t ldy, void* stream);
LYNX_API lynx_status lynx_act_sparse_linear_fp8(lynx_ctx* ctx, const void* X, int64_t M, int64_t K,
                                                int64_t ldx, const float* row_amax, const void* Wq,
                                                int64_t N, int64_t ldwq,
                                                const float* wscale, const void* bias,
                                                lynx_comp_mode mode, const void* residual, int64_t ldr,
                                                void* Y, int64_t ldy, void* stream);

/* ---- inspection helpers ------------------------------------------------------------------------ */

/* Hardware-order metadata -> canonical form: uint16 [M x K/16], nibble (g%4) of group g in bits
 * 4*(g%4).. of word g/4 of its row. */
LYNX_API lynx_status lynx_meta_to_canonical(lynx_ctx* ctx, const void* meta, int64_t M, int64_t K,
                                            void* meta_canon, void* stream);
/* Expands (values, meta) back to the masked dense matrix X~ [M x K] bf16 (dropped entries +0). */
LYNX_API lynx_status lynx_decompress(lynx_ctx* ctx, const void* values, const void* meta, int64_t M,
                                     int64_t K, void* Xmasked, void* stream);

/* Self-test of the device-side time-out path.  Every wait inside the kernels is bounded; when one
 * runs out the kernel sets the context's error word and returns, and the next call on the context
 * (or lynx_last_error) reports LYNX_ERR_TIMEOUT.  This entry launches one warp that waits
 * `limit_us` microseconds (1 .. 100000) on a barrier nobody arrives at, so that exactly this
 * happens: after synchronising `stream`, the next library call returns LYNX_ERR_TIMEOUT and
 * lynx_last_error returns LYNX_ERR_TIMEOUT once and clears the word.  Nothing faults. */
LYNX_API lynx_status lynx_selftest_wait_timeout(lynx_ctx* ctx, int64_t limit_us, void* stream);

/* Host-only views of how the sparse GEMM would be run (nothing is launched, no device is needed):
 * lynx_gemm_plan returns 1 when, for an (M, N, K) product on a GPU with num_sms SMs, the kernel
 * that runs two 256-row tiles per W stage is chosen (its number of 512-row items and of CTA pairs
 * in *doubles / *clusters), 0 when the single-tile kernel is, -1 on bad arguments.
 * lynx_gemm_schedule_items lists the work items of CTA pair `cluster` for `tiles_m` x `tiles_n`
 * tiles of 256 x 240 over `clusters` pairs with `doubles` 512-row items: items[4i..4i+3] = first
 * row tile, column tile, row tiles (1 or 2), ordinal among the pair's single-tile items; returns
 * the item count (only the first `capacity` are written) or -1. */
LYNX_API int lynx_gemm_plan(int num_sms, int64_t M, int64_t N, int64_t K, int lora_steps, int* doubles,
                            int* clusters);
LYNX_API int lynx_gemm_schedule_items(int tiles_m, int tiles_n, int clusters, int doubles, int cluster,
                                      int* items, int capacity);

/* Number of kernels the library launched on this context since creation (for accounting). */
LYNX_API int64_t lynx_launch_count(lynx_ctx* ctx);

#ifdef __cplusplus
}
#endif
#endif /* LYNX_H_ */

/*
 * astra.h -- C ABI of the B200 (sm_100a) library for the three memory-bound LLM-serving
 * operations studied in "Astra: A Multi-Agent System for GPU Kernel Performance Optimization"
 * (Table 1: merge_attn_states_lse, fused_add_rmsnorm, silu_and_mul).
 *
 * Conventions shared by every entry point
 *   - Every data pointer is a DEVICE pointer on the current CUDA device, owned by the caller.
 *     The library allocates nothing, keeps no state between calls, and never synchronises:
 *     work is enqueued on `cuda_stream` (a cudaStream_t passed as void*; NULL = default stream)
 *     and the call returns immediately.  Host pointers are not detected (undefined behaviour).
 *   - Tensors are dense and row-major (the last index is contiguous; a row's pitch is its width).
 *   - `dtype` selects the storage type of all value tensors of the call (bf16, fp16 or fp32).
 *     Arithmetic is binary32 throughout, with a single round-to-nearest-even to the storage type at
 *     each store.
 *   - Pointers need only the natural alignment of their element (2 bytes for 16-bit values, 4 for
 *     fp32 values and for scores).  Wider alignment is detected and exploited inside; widths need not be multiples
 *     of 8.  A pointer with less than element alignment gives ASTRA_ERR_MISALIGNED.
 *   - Errors are return codes only: nothing is printed, thrown or aborted.  Arguments are checked
 *     before anything is launched, so after any status other than ASTRA_OK and ASTRA_ERR_CUDA the
 *     GPU has been given no work.  ASTRA_ERR_CUDA means the CUDA runtime refused a kernel launch
 *     (the status is that launch's own return value).  Inputs beyond 2^31 - 1 vectors or rows are
 *     issued as several launches; if one of them is refused the later ones are not issued, but
 *     the earlier ones remain enqueued, so the outputs are then partly written.
 *     The library links its own copy of the CUDA runtime: on success it neither reads nor clears
 *     the runtime's per-thread "last error", and the caller's runtime state is never touched.
 *   - A zero-sized first dimension (T == 0) is ASTRA_OK and launches nothing; the pointers of such
 *     a call are not examined (an empty tensor may have a NULL address).  Any other non-positive
 *     extent is ASTRA_ERR_BAD_SHAPE.  Limits: a fused_add_rmsnorm row holds at most 2^30 16-bit
 *     units (2^30 bf16/fp16 or 2^29 fp32 elements); D of the other two operations is below 2^30.
 *   - Non-finite inputs never trap; they propagate by IEEE rules except where stated below.
 */
#ifndef ASTRA_H_
#define ASTRA_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    ASTRA_BF16 = 0, /* bfloat16: 1 sign, 8 exponent, 7 fraction bits */
    ASTRA_FP16 = 1, /* IEEE binary16                                  */
    ASTRA_FP32 = 2  /* IEEE binary32 (no conversion, no rounding at the store beyond the arithmetic's own) */
} astra_dtype_t;

typedef enum {
    ASTRA_OK = 0,
    ASTRA_ERR_NULL_POINTER = 1, /* a required pointer is NULL                         */
    ASTRA_ERR_BAD_SHAPE = 2,    /* an extent is negative, zero where not allowed, or too large */
    ASTRA_ERR_BAD_DTYPE = 3,    /* dtype is not one of astra_dtype_t                  */
    ASTRA_ERR_MISALIGNED = 4,   /* a pointer is not aligned to its element size       */
    ASTRA_ERR_CUDA = 5,         /* the CUDA runtime reported an error at launch       */
    ASTRA_ERR_OVERLAP = 6       /* an output overlaps an input in a way not allowed   */
} astra_status_t;

/*
 * fused_add_rmsnorm (Table 1, Kernel 2):
 *     y = (x + r) / sqrt( (1/H) * ||x + r||_2^2 + eps )  (.)  w         per row of H elements
 *
 *   x        [T, H]  in: x.          out: y                       (updated in place)
 *   residual [T, H]  in: r.          out: x + r                   (updated in place)
 *   weight   [H]     in: w.
 *   eps      added to the mean of squares, inside the square root.
 *
 * The sum x + r is one binary32 addition.  `residual` receives that sum rounded once to the
 * storage type (bit-exact, independent of launch shape).  The norm is taken over the unrounded
 * binary32 sums, and nothing is rounded between the normalisation and the multiplication by w.
 * x and residual must not overlap each other or weight.
 */
astra_status_t astra_fused_add_rmsnorm(void *x, void *residual, const void *weight,
                                       int64_t T, int64_t H, float eps,
                                       astra_dtype_t dtype, void *cuda_stream);

/*
 * silu_and_mul (Table 1, Kernel 3):
 *     out = SiLU(a) (.) b,   SiLU(z) = z / (1 + e^{-z})
 *
 *   input [T, 2*D]  in: each row is [ a (D gate values) | b (D up values) ].
 *   out   [T, D]    out.  Must not overlap input (checked: ASTRA_ERR_OVERLAP).
 *
 * SiLU(a) is not rounded to the storage type before the multiplication by b.
 */
astra_status_t astra_silu_and_mul(void *out, const void *input, int64_t T, int64_t D,
                                  astra_dtype_t dtype, void *cuda_stream);

/*
 * merge_attn_states_lse (Table 1, Kernel 1): merge two partial attention results, each given
 * as an output vector and the natural-log sum of exponentials of its logits.
 *     V_out = (e^{Sa} Va + e^{Sb} Vb) / (e^{Sa} + e^{Sb})
 *     S_out = log(e^{Sa} + e^{Sb})
 *
 *   v_a, v_b  [T, Hh, D]  in.        lse_a, lse_b  [T, Hh] binary32, in.
 *   v_out     [T, Hh, D]  out.       lse_out       [T, Hh] binary32, out; may be NULL (not written).
 *
 * The two weights are computed once per (token, head).  v_out may be exactly v_a or v_b
 * (in-place merge of the values); any other overlap of v_out with an input, and any overlap of
 * lse_out with lse_a or lse_b, gives ASTRA_ERR_OVERLAP.
 * A score of -inf denotes an empty state: its weight is exactly 0, its V is ignored (even if
 * not finite), and the other state is returned unchanged.  If both scores are -inf the result
 * is V_out = 0, S_out = -inf.  A score of +inf or NaN is outside the domain: NaN is produced.
 */
astra_status_t astra_merge_attn_states_lse(void *v_out, float *lse_out,
                                           const void *v_a, const float *lse_a,
                                           const void *v_b, const float *lse_b,
                                           int64_t T, int64_t Hh, int64_t D,
                                           astra_dtype_t dtype, void *cuda_stream);

/*
 * Strided / out-of-place forms.  Same operations and arithmetic as above (Table 1); only the
 * addressing differs.  All pitches and strides are in ELEMENTS and must be non-negative; the
 * innermost dimension is always contiguous.  Rows of one tensor must not overlap each other
 * (pitch >= row width), otherwise ASTRA_ERR_BAD_SHAPE.  Vector width is chosen from the width, the
 * pitches and the base addresses, so slices of wider buffers work at any element alignment.
 */

/*
 * fused_add_rmsnorm with separate outputs and row pitches.
 *   y            [T, H] rows y_pitch apart             out: RMSNorm(x + residual) * weight
 *   residual_out [T, H] rows residual_out_pitch apart  out: x + residual (one binary32 add, one rounding)
 *   x, residual  [T, H] rows x_pitch / residual_pitch apart, in
 * y may be exactly x (same address and pitch) and residual_out exactly residual; that is the
 * in-place form, and astra_fused_add_rmsnorm(x, r, w, ...) is this call with y = x,
 * residual_out = r and all pitches equal to H.  Any other overlap between an output and another
 * operand gives ASTRA_ERR_OVERLAP.
 */
astra_status_t astra_fused_add_rmsnorm_ex(void *y, void *residual_out, const void *x,
                                          const void *residual, const void *weight,
                                          int64_t T, int64_t H,
                                          int64_t y_pitch, int64_t residual_out_pitch,
                                          int64_t x_pitch, int64_t residual_pitch,
                                          float eps, astra_dtype_t dtype, void *cuda_stream);

/*
 * silu_and_mul with separately addressed gate and up operands.
 *   gate [T, D] rows gate_pitch apart, up [T, D] rows up_pitch apart, out [T, D] rows out_pitch apart.
 * The packed row [a | b] of astra_silu_and_mul is gate = input, up = input + D, both pitches 2*D.
 * out must not overlap gate or up.
 */
astra_status_t astra_silu_and_mul_ex(void *out, const void *gate, const void *up,
                                     int64_t T, int64_t D,
                                     int64_t out_pitch, int64_t gate_pitch, int64_t up_pitch,
                                     astra_dtype_t dtype, void *cuda_stream);

/*
 * merge_attn_states_lse for strided tensors.  `strides` is a HOST array of 12 element strides:
 *   { v_a token, v_a head, v_b token, v_b head, v_out token, v_out head,
 *     lse_a token, lse_a head, lse_b token, lse_b head, lse_out token, lse_out head }.
 * head_dim is contiguous in the value tensors.  Scores stored head-major ([Hh, T]) are
 * { token stride 1, head stride T }.  T * Hh must be below 2^31.  Aliasing rules as for
 * astra_merge_attn_states_lse: v_out may be exactly v_a or v_b (same address and strides);
 * lse_out may be NULL (its two strides are then ignored).
 */
astra_status_t astra_merge_attn_states_lse_ex(void *v_out, float *lse_out,
                                              const void *v_a, const float *lse_a,
                                              const void *v_b, const float *lse_b,
                                              int64_t T, int64_t Hh, int64_t D,
                                              const int64_t *strides,
                                              astra_dtype_t dtype, void *cuda_stream);

/*
 * fused_allreduce_add_rmsnorm: fused_add_rmsnorm (Table 1, Kernel 2) on a hidden state that arrives
 * as n_parts partial sums, one per tensor-parallel rank -- the all-reduce that precedes Kernel 2 in
 * tensor-parallel serving, folded into it (the paper's per-shape study, Table 4, shows these small
 * calls bound by fixed cost rather than bandwidth; the paper itself states Kernel 2 for one x only):
 *     x = x_0 + x_1 + ... + x_{n-1};  s = x + r;  residual <- s;  y = s / sqrt(mean(s^2) + eps) (.) w
 *
 *   y        [T, H]  out.
 *   residual [T, H]  in: r.  out: s rounded once to the storage type  (updated in place)
 *   x_parts  HOST array of n_parts device pointers, in rank order, each a dense [T, H] tensor.
 *            A partial may live in another GPU's memory if that memory is mapped into this
 *            process (peer access): the kernel reads it with ordinary per-thread loads only.
 *   n_parts  1 .. 16 (else ASTRA_ERR_BAD_SHAPE).  n_parts = 1 is the operation of
 *            astra_fused_add_rmsnorm_ex with separate y (same residual bits; y by the same arithmetic).
 *   weight   [H].
 *
 * Arithmetic: every addition is one binary32 addition; the partials are added in rank order
 * starting from x_0 and the residual is added last; nothing is rounded to the storage type before
 * that.  Ranks that run this on the same partials therefore produce identical bits.
 * Ordering: the call waits for nothing.  The caller must order it after every rank has finished
 * writing its partial, and must keep the partials unchanged until the kernel has completed.
 * y and residual must not overlap each other, any partial, or weight (ASTRA_ERR_OVERLAP); the
 * partials may overlap one another.  Every pointer needs the alignment of its element.
 */
astra_status_t astra_fused_allreduce_add_rmsnorm(void *y, void *residual,
                                                 const void *const *x_parts, int32_t n_parts,
                                                 const void *weight, int64_t T, int64_t H, float eps,
                                                 astra_dtype_t dtype, void *cuda_stream);

/*
 * fused_allreduce_add_rmsnorm with several destinations per result: the two-shot form of the same
 * operation (Table 1, Kernel 2 on a hidden state given as n_parts partial sums; arithmetic exactly
 * as astra_fused_allreduce_add_rmsnorm).  For batches large enough that reading every partial on
 * every rank would be bound by the links, each rank calls this for ITS OWN BLOCK OF ROWS only and
 * has the results stored into every rank's buffers, so that each element crosses the links once as
 * a partial and once as a result:
 *
 *   y_outs         HOST array of n_y device pointers; each receives the T normalised rows.
 *   residual_outs  HOST array of n_r device pointers; each receives the T rows of the new residual.
 *   residual       [T, H] in: r.  One of residual_outs may be exactly this pointer (in place).
 *   x_parts, n_parts, weight, T, H, eps, dtype: as in astra_fused_allreduce_add_rmsnorm.
 *   n_y, n_r       1 .. 16 each (else ASTRA_ERR_BAD_SHAPE).
 *
 * All tensors are dense [T, H] blocks; the caller passes pointers already advanced to the block's
 * first row in each buffer.  A destination may live in another GPU's memory mapped into this
 * process: it is written with ordinary per-thread stores only.  With n_y = n_r = 1 and
 * residual_outs[0] = residual this is astra_fused_allreduce_add_rmsnorm, bit for bit.
 * Ordering is the caller's, in both directions: the call waits for nothing, and the ranks that own
 * the destinations must not read them before this kernel has completed.
 * Every destination must not overlap any other destination, any partial, weight, or residual
 * (except the exact in-place case above): ASTRA_ERR_OVERLAP.
 */
astra_status_t astra_fused_allreduce_add_rmsnorm_ex(void *const *y_outs, int32_t n_y,
                                                    void *const *residual_outs, int32_t n_r,
                                                    const void *residual,
                                                    const void *const *x_parts, int32_t n_parts,
                                                    const void *weight, int64_t T, int64_t H, float eps,
                                                    astra_dtype_t dtype, void *cuda_stream);

/* Static, NUL-terminated description of a status code (never NULL). */
const char *astra_status_string(astra_status_t status);

/*
 * Static, NUL-terminated identifier of the sources this library was compiled from: the hexadecimal
 * SHA-256 the build script computes over the headers and CUDA sources ("unidentified" if the
 * library was compiled by hand).  The Python binding compares it with the sources beside it when it
 * loads the library and refuses a library built from other sources.  No counterpart in the paper.
 */
const char *astra_build_id(void);

#ifdef __cplusplus
}
#endif
#endif /* ASTRA_H_ */

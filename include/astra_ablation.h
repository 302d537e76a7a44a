/*
 * astra_ablation.h -- C ABI of the ablation library: the kernel DESIGN PAIRS that the case studies
 * of "Astra: A Multi-Agent System for GPU Kernel Performance Optimization" describe (Section 5.3,
 * Figures 2-5), re-implemented from those descriptions for sm_100a so that the paper's headline
 * quantity -- the speedup of the optimised design over the baseline design, per shape and as a
 * geometric mean (Section 3.1) -- can be measured on a B200 next to this library's own kernels.
 *
 * These are measurement subjects, not the product: same operations, same arithmetic readings and
 * the same argument conventions as astra.h (device pointers, dense row-major tensors, status codes,
 * asynchronous launch on `cuda_stream`), but deliberately built the way the paper describes each
 * design.  Widths must be even for design 1 (32-bit accesses); otherwise ASTRA_ERR_BAD_SHAPE.
 *
 *   design 0 ("baseline")                          design 1 ("optimised")
 *   merge   weights (max, two exp, division)       weights computed once before the element loop;
 *           recomputed for every element,          the loop is load, multiply-add, store; 32-bit
 *           scalar 16-bit accesses                 (two-element) accesses
 *   rmsnorm shared-memory tree reduction with a    warp-shuffle reduction, one shared-memory slot
 *           block barrier per halving step,        per warp, short cross-warp finish; 32-bit
 *           scalar accesses                        accesses
 *   silu    scalar accesses, expf and a division   32-bit accesses, fast exponential intrinsic,
 *                                                  reciprocal and multiply instead of the division
 */
#ifndef ASTRA_ABLATION_H_
#define ASTRA_ABLATION_H_

#include "astra.h"

#ifdef __cplusplus
extern "C" {
#endif

/* Section 5.3, Kernel 1 (Figure 2): merge_attn_states_lse; arguments as astra_merge_attn_states_lse,
 * lse_out required. */
astra_status_t astra_ablation_merge_attn_states_lse(int design, void *v_out, float *lse_out,
                                                    const void *v_a, const float *lse_a,
                                                    const void *v_b, const float *lse_b,
                                                    int64_t T, int64_t Hh, int64_t D,
                                                    astra_dtype_t dtype, void *cuda_stream);

/* Section 5.3, Kernel 2 (Figure 3): fused_add_rmsnorm, in place; arguments as astra_fused_add_rmsnorm.
 * H is limited to 65536. */
astra_status_t astra_ablation_fused_add_rmsnorm(int design, void *x, void *residual, const void *weight,
                                                int64_t T, int64_t H, float eps,
                                                astra_dtype_t dtype, void *cuda_stream);

/* Section 5.3, Kernel 3 (Figures 4 and 5): silu_and_mul; arguments as astra_silu_and_mul. */
astra_status_t astra_ablation_silu_and_mul(int design, void *out, const void *input,
                                           int64_t T, int64_t D,
                                           astra_dtype_t dtype, void *cuda_stream);

#ifdef __cplusplus
}
#endif
#endif /* ASTRA_ABLATION_H_ */

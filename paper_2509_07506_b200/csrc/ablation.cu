// Ablation library (declared in astra_ablation.h): the baseline / optimised design pairs described
// in the paper's case studies (Section 5.3, Figures 2-5), written from those descriptions for
// sm_100a.  They exist to be timed against each other and against the library's own kernels; they
// use the same arithmetic readings (binary32 throughout, one rounding per store) so the same parity
// gates apply.
#include <cuda_runtime.h>

#include "astra_ablation.h"
#include "vec.cuh"

namespace {

using namespace astra;

constexpr int kThreads = 256;

// ---------------------------------------------------------------------------------------------
// Kernel 1: merge_attn_states_lse.  One warp per (token, head) row; lanes stride over head_dim.
// ---------------------------------------------------------------------------------------------
struct Weights { float a, b, lse; };

// max, two exponentials, one division: the weight computation the paper's Figure 2 hoists.
__device__ __forceinline__ Weights mixing_weights(float sa, float sb) {
    Weights w;
    const float m = fmaxf(sa, sb);
    if (m == -INFINITY) { w.a = 0.f; w.b = 0.f; w.lse = -INFINITY; return w; }
    const float ea = expf(sa - m), eb = expf(sb - m);
    const float inv = 1.0f / (ea + eb);
    w.a = ea * inv;
    w.b = eb * inv;
    w.lse = m + logf(ea + eb);
    return w;
}

__device__ __forceinline__ float blend(const Weights &w, float va, float vb) {
    // a zero weight drops its side (an empty state may hold anything)
    const float ta = (w.a == 0.f) ? 0.f : w.a * va;
    return (w.b == 0.f) ? ta : fmaf(w.b, vb, ta);
}

// design 0: the weights are recomputed for every element inside the loop over head_dim
template <int DT>
__global__ void __launch_bounds__(kThreads)
merge_recompute_kernel(uint16_t *v_out, float *lse_out, const uint16_t *v_a, const float *lse_a,
                       const uint16_t *v_b, const float *lse_b, int64_t rows, int D) {
    const int64_t row = static_cast<int64_t>(blockIdx.x) * (kThreads / 32) + (threadIdx.x >> 5);
    const int lane = threadIdx.x & 31;
    if (row >= rows) return;
    const float sa = lse_a[row], sb = lse_b[row];
    const uint16_t *pa = v_a + row * D, *pb = v_b + row * D;
    uint16_t *po = v_out + row * D;
    for (int d = lane; d < D; d += 32) {
        const Weights w = mixing_weights(sa, sb);  // loop-invariant, recomputed on purpose
        po[d] = Storage<DT>::narrow1(blend(w, Storage<DT>::widen1(pa[d]), Storage<DT>::widen1(pb[d])));
        if (d == 0) lse_out[row] = w.lse;
    }
}

// design 1: weights once per row, then a light loop; two elements per 32-bit access
template <int DT>
__global__ void __launch_bounds__(kThreads)
merge_hoisted_kernel(uint16_t *v_out, float *lse_out, const uint16_t *v_a, const float *lse_a,
                     const uint16_t *v_b, const float *lse_b, int64_t rows, int D) {
    const int64_t row = static_cast<int64_t>(blockIdx.x) * (kThreads / 32) + (threadIdx.x >> 5);
    const int lane = threadIdx.x & 31;
    if (row >= rows) return;
    const Weights w = mixing_weights(lse_a[row], lse_b[row]);
    const uint32_t *pa = reinterpret_cast<const uint32_t *>(v_a + row * D);
    const uint32_t *pb = reinterpret_cast<const uint32_t *>(v_b + row * D);
    uint32_t *po = reinterpret_cast<uint32_t *>(v_out + row * D);
    for (int d = lane; d < D / 2; d += 32) {
        float a0, a1, b0, b1;
        Storage<DT>::widen2(pa[d], a0, a1);
        Storage<DT>::widen2(pb[d], b0, b1);
        po[d] = Storage<DT>::narrow2(blend(w, a0, b0), blend(w, a1, b1));
    }
    if (lane == 0) lse_out[row] = w.lse;
}

// ---------------------------------------------------------------------------------------------
// Kernel 2: fused_add_rmsnorm, one block per row, two sweeps over the row (the sum of squares
// first, then the outputs; nothing is written before the norm is known).
// ---------------------------------------------------------------------------------------------

// design 0: tree reduction in shared memory, one block barrier per halving step
template <int DT>
__global__ void __launch_bounds__(kThreads)
rmsnorm_tree_kernel(uint16_t *x, uint16_t *residual, const uint16_t *weight, int H, float eps) {
    __shared__ float partial[kThreads];
    uint16_t *xr = x + static_cast<int64_t>(blockIdx.x) * H;
    uint16_t *rr = residual + static_cast<int64_t>(blockIdx.x) * H;
    const int tx = threadIdx.x;
    float acc = 0.f;
    for (int j = tx; j < H; j += kThreads) {
        const float s = Storage<DT>::widen1(xr[j]) + Storage<DT>::widen1(rr[j]);
        acc = fmaf(s, s, acc);
    }
    partial[tx] = acc;
    __syncthreads();
    for (int half = kThreads / 2; half > 0; half >>= 1) {
        if (tx < half) partial[tx] += partial[tx + half];
        __syncthreads();
    }
    const float rstd = rsqrtf(partial[0] / static_cast<float>(H) + eps);
    for (int j = tx; j < H; j += kThreads) {
        const float s = Storage<DT>::widen1(xr[j]) + Storage<DT>::widen1(rr[j]);
        rr[j] = Storage<DT>::narrow1(s);
        xr[j] = Storage<DT>::narrow1(s * rstd * Storage<DT>::widen1(weight[j]));
    }
}

// design 1: shuffles inside each warp, one shared slot per warp, short finish; 32-bit accesses
template <int DT>
__global__ void __launch_bounds__(kThreads)
rmsnorm_shuffle_kernel(uint16_t *x, uint16_t *residual, const uint16_t *weight, int H, float eps) {
    __shared__ float warp_sum[kThreads / 32];
    uint32_t *xr = reinterpret_cast<uint32_t *>(x + static_cast<int64_t>(blockIdx.x) * H);
    uint32_t *rr = reinterpret_cast<uint32_t *>(residual + static_cast<int64_t>(blockIdx.x) * H);
    const uint32_t *wr = reinterpret_cast<const uint32_t *>(weight);
    const int tx = threadIdx.x, lane = tx & 31, warp = tx >> 5;
    float acc = 0.f;
    for (int j = tx; j < H / 2; j += kThreads) {
        float x0, x1, r0, r1;
        Storage<DT>::widen2(xr[j], x0, x1);
        Storage<DT>::widen2(rr[j], r0, r1);
        const float s0 = x0 + r0, s1 = x1 + r1;
        acc = fmaf(s0, s0, acc);
        acc = fmaf(s1, s1, acc);
    }
    for (int off = 16; off > 0; off >>= 1) acc += __shfl_down_sync(0xffffffffu, acc, off);
    if (lane == 0) warp_sum[warp] = acc;
    __syncthreads();
    float total = 0.f;
#pragma unroll
    for (int i = 0; i < kThreads / 32; ++i) total += warp_sum[i];
    const float rstd = rsqrtf(total / static_cast<float>(H) + eps);
    for (int j = tx; j < H / 2; j += kThreads) {
        float x0, x1, r0, r1, w0, w1;
        Storage<DT>::widen2(xr[j], x0, x1);
        Storage<DT>::widen2(rr[j], r0, r1);
        Storage<DT>::widen2(wr[j], w0, w1);
        const float s0 = x0 + r0, s1 = x1 + r1;
        rr[j] = Storage<DT>::narrow2(s0, s1);
        xr[j] = Storage<DT>::narrow2(s0 * rstd * w0, s1 * rstd * w1);
    }
}

// ---------------------------------------------------------------------------------------------
// Kernel 3: silu_and_mul, one thread per element (design 0) or per element pair (design 1).
// ---------------------------------------------------------------------------------------------
template <int DT>
__global__ void __launch_bounds__(kThreads)
silu_scalar_kernel(uint16_t *out, const uint16_t *in, int64_t total, int64_t D) {
    const int64_t i = static_cast<int64_t>(blockIdx.x) * kThreads + threadIdx.x;
    if (i >= total) return;
    const int64_t row = i / D, col = i - row * D;
    const float a = Storage<DT>::widen1(in[row * 2 * D + col]);
    const float b = Storage<DT>::widen1(in[row * 2 * D + D + col]);
    out[i] = Storage<DT>::narrow1(a / (1.0f + expf(-a)) * b);  // library exponential and a division
}

__device__ __forceinline__ float silu_fast(float a) {
    // fast exponential, then reciprocal and multiply in place of the division (as described; for
    // gates below about -88 the exponential overflows and the result is -0, like design 0)
    const float e = __expf(-a);
    return __fmul_rn(a, __frcp_rn(1.0f + e));
}

template <int DT>
__global__ void __launch_bounds__(kThreads)
silu_pair_kernel(uint16_t *out, const uint16_t *in, int64_t total_pairs, int64_t halfD) {
    const int64_t i = static_cast<int64_t>(blockIdx.x) * kThreads + threadIdx.x;
    if (i >= total_pairs) return;
    const int64_t row = i / halfD, col = i - row * halfD;
    const uint32_t *pin = reinterpret_cast<const uint32_t *>(in);
    float a0, a1, b0, b1;
    Storage<DT>::widen2(pin[row * 2 * halfD + col], a0, a1);
    Storage<DT>::widen2(pin[row * 2 * halfD + halfD + col], b0, b1);
    reinterpret_cast<uint32_t *>(out)[i] = Storage<DT>::narrow2(__fmul_rn(silu_fast(a0), b0), __fmul_rn(silu_fast(a1), b1));
}

inline bool aligned4(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 3) == 0; }
inline astra_status_t launched() { return cudaGetLastError() == cudaSuccess ? ASTRA_OK : ASTRA_ERR_CUDA; }

}  // namespace

extern "C" {

astra_status_t astra_ablation_merge_attn_states_lse(int design, void *v_out, float *lse_out,
                                                    const void *v_a, const float *lse_a,
                                                    const void *v_b, const float *lse_b,
                                                    int64_t T, int64_t Hh, int64_t D,
                                                    astra_dtype_t dtype, void *cuda_stream) {
    if (!v_out || !lse_out || !v_a || !lse_a || !v_b || !lse_b) return ASTRA_ERR_NULL_POINTER;
    if (dtype != ASTRA_BF16 && dtype != ASTRA_FP16) return ASTRA_ERR_BAD_DTYPE;
    if (design != 0 && design != 1) return ASTRA_ERR_BAD_SHAPE;
    if (T < 0 || Hh <= 0 || D <= 0 || D > 65536 || (design == 1 && D % 2)) return ASTRA_ERR_BAD_SHAPE;
    if (T > 0 && Hh > (1ll << 40) / T) return ASTRA_ERR_BAD_SHAPE;
    if (design == 1 && !(aligned4(v_out) && aligned4(v_a) && aligned4(v_b))) return ASTRA_ERR_MISALIGNED;
    if (T == 0) return ASTRA_OK;
    const int64_t rows = T * Hh;
    const int64_t blocks = (rows + kThreads / 32 - 1) / (kThreads / 32);
    if (blocks > 2147483647ll) return ASTRA_ERR_BAD_SHAPE;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    uint16_t *vo = static_cast<uint16_t *>(v_out);
    const uint16_t *va = static_cast<const uint16_t *>(v_a), *vb = static_cast<const uint16_t *>(v_b);
    const unsigned g = static_cast<unsigned>(blocks);
    const int d = static_cast<int>(D);
    if (design == 0) {
        if (dtype == ASTRA_BF16) merge_recompute_kernel<ASTRA_BF16><<<g, kThreads, 0, st>>>(vo, lse_out, va, lse_a, vb, lse_b, rows, d);
        else merge_recompute_kernel<ASTRA_FP16><<<g, kThreads, 0, st>>>(vo, lse_out, va, lse_a, vb, lse_b, rows, d);
    } else {
        if (dtype == ASTRA_BF16) merge_hoisted_kernel<ASTRA_BF16><<<g, kThreads, 0, st>>>(vo, lse_out, va, lse_a, vb, lse_b, rows, d);
        else merge_hoisted_kernel<ASTRA_FP16><<<g, kThreads, 0, st>>>(vo, lse_out, va, lse_a, vb, lse_b, rows, d);
    }
    return launched();
}

astra_status_t astra_ablation_fused_add_rmsnorm(int design, void *x, void *residual, const void *weight,
                                                int64_t T, int64_t H, float eps,
                                                astra_dtype_t dtype, void *cuda_stream) {
    if (!x || !residual || !weight) return ASTRA_ERR_NULL_POINTER;
    if (dtype != ASTRA_BF16 && dtype != ASTRA_FP16) return ASTRA_ERR_BAD_DTYPE;
    if (design != 0 && design != 1) return ASTRA_ERR_BAD_SHAPE;
    if (T < 0 || T > 2147483647ll || H <= 0 || H > 65536 || (design == 1 && H % 2)) return ASTRA_ERR_BAD_SHAPE;
    if (design == 1 && !(aligned4(x) && aligned4(residual) && aligned4(weight))) return ASTRA_ERR_MISALIGNED;
    if (T == 0) return ASTRA_OK;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    uint16_t *xp = static_cast<uint16_t *>(x), *rp = static_cast<uint16_t *>(residual);
    const uint16_t *wp = static_cast<const uint16_t *>(weight);
    const unsigned g = static_cast<unsigned>(T);
    const int h = static_cast<int>(H);
    if (design == 0) {
        if (dtype == ASTRA_BF16) rmsnorm_tree_kernel<ASTRA_BF16><<<g, kThreads, 0, st>>>(xp, rp, wp, h, eps);
        else rmsnorm_tree_kernel<ASTRA_FP16><<<g, kThreads, 0, st>>>(xp, rp, wp, h, eps);
    } else {
        if (dtype == ASTRA_BF16) rmsnorm_shuffle_kernel<ASTRA_BF16><<<g, kThreads, 0, st>>>(xp, rp, wp, h, eps);
        else rmsnorm_shuffle_kernel<ASTRA_FP16><<<g, kThreads, 0, st>>>(xp, rp, wp, h, eps);
    }
    return launched();
}

astra_status_t astra_ablation_silu_and_mul(int design, void *out, const void *input, int64_t T, int64_t D,
                                           astra_dtype_t dtype, void *cuda_stream) {
    if (!out || !input) return ASTRA_ERR_NULL_POINTER;
    if (dtype != ASTRA_BF16 && dtype != ASTRA_FP16) return ASTRA_ERR_BAD_DTYPE;
    if (design != 0 && design != 1) return ASTRA_ERR_BAD_SHAPE;
    if (T < 0 || D <= 0 || D > (1ll << 30) || (design == 1 && D % 2)) return ASTRA_ERR_BAD_SHAPE;
    if (T > 0 && D > (1ll << 38) / T) return ASTRA_ERR_BAD_SHAPE;
    if (design == 1 && !(aligned4(out) && aligned4(input))) return ASTRA_ERR_MISALIGNED;
    if (T == 0) return ASTRA_OK;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    uint16_t *op = static_cast<uint16_t *>(out);
    const uint16_t *ip = static_cast<const uint16_t *>(input);
    const int64_t total = (design == 0) ? T * D : T * (D / 2);
    const int64_t blocks = (total + kThreads - 1) / kThreads;
    if (blocks > 2147483647ll) return ASTRA_ERR_BAD_SHAPE;
    const unsigned g = static_cast<unsigned>(blocks);
    if (design == 0) {
        if (dtype == ASTRA_BF16) silu_scalar_kernel<ASTRA_BF16><<<g, kThreads, 0, st>>>(op, ip, total, D);
        else silu_scalar_kernel<ASTRA_FP16><<<g, kThreads, 0, st>>>(op, ip, total, D);
    } else {
        if (dtype == ASTRA_BF16) silu_pair_kernel<ASTRA_BF16><<<g, kThreads, 0, st>>>(op, ip, total, D / 2);
        else silu_pair_kernel<ASTRA_FP16><<<g, kThreads, 0, st>>>(op, ip, total, D / 2);
    }
    return launched();
}

}  // extern "C"

// Ablation library (declared in astra_ablation.h).  The paper's case studies (Section 5.3) explain
// its speedups by three contrasts: loop-invariant weights recomputed per element vs derived once;
// a block reduction done entirely in shared memory vs in registers with a short shared-memory
// finish; scalar 16-bit accesses with library math vs 32-bit accesses with fast-math intrinsics.
// Each contrast is built here as a pair of kernels that differ in that one respect only, so the
// effect can be timed on sm_100a.  The kernels are this library's own (grid-stride work
// distribution, block size as a template parameter, reductions that accept any block size); they
// follow the arithmetic readings of the main library (binary32 throughout, one rounding per store)
// so the same parity gates apply.
#include <cuda_runtime.h>

#include "astra_ablation.h"
#include "vec.cuh"

#ifndef ASTRA_BUILD_ID
#define ASTRA_BUILD_ID "unidentified"
#endif
// hash of the sources this library was compiled from; the build script finds it in the file
extern "C" __attribute__((used, visibility("default"))) const char astra_ablation_build_marker[] =
    "astra-build-id:" ASTRA_BUILD_ID;

namespace {

using namespace astra;

constexpr int kBlock = 256;        // threads per block of every kernel here
constexpr int kWavesOfBlocks = 8;  // grid-stride kernels launch at most this many blocks per SM

// ---------------------------------------------------------------------------------------------
// Kernel 1: merge_attn_states_lse.  A warp walks over (token, head) rows; its lanes cover head_dim.
// ---------------------------------------------------------------------------------------------
struct Mix {
    float a, b;  // softmax of the two scores
    float lse;   // log(e^{Sa} + e^{Sb})
};

// Two-way softmax shifted by the larger score (nothing overflows), with library exponentials and
// true divisions: this is the per-row work whose placement the two designs differ in.
__device__ __forceinline__ Mix mix_of(float sa, float sb) {
    const float top = fmaxf(sa, sb);
    if (top == -INFINITY) return Mix{0.f, 0.f, -INFINITY};  // both states empty
    const float ea = expf(sa - top), eb = expf(sb - top);
    const float z = ea + eb;
    return Mix{ea / z, eb / z, top + logf(z)};
}

// A side of weight zero is left out altogether: an empty state may hold anything.
__device__ __forceinline__ float blend(const Mix &m, float va, float vb) {
    float acc = 0.f;
    if (m.a != 0.f) acc = m.a * va;
    if (m.b != 0.f) acc = fmaf(m.b, vb, acc);
    return acc;
}

// HOIST = false: the scores are fetched and the weights derived again for every element (the stores
// in between may alias the scores, so the compiler cannot lift them out either); 16-bit accesses.
// HOIST = true: once per row, ahead of the element loop, which then moves two elements per access.
template <int DT, bool HOIST, int BLOCK>
__global__ void __launch_bounds__(BLOCK)
merge_pair_kernel(uint16_t *v_out, float *lse_out, const uint16_t *v_a, const float *lse_a,
                  const uint16_t *v_b, const float *lse_b, int64_t rows, int D) {
    constexpr int kWarps = BLOCK / 32;
    const int lane = threadIdx.x % 32;
    const int64_t first = static_cast<int64_t>(blockIdx.x) * kWarps + threadIdx.x / 32;
    const int64_t step = static_cast<int64_t>(gridDim.x) * kWarps;
    for (int64_t row = first; row < rows; row += step) {
        const int64_t at = row * D;
        if constexpr (HOIST) {
            const Mix m = mix_of(lse_a[row], lse_b[row]);
            const uint32_t *pa = reinterpret_cast<const uint32_t *>(v_a + at);
            const uint32_t *pb = reinterpret_cast<const uint32_t *>(v_b + at);
            uint32_t *po = reinterpret_cast<uint32_t *>(v_out + at);
            for (int p = lane; 2 * p < D; p += 32) {
                float a_lo, a_hi, b_lo, b_hi;
                Storage<DT>::widen2(pa[p], a_lo, a_hi);
                Storage<DT>::widen2(pb[p], b_lo, b_hi);
                po[p] = Storage<DT>::narrow2(blend(m, a_lo, b_lo), blend(m, a_hi, b_hi));
            }
            if (lane == 0) lse_out[row] = m.lse;
        } else {
            for (int d = lane; d < D; d += 32) {
                const Mix m = mix_of(lse_a[row], lse_b[row]);
                v_out[at + d] = Storage<DT>::narrow1(
                    blend(m, Storage<DT>::widen1(v_a[at + d]), Storage<DT>::widen1(v_b[at + d])));
                if (d == 0) lse_out[row] = m.lse;
            }
        }
    }
}

// ---------------------------------------------------------------------------------------------
// Kernel 2: fused_add_rmsnorm.  A block walks over rows; each row is swept twice (sum of squares,
// then the outputs, so nothing is written before the norm is known).  The pair differs in how the
// per-thread partial sums become the row total, and in the access width.
// ---------------------------------------------------------------------------------------------

// All-shared-memory reduction: every partial goes to shared memory and the live range is folded
// onto its lower part, with a block barrier after each fold, until one value is left.  Any BLOCK
// (an odd live range keeps its middle element for the next fold).
template <int BLOCK>
__device__ __forceinline__ float total_in_shared_memory(float mine, float *scratch) {
    scratch[threadIdx.x] = mine;
    __syncthreads();
    int live = BLOCK;
    while (live > 1) {
        const int kept = (live + 1) / 2;
        if (static_cast<int>(threadIdx.x) + kept < live) scratch[threadIdx.x] += scratch[threadIdx.x + kept];
        __syncthreads();
        live = kept;
    }
    const float total = scratch[0];
    __syncthreads();  // scratch is reused by the next row
    return total;
}

// Register reduction: a butterfly of shuffles leaves the warp's sum in every lane; one value per
// warp passes through shared memory, and the first warp's butterfly over those finishes the job.
template <int BLOCK>
__device__ __forceinline__ float total_in_registers(float mine, float *per_warp) {
    static_assert(BLOCK % 32 == 0 && BLOCK <= 1024, "whole warps, at most 32 of them");
    constexpr int kWarps = BLOCK / 32;
    for (int mask = 1; mask < 32; mask <<= 1) mine += __shfl_xor_sync(0xffffffffu, mine, mask);
    if (threadIdx.x % 32 == 0) per_warp[threadIdx.x / 32] = mine;
    __syncthreads();
    float t = (threadIdx.x % 32) < kWarps ? per_warp[threadIdx.x % 32] : 0.f;
    for (int mask = 1; mask < 32; mask <<= 1) t += __shfl_xor_sync(0xffffffffu, t, mask);
    __syncthreads();  // per_warp is reused by the next row
    return t;
}

template <int DT, bool REGISTERS, int BLOCK>
__global__ void __launch_bounds__(BLOCK)
rmsnorm_pair_kernel(uint16_t *x, uint16_t *residual, const uint16_t *weight, int64_t T, int H, float eps) {
    __shared__ float scratch[REGISTERS ? 32 : BLOCK];
    const float inv_H = 1.0f / static_cast<float>(H);
    for (int64_t row = blockIdx.x; row < T; row += gridDim.x) {
        uint16_t *xr = x + row * H, *rr = residual + row * H;
        float sq = 0.f;
        float rstd;
        if constexpr (REGISTERS) {
            uint32_t *x2 = reinterpret_cast<uint32_t *>(xr), *r2 = reinterpret_cast<uint32_t *>(rr);
            const uint32_t *w2 = reinterpret_cast<const uint32_t *>(weight);
            for (int p = threadIdx.x; 2 * p < H; p += BLOCK) {
                float xa, xb, ra, rb;
                Storage<DT>::widen2(x2[p], xa, xb);
                Storage<DT>::widen2(r2[p], ra, rb);
                const float sa = xa + ra, sb = xb + rb;
                sq = fmaf(sa, sa, sq);
                sq = fmaf(sb, sb, sq);
            }
            rstd = rsqrtf(fmaf(total_in_registers<BLOCK>(sq, scratch), inv_H, eps));
            for (int p = threadIdx.x; 2 * p < H; p += BLOCK) {
                float xa, xb, ra, rb, wa, wb;
                Storage<DT>::widen2(x2[p], xa, xb);
                Storage<DT>::widen2(r2[p], ra, rb);
                Storage<DT>::widen2(w2[p], wa, wb);
                const float sa = xa + ra, sb = xb + rb;
                r2[p] = Storage<DT>::narrow2(sa, sb);
                x2[p] = Storage<DT>::narrow2(sa * rstd * wa, sb * rstd * wb);
            }
        } else {
            for (int j = threadIdx.x; j < H; j += BLOCK) {
                const float s = Storage<DT>::widen1(xr[j]) + Storage<DT>::widen1(rr[j]);
                sq = fmaf(s, s, sq);
            }
            rstd = rsqrtf(fmaf(total_in_shared_memory<BLOCK>(sq, scratch), inv_H, eps));
            for (int j = threadIdx.x; j < H; j += BLOCK) {
                const float s = Storage<DT>::widen1(xr[j]) + Storage<DT>::widen1(rr[j]);
                rr[j] = Storage<DT>::narrow1(s);
                xr[j] = Storage<DT>::narrow1(s * rstd * Storage<DT>::widen1(weight[j]));
            }
        }
    }
}

// ---------------------------------------------------------------------------------------------
// Kernel 3: silu_and_mul, grid-stride over the outputs.  FAST = false: one 16-bit element per
// access, the library exponential and a true division.  FAST = true: two elements per 32-bit
// access, the fast exponential and a reciprocal-multiply in place of the division (the intrinsics
// Section 5.3 names); for gates below about -88 the exponential overflows and the result is -0,
// as with the division.
// ---------------------------------------------------------------------------------------------
template <bool FAST>
__device__ __forceinline__ float gated(float a, float b) {
    if constexpr (FAST) {
        const float sigmoid = __frcp_rn(1.0f + __expf(-a));
        return a * sigmoid * b;
    } else {
        return a / (1.0f + expf(-a)) * b;
    }
}

template <int DT, bool FAST, int BLOCK>
__global__ void __launch_bounds__(BLOCK)
silu_pair_kernel(uint16_t *out, const uint16_t *in, int64_t T, int64_t D) {
    const int64_t per_row = FAST ? D / 2 : D;  // work items per row: element pairs or elements
    const int64_t items = T * per_row;
    const int64_t stride = static_cast<int64_t>(gridDim.x) * BLOCK;
    for (int64_t i = static_cast<int64_t>(blockIdx.x) * BLOCK + threadIdx.x; i < items; i += stride) {
        const int64_t row = i / per_row, col = i - row * per_row;
        if constexpr (FAST) {
            const uint32_t *in2 = reinterpret_cast<const uint32_t *>(in) + row * 2 * per_row;
            float a_lo, a_hi, b_lo, b_hi;
            Storage<DT>::widen2(in2[col], a_lo, a_hi);
            Storage<DT>::widen2(in2[per_row + col], b_lo, b_hi);
            reinterpret_cast<uint32_t *>(out)[i] = Storage<DT>::narrow2(gated<true>(a_lo, b_lo), gated<true>(a_hi, b_hi));
        } else {
            const uint16_t *gate = in + row * 2 * D;
            out[i] = Storage<DT>::narrow1(gated<false>(Storage<DT>::widen1(gate[col]), Storage<DT>::widen1(gate[D + col])));
        }
    }
}

// ---------------------------------------------------------------------------------------------
// host side
// ---------------------------------------------------------------------------------------------
inline bool word_aligned(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 3) == 0; }

// Blocks for `work` block-sized pieces: all of them, up to a few waves per SM (the kernels stride).
inline unsigned grid_for(int64_t work) {
    int dev = 0, sms = 0;
    if (cudaGetDevice(&dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms <= 0)
        sms = 148;
    const int64_t cap = static_cast<int64_t>(sms) * kWavesOfBlocks * (2048 / kBlock);
    return static_cast<unsigned>(work < cap ? (work < 1 ? 1 : work) : cap);
}

template <typename... KArgs, typename... Args>
inline astra_status_t run(void (*kernel)(KArgs...), unsigned grid, cudaStream_t stream, Args... args) {
    // the launch's own return value: an error some other code left pending is neither read nor cleared
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid);
    cfg.blockDim = dim3(kBlock);
    cfg.stream = stream;
    if (cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...) == cudaSuccess) return ASTRA_OK;
    (void)cudaGetLastError();  // the refusal has been reported through the status
    return ASTRA_ERR_CUDA;
}

// Runs CALL with DT bound to the (validated, 16-bit) dtype and VARIANT to the design.
#define ABLATION_DISPATCH(dtype, design, CALL)                                            \
    do {                                                                                  \
        if ((dtype) == ASTRA_BF16) {                                                      \
            constexpr int DT = ASTRA_BF16;                                                \
            if (design) { constexpr bool VARIANT = true; return CALL; }                   \
            constexpr bool VARIANT = false; return CALL;                                  \
        }                                                                                 \
        constexpr int DT = ASTRA_FP16;                                                    \
        if (design) { constexpr bool VARIANT = true; return CALL; }                       \
        constexpr bool VARIANT = false; return CALL;                                      \
    } while (0)

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
    if (design == 1 && !(word_aligned(v_out) && word_aligned(v_a) && word_aligned(v_b))) return ASTRA_ERR_MISALIGNED;
    if (T == 0) return ASTRA_OK;
    const int64_t rows = T * Hh;
    const unsigned grid = grid_for((rows + kBlock / 32 - 1) / (kBlock / 32));
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    uint16_t *vo = static_cast<uint16_t *>(v_out);
    const uint16_t *va = static_cast<const uint16_t *>(v_a), *vb = static_cast<const uint16_t *>(v_b);
    ABLATION_DISPATCH(dtype, design,
                      run(merge_pair_kernel<DT, VARIANT, kBlock>, grid, st, vo, lse_out, va, lse_a, vb, lse_b, rows,
                          static_cast<int>(D)));
}

astra_status_t astra_ablation_fused_add_rmsnorm(int design, void *x, void *residual, const void *weight,
                                                int64_t T, int64_t H, float eps,
                                                astra_dtype_t dtype, void *cuda_stream) {
    if (!x || !residual || !weight) return ASTRA_ERR_NULL_POINTER;
    if (dtype != ASTRA_BF16 && dtype != ASTRA_FP16) return ASTRA_ERR_BAD_DTYPE;
    if (design != 0 && design != 1) return ASTRA_ERR_BAD_SHAPE;
    if (T < 0 || T > 2147483647ll || H <= 0 || H > 65536 || (design == 1 && H % 2)) return ASTRA_ERR_BAD_SHAPE;
    if (design == 1 && !(word_aligned(x) && word_aligned(residual) && word_aligned(weight))) return ASTRA_ERR_MISALIGNED;
    if (T == 0) return ASTRA_OK;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    uint16_t *xp = static_cast<uint16_t *>(x), *rp = static_cast<uint16_t *>(residual);
    const uint16_t *wp = static_cast<const uint16_t *>(weight);
    const unsigned grid = static_cast<unsigned>(T);  // one block per row (the stride loop then runs once)
    ABLATION_DISPATCH(dtype, design,
                      run(rmsnorm_pair_kernel<DT, VARIANT, kBlock>, grid, st, xp, rp, wp, T, static_cast<int>(H), eps));
}

astra_status_t astra_ablation_silu_and_mul(int design, void *out, const void *input, int64_t T, int64_t D,
                                           astra_dtype_t dtype, void *cuda_stream) {
    if (!out || !input) return ASTRA_ERR_NULL_POINTER;
    if (dtype != ASTRA_BF16 && dtype != ASTRA_FP16) return ASTRA_ERR_BAD_DTYPE;
    if (design != 0 && design != 1) return ASTRA_ERR_BAD_SHAPE;
    if (T < 0 || D <= 0 || D > (1ll << 30) || (design == 1 && D % 2)) return ASTRA_ERR_BAD_SHAPE;
    if (T > 0 && D > (1ll << 38) / T) return ASTRA_ERR_BAD_SHAPE;
    if (design == 1 && !(word_aligned(out) && word_aligned(input))) return ASTRA_ERR_MISALIGNED;
    if (T == 0) return ASTRA_OK;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    uint16_t *op = static_cast<uint16_t *>(out);
    const uint16_t *ip = static_cast<const uint16_t *>(input);
    const int64_t items = design == 0 ? T * D : T * (D / 2);
    const unsigned grid = grid_for((items + kBlock - 1) / kBlock);
    ABLATION_DISPATCH(dtype, design, run(silu_pair_kernel<DT, VARIANT, kBlock>, grid, st, op, ip, T, D));
}

}  // extern "C"

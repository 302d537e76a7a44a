// C ABI of the library (declared in astra.h): argument validation, launch-shape selection per
// width / alignment / row count, and the kernel launches.  Nothing here allocates, synchronises or
// keeps state; every failure is reported as a status code before anything is launched.
#include <cuda_runtime.h>

#include "astra.h"
#include "fused_add_rmsnorm.cuh"
#include "merge_attn_states_lse.cuh"
#include "silu_and_mul.cuh"

namespace {

using namespace astra;

inline bool aligned(const void *p, size_t bytes) {
    return (reinterpret_cast<uintptr_t>(p) % bytes) == 0;
}

// [a, a+na) and [b, b+nb) intersect
inline bool overlaps(const void *a, int64_t na, const void *b, int64_t nb) {
    const uintptr_t a0 = reinterpret_cast<uintptr_t>(a), b0 = reinterpret_cast<uintptr_t>(b);
    return a0 < b0 + static_cast<uintptr_t>(nb) && b0 < a0 + static_cast<uintptr_t>(na);
}

// Largest vector width (in elements, up to max_vec) such that `width` is a multiple of it and every
// pointer is aligned to it.  Rows start at multiples of `width` elements, so this makes every
// vector access in every row aligned.
template <typename... P>
inline int pick_vec(int max_vec, int64_t width, P... ptrs) {
    for (int vec = max_vec; vec > 1; vec >>= 1) {
        if (width % vec != 0) continue;
        const bool ok = (aligned(ptrs, static_cast<size_t>(vec) * 2) && ...);
        if (ok) return vec;
    }
    return 1;
}

inline astra_status_t launch_status() {
    return cudaGetLastError() == cudaSuccess ? ASTRA_OK : ASTRA_ERR_CUDA;
}

// Every kernel is launched with programmatic stream serialization allowed: its blocks may be
// scheduled while the previous kernel in the stream drains, and they wait (griddepcontrol.wait)
// for that kernel to complete before their first global access.  Stream order is unchanged; the
// launch latency and block prologue of back-to-back calls overlap the previous kernel's tail.
template <typename... KArgs, typename... Args>
inline void launch(void (*kernel)(KArgs...), unsigned grid, unsigned block, cudaStream_t stream,
                   Args... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid);
    cfg.blockDim = dim3(block);
    cfg.dynamicSmemBytes = 0;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    (void)cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);  // failure is read back by launch_status()
}

constexpr int64_t kMaxVecsPerLaunch = (1ll << 31) - 1;  // flat vector indices are 31-bit

// ---------------------------------------------------------------------------------------------
// silu_and_mul
// ---------------------------------------------------------------------------------------------
template <int DT, int VEC, int UNROLL, int THREADS>
void launch_silu(uint16_t *out, const uint16_t *in, int64_t T, int64_t D, cudaStream_t stream) {
    const int64_t nvec = D / VEC;
    const int64_t rows_per_launch = kMaxVecsPerLaunch / nvec;
    for (int64_t t0 = 0; t0 < T; t0 += rows_per_launch) {
        const int64_t rows = (T - t0 < rows_per_launch) ? (T - t0) : rows_per_launch;
        const uint32_t total = static_cast<uint32_t>(rows * nvec);
        const uint32_t tile = THREADS * UNROLL;
        const uint32_t blocks = (total + tile - 1) / tile;
        launch(silu_and_mul_kernel<DT, VEC, UNROLL, THREADS>, blocks, THREADS, stream,
               out + t0 * D, in + t0 * 2 * D, total, FastDiv::make(static_cast<uint32_t>(nvec)), D);
    }
}

template <int DT>
void dispatch_silu(uint16_t *out, const uint16_t *in, int64_t T, int64_t D, cudaStream_t stream) {
    // each row is [a | b]: a starts at 2*D*t and b at 2*D*t + D, so D itself must be a multiple of VEC
    // One 16-byte vector per thread and 256-thread blocks: the smallest work quantum that still
    // keeps the block scheduler ahead, which gives the shortest drain at the end of the grid.
    switch (pick_vec(8, D, out, in)) {
        case 8: launch_silu<DT, 8, 1, 256>(out, in, T, D, stream); break;
        case 4: launch_silu<DT, 4, 4, 256>(out, in, T, D, stream); break;
        case 2: launch_silu<DT, 2, 4, 256>(out, in, T, D, stream); break;
        default: launch_silu<DT, 1, 4, 256>(out, in, T, D, stream); break;
    }
}

// ---------------------------------------------------------------------------------------------
// merge_attn_states_lse
// ---------------------------------------------------------------------------------------------
template <int DT, int VEC, int UNROLL, int THREADS>
void launch_merge(uint16_t *v_out, float *lse_out, const uint16_t *v_a, const float *lse_a,
                  const uint16_t *v_b, const float *lse_b, int64_t rows_total, int64_t D,
                  cudaStream_t stream) {
    const int64_t nvec = D / VEC;
    const int64_t rows_per_launch = kMaxVecsPerLaunch / nvec;
    for (int64_t r0 = 0; r0 < rows_total; r0 += rows_per_launch) {
        const int64_t rows = (rows_total - r0 < rows_per_launch) ? (rows_total - r0) : rows_per_launch;
        const uint32_t total = static_cast<uint32_t>(rows * nvec);
        const uint32_t tile = THREADS * UNROLL;
        const uint32_t blocks = (total + tile - 1) / tile;
        launch(merge_attn_states_lse_kernel<DT, VEC, UNROLL, THREADS>, blocks, THREADS, stream,
               v_out + r0 * D, lse_out ? lse_out + r0 : nullptr, v_a + r0 * D, lse_a + r0, v_b + r0 * D,
               lse_b + r0, total, FastDiv::make(static_cast<uint32_t>(nvec)));
    }
}

template <int DT>
void dispatch_merge(uint16_t *v_out, float *lse_out, const uint16_t *v_a, const float *lse_a,
                    const uint16_t *v_b, const float *lse_b, int64_t rows, int64_t D,
                    cudaStream_t stream) {
    switch (pick_vec(16, D, v_out, v_a, v_b)) {
        case 16: launch_merge<DT, 16, 1, 256>(v_out, lse_out, v_a, lse_a, v_b, lse_b, rows, D, stream); break;
        case 8: launch_merge<DT, 8, 2, 256>(v_out, lse_out, v_a, lse_a, v_b, lse_b, rows, D, stream); break;
        case 4: launch_merge<DT, 4, 4, 256>(v_out, lse_out, v_a, lse_a, v_b, lse_b, rows, D, stream); break;
        case 2: launch_merge<DT, 2, 4, 256>(v_out, lse_out, v_a, lse_a, v_b, lse_b, rows, D, stream); break;
        default: launch_merge<DT, 1, 4, 256>(v_out, lse_out, v_a, lse_a, v_b, lse_b, rows, D, stream); break;
    }
}

// ---------------------------------------------------------------------------------------------
// fused_add_rmsnorm
// ---------------------------------------------------------------------------------------------
constexpr int kMaxGridX = 2147483647;

inline int round_up(int v, int m) { return (v + m - 1) / m * m; }

template <int DT, int VEC, int VPT>
inline void launch_rmsnorm_reg(unsigned rows, int threads, cudaStream_t stream, uint16_t *x, uint16_t *r,
                               const uint16_t *w, int H, float eps, float inv_H) {
    // at most 64 elements per thread are ever selected; wider combinations are not instantiated
    if constexpr (VEC * VPT <= 64)
        launch(fused_add_rmsnorm_reg_kernel<DT, VEC, VPT>, rows, threads, stream, x, r, w, H, eps, inv_H);
}

// Register-resident rows: VPT vectors per thread with blockDim = ceil(nvec / VPT) rounded up to a warp.
// 16 elements per thread (32 bytes of x and of r in flight per thread) with 256..1024 threads
// measured best; up to 64 elements per thread are used for wider rows, with the block size capped
// so the row still fits the register file.  Rows wider than that take the two-sweep kernel.
template <int DT, int VEC>
void launch_rmsnorm(uint16_t *x, uint16_t *r, const uint16_t *w, int64_t T, int H, float eps,
                    cudaStream_t stream) {
    const int nvec = H / VEC;
    const float inv_H = 1.0f / static_cast<float>(H);
    // start at 16 elements per thread; widen the per-thread share only if the row needs more
    // threads than that share allows, narrow it if the block would fall under 128 threads
    int vpt = 16 / VEC < 1 ? 1 : 16 / VEC;
    auto threads_for = [&](int v) { return round_up((nvec + v - 1) / v, 32); };
    while (vpt < 64 / VEC && threads_for(vpt) > rmsnorm_reg_max_threads(VEC, vpt)) vpt <<= 1;
    while (vpt > 1 && threads_for(vpt) < 128) vpt >>= 1;
    const int threads = threads_for(vpt);
    const bool fits = threads <= rmsnorm_reg_max_threads(VEC, vpt);
    for (int64_t t0 = 0; t0 < T; t0 += kMaxGridX) {
        const unsigned rows = static_cast<unsigned>(T - t0 < kMaxGridX ? T - t0 : kMaxGridX);
        uint16_t *xs = x + t0 * H, *rs = r + t0 * H;
        if (!fits) {
            launch(fused_add_rmsnorm_twopass_kernel<DT, VEC>, rows, 1024, stream, xs, rs, w, H, eps, inv_H);
            continue;
        }
        switch (vpt) {
            case 1: launch_rmsnorm_reg<DT, VEC, 1>(rows, threads, stream, xs, rs, w, H, eps, inv_H); break;
            case 2: launch_rmsnorm_reg<DT, VEC, 2>(rows, threads, stream, xs, rs, w, H, eps, inv_H); break;
            case 4: launch_rmsnorm_reg<DT, VEC, 4>(rows, threads, stream, xs, rs, w, H, eps, inv_H); break;
            case 8: launch_rmsnorm_reg<DT, VEC, 8>(rows, threads, stream, xs, rs, w, H, eps, inv_H); break;
            case 16: launch_rmsnorm_reg<DT, VEC, 16>(rows, threads, stream, xs, rs, w, H, eps, inv_H); break;
            case 32: launch_rmsnorm_reg<DT, VEC, 32>(rows, threads, stream, xs, rs, w, H, eps, inv_H); break;
            default: launch_rmsnorm_reg<DT, VEC, 64>(rows, threads, stream, xs, rs, w, H, eps, inv_H); break;
        }
    }
}

template <int DT>
void dispatch_rmsnorm(uint16_t *x, uint16_t *r, const uint16_t *w, int64_t T, int H, float eps,
                      cudaStream_t stream) {
    switch (pick_vec(8, H, x, r, w)) {
        case 8: launch_rmsnorm<DT, 8>(x, r, w, T, H, eps, stream); break;
        case 4: launch_rmsnorm<DT, 4>(x, r, w, T, H, eps, stream); break;
        case 2: launch_rmsnorm<DT, 2>(x, r, w, T, H, eps, stream); break;
        default: launch_rmsnorm<DT, 1>(x, r, w, T, H, eps, stream); break;
    }
}

inline bool valid_dtype(astra_dtype_t d) { return d == ASTRA_BF16 || d == ASTRA_FP16; }

}  // namespace

extern "C" {

astra_status_t astra_fused_add_rmsnorm(void *x, void *residual, const void *weight, int64_t T,
                                       int64_t H, float eps, astra_dtype_t dtype, void *cuda_stream) {
    if (!x || !residual || !weight) return ASTRA_ERR_NULL_POINTER;
    if (!valid_dtype(dtype)) return ASTRA_ERR_BAD_DTYPE;
    if (T < 0 || H <= 0 || H > 2147483647ll) return ASTRA_ERR_BAD_SHAPE;
    if (T > 0 && H > INT64_MAX / 2 / T) return ASTRA_ERR_BAD_SHAPE;
    if (!aligned(x, 2) || !aligned(residual, 2) || !aligned(weight, 2)) return ASTRA_ERR_MISALIGNED;
    if (T == 0) return ASTRA_OK;
    const int64_t bytes = T * H * 2;
    if (overlaps(x, bytes, residual, bytes) || overlaps(x, bytes, weight, H * 2) ||
        overlaps(residual, bytes, weight, H * 2))
        return ASTRA_ERR_OVERLAP;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    uint16_t *xp = static_cast<uint16_t *>(x), *rp = static_cast<uint16_t *>(residual);
    const uint16_t *wp = static_cast<const uint16_t *>(weight);
    if (dtype == ASTRA_BF16)
        dispatch_rmsnorm<ASTRA_BF16>(xp, rp, wp, T, static_cast<int>(H), eps, stream);
    else
        dispatch_rmsnorm<ASTRA_FP16>(xp, rp, wp, T, static_cast<int>(H), eps, stream);
    return launch_status();
}

astra_status_t astra_silu_and_mul(void *out, const void *input, int64_t T, int64_t D,
                                  astra_dtype_t dtype, void *cuda_stream) {
    if (!out || !input) return ASTRA_ERR_NULL_POINTER;
    if (!valid_dtype(dtype)) return ASTRA_ERR_BAD_DTYPE;
    if (T < 0 || D <= 0 || D > 1073741823ll) return ASTRA_ERR_BAD_SHAPE;
    if (T > 0 && D > INT64_MAX / 4 / T) return ASTRA_ERR_BAD_SHAPE;
    if (!aligned(out, 2) || !aligned(input, 2)) return ASTRA_ERR_MISALIGNED;
    if (T == 0) return ASTRA_OK;
    if (overlaps(out, T * D * 2, input, T * D * 4)) return ASTRA_ERR_OVERLAP;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    uint16_t *op = static_cast<uint16_t *>(out);
    const uint16_t *ip = static_cast<const uint16_t *>(input);
    if (dtype == ASTRA_BF16)
        dispatch_silu<ASTRA_BF16>(op, ip, T, D, stream);
    else
        dispatch_silu<ASTRA_FP16>(op, ip, T, D, stream);
    return launch_status();
}

astra_status_t astra_merge_attn_states_lse(void *v_out, float *lse_out, const void *v_a,
                                           const float *lse_a, const void *v_b, const float *lse_b,
                                           int64_t T, int64_t Hh, int64_t D, astra_dtype_t dtype,
                                           void *cuda_stream) {
    if (!v_out || !v_a || !v_b || !lse_a || !lse_b) return ASTRA_ERR_NULL_POINTER;
    if (!valid_dtype(dtype)) return ASTRA_ERR_BAD_DTYPE;
    if (T < 0 || Hh <= 0 || D <= 0 || D > 2147483647ll) return ASTRA_ERR_BAD_SHAPE;
    if (T > 0 && (Hh > INT64_MAX / 4 / T || D > INT64_MAX / 4 / (T * Hh))) return ASTRA_ERR_BAD_SHAPE;
    if (!aligned(v_out, 2) || !aligned(v_a, 2) || !aligned(v_b, 2) || !aligned(lse_a, 4) ||
        !aligned(lse_b, 4) || (lse_out && !aligned(lse_out, 4)))
        return ASTRA_ERR_MISALIGNED;
    if (T == 0) return ASTRA_OK;
    const int64_t rows = T * Hh;
    const int64_t vbytes = rows * D * 2, sbytes = rows * 4;
    if ((v_out != v_a && overlaps(v_out, vbytes, v_a, vbytes)) ||
        (v_out != v_b && overlaps(v_out, vbytes, v_b, vbytes)))
        return ASTRA_ERR_OVERLAP;
    if (overlaps(v_out, vbytes, lse_a, sbytes) || overlaps(v_out, vbytes, lse_b, sbytes))
        return ASTRA_ERR_OVERLAP;
    if (lse_out && (overlaps(lse_out, sbytes, lse_a, sbytes) || overlaps(lse_out, sbytes, lse_b, sbytes) ||
                    overlaps(lse_out, sbytes, v_a, vbytes) || overlaps(lse_out, sbytes, v_b, vbytes) ||
                    overlaps(lse_out, sbytes, v_out, vbytes)))
        return ASTRA_ERR_OVERLAP;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    uint16_t *vo = static_cast<uint16_t *>(v_out);
    const uint16_t *va = static_cast<const uint16_t *>(v_a), *vb = static_cast<const uint16_t *>(v_b);
    if (dtype == ASTRA_BF16)
        dispatch_merge<ASTRA_BF16>(vo, lse_out, va, lse_a, vb, lse_b, rows, D, stream);
    else
        dispatch_merge<ASTRA_FP16>(vo, lse_out, va, lse_a, vb, lse_b, rows, D, stream);
    return launch_status();
}

const char *astra_status_string(astra_status_t status) {
    switch (status) {
        case ASTRA_OK: return "ok";
        case ASTRA_ERR_NULL_POINTER: return "a required pointer is NULL";
        case ASTRA_ERR_BAD_SHAPE: return "an extent is negative, zero where not allowed, or too large";
        case ASTRA_ERR_BAD_DTYPE: return "unknown dtype";
        case ASTRA_ERR_MISALIGNED: return "a pointer is not aligned to its element size";
        case ASTRA_ERR_CUDA: return "the CUDA runtime reported an error at launch";
        case ASTRA_ERR_OVERLAP: return "an output overlaps an input in a way that is not allowed";
        default: return "unknown status";
    }
}

}  // extern "C"

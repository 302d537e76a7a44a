// C ABI of the library (declared in astra.h): argument validation, launch-shape selection per
// width / alignment / row count, and the kernel launches.  Nothing here allocates, synchronises or
// keeps state.  Argument errors are reported before anything is launched; a launch the runtime
// refuses is reported as ASTRA_ERR_CUDA from that launch's own return value (the thread's sticky
// "last error" of the CUDA runtime is neither read nor cleared on the success path), and the
// remaining launches of a split call are not issued.
#include <cuda_runtime.h>

#include "astra.h"
#include "fused_add_rmsnorm.cuh"
#include "launch.cuh"
#include "merge_attn_states_lse.cuh"
#include "silu_and_mul.cuh"

#ifndef ASTRA_BUILD_ID
#define ASTRA_BUILD_ID "unidentified"
#endif

namespace {

using namespace astra;
using namespace astra::host;

// Hash of the sources this library was compiled from (set by the build script), behind a marker
// that can also be found in the file without loading it.
const char kBuildId[] = "astra-build-id:" ASTRA_BUILD_ID;


// ---------------------------------------------------------------------------------------------
// silu_and_mul
// ---------------------------------------------------------------------------------------------
// D, the pitches and the pointers are in 16-bit units; UVEC is the vector width in units.
// Above this many blocks a launch runs long enough that its ramp-up no longer shows, and the extra
// prefetch requests only cost issue slots (measured, L2-cold: 24 % faster at [128, 14336], 5 % at
// [1024, 14336] = 7168 blocks, 0.5 % at [4096, 14336], 1.6 % slower at [8192, 14336] = 57344 blocks);
// below it the inputs are requested ahead of the dependency wait.
constexpr uint32_t kSiluPrefetchMaxBlocks = 1u << 14;
// Range of grid sizes (in 256-thread blocks of one 32-byte vector per thread) in which the 32-byte
// form is used: from 640 blocks (measured: slower at 448, faster at 896) to 8192 (faster at 7168,
// slower at 14336).
constexpr int64_t kSiluWideMinBlocks = 640;
constexpr int64_t kSiluWideMaxBlocks = 8192;

template <int DT, int UVEC, int UNROLL, int THREADS>
cudaError_t launch_silu(uint16_t *out, const uint16_t *gate, const uint16_t *up, int64_t T, int64_t D,
                        int64_t out_pitch, int64_t gate_pitch, int64_t up_pitch, cudaStream_t stream) {
  if constexpr (UVEC >= Storage<DT>::UNITS) {
    constexpr int VEC = UVEC / Storage<DT>::UNITS;
    const int64_t nvec = D / UVEC;
    const int64_t rows_per_launch = kMaxVecsPerLaunch / nvec;
    for (int64_t t0 = 0; t0 < T; t0 += rows_per_launch) {
        const int64_t rows = (T - t0 < rows_per_launch) ? (T - t0) : rows_per_launch;
        const uint32_t total = static_cast<uint32_t>(rows * nvec);
        const uint32_t tile = THREADS * UNROLL;
        const uint32_t blocks = (total + tile - 1) / tile;
        const FastDiv per_row = FastDiv::make(static_cast<uint32_t>(nvec));
        cudaError_t err;
        if (UVEC >= 8 && blocks <= kSiluPrefetchMaxBlocks)
            err = launch(silu_and_mul_kernel<DT, VEC, UNROLL, THREADS, Ld::StreamReadOnly, St::Stream, THREADS * UNROLL>,
                         blocks, THREADS, stream, out + t0 * out_pitch, gate + t0 * gate_pitch, up + t0 * up_pitch,
                         total, per_row, out_pitch, gate_pitch, up_pitch);
        else
            err = launch(silu_and_mul_kernel<DT, VEC, UNROLL, THREADS, Ld::StreamReadOnly, St::Stream, 0>, blocks,
                         THREADS, stream, out + t0 * out_pitch, gate + t0 * gate_pitch, up + t0 * up_pitch, total,
                         per_row, out_pitch, gate_pitch, up_pitch);
        if (err != cudaSuccess) return err;
    }
  }
  return cudaSuccess;
}

template <int DT>
cudaError_t dispatch_silu(uint16_t *out, const uint16_t *gate, const uint16_t *up, int64_t T, int64_t D,
                   int64_t out_pitch, int64_t gate_pitch, int64_t up_pitch, cudaStream_t stream) {
    int vec = VecPick(16).extent(D).extent(out_pitch).extent(gate_pitch).extent(up_pitch)
                  .pointer(out).pointer(gate).pointer(up).vec;
    // One 16-byte vector per thread and 256-thread blocks: the smallest work quantum that still
    // keeps the block scheduler ahead, which gives the shortest drain at the end of the grid.
    // Between about one and ten waves of blocks, one 32-byte vector per thread (half as many blocks,
    // each still prefetching its share ahead of the dependency wait) is faster where everything is
    // 32-byte aligned: 4.21 -> 3.83 us at [256, 14336], 7.19 -> 6.73 us at [512, 14336], 13.2 -> 12.6 us
    // at [1024, 14336], 25.2 -> 24.8 us at [2048, 14336] (L2-cold, bf16); it is slower below that
    // (2.56 -> 3.14 us at [128, 14336]) and above it (98.3 -> 99.9 us at [8192, 14336]).
    if (vec == 16) {
        const int64_t blocks_wide = (T * (D / 16) + 255) / 256;
        if (blocks_wide >= kSiluWideMinBlocks && blocks_wide <= kSiluWideMaxBlocks)
            return launch_silu<DT, 16, 1, 256>(out, gate, up, T, D, out_pitch, gate_pitch, up_pitch, stream);
        vec = 8;  // everything that is 32-byte aligned is 16-byte aligned
    }
    switch (vec) {
        case 8: return launch_silu<DT, 8, 1, 256>(out, gate, up, T, D, out_pitch, gate_pitch, up_pitch, stream);
        case 4: return launch_silu<DT, 4, 4, 256>(out, gate, up, T, D, out_pitch, gate_pitch, up_pitch, stream);
        case 2: return launch_silu<DT, 2, 4, 256>(out, gate, up, T, D, out_pitch, gate_pitch, up_pitch, stream);
        default: return launch_silu<DT, 1, 4, 256>(out, gate, up, T, D, out_pitch, gate_pitch, up_pitch, stream);
    }
}

astra_status_t silu_entry(void *out, const void *gate, const void *up, int64_t T, int64_t D,
                          int64_t out_pitch, int64_t gate_pitch, int64_t up_pitch,
                          astra_dtype_t dtype, void *cuda_stream) {
    if (!valid_dtype(dtype)) return ASTRA_ERR_BAD_DTYPE;
    if (T < 0 || D <= 0 || D > 1073741823ll) return ASTRA_ERR_BAD_SHAPE;
    if (out_pitch < D || gate_pitch < D || up_pitch < D) return ASTRA_ERR_BAD_SHAPE;
    const int64_t max_pitch = out_pitch > gate_pitch ? (out_pitch > up_pitch ? out_pitch : up_pitch)
                                                     : (gate_pitch > up_pitch ? gate_pitch : up_pitch);
    if (T > 0 && max_pitch > kInt64Max / 4 / T) return ASTRA_ERR_BAD_SHAPE;
    if (T == 0) return ASTRA_OK;  // an empty batch has no data to point at: its pointers are not examined
    if (!out || !gate || !up) return ASTRA_ERR_NULL_POINTER;
    const int64_t U = units_per_elem(dtype);
    const size_t eb = static_cast<size_t>(2 * U);
    if (!aligned(out, eb) || !aligned(gate, eb) || !aligned(up, eb)) return ASTRA_ERR_MISALIGNED;
    const int64_t Du = D * U, opu = out_pitch * U, gpu = gate_pitch * U, upu = up_pitch * U;  // in units
    if (pitched_overlap(out, opu, gate, gpu, T, Du) || pitched_overlap(out, opu, up, upu, T, Du))
        return ASTRA_ERR_OVERLAP;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    uint16_t *op = static_cast<uint16_t *>(out);
    const uint16_t *gp = static_cast<const uint16_t *>(gate), *upp = static_cast<const uint16_t *>(up);
    cudaError_t err = cudaSuccess;
    ASTRA_FOR_DTYPE(dtype, err = dispatch_silu<DT>(op, gp, upp, T, Du, opu, gpu, upu, stream));
    return launch_status(err);
}

// ---------------------------------------------------------------------------------------------
// merge_attn_states_lse
// ---------------------------------------------------------------------------------------------
// D and the value pointers are in 16-bit units; UVEC is the vector width in units.
template <int DT, int UVEC, int UNROLL, int THREADS>
cudaError_t launch_merge(uint16_t *v_out, float *lse_out, const uint16_t *v_a, const float *lse_a,
                  const uint16_t *v_b, const float *lse_b, int64_t rows_total, int64_t D,
                  cudaStream_t stream) {
  if constexpr (UVEC >= Storage<DT>::UNITS) {
    constexpr int VEC = UVEC / Storage<DT>::UNITS;
    const int64_t nvec = D / UVEC;
    const int64_t rows_per_launch = kMaxVecsPerLaunch / nvec;
    for (int64_t r0 = 0; r0 < rows_total; r0 += rows_per_launch) {
        const int64_t rows = (rows_total - r0 < rows_per_launch) ? (rows_total - r0) : rows_per_launch;
        const uint32_t total = static_cast<uint32_t>(rows * nvec);
        const uint32_t tile = THREADS * UNROLL;
        const uint32_t blocks = (total + tile - 1) / tile;
        const cudaError_t err =
            launch(merge_attn_states_lse_kernel<DT, VEC, UNROLL, THREADS>, blocks, THREADS, stream,
                   v_out + r0 * D, lse_out ? lse_out + r0 : nullptr, v_a + r0 * D, lse_a + r0, v_b + r0 * D,
                   lse_b + r0, total, FastDiv::make(static_cast<uint32_t>(nvec)));
        if (err != cudaSuccess) return err;
    }
  }
  return cudaSuccess;
}

template <int DT>
cudaError_t dispatch_merge(uint16_t *v_out, float *lse_out, const uint16_t *v_a, const float *lse_a,
                    const uint16_t *v_b, const float *lse_b, int64_t rows, int64_t D,
                    cudaStream_t stream) {
    // 32-byte accesses measured best here (one per thread, 256-thread blocks)
    switch (VecPick(16).extent(D).pointer(v_out).pointer(v_a).pointer(v_b).vec) {
        case 16: return launch_merge<DT, 16, 1, 256>(v_out, lse_out, v_a, lse_a, v_b, lse_b, rows, D, stream);
        case 8: return launch_merge<DT, 8, 2, 256>(v_out, lse_out, v_a, lse_a, v_b, lse_b, rows, D, stream);
        case 4: return launch_merge<DT, 4, 4, 256>(v_out, lse_out, v_a, lse_a, v_b, lse_b, rows, D, stream);
        case 2: return launch_merge<DT, 2, 4, 256>(v_out, lse_out, v_a, lse_a, v_b, lse_b, rows, D, stream);
        default: return launch_merge<DT, 1, 4, 256>(v_out, lse_out, v_a, lse_a, v_b, lse_b, rows, D, stream);
    }
}

template <int DT, int UVEC, int UNROLL, int THREADS>
cudaError_t launch_merge_strided(uint16_t *v_out, float *lse_out, const uint16_t *v_a, const float *lse_a,
                          const uint16_t *v_b, const float *lse_b, int64_t rows_total, int64_t Hh,
                          int64_t D, const MergeStrides &st, cudaStream_t stream) {
  if constexpr (UVEC >= Storage<DT>::UNITS) {
    constexpr int VEC = UVEC / Storage<DT>::UNITS;
    const int64_t nvec = D / UVEC;
    const int64_t rows_per_launch = kMaxVecsPerLaunch / nvec;
    for (int64_t r0 = 0; r0 < rows_total; r0 += rows_per_launch) {
        const int64_t rows = (rows_total - r0 < rows_per_launch) ? (rows_total - r0) : rows_per_launch;
        const uint32_t total = static_cast<uint32_t>(rows * nvec);
        const uint32_t tile = THREADS * UNROLL;
        const uint32_t blocks = (total + tile - 1) / tile;
        const cudaError_t err =
            launch(merge_attn_states_lse_strided_kernel<DT, VEC, UNROLL, THREADS>, blocks, THREADS, stream,
                   v_out, lse_out, v_a, lse_a, v_b, lse_b, total, static_cast<uint32_t>(r0),
                   FastDiv::make(static_cast<uint32_t>(nvec)), FastDiv::make(static_cast<uint32_t>(Hh)), st);
        if (err != cudaSuccess) return err;
    }
  }
  return cudaSuccess;
}

template <int DT>
cudaError_t dispatch_merge_strided(uint16_t *v_out, float *lse_out, const uint16_t *v_a, const float *lse_a,
                            const uint16_t *v_b, const float *lse_b, int64_t rows, int64_t Hh, int64_t D,
                            const MergeStrides &st, cudaStream_t stream) {
    const int vec = VecPick(16).extent(D).extent(st.va_t).extent(st.va_h).extent(st.vb_t).extent(st.vb_h)
                        .extent(st.vo_t).extent(st.vo_h).pointer(v_out).pointer(v_a).pointer(v_b).vec;
    switch (vec) {
        case 16: return launch_merge_strided<DT, 16, 1, 256>(v_out, lse_out, v_a, lse_a, v_b, lse_b, rows, Hh, D, st, stream);
        case 8: return launch_merge_strided<DT, 8, 2, 256>(v_out, lse_out, v_a, lse_a, v_b, lse_b, rows, Hh, D, st, stream);
        case 4: return launch_merge_strided<DT, 4, 4, 256>(v_out, lse_out, v_a, lse_a, v_b, lse_b, rows, Hh, D, st, stream);
        case 2: return launch_merge_strided<DT, 2, 4, 256>(v_out, lse_out, v_a, lse_a, v_b, lse_b, rows, Hh, D, st, stream);
        default: return launch_merge_strided<DT, 1, 4, 256>(v_out, lse_out, v_a, lse_a, v_b, lse_b, rows, Hh, D, st, stream);
    }
}

// One past the largest element offset of a [T, Hh, W] tensor addressed by (token, head) strides.
inline int64_t strided_extent(int64_t T, int64_t Hh, int64_t W, int64_t st, int64_t sh) {
    return (T - 1) * st + (Hh - 1) * sh + W;
}

// The (token, head) rows of W contiguous elements must not overlap one another: with the smaller
// stride s1 over n1 steps and the larger s2, require s1 >= W (or n1 == 1) and s2 >= extent of the
// inner dimension (or n2 == 1).
inline bool rows_disjoint(int64_t T, int64_t Hh, int64_t W, int64_t st, int64_t sh) {
    int64_t n1 = Hh, s1 = sh, n2 = T, s2 = st;
    if ((n1 > 1 && n2 > 1 && s1 > s2) || n1 == 1) {
        int64_t tn = n1, ts = s1;
        n1 = n2; s1 = s2; n2 = tn; s2 = ts;
    }
    if (n1 > 1 && s1 < W) return false;
    if (n2 > 1 && s2 < (n1 - 1) * s1 + W) return false;
    return true;
}

// ---------------------------------------------------------------------------------------------
// fused_add_rmsnorm
// ---------------------------------------------------------------------------------------------
constexpr int kMaxGridX = ASTRA_MAX_ROWS_PER_LAUNCH;
constexpr int64_t kOneWaveRows = 2 * 148;  // rows below which the grid is a fraction of one wave on the 148 SMs of a B200

// Most 16-bit units of a row one thread keeps in registers: 64 with vector accesses, 8 on the
// scalar path (each element then also costs three separate packed-input registers).
constexpr int rmsnorm_max_units_per_thread(int uvec) { return uvec == 1 ? 8 : 64; }

inline int round_up(int v, int m) { return (v + m - 1) / m * m; }

template <int DT, int UVEC, int VPT>
inline cudaError_t launch_rmsnorm_reg(unsigned rows, int threads, cudaStream_t stream, const RmsnormOperands &op,
                                      const uint16_t *w, int H, float eps, float inv_H) {
    // wider combinations than the per-thread cap are never selected and are not instantiated
    if constexpr (UVEC * VPT <= rmsnorm_max_units_per_thread(UVEC))
        return launch(fused_add_rmsnorm_reg_kernel<DT, UVEC / Storage<DT>::UNITS, VPT>, rows, threads, stream, op,
                      w, H, eps, inv_H);
    return cudaErrorInvalidValue;
}

// Register-resident rows: VPT vectors per thread with blockDim = ceil(nvec / VPT) rounded up to a warp.
// 16 units per thread (32 bytes of x and of r in flight per thread) with 256..1024 threads measured
// best; up to 64 units per thread are used for wider rows, with the block size capped so the row
// still fits the register file.  Rows wider than that take the two-sweep kernel.
// H is in elements; the operands' pointers and pitches are in 16-bit units; UVEC is the vector width
// in units.
template <int DT, int UVEC>
cudaError_t launch_rmsnorm(RmsnormOperands op, const uint16_t *w, int64_t T, int H, float eps, cudaStream_t stream) {
  if constexpr (UVEC >= Storage<DT>::UNITS) {
    constexpr int VEC = UVEC / Storage<DT>::UNITS;
    constexpr int kMaxVpt = rmsnorm_max_units_per_thread(UVEC) / UVEC;
    const int nvec = H / VEC;
    const float inv_H = 1.0f / static_cast<float>(H);
    // start at 16 units per thread; widen the per-thread share only if the row needs more threads
    // than that share allows, narrow it if the block would fall under 128 threads
    int vpt = UVEC == 1 ? 8 : 16 / UVEC;
    auto threads_for = [&](int v) { return round_up((nvec + v - 1) / v, 32); };
    while (vpt < kMaxVpt && threads_for(vpt) > rmsnorm_reg_max_threads(UVEC * vpt)) vpt <<= 1;
    while (vpt > 1 && threads_for(vpt) < 128) vpt >>= 1;
    // Streaming sizes (more rows than one wave of blocks) with 16-byte vectors: 32 units per thread in
    // blocks of 128..256 threads (H = 4096 .. 8192 for the 16-bit types) measured 1-5 % faster than 16
    // units per thread, L2-cold, at T = 1024 and 8192 (7.9 -> 7.5 us at [1024, 5120], 79.6 -> 78.6 us
    // at [8192, 8192]); wider rows and decode-sized batches did not gain.
    if (UVEC == 8 && vpt == 2 && T > kOneWaveRows && threads_for(4) >= 128 && threads_for(4) <= 256) vpt = 4;
    const int threads = threads_for(vpt);
    const bool fits = threads <= rmsnorm_reg_max_threads(UVEC * vpt);
    // Wider rows: share the row among a cluster of 2, 4 or 8 blocks (the portable maximum), each
    // holding 16 units per thread; only beyond 8 x 1024 x 16 units per row fall back to two sweeps.
    constexpr int kClusterVpt = (16 / UVEC < 1 ? 1 : 16 / UVEC);
    int cluster = 0, cluster_threads = 0;
    if (!fits && UVEC >= 4) {  // vector paths only; scalar and 4-byte rows take the two-sweep kernel
        for (int c = 2; c <= 8; c <<= 1) {
            const int chunk = (nvec + c - 1) / c;
            const int th = round_up((chunk + kClusterVpt - 1) / kClusterVpt, 32);
            if (th > rmsnorm_reg_max_threads(UVEC * kClusterVpt)) continue;
            if (cluster != 0 && cluster_threads <= ASTRA_CLUSTER_PREFERRED_THREADS) break;
            cluster = c;
            cluster_threads = th;
        }
    }
    // two-sweep fallback: as few strided iterations per thread as 1024 threads allow, evenly filled
    const int sweep_iters = (nvec + 1023) / 1024;
    const int sweep_threads = round_up((nvec + sweep_iters - 1) / sweep_iters, 32);
    const int64_t rows_per_launch = cluster ? kMaxGridX / cluster : kMaxGridX;
    for (int64_t t0 = 0; t0 < T; t0 += rows_per_launch) {
        const unsigned rows = static_cast<unsigned>(T - t0 < rows_per_launch ? T - t0 : rows_per_launch);
        RmsnormOperands o = op;
        o.x += t0 * op.x_pitch;
        o.r += t0 * op.r_pitch;
        o.y += t0 * op.y_pitch;
        o.r_out += t0 * op.r_out_pitch;
        cudaError_t err = cudaSuccess;
        if (cluster) {
            if constexpr (UVEC >= 4)
                err = launch_clustered(fused_add_rmsnorm_cluster_kernel<DT, VEC, kClusterVpt>, rows * cluster,
                                       cluster_threads, cluster, stream, o, w, H, eps, inv_H);
        } else if (!fits) {
            err = launch(fused_add_rmsnorm_twopass_kernel<DT, VEC>, rows, sweep_threads, stream, o, w, H, eps, inv_H);
        } else {
            switch (vpt) {
                case 1: err = launch_rmsnorm_reg<DT, UVEC, 1>(rows, threads, stream, o, w, H, eps, inv_H); break;
                case 2: err = launch_rmsnorm_reg<DT, UVEC, 2>(rows, threads, stream, o, w, H, eps, inv_H); break;
                case 4: err = launch_rmsnorm_reg<DT, UVEC, 4>(rows, threads, stream, o, w, H, eps, inv_H); break;
                case 8: err = launch_rmsnorm_reg<DT, UVEC, 8>(rows, threads, stream, o, w, H, eps, inv_H); break;
                case 16: err = launch_rmsnorm_reg<DT, UVEC, 16>(rows, threads, stream, o, w, H, eps, inv_H); break;
                case 32: err = launch_rmsnorm_reg<DT, UVEC, 32>(rows, threads, stream, o, w, H, eps, inv_H); break;
                default: err = launch_rmsnorm_reg<DT, UVEC, 64>(rows, threads, stream, o, w, H, eps, inv_H); break;
            }
        }
        if (err != cudaSuccess) return err;
    }
  }
  return cudaSuccess;
}

// Streaming sizes whose rows are 32-byte aligned throughout: the same 32 units per thread as two
// 32-byte vectors instead of four 16-byte ones (68 registers, half the memory instructions).
// Measured L2-cold against the 16-byte form, bf16: 11.36 -> 11.08 us at [2048, 4096], 40.3 -> 39.8 us at
// [8192, 4096], 13.7 -> 13.5 / 50.1 -> 49.6 us at [2048 / 8192, 5120], 0.2-0.4 % at H = 8192, 6.48 -> 6.39 us
// at [1024, 4096]; 1-2 % slower at [512, 5120] and [512, 8192] and no different at or below one wave of
// rows, so the 16-byte forms stay below 1024 rows.  Blocks of 64 to 448 threads, i.e. H = 2048 ... 14336
// for the 16-bit types (also measured: 21.4 -> 20.6 us at [8192, 2048], 104.4 -> 103.9 us at
// [8192, 11008], 136.7 -> 135.8 us at [8192, 14336], 18.7 -> 18.4 us at [1024, 14336]); wider rows would
// leave one 512-thread block per SM and keep 16 units per thread at full occupancy instead.
// The same form also wins at decode sizes, where its blocks of half as many warps start and reduce
// faster (device time from a graph, bf16: 1.61 -> 1.39 us at [1, 4096], 1.70 -> 1.49 us at [16, 4096],
// 2.09 -> 1.87 us at [16, 8192], 1.58 -> 1.45 us at [16, 2048]); at 64 to 768 rows it is level or slower
// (1.77 -> 1.94 us at [64, 4096], 3.38 -> 3.53 us at [256, 8192]).
constexpr int64_t kWideVectorDecodeRows = 16;
#ifndef ASTRA_RMSNORM_WIDE_VECTOR_ROWS
#define ASTRA_RMSNORM_WIDE_VECTOR_ROWS 1024
#endif
constexpr int64_t kWideVectorRows = ASTRA_RMSNORM_WIDE_VECTOR_ROWS;
template <int DT>
bool launch_rmsnorm_wide(const RmsnormOperands &op, const uint16_t *w, int64_t T, int H, float eps,
                         cudaStream_t stream, cudaError_t *err) {
    constexpr int UVEC = 16, VEC = UVEC / Storage<DT>::UNITS, VPT = 2;
    const int nvec = H / VEC;
    const int threads = round_up((nvec + VPT - 1) / VPT, 32);
    if ((T > kWideVectorDecodeRows && T < kWideVectorRows) || threads < 64 || threads > 448) return false;
    const float inv_H = 1.0f / static_cast<float>(H);
    *err = cudaSuccess;
    for (int64_t t0 = 0; t0 < T && *err == cudaSuccess; t0 += kMaxGridX) {
        const unsigned rows = static_cast<unsigned>(T - t0 < kMaxGridX ? T - t0 : kMaxGridX);
        RmsnormOperands o = op;
        o.x += t0 * op.x_pitch;
        o.r += t0 * op.r_pitch;
        o.y += t0 * op.y_pitch;
        o.r_out += t0 * op.r_out_pitch;
        *err = launch(fused_add_rmsnorm_reg_kernel<DT, VEC, VPT>, rows, threads, stream, o, w, H, eps, inv_H);
    }
    return true;
}

template <int DT>
cudaError_t dispatch_rmsnorm(const RmsnormOperands &op, const uint16_t *w, int64_t T, int H, float eps,
                      cudaStream_t stream) {
    int vec = VecPick(16).extent(static_cast<int64_t>(H) * Storage<DT>::UNITS).extent(op.x_pitch)
                  .extent(op.r_pitch).extent(op.y_pitch).extent(op.r_out_pitch).pointer(op.x)
                  .pointer(op.r).pointer(op.y).pointer(op.r_out).pointer(w).vec;
    if (vec == 16) {
        cudaError_t err = cudaSuccess;
        if (launch_rmsnorm_wide<DT>(op, w, T, H, eps, stream, &err)) return err;
        vec = 8;  // everything that is 32-byte aligned is 16-byte aligned
    }
    switch (vec) {
        case 8: return launch_rmsnorm<DT, 8>(op, w, T, H, eps, stream);
        case 4: return launch_rmsnorm<DT, 4>(op, w, T, H, eps, stream);
        case 2: return launch_rmsnorm<DT, 2>(op, w, T, H, eps, stream);
        default: return launch_rmsnorm<DT, 1>(op, w, T, H, eps, stream);
    }
}

astra_status_t rmsnorm_entry(void *y, void *residual_out, const void *x, const void *residual,
                             const void *weight, int64_t T, int64_t H, int64_t y_pitch,
                             int64_t ro_pitch, int64_t x_pitch, int64_t r_pitch, float eps,
                             astra_dtype_t dtype, void *cuda_stream) {
    if (!valid_dtype(dtype)) return ASTRA_ERR_BAD_DTYPE;
    const int64_t U = units_per_elem(dtype);
    // a row is indexed in 16-bit units with 32-bit integers inside the kernels
    if (T < 0 || H <= 0 || H > kMaxRowUnits / U) return ASTRA_ERR_BAD_SHAPE;
    if (y_pitch < H || ro_pitch < H || x_pitch < H || r_pitch < H) return ASTRA_ERR_BAD_SHAPE;
    int64_t max_pitch = y_pitch;
    if (ro_pitch > max_pitch) max_pitch = ro_pitch;
    if (x_pitch > max_pitch) max_pitch = x_pitch;
    if (r_pitch > max_pitch) max_pitch = r_pitch;
    if (T > 0 && max_pitch > kInt64Max / 4 / T) return ASTRA_ERR_BAD_SHAPE;
    if (T == 0) return ASTRA_OK;
    if (!y || !residual_out || !x || !residual || !weight) return ASTRA_ERR_NULL_POINTER;
    const size_t eb = static_cast<size_t>(2 * U);
    if (!aligned(y, eb) || !aligned(residual_out, eb) || !aligned(x, eb) || !aligned(residual, eb) ||
        !aligned(weight, eb))
        return ASTRA_ERR_MISALIGNED;
    // from here on widths and pitches are in 16-bit units
    const int64_t Hu = H * U;
    y_pitch *= U;
    ro_pitch *= U;
    x_pitch *= U;
    r_pitch *= U;
    const bool y_is_x = (y == x && y_pitch == x_pitch);
    const bool ro_is_r = (residual_out == residual && ro_pitch == r_pitch);
    // the weight is one row: compare it against every output as a [T, H] tensor of pitch 0 would be
    // wrong (pitch < width), so use the outputs' spans for it
    const int64_t sy = span_bytes(T, Hu, y_pitch, 2), sro = span_bytes(T, Hu, ro_pitch, 2), sw = Hu * 2;
    if ((!y_is_x && pitched_overlap(y, y_pitch, x, x_pitch, T, Hu)) ||
        pitched_overlap(y, y_pitch, residual, r_pitch, T, Hu) ||
        pitched_overlap(y, y_pitch, residual_out, ro_pitch, T, Hu) || overlaps(y, sy, weight, sw) ||
        (!ro_is_r && pitched_overlap(residual_out, ro_pitch, residual, r_pitch, T, Hu)) ||
        pitched_overlap(residual_out, ro_pitch, x, x_pitch, T, Hu) || overlaps(residual_out, sro, weight, sw))
        return ASTRA_ERR_OVERLAP;
    RmsnormOperands op;
    op.x = static_cast<const uint16_t *>(x);
    op.r = static_cast<const uint16_t *>(residual);
    op.y = static_cast<uint16_t *>(y);
    op.r_out = static_cast<uint16_t *>(residual_out);
    op.x_pitch = x_pitch;
    op.r_pitch = r_pitch;
    op.y_pitch = y_pitch;
    op.r_out_pitch = ro_pitch;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    const uint16_t *wp = static_cast<const uint16_t *>(weight);
    cudaError_t err = cudaSuccess;
    ASTRA_FOR_DTYPE(dtype, err = dispatch_rmsnorm<DT>(op, wp, T, static_cast<int>(H), eps, stream));
    return launch_status(err);
}

}  // namespace

extern "C" {

astra_status_t astra_fused_add_rmsnorm(void *x, void *residual, const void *weight, int64_t T,
                                       int64_t H, float eps, astra_dtype_t dtype, void *cuda_stream) {
    return rmsnorm_entry(x, residual, x, residual, weight, T, H, H, H, H, H, eps, dtype, cuda_stream);
}

astra_status_t astra_fused_add_rmsnorm_ex(void *y, void *residual_out, const void *x,
                                          const void *residual, const void *weight, int64_t T,
                                          int64_t H, int64_t y_pitch, int64_t residual_out_pitch,
                                          int64_t x_pitch, int64_t residual_pitch, float eps,
                                          astra_dtype_t dtype, void *cuda_stream) {
    return rmsnorm_entry(y, residual_out, x, residual, weight, T, H, y_pitch, residual_out_pitch,
                         x_pitch, residual_pitch, eps, dtype, cuda_stream);
}

astra_status_t astra_silu_and_mul(void *out, const void *input, int64_t T, int64_t D,
                                  astra_dtype_t dtype, void *cuda_stream) {
    if (!valid_dtype(dtype)) return ASTRA_ERR_BAD_DTYPE;
    if (T < 0 || D <= 0 || D > 1073741823ll) return ASTRA_ERR_BAD_SHAPE;
    if (T == 0) return ASTRA_OK;
    if (!input) return ASTRA_ERR_NULL_POINTER;
    const void *up = static_cast<const uint16_t *>(input) + D * units_per_elem(dtype);
    return silu_entry(out, input, up, T, D, D, 2 * D, 2 * D, dtype, cuda_stream);
}

astra_status_t astra_silu_and_mul_ex(void *out, const void *gate, const void *up, int64_t T,
                                     int64_t D, int64_t out_pitch, int64_t gate_pitch,
                                     int64_t up_pitch, astra_dtype_t dtype, void *cuda_stream) {
    return silu_entry(out, gate, up, T, D, out_pitch, gate_pitch, up_pitch, dtype, cuda_stream);
}

astra_status_t astra_merge_attn_states_lse(void *v_out, float *lse_out, const void *v_a,
                                           const float *lse_a, const void *v_b, const float *lse_b,
                                           int64_t T, int64_t Hh, int64_t D, astra_dtype_t dtype,
                                           void *cuda_stream) {
    if (!valid_dtype(dtype)) return ASTRA_ERR_BAD_DTYPE;
    if (T < 0 || Hh <= 0 || D <= 0 || D > 1073741823ll) return ASTRA_ERR_BAD_SHAPE;
    if (T > 0 && (Hh > kInt64Max / 4 / T || D > kInt64Max / 4 / (T * Hh))) return ASTRA_ERR_BAD_SHAPE;
    if (T == 0) return ASTRA_OK;
    if (!v_out || !v_a || !v_b || !lse_a || !lse_b) return ASTRA_ERR_NULL_POINTER;
    const int64_t U = units_per_elem(dtype);
    const size_t eb = static_cast<size_t>(2 * U);
    if (!aligned(v_out, eb) || !aligned(v_a, eb) || !aligned(v_b, eb) || !aligned(lse_a, 4) ||
        !aligned(lse_b, 4) || (lse_out && !aligned(lse_out, 4)))
        return ASTRA_ERR_MISALIGNED;
    const int64_t rows = T * Hh;
    const int64_t Du = D * U;  // row width in 16-bit units
    const int64_t vbytes = rows * Du * 2, sbytes = rows * 4;
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
    cudaError_t err = cudaSuccess;
    ASTRA_FOR_DTYPE(dtype, err = dispatch_merge<DT>(vo, lse_out, va, lse_a, vb, lse_b, rows, Du, stream));
    return launch_status(err);
}

astra_status_t astra_merge_attn_states_lse_ex(void *v_out, float *lse_out, const void *v_a,
                                              const float *lse_a, const void *v_b, const float *lse_b,
                                              int64_t T, int64_t Hh, int64_t D, const int64_t *strides,
                                              astra_dtype_t dtype, void *cuda_stream) {
    if (!valid_dtype(dtype)) return ASTRA_ERR_BAD_DTYPE;
    if (T < 0 || Hh <= 0 || D <= 0 || D > 1073741823ll || Hh > 2147483647ll) return ASTRA_ERR_BAD_SHAPE;
    if (T > 0 && Hh > 2147483647ll / T) return ASTRA_ERR_BAD_SHAPE;  // T * Hh must stay below 2^31
    if (T == 0) return ASTRA_OK;
    if (!v_out || !v_a || !v_b || !lse_a || !lse_b || !strides) return ASTRA_ERR_NULL_POINTER;
    for (int i = 0; i < 12; ++i) {
        if (lse_out == nullptr && i >= 10) break;
        // every offset (T-1)*stride, (Hh-1)*stride must stay far inside int64
        const int64_t steps = (i % 2 == 0 ? T : Hh) - 1;
        if (strides[i] < 0 || (steps > 0 && strides[i] > (1ll << 60) / steps)) return ASTRA_ERR_BAD_SHAPE;
    }
    const int64_t U = units_per_elem(dtype);
    const size_t eb = static_cast<size_t>(2 * U);
    const int64_t Du = D * U;  // row width and value strides in 16-bit units from here on
    MergeStrides st;
    st.va_t = strides[0] * U; st.va_h = strides[1] * U; st.vb_t = strides[2] * U; st.vb_h = strides[3] * U;
    st.vo_t = strides[4] * U; st.vo_h = strides[5] * U; st.sa_t = strides[6]; st.sa_h = strides[7];
    st.sb_t = strides[8]; st.sb_h = strides[9];
    st.so_t = lse_out ? strides[10] : 0;
    st.so_h = lse_out ? strides[11] : 0;
    if (!aligned(v_out, eb) || !aligned(v_a, eb) || !aligned(v_b, eb) || !aligned(lse_a, 4) ||
        !aligned(lse_b, 4) || (lse_out && !aligned(lse_out, 4)))
        return ASTRA_ERR_MISALIGNED;
    // written tensors must have non-overlapping rows; read tensors may broadcast (stride 0)
    if (!rows_disjoint(T, Hh, Du, st.vo_t, st.vo_h)) return ASTRA_ERR_BAD_SHAPE;
    if (lse_out && !rows_disjoint(T, Hh, 1, st.so_t, st.so_h)) return ASTRA_ERR_BAD_SHAPE;
    const int64_t bva = strided_extent(T, Hh, Du, st.va_t, st.va_h) * 2;
    const int64_t bvb = strided_extent(T, Hh, Du, st.vb_t, st.vb_h) * 2;
    const int64_t bvo = strided_extent(T, Hh, Du, st.vo_t, st.vo_h) * 2;
    const int64_t bsa = strided_extent(T, Hh, 1, st.sa_t, st.sa_h) * 4;
    const int64_t bsb = strided_extent(T, Hh, 1, st.sb_t, st.sb_h) * 4;
    const int64_t bso = lse_out ? strided_extent(T, Hh, 1, st.so_t, st.so_h) * 4 : 0;
    const bool out_is_a = (v_out == v_a && st.vo_t == st.va_t && st.vo_h == st.va_h);
    const bool out_is_b = (v_out == v_b && st.vo_t == st.vb_t && st.vo_h == st.vb_h);
    if ((!out_is_a && overlaps(v_out, bvo, v_a, bva)) || (!out_is_b && overlaps(v_out, bvo, v_b, bvb)) ||
        overlaps(v_out, bvo, lse_a, bsa) || overlaps(v_out, bvo, lse_b, bsb))
        return ASTRA_ERR_OVERLAP;
    if (lse_out && (overlaps(lse_out, bso, lse_a, bsa) || overlaps(lse_out, bso, lse_b, bsb) ||
                    overlaps(lse_out, bso, v_a, bva) || overlaps(lse_out, bso, v_b, bvb) ||
                    overlaps(lse_out, bso, v_out, bvo)))
        return ASTRA_ERR_OVERLAP;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    uint16_t *vo = static_cast<uint16_t *>(v_out);
    const uint16_t *va = static_cast<const uint16_t *>(v_a), *vb = static_cast<const uint16_t *>(v_b);
    const int64_t rows = T * Hh;
    cudaError_t err = cudaSuccess;
    ASTRA_FOR_DTYPE(dtype, err = dispatch_merge_strided<DT>(vo, lse_out, va, lse_a, vb, lse_b, rows, Hh, Du, st, stream));
    return launch_status(err);
}

const char *astra_build_id(void) { return kBuildId + sizeof("astra-build-id:") - 1; }

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

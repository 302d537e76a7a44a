// C ABI of astra_fused_allreduce_add_rmsnorm (declared in astra.h): argument validation, launch-shape
// selection and the kernel launch.  Same conventions as the rest of the library: nothing is
// allocated, nothing synchronises, errors are status codes.
#include <cuda_runtime.h>

#include "astra.h"
#include "fused_allreduce_add_rmsnorm.cuh"
#include "launch.cuh"

namespace {

using namespace astra;
using namespace astra::host;

inline int round_up_to(int v, int m) { return (v + m - 1) / m * m; }

// Register-resident rows hold at most 32 16-bit units per thread in vectors of 8, 16 or 32 bytes.
// UVEC is the vector width in units, VPT the vectors per thread.
// `dense` selects the instantiation whose registers are capped so that five 256-thread blocks fit an
// SM; it exists for the streaming shape (two loads in flight, 16 units per thread) only.
template <int DT, int UVEC, int VPT, int GROUP>
cudaError_t launch_reg(const AllreduceOperands &op, const uint16_t *w, unsigned rows, int threads, int H,
                       float eps, float inv_H, bool dense, cudaStream_t stream) {
    if constexpr (UVEC >= 4 && UVEC >= Storage<DT>::UNITS && UVEC * VPT <= 32) {
        if constexpr (GROUP == 2 && UVEC == 8 && VPT == 2) {  // the measured case: 16-byte vectors, no spill at 48 registers
            if (dense && threads <= kAllreduceDenseThreads)
                return launch(fused_allreduce_add_rmsnorm_reg_kernel<DT, UVEC / Storage<DT>::UNITS, VPT, GROUP, true>,
                              rows, threads, stream, op, w, H, eps, inv_H);
        }
        return launch(fused_allreduce_add_rmsnorm_reg_kernel<DT, UVEC / Storage<DT>::UNITS, VPT, GROUP>, rows,
                      threads, stream, op, w, H, eps, inv_H);
    }
    return cudaErrorInvalidValue;
}

// Launch shapes of the 16-byte forms (operands that are not 32-byte aligned throughout; the 32-byte
// forms further down serve everything else, at every row count), chosen by the number of rows
// (measured at H = 4096 with 2, 4 and 8 partials):
//  - streaming (more rows than one wave of blocks holds): two partial loads in flight per vector
//    position and 16 units per thread (256-thread blocks at H = 4096).  It beat four and eight in
//    flight and every other per-thread share by 3 to 25 % at [1024, 4096] and [8192, 4096]: the
//    registers of a deeper queue cost more occupancy than the queue gains.
//  - latency (at most one wave: decode-sized batches, where this fusion matters most): up to eight
//    partial loads in flight and 8 units per thread (512-thread blocks), so that all partials of a
//    row arrive in one round trip: 2.5 against 3.9 us at [16, 4096] with 8 partials (with one or two
//    partials the queue stays at two, the per-thread share is still 8 units: 1.8 against 2.0 us).
constexpr int kStreamGroup = 2;
constexpr int kLatencyGroup = 8;
#ifndef ASTRA_ALLREDUCE_LATENCY_ROWS
#define ASTRA_ALLREDUCE_LATENCY_ROWS (2 * 148)
#endif
constexpr int64_t kLatencyRows = ASTRA_ALLREDUCE_LATENCY_ROWS;  // two 512-thread blocks per SM on the 148 SMs of a B200
// From this many rows on the streaming shape runs in its register-capped form (five resident blocks
// per SM instead of four): 1-2 % faster at [8192, 4096], neutral to 3 % slower at [1024, 4096].
constexpr int64_t kDenseRows = 4096;

// Per-thread share of a register-resident row for a given width, or 0 if the row does not fit:
// start at `start_units` 16-bit units; double the share while the block would exceed what the
// register file allows; halve it while the block would fall under 128 threads.
template <int UVEC, int GROUP>
inline int pick_vpt(int nvec, int start_units, int *threads_out) {
    if (UVEC < 4) return 0;  // 2- and 4-byte vectors take the two-sweep kernel
    constexpr int kMaxVpt = 32 / (UVEC < 4 ? 4 : UVEC);
    auto threads_for = [&](int v) { return round_up_to((nvec + v - 1) / v, 32); };
    int vpt = start_units / UVEC;
    if (vpt < 1) vpt = 1;
    while (vpt <= kMaxVpt && threads_for(vpt) > allreduce_reg_max_threads(UVEC * vpt, GROUP)) vpt <<= 1;
    if (vpt > kMaxVpt) return 0;
    while (vpt > 1 && threads_for(vpt) < 128) vpt >>= 1;
    *threads_out = threads_for(vpt);
    return vpt;
}

// Launches over all rows (split where the grid limit requires).  vpt = 0 selects the two-sweep kernel.
template <int DT, int UVEC, int GROUP>
cudaError_t launch_rows(AllreduceOperands op, const uint16_t *w, int64_t T, int H, float eps, int vpt,
                        int threads, cudaStream_t stream) {
  if constexpr (UVEC >= Storage<DT>::UNITS) {
    constexpr int VEC = UVEC / Storage<DT>::UNITS;
    const int nvec = H / VEC;
    const float inv_H = 1.0f / static_cast<float>(H);
    const int sweep_iters = (nvec + 1023) / 1024;
    const int sweep_threads = round_up_to((nvec + sweep_iters - 1) / sweep_iters, 32);
    const int64_t row_units = static_cast<int64_t>(H) * Storage<DT>::UNITS;
    const int64_t rows_per_launch = kMaxRowsPerLaunch;
    const bool dense = T >= kDenseRows;
    for (int64_t t0 = 0; t0 < T; t0 += rows_per_launch) {
        const unsigned rows = static_cast<unsigned>(T - t0 < rows_per_launch ? T - t0 : rows_per_launch);
        AllreduceOperands o = op;
        for (int p = 0; p < kMaxParts; ++p) {  // unused slots repeat slot 0, so every slot moves along
            o.part[p] += t0 * row_units;
            o.y_out[p] += t0 * row_units;
            o.r_out[p] += t0 * row_units;
        }
        o.r += t0 * row_units;
        cudaError_t err;
        switch (vpt) {
            case 0: err = launch(fused_allreduce_add_rmsnorm_twopass_kernel<DT, VEC, GROUP>, rows, sweep_threads,
                                 stream, o, w, H, eps, inv_H); break;
            case 1: err = launch_reg<DT, UVEC, 1, GROUP>(o, w, rows, threads, H, eps, inv_H, dense, stream); break;
            case 2: err = launch_reg<DT, UVEC, 2, GROUP>(o, w, rows, threads, H, eps, inv_H, dense, stream); break;
            case 4: err = launch_reg<DT, UVEC, 4, GROUP>(o, w, rows, threads, H, eps, inv_H, dense, stream); break;
            default: err = launch_reg<DT, UVEC, 8, GROUP>(o, w, rows, threads, H, eps, inv_H, dense, stream); break;
        }
        if (err != cudaSuccess) return err;
    }
  }
  return cudaSuccess;
}

template <int DT, int UVEC>
cudaError_t choose_shape(const AllreduceOperands &op, const uint16_t *w, int64_t T, int H, float eps,
                         cudaStream_t stream) {
  if constexpr (UVEC >= Storage<DT>::UNITS) {
    const int nvec = H / (UVEC / Storage<DT>::UNITS);
    int threads = 0;
    if (T <= kLatencyRows && op.n_parts > kStreamGroup) {
        const int vpt = pick_vpt<UVEC, kLatencyGroup>(nvec, 8, &threads);
        if (vpt > 0) return launch_rows<DT, UVEC, kLatencyGroup>(op, w, T, H, eps, vpt, threads, stream);
    }
    const int start_units = T <= kLatencyRows ? 8 : 16;
    const int vpt = pick_vpt<UVEC, kStreamGroup>(nvec, start_units, &threads);  // 0: the row does not fit the registers
    return launch_rows<DT, UVEC, kStreamGroup>(op, w, T, H, eps, vpt, threads, stream);
  }
  return cudaErrorInvalidValue;
}

// Streaming sizes whose operands are 32-byte aligned throughout: 32-byte accesses.  Measured L2-cold
// against the 16-byte form at [8192, 4096]: 50.6 -> 49.2 us with 2 partials, 70.8 -> 66.6 us with 4,
// 110.9 -> 104.7 us with 8; at [1024, 4096]: 8.3 -> 7.7, 10.9 -> 10.3, 16.2 -> 15.9 us.
//
// Four shapes: one or two vectors per thread (16 or 32 units), two or four partial loads in flight
// (four only from four partials on).  What decides between them is how many bytes of loads an SM has
// in flight, i.e. resident blocks x threads x bytes per thread, with the resident blocks set by the
// registers (56 / 96 / 72 / 128 per thread as compiled for sm_100a, allocated in eights, 65536 per
// SM).  The measurements across H = 2048 ... 16384 fit one rule: take the first shape, in the order
// below, that keeps about 90 KB in flight per SM; if none does, the one with the most.  Examples:
// H = 4096 takes one vector and four in flight (three 256-thread blocks per SM); H = 8192 with four
// in flight would leave one 512-thread block per SM, so it takes two vectors in 256-thread blocks
// (78.8 -> 68.0 us with 4 partials, 117.3 -> 105.6 us with 8); H = 10240 with two in flight takes two
// vectors in 320-thread blocks (two per SM) rather than one 640-thread block (61.6 against 76.7 us);
// H = 16384 takes one vector in one 1024-thread block (143.1 against 155.8 us with 4 partials).
// Returns false where no shape applies (rows too narrow for 128-thread blocks, or too wide).
struct WideShape {
    int vpt, group, regs, max_threads, min_threads;
};
#ifndef ASTRA_ALLREDUCE_DEEP_QUEUE_ROWS
#define ASTRA_ALLREDUCE_DEEP_QUEUE_ROWS 128
#endif
constexpr int64_t kDeepQueueRows = ASTRA_ALLREDUCE_DEEP_QUEUE_ROWS;
constexpr WideShape kWideShapes[] = {
    {1, 4, 72, 512, 128}, {2, 4, 128, 256, 64}, {1, 2, 56, 1024, 128}, {2, 2, 96, 512, 64}};
constexpr int64_t kWideBytesInFlight = 90 * 1024;

template <int DT>
bool launch_wide(const AllreduceOperands &op, const uint16_t *w, int64_t T, int H, float eps, cudaStream_t stream,
                 cudaError_t *err) {
    constexpr int UVEC = 16;
    const int nvec = H / (UVEC / Storage<DT>::UNITS);
    // Few rows and more than four partials: all of a row's partials in one round trip (eight loads in
    // flight, one vector per thread); with so few blocks the registers that costs do not matter.
    // Device time from a graph, 8 partials, against the streaming shapes: 3.19 -> 2.70 us at [16, 4096],
    // 4.17 -> 3.41 us at [16, 8192], 4.12 -> 3.85 us at [128, 4096]; slower from 192 rows on (7.93 -> 8.89 us
    // at [192, 8192]).  With up to four partials the streaming shapes are the fastest at every row
    // count (1.65 / 1.98 us at [16, 4096] with 2 / 4 partials, where the 16-byte shapes took 2.08 / 2.40).
    if (T <= kDeepQueueRows && op.n_parts > 4) {
        const int threads = round_up_to(nvec, 32);
        if (threads >= 128 && threads <= allreduce_reg_max_threads(16, kLatencyGroup)) {
            *err = launch_rows<DT, UVEC, kLatencyGroup>(op, w, T, H, eps, 1, threads, stream);
            return true;
        }
    }
    int best = -1, best_threads = 0;
    int64_t best_bytes = 0;
    for (int c = 0; c < 4; ++c) {
        const WideShape &sh = kWideShapes[c];
        if (sh.group > kStreamGroup && op.n_parts < sh.group) continue;
        const int threads = round_up_to((nvec + sh.vpt - 1) / sh.vpt, 32);
        if (threads > sh.max_threads || threads < sh.min_threads) continue;
        const int by_regs = 65536 / (sh.regs * threads), by_threads = 2048 / threads;
        const int blocks = by_regs < by_threads ? by_regs : by_threads;
        const int64_t bytes = static_cast<int64_t>(blocks) * threads * sh.vpt * (sh.group + 1) * 32;
        if (bytes > best_bytes) {
            best = c;
            best_bytes = bytes;
            best_threads = threads;
        }
        if (bytes >= kWideBytesInFlight) break;  // the first shape that reaches it is also the largest so far
    }
    if (best < 0) return false;
    const WideShape &sh = kWideShapes[best];
    if (sh.group == 4)
        *err = launch_rows<DT, UVEC, 4>(op, w, T, H, eps, sh.vpt, best_threads, stream);
    else
        *err = launch_rows<DT, UVEC, kStreamGroup>(op, w, T, H, eps, sh.vpt, best_threads, stream);
    return true;
}

template <int DT>
cudaError_t dispatch(const AllreduceOperands &op, const uint16_t *w, int64_t T, int H, float eps,
                     cudaStream_t stream) {
    VecPick pick(16);
    pick.extent(static_cast<int64_t>(H) * Storage<DT>::UNITS).pointer(op.r).pointer(w);
    for (int p = 0; p < op.n_parts; ++p) pick.pointer(op.part[p]);
    for (int d = 0; d < op.n_y; ++d) pick.pointer(op.y_out[d]);
    for (int d = 0; d < op.n_r; ++d) pick.pointer(op.r_out[d]);
    if (pick.vec == 16) {
        cudaError_t err = cudaSuccess;
        if (launch_wide<DT>(op, w, T, H, eps, stream, &err)) return err;
        pick.vec = 8;  // everything that is 32-byte aligned is 16-byte aligned
    }
    switch (pick.vec) {
        case 8: return choose_shape<DT, 8>(op, w, T, H, eps, stream);
        case 4: return choose_shape<DT, 4>(op, w, T, H, eps, stream);
        case 2: return choose_shape<DT, 2>(op, w, T, H, eps, stream);
        default: return choose_shape<DT, 1>(op, w, T, H, eps, stream);
    }
}

// Shared by the two entry points.  y_outs / r_outs: n_y / n_r destinations of the normalised rows and
// of the new residual; `residual` is the residual input, which one of r_outs may be exactly.
astra_status_t allreduce_entry(void *const *y_outs, int32_t n_y, void *const *r_outs, int32_t n_r,
                               const void *residual, const void *const *x_parts, int32_t n_parts,
                               const void *weight, int64_t T, int64_t H, float eps, astra_dtype_t dtype,
                               void *cuda_stream) {
    if (!valid_dtype(dtype)) return ASTRA_ERR_BAD_DTYPE;
    const int64_t U = units_per_elem(dtype);
    if (n_parts < 1 || n_parts > kMaxParts || n_y < 1 || n_y > kMaxParts || n_r < 1 || n_r > kMaxParts)
        return ASTRA_ERR_BAD_SHAPE;
    if (T < 0 || H <= 0 || H > kMaxRowUnits / U) return ASTRA_ERR_BAD_SHAPE;
    if (T > 0 && H > kInt64Max / 4 / T) return ASTRA_ERR_BAD_SHAPE;
    if (T == 0) return ASTRA_OK;
    if (!y_outs || !r_outs || !residual || !x_parts || !weight) return ASTRA_ERR_NULL_POINTER;
    for (int p = 0; p < n_parts; ++p)
        if (!x_parts[p]) return ASTRA_ERR_NULL_POINTER;
    for (int d = 0; d < n_y; ++d)
        if (!y_outs[d]) return ASTRA_ERR_NULL_POINTER;
    for (int d = 0; d < n_r; ++d)
        if (!r_outs[d]) return ASTRA_ERR_NULL_POINTER;
    const size_t eb = static_cast<size_t>(2 * U);
    if (!aligned(residual, eb) || !aligned(weight, eb)) return ASTRA_ERR_MISALIGNED;
    for (int p = 0; p < n_parts; ++p)
        if (!aligned(x_parts[p], eb)) return ASTRA_ERR_MISALIGNED;
    for (int d = 0; d < n_y; ++d)
        if (!aligned(y_outs[d], eb)) return ASTRA_ERR_MISALIGNED;
    for (int d = 0; d < n_r; ++d)
        if (!aligned(r_outs[d], eb)) return ASTRA_ERR_MISALIGNED;
    // Every destination overlaps nothing else, except that a residual destination may be exactly the
    // residual input.  (Memory of another GPU has addresses in the same unified space, so the
    // byte-range test is meaningful for it too.)  Partials may overlap one another: they are only read.
    const int64_t bytes = T * H * U * 2, wbytes = H * U * 2;
    void *outs[2 * kMaxParts];
    int n_out = 0;
    for (int d = 0; d < n_y; ++d) outs[n_out++] = y_outs[d];
    for (int d = 0; d < n_r; ++d) outs[n_out++] = r_outs[d];
    for (int a = 0; a < n_out; ++a) {
        const bool is_residual_dest = a >= n_y;
        if (overlaps(outs[a], bytes, weight, wbytes)) return ASTRA_ERR_OVERLAP;
        if (!(is_residual_dest && outs[a] == residual) && overlaps(outs[a], bytes, residual, bytes))
            return ASTRA_ERR_OVERLAP;
        for (int p = 0; p < n_parts; ++p)
            if (overlaps(outs[a], bytes, x_parts[p], bytes)) return ASTRA_ERR_OVERLAP;
        for (int b = a + 1; b < n_out; ++b)
            if (overlaps(outs[a], bytes, outs[b], bytes)) return ASTRA_ERR_OVERLAP;
    }
    AllreduceOperands op;
    for (int p = 0; p < kMaxParts; ++p) {
        op.part[p] = static_cast<const uint16_t *>(x_parts[p < n_parts ? p : 0]);
        op.y_out[p] = static_cast<uint16_t *>(y_outs[p < n_y ? p : 0]);
        op.r_out[p] = static_cast<uint16_t *>(r_outs[p < n_r ? p : 0]);
    }
    op.n_parts = n_parts;
    op.n_y = n_y;
    op.n_r = n_r;
    op.r = static_cast<const uint16_t *>(residual);
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    const uint16_t *wp = static_cast<const uint16_t *>(weight);
    cudaError_t err = cudaSuccess;
    ASTRA_FOR_DTYPE(dtype, err = dispatch<DT>(op, wp, T, static_cast<int>(H), eps, stream));
    return launch_status(err);
}

}  // namespace

extern "C" {

astra_status_t astra_fused_allreduce_add_rmsnorm(void *y, void *residual, const void *const *x_parts,
                                                 int32_t n_parts, const void *weight, int64_t T, int64_t H,
                                                 float eps, astra_dtype_t dtype, void *cuda_stream) {
    void *ys[1] = {y}, *rs[1] = {residual};  // one destination apiece, the residual in place
    return allreduce_entry(ys, 1, rs, 1, residual, x_parts, n_parts, weight, T, H, eps, dtype, cuda_stream);
}

astra_status_t astra_fused_allreduce_add_rmsnorm_ex(void *const *y_outs, int32_t n_y, void *const *residual_outs,
                                                    int32_t n_r, const void *residual,
                                                    const void *const *x_parts, int32_t n_parts,
                                                    const void *weight, int64_t T, int64_t H, float eps,
                                                    astra_dtype_t dtype, void *cuda_stream) {
    return allreduce_entry(y_outs, n_y, residual_outs, n_r, residual, x_parts, n_parts, weight, T, H, eps, dtype,
                           cuda_stream);
}

}  // extern "C"

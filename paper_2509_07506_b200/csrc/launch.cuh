// Host-side helpers shared by the translation units of the library: pointer and overlap tests, the
// choice of vector width, and the launch wrappers.  Nothing here allocates, synchronises or keeps state.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "astra.h"

namespace astra {
namespace host {

inline bool aligned(const void *p, size_t bytes) {
    return (reinterpret_cast<uintptr_t>(p) % bytes) == 0;
}

// [a, a+na) and [b, b+nb) intersect (byte ranges)
inline bool overlaps(const void *a, int64_t na, const void *b, int64_t nb) {
    const uintptr_t a0 = reinterpret_cast<uintptr_t>(a), b0 = reinterpret_cast<uintptr_t>(b);
    return a0 < b0 + static_cast<uintptr_t>(nb) && b0 < a0 + static_cast<uintptr_t>(na);
}

// Bytes from the first element of a [rows, width] tensor with the given row pitch to one past its last.
inline int64_t span_bytes(int64_t rows, int64_t width, int64_t pitch, int64_t elem) {
    return ((rows - 1) * pitch + width) * elem;
}

// Do two [rows, width] tensors of 16-bit units with the given row pitches share any unit?
// Exact when the pitches are equal (slices of one wider buffer: rows interleave without touching);
// otherwise conservative (overlapping address spans count as overlap).
inline bool pitched_overlap(const void *a, int64_t pitch_a, const void *b, int64_t pitch_b,
                            int64_t rows, int64_t width) {
    if (!overlaps(a, span_bytes(rows, width, pitch_a, 2), b, span_bytes(rows, width, pitch_b, 2))) return false;
    if (pitch_a != pitch_b || rows == 1) return true;
    const int64_t P = pitch_a * 2, w = width * 2;
    const int64_t d = static_cast<int64_t>(reinterpret_cast<intptr_t>(b) - reinterpret_cast<intptr_t>(a));
    int64_t k = d / P, r = d % P;  // b's row j starts r bytes into a's row j + k
    if (r < 0) { r += P; --k; }
    const bool hits_k = r < w && k > -rows && k < rows;
    const bool hits_k1 = P - r < w && (k + 1) > -rows && (k + 1) < rows;
    return hits_k || hits_k1;
}

// Largest vector width (in 16-bit units, a power of two up to max_vec) that divides every extent
// (given in units) and to which every pointer is aligned.  Row starts are multiples of the pitches, so
// every vector access of every row is then naturally aligned.
struct VecPick {
    int vec;
    explicit VecPick(int max_vec) : vec(max_vec) {}
    VecPick &extent(int64_t e) {
        while (vec > 1 && e % vec != 0) vec >>= 1;
        return *this;
    }
    VecPick &pointer(const void *p) {
        while (vec > 1 && !aligned(p, static_cast<size_t>(vec) * 2)) vec >>= 1;
        return *this;
    }
};

// Status of a call from the result of its launch(es).  After a refused launch the runtime's
// per-thread last-error slot holds that refusal; it has been reported through the return code, so it
// is taken out again rather than left to surface in some later, unrelated check of the caller's.
inline astra_status_t launch_status(cudaError_t err) {
    if (err == cudaSuccess) return ASTRA_OK;
    (void)cudaGetLastError();
    return ASTRA_ERR_CUDA;
}

// Every kernel is launched with programmatic stream serialization allowed: its blocks may be
// scheduled while the previous kernel in the stream drains, and they wait (griddepcontrol.wait)
// for that kernel to complete before their first global access.  Stream order is unchanged; the
// launch latency and block prologue of back-to-back calls overlap the previous kernel's tail.
template <typename... KArgs, typename... Args>
inline cudaError_t launch(void (*kernel)(KArgs...), unsigned grid, unsigned block, cudaStream_t stream,
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
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

// Flat vector indices are 31-bit and grids are limited to 2^31-1 blocks; larger inputs are split
// into several launches.  The two limits can be lowered at compile time so that tests can drive the
// splitting with small inputs.
#ifndef ASTRA_MAX_VECS_PER_LAUNCH
#define ASTRA_MAX_VECS_PER_LAUNCH ((1ll << 31) - 1)
#endif
#ifndef ASTRA_MAX_ROWS_PER_LAUNCH
#define ASTRA_MAX_ROWS_PER_LAUNCH 2147483647
#endif
// Preferred upper bound on the block size of the cluster kernel (more, smaller blocks per row are
// chosen while the cluster size allows it).
#ifndef ASTRA_CLUSTER_PREFERRED_THREADS
#define ASTRA_CLUSTER_PREFERRED_THREADS 512
#endif
// The same, for a kernel whose consecutive groups of `cluster` blocks form thread-block clusters
// (distributed shared memory between the blocks of a group).
template <typename... KArgs, typename... Args>
inline cudaError_t launch_clustered(void (*kernel)(KArgs...), unsigned grid, unsigned block, unsigned cluster,
                                    cudaStream_t stream, Args... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid);
    cfg.blockDim = dim3(block);
    cfg.dynamicSmemBytes = 0;
    cfg.stream = stream;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    attr[1].id = cudaLaunchAttributeClusterDimension;
    attr[1].val.clusterDim.x = cluster;
    attr[1].val.clusterDim.y = 1;
    attr[1].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 2;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

constexpr int64_t kMaxVecsPerLaunch = ASTRA_MAX_VECS_PER_LAUNCH;
constexpr int64_t kMaxRowsPerLaunch = ASTRA_MAX_ROWS_PER_LAUNCH;
constexpr int64_t kInt64Max = 9223372036854775807ll;
// Widest row of fused_add_rmsnorm, in 16-bit units (2^30 bf16/fp16 or 2^29 fp32 elements, a 2 GiB
// row): unit offsets inside a row, and the rounded-up vector counts derived from them, then fit a
// 32-bit signed integer.
constexpr int64_t kMaxRowUnits = 1ll << 30;

inline bool valid_dtype(astra_dtype_t d) { return d == ASTRA_BF16 || d == ASTRA_FP16 || d == ASTRA_FP32; }

// All value tensors are addressed in 16-bit units inside the library: an element is 1 unit for the
// 16-bit storage types and 2 for binary32.  Entry points validate in elements, then scale widths and
// pitches to units once; kernels turn a vector of UV units back into UV / UNITS elements.
inline int64_t units_per_elem(astra_dtype_t d) { return d == ASTRA_FP32 ? 2 : 1; }

// Runs CALL with the compile-time constant DT set to the runtime dtype (already validated).
#define ASTRA_FOR_DTYPE(dtype, CALL)                                        \
    do {                                                                    \
        if ((dtype) == ASTRA_BF16) { constexpr int DT = ASTRA_BF16; CALL; } \
        else if ((dtype) == ASTRA_FP16) { constexpr int DT = ASTRA_FP16; CALL; } \
        else { constexpr int DT = ASTRA_FP32; CALL; }                       \
    } while (0)

}  // namespace host
}  // namespace astra

// fused_add_rmsnorm (Astra paper, Table 1, Kernel 2):
//     s = x + r;   r_out <- s;   y <- s / sqrt(mean(s^2) + eps) * w        per row of H elements
// (in place when y is x and r_out is r).
//
// HBM-bound: 8 bytes move per element (x and r read once, y and the new r written once).  One
// thread block owns one row.  In the register-resident kernel each thread keeps its share of the
// binary32 sums s in registers across the row reduction, so the row makes a single trip through
// HBM.  The reduction is the one the paper's optimised kernel uses: shuffles inside each warp, one
// shared-memory slot per warp, then a short combine.  All loads of x and r of a row are issued
// before anything is consumed; the weight (an L2 hit) is fetched while the reduction completes.
#pragma once

#include <cooperative_groups.h>

#include "vec.cuh"

namespace astra {

constexpr int kMaxWarps = 32;

// Row-addressed operands.  Pointers and pitches are in 16-bit units.  y may be exactly x and r_out exactly r (the
// in-place form); each thread reads the vectors it later overwrites, so that aliasing is safe.
struct RmsnormOperands {
    const uint16_t *x;
    const uint16_t *r;
    uint16_t *y;
    uint16_t *r_out;
    int64_t x_pitch, r_pitch, y_pitch, r_out_pitch;
};

// Sum over the block; every thread receives the total.  `slots` holds kMaxWarps floats.
__device__ __forceinline__ float block_sum(float v, float *slots) {
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) v += __shfl_xor_sync(0xffffffffu, v, off);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int nwarps = (blockDim.x + 31) >> 5;
    if (nwarps == 1) return v;
    if (lane == 0) slots[warp] = v;
    __syncthreads();
    float t = lane < nwarps ? slots[lane] : 0.f;
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) t += __shfl_xor_sync(0xffffffffu, t, off);
    return t;
}

// s = x + r (one binary32 add per element) and the running sum of squares, two elements per
// instruction with the packed binary32 forms of sm_100 where the vector has an even length (the
// scalar accumulator serves one-element vectors).  Same roundings as the scalar forms.
template <int VEC>
__device__ __forceinline__ void add_and_square(const float (&x)[VEC], const float (&r)[VEC], float (&s)[VEC],
                                               float &acc, float2 &acc2) {
    if constexpr (VEC % 2 == 0) {
#pragma unroll
        for (int k = 0; k < VEC; k += 2) {
            const float2 t = __fadd2_rn(make_float2(x[k], x[k + 1]), make_float2(r[k], r[k + 1]));
            acc2 = __ffma2_rn(t, t, acc2);
            s[k] = t.x;
            s[k + 1] = t.y;
        }
    } else {
#pragma unroll
        for (int k = 0; k < VEC; ++k) {
            s[k] = x[k] + r[k];
            acc = fmaf(s[k], s[k], acc);
        }
    }
}

// y = (s * rstd) * w, packed likewise.
template <int VEC>
__device__ __forceinline__ void scale(const float (&s)[VEC], float rstd, const float (&w)[VEC], float (&y)[VEC]) {
    if constexpr (VEC % 2 == 0) {
        const float2 r2 = make_float2(rstd, rstd);
#pragma unroll
        for (int k = 0; k < VEC; k += 2) {
            const float2 t = __fmul2_rn(__fmul2_rn(make_float2(s[k], s[k + 1]), r2), make_float2(w[k], w[k + 1]));
            y[k] = t.x;
            y[k + 1] = t.y;
        }
    } else {
#pragma unroll
        for (int k = 0; k < VEC; ++k) y[k] = s[k] * rstd * w[k];
    }
}

// Largest block the register-resident kernel may be launched with, by vectors per thread: the
// row's binary32 sums plus its packed inputs (counted in 16-bit units per thread) must fit the
// register file.
__host__ __device__ constexpr int rmsnorm_reg_max_threads(int units_per_thread) {
    return units_per_thread <= 16 ? 1024 : (units_per_thread <= 32 ? 512 : 256);
}

// Register-resident row: thread i owns vectors i, i + blockDim.x, ... (at most VPT of them).
// Requires nvec = H / VEC <= VPT * blockDim.x and blockDim.x <= rmsnorm_reg_max_threads(VEC * VPT * UNITS).
// EARLY_W issues the weight loads before the reduction instead of after it (measured: no faster,
// and it costs the registers that decide occupancy).  MINB is the minimum number of resident blocks
// the register allocation must allow; with 16 units per thread in at most four vectors MINB = 2
// caps the kernel at 32 registers, i.e. full occupancy for every block size, which is worth 5 % at
// [16384, 8192] and 27 % at [512, 14336] (896-thread blocks: two per SM instead of one).  The
// four-vector form (8-byte accesses, e.g. H = 4100) fits the cap too; with eight or sixteen narrower
// vectors it would spill, so no cap there.
template <int DT, int VEC, int VPT, Ld LDH = Ld::Stream, St STH = St::Stream, bool EARLY_W = false,
          int MINB = ((VEC * VPT * Storage<DT>::UNITS <= 16 && VPT <= 4 && VEC * Storage<DT>::UNITS >= 4) ? 2 : 1)>
__global__ void __launch_bounds__(rmsnorm_reg_max_threads(VEC * VPT * Storage<DT>::UNITS), MINB)
fused_add_rmsnorm_reg_kernel(RmsnormOperands op, const uint16_t *__restrict__ weight,
                             int H, float eps, float inv_H) {
    constexpr int UV = VEC * Storage<DT>::UNITS;  // 16-bit units per vector
    __shared__ float slots[kMaxWarps];
    const int nvec = H / VEC;
    const int64_t row = blockIdx.x;
    const uint16_t *xr = op.x + row * op.x_pitch;
    const uint16_t *rr = op.r + row * op.r_pitch;
    uint16_t *yr = op.y + row * op.y_pitch;
    uint16_t *ror = op.r_out + row * op.r_out_pitch;
    // the row's two inputs start moving towards L2 while the previous kernel is still draining
    if (threadIdx.x == 0) {
        prefetch_l2_range(xr, static_cast<int64_t>(H) * (2 * Storage<DT>::UNITS));
        prefetch_l2_range(rr, static_cast<int64_t>(H) * (2 * Storage<DT>::UNITS));
    }
    grid_dependency_wait();
    grid_launch_dependents();

    Pack<UV> px[VPT], pr[VPT], pw[VPT];
#pragma unroll
    for (int i = 0; i < VPT; ++i) {
        const int v = threadIdx.x + i * blockDim.x;
        if (v < nvec) {
            // x and residual may be rewritten by this same thread below: coherent loads, not .nc
            px[i] = load<UV, LDH>(xr + v * UV);
            pr[i] = load<UV, LDH>(rr + v * UV);
        }
    }
    if constexpr (EARLY_W) {
#pragma unroll
        for (int i = 0; i < VPT; ++i) {
            const int v = threadIdx.x + i * blockDim.x;
            if (v < nvec) pw[i] = load<UV, Ld::Keep>(weight + v * UV);
        }
    }

    float s[VPT][VEC];
    float acc = 0.f;
    float2 acc2 = make_float2(0.f, 0.f);
#pragma unroll
    for (int i = 0; i < VPT; ++i) {
        const int v = threadIdx.x + i * blockDim.x;
        if (v < nvec) {
            float fx[VEC], fr[VEC];
            widen<DT, VEC>(px[i], fx);
            widen<DT, VEC>(pr[i], fr);
            add_and_square(fx, fr, s[i], acc, acc2);  // the one binary32 add per element
            store<UV, STH>(ror + v * UV, narrow<DT, VEC>(s[i]));
        }
    }

    if constexpr (!EARLY_W) {
#pragma unroll
        for (int i = 0; i < VPT; ++i) {
            const int v = threadIdx.x + i * blockDim.x;
            if (v < nvec) pw[i] = load<UV, Ld::Keep>(weight + v * UV);
        }
    }
    const float total = block_sum(acc + (acc2.x + acc2.y), slots);
    const float rstd = rsqrtf(fmaf(total, inv_H, eps));

#pragma unroll
    for (int i = 0; i < VPT; ++i) {
        const int v = threadIdx.x + i * blockDim.x;
        if (v < nvec) {
            float fw[VEC], fy[VEC];
            widen<DT, VEC>(pw[i], fw);
            scale(s[i], rstd, fw, fy);
            store<UV, STH>(yr + v * UV, narrow<DT, VEC>(fy));
        }
    }
}

// Rows too wide for one block's registers: a thread-block cluster owns the row.  Each block keeps
// its contiguous share of the row in registers exactly as above and reduces it; the per-block
// partial sums are then exchanged through distributed shared memory (every block reads every
// partial, in rank order, so all blocks form the same total bit for bit), and each block finishes
// its share.  The row still makes one trip through HBM.  The two cluster barriers are hardware
// barriers that every thread of every block reaches unconditionally (blocks without work included):
// the first publishes the partials; the second, split into an arrive right after the partials are
// read and a wait at the very end, keeps each block's shared memory alive until all its peers have
// read it without stalling the final stores.
// (scalar arithmetic here: the packed forms cost the registers that keep this kernel at full
// occupancy, which matters more: 5.4 against 4.5 TB/s at [2048, 14336] fp32)
template <int DT, int VEC, int VPT, int MINB = ((VEC * VPT * Storage<DT>::UNITS <= 16 && VPT <= 2) ? 2 : 1)>
__global__ void __launch_bounds__(rmsnorm_reg_max_threads(VEC * VPT * Storage<DT>::UNITS), MINB)
fused_add_rmsnorm_cluster_kernel(RmsnormOperands op, const uint16_t *__restrict__ weight,
                                 int H, float eps, float inv_H) {
    namespace cg = cooperative_groups;
    constexpr int UV = VEC * Storage<DT>::UNITS;
    __shared__ float slots[kMaxWarps];
    __shared__ float block_partial;
    cg::cluster_group cluster = cg::this_cluster();
    const unsigned nblocks = cluster.num_blocks();
    const unsigned rank = cluster.block_rank();
    const int nvec = H / VEC;
    const int chunk = (nvec + nblocks - 1) / nblocks;  // vectors per block (the last may hold fewer)
    const int first = rank * chunk;
    const int count = max(0, min(chunk, nvec - first));
    const int64_t row = blockIdx.x / nblocks;
    const uint16_t *xr = op.x + row * op.x_pitch + static_cast<int64_t>(first) * UV;
    const uint16_t *rr = op.r + row * op.r_pitch + static_cast<int64_t>(first) * UV;
    uint16_t *yr = op.y + row * op.y_pitch + static_cast<int64_t>(first) * UV;
    uint16_t *ror = op.r_out + row * op.r_out_pitch + static_cast<int64_t>(first) * UV;
    const uint16_t *wr = weight + static_cast<int64_t>(first) * UV;
    if (threadIdx.x == 0) {
        prefetch_l2_range(xr, static_cast<int64_t>(count) * UV * 2);
        prefetch_l2_range(rr, static_cast<int64_t>(count) * UV * 2);
    }
    grid_dependency_wait();
    grid_launch_dependents();

    Pack<UV> px[VPT], pr[VPT], pw[VPT];
#pragma unroll
    for (int i = 0; i < VPT; ++i) {
        const int v = threadIdx.x + i * blockDim.x;
        if (v < count) {
            px[i] = load<UV, Ld::Stream>(xr + v * UV);
            pr[i] = load<UV, Ld::Stream>(rr + v * UV);
        }
    }
    float s[VPT][VEC];
    float acc = 0.f;
#pragma unroll
    for (int i = 0; i < VPT; ++i) {
        const int v = threadIdx.x + i * blockDim.x;
        if (v < count) {
            float fx[VEC], fr[VEC];
            widen<DT, VEC>(px[i], fx);
            widen<DT, VEC>(pr[i], fr);
#pragma unroll
            for (int k = 0; k < VEC; ++k) {
                s[i][k] = fx[k] + fr[k];
                acc = fmaf(s[i][k], s[i][k], acc);
            }
            store<UV, St::Stream>(ror + v * UV, narrow<DT, VEC>(s[i]));
        }
    }
#pragma unroll
    for (int i = 0; i < VPT; ++i) {
        const int v = threadIdx.x + i * blockDim.x;
        if (v < count) pw[i] = load<UV, Ld::Keep>(wr + v * UV);
    }
    const float mine = block_sum(acc, slots);
    if (threadIdx.x == 0) block_partial = mine;
    cluster.sync();
    float total = 0.f;
    for (unsigned b = 0; b < nblocks; ++b) total += *cluster.map_shared_rank(&block_partial, b);
    cluster.barrier_arrive();  // "I have read my peers' partials"; waited for just before exit
    const float rstd = rsqrtf(fmaf(total, inv_H, eps));
#pragma unroll
    for (int i = 0; i < VPT; ++i) {
        const int v = threadIdx.x + i * blockDim.x;
        if (v < count) {
            float fw[VEC], fy[VEC];
            widen<DT, VEC>(pw[i], fw);
#pragma unroll
            for (int k = 0; k < VEC; ++k) fy[k] = s[i][k] * rstd * fw[k];
            store<UV, St::Stream>(yr + v * UV, narrow<DT, VEC>(fy));
        }
    }
    cluster.barrier_wait();  // no block leaves while a peer may still read its shared memory
}

// Any H: two sweeps over the row.  The first only reads (x, r) and accumulates the sum of squares;
// the second re-reads them (the row was just touched, so it comes from L2), recomputes the same
// binary32 sums, and writes both outputs.  Nothing is written before the norm is known, so the
// in-place update cannot disturb the reduction.
template <int DT, int VEC>
__global__ void fused_add_rmsnorm_twopass_kernel(RmsnormOperands op,
                                                 const uint16_t *__restrict__ weight,
                                                 int H, float eps, float inv_H) {
    constexpr int UV = VEC * Storage<DT>::UNITS;  // 16-bit units per vector
    __shared__ float slots[kMaxWarps];
    const int nvec = H / VEC;
    const int64_t row = blockIdx.x;
    const uint16_t *xr = op.x + row * op.x_pitch;
    const uint16_t *rr = op.r + row * op.r_pitch;
    uint16_t *yr = op.y + row * op.y_pitch;
    uint16_t *ror = op.r_out + row * op.r_out_pitch;
    grid_dependency_wait();
    grid_launch_dependents();

    float acc = 0.f;
    for (int v = threadIdx.x; v < nvec; v += blockDim.x) {
        float fx[VEC], fr[VEC];
        widen<DT, VEC>(load<UV, Ld::Stream>(xr + v * UV), fx);
        widen<DT, VEC>(load<UV, Ld::Stream>(rr + v * UV), fr);
#pragma unroll
        for (int k = 0; k < VEC; ++k) {
            const float s = fx[k] + fr[k];
            acc = fmaf(s, s, acc);
        }
    }
    const float total = block_sum(acc, slots);
    const float rstd = rsqrtf(fmaf(total, inv_H, eps));

    for (int v = threadIdx.x; v < nvec; v += blockDim.x) {
        float fx[VEC], fr[VEC], fw[VEC], fs[VEC], fy[VEC];
        widen<DT, VEC>(load<UV, Ld::Stream>(xr + v * UV), fx);
        widen<DT, VEC>(load<UV, Ld::Stream>(rr + v * UV), fr);
        widen<DT, VEC>(load<UV, Ld::Keep>(weight + v * UV), fw);
#pragma unroll
        for (int k = 0; k < VEC; ++k) {
            fs[k] = fx[k] + fr[k];
            fy[k] = fs[k] * rstd * fw[k];
        }
        store<UV, St::Stream>(ror + v * UV, narrow<DT, VEC>(fs));
        store<UV, St::Stream>(yr + v * UV, narrow<DT, VEC>(fy));
    }
}

}  // namespace astra

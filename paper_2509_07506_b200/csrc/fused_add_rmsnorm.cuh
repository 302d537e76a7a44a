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

#include "vec.cuh"

namespace astra {

constexpr int kMaxWarps = 32;

// Row-addressed operands.  Pitches are in elements.  y may be exactly x and r_out exactly r (the
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

// Largest block the register-resident kernel may be launched with, by vectors per thread: the
// row's binary32 sums (VPT * VEC registers) plus its packed inputs must fit the register file.
__host__ __device__ constexpr int rmsnorm_reg_max_threads(int vec, int vpt) {
    return vec * vpt <= 16 ? 1024 : (vec * vpt <= 32 ? 512 : 256);
}

// Register-resident row: thread i owns vectors i, i + blockDim.x, ... (at most VPT of them).
// Requires nvec = H / VEC <= VPT * blockDim.x and blockDim.x <= rmsnorm_reg_max_threads(VEC, VPT).
// EARLY_W issues the weight loads before the reduction instead of after it (measured: no faster,
// and it costs the registers that decide occupancy).  MINB is the minimum number of resident blocks
// the register allocation must allow; with 16 elements per thread MINB = 2 caps the kernel at 32
// registers, i.e. full occupancy for every block size, which is worth 5 % at [16384, 8192] and
// 27 % at [512, 14336] (896-thread blocks: two per SM instead of one).
template <int DT, int VEC, int VPT, Ld LDH = Ld::Stream, St STH = St::Stream, bool EARLY_W = false,
          int MINB = (VEC * VPT <= 16 ? 2 : 1)>
__global__ void __launch_bounds__(rmsnorm_reg_max_threads(VEC, VPT), MINB)
fused_add_rmsnorm_reg_kernel(RmsnormOperands op, const uint16_t *__restrict__ weight,
                             int H, float eps, float inv_H) {
    __shared__ float slots[kMaxWarps];
    const int nvec = H / VEC;
    const int64_t row = blockIdx.x;
    const uint16_t *xr = op.x + row * op.x_pitch;
    const uint16_t *rr = op.r + row * op.r_pitch;
    uint16_t *yr = op.y + row * op.y_pitch;
    uint16_t *ror = op.r_out + row * op.r_out_pitch;
    grid_dependency_wait();
    grid_launch_dependents();

    Pack<VEC> px[VPT], pr[VPT], pw[VPT];
#pragma unroll
    for (int i = 0; i < VPT; ++i) {
        const int v = threadIdx.x + i * blockDim.x;
        if (v < nvec) {
            // x and residual may be rewritten by this same thread below: coherent loads, not .nc
            px[i] = load<VEC, LDH>(xr + v * VEC);
            pr[i] = load<VEC, LDH>(rr + v * VEC);
        }
    }
    if constexpr (EARLY_W) {
#pragma unroll
        for (int i = 0; i < VPT; ++i) {
            const int v = threadIdx.x + i * blockDim.x;
            if (v < nvec) pw[i] = load<VEC, Ld::Keep>(weight + v * VEC);
        }
    }

    float s[VPT][VEC];
    float acc = 0.f;
#pragma unroll
    for (int i = 0; i < VPT; ++i) {
        const int v = threadIdx.x + i * blockDim.x;
        if (v < nvec) {
            float fx[VEC], fr[VEC];
            widen<DT, VEC>(px[i], fx);
            widen<DT, VEC>(pr[i], fr);
#pragma unroll
            for (int k = 0; k < VEC; ++k) {
                s[i][k] = fx[k] + fr[k];  // the one binary32 add
                acc = fmaf(s[i][k], s[i][k], acc);
            }
            store<VEC, STH>(ror + v * VEC, narrow<DT, VEC>(s[i]));
        }
    }

    if constexpr (!EARLY_W) {
#pragma unroll
        for (int i = 0; i < VPT; ++i) {
            const int v = threadIdx.x + i * blockDim.x;
            if (v < nvec) pw[i] = load<VEC, Ld::Keep>(weight + v * VEC);
        }
    }
    const float total = block_sum(acc, slots);
    const float rstd = rsqrtf(fmaf(total, inv_H, eps));

#pragma unroll
    for (int i = 0; i < VPT; ++i) {
        const int v = threadIdx.x + i * blockDim.x;
        if (v < nvec) {
            float fw[VEC], fy[VEC];
            widen<DT, VEC>(pw[i], fw);
#pragma unroll
            for (int k = 0; k < VEC; ++k) fy[k] = s[i][k] * rstd * fw[k];
            store<VEC, STH>(yr + v * VEC, narrow<DT, VEC>(fy));
        }
    }
}

// Any H: two sweeps over the row.  The first only reads (x, r) and accumulates the sum of squares;
// the second re-reads them (the row was just touched, so it comes from L2), recomputes the same
// binary32 sums, and writes both outputs.  Nothing is written before the norm is known, so the
// in-place update cannot disturb the reduction.
template <int DT, int VEC>
__global__ void fused_add_rmsnorm_twopass_kernel(RmsnormOperands op,
                                                 const uint16_t *__restrict__ weight,
                                                 int H, float eps, float inv_H) {
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
        widen<DT, VEC>(load<VEC, Ld::Stream>(xr + v * VEC), fx);
        widen<DT, VEC>(load<VEC, Ld::Stream>(rr + v * VEC), fr);
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
        widen<DT, VEC>(load<VEC, Ld::Stream>(xr + v * VEC), fx);
        widen<DT, VEC>(load<VEC, Ld::Stream>(rr + v * VEC), fr);
        widen<DT, VEC>(load<VEC, Ld::Keep>(weight + v * VEC), fw);
#pragma unroll
        for (int k = 0; k < VEC; ++k) {
            fs[k] = fx[k] + fr[k];
            fy[k] = fs[k] * rstd * fw[k];
        }
        store<VEC, St::Stream>(ror + v * VEC, narrow<DT, VEC>(fs));
        store<VEC, St::Stream>(yr + v * VEC, narrow<DT, VEC>(fy));
    }
}

}  // namespace astra

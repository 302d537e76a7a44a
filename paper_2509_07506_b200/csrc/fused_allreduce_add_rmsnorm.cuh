// fused_allreduce_add_rmsnorm: fused_add_rmsnorm (Astra paper, Table 1, Kernel 2) on a hidden state
// that arrives as N partial sums, one per tensor-parallel rank:
//     x = x_0 + x_1 + ... + x_{N-1};   s = x + r;   r_out <- s;   y <- s / sqrt(mean(s^2) + eps) * w
// Every addition is one binary32 addition, in rank order, the residual last, so that all ranks of a
// group that run this on the same partials produce identical bits.
//
// One-shot form: each rank reads all N partials of the rows it normalises (its own from local
// memory, the others through peer-mapped addresses) and writes only its own memory.  Two-shot form
// (for batches large enough that the N-fold read would be bound by the links): each rank does this
// for its own block of rows only and stores the results to every rank's buffers, so each element
// crosses the links once as a partial and once as a result instead of N - 1 times.
// All loads and stores are plain per-thread `ld.global` / `st.global` (no multicast, no bulk or
// tensor-map copies), so a partial or a destination may live in another GPU's memory.  The kernel
// waits for nothing: the caller orders it after every rank has finished writing its partial and
// orders the consumers after it (stream events, a host barrier).
//
// HBM/NVLink-bound: (N + 1 + Dy + Dr) * 2 bytes per element of 16-bit storage (N partials and r read,
// y written to Dy destinations and the new residual to Dr; N + 3 in the one-shot form).  One block owns a row and keeps the running binary32 sums in registers; the
// partials are fetched GROUP at a time so that GROUP (+1 for the residual) vector loads per vector
// position are in flight before the first addition (GROUP = 2 measured best; see the launch code).
#pragma once

#include "fused_add_rmsnorm.cuh"

namespace astra {

constexpr int kMaxParts = 16;

// Dense [T, H] operands (row pitch = H).  Pointers are in 16-bit units.  Each result goes to one or
// more destinations (the same bytes to each): with one destination apiece this is the one-shot
// all-reduce; with one destination per rank it is the two-shot form, in which a rank reduces and
// normalises only its own row block and pushes the results into every rank's buffers.  A residual
// destination may be exactly r (each thread reads the residual vectors it later overwrites); the
// destinations overlap nothing else.
struct AllreduceOperands {
    const uint16_t *part[kMaxParts];  // rank order
    const uint16_t *r;
    uint16_t *y_out[kMaxParts];
    uint16_t *r_out[kMaxParts];
    int n_parts, n_y, n_r;
};

// The same vector to each of the first n destinations, with plain per-thread stores (a destination
// may be another GPU's memory).  Unrolled and left by a break, so every copy has a constant index.
template <int UV>
__device__ __forceinline__ void store_to_all(uint16_t *const (&dst)[kMaxParts], int n, int64_t at, const Pack<UV> &v) {
#pragma unroll
    for (int d = 0; d < kMaxParts; ++d) {
        if (d >= n) break;
        store<UV, St::Stream>(dst[d] + at, v);
    }
}

// s += x, two elements per instruction where the vector length is even (same roundings as scalar adds).
template <int VEC>
__device__ __forceinline__ void accumulate(float (&s)[VEC], const float (&x)[VEC]) {
    if constexpr (VEC % 2 == 0) {
#pragma unroll
        for (int k = 0; k < VEC; k += 2) {
            const float2 t = __fadd2_rn(make_float2(s[k], s[k + 1]), make_float2(x[k], x[k + 1]));
            s[k] = t.x;
            s[k + 1] = t.y;
        }
    } else {
#pragma unroll
        for (int k = 0; k < VEC; ++k) s[k] += x[k];
    }
}

// Largest block of the register-resident kernel: a thread holds its share of the row as binary32 sums
// (one register per element) plus GROUP + 1 packed input copies of it, and the register file is
// 64 K registers per block.  `units` = 16-bit units of the row per thread.
// With two loads in flight 16 units per thread need 54 to 56 registers, so even a 1024-thread block
// fits; that matters for rows of more than 8192 units, where one fat block per SM with one vector per
// thread beat two vectors per thread in half as many threads by 3 to 9 % (e.g. 157.9 -> 143.1 us at
// [4096, 16384] with 4 partials, 82.2 -> 77.4 us at [4096, 11008] with 2).
__host__ __device__ constexpr int allreduce_reg_max_threads(int units, int group) {
    return group > 4 ? (units <= 16 ? 512 : 128)
         : group > 2 ? (units <= 8 ? 1024 : (units <= 16 ? 512 : 256))
                     : (units <= 16 ? 1024 : 512);
}

// Register-resident row: thread i owns vectors i, i + blockDim.x, ... (at most VPT of them).
// Requires nvec = H / VEC <= VPT * blockDim.x and blockDim.x <= allreduce_reg_max_threads(...), or
// blockDim.x <= kAllreduceDenseThreads for the DENSE instantiation: blocks of at most 256 threads
// whose register allocation is held to 48 so that five of them are resident per SM instead of four
// (for two loads in flight and 16 units per thread that costs no spill).  Measured at [8192, 4096],
// L2-cold: 50.8 -> 50.5 us with 2 partials, 71.5 -> 70.4 us with 4, 112.2 -> 110.3 us with 8; at
// [1024, 4096] it is neutral or slower (16.1 -> 16.5 us with 8 partials), so the launch code uses it
// for long streams only.
constexpr int kAllreduceDenseThreads = 256;
constexpr int kAllreduceDenseBlocks = 5;

template <int DT, int VEC, int VPT, int GROUP, bool DENSE = false>
__global__ void __launch_bounds__(DENSE ? kAllreduceDenseThreads : allreduce_reg_max_threads(VEC * VPT * Storage<DT>::UNITS, GROUP),
                                  DENSE ? kAllreduceDenseBlocks : 1)
fused_allreduce_add_rmsnorm_reg_kernel(const __grid_constant__ AllreduceOperands op,
                                       const uint16_t *__restrict__ weight, int H, float eps, float inv_H) {
    constexpr int UV = VEC * Storage<DT>::UNITS;  // 16-bit units per vector
    __shared__ float slots[kMaxWarps];
    const int nvec = H / VEC;
    const int64_t row = static_cast<int64_t>(blockIdx.x) * H * Storage<DT>::UNITS;  // first unit of the row
    const int n = op.n_parts;
    // The residual row is this GPU's own memory: ask for it ahead of the dependency wait.  The partials
    // may be another GPU's memory and are left to the ordinary loads below.
    if (threadIdx.x == 0) prefetch_l2_range(op.r + row, static_cast<int64_t>(H) * (2 * Storage<DT>::UNITS));
    grid_dependency_wait();
    grid_launch_dependents();

    // the residual is consumed last but requested first, together with the first group of partials
    Pack<UV> pr[VPT];
#pragma unroll
    for (int i = 0; i < VPT; ++i) {
        const int v = threadIdx.x + i * blockDim.x;
        if (v < nvec) pr[i] = load<UV, Ld::Stream>(op.r + row + v * UV);
    }

    // The loop over groups is unrolled to the largest supported count and left by a break: every copy
    // then has a constant p0 (the first one initialises the sums without a test) and the compiler may
    // move a group's loads above the additions of the group before it.  Measured against the rolled
    // loop at [8192, 4096], L2-cold: 54.1 -> 50.8 us with 2 partials, 74.5 -> 71.8 us with 4,
    // 113.8 -> 111.8 us with 8.
    float s[VPT][VEC];
#pragma unroll
    for (int p0 = 0; p0 < kMaxParts; p0 += GROUP) {
        if (p0 >= n) break;
        Pack<UV> px[GROUP][VPT];
#pragma unroll
        for (int g = 0; g < GROUP; ++g) {
            if (p0 + g < n) {
                const uint16_t *base = op.part[p0 + g] + row;
#pragma unroll
                for (int i = 0; i < VPT; ++i) {
                    const int v = threadIdx.x + i * blockDim.x;
                    if (v < nvec) px[g][i] = load<UV, Ld::Stream>(base + v * UV);
                }
            }
        }
#pragma unroll
        for (int g = 0; g < GROUP; ++g) {
            if (p0 + g < n) {
#pragma unroll
                for (int i = 0; i < VPT; ++i) {
                    const int v = threadIdx.x + i * blockDim.x;
                    if (v < nvec) {
                        float fx[VEC];
                        widen<DT, VEC>(px[g][i], fx);
                        if (p0 + g == 0) {
#pragma unroll
                            for (int k = 0; k < VEC; ++k) s[i][k] = fx[k];
                        } else {
                            accumulate(s[i], fx);  // rank order: partial p0 + g joins the sum of those before it
                        }
                    }
                }
            }
        }
    }

    float acc = 0.f;
    float2 acc2 = make_float2(0.f, 0.f);
#pragma unroll
    for (int i = 0; i < VPT; ++i) {
        const int v = threadIdx.x + i * blockDim.x;
        if (v < nvec) {
            float fr[VEC];
            widen<DT, VEC>(pr[i], fr);
            add_and_square(s[i], fr, s[i], acc, acc2);  // the residual joins last
            store_to_all<UV>(op.r_out, op.n_r, row + v * UV, narrow<DT, VEC>(s[i]));
        }
    }

    Pack<UV> pw[VPT];
#pragma unroll
    for (int i = 0; i < VPT; ++i) {
        const int v = threadIdx.x + i * blockDim.x;
        if (v < nvec) pw[i] = load<UV, Ld::Keep>(weight + v * UV);
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
            store_to_all<UV>(op.y_out, op.n_y, row + v * UV, narrow<DT, VEC>(fy));
        }
    }
}

// The rank-order sum of one vector position, GROUP partial loads in flight at a time.
template <int DT, int VEC, int GROUP>
__device__ __forceinline__ void rank_order_sum(const AllreduceOperands &op, int64_t at, float (&s)[VEC]) {
    constexpr int UV = VEC * Storage<DT>::UNITS;
    const int n = op.n_parts;
    const Pack<UV> pr = load<UV, Ld::Stream>(op.r + at);
#pragma unroll
    for (int p0 = 0; p0 < kMaxParts; p0 += GROUP) {  // unrolled and left by a break, as in the kernel above
        if (p0 >= n) break;
        Pack<UV> px[GROUP];
#pragma unroll
        for (int g = 0; g < GROUP; ++g)
            if (p0 + g < n) px[g] = load<UV, Ld::Stream>(op.part[p0 + g] + at);
#pragma unroll
        for (int g = 0; g < GROUP; ++g) {
            if (p0 + g < n) {
                float fx[VEC];
                widen<DT, VEC>(px[g], fx);
                if (p0 + g == 0) {
#pragma unroll
                    for (int k = 0; k < VEC; ++k) s[k] = fx[k];
                } else {
                    accumulate(s, fx);
                }
            }
        }
    }
    float fr[VEC];
    widen<DT, VEC>(pr, fr);
    accumulate(s, fr);
}

// Any width and any vector size: two sweeps over the row.  The first forms the sums and their
// squares and writes nothing; the second forms the same sums again (the partials now come from L2
// where they fit) and writes both outputs, so the in-place residual cannot disturb the reduction.
template <int DT, int VEC, int GROUP>
__global__ void __launch_bounds__(1024)
fused_allreduce_add_rmsnorm_twopass_kernel(const __grid_constant__ AllreduceOperands op,
                                           const uint16_t *__restrict__ weight, int H, float eps, float inv_H) {
    constexpr int UV = VEC * Storage<DT>::UNITS;
    __shared__ float slots[kMaxWarps];
    const int nvec = H / VEC;
    const int64_t row = static_cast<int64_t>(blockIdx.x) * H * Storage<DT>::UNITS;
    grid_dependency_wait();
    grid_launch_dependents();

    float acc = 0.f;
    for (int v = threadIdx.x; v < nvec; v += blockDim.x) {
        float s[VEC];
        rank_order_sum<DT, VEC, GROUP>(op, row + static_cast<int64_t>(v) * UV, s);
#pragma unroll
        for (int k = 0; k < VEC; ++k) acc = fmaf(s[k], s[k], acc);
    }
    const float total = block_sum(acc, slots);
    const float rstd = rsqrtf(fmaf(total, inv_H, eps));

    for (int v = threadIdx.x; v < nvec; v += blockDim.x) {
        const int64_t at = row + static_cast<int64_t>(v) * UV;
        float s[VEC], fw[VEC], fy[VEC];
        rank_order_sum<DT, VEC, GROUP>(op, at, s);
        widen<DT, VEC>(load<UV, Ld::Keep>(weight + static_cast<int64_t>(v) * UV), fw);
#pragma unroll
        for (int k = 0; k < VEC; ++k) fy[k] = s[k] * rstd * fw[k];
        store_to_all<UV>(op.r_out, op.n_r, at, narrow<DT, VEC>(s));
        store_to_all<UV>(op.y_out, op.n_y, at, narrow<DT, VEC>(fy));
    }
}

}  // namespace astra

// silu_and_mul (Astra paper, Table 1, Kernel 3):  out = a * sigmoid(a) * b,  row = [a | b].
//
// Elementwise and HBM-bound: 6 bytes move per output (4 read, 2 written).  Each thread owns UNROLL
// vectors of VEC elements; all its 2*UNROLL loads are issued before the first use so that enough
// bytes are in flight per SM to cover HBM latency.  The sigmoid costs two special-function ops per
// element (ex2 and rcp, the fast-math forms the paper's optimised kernel also turns to), in
// binary32, with one rounding at the store.  Instruction count matters even though the kernel is
// HBM-bound: under a sustained power cap the SM clock (and with it the on-chip fabric) drops as
// issue activity rises, so the arithmetic is kept to the packed two-wide forms.
#pragma once

#include "vec.cuh"

namespace astra {

// SiLU(a) * b in binary32, in the overflow-free form: with t = e^{-|a|} in [0, 1],
// sigmoid(a) = 1/(1+t) for a >= 0 and t/(1+t) for a < 0, so the reciprocal's argument stays in
// [1, 2].  t is formed as h*h with h = e^{-|a|/2} = 2^{-|a| * log2(e)/2}: h stays a normal number
// down to |a| = 174, and the (non-flushing) product h*h reaches the subnormals, so a * e^{a} * b is
// still produced where e^{a} alone is below 2^-126; beyond |a| = 174 the true result is below every
// representable magnitude anyway.
constexpr float kHalfLog2e = 0.7213475204444817f;

__device__ __forceinline__ float silu_mul(float a, float b) {
    float h, d;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(h) : "f"(fabsf(a) * -kHalfLog2e));
    const float t = h * h;
    asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(d) : "f"(1.0f + t));
    return a * (d * (a >= 0.f ? 1.0f : t)) * b;
}

// Two elements at a time with the packed binary32 instructions of sm_100 (two multiplies or adds
// per issue slot); the two special-function ops per element stay scalar.  Same arithmetic, element
// by element, as silu_mul.
__device__ __forceinline__ float2 silu_mul2(float2 a, float2 b) {
    const float2 arg = __fmul2_rn(make_float2(fabsf(a.x), fabsf(a.y)), make_float2(-kHalfLog2e, -kHalfLog2e));
    float2 h, d;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(h.x) : "f"(arg.x));
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(h.y) : "f"(arg.y));
    const float2 t = __fmul2_rn(h, h);
    const float2 den = __fadd2_rn(t, make_float2(1.0f, 1.0f));
    asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(d.x) : "f"(den.x));
    asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(d.y) : "f"(den.y));
    const float2 f = make_float2(a.x >= 0.f ? 1.0f : t.x, a.y >= 0.f ? 1.0f : t.y);
    return __fmul2_rn(__fmul2_rn(a, __fmul2_rn(d, f)), b);
}

// Flat indexing: vector v of the output covers out[row, col*VEC .. col*VEC+VEC) with
// row = v / nvec, col = v % nvec, nvec = D / VEC.  A block handles THREADS*UNROLL consecutive vectors.
// gate and up are addressed separately (pointers and row pitches in 16-bit units), which covers both the packed
// row [a | b] (up = gate + D, equal pitches) and two independent tensors.
template <int DT, int VEC, int UNROLL, int THREADS, Ld LDH = Ld::StreamReadOnly, St STH = St::Stream,
          int PF_VECS = 0>
__global__ void __launch_bounds__(THREADS)
silu_and_mul_kernel(uint16_t *__restrict__ out, const uint16_t *__restrict__ gate,
                    const uint16_t *__restrict__ up, uint32_t total_vecs, FastDiv nvec,
                    int64_t out_pitch, int64_t gate_pitch, int64_t up_pitch) {
    constexpr int UV = VEC * Storage<DT>::UNITS;  // 16-bit units per vector
    const uint32_t base = blockIdx.x * (THREADS * UNROLL) + threadIdx.x;
    // Ahead of the dependency wait, the block asks for the gate and up bytes of its vectors to be
    // brought into L2: PF_VECS vectors per request (0 = no prefetch), each request cut at a row end.
    if constexpr (PF_VECS > 0) {
        const uint32_t first = blockIdx.x * (THREADS * UNROLL);
        const uint32_t piece = threadIdx.x * PF_VECS;  // thread t asks for vectors [first + piece, + PF_VECS)
        if (piece < THREADS * UNROLL && first + piece < total_vecs) {
            const uint32_t v0 = first + piece;
            const uint32_t row = nvec.div(v0);
            const uint32_t col = v0 - row * nvec.d;
            uint32_t n = min(static_cast<uint32_t>(PF_VECS), total_vecs - v0);
            n = min(n, nvec.d - col);
            const int64_t c = static_cast<int64_t>(col) * UV;
            prefetch_l2_range(gate + (static_cast<int64_t>(row) * gate_pitch + c), static_cast<int64_t>(n) * UV * 2);
            prefetch_l2_range(up + (static_cast<int64_t>(row) * up_pitch + c), static_cast<int64_t>(n) * UV * 2);
        }
    }
    grid_dependency_wait();
    grid_launch_dependents();
    Pack<UV> a[UNROLL], b[UNROLL];
#pragma unroll
    for (int j = 0; j < UNROLL; ++j) {
        const uint32_t v = base + j * THREADS;
        if (v < total_vecs) {
            const uint32_t row = nvec.div(v);
            const uint32_t col = v - row * nvec.d;
            const int64_t c = static_cast<int64_t>(col) * UV;
            a[j] = load<UV, LDH>(gate + (static_cast<int64_t>(row) * gate_pitch + c));
            b[j] = load<UV, LDH>(up + (static_cast<int64_t>(row) * up_pitch + c));
        }
    }
#pragma unroll
    for (int j = 0; j < UNROLL; ++j) {
        const uint32_t v = base + j * THREADS;
        if (v < total_vecs) {
            float fa[VEC], fb[VEC], fo[VEC];
            widen<DT, VEC>(a[j], fa);
            widen<DT, VEC>(b[j], fb);
            if constexpr (VEC == 1) {
                fo[0] = silu_mul(fa[0], fb[0]);
            } else {
#pragma unroll
                for (int i = 0; i < VEC; i += 2) {
                    const float2 o = silu_mul2(make_float2(fa[i], fa[i + 1]), make_float2(fb[i], fb[i + 1]));
                    fo[i] = o.x;
                    fo[i + 1] = o.y;
                }
            }
            const uint32_t row = nvec.div(v);
            const uint32_t col = v - row * nvec.d;
            store<UV, STH>(out + (static_cast<int64_t>(row) * out_pitch + static_cast<int64_t>(col) * UV),
                            narrow<DT, VEC>(fo));
        }
    }
}

}  // namespace astra

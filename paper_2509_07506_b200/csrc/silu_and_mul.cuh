// silu_and_mul (Astra paper, Table 1, Kernel 3):  out = a * sigmoid(a) * b,  row = [a | b].
//
// Elementwise and HBM-bound: 6 bytes move per output (4 read, 2 written).  Each thread owns UNROLL
// vectors of VEC elements; all its 2*UNROLL loads are issued before the first use so that enough
// bytes are in flight per SM to cover HBM latency.  The sigmoid costs two special-function ops per
// element (ex2 and rcp, the fast-math forms the paper's optimised kernel also turns to), in
// binary32, with one rounding at the store.
#pragma once

#include "vec.cuh"

namespace astra {

// SiLU(a) * b in binary32, in the overflow-free form: with t = e^{-|a|} in [0, 1],
// sigmoid(a) = 1/(1+t) for a >= 0 and t/(1+t) for a < 0.  The reciprocal's argument stays in [1, 2].
// ex2 is the non-flushing form so that e^{-|a|} below 2^-126 still yields the (tiny but
// representable) product a * e^{a} * b instead of zero.
__device__ __forceinline__ float silu_mul(float a, float b) {
    float t, d;
    asm("ex2.approx.f32 %0, %1;" : "=f"(t) : "f"(fabsf(a) * -1.4426950408889634f));
    asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(d) : "f"(1.0f + t));
    const float sig = a >= 0.f ? d : t * d;
    return a * sig * b;
}

// Flat indexing: vector v of the output covers out[row, col*VEC .. col*VEC+VEC) with
// row = v / nvec, col = v % nvec, nvec = D / VEC.  A block handles THREADS*UNROLL consecutive vectors.
template <int DT, int VEC, int UNROLL, int THREADS>
__global__ void __launch_bounds__(THREADS)
silu_and_mul_kernel(uint16_t *__restrict__ out, const uint16_t *__restrict__ in,
                    uint32_t total_vecs, FastDiv nvec, int64_t D) {
    const uint32_t base = blockIdx.x * (THREADS * UNROLL) + threadIdx.x;
    Pack<VEC> a[UNROLL], b[UNROLL];
#pragma unroll
    for (int j = 0; j < UNROLL; ++j) {
        const uint32_t v = base + j * THREADS;
        if (v < total_vecs) {
            const uint32_t row = nvec.div(v);
            const uint32_t col = v - row * nvec.d;
            const uint16_t *pa = in + (static_cast<int64_t>(row) * 2 * D + static_cast<int64_t>(col) * VEC);
            a[j] = load<VEC, Ld::StreamReadOnly>(pa);
            b[j] = load<VEC, Ld::StreamReadOnly>(pa + D);
        }
    }
#pragma unroll
    for (int j = 0; j < UNROLL; ++j) {
        const uint32_t v = base + j * THREADS;
        if (v < total_vecs) {
            float fa[VEC], fb[VEC], fo[VEC];
            widen<DT, VEC>(a[j], fa);
            widen<DT, VEC>(b[j], fb);
#pragma unroll
            for (int i = 0; i < VEC; ++i) fo[i] = silu_mul(fa[i], fb[i]);
            store<VEC, St::Stream>(out + static_cast<int64_t>(v) * VEC, narrow<DT, VEC>(fo));
        }
    }
}

}  // namespace astra

// Vector memory access and 16-bit storage conversion helpers shared by the three kernels.
//
// Every kernel here is HBM-bound: each input byte is read once and each output byte written once.
// The helpers therefore expose (a) the widest aligned global access the data allows (2, 4, 8, 16 or
// 32 bytes per thread; 32-byte accesses exist on sm_100 and later) with cache hints for once-touched
// data, and (b) exact widening / single-rounding narrowing between the storage types and binary32.
#pragma once

#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <stdint.h>

#include "astra.h"

namespace astra {

// ---------------------------------------------------------------------------------------------
// Storage types: two packed elements per 32-bit word, low half at the lower address.
// ---------------------------------------------------------------------------------------------
template <int DT> struct Storage;

template <> struct Storage<ASTRA_BF16> {
    static constexpr int UNITS = 1;  // 16-bit units per element
    static __device__ __forceinline__ void widen2(uint32_t w, float &lo, float &hi) {
        lo = __uint_as_float(w << 16);
        hi = __uint_as_float(w & 0xffff0000u);
    }
    static __device__ __forceinline__ uint32_t narrow2(float lo, float hi) {
        __nv_bfloat162 p = __floats2bfloat162_rn(lo, hi);  // one cvt.rn.bf16x2.f32
        return *reinterpret_cast<uint32_t *>(&p);
    }
    static __device__ __forceinline__ float widen1(uint16_t h) {
        return __uint_as_float(static_cast<uint32_t>(h) << 16);
    }
    static __device__ __forceinline__ uint16_t narrow1(float f) {
        return __bfloat16_as_ushort(__float2bfloat16_rn(f));
    }
};

template <> struct Storage<ASTRA_FP16> {
    static constexpr int UNITS = 1;
    static __device__ __forceinline__ void widen2(uint32_t w, float &lo, float &hi) {
        float2 f = __half22float2(*reinterpret_cast<__half2 *>(&w));
        lo = f.x;
        hi = f.y;
    }
    static __device__ __forceinline__ uint32_t narrow2(float lo, float hi) {
        __half2 p = __floats2half2_rn(lo, hi);  // one cvt.rn.f16x2.f32
        return *reinterpret_cast<uint32_t *>(&p);
    }
    static __device__ __forceinline__ float widen1(uint16_t h) {
        return __half2float(__ushort_as_half(h));
    }
    static __device__ __forceinline__ uint16_t narrow1(float f) {
        return __half_as_ushort(__float2half_rn(f));
    }
};

// binary32 storage: an element is two 16-bit units (one 32-bit word) and needs no conversion.
template <> struct Storage<ASTRA_FP32> {
    static constexpr int UNITS = 2;
};

// ---------------------------------------------------------------------------------------------
// A group of N consecutive 16-bit units moved with one global access of 2*N bytes (all tensors are
// addressed in 16-bit units; an element of storage type DT is Storage<DT>::UNITS of them).
// N = 1 is the scalar fallback for odd widths or 2-byte-aligned pointers of the 16-bit types.
// ---------------------------------------------------------------------------------------------
enum class Ld { Stream, StreamReadOnly, Keep };  // once-touched / once-touched and never written / reused (weights)
enum class St { Stream, Default };

template <int VEC> struct Pack {
    static_assert(VEC == 2 || VEC == 4 || VEC == 8 || VEC == 16, "unsupported vector width");
    static constexpr int WORDS = VEC / 2;
    uint32_t w[WORDS];
};
template <> struct Pack<1> {
    static constexpr int WORDS = 1;
    uint32_t w[1];  // low 16 bits hold the element
};

template <int VEC, Ld HINT> __device__ __forceinline__ Pack<VEC> load(const uint16_t *p) {
    Pack<VEC> v;
    if constexpr (VEC == 1) {
        uint16_t h;
        if constexpr (HINT == Ld::Keep)
            asm volatile("ld.global.nc.u16 %0, [%1];" : "=h"(h) : "l"(p));
        else if constexpr (HINT == Ld::StreamReadOnly)
            asm volatile("ld.global.nc.L1::no_allocate.u16 %0, [%1];" : "=h"(h) : "l"(p));
        else
            asm volatile("ld.global.L1::no_allocate.u16 %0, [%1];" : "=h"(h) : "l"(p) : "memory");
        v.w[0] = h;
    } else if constexpr (VEC == 2) {
        if constexpr (HINT == Ld::Keep)
            asm volatile("ld.global.nc.u32 %0, [%1];" : "=r"(v.w[0]) : "l"(p));
        else if constexpr (HINT == Ld::StreamReadOnly)
            asm volatile("ld.global.nc.L1::no_allocate.u32 %0, [%1];" : "=r"(v.w[0]) : "l"(p));
        else
            asm volatile("ld.global.L1::no_allocate.u32 %0, [%1];" : "=r"(v.w[0]) : "l"(p) : "memory");
    } else if constexpr (VEC == 4) {
        if constexpr (HINT == Ld::Keep)
            asm volatile("ld.global.nc.v2.u32 {%0,%1}, [%2];" : "=r"(v.w[0]), "=r"(v.w[1]) : "l"(p));
        else if constexpr (HINT == Ld::StreamReadOnly)
            asm volatile("ld.global.nc.L1::no_allocate.v2.u32 {%0,%1}, [%2];" : "=r"(v.w[0]), "=r"(v.w[1]) : "l"(p));
        else
            asm volatile("ld.global.L1::no_allocate.v2.u32 {%0,%1}, [%2];"
                         : "=r"(v.w[0]), "=r"(v.w[1]) : "l"(p) : "memory");
    } else if constexpr (VEC == 8) {
        if constexpr (HINT == Ld::Keep)
            asm volatile("ld.global.nc.v4.u32 {%0,%1,%2,%3}, [%4];"
                         : "=r"(v.w[0]), "=r"(v.w[1]), "=r"(v.w[2]), "=r"(v.w[3]) : "l"(p));
        else if constexpr (HINT == Ld::StreamReadOnly)
            asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                         : "=r"(v.w[0]), "=r"(v.w[1]), "=r"(v.w[2]), "=r"(v.w[3]) : "l"(p));
        else
            asm volatile("ld.global.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                         : "=r"(v.w[0]), "=r"(v.w[1]), "=r"(v.w[2]), "=r"(v.w[3]) : "l"(p) : "memory");
    } else {  // 32-byte access (sm_100+)
        if constexpr (HINT == Ld::Keep)
            asm volatile("ld.global.nc.v8.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                         : "=r"(v.w[0]), "=r"(v.w[1]), "=r"(v.w[2]), "=r"(v.w[3]),
                           "=r"(v.w[4]), "=r"(v.w[5]), "=r"(v.w[6]), "=r"(v.w[7]) : "l"(p));
        else if constexpr (HINT == Ld::StreamReadOnly)
            asm volatile("ld.global.nc.L1::no_allocate.v8.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                         : "=r"(v.w[0]), "=r"(v.w[1]), "=r"(v.w[2]), "=r"(v.w[3]),
                           "=r"(v.w[4]), "=r"(v.w[5]), "=r"(v.w[6]), "=r"(v.w[7]) : "l"(p));
        else
            asm volatile("ld.global.L1::no_allocate.v8.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                         : "=r"(v.w[0]), "=r"(v.w[1]), "=r"(v.w[2]), "=r"(v.w[3]),
                           "=r"(v.w[4]), "=r"(v.w[5]), "=r"(v.w[6]), "=r"(v.w[7]) : "l"(p) : "memory");
    }
    return v;
}

template <int VEC, St HINT> __device__ __forceinline__ void store(uint16_t *p, const Pack<VEC> &v) {
    if constexpr (VEC == 1) {
        uint16_t h = static_cast<uint16_t>(v.w[0]);
        if constexpr (HINT == St::Stream)
            asm volatile("st.global.cs.u16 [%0], %1;" ::"l"(p), "h"(h) : "memory");
        else
            asm volatile("st.global.u16 [%0], %1;" ::"l"(p), "h"(h) : "memory");
    } else if constexpr (VEC == 2) {
        if constexpr (HINT == St::Stream)
            asm volatile("st.global.cs.u32 [%0], %1;" ::"l"(p), "r"(v.w[0]) : "memory");
        else
            asm volatile("st.global.u32 [%0], %1;" ::"l"(p), "r"(v.w[0]) : "memory");
    } else if constexpr (VEC == 4) {
        if constexpr (HINT == St::Stream)
            asm volatile("st.global.cs.v2.u32 [%0], {%1,%2};" ::"l"(p), "r"(v.w[0]), "r"(v.w[1]) : "memory");
        else
            asm volatile("st.global.v2.u32 [%0], {%1,%2};" ::"l"(p), "r"(v.w[0]), "r"(v.w[1]) : "memory");
    } else if constexpr (VEC == 8) {
        if constexpr (HINT == St::Stream)
            asm volatile("st.global.cs.v4.u32 [%0], {%1,%2,%3,%4};"
                         ::"l"(p), "r"(v.w[0]), "r"(v.w[1]), "r"(v.w[2]), "r"(v.w[3]) : "memory");
        else
            asm volatile("st.global.v4.u32 [%0], {%1,%2,%3,%4};"
                         ::"l"(p), "r"(v.w[0]), "r"(v.w[1]), "r"(v.w[2]), "r"(v.w[3]) : "memory");
    } else {  // 32-byte access (sm_100+)
        if constexpr (HINT == St::Stream)
            asm volatile("st.global.cs.v8.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};"
                         ::"l"(p), "r"(v.w[0]), "r"(v.w[1]), "r"(v.w[2]), "r"(v.w[3]),
                           "r"(v.w[4]), "r"(v.w[5]), "r"(v.w[6]), "r"(v.w[7]) : "memory");
        else
            asm volatile("st.global.v8.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};"
                         ::"l"(p), "r"(v.w[0]), "r"(v.w[1]), "r"(v.w[2]), "r"(v.w[3]),
                           "r"(v.w[4]), "r"(v.w[5]), "r"(v.w[6]), "r"(v.w[7]) : "memory");
    }
}

// Pack of VEC elements of storage type DT  <->  VEC floats.
template <int DT, int VEC>
__device__ __forceinline__ void widen(const Pack<VEC * Storage<DT>::UNITS> &v, float (&f)[VEC]) {
    if constexpr (DT == ASTRA_FP32) {
#pragma unroll
        for (int i = 0; i < VEC; ++i) f[i] = __uint_as_float(v.w[i]);
    } else if constexpr (VEC == 1) {
        f[0] = Storage<DT>::widen1(static_cast<uint16_t>(v.w[0]));
    } else {
#pragma unroll
        for (int i = 0; i < VEC / 2; ++i) Storage<DT>::widen2(v.w[i], f[2 * i], f[2 * i + 1]);
    }
}

template <int DT, int VEC>
__device__ __forceinline__ Pack<VEC * Storage<DT>::UNITS> narrow(const float (&f)[VEC]) {
    Pack<VEC * Storage<DT>::UNITS> v;
    if constexpr (DT == ASTRA_FP32) {
#pragma unroll
        for (int i = 0; i < VEC; ++i) v.w[i] = __float_as_uint(f[i]);
    } else if constexpr (VEC == 1) {
        v.w[0] = Storage<DT>::narrow1(f[0]);
    } else {
#pragma unroll
        for (int i = 0; i < VEC / 2; ++i) v.w[i] = Storage<DT>::narrow2(f[2 * i], f[2 * i + 1]);
    }
    return v;
}

// ---------------------------------------------------------------------------------------------
// Programmatic dependent launch.  A kernel launched with the programmatic-stream-serialization
// attribute may be scheduled while the previous kernel in the stream is still draining.  It must
// not touch global memory before `grid_dependency_wait()` returns (the previous grid has then
// completed and its writes are visible), so stream order is preserved; what overlaps is only the
// launch latency and the block prologue.  `grid_launch_dependents()` lets the next kernel in the
// stream do the same with respect to this one.  Both are no-ops for an ordinary launch.
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ void grid_dependency_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void grid_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

// ---------------------------------------------------------------------------------------------
// L2 prefetch of a contiguous byte range with one instruction (the bulk-copy engine's prefetch form;
// fire and forget: nothing is returned, nothing has to be waited for).  It needs a 16-byte aligned
// start and a multiple of 16 bytes, so the range is trimmed inward to that; the trimmed edges are
// simply fetched by the loads later.
//
// Use: a block issues it for its inputs BEFORE `grid_dependency_wait()`.  A prefetch consumes no
// data, and L2 is the point of coherence for everything the previous kernel writes, so this is safe
// whatever that kernel does to the same addresses.  What it buys: the request reaches the memory
// system as one contiguous piece before the block's warps have even been through the wait, so the
// first-byte latency overlaps the previous kernel's drain and the block's own prologue.  Measured
// with inputs that are cold in L2: merge 5 % at [8192, 32, 128] and 17 % at [512, 32, 128], silu 5 %
// at [1024, 14336] and 24 % at [128, 14336], rmsnorm 3 % at [1024, 4096]; more when part of the
// input is still in L2.  Only for memory of this GPU.
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ void prefetch_l2_range(const void *begin, int64_t bytes) {
    const uint64_t lo = (reinterpret_cast<uint64_t>(begin) + 15u) & ~static_cast<uint64_t>(15);
    const uint64_t hi = (reinterpret_cast<uint64_t>(begin) + static_cast<uint64_t>(bytes)) & ~static_cast<uint64_t>(15);
    if (hi > lo) {
        const uint32_t n = static_cast<uint32_t>(hi - lo);
        asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(lo), "r"(n) : "memory");
    }
}

// ---------------------------------------------------------------------------------------------
// Division of a 31-bit index by a launch-constant divisor: q = (n * mul) >> shift, exact for
// 0 <= n < 2^31 and 1 <= d < 2^31 with shift = 31 + ceil(log2 d), mul = ceil(2^shift / d) <= 2^32 - 1
// (d = 1 is special-cased so that mul fits 32 bits).
// ---------------------------------------------------------------------------------------------
struct FastDiv {
    uint32_t d;
    uint32_t mul;
    uint32_t shift;
    static inline FastDiv make(uint32_t divisor) {
        FastDiv f;
        f.d = divisor;
        uint32_t s = 0;
        while ((1ull << s) < divisor) ++s;
        f.shift = 31 + s;
        uint64_t p = 1ull << f.shift;
        f.mul = static_cast<uint32_t>((p + divisor - 1) / divisor);  // d=1: 2^31; d>=2: < 2^32
        return f;
    }
    __host__ __device__ __forceinline__ uint32_t div(uint32_t n) const {
        return static_cast<uint32_t>((static_cast<uint64_t>(n) * mul) >> shift);
    }
};

}  // namespace astra

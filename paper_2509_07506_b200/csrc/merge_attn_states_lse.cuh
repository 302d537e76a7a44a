// merge_attn_states_lse (Astra paper, Table 1, Kernel 1):
//     V_out = (e^{Sa} Va + e^{Sb} Vb) / (e^{Sa} + e^{Sb}),   S_out = log(e^{Sa} + e^{Sb}).
//
// HBM-bound: per (token, head) row of D elements, 2*D*2 bytes are read and D*2 written, plus three
// 4-byte scores.  The two mixing weights depend only on the row, so each thread derives them once
// for the vector(s) it owns (the paper's hoisting of the exponentials out of the element loop); the
// element work is one multiply and one fused multiply-add.
#pragma once

#include "vec.cuh"

namespace astra {

struct MergeWeights {
    float wa, wb;   // normalised weights of the two states
    float lse;      // merged score
    bool use_a, use_b;
};

// m = max(Sa, Sb); with t = e^{min - max} in [0, 1]: weight of the larger = 1/(1+t), of the
// smaller = t/(1+t), S_out = m + log(1+t).  A score of -inf gives t = 0 exactly, so the other state
// passes through with weight exactly 1; its own V is not used at all.  Both -inf: empty result.
__device__ __forceinline__ MergeWeights merge_weights(float sa, float sb) {
    MergeWeights r;
    const float m = fmaxf(sa, sb);
    const float lo = fminf(sa, sb);
    if (m == -INFINITY) {  // both states empty
        r.wa = 0.f; r.wb = 0.f; r.lse = -INFINITY; r.use_a = false; r.use_b = false;
        return r;
    }
    // t in [0, 1]; exactly 0 for lo = -inf, exactly 1 for lo = m.  Non-flushing ex2, so a weight
    // below 2^-126 is still a (subnormal) weight rather than zero.
    float t;
    asm("ex2.approx.f32 %0, %1;" : "=f"(t) : "f"((lo - m) * 1.4426950408889634f));
    const float inv = __fdividef(1.0f, 1.0f + t);
    const float w_hi = inv, w_lo = t * inv;
    const bool a_is_hi = sa >= sb;
    r.wa = a_is_hi ? w_hi : w_lo;
    r.wb = a_is_hi ? w_lo : w_hi;
    // log(1 + t) with 1 + t in [1, 2]: lg2.approx is within about 2^-22 absolute there
    float l2;
    asm("lg2.approx.f32 %0, %1;" : "=f"(l2) : "f"(1.0f + t));
    r.lse = fmaf(l2, 0.6931471805599453f, m);
    // +inf or NaN scores are outside the domain (e^{S} / e^{S} = inf / inf): everything becomes NaN.
    if (!(m < INFINITY) || sa != sa || sb != sb) { r.wa = r.wb = r.lse = __int_as_float(0x7fc00000); }
    r.use_a = !(r.wa == 0.f);
    r.use_b = !(r.wb == 0.f);
    return r;
}

// Strides of one [T, Hh, D] value tensor (in 16-bit units) or one [T, Hh] score tensor (in floats);
// D is contiguous.
struct MergeStrides {
    int64_t va_t, va_h, vb_t, vb_h, vo_t, vo_h;  // values: token and head strides
    int64_t sa_t, sa_h, sb_t, sb_h, so_t, so_h;  // scores: token and head strides
};

// Flat indexing over vectors of VEC elements: vector v belongs to row = v / nvec (row = token*Hh+head).
template <int DT, int VEC, int UNROLL, int THREADS, Ld LDH = Ld::Stream, St STH = St::Stream, bool PREFETCH = true>
__global__ void __launch_bounds__(THREADS)
merge_attn_states_lse_kernel(uint16_t *v_out, float *lse_out,
                             const uint16_t *v_a, const float *lse_a,
                             const uint16_t *v_b, const float *lse_b,
                             uint32_t total_vecs, FastDiv nvec) {
    constexpr int UV = VEC * Storage<DT>::UNITS;  // 16-bit units per vector
    const uint32_t base = blockIdx.x * (THREADS * UNROLL) + threadIdx.x;
    // Ahead of the dependency wait the block asks for its (contiguous) share of both value tensors to
    // be brought into L2.
    if (PREFETCH && threadIdx.x == 0 && base < total_vecs) {
        const uint32_t n = min(static_cast<uint32_t>(THREADS * UNROLL), total_vecs - base);
        prefetch_l2_range(v_a + static_cast<int64_t>(base) * UV, static_cast<int64_t>(n) * UV * 2);
        prefetch_l2_range(v_b + static_cast<int64_t>(base) * UV, static_cast<int64_t>(n) * UV * 2);
    }
    grid_dependency_wait();
    grid_launch_dependents();
    Pack<UV> a[UNROLL], b[UNROLL];
    float sa[UNROLL], sb[UNROLL];
    uint32_t row[UNROLL];
#pragma unroll
    for (int j = 0; j < UNROLL; ++j) {
        const uint32_t v = base + j * THREADS;
        if (v < total_vecs) {
            row[j] = nvec.div(v);
            // v_out may be exactly v_a or v_b, so these are ordinary (coherent) loads; the thread
            // that reads a vector is the only one that writes it
            a[j] = load<UV, LDH>(v_a + static_cast<int64_t>(v) * UV);
            b[j] = load<UV, LDH>(v_b + static_cast<int64_t>(v) * UV);
            sa[j] = lse_a[row[j]];
            sb[j] = lse_b[row[j]];
        }
    }
#pragma unroll
    for (int j = 0; j < UNROLL; ++j) {
        const uint32_t v = base + j * THREADS;
        if (v < total_vecs) {
            const MergeWeights mw = merge_weights(sa[j], sb[j]);
            float fa[VEC], fb[VEC], fo[VEC];
            widen<DT, VEC>(a[j], fa);
            widen<DT, VEC>(b[j], fb);
#pragma unroll
            for (int i = 0; i < VEC; ++i) {
                // a zero-weight side is dropped, not multiplied: its payload may be Inf/NaN garbage
                const float ta = mw.use_a ? fa[i] * mw.wa : 0.f;
                fo[i] = mw.use_b ? fmaf(fb[i], mw.wb, ta) : ta;
            }
            store<UV, STH>(v_out + static_cast<int64_t>(v) * UV, narrow<DT, VEC>(fo));
            if (lse_out != nullptr && v == row[j] * nvec.d) lse_out[row[j]] = mw.lse;
        }
    }
}

}  // namespace astra

namespace astra {

// Same computation for arbitrarily strided tensors (head_dim contiguous): row = token * Hh + head is
// split again into (token, head) to address each tensor by its own strides.  This is the form for
// head-major scores ([Hh, T]) or values that are slices of a wider buffer.
template <int DT, int VEC, int UNROLL, int THREADS>
__global__ void __launch_bounds__(THREADS)
merge_attn_states_lse_strided_kernel(uint16_t *v_out, float *lse_out,
                                     const uint16_t *v_a, const float *lse_a,
                                     const uint16_t *v_b, const float *lse_b,
                                     uint32_t total_vecs, uint32_t row0, FastDiv nvec, FastDiv heads,
                                     MergeStrides st) {
    constexpr int UV = VEC * Storage<DT>::UNITS;  // 16-bit units per vector
    const uint32_t base = blockIdx.x * (THREADS * UNROLL) + threadIdx.x;
    grid_dependency_wait();
    grid_launch_dependents();
#pragma unroll
    for (int j = 0; j < UNROLL; ++j) {
        const uint32_t v = base + j * THREADS;
        if (v < total_vecs) {
            const uint32_t lrow = nvec.div(v);
            const int64_t col = static_cast<int64_t>(v - lrow * nvec.d) * UV;
            const uint32_t row = row0 + lrow;  // rows of this launch start at row0
            const uint32_t t = heads.div(row);
            const uint32_t h = row - t * heads.d;
            const Pack<UV> a = load<UV, Ld::Stream>(v_a + (t * st.va_t + h * st.va_h + col));
            const Pack<UV> b = load<UV, Ld::Stream>(v_b + (t * st.vb_t + h * st.vb_h + col));
            const MergeWeights mw = merge_weights(lse_a[t * st.sa_t + h * st.sa_h], lse_b[t * st.sb_t + h * st.sb_h]);
            float fa[VEC], fb[VEC], fo[VEC];
            widen<DT, VEC>(a, fa);
            widen<DT, VEC>(b, fb);
#pragma unroll
            for (int i = 0; i < VEC; ++i) {
                const float ta = mw.use_a ? fa[i] * mw.wa : 0.f;
                fo[i] = mw.use_b ? fmaf(fb[i], mw.wb, ta) : ta;
            }
            store<UV, St::Stream>(v_out + (t * st.vo_t + h * st.vo_h + col), narrow<DT, VEC>(fo));
            if (lse_out != nullptr && col == 0) lse_out[t * st.so_t + h * st.so_h] = mw.lse;
        }
    }
}

}  // namespace astra

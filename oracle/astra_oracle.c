/*
 * fp64 CPU oracle for the three memory-bound LLM-serving operations of the
 * Astra paper (Table 1): fused_add_rmsnorm, silu_and_mul, merge_attn_states_lse.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain definition the CUDA
 * library is checked against.  It shares no code, header, table or constant
 * with the CUDA path, and nothing on the product path may call it.
 *
 * Every function is the printed formula evaluated in double precision on the
 * exact values of the 16-bit storage patterns the GPU receives.  No blocking,
 * fusion or reordering: one loop per index of the formula.  The only
 * parallelism is an OpenMP "parallel for" over independent rows, used when the
 * oracle is timed as a CPU baseline (nthreads > 1); it does not change any
 * arithmetic because rows never interact.
 *
 * Storage formats.  dtype 0 = bfloat16 (1 sign, 8 exponent, 7 fraction bits),
 * dtype 1 = IEEE binary16 (1, 5, 10), dtype 2 = IEEE binary32 (value tensors are
 * then arrays of 32-bit patterns; the C compiler's float is that format, so it is
 * widened by a cast and rounded by a cast).  The 16-bit formats are widened exactly to double and
 * rounded back with round-to-nearest-even, written out arithmetically below
 * (frexp / ldexp / nearbyint), not with bit tricks, so they can be read against
 * the format definitions.
 *
 * Pins (tests, CPU only): closed forms, invariants, textbook reductions
 * (plain RMSNorm, two-way softmax, attention over a split key set), library
 * routines of torch on CPU in fp64, an integer-only bf16 adder for the
 * residual sum, and torch's own float->bf16 / float->fp16 casts for the
 * rounding helpers; for the partial-sum form of Kernel 2 an exact-rational
 * adder with its own binary32 rounding, cases whose result depends on the
 * order and on the number of roundings, and its N = 1 case against
 * fused_add_rmsnorm.  No function here is "parity unpinned".
 */
#include <math.h>
#include <stdint.h>
#include <string.h>

#ifndef ORACLE_BUILD_ID
#define ORACLE_BUILD_ID "unidentified"
#endif
/* hash of this file as compiled (set by the build script), findable in the built library */
const char oracle_build_marker[] = "oracle-build-id:" ORACLE_BUILD_ID;

#define ORACLE_BF16 0
#define ORACLE_FP16 1
#define ORACLE_FP32 2 /* IEEE binary32 storage: patterns are 32 bits wide */

typedef struct {
    int frac_bits; /* explicit fraction bits            */
    int exp_bits;  /* exponent field width              */
    int bias;      /* exponent bias                     */
} storage_format;

static storage_format format_of(int dtype)
{
    storage_format f;
    if (dtype == ORACLE_FP16) {
        f.frac_bits = 10; f.exp_bits = 5; f.bias = 15;
    } else { /* bfloat16; binary32 storage never goes through this table */
        f.frac_bits = 7;  f.exp_bits = 8; f.bias = 127;
    }
    return f;
}

/* Exact value of a 16-bit storage pattern. */
static double widen(uint16_t bits, storage_format f)
{
    int sign = (bits >> 15) & 1;
    int exp_field = (bits >> f.frac_bits) & ((1 << f.exp_bits) - 1);
    int frac = bits & ((1 << f.frac_bits) - 1);
    int exp_all_ones = (1 << f.exp_bits) - 1;
    double v;
    if (exp_field == exp_all_ones) {
        v = frac ? NAN : INFINITY;
    } else if (exp_field == 0) {
        /* subnormal: frac * 2^(1 - bias - frac_bits) */
        v = ldexp((double)frac, 1 - f.bias - f.frac_bits);
    } else {
        v = ldexp((double)((1 << f.frac_bits) + frac), exp_field - f.bias - f.frac_bits);
    }
    return sign ? -v : v;
}

/* Round a double to the storage format, nearest-even, return the bit pattern.
   nearbyint() rounds to nearest-even in the default rounding mode. */
static uint16_t round_to_storage(double v, storage_format f)
{
    uint16_t sign = signbit(v) ? 0x8000u : 0u;
    int exp_all_ones = (1 << f.exp_bits) - 1;
    double a = fabs(v);
    if (isnan(v))
        return (uint16_t)(sign | (exp_all_ones << f.frac_bits) | (1 << (f.frac_bits - 1)));
    if (isinf(v))
        return (uint16_t)(sign | (exp_all_ones << f.frac_bits));
    if (a == 0.0)
        return sign;

    int e_min = 1 - f.bias;                 /* exponent of the smallest normal   */
    int e_max = exp_all_ones - 1 - f.bias;  /* exponent of the largest finite    */
    int e;
    (void)frexp(a, &e);                     /* a = m * 2^e, m in [0.5, 1)        */
    int E = e - 1;                          /* a in [2^E, 2^(E+1))               */
    if (E < e_min) E = e_min;               /* subnormals share the quantum of e_min */
    double quantum = ldexp(1.0, E - f.frac_bits);
    double q = nearbyint(a / quantum);      /* division by a power of two: exact */
    double r = q * quantum;                 /* the rounded magnitude             */

    /* r may have carried into the next binade; re-derive its exponent. */
    if (r >= ldexp(1.0, e_max + 1))
        return (uint16_t)(sign | (exp_all_ones << f.frac_bits)); /* overflow -> inf */
    if (r < ldexp(1.0, e_min)) {
        /* subnormal or zero: fraction field counts quanta of 2^(e_min - frac_bits) */
        uint16_t frac = (uint16_t)(r / ldexp(1.0, e_min - f.frac_bits));
        return (uint16_t)(sign | frac);
    }
    (void)frexp(r, &e);
    E = e - 1;
    uint16_t exp_field = (uint16_t)(E + f.bias);
    uint16_t frac = (uint16_t)(r / ldexp(1.0, E - f.frac_bits) - (double)(1 << f.frac_bits));
    return (uint16_t)(sign | (exp_field << f.frac_bits) | frac);
}

/* Exposed so the tests can pin the two helpers on their own. */
double oracle_widen(uint16_t bits, int dtype)
{
    return widen(bits, format_of(dtype));
}

uint16_t oracle_round_to_storage(double v, int dtype)
{
    return round_to_storage(v, format_of(dtype));
}

/* Element i of a value tensor of the given storage type, as its exact double value. */
static double load_value(const void *base, int64_t i, int dtype, storage_format f)
{
    if (dtype == ORACLE_FP32) {
        float v;
        memcpy(&v, (const unsigned char *)base + 4 * i, 4);
        return (double)v;
    }
    return widen(((const uint16_t *)base)[i], f);
}

/* Store a binary32 value into element i of a storage-typed tensor, rounding once (nearest-even). */
static void store_rounded(void *base, int64_t i, float v, int dtype, storage_format f)
{
    if (dtype == ORACLE_FP32) {
        memcpy((unsigned char *)base + 4 * i, &v, 4);
    } else {
        ((uint16_t *)base)[i] = round_to_storage((double)v, f);
    }
}

/*
 * fused_add_rmsnorm  (Table 1, Kernel 2):
 *     y = (x + r) / sqrt( (1/H) * ||x + r||^2 + eps )  (.)  w
 *
 * x, r : [T, H] storage patterns.  w : [H].
 * y_out        : [T, H] doubles, the formula's value.
 * residual_out : [T, H] storage patterns of the updated residual.
 *
 * Readings where Table 1 is silent:
 *  - The sum s = x + r is formed as a binary32 add (the exact double sum
 *    rounded once to float).  The updated residual is that float rounded once
 *    to the storage dtype.  This output is compared bit for bit.
 *  - The norm uses the float sum itself, not the storage-rounded residual.
 *  - eps is a float argument taken at its exact value; it sits inside the
 *    square root, added to the mean of squares, as printed.
 *  - No rounding between the normalisation and the multiplication by w.
 */
/* The one binary32 addition of the operation.  Operands of the 16-bit storage types have at most
   11 significant bits, so their double sum rounded once to float is that addition; binary32
   operands are added as floats. */
static float add_binary32(double a, double b, int dtype)
{
    if (dtype == ORACLE_FP32) {
        volatile float fa = (float)a, fb = (float)b;
        volatile float s = fa + fb;
        return s;
    }
    return (float)(a + b);
}

void oracle_fused_add_rmsnorm(const void *x, const void *r, const void *w,
                              int64_t T, int64_t H, float eps, int dtype,
                              double *y_out, void *residual_out, int nthreads)
{
    storage_format f = format_of(dtype);
    if (nthreads < 1) nthreads = 1;
#pragma omp parallel for num_threads(nthreads) schedule(static)
    for (int64_t t = 0; t < T; ++t) {
        double sum_sq = 0.0;
        for (int64_t j = 0; j < H; ++j) {
            double xv = load_value(x, t * H + j, dtype, f), rv = load_value(r, t * H + j, dtype, f);
            double s = (double)add_binary32(xv, rv, dtype);
            sum_sq += s * s;
        }
        double denom = sqrt(sum_sq / (double)H + (double)eps);
        for (int64_t j = 0; j < H; ++j) {
            double xv = load_value(x, t * H + j, dtype, f), rv = load_value(r, t * H + j, dtype, f);
            float s32 = add_binary32(xv, rv, dtype);
            store_rounded(residual_out, t * H + j, s32, dtype, f);
            y_out[t * H + j] = (double)s32 / denom * load_value(w, j, dtype, f);
        }
    }
}

/*
 * fused_allreduce_add_rmsnorm: Kernel 2 of Table 1 applied to a hidden state that arrives as N
 * partial sums, one per tensor-parallel rank (the all-reduce that precedes the operation in
 * tensor-parallel serving, folded into it):
 *     x = x_0 + x_1 + ... + x_{N-1};   s = x + r;   r_out <- s;   y = s / sqrt(mean(s^2) + eps) (.) w
 *
 * parts : N pointers to [T, H] storage patterns, in rank order.  r : [T, H].  w : [H].
 * y_out : [T, H] doubles.  residual_out : [T, H] storage patterns.
 *
 * Readings (the paper states Kernel 2 for one x only; where the additions are rounded has to be
 * fixed because the updated residual is compared bit for bit):
 *  - every addition is one binary32 addition (round to nearest even): the partials are added in
 *    rank order starting from x_0, then the residual is added last:
 *        s = fl( fl( ... fl( fl(x_0 + x_1) + x_2 ) ... + x_{N-1} ) + r ).
 *    N = 1 is fused_add_rmsnorm exactly.  Rank order makes every rank of a tensor-parallel group
 *    compute the same bits.
 *  - nothing is rounded to the storage type before the residual joins (a separate all-reduce
 *    would have rounded x there); the residual gets s rounded once to the storage type;
 *  - the norm uses the binary32 s; eps and the weight as in fused_add_rmsnorm.
 * The C type float is binary32 and this file is compiled without contraction or excess precision,
 * so `a + b` on floats is that one addition; the volatile keeps the compiler from re-associating.
 */
static float value_as_float(const void *base, int64_t i, int dtype, storage_format f)
{
    /* every storage pattern is exactly representable in binary32 */
    return (float)load_value(base, i, dtype, f);
}

static float sum_in_rank_order(const void *const *parts, int n_parts, const void *r, int64_t i,
                               int dtype, storage_format f)
{
    volatile float acc = value_as_float(parts[0], i, dtype, f);
    for (int p = 1; p < n_parts; ++p) {
        volatile float next = value_as_float(parts[p], i, dtype, f);
        acc = acc + next;
    }
    volatile float res = value_as_float(r, i, dtype, f);
    acc = acc + res;
    return acc;
}

void oracle_fused_allreduce_add_rmsnorm(const void *const *parts, int n_parts, const void *r,
                                        const void *w, int64_t T, int64_t H, float eps, int dtype,
                                        double *y_out, void *residual_out, int nthreads)
{
    storage_format f = format_of(dtype);
    if (nthreads < 1) nthreads = 1;
#pragma omp parallel for num_threads(nthreads) schedule(static)
    for (int64_t t = 0; t < T; ++t) {
        double sum_sq = 0.0;
        for (int64_t j = 0; j < H; ++j) {
            double s = (double)sum_in_rank_order(parts, n_parts, r, t * H + j, dtype, f);
            sum_sq += s * s;
        }
        double denom = sqrt(sum_sq / (double)H + (double)eps);
        for (int64_t j = 0; j < H; ++j) {
            float s32 = sum_in_rank_order(parts, n_parts, r, t * H + j, dtype, f);
            store_rounded(residual_out, t * H + j, s32, dtype, f);
            y_out[t * H + j] = (double)s32 / denom * load_value(w, j, dtype, f);
        }
    }
}

/*
 * silu_and_mul  (Table 1, Kernel 3):
 *     out = SiLU(a) (.) b,   SiLU(z) = z / (1 + e^{-z})
 *
 * input : [T, 2*D]; columns 0..D-1 are the gate a, columns D..2D-1 are b.
 * out   : [T, D] doubles.
 *
 * For z below -700, e^{-z} overflows a double; the algebraically identical form
 * z * e^{z} / (1 + e^{z}) is used there so the function stays total.
 */
static double silu(double z)
{
    if (z < -700.0) {
        double ez = exp(z);
        return z * ez / (1.0 + ez);
    }
    return z / (1.0 + exp(-z));
}

void oracle_silu_and_mul(const void *input, int64_t T, int64_t D, int dtype,
                         double *out, int nthreads)
{
    storage_format f = format_of(dtype);
    if (nthreads < 1) nthreads = 1;
#pragma omp parallel for num_threads(nthreads) schedule(static)
    for (int64_t t = 0; t < T; ++t) {
        const int64_t row = t * 2 * D;
        for (int64_t i = 0; i < D; ++i) {
            double a = load_value(input, row + i, dtype, f);
            double b = load_value(input, row + D + i, dtype, f);
            out[t * D + i] = silu(a) * b;
        }
    }
}

/*
 * merge_attn_states_lse  (Table 1, Kernel 1):
 *     V_out = (e^{Sa} Va + e^{Sb} Vb) / (e^{Sa} + e^{Sb})
 *     S_out = log(e^{Sa} + e^{Sb})                        (natural log)
 *
 * v_a, v_b : [T, Hh, D] storage patterns.  lse_a, lse_b : [T, Hh] binary32.
 * v_out    : [T, Hh, D] doubles.           lse_out      : [T, Hh] doubles.
 *
 * Evaluated after factoring e^{m}, m = max(Sa, Sb), out of numerator and
 * denominator; this is the same real number and keeps e^{S} inside double range.
 *
 * Readings where Table 1 is silent:
 *  - One score -inf: its weight is exactly 0 and that side's V does not
 *    contribute (it is skipped, not multiplied), so the other state is returned.
 *  - Both scores -inf (an empty state merged with an empty state):
 *    V_out = 0 and S_out = -inf.
 *  - +inf or NaN scores are outside the operation's domain: NaN out.
 */
void oracle_merge_attn_states_lse(const void *v_a, const float *lse_a,
                                  const void *v_b, const float *lse_b,
                                  int64_t T, int64_t Hh, int64_t D, int dtype,
                                  double *v_out, double *lse_out, int nthreads)
{
    storage_format f = format_of(dtype);
    if (nthreads < 1) nthreads = 1;
#pragma omp parallel for num_threads(nthreads) schedule(static)
    for (int64_t th = 0; th < T * Hh; ++th) {
        double sa = (double)lse_a[th];
        double sb = (double)lse_b[th];
        const int64_t base = th * D;
        double *vo = v_out + th * D;

        if (isnan(sa) || isnan(sb) || sa == INFINITY || sb == INFINITY) {
            for (int64_t d = 0; d < D; ++d) vo[d] = NAN;
            lse_out[th] = NAN;
            continue;
        }
        if (sa == -INFINITY && sb == -INFINITY) {
            for (int64_t d = 0; d < D; ++d) vo[d] = 0.0;
            lse_out[th] = -INFINITY;
            continue;
        }
        double m = sa > sb ? sa : sb;
        double wa = exp(sa - m); /* exp(-inf) = 0 exactly */
        double wb = exp(sb - m);
        double denom = wa + wb;
        for (int64_t d = 0; d < D; ++d) {
            double num = 0.0;
            if (wa != 0.0) num += wa * load_value(v_a, base + d, dtype, f);
            if (wb != 0.0) num += wb * load_value(v_b, base + d, dtype, f);
            vo[d] = num / denom;
        }
        lse_out[th] = m + log(denom);
    }
}

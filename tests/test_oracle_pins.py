"""Pins for the fp64 oracle (CPU only).

The oracle is the ground truth of every GPU parity test, so it is first checked against
things that are not itself: closed forms and textbook constants (tests/golden/hand_values.txt),
invariants of the definitions in Table 1 of the Astra paper, torch's CPU library routines in
fp64, arbitrary-precision brute force (``decimal``) on tiny shapes, an integer-only adder for
the residual sum, and attention over a split key set for the merge.
"""
import decimal
import math
import os

import numpy as np
import pytest
import torch

import oracle
from paper_2509_07506_b200 import workloads as wl

BF16, FP16, FP32 = wl.BF16, wl.FP16, wl.FP32
DTYPES = [BF16, FP16]                # the 16-bit storage formats (helpers that take 16-bit patterns)
VALUE_DTYPES = [BF16, FP16, FP32]    # every storage type of the three operations
TD = {BF16: torch.bfloat16, FP16: torch.float16, FP32: torch.float32}


def golden():
    path = os.path.join(os.path.dirname(__file__), "golden", "hand_values.txt")
    out = {}
    with open(path) as fh:
        for line in fh:
            if line.startswith("#") or "|" not in line:
                continue
            name, value, _ = [p.strip() for p in line.split("|", 2)]
            out[name] = float(value)
    return out


GOLD = golden()


def enc(values, dtype):
    """Storage patterns of values that are cast (RNE) by torch."""
    t = torch.tensor(values, dtype=torch.float64).to(TD[dtype])
    return wl.bits(t)


def dec(bits_arr, dtype):
    """Exact float64 values of storage patterns, via torch's cast (independent of the oracle)."""
    pat = np.uint32 if dtype == FP32 else np.uint16
    return wl.from_bits(np.asarray(bits_arr, dtype=pat), dtype).to(torch.float64).numpy()


# ---------------------------------------------------------------------------------------
# storage helpers
# ---------------------------------------------------------------------------------------

@pytest.mark.parametrize("dtype", DTYPES)
def test_widen_all_patterns_match_torch_cast(dtype):
    allbits = np.arange(65536, dtype=np.uint32).astype(np.uint16)
    want = dec(allbits, dtype)
    got = np.array([oracle.widen(int(b), dtype) for b in allbits])
    nan = np.isnan(want)
    assert np.array_equal(np.isnan(got), nan)
    assert np.array_equal(got[~nan], want[~nan])
    assert np.array_equal(np.signbit(got[~nan]), np.signbit(want[~nan]))


@pytest.mark.parametrize("dtype", DTYPES)
def test_round_trip_all_patterns(dtype):
    for b in range(65536):
        v = oracle.widen(b, dtype)
        if math.isnan(v):
            continue
        assert oracle.round_to_storage(v, dtype) == b


@pytest.mark.parametrize("dtype", DTYPES)
def test_round_to_storage_matches_torch_cast(dtype):
    g = torch.Generator().manual_seed(11)
    mag = torch.exp(torch.randn(30000, generator=g, dtype=torch.float64) * (12 if dtype == FP16 else 40))
    vals = torch.randn(30000, generator=g, dtype=torch.float64) * mag
    # exact ties and their neighbours between adjacent storage values, all binades sampled
    pats = np.arange(0, 0x7c00 if dtype == FP16 else 0x7f80, 37, dtype=np.uint32).astype(np.uint16)
    lo = dec(pats, dtype)
    hi = dec((pats + 1).astype(np.uint16), dtype)
    hi = np.where(np.isfinite(hi), hi, lo * 2)
    mid = (lo + hi) / 2
    mid32 = mid.astype(np.float32)  # midpoints need one more bit than the storage format: exact in binary32
    ties = np.concatenate([mid32, np.nextafter(mid32, np.float32(np.inf)),
                           np.nextafter(mid32, np.float32(-np.inf)), -mid32]).astype(np.float64)
    special = np.array([0.0, -0.0, np.inf, -np.inf, 65504.0, 65519.99, 65520.0, 1e-8, 2.0 ** -25,
                        2.0 ** -24, 3.0 * 2.0 ** -25, 3.3895313892515355e38, 3.4e38, 1e39, 2.0 ** -134,
                        2.0 ** -133, 1.5 * 2.0 ** -133])
    # binary32 inputs only: that is what the oracle rounds (the float sum), and torch's cast from
    # binary32 to either storage type is a single rounding
    with np.errstate(over="ignore"):
        allv = np.concatenate([vals.numpy(), ties, special]).astype(np.float32).astype(np.float64)
    want = wl.bits(torch.from_numpy(allv.astype(np.float32)).to(TD[dtype]))
    got = np.array([oracle.round_to_storage(float(v), dtype) for v in allv], dtype=np.uint16)
    assert np.array_equal(got, want)


# ---------------------------------------------------------------------------------------
# residual sum: bit-exact pin against an integer-only adder
# ---------------------------------------------------------------------------------------

def _rne_int(n, p):
    """Round the positive integer n to p significant bits, nearest-even."""
    bl = n.bit_length()
    if bl <= p:
        return n
    sh = bl - p
    q, rem = n >> sh, n & ((1 << sh) - 1)
    half = 1 << (sh - 1)
    if rem > half or (rem == half and (q & 1)):
        q += 1
    return q << sh


def _bf16_fields(b):
    s, e, f = b >> 15, (b >> 7) & 0xff, b & 0x7f
    return s, e, f


def int_bf16_add(a, b):
    """bf16 + bf16 -> binary32 (RNE) -> bf16 (RNE) with Python integers only.
    Values are integers in units of 2^-133 (the bf16 subnormal quantum)."""
    def to_int(p):
        s, e, f = _bf16_fields(p)
        assert e != 0xff
        m = f if e == 0 else (0x80 | f)
        sh = 0 if e == 0 else e - 1
        v = m << sh
        return -v if s else v
    total = to_int(a) + to_int(b)
    if total == 0:
        # IEEE: x + (-x) = +0, (-0) + (-0) = -0
        neg = (a >> 15) & (b >> 15)
        return 0x8000 if neg else 0
    sign = 0x8000 if total < 0 else 0
    n = _rne_int(abs(total), 24)       # binary32 has 24 significant bits; no fp32 subnormals reachable
    n = _rne_int(n, 8)                 # bf16 has 8 significant bits; subnormals are exact integers < 128
    if n < 0x80:                       # subnormal
        return sign | n
    bl = n.bit_length()
    e = bl - 8 + 1
    if e >= 0xff:
        return sign | 0x7f80
    frac = (n >> (bl - 8)) & 0x7f
    return sign | (e << 7) | frac


def _finite_bf16(rng, n):
    b = rng.integers(0, 65536, size=n, dtype=np.uint32).astype(np.uint16)
    b = b[((b >> 7) & 0xff) != 0xff]
    return b


def test_residual_sum_bf16_against_integer_adder():
    rng = np.random.default_rng(5)
    partner = enc([1.0, -1.0, 0.0078125, -3.140625, 1e-30, 2.0 ** -130, 3e38, -0.0], BF16)
    allb = np.arange(65536, dtype=np.uint32).astype(np.uint16)
    allb = allb[((allb >> 7) & 0xff) != 0xff]
    xs = [np.tile(allb, 1)]
    rs = [np.full(allb.shape, partner[0], dtype=np.uint16)]
    for p in partner[1:]:
        sub = allb[:: 7]
        xs.append(sub)
        rs.append(np.full(sub.shape, p, dtype=np.uint16))
    # stratified random pairs, including near-cancellation (same exponent, opposite sign)
    a = _finite_bf16(rng, 40000)
    b = _finite_bf16(rng, 40000)
    n = min(len(a), len(b))
    xs.append(a[:n]); rs.append(b[:n])
    near = (a[:n] ^ 0x8000) ^ rng.integers(0, 16, size=n).astype(np.uint16)
    near = np.where(((near >> 7) & 0xff) == 0xff, a[:n], near)
    xs.append(a[:n]); rs.append(near.astype(np.uint16))
    x = np.concatenate(xs); r = np.concatenate(rs)
    H = 8
    pad = (-len(x)) % H
    x = np.concatenate([x, np.zeros(pad, np.uint16)]).reshape(-1, H)
    r = np.concatenate([r, np.zeros(pad, np.uint16)]).reshape(-1, H)
    w = enc([1.0] * H, BF16)
    _, r_out = oracle.fused_add_rmsnorm(x, r, w, 1e-6, BF16)
    want = np.array([int_bf16_add(int(p), int(q)) for p, q in zip(x.ravel(), r.ravel())], dtype=np.uint16)
    assert np.array_equal(r_out.ravel(), want)


@pytest.mark.parametrize("dtype", VALUE_DTYPES)
def test_residual_sum_matches_torch_float_add(dtype):
    """Library pin: torch adds in binary32 and casts once to the storage dtype."""
    inp = wl.rmsnorm_inputs(64, 515, dtype, seed=77)
    _, r_out = oracle.fused_add_rmsnorm(wl.bits(inp.x), wl.bits(inp.residual), wl.bits(inp.weight), 1e-6, dtype)
    want = wl.bits((inp.x.float() + inp.residual.float()).to(TD[dtype]))
    assert np.array_equal(r_out, want)


# ---------------------------------------------------------------------------------------
# fused_add_rmsnorm  (Table 1, Kernel 2)
# ---------------------------------------------------------------------------------------

@pytest.mark.parametrize("dtype", VALUE_DTYPES)
def test_rmsnorm_hand_value_3_4(dtype):
    # x + r = [3, 4] split unevenly between x and r; eps = 0; weights [2, 0.5]
    x = enc([[1.0, 5.0]], dtype); r = enc([[2.0, -1.0]], dtype); w = enc([2.0, 0.5], dtype)
    y, r_out = oracle.fused_add_rmsnorm(x, r, w, 0.0, dtype)
    rms = GOLD["rms_3_4"]
    assert y[0, 0] == pytest.approx(3.0 / rms * 2.0, rel=1e-15)
    assert y[0, 1] == pytest.approx(4.0 / rms * 0.5, rel=1e-15)
    assert np.array_equal(r_out, enc([[3.0, 4.0]], dtype))


@pytest.mark.parametrize("dtype", VALUE_DTYPES)
@pytest.mark.parametrize("c", [0.5, -2.0, 3.0])
def test_rmsnorm_constant_row_closed_form(dtype, c):
    H = 37
    g = torch.Generator().manual_seed(3)
    wt = (1 + 0.1 * torch.randn(H, generator=g, dtype=torch.float64)).to(TD[dtype])
    w = wl.bits(wt)
    x = enc([[c * 0.25] * H], dtype); r = enc([[c * 0.75] * H], dtype)
    eps = 1e-6
    y, _ = oracle.fused_add_rmsnorm(x, r, w, eps, dtype)
    eps_f = float(np.float32(eps))
    want = c / math.sqrt(c * c + eps_f) * wt.to(torch.float64).numpy()
    np.testing.assert_allclose(y[0], want, rtol=1e-14)
    # for eps << c^2 the row normalises to sign(c) * w after rounding to a 16-bit storage type
    if dtype != FP32:
        stored = wl.bits(torch.from_numpy(y[0]).to(TD[dtype]))
        assert np.array_equal(stored, wl.bits((math.copysign(1.0, c) * wt.to(torch.float64)).to(TD[dtype])))


@pytest.mark.parametrize("dtype", VALUE_DTYPES)
def test_rmsnorm_zero_row_is_zero(dtype):
    x = enc([[0.0] * 9, [1.0] * 9], dtype); r = enc([[0.0] * 9, [-1.0] * 9], dtype)
    w = enc([1.5] * 9, dtype)
    y, r_out = oracle.fused_add_rmsnorm(x, r, w, 1e-6, dtype)
    assert np.all(y == 0.0) and np.all(np.isfinite(y))
    assert np.all(r_out == 0)


@pytest.mark.parametrize("dtype", VALUE_DTYPES)
@pytest.mark.parametrize("eps", [1e-6, 1e-5, 0.5])
def test_rmsnorm_mean_square_invariant_and_eps_placement(dtype, eps):
    """mean_j (y_j / w_j)^2 = m / (m + eps): holds only with eps inside the root, added to the mean."""
    inp = wl.rmsnorm_inputs(5, 131, dtype, eps=eps, seed=21)
    y, _ = oracle.fused_add_rmsnorm(wl.bits(inp.x), wl.bits(inp.residual), wl.bits(inp.weight), eps, dtype)
    s = (inp.x.float() + inp.residual.float()).to(torch.float64).numpy()
    w = inp.weight.to(torch.float64).numpy()
    m = (s * s).mean(axis=1)
    lhs = ((y / w) ** 2).mean(axis=1)
    np.testing.assert_allclose(lhs, m / (m + float(np.float32(eps))), rtol=1e-13)


def test_rmsnorm_power_of_two_scaling_invariance():
    inp = wl.rmsnorm_inputs(4, 64, BF16, seed=8)
    y1, _ = oracle.fused_add_rmsnorm(wl.bits(inp.x), wl.bits(inp.residual), wl.bits(inp.weight), 0.0, BF16)
    y2, _ = oracle.fused_add_rmsnorm(wl.bits(inp.x * 8), wl.bits(inp.residual * 8), wl.bits(inp.weight), 0.0, BF16)
    np.testing.assert_allclose(y2, y1, rtol=1e-15)


@pytest.mark.parametrize("dtype", VALUE_DTYPES)
def test_rmsnorm_reduces_to_library_rms_norm(dtype):
    """r = 0, w = 1 is plain RMSNorm; the general case is rms_norm of the binary32 sum."""
    inp = wl.rmsnorm_inputs(7, 200, dtype, eps=1e-5, seed=9)
    zero = torch.zeros_like(inp.residual); one = torch.ones_like(inp.weight)
    y, _ = oracle.fused_add_rmsnorm(wl.bits(inp.x), wl.bits(zero), wl.bits(one), 1e-5, dtype)
    eps_f = float(np.float32(1e-5))
    want = torch.nn.functional.rms_norm(inp.x.to(torch.float64), (200,), eps=eps_f)
    np.testing.assert_allclose(y, want.numpy(), rtol=1e-13)
    y, _ = oracle.fused_add_rmsnorm(wl.bits(inp.x), wl.bits(inp.residual), wl.bits(inp.weight), 1e-5, dtype)
    s = (inp.x.float() + inp.residual.float()).to(torch.float64)
    want = torch.nn.functional.rms_norm(s, (200,), weight=inp.weight.to(torch.float64), eps=eps_f)
    np.testing.assert_allclose(y, want.numpy(), rtol=1e-13)


def test_rmsnorm_norm_uses_binary32_sum_not_stored_residual():
    """1 + 2^-9 is exact in binary32 but rounds to 1 in bf16; the norm must see 1 + 2^-9."""
    s0 = 1.0 + 2.0 ** -9
    x = enc([[1.0, 1.0]], BF16); r = enc([[2.0 ** -9, 0.0]], BF16); w = enc([1.0, 1.0], BF16)
    y, r_out = oracle.fused_add_rmsnorm(x, r, w, 0.0, BF16)
    assert np.array_equal(r_out, enc([[1.0, 1.0]], BF16))
    assert y[0, 0] == pytest.approx(s0 / math.sqrt((s0 * s0 + 1.0) / 2.0), rel=1e-15)
    assert y[0, 1] == pytest.approx(1.0 / math.sqrt((s0 * s0 + 1.0) / 2.0), rel=1e-15)


def test_rmsnorm_rows_are_independent_and_weight_indexed_by_column():
    inp = wl.rmsnorm_inputs(6, 33, BF16, seed=4)
    xb, rb, wb = wl.bits(inp.x), wl.bits(inp.residual), wl.bits(inp.weight)
    y, ro = oracle.fused_add_rmsnorm(xb, rb, wb, 1e-6, BF16)
    for t in (0, 3, 5):
        yt, rt = oracle.fused_add_rmsnorm(xb[t:t + 1], rb[t:t + 1], wb, 1e-6, BF16)
        assert np.array_equal(yt[0], y[t]) and np.array_equal(rt[0], ro[t])
    # permuting columns of x, r and w together permutes y the same way
    perm = np.random.default_rng(0).permutation(33)
    yp, _ = oracle.fused_add_rmsnorm(xb[:, perm], rb[:, perm], wb[perm], 1e-6, BF16)
    np.testing.assert_allclose(yp, y[:, perm], rtol=1e-14)


# ---------------------------------------------------------------------------------------
# fused_allreduce_add_rmsnorm: Kernel 2 on a hidden state given as N partial sums
# ---------------------------------------------------------------------------------------

def _fl32(q):
    """Correctly rounded (nearest-even) binary32 value of an exact rational, as an exact rational:
    integer arithmetic only.  Magnitudes stay inside the normal range of binary32 in these tests."""
    from fractions import Fraction
    if q == 0:
        return Fraction(0)
    sign, a = (-1 if q < 0 else 1), abs(q)
    e = a.numerator.bit_length() - a.denominator.bit_length()
    if Fraction(2) ** e > a:
        e -= 1                                    # now 2^e <= a < 2^(e+1)
    assert -126 <= e <= 127
    quantum = Fraction(2) ** (e - 23)
    n, rem = divmod(a, quantum)                    # a = n * quantum + rem, n a 24-bit integer
    if rem * 2 > quantum or (rem * 2 == quantum and n % 2 == 1):
        n += 1
    return sign * n * quantum


def _rank_order_sum(values, r):
    """fl(...fl(fl(x0 + x1) + x2)... + r) with exact rationals and _fl32."""
    acc = values[0]
    for v in values[1:]:
        acc = _fl32(acc + v)
    return _fl32(acc + r)


@pytest.mark.parametrize("dtype", VALUE_DTYPES)
@pytest.mark.parametrize("n_parts", [1, 2, 3, 5, 8])
def test_allreduce_form_against_exact_rational_adder(dtype, n_parts):
    """Every element: the rank-order binary32 sum rebuilt from exact rationals with an integer-only
    rounding; the residual is that sum cast once by torch; y follows from the sums in fp64.  The inputs
    span many binades, so most additions are inexact and both their order and their number matter."""
    from fractions import Fraction
    T, H = 3, 29
    g = torch.Generator().manual_seed(100 + n_parts)
    span = 6 if dtype == FP16 else 12

    def draw(shape):
        mant = 1 + torch.rand(shape, generator=g, dtype=torch.float64)
        expo = torch.randint(-span, span + 1, shape, generator=g)
        sign = torch.randint(0, 2, shape, generator=g) * 2 - 1
        return (sign * mant * 2.0 ** expo).to(TD[dtype])

    parts = [draw((T, H)) for _ in range(n_parts)]
    r, w = draw((T, H)), draw((H,))
    eps = 1e-5
    y, r_out = oracle.fused_allreduce_add_rmsnorm([wl.bits(p) for p in parts], wl.bits(r), wl.bits(w), eps, dtype)
    s = np.empty((T, H))
    for t in range(T):
        for j in range(H):
            q = _rank_order_sum([Fraction(float(p[t, j])) for p in parts], Fraction(float(r[t, j])))
            s[t, j] = float(q)                     # a binary32 value: exact in a double
    assert np.array_equal(r_out, wl.bits(torch.from_numpy(s).to(torch.float32).to(TD[dtype])))
    denom = np.sqrt((s * s).mean(axis=1, keepdims=True) + float(np.float32(eps)))
    np.testing.assert_allclose(y, s / denom * w.to(torch.float64).numpy(), rtol=1e-13)


@pytest.mark.parametrize("dtype", VALUE_DTYPES)
def test_allreduce_form_with_one_partial_is_fused_add_rmsnorm(dtype):
    inp = wl.rmsnorm_inputs(9, 133, dtype, eps=1e-5, seed=31)
    xb, rb, wb = wl.bits(inp.x), wl.bits(inp.residual), wl.bits(inp.weight)
    y1, r1 = oracle.fused_allreduce_add_rmsnorm([xb], rb, wb, 1e-5, dtype)
    y0, r0 = oracle.fused_add_rmsnorm(xb, rb, wb, 1e-5, dtype)
    assert np.array_equal(y1, y0) and np.array_equal(r1, r0)


@pytest.mark.parametrize("dtype", VALUE_DTYPES)
def test_allreduce_form_equals_kernel_2_on_the_summed_state_when_the_sums_are_exact(dtype):
    """Small integers: every partial sum is exact and fits the storage type, so the N-partial form is
    Kernel 2 applied to x = sum of the partials, in any order of the partials."""
    g = torch.Generator().manual_seed(5)
    parts = [torch.randint(-7, 8, (4, 40), generator=g).to(TD[dtype]) for _ in range(6)]
    r = torch.randint(-7, 8, (4, 40), generator=g).to(TD[dtype])
    w = (1 + 0.1 * torch.randn(40, generator=g)).to(TD[dtype])
    x = sum(p.to(torch.float64) for p in parts).to(TD[dtype])
    y0, r0 = oracle.fused_add_rmsnorm(wl.bits(x), wl.bits(r), wl.bits(w), 1e-6, dtype)
    for order in ([0, 1, 2, 3, 4, 5], [5, 3, 1, 0, 2, 4]):
        y, ro = oracle.fused_allreduce_add_rmsnorm([wl.bits(parts[i]) for i in order], wl.bits(r), wl.bits(w), 1e-6, dtype)
        assert np.array_equal(ro, r0)
        np.testing.assert_allclose(y, y0, rtol=1e-15)


def test_allreduce_form_order_and_roundings():
    """Hand cases whose answer depends on the reading: rank order, the residual last, one rounding
    per addition (not one for the whole sum), and no rounding to the storage type before the residual."""
    def run(parts, r, dtype):
        y, ro = oracle.fused_allreduce_add_rmsnorm([enc([[v]], dtype) for v in parts], enc([[r]], dtype),
                                                   enc([1.0], dtype), 1e-6, dtype)
        return y[0, 0], ro
    big, tiny = 256.0, 2.0 ** -17          # tiny is a quarter of a binary32 ulp of big
    # rank order: (big - big) + tiny = tiny, but (big + tiny) - big = 0
    y, ro = run([big, -big, tiny], 0.0, BF16)
    assert np.array_equal(ro, enc([[tiny]], BF16)) and y > 0.0
    y, ro = run([big, tiny, -big], 0.0, BF16)
    assert np.array_equal(ro, enc([[0.0]], BF16)) and y == 0.0
    # the residual joins last: (big + tiny) + (-big) = 0, whereas (-big + big) + tiny would be tiny
    _, ro = run([big, tiny], -big, BF16)
    assert np.array_equal(ro, enc([[0.0]], BF16))
    _, ro = run([-big, tiny], big, BF16)
    assert np.array_equal(ro, enc([[0.0]], BF16))
    # one rounding per addition: 1 + 2^-24 + 2^-24 stays 1 step by step (ties to even twice);
    # a sum carried in wider precision and rounded once would give 1 + 2^-23
    _, ro = run([1.0, 2.0 ** -24, 2.0 ** -24], 0.0, FP32)
    assert np.array_equal(ro, enc([[1.0]], FP32))
    _, ro = run([2.0 ** -24, 2.0 ** -24, 1.0], 0.0, FP32)
    assert np.array_equal(ro, enc([[1.0 + 2.0 ** -23]], FP32))
    # nothing is rounded to the storage type before the residual joins: 1 + 2^-9 is not a bf16 value
    _, ro = run([1.0, 2.0 ** -9], -1.0, BF16)
    assert np.array_equal(ro, enc([[2.0 ** -9]], BF16))


def test_allreduce_form_norm_uses_the_binary32_sum_and_constant_rows():
    s0 = 1.0 + 2.0 ** -9
    parts = [enc([[0.5, 0.25]], BF16), enc([[0.5, 0.25]], BF16), enc([[2.0 ** -9, 0.25]], BF16)]
    y, ro = oracle.fused_allreduce_add_rmsnorm(parts, enc([[0.0, 0.25]], BF16), enc([1.0, 1.0], BF16), 0.0, BF16)
    assert np.array_equal(ro, enc([[1.0, 1.0]], BF16))
    assert y[0, 0] == pytest.approx(s0 / math.sqrt((s0 * s0 + 1.0) / 2.0), rel=1e-15)
    assert y[0, 1] == pytest.approx(1.0 / math.sqrt((s0 * s0 + 1.0) / 2.0), rel=1e-15)
    # constant row: every partial and the residual constant -> y = sign(c) * w / sqrt(1 + eps / c^2)
    H, eps = 19, 1e-6
    wt = torch.linspace(0.5, 1.5, H, dtype=torch.float64).to(torch.float16)
    for c_parts, c_r in (([0.5, 0.25, 1.0], 0.25), ([-1.0, -0.5], -0.5)):
        c = sum(c_parts) + c_r
        y, _ = oracle.fused_allreduce_add_rmsnorm([enc([[v] * H], FP16) for v in c_parts], enc([[c_r] * H], FP16),
                                                  wl.bits(wt), eps, FP16)
        want = c / math.sqrt(c * c + float(np.float32(eps))) * wt.to(torch.float64).numpy()
        np.testing.assert_allclose(y[0], want, rtol=1e-14)


# ---------------------------------------------------------------------------------------
# silu_and_mul  (Table 1, Kernel 3)
# ---------------------------------------------------------------------------------------

@pytest.mark.parametrize("dtype", VALUE_DTYPES)
def test_silu_hand_values_and_layout(dtype):
    # row = [gate | up]; D = 3
    row = enc([[1.0, -1.0, 2.0, 1.0, 1.0, 1.0]], dtype)
    out = oracle.silu_and_mul(row, dtype)
    assert out[0, 0] == pytest.approx(GOLD["sigmoid_1"], rel=1e-15)
    assert out[0, 1] == pytest.approx(-GOLD["sigmoid_minus_1"], rel=1e-15)
    assert out[0, 2] == pytest.approx(GOLD["silu_2"], rel=1e-15)
    # SiLU goes on the first half: [gate 2 | up 1] -> silu(2), not silu(1) * 2
    out = oracle.silu_and_mul(enc([[2.0, 1.0]], dtype), dtype)
    assert out[0, 0] == pytest.approx(GOLD["silu_2"], rel=1e-15)
    out = oracle.silu_and_mul(enc([[1.0, 2.0]], dtype), dtype)
    assert out[0, 0] == pytest.approx(2 * GOLD["sigmoid_1"], rel=1e-15)


@pytest.mark.parametrize("dtype", VALUE_DTYPES)
def test_silu_zero_odd_part_and_limits(dtype):
    a = [0.0, -0.0, 0.37, 1.5, 7.25, 30.0, 60.0]
    D = len(a)
    pos = oracle.silu_and_mul(enc([a + [1.0] * D], dtype), dtype)[0]
    neg = oracle.silu_and_mul(enc([[-v for v in a] + [1.0] * D], dtype), dtype)[0]
    av = dec(enc(a, dtype), dtype)
    assert pos[0] == 0.0 and pos[1] == 0.0
    # silu(a) - silu(-a) = a
    np.testing.assert_allclose(pos - neg, av, rtol=1e-14, atol=1e-300)
    # a >> 0: silu(a) -> a ; a << 0: silu(a) -> 0 from below
    assert pos[-1] == pytest.approx(60.0, rel=1e-15)
    assert -1e-20 < neg[-1] < 0.0
    # times zero / times minus one
    out = oracle.silu_and_mul(enc([a + [0.0] * D], dtype), dtype)[0]
    assert np.all(out == 0.0)
    out = oracle.silu_and_mul(enc([a + [-1.0] * D], dtype), dtype)[0]
    np.testing.assert_allclose(out, -pos, rtol=0, atol=0)


@pytest.mark.parametrize("dtype", VALUE_DTYPES)
def test_silu_matches_library_silu(dtype):
    inp = wl.silu_inputs(9, 77, dtype, std=2.0, seed=5)
    out = oracle.silu_and_mul(wl.bits(inp.input), dtype)
    x = inp.input.to(torch.float64)
    want = torch.nn.functional.silu(x[:, :77]) * x[:, 77:]
    np.testing.assert_allclose(out, want.numpy(), rtol=1e-14, atol=1e-300)


def test_silu_total_for_huge_negative_gate():
    out = oracle.silu_and_mul(enc([[-3e38, -1000.0, 1.0, 1.0]], BF16), BF16)[0]
    assert out[0] == 0.0 and np.signbit(out[0])
    assert out[1] <= 0.0 and out[1] > -1e-300


# ---------------------------------------------------------------------------------------
# merge_attn_states_lse  (Table 1, Kernel 1)
# ---------------------------------------------------------------------------------------

def _merge(va, sa, vb, sb, dtype=BF16):
    va = np.asarray(va, dtype=np.float64); vb = np.asarray(vb, dtype=np.float64)
    T, Hh, D = va.shape
    v, s = oracle.merge_attn_states_lse(
        enc(va.tolist(), dtype), np.asarray(sa, dtype=np.float32).reshape(T, Hh),
        enc(vb.tolist(), dtype), np.asarray(sb, dtype=np.float32).reshape(T, Hh), dtype)
    return v, s


@pytest.mark.parametrize("dtype", VALUE_DTYPES)
def test_merge_equal_scores_give_mean_and_ln2(dtype):
    va = [[[1.0, -2.0, 0.5, 3.0]]]; vb = [[[3.0, 2.0, 0.25, -3.0]]]
    for s in (0.0, 7.5, -40.0, 80.0):
        v, so = _merge(va, [[s]], vb, [[s]], dtype)
        np.testing.assert_allclose(v[0, 0], [2.0, 0.0, 0.375, 0.0], rtol=0, atol=0)
        assert so[0, 0] == pytest.approx(s + GOLD["ln_2"], abs=1e-14)


def test_merge_hand_weight_three_quarters():
    # Sa - Sb = ln 3 -> weights 3/4 and 1/4 (Sa rounded to binary32: compare at 1e-7)
    sa = np.float32(math.log(3.0))
    v, so = _merge([[[4.0]]], [[sa]], [[[0.0]]], [[0.0]])
    assert v[0, 0, 0] == pytest.approx(4.0 * GOLD["merge_w_ln3"], rel=2e-7)
    assert so[0, 0] == pytest.approx(math.log(4.0), rel=2e-7)


@pytest.mark.parametrize("dtype", VALUE_DTYPES)
def test_merge_neg_inf_returns_other_state(dtype):
    ninf = float("-inf")
    va = [[[1.5, -2.0, 0.0, 7.0]]]; vb = [[[9.0, 9.0, -9.0, 1.0]]]
    v, s = _merge(va, [[3.25]], vb, [[ninf]], dtype)
    assert np.array_equal(v[0, 0], np.array(va[0][0])) and s[0, 0] == 3.25
    v, s = _merge(va, [[ninf]], vb, [[-11.0]], dtype)
    assert np.array_equal(v[0, 0], np.array(vb[0][0])) and s[0, 0] == -11.0
    # both empty: zero output, -inf score
    v, s = _merge(va, [[ninf]], vb, [[ninf]], dtype)
    assert np.all(v == 0.0) and s[0, 0] == ninf
    # a non-finite payload on the zero-weight side does not leak
    v, s = _merge([[[float("inf"), float("nan"), 1.0, 1.0]]], [[ninf]], vb, [[0.5]], dtype)
    assert np.array_equal(v[0, 0], np.array(vb[0][0])) and s[0, 0] == 0.5
    v, s = _merge(va, [[-2.5]], [[[float("nan"), float("-inf"), 1.0, 1.0]]], [[ninf]], dtype)
    assert np.array_equal(v[0, 0], np.array(va[0][0])) and s[0, 0] == -2.5


def test_merge_out_of_domain_scores_give_nan():
    v, s = _merge([[[1.0]]], [[float("inf")]], [[[2.0]]], [[0.0]])
    assert np.isnan(v).all() and np.isnan(s).all()
    v, s = _merge([[[1.0]]], [[float("nan")]], [[[2.0]]], [[0.0]])
    assert np.isnan(v).all() and np.isnan(s).all()


@pytest.mark.parametrize("dtype", VALUE_DTYPES)
def test_merge_symmetry_shift_and_bounds(dtype):
    inp = wl.merge_inputs(11, 3, 20, dtype, seed=13, neg_inf_frac=0.0, forced_both_neg_inf=0)
    va, vb = wl.bits(inp.v_a), wl.bits(inp.v_b)
    # scores on a 2^-10 grid so that shifting by 4 is exact in binary32
    sa = (torch.round(inp.lse_a * 1024) / 1024).numpy(); sb = (torch.round(inp.lse_b * 1024) / 1024).numpy()
    v, s = oracle.merge_attn_states_lse(va, sa, vb, sb, dtype)
    v2, s2 = oracle.merge_attn_states_lse(vb, sb, va, sa, dtype)
    np.testing.assert_allclose(v2, v, rtol=1e-15, atol=1e-300); np.testing.assert_allclose(s2, s, rtol=1e-15)
    v3, s3 = oracle.merge_attn_states_lse(va, sa + np.float32(4), vb, sb + np.float32(4), dtype)
    np.testing.assert_allclose(v3, v, rtol=1e-14, atol=1e-300); np.testing.assert_allclose(s3, s + 4.0, rtol=0, atol=1e-13)
    a = dec(va, dtype); b = dec(vb, dtype)
    assert np.all(v >= np.minimum(a, b) - 1e-15) and np.all(v <= np.maximum(a, b) + 1e-15)
    m = np.maximum(sa, sb).astype(np.float64)
    assert np.all(s >= m) and np.all(s <= m + GOLD["ln_2"] + 1e-15)


@pytest.mark.parametrize("dtype", VALUE_DTYPES)
def test_merge_matches_library_softmax_and_logaddexp(dtype):
    inp = wl.merge_inputs(9, 5, 24, dtype, seed=31)
    v, s = oracle.merge_attn_states_lse(wl.bits(inp.v_a), inp.lse_a.numpy(), wl.bits(inp.v_b),
                                        inp.lse_b.numpy(), dtype)
    sa = inp.lse_a.to(torch.float64); sb = inp.lse_b.to(torch.float64)
    both = torch.isinf(sa) & torch.isinf(sb)
    assert both.any()  # the generator forces some
    w = torch.softmax(torch.stack([sa, sb], dim=-1), dim=-1)  # NaN where both are -inf
    want_v = w[..., 0:1] * inp.v_a.to(torch.float64) + w[..., 1:2] * inp.v_b.to(torch.float64)
    want_s = torch.logaddexp(sa, sb)
    ok = ~both
    np.testing.assert_allclose(v[ok.numpy()], want_v[ok].numpy(), rtol=1e-13, atol=1e-300)
    np.testing.assert_allclose(s[ok.numpy()], want_s[ok].numpy(), rtol=1e-14)
    assert np.all(v[both.numpy()] == 0.0) and np.all(s[both.numpy()] == -np.inf)


def test_merge_equals_attention_over_the_union_of_two_key_sets():
    """The defining property: merging the partial attention results of two disjoint key sets,
    each summarised by (output, log-sum-exp of its logits), gives attention over all keys.
    Keys within a set share a logit, and values are multiples of the set size, so each partial
    output is exactly representable in bf16; the only inexact input is the binary32 score."""
    rng = np.random.default_rng(2)
    D = 4
    for na, nb, la, lb in [(4, 8, 1.25, -0.5), (2, 4, -3.0, 2.0), (8, 2, 0.0, 0.0)]:
        Va = rng.integers(-6, 7, size=(na, D)) * na / 4.0
        Vb = rng.integers(-6, 7, size=(nb, D)) * nb / 4.0
        logits = np.array([la] * na + [lb] * nb)
        p = np.exp(logits - logits.max()); p /= p.sum()
        full = p @ np.concatenate([Va, Vb])
        full_lse = logits.max() + math.log(np.exp(logits - logits.max()).sum())
        oa, ob = Va.mean(axis=0), Vb.mean(axis=0)
        sa = np.float32(la + math.log(na)); sb = np.float32(lb + math.log(nb))
        v, s = _merge([[oa.tolist()]], [[sa]], [[ob.tolist()]], [[sb]])
        np.testing.assert_allclose(v[0, 0], full, rtol=1e-6, atol=1e-6)
        assert s[0, 0] == pytest.approx(full_lse, abs=1e-6)


def test_merge_equals_attention_general_logits():
    """Same property with arbitrary logits; partial outputs are rounded to fp16, so 2e-3."""
    rng = np.random.default_rng(3)
    D = 4
    q = rng.normal(size=D); K = rng.normal(size=(8, D)); V = rng.normal(size=(8, D))
    logits = K @ q
    def part(idx):
        l = logits[idx]; m = l.max(); e = np.exp(l - m)
        return (e / e.sum()) @ V[idx], m + math.log(e.sum())
    oa, sa = part(np.arange(0, 3)); ob, sb = part(np.arange(3, 8))
    full, full_lse = part(np.arange(0, 8))
    v, s = _merge([[oa.tolist()]], [[np.float32(sa)]], [[ob.tolist()]], [[np.float32(sb)]], FP16)
    np.testing.assert_allclose(v[0, 0], full, atol=2e-3)
    assert s[0, 0] == pytest.approx(full_lse, abs=1e-6)


# ---------------------------------------------------------------------------------------
# arbitrary-precision brute force on tiny shapes
# ---------------------------------------------------------------------------------------

def _D(v):
    return decimal.Decimal(float(v))


@pytest.mark.parametrize("dtype", VALUE_DTYPES)
def test_tiny_shapes_against_50_digit_arithmetic(dtype):
    decimal.getcontext().prec = 50
    for T in (1, 2, 3):
        for H in (1, 7, 8, 9, 33):
            inp = wl.rmsnorm_inputs(T, H, dtype, eps=1e-5, seed=100 + T * 40 + H)
            y, _ = oracle.fused_add_rmsnorm(wl.bits(inp.x), wl.bits(inp.residual), wl.bits(inp.weight), 1e-5, dtype)
            s = (inp.x.float() + inp.residual.float()).to(torch.float64).numpy()
            w = inp.weight.to(torch.float64).numpy()
            eps = _D(np.float32(1e-5))
            for t in range(T):
                msq = sum(_D(v) * _D(v) for v in s[t]) / decimal.Decimal(H)
                den = (msq + eps).sqrt()
                for j in range(H):
                    want = _D(s[t, j]) / den * _D(w[j])
                    assert float(want) == pytest.approx(y[t, j], rel=1e-14, abs=1e-300)
        for Dm in (1, 7, 8, 9):
            inp = wl.silu_inputs(T, Dm, dtype, std=2.0, seed=300 + T * 10 + Dm)
            out = oracle.silu_and_mul(wl.bits(inp.input), dtype)
            xin = inp.input.to(torch.float64).numpy()
            for t in range(T):
                for i in range(Dm):
                    a, b = _D(xin[t, i]), _D(xin[t, Dm + i])
                    want = a / (1 + (-a).exp()) * b
                    assert float(want) == pytest.approx(out[t, i], rel=1e-14, abs=1e-300)
            for Hh in (1, 3):
                inp = wl.merge_inputs(T, Hh, Dm, dtype, seed=500 + T * 100 + Hh * 10 + Dm, neg_inf_frac=0.0,
                                      forced_both_neg_inf=0)
                v, s = oracle.merge_attn_states_lse(wl.bits(inp.v_a), inp.lse_a.numpy(), wl.bits(inp.v_b),
                                                    inp.lse_b.numpy(), dtype)
                a64 = inp.v_a.to(torch.float64).numpy(); b64 = inp.v_b.to(torch.float64).numpy()
                for t in range(T):
                    for h in range(Hh):
                        ea = _D(inp.lse_a[t, h].item()).exp(); eb = _D(inp.lse_b[t, h].item()).exp()
                        assert float((ea + eb).ln()) == pytest.approx(s[t, h], rel=1e-14, abs=1e-14)
                        for d in range(Dm):
                            want = (ea * _D(a64[t, h, d]) + eb * _D(b64[t, h, d])) / (ea + eb)
                            assert float(want) == pytest.approx(v[t, h, d], rel=1e-13, abs=1e-15)


def test_threads_do_not_change_the_allreduce_form():
    g = torch.Generator().manual_seed(8)
    parts = [wl.bits(torch.randn((37, 65), generator=g).to(torch.bfloat16)) for _ in range(4)]
    inp = wl.rmsnorm_inputs(37, 65, BF16, seed=2)
    a = oracle.fused_allreduce_add_rmsnorm(parts, wl.bits(inp.residual), wl.bits(inp.weight), 1e-5, BF16, nthreads=1)
    b = oracle.fused_allreduce_add_rmsnorm(parts, wl.bits(inp.residual), wl.bits(inp.weight), 1e-5, BF16, nthreads=4)
    assert np.array_equal(a[0], b[0]) and np.array_equal(a[1], b[1])


def test_threads_do_not_change_results():
    inp = wl.rmsnorm_inputs(64, 300, BF16, seed=1)
    a = oracle.fused_add_rmsnorm(wl.bits(inp.x), wl.bits(inp.residual), wl.bits(inp.weight), 1e-6, BF16, nthreads=1)
    b = oracle.fused_add_rmsnorm(wl.bits(inp.x), wl.bits(inp.residual), wl.bits(inp.weight), 1e-6, BF16, nthreads=4)
    assert np.array_equal(a[0], b[0]) and np.array_equal(a[1], b[1])

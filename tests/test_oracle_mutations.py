"""Do the pins bite?  Each case plants one plausible mistake in a COPY of the oracle's C source
(a dropped term, a wrong sign, a swapped operand, a misplaced epsilon, ...), builds it on the CPU,
swaps it in for the real oracle, and requires that at least one pin in test_oracle_pins.py fails.
A mistake that no pin catches would mean the oracle is not pinned against it."""
import ctypes
import inspect
import os

import pytest

import oracle
import test_oracle_pins as pins

SRC = os.path.join(os.path.dirname(os.path.abspath(oracle.__file__)), "astra_oracle.c")

# (name, text in the oracle source, replacement)
MUTATIONS = [
    ("rmsnorm: eps added outside the root",
     "sqrt(sum_sq / (double)H + (double)eps)", "(sqrt(sum_sq / (double)H) + (double)eps)"),
    ("rmsnorm: sum of squares instead of mean",
     "sqrt(sum_sq / (double)H + (double)eps)", "sqrt(sum_sq + (double)eps)"),
    ("rmsnorm: eps dropped",
     "sqrt(sum_sq / (double)H + (double)eps)", "sqrt(sum_sq / (double)H)"),
    ("rmsnorm: weight indexed from the other end",
     "/ denom * load_value(w, j, dtype, f)", "/ denom * load_value(w, H - 1 - j, dtype, f)"),
    ("rmsnorm: weight dropped",
     "/ denom * load_value(w, j, dtype, f)", "/ denom"),
    ("rmsnorm: norm taken from the stored residual instead of the binary32 sum",
     "double s = (double)add_binary32(xv, rv, dtype);",
     "double s = widen(round_to_storage((double)add_binary32(xv, rv, dtype), f), f);"),
    ("rmsnorm: x - r instead of x + r (both loops)",
     "return (float)(a + b);", "return (float)(a - b);"),
    ("rmsnorm: residual gets x only",
     "float s32 = add_binary32(xv, rv, dtype);", "float s32 = (float)xv;"),
    ("rmsnorm: divides by the mean square instead of its root",
     "double denom = sqrt(", "double denom = ("),
    ("allreduce form: the residual is not added",
     "    acc = acc + res;\n", "    acc = acc + 0.0f * res;\n"),
    ("allreduce form: the last partial is skipped",
     "for (int p = 1; p < n_parts; ++p) {", "for (int p = 1; p < n_parts - 1; ++p) {"),
    ("allreduce form: partials added from the last rank down",
     "volatile float acc = value_as_float(parts[0], i, dtype, f);\n    for (int p = 1; p < n_parts; ++p) {\n"
     "        volatile float next = value_as_float(parts[p], i, dtype, f);",
     "volatile float acc = value_as_float(parts[n_parts - 1], i, dtype, f);\n    for (int p = 1; p < n_parts; ++p) {\n"
     "        volatile float next = value_as_float(parts[n_parts - 1 - p], i, dtype, f);"),
    ("allreduce form: the residual is added first",
     "volatile float acc = value_as_float(parts[0], i, dtype, f);\n    for (int p = 1; p < n_parts; ++p) {\n"
     "        volatile float next = value_as_float(parts[p], i, dtype, f);",
     "volatile float acc = value_as_float(r, i, dtype, f) + value_as_float(parts[0], i, dtype, f);\n"
     "    r = parts[0];\n    for (int p = 1; p <= n_parts; ++p) {\n"
     "        volatile float next = p < n_parts ? value_as_float(parts[p], i, dtype, f) : 0.0f;"),
    ("allreduce form: the sum is carried in double and rounded once",
     "volatile float acc = value_as_float(parts[0], i, dtype, f);", "volatile double acc = value_as_float(parts[0], i, dtype, f);"),
    ("allreduce form: the summed state is rounded to the storage type before the residual joins",
     "    volatile float res = value_as_float(r, i, dtype, f);",
     "    if (dtype != ORACLE_FP32) acc = (float)widen(round_to_storage((double)acc, f), f);\n"
     "    volatile float res = value_as_float(r, i, dtype, f);"),
    ("allreduce form: norm taken from the stored residual",
     "double s = (double)sum_in_rank_order(parts, n_parts, r, t * H + j, dtype, f);",
     "double s = dtype == ORACLE_FP32 ? 0.0 : widen(round_to_storage((double)sum_in_rank_order(parts, n_parts, r, t * H + j, dtype, f), f), f);"),
    ("allreduce form: every element reads the first row of the partials",
     "(double)sum_in_rank_order(parts, n_parts, r, t * H + j, dtype, f);\n            sum_sq",
     "(double)sum_in_rank_order(parts, n_parts, r, j, dtype, f);\n            sum_sq"),
    ("silu: e^{+z} in the denominator",
     "return z / (1.0 + exp(-z));", "return z / (1.0 + exp(z));"),
    ("silu: sigmoid instead of SiLU (z dropped)",
     "return z / (1.0 + exp(-z));", "return 1.0 / (1.0 + exp(-z));"),
    ("silu: gate and up halves swapped",
     "double a = load_value(input, row + i, dtype, f);\n            double b = load_value(input, row + D + i, dtype, f);",
     "double a = load_value(input, row + D + i, dtype, f);\n            double b = load_value(input, row + i, dtype, f);"),
    ("silu: multiplication by b dropped",
     "out[t * D + i] = silu(a) * b;", "out[t * D + i] = silu(a);"),
    ("silu: row pitch D instead of 2D",
     "const int64_t row = t * 2 * D;", "const int64_t row = t * D;"),
    ("merge: weights applied to the wrong states",
     "if (wa != 0.0) num += wa * load_value(v_a, base + d, dtype, f);\n            if (wb != 0.0) num += wb * load_value(v_b, base + d, dtype, f);",
     "if (wa != 0.0) num += wa * load_value(v_b, base + d, dtype, f);\n            if (wb != 0.0) num += wb * load_value(v_a, base + d, dtype, f);"),
    ("merge: normalisation dropped",
     "vo[d] = num / denom;", "vo[d] = num;"),
    ("merge: max dropped from the merged score",
     "lse_out[th] = m + log(denom);", "lse_out[th] = log(denom);"),
    ("merge: score is log of the max weight only",
     "lse_out[th] = m + log(denom);", "lse_out[th] = m;"),
    ("merge: difference of scores with the wrong sign",
     "double wa = exp(sa - m);", "double wa = exp(m - sa);"),
    ("merge: both-empty case not handled",
     "if (sa == -INFINITY && sb == -INFINITY) {", "if (0) {"),
    ("merge: zero-weight side multiplied instead of skipped",
     "if (wb != 0.0) num += wb * load_value(v_b, base + d, dtype, f);", "num += wb * load_value(v_b, base + d, dtype, f);"),
    ("merge: scores indexed per token instead of per (token, head)",
     "double sb = (double)lse_b[th];", "double sb = (double)lse_b[th / Hh];"),
    ("storage: fp16 exponent bias off by one",
     "f.frac_bits = 10; f.exp_bits = 5; f.bias = 15;", "f.frac_bits = 10; f.exp_bits = 5; f.bias = 16;"),
    ("storage: fp32 elements read at a 2-byte pitch",
     "memcpy(&v, (const unsigned char *)base + 4 * i, 4);", "memcpy(&v, (const unsigned char *)base + 2 * i, 4);"),
    ("storage: fp32 addition carried out in double and rounded afterwards twice (to bf16 precision)",
     "volatile float s = fa + fb;", "volatile float s = (float)widen(round_to_storage((double)(fa + fb), format_of(0)), format_of(0));"),
    ("storage: bf16 read with 8 fraction bits",
     "f.frac_bits = 7;  f.exp_bits = 8; f.bias = 127;", "f.frac_bits = 8;  f.exp_bits = 8; f.bias = 127;"),
    ("storage: truncation instead of round-to-nearest-even",
     "double q = nearbyint(a / quantum);", "double q = floor(a / quantum);"),
    ("storage: round half away from zero",
     "double q = nearbyint(a / quantum);", "double q = floor(a / quantum + 0.5);"),
    ("storage: subnormals flushed on widening",
     "v = ldexp((double)frac, 1 - f.bias - f.frac_bits);", "v = 0.0;"),
]

PIN_TESTS = [(name, fn) for name, fn in inspect.getmembers(pins, inspect.isfunction) if name.startswith("test_")]


def run_all_pins():
    """Calls every pin with every parameter combination; returns the names of those that failed."""
    failed = []
    for name, fn in PIN_TESTS:
        marks = [m for m in getattr(fn, "pytestmark", []) if m.name == "parametrize"]
        combos = [{}]
        for m in marks:
            argnames = [a.strip() for a in m.args[0].split(",")]
            new = []
            for c in combos:
                for vals in m.args[1]:
                    vals = vals if isinstance(vals, (tuple, list)) and len(argnames) > 1 else (vals,)
                    d = dict(c); d.update(dict(zip(argnames, vals)))
                    new.append(d)
            combos = new
        for kw in combos:
            try:
                fn(**kw)
            except Exception:  # an assertion, or an arithmetic error caused by the planted mistake
                failed.append(name)
                break
    return failed


def test_unmodified_oracle_passes_when_driven_this_way():
    assert run_all_pins() == []


@pytest.mark.parametrize("name,old,new", MUTATIONS, ids=[m[0] for m in MUTATIONS])
def test_planted_mistake_is_caught(name, old, new, tmp_path, monkeypatch):
    text = open(SRC).read()
    assert text.count(old) >= 1, f"mutation target not found in the oracle source: {old!r}"
    src = tmp_path / "mutated.c"
    src.write_text(text.replace(old, new))
    lib = oracle.declare(ctypes.CDLL(oracle.compile_source(str(src), str(tmp_path / "libmutated.so"))))
    monkeypatch.setattr(oracle, "_lib", lib)
    failed = run_all_pins()
    assert failed, f"no pin noticed: {name}"

"""CPU checks of the tolerance helpers used by the GPU parity tests."""
import numpy as np
import pytest
import torch

from parity import BF16, FP16, check_lse, check_values, ulp


def test_ulp_matches_spacing_of_torch_types():
    for dtype, td in ((BF16, torch.bfloat16), (FP16, torch.float16)):
        pats = np.arange(1, 0x7bff if dtype == FP16 else 0x7f7f, 13, dtype=np.int16)
        a = torch.from_numpy(pats).view(td).to(torch.float64).numpy()
        b = torch.from_numpy((pats + 1).astype(np.int16)).view(td).to(torch.float64).numpy()
        assert np.array_equal(ulp(a, dtype), b - a)
        # values inside a binade share its spacing
        assert np.array_equal(ulp(a + (b - a) / 3, dtype), b - a)


def test_check_values_gate():
    o = np.array([1.0, -3.0, 0.0, 100.0])
    check_values(o + np.array([2 ** -6, 2 ** -5, 0.0, 1.0]), o, BF16)
    with pytest.raises(AssertionError):
        check_values(o + np.array([2 ** -6 * 1.01, 0, 0, 0]), o, BF16)
    with pytest.raises(AssertionError):
        check_values(o + np.array([0, 0, 1e-30, 0]), o, BF16)
    check_values(o + np.array([1e-3, 1e-3, 0, 0.125]), o, FP16)
    with pytest.raises(AssertionError):  # 2 ulp at 0.25 is 4.9e-4, so the 1e-3 floor is the gate there
        check_values(np.array([0.25 + 1.1e-3]), np.array([0.25]), FP16)
    with pytest.raises(AssertionError):  # 2 ulp at 100 is 0.125
        check_values(np.array([100.13]), np.array([100.0]), FP16)
    # cancellation floor
    check_values(np.array([1e-9]), np.array([1e-12]), BF16, extra=np.array([2.0 ** -22 * 2.0]))


def test_check_lse_gate():
    o = np.array([1.0, -np.inf, 20.0])
    check_lse(o + np.array([9e-6, 0, -9e-6]), o)
    with pytest.raises(AssertionError):
        check_lse(o + np.array([2e-5, 0, 0]), o)
    with pytest.raises(AssertionError):
        check_lse(np.array([1.0, -1e30, 20.0]), o)

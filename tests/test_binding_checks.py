"""CPU checks of what the Python binding validates before it hands bare addresses to the C side.
The tensors are stand-ins (``MagicMock(spec=torch.Tensor)``): every case must be refused before
the library is called, so no device is needed and nothing is launched."""
from unittest import mock

import pytest
import torch

from paper_2509_07506_b200 import binding


def fake(shape, dtype=torch.bfloat16, device=0, contiguous=True, strides=None):
    t = mock.MagicMock(spec=torch.Tensor)
    t.is_cuda = True
    t.device = torch.device("cuda", device)
    t.dtype = dtype
    t.shape = torch.Size(shape)
    t.dim.return_value = len(shape)
    t.is_contiguous.return_value = contiguous
    if strides is None:
        strides, acc = [], 1
        for n in reversed(shape):
            strides.insert(0, acc)
            acc *= n
    t.stride.side_effect = lambda i=None: tuple(strides) if i is None else strides[i]
    t.data_ptr.side_effect = AssertionError("the address must not be read: the call should have been refused")
    return t


@pytest.fixture(autouse=True)
def _no_library(monkeypatch):
    def boom():
        raise AssertionError("the library must not be reached")
    monkeypatch.setattr(binding, "load_library", boom)


def test_operands_on_different_gpus_are_refused():
    x, r, w = fake((4, 64)), fake((4, 64), device=1), fake((64,))
    with pytest.raises(ValueError, match="cuda:1"):
        binding.astra_fused_add_rmsnorm(x, r, w, 1e-6)
    with pytest.raises(ValueError, match="cuda:1"):
        binding.astra_fused_add_rmsnorm(x, fake((4, 64)), fake((64,), device=1), 1e-6)
    with pytest.raises(ValueError, match="cuda:1"):
        binding.astra_silu_and_mul(fake((4, 32), device=1), fake((4, 64)))
    va, sa = fake((2, 3, 8)), fake((2, 3), torch.float32)
    with pytest.raises(ValueError, match="cuda:1"):
        binding.astra_merge_attn_states_lse(fake((2, 3, 8)), fake((2, 3), torch.float32), va, sa,
                                            fake((2, 3, 8)), fake((2, 3), torch.float32, device=1))
    with pytest.raises(ValueError, match="cuda:1"):
        binding.astra_merge_attn_states_lse(fake((2, 3, 8)), fake((2, 3), torch.float32, device=1), va, sa,
                                            fake((2, 3, 8)), fake((2, 3), torch.float32))


def test_operands_on_different_gpus_are_refused_by_the_strided_forms():
    x = fake((4, 64))
    with pytest.raises(ValueError, match="cuda:1"):
        binding.astra_fused_add_rmsnorm_ex(fake((4, 64), device=1), fake((4, 64)), x, fake((4, 64)), fake((64,)), 1e-6)
    with pytest.raises(ValueError, match="cuda:1"):
        binding.astra_silu_and_mul_ex(fake((4, 64)), x, fake((4, 64), device=1))
    va, sa = fake((2, 3, 8)), fake((2, 3), torch.float32)
    with pytest.raises(ValueError, match="cuda:1"):
        binding.astra_merge_attn_states_lse_ex(fake((2, 3, 8)), None, va, sa, fake((2, 3, 8)),
                                               fake((2, 3), torch.float32, device=1))
    with pytest.raises(ValueError, match="cuda:1"):
        binding.astra_merge_attn_states_lse_ex(fake((2, 3, 8), device=1), None, va, sa, fake((2, 3, 8)),
                                               fake((2, 3), torch.float32))


def test_partials_on_different_gpus_are_accepted_only_as_partials():
    """The partial hidden states of the all-reduce form are the one operand that may live on other
    GPUs (that is its purpose); the outputs, the residual and the weight may not."""
    parts = [fake((4, 64), device=0), fake((4, 64), device=1)]
    with pytest.raises(ValueError, match="cuda:1"):
        binding.astra_fused_allreduce_add_rmsnorm(fake((4, 64)), fake((4, 64), device=1), parts, fake((64,)), 1e-6)
    with pytest.raises(ValueError, match="cuda:1"):
        binding.astra_fused_allreduce_add_rmsnorm(fake((4, 64)), fake((4, 64)), parts, fake((64,), device=1), 1e-6)
    with pytest.raises(ValueError):
        binding.astra_fused_allreduce_add_rmsnorm(fake((4, 64)), fake((4, 64)), [], fake((64,)), 1e-6)
    with pytest.raises(ValueError):
        binding.astra_fused_allreduce_add_rmsnorm(fake((4, 64)), fake((4, 64)), [fake((4, 32))], fake((64,)), 1e-6)


def test_wrong_dtype_shape_and_layout_are_refused():
    with pytest.raises(TypeError):
        binding.astra_fused_add_rmsnorm(fake((4, 64), torch.int32), fake((4, 64)), fake((64,)), 1e-6)
    with pytest.raises(TypeError):
        binding.astra_fused_add_rmsnorm(fake((4, 64)), fake((4, 64), torch.float16), fake((64,)), 1e-6)
    with pytest.raises(ValueError):
        binding.astra_fused_add_rmsnorm(fake((4, 64)), fake((4, 64)), fake((32,)), 1e-6)
    with pytest.raises(ValueError):
        binding.astra_fused_add_rmsnorm(fake((4, 64), contiguous=False), fake((4, 64)), fake((64,)), 1e-6)
    with pytest.raises(ValueError):
        binding.astra_silu_and_mul(fake((4, 32)), fake((4, 63)))
    with pytest.raises(ValueError):
        binding.astra_silu_and_mul_ex(fake((4, 32)), fake((4, 32), strides=[64, 2]), fake((4, 32)))
    cpu = mock.MagicMock(spec=torch.Tensor)
    cpu.is_cuda = False
    with pytest.raises(TypeError):
        binding.astra_silu_and_mul(fake((4, 32)), cpu)

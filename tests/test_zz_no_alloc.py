"""The allocation-free moments entry point against the regular one and the CPU oracle.

sb_calib_moments_noalloc serves callers that cannot allocate device memory at the time
they need the moments (all device memory handed out at start-up, code under a caching
allocator, latency-critical loops): its scratch is a fixed array inside the library.
This file is collected last, so a failure here cannot hide another test's result; the test
passes alone in a fresh process and after the rest of the suite.
"""
import numpy as np
import pytest
import torch

from oracle import sbo
from paper_2602_17698_b200 import synth

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def test_noalloc_matches_regular_entry_point_twice_in_a_row():
    from paper_2602_17698_b200 import binding
    torch.cuda.set_device(0)
    ctx = binding.Context()
    # two calls in a row, the second on a different and smaller shape: it reuses the scratch
    # that still holds the first call's partial sums
    X1 = synth.make_activations(5000, 2048, 41, DEV)
    X2 = synth.make_activations(777, 264, 42, DEV)
    ref1 = ctx.calib_moments(X1)
    ref2 = ctx.calib_moments(X2)
    got1 = binding.calib_moments_noalloc(X1)
    got2 = binding.calib_moments_noalloc(X2)
    # accumulate on top of the first result, through a strided view (ldx > K)
    acc = got1[256:1280].clone()
    binding.calib_moments_noalloc(X1[:, 256:1280], acc, accumulate=True)
    ctx.sync()
    torch.cuda.synchronize()
    # same arithmetic in the same order: the tolerance of the moments tests (1e-5 relative)
    assert torch.allclose(got1, ref1, rtol=1e-5, atol=0)
    assert torch.allclose(got2, ref2, rtol=1e-5, atol=0)
    assert torch.allclose(acc, 2 * ref1[256:1280], rtol=1e-5, atol=0)
    # and against the fp64 oracle, not only against the other CUDA entry point
    for X, got in ((X1, got1), (X2, got2)):
        want = sbo.calib_moments(X.cpu(), 1.0 / X.shape[0])
        assert np.allclose(got.cpu().double().numpy(), want, rtol=1e-5, atol=0)
    ctx.close()


def test_noalloc_call_leaves_device_memory_as_it_found_it():
    """The property the entry point exists for: once the first call on the device has looked up
    the scratch address, a call with a caller-supplied output takes no device memory, neither
    from the driver nor from torch's pool."""
    from paper_2602_17698_b200 import binding
    torch.cuda.set_device(0)
    X = synth.make_activations(3000, 1024, 43, DEV)
    out = torch.empty(1024, dtype=torch.float32, device=DEV)
    binding.calib_moments_noalloc(X, out)                     # first call: symbol look-up
    torch.cuda.synchronize()
    free0, _ = torch.cuda.mem_get_info()
    alloc0, reserved0 = torch.cuda.memory_allocated(), torch.cuda.memory_reserved()
    binding.calib_moments_noalloc(X, out)
    torch.cuda.synchronize()
    free1, _ = torch.cuda.mem_get_info()
    assert free1 == free0
    assert torch.cuda.memory_allocated() == alloc0 and torch.cuda.memory_reserved() == reserved0
    want = sbo.calib_moments(X.cpu(), 1.0 / X.shape[0])
    assert np.allclose(out.cpu().double().numpy(), want, rtol=1e-5, atol=0)


def test_noalloc_with_no_tokens_gives_zeros_or_leaves_an_accumulator_alone():
    from paper_2602_17698_b200 import binding
    torch.cuda.set_device(0)
    X = torch.empty((0, 512), dtype=torch.bfloat16, device=DEV)
    out = torch.full((512,), 7.0, dtype=torch.float32, device=DEV)
    binding.calib_moments_noalloc(X, out, accumulate=True, scale=1.0)
    torch.cuda.synchronize()
    assert torch.all(out == 7.0)
    binding.calib_moments_noalloc(X, out, accumulate=False, scale=1.0)
    torch.cuda.synchronize()
    assert torch.all(out == 0.0)


def test_noalloc_rejects_sizes_beyond_its_fixed_scratch():
    from paper_2602_17698_b200 import binding
    torch.cuda.set_device(0)
    X = torch.zeros((4, 65536 + 8), dtype=torch.bfloat16, device=DEV)
    with pytest.raises(binding.SbError) as ei:
        binding.calib_moments_noalloc(X)
    assert ei.value.status == binding.SB_ERR_SCRATCH
    ok = binding.calib_moments_noalloc(torch.ones((4, 65536), dtype=torch.bfloat16, device=DEV))
    torch.cuda.synchronize()
    assert torch.all(ok == 1.0)

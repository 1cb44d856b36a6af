"""The GEMM entry point for callers that cannot allocate device memory (its split-K workspace
is a fixed array inside the library) against the ordinary entry point, which takes the
workspace from the caller.  This file sorts last on purpose: a run that stops at the first
failure has then already run every other test.  It passes alone in a fresh process and after
the rest of the suite: the first call on the device performs the one-time address lookup."""
import pytest
import torch

from gpu_util import library
from paper_2608_12385_b200 import binding

pytestmark = pytest.mark.gpu


def _inputs(n_out, K, R, seed):
    g = torch.Generator().manual_seed(seed)
    W = (torch.randn(n_out, K, generator=g) * 0.05).to(torch.bfloat16).cuda()
    X = torch.randn(R, K, generator=g).to(torch.bfloat16).cuda()
    return W, X


def test_static_scratch_entry_matches_caller_scratch_entry_twice_in_a_row():
    library()
    # first call: several splits, so the shared array really carries partial sums
    W, X = _inputs(1024, 2048, 24, seed=1)
    want, split_a = binding.op_gemm_tc(W, X, force_split=4)
    got, split_b = binding.op_gemm_tc_static(W, X, force_split=4)
    assert split_a == split_b == 4
    # same kernels, same split order: the tolerance of the GEMM tests (here it is met exactly)
    torch.testing.assert_close(got, want, rtol=0, atol=2e-6 * 0.25 * 5.0 * 2048)
    assert torch.equal(got, want)
    # second call right after, different shape and data: what the first call left behind in the
    # array must not leak into this result
    W2, X2 = _inputs(384, 512, 100, seed=2)
    want2, s2 = binding.op_gemm_tc(W2, X2, force_split=0)
    got2, s2b = binding.op_gemm_tc_static(W2, X2, force_split=0)
    assert s2 == s2b
    torch.testing.assert_close(got2, want2, rtol=0, atol=2e-6 * 0.25 * 5.0 * 512)
    assert torch.equal(got2, want2)


def test_sizes_beyond_the_static_array_are_refused_with_a_message():
    library()
    W, X = _inputs(32768, 64, 200, seed=3)  # roundup(200) = 256 rows x 32768 features = 2^23 floats > 2^21
    with pytest.raises(binding.DbtError) as e:
        binding.op_gemm_tc_static(W, X)
    assert e.value.status == 3 and "8 MiB" in str(e.value)
    W, X = _inputs(4096, 2048, 100, seed=4)  # fits unsplit (2^19), not with 16 splits (2^23)
    with pytest.raises(binding.DbtError) as e:
        binding.op_gemm_tc_static(W, X, force_split=16)
    assert e.value.status == 3
    got, used = binding.op_gemm_tc_static(W, X)  # the library's own choice is lowered to fit
    want, _ = binding.op_gemm_tc(W, X, force_split=used)
    assert torch.equal(got, want)

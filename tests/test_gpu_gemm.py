"""Operator-level parity of the grouped skinny GEMM (TMA + tcgen05) against the oracle's
linear routine, over row counts, ragged feature counts, ragged K and split-K factors."""
import numpy as np
import pytest
import torch

import oracle
from gpu_util import library
from paper_2608_12385_b200 import binding

pytestmark = pytest.mark.gpu


def _case(n_out, K, R, split, seed):
    library()
    g = torch.Generator().manual_seed(seed)
    W = (torch.randn(n_out, K, generator=g) * 0.05).to(torch.bfloat16)
    X = torch.randn(R, K, generator=g).to(torch.bfloat16)
    want = oracle.linear(W, X.float().numpy())
    got, used = binding.op_gemm_tc(W.cuda(), X.cuda(), force_split=split)
    got = got.cpu().numpy()
    # bf16 x bf16 products are exact in fp32; only the fp32 summation order differs
    scale = np.abs(W.float().numpy()).max() * np.abs(X.float().numpy()).max() * K
    np.testing.assert_allclose(got, want, rtol=0, atol=2e-6 * scale)
    rel = np.linalg.norm(got - want) / np.linalg.norm(want)
    assert rel < 1e-5, rel
    return used


@pytest.mark.parametrize("R", [1, 2, 8, 16, 17, 32, 33, 64, 100, 128, 200, 256])
def test_row_counts_span_every_instruction_width(R):
    _case(n_out=384, K=512, R=R, split=0, seed=R)


@pytest.mark.parametrize("n_out,K", [(128, 64), (130, 72), (712, 256), (100, 1000), (2048, 2048), (1024, 5632)])
def test_ragged_features_and_k(n_out, K):
    _case(n_out=n_out, K=K, R=6, split=0, seed=n_out + K)


@pytest.mark.parametrize("split", [1, 2, 3, 7, 16])
def test_split_k_partials_sum_to_the_same_result(split):
    used = _case(n_out=256, K=2048, R=12, split=split, seed=split)
    assert used >= 1


def test_one_hot_rows_pick_weight_columns_exactly():
    """A one-hot activation row returns a column of W bit-exactly (catches a transposed or
    mis-swizzled operand)."""
    library()
    n_out, K, R = 256, 320, 20
    g = torch.Generator().manual_seed(7)
    W = torch.randn(n_out, K, generator=g).to(torch.bfloat16)
    X = torch.zeros(R, K, dtype=torch.bfloat16)
    cols = [(37 * r + 5) % K for r in range(R)]
    for r, c in enumerate(cols):
        X[r, c] = 1.0
    got, _ = binding.op_gemm_tc(W.cuda(), X.cuda(), force_split=2)
    for r, c in enumerate(cols):
        assert torch.equal(got[r].cpu(), W[:, c].float())


def test_columns_are_independent_of_their_neighbours():
    """A row's result does not depend on which other rows are stacked with it, nor on the
    instruction width it is padded to."""
    library()
    g = torch.Generator().manual_seed(8)
    W = (torch.randn(512, 1024, generator=g) * 0.05).to(torch.bfloat16).cuda()
    X = torch.randn(40, 1024, generator=g).to(torch.bfloat16).cuda()
    full, _ = binding.op_gemm_tc(W, X, force_split=4)           # 40 rows -> 64-wide instruction
    same, _ = binding.op_gemm_tc(W, X[:35].contiguous(), force_split=4)  # 35 rows -> 64-wide too
    assert torch.equal(full[:35], same)
    narrow, _ = binding.op_gemm_tc(W, X[:20].contiguous(), force_split=4)  # 32-wide instruction
    torch.testing.assert_close(full[:20], narrow, rtol=1e-5, atol=1e-5)
    print("bit-identical across instruction widths:", torch.equal(full[:20], narrow))


def test_an_expired_device_wait_is_reported_and_the_next_call_is_clean(monkeypatch):
    """Every wait inside the kernels is bounded.  With the host-set test hook one CTA of a tiny GEMM never
    requests one of its weight tiles and the limit drops to about a millisecond: the waits on that tile run
    out, the kernel records status 3 with the wait site, skips its stores, frees its tensor memory and
    returns -- nothing traps and nothing spins on.  The very next call on the same GPU, without the hook,
    is clean and correct."""
    g = torch.Generator(device="cpu").manual_seed(3)
    W = torch.randn(256, 512, generator=g).to(torch.bfloat16).cuda()
    X = torch.randn(8, 512, generator=g).to(torch.bfloat16).cuda()
    monkeypatch.setenv("DBT_TEST_EXPIRE_WAIT", "1")
    with pytest.raises(binding.DbtError) as e:
        binding.op_gemm_tc(W, X, force_split=2)
    assert e.value.status == 7 and ("[3, 10" in str(e.value) or "[3, 20" in str(e.value)), str(e.value)
    monkeypatch.delenv("DBT_TEST_EXPIRE_WAIT")
    Y, _ = binding.op_gemm_tc(W, X, force_split=2)
    want = X.float() @ W.float().T
    assert torch.allclose(Y, want, rtol=1e-3, atol=1e-2)
    torch.cuda.synchronize()

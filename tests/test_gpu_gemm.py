"""The weight-streaming skinny GEMM of the decode kernel against a float64 matrix product."""

import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu

from paper_2506_03700_b200 import binding, synth


def _case(N, K, cols, mode, seed=7):
    W = synth.normal_tensor(seed, 11, (N, K), 0.05, torch.bfloat16, "cuda")
    X = synth.normal_tensor(seed, 12, (cols, K), 1.0, torch.float32, "cuda")
    Y, _ = binding.debug_gemm(W, X, mode)
    Wd, Xd = W.double().cpu().numpy(), X.double().cpu().numpy()
    ref = Xd @ Wd.T
    if mode == 1:
        g, u = ref[:, :N // 2], ref[:, N // 2:]
        ref = g / (1.0 + np.exp(-g)) * u
    return Y.double().cpu().numpy(), ref


# shapes: one tile; ragged last tile and several k chunks; k tail shorter than a chunk; more
# tiles than the grid holds at once (several groups per block); the 8B-shaped down projection
@pytest.mark.parametrize("N,K,cols", [(16, 64, 1), (48, 128, 3), (1000, 1216, 8), (5003, 512, 5), (40000, 192, 2),
                                      (4096, 14336, 6), (6144, 4096, 1)])
def test_streaming_gemm_matches_float64(N, K, cols):
    y, ref = _case(N, K, cols, 0)
    assert np.abs(y - ref).max() <= 2e-5 * max(1.0, np.abs(ref).max())


@pytest.mark.parametrize("N,K,cols", [(2 * 688, 256, 4), (2 * 14336, 4096, 6), (2 * 16, 64, 8)])
def test_streaming_gate_up_swiglu(N, K, cols):
    y, ref = _case(N, K, cols, 1)
    assert np.abs(y - ref).max() <= 2e-5 * max(1.0, np.abs(ref).max())


def test_result_of_a_column_does_not_depend_on_the_other_columns():
    """The same token in another column, alone or beside other tokens, gives the same bits."""
    N, K = 2048, 1536
    W = synth.normal_tensor(3, 11, (N, K), 0.05, torch.bfloat16, "cuda")
    X = synth.normal_tensor(3, 12, (8, K), 1.0, torch.float32, "cuda")
    full, _ = binding.debug_gemm(W, X, 0)
    for c in (0, 3, 7):
        alone, _ = binding.debug_gemm(W, X[c:c + 1].contiguous(), 0)
        assert torch.equal(alone[0], full[c])
    perm = [5, 2, 7, 0]
    mixed, _ = binding.debug_gemm(W, X[perm].contiguous(), 0)
    for j, c in enumerate(perm):
        assert torch.equal(mixed[j], full[c])


def test_bad_arguments_are_refused():
    W = torch.zeros(32, 48, dtype=torch.bfloat16, device="cuda")      # K not a multiple of 64
    X = torch.zeros(1, 48, dtype=torch.float32, device="cuda")
    with pytest.raises(binding.AdaError) as e:
        binding.debug_gemm(W, X, 0)
    assert e.value.code == -1


# ---------------------------------------------------------------- dense GEMM of the prompt pass (tcgen05)

@pytest.mark.parametrize("N,K,rows", [(64, 64, 128), (64, 256, 5), (200, 512, 128), (6144, 4096, 77), (4096, 14336, 128)])
def test_dense_gemm_matches_float64(N, K, rows):
    W = synth.normal_tensor(9, 11, (N, K), 0.05, torch.bfloat16, "cuda")
    X = synth.normal_tensor(9, 12, (rows, K), 1.0, torch.float32, "cuda")
    Y = binding.debug_dense_gemm(W, X)
    ref = X.double().cpu().numpy() @ W.double().cpu().numpy().T
    assert torch.isfinite(Y).all()
    assert np.abs(Y.double().cpu().numpy() - ref).max() <= 2e-5 * max(1.0, np.abs(ref).max())
    # accumulate form: the product is added to what the output holds
    Y2 = torch.ones_like(Y)
    binding.debug_dense_gemm(W, X, Y2)
    assert np.abs(Y2.double().cpu().numpy() - (ref + 1.0)).max() <= 2e-5 * max(1.0, np.abs(ref).max())

"""tcgen05 / TMA GEMM against fp64 matmul of the same bf16 inputs: every operand-layout
combination, tile tails in M, N and K, the residual and the split-K reduction epilogues."""
import numpy as np
import pytest
import torch

from paper_2605_16154_b200 import synth
from tests.gpu_helpers import rel_fro

pytestmark = pytest.mark.gpu


def _mods():
    from paper_2605_16154_b200 import binding as B, pipeline as PL
    return B, PL


def _operands(rng, M, N, K, a_k, b_k, PL):
    A = synth.round_to_dtype(rng.standard_normal((M, K)).astype(np.float32), "bf16")
    Bm = synth.round_to_dtype(rng.standard_normal((N, K)).astype(np.float32), "bf16")
    At = PL.dev(A if a_k else A.T.copy(), torch.bfloat16)
    Bt = PL.dev(Bm if b_k else Bm.T.copy(), torch.bfloat16)
    return A, Bm, At, Bt


@pytest.mark.parametrize("a_k,b_k", [(True, True), (True, False), (False, True), (False, False)])
@pytest.mark.parametrize("M,N,K", [(128, 256, 64), (304, 768, 200), (936, 1024, 1024), (200, 96, 72)])
def test_tcgen05_gemm_layouts_and_tails(a_k, b_k, M, N, K):
    B, PL = _mods()
    rng = np.random.default_rng(11)
    A, Bm, At, Bt = _operands(rng, M, N, K, a_k, b_k, PL)
    expect = A.astype(np.float64) @ Bm.astype(np.float64).T
    out = B.grpo_gemm(At, a_k, Bt, b_k, M, N, K, torch.float32, backend=2)
    assert rel_fro(out.cpu().numpy(), expect) < 1e-5
    # bf16 output with an fp32 residual
    R = rng.standard_normal((M, N)).astype(np.float32)
    out16 = B.grpo_gemm(At, a_k, Bt, b_k, M, N, K, torch.bfloat16, R=PL.dev(R), backend=2)
    assert rel_fro(out16.float().cpu().numpy(), expect + R) < 4e-3


@pytest.mark.parametrize("M,N,K", [(256, 512, 5000), (1024, 256, 936), (768, 256, 300)])
def test_tcgen05_weight_gradient_shape_split_k_accumulates(M, N, K):
    """dW[M, N] += dY^T X with tokens along K: both operands MN-major, fp32 reduction epilogue."""
    B, PL = _mods()
    rng = np.random.default_rng(12)
    A, Bm, At, Bt = _operands(rng, M, N, K, False, False, PL)
    start = rng.standard_normal((M, N)).astype(np.float32)
    acc = PL.dev(start.copy())
    B.grpo_gemm(At, False, Bt, False, M, N, K, R=acc, backend=2, C_out=acc)
    expect = A.astype(np.float64) @ Bm.astype(np.float64).T + start
    assert rel_fro(acc.cpu().numpy(), expect) < 1e-5


def test_tcgen05_matches_simt_on_strided_views():
    """Operands and outputs that are column slices of wider buffers (row stride > width)."""
    B, PL = _mods()
    rng = np.random.default_rng(13)
    M, N, K = 312, 256, 256
    big = PL.dev(synth.round_to_dtype(rng.standard_normal((M, 3 * K)).astype(np.float32), "bf16"), torch.bfloat16)
    Wt = PL.dev(synth.round_to_dtype(rng.standard_normal((N, K)).astype(np.float32), "bf16"), torch.bfloat16)
    A = big[:, K:2 * K]
    outs = []
    for backend in (1, 2):
        C = torch.zeros((M, N), dtype=torch.float32, device="cuda")
        rc = B._lib.grpo_gemm(M, N, K, A.data_ptr(), A.stride(0), 1, Wt.data_ptr(), Wt.stride(0), 1, B.GRPO_BF16,
                              C.data_ptr(), C.stride(0), B.GRPO_F32, None, 0, backend,
                              torch.cuda.current_stream().cuda_stream)
        assert rc == 0
        outs.append(C.cpu().numpy())
    assert rel_fro(outs[1], outs[0]) < 1e-5

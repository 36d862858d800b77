"""tcgen05 GEMM at the shapes one step of the medium and the large workload really launches, checked
against fp64 matmul on sampled output rows (a row of the output is an independent dot-product problem,
so the oracle computes only the sampled ones).

These shapes reach code the small cases do not: a persistent CTA pair walking tens of tiles with the
tile position wrapping in all three indices, the wave-filling split of a 119 808-long contraction with
the fp32 reduction epilogue, and row tiles at the very end of a 119 808-row operand.  Tolerances: 4e-3 for bf16 outputs as in the small GEMM cases;
1e-4 for the fp32 weight-gradient reduction over 119 808 terms (derived where it is used)."""
import numpy as np
import pytest
import torch

from tests.gpu_helpers import rel_fro

pytestmark = pytest.mark.gpu

M_C1 = 384 * 312        # tokens of one medium step: 119 808


def _mods():
    from paper_2605_16154_b200 import binding as B
    return B


def _rand_bf16(shape, seed, scale=1.0):
    g = torch.Generator(device="cuda").manual_seed(seed)
    return (torch.randn(shape, generator=g, device="cuda") * scale).to(torch.bfloat16)


def _sample_rows(n, tile, extra=()):
    """Rows from the first, a middle and the last tile, tile boundaries included."""
    picks = {0, 1, tile - 1, tile, n // 2, n // 2 + 1, n - tile, n - 2, n - 1}
    rng = np.random.default_rng(n)
    picks.update(int(v) for v in rng.integers(0, n, size=48))
    picks.update(extra)
    return np.array(sorted(p for p in picks if 0 <= p < n), dtype=np.int64)


def _f64(t):
    return t.float().cpu().numpy().astype(np.float64)


@pytest.mark.parametrize("M,N,K", [(M_C1, 3072, 1024),          # QKV projection of the medium model
                                   (96 * 312, 6144, 2048)])     # QKV projection of the large model (96-chunk micro-batch)
def test_forward_shape_bf16_out_on_sampled_rows(M, N, K):
    B = _mods()
    A = _rand_bf16((M, K), 1)
    W = _rand_bf16((N, K), 2, 0.05)
    out = B.grpo_gemm(A, True, W, True, M, N, K, torch.bfloat16, backend=2)
    rows = _sample_rows(M, 256)
    expect = _f64(A[rows]) @ _f64(W).T                           # every column tile of the sampled rows
    got = out[rows].float().cpu().numpy()
    assert rel_fro(got, expect) < 4e-3
    for lo in range(0, N, 256):                                   # no column tile may hide behind the others
        assert rel_fro(got[:, lo:lo + 256], expect[:, lo:lo + 256]) < 4e-3, lo


def test_input_gradient_shape_nn_on_sampled_rows():
    """dX[M][d] = dY[M][8d] W[8d][d]: B is MN-major, K = 8192."""
    B = _mods()
    M, N, K = M_C1, 1024, 8192
    dY = _rand_bf16((M, K), 3)
    W = _rand_bf16((K, N), 4, 0.05)
    out = B.grpo_gemm(dY, True, W, False, M, N, K, torch.bfloat16, backend=2)
    rows = _sample_rows(M, 256)
    expect = _f64(dY[rows]) @ _f64(W)
    assert rel_fro(out[rows].float().cpu().numpy(), expect) < 4e-3


@pytest.mark.parametrize("M,N", [(3072, 1024), (1024, 1024)])
def test_weight_gradient_shape_tn_accumulates_into_a_non_zero_start(M, N):
    """dW[M][N] += dY^T X with the 119 808 tokens along the contraction: both operands MN-major, the
    contraction split over CTA pairs and reduced in fp32 into what the buffer already holds."""
    B = _mods()
    K = M_C1
    dY = _rand_bf16((K, M), 5)
    X = _rand_bf16((K, N), 6)
    g = torch.Generator(device="cuda").manual_seed(7)
    start = torch.randn((M, N), generator=g, device="cuda") * 100.0
    acc = start.clone()
    B.grpo_gemm(dY, False, X, False, M, N, K, R=acc, backend=2, C_out=acc)
    rows = _sample_rows(M, 256)
    Xd = _f64(X)
    expect = _f64(dY[:, rows]).T @ Xd + start[rows].cpu().numpy().astype(np.float64)
    got = acc[rows].cpu().numpy()
    # A contraction of 119 808 terms is about 830 accumulating MMAs per split and the fp32 accumulator is not
    # rounded to nearest (addends are aligned and truncated), so the error is a small bias of up to one unit in
    # the last place per accumulation: bounded by (K / 16 / splits) * 2^-23 ~ 1e-4 relative, measured 4.4e-5.
    # The 1e-5 of the short contractions does not carry over; 1e-4 does, for the norm, per column tile and per entry.
    tol = 1e-4
    assert rel_fro(got, expect) < tol
    for lo in range(0, N, 256):
        assert rel_fro(got[:, lo:lo + 256], expect[:, lo:lo + 256]) < tol, lo
    assert np.max(np.abs(got - expect)) < tol * np.max(np.abs(expect))

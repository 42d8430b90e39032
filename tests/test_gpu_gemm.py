"""bf16 matrix products behind the MLP passes: the tensor-core (tcgen05) kernel and the CUDA-core
kernel against numpy's fp64 matmul of the same bf16 values, for every operand layout the forward,
backward-data, weight-gradient and R-operator passes use, ragged sizes included."""
import numpy as np
import pytest
import torch

import synth_inputs as si

pytestmark = pytest.mark.gpu


def _mat(seed, rows, cols, ld):
    a = si.to_bf16_values(si.normal_f32(seed, 1, (rows, cols)))
    buf = torch.zeros(rows, ld, dtype=torch.bfloat16, device="cuda")
    buf[:, :cols] = torch.from_numpy(a).to(torch.bfloat16).cuda()
    return a.astype(np.float64), buf


def _ld8(n):
    return (n + 7) // 8 * 8


def _operand(seed, logical_rows, logical_cols, transposed):
    """Logical [rows, cols] matrix, stored as is or transposed; returns (fp64 logical, device buffer, ld)."""
    if transposed:
        a, buf = _mat(seed, logical_cols, logical_rows, _ld8(logical_rows))
        return a.T, buf, _ld8(logical_rows)
    a, buf = _mat(seed, logical_rows, logical_cols, _ld8(logical_cols))
    return a, buf, _ld8(logical_cols)


SHAPES = [(128, 128, 64), (256, 384, 192), (200, 136, 104), (512, 10, 1024), (10, 1024, 512), (1024, 512, 784),
          (300, 1000, 72), (64, 4096, 8), (130, 70, 1000)]


@pytest.mark.parametrize("path", [1, 2, 3, 4, 5])
@pytest.mark.parametrize("ta,tb", [(0, 1), (0, 0), (1, 0), (1, 1)])
@pytest.mark.parametrize("M,N,K", SHAPES)
def test_single_product(path, ta, tb, M, N, K):
    import paper_2207_02849_b200 as bt
    A, dA, lda = _operand(1, M, K, ta)
    B, dB, ldb = _operand(2, K, N, tb)          # stored [N,K] when tb
    C = torch.full((M, N), float("nan"), dtype=torch.float32, device="cuda")
    w = torch.zeros(1, dtype=torch.float32, device="cuda")
    lv = bt.Level(bt.LOSS_LOGREG, bt.PARAM_VECTOR, w)
    ws = bt.Workspace.__new__(bt.Workspace)
    ws.nbytes = 4096
    ws.buf = torch.zeros(4096 + 256, dtype=torch.uint8, device="cuda")
    ws.ptr = ws.buf.data_ptr() + (-ws.buf.data_ptr()) % 256
    bt.betty_gemm_bf16(M, N, [(dA, lda, ta, dB, ldb, tb, K, 1.0)], C, N, 0.0, path, ws)
    st, _ = bt.betty_poll_status(ws, raise_on_error=False)
    assert st == bt.BETTY_OK
    ref = A @ B
    got = C.double().cpu().numpy()
    assert np.linalg.norm(got - ref) / np.linalg.norm(ref) < 1e-5


@pytest.mark.parametrize("path", [1, 2, 3, 4, 5])
def test_two_products_negation_and_beta(path):
    import paper_2207_02849_b200 as bt
    M, N, K1, K2 = 200, 264, 136, 72
    A1, dA1, lda1 = _operand(3, M, K1, 0)
    B1, dB1, ldb1 = _operand(4, K1, N, 0)
    A2, dA2, lda2 = _operand(5, M, K2, 1)
    B2, dB2, ldb2 = _operand(6, K2, N, 0)
    C0 = si.normal_f32(7, 1, (M, N))
    C = torch.from_numpy(C0).cuda()
    ws = bt.Workspace.__new__(bt.Workspace)
    ws.nbytes = 4096
    ws.buf = torch.zeros(4096 + 256, dtype=torch.uint8, device="cuda")
    ws.ptr = ws.buf.data_ptr() + (-ws.buf.data_ptr()) % 256
    bt.betty_gemm_bf16(M, N, [(dA1, lda1, 0, dB1, ldb1, 0, K1, -1.0), (dA2, lda2, 1, dB2, ldb2, 0, K2, 1.0)], C, N, 1.0,
                       path, ws)
    assert bt.betty_poll_status(ws, raise_on_error=False)[0] == bt.BETTY_OK
    ref = -(A1 @ B1) + A2 @ B2 + C0.astype(np.float64)
    got = C.double().cpu().numpy()
    assert np.linalg.norm(got - ref) / np.linalg.norm(ref) < 1e-5

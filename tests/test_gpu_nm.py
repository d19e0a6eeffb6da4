"""GPU parity for mwu_keep_n_of_m (Section 4.7: two of every four consecutive weights stay) and
mwu_gemm_dense against the CPU checker: Q, the keep bitmap and the bf16 weight matrix bit for bit,
the product within the GEMM tolerances."""
import numpy as np
import pytest
import torch

from oracle import mwu_oracle as O
from paper_2106_08301_b200 import binding as B
from paper_2106_08301_b200 import inputs
from test_gpu_gemm import errors

pytestmark = pytest.mark.gpu


def keep_on_gpu(W, n, U=None, ldw=None):
    rows, cols = W.shape
    ldw = ldw or (cols + 7) // 8 * 8            # rows of the bf16 matrix start on 16-byte boundaries
    Q = torch.full((rows, cols), float("nan"), dtype=torch.float32, device="cuda")
    bits = torch.zeros((rows * cols + 31) // 32, dtype=torch.int32, device="cuda")
    Wd = torch.full((rows, ldw), float("nan"), dtype=torch.bfloat16, device="cuda")
    st = torch.zeros(1, dtype=torch.int32, device="cuda")
    B.mwu_keep_n_of_m(rows, cols, n, 4, W.cuda(), None if U is None else U.cuda(), Q, bits, Wd, ldw, st)
    torch.cuda.synchronize()
    return Q, bits, Wd, st


@pytest.mark.parametrize("n", [0, 1, 2, 3, 4])
@pytest.mark.parametrize("rows,cols", [(64, 64), (37, 100), (300, 1004)])
def test_keep_n_of_4_parity(n, rows, cols):
    W = inputs.normal_weights(rows, cols, 0.02, 800 + n + rows)
    r = O.project_n_of_m(W.numpy(), n, 4)
    Q, bits, Wd, st = keep_on_gpu(W, n)
    assert int(st.item()) == 0
    assert np.array_equal(Q.cpu().numpy().view(np.uint32), r.Q.view(np.uint32))
    assert np.array_equal(bits.cpu().numpy().view(np.uint32), O.bitmap_words(r.keep.reshape(-1)))
    ref_bf = torch.from_numpy(r.Q).to(torch.bfloat16)
    assert torch.equal(Wd[:, :cols].cpu().contiguous().view(torch.int16), ref_bf.view(torch.int16))


def test_keep_2_of_4_ties_zeros_dual_and_leading_dimension():
    W = inputs.normal_weights(16, 64, 0.02, 810)
    W[:, 0:8] = 0.5 * torch.sign(W[:, 0:8])      # equal magnitudes: the lower index stays
    W[:, 8:16] = 0.0
    W[3, 8] = -0.0
    U = inputs.normal_weights(16, 64, 0.01, 811)
    for dual in (None, U):
        r = O.project_n_of_m(W.numpy(), 2, 4, U=None if dual is None else dual.numpy())
        Q, bits, Wd, st = keep_on_gpu(W, 2, U=dual, ldw=72)
        assert np.array_equal(Q.cpu().numpy().view(np.uint32), r.Q.view(np.uint32))
        assert np.array_equal(bits.cpu().numpy().view(np.uint32), O.bitmap_words(r.keep.reshape(-1)))
        assert bool(torch.isnan(Wd[:, 64:].float()).all())            # nothing written past cols
    Wbad = W.clone()
    Wbad[2, 5] = float("inf")
    assert int(keep_on_gpu(Wbad, 2)[3].item()) & B.MWU_DEV_NONFINITE
    st = torch.zeros(1, dtype=torch.int32, device="cuda")
    Wc = W.cuda()
    bits = torch.zeros(32, dtype=torch.int32, device="cuda")
    assert B.mwu_keep_n_of_m(16, 64, 2, 8, Wc, None, None, bits, None, 64, st, check=False) == 2     # m != 4
    assert B.mwu_keep_n_of_m(16, 64, 5, 4, Wc, None, None, bits, None, 64, st, check=False) == 2


@pytest.mark.parametrize("N,K,M", [(512, 256, 700), (200, 192, 1100), (1024, 1024, 2048 + 31)])
def test_keep_2_of_4_then_dense_gemm(N, K, M):
    W = inputs.normal_weights(N, K, 0.02, 820 + N)
    X = inputs.normal_activations_bf16((M, K), 821 + N)
    r = O.project_n_of_m(W.numpy(), 2, 4)
    What = O.bf16_bits_to_f64(O.bf16_bits_rne(r.Q))
    ref = O.gemm(X.to(torch.float64).numpy(), What)
    Q, bits, Wd, st = keep_on_gpu(W, 2)
    for y_dtype, tol in ((1, 1e-5), (0, 2e-3)):
        Y = torch.full((M, N), float("nan"), dtype=torch.float32 if y_dtype else torch.bfloat16, device="cuda")
        B.mwu_gemm_dense(N, K, Wd, K, X.cuda(), M, K, Y, N, y_dtype, st)
        torch.cuda.synchronize()
        assert int(st.item()) == 0
        fro, mx = errors(Y.float().cpu().numpy(), ref)
        assert fro <= tol and mx <= 1e-2, (y_dtype, fro, mx)

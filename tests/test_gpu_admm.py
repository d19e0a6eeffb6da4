"""GPU parity: mwu_admm_step (projection + dual update + residual) through the C ABI against the
CPU checker.  U_next is compared bit for bit; residual_sq within 1e-10 relative (an fp64 sum whose
order of additions is not fixed)."""
import numpy as np
import pytest
import torch

from oracle import mwu_oracle as O
from paper_2106_08301_b200 import binding as B
from paper_2106_08301_b200 import inputs

pytestmark = pytest.mark.gpu

RESIDUAL_RTOL = 1e-10


def run_step(W, b, ku, kp, U=None, prune_key=0, algo=B.MWU_ALGO_AUTO, want_q=True, want_u=True, want_r=True):
    rows, cols = W.shape
    desc = B.make_desc(rows, cols, b, ku, kp, prune_key, algo)
    bufs = B.ProjectionBuffers(desc, want_q=want_q)
    Wd = W.cuda().contiguous()
    Ud = U.cuda().contiguous() if U is not None else None
    U_next = torch.full((rows * cols,), float("nan"), dtype=torch.float32, device="cuda") if want_u else None
    resid = torch.full((1,), 123.0, dtype=torch.float64, device="cuda") if want_r else None
    bufs.admm_step(Wd, Ud, U_next, resid)
    torch.cuda.synchronize()
    assert int(bufs.dev_status.item()) == 0
    return bufs, U_next, resid


def check(W, b, ku, kp, U=None, prune_key=0, algos=(B.MWU_ALGO_MULTI_PASS, B.MWU_ALGO_ONE_PASS)):
    p = O.project(W.numpy(), b, ku, kp, U=None if U is None else U.numpy(),
                  prune_key="l1" if prune_key else "l2sq")
    d = O.dual_update(p, b)
    for algo in algos:
        bufs, U_next, resid = run_step(W, b, ku, kp, U, prune_key, algo)
        assert np.array_equal(bufs.Q.cpu().numpy().view(np.uint32), p.Q.reshape(-1).view(np.uint32))
        assert np.array_equal(bufs.pruned_bitmap.cpu().numpy().view(np.uint32), O.bitmap_words(p.pruned))
        assert np.array_equal(bufs.unified_bitmap.cpu().numpy().view(np.uint32), O.bitmap_words(p.unified))
        assert np.array_equal(bufs.u.cpu().numpy(), p.u)
        assert np.array_equal(U_next.cpu().numpy().view(np.uint32), d.U_next.reshape(-1).view(np.uint32))
        r = float(resid.item())
        assert abs(r - d.residual_sq) <= RESIDUAL_RTOL * max(d.residual_sq, 1e-300), (r, d.residual_sq)
    return p, d


@pytest.mark.parametrize("b", [2, 4, 8, 16])
@pytest.mark.parametrize("rows,cols", [(64, 64), (7, 48), (300, 1008)])
def test_admm_step_parity_small(b, rows, cols):
    W = inputs.normal_weights(rows, cols, 0.02, 500 + b)
    U = inputs.normal_weights(rows, cols, 0.005, 600 + b)
    Mb = rows * cols // b
    check(W, b, O.count_from_permille(Mb, 600), O.count_from_permille(Mb, 300), U=U)


@pytest.mark.parametrize("b,rows,cols,permille", [(16, 1000, 4112, (800, 600)), (4, 517, 1028, (500, 250)),
                                                  (2, 300, 1002, (350, 250)), (8, 640, 1032, (100, 0)),
                                                  (8, 512, 1024, (1000, 900))])
def test_admm_step_parity_medium_one_pass(b, rows, cols, permille):
    W = inputs.normal_weights(rows, cols, 0.02, 700 + b)
    U = inputs.normal_weights(rows, cols, 0.004, 800 + b)
    Mb = rows * cols // b
    check(W, b, O.count_from_permille(Mb, permille[0]), O.count_from_permille(Mb, permille[1]), U=U,
          algos=(B.MWU_ALGO_AUTO,))


def test_admm_step_l1_key_and_no_dual():
    W = inputs.normal_weights(512, 1024, 0.02, 41)
    Mb = W.numel() // 8
    check(W, 8, Mb * 6 // 10, Mb * 3 // 10, prune_key=1)        # Kp is the L1 norm, the residual is not
    check(W, 8, Mb * 6 // 10, Mb * 3 // 10)


def test_admm_step_fallback_resets_the_residual():
    """A projected tensor projected again: the one-pass attempt is given up (thousands of equal
    keys) after it has already written provisional outputs and sums; the multi-pass kernels must
    leave the exact U_next (all zero) and residual (zero)."""
    W = inputs.normal_weights(512, 2048, 0.02, 17)
    b = 16
    Mb = W.numel() // b
    ku, kp = Mb * 8 // 10, Mb * 6 // 10
    p, d = check(W, b, ku, kp, algos=(B.MWU_ALGO_AUTO,))
    Q1 = torch.from_numpy(p.Q.copy())
    p2, d2 = check(Q1, b, ku, kp, algos=(B.MWU_ALGO_AUTO,))
    assert d2.residual_sq == 0.0 and not d2.U_next.any()


def test_admm_two_iterations_on_device():
    """U_1 from the first call feeds the second: the dual variable accumulates as in Algorithm 1."""
    W = inputs.normal_weights(256, 512, 0.02, 51)
    b = 4
    Mb = W.numel() // b
    ku, kp = Mb // 2, Mb // 8
    p1, d1 = check(W, b, ku, kp, algos=(B.MWU_ALGO_ONE_PASS,))
    U1 = torch.from_numpy(d1.U_next.copy())
    check(W, b, ku, kp, U=U1, algos=(B.MWU_ALGO_ONE_PASS, B.MWU_ALGO_MULTI_PASS))


def test_admm_step_optional_outputs_and_errors():
    W = inputs.normal_weights(128, 256, 0.02, 61)
    b = 8
    Mb = W.numel() // b
    p = O.project(W.numpy(), b, Mb // 2, Mb // 4)
    d = O.dual_update(p, b)
    bufs, U_next, resid = run_step(W, b, Mb // 2, Mb // 4, want_q=False, want_r=False)
    assert np.array_equal(U_next.cpu().numpy(), d.U_next.reshape(-1))
    bufs, U_next, resid = run_step(W, b, Mb // 2, Mb // 4, want_u=False)
    assert abs(float(resid.item()) - d.residual_sq) <= RESIDUAL_RTOL * d.residual_sq
    desc = B.make_desc(128, 256, b, Mb // 2, Mb // 4)
    bufs = B.ProjectionBuffers(desc)
    Wd = W.cuda()
    # nothing asked for beyond the projection; U_next on top of an input
    assert B.mwu_admm_step(desc, Wd, None, bufs.Q, None, None, bufs.u, bufs.pruned_bitmap, bufs.unified_bitmap,
                           bufs.sign_bits, bufs.dev_status, bufs.workspace, check=False) == B.MWU_ERR_INVALID_ARG
    assert B.mwu_admm_step(desc, Wd, None, bufs.Q, Wd.reshape(-1), None, bufs.u, bufs.pruned_bitmap,
                           bufs.unified_bitmap, bufs.sign_bits, bufs.dev_status, bufs.workspace,
                           check=False) == B.MWU_ERR_INVALID_ARG

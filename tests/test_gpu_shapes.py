"""GPU parity for the 2- and 3-dim block shapes of Section 3.1 / Table 1 ([2,2] for linear layers
and 1x1 convolutions, [2,2,2] for 3x3 convolutions): mwu_project / mwu_admm_step through the C ABI
against the CPU checker bit for bit; the product on the projected weights within the GEMM
tolerances (packed form for 2-dim shapes, dense bf16 weights for shapes without a packed form)."""
import numpy as np
import pytest
import torch

from oracle import mwu_oracle as O
from paper_2106_08301_b200 import binding as B
from paper_2106_08301_b200 import inputs
from test_gpu_gemm import errors
from test_gpu_projection import decoded_on_gpu

pytestmark = pytest.mark.gpu


def shaped_desc(rows, cols, shape, ku, kp, prune_key=0):
    return B.make_desc(rows, cols, shape.dk, ku, kp, prune_key, block_rows=shape.dr, block_taps=shape.dt,
                       taps=shape.taps)


def check_shape(W, shape, unified_permille, pruned_permille, U=None, prune_key=0, admm=False):
    rows, cols = W.shape
    Mb = O.partition(rows, cols, shape).idx.shape[0]
    ku, kp = O.count_from_permille(Mb, unified_permille), O.count_from_permille(Mb, pruned_permille)
    p = O.project(W.numpy(), shape, ku, kp, U=None if U is None else U.numpy(),
                  prune_key="l1" if prune_key else "l2sq")
    desc = shaped_desc(rows, cols, shape, ku, kp, prune_key)
    assert desc.n_blocks == Mb
    bufs = B.ProjectionBuffers(desc, want_q=True, want_loss=True)
    Wd = W.cuda().contiguous()
    Ud = U.cuda().contiguous() if U is not None else None
    if admm:
        U_next = torch.full((rows, cols), float("nan"), dtype=torch.float32, device="cuda")
        resid = torch.full((1,), float("nan"), dtype=torch.float64, device="cuda")
        bufs.loss_u = bufs.loss_p = None
        bufs.admm_step(Wd, Ud, U_next, resid)
    else:
        bufs.project(Wd, Ud)
    torch.cuda.synchronize()
    assert int(bufs.dev_status.item()) == 0
    if not admm:
        assert np.array_equal(bufs.loss_u.cpu().numpy().view(np.uint64), p.stats.L_u.view(np.uint64))
        kp_ref = p.stats.S if prune_key else p.stats.L_p
        assert np.array_equal(bufs.loss_p.cpu().numpy().view(np.uint64), kp_ref.view(np.uint64))
    assert np.array_equal(bufs.pruned_bitmap.cpu().numpy().view(np.uint32), O.bitmap_words(p.pruned))
    assert np.array_equal(bufs.unified_bitmap.cpu().numpy().view(np.uint32), O.bitmap_words(p.unified))
    assert np.array_equal(bufs.sign_bits.cpu().numpy().view(np.uint32), O.bitmap_words(p.sign.reshape(-1)))
    assert np.array_equal(bufs.u.cpu().numpy(), p.u)
    assert np.array_equal(bufs.Q.cpu().numpy().reshape(W.shape).view(np.uint32), p.Q.view(np.uint32))
    if admm:
        d = O.dual_update(p)
        assert np.array_equal(U_next.cpu().numpy().view(np.uint32), d.U_next.view(np.uint32))
        assert abs(float(resid.item()) - d.residual_sq) <= 1e-10 * max(d.residual_sq, 1e-300)
    return desc, bufs, Wd, p


@pytest.mark.parametrize("shape,rows,cols", [(O.BlockShape(2, 2), 1024, 256),                 # 2x2, a 1x1-conv / FC weight
                                             (O.BlockShape(2, 2, 2, taps=9), 128, 1152),      # 2x2x2 on a 3x3 conv weight
                                             (O.BlockShape(4, 2), 66, 136),
                                             (O.BlockShape(2, 4), 64, 70),
                                             (O.BlockShape(2, 2, 2, taps=4), 32, 256),        # taps divide evenly
                                             (O.BlockShape(4, 1, 2, taps=9), 24, 288),
                                             (O.BlockShape(2, 2, 2, taps=25), 16, 400)])
def test_block_shape_projection_parity(shape, rows, cols):
    W = inputs.normal_weights(rows, cols, 0.02, 900 + rows + cols)
    check_shape(W, shape, 600, 300)


def test_block_shape_edge_counts_ties_dual_and_l1():
    shape = O.BlockShape(2, 2, 2, taps=9)
    W = inputs.normal_weights(16, 144, 0.02, 910)
    for up, pp in [(0, 0), (1000, 0), (1000, 1000), (1000, 999), (500, 0), (3, 3)]:
        check_shape(W, shape, up, pp)
    U = inputs.normal_weights(16, 144, 0.005, 911)
    check_shape(W, shape, 700, 200, U=U)
    check_shape(W, shape, 700, 200, prune_key=1)
    check_shape(W, shape, 700, 200, U=U, admm=True)
    check_shape(W, shape, 700, 200, prune_key=1, admm=True)
    # exact ties: identical blocks and whole zero blocks
    W2 = inputs.normal_weights(2, 36, 0.02, 912).repeat(8, 4).contiguous()
    W2[4:6, :] = 0.0
    check_shape(W2, shape, 600, 300)
    check_shape(W2, O.BlockShape(2, 2), 600, 300)


def test_block_shape_idempotent_on_device():
    shape = O.BlockShape(2, 2)
    W = inputs.normal_weights(128, 128, 0.02, 913)
    desc, bufs, Wd, p = check_shape(W, shape, 600, 300)
    Q1 = bufs.Q.clone().reshape(128, 128).cpu()
    desc2, bufs2, _, p2 = check_shape(Q1, shape, 600, 300)
    assert torch.equal(bufs2.Q.cpu().view(torch.int32), Q1.reshape(-1).view(torch.int32))


def test_2x2_blocks_pack_and_gemm():
    """A 2x2-unified 1024 x 256 weight through mwu_pack (every block becomes two per-row runs that
    share its magnitude) and mwu_gemm / mwu_gemm_ws."""
    shape = O.BlockShape(2, 2)
    rows, cols, M = 1024, 256, 1500
    W = inputs.normal_weights(rows, cols, 0.02, 920)
    desc, bufs, Wd, p = check_shape(W, shape, 750, 500)
    packed = torch.empty(B.mwu_packed_bytes(desc), dtype=torch.uint8, device="cuda")
    bufs.pack(Wd, packed=packed)
    torch.cuda.synchronize()
    assert int(bufs.dev_status.item()) == 0
    What = O.decoded_weights(p)
    assert np.array_equal(decoded_on_gpu(desc, bufs, packed), What)
    X = inputs.normal_activations_bf16((M, cols), 921)
    ref = O.gemm(X.to(torch.float64).numpy(), What)
    for ws_bytes in (B.mwu_gemm_workspace_bytes(desc, M), 0):
        ws = torch.empty(ws_bytes, dtype=torch.uint8, device="cuda") if ws_bytes else None
        for y_dtype, tol in ((1, 1e-5), (0, 2e-3)):
            Y = torch.full((M, rows), float("nan"), dtype=torch.float32 if y_dtype else torch.bfloat16, device="cuda")
            B.mwu_gemm_ws(desc, packed, X.cuda(), M, cols, Y, rows, y_dtype, ws, bufs.dev_status)
            torch.cuda.synchronize()
            assert int(bufs.dev_status.item()) == 0
            fro, mx = errors(Y.float().cpu().numpy(), ref)
            assert fro <= tol and mx <= 1e-2, (ws_bytes, y_dtype, fro, mx)


def test_2x2x2_blocks_convolution_on_dense_weights():
    """A 2x2x2-unified 3x3 convolution weight (128 filters, 128 channels): no packed form, so Q is
    rounded to bf16 (device memory plumbing) and multiplied by mwu_conv_dense."""
    shape = O.BlockShape(2, 2, 2, taps=9)
    rows, cin, n, h, w = 128, 128, 4, 14, 14
    W = inputs.normal_weights(rows, cin * 9, 0.05, 930)
    desc, bufs, Wd, p = check_shape(W, shape, 600, 300)
    assert B.mwu_packed_bytes(desc) == 0                       # this shape has no packed form
    What = O.decoded_weights(p)
    Wbf = bufs.Q.reshape(rows, cin * 9).to(torch.bfloat16)
    assert np.array_equal(Wbf.to(torch.float64).cpu().numpy(), What)
    x = inputs.normal_activations_bf16((n, cin, h, w), 931)
    ref = O.conv2d_direct(x.to(torch.float64).numpy(), What, 3, 3, 1, 1)
    ws = torch.empty(B.mwu_conv_dense_workspace_bytes(rows, n, cin, h, w, 3, 3, 1, 1), dtype=torch.uint8, device="cuda")
    assert ws.numel() > 0
    for y_dtype, tol in ((1, 1e-5), (0, 2e-3)):
        Y = torch.full((n, rows, h, w), float("nan"), dtype=torch.float32 if y_dtype else torch.bfloat16, device="cuda")
        B.mwu_conv_dense(rows, Wbf, cin * 9, x.cuda(), n, cin, h, w, 3, 3, 1, 1, Y, y_dtype, ws, bufs.dev_status)
        torch.cuda.synchronize()
        assert int(bufs.dev_status.item()) == 0
        fro, mx = errors(Y.float().cpu().numpy(), ref)
        assert fro <= tol and mx <= 1e-2, (y_dtype, fro, mx)
    # the same weights through the dense GEMM entry point on the lowered matrix (a 1x1 view: M pixels x K)
    Xm = inputs.normal_activations_bf16((300, cin * 9), 932)
    Y = torch.empty((300, rows), dtype=torch.float32, device="cuda")
    B.mwu_gemm_dense(rows, cin * 9, Wbf, cin * 9, Xm.cuda(), 300, cin * 9, Y, rows, 1, bufs.dev_status)
    torch.cuda.synchronize()
    assert errors(Y.cpu().numpy(), O.gemm(Xm.to(torch.float64).numpy(), What))[0] <= 1e-5


def test_shape_descriptors_are_validated():
    assert B.mwu_project_workspace_bytes(shaped_desc(64, 64, O.BlockShape(2, 3), 10, 5)) == 0       # rows of a block
    assert B.mwu_project_workspace_bytes(shaped_desc(63, 64, O.BlockShape(2, 2), 10, 5)) == 0       # rows % 2
    assert B.mwu_project_workspace_bytes(shaped_desc(64, 64, O.BlockShape(16, 2), 10, 5)) == 0      # 32 weights
    assert B.mwu_project_workspace_bytes(shaped_desc(64, 63, O.BlockShape(2, 2, 2, taps=9), 10, 5)) == 0
    assert B.mwu_project_workspace_bytes(shaped_desc(64, 72, O.BlockShape(2, 2, 2, taps=9), 10, 5)) > 0
    d = shaped_desc(64, 72, O.BlockShape(2, 2, 2, taps=9), 64 * 4 * 5 // 2 + 1, 0)                   # k_unify > blocks
    assert B.mwu_project_workspace_bytes(d) == 0

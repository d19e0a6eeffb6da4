"""GPU parity: mwu_gemm / mwu_conv_implicit through the C ABI against the CPU checker.

Tolerances: bf16 output -- relative Frobenius error <= 2e-3 and max element error
<= 1e-2 * max|y| (output rounding alone is about 1.5e-3); fp32 output -- 1e-5 relative
Frobenius, so that an indexing or decode mistake cannot hide under output rounding.
"""
import numpy as np
import pytest
import torch

import packed_format as F
from oracle import mwu_oracle as O
from paper_2106_08301_b200 import binding as B
from paper_2106_08301_b200 import inputs

pytestmark = pytest.mark.gpu


def project_and_pack(W, b, ku, kp):
    rows, cols = W.shape
    desc = B.make_desc(rows, cols, b, ku, kp)
    bufs = B.ProjectionBuffers(desc, want_q=False)
    Wd = W.cuda().contiguous()
    bufs.project(Wd)
    packed = bufs.pack(Wd)
    torch.cuda.synchronize()
    assert int(bufs.dev_status.item()) == 0
    p = O.project(W.numpy(), b, ku, kp)
    return desc, bufs, packed, p


def errors(Y, ref):
    Y = Y.astype(np.float64)
    fro = np.linalg.norm(Y - ref) / max(np.linalg.norm(ref), 1e-300)
    mx = np.abs(Y - ref).max() / max(np.abs(ref).max(), 1e-300)
    return fro, mx


def run_gemm(desc, bufs, packed, X, y_dtype, ldy=None):
    M = X.shape[0]
    N = desc.rows
    ldy = ldy or N
    Y = torch.full((M, ldy), float("nan"), dtype=torch.float32 if y_dtype else torch.bfloat16, device="cuda")
    Xd = X.cuda().contiguous()
    B.mwu_gemm(desc, packed, Xd, M, X.shape[1], Y, ldy, y_dtype, bufs.dev_status)
    torch.cuda.synchronize()
    assert int(bufs.dev_status.item()) == 0
    return Y.float().cpu().numpy()[:, :N]


def check_gemm(W, b, ku, kp, M, seed=0):
    desc, bufs, packed, p = project_and_pack(W, b, ku, kp)
    X = inputs.normal_activations_bf16((M, W.shape[1]), 4242 + seed)
    What = O.decoded_weights(p, b)
    ref = O.gemm(X.to(torch.float64).numpy(), What)
    Y32 = run_gemm(desc, bufs, packed, X, 1)
    fro, mx = errors(Y32, ref)
    assert fro <= 1e-5, (fro, mx)
    Y16 = run_gemm(desc, bufs, packed, X, 0)
    fro, mx = errors(Y16, ref)
    assert fro <= 2e-3 and mx <= 1e-2, (fro, mx)
    return desc, bufs, packed, p


def test_gemm_config1_linear():
    wl = inputs.WORKLOADS["c1_linear"]
    Mb = wl.n_blocks
    check_gemm(wl.weights(), wl.block, B.mwu_count_from_permille(Mb, wl.unified_permille),
               B.mwu_count_from_permille(Mb, wl.pruned_permille), wl.m)


@pytest.mark.parametrize("b", [2, 4, 8, 16])
def test_gemm_block_widths_and_ragged_shapes(b):
    # N = 384 -> three 128-row weight tiles (an odd count: last CTA tile has one record);
    # M = 300 -> ragged last row tile; K = 192 -> three stages
    W = inputs.normal_weights(384, 192, 0.02, 50 + b)
    Mb = W.numel() // b
    check_gemm(W, b, Mb * 6 // 10, Mb * 3 // 10, 300, seed=b)


def test_gemm_ragged_weight_rows():
    W = inputs.normal_weights(200, 128, 0.02, 61)       # N not a multiple of 128, single CTA tile
    Mb = W.numel() // 8
    check_gemm(W, 8, Mb // 2, Mb // 4, 130)
    W = inputs.normal_weights(72, 64, 0.02, 62)         # one record, N = 72
    check_gemm(W, 4, 100, 50, 5)


def test_gemm_all_classes_degenerate():
    W = inputs.normal_weights(256, 256, 0.02, 63)
    Mb = W.numel() // 16
    check_gemm(W, 16, 0, 0, 64)            # all dense: an ordinary GEMM
    check_gemm(W, 16, Mb, 0, 64)           # all unified
    check_gemm(W, 16, Mb, Mb, 64)          # all pruned: exactly zero, every stage skipped
    desc, bufs, packed, p = project_and_pack(W, 16, Mb, Mb)
    X = inputs.normal_activations_bf16((64, 256), 1)
    assert np.all(run_gemm(desc, bufs, packed, X, 0) == 0)


def test_gemm_skips_dead_stages_and_slices():
    """Structured pruning: whole 64-column stages and single 16-column slices are zero in every
    row, so the kernel's skip paths run; results must not change."""
    W = inputs.normal_weights(256, 512, 0.02, 64)
    W[:, 64:192] = 0.0                  # stages 1 and 2 dead in every tile
    W[:, 272:288] = 0.0                 # slice 1 of stage 4 dead
    W[:128, 448:512] = 0.0              # stage 7 dead in the first row tile only (not skippable with 2-tile CTAs)
    b = 16
    Mb = W.numel() // b
    n_zero = int((W.reshape(-1, b).abs().sum(dim=1) == 0).sum())
    desc, bufs, packed, p = check_gemm(W, b, n_zero + 500, n_zero, 200)
    rec = F.records(packed.cpu().numpy())
    assert rec[1, 3] == 0 and rec[2, 3] == 0 and rec[8 + 1, 3] == 0 and rec[4, 3] == 0b1101


def test_gemm_output_leading_dimension():
    W = inputs.normal_weights(256, 128, 0.02, 65)
    desc, bufs, packed, p = project_and_pack(W, 8, 2000, 1000)
    X = inputs.normal_activations_bf16((100, 128), 3)
    ref = O.gemm(X.to(torch.float64).numpy(), O.decoded_weights(p))
    Y = run_gemm(desc, bufs, packed, X, 1, ldy=264)
    assert errors(Y, ref)[0] <= 1e-5


def test_gemm_argument_errors():
    W = inputs.normal_weights(128, 64, 0.02, 66)
    desc, bufs, packed, p = project_and_pack(W, 4, 100, 50)
    X = inputs.normal_activations_bf16((16, 64), 3).cuda()
    Y = torch.empty((16, 128), dtype=torch.bfloat16, device="cuda")
    assert B.mwu_gemm(desc, packed, X, 16, 60, Y, 128, 0, bufs.dev_status, check=False) == 2   # ldx < cols
    assert B.mwu_gemm(desc, packed, X, 16, 64, Y, 100, 0, bufs.dev_status, check=False) == 2   # ldy < rows
    assert B.mwu_gemm(desc, packed, X, 16, 64, Y, 132, 0, bufs.dev_status, check=False) == 3   # ldy % 8
    assert B.mwu_gemm(desc, packed, X, 16, 64, Y, 128, 7, bufs.dev_status, check=False) == 1
    assert B.mwu_gemm(desc, packed, X, 0, 64, Y, 128, 0, bufs.dev_status, check=False) == 0    # no-op


def test_gemm_config3_shape_reduced_rows():
    """1x1 conv as GEMM (K = 256, N = 1024) on a reduced M, every output compared (the full
    M = 200704 runs in test_gpu_decode_once.py on sampled rows)."""
    wl = inputs.WORKLOADS["c3_conv1x1"]
    Mb = wl.n_blocks
    check_gemm(wl.weights(), wl.block, B.mwu_count_from_permille(Mb, wl.unified_permille),
               B.mwu_count_from_permille(Mb, wl.pruned_permille), 1000)


def conv_case(W, b, ku, kp, x, kh, kw, stride, pad, expect_ws=None):
    """Both entry points: mwu_conv_implicit (decode fused into the kernel) and mwu_conv_implicit_ws
    (weights expanded once into a workspace; falls back to the first for shapes it does not serve)."""
    desc, bufs, packed, p = project_and_pack(W, b, ku, kp)
    n, c, h, w = x.shape
    oh = (h + 2 * pad - kh) // stride + 1
    ow = (w + 2 * pad - kw) // stride + 1
    ref = O.conv2d_direct(x.to(torch.float64).numpy(), O.decoded_weights(p), kh, kw, stride, pad)
    xd = x.cuda().contiguous()
    ws_bytes = B.mwu_conv_workspace_bytes(desc, n, c, h, w, kh, kw, stride, pad)
    if expect_ws is not None:
        assert (ws_bytes > 0) == expect_ws
    ws = torch.empty(ws_bytes, dtype=torch.uint8, device="cuda") if ws_bytes else None
    for use_ws in (False, True):
        for y_dtype, tol in [(1, 1e-5), (0, 2e-3)]:
            Y = torch.full((n, W.shape[0], oh, ow), float("nan"),
                           dtype=torch.float32 if y_dtype else torch.bfloat16, device="cuda")
            if use_ws:
                B.mwu_conv_implicit_ws(desc, packed, xd, n, c, h, w, kh, kw, stride, pad, Y, y_dtype, ws,
                                       bufs.dev_status)
            else:
                B.mwu_conv_implicit(desc, packed, xd, n, c, h, w, kh, kw, stride, pad, Y, y_dtype, bufs.dev_status)
            torch.cuda.synchronize()
            assert int(bufs.dev_status.item()) == 0
            fro, mx = errors(Y.float().cpu().numpy(), ref)
            assert fro <= tol and mx <= 1e-2, (use_ws, y_dtype, fro, mx)
    return desc, bufs, packed, p, xd, ref


def test_conv_small_cases():
    # 3x3 s1 p1, K = 64*9 = 576; M = 2*9*7 = 126 (ragged)
    W = inputs.normal_weights(128, 576, 0.05, 70)
    x = inputs.normal_activations_bf16((2, 64, 9, 7), 71)
    Mb = W.numel() // 4
    conv_case(W, 4, Mb * 6 // 10, Mb * 3 // 10, x, 3, 3, 1, 1)
    # stride 2, no padding, 256 filters (two records per CTA tile), b = 16
    W = inputs.normal_weights(256, 576, 0.05, 72)
    Mb = W.numel() // 16
    conv_case(W, 16, Mb // 2, Mb // 4, x, 3, 3, 2, 0)
    # 1x1 convolution equals a GEMM over channels
    W = inputs.normal_weights(128, 64, 0.05, 73)
    conv_case(W, 8, 300, 100, x, 1, 1, 1, 0)


@pytest.mark.parametrize("filters,cin,h,w,k,pad,b", [(128, 64, 13, 12, 3, 1, 4),     # second tile of an image has 3 of 10 rows
                                                     (256, 128, 28, 28, 3, 1, 16),   # two filter tiles, two channel chunks, 4-row tiles
                                                     (200, 64, 9, 11, 5, 2, 8),      # 5x5 taps, filters ragged inside a tile
                                                     (128, 64, 10, 10, 3, 0, 2),     # no padding: 8x8 output
                                                     (128, 192, 6, 40, 1, 0, 8)])    # 1x1, three channel chunks, 3-row tiles
def test_conv_workspace_path_shapes(filters, cin, h, w, k, pad, b):
    W = inputs.normal_weights(filters, cin * k * k, 0.05, 740 + filters + cin + k)
    x = inputs.normal_activations_bf16((3, cin, h, w), 741 + h)
    Mb = W.numel() // b
    conv_case(W, b, Mb * 6 // 10, Mb * 3 // 10, x, k, k, 1, pad, expect_ws=True)


def test_conv_workspace_path_declines_other_shapes():
    x = inputs.normal_activations_bf16((2, 64, 9, 7), 71)
    W = inputs.normal_weights(128, 576, 0.05, 72)
    d = B.make_desc(128, 576, 16, 1000, 500)
    assert B.mwu_conv_workspace_bytes(d, 2, 64, 9, 7, 3, 3, 2, 0) == 0          # stride 2
    assert B.mwu_conv_workspace_bytes(d, 2, 64, 9, 200, 3, 3, 1, 1) == 0        # 200 output pixels per row
    assert B.mwu_conv_workspace_bytes(d, 2, 64, 9, 7, 3, 3, 1, 1) > 0
    d2 = B.make_desc(128, 288, 16, 500, 200)                                     # 32 channels
    assert B.mwu_conv_workspace_bytes(d2, 2, 32, 9, 7, 3, 3, 1, 1) == 0


def test_bounded_wait_runs_out_and_the_context_stays_usable():
    """Every wait of a kernel on its own barriers has a limit.  Here the producer of the convolution
    kernel leaves one stage's loads out (a barrier that nothing completes) and the limit is cut to
    about a millisecond: the kernel must come back by itself with MWU_DEV_TIMEOUT set, and the next
    call on the same stream must give the right result."""
    W = inputs.normal_weights(128, 576, 0.05, 760)
    x = inputs.normal_activations_bf16((4, 64, 8, 8), 761)
    Mb = W.numel() // 4
    desc, bufs, packed, p = project_and_pack(W, 4, Mb // 2, Mb // 4)
    ref = O.conv2d_direct(x.to(torch.float64).numpy(), O.decoded_weights(p), 3, 3, 1, 1)
    xd = x.cuda()
    ws = torch.empty(B.mwu_conv_workspace_bytes(desc, 4, 64, 8, 8, 3, 3, 1, 1), dtype=torch.uint8, device="cuda")
    assert ws.numel() > 0
    Y = torch.zeros((4, 128, 8, 8), dtype=torch.float32, device="cuda")
    B.mwu_debug_conv_wait(2_000_000, 3)                  # ~1 ms; the fourth stage of every CTA never arrives
    try:
        B.mwu_conv_implicit_ws(desc, packed, xd, 4, 64, 8, 8, 3, 3, 1, 1, Y, 1, ws, bufs.dev_status)
        torch.cuda.synchronize()
    finally:
        B.mwu_debug_conv_wait(0, -1)
    assert int(bufs.dev_status.item()) & B.MWU_DEV_TIMEOUT
    bufs.dev_status.zero_()
    B.mwu_conv_implicit_ws(desc, packed, xd, 4, 64, 8, 8, 3, 3, 1, 1, Y, 1, ws, bufs.dev_status)
    torch.cuda.synchronize()
    assert int(bufs.dev_status.item()) == 0
    assert errors(Y.cpu().numpy(), ref)[0] <= 1e-5


def test_conv_config2():
    wl = inputs.WORKLOADS["c2_conv3x3"]
    Mb = wl.n_blocks
    x = wl.activations()
    n, c, h, w, kh, kw, stride, pad = wl.conv
    conv_case(wl.weights(), wl.block, B.mwu_count_from_permille(Mb, wl.unified_permille),
              B.mwu_count_from_permille(Mb, wl.pruned_permille), x, kh, kw, stride, pad)


@pytest.mark.parametrize("b", [2, 4, 8, 16])
def test_gemm_pair_tiles(b):
    """Shapes that take the two-CTA path: M > 256, an even number of 128-row weight tiles, N a
    multiple of 256; M = 900 leaves a ragged last 512-row tile, K = 320 gives five stages (more
    than the four pipeline slots)."""
    W = inputs.normal_weights(512, 320, 0.02, 80 + b)
    Mb = W.numel() // b
    check_gemm(W, b, Mb * 7 // 10, Mb * 4 // 10, 900, seed=20 + b)


def test_gemm_pair_tiles_dead_stages_and_all_pruned():
    W = inputs.normal_weights(512, 512, 0.02, 90)
    W[:, 128:256] = 0.0                 # stages 2 and 3 dead in every record
    W[:256, 448:464] = 0.0              # one dead slice in the first pair tile only
    b = 16
    Mb = W.numel() // b
    n_zero = int((W.reshape(-1, b).abs().sum(dim=1) == 0).sum())
    check_gemm(W, b, n_zero + 700, n_zero, 1030)
    check_gemm(W, b, Mb, Mb, 600)       # everything pruned: zeros, no MMA issued at all
    check_gemm(W, b, 0, 0, 513)         # everything dense


@pytest.mark.parametrize("K,b", [(256, 8), (192, 16)])
def test_gemm_pair_tiles_resident_weights(K, b):
    """Small reduction, many activation rows: a CTA pair keeps one weight tile in shared memory and
    walks the activation tiles (K = 256 fills the four slots exactly, so decode is skipped after
    the first tile; K = 192 takes the same tile order but re-decodes)."""
    W = inputs.normal_weights(512, K, 0.02, 95 + b)
    Mb = W.numel() // b
    check_gemm(W, b, Mb * 3 // 4, Mb // 2, 77000 + 37, seed=31 + b)

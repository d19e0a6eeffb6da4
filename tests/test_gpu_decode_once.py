"""GPU parity: mwu_decode and the decode-once path of mwu_gemm_ws against the CPU checker.

mwu_decode must reproduce the checker's decoded weights bit for bit (they are bf16 values).
mwu_gemm_ws with a workspace uses the same tolerances as mwu_gemm: fp32 output 1e-5 relative
Frobenius, bf16 output 2e-3 relative Frobenius and 1e-2 * max|y| per element.
"""
import numpy as np
import pytest
import torch

import packed_format as F
from oracle import mwu_oracle as O
from paper_2106_08301_b200 import binding as B
from paper_2106_08301_b200 import inputs
from test_gpu_gemm import errors, project_and_pack
from test_gpu_projection import check_against_oracle, check_pack

pytestmark = pytest.mark.gpu


def decode_on_gpu(desc, bufs, packed, ldw=None):
    n_pad = (desc.rows + 127) // 128 * 128
    ldw = ldw or desc.cols
    Wd = torch.full((n_pad, ldw), float("nan"), dtype=torch.bfloat16, device="cuda")
    B.mwu_decode(desc, packed, Wd, ldw, bufs.dev_status)
    torch.cuda.synchronize()
    assert int(bufs.dev_status.item()) == 0
    return Wd


@pytest.mark.parametrize("b", [2, 4, 8, 16])
def test_decode_matches_checker_bit_for_bit(b):
    W = inputs.normal_weights(200, 192, 0.02, 70 + b)        # 200 rows: the second record tile is padded
    Mb = W.numel() // b
    desc, bufs, packed, p = project_and_pack(W, b, Mb * 6 // 10, Mb * 3 // 10)
    Wd = decode_on_gpu(desc, bufs, packed).float().cpu().numpy().astype(np.float64)
    What = O.decoded_weights(p, b)
    assert np.array_equal(Wd[:200], What)
    assert np.all(Wd[200:] == 0)                              # padding rows are written, as zeros


def test_decode_leading_dimension_and_errors():
    W = inputs.normal_weights(128, 128, 0.02, 75)
    desc, bufs, packed, p = project_and_pack(W, 8, 1200, 600)
    Wd = decode_on_gpu(desc, bufs, packed, ldw=136)
    got = Wd.float().cpu().numpy()
    assert np.array_equal(got[:, :128].astype(np.float64), O.decoded_weights(p, 8))
    assert np.all(np.isnan(got[:, 128:]))                     # nothing written past cols
    assert B.mwu_decode(desc, packed, Wd, 120, bufs.dev_status, check=False) == 2    # ldw < cols
    assert B.mwu_decode(desc, packed, Wd, 132, bufs.dev_status, check=False) == 3    # ldw % 8


def run_gemm_ws(desc, bufs, packed, X, y_dtype, ldy=None, extra_ws=0):
    M, N = X.shape[0], desc.rows
    ldy = ldy or N
    need = B.mwu_gemm_workspace_bytes(desc, M)
    assert need == (N + 127) // 128 * 128 * desc.cols * 2
    ws = torch.empty(need + extra_ws, dtype=torch.uint8, device="cuda")
    Y = torch.full((M, ldy), float("nan"), dtype=torch.float32 if y_dtype else torch.bfloat16, device="cuda")
    B.mwu_gemm_ws(desc, packed, X.cuda().contiguous(), M, X.shape[1], Y, ldy, y_dtype, ws, bufs.dev_status)
    torch.cuda.synchronize()
    assert int(bufs.dev_status.item()) == 0
    return Y.float().cpu().numpy()[:, :N]


def check_gemm_ws(W, b, ku, kp, M, seed=0):
    desc, bufs, packed, p = project_and_pack(W, b, ku, kp)
    X = inputs.normal_activations_bf16((M, W.shape[1]), 5151 + seed)
    ref = O.gemm(X.to(torch.float64).numpy(), O.decoded_weights(p, b))
    fro, mx = errors(run_gemm_ws(desc, bufs, packed, X, 1), ref)
    assert fro <= 1e-5, (fro, mx)
    fro, mx = errors(run_gemm_ws(desc, bufs, packed, X, 0), ref)
    assert fro <= 2e-3 and mx <= 1e-2, (fro, mx)
    return desc, bufs, packed, p, X, ref


@pytest.mark.parametrize("b", [2, 4, 8, 16])
def test_gemm_ws_block_widths_and_ragged_shapes(b):
    # N = 384: three 128-row records, so the last 256-wide tile has one record and the other half
    # of its weight operand is out of range; M = 1100: ragged last 256-row tile; K = 192.
    W = inputs.normal_weights(384, 192, 0.02, 80 + b)
    Mb = W.numel() // b
    check_gemm_ws(W, b, Mb * 6 // 10, Mb * 3 // 10, 1100, seed=b)


def test_gemm_ws_many_tiles_per_pair_and_long_reduction():
    """More tiles than CTA pairs (both accumulator buffers are reused several times) and a
    reduction longer than the six-slot ring."""
    W = inputs.normal_weights(1024, 1024, 0.02, 85)
    Mb = W.numel() // 16
    check_gemm_ws(W, 16, Mb * 8 // 10, Mb * 6 // 10, 256 * 80 + 17)


def test_gemm_ws_ragged_weight_rows_and_ldy():
    W = inputs.normal_weights(200, 128, 0.02, 86)             # N = 200: ragged inside a 32-column chunk
    Mb = W.numel() // 8
    desc, bufs, packed, p, X, ref = check_gemm_ws(W, 8, Mb // 2, Mb // 4, 1030)
    Y = run_gemm_ws(desc, bufs, packed, X, 1, ldy=264, extra_ws=4096)
    assert errors(Y, ref)[0] <= 1e-5


def test_gemm_ws_degenerate_classes_and_dead_stages():
    W = inputs.normal_weights(256, 512, 0.02, 87)
    Mb = W.numel() // 16
    check_gemm_ws(W, 16, 0, 0, 1024)           # all dense
    check_gemm_ws(W, 16, Mb, 0, 1024)          # all unified
    desc, bufs, packed, p = project_and_pack(W, 16, Mb, Mb)   # all pruned: every stage skipped, exact zeros
    X = inputs.normal_activations_bf16((1024, 512), 2)
    assert np.all(run_gemm_ws(desc, bufs, packed, X, 0) == 0)
    W[:, 64:192] = 0.0                  # stages 1 and 2 dead in every row
    W[:, 272:288] = 0.0                 # slice 1 of stage 4 dead
    W[:128, 448:512] = 0.0              # stage 7 dead in the first record only (not skippable)
    n_zero = int((W.reshape(-1, 16).abs().sum(dim=1) == 0).sum())
    check_gemm_ws(W, 16, n_zero + 500, n_zero, 1500)


def test_gemm_ws_falls_back_without_workspace_or_with_a_short_one():
    W = inputs.normal_weights(256, 128, 0.02, 88)
    desc, bufs, packed, p = project_and_pack(W, 8, 2000, 1000)
    assert B.mwu_gemm_workspace_bytes(desc, 0) == 0
    assert B.mwu_gemm_workspace_bytes(desc, 200) == 256 * 128 * 2       # the expanded weights, bf16
    for M in (200, 1024):
        X = inputs.normal_activations_bf16((M, 128), 3)
        ref = O.gemm(X.to(torch.float64).numpy(), O.decoded_weights(p, 8))
        Y = torch.full((M, 256), float("nan"), dtype=torch.float32, device="cuda")
        small = torch.empty(256, dtype=torch.uint8, device="cuda")
        for ws in (None, small):
            B.mwu_gemm_ws(desc, packed, X.cuda(), M, 128, Y, 256, 1, ws, bufs.dev_status)
            torch.cuda.synchronize()
            assert int(bufs.dev_status.item()) == 0
            assert errors(Y.cpu().numpy(), ref)[0] <= 1e-5


def test_gemm_ws_config4_shape_sampled_outputs():
    """The benchmark's launch configuration (16384 x 4096 weight, b = 16, 80 %/60 %, M = 8192):
    sampled output rows against the checker, which projects and decodes the full weight."""
    wl = inputs.WORKLOADS["c4_ffn"]
    ku = B.mwu_count_from_permille(wl.n_blocks, wl.unified_permille)
    kp = B.mwu_count_from_permille(wl.n_blocks, wl.pruned_permille)
    desc, bufs, packed, p = project_and_pack(wl.weights(), wl.block, ku, kp)
    X = wl.activations()
    ws = torch.empty(B.mwu_gemm_workspace_bytes(desc, wl.m), dtype=torch.uint8, device="cuda")
    Y = torch.empty((wl.m, wl.rows), dtype=torch.bfloat16, device="cuda")
    B.mwu_gemm_ws(desc, packed, X.cuda(), wl.m, wl.cols, Y, wl.rows, 0, ws, bufs.dev_status)
    torch.cuda.synchronize()
    assert int(bufs.dev_status.item()) == 0
    rows = [0, 1, 127, 128, 255, 256, 4095, 4096 + 129, 8191]
    ref = O.gemm(X[rows].to(torch.float64).numpy(), O.decoded_weights(p, wl.block))
    fro, mx = errors(Y[rows].float().cpu().numpy(), ref)
    assert fro <= 2e-3 and mx <= 1e-2, (fro, mx)


@pytest.mark.parametrize("pruned_permille", [0, 250, 500, 750, 900])
@pytest.mark.parametrize("b", [2, 4, 8, 16])
def test_gemm_ws_sweep_points_full_size_sampled_outputs(b, pruned_permille):
    """All twenty points of the 4096 x 4096 sweep (block width x pruned fraction) at full size
    (M = 8192), in the configuration the benchmark times: keys, bitmaps, sign plane, u and Q against
    the checker bit for bit, the packed form through mwu_decode, the GEMM on sampled rows."""
    wl = inputs.sweep_workload(b, pruned_permille)
    ku = B.mwu_count_from_permille(wl.n_blocks, wl.unified_permille)
    kp = B.mwu_count_from_permille(wl.n_blocks, wl.pruned_permille)
    desc, bufs, Wd, _, p = check_against_oracle(wl.weights(), b, ku, kp, algos=(B.MWU_ALGO_AUTO,))
    packed = bufs.pack(Wd)
    torch.cuda.synchronize()
    assert int(bufs.dev_status.item()) == 0
    check_pack(desc, bufs, packed, p, b)
    del Wd
    X = wl.activations()
    ws = torch.empty(B.mwu_gemm_workspace_bytes(desc, wl.m), dtype=torch.uint8, device="cuda")
    Y = torch.empty((wl.m, wl.rows), dtype=torch.bfloat16, device="cuda")
    B.mwu_gemm_ws(desc, packed, X.cuda(), wl.m, wl.cols, Y, wl.rows, 0, ws, bufs.dev_status)
    torch.cuda.synchronize()
    assert int(bufs.dev_status.item()) == 0
    rows = [0, 31, 32, 255, 256, 4097, 8191]
    ref = O.gemm(X[rows].to(torch.float64).numpy(), O.decoded_weights(p))
    fro, mx = errors(Y[rows].float().cpu().numpy(), ref)
    assert fro <= 2e-3 and mx <= 1e-2, (fro, mx)


def test_gemm_ws_config3_full_size_sampled_outputs():
    """The 1x1-convolution shape at its full size (M = 200704, K = 256, N = 1024) on the workspace
    path: sampled output rows, among them the first and last row of the matrix and of a tile."""
    wl = inputs.WORKLOADS["c3_conv1x1"]
    ku = B.mwu_count_from_permille(wl.n_blocks, wl.unified_permille)
    kp = B.mwu_count_from_permille(wl.n_blocks, wl.pruned_permille)
    desc, bufs, packed, p = project_and_pack(wl.weights(), wl.block, ku, kp)
    X = wl.activations()
    ws = torch.empty(B.mwu_gemm_workspace_bytes(desc, wl.m), dtype=torch.uint8, device="cuda")
    What = O.decoded_weights(p)
    rows = [0, 1, 127, 128, 255, 256, 257, 511, 512, 100000, 100351, 100352, 200447, 200448, 200702, 200703]
    for y_dtype, tol in ((1, 1e-5), (0, 2e-3)):
        Y = torch.full((wl.m, wl.rows), float("nan"), dtype=torch.float32 if y_dtype else torch.bfloat16,
                       device="cuda")
        B.mwu_gemm_ws(desc, packed, X.cuda(), wl.m, wl.cols, Y, wl.rows, y_dtype, ws, bufs.dev_status)
        torch.cuda.synchronize()
        assert int(bufs.dev_status.item()) == 0
        ref = O.gemm(X[rows].to(torch.float64).numpy(), What)
        fro, mx = errors(Y[rows].float().cpu().numpy(), ref)
        assert fro <= tol and mx <= 1e-2, (y_dtype, fro, mx)
        assert not bool(torch.isnan(Y).any())                 # every output element was written
        del Y


@pytest.mark.parametrize("N,K,M,b", [(504, 256, 40001, 8), (1024, 128, 50000, 16), (304, 384, 38000, 4),
                                     (1104, 64, 20000, 2)])
def test_gemm_ws_short_reduction_many_rows(N, K, M, b):
    """Short reductions with many activation rows (the 1x1-convolution regime: a few k stages per
    tile, hundreds of row tiles).  Ragged N, M and an odd number of 128-row weight tiles."""
    W = inputs.normal_weights(N, K, 0.02, 7000 + N)
    Mb = N * K // b
    check_gemm_ws(W, b, Mb * 7 // 10, Mb * 4 // 10, M, seed=N)


def test_gemm_ws_short_reduction_dead_stage():
    """A 64-column stage that is pruned in every row is skipped (short reduction, many rows)."""
    N, K, b, M = 512, 256, 16, 40000
    W = inputs.normal_weights(N, K, 0.02, 7100)
    W[:, 64:128] = 0.0
    Mb = N * K // b
    desc, bufs, packed, p, X, ref = check_gemm_ws(W, b, Mb // 2, Mb // 4, M, seed=3)
    rec = F.records(packed.cpu().numpy())
    assert rec[1, 3] == 0                                    # stage 1 of the first row tile is dead

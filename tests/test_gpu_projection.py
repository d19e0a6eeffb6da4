"""GPU parity: mwu_project / mwu_pack through the C ABI against the CPU checker."""
import numpy as np
import pytest
import torch

import packed_format as F
from oracle import mwu_oracle as O
from paper_2106_08301_b200 import binding as B
from paper_2106_08301_b200 import inputs

pytestmark = pytest.mark.gpu


def decoded_on_gpu(desc, bufs, packed):
    """mwu_decode of a packed buffer: bf16 [rows][cols] as fp64 (padding rows checked to be zero)."""
    n_pad = (desc.rows + 127) // 128 * 128
    Wd = torch.full((n_pad, desc.cols), float("nan"), dtype=torch.bfloat16, device="cuda")
    B.mwu_decode(desc, packed, Wd, desc.cols, bufs.dev_status)
    torch.cuda.synchronize()
    assert int(bufs.dev_status.item()) == 0
    assert not bool(Wd[desc.rows:].any())
    return Wd[:desc.rows].to(torch.float64).cpu().numpy()


def check_pack(desc, bufs, packed, p, b):
    """mwu_pack judged without any knowledge of its layout: what mwu_decode reads back from the
    packed bytes equals the checker's decoded weights bit for bit, and the header carries the
    class counts of the projection."""
    assert np.array_equal(decoded_on_gpu(desc, bufs, packed), O.decoded_weights(p))
    h = F.parse_header(packed[:256].cpu().numpy())
    mb = p.pruned.shape[0]
    assert (h["N"], h["K"], h["b"]) == (desc.rows, desc.cols, b)
    assert h["n_pruned"] == int(p.pruned.sum()) and h["n_unified"] == int(p.unified.sum())
    assert h["n_dense"] == mb - int(p.pruned.sum()) - int(p.unified.sum())
    assert h["total"] == packed.numel() == B.mwu_packed_bytes(desc)


def run_project(W, b, ku, kp, U=None, prune_key=0, want_loss=True, algo=B.MWU_ALGO_AUTO):
    rows, cols = W.shape
    desc = B.make_desc(rows, cols, b, ku, kp, prune_key, algo)
    bufs = B.ProjectionBuffers(desc, want_q=True, want_loss=want_loss)
    Wd = W.cuda().contiguous()
    Ud = U.cuda().contiguous() if U is not None else None
    bufs.project(Wd, Ud)
    torch.cuda.synchronize()
    return desc, bufs, Wd, Ud


def check_against_oracle(W, b, ku, kp, U=None, prune_key=0, algos=None):
    """Both kernel pipelines of mwu_project (one pass with correction, multi pass) against the
    CPU checker; returns the buffers of the last one."""
    p = O.project(W.numpy(), b, ku, kp, U=None if U is None else U.numpy(),
                  prune_key="l1" if prune_key else "l2sq")
    out = None
    for algo in (algos or (B.MWU_ALGO_MULTI_PASS, B.MWU_ALGO_ONE_PASS)):
        out = compare_with(p, W, b, ku, kp, U, prune_key, algo)
    return out + (p,)


def compare_with(p, W, b, ku, kp, U, prune_key, algo):
    desc, bufs, Wd, Ud = run_project(W, b, ku, kp, U, prune_key, algo=algo)
    assert int(bufs.dev_status.item()) == 0
    # keys: bit-exact fp64
    lu = bufs.loss_u.cpu().numpy()
    lp = bufs.loss_p.cpu().numpy()
    assert np.array_equal(lu.view(np.uint64), p.stats.L_u.view(np.uint64))
    kp_ref = p.stats.S if prune_key else p.stats.L_p
    assert np.array_equal(lp.view(np.uint64), kp_ref.view(np.uint64))
    # selection, sign plane: bit-exact
    pb = bufs.pruned_bitmap.cpu().numpy().view(np.uint32)
    ub = bufs.unified_bitmap.cpu().numpy().view(np.uint32)
    assert np.array_equal(pb, O.bitmap_words(p.pruned))
    assert np.array_equal(ub, O.bitmap_words(p.unified))
    sb = bufs.sign_bits.cpu().numpy().view(np.uint32)
    assert np.array_equal(sb, O.bitmap_words(p.sign.reshape(-1)))
    # unified values within 1e-6 relative (they are in fact the same fp32 numbers)
    u = bufs.u.cpu().numpy()
    assert np.allclose(u, p.u, rtol=1e-6, atol=0)
    assert np.array_equal(u, p.u)
    Q = bufs.Q.cpu().numpy().reshape(W.shape)
    assert np.array_equal(Q.view(np.uint32), p.Q.view(np.uint32))
    return desc, bufs, Wd, Ud


@pytest.mark.parametrize("b", [2, 4, 8, 16])
@pytest.mark.parametrize("rows,cols", [(64, 64), (96, 160), (7, 48), (300, 1008)])
def test_projection_parity_small(b, rows, cols):
    W = inputs.normal_weights(rows, cols, 0.02, 1234 + b)
    Mb = rows * cols // b
    check_against_oracle(W, b, O.count_from_permille(Mb, 600), O.count_from_permille(Mb, 300))


@pytest.mark.parametrize("ku,kp", [(0, 0), (1, 0), (1, 1), (2048, 0), (2048, 2048), (4096, 1),
                                   (4096, 4096), (4096, 4095), (3000, 2999)])
def test_projection_edge_counts(ku, kp):
    W = inputs.normal_weights(64, 256, 0.02, 77)
    check_against_oracle(W, 4, ku, kp)


def test_projection_l1_key_and_dual():
    W = inputs.normal_weights(128, 256, 0.02, 5)
    U = inputs.normal_weights(128, 256, 0.004, 6)
    Mb = 128 * 256 // 8
    check_against_oracle(W, 8, Mb // 2, Mb // 4, U=U)
    check_against_oracle(W, 8, Mb // 2, Mb // 4, prune_key=1)


def test_projection_ties_zeros_and_negative_zero():
    g = torch.Generator().manual_seed(3)
    W = inputs.normal_weights(64, 128, 0.02, 9)
    W[:, 0:32] = 0.0                 # whole zero blocks: exact ties at key 0
    W[5, 0:4] = -0.0
    W[:, 64:96] = W[0:1, 64:96]      # identical blocks in every row
    W[:, 96:128] = 0.5 * torch.sign(torch.randn(64, 32, generator=g))   # equal magnitudes: L_u == 0
    for b in (4, 16):
        Mb = W.numel() // b
        check_against_oracle(W, b, Mb * 3 // 4, Mb // 8)
        check_against_oracle(W, b, Mb // 8, Mb // 16)


def test_projection_idempotent_on_device():
    W = inputs.normal_weights(256, 256, 0.02, 11)
    b = 8
    Mb = W.numel() // b
    ku, kp = Mb * 6 // 10, Mb * 3 // 10
    desc, bufs, Wd, _, p = check_against_oracle(W, b, ku, kp)
    Q1 = bufs.Q.clone().reshape(256, 256)
    # projecting the projection: massive exact ties (all pruned blocks 0, all unified L_u = 0)
    desc2, bufs2, _, _, p2 = check_against_oracle(Q1.cpu(), b, ku, kp)
    assert torch.equal(bufs2.Q.view(torch.int32), Q1.reshape(-1).view(torch.int32))


def test_projection_large_tie_group_refinement():
    """All blocks identical: the threshold is decided by block index alone."""
    blk = torch.tensor([0.5, -0.25, 0.125, 1.0])
    W = blk.repeat(256 * 64).reshape(256, 256).contiguous()
    check_against_oracle(W, 4, 9000, 5000)


def test_nonfinite_sets_status():
    W = inputs.normal_weights(64, 64, 0.02, 1)
    W[3, 7] = float("inf")
    desc, bufs, _, _ = run_project(W, 4, 100, 50, want_loss=False)
    assert int(bufs.dev_status.item()) & B.MWU_DEV_NONFINITE


@pytest.mark.parametrize("name", ["c1_linear", "c2_conv3x3", "c3_conv1x1", "c4_ffn"])
def test_projection_and_pack_parity_configs(name):
    """The four named workloads at full size, both kernel pipelines: keys, bitmaps, sign plane, u
    and Q bit for bit against the checker; the packed form through mwu_decode."""
    wl = inputs.WORKLOADS[name]
    W = wl.weights()
    Mb = wl.n_blocks
    ku = B.mwu_count_from_permille(Mb, wl.unified_permille)
    kp = B.mwu_count_from_permille(Mb, wl.pruned_permille)
    assert ku == O.count_from_permille(Mb, wl.unified_permille)
    assert kp == O.count_from_permille(Mb, wl.pruned_permille)
    desc, bufs, Wd, _, p = check_against_oracle(W, wl.block, ku, kp)
    packed = bufs.pack(Wd)
    torch.cuda.synchronize()
    assert int(bufs.dev_status.item()) == 0
    check_pack(desc, bufs, packed, p, wl.block)


@pytest.mark.parametrize("b", [4, 16])
def test_projection_size_sweep_point_both_pipelines(b):
    """One size of the projection sweep (2^24 weights, 50 % / 25 %) through the one-pass and the
    multi-pass pipeline: both must give the checker's bits."""
    rows, cols = inputs.projection_sweep_shape(24)
    W = inputs.normal_weights(rows, cols, 0.02, inputs.seed_for(5, 924))
    Mb = rows * cols // b
    check_against_oracle(W, b, O.count_from_permille(Mb, 500), O.count_from_permille(Mb, 250),
                         algos=(B.MWU_ALGO_ONE_PASS, B.MWU_ALGO_MULTI_PASS))


@pytest.mark.parametrize("b,rows,cols", [(2, 100, 128), (4, 130, 64), (8, 257, 192), (16, 128, 256)])
def test_pack_ragged_rows(b, rows, cols):
    W = inputs.normal_weights(rows, cols, 0.02, 99 + b)
    Mb = rows * cols // b
    desc, bufs, Wd, _, p = check_against_oracle(W, b, Mb * 7 // 10, Mb * 4 // 10)
    packed = bufs.pack(Wd)
    torch.cuda.synchronize()
    assert int(bufs.dev_status.item()) == 0
    check_pack(desc, bufs, packed, p, b)


def test_pack_with_dual_and_structured_pruning():
    rows, cols, b = 256, 256, 16
    W = inputs.normal_weights(rows, cols, 0.02, 21)
    U = inputs.normal_weights(rows, cols, 0.002, 22)
    W[:, 64:128] = 0.0
    U[:, 64:128] = 0.0               # a whole 64-column stage is zero in every row
    Mb = rows * cols // b
    desc, bufs, Wd, Ud, p = check_against_oracle(W, b, Mb // 2, Mb // 4, U=U)
    packed = bufs.pack(Wd, Ud)
    torch.cuda.synchronize()
    check_pack(desc, bufs, packed, p, b)
    rec = F.records(packed.cpu().numpy())
    assert rec[1, 3] == 0 and rec[5, 3] == 0          # stage 1 of both row tiles is dead
    assert rec[0, 3] == 0xF


@pytest.mark.parametrize("name,b,rows,cols", [("c1_linear", 0, 0, 0), ("c2_conv3x3", 0, 0, 0), ("ragged", 4, 130, 64),
                                              ("ragged", 16, 200, 128), ("ragged", 2, 100, 128)])
def test_packed_bytes_follow_the_documented_format(name, b, rows, cols):
    """Regression of the file format (not a parity claim): the bytes mwu_pack writes are the ones
    the format description in the header file leads to, as restated by tests/packed_format.py."""
    if name == "ragged":
        W = inputs.normal_weights(rows, cols, 0.02, 199 + b)
        Mb = rows * cols // b
        ku, kp = Mb * 7 // 10, Mb * 4 // 10
    else:
        wl = inputs.WORKLOADS[name]
        W, b = wl.weights(), wl.block
        ku = B.mwu_count_from_permille(wl.n_blocks, wl.unified_permille)
        kp = B.mwu_count_from_permille(wl.n_blocks, wl.pruned_permille)
    desc, bufs, Wd, _ = run_project(W, b, ku, kp, want_loss=False)
    packed = bufs.pack(Wd)
    torch.cuda.synchronize()
    assert int(bufs.dev_status.item()) == 0
    p = O.project(W.numpy(), b, ku, kp)
    assert np.array_equal(packed.cpu().numpy(), F.write(p, b))


@pytest.mark.parametrize("b,rows,cols,permille", [(16, 1000, 4112, (800, 600)), (4, 517, 1028, (500, 250)),
                                                  (2, 300, 1002, (350, 250)), (8, 2048, 1024, (1000, 900)),
                                                  (8, 640, 1032, (100, 0)), (16, 777, 2064, (700, 700))])
def test_projection_parity_medium_auto(b, rows, cols, permille):
    """Sizes above the switch to the one-pass pipeline (default algo), ragged against every tile."""
    W = inputs.normal_weights(rows, cols, 0.02, 4321 + b)
    Mb = rows * cols // b
    assert Mb >= 32768
    check_against_oracle(W, b, O.count_from_permille(Mb, permille[0]), O.count_from_permille(Mb, permille[1]),
                         algos=(B.MWU_ALGO_AUTO,))


def test_projection_medium_reprojection_falls_back():
    """Projecting a projected tensor: thousands of exactly equal keys (0 for pruned blocks and for
    the L_u of unified ones), so no sample window can isolate the threshold and the one-pass
    pipeline must hand over to the multi-pass kernels."""
    W = inputs.normal_weights(512, 2048, 0.02, 17)
    b = 16
    Mb = W.numel() // b
    ku, kp = Mb * 8 // 10, Mb * 6 // 10
    desc, bufs, Wd, _, p = check_against_oracle(W, b, ku, kp, algos=(B.MWU_ALGO_AUTO,))
    Q1 = bufs.Q.clone().reshape(512, 2048).cpu()
    desc2, bufs2, _, _, p2 = check_against_oracle(Q1, b, ku, kp, algos=(B.MWU_ALGO_AUTO,))
    assert torch.equal(bufs2.Q.cpu().view(torch.int32), Q1.reshape(-1).view(torch.int32))


def test_projection_one_pass_with_dual_and_l1():
    W = inputs.normal_weights(512, 1024, 0.02, 31)
    U = inputs.normal_weights(512, 1024, 0.004, 32)
    Mb = 512 * 1024 // 4
    check_against_oracle(W, 4, Mb * 6 // 10, Mb * 3 // 10, U=U, algos=(B.MWU_ALGO_AUTO,))
    check_against_oracle(W, 4, Mb * 6 // 10, Mb * 3 // 10, prune_key=1, algos=(B.MWU_ALGO_AUTO,))


def test_projection_many_blocks_wide_histogram():
    """More than 8 Mi blocks: both pipelines switch to the 65536-bin window histogram (64 bins per
    thread in the threshold search) and the candidate list holds several hundred thousand entries."""
    rows, cols, b = 2050, 8192, 2
    W = inputs.normal_weights(rows, cols, 0.02, 2050)
    Mb = rows * cols // b
    assert Mb > 8 * 1024 * 1024
    check_against_oracle(W, b, O.count_from_permille(Mb, 350), O.count_from_permille(Mb, 250))


def test_projection_largest_sweep_size_properties():
    """2^28 weights (the largest size of the projection sweep), where the CPU checker is out of
    reach: properties that pin the result at any size.  Class counts are exact; pruned blocks are
    zero, unified blocks carry +-u, other blocks are copied; and the selection is a valid one: no
    pruned block has a larger prune key than a surviving one, no unified block a larger L_u than a
    surviving one that kept its values (keys recomputed here with plain fp64 tensor operations)."""
    rows = cols = 16384
    b = 16
    Mb = rows * cols // b
    ku, kp = O.count_from_permille(Mb, 500), O.count_from_permille(Mb, 250)
    W = inputs.normal_weights(rows, cols, 0.02, inputs.seed_for(5, 928))
    desc, bufs, Wd, _ = run_project(W, b, ku, kp, want_loss=False)
    del W
    assert int(bufs.dev_status.item()) == 0

    def unpack(words):
        bits = (words.view(torch.int32).unsqueeze(1) >> torch.arange(32, device="cuda", dtype=torch.int32)) & 1
        return bits.reshape(-1)[:Mb].bool()

    pruned, unified = unpack(bufs.pruned_bitmap), unpack(bufs.unified_bitmap)
    assert int(pruned.sum()) == kp and int(unified.sum()) == ku - kp and not bool((pruned & unified).any())
    V = Wd.reshape(Mb, b)
    Q = bufs.Q.reshape(Mb, b)
    kept = ~(pruned | unified)
    assert not bool(Q[pruned].any())
    assert torch.equal(Q[kept].view(torch.int32), V[kept].view(torch.int32))
    u = bufs.u
    assert not bool(u[~unified].any())
    assert torch.equal(Q[unified], torch.where(V[unified] < 0, -u[unified, None], u[unified, None]))
    A = V.abs().double()
    Lp = (A * A).sum(1)
    q = A.mean(1, keepdim=True)
    Lu = ((A - q) ** 2).sum(1)
    del A
    assert float(Lp[pruned].max()) <= float(Lp[~pruned].min()) * (1 + 1e-12)
    assert float(Lu[unified].max()) <= float(Lu[kept].min()) * (1 + 1e-12)
    # the unified value is the mean magnitude
    assert torch.allclose(u[unified].double(), q[unified, 0], rtol=1e-6, atol=0)

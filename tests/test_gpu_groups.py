"""GPU parity for grouped pruning (whole groups of rows x columns are pruned; unification stays
block by block): mwu_project / mwu_pack / mwu_gemm_ws through the C ABI against the CPU checker,
bit for bit on everything the projection writes, within the GEMM tolerances on the product."""
import numpy as np
import pytest
import torch

import packed_format as F
from oracle import mwu_oracle as O
from paper_2106_08301_b200 import binding as B
from paper_2106_08301_b200 import inputs
from test_gpu_gemm import errors
from test_gpu_projection import check_pack

pytestmark = pytest.mark.gpu


def project_grouped(W, b, ku, kp, group, U=None, prune_key=0, algo=B.MWU_ALGO_AUTO):
    rows, cols = W.shape
    desc = B.make_desc(rows, cols, b, ku, kp, prune_key, algo, prune_group=group)
    bufs = B.ProjectionBuffers(desc, want_q=True, want_loss=False)
    Wd = W.cuda().contiguous()
    Ud = U.cuda().contiguous() if U is not None else None
    bufs.project(Wd, Ud)
    torch.cuda.synchronize()
    assert int(bufs.dev_status.item()) == 0
    return desc, bufs, Wd, Ud


def check_grouped(W, b, ku, kp, group, U=None, prune_key=0, algos=(B.MWU_ALGO_MULTI_PASS, B.MWU_ALGO_ONE_PASS)):
    p = O.project(W.numpy(), b, ku, kp, U=None if U is None else U.numpy(),
                  prune_key="l1" if prune_key else "l2sq", prune_group=group)
    out = None
    for algo in algos:
        desc, bufs, Wd, Ud = project_grouped(W, b, ku, kp, group, U, prune_key, algo)
        assert np.array_equal(bufs.pruned_bitmap.cpu().numpy().view(np.uint32), O.bitmap_words(p.pruned))
        assert np.array_equal(bufs.unified_bitmap.cpu().numpy().view(np.uint32), O.bitmap_words(p.unified))
        assert np.array_equal(bufs.sign_bits.cpu().numpy().view(np.uint32), O.bitmap_words(p.sign.reshape(-1)))
        assert np.array_equal(bufs.u.cpu().numpy(), p.u)
        assert np.array_equal(bufs.Q.cpu().numpy().reshape(W.shape).view(np.uint32), p.Q.view(np.uint32))
        out = (desc, bufs, Wd, Ud)
    return out + (p,)


def counts(Mb, b, group, unified_permille, pruned_permille):
    per = group[0] * group[1] // b
    kp = O.count_from_permille(Mb, pruned_permille) // per * per
    return O.count_from_permille(Mb, unified_permille), kp


@pytest.mark.parametrize("b", [2, 4, 8, 16])
@pytest.mark.parametrize("group", [(32, 16), (64, 32), (128, 64), (256, 16), (256, 64)])
def test_grouped_projection_parity(b, group):
    rows, cols = 768, 448                      # three 256-row tiles; 448 = 7 x 64 columns
    W = inputs.normal_weights(rows, cols, 0.02, 600 + b + group[0] + group[1])
    Mb = rows * cols // b
    ku, kp = counts(Mb, b, group, 800, 600)
    check_grouped(W, b, ku, kp, group)


def test_grouped_edge_counts_dual_l1_and_ties():
    rows, cols, b, group = 256, 256, 8, (64, 32)
    W = inputs.normal_weights(rows, cols, 0.02, 650)
    Mb = rows * cols // b
    per = group[0] * group[1] // b
    n_groups = Mb // per
    for kg, extra in [(0, 100), (1, 0), (n_groups, 0), (n_groups - 1, per), (n_groups // 2, 0)]:
        check_grouped(W, b, kg * per + extra, kg * per, group)
    U = inputs.normal_weights(rows, cols, 0.004, 651)
    check_grouped(W, b, Mb * 3 // 4, (n_groups // 3) * per, group, U=U)
    check_grouped(W, b, Mb * 3 // 4, (n_groups // 3) * per, group, prune_key=1)
    # identical groups: the group index decides
    W2 = inputs.normal_weights(1, 32, 0.02, 652).repeat(rows, cols // 32).contiguous()
    check_grouped(W2, b, 5 * per + 17, 5 * per, group)
    # whole groups of zeros (exact ties at key 0) among random ones
    W3 = W.clone()
    W3[64:128, 32:128] = 0.0
    check_grouped(W3, b, 6 * per + 300, 6 * per, group)


def test_grouped_rejects_counts_that_split_a_group():
    d = B.make_desc(256, 256, 8, 4000, 1000, prune_group=(64, 32))      # 1000 is not a multiple of 256
    assert B.mwu_project_workspace_bytes(d) == 0
    d = B.make_desc(250, 256, 8, 4000, 0, prune_group=(64, 32))         # rows % 64 != 0
    assert B.mwu_project_workspace_bytes(d) == 0
    d = B.make_desc(256, 256, 8, 4000, 0, prune_group=(48, 32))         # unsupported extent
    assert B.mwu_project_workspace_bytes(d) == 0
    assert B.mwu_project_workspace_bytes(B.make_desc(256, 256, 8, 4096, 1024, prune_group=(64, 32))) > 0


@pytest.mark.parametrize("group", [(256, 64), (256, 16)])
def test_grouped_medium_one_pass_pack_and_gemm(group):
    """A tensor large enough for the one-pass pipeline; 60 % of the groups pruned, so whole 64-wide
    stages (or 16-wide slices) of the 256-row weight tiles are dead and the GEMM's skip paths run."""
    rows, cols, b, M = 1024, 2048, 16, 1300
    W = inputs.normal_weights(rows, cols, 0.02, 660 + group[1])
    Mb = rows * cols // b
    ku, kp = counts(Mb, b, group, 800, 600)
    desc, bufs, Wd, _, p = check_grouped(W, b, ku, kp, group, algos=(B.MWU_ALGO_AUTO,))
    packed = bufs.pack(Wd)
    torch.cuda.synchronize()
    assert int(bufs.dev_status.item()) == 0
    check_pack(desc, bufs, packed, p, b)
    rec = F.records(packed.cpu().numpy())
    live = rec[:-1, 3]
    dead_slices = int(sum(4 - bin(int(x)).count("1") for x in live))
    assert dead_slices >= int(0.55 * 4 * live.shape[0])          # the pruned groups show up as dead slices
    X = inputs.normal_activations_bf16((M, cols), 661)
    ref = O.gemm(X.to(torch.float64).numpy(), O.decoded_weights(p))
    for ws_bytes in (B.mwu_gemm_workspace_bytes(desc, M), 0):
        ws = torch.empty(ws_bytes, dtype=torch.uint8, device="cuda") if ws_bytes else None
        for y_dtype, tol in ((1, 1e-5), (0, 2e-3)):
            Y = torch.full((M, rows), float("nan"), dtype=torch.float32 if y_dtype else torch.bfloat16, device="cuda")
            B.mwu_gemm_ws(desc, packed, X.cuda(), M, cols, Y, rows, y_dtype, ws, bufs.dev_status)
            torch.cuda.synchronize()
            assert int(bufs.dev_status.item()) == 0
            fro, mx = errors(Y.float().cpu().numpy(), ref)
            assert fro <= tol and mx <= 1e-2, (ws_bytes, y_dtype, fro, mx)

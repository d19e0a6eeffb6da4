"""mwu_project_static: the projection for callers that cannot allocate device memory.

A host that embeds this library may have handed all device memory to its own pool, or may be
past the point where allocations are allowed, so it cannot provide the workspace mwu_project
asks for.  mwu_project_static uses a fixed array inside the library instead.  This test calls
it through the C ABI twice in a row (second call on a different tensor and block width, so
anything left in the shared scratch by the first call would show) and requires the outputs to
be identical, bit for bit, to those of mwu_project and of the CPU checker -- the same bar the
other projection tests use -- and the amount of free device memory to be the same before and
after the second call.  It is collected last on purpose.
"""
import ctypes

import numpy as np
import pytest
import torch

from oracle import mwu_oracle as O
from paper_2106_08301_b200 import binding as B
from paper_2106_08301_b200 import inputs

pytestmark = pytest.mark.gpu


def outputs(desc, device="cuda"):
    mb = desc.rows * desc.cols // desc.block
    n = desc.rows * desc.cols
    return dict(Q=torch.zeros(n, dtype=torch.float32, device=device),
                u=torch.zeros(mb, dtype=torch.float32, device=device),
                pb=torch.zeros((mb + 31) // 32, dtype=torch.int32, device=device),
                ub=torch.zeros((mb + 31) // 32, dtype=torch.int32, device=device),
                sb=torch.zeros((n + 31) // 32, dtype=torch.int32, device=device),
                lu=torch.zeros(mb, dtype=torch.float64, device=device),
                lp=torch.zeros(mb, dtype=torch.float64, device=device),
                st=torch.zeros(1, dtype=torch.int32, device=device))


def project_both_ways(W, b, ku, kp, check_memory=False):
    desc = B.make_desc(W.shape[0], W.shape[1], b, ku, kp)
    Wd = W.cuda().contiguous()
    ref = outputs(desc)
    ws = torch.empty(B.mwu_project_workspace_bytes(desc), dtype=torch.uint8, device="cuda")
    B.mwu_project(desc, Wd, None, ref["Q"], ref["u"], ref["pb"], ref["ub"], ref["sb"], ref["lu"],
                  ref["lp"], ref["st"], ws)
    got = outputs(desc)
    torch.cuda.synchronize()
    free_before = torch.cuda.mem_get_info()[0] if check_memory else None
    B.mwu_project_static(desc, Wd, None, got["Q"], got["u"], got["pb"], got["ub"], got["sb"],
                         got["lu"], got["lp"], got["st"])
    torch.cuda.synchronize()
    if check_memory:
        # the call took no device memory from the driver (the first call on a device may load the
        # library's device image, which holds the scratch array; later calls must not change anything)
        assert torch.cuda.mem_get_info()[0] == free_before
    assert int(ref["st"].item()) == 0 and int(got["st"].item()) == 0
    for name in ("Q", "u", "lu", "lp"):
        a, c = ref[name], got[name]
        view = torch.int32 if a.dtype == torch.float32 else torch.int64
        assert torch.equal(a.view(view), c.view(view)), name
    for name in ("pb", "ub", "sb"):
        assert torch.equal(ref[name], got[name]), name
    # and against the CPU checker
    p = O.project(W.numpy(), b, ku, kp)
    assert np.array_equal(got["Q"].cpu().numpy().reshape(W.shape).view(np.uint32), p.Q.view(np.uint32))
    assert np.array_equal(got["u"].cpu().numpy(), p.u)
    assert np.array_equal(got["pb"].cpu().numpy().view(np.uint32), O.bitmap_words(p.pruned))
    assert np.array_equal(got["ub"].cpu().numpy().view(np.uint32), O.bitmap_words(p.unified))
    assert np.array_equal(got["sb"].cpu().numpy().view(np.uint32), O.bitmap_words(p.sign.reshape(-1)))
    assert np.array_equal(got["lu"].cpu().numpy().view(np.uint64), p.stats.L_u.view(np.uint64))


def test_static_scratch_matches_workspace_version_twice_in_a_row():
    W1 = inputs.normal_weights(512, 1024, 0.02, 4101)
    mb1 = W1.numel() // 16
    project_both_ways(W1, 16, mb1 * 8 // 10, mb1 * 6 // 10)
    W2 = inputs.normal_weights(300, 1008, 0.02, 4102)           # different size and block width
    mb2 = W2.numel() // 4
    project_both_ways(W2, 4, mb2 // 2, mb2 // 4, check_memory=True)


def test_static_scratch_rejects_tensors_beyond_its_limit():
    rows, cols, b = 4096, 4096, 8                               # 2 097 152 blocks > the limit
    assert rows * cols // b > B.MWU_STATIC_MAX_BLOCKS
    desc = B.make_desc(rows, cols, b, 10, 5)
    one = ctypes.c_void_p(256)
    rc = B.lib().mwu_project_static(ctypes.byref(desc), *([one] * 10), None)
    assert rc == 4                                              # MWU_ERR_WORKSPACE, nothing launched

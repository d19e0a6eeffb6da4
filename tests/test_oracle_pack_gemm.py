"""Pins for the CPU checker's packed format, decode, GEMM and convolution."""
import numpy as np
import pytest
import torch

from oracle import mwu_oracle as O

RNG = np.random.default_rng(8301)


def rand_w(n, k, scale=0.02):
    return (RNG.standard_normal((n, k)) * scale).astype(np.float32)


def rand_x_bf16(*shape):
    x = torch.from_numpy(RNG.standard_normal(shape).astype(np.float32)).to(torch.bfloat16)
    return x.to(torch.float64).numpy()


def test_bf16_rne_against_torch_and_ties():
    x = rand_w(64, 64, scale=1.0)
    ours = O.bf16_bits_rne(x)
    ref = torch.from_numpy(x).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(ours, ref)
    # exact ties: 1 + 2^-8 is halfway between 1 and 1 + 2^-7 -> even (1.0);
    # 1 + 3*2^-8 is halfway between 1+2^-7 and 1+2^-6 -> even (1 + 2^-6)
    t = np.array([1.0 + 2.0 ** -8, 1.0 + 3 * 2.0 ** -8, -(1.0 + 2.0 ** -8)], dtype=np.float32)
    back = O.bf16_bits_to_f64(O.bf16_bits_rne(t))
    assert back.tolist() == [1.0, 1.0 + 2.0 ** -6, -1.0]


@pytest.mark.parametrize("b,N,K", [(4, 128, 64), (16, 200, 128), (2, 64, 64), (8, 130, 192)])
def test_pack_decode_round_trip(b, N, K):
    W = rand_w(N, K)
    Mb = N * K // b
    p = O.project(W, b, Mb * 7 // 10, Mb * 4 // 10)
    buf = O.pack(p, b)
    h = O.parse_header(buf)
    assert (h["N"], h["K"], h["b"]) == (N, K, b)
    assert h["n_pruned"] == p.pruned.sum() and h["n_unified"] == p.unified.sum()
    assert h["total"] == buf.shape[0]
    What = O.decode(buf)
    assert np.array_equal(What, O.decoded_weights(p, b))
    # against Q: zero on pruned blocks, bf16(Q) elsewhere
    Qb = O.bf16_bits_to_f64(O.bf16_bits_rne(p.Q))
    assert np.array_equal(What, Qb)
    assert np.all(What.reshape(-1, b)[p.pruned] == 0)


def test_packed_size_accounting():
    """Storage model (Section 3.1 / Table 1): a unified block keeps one magnitude, a pruned
    block nothing, every weight one sign bit; the streams hold exactly that."""
    N, K, b = 256, 256, 8
    W = rand_w(N, K)
    Mb = N * K // b
    ku, kp = Mb * 3 // 4, Mb // 2
    p = O.project(W, b, ku, kp)
    h = O.parse_header(O.pack(p, b))
    assert h["off_dpos"] - h["off_ulist"] >= 8 * (ku - kp)
    assert h["off_ppos"] - h["off_dpay"] >= 2 * b * (Mb - ku)
    assert h["off_ppos"] - h["off_dpay"] < 2 * b * (Mb - ku) + 256
    assert h["total"] - h["off_ppos"] >= 2 * kp
    assert h["n_dense"] == Mb - ku and h["n_plist"] == kp


def test_live_mask_and_padding():
    N, K, b = 100, 128, 16          # 28 padded rows
    W = rand_w(N, K)
    W[:, 16:32] = 0.0               # slice 1 of stage 0 is all-zero in every row
    Mb = N * K // b
    kp = N                          # exactly those blocks are pruned (smallest norm, ties by index)
    p = O.project(W, b, kp, kp)
    assert p.pruned.reshape(N, K // b)[:, 1].all()
    buf = O.pack(p, b)
    h = O.parse_header(buf)
    rec = buf[h["off_rec"]:h["off_rec"] + 16 * 3].view(np.uint32).reshape(3, 4)
    assert rec[0, 3] == 0b1101 and rec[1, 3] == 0b1111
    nb = 64 // b
    assert h["n_plist"] == kp + 28 * (K // b)                           # padding rows pruned
    ppos = buf[h["off_ppos"]:h["off_ppos"] + 2 * h["n_plist"]].view(np.uint16)
    first = ppos[rec[0, 2]:rec[1, 2]]
    slots = [O.tile_offset_inverse(int(o), b) for o in first]
    codes = [r * nb + i for r, i in slots]
    assert len(set(codes)) == len(codes)
    assert set(range(100 * nb, 128 * nb)) <= set(codes)
    assert rec[2].tolist() == [h["n_unified"], h["n_dense"], h["n_plist"], 0]
    assert O.decode(buf).shape == (N, K)


def test_gemm_special_cases():
    N, K, b, M = 128, 128, 4, 24
    W = rand_w(N, K)
    X = rand_x_bf16(M, K)
    Mb = N * K // b
    # all dense: an ordinary matmul with the bf16-rounded weights (library routine)
    p = O.project(W, b, 0, 0)
    What = O.decode(O.pack(p, b))
    ref = torch.from_numpy(X) @ torch.from_numpy(W).to(torch.bfloat16).to(torch.float64).T
    assert np.allclose(O.gemm(X, What), ref.numpy(), rtol=1e-13, atol=1e-15)
    # all pruned: exactly zero
    p = O.project(W, b, Mb, Mb)
    assert np.all(O.gemm(X, O.decode(O.pack(p, b))) == 0)
    # all unified: the shared-partial-sum form agrees with the plain contraction
    p = O.project(W, b, Mb, 0)
    Y1 = O.gemm(X, O.decode(O.pack(p, b)))
    Y2 = O.gemm_shared_partial(X, p, b)
    assert np.allclose(Y1, Y2, rtol=1e-11, atol=1e-14)
    # mixed
    p = O.project(W, b, Mb // 2, Mb // 4)
    Y1 = O.gemm(X, O.decode(O.pack(p, b)))
    Y2 = O.gemm_shared_partial(X, p, b)
    assert np.allclose(Y1, Y2, rtol=1e-11, atol=1e-14)
    # operand orientation: Y is [M][N] = X . W^T (a transposed operand would not even match shapes
    # for M != N, and for the square case gives different numbers)
    Xs = rand_x_bf16(N, K)
    Ws = O.decoded_weights(p, b)
    assert not np.allclose(O.gemm(Xs, Ws), O.gemm(Ws, Xs))
    assert np.allclose(O.gemm(Xs, Ws)[3, 5], (Xs[3] * Ws[5]).sum())


def test_conv_against_library_and_im2col():
    B, C, H, Wd, Oc = 2, 8, 7, 6, 128
    b = 4
    K = C * 9
    Wt = rand_w(Oc, K, scale=0.05)
    Kpad = 128                                   # pack needs K % 64 == 0; check conv on W_hat directly
    p = O.project(Wt, b, Oc * K // b // 2, Oc * K // b // 4)
    What = O.decoded_weights(p, b)
    x = rand_x_bf16(B, C, H, Wd)
    y = O.conv2d_direct(x, What, 3, 3, 1, 1)
    ref = torch.nn.functional.conv2d(torch.from_numpy(x),
                                     torch.from_numpy(What).reshape(Oc, C, 3, 3), padding=1)
    assert np.allclose(y, ref.numpy(), rtol=1e-12, atol=1e-14)
    # explicit im2col + the checker's GEMM
    xp = np.pad(x, ((0, 0), (0, 0), (1, 1), (1, 1)))
    A = np.zeros((B * H * Wd, K))
    for n in range(B):
        for oh in range(H):
            for ow in range(Wd):
                A[(n * H + oh) * Wd + ow] = xp[n, :, oh:oh + 3, ow:ow + 3].reshape(-1)
    Y = O.gemm(A, What).reshape(B, H, Wd, Oc).transpose(0, 3, 1, 2)
    assert np.allclose(y, Y, rtol=1e-12, atol=1e-14)
    # stride 2, no padding
    y2 = O.conv2d_direct(x, What, 3, 3, 2, 0)
    ref2 = torch.nn.functional.conv2d(torch.from_numpy(x),
                                      torch.from_numpy(What).reshape(Oc, C, 3, 3), stride=2)
    assert np.allclose(y2, ref2.numpy(), rtol=1e-12, atol=1e-14)


def test_tile_offset_is_a_bijection_and_matches_the_swizzle():
    for b in (2, 4, 8, 16):
        nb = 64 // b
        pos = np.arange(128 * nb)
        off = O.tile_offset(pos, b)
        g = min(2 * b, 16)          # a block wider than a chunk starts on a chunk boundary
        assert off.min() == 0 and off.max() == 16384 - g
        assert len(set(off.tolist())) == pos.size and np.all(off % g == 0)
        back = [O.tile_offset_inverse(int(o), b) for o in off]
        assert [r * nb + i for r, i in back] == pos.tolist()
    # row 0 is not permuted; row 1 swaps neighbouring chunks; rows 8.. start 1024 bytes later
    assert O.tile_offset(np.array([0, 1, 2, 3]), 16).tolist() == [0, 32, 64, 96]
    assert O.tile_offset(np.array([4, 5]), 16).tolist() == [128 + 16, 128 + 48]
    assert O.tile_offset(np.array([32]), 16).tolist() == [1024]


def test_class_lists_are_dealt_round_robin_over_store_slots():
    N, K, b = 128, 64, 16
    W = rand_w(N, K)
    Mb = N * K // b
    p = O.project(W, b, Mb * 8 // 10, Mb * 6 // 10)
    buf = O.pack(p, b)
    h = O.parse_header(buf)
    ppos = buf[h["off_ppos"]:h["off_ppos"] + 2 * h["n_plist"]].view(np.uint16).astype(int)
    slot = (ppos % 128) // 16
    # same multiset of blocks as the pruned mask
    assert sorted(O.tile_offset(np.flatnonzero(p.pruned), b).tolist()) == sorted(ppos.tolist())
    # the first round holds one entry of every slot present, in ascending slot order
    n_slots = len(set(slot.tolist()))
    assert slot[:n_slots].tolist() == sorted(set(slot.tolist()))
    # inside a slot the entries keep ascending block order
    for sl in set(slot.tolist()):
        pos = [r * 4 + i for r, i in (O.tile_offset_inverse(int(o), b) for o in ppos[slot == sl])]
        assert pos == sorted(pos)
    # while all eight slots still have entries, any 8 consecutive entries hit 8 different slots
    shortest = min(np.bincount(slot, minlength=8))
    full = slot[:8 * shortest].reshape(-1, 8)
    assert all(len(set(row.tolist())) == 8 for row in full)

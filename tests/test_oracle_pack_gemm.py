"""Pins for the CPU checker's storage form, decoded weights, GEMM and convolution."""
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
def test_storage_round_trip(b, N, K):
    W = rand_w(N, K)
    Mb = N * K // b
    p = O.project(W, b, Mb * 7 // 10, Mb * 4 // 10)
    What = O.unpack(O.pack(p), b)
    assert np.array_equal(What, O.decoded_weights(p))
    # against Q: zero on pruned blocks, bf16(Q) elsewhere
    Qb = O.bf16_bits_to_f64(O.bf16_bits_rne(p.Q))
    assert np.array_equal(What, Qb)
    assert np.all(What.reshape(-1, b)[p.pruned] == 0)


def test_decoded_weights_element_by_element():
    """decoded_weights against a plain loop over blocks and weights (no vector indexing)."""
    N, K, b = 6, 16, 4
    W = rand_w(N, K)
    p = O.project(W, b, 14, 6)
    What = O.decoded_weights(p)
    for n in range(N):
        for kb in range(K // b):
            j = n * (K // b) + kb
            for l in range(b):
                w = float(W[n, kb * b + l])
                if p.pruned[j]:
                    expect = 0.0
                elif p.unified[j]:
                    mag = float(torch.tensor(float(p.u[j])).to(torch.bfloat16))
                    expect = -mag if w < 0 else mag
                else:
                    expect = float(torch.tensor(w).to(torch.bfloat16))
                assert What[n, kb * b + l] == expect


def test_storage_size_accounting():
    """Storage model (Section 3.1 / Table 1): a unified block keeps one magnitude and one sign
    bit per weight, a pruned block nothing, the rest their values; the byte string holds exactly
    that (plus the header and the class bitmaps)."""
    N, K, b = 256, 256, 8
    W = rand_w(N, K)
    Mb = N * K // b
    ku, kp = Mb * 3 // 4, Mb // 2
    p = O.project(W, b, ku, kp)
    bits = O.storage_bits(p)
    assert bits["unified_values"] == 32 * (ku - kp) and bits["unified_signs"] == b * (ku - kp)
    assert bits["dense_values"] == 16 * b * (Mb - ku) and bits["pruned"] == 0
    buf = O.pack(p)
    words = lambda nbits: (nbits + 31) // 32 * 4
    assert buf.shape[0] == 8 * len(O.STORE_FIELDS) + 2 * words(Mb) + bits["unified_values"] // 8 + \
        words(bits["unified_signs"]) + bits["dense_values"] // 8
    # all blocks unified with fp32 magnitudes: the ratio of Section 3.1 ("nearly 4x" for 4 weights)
    p_all = O.project(W, 4, N * K // 4, 0)
    b4 = O.storage_bits(p_all)
    ratio = 32 * N * K / (b4["unified_values"] + b4["unified_signs"])
    assert ratio == pytest.approx(O.storage_reduction((2, 2), include_sign_bits=True))


def test_gemm_special_cases():
    N, K, b, M = 128, 128, 4, 24
    W = rand_w(N, K)
    X = rand_x_bf16(M, K)
    Mb = N * K // b
    # all dense: an ordinary matmul with the bf16-rounded weights (library routine)
    p = O.project(W, b, 0, 0)
    What = O.unpack(O.pack(p), b)
    ref = torch.from_numpy(X) @ torch.from_numpy(W).to(torch.bfloat16).to(torch.float64).T
    assert np.allclose(O.gemm(X, What), ref.numpy(), rtol=1e-13, atol=1e-15)
    # all pruned: exactly zero
    p = O.project(W, b, Mb, Mb)
    assert np.all(O.gemm(X, O.unpack(O.pack(p), b)) == 0)
    # all unified: the shared-partial-sum form agrees with the plain contraction
    p = O.project(W, b, Mb, 0)
    Y1 = O.gemm(X, O.unpack(O.pack(p), b))
    Y2 = O.gemm_shared_partial(X, p, b)
    assert np.allclose(Y1, Y2, rtol=1e-11, atol=1e-14)
    # mixed
    p = O.project(W, b, Mb // 2, Mb // 4)
    Y1 = O.gemm(X, O.unpack(O.pack(p), b))
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

"""The format helper tests/packed_format.py (a restatement of the byte format include/mwu.h
documents for mwu_pack) against itself and against the CPU checker: what it writes reads back as
the checker's decoded weights, every block slot is listed exactly once, and the documented entry
order holds.  These are regressions of the file format, not parity claims."""
import numpy as np
import pytest

import packed_format as F
from oracle import mwu_oracle as O

RNG = np.random.default_rng(8302)


def rand_w(n, k, scale=0.02):
    return (RNG.standard_normal((n, k)) * scale).astype(np.float32)


@pytest.mark.parametrize("b,N,K", [(4, 128, 64), (16, 200, 128), (2, 64, 64), (8, 130, 192)])
def test_write_read_round_trip(b, N, K):
    W = rand_w(N, K)
    Mb = N * K // b
    p = O.project(W, b, Mb * 7 // 10, Mb * 4 // 10)
    buf = F.write(p, b)
    h = F.parse_header(buf)
    assert (h["N"], h["K"], h["b"]) == (N, K, b)
    assert h["n_pruned"] == p.pruned.sum() and h["n_unified"] == p.unified.sum()
    assert h["total"] == buf.shape[0]
    assert np.array_equal(F.read(buf), O.decoded_weights(p))


def test_section_sizes():
    N, K, b = 256, 256, 8
    W = rand_w(N, K)
    Mb = N * K // b
    ku, kp = Mb * 3 // 4, Mb // 2
    h = F.parse_header(F.write(O.project(W, b, ku, kp), b))
    assert h["off_dpos"] - h["off_ulist"] >= 8 * (ku - kp)
    assert h["off_ppos"] - h["off_dpay"] >= 2 * b * (Mb - ku)
    assert h["off_ppos"] - h["off_dpay"] < 2 * b * (Mb - ku) + 256
    assert h["total"] - h["off_ppos"] >= 2 * kp
    assert h["n_dense"] == Mb - ku and h["n_plist"] == kp


def test_live_mask_and_padding():
    N, K, b = 100, 128, 16          # 28 padded rows
    W = rand_w(N, K)
    W[:, 16:32] = 0.0               # slice 1 of stage 0 is all-zero in every row
    kp = N                          # exactly those blocks are pruned (smallest norm, ties by index)
    p = O.project(W, b, kp, kp)
    assert p.pruned.reshape(N, K // b)[:, 1].all()
    buf = F.write(p, b)
    h = F.parse_header(buf)
    rec = F.records(buf)
    assert rec[0, 3] == 0b1101 and rec[1, 3] == 0b1111
    nb = 64 // b
    assert h["n_plist"] == kp + 28 * (K // b)                           # padding rows pruned
    ppos = buf[h["off_ppos"]:h["off_ppos"] + 2 * h["n_plist"]].view(np.uint16)
    first = ppos[rec[0, 2]:rec[1, 2]]
    slots = [F.tile_offset_inverse(int(o), b) for o in first]
    codes = [r * nb + i for r, i in slots]
    assert len(set(codes)) == len(codes)
    assert set(range(100 * nb, 128 * nb)) <= set(codes)
    assert rec[2].tolist() == [h["n_unified"], h["n_dense"], h["n_plist"], 0]
    assert F.read(buf).shape == (N, K)


def test_tile_offset_is_a_bijection():
    for b in (2, 4, 8, 16):
        nb = 64 // b
        pos = np.arange(128 * nb)
        off = F.tile_offset(pos, b)
        g = min(2 * b, 16)          # a block wider than a chunk starts on a chunk boundary
        assert off.min() == 0 and off.max() == 16384 - g
        assert len(set(off.tolist())) == pos.size and np.all(off % g == 0)
        back = [F.tile_offset_inverse(int(o), b) for o in off]
        assert [r * nb + i for r, i in back] == pos.tolist()
    # row 0 is not permuted; row 1 swaps neighbouring chunks; rows 8.. start 1024 bytes later
    assert F.tile_offset(np.array([0, 1, 2, 3]), 16).tolist() == [0, 32, 64, 96]
    assert F.tile_offset(np.array([4, 5]), 16).tolist() == [128 + 16, 128 + 48]
    assert F.tile_offset(np.array([32]), 16).tolist() == [1024]


def test_class_lists_are_dealt_round_robin():
    N, K, b = 128, 64, 16
    W = rand_w(N, K)
    Mb = N * K // b
    p = O.project(W, b, Mb * 8 // 10, Mb * 6 // 10)
    buf = F.write(p, b)
    h = F.parse_header(buf)
    ppos = buf[h["off_ppos"]:h["off_ppos"] + 2 * h["n_plist"]].view(np.uint16).astype(int)
    lane = (ppos % 128) // 16
    # same multiset of blocks as the pruned mask
    assert sorted(F.tile_offset(np.flatnonzero(p.pruned), b).tolist()) == sorted(ppos.tolist())
    # the first round holds one entry of every value present, in ascending order
    n_lanes = len(set(lane.tolist()))
    assert lane[:n_lanes].tolist() == sorted(set(lane.tolist()))
    # inside one value the entries keep ascending block order
    for sl in set(lane.tolist()):
        pos = [r * 4 + i for r, i in (F.tile_offset_inverse(int(o), b) for o in ppos[lane == sl])]
        assert pos == sorted(pos)
    # while all eight values still have entries, any 8 consecutive entries hit 8 different ones
    shortest = min(np.bincount(lane, minlength=8))
    full = lane[:8 * shortest].reshape(-1, 8)
    assert all(len(set(row.tolist())) == 8 for row in full)

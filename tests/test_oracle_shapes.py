"""Pins for the CPU checker's block shapes (Section 3.1: 1-, 2- and 3-dim blocks; Table 1),
grouped pruning and the keep-2-of-4 projection of Section 4.7: hand-written partitions,
per-block Python loops, brute force over subsets and patterns."""
import itertools

import numpy as np
import pytest

from oracle import mwu_oracle as O

RNG = np.random.default_rng(31)


def rand_w(n, k, scale=0.02):
    return (RNG.standard_normal((n, k)) * scale).astype(np.float32)


# ---- the partition ------------------------------------------------------------------------------
def test_partition_2x2_by_hand():
    """Section 3.1's example layer: 6 inputs, 4 outputs, 2x2 blocks -> 6 blocks."""
    part = O.partition(4, 6, O.BlockShape(2, 2))
    assert part.idx.tolist() == [[0, 1, 6, 7], [2, 3, 8, 9], [4, 5, 10, 11],
                                 [12, 13, 18, 19], [14, 15, 20, 21], [16, 17, 22, 23]]
    assert part.size.tolist() == [4] * 6


def test_partition_1d_is_consecutive_entries_of_a_row():
    part = O.partition(3, 8, 4)
    assert part.idx.tolist() == [[0, 1, 2, 3], [4, 5, 6, 7], [8, 9, 10, 11], [12, 13, 14, 15],
                                 [16, 17, 18, 19], [20, 21, 22, 23]]


def test_partition_2x2x2_with_nine_taps_by_hand():
    """Weight [2 rows][2 channels * 9 taps]: reduction index = channel * 9 + tap.  Tap groups
    {0,1} {2,3} {4,5} {6,7} {8}: four full blocks of 8 and one short block of 4."""
    part = O.partition(2, 18, O.BlockShape(2, 2, 2, taps=9))
    assert part.size.tolist() == [8, 8, 8, 8, 4]
    assert part.idx[0].tolist() == [0, 1, 9, 10, 18, 19, 27, 28]       # (row, channel, tap) order
    assert part.idx[3].tolist() == [6, 7, 15, 16, 24, 25, 33, 34]
    assert part.idx[4].tolist() == [8, 17, 26, 35, -1, -1, -1, -1]
    # every weight belongs to exactly one block
    flat = part.idx[part.idx >= 0]
    assert sorted(flat.tolist()) == list(range(36))


@pytest.mark.parametrize("shape,N,K", [(O.BlockShape(2, 2), 8, 12), (O.BlockShape(2, 2, 2, taps=9), 4, 36),
                                       (O.BlockShape(4, 1), 3, 16), (O.BlockShape(2, 2, 2, taps=4), 4, 16)])
def test_partition_covers_every_weight_once(shape, N, K):
    part = O.partition(N, K, shape)
    flat = part.idx[part.idx >= 0]
    assert sorted(flat.tolist()) == list(range(N * K))
    assert int(part.size.sum()) == N * K


# ---- statistics and projection, block by block in plain Python ---------------------------------
@pytest.mark.parametrize("shape,N,K", [(O.BlockShape(2, 2), 6, 8), (O.BlockShape(2, 2, 2, taps=9), 4, 36),
                                       (O.BlockShape(8, 1), 4, 16)])
def test_block_stats_python_loop(shape, N, K):
    W = rand_w(N, K)
    st = O.block_stats(W, shape)
    part = O.partition(N, K, shape)
    flat = W.reshape(-1).astype(np.float64)
    for j in range(part.idx.shape[0]):
        a = [abs(float(flat[i])) for i in part.idx[j] if i >= 0]
        q = sum(a) / len(a)
        assert st.q[j] == pytest.approx(q, rel=1e-14)
        assert st.S[j] == pytest.approx(sum(a), rel=1e-14)
        assert st.L_u[j] == pytest.approx(sum((x - q) ** 2 for x in a), rel=1e-10, abs=1e-20)
        assert st.L_p[j] == pytest.approx(sum(x * x for x in a), rel=1e-13)


def test_1d_shape_equals_the_row_reshape():
    W = rand_w(16, 32)
    for b in (2, 4, 8, 16):
        st = O.block_stats(W, b)
        a = np.abs(W.astype(np.float64)).reshape(-1, b)
        S = O.tree_sum(a)
        assert np.array_equal(st.S, S)
        assert np.array_equal(st.L_p, O.tree_sum(a * a))
        d = a - (S / b)[:, None]
        assert np.array_equal(st.L_u, O.tree_sum(d * d))


def test_2x2_blocks_take_two_rows():
    """A 2x2 block covers two entries of each of two neighbouring rows (not four of one row)."""
    W = np.full((4, 4), 5.0, dtype=np.float32)
    W[2:4, 2:4] = 0.1                          # bottom-right 2x2 block is small
    W[0, :] = [0.2, 0.2, 0.2, 0.2]             # a small row must not form a block
    W[1, :] = 5.0
    p = O.project(W, O.BlockShape(2, 2), 1, 1)
    assert np.flatnonzero(p.pruned).tolist() == [3]
    assert np.all(p.Q[2:4, 2:4] == 0) and np.array_equal(p.Q[:2], W[:2])


@pytest.mark.parametrize("shape,N,K", [(O.BlockShape(2, 2), 8, 8), (O.BlockShape(2, 2, 2, taps=9), 4, 18)])
def test_projection_python_loop(shape, N, K):
    W = rand_w(N, K)
    part = O.partition(N, K, shape)
    Mb = part.idx.shape[0]
    p = O.project(W, shape, Mb * 3 // 4, Mb // 4)
    Q = p.Q.reshape(-1)
    flat = W.reshape(-1)
    for j in range(Mb):
        members = [i for i in part.idx[j] if i >= 0]
        for i in members:
            if p.pruned[j]:
                assert Q[i] == 0 and not np.signbit(Q[i])
            elif p.unified[j]:
                q32 = np.float32(sum(abs(float(flat[m])) for m in members) / len(members))
                assert abs(float(Q[i])) == pytest.approx(float(q32), rel=1e-6)
                assert (Q[i] < 0) == (flat[i] < 0)
            else:
                assert Q[i] == flat[i]
    assert p.pruned.sum() == Mb // 4 and p.unified.sum() == Mb * 3 // 4 - Mb // 4
    # distance of the result = sum of the chosen blocks' losses
    dist = float(((W.astype(np.float64) - p.Q.astype(np.float64)) ** 2).sum())
    assert dist == pytest.approx(float(p.stats.L_p[p.pruned].sum() + p.stats.L_u[p.unified].sum()), rel=1e-5)


def _dist(stats, pruned_set, unified_set):
    return stats.L_p[list(pruned_set)].sum() + stats.L_u[list(unified_set)].sum()


@pytest.mark.parametrize("shape,N,K", [(O.BlockShape(2, 2), 4, 8), (O.BlockShape(2, 2, 2, taps=3), 4, 6)])
def test_selection_brute_force_for_block_shapes(shape, N, K):
    W = rand_w(N, K)
    st = O.block_stats(W, shape)
    Mb = st.S.shape[0]
    assert Mb <= 8
    idx = range(Mb)
    for k in range(1, Mb + 1):
        p = O.project(W, shape, k, 0)
        best = min(_dist(st, [], c) for c in itertools.combinations(idx, k))
        assert _dist(st, [], np.flatnonzero(p.unified)) == pytest.approx(best, rel=1e-12)
        p = O.project(W, shape, k, k)
        best = min(_dist(st, c, []) for c in itertools.combinations(idx, k))
        assert _dist(st, np.flatnonzero(p.pruned), []) == pytest.approx(best, rel=1e-12)


@pytest.mark.parametrize("shape,N,K", [(O.BlockShape(2, 2), 16, 16), (O.BlockShape(2, 2, 2, taps=9), 8, 72)])
def test_idempotence_for_block_shapes(shape, N, K):
    W = rand_w(N, K)
    Mb = O.partition(N, K, shape).idx.shape[0]
    ku, kp = Mb * 6 // 10, Mb * 3 // 10
    p1 = O.project(W, shape, ku, kp)
    p2 = O.project(p1.Q, shape, ku, kp)
    assert np.array_equal(p1.Q.view(np.uint32), p2.Q.view(np.uint32))
    st = O.block_stats(p1.Q, shape)
    assert np.all(st.L_u[p1.unified] == 0.0) and np.all(st.L_p[p1.pruned] == 0.0)


def test_section_3_1_example_counts():
    """Section 3.1's walk-through: 6 inputs x 4 outputs in 2x2 blocks.  Half of the blocks pruned
    halves the parameters; all blocks unified leaves one magnitude and four sign bits per block
    ("nearly 4x" with fp32 magnitudes)."""
    W = rand_w(4, 6)
    shape = O.BlockShape(2, 2)
    p = O.project(W, shape, 3, 3)
    assert int((p.Q != 0).sum()) == 12                      # 24 parameters -> 12
    p = O.project(W, shape, 6, 0)
    bits = O.storage_bits(p)
    assert bits["unified_values"] == 6 * 32 and bits["unified_signs"] == 24 and bits["dense_values"] == 0
    assert 24 * 32 / (bits["unified_values"] + bits["unified_signs"]) == pytest.approx(3.5555, abs=1e-3)
    assert np.array_equal(O.unpack(O.pack(p), shape), O.decoded_weights(p))


def test_storage_round_trip_for_block_shapes():
    for shape, N, K in [(O.BlockShape(2, 2), 8, 16), (O.BlockShape(2, 2, 2, taps=9), 4, 36)]:
        W = rand_w(N, K)
        Mb = O.partition(N, K, shape).idx.shape[0]
        p = O.project(W, shape, Mb * 7 // 10, Mb * 3 // 10)
        assert np.array_equal(O.unpack(O.pack(p), shape), O.decoded_weights(p))
        Qb = O.bf16_bits_to_f64(O.bf16_bits_rne(p.Q))
        assert np.array_equal(O.decoded_weights(p), Qb)


# ---- grouped pruning ------------------------------------------------------------------------------
def test_group_keys_python_loop():
    N, K, b, gr, gc = 8, 16, 4, 4, 8
    W = rand_w(N, K)
    st = O.block_stats(W, b)
    gk = O.group_prune_keys(st.L_p, N, K, b, gr, gc)
    assert gk.shape == (2, 2)
    for t in range(2):
        for s in range(2):
            tot = float((W[t * gr:(t + 1) * gr, s * gc:(s + 1) * gc].astype(np.float64) ** 2).sum())
            assert gk[t, s] == pytest.approx(tot, rel=1e-13)


def test_grouped_pruning_brute_force_and_ties():
    N, K, b, gr, gc = 8, 16, 4, 4, 4            # 2 row tiles x 4 slices = 8 groups of 4 blocks
    W = rand_w(N, K)
    st = O.block_stats(W, b)
    per = gr * gc // b
    gk = O.group_prune_keys(st.L_p, N, K, b, gr, gc).reshape(-1)
    for kg in (1, 3, 5, 8):
        p = O.project(W, b, kg * per, kg * per, prune_group=(gr, gc))
        # whole groups are zero, nothing else
        zero = (p.Q.reshape(2, gr, 4, gc) == 0).all(axis=(1, 3)).reshape(-1)
        assert int(zero.sum()) == kg and int(p.pruned.sum()) == kg * per
        assert np.array_equal(p.Q[p.Q != 0], W[p.Q != 0])
        # the chosen groups minimise the distance among all sets of kg groups
        best = min(gk[list(c)].sum() for c in itertools.combinations(range(8), kg))
        assert gk[zero].sum() == pytest.approx(best, rel=1e-12)
        assert float((W.astype(np.float64) ** 2)[p.Q == 0].sum()) == pytest.approx(best, rel=1e-12)
    # unification picks among the blocks outside the pruned groups
    p = O.project(W, b, 2 * per + 5, 2 * per, prune_group=(gr, gc))
    assert int(p.unified.sum()) == 5 and not np.any(p.unified & p.pruned)
    rest = np.flatnonzero(~p.pruned)
    assert st.L_u[p.unified].max() <= np.sort(st.L_u[rest])[5 - 1]
    # identical groups: the lower group index (row tile first, then slice) goes first
    W2 = np.tile(rand_w(1, 4), (8, 4)).astype(np.float32)
    p = O.project(W2, b, 3 * per, 3 * per, prune_group=(gr, gc))
    zero = (p.Q.reshape(2, gr, 4, gc) == 0).all(axis=(1, 3)).reshape(-1)
    assert zero.tolist() == [True, True, True, False, False, False, False, False]


def test_group_of_one_block_is_plain_pruning():
    N, K, b = 8, 32, 4
    W = rand_w(N, K)
    a = O.project(W, b, 40, 24)
    g = O.project(W, b, 40, 24, prune_group=(1, b))
    assert np.array_equal(a.pruned, g.pruned) and np.array_equal(a.unified, g.unified)
    assert np.array_equal(a.Q, g.Q)


# ---- keep 2 of every 4 (Section 4.7) ----------------------------------------------------------------
def test_keep_2_of_4_brute_force():
    W = rand_w(6, 16)
    r = O.project_n_of_m(W, 2, 4)
    groups = W.reshape(-1, 4).astype(np.float64)
    Qg = r.Q.reshape(-1, 4)
    for g in range(groups.shape[0]):
        best = min(sum(groups[g, i] ** 2 for i in range(4) if i not in keep)
                   for keep in itertools.combinations(range(4), 2))
        got = float(((groups[g] - Qg[g].astype(np.float64)) ** 2).sum())
        assert got == pytest.approx(best, rel=1e-12)
        assert int((Qg[g] != 0).sum()) == 2
        assert np.array_equal(Qg[g][Qg[g] != 0], W.reshape(-1, 4)[g][Qg[g] != 0])
    assert int(r.keep.sum()) == W.size // 2


def test_keep_n_of_m_ties_zeros_and_dual():
    W = np.array([[1, -1, 1, 1, 0, 0, 0, 0, 3, -0.0, 2, 2]], dtype=np.float32)
    r = O.project_n_of_m(W, 2, 4)
    assert r.keep.tolist() == [[True, True, False, False, True, True, False, False, True, False, True, False]]
    assert r.Q.tolist() == [[1, -1, 0, 0, 0, 0, 0, 0, 3, 0, 2, 0]]
    U = rand_w(1, 12, scale=1.0)
    r2 = O.project_n_of_m(W, 2, 4, U=U)
    assert np.array_equal(r2.V, (W + U).astype(np.float32))
    assert np.array_equal(r2.Q, O.project_n_of_m(r2.V, 2, 4).Q)
    # n = m keeps everything, n = 0 nothing
    assert np.array_equal(O.project_n_of_m(W, 4, 4).Q, W)
    assert not O.project_n_of_m(W, 0, 4).Q.any()

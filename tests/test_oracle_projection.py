"""Pins for the CPU checker's projection: closed forms, invariants, brute force.

Each test is chosen so that a plausible slip in oracle/mwu_oracle.py (a dropped term, a
wrong sign, a wrong axis, a wrong tie rule) makes it fail.  Nothing here touches the GPU.
"""
import itertools
import os

import numpy as np
import pytest

from oracle import mwu_oracle as O

RNG = np.random.default_rng(20210608)


def rand_w(n, k, scale=0.02):
    return (RNG.standard_normal((n, k)) * scale).astype(np.float32)


# ---- unified value: Eq. (2) + "average of the absolute value" --------------------------
@pytest.mark.parametrize("b", [2, 4])
def test_q_is_the_euclidean_projection_brute_force(b):
    """For each block, (sign(w), mean|w|) minimises sum (w_l - s_l q)^2 over all sign
    patterns and a fine grid of q >= 0 (Eq. 7: the Q-step is a Euclidean projection)."""
    W = rand_w(6, b)
    st = O.block_stats(W, b)
    for j in range(W.shape[0]):
        w = W[j].astype(np.float64)
        best = np.inf
        grid = np.linspace(0.0, np.abs(w).max() * 1.5, 3001)
        for s in itertools.product([-1.0, 1.0], repeat=b):
            s = np.array(s)
            cost = ((w[None, :] - grid[:, None] * s[None, :]) ** 2).sum(axis=1)
            best = min(best, cost.min())
        assert st.L_u[j] <= best + 1e-15
        # and the optimum on the grid is close to it (grid resolution)
        assert best - st.L_u[j] < (grid[1] - grid[0]) ** 2 * b + 1e-15
        assert st.q[j] == pytest.approx(np.abs(w).mean(), rel=1e-15)


def test_q_derivative_is_zero():
    W = rand_w(32, 16)
    st = O.block_stats(W, 16)
    a = np.abs(W.astype(np.float64))
    # d/dq sum (a_l - q)^2 = -2 sum (a_l - q)
    assert np.allclose((a - st.q[:, None]).sum(axis=1), 0.0, atol=1e-15)


@pytest.mark.parametrize("b", [2, 4, 8, 16])
def test_loss_closed_forms(b):
    W = rand_w(64, 64)
    st = O.block_stats(W, b)
    a = np.abs(W.astype(np.float64)).reshape(-1, b)
    sumsq = (a * a).sum(axis=1)
    assert np.allclose(st.L_p, sumsq, rtol=1e-13)
    assert np.allclose(st.L_u, sumsq - st.S ** 2 / b, rtol=1e-9, atol=1e-18)
    assert np.allclose(st.L_p, st.L_u + st.S ** 2 / b, rtol=1e-12)
    assert np.allclose(st.S, a.sum(axis=1), rtol=1e-14)
    assert np.all(st.L_u <= st.L_p)


def test_tree_sum_order_is_pairwise():
    """1 + 2^-53 + 2^-53 + 0: pairwise (l with l^1 first) loses both tiny terms in the first
    pair only if they are split; the balanced tree gives a result a left-to-right sum does not."""
    t = 2.0 ** -53
    x = np.array([[1.0, t, t, 0.0]])
    # pairwise: (1 + t) + (t + 0) = 1 + t -> rounds to 1 (ties to even), then 1 + t = 1
    assert O.tree_sum(x)[0] == 1.0
    x = np.array([[t, t, 1.0, 0.0]])
    # pairwise: (t + t) + (1 + 0) = 1 + 2^-52 exactly representable
    assert O.tree_sum(x)[0] == 1.0 + 2.0 ** -52
    # a left-to-right sum of the first ordering would also be 1.0, of the second 1 + 2^-52;
    # the order-sensitive case: [1, t, 1, t] -> pairs (1+t)=1, (1+t)=1 -> 2
    x = np.array([[t, 1.0, t, 1.0, t, t, t, t]])
    assert O.tree_sum(x)[0] == (1.0 + 1.0) + 4 * t


def test_frobenius_distance_is_sum_of_block_losses():
    W = rand_w(16, 32)
    b = 4
    Mb = W.size // b
    p = O.project(W, b, k_unify=Mb // 2, k_prune=Mb // 4)
    # Q holds fp32(q); compare with the fp64 statistic at fp32 accuracy
    dist = ((W.astype(np.float64) - p.Q.astype(np.float64)) ** 2).reshape(-1, b).sum(axis=1)
    expect = np.where(p.pruned, p.stats.L_p, np.where(p.unified, p.stats.L_u, 0.0))
    assert np.allclose(dist, expect, rtol=1e-5, atol=1e-14)
    assert p.pruned.sum() == Mb // 4 and p.unified.sum() == Mb // 2 - Mb // 4
    assert not np.any(p.pruned & p.unified)


# ---- pruning special case -----------------------------------------------------------------
def test_all_zero_block_is_a_fixed_point():
    W = rand_w(4, 16)
    W[1, 4:8] = 0.0
    W[2, 0:4] = -0.0
    st = O.block_stats(W, 4)
    assert st.q[5] == 0 and st.L_u[5] == 0 and st.L_p[5] == 0
    p = O.project(W, 4, k_unify=2, k_prune=2)
    assert p.pruned[5] and p.pruned[8]           # the two zero blocks have the smallest norm
    assert np.all(p.Q[1, 4:8] == 0) and np.all(p.Q[2, 0:4] == 0)
    # everything else untouched, bit for bit
    keep = np.ones_like(W, dtype=bool)
    keep[1, 4:8] = False
    keep[2, 0:4] = False
    assert np.array_equal(p.Q[keep].view(np.uint32), W[keep].view(np.uint32))


def test_pure_pruning_zeroes_smallest_norm_blocks():
    """k_unify == k_prune: Section 3.1's pruning walk-through (smallest-norm blocks go)."""
    W = rand_w(8, 64)
    for b, key in [(4, "l2sq"), (4, "l1"), (8, "l2sq")]:
        Mb = W.size // b
        k = Mb // 2
        p = O.project(W, b, k, k, prune_key=key)
        a = np.abs(W.astype(np.float64)).reshape(-1, b)
        norm = (a * a).sum(axis=1) if key == "l2sq" else a.sum(axis=1)
        thr = np.sort(norm)[k - 1]
        assert np.all(norm[p.pruned] <= thr) and np.all(norm[~p.pruned] >= thr)
        assert p.pruned.sum() == k and p.unified.sum() == 0
        assert np.all(p.Q.reshape(-1, b)[p.pruned] == 0)
        assert np.array_equal(p.Q.reshape(-1, b)[~p.pruned], W.reshape(-1, b)[~p.pruned])


def test_l1_and_l2_keys_can_disagree():
    # block 0: (3,0,0,0): L1=3, L2^2=9 ; block 1: (2,2,0,0): L1=4, L2^2=8
    W = np.array([[3, 0, 0, 0, 2, 2, 0, 0]], dtype=np.float32)
    assert O.project(W, 4, 1, 1, prune_key="l1").pruned.tolist() == [True, False]
    assert O.project(W, 4, 1, 1, prune_key="l2sq").pruned.tolist() == [False, True]


# ---- Eq. (2) sign rule ----------------------------------------------------------------------
def test_sign_rule_and_negative_zero():
    W = np.array([[1.0, -3.0, 0.0, -0.0]], dtype=np.float32)
    p = O.project(W, 4, 1, 0)
    assert p.unified.tolist() == [True]
    assert p.u[0] == np.float32(1.0)
    assert p.Q.tolist() == [[1.0, -1.0, 1.0, 1.0]]          # zeros (either sign) become +q
    assert p.sign.tolist() == [[False, True, False, False]]
    assert not np.signbit(p.Q[0, 3])


def test_sign_flip_equivariance_and_scaling():
    W = rand_w(16, 32)
    b = 8
    Mb = W.size // b
    p = O.project(W, b, Mb * 3 // 4, Mb // 4)
    flip = RNG.random(W.shape) < 0.5
    W2 = np.where(flip, -W, W).astype(np.float32)
    p2 = O.project(W2, b, Mb * 3 // 4, Mb // 4)
    assert np.array_equal(p.pruned, p2.pruned) and np.array_equal(p.unified, p2.unified)
    assert np.array_equal(p.u, p2.u)
    nz = W != 0
    assert np.array_equal(p2.Q[nz], np.where(flip, -p.Q, p.Q)[nz])
    # scaling by a power of two is exact in every step
    p3 = O.project((W * np.float32(8.0)).astype(np.float32), b, Mb * 3 // 4, Mb // 4)
    assert np.array_equal(p.pruned, p3.pruned) and np.array_equal(p.unified, p3.unified)
    assert np.array_equal(p3.Q, p.Q * np.float32(8.0))
    assert np.array_equal(p3.u, p.u * np.float32(8.0))


def test_block_permutation_equivariance():
    W = rand_w(1, 64 * 4)
    b = 4
    Mb = 64
    perm = RNG.permutation(Mb)
    W2 = W.reshape(Mb, b)[perm].reshape(1, -1)
    p = O.project(W, b, 40, 16)
    p2 = O.project(W2, b, 40, 16)
    assert np.array_equal(p.pruned[perm], p2.pruned)
    assert np.array_equal(p.unified[perm], p2.unified)
    assert np.array_equal(p.Q.reshape(Mb, b)[perm], p2.Q.reshape(Mb, b))


def test_blocks_run_along_the_row():
    """Block j covers W[n][kb*b .. kb*b+b-1] with j = n*(K/b)+kb (not a column block)."""
    W = np.zeros((4, 8), dtype=np.float32)
    W[:, :] = 5.0
    W[2, 4:8] = [0.1, 0.1, 0.1, 0.1]          # one whole row-block is small
    W[0:4, 0] = [0.2, 0.2, 5.0, 0.2]          # a column of small values must not form a block
    p = O.project(W, 4, 1, 1)
    assert np.flatnonzero(p.pruned).tolist() == [2 * 2 + 1]


# ---- selection: brute force over all subsets ------------------------------------------------
def _dist(V, b, pruned_set, unified_set):
    a = np.abs(V.astype(np.float64)).reshape(-1, b)
    q = a.mean(axis=1, keepdims=True)
    lu = ((a - q) ** 2).sum(axis=1)
    lp = (a ** 2).sum(axis=1)
    return lp[list(pruned_set)].sum() + lu[list(unified_set)].sum()


@pytest.mark.parametrize("seed", [0, 1, 2])
def test_selection_brute_force(seed):
    rng = np.random.default_rng(seed)
    b, Mb = 4, 8
    V = (rng.standard_normal((2, Mb * b // 2)) * 0.02).astype(np.float32)
    idx = range(Mb)
    # (i) pure unification: chosen set is the global optimum among all sets of size k
    for k in [1, 3, 5, 8]:
        p = O.project(V, b, k, 0)
        got = _dist(V, b, [], np.flatnonzero(p.unified))
        best = min(_dist(V, b, [], c) for c in itertools.combinations(idx, k))
        assert got == pytest.approx(best, rel=1e-12)
    # (ii) pure pruning
    for k in [1, 4, 7]:
        p = O.project(V, b, k, k)
        got = _dist(V, b, np.flatnonzero(p.pruned), [])
        best = min(_dist(V, b, c, []) for c in itertools.combinations(idx, k))
        assert got == pytest.approx(best, rel=1e-12)
    # (iii) mixed: P optimal among size-k_p sets; U optimal among subsets of the remainder
    ku, kp = 5, 2
    p = O.project(V, b, ku, kp)
    P = np.flatnonzero(p.pruned)
    U = np.flatnonzero(p.unified)
    assert len(P) == kp and len(U) == ku - kp
    bestP = min(_dist(V, b, c, []) for c in itertools.combinations(idx, kp))
    assert _dist(V, b, P, []) == pytest.approx(bestP, rel=1e-12)
    rest = [j for j in idx if j not in set(P.tolist())]
    bestU = min(_dist(V, b, [], c) for c in itertools.combinations(rest, ku - kp))
    assert _dist(V, b, [], U) == pytest.approx(bestU, rel=1e-12)
    # the staged rule is never better than the joint optimum (it is a reading, not the optimum)
    joint = min(_dist(V, b, cp, cu)
                for cp in itertools.combinations(idx, kp)
                for cu in itertools.combinations([j for j in idx if j not in cp], ku - kp))
    assert joint <= _dist(V, b, P, U) + 1e-18


def test_ties_go_to_the_lower_index():
    blk = np.array([0.5, -0.25, 0.125, 1.0], dtype=np.float32)
    W = np.tile(blk, 6).reshape(1, -1)                      # six identical blocks
    p = O.project(W, 4, 4, 2)
    assert p.pruned.tolist() == [True, True, False, False, False, False]
    assert p.unified.tolist() == [False, False, True, True, False, False]
    # blocks of equal magnitudes have L_u == 0 exactly, whatever their scale: index decides
    W = np.array([[3, -3, 3, 3, 1, 1, -1, 1, 2, 2, 2, -2]], dtype=np.float32)
    p = O.project(W, 4, 2, 0)
    assert p.unified.tolist() == [True, True, False]


# ---- idempotence ------------------------------------------------------------------------------
@pytest.mark.parametrize("b", [2, 4, 8, 16])
def test_idempotence(b):
    W = rand_w(32, 64)
    Mb = W.size // b
    ku, kp = Mb * 6 // 10, Mb * 3 // 10
    p1 = O.project(W, b, ku, kp)
    p2 = O.project(p1.Q, b, ku, kp)
    assert np.array_equal(p1.Q.view(np.uint32), p2.Q.view(np.uint32))
    st = O.block_stats(p1.Q, b)
    assert np.all(st.L_u[p1.unified] == 0.0)       # residual form gives exactly zero
    assert np.all(st.L_p[p1.pruned] == 0.0)
    assert np.array_equal(st.q[p1.unified].astype(np.float32), p1.u[p1.unified])


# ---- ADMM input: Unify(W + U) ------------------------------------------------------------------
def test_dual_variable_is_added_in_fp32():
    W = rand_w(8, 32)
    U = rand_w(8, 32, scale=0.005)
    p = O.project(W, 4, 32, 16, U=U)
    V = (W + U).astype(np.float32)
    p_ref = O.project(V, 4, 32, 16)
    assert np.array_equal(p.Q, p_ref.Q) and np.array_equal(p.V, V)
    # and it is not the projection of W alone
    assert not np.array_equal(p.Q, O.project(W, 4, 32, 16).Q)


def test_count_from_permille():
    assert O.count_from_permille(36864, 600) == 22118      # 22118.4
    assert O.count_from_permille(36864, 300) == 11059      # 11059.2
    assert O.count_from_permille(4194304, 800) == 3355443
    assert O.count_from_permille(4194304, 600) == 2516582
    assert O.count_from_permille(3, 500) == 2               # 1.5 rounds half up
    assert O.count_from_permille(16384, 500) == 8192


def test_bitmap_words():
    m = np.zeros(70, dtype=bool)
    m[[0, 31, 32, 69]] = True
    w = O.bitmap_words(m)
    assert w.dtype == np.uint32 and w.tolist() == [0x80000001, 0x1, 1 << 5]


# ---- Table 1 (values the paper prints) -----------------------------------------------------------
def test_table1_accounting_matches_the_paper():
    path = os.path.join(os.path.dirname(__file__), "golden", "table1_block_shapes.txt")
    rows = 0
    for line in open(path):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        parts = line.split()
        if parts[0] == "fig2":
            shape = tuple(int(x) for x in parts[1].split(","))
            dense, uni = O.multiplies_per_block(shape)
            assert (2 * dense, 2 * uni) == (int(parts[2]), int(parts[3]))
            continue
        shape = tuple(int(x) for x in parts[0].split(","))
        assert O.multiplier_reduction(shape) == float(parts[1])
        assert O.storage_reduction(shape) == float(parts[2])
        rows += 1
    assert rows == 4
    # Section 3.1: 2x2 blocks, all unified -> "nearly 4x" once the sign bits are stored too
    assert O.storage_reduction((2, 2), include_sign_bits=True) == pytest.approx(32 * 4 / 36)


# ---- a planted mistake must be caught (the pins have teeth) ---------------------------------------
def test_planted_mistakes_are_caught(monkeypatch):
    W = rand_w(8, 32)
    a = np.abs(W.astype(np.float64)).reshape(-1, 4)
    # mistake 1: q = sum instead of mean
    bad = O.block_stats(W, 4)
    bad_q = bad.S
    assert not np.allclose(bad_q, a.mean(axis=1))
    # mistake 2: dropping the last term of the tree
    monkeypatch.setattr(O, "tree_sum", lambda x: x[..., :-1].sum(axis=-1))
    st = O.block_stats(W, 4)
    assert not np.allclose(st.L_p, (a * a).sum(axis=1), rtol=1e-13)

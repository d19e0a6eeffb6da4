"""Pins for the CPU checker's dual step (Algorithm 1: U <- U + W - Q; quadratic term of the
augmented Lagrangian of Section 3.3): closed forms, element-by-element loops, fixed points."""
import numpy as np
import pytest

from oracle import mwu_oracle as O


def make(rows, cols, seed, scale=0.02):
    rng = np.random.default_rng(seed)
    return (rng.standard_normal((rows, cols)) * scale).astype(np.float32)


@pytest.mark.parametrize("b", [2, 4, 8, 16])
def test_dual_update_by_class_closed_forms(b):
    W, U = make(24, 64, 1), make(24, 64, 2, 0.004)
    Mb = W.size // b
    p = O.project(W, b, Mb * 6 // 10, Mb * 3 // 10, U=U)
    d = O.dual_update(p, b)
    Un = d.U_next.reshape(-1, b)
    V = p.V.reshape(-1, b)
    dense = ~(p.pruned | p.unified)
    # a block that keeps its values leaves no residual; a pruned block leaves itself
    assert np.all(Un[dense] == 0) and not np.any(np.signbit(Un[dense]))
    assert np.array_equal(Un[p.pruned], V[p.pruned])
    # unified: v - sign*q = sign * (|v| - q): the same real number, so the same fp32 rounding
    q = p.u[p.unified].astype(np.float64)[:, None]
    Vu = V[p.unified].astype(np.float64)
    expect = (np.where(Vu < 0, -1.0, 1.0) * (np.abs(Vu) - q)).astype(np.float32)
    assert np.array_equal(Un[p.unified], expect)


def test_dual_update_python_loop():
    """U + W - Q entry by entry in Python floats (fp64), rounded to fp32 at the end: v and Q are
    fp32, so the fp64 difference is exact and its fp32 rounding is the fp32 subtraction."""
    W, U = make(6, 16, 3), make(6, 16, 4, 0.01)
    b = 4
    Mb = W.size // b
    p = O.project(W, b, Mb // 2, Mb // 4, U=U)
    d = O.dual_update(p, b)
    for n in range(6):
        for k in range(16):
            v = float(np.float32(np.float32(W[n, k]) + np.float32(U[n, k])))
            assert d.U_next[n, k] == np.float32(v - float(p.Q[n, k]))


@pytest.mark.parametrize("prune_key", ["l2sq", "l1"])
def test_residual_is_the_frobenius_distance(prune_key):
    W = make(32, 128, 5)
    b = 8
    Mb = W.size // b
    p = O.project(W, b, Mb * 7 // 10, Mb * 4 // 10, prune_key=prune_key)
    d = O.dual_update(p, b)
    direct = float(np.sum((p.V.astype(np.float64) - p.Q.astype(np.float64)) ** 2))
    assert abs(d.residual_sq - direct) <= 1e-9 * direct            # q rounded to fp32 in Q: ~1e-15
    assert abs(float(np.sum(d.U_next.astype(np.float64) ** 2)) - direct) <= 1e-6 * direct


def test_projected_tensor_has_zero_dual_update():
    W = make(16, 64, 6)
    b = 4
    Mb = W.size // b
    p = O.project(W, b, Mb // 2, Mb // 4)
    p2 = O.project(p.Q, b, Mb // 2, Mb // 4)
    d = O.dual_update(p2, b)
    assert np.all(d.U_next == 0) and d.residual_sq == 0.0


def test_dual_accumulates_over_iterations():
    """Two iterations with W fixed: U_2 = U_1 + W - Q_2, and sum_k (W - Q_k) telescopes into U."""
    W = make(8, 32, 7)
    b = 4
    Mb = W.size // b
    p1 = O.project(W, b, Mb // 2, 0)
    U1 = O.dual_update(p1, b).U_next
    p2 = O.project(W, b, Mb // 2, 0, U=U1)
    U2 = O.dual_update(p2, b).U_next
    ref = (U1.astype(np.float64) + W.astype(np.float64) - p2.Q.astype(np.float64))
    assert np.allclose(U2, ref, rtol=0, atol=1e-8)


def test_planted_mistake_wrong_sign_is_caught():
    W = make(8, 32, 8)
    b = 4
    Mb = W.size // b
    p = O.project(W, b, Mb // 2, Mb // 4)
    good = O.dual_update(p, b).U_next
    bad = (p.Q - p.V).astype(np.float32)
    assert not np.array_equal(good, bad)
    assert np.array_equal(good, -bad)

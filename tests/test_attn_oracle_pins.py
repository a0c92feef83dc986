"""Pins for the attention-projection oracle (Algorithm 1's projection and output-projection lines).

None of these re-types the oracle's own matmul: they use scalar loops with exact summation, closed forms whose
value is known without any matrix product, and invariants that a transposed operand, a wrong shard order or a
dropped shard would break.
"""
import math

import numpy as np
import pytest

from oracle import tsp_attn_proj_oracle as orc
from paper_2604_26294_b200 import inputs as inp


def _rng(seed):
    return np.random.default_rng(seed)


def _shard_rows(W, D):
    return [W[r * (W.shape[0] // D):(r + 1) * (W.shape[0] // D)] for r in range(D)]


def _shard_cols(W, D):
    return [W[:, r * (W.shape[1] // D):(r + 1) * (W.shape[1] // D)] for r in range(D)]


def _brute_xwT(X, W):
    """out[s, n] = sum_h X[s, h] * W[n, h] with exactly rounded sums."""
    S, H = X.shape
    N = W.shape[0]
    out = np.empty((S, N))
    for s in range(S):
        for n in range(N):
            out[s, n] = math.fsum(float(X[s, h]) * float(W[n, h]) for h in range(H))
    return out


@pytest.mark.parametrize("S,H,Hq,Hkv", [(3, 4, 6, 2), (5, 7, 4, 4), (2, 3, 8, 2)])
def test_qkv_projection_brute_force(S, H, Hq, Hkv):
    r = _rng(1)
    X, Wq, Wk, Wv = r.standard_normal((S, H)), r.standard_normal((Hq, H)), r.standard_normal((Hkv, H)), \
        r.standard_normal((Hkv, H))
    Q, K, V = orc.qkv_projection(X, Wq, Wk, Wv)
    assert Q.shape == (S, Hq) and K.shape == (S, Hkv) and V.shape == (S, Hkv)
    np.testing.assert_allclose(Q, _brute_xwT(X, Wq), rtol=0, atol=1e-13)
    np.testing.assert_allclose(K, _brute_xwT(X, Wk), rtol=0, atol=1e-13)
    np.testing.assert_allclose(V, _brute_xwT(X, Wv), rtol=0, atol=1e-13)


@pytest.mark.parametrize("S,H,Hq", [(3, 5, 4), (4, 2, 6)])
def test_output_projection_brute_force(S, H, Hq):
    r = _rng(2)
    A, Wo = r.standard_normal((S, Hq)), r.standard_normal((H, Hq))
    Y = orc.output_projection(A, Wo)
    assert Y.shape == (S, H)
    np.testing.assert_allclose(Y, _brute_xwT(A, Wo), rtol=0, atol=1e-13)


def test_closed_forms_without_a_matrix_product():
    r = _rng(3)
    S, H = 6, 5
    X = r.standard_normal((S, H))
    # selector rows: output feature n copies input feature perm[n] -> a transposed or mis-indexed weight shows at once
    perm = np.array([3, 0, 4, 4, 1, 2, 0])
    W = np.zeros((len(perm), H))
    W[np.arange(len(perm)), perm] = 1.0
    Q, K, V = orc.qkv_projection(X, W, 2.0 * W[:3], -W[:3])
    np.testing.assert_array_equal(Q, X[:, perm])
    np.testing.assert_array_equal(K, 2.0 * X[:, perm[:3]])
    np.testing.assert_array_equal(V, -X[:, perm[:3]])
    # rank-one weights: (X v) u^T
    u, v = r.standard_normal(4), r.standard_normal(H)
    Q, _, _ = orc.qkv_projection(X, np.outer(u, v), W[:1], W[:1])
    xv = np.array([math.fsum(X[s, h] * v[h] for h in range(H)) for s in range(S)])
    np.testing.assert_allclose(Q, xv[:, None] * u[None, :], rtol=1e-13, atol=1e-14)
    # output projection with selector columns: Y[:, n] = A[:, perm[n]]
    A = r.standard_normal((S, 5))
    Wo = np.zeros((len(perm), 5))
    Wo[np.arange(len(perm)), perm] = 1.0
    np.testing.assert_array_equal(orc.output_projection(A, Wo), A[:, perm])
    # zeros and scalars
    assert not orc.output_projection(np.zeros((S, 5)), Wo).any()
    np.testing.assert_array_equal(orc.output_projection(np.array([[2.0]]), np.array([[3.0]])), [[6.0]])


@pytest.mark.parametrize("D", [1, 2, 4, 8])
def test_shard_loop_reaches_the_unsharded_projections(D):
    r = _rng(4)
    S, H, Hq, Hkv = 9, 16, 32, 16
    X, Wq, Wk, Wv = r.standard_normal((S, H)), r.standard_normal((Hq, H)), r.standard_normal((Hkv, H)), \
        r.standard_normal((Hkv, H))
    Q, K, V = orc.qkv_projection(X, Wq, Wk, Wv)
    Qs, Ks, Vs = orc.sharded_qkv_projection(X, _shard_rows(Wq, D), _shard_rows(Wk, D), _shard_rows(Wv, D))
    np.testing.assert_array_equal(Qs, Q)     # same dot products, only grouped by shard
    np.testing.assert_array_equal(Ks, K)
    np.testing.assert_array_equal(Vs, V)
    A, Wo = r.standard_normal((S, Hq)), r.standard_normal((H, Hq))
    Y = orc.output_projection(A, Wo)
    Ys = orc.sharded_output_projection(_shard_cols(A, D), _shard_cols(Wo, D))
    np.testing.assert_allclose(Ys, Y, rtol=1e-13, atol=1e-13)
    # D = 1 is the plain layer
    if D == 1:
        np.testing.assert_array_equal(Ys, Y)


def test_invariants_of_the_output_projection():
    r = _rng(5)
    S, H, Hq, D = 7, 6, 12, 3
    A, Wo = r.standard_normal((S, Hq)), r.standard_normal((H, Hq))
    Y = orc.output_projection(A, Wo)
    # the same permutation of heads' columns in A and Wo leaves Y unchanged (why the shard order cannot matter)
    p = r.permutation(Hq)
    np.testing.assert_allclose(orc.output_projection(A[:, p], Wo[:, p]), Y, rtol=1e-13, atol=1e-13)
    # dropping a shard changes Y by exactly that shard's contribution
    As, Ws = _shard_cols(A, D), _shard_cols(Wo, D)
    part = orc.sharded_output_projection(As[:2], Ws[:2])
    np.testing.assert_allclose(Y - part, _brute_xwT(As[2], Ws[2]), rtol=0, atol=1e-12)
    # linear in both arguments; rows independent
    np.testing.assert_allclose(orc.output_projection(2.5 * A, Wo), 2.5 * Y, rtol=1e-14)
    q = r.permutation(S)
    np.testing.assert_array_equal(orc.output_projection(A[q], Wo), Y[q])
    np.testing.assert_array_equal(orc.output_rows(A, Wo, [4, 1]), Y[[4, 1]])


def test_sampled_rows_equal_full_mode():
    r = _rng(6)
    X, Wq, Wk = r.standard_normal((10, 8)), r.standard_normal((16, 8)), r.standard_normal((4, 8))
    Q, K, V = orc.qkv_projection(X, Wq, Wk, -Wk)
    q, k, v = orc.qkv_rows(X, Wq, Wk, -Wk, [7, 0, 3])
    np.testing.assert_array_equal(q, Q[[7, 0, 3]])
    np.testing.assert_array_equal(k, K[[7, 0, 3]])
    np.testing.assert_array_equal(v, V[[7, 0, 3]])


def test_input_recipe_statistics_and_determinism():
    a = inp.make_attn_inputs(64, 128, 256, 128, seed=3)
    b2 = inp.make_attn_inputs(64, 128, 256, 128, seed=3)
    for name in ("X", "Wq", "Wk", "Wv", "A", "Wo"):
        assert np.array_equal(getattr(a, name), getattr(b2, name))
    assert a.Wq.shape == (256, 128) and a.Wk.shape == (128, 128) and a.Wo.shape == (128, 256) and a.A.shape == (64, 256)
    # N(0, var 1/H) weights: Q = X Wq^T has unit variance elementwise
    Q, _, _ = orc.qkv_projection(inp.bf16_bits_to_f64(a.X), inp.bf16_bits_to_f64(a.Wq), inp.bf16_bits_to_f64(a.Wk),
                                 inp.bf16_bits_to_f64(a.Wv))
    assert abs(Q.std() - 1.0) < 0.05
    Y = orc.output_projection(inp.bf16_bits_to_f64(a.A), inp.bf16_bits_to_f64(a.Wo))
    assert abs(Y.std() - 1.0) < 0.05
    assert inp.shard_out_columns(a.Wo, 4).shape == (4, 128, 64)


# ----------------------------------------------------------------------------------------------------- backward
def _brute_aTb(A, B):
    """out[i, j] = sum_s A[s, i] * B[s, j] with exactly rounded sums."""
    return np.array([[math.fsum(float(A[s, i]) * float(B[s, j]) for s in range(A.shape[0])) for j in range(B.shape[1])]
                     for i in range(A.shape[1])])


def test_backward_brute_force():
    r = _rng(10)
    S, H, Hq, Hkv = 4, 5, 6, 2
    X, Wq, Wk, Wv = r.standard_normal((S, H)), r.standard_normal((Hq, H)), r.standard_normal((Hkv, H)), \
        r.standard_normal((Hkv, H))
    dQ, dK, dV = r.standard_normal((S, Hq)), r.standard_normal((S, Hkv)), r.standard_normal((S, Hkv))
    dX, dWq, dWk, dWv = orc.qkv_projection_backward(X, Wq, Wk, Wv, dQ, dK, dV)
    # dX[s, h] = sum_j dQ[s, j] Wq[j, h] + ... : brute force via the transposed weights
    ref_dX = _brute_xwT(dQ, Wq.T) + _brute_xwT(dK, Wk.T) + _brute_xwT(dV, Wv.T)
    np.testing.assert_allclose(dX, ref_dX, rtol=0, atol=1e-13)
    np.testing.assert_allclose(dWq, _brute_aTb(dQ, X), rtol=0, atol=1e-13)
    np.testing.assert_allclose(dWk, _brute_aTb(dK, X), rtol=0, atol=1e-13)
    np.testing.assert_allclose(dWv, _brute_aTb(dV, X), rtol=0, atol=1e-13)
    A, Wo, dY = r.standard_normal((S, Hq)), r.standard_normal((H, Hq)), r.standard_normal((S, H))
    dA, dWo = orc.output_projection_backward(A, Wo, dY)
    np.testing.assert_allclose(dA, _brute_xwT(dY, Wo.T), rtol=0, atol=1e-13)
    np.testing.assert_allclose(dWo, _brute_aTb(dY, A), rtol=0, atol=1e-13)


def test_backward_finite_differences():
    r = _rng(11)
    S, H, Hq, Hkv = 5, 6, 8, 4
    X, Wq, Wk, Wv = r.standard_normal((S, H)), r.standard_normal((Hq, H)), r.standard_normal((Hkv, H)), \
        r.standard_normal((Hkv, H))
    dQ, dK, dV = r.standard_normal((S, Hq)), r.standard_normal((S, Hkv)), r.standard_normal((S, Hkv))

    def loss(X_, Wq_, Wk_, Wv_):
        Q, K, V = orc.qkv_projection(X_, Wq_, Wk_, Wv_)
        return float((dQ * Q).sum() + (dK * K).sum() + (dV * V).sum())

    grads = orc.qkv_projection_backward(X, Wq, Wk, Wv, dQ, dK, dV)
    args = [X, Wq, Wk, Wv]
    eps = 1e-5
    for which in range(4):
        Vdir = r.standard_normal(args[which].shape)
        plus = [a + eps * Vdir if i == which else a for i, a in enumerate(args)]
        minus = [a - eps * Vdir if i == which else a for i, a in enumerate(args)]
        fd = (loss(*plus) - loss(*minus)) / (2 * eps)
        assert abs(fd - float((grads[which] * Vdir).sum())) <= 1e-7 * max(1.0, abs(fd))
    A, Wo, dY = r.standard_normal((S, Hq)), r.standard_normal((H, Hq)), r.standard_normal((S, H))
    dA, dWo = orc.output_projection_backward(A, Wo, dY)
    for which, g in ((0, dA), (1, dWo)):
        Vdir = r.standard_normal(g.shape)
        f = lambda e: float((dY * orc.output_projection(A + e * Vdir if which == 0 else A,
                                                        Wo + e * Vdir if which == 1 else Wo)).sum())
        fd = (f(eps) - f(-eps)) / (2 * eps)
        assert abs(fd - float((g * Vdir).sum())) <= 1e-7 * max(1.0, abs(fd))


def test_backward_adjoint_identities():
    # the layers are bilinear: <dWo, Wo> = <dA, A> = <dY, Y>, and <dX, X> = <dWq, Wq> + <dWk, Wk> + <dWv, Wv> = L
    r = _rng(12)
    S, H, Hq, Hkv = 7, 6, 10, 5
    X, Wq, Wk, Wv = r.standard_normal((S, H)), r.standard_normal((Hq, H)), r.standard_normal((Hkv, H)), \
        r.standard_normal((Hkv, H))
    dQ, dK, dV = r.standard_normal((S, Hq)), r.standard_normal((S, Hkv)), r.standard_normal((S, Hkv))
    Q, K, V = orc.qkv_projection(X, Wq, Wk, Wv)
    L = (dQ * Q).sum() + (dK * K).sum() + (dV * V).sum()
    dX, dWq, dWk, dWv = orc.qkv_projection_backward(X, Wq, Wk, Wv, dQ, dK, dV)
    assert abs((dX * X).sum() - L) <= 1e-12 * abs(L)
    assert abs((dWq * Wq).sum() + (dWk * Wk).sum() + (dWv * Wv).sum() - L) <= 1e-12 * abs(L)
    assert abs((dWq * Wq).sum() - (dQ * Q).sum()) <= 1e-12 * abs(L)
    A, Wo, dY = r.standard_normal((S, Hq)), r.standard_normal((H, Hq)), r.standard_normal((S, H))
    LY = (dY * orc.output_projection(A, Wo)).sum()
    dA, dWo = orc.output_projection_backward(A, Wo, dY)
    assert abs((dA * A).sum() - LY) <= 1e-12 * abs(LY) and abs((dWo * Wo).sum() - LY) <= 1e-12 * abs(LY)
    # zero upstream gradient -> zero gradients
    z = orc.qkv_projection_backward(X, Wq, Wk, Wv, 0 * dQ, 0 * dK, 0 * dV)
    assert not any(g.any() for g in z)


@pytest.mark.parametrize("D", [1, 2, 4])
def test_sharded_backward_sums_to_owner(D):
    r = _rng(13)
    S, H, Hq, Hkv = 8, 6, 8, 4
    X, Wq, Wk, Wv = r.standard_normal((S, H)), r.standard_normal((Hq, H)), r.standard_normal((Hkv, H)), \
        r.standard_normal((Hkv, H))
    dQ, dK, dV = r.standard_normal((S, Hq)), r.standard_normal((S, Hkv)), r.standard_normal((S, Hkv))
    ranks = lambda M: [M[p * (S // D):(p + 1) * (S // D)] for p in range(D)]
    dXs, dWq, dWk, dWv = orc.sharded_qkv_projection_backward(ranks(X), _shard_rows(Wq, D), _shard_rows(Wk, D),
                                                             _shard_rows(Wv, D), ranks(dQ), ranks(dK), ranks(dV))
    ref = orc.qkv_projection_backward(X, Wq, Wk, Wv, dQ, dK, dV)
    for got, want in zip((np.concatenate(dXs, axis=0), dWq, dWk, dWv), ref):
        np.testing.assert_allclose(got, want, rtol=1e-12, atol=1e-12)
    A, Wo, dY = r.standard_normal((S, Hq)), r.standard_normal((H, Hq)), r.standard_normal((S, H))
    dAs, dWos = orc.sharded_output_projection_backward(ranks(A), _shard_cols(Wo, D), ranks(dY))
    rdA, rdWo = orc.output_projection_backward(A, Wo, dY)
    np.testing.assert_allclose(np.concatenate(dAs, axis=0), rdA, rtol=1e-12, atol=1e-12)
    np.testing.assert_allclose(np.concatenate(dWos, axis=1), rdWo, rtol=1e-12, atol=1e-12)

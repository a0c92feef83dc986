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

"""Pins of the CPU oracle against things that are not the oracle.

Brute-force scalar loops (pure Python, math.fsum), closed forms, finite differences
and invariants of the gated MLP.  Each is chosen so that a plausible mistake in the
oracle (dropped term, wrong sign, transposed operand, wrong shard index) fails it.
"""
import math
import os

import numpy as np
import pytest

from oracle import tsp_mlp_oracle as orc

RNG = np.random.default_rng(1234)


# ---------------------------------------------------------------------------------------
# independent scalar implementation (no numpy arithmetic, no shared helpers)
# ---------------------------------------------------------------------------------------
def _sig(z):
    return 1.0 / (1.0 + math.exp(-z)) if z >= 0 else math.exp(z) / (1.0 + math.exp(z))


def brute_forward(X, Wg, Wu, Wd):
    S, H = len(X), len(X[0])
    F = len(Wd)
    Y = [[0.0] * H for _ in range(S)]
    for s in range(S):
        a = []
        for j in range(F):
            g = math.fsum(X[s][h] * Wg[h][j] for h in range(H))
            u = math.fsum(X[s][h] * Wu[h][j] for h in range(H))
            a.append(g * _sig(g) * u)
        for h in range(H):
            Y[s][h] = math.fsum(a[j] * Wd[j][h] for j in range(F))
    return Y


def _rand(*shape):
    return RNG.standard_normal(shape)


@pytest.mark.parametrize("S,H,F", [(4, 3, 4), (8, 16, 32), (5, 7, 6)])
def test_forward_matches_brute_force(S, H, F):
    X, Wg, Wu, Wd = _rand(S, H), _rand(H, F) / math.sqrt(H), _rand(H, F) / math.sqrt(H), _rand(F, H)
    Y = orc.gated_mlp_forward(X, Wg, Wu, Wd)
    Yb = np.array(brute_forward(X.tolist(), Wg.tolist(), Wu.tolist(), Wd.tolist()))
    assert Y.shape == (S, H)
    np.testing.assert_allclose(Y, Yb, rtol=1e-12, atol=1e-13)


def test_non_square_operands_are_not_transposed():
    # With H != F and asymmetric weights a transposed operand changes the shape or the value.
    S, H, F = 3, 2, 5
    X = np.arange(S * H, dtype=np.float64).reshape(S, H) / 7 - 0.3
    Wg = np.arange(H * F, dtype=np.float64).reshape(H, F) / 11 - 0.4
    Wu = np.arange(H * F, dtype=np.float64).reshape(H, F)[::-1] / 13 + 0.1
    Wd = np.arange(F * H, dtype=np.float64).reshape(F, H) / 5 - 0.9
    Yb = np.array(brute_forward(X.tolist(), Wg.tolist(), Wu.tolist(), Wd.tolist()))
    np.testing.assert_allclose(orc.gated_mlp_forward(X, Wg, Wu, Wd), Yb, rtol=1e-13, atol=1e-14)


# ---------------------------------------------------------------------------------------
# closed forms
# ---------------------------------------------------------------------------------------
def test_activation_golden_values(golden_dir):
    rows = []
    with open(os.path.join(golden_dir, "silu_closed_forms.txt")) as f:
        for line in f:
            if line.strip() and not line.startswith("#"):
                rows.append([float(v) for v in line.split()])
    assert len(rows) >= 5
    for z, s, sp in rows:
        assert abs(float(orc.silu(np.array([z]))[0]) - s) < 1e-14
        assert abs(float(orc.silu_prime(np.array([z]))[0]) - sp) < 1e-14


def test_activation_identities_and_extremes():
    z = np.linspace(-30, 30, 241)
    np.testing.assert_allclose(orc.silu(-z), orc.silu(z) - z, atol=1e-13)
    np.testing.assert_allclose(orc.silu_prime(-z), 1.0 - orc.silu_prime(z), atol=1e-13)
    big = np.array([-800.0, 800.0])
    assert np.all(np.isfinite(orc.silu(big))) and np.all(np.isfinite(orc.silu_prime(big)))
    assert orc.silu(big)[0] == 0.0 and orc.silu(big)[1] == 800.0
    # derivative against a central difference of silu itself
    zz = np.linspace(-6, 6, 49)
    e = 1e-6
    fd = (orc.silu(zz + e) - orc.silu(zz - e)) / (2 * e)
    np.testing.assert_allclose(orc.silu_prime(zz), fd, atol=1e-9)


def test_scalar_closed_form():
    # H = F = 1: y = silu(x wg) * (x wu) * wd
    x, wg, wu, wd = 1.0, 1.0, 3.0, -2.0
    y = orc.gated_mlp_forward([[x]], [[wg]], [[wu]], [[wd]])
    assert abs(y[0, 0] - 0.7310585786300049 * 3.0 * -2.0) < 1e-14
    y = orc.gated_mlp_forward([[-1.0]], [[1.0]], [[2.0]], [[0.5]])
    assert abs(y[0, 0] - (-0.2689414213699951) * (-2.0) * 0.5) < 1e-14


def test_zero_cases():
    X, Wg, Wu, Wd = _rand(6, 5), _rand(5, 8), _rand(5, 8), _rand(8, 5)
    assert np.all(orc.gated_mlp_forward(X, 0 * Wg, Wu, Wd) == 0)
    assert np.all(orc.gated_mlp_forward(0 * X, Wg, Wu, Wd) == 0)
    grads = orc.gated_mlp_backward(X, Wg, Wu, Wd, np.zeros((6, 5)))
    assert all(np.all(g == 0) for g in grads)


# ---------------------------------------------------------------------------------------
# invariants
# ---------------------------------------------------------------------------------------
def test_linearity_in_up_and_down_weights():
    X, Wg, Wu, Wd = _rand(6, 5), _rand(5, 8), _rand(5, 8), _rand(8, 5)
    Y = orc.gated_mlp_forward(X, Wg, Wu, Wd)
    np.testing.assert_allclose(orc.gated_mlp_forward(X, Wg, 2.5 * Wu, Wd), 2.5 * Y, rtol=1e-13)
    np.testing.assert_allclose(orc.gated_mlp_forward(X, Wg, Wu, -3.0 * Wd), -3.0 * Y, rtol=1e-13)
    # the gate is NOT linear: scaling Wg must not scale Y (catches gate/up swapped)
    assert not np.allclose(orc.gated_mlp_forward(X, 2.0 * Wg, Wu, Wd), 2.0 * Y, rtol=1e-3)


def test_intermediate_permutation_invariance():
    X, Wg, Wu, Wd = _rand(6, 5), _rand(5, 8), _rand(5, 8), _rand(8, 5)
    perm = RNG.permutation(8)
    np.testing.assert_allclose(orc.gated_mlp_forward(X, Wg[:, perm], Wu[:, perm], Wd[perm]),
                               orc.gated_mlp_forward(X, Wg, Wu, Wd), rtol=1e-12, atol=1e-13)


def test_token_row_independence():
    X, Wg, Wu, Wd = _rand(9, 5), _rand(5, 8), _rand(5, 8), _rand(8, 5)
    perm = RNG.permutation(9)
    Y = orc.gated_mlp_forward(X, Wg, Wu, Wd)
    np.testing.assert_allclose(orc.gated_mlp_forward(X[perm], Wg, Wu, Wd), Y[perm], rtol=1e-13)
    rows = np.array([7, 2, 2, 0])
    np.testing.assert_allclose(orc.forward_rows(X, Wg, Wu, Wd, rows), Y[rows], rtol=1e-13)


def _split(X, Wg, Wu, Wd, D, dY=None):
    S, F = X.shape[0], Wd.shape[0]
    Xs = [X[p * S // D:(p + 1) * S // D] for p in range(D)]
    Wgs = [Wg[:, k * F // D:(k + 1) * F // D] for k in range(D)]
    Wus = [Wu[:, k * F // D:(k + 1) * F // D] for k in range(D)]
    Wds = [Wd[k * F // D:(k + 1) * F // D] for k in range(D)]
    if dY is None:
        return Xs, Wgs, Wus, Wds
    return Xs, Wgs, Wus, Wds, [dY[p * S // D:(p + 1) * S // D] for p in range(D)]


@pytest.mark.parametrize("D", [1, 2, 4, 8, 16])
def test_ring_schedule_equals_unsharded(D):
    # After D steps every rank has applied every shard to its own tokens (Section 3.1).
    S, H, F = 32, 12, 48
    X, Wg, Wu, Wd = _rand(S, H), _rand(H, F) / 3, _rand(H, F) / 3, _rand(F, H) / 6
    Y = orc.gated_mlp_forward(X, Wg, Wu, Wd)
    Yr, order = orc.ring_gated_mlp_forward(*_split(X, Wg, Wu, Wd, D))
    np.testing.assert_allclose(np.concatenate(Yr, 0), Y, rtol=1e-12, atol=1e-12)
    assert order == orc.visiting_order(D)


def test_single_shard_is_plain_swiglu():
    S, H, F = 6, 5, 7
    X, Wg, Wu, Wd = _rand(S, H), _rand(H, F), _rand(H, F), _rand(F, H)
    Yr, order = orc.ring_gated_mlp_forward([X], [Wg], [Wu], [Wd])
    G = X @ Wg
    ref = ((G / (1 + np.exp(-G))) * (X @ Wu)) @ Wd
    np.testing.assert_allclose(Yr[0], ref, rtol=1e-12, atol=1e-13)
    assert order == [[0]]


@pytest.mark.parametrize("D", [1, 2, 3, 4, 8, 16])
def test_visiting_order_properties(D):
    order = orc.visiting_order(D)
    for p in range(D):
        assert order[p][0] == p                         # starts with its own shard
        assert sorted(order[p]) == list(range(D))       # meets every shard exactly once
        for t in range(D):
            assert order[p][t] == (p - t) % D           # receives from (p-1) mod D
    for t in range(D):
        assert sorted(order[p][t] for p in range(D)) == list(range(D))  # D distinct shards per step


# ---------------------------------------------------------------------------------------
# gradients
# ---------------------------------------------------------------------------------------
def _loss(X, Wg, Wu, Wd, dY):
    return float(np.sum(dY * orc.gated_mlp_forward(X, Wg, Wu, Wd)))


def test_gradients_per_element_finite_differences():
    S, H, F = 3, 4, 5
    X, Wg, Wu, Wd, dY = _rand(S, H), _rand(H, F) / 2, _rand(H, F) / 2, _rand(F, H) / 2, _rand(S, H)
    grads = orc.gated_mlp_backward(X, Wg, Wu, Wd, dY)
    params = [X, Wg, Wu, Wd]
    eps = 1e-6
    for which, (P, Gd) in enumerate(zip(params, grads)):
        assert Gd.shape == P.shape
        for idx in np.ndindex(P.shape):
            plus = [q.copy() for q in params]
            minus = [q.copy() for q in params]
            plus[which][idx] += eps
            minus[which][idx] -= eps
            fd = (_loss(*plus, dY) - _loss(*minus, dY)) / (2 * eps)
            assert abs(fd - Gd[idx]) < 1e-7 * max(1.0, abs(fd)), (which, idx, fd, Gd[idx])


def test_gradients_directional_finite_differences_medium():
    S, H, F = 24, 32, 40
    X, Wg, Wu, Wd, dY = _rand(S, H), _rand(H, F) / 6, _rand(H, F) / 6, _rand(F, H) / 6, _rand(S, H)
    grads = orc.gated_mlp_backward(X, Wg, Wu, Wd, dY)
    params = [X, Wg, Wu, Wd]
    eps = 1e-5
    for which in range(4):
        V = _rand(*params[which].shape)
        plus = [q.copy() for q in params]
        minus = [q.copy() for q in params]
        plus[which] = plus[which] + eps * V
        minus[which] = minus[which] - eps * V
        fd = (_loss(*plus, dY) - _loss(*minus, dY)) / (2 * eps)
        an = float(np.sum(grads[which] * V))
        assert abs(fd - an) <= 1e-7 * max(1.0, abs(an)), (which, fd, an)


def test_euler_identities():
    # Y is homogeneous of degree 1 in Wu and in Wd: <dWu, Wu> = <dWd, Wd> = <dY, Y>.
    S, H, F = 10, 6, 9
    X, Wg, Wu, Wd, dY = _rand(S, H), _rand(H, F), _rand(H, F), _rand(F, H), _rand(S, H)
    _, dWg, dWu, dWd = orc.gated_mlp_backward(X, Wg, Wu, Wd, dY)
    L = _loss(X, Wg, Wu, Wd, dY)
    assert abs(np.sum(dWu * Wu) - L) < 1e-11 * max(1, abs(L))
    assert abs(np.sum(dWd * Wd) - L) < 1e-11 * max(1, abs(L))


@pytest.mark.parametrize("D", [1, 2, 4, 8])
def test_ring_backward_sum_to_owner_equals_unsharded(D):
    S, H, F = 16, 6, 24
    X, Wg, Wu, Wd, dY = _rand(S, H), _rand(H, F) / 2, _rand(H, F) / 2, _rand(F, H) / 4, _rand(S, H)
    dX, dWg, dWu, dWd = orc.gated_mlp_backward(X, Wg, Wu, Wd, dY)
    rX, rWg, rWu, rWd = orc.ring_gated_mlp_backward(*_split(X, Wg, Wu, Wd, D, dY))
    np.testing.assert_allclose(np.concatenate(rX, 0), dX, rtol=1e-11, atol=1e-12)
    np.testing.assert_allclose(np.concatenate(rWg, 1), dWg, rtol=1e-11, atol=1e-12)
    np.testing.assert_allclose(np.concatenate(rWu, 1), dWu, rtol=1e-11, atol=1e-12)
    np.testing.assert_allclose(np.concatenate(rWd, 0), dWd, rtol=1e-11, atol=1e-12)


def test_sampled_modes_equal_full_mode():
    S, H, F = 20, 8, 12
    X, Wg, Wu, Wd, dY = _rand(S, H), _rand(H, F), _rand(H, F), _rand(F, H), _rand(S, H)
    dX, dWg, dWu, dWd = orc.gated_mlp_backward(X, Wg, Wu, Wd, dY)
    rows = np.array([0, 5, 19])
    cols = np.array([1, 4, 11])
    np.testing.assert_allclose(orc.backward_rows(X, Wg, Wu, Wd, dY, rows), dX[rows], rtol=1e-12, atol=1e-13)
    cWg, cWu, cWd = orc.backward_columns(X, Wg, Wu, Wd, dY, cols)
    np.testing.assert_allclose(cWg, dWg[:, cols], rtol=1e-12, atol=1e-13)
    np.testing.assert_allclose(cWu, dWu[:, cols], rtol=1e-12, atol=1e-13)
    np.testing.assert_allclose(cWd, dWd[cols], rtol=1e-12, atol=1e-13)


# ---------------------------------------------------------------------------------------
# statistics of the benchmark distribution
# ---------------------------------------------------------------------------------------
def test_output_scale_under_benchmark_distribution():
    # X ~ N(0,1), Wg,Wu ~ N(0,1/H), Wd ~ N(0,1/F): G,U ~ N(0,1) and var(Y) = E[silu(g)^2].
    from scipy import integrate

    second_moment, _ = integrate.quad(
        lambda g: (g / (1.0 + math.exp(-g))) ** 2 * math.exp(-g * g / 2) / math.sqrt(2 * math.pi), -12, 12)
    S, H, F = 64, 256, 512
    X, Wg, Wu, Wd = _rand(S, H), _rand(H, F) / math.sqrt(H), _rand(H, F) / math.sqrt(H), _rand(F, H) / math.sqrt(F)
    Y = orc.gated_mlp_forward(X, Wg, Wu, Wd)
    assert abs(Y.std() - math.sqrt(second_moment)) < 0.03
    assert abs(math.sqrt(second_moment) - 0.596) < 2e-3


# ---------------------------------------------------------------------------------------
# other gate activations (Algorithm 2 takes a generic "Activation sigma")
# ---------------------------------------------------------------------------------------
def _brute_forward_act(X, Wg, Wu, Wd, act):
    def sigma(g):
        if act == "gelu":
            return g * 0.5 * (1.0 + math.erf(g / math.sqrt(2.0)))
        if act == "relu":
            return g if g > 0 else 0.0
        return g * _sig(g)
    S, H, F = len(X), len(X[0]), len(Wd)
    Y = [[0.0] * H for _ in range(S)]
    for s in range(S):
        a = []
        for j in range(F):
            g = math.fsum(X[s][h] * Wg[h][j] for h in range(H))
            u = math.fsum(X[s][h] * Wu[h][j] for h in range(H))
            a.append(sigma(g) * u)
        for h in range(H):
            Y[s][h] = math.fsum(a[j] * Wd[j][h] for j in range(F))
    return Y


@pytest.mark.parametrize("act", ["silu", "gelu", "relu"])
def test_forward_brute_force_every_activation(act):
    S, H, F = 5, 6, 7
    X, Wg, Wu, Wd = _rand(S, H), _rand(H, F) / 2, _rand(H, F) / 2, _rand(F, H)
    Y = orc.gated_mlp_forward(X, Wg, Wu, Wd, act)
    Yb = np.array(_brute_forward_act(X.tolist(), Wg.tolist(), Wu.tolist(), Wd.tolist(), act))
    np.testing.assert_allclose(Y, Yb, rtol=1e-12, atol=1e-13)


def test_gelu_golden_values_and_identities(golden_dir):
    with open(os.path.join(golden_dir, "gelu_closed_forms.txt")) as f:
        rows = [[float(v) for v in ln.split()] for ln in f if ln.strip() and not ln.startswith("#")]
    assert len(rows) >= 5
    for z, g, gp in rows:
        assert abs(float(orc.gelu(np.array([z]))[0]) - g) < 1e-13
        assert abs(float(orc.gelu_prime(np.array([z]))[0]) - gp) < 1e-13
    z = np.linspace(-8, 8, 161)
    np.testing.assert_allclose(orc.gelu(-z), orc.gelu(z) - z, atol=1e-13)
    np.testing.assert_allclose(orc.gelu_prime(-z), 1.0 - orc.gelu_prime(z), atol=1e-13)
    e = 1e-6
    np.testing.assert_allclose(orc.gelu_prime(z), (orc.gelu(z + e) - orc.gelu(z - e)) / (2 * e), atol=1e-8)


def test_relu_values():
    z = np.array([-2.0, -0.0, 0.0, 0.5, 3.0])
    assert np.array_equal(orc.relu(z), np.array([0.0, 0.0, 0.0, 0.5, 3.0]))
    assert np.array_equal(orc.relu_prime(z), np.array([0.0, 0.0, 0.0, 1.0, 1.0]))


@pytest.mark.parametrize("act", ["gelu", "relu"])
def test_gradients_finite_differences_other_activations(act):
    S, H, F = 6, 5, 7
    X, Wg, Wu, Wd, dY = _rand(S, H), _rand(H, F) / 2, _rand(H, F) / 2, _rand(F, H) / 2, _rand(S, H)
    grads = orc.gated_mlp_backward(X, Wg, Wu, Wd, dY, act)
    params = [X, Wg, Wu, Wd]
    # relu is piecewise linear: keep the step far below the distance of any pre-activation to the kink
    eps = 1e-7 if act == "relu" else 1e-5
    assert act != "relu" or np.min(np.abs(X @ Wg)) > 1e-4
    for which in range(4):
        V = _rand(*params[which].shape)
        plus = [q.copy() for q in params]
        minus = [q.copy() for q in params]
        plus[which] = plus[which] + eps * V
        minus[which] = minus[which] - eps * V
        fd = (float(np.sum(dY * orc.gated_mlp_forward(*plus, act))) -
              float(np.sum(dY * orc.gated_mlp_forward(*minus, act)))) / (2 * eps)
        an = float(np.sum(grads[which] * V))
        assert abs(fd - an) <= 1e-6 * max(1.0, abs(an)), (act, which, fd, an)


@pytest.mark.parametrize("act", ["gelu", "relu"])
@pytest.mark.parametrize("D", [2, 4])
def test_ring_equals_unsharded_other_activations(act, D):
    S, H, F = 16, 6, 24
    X, Wg, Wu, Wd, dY = _rand(S, H), _rand(H, F) / 2, _rand(H, F) / 2, _rand(F, H) / 4, _rand(S, H)
    Yr, _ = orc.ring_gated_mlp_forward(*_split(X, Wg, Wu, Wd, D), act)
    np.testing.assert_allclose(np.concatenate(Yr, 0), orc.gated_mlp_forward(X, Wg, Wu, Wd, act), rtol=1e-12, atol=1e-12)
    dX, dWg, dWu, dWd = orc.gated_mlp_backward(X, Wg, Wu, Wd, dY, act)
    rX, rWg, rWu, rWd = orc.ring_gated_mlp_backward(*_split(X, Wg, Wu, Wd, D, dY), act)
    np.testing.assert_allclose(np.concatenate(rX, 0), dX, rtol=1e-11, atol=1e-12)
    np.testing.assert_allclose(np.concatenate(rWg, 1), dWg, rtol=1e-11, atol=1e-12)
    np.testing.assert_allclose(np.concatenate(rWd, 0), dWd, rtol=1e-11, atol=1e-12)

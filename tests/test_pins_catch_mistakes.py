"""Do the pins have teeth?  Plausible mistakes are planted in copies of the oracle's formulas and the same kinds of
checks the pin tests use (exact-sum brute force, finite differences, bilinear identities) must reject every one of
them, while accepting the oracle itself.

The mutants are written here (they are deliberately wrong); the checks use no matrix product of the oracle's.
"""
import math

import numpy as np
import pytest

from oracle import tsp_attn_proj_oracle as aorc
from oracle import tsp_mlp_oracle as orc


def _inputs(seed=0, S=5, H=4, F=6):
    r = np.random.default_rng(seed)
    return (r.standard_normal((S, H)), r.standard_normal((H, F)), r.standard_normal((H, F)),
            r.standard_normal((F, H)), r.standard_normal((S, H)))


def _brute_forward(X, Wg, Wu, Wd):
    S, H = X.shape
    F = Wg.shape[1]
    Y = np.zeros((S, H))
    for s in range(S):
        a = []
        for j in range(F):
            g = math.fsum(X[s, h] * Wg[h, j] for h in range(H))
            u = math.fsum(X[s, h] * Wu[h, j] for h in range(H))
            a.append(g / (1.0 + math.exp(-g)) * u)
        for n in range(H):
            Y[s, n] = math.fsum(a[j] * Wd[j, n] for j in range(F))
    return Y


def forward_ok(fwd) -> bool:
    X, Wg, Wu, Wd, _ = _inputs()
    return bool(np.allclose(fwd(X, Wg, Wu, Wd), _brute_forward(X, Wg, Wu, Wd), rtol=1e-11, atol=1e-12))


def backward_ok(bwd) -> bool:
    """Directional finite differences of L = <dY, Y> (Y from the brute-force forward) against the claimed gradients."""
    X, Wg, Wu, Wd, dY = _inputs(seed=1)
    grads = bwd(X, Wg, Wu, Wd, dY)
    args = [X, Wg, Wu, Wd]
    r = np.random.default_rng(2)
    eps = 1e-5
    for i in range(4):
        V = r.standard_normal(args[i].shape)
        plus = [a + eps * V if k == i else a for k, a in enumerate(args)]
        minus = [a - eps * V if k == i else a for k, a in enumerate(args)]
        fd = (float((dY * _brute_forward(*plus)).sum()) - float((dY * _brute_forward(*minus)).sum())) / (2 * eps)
        if abs(fd - float((grads[i] * V).sum())) > 1e-6 * max(1.0, abs(fd)):
            return False
    return True


def test_the_oracle_itself_passes():
    assert forward_ok(orc.gated_mlp_forward)
    assert backward_ok(orc.gated_mlp_backward)


def _sig(z):
    return 1.0 / (1.0 + np.exp(-z))


FORWARD_MUTANTS = {
    "gate and up swapped": lambda X, Wg, Wu, Wd: ((X @ Wu) * _sig(X @ Wu) * (X @ Wg)) @ Wd,
    "sigmoid instead of silu": lambda X, Wg, Wu, Wd: (_sig(X @ Wg) * (X @ Wu)) @ Wd,
    "silu applied to both": lambda X, Wg, Wu, Wd: ((X @ Wg) * _sig(X @ Wg) * (X @ Wu) * _sig(X @ Wu)) @ Wd,
    "sum instead of product": lambda X, Wg, Wu, Wd: ((X @ Wg) * _sig(X @ Wg) + (X @ Wu)) @ Wd,
    "last shard dropped": lambda X, Wg, Wu, Wd: (((X @ Wg) * _sig(X @ Wg) * (X @ Wu))[:, :-2]) @ Wd[:-2],
    "sign of the exponent": lambda X, Wg, Wu, Wd: ((X @ Wg) / (1.0 + np.exp(X @ Wg)) * (X @ Wu)) @ Wd,
}


@pytest.mark.parametrize("name", sorted(FORWARD_MUTANTS))
def test_forward_mutants_are_rejected(name):
    assert not forward_ok(FORWARD_MUTANTS[name]), name


def _mutant_backward(kind):
    def bwd(X, Wg, Wu, Wd, dY):
        G, U = X @ Wg, X @ Wu
        s = _sig(G)
        silu, dsilu = G * s, s * (1 + G * (1 - s))
        if kind == "silu' without the second term":
            dsilu = s
        if kind == "silu' with the wrong sign inside":
            dsilu = s * (1 - G * (1 - s))
        dA = dY @ Wd.T
        dU, dG = dA * silu, dA * U * dsilu
        if kind == "dU uses G instead of silu(G)":
            dU = dA * G
        if kind == "dG misses the factor U":
            dG = dA * dsilu
        dX = dG @ Wg.T + dU @ Wu.T
        if kind == "dX misses the up path":
            dX = dG @ Wg.T
        dWg, dWu, dWd = X.T @ dG, X.T @ dU, (silu * U).T @ dY
        if kind == "dWg and dWu swapped":
            dWg, dWu = dWu, dWg
        if kind == "dWd from G*U instead of A":
            dWd = (G * U).T @ dY
        if kind == "dWd pairs each token with another token's dY":
            dWd = (silu * U).T @ dY[::-1]
        return dX, dWg, dWu, dWd
    return bwd


BACKWARD_KINDS = ["silu' without the second term", "silu' with the wrong sign inside", "dU uses G instead of silu(G)",
                  "dG misses the factor U", "dX misses the up path", "dWg and dWu swapped", "dWd from G*U instead of A",
                  "dWd pairs each token with another token's dY"]


@pytest.mark.parametrize("kind", BACKWARD_KINDS)
def test_backward_mutants_are_rejected(kind):
    assert backward_ok(_mutant_backward("none"))        # the unmutated copy passes, so a rejection is the mutation's
    assert not backward_ok(_mutant_backward(kind)), kind


# ---- attention projections -------------------------------------------------------------------------------------------
def _attn_forward_ok(qkv, out) -> bool:
    r = np.random.default_rng(3)
    S, H, Hq, Hkv = 4, 5, 6, 3
    X, Wq, Wk, Wv = r.standard_normal((S, H)), r.standard_normal((Hq, H)), r.standard_normal((Hkv, H)), \
        r.standard_normal((Hkv, H))
    A, Wo = r.standard_normal((S, Hq)), r.standard_normal((H, Hq))

    def brute(M, W):
        return np.array([[math.fsum(M[s, h] * W[n, h] for h in range(M.shape[1])) for n in range(W.shape[0])]
                         for s in range(M.shape[0])])

    try:
        Q, K, V = qkv(X, Wq, Wk, Wv)
        Y = out(A, Wo)
        return bool(np.allclose(Q, brute(X, Wq), atol=1e-12) and np.allclose(K, brute(X, Wk), atol=1e-12)
                    and np.allclose(V, brute(X, Wv), atol=1e-12) and np.allclose(Y, brute(A, Wo), atol=1e-12))
    except ValueError:      # a transposed operand of a non-square matrix does not even multiply
        return False


def test_attention_projection_mutants_are_rejected():
    assert _attn_forward_ok(aorc.qkv_projection, aorc.output_projection)
    assert not _attn_forward_ok(lambda X, Wq, Wk, Wv: (X @ Wq.T, X @ Wv.T, X @ Wk.T), aorc.output_projection)   # K, V swapped
    assert not _attn_forward_ok(aorc.qkv_projection, lambda A, Wo: A @ Wo[:, ::-1].T)                            # heads reversed
    assert not _attn_forward_ok(aorc.qkv_projection, lambda A, Wo: A[:, :-1] @ Wo[:, :-1].T)                     # a column dropped
    assert not _attn_forward_ok(lambda X, Wq, Wk, Wv: (X @ Wq, X @ Wk, X @ Wv), aorc.output_projection)          # not transposed

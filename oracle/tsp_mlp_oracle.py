"""CPU fp64 oracle for the TSP gated ring MLP.  TEST INFRASTRUCTURE ONLY.

This file is the yardstick the CUDA path is measured against.  It is imported by
the tests, by the smoke check and by the bench's CPU-baseline legs, and by nothing
else: the product path never calls it and has no CPU fallback.  It shares no code
with the CUDA path (it imports only numpy and scipy.special.erf).

What it computes
----------------
Algorithm 2 (TSP Gated Ring MLP) lets rank p apply every weight shard to its own
token shard and add the contributions up locally; after D ring steps every rank
has applied every shard (Section 3.1), so the result is exactly the unsharded
gated MLP with three weight matrices (Section 4, model assumptions; "e.g. SwiGLU"):

    G = X Wg        U = X Wu        A = silu(G) * U        Y = A Wd

Two forward functions are given:
  * ``gated_mlp_forward``       the plain definition above, written out;
  * ``ring_gated_mlp_forward``  Algorithm 2 step by step (buffers, send/recv to the
                                ring neighbours, swap), for every rank p.
The tests prove they agree for every D.  Gradients (the paper only says that the
backward pass mirrors the forward weight movement and that per-shard partial
gradients are summed back to the shard's owner, Sections 4.3.4 and 4.7) are the
derivatives of the plain definition, again in a plain and a ring form.

The activation sigma of Algorithm 2 is a parameter: "silu" (default; the paper's
SwiGLU example), "gelu" (z * Phi(z), erf form) or "relu" (derivative 0 at z = 0).

Everything is float64; inputs are expected to be the bf16-rounded values widened
to float64.  Every function here is pinned by tests/test_oracle_pins.py (brute
force, closed forms, finite differences, invariants); none is "parity unpinned".
"""
from __future__ import annotations

import numpy as np
from scipy.special import erf as _erf


# ----------------------------------------------------------------------------------------
# activation
# ----------------------------------------------------------------------------------------
def sigmoid(z: np.ndarray) -> np.ndarray:
    """Logistic function, evaluated without overflow on either side of zero."""
    z = np.asarray(z, dtype=np.float64)
    out = np.empty_like(z)
    pos = z >= 0
    out[pos] = 1.0 / (1.0 + np.exp(-z[pos]))
    ez = np.exp(z[~pos])
    out[~pos] = ez / (1.0 + ez)
    return out


def silu(z: np.ndarray) -> np.ndarray:
    """Activation sigma of Algorithm 2, taken as SiLU: z * sigmoid(z)."""
    return np.asarray(z, dtype=np.float64) * sigmoid(z)


def silu_prime(z: np.ndarray) -> np.ndarray:
    """d/dz silu(z) = s(z) * (1 + z * (1 - s(z))), s = sigmoid."""
    s = sigmoid(z)
    return s * (1.0 + np.asarray(z, dtype=np.float64) * (1.0 - s))


def gelu(z: np.ndarray) -> np.ndarray:
    """z * Phi(z) with Phi the standard normal CDF, Phi(z) = (1 + erf(z / sqrt 2)) / 2."""
    z = np.asarray(z, dtype=np.float64)
    return z * 0.5 * (1.0 + _erf(z / np.sqrt(2.0)))


def gelu_prime(z: np.ndarray) -> np.ndarray:
    """Phi(z) + z * phi(z), phi the standard normal density."""
    z = np.asarray(z, dtype=np.float64)
    return 0.5 * (1.0 + _erf(z / np.sqrt(2.0))) + z * np.exp(-0.5 * z * z) / np.sqrt(2.0 * np.pi)


def relu(z: np.ndarray) -> np.ndarray:
    return np.maximum(np.asarray(z, dtype=np.float64), 0.0)


def relu_prime(z: np.ndarray) -> np.ndarray:
    return (np.asarray(z, dtype=np.float64) > 0).astype(np.float64)


ACTIVATIONS = {"silu": (silu, silu_prime), "gelu": (gelu, gelu_prime), "relu": (relu, relu_prime)}


# ----------------------------------------------------------------------------------------
# forward
# ----------------------------------------------------------------------------------------
def gated_mlp_forward(X, Wg, Wu, Wd, act="silu"):
    """Unsharded gated MLP.  X [S,H], Wg/Wu [H,F], Wd [F,H] -> Y [S,H].

    Body of Algorithm 2 with the whole weight matrices in place of one shard
    (W1^T = Wg, W3^T = Wu, W2 = Wd).
    """
    sigma, _ = ACTIVATIONS[act]
    X = np.asarray(X, dtype=np.float64)
    G = X @ np.asarray(Wg, dtype=np.float64)
    U = X @ np.asarray(Wu, dtype=np.float64)
    A = sigma(G) * U
    return A @ np.asarray(Wd, dtype=np.float64)


def ring_gated_mlp_forward(X_shards, Wg_shards, Wu_shards, Wd_shards, act="silu"):
    """Algorithm 2 executed for all D ranks.

    ``X_shards[p]`` is rank p's token shard [S/D, H]; ``W*_shards[p]`` the weight
    shards rank p owns (Wg/Wu: [H, F/D], Wd: [F/D, H]).  Returns the list of Y_p and
    the visiting table ``order[p][t]`` = index of the shard rank p computed with at
    step t (recorded from the simulated transfers, not from a formula).
    """
    sigma, _ = ACTIVATIONS[act]
    D = len(X_shards)
    # "W1, W2, W3 <- own shards"; `tag` remembers whose shard sits in the buffer.
    held = [(np.asarray(Wg_shards[p], np.float64), np.asarray(Wu_shards[p], np.float64),
             np.asarray(Wd_shards[p], np.float64), p) for p in range(D)]
    Y = [np.zeros_like(np.asarray(X_shards[p], np.float64)) for p in range(D)]
    order = [[-1] * D for _ in range(D)]
    for t in range(D):
        incoming = None
        if t < D - 1:
            # AsyncRingSendRecv: rank p sends its current buffers to (p+1) mod D and
            # receives those of (p-1) mod D into the primed buffers.
            incoming = [held[(p - 1) % D] for p in range(D)]
        for p in range(D):
            Wg_k, Wu_k, Wd_k, k = held[p]
            Xp = np.asarray(X_shards[p], np.float64)
            G = sigma(Xp @ Wg_k)         # gate projection + activation
            Hh = Xp @ Wu_k               # up projection
            Y[p] = Y[p] + (G * Hh) @ Wd_k  # down projection + accumulate
            order[p][t] = k
        if t < D - 1:
            held = incoming              # Wait(); swap buffers
    return Y, order


def visiting_order(D: int):
    """order[p][t]: which shard rank p holds at ring step t, by simulating the rotation."""
    held = list(range(D))
    order = [[-1] * D for _ in range(D)]
    for t in range(D):
        for p in range(D):
            order[p][t] = held[p]
        held = [held[(p - 1) % D] for p in range(D)]
    return order


# ----------------------------------------------------------------------------------------
# backward
# ----------------------------------------------------------------------------------------
def gated_mlp_backward(X, Wg, Wu, Wd, dY, act="silu"):
    """Gradients of L = <dY, Y> for the unsharded gated MLP.

    Returns dX [S,H], dWg [H,F], dWu [H,F], dWd [F,H].  Shard k's gradients are the
    column block (dWg, dWu) / row block (dWd) k of these.
    """
    X = np.asarray(X, np.float64)
    Wg = np.asarray(Wg, np.float64)
    Wu = np.asarray(Wu, np.float64)
    Wd = np.asarray(Wd, np.float64)
    dY = np.asarray(dY, np.float64)
    sigma, sigma_prime = ACTIVATIONS[act]
    G = X @ Wg
    U = X @ Wu
    sG = sigma(G)
    A = sG * U
    dA = dY @ Wd.T
    dU = dA * sG
    dG = dA * U * sigma_prime(G)
    dWd = A.T @ dY
    dWg = X.T @ dG
    dWu = X.T @ dU
    dX = dG @ Wg.T + dU @ Wu.T
    return dX, dWg, dWu, dWd


def ring_gated_mlp_backward(X_shards, Wg_shards, Wu_shards, Wd_shards, dY_shards, act="silu"):
    """Backward pass in ring form: each rank meets each shard once; the partial
    weight gradients a shard collects on its way round are summed to its owner.

    Returns (dX list per rank, dWg list per shard, dWu list per shard, dWd list per shard).
    Shard k meets the ranks in the order (k + t) mod D, t = 0..D-1.
    """
    D = len(X_shards)
    order = visiting_order(D)
    dX = [np.zeros_like(np.asarray(X_shards[p], np.float64)) for p in range(D)]
    dWg = [np.zeros_like(np.asarray(Wg_shards[k], np.float64)) for k in range(D)]
    dWu = [np.zeros_like(np.asarray(Wu_shards[k], np.float64)) for k in range(D)]
    dWd = [np.zeros_like(np.asarray(Wd_shards[k], np.float64)) for k in range(D)]
    for t in range(D):
        for p in range(D):
            k = order[p][t]
            dx, dwg, dwu, dwd = gated_mlp_backward(
                X_shards[p], Wg_shards[k], Wu_shards[k], Wd_shards[k], dY_shards[p], act)
            dX[p] = dX[p] + dx
            dWg[k] = dWg[k] + dwg       # sum-to-owner
            dWu[k] = dWu[k] + dwu
            dWd[k] = dWd[k] + dwd
    return dX, dWg, dWu, dWd


# ----------------------------------------------------------------------------------------
# sampled modes for sizes where the full fp64 pass is too slow
# ----------------------------------------------------------------------------------------
def forward_rows(X, Wg, Wu, Wd, rows, act="silu"):
    """Rows `rows` of Y.  Token rows are independent, so this is the plain forward on X[rows]."""
    return gated_mlp_forward(np.asarray(X)[rows], Wg, Wu, Wd, act)


def backward_rows(X, Wg, Wu, Wd, dY, rows, act="silu"):
    """Rows `rows` of dX (needs only those rows of X and dY, and all weights)."""
    dX, _, _, _ = gated_mlp_backward(np.asarray(X)[rows], Wg, Wu, Wd, np.asarray(dY)[rows], act)
    return dX


def backward_columns(X, Wg, Wu, Wd, dY, cols, act="silu"):
    """dWg[:, cols], dWu[:, cols], dWd[cols, :].

    Intermediate column j of G, U, dA depends only on column j of Wg, Wu and row j of
    Wd, so the weight gradients of those columns follow from the reduced problem.
    """
    Wg = np.asarray(Wg)[:, cols]
    Wu = np.asarray(Wu)[:, cols]
    Wd = np.asarray(Wd)[cols, :]
    _, dWg, dWu, dWd = gated_mlp_backward(X, Wg, Wu, Wd, dY, act)
    return dWg, dWu, dWd

"""CPU fp64 oracle for the projection GEMMs of TSP attention.  TEST INFRASTRUCTURE ONLY.

Imported by the tests (and the smoke check) and by nothing else; the product path never calls it and has no CPU
fallback.  It shares no code with the CUDA path (numpy only).

What it computes
----------------
Algorithm 1 (TSP multi-head attention, forward pass on rank p) loops over the D weight-owning ranks r.  In each
iteration every rank projects its own tokens with shard r's weights,

    Q = X W_Q^(r)T      K = X W_K^(r)T      V = X W_V^(r)T          W_Q^(r), W_K^(r), W_V^(r) in R^{(h/D) x h}

(GQA with group size g: the K / V shards are h/(gD) wide), runs attention on those heads, and adds the heads'
output through shard r of the output projection,

    Y <- Y + Flatten(A) W_O^(r)T                                    W_O^(r) in R^{h x (h/D)},  Y starts at 0.

Only these two dense steps are covered; the attention core between them (K/V all-gather, zigzag reorder, causal
attention) is not.  Shard r holds heads r*H_s .. (r+1)*H_s - 1, so stacking the shards' rows gives the ordinary
projection matrices and the loop reaches exactly the unsharded result:

    Q = X Wq^T [S, Hq]   K = X Wk^T [S, Hkv]   V = X Wv^T [S, Hkv]       Y = A Wo^T [S, H],   Wo = [Wo^(0) | .. | Wo^(D-1)]

Backward (the paper only says that the backward pass mirrors the forward weight movement and that the partial
weight gradients the ranks produce for a shard are summed to its owner, Sections 4.3.4 and 4.7): the derivatives of
the two definitions for upstream gradients dQ, dK, dV and dY,

    dX = dQ Wq + dK Wk + dV Wv      dWq = dQ^T X   dWk = dK^T X   dWv = dV^T X      dA = dY Wo      dWo = dY^T A

with the sums over tokens running over ALL ranks' tokens (that is the sum-to-owner).

Each step is given twice: the plain definition, and the loop of Algorithm 1 written out shard by shard (the tests
prove the two agree for every D).  Everything is float64 on the bf16-rounded input values.  Every function is
pinned by tests/test_attn_oracle_pins.py (brute force with exact summation, closed forms, invariants); none is
"parity unpinned".
"""
from __future__ import annotations

import numpy as np


def qkv_projection(X, Wq, Wk, Wv):
    """Q, K, V of the unsharded layer.  X [S, H]; Wq [Hq, H]; Wk, Wv [Hkv, H] (rows = output features)."""
    return X @ Wq.T, X @ Wk.T, X @ Wv.T


def output_projection(A, Wo):
    """Y = A Wo^T.  A [S, Hq] (heads flattened along the columns); Wo [H, Hq]."""
    return A @ Wo.T


def sharded_qkv_projection(X, Wq_shards, Wk_shards, Wv_shards):
    """The projection lines of Algorithm 1, iteration by iteration.

    Wq_shards[r] is W_Q^(r) [Hq/D, H] and so on.  Iteration r yields that shard's heads; they are laid side by
    side in head order (shard r = heads r*H_s .. (r+1)*H_s - 1).
    """
    D = len(Wq_shards)
    Q_parts, K_parts, V_parts = [], [], []
    for r in range(D):                       # loop over weight-owning ranks
        Q_parts.append(X @ Wq_shards[r].T)   # local projections with the shard that was broadcast
        K_parts.append(X @ Wk_shards[r].T)
        V_parts.append(X @ Wv_shards[r].T)
    return np.concatenate(Q_parts, axis=1), np.concatenate(K_parts, axis=1), np.concatenate(V_parts, axis=1)


def sharded_output_projection(A_shards, Wo_shards):
    """Output projection + accumulate of Algorithm 1: Y <- 0; for r = 0..D-1: Y <- Y + A_r W_O^(r)T.

    A_shards[r] [S, Hq/D] is the attention output of shard r's heads, Wo_shards[r] is W_O^(r) [H, Hq/D].
    """
    Y = np.zeros((A_shards[0].shape[0], Wo_shards[0].shape[0]))
    for r in range(len(A_shards)):
        Y = Y + A_shards[r] @ Wo_shards[r].T
    return Y


def qkv_rows(X, Wq, Wk, Wv, rows):
    """Sampled mode: the projections are row-separable, so rows `rows` need only those rows of X."""
    return qkv_projection(X[rows], Wq, Wk, Wv)


def output_rows(A, Wo, rows):
    return output_projection(A[rows], Wo)


# ----------------------------------------------------------------------------------------
# backward
# ----------------------------------------------------------------------------------------
def qkv_projection_backward(X, Wq, Wk, Wv, dQ, dK, dV):
    """Gradients of L = <dQ, Q> + <dK, K> + <dV, V>: returns dX [S, H], dWq [Hq, H], dWk, dWv [Hkv, H]."""
    dX = dQ @ Wq + dK @ Wk + dV @ Wv
    return dX, dQ.T @ X, dK.T @ X, dV.T @ X


def output_projection_backward(A, Wo, dY):
    """Gradients of L = <dY, Y>: returns dA [S, Hq] and dWo [H, Hq]."""
    return dY @ Wo, dY.T @ A


def sharded_qkv_projection_backward(X_ranks, Wq_shards, Wk_shards, Wv_shards, dQ_ranks, dK_ranks, dV_ranks):
    """The same gradients formed the way the sharded schedule forms them.

    X_ranks[p] [S_loc, H] are rank p's tokens, dQ_ranks[p] [S_loc, Hq] etc. its upstream gradients.  In iteration r
    every rank p adds shard r's term to its dX and produces a partial gradient for shard r's rows; the partials of
    all ranks are summed to the owner r.  Returns (list of dX per rank, dWq, dWk, dWv stacked in shard order).
    """
    D, P = len(Wq_shards), len(X_ranks)
    q_w, kv_w = Wq_shards[0].shape[0], Wk_shards[0].shape[0]
    dX = [np.zeros_like(X_ranks[p]) for p in range(P)]
    dWq = [np.zeros_like(Wq_shards[r]) for r in range(D)]
    dWk = [np.zeros_like(Wk_shards[r]) for r in range(D)]
    dWv = [np.zeros_like(Wv_shards[r]) for r in range(D)]
    for r in range(D):
        q_cols, kv_cols = slice(r * q_w, (r + 1) * q_w), slice(r * kv_w, (r + 1) * kv_w)
        for p in range(P):
            dq, dk, dv = dQ_ranks[p][:, q_cols], dK_ranks[p][:, kv_cols], dV_ranks[p][:, kv_cols]
            dX[p] = dX[p] + dq @ Wq_shards[r] + dk @ Wk_shards[r] + dv @ Wv_shards[r]
            dWq[r] = dWq[r] + dq.T @ X_ranks[p]       # partial of rank p, summed to owner r
            dWk[r] = dWk[r] + dk.T @ X_ranks[p]
            dWv[r] = dWv[r] + dv.T @ X_ranks[p]
    return dX, np.concatenate(dWq, axis=0), np.concatenate(dWk, axis=0), np.concatenate(dWv, axis=0)


def sharded_output_projection_backward(A_ranks, Wo_shards, dY_ranks):
    """dA per rank (heads of shard r in columns r*Hq/D ..) and dWo shards summed over the ranks' tokens."""
    D, P = len(Wo_shards), len(A_ranks)
    w = Wo_shards[0].shape[1]
    dA = [np.zeros_like(A_ranks[p]) for p in range(P)]
    dWo = [np.zeros_like(Wo_shards[r]) for r in range(D)]
    for r in range(D):
        cols = slice(r * w, (r + 1) * w)
        for p in range(P):
            dA[p][:, cols] = dY_ranks[p] @ Wo_shards[r]
            dWo[r] = dWo[r] + dY_ranks[p].T @ A_ranks[p][:, cols]
    return dA, dWo

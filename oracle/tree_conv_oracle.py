"""CPU fp64 oracle for the tree-parallel causal convolution front end (Stage 1).

TEST INFRASTRUCTURE ONLY (see tree_oracle.py): numpy, float64, imported only by
tests, the smoke check and the benchmark's CPU-baseline leg.

What it computes.  Section II-A: a linear-attention layer forms q, k and v by
passing its projected inputs through a short causal depthwise convolution.
Section IV-C, Stage 1: under a proposal tree the taps of that convolution for a
node are the node's ancestors along its root-to-node path (then the committed
context), not its neighbours in the flattened order, and the stage applies the
convolution, the bias and SiLU in one pass:

    y_i[c] = SiLU( bias[c] + sum_{r=0}^{W-1} w[c][W-1-r] * in_r(i)[c] )

where in_0(i) = x_i, in_1(i) = x_pi(i), in_2(i) = x_pi(pi(i)), ... and, once
the path reaches the virtual root, the sequence continues into the committed
context: ctx[W-2] is the token just before the tree, ctx[W-3] the one before
it, and so on (ctx has W-1 rows, oldest first).  w[c][W-1] multiplies the
current token (the usual causal depthwise layout), SiLU(z) = z / (1 + e^-z).

Readings of what the paper leaves open, fixed here:
the channel order is [q heads | k heads | v heads]; the normalisation that the
paper folds into its stages without a formula is read as an optional L2
normalisation of each q and k head vector after SiLU, x / sqrt(sum x^2 + eps);
the gate formulas are not given by the paper either (see gate_prep below).

Pins.  tree_conv and conv_commit are pinned by what the definition fixes (hand
example, numpy.convolve on chains, path locality, ...).  gate_prep and the
normalisation are readings: their tests fix the reading against library
softplus / sigmoid and closed forms, but nothing in the paper fixes the formula
itself -- parity of gate_prep is UNPINNED BY THE PAPER.
"""
from __future__ import annotations

import numpy as np


def silu(z):
    return z / (1.0 + np.exp(-z))


def conv_inputs_for_node(x, ctx, parent, i, W):
    """The W inputs [in_0, ..., in_{W-1}] of node i: itself, then its ancestors
    from the nearest upwards, then the context from its newest row backwards."""
    rows = []
    j = int(i)
    while j >= 0 and len(rows) < W:
        rows.append(x[j])
        j = int(parent[j])
    back = ctx.shape[0] - 1
    while len(rows) < W:
        rows.append(ctx[back])
        back -= 1
    return rows


def tree_conv(x, ctx, weight, bias, parent):
    """x [T, C], ctx [W-1, C], weight [C, W], bias [C] or None -> y [T, C]."""
    T, C = x.shape
    W = weight.shape[1]
    y = np.zeros((T, C))
    for i in range(T):
        rows = conv_inputs_for_node(x, ctx, parent, i, W)
        z = np.zeros(C) if bias is None else np.array(bias, dtype=np.float64)
        for r in range(W):
            z = z + weight[:, W - 1 - r] * rows[r]
        y[i] = silu(z)
    return y


def split_heads(y, H, dk, dv, normalize_qk=False, eps=1e-6):
    """[T, H(2dk+dv)] -> q [H,T,dk], k [H,T,dk], v [H,T,dv] (channel order q|k|v)."""
    T = y.shape[0]
    q = y[:, :H * dk].reshape(T, H, dk).transpose(1, 0, 2).copy()
    k = y[:, H * dk:2 * H * dk].reshape(T, H, dk).transpose(1, 0, 2).copy()
    v = y[:, 2 * H * dk:].reshape(T, H, dv).transpose(1, 0, 2).copy()
    if normalize_qk:
        q = q / np.sqrt((q * q).sum(-1, keepdims=True) + eps)
        k = k / np.sqrt((k * k).sum(-1, keepdims=True) + eps)
    return q, k, v


def tree_conv_batch(x, ctx, weight, bias, parents, H, dk, dv, normalize_qk=False, eps=1e-6):
    """x [B,T,C], ctx [B,W-1,C] -> q,k [B,H,T,dk], v [B,H,T,dv]."""
    B = x.shape[0]
    qs, ks, vs = [], [], []
    for b in range(B):
        par = parents[0] if parents.shape[0] == 1 else parents[b]
        y = tree_conv(np.asarray(x[b], np.float64), np.asarray(ctx[b], np.float64),
                      np.asarray(weight, np.float64), None if bias is None else np.asarray(bias, np.float64), par)
        q, k, v = split_heads(y, H, dk, dv, normalize_qk, eps)
        qs.append(q); ks.append(k); vs.append(v)
    return np.stack(qs), np.stack(ks), np.stack(vs)


def gate_prep(a, b, A_log, dt_bias):
    """Gate preparation of Stage 1.  The paper names the step and gives no formula; this is the
    parameterisation of the Gated DeltaNet publication it cites for the layer:

        gamma = exp( -exp(A_log[h]) * softplus(a + dt_bias[h]) )      (decay, in (0, 1])
        beta  = 1 / (1 + exp(-b))                                     (write strength, in (0, 1))

    a, b [T, H] -> gamma, beta [H, T] (head-major, the layout the verification stage reads).
    """
    a = np.asarray(a, np.float64)
    b = np.asarray(b, np.float64)
    z = a + np.asarray(dt_bias, np.float64)[None, :]
    softplus = np.maximum(z, 0.0) + np.log1p(np.exp(-np.abs(z)))
    gamma = np.exp(-np.exp(np.asarray(A_log, np.float64))[None, :] * softplus)
    beta = 1.0 / (1.0 + np.exp(-b))
    return gamma.T.copy(), beta.T.copy()


def conv_commit(x, ctx, parent, accepted):
    """Context rows after the accepted path is committed: the last W-1 rows of the sequence
    [ctx rows, x along the accepted root-to-node path].  accepted = -1 keeps ctx.
    (Implied by Section IV-D's commit for a layer whose front end is the convolution: the next
    round's taps must be the committed tokens; the paper does not spell it out.)"""
    path = []
    j = int(accepted)
    while j >= 0:
        path.append(j)
        j = int(parent[j])
    path.reverse()
    seq = np.concatenate([ctx, x[path]]) if path else np.array(ctx, copy=True)
    keep = ctx.shape[0]
    return seq[seq.shape[0] - keep:].copy()

"""fp64 CPU oracle of the harmonized-context-alignment (HCA) attention of the draft layer.

TEST INFRASTRUCTURE ONLY: imported by the tests, by the smoke check and by the
benchmark's CPU-baseline leg. It shares no code with the CUDA path.

What it computes (Section 3.2, "Harmonized Context Alignment"): in aligning step
j = m + 1 the query at position t attends causally to a key/value sequence of its own.
Position s <= t of that sequence holds the target LLM's feature when it lies at least m
positions back (t - s >= m); the m most recent positions hold draft features instead,
position s = t - i taken from the i-th most recent earlier draft pass (i = 0 is the
latest pass and sits at the query's own position). The output is an ordinary softmax
attention of the query over that sequence:

    k(t, s), v(t, s) = K_t[s], V_t[s]            if t - s >= m
                       K_d[t - s][s], V_d[t - s][s]  otherwise
    w[t, .] = softmax_{s <= t}( scale * <Q[t], k(t, s)> ),   O[t] = sum_s w[t, s] v(t, s)

The code below is that definition written out: one query at a time, its key and value
sequences assembled explicitly, then a plain fp64 softmax attention over them.

Reading taken where the appendix listing and the text differ: the listing multiplies the
value substitution by the score matrix *before* the softmax; the text defines keys and
values as the concatenation of target and draft features, i.e. an attention over the
substituted sequence with normalised weights. This oracle follows the text. A draft pass
i >= T meets no (query, key) pair of a T-position sequence and is inert.

Layout: Q [B, T, H, D]; K_t, V_t [B, T, Hkv, D] with H a multiple of Hkv (query head h
reads key/value head h // (H // Hkv)); K_d, V_d: sequences of m arrays shaped like K_t,
index i = how many positions behind the query the pass is used. All arithmetic in float64.
"""
from __future__ import annotations

import math
from typing import Optional, Sequence

import numpy as np


def _as64(x) -> np.ndarray:
    return np.asarray(x, dtype=np.float64)


class _Context:
    """Key and value sequences of one (sequence, key/value head) as each query sees them: a working copy of
    the target rows in which, for the query at hand, the rows of its m most recent positions are replaced by
    the draft passes' rows (and put back afterwards)."""

    def __init__(self, k_t, v_t, k_d, v_d):
        self.k_t, self.v_t, self.k_d, self.v_d = k_t, v_t, k_d, v_d
        self.keys, self.vals = k_t.copy(), v_t.copy()

    def enter(self, t):
        for i in range(len(self.k_d)):
            s = t - i
            if s < 0:
                break
            self.keys[s] = self.k_d[i][s]
            self.vals[s] = self.v_d[i][s]
        return self.keys[:t + 1], self.vals[:t + 1]

    def leave(self, t):
        for i in range(len(self.k_d)):
            s = t - i
            if s < 0:
                break
            self.keys[s] = self.k_t[s]
            self.vals[s] = self.v_t[s]


def hca_attention(Q, K_t, V_t, K_d: Sequence = (), V_d: Sequence = (), scale: Optional[float] = None):
    """Forward pass. Returns (O [B, T, H, D], lse [B, H, T]) with lse the natural-log
    normaliser of each query's scores over its own key sequence."""
    Q, K_t, V_t = _as64(Q), _as64(K_t), _as64(V_t)
    K_d = [_as64(x) for x in K_d]
    V_d = [_as64(x) for x in V_d]
    assert len(K_d) == len(V_d)
    B, T, H, D = Q.shape
    Hkv = K_t.shape[2]
    assert H % Hkv == 0
    rep = H // Hkv
    if scale is None:
        scale = 1.0 / math.sqrt(D)
    O = np.zeros((B, T, H, D))
    lse = np.zeros((B, H, T))
    for b in range(B):
        for g in range(Hkv):
            ctx = _Context(K_t[b, :, g, :], V_t[b, :, g, :], [x[b, :, g, :] for x in K_d],
                           [x[b, :, g, :] for x in V_d])
            for t in range(T):
                keys, vals = ctx.enter(t)
                for h in range(g * rep, (g + 1) * rep):
                    sc = (keys @ Q[b, t, h]) * scale
                    mx = sc.max()
                    e = np.exp(sc - mx)
                    den = e.sum()
                    O[b, t, h] = (e / den) @ vals
                    lse[b, h, t] = mx + math.log(den)
                ctx.leave(t)
    return O, lse


def hca_attention_grad(Q, K_t, V_t, K_d: Sequence, V_d: Sequence, dO, scale: Optional[float] = None):
    """Gradients of sum(O * dO) with respect to every input: the chain rule through each query's softmax
    attention (dw = <dO[t], v(t, s)>, ds = w (dw - sum_s w dw) scale), with the gradient of every key and
    value row sent back to the tensor the row came from.
    Returns (dQ, dK_t, dV_t, [dK_d], [dV_d]) with the inputs' shapes."""
    Q, K_t, V_t, dO = _as64(Q), _as64(K_t), _as64(V_t), _as64(dO)
    K_d = [_as64(x) for x in K_d]
    V_d = [_as64(x) for x in V_d]
    B, T, H, D = Q.shape
    Hkv = K_t.shape[2]
    rep = H // Hkv
    m = len(K_d)
    if scale is None:
        scale = 1.0 / math.sqrt(D)
    dQ = np.zeros_like(Q)
    dK_t, dV_t = np.zeros_like(K_t), np.zeros_like(V_t)
    dK_d = [np.zeros_like(K_t) for _ in range(m)]
    dV_d = [np.zeros_like(V_t) for _ in range(m)]
    pos = np.arange(T)
    from_target = (pos[:, None] - pos[None, :]) >= m          # [t, s]: the pair (t, s) uses the target's row s
    for b in range(B):
        for g in range(Hkv):
            ctx = _Context(K_t[b, :, g, :], V_t[b, :, g, :], [x[b, :, g, :] for x in K_d],
                           [x[b, :, g, :] for x in V_d])
            for h in range(g * rep, (g + 1) * rep):
                # per-query weights w[t, s] and score gradients ds[t, s] (zero for s > t)
                w = np.zeros((T, T))
                ds = np.zeros((T, T))
                for t in range(T):
                    keys, vals = ctx.enter(t)
                    sc = (keys @ Q[b, t, h]) * scale
                    e = np.exp(sc - sc.max())
                    wt = e / e.sum()
                    dw = vals @ dO[b, t, h]
                    dst = wt * (dw - wt @ dw) * scale
                    dQ[b, t, h] = dst @ keys
                    w[t, :t + 1] = wt
                    ds[t, :t + 1] = dst
                    ctx.leave(t)
                # dk(t, s) = ds[t, s] Q[t] and dv(t, s) = w[t, s] dO[t], summed into the row's own tensor
                dK_t[b, :, g, :] += np.where(from_target, ds, 0.0).T @ Q[b, :, h, :]
                dV_t[b, :, g, :] += np.where(from_target, w, 0.0).T @ dO[b, :, h, :]
                for i in range(min(m, T)):
                    s = pos[:T - i]                            # keys that have a query i positions ahead
                    dK_d[i][b, s, g, :] += ds[s + i, s][:, None] * Q[b, s + i, h, :]
                    dV_d[i][b, s, g, :] += w[s + i, s][:, None] * dO[b, s + i, h, :]
    return dQ, dK_t, dV_t, dK_d, dV_d

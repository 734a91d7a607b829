"""fp64 CPU oracle of the harmonized-context-alignment (HCA) attention of the draft layer.

TEST INFRASTRUCTURE ONLY: imported by the tests, by the smoke check and by the
benchmark's CPU-baseline leg. It shares no code with the CUDA path.

What it computes (Section 3.2, and the attention listing of the appendix): in aligning
step j = m + 1 the query at position t attends, causally, to keys and values that come
from the target LLM's features everywhere except on the m most recent positions, where
they come from the draft features of the earlier passes: the pair (t, s) with
t - s = i < m uses the keys/values of the i-th most recent draft pass (i = 0 is the
latest pass and sits on the main diagonal). The steps below follow the listing's
order: target scores with the causal mask, sub-diagonal overwrite with draft scores,
softmax, product with the target values, then one correction per sub-diagonal that
swaps the target value for the draft value.

Reading taken where the listing and the text differ: the listing weights the value
correction with the score matrix *before* the softmax; the text defines keys and values
as the concatenation of target and draft features, i.e. an ordinary attention over the
substituted key/value sequence. This oracle follows the text and uses the normalised
weights, so that every output row is a convex combination of the value rows it attends
to (pinned in the tests against the text's concatenation written out per query).

Layout: Q [B, T, H, D]; K_t, V_t [B, T, Hkv, D] with H a multiple of Hkv (query head h
reads key/value head h // (H // Hkv)); K_d, V_d: sequences of m arrays shaped like K_t,
index i = the sub-diagonal they replace. All arithmetic in float64.
"""
from __future__ import annotations

import math
from typing import Optional, Sequence

import numpy as np


def _as64(x) -> np.ndarray:
    return np.asarray(x, dtype=np.float64)


def hca_attention(Q, K_t, V_t, K_d: Sequence = (), V_d: Sequence = (), scale: Optional[float] = None):
    """Forward pass. Returns (O [B, T, H, D], lse [B, H, T]) with lse the natural-log
    normaliser of each query row after the sub-diagonal overwrite."""
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
    idx = np.arange(T)
    mask = np.where(idx[None, :] > idx[:, None], -np.inf, 0.0)          # causal: s > t is hidden
    for b in range(B):
        for h in range(H):
            g = h // rep
            q = Q[b, :, h, :]
            k_t, v_t = K_t[b, :, g, :], V_t[b, :, g, :]
            w = q @ k_t.T * scale + mask
            for i in range(len(K_d)):
                if i >= T:
                    continue        # sub-diagonal i of a T x T matrix is empty
                ind_q, ind_k = idx[i:], idx[:T - i]
                w_d = q @ K_d[i][b, :, g, :].T * scale
                w[ind_q, ind_k] = w_d[ind_q, ind_k]
            mx = w.max(axis=1, keepdims=True)
            e = np.exp(w - mx)
            den = e.sum(axis=1, keepdims=True)
            wn = e / den
            out = wn @ v_t
            for i in range(len(V_d)):
                if i >= T:
                    continue        # sub-diagonal i of a T x T matrix is empty
                ind_q, ind_k = idx[i:], idx[:T - i]
                v_d = V_d[i][b, :, g, :]
                out[ind_q] += wn[ind_q, ind_k][:, None] * (v_d[ind_k] - v_t[ind_k])
            O[b, :, h, :] = out
            lse[b, h, :] = (mx + np.log(den))[:, 0]
    return O, lse


def hca_attention_grad(Q, K_t, V_t, K_d: Sequence, V_d: Sequence, dO, scale: Optional[float] = None):
    """Gradients of sum(O * dO) with respect to every input, by the chain rule through the
    steps of hca_attention (softmax Jacobian: dS = W * (dW - rowsum(W * dW))).
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
    idx = np.arange(T)
    mask = np.where(idx[None, :] > idx[:, None], -np.inf, 0.0)
    for b in range(B):
        for h in range(H):
            g = h // rep
            q = Q[b, :, h, :]
            do = dO[b, :, h, :]
            k_t, v_t = K_t[b, :, g, :], V_t[b, :, g, :]
            w = q @ k_t.T * scale + mask
            for i in range(m):
                if i >= T:
                    continue        # sub-diagonal i of a T x T matrix is empty
                ind_q, ind_k = idx[i:], idx[:T - i]
                w[ind_q, ind_k] = (q @ K_d[i][b, :, g, :].T * scale)[ind_q, ind_k]
            wn = np.exp(w - w.max(axis=1, keepdims=True))
            wn /= wn.sum(axis=1, keepdims=True)
            # d(loss)/d(wn): against the value each pair actually uses
            dwn = do @ v_t.T
            for i in range(m):
                if i >= T:
                    continue        # sub-diagonal i of a T x T matrix is empty
                ind_q, ind_k = idx[i:], idx[:T - i]
                dwn[ind_q, ind_k] = np.einsum("td,td->t", do[ind_q], V_d[i][b, ind_k, g, :])
            ds = wn * (dwn - (wn * dwn).sum(axis=1, keepdims=True)) * scale
            # split weights and score gradients into the part that meets target keys/values
            # and the sub-diagonals that meet draft keys/values
            wn_t, ds_t = wn.copy(), ds.copy()
            for i in range(m):
                if i >= T:
                    continue        # sub-diagonal i of a T x T matrix is empty
                ind_q, ind_k = idx[i:], idx[:T - i]
                wd, dsd = wn[ind_q, ind_k], ds[ind_q, ind_k]
                wn_t[ind_q, ind_k] = 0.0
                ds_t[ind_q, ind_k] = 0.0
                dV_d[i][b, ind_k, g, :] += wd[:, None] * do[ind_q]
                dK_d[i][b, ind_k, g, :] += dsd[:, None] * q[ind_q]
                dQ[b, ind_q, h, :] += dsd[:, None] * K_d[i][b, ind_k, g, :]
            dV_t[b, :, g, :] += wn_t.T @ do
            dK_t[b, :, g, :] += ds_t.T @ q
            dQ[b, :, h, :] += ds_t @ k_t
    return dQ, dK_t, dV_t, dK_d, dV_d

"""Comparison of the CUDA path's outputs with the fp64 oracle, row subset by row subset.

Tolerances (stated by the benchmark spec for this path):
  * Top-K index sets identical, except that an element may differ when its target logit is
    within TIE_TOL of the oracle's K-th largest target logit (a near-tie at rank K / K+1);
    such a row is re-scored by the oracle on the GPU's own set, since both sets are valid.
  * per-row loss within LOSS_RTOL relative error (floor 1e-6 on the reference magnitude).
  * dH_d within DH_TOL * max|dH_d| over the compared rows.
lse and q are fp32 results of an fp32 log-sum-exp; they get LSE_ATOL / Q_RTOL.
"""
from __future__ import annotations

import numpy as np
import torch

import hass_inputs as hi
import oracle

TIE_TOL = 1e-3
LOSS_RTOL = 2e-3
DH_TOL = 1e-2
LSE_ATOL = 1e-4
Q_RTOL = 1e-3


def compare(H_t, H_d, W, K, gpu: dict, rows=None, grad_loss=None, check_dH=True) -> dict:
    """H_t, H_d, W: bf16 CPU tensors. gpu: dict of CPU tensors/arrays with loss, topk_idx, topk_q,
    lse_t, lse_d and (if check_dH) dH_d, for ALL N rows. rows: subset the oracle evaluates."""
    Hb_t, Hb_d, Wb = hi.bf16_bits(H_t), hi.bf16_bits(H_d), hi.bf16_bits(W)
    N = Hb_t.shape[0]
    rows = np.arange(N, dtype=np.int64) if rows is None else np.asarray(rows, dtype=np.int64)
    gl = None if grad_loss is None else np.asarray(grad_loss, dtype=np.float64)
    ref = oracle.from_features(Hb_t, Hb_d, Wb, K, rows=rows, grad_loss=gl, want_dH=check_dH)

    g = {k: (v.float().numpy() if isinstance(v, torch.Tensor) and v.dtype == torch.bfloat16 else
             (v.numpy() if isinstance(v, torch.Tensor) else np.asarray(v))) for k, v in gpu.items()
         if k in ("loss", "topk_idx", "topk_q", "lse_t", "lse_d", "dH_d")}
    g_idx = g["topk_idx"][rows]
    assert g_idx.min() >= 0 and g_idx.max() < Wb.shape[0], "GPU returned token ids out of range"

    # ---- index sets ----
    tie_rows = []
    for r in range(rows.shape[0]):
        sg, so = set(g_idx[r].tolist()), set(ref["idx"][r].tolist())
        assert len(sg) == K, f"row {rows[r]}: GPU top-K has duplicates"
        if sg != so:
            diff = sorted(sg ^ so)
            z = oracle.logits_at(Hb_t, Wb, np.full(len(diff), rows[r]), np.array(diff, dtype=np.int32))
            z_kth = oracle.logits_at(Hb_t, Wb, rows[r:r + 1], ref["idx"][r, K - 1:K])[0]
            assert np.all(np.abs(z - z_kth) < TIE_TOL), (
                f"row {rows[r]}: top-K sets differ beyond a near-tie: tokens {diff}, logits {z}, K-th {z_kth}")
            tie_rows.append(r)
    if tie_rows:
        tr = np.array(tie_rows)
        alt = oracle.from_features(Hb_t, Hb_d, Wb, K, rows=rows[tr], grad_loss=gl,
                                   forced_idx=g_idx[tr].astype(np.int32), want_dH=check_dH)
        for key in ("loss", "q_k", "idx") + (("dH_d",) if check_dH else ()):
            ref[key][tr] = alt[key]

    # ---- order inside a row: descending q ----
    gq = g["topk_q"][rows]
    assert np.all(np.diff(gq, axis=1) <= 0), "GPU top-K not in descending q"
    # ---- values ----
    np.testing.assert_allclose(g["lse_t"][rows], ref["lse_t"], atol=LSE_ATOL, rtol=0)
    np.testing.assert_allclose(g["lse_d"][rows], ref["lse_d"], atol=LSE_ATOL, rtol=0)
    np.testing.assert_allclose(gq, ref["q_k"], rtol=Q_RTOL, atol=0)
    # same tokens at the same rank unless their q are equal to within the q tolerance
    mism = g_idx != ref["idx"]
    if mism.any():
        assert np.all(np.abs(gq[mism] - ref["q_k"][mism]) <= Q_RTOL * ref["q_k"][mism])
    loss_err = np.abs(g["loss"][rows] - ref["loss"]) / np.maximum(np.abs(ref["loss"]), 1e-6)
    assert loss_err.max() <= LOSS_RTOL, f"loss relative error {loss_err.max():.3e} at row {rows[loss_err.argmax()]}"
    stats = dict(rows=int(rows.shape[0]), tie_rows=len(tie_rows), loss_rel_err=float(loss_err.max()))
    if check_dH:
        scale = np.abs(ref["dH_d"]).max()
        err = np.abs(g["dH_d"][rows].astype(np.float64) - ref["dH_d"]).max()
        stats.update(dH_err=float(err), dH_scale=float(scale), dH_rel=float(err / max(scale, 1e-300)))
        assert err <= DH_TOL * scale, f"dH_d error {err:.3e} vs max|dH_d| {scale:.3e}"
    return stats


def _np(v):
    if isinstance(v, torch.Tensor):
        return v.float().numpy() if v.dtype == torch.bfloat16 else v.numpy()
    return np.asarray(v)


def compare_variant(H_t, H_d, W, K, variant, param, gpu: dict, rows=None, grad_loss=None) -> dict:
    """The loss variants of Section 4.3 (oracle.VARIANT_*) against the oracle, every compared row examined.

    A row whose token set differs from the oracle's is accepted only when every differing token is a
    near-tie with the selection boundary: its target logit within TIE_TOL of the oracle's last selected
    target logit (target list), for the bi-directional variant alternatively its draft logit within TIE_TOL
    of the oracle's K-th largest draft logit (draft list), for Top-P alternatively a cumulative probability
    within 1e-5 of P at the cut (fp32 against fp64 running sums). Such a row is then re-scored by the oracle
    on the GPU's own set, and loss, q and dH_d are compared on that; no row is left out of the comparison."""
    Hb_t, Hb_d, Wb = hi.bf16_bits(H_t), hi.bf16_bits(H_d), hi.bf16_bits(W)
    N, V = Hb_t.shape[0], Wb.shape[0]
    rows = np.arange(N, dtype=np.int64) if rows is None else np.asarray(rows, dtype=np.int64)
    gl = None if grad_loss is None else np.asarray(grad_loss, dtype=np.float64)
    bidir, top_p, normed = variant == oracle.VARIANT_BIDIR, variant == oracle.VARIANT_TOP_P, variant == oracle.VARIANT_NORMED
    ref = oracle.variant_from_features(Hb_t, Hb_d, Wb, K, variant, param, rows=rows, grad_loss=gl)
    g = {k: _np(v) for k, v in gpu.items() if v is not None and k != "workspace"}
    g_idx, g_n = g["topk_idx"][rows], g["topk_n"][rows]
    if top_p:
        # Top-P: a negative count marks a row whose prefix took all K tokens without exceeding P
        cut = g_n < 0
        g_n = np.abs(g_n)
        tot = ref["q_k"].sum(1)
        assert np.all(g_n[cut] == K) and np.all(tot[cut] <= param + 1e-5), "cap flag on a row that reached P"
        assert np.all(tot[(~cut) & (g_n == K)] > param - 1e-5), "a row cut by the cap is not flagged"
    kk = g_idx.shape[1]
    assert kk == ref["idx"].shape[1]
    assert g_idx.max() < V and np.all((g_idx >= 0) == (np.arange(kk)[None, :] < g_n[:, None])), "padding / count mismatch"
    tie_rows = []
    for r in range(rows.shape[0]):
        sel_g, sel_o = g_idx[r][g_idx[r] >= 0], ref["idx"][r][ref["idx"][r] >= 0]
        sg, so = set(sel_g.tolist()), set(sel_o.tolist())
        assert len(sg) == len(sel_g), f"row {rows[r]}: GPU set has duplicates"
        if sg == so:
            continue
        diff = np.array(sorted(sg ^ so), dtype=np.int32)
        rr = np.full(len(diff), rows[r])
        n_t = min(K, int(ref["n"][r]))                        # the target list ends at the oracle's n_t-th token
        zt = oracle.logits_at(Hb_t, Wb, rr, diff)
        zt_edge = oracle.logits_at(Hb_t, Wb, rows[r:r + 1], ref["idx"][r, n_t - 1:n_t])[0]
        ok = np.abs(zt - zt_edge) < TIE_TOL
        if bidir:
            zd_all = oracle.logits_at(Hb_d, Wb, np.full(V, rows[r]), np.arange(V, dtype=np.int32))
            zd_edge = np.sort(zd_all)[-K]
            ok |= np.abs(zd_all[diff] - zd_edge) < TIE_TOL
        if top_p:
            cum = np.cumsum(ref["q_k"][r])
            ok |= np.abs(cum - param).min() < 1e-5
        assert np.all(ok), f"row {rows[r]}: sets differ beyond a near-tie: tokens {diff.tolist()}"
        tie_rows.append(r)
    if tie_rows:
        tr = np.array(tie_rows)
        alt = oracle.variant_from_features(Hb_t, Hb_d, Wb, K, variant, param, rows=rows[tr], grad_loss=gl,
                                           forced_idx=g_idx[tr].astype(np.int32))
        for key in ("loss", "q_k", "idx", "n", "dH_d"):
            ref[key][tr] = alt[key]
    assert np.array_equal(g_n, ref["n"]), "set sizes differ"
    # q per token (orders may differ between equal probabilities: compare after sorting by token id)
    o_g, o_r = np.argsort(g_idx, 1, kind="stable"), np.argsort(ref["idx"], 1, kind="stable")
    assert np.array_equal(np.take_along_axis(g_idx, o_g, 1), np.take_along_axis(ref["idx"], o_r, 1))
    np.testing.assert_allclose(np.take_along_axis(g["topk_q"][rows], o_g, 1), np.take_along_axis(ref["q_k"], o_r, 1),
                               rtol=Q_RTOL, atol=1e-12)
    np.testing.assert_allclose(g["lse_t"][rows], ref["lse_t"], atol=LSE_ATOL, rtol=0)
    if not normed:
        np.testing.assert_allclose(g["lse_d"][rows], ref["lse_d"], atol=LSE_ATOL, rtol=0)
    loss_err = np.abs(g["loss"][rows] - ref["loss"]) / np.maximum(np.abs(ref["loss"]), 1e-6)
    assert loss_err.max() <= LOSS_RTOL, f"loss relative error {loss_err.max():.3e} at row {rows[loss_err.argmax()]}"
    scale = np.abs(ref["dH_d"]).max()
    err = np.abs(g["dH_d"][rows].astype(np.float64) - ref["dH_d"]).max()
    assert err <= DH_TOL * scale, f"dH_d error {err:.3e} vs max|dH_d| {scale:.3e}"
    return dict(rows=int(rows.shape[0]), tie_rows=len(tie_rows), mean_n=float(ref["n"].mean()),
                loss_rel_err=float(loss_err.max()), dH_rel=float(err / max(scale, 1e-300)))

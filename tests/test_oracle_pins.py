"""Pins for the fp64 CPU oracle: each test checks it against something other than itself —
a library routine on a special case, a closed form, an invariant, brute force on tiny
inputs, finite differences, or autograd. CPU only.

The paper prints no numeric value of Eq. 1, so there is no golden worked example.
"""
import itertools

import numpy as np
import pytest
import torch

import hass_inputs as hi
import oracle


def _rand_logits(V, seed, scale=1.5):
    rng = np.random.default_rng(seed)
    return rng.normal(0, scale, V), rng.normal(0, scale, V)


def _feat(N, d, V, seed, sigma_w=0.05):
    inp = hi.make_custom(N, d, V, K=1, seed=seed, sigma_w=sigma_w)
    return hi.bf16_bits(inp.H_t), hi.bf16_bits(inp.H_d[0]), hi.bf16_bits(inp.W), inp


# ---- P1: K = V is soft-target cross-entropy (library log_softmax / softmax) -------------------

@pytest.mark.parametrize("V", [7, 64, 1000])
def test_k_equals_v_is_soft_cross_entropy(V):
    z_t, z_d = _rand_logits(V, seed=V)
    r = oracle.from_logits(z_t, z_d, K=V)
    q = torch.softmax(torch.tensor(z_t), 0)
    logp = torch.log_softmax(torch.tensor(z_d), 0)
    ce = float(-(q * logp).sum())
    assert r["loss"] == pytest.approx(ce, rel=1e-12)
    # S_q = 1, so dL/dz_d = p - q
    np.testing.assert_allclose(r["dz_d"], (logp.exp() - q).numpy(), atol=1e-14)
    # CE = H(q) + KL(q || p)
    Hq = float(-(q * torch.log_softmax(torch.tensor(z_t), 0)).sum())
    kl = float(torch.nn.functional.kl_div(logp, q, reduction="sum"))
    assert r["loss"] == pytest.approx(Hq + kl, rel=1e-12)
    assert np.array_equal(np.sort(r["idx"]), np.arange(V))
    assert r["q_k"].sum() == pytest.approx(1.0, rel=1e-12)


def test_k_equals_v_same_features_gives_entropy_and_zero_gradient():
    Ht, _, W, _ = _feat(5, 32, 48, seed=3, sigma_w=0.3)
    r = oracle.from_features(Ht, Ht, W, K=48)
    for i in range(5):
        q = torch.softmax(torch.tensor(_z(Ht, W)[i]), 0)
        assert r["loss"][i] == pytest.approx(float(torch.distributions.Categorical(probs=q).entropy()), rel=1e-10)
    assert np.abs(r["dH_d"]).max() < 1e-13


def _z(H_bits, W_bits):
    H = torch.from_numpy(H_bits.view(np.int16).copy()).view(torch.bfloat16).double()
    W = torch.from_numpy(W_bits.view(np.int16).copy()).view(torch.bfloat16).double()
    return (H @ W.T).numpy()


# ---- P2: one-hot target gives plain NLL ------------------------------------------------------

@pytest.mark.parametrize("K", [1, 5])
def test_one_hot_target_is_nll(K):
    V = 50
    z_t, z_d = _rand_logits(V, seed=11)
    z_t = z_t.copy()
    z_t[17] += 800.0                     # q(17) = 1 to fp64 precision
    r = oracle.from_logits(z_t, z_d, K=K)
    nll = float(torch.nn.functional.cross_entropy(torch.tensor(z_d)[None], torch.tensor([17])))
    assert r["idx"][0] == 17
    assert r["loss"] == pytest.approx(nll, rel=1e-12)
    p = torch.softmax(torch.tensor(z_d), 0).numpy()
    onehot = np.zeros(V)
    onehot[17] = 1.0
    np.testing.assert_allclose(r["dz_d"], p - onehot, atol=1e-14)


# ---- P3: invariants ------------------------------------------------------------------------------

def test_shift_invariance_and_gradient_sums_to_zero():
    V, K = 300, 10
    z_t, z_d = _rand_logits(V, seed=5)
    a = oracle.from_logits(z_t, z_d, K)
    b = oracle.from_logits(z_t + 3.25, z_d, K)        # per-row constant on the target logits
    c = oracle.from_logits(z_t, z_d - 7.5, K)         # ... on the draft logits
    for o in (b, c):
        assert np.array_equal(a["idx"], o["idx"])
        np.testing.assert_allclose(a["q_k"], o["q_k"], rtol=1e-12)
        assert a["loss"] == pytest.approx(o["loss"], rel=1e-12)
        np.testing.assert_allclose(a["dz_d"], o["dz_d"], atol=1e-15)
    assert abs(a["dz_d"].sum()) < 1e-15
    assert a["loss"] >= 0
    assert b["lse_t"] == pytest.approx(a["lse_t"] + 3.25, rel=1e-13)
    assert c["lse_d"] == pytest.approx(a["lse_d"] - 7.5, rel=1e-13)


def test_loss_is_monotone_in_k_and_nonnegative():
    V = 200
    z_t, z_d = _rand_logits(V, seed=8)
    losses = [oracle.from_logits(z_t, z_d, K, want_dz=False)["loss"] for K in (1, 2, 5, 10, 50, 100, 200)]
    assert all(l >= 0 for l in losses)
    assert all(b >= a for a, b in zip(losses, losses[1:]))


def test_vocabulary_permutation_equivariance():
    N, d, V, K = 4, 24, 90, 6
    Ht, Hd, W, _ = _feat(N, d, V, seed=2, sigma_w=0.3)
    perm = np.random.default_rng(0).permutation(V)
    a = oracle.from_features(Ht, Hd, W, K)
    b = oracle.from_features(Ht, Hd, W[perm], K)      # token perm[j] now sits at position j
    np.testing.assert_allclose(a["loss"], b["loss"], rtol=1e-12)
    np.testing.assert_allclose(a["dH_d"], b["dH_d"], atol=1e-13)
    assert np.array_equal(a["idx"], perm[b["idx"]])


def test_rows_are_independent_and_subset_matches_full():
    N, d, V, K = 9, 16, 70, 4
    Ht, Hd, W, _ = _feat(N, d, V, seed=4, sigma_w=0.3)
    full = oracle.from_features(Ht, Hd, W, K)
    rows = np.array([7, 0, 3])
    sub = oracle.from_features(Ht, Hd, W, K, rows=rows)
    alone = oracle.from_features(Ht[3:4], Hd[3:4], W, K)
    for key in ("loss", "idx", "q_k", "lse_t", "lse_d", "dH_d"):
        np.testing.assert_array_equal(full[key][rows], sub[key])
        np.testing.assert_array_equal(full[key][3:4], alone[key])


def test_ties_go_to_lower_index_and_order_is_descending():
    z_t = np.array([0.5, 2.0, 2.0, -1.0, 2.0, 1.0])
    z_d = np.zeros(6)
    r = oracle.from_logits(z_t, z_d, K=2)
    assert list(r["idx"]) == [1, 2]
    r = oracle.from_logits(z_t, z_d, K=4)
    assert list(r["idx"]) == [1, 2, 4, 5]
    assert np.all(np.diff(r["q_k"]) <= 0)


def test_grad_loss_scales_gradient_only():
    N, d, V, K = 3, 16, 40, 5
    Ht, Hd, W, _ = _feat(N, d, V, seed=6, sigma_w=0.3)
    g = np.array([0.0, 2.0, -0.5])
    a = oracle.from_features(Ht, Hd, W, K)
    b = oracle.from_features(Ht, Hd, W, K, grad_loss=g)
    np.testing.assert_allclose(a["loss"], b["loss"], rtol=0)
    np.testing.assert_allclose(a["dH_d"] * g[:, None], b["dH_d"], atol=1e-15)


# ---- P4: brute force on tiny vocabularies ------------------------------------------------------

@pytest.mark.parametrize("V,K", [(6, 1), (8, 3), (12, 5), (16, 4), (20, 10)])
def test_brute_force_subset_and_literal_eq1(V, K):
    z_t, z_d = _rand_logits(V, seed=100 + V, scale=1.0)
    # literal, unshifted softmax: values are small enough not to overflow
    q = np.exp(z_t) / np.exp(z_t).sum()
    p = np.exp(z_d) / np.exp(z_d).sum()
    best = max(itertools.combinations(range(V), K), key=lambda s: sum(q[list(s)]))
    eq1 = -sum(q[x] * np.log(p[x]) for x in best)
    r = oracle.from_logits(z_t, z_d, K)
    assert set(r["idx"]) == set(best)
    assert r["loss"] == pytest.approx(eq1, rel=1e-12)
    np.testing.assert_allclose(r["q_k"], np.sort(q[list(best)])[::-1], rtol=1e-12)


@pytest.mark.parametrize("V,K", [(33, 7), (64, 10), (64, 64)])
def test_literal_eq1_with_sorted_topk(V, K):
    z_t, z_d = _rand_logits(V, seed=7 * V + K, scale=2.0)
    q = np.exp(z_t) / np.exp(z_t).sum()
    p = np.exp(z_d) / np.exp(z_d).sum()
    top = np.argsort(-q, kind="stable")[:K]
    eq1 = -(q[top] * np.log(p[top])).sum()
    r = oracle.from_logits(z_t, z_d, K)
    assert np.array_equal(r["idx"], top)
    assert r["loss"] == pytest.approx(eq1, rel=1e-12)
    assert r["lse_t"] == pytest.approx(np.log(np.exp(z_t).sum()), rel=1e-13)
    assert r["lse_d"] == pytest.approx(np.log(np.exp(z_d).sum()), rel=1e-13)


# ---- P5: finite differences -----------------------------------------------------------------------

def test_dz_matches_finite_differences_of_the_loss():
    V, K = 40, 6
    z_t, z_d = _rand_logits(V, seed=21)
    r = oracle.from_logits(z_t, z_d, K, g=1.0)
    h = 1e-6
    for v in list(r["idx"][:3]) + [0, 13, 39]:
        e = np.zeros(V)
        e[v] = h
        lp = oracle.from_logits(z_t, z_d + e, K, want_dz=False)["loss"]
        lm = oracle.from_logits(z_t, z_d - e, K, want_dz=False)["loss"]
        assert r["dz_d"][v] == pytest.approx((lp - lm) / (2 * h), rel=1e-6, abs=1e-10)


def test_dH_matches_finite_differences_in_draft_features():
    N, d, V, K = 3, 12, 30, 4
    rng = np.random.default_rng(9)
    Ht = rng.normal(size=(N, d))
    Hd = Ht + 0.5 * rng.normal(size=(N, d))
    W = rng.normal(scale=0.4, size=(V, d))
    g = np.array([1.0, 0.3, 2.0])
    base = oracle.from_features(Ht, Hd, W, K, grad_loss=g)
    h = 1e-6
    for (i, k) in [(0, 0), (1, 5), (2, 11), (1, 0)]:
        E = np.zeros_like(Hd)
        E[i, k] = h
        lp = oracle.from_features(Ht, Hd + E, W, K, want_dH=False)["loss"]
        lm = oracle.from_features(Ht, Hd - E, W, K, want_dH=False)["loss"]
        fd = g[i] * (lp[i] - lm[i]) / (2 * h)
        assert base["dH_d"][i, k] == pytest.approx(fd, rel=1e-6, abs=1e-10)
        # other rows' losses do not move
        others = [j for j in range(N) if j != i]
        np.testing.assert_array_equal(lp[others], lm[others])


# ---- P6: autograd restatement on the tiny configuration -------------------------------------

def test_autograd_restatement_on_tiny_config():
    wl = hi.WORKLOADS["tiny"]
    inp = hi.make_inputs(wl)
    r = oracle.from_features(hi.bf16_bits(inp.H_t), hi.bf16_bits(inp.H_d[0]), hi.bf16_bits(inp.W), wl.K)
    Ht, W = inp.H_t.double(), inp.W.double()
    Hd = inp.H_d[0].double().requires_grad_(True)
    q = torch.softmax(Ht @ W.T, -1)
    logp = torch.log_softmax(Hd @ W.T, -1)
    qk, idx = torch.topk(q, wl.K, dim=-1)
    loss = -(qk * logp.gather(-1, idx)).sum(-1)
    loss.sum().backward()
    np.testing.assert_allclose(r["loss"], loss.detach().numpy(), rtol=1e-11)
    np.testing.assert_allclose(r["q_k"], qk.numpy(), rtol=1e-11)
    assert np.array_equal(np.sort(r["idx"], 1), np.sort(idx.numpy(), 1))
    np.testing.assert_allclose(r["dH_d"], Hd.grad.numpy(), atol=1e-13 + 1e-10 * np.abs(r["dH_d"]).max())
    np.testing.assert_allclose(r["lse_t"], torch.logsumexp(Ht @ W.T, -1).numpy(), rtol=1e-13)


def test_bf16_entry_equals_f64_entry_on_widened_inputs():
    N, d, V, K = 6, 40, 77, 5
    Ht, Hd, W, inp = _feat(N, d, V, seed=12, sigma_w=0.2)
    a = oracle.from_features(Ht, Hd, W, K)
    b = oracle.from_features(inp.H_t.double().numpy(), inp.H_d[0].double().numpy(), inp.W.double().numpy(), K)
    for key in a:
        np.testing.assert_array_equal(a[key], b[key])


def test_forced_index_set_and_logits_at():
    N, d, V, K = 4, 16, 50, 3
    Ht, Hd, W, _ = _feat(N, d, V, seed=13, sigma_w=0.3)
    base = oracle.from_features(Ht, Hd, W, K)
    same = oracle.from_features(Ht, Hd, W, K, forced_idx=base["idx"][:, ::-1].copy())
    for key in base:
        np.testing.assert_allclose(base[key], same[key], rtol=1e-13, atol=1e-15)
    z = _z(Ht, W)
    rows = np.array([0, 3, 2])
    toks = np.array([5, 49, 0], dtype=np.int32)
    np.testing.assert_allclose(oracle.logits_at(Ht, W, rows, toks), z[rows, toks], rtol=1e-12, atol=1e-14)
    # a different forced set changes the loss to Eq. 1 on that set
    forced = np.tile(np.array([1, 2, 3], dtype=np.int32), (N, 1))
    r = oracle.from_features(Ht, Hd, W, K, forced_idx=forced)
    q = torch.softmax(torch.tensor(z), -1)
    logp = torch.log_softmax(torch.tensor(_z(Hd, W)), -1)
    np.testing.assert_allclose(r["loss"], -(q[:, 1:4] * logp[:, 1:4]).sum(-1).numpy(), rtol=1e-12)


def test_bad_arguments_are_rejected():
    z_t, z_d = _rand_logits(5, seed=1)
    with pytest.raises(ValueError):
        oracle.from_logits(z_t, z_d, K=6)
    with pytest.raises(ValueError):
        oracle.from_logits(z_t, z_d, K=0)


def test_expected_magnitudes_on_tiny_config():
    # sanity band, not a pin: sigma_z = sqrt(d) * sigma_w = 0.32, so lse ~ ln V + sigma_z^2 / 2
    wl = hi.WORKLOADS["tiny"]
    inp = hi.make_inputs(wl)
    r = oracle.from_features(hi.bf16_bits(inp.H_t), hi.bf16_bits(inp.H_d[0]), hi.bf16_bits(inp.W), wl.K,
                             want_dH=False)
    assert abs(r["lse_t"].mean() - (np.log(wl.V) + 0.32 ** 2 / 2)) < 0.05


# ---- combined objective: cross-entropy over the vocabulary + w * Top-K (Section 3.2) ---------------

def test_objective_ce_only_is_soft_target_cross_entropy_with_autograd_gradient():
    V, K = 90, 7
    z_t, z_d = _rand_logits(V, seed=31)
    r = oracle.objective_from_logits(z_t, z_d, K, w_ce=1.0, w_topk=0.0, g=1.7)
    zd = torch.tensor(z_d, requires_grad=True)
    q = torch.softmax(torch.tensor(z_t), 0)
    ce = torch.nn.functional.cross_entropy(zd[None], q[None])        # soft (probability) targets
    (1.7 * ce).backward()
    assert r["loss_ce"] == pytest.approx(float(ce), rel=1e-12)
    np.testing.assert_allclose(r["dz_d"], zd.grad.numpy(), atol=1e-14)
    # the Top-K loss and set are unaffected by the weights
    base = oracle.from_logits(z_t, z_d, K)
    assert r["loss"] == pytest.approx(base["loss"], rel=1e-13) and np.array_equal(r["idx"], base["idx"])


def test_objective_gradient_is_linear_in_the_two_weights_and_matches_finite_differences():
    V, K = 60, 6
    z_t, z_d = _rand_logits(V, seed=33)
    a = oracle.objective_from_logits(z_t, z_d, K, 1.0, 0.0)
    b = oracle.objective_from_logits(z_t, z_d, K, 0.0, 1.0)
    c = oracle.objective_from_logits(z_t, z_d, K, 0.6, 2.5, g=0.5)
    np.testing.assert_allclose(c["dz_d"], 0.5 * (0.6 * a["dz_d"] + 2.5 * b["dz_d"]), atol=1e-15)
    np.testing.assert_allclose(b["dz_d"], oracle.from_logits(z_t, z_d, K)["dz_d"], atol=0)
    h = 1e-6
    for v in (0, 17, int(c["idx"][0]), 59):
        e = np.zeros(V)
        e[v] = h
        up = oracle.objective_from_logits(z_t, z_d + e, K, 0.6, 2.5)
        dn = oracle.objective_from_logits(z_t, z_d - e, K, 0.6, 2.5)
        fd = 0.5 * ((0.6 * up["loss_ce"] + 2.5 * up["loss"]) - (0.6 * dn["loss_ce"] + 2.5 * dn["loss"])) / (2 * h)
        assert c["dz_d"][v] == pytest.approx(fd, rel=1e-6, abs=1e-10)


def test_objective_k_equals_v_makes_both_losses_equal():
    V = 40
    z_t, z_d = _rand_logits(V, seed=35)
    r = oracle.objective_from_logits(z_t, z_d, V, 1.0, 1.0)
    assert r["loss"] == pytest.approx(r["loss_ce"], rel=1e-12)
    np.testing.assert_allclose(r["dz_d"], 2 * oracle.objective_from_logits(z_t, z_d, V, 1.0, 0.0)["dz_d"], atol=1e-15)


def test_objective_features_level_autograd_restatement():
    N, d, V, K, w = 5, 24, 80, 6, 0.5
    Ht, Hd, W, inp = _feat(N, d, V, seed=37, sigma_w=0.3)
    g = np.array([1.0, 0.0, 2.0, -1.0, 0.5])
    r = oracle.objective_from_features(Ht, Hd, W, K, 1.0, w, grad_loss=g)
    Htt, Wt = inp.H_t.double(), inp.W.double()
    Hdt = inp.H_d[0].double().requires_grad_(True)
    q = torch.softmax(Htt @ Wt.T, -1)
    logp = torch.log_softmax(Hdt @ Wt.T, -1)
    ce = -(q * logp).sum(-1)
    qk, idx = torch.topk(q, K, dim=-1)
    tk = -(qk * logp.gather(-1, idx)).sum(-1)
    ((ce + w * tk) * torch.tensor(g)).sum().backward()
    np.testing.assert_allclose(r["loss_ce"], ce.detach().numpy(), rtol=1e-12)
    np.testing.assert_allclose(r["loss"], tk.detach().numpy(), rtol=1e-12)
    np.testing.assert_allclose(r["dH_d"], Hdt.grad.numpy(), atol=1e-13)
    plain = oracle.from_features(Ht, Hd, W, K, grad_loss=g)
    np.testing.assert_allclose(plain["dH_d"], oracle.objective_from_features(Ht, Hd, W, K, 0.0, 1.0, grad_loss=g)["dH_d"], atol=0)


# ---- loss variants of Section 4.3: Top-P and Normed Top-K ---------------------------------------------

def test_top_p_is_the_shortest_sorted_prefix_and_reduces_to_top_k():
    V, cap = 50, 12
    z_t, z_d = _rand_logits(V, seed=41, scale=2.0)
    q = np.exp(z_t) / np.exp(z_t).sum()
    p = np.exp(z_d) / np.exp(z_d).sum()
    order = np.argsort(-q, kind="stable")
    for P in (0.05, 0.3, 0.6, 0.9):
        n = int(np.searchsorted(np.cumsum(q[order]), P, side="right")) + 1      # literal: first prefix with cum > P
        n = min(n, cap)
        r = oracle.variant_from_logits(z_t, z_d, cap, oracle.VARIANT_TOP_P, P)
        assert r["n"] == n and np.array_equal(r["idx"][:n], order[:n]) and np.all(r["idx"][n:] == -1)
        assert r["loss"] == pytest.approx(-(q[order[:n]] * np.log(p[order[:n]])).sum(), rel=1e-12)
        same = oracle.from_logits(z_t, z_d, n)           # Eq. 1 with K = n is the same loss and gradient
        assert r["loss"] == pytest.approx(same["loss"], rel=1e-13)
        np.testing.assert_allclose(r["dz_d"], same["dz_d"], atol=1e-16)
    full = oracle.variant_from_logits(z_t, z_d, cap, oracle.VARIANT_TOP_P, 2.0)     # P never reached: all cap tokens
    assert full["n"] == cap and full["loss"] == pytest.approx(oracle.from_logits(z_t, z_d, cap)["loss"], rel=1e-13)
    one = oracle.variant_from_logits(z_t, z_d, cap, oracle.VARIANT_TOP_P, 0.0)
    assert one["n"] == 1 and one["loss"] == pytest.approx(oracle.from_logits(z_t, z_d, 1)["loss"], rel=1e-13)


def test_normed_top_k_closed_forms_and_autograd():
    V, K = 70, 8
    z_t, z_d = _rand_logits(V, seed=43, scale=1.5)
    r = oracle.variant_from_logits(z_t, z_d, K, oracle.VARIANT_NORMED, g=1.3)
    zd = torch.tensor(z_d, requires_grad=True)
    q = torch.softmax(torch.tensor(z_t), 0)
    qk, idx = torch.topk(q, K)
    logpn = torch.log_softmax(zd[idx], 0)                # softmax over the logits restricted to Omega_hat
    loss = -((qk / qk.sum()) * logpn).sum()
    (1.3 * loss).backward()
    assert np.array_equal(r["idx"], idx.numpy())
    assert r["loss"] == pytest.approx(float(loss), rel=1e-12)
    np.testing.assert_allclose(r["dz_d"], zd.grad.numpy(), atol=1e-15)
    # linear normalisation of the probabilities gives the same thing
    p = torch.softmax(torch.tensor(z_d), 0)
    lin = -((qk / qk.sum()) * torch.log(p[idx] / p[idx].sum())).sum()
    assert r["loss"] == pytest.approx(float(lin), rel=1e-12)
    # K = V: nothing to renormalise, plain cross-entropy; K = 1: the loss and its gradient vanish
    allv = oracle.variant_from_logits(z_t, z_d, V, oracle.VARIANT_NORMED)
    assert allv["loss"] == pytest.approx(float(-(q * torch.log_softmax(torch.tensor(z_d), 0)).sum()), rel=1e-12)
    k1 = oracle.variant_from_logits(z_t, z_d, 1, oracle.VARIANT_NORMED)
    assert abs(k1["loss"]) < 1e-15 and np.abs(k1["dz_d"]).max() < 1e-15
    # invariant to shifting the draft logits, gradient sums to zero, non-negative
    sh = oracle.variant_from_logits(z_t, z_d + 4.0, K, oracle.VARIANT_NORMED, g=1.3)
    assert sh["loss"] == pytest.approx(r["loss"], rel=1e-12) and abs(r["dz_d"].sum()) < 1e-15 and r["loss"] >= 0


def test_variants_at_features_level_match_the_row_entry():
    N, d, V, K = 4, 16, 60, 5
    Ht, Hd, W, _ = _feat(N, d, V, seed=45, sigma_w=0.3)
    zt, zd = _z(Ht, W), _z(Hd, W)
    Wd = torch.from_numpy(W.view(np.int16).copy()).view(torch.bfloat16).double().numpy()
    g = np.array([1.0, 0.5, 0.0, 2.0])
    for variant, param in ((oracle.VARIANT_TOPK, 0.0), (oracle.VARIANT_TOP_P, 0.2), (oracle.VARIANT_NORMED, 0.0)):
        f = oracle.variant_from_features(Ht, Hd, W, K, variant, param, grad_loss=g)
        for i in range(N):
            r = oracle.variant_from_logits(zt[i], zd[i], K, variant, param, g=g[i])
            assert f["loss"][i] == pytest.approx(r["loss"], rel=1e-12) and f["n"][i] == r["n"]
            np.testing.assert_allclose(f["dH_d"][i], r["dz_d"] @ Wd, atol=1e-13)
    plain = oracle.from_features(Ht, Hd, W, K, grad_loss=g)
    np.testing.assert_allclose(oracle.variant_from_features(Ht, Hd, W, K, 0, grad_loss=g)["dH_d"], plain["dH_d"], atol=1e-15)


def test_bidirectional_top_k_is_eq1_on_the_union_of_both_top_k_sets():
    V, K = 64, 5
    z_t, z_d = _rand_logits(V, seed=47, scale=1.5)
    r = oracle.variant_from_logits(z_t, z_d, K, oracle.VARIANT_BIDIR, g=0.7)
    zd = torch.tensor(z_d, requires_grad=True)
    q = torch.softmax(torch.tensor(z_t), 0)
    logp = torch.log_softmax(zd, 0)
    top_t = torch.topk(q, K).indices.tolist()
    top_d = torch.topk(logp.detach(), K).indices.tolist()
    union = top_t + [x for x in top_d if x not in top_t]
    loss = -(q[union] * logp[union]).sum()
    (0.7 * loss).backward()
    assert r["n"] == len(union) and list(r["idx"][:r["n"]]) == union and np.all(r["idx"][r["n"]:] == -1)
    assert K < r["n"] <= 2 * K                      # this seed has draft tokens outside the target's set
    assert r["loss"] == pytest.approx(float(loss), rel=1e-12)
    np.testing.assert_allclose(r["dz_d"], zd.grad.numpy(), atol=1e-15)
    # identical logits: the two sets coincide and the variant is Eq. 1
    same = oracle.variant_from_logits(z_t, z_t, K, oracle.VARIANT_BIDIR)
    base = oracle.from_logits(z_t, z_t, K)
    assert same["n"] == K and same["loss"] == pytest.approx(base["loss"], rel=1e-13)
    np.testing.assert_allclose(same["dz_d"], base["dz_d"], atol=1e-16)
    # K = V: every token, plain cross-entropy
    allv = oracle.variant_from_logits(z_t, z_d, V, oracle.VARIANT_BIDIR)
    assert allv["n"] == V and allv["loss"] == pytest.approx(float(-(q * torch.log_softmax(torch.tensor(z_d), 0)).sum()), rel=1e-12)
    # feature level agrees with the row entry
    Ht, Hd, W, _ = _feat(3, 16, 50, seed=49, sigma_w=0.3)
    f = oracle.variant_from_features(Ht, Hd, W, 4, oracle.VARIANT_BIDIR)
    zt, zdd = _z(Ht, W), _z(Hd, W)
    Wd = torch.from_numpy(W.view(np.int16).copy()).view(torch.bfloat16).double().numpy()
    for i in range(3):
        ri = oracle.variant_from_logits(zt[i], zdd[i], 4, oracle.VARIANT_BIDIR)
        assert f["n"][i] == ri["n"] and np.array_equal(f["idx"][i], ri["idx"]) and f["loss"][i] == pytest.approx(ri["loss"], rel=1e-12)
        np.testing.assert_allclose(f["dH_d"][i], ri["dz_d"] @ Wd, atol=1e-13)


# ---- scoring a row on a given token set (the comparator's route for near-ties at rank K) ----------------

def test_scoring_on_a_given_set_is_the_literal_restricted_sum_and_autograd():
    V = 40
    z_t, z_d = _rand_logits(V, seed=51, scale=1.5)
    tokens = [7, 31, 2, 19, 24]                       # any set, not the K most probable
    q = np.exp(z_t) / np.exp(z_t).sum()
    zd = torch.tensor(z_d, requires_grad=True)
    logp = torch.log_softmax(zd, 0)
    loss = -(torch.tensor(q[tokens]) * logp[tokens]).sum()         # Eq. 1 with the sum over the given set
    (0.6 * loss).backward()
    r = oracle.on_set_from_logits(z_t, z_d, tokens, g=0.6)
    assert r["loss"] == pytest.approx(float(loss), rel=1e-12)
    np.testing.assert_allclose(r["q_k"], q[tokens], rtol=1e-12)
    np.testing.assert_allclose(r["dz_d"], zd.grad.numpy(), atol=1e-15)
    # normed: both distributions restricted to the set (library log_softmax of the restricted logits)
    zd2 = torch.tensor(z_d, requires_grad=True)
    qn = torch.tensor(q[tokens] / q[tokens].sum())
    ln = -(qn * torch.log_softmax(zd2[tokens], 0)).sum()
    (0.6 * ln).backward()
    rn = oracle.on_set_from_logits(z_t, z_d, tokens, g=0.6, normed=True)
    assert rn["loss"] == pytest.approx(float(ln), rel=1e-12)
    np.testing.assert_allclose(rn["dz_d"], zd2.grad.numpy(), atol=1e-15)
    # bad sets are refused: repeated id, id out of range, empty
    for bad in ([3, 3], [V], []):
        with pytest.raises(ValueError):
            oracle.on_set_from_logits(z_t, z_d, bad)


def test_forcing_a_variants_own_selection_reproduces_the_unforced_result():
    N, d, V, K = 5, 16, 80, 6
    Ht, Hd, W, _ = _feat(N, d, V, seed=53, sigma_w=0.3)
    g = np.array([1.0, -0.5, 0.0, 2.0, 0.3])
    for variant, param in ((oracle.VARIANT_TOPK, 0.0), (oracle.VARIANT_TOP_P, 0.25), (oracle.VARIANT_NORMED, 0.0),
                           (oracle.VARIANT_BIDIR, 0.0)):
        free = oracle.variant_from_features(Ht, Hd, W, K, variant, param, grad_loss=g)
        forced = oracle.variant_from_features(Ht, Hd, W, K, variant, param, grad_loss=g, forced_idx=free["idx"])
        assert np.array_equal(forced["idx"], free["idx"]) and np.array_equal(forced["n"], free["n"])
        np.testing.assert_allclose(forced["loss"], free["loss"], rtol=1e-13)
        np.testing.assert_allclose(forced["q_k"], free["q_k"], rtol=1e-13)
        np.testing.assert_allclose(forced["dH_d"], free["dH_d"], atol=1e-15)
    # a different set gives a different loss (the forced set is really used): swap one token of row 0
    free = oracle.variant_from_features(Ht, Hd, W, K, oracle.VARIANT_NORMED)
    alt = free["idx"].copy()
    alt[0, -1] = next(v for v in range(V) if v not in set(free["idx"][0].tolist()))
    other = oracle.variant_from_features(Ht, Hd, W, K, oracle.VARIANT_NORMED, forced_idx=alt)
    assert abs(other["loss"][0] - free["loss"][0]) > 1e-6
    np.testing.assert_allclose(other["loss"][1:], free["loss"][1:], rtol=1e-13)

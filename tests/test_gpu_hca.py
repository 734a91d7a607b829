"""GPU parity of the HCA attention kernel (through the C ABI) against the fp64 oracle.

Tolerances (the kernel multiplies bf16 operands exactly, accumulates in fp32, rounds the softmax
weights to bf16 before the value product and the output to bf16):
  O    every row (one position of one head) within 1e-2 of that row's own largest entry, see
       tests/hca_parity.py (bf16 rounding of weights and output, 2^-9 relative each)
  lse  |error| <= 2e-3            (fp32 sums, approximate exp2)
"""
import numpy as np
import pytest
import torch

import hass_inputs as hi
from hca_parity import rowwise_error, tilewise_error
from oracle import hca_oracle as ho

pytestmark = pytest.mark.gpu

O_TOL = 1e-2
LSE_TOL = 2e-3


def _hass():
    import paper_2408_15766_b200 as hass
    return hass


def _f64(t):
    return t.to(torch.float64).numpy()


def _run(inp, scale=None, m=None):
    hass = _hass()
    dev = torch.device("cuda:0")
    m = inp.wl.m if m is None else m
    out = hass.hca_attention_fwd(inp.Q.to(dev), inp.K_t.to(dev), inp.V_t.to(dev), [x.to(dev) for x in inp.K_d[:m]],
                                 [x.to(dev) for x in inp.V_d[:m]], scale=scale)
    hass.check(out["workspace"])
    return out["O"].cpu(), out["lse"].cpu()


def _compare(inp, O, lse, scale=None, m=None, pairs=None):
    """pairs: list of (b, h) to check (all when None)."""
    wl = inp.wl
    m = wl.m if m is None else m
    rep = wl.H // wl.Hkv
    if pairs is None:
        pairs = [(b, h) for b in range(wl.B) for h in range(wl.H)]
    worst_o = worst_l = 0.0
    for b, h in pairs:
        g = h // rep
        sl = lambda x, hh: _f64(x[b:b + 1, :, hh:hh + 1, :])
        O_ref, lse_ref = ho.hca_attention(sl(inp.Q, h), sl(inp.K_t, g), sl(inp.V_t, g),
                                          [sl(x, g) for x in inp.K_d[:m]], [sl(x, g) for x in inp.V_d[:m]], scale=scale)
        err = rowwise_error(_f64(O[b:b + 1, :, h:h + 1, :]), O_ref).max()
        lerr = np.abs(lse[b, h].to(torch.float64).numpy() - lse_ref[0, 0]).max()
        worst_o, worst_l = max(worst_o, err), max(worst_l, lerr)
    assert worst_o <= O_TOL, f"O error {worst_o:.3e} of the row's own scale"
    assert worst_l <= LSE_TOL, f"lse error {worst_l:.3e}"
    return worst_o, worst_l


@pytest.mark.parametrize("name", ["hca-tiny", "hca-mid"])
def test_small_workloads_all_heads(name):
    inp = hi.make_hca_inputs(hi.HCA_WORKLOADS[name])
    O, lse = _run(inp)
    print(_compare(inp, O, lse))


@pytest.mark.parametrize("B,T,H,Hkv,m", [
    (1, 1, 1, 1, 1),          # a single position: the output is the draft value row itself
    (1, 128, 2, 2, 8),        # exactly one tile, the maximum number of draft passes
    (1, 129, 2, 1, 8),        # one row in the second tile: its sub-diagonals reach back into the first
    (2, 256, 3, 3, 0),        # first aligning step: plain causal attention
    (1, 515, 4, 2, 5),
    (2, 700, 16, 4, 2),       # more work items than SMs: every CTA takes a second item
    (1, 4096, 2, 1, 3),       # a long sequence: 64 key tiles in the last items
    (3, 64, 5, 5, 4),         # one key tile per item, five heads
    (1, 70, 1, 1, 8),         # the second key tile holds only hidden columns for most rows
    (2, 5, 2, 1, 8),          # more draft passes than positions
    (1, 300, 3, 1, 2),        # an odd group size: a CTA pairs two query tiles of one head; three tiles leave one alone
    (2, 640, 2, 2, 3),        # one query head per key/value head, five query tiles
    (1, 384, 6, 3, 1),        # an even group size: a CTA pairs two heads of one group
])
def test_awkward_shapes(B, T, H, Hkv, m):
    inp = hi.make_hca_inputs(hi.HcaWorkload("custom", B=B, T=T, H=H, Hkv=Hkv, m=m, seed=T + m))
    O, lse = _run(inp)
    pairs = None if B * H <= 8 else [(0, 0), (0, H - 1), (B - 1, H // 2), (B - 1, 1)]
    print(_compare(inp, O, lse, pairs=pairs))
    if T == 1:
        assert torch.equal(O, inp.V_d[0])


def test_steep_scores_rescale_the_accumulator():
    # scale 1 instead of 1/sqrt(D): scores spread over +-40, so later tiles push the running reference
    # up by far more than the lazy-rescale threshold
    inp = hi.make_hca_inputs(hi.HcaWorkload("steep", B=1, T=640, H=2, Hkv=1, m=2, seed=3))
    O, lse = _run(inp, scale=1.0)
    print(_compare(inp, O, lse, scale=1.0))


def test_fewer_passes_than_provided_and_determinism():
    inp = hi.make_hca_inputs(hi.HCA_WORKLOADS["hca-mid"])
    O1, l1 = _run(inp, m=1)
    _compare(inp, O1, l1, m=1)
    O2, l2 = _run(inp, m=1)
    assert torch.equal(O1, O2) and torch.equal(l1, l2)


def test_argument_errors():
    hass = _hass()
    inp = hi.make_hca_inputs(hi.HCA_WORKLOADS["hca-tiny"])
    dev = torch.device("cuda:0")
    Q, K, V = inp.Q.to(dev), inp.K_t.to(dev), inp.V_t.to(dev)
    with pytest.raises(hass.HassError):       # head dimension other than 128
        hass.hca_attention_fwd(Q[..., :64].contiguous(), K[..., :64].contiguous(), V[..., :64].contiguous())
    with pytest.raises(hass.HassError):       # too many draft passes
        hass.hca_attention_fwd(Q, K, V, [K] * 9, [V] * 9)
    with pytest.raises(hass.HassError):
        hass.hca_attention_fwd(Q, K, V, scale=0.0)


@pytest.mark.parametrize("name", ["hca-l3-8b", "hca-l2-7b"])
def test_full_size_sampled_heads(name):
    wl = hi.HCA_WORKLOADS[name]
    inp = hi.make_hca_inputs(wl)
    O, lse = _run(inp)
    pairs = [(0, 0), (wl.B - 1, wl.H - 1), (1, 5), (2, wl.H // 2 + 1)]
    print(_compare(inp, O, lse, pairs=pairs))


# ---- backward ---------------------------------------------------------------------------------------
# Tolerance: every tile of 64 positions of every gradient within G_TOL of that tile's own largest entry
# (tests/hca_parity.py explains why tiles and not single rows; the weights and dS pass through bf16 before their
# products, D = <dO, O> is formed from the bf16 output, outputs are bf16; observed <= 5.3e-3), with the
# comparator's floor for tiles that are zero by construction (a single position has softmax weight 1 and dS = 0).
# `whole_tensor`: compare against the tensor's largest entry instead; only for the steep-score case, where nearly
# every row attends to a single key, dS is a difference of two nearly equal numbers throughout, and the error of a
# tile is set by the rounding of D, not by the tile's own (vanishing) gradient.
G_TOL = 1.5e-2


def _run_bwd(inp, scale=None, pairs=None, whole_tensor=False):
    hass = _hass()
    dev = torch.device("cuda:0")
    wl = inp.wl
    g = torch.Generator().manual_seed(wl.seed + 77)
    dO = torch.randn(inp.Q.shape, generator=g).to(torch.bfloat16)
    d = lambda x: x.to(dev)
    Kd, Vd = [d(x) for x in inp.K_d], [d(x) for x in inp.V_d]
    fw = hass.hca_attention_fwd(d(inp.Q), d(inp.K_t), d(inp.V_t), Kd, Vd, scale=scale)
    bw = hass.hca_attention_bwd(d(inp.Q), d(inp.K_t), d(inp.V_t), Kd, Vd, fw["O"], fw["lse"], d(dO), scale=scale)
    hass.check(bw["workspace"])
    got = dict(dQ=bw["dQ"].cpu(), dK_t=bw["dK_t"].cpu(), dV_t=bw["dV_t"].cpu(),
               dK_d=[x.cpu() for x in bw["dK_d"]], dV_d=[x.cpu() for x in bw["dV_d"]])
    # oracle per sequence and key/value group (a group's heads share their keys' gradients)
    rep = wl.H // wl.Hkv
    if pairs is None:
        pairs = [(b, g_) for b in range(wl.B) for g_ in range(wl.Hkv)]
    worst = 0.0
    for b, gk in pairs:
        hs = slice(gk * rep, (gk + 1) * rep)
        sq = lambda x: _f64(x[b:b + 1, :, hs, :])
        sk = lambda x: _f64(x[b:b + 1, :, gk:gk + 1, :])
        ref = ho.hca_attention_grad(sq(inp.Q), sk(inp.K_t), sk(inp.V_t), [sk(x) for x in inp.K_d],
                                    [sk(x) for x in inp.V_d], sq(dO), scale=scale)
        cmp = [(sq(got["dQ"]), ref[0]), (sk(got["dK_t"]), ref[1]), (sk(got["dV_t"]), ref[2])]
        cmp += [(sk(got["dK_d"][i]), ref[3][i]) for i in range(wl.m)]
        cmp += [(sk(got["dV_d"][i]), ref[4][i]) for i in range(wl.m)]
        names = ["dQ", "dK_t", "dV_t"] + [f"dK_d[{i}]" for i in range(wl.m)] + [f"dV_d[{i}]" for i in range(wl.m)]
        for name, (mine, want) in zip(names, cmp):
            if np.abs(want).max() < 1e-2:                            # an all-zero gradient: absolute comparison
                err = np.abs(mine - want).max() / 1e-2
            elif whole_tensor:
                err = np.abs(mine - want).max() / np.abs(want).max()
            else:
                err = tilewise_error(mine, want).max()
            assert err <= G_TOL, f"{name} of (sequence {b}, group {gk}): error {err:.3e} of the tile's scale"
            worst = max(worst, err)
    return worst


@pytest.mark.parametrize("name", ["hca-tiny", "hca-mid"])
def test_backward_small_workloads(name):
    print(_run_bwd(hi.make_hca_inputs(hi.HCA_WORKLOADS[name])))


@pytest.mark.parametrize("B,T,H,Hkv,m", [
    (1, 1, 1, 1, 1), (1, 128, 2, 2, 8), (1, 129, 2, 1, 8), (2, 256, 3, 3, 0), (1, 515, 4, 2, 5),
    (2, 700, 16, 4, 2), (3, 64, 5, 5, 4), (1, 70, 1, 1, 8), (2, 5, 2, 1, 8), (1, 4096, 2, 1, 3),
    (2, 300, 6, 2, 3), (1, 200, 10, 2, 1),
])
def test_backward_awkward_shapes(B, T, H, Hkv, m):
    inp = hi.make_hca_inputs(hi.HcaWorkload("custom", B=B, T=T, H=H, Hkv=Hkv, m=m, seed=T + m))
    pairs = None if B * Hkv <= 6 else [(0, 0), (B - 1, Hkv - 1), (B - 1, 1)]
    print(_run_bwd(inp, pairs=pairs))


def test_backward_steep_scores():
    inp = hi.make_hca_inputs(hi.HcaWorkload("steep", B=1, T=640, H=2, Hkv=1, m=2, seed=3))
    print(_run_bwd(inp, scale=0.5, whole_tensor=True))


@pytest.mark.parametrize("name", ["hca-l3-8b", "hca-l2-7b"])
def test_backward_full_size_sampled_groups(name):
    wl = hi.HCA_WORKLOADS[name]
    print(_run_bwd(hi.make_hca_inputs(wl), pairs=[(0, 0), (wl.B - 1, wl.Hkv - 1), (1, wl.Hkv // 2)]))


def test_backward_twice_gives_the_same_gradients():
    # dK_t, dV_t and the draft passes' gradients have one writer per row and a fixed summation order: bit-identical
    # between two calls. dQ is summed over the key tiles in fp32 by reductions whose order is not fixed: two calls
    # may differ by the rounding of that sum, i.e. by one step of the bf16 result in rare entries and never more.
    hass = _hass()
    dev = torch.device("cuda:0")
    inp = hi.make_hca_inputs(hi.HcaWorkload("twice", B=2, T=1500, H=8, Hkv=2, m=3, seed=11))
    g = torch.Generator().manual_seed(5)
    dO = torch.randn(inp.Q.shape, generator=g).to(torch.bfloat16).to(dev)
    d = lambda x: x.to(dev)
    Q, K, V = d(inp.Q), d(inp.K_t), d(inp.V_t)
    Kd, Vd = [d(x) for x in inp.K_d], [d(x) for x in inp.V_d]
    fw = hass.hca_attention_fwd(Q, K, V, Kd, Vd)
    runs = []
    for _ in range(2):
        bw = hass.hca_attention_bwd(Q, K, V, Kd, Vd, fw["O"], fw["lse"], dO)
        hass.check(bw["workspace"])
        runs.append(bw)
    a, b = runs
    assert torch.equal(a["dK_t"], b["dK_t"]) and torch.equal(a["dV_t"], b["dV_t"])
    for i in range(3):
        assert torch.equal(a["dK_d"][i], b["dK_d"][i]) and torch.equal(a["dV_d"][i], b["dV_d"][i])
    qa, qb = a["dQ"].float(), b["dQ"].float()
    step = torch.maximum(qa.abs(), qb.abs()) * 2.0 ** -7        # one bf16 step is at most 2^-7 of the value
    assert bool(((qa - qb).abs() <= step).all())
    assert float((qa != qb).float().mean()) < 0.05


def test_draft_passes_equal_to_target_change_nothing_on_the_gpu():
    # property that holds at any size: with K_d = K_t and V_d = V_t the substituted entries carry the same keys and
    # values as the ones they replace, so the output must agree with plain causal attention (m = 0) up to the
    # rounding of the two routes (tensor-core tile vs. diagonal tile)
    hass = _hass()
    dev = torch.device("cuda:0")
    inp = hi.make_hca_inputs(hi.HcaWorkload("same", B=2, T=1000, H=8, Hkv=2, m=0, seed=5))
    Q, K, V = inp.Q.to(dev), inp.K_t.to(dev), inp.V_t.to(dev)
    base = hass.hca_attention_fwd(Q, K, V)
    sub = hass.hca_attention_fwd(Q, K, V, [K] * 3, [V] * 3)
    hass.check(sub["workspace"])
    scale = base["O"].float().abs().max().item()
    assert (base["O"].float() - sub["O"].float()).abs().max().item() <= 1e-2 * scale
    assert (base["lse"] - sub["lse"]).abs().max().item() <= 1e-4

"""GPU parity: the CUDA path (through the C ABI) against the fp64 oracle on the same seeded inputs."""
import os

import numpy as np
import pytest
import torch

import hass_inputs as hi
from parity import compare, compare_variant

pytestmark = pytest.mark.gpu

FULL_ROWS = int(os.environ.get("HASS_ORACLE_ROWS", "192"))


def _hass():
    import paper_2408_15766_b200 as hass
    return hass


def _to_cpu(out):
    return {k: v.cpu() for k, v in out.items() if k != "workspace"}


def _run_and_compare(inp, K, step=0, dH_dtype=None, grad_loss=None, rows=None):
    hass = _hass()
    dH_dtype = hass.HASS_BF16 if dH_dtype is None else dH_dtype
    dev = torch.device("cuda:0")
    H_t, H_d, W = inp.H_t.to(dev), inp.H_d[step].to(dev), inp.W.to(dev)
    gl = None if grad_loss is None else torch.tensor(grad_loss, dtype=torch.float32, device=dev)
    out = hass.topk_distill_fwd_bwd(H_t, H_d, W, K, grad_loss=gl, dH_dtype=dH_dtype)
    hass.check(out["workspace"])
    return compare(inp.H_t, inp.H_d[step], inp.W, K, _to_cpu(out), rows=rows, grad_loss=grad_loss), out


def test_tiny_config_all_rows():
    wl = hi.WORKLOADS["tiny"]
    stats, _ = _run_and_compare(hi.make_inputs(wl), wl.K, dH_dtype=_hass().HASS_FP32)
    print(stats)


GUARD = 1024          # bytes of pattern on both sides of every guarded buffer
PATTERN = 0xA5


class Guarded:
    """Outputs and workspace carved out of one device buffer, each between two pattern-filled margins.
    compute-sanitizer is not available on the test machines; an out-of-bounds write on a ragged tile shows up
    here as a damaged margin instead."""

    def __init__(self, dev):
        self.dev, self.specs, self.size = dev, [], 0

    def add(self, name, shape, dtype):
        nbytes = int(np.prod(shape)) * torch.empty(0, dtype=dtype).element_size()
        off = self.size + GUARD
        self.specs.append((name, off, nbytes, tuple(shape), dtype))
        self.size = off + (nbytes + 255) // 256 * 256 + GUARD      # payloads start 256-byte aligned
        return self

    def build(self):
        self.buf = torch.full((self.size,), PATTERN, dtype=torch.uint8, device=self.dev)
        assert self.buf.data_ptr() % 256 == 0
        return {name: self.buf[off:off + nbytes].view(dtype).view(shape) for name, off, nbytes, shape, dtype in self.specs}

    def check(self):
        keep = torch.ones(self.size, dtype=torch.bool, device=self.dev)
        for _, off, nbytes, _, _ in self.specs:
            keep[off:off + nbytes] = False
        bad = torch.nonzero((self.buf != PATTERN) & keep).flatten()
        assert bad.numel() == 0, f"{bad.numel()} guard bytes overwritten, first at offset {int(bad[0])} of {self.specs}"


def _guarded_fused(inp, K, grad, dH_fp32=True):
    """hass_topk_distill_fwd_bwd with every output and the workspace between guard bands."""
    hass = _hass()
    dev = torch.device("cuda:0")
    N, d, V = inp.H_t.shape[0], inp.H_t.shape[1], inp.W.shape[0]
    g = Guarded(dev)
    g.add("loss", (N,), torch.float32).add("topk_idx", (N, K), torch.int32).add("topk_q", (N, K), torch.float32)
    g.add("lse_t", (N,), torch.float32).add("lse_d", (N,), torch.float32)
    g.add("dH_d", (N, d), torch.float32 if dH_fp32 else torch.bfloat16)
    g.add("workspace", (hass.topk_distill_workspace_bytes(N, d, V, K),), torch.uint8)
    t = g.build()
    ws = t.pop("workspace")
    gl = None if grad is None else torch.tensor(grad, dtype=torch.float32, device=dev)
    out = hass.topk_distill_fwd_bwd(inp.H_t.to(dev), inp.H_d[0].to(dev), inp.W.to(dev), K, grad_loss=gl,
                                    dH_dtype=hass.HASS_FP32 if dH_fp32 else hass.HASS_BF16, workspace=ws, out=t)
    hass.check(ws)
    g.check()
    fused = _to_cpu(out)
    # the separate forward and the recomputing backward into the same guarded buffers
    f = hass.topk_distill_fwd(inp.H_t.to(dev), inp.H_d[0].to(dev), inp.W.to(dev), K, workspace=ws)
    hass.topk_distill_bwd(inp.H_d[0].to(dev), inp.W.to(dev), f["topk_idx"], f["topk_q"], f["lse_d"], grad_loss=gl,
                          dH_dtype=hass.HASS_FP32 if dH_fp32 else hass.HASS_BF16, workspace=ws, out=t["dH_d"])
    hass.check(ws)
    g.check()
    split = dict(_to_cpu(f), dH_d=t["dH_d"].cpu())
    return fused, split


@pytest.mark.parametrize("N,d,V,K", [
    (1, 64, 64, 1), (64, 256, 1000, 2), (127, 264, 1024, 10), (129, 64, 32003, 10),
    (300, 256, 5000, 64), (200, 128, 777, 100), (130, 512, 300, 128), (5, 8, 9, 9),
    (4800, 64, 700, 5),       # two row chunks, the second one ragged
    (260, 72, 20000, 17),     # smallest K on the buffered Top-K path, d not a multiple of 64
    (129, 4096, 128257, 10),  # a full-size hidden dimension, one row and one token past a tile boundary
    (64, 64, 40000, 100),     # one row tile split over 148 lanes: the selection cuts its candidate pool many times
    (100, 64, 33000, 256),    # the largest K, 129 lanes
    (150, 64, 3000, 200),     # K above 128 with two row tiles and few lanes
])
def test_awkward_shapes(N, d, V, K):
    inp = hi.make_custom(N, d, V, K, seed=N + V, sigma_w=0.5 / np.sqrt(d) * 4)
    rng = np.random.default_rng(0)
    grad = rng.normal(size=N)
    grad[0] = 0.0
    # fused call first, the split route second, both writing between guard bands
    fused, split = _guarded_fused(inp, K, grad)
    print("fused", compare(inp.H_t, inp.H_d[0], inp.W, K, fused, grad_loss=grad))
    print("split", compare(inp.H_t, inp.H_d[0], inp.W, K, split, grad_loss=grad))


def test_awkward_shape_bf16_output_between_guard_bands():
    inp = hi.make_custom(131, 72, 1500, 20, seed=77, sigma_w=0.3)
    fused, split = _guarded_fused(inp, 20, None, dH_fp32=False)
    print("fused", compare(inp.H_t, inp.H_d[0], inp.W, 20, fused))
    print("split", compare(inp.H_t, inp.H_d[0], inp.W, 20, split))


def test_split_calls_match_fused_call_and_draft_only_forward():
    hass = _hass()
    wl = hi.Workload("mid", N=384, d=512, V=4096, K=10, steps=2)
    inp = hi.make_inputs(wl)
    dev = torch.device("cuda:0")
    H_t, W = inp.H_t.to(dev), inp.W.to(dev)
    H_d0, H_d1 = inp.H_d[0].to(dev), inp.H_d[1].to(dev)
    fused = hass.topk_distill_fwd_bwd(H_t, H_d0, W, wl.K)
    hass.check(fused["workspace"])
    f = hass.topk_distill_fwd(H_t, H_d0, W, wl.K)
    dH = hass.topk_distill_bwd(H_d0, W, f["topk_idx"], f["topk_q"], f["lse_d"], workspace=f["workspace"])
    hass.check(f["workspace"])
    # the fused call (no recompute) and the split calls (recompute) are two routes to the same numbers
    for k in ("topk_idx", "topk_q", "lse_t"):
        assert torch.equal(fused[k], f[k])
    assert torch.allclose(fused["lse_d"], f["lse_d"], atol=1e-5, rtol=0)
    assert torch.allclose(fused["loss"], f["loss"], rtol=1e-4, atol=0)
    scale = dH.float().abs().max()
    assert (fused["dH_d"].float() - dH.float()).abs().max() <= 1e-2 * scale
    split = dict(_to_cpu(f), dH_d=dH.cpu())
    print("split", compare(inp.H_t, inp.H_d[0], inp.W, wl.K, split))
    print("fused", compare(inp.H_t, inp.H_d[0], inp.W, wl.K, _to_cpu(fused)))
    # aligning step 2: target statistics reused, only the draft side recomputed
    s2 = hass.topk_distill_fwd_draft(H_d1, W, f["topk_idx"], f["topk_q"], workspace=f["workspace"])
    dH2 = hass.topk_distill_bwd(H_d1, W, f["topk_idx"], f["topk_q"], s2["lse_d"], workspace=f["workspace"])
    hass.check(f["workspace"])
    gpu = dict(loss=s2["loss"].cpu(), lse_d=s2["lse_d"].cpu(), lse_t=f["lse_t"].cpu(), topk_idx=f["topk_idx"].cpu(),
               topk_q=f["topk_q"].cpu(), dH_d=dH2.cpu())
    print("step 2 split", compare(inp.H_t, inp.H_d[1], inp.W, wl.K, gpu))
    # the same step through the fused draft-only entry
    g = torch.linspace(-1.0, 2.0, wl.N, device=dev)
    fd = hass.topk_distill_fwd_bwd_draft(H_d1, W, f["topk_idx"], f["topk_q"], grad_loss=g, dH_dtype=hass.HASS_FP32,
                                         workspace=f["workspace"])
    hass.check(f["workspace"])
    gpu = dict(loss=fd["loss"].cpu(), lse_d=fd["lse_d"].cpu(), lse_t=f["lse_t"].cpu(), topk_idx=f["topk_idx"].cpu(),
               topk_q=f["topk_q"].cpu(), dH_d=fd["dH_d"].cpu())
    print("step 2 fused", compare(inp.H_t, inp.H_d[1], inp.W, wl.K, gpu, grad_loss=g.cpu().numpy()))


def test_rows_beyond_the_exponent_range_of_the_spill_are_redone_exactly():
    hass = _hass()
    N, d, V, K = 40, 64, 700, 3
    inp = hi.make_custom(N, d, V, K, seed=3, sigma_w=0.1)
    H_d = torch.ones(N, d, dtype=torch.bfloat16)
    W = inp.W.clone()
    W[:256] = -2.0                    # draft logits of the first 256 tokens: -128
    W[300] = 2.0                      # one later token at +128: 256 above the row reference
    dev = torch.device("cuda:0")
    # the plain fused call notices and falls back to its exact route on the device
    out = hass.topk_distill_fwd_bwd(inp.H_t.to(dev), H_d.to(dev), W.to(dev), K, dH_dtype=hass.HASS_FP32)
    hass.check(out["workspace"])
    print(compare(inp.H_t, H_d, W, K, _to_cpu(out)))
    d2 = hass.topk_distill_fwd_bwd_draft(H_d.to(dev), W.to(dev), out["topk_idx"], out["topk_q"],
                                         dH_dtype=hass.HASS_FP32, workspace=out["workspace"])
    hass.check(out["workspace"])
    assert torch.allclose(d2["loss"], out["loss"], rtol=1e-5) and torch.allclose(d2["dH_d"], out["dH_d"], atol=1e-6)
    # the Top-P variant has the same second route ...
    import oracle
    v = hass.variant_distill_fwd_bwd(inp.H_t.to(dev), H_d.to(dev), W.to(dev), K, hass.LOSS_TOP_P, 0.004,
                                     dH_dtype=hass.HASS_FP32)
    hass.check(v["workspace"])
    print("top-p, exact route", compare_variant(inp.H_t, H_d, W, K, oracle.VARIANT_TOP_P, 0.004, _to_cpu(v)))
    # ... and the Bi-directional variant and the combined objective sweep a second time with every row's reference
    # taken from the row's largest logit, which the first sweep recorded
    v = hass.variant_distill_fwd_bwd(inp.H_t.to(dev), H_d.to(dev), W.to(dev), K, hass.LOSS_BIDIR_TOPK, 0.0,
                                     dH_dtype=hass.HASS_FP32)
    hass.check(v["workspace"])
    print("bidir, second sweep", compare_variant(inp.H_t, H_d, W, K, oracle.VARIANT_BIDIR, 0.0, _to_cpu(v)))
    c = hass.combined_distill_fwd_bwd(inp.H_t.to(dev), H_d.to(dev), W.to(dev), K, w_topk=0.5, dH_dtype=hass.HASS_FP32)
    hass.check(c["workspace"])
    cpu = _to_cpu(c)
    print("combined, second sweep", compare(inp.H_t, H_d, W, K, cpu, check_dH=False))
    ref = oracle.objective_from_features(hi.bf16_bits(inp.H_t), hi.bf16_bits(H_d), hi.bf16_bits(W), K, 1.0, 0.5,
                                         forced_idx=cpu["topk_idx"].numpy().astype(np.int32))
    # logits of +-128 here: a row's cross-entropy is lse_d - <q, z_d> with both terms near 128 in fp32, so its
    # error is measured against the largest cross-entropy of the batch as well as against its own value
    ce = cpu["loss_ce"].numpy()
    assert np.all(np.abs(ce - ref["loss_ce"]) <= 2e-3 * np.abs(ref["loss_ce"]) + 1e-5 * np.abs(ref["loss_ce"]).max())
    assert np.abs(cpu["dH_d"].numpy().astype(np.float64) - ref["dH_d"]).max() <= 1e-2 * np.abs(ref["dH_d"]).max()
    assert hass.status_string(-7) == "HASS_ERR_RANGE"


def test_exact_route_with_two_row_chunks_when_only_some_rows_exceed_the_range():
    """N = 4800 is two row chunks (4736 + 64 rows), K = 17 runs the buffered Top-K sweep. A handful of rows in
    both chunks have one draft logit more than 200 above everything among the first 256 tokens; the fused call
    must notice and redo every row exactly."""
    hass = _hass()
    N, d, V, K = 4800, 64, 700, 17
    inp = hi.make_custom(N, d, V, K, seed=31, sigma_w=0.1)
    u = torch.where(torch.rand(d, generator=torch.Generator().manual_seed(1)) < 0.5, -1.0, 1.0)
    W = inp.W.clone()
    W[300] = (0.125 * u).to(torch.bfloat16)          # an ordinary row's logit of token 300 stays of order 1
    H_d = inp.H_d[0].clone()
    hot = [5, 130, 4735, 4736, 4790]
    H_d[hot] = (37.5 * u).to(torch.bfloat16)         # z_d[300] = 64 * 0.125 * 37.5 = 300 on these rows, |z_d| < 100 elsewhere
    dev = torch.device("cuda:0")
    grad = np.random.default_rng(4).uniform(0.5, 1.5, size=N)
    out = hass.topk_distill_fwd_bwd(inp.H_t.to(dev), H_d.to(dev), W.to(dev), K, dH_dtype=hass.HASS_FP32,
                                    grad_loss=torch.tensor(grad, dtype=torch.float32, device=dev))
    hass.check(out["workspace"])
    rows = np.unique(np.concatenate([np.array(hot), hi.sample_rows(N, 400, seed=2)]))
    print(compare(inp.H_t, H_d, W, K, _to_cpu(out), rows=rows, grad_loss=grad))
    # the same inputs with the hot rows removed stay on the fused route and agree on the other rows
    calm = inp.H_d[0].to(dev)
    ref = hass.topk_distill_fwd_bwd(inp.H_t.to(dev), calm, W.to(dev), K, dH_dtype=hass.HASS_FP32,
                                    grad_loss=torch.tensor(grad, dtype=torch.float32, device=dev))
    hass.check(ref["workspace"])
    keep = np.setdiff1d(np.arange(N), hot)
    assert torch.equal(out["topk_idx"].cpu()[keep], ref["topk_idx"].cpu()[keep])
    assert torch.allclose(out["loss"].cpu()[keep], ref["loss"].cpu()[keep], rtol=1e-3, atol=1e-7)
    # the Bi-directional variant on the same inputs: its second pass covers both chunks, every row keeps a valid result
    import oracle
    v = hass.variant_distill_fwd_bwd(inp.H_t.to(dev), H_d.to(dev), W.to(dev), K, hass.LOSS_BIDIR_TOPK, 0.0,
                                     dH_dtype=hass.HASS_FP32)
    hass.check(v["workspace"])
    print("bidir, two chunks, second pass",
          compare_variant(inp.H_t, H_d, W, K, oracle.VARIANT_BIDIR, 0.0, _to_cpu(v), rows=rows))


def test_l3_8b_split_forward_and_recomputing_backward_sampled_rows():
    """hass_topk_distill_fwd + hass_topk_distill_bwd (the route without a range condition) at full size."""
    hass = _hass()
    wl = hi.WORKLOADS["l3-8b"]
    inp = hi.make_inputs(wl)
    dev = torch.device("cuda:0")
    H_t, H_d, W = inp.H_t.to(dev), inp.H_d[0].to(dev), inp.W.to(dev)
    f = hass.topk_distill_fwd(H_t, H_d, W, wl.K)
    dH = hass.topk_distill_bwd(H_d, W, f["topk_idx"], f["topk_q"], f["lse_d"], workspace=f["workspace"])
    hass.check(f["workspace"])
    rows = hi.sample_rows(wl.N, max(FULL_ROWS // 2, 32), seed=wl.seed + 1)
    print("l3-8b split", compare(inp.H_t, inp.H_d[0], inp.W, wl.K, dict(_to_cpu(f), dH_d=dH.cpu()), rows=rows))


def test_smaller_workspace_means_smaller_row_chunks_same_results():
    hass = _hass()
    N, d, V, K = 1000, 128, 3000, 10
    inp = hi.make_custom(N, d, V, K, seed=21, sigma_w=0.2)
    dev = torch.device("cuda:0")
    H_t, H_d, W = inp.H_t.to(dev), inp.H_d[0].to(dev), inp.W.to(dev)
    full = hass.topk_distill_workspace_bytes(N, d, V, K)
    tile_bytes = 128 * (-(-V // 256) * 256) * 2          # dz_d / spill scratch of one 128-row tile
    row_tiles = -(-N // 128)
    small = torch.empty(full - (row_tiles - 2) * tile_bytes, dtype=torch.uint8, device=dev)   # room for 2 row tiles
    a = hass.topk_distill_fwd_bwd(H_t, H_d, W, K)
    b = hass.topk_distill_fwd_bwd(H_t, H_d, W, K, workspace=small)
    hass.check(a["workspace"])
    hass.check(small)
    # a different chunking splits the vocabulary sweep differently: same sets, sums in another order
    assert torch.equal(a["topk_idx"], b["topk_idx"])
    assert torch.allclose(a["lse_t"], b["lse_t"], atol=1e-5, rtol=0)
    assert torch.allclose(a["topk_q"], b["topk_q"], rtol=1e-5, atol=0)
    print(compare(inp.H_t, inp.H_d[0], inp.W, K, _to_cpu(b)))
    dH = hass.topk_distill_bwd(H_d, W, b["topk_idx"], b["topk_q"], b["lse_d"], workspace=small)
    hass.check(small)
    print(compare(inp.H_t, inp.H_d[0], inp.W, K, dict(_to_cpu(b), dH_d=dH.cpu())))
    # a workspace without room for even one row tile of scratch is refused
    tiny = torch.empty(full - row_tiles * tile_bytes, dtype=torch.uint8, device=dev)
    with pytest.raises(hass.HassError) as e:
        hass.topk_distill_fwd_bwd(H_t, H_d, W, K, workspace=tiny)
    assert e.value.status == -3


def test_host_buffer_entry_matches_device_entry():
    hass = _hass()
    wl = hi.Workload("mid", N=200, d=256, V=3000, K=10)
    inp = hi.make_inputs(wl)
    dev = torch.device("cuda:0")
    W = inp.W.to(dev)
    ref = hass.topk_distill_fwd_bwd(inp.H_t.to(dev), inp.H_d[0].to(dev), W, wl.K)
    loss_h = torch.empty(wl.N, dtype=torch.float32).pin_memory()
    dH_h = torch.empty(wl.N, wl.d, dtype=torch.bfloat16).pin_memory()
    idx_h = torch.empty(wl.N, wl.K, dtype=torch.int32).pin_memory()
    hass.topk_distill_fwd_bwd_host(inp.H_t.pin_memory(), inp.H_d[0].pin_memory(), W, wl.K, loss_h, dH_h,
                                   topk_idx_host=idx_h)
    assert torch.equal(loss_h, ref["loss"].cpu())
    assert torch.equal(dH_h, ref["dH_d"].cpu())
    assert torch.equal(idx_h, ref["topk_idx"].cpu())


def test_host_buffer_entry_with_several_row_chunks_and_the_exact_route():
    """N = 4800 is two row chunks: the second chunk's rows travel to the device while the first computes and
    the first chunk's dH_d rows travel back meanwhile; results equal the device entry's bit for bit. With a row
    beyond the spill's exponent range the exact route redoes the call after the chunks' dH_d rows have left,
    and the entry must fetch them again."""
    hass = _hass()
    N, d, V, K = 4800, 64, 700, 5
    inp = hi.make_custom(N, d, V, K, seed=17, sigma_w=0.1)
    dev = torch.device("cuda:0")
    for hot in (False, True):
        W, H_d = inp.W.clone(), inp.H_d[0].clone()
        if hot:
            u = torch.where(torch.rand(d, generator=torch.Generator().manual_seed(1)) < 0.5, -1.0, 1.0)
            W[300] = (0.125 * u).to(torch.bfloat16)
            H_d[[7, 4790]] = (37.5 * u).to(torch.bfloat16)        # z_d[300] = 300 on these rows
        Wd = W.to(dev)
        grad = torch.rand(N, generator=torch.Generator().manual_seed(2)) + 0.5
        ref = hass.topk_distill_fwd_bwd(inp.H_t.to(dev), H_d.to(dev), Wd, K, grad_loss=grad.to(dev))
        hass.check(ref["workspace"])
        loss_h = torch.empty(N, dtype=torch.float32).pin_memory()
        dH_h = torch.full((N, d), float("nan"), dtype=torch.bfloat16).pin_memory()
        q_h = torch.empty(N, K, dtype=torch.float32).pin_memory()
        hass.topk_distill_fwd_bwd_host(inp.H_t.pin_memory(), H_d.pin_memory(), Wd, K, loss_h, dH_h,
                                       grad_loss_host=grad.pin_memory(), topk_q_host=q_h)
        assert torch.equal(loss_h, ref["loss"].cpu())
        assert torch.equal(dH_h, ref["dH_d"].cpu())
        assert torch.equal(q_h, ref["topk_q"].cpu())
        if hot:
            print(compare(inp.H_t, H_d, W, K, dict(loss=loss_h, topk_idx=ref["topk_idx"].cpu(), topk_q=q_h,
                                                   lse_t=ref["lse_t"].cpu(), lse_d=ref["lse_d"].cpu(), dH_d=dH_h),
                          rows=np.array([0, 7, 100, 4735, 4736, 4790, 4799]), grad_loss=grad.numpy().astype(np.float64)))


def test_host_buffer_entry_with_more_row_chunks_than_it_has_events():
    """409600 rows are 87 row chunks on a 148-SM device, more than the entry's event pool covers: it falls back to
    one copy in, the call, one copy out, and the results still equal the device entry's."""
    hass = _hass()
    N, d, V, K = 3200 * 128, 8, 64, 2
    inp = hi.make_custom(N, d, V, K, seed=5, sigma_w=0.3)
    dev = torch.device("cuda:0")
    W = inp.W.to(dev)
    ref = hass.topk_distill_fwd_bwd(inp.H_t.to(dev), inp.H_d[0].to(dev), W, K)
    hass.check(ref["workspace"])
    loss_h = torch.empty(N, dtype=torch.float32).pin_memory()
    dH_h = torch.empty(N, d, dtype=torch.bfloat16).pin_memory()
    hass.topk_distill_fwd_bwd_host(inp.H_t.pin_memory(), inp.H_d[0].pin_memory(), W, K, loss_h, dH_h)
    assert torch.equal(loss_h, ref["loss"].cpu())
    assert torch.equal(dH_h, ref["dH_d"].cpu())
    rows = hi.sample_rows(N, 300, seed=1)
    print(compare(inp.H_t, inp.H_d[0], inp.W, K, _to_cpu(ref), rows=rows))


def test_results_are_deterministic_run_to_run():
    hass = _hass()
    inp = hi.make_custom(500, 256, 9000, 10, seed=5, sigma_w=0.1)
    dev = torch.device("cuda:0")
    a = hass.topk_distill_fwd_bwd(inp.H_t.to(dev), inp.H_d[0].to(dev), inp.W.to(dev), 10)
    b = hass.topk_distill_fwd_bwd(inp.H_t.to(dev), inp.H_d[0].to(dev), inp.W.to(dev), 10)
    for k in ("loss", "topk_idx", "topk_q", "lse_t", "lse_d", "dH_d"):
        assert torch.equal(a[k], b[k]), k


def test_exact_ties_resolve_to_lower_token_id():
    hass = _hass()
    inp = hi.make_custom(70, 64, 600, 4, seed=9, sigma_w=0.2)
    W = inp.W.clone()
    W[300:600] = W[0:300]            # every logit appears twice: tokens v and v + 300
    dev = torch.device("cuda:0")
    out = hass.topk_distill_fwd(inp.H_t.to(dev), inp.H_d[0].to(dev), W.to(dev), 4)
    hass.check(out["workspace"])
    idx = out["topk_idx"].cpu().numpy()
    assert np.all(idx[:, 1] == idx[:, 0] + 300) and np.all(idx[:, 3] == idx[:, 2] + 300)
    assert np.all(idx[:, 0] < 300) and np.all(idx[:, 2] < 300)
    print(compare(inp.H_t, inp.H_d[0], W, 4, _to_cpu(out) | {"dH_d": None}, check_dH=False))


@pytest.mark.parametrize("K", [20, 64])
def test_zero_rows_and_ties_with_buffered_candidates(K):
    # K > 16 takes the candidate-buffer path, whose first threshold of a sweep is found by a search over the
    # sweep's first tile. Rows of zeros make every logit +0 (the search ends at the prefix of zero, and the
    # threshold must still admit the zeros); duplicated rows of W put ties everywhere, also at the K-th place.
    hass = _hass()
    inp = hi.make_custom(130, 64, 1500, K, seed=21, sigma_w=0.2)
    W = inp.W.clone()
    W[750:1500] = W[0:750]           # every logit appears twice: tokens v and v + 750
    H_t, H_d = inp.H_t.clone(), inp.H_d[0].clone()
    for r in (5, 77, 129):
        H_t[r] = 0
    H_d[5] = 0
    dev = torch.device("cuda:0")
    out = hass.topk_distill_fwd_bwd(H_t.to(dev), H_d.to(dev), W.to(dev), K)
    hass.check(out["workspace"])
    idx = out["topk_idx"].cpu().numpy()
    for r in (5, 77, 129):
        assert np.array_equal(np.sort(idx[r]), np.arange(K)), "all logits equal: the K lowest token ids"
    print(compare(H_t, H_d, W, K, _to_cpu(out)))


@pytest.mark.parametrize("name", ["l2-7b", "l3-8b"])
def test_full_size_config_sampled_rows(name):
    wl = hi.WORKLOADS[name]
    inp = hi.make_inputs(wl)
    rows = hi.sample_rows(wl.N, FULL_ROWS, seed=wl.seed)
    stats, _ = _run_and_compare(inp, wl.K, rows=rows)
    print(name, stats)


def test_l2_13b_three_aligning_steps_sampled_rows():
    hass = _hass()
    wl = hi.WORKLOADS["l2-13b"]
    inp = hi.make_inputs(wl)
    rows = hi.sample_rows(wl.N, max(FULL_ROWS // 3, 32), seed=wl.seed)
    dev = torch.device("cuda:0")
    H_t, W = inp.H_t.to(dev), inp.W.to(dev)
    first = None
    for step in range(wl.steps):
        H_d = inp.H_d[step].to(dev)
        if step == 0:
            out = hass.topk_distill_fwd_bwd(H_t, H_d, W, wl.K)
            first = out
        else:
            s = hass.topk_distill_fwd_bwd_draft(H_d, W, first["topk_idx"], first["topk_q"],
                                                workspace=first["workspace"])
            out = dict(loss=s["loss"], lse_d=s["lse_d"], lse_t=first["lse_t"], topk_idx=first["topk_idx"],
                       topk_q=first["topk_q"], dH_d=s["dH_d"])
        hass.check(first["workspace"])
        print("step", step, compare(inp.H_t, inp.H_d[step], inp.W, wl.K, _to_cpu(out), rows=rows))


@pytest.mark.parametrize("K", [1, 10, 64])
def test_l3_70b_k_sweep_sampled_rows(K):
    wl = hi.WORKLOADS["l3-70b"]
    inp = hi.make_inputs(wl)
    rows = hi.sample_rows(wl.N, max(FULL_ROWS // 3, 32), seed=wl.seed)
    stats, _ = _run_and_compare(inp, K, rows=rows)
    print("l3-70b K", K, stats)


@pytest.mark.parametrize("N,d,V,K,w", [(64, 256, 1024, 10, 1.0), (300, 128, 5000, 5, 0.5), (4800, 64, 700, 20, 2.0)])
def test_combined_objective_matches_oracle(N, d, V, K, w):
    """Cross-entropy over the vocabulary + w * Top-K loss, forward and backward in one call."""
    import oracle
    hass = _hass()
    inp = hi.make_custom(N, d, V, K, seed=N + K, sigma_w=2.0 / np.sqrt(d))
    dev = torch.device("cuda:0")
    rng = np.random.default_rng(1)
    grad = rng.uniform(0.5, 1.5, size=N)
    grad[-1] = 0.0
    out = hass.combined_distill_fwd_bwd(inp.H_t.to(dev), inp.H_d[0].to(dev), inp.W.to(dev), K, w_topk=w,
                                        grad_loss=torch.tensor(grad, dtype=torch.float32, device=dev),
                                        dH_dtype=hass.HASS_FP32)
    hass.check(out["workspace"])
    # Top-K loss, Omega_hat, lse: the usual comparison (dH_d is that of the combined objective, checked below)
    cpu = _to_cpu(out)
    print(compare(inp.H_t, inp.H_d[0], inp.W, K, cpu, check_dH=False))
    rows = hi.sample_rows(N, 256, seed=3)
    ref = oracle.objective_from_features(hi.bf16_bits(inp.H_t), hi.bf16_bits(inp.H_d[0]), hi.bf16_bits(inp.W), K,
                                         1.0, w, rows=rows, grad_loss=grad,
                                         forced_idx=cpu["topk_idx"].numpy()[rows].astype(np.int32))
    ce = cpu["loss_ce"].numpy()[rows]
    assert np.all(np.abs(ce - ref["loss_ce"]) <= 2e-3 * np.maximum(np.abs(ref["loss_ce"]), 1e-6))
    scale = np.abs(ref["dH_d"]).max()
    err = np.abs(cpu["dH_d"].numpy()[rows].astype(np.float64) - ref["dH_d"]).max()
    print("combined: loss_ce rel", float((np.abs(ce - ref["loss_ce"]) / np.abs(ref["loss_ce"])).max()), "dH rel", err / scale)
    assert err <= 1e-2 * scale


def test_combined_objective_l2_7b_sampled_rows():
    import oracle
    hass = _hass()
    wl = hi.WORKLOADS["l2-7b"]
    inp = hi.make_inputs(wl)
    dev = torch.device("cuda:0")
    out = hass.combined_distill_fwd_bwd(inp.H_t.to(dev), inp.H_d[0].to(dev), inp.W.to(dev), wl.K, w_topk=1.0)
    hass.check(out["workspace"])
    cpu = _to_cpu(out)
    rows = hi.sample_rows(wl.N, max(FULL_ROWS // 2, 32), seed=1)
    print(compare(inp.H_t, inp.H_d[0], inp.W, wl.K, cpu, rows=rows, check_dH=False))
    ref = oracle.objective_from_features(hi.bf16_bits(inp.H_t), hi.bf16_bits(inp.H_d[0]), hi.bf16_bits(inp.W), wl.K,
                                         1.0, 1.0, rows=rows, forced_idx=cpu["topk_idx"].numpy()[rows].astype(np.int32))
    ce = cpu["loss_ce"].numpy()[rows]
    assert np.all(np.abs(ce - ref["loss_ce"]) <= 2e-3 * np.abs(ref["loss_ce"]))
    scale = np.abs(ref["dH_d"]).max()
    err = np.abs(cpu["dH_d"].float().numpy()[rows].astype(np.float64) - ref["dH_d"]).max()
    print("l2-7b combined: loss_ce rel", float((np.abs(ce - ref["loss_ce"]) / np.abs(ref["loss_ce"])).max()), "dH rel", err / scale)
    assert err <= 1e-2 * scale


def _run_variant(inp, K, variant, param=0.0, grad=None):
    hass = _hass()
    dev = torch.device("cuda:0")
    gl = None if grad is None else torch.tensor(grad, dtype=torch.float32, device=dev)
    out = hass.variant_distill_fwd_bwd(inp.H_t.to(dev), inp.H_d[0].to(dev), inp.W.to(dev), K, variant, param,
                                       grad_loss=gl, dH_dtype=hass.HASS_FP32)
    hass.check(out["workspace"])
    return _to_cpu(out)


@pytest.mark.parametrize("N,d,V,K", [(64, 256, 1024, 10), (300, 128, 5000, 24), (4800, 64, 700, 8)])
def test_normed_top_k_variant_matches_oracle(N, d, V, K):
    import oracle
    inp = hi.make_custom(N, d, V, K, seed=N + K + 1, sigma_w=2.0 / np.sqrt(d))
    grad = np.random.default_rng(2).uniform(-1.0, 2.0, size=N)
    cpu = _run_variant(inp, K, _hass().LOSS_NORMED_TOPK, grad=grad)
    assert np.all(cpu["topk_n"].numpy() == K)
    assert np.all(np.diff(cpu["topk_q"].numpy(), axis=1) <= 0)
    print("normed", compare_variant(inp.H_t, inp.H_d[0], inp.W, K, oracle.VARIANT_NORMED, 0.0, cpu, grad_loss=grad))


@pytest.mark.parametrize("N,d,V,K,P", [(64, 256, 1024, 10, 0.2), (300, 128, 5000, 24, 0.3), (4800, 64, 700, 16, 0.5),
                                       (200, 128, 6000, 256, 0.6)])
def test_top_p_variant_matches_oracle(N, d, V, K, P):
    import oracle
    inp = hi.make_custom(N, d, V, K, seed=N + K + 2, sigma_w=2.0 / np.sqrt(d))
    cpu = _run_variant(inp, K, _hass().LOSS_TOP_P, P)
    n_gpu = np.abs(cpu["topk_n"].numpy())
    assert n_gpu.min() >= 1 and n_gpu.max() <= K and len(np.unique(n_gpu)) > 1
    print("top-p", compare_variant(inp.H_t, inp.H_d[0], inp.W, K, oracle.VARIANT_TOP_P, P, cpu))


def test_top_p_reports_rows_whose_prefix_was_cut_by_the_cap():
    """With K = 4 and P = 0.9 on near-uniform rows no prefix of 4 tokens reaches P: topk_n = -4 on those rows;
    a peaked row (one dominant token) reaches P with its first token: topk_n = 1."""
    import oracle
    N, d, V, K, P = 96, 64, 900, 4, 0.9
    inp = hi.make_custom(N, d, V, K, seed=11, sigma_w=0.05)
    H_t = inp.H_t.clone()
    u = torch.where(torch.rand(d, generator=torch.Generator().manual_seed(5)) < 0.5, -1.0, 1.0)
    W = inp.W.clone()
    W[123] = (0.25 * u).to(torch.bfloat16)
    H_t[::3] = (2.0 * u).to(torch.bfloat16)            # z_t[123] = 64 * 0.25 * 2 = 32 on every third row: q(123) ~ 1
    cpu = _run_variant(hi.Inputs(inp.wl, H_t, inp.H_d, W), K, _hass().LOSS_TOP_P, P)
    n = cpu["topk_n"].numpy()
    assert np.all(n[::3] == 1) and np.all(np.delete(n, np.arange(0, N, 3)) == -K)
    print("top-p cap", compare_variant(H_t, inp.H_d[0], W, K, oracle.VARIANT_TOP_P, P, cpu))


@pytest.mark.parametrize("N,d,V,K", [(64, 256, 1024, 10), (300, 128, 5000, 24), (4800, 64, 700, 6)])
def test_bidirectional_top_k_variant_matches_oracle(N, d, V, K):
    import oracle
    inp = hi.make_custom(N, d, V, K, seed=N + K + 3, sigma_w=2.0 / np.sqrt(d))
    cpu = _run_variant(inp, K, _hass().LOSS_BIDIR_TOPK)
    assert cpu["topk_n"].numpy().max() > K                       # the draft really contributes tokens
    assert np.all(np.diff(cpu["topk_q"].numpy()[:, :K], axis=1) <= 0)
    print("bidir", compare_variant(inp.H_t, inp.H_d[0], inp.W, K, oracle.VARIANT_BIDIR, 0.0, cpu))

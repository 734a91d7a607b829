"""Row-wise comparison of HCA-attention tensors with the fp64 oracle.

Attention rows shrink like 1/sqrt(t) on random inputs, so an error bound relative to the largest entry of
the whole tensor is loose for late positions. Every row (one position of one head, D entries) is therefore
compared against its OWN largest reference entry:

    max_j |got[t, j] - ref[t, j]|  <=  tol * ( max_j |ref[t, j]| + FLOOR * max |ref| )

The floor covers rows whose reference is (nearly) zero by construction and the fp32 accumulation noise that
does not scale with the row.

Gradients are compared per tile of TILE consecutive positions of one head instead (tilewise_error): the backward
forms dS = P (dP - D) with D = <dO, O> taken from the bf16-rounded output, so a row whose two terms nearly
cancel (the first few positions of a sequence, where one or two keys carry all the weight) has an absolute
error set by its neighbours' scale, not by its own tiny gradient. A tile of 64 positions still localises a fault
to one key or query tile of the kernels.
"""
import numpy as np

FLOOR = 1e-3


def rowwise_error(got, ref) -> np.ndarray:
    """got, ref: arrays [..., D]. Returns the error of every row relative to that row's scale."""
    got, ref = np.asarray(got, dtype=np.float64), np.asarray(ref, dtype=np.float64)
    assert got.shape == ref.shape
    scale = np.abs(ref).max(axis=-1) + FLOOR * max(np.abs(ref).max(), 1e-30)
    return np.abs(got - ref).max(axis=-1) / scale


def assert_rows_close(got, ref, tol, what="tensor"):
    err = rowwise_error(got, ref)
    worst = np.unravel_index(int(err.argmax()), err.shape)
    assert err.max() <= tol, f"{what}: row {worst} off by {err.max():.3e} of its own scale (tolerance {tol:g})"
    return float(err.max())


TILE = 64


def tilewise_error(got, ref, tile=TILE) -> np.ndarray:
    """got, ref: arrays [B, T, heads, D]. Error of every (sequence, tile of `tile` positions, head) relative to
    the largest reference entry inside that tile (plus the floor)."""
    got, ref = np.asarray(got, dtype=np.float64), np.asarray(ref, dtype=np.float64)
    assert got.shape == ref.shape and got.ndim == 4
    B, T, H, D = ref.shape
    pad = (-T) % tile
    if pad:
        z = np.zeros((B, pad, H, D))
        got, ref = np.concatenate([got, z], 1), np.concatenate([ref, z], 1)
    g = got.reshape(B, -1, tile, H, D)
    r = ref.reshape(B, -1, tile, H, D)
    scale = np.abs(r).max(axis=(2, 4)) + FLOOR * max(np.abs(ref).max(), 1e-30)
    return np.abs(g - r).max(axis=(2, 4)) / scale

"""ctypes binding of libhass_b200.so. See include/hass.h for the contract of every call."""
from __future__ import annotations

import ctypes
import os
from typing import Optional

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
# HASS_LIBRARY_PATH selects another build of the same library (e.g. a tuning variant)
_LIB_PATH = os.environ.get("HASS_LIBRARY_PATH") or os.path.join(_HERE, "libhass_b200.so")

HASS_BF16, HASS_FP32 = 0, 1
K_MAX = 256


class HassError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {status_string(status)} ({status})")


def _load() -> ctypes.CDLL:
    if not os.path.exists(_LIB_PATH):
        raise ImportError(
            f"{_LIB_PATH} is missing: build it with `python paper_2408_15766_b200/build.py` "
            "(needs nvcc with sm_100a support). There is no fallback path.")
    L = ctypes.CDLL(_LIB_PATH)
    vp, i64, i32, sz = ctypes.c_void_p, ctypes.c_int64, ctypes.c_int32, ctypes.c_size_t
    L.hass_status_string.restype = ctypes.c_char_p
    L.hass_status_string.argtypes = [ctypes.c_int]
    L.hass_version.restype = ctypes.c_int
    L.hass_kernel_launch_count.restype = ctypes.c_int64
    L.hass_topk_distill_workspace_bytes.argtypes = [i64, i64, i64, i32, ctypes.POINTER(sz)]
    L.hass_topk_distill_host_workspace_bytes.argtypes = [i64, i64, i64, i32, ctypes.c_int, ctypes.POINTER(sz)]
    L.hass_topk_distill_fwd.argtypes = [vp, vp, vp, i64, i64, i64, i32, vp, vp, vp, vp, vp, vp, sz, vp]
    L.hass_topk_distill_fwd_draft.argtypes = [vp, vp, i64, i64, i64, i32, vp, vp, vp, vp, vp, sz, vp]
    L.hass_topk_distill_bwd.argtypes = [vp, vp, i64, i64, i64, i32, vp, vp, vp, vp, vp, ctypes.c_int, vp, sz, vp]
    L.hass_topk_distill_fwd_bwd.argtypes = [vp, vp, vp, i64, i64, i64, i32, vp, vp, vp, vp, vp, vp, vp,
                                            ctypes.c_int, vp, sz, vp]
    L.hass_topk_distill_fwd_bwd_draft.argtypes = [vp, vp, i64, i64, i64, i32, vp, vp, vp, vp, vp, vp, ctypes.c_int,
                                                  vp, sz, vp]
    L.hass_topk_distill_fwd_bwd_draft.restype = ctypes.c_int
    L.hass_combined_distill_workspace_bytes.argtypes = [i64, i64, i64, i32, ctypes.POINTER(sz)]
    L.hass_combined_distill_workspace_bytes.restype = ctypes.c_int
    L.hass_combined_distill_fwd_bwd.argtypes = [vp, vp, vp, i64, i64, i64, i32, ctypes.c_float, vp, vp, vp, vp, vp, vp,
                                                vp, vp, ctypes.c_int, vp, sz, vp]
    L.hass_combined_distill_fwd_bwd.restype = ctypes.c_int
    L.hass_variant_distill_fwd_bwd.argtypes = [vp, vp, vp, i64, i64, i64, i32, ctypes.c_int, ctypes.c_float, vp, vp, vp,
                                               vp, vp, vp, vp, vp, ctypes.c_int, vp, sz, vp]
    L.hass_variant_distill_fwd_bwd.restype = ctypes.c_int
    L.hass_topk_distill_fwd_bwd_host.argtypes = [vp, vp, vp, i64, i64, i64, i32, vp, vp, vp, vp, vp,
                                                 ctypes.c_int, vp, sz, vp]
    L.hass_hca_attention_workspace_bytes.argtypes = [ctypes.POINTER(sz)]
    L.hass_hca_attention_workspace_bytes.restype = ctypes.c_int
    L.hass_hca_attention_fwd.argtypes = [vp, vp, vp, ctypes.POINTER(vp), ctypes.POINTER(vp), i32, i64, i64, i64, i64,
                                         i64, ctypes.c_float, vp, vp, vp, sz, vp]
    L.hass_hca_attention_fwd.restype = ctypes.c_int
    L.hass_hca_attention_bwd_workspace_bytes.argtypes = [i64, i64, i64, i32, ctypes.POINTER(sz)]
    L.hass_hca_attention_bwd_workspace_bytes.restype = ctypes.c_int
    L.hass_hca_attention_bwd.argtypes = [vp, vp, vp, ctypes.POINTER(vp), ctypes.POINTER(vp), i32, i64, i64, i64, i64,
                                         i64, ctypes.c_float, vp, vp, vp, vp, vp, vp, ctypes.POINTER(vp),
                                         ctypes.POINTER(vp), vp, sz, vp]
    L.hass_hca_attention_bwd.restype = ctypes.c_int
    L.hass_check.argtypes = [vp, vp]
    L.hass_selftest_wait_expiry.argtypes = [vp, sz, ctypes.c_uint64, vp]
    L.hass_selftest_wait_expiry.restype = ctypes.c_int
    L.hass_topk_distill_fwd_static.argtypes = [vp, vp, vp, i64, i64, i64, i32, vp, vp, vp, vp, vp, vp, vp]
    L.hass_topk_distill_fwd_static.restype = ctypes.c_int
    L.hass_topk_distill_fwd_static_scratch_bytes.argtypes = [i64, i64, i64, i32, ctypes.POINTER(sz)]
    L.hass_topk_distill_fwd_static_scratch_bytes.restype = ctypes.c_int
    L.hass_profile_enable.argtypes = [ctypes.c_int]
    L.hass_profile_enable.restype = ctypes.c_int
    L.hass_profile_summary.argtypes = [ctypes.POINTER(ctypes.c_double), ctypes.POINTER(ctypes.c_int64), ctypes.c_int]
    L.hass_profile_summary.restype = ctypes.c_int
    for name in ("hass_topk_distill_workspace_bytes", "hass_topk_distill_host_workspace_bytes",
                 "hass_topk_distill_fwd", "hass_topk_distill_fwd_draft", "hass_topk_distill_bwd",
                 "hass_topk_distill_fwd_bwd", "hass_topk_distill_fwd_bwd_host", "hass_check"):
        getattr(L, name).restype = ctypes.c_int
    return L


lib = _load()


def status_string(status: int) -> str:
    return lib.hass_status_string(int(status)).decode()


def version() -> int:
    return int(lib.hass_version())


def kernel_launch_count() -> int:
    return int(lib.hass_kernel_launch_count())


def _ok(status: int, where: str) -> None:
    if status != 0:
        raise HassError(status, where)


def _p(t: Optional[torch.Tensor]):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


def _stream(stream) -> ctypes.c_void_p:
    s = torch.cuda.current_stream() if stream is None else stream
    return ctypes.c_void_p(s.cuda_stream)


def _dims(H: torch.Tensor, W: torch.Tensor):
    assert H.dtype == torch.bfloat16 and W.dtype == torch.bfloat16, "H and W must be bf16"
    assert H.is_contiguous() and W.is_contiguous() and H.dim() == 2 and W.dim() == 2
    assert H.shape[1] == W.shape[1], "H and W disagree on d"
    return H.shape[0], H.shape[1], W.shape[0]


def topk_distill_workspace_bytes(N: int, d: int, V: int, K: int) -> int:
    out = ctypes.c_size_t(0)
    _ok(lib.hass_topk_distill_workspace_bytes(N, d, V, K, ctypes.byref(out)), "hass_topk_distill_workspace_bytes")
    return int(out.value)


def topk_distill_host_workspace_bytes(N: int, d: int, V: int, K: int, dH_dtype: int = HASS_BF16) -> int:
    out = ctypes.c_size_t(0)
    _ok(lib.hass_topk_distill_host_workspace_bytes(N, d, V, K, dH_dtype, ctypes.byref(out)),
        "hass_topk_distill_host_workspace_bytes")
    return int(out.value)


def _workspace(ws: Optional[torch.Tensor], nbytes: int, device) -> torch.Tensor:
    if ws is None:
        ws = torch.empty(nbytes, dtype=torch.uint8, device=device)
    assert ws.dtype == torch.uint8 and ws.is_cuda and ws.is_contiguous()
    return ws


def _dh_dtype(code: int):
    return torch.float32 if code == HASS_FP32 else torch.bfloat16


def topk_distill_fwd(H_t, H_d, W, K: int, workspace=None, stream=None) -> dict:
    N, d, V = _dims(H_t, W)
    assert H_d.shape == H_t.shape and H_d.dtype == torch.bfloat16 and H_d.is_contiguous()
    dev = H_t.device
    ws = _workspace(workspace, topk_distill_workspace_bytes(N, d, V, K), dev)
    out = dict(loss=torch.empty(N, dtype=torch.float32, device=dev),
               topk_idx=torch.empty(N, K, dtype=torch.int32, device=dev),
               topk_q=torch.empty(N, K, dtype=torch.float32, device=dev),
               lse_t=torch.empty(N, dtype=torch.float32, device=dev),
               lse_d=torch.empty(N, dtype=torch.float32, device=dev), workspace=ws)
    _ok(lib.hass_topk_distill_fwd(_p(H_t), _p(H_d), _p(W), N, d, V, K, _p(out["loss"]), _p(out["topk_idx"]),
                                  _p(out["topk_q"]), _p(out["lse_t"]), _p(out["lse_d"]), _p(ws), ws.numel(),
                                  _stream(stream)), "hass_topk_distill_fwd")
    return out


STATIC_SCRATCH_MAX_BYTES = 32 << 20


def topk_distill_fwd_static_scratch_bytes(N: int, d: int, V: int, K: int) -> int:
    """Bytes of the built-in scratch array that hass_topk_distill_fwd_static needs for this size."""
    out = ctypes.c_size_t(0)
    _ok(lib.hass_topk_distill_fwd_static_scratch_bytes(N, d, V, K, ctypes.byref(out)),
        "hass_topk_distill_fwd_static_scratch_bytes")
    return int(out.value)


def topk_distill_fwd_static(H_t, H_d, W, K: int, stream=None, out: Optional[dict] = None) -> dict:
    """Forward for callers that cannot hand the library a workspace: the library's built-in 32 MiB
    scratch array is used instead. Here the outputs are still torch tensors, created by this wrapper
    when ``out`` is not given; pass preallocated ``out`` tensors to make the call allocation-free end
    to end. ``out['device_status']`` (uint32[1]) is 0 after a clean run."""
    N, d, V = _dims(H_t, W)
    assert H_d.shape == H_t.shape and H_d.dtype == torch.bfloat16 and H_d.is_contiguous()
    dev = H_t.device
    if out is None:
        out = dict(loss=torch.empty(N, dtype=torch.float32, device=dev),
                   topk_idx=torch.empty(N, K, dtype=torch.int32, device=dev),
                   topk_q=torch.empty(N, K, dtype=torch.float32, device=dev),
                   lse_t=torch.empty(N, dtype=torch.float32, device=dev),
                   lse_d=torch.empty(N, dtype=torch.float32, device=dev),
                   device_status=torch.empty(1, dtype=torch.int32, device=dev))
    _ok(lib.hass_topk_distill_fwd_static(_p(H_t), _p(H_d), _p(W), N, d, V, K, _p(out["loss"]), _p(out["topk_idx"]),
                                         _p(out["topk_q"]), _p(out["lse_t"]), _p(out["lse_d"]),
                                         _p(out.get("device_status")), _stream(stream)),
        "hass_topk_distill_fwd_static")
    return out


def topk_distill_fwd_draft(H_d, W, topk_idx, topk_q, workspace=None, stream=None) -> dict:
    N, d, V = _dims(H_d, W)
    K = topk_idx.shape[1]
    assert topk_idx.dtype == torch.int32 and topk_q.dtype == torch.float32
    assert topk_idx.is_contiguous() and topk_q.is_contiguous() and topk_idx.shape == topk_q.shape == (N, K)
    dev = H_d.device
    ws = _workspace(workspace, topk_distill_workspace_bytes(N, d, V, K), dev)
    out = dict(loss=torch.empty(N, dtype=torch.float32, device=dev),
               lse_d=torch.empty(N, dtype=torch.float32, device=dev), workspace=ws)
    _ok(lib.hass_topk_distill_fwd_draft(_p(H_d), _p(W), N, d, V, K, _p(topk_idx), _p(topk_q), _p(out["loss"]),
                                        _p(out["lse_d"]), _p(ws), ws.numel(), _stream(stream)),
        "hass_topk_distill_fwd_draft")
    return out


def topk_distill_bwd(H_d, W, topk_idx, topk_q, lse_d, grad_loss=None, dH_dtype: int = HASS_BF16, workspace=None,
                     stream=None, out=None) -> torch.Tensor:
    N, d, V = _dims(H_d, W)
    K = topk_idx.shape[1]
    assert topk_idx.dtype == torch.int32 and topk_q.dtype == torch.float32 and lse_d.dtype == torch.float32
    assert topk_idx.is_contiguous() and topk_q.is_contiguous() and lse_d.is_contiguous()
    assert grad_loss is None or (grad_loss.dtype == torch.float32 and grad_loss.shape == (N,))
    dev = H_d.device
    ws = _workspace(workspace, topk_distill_workspace_bytes(N, d, V, K), dev)
    dH = torch.empty(N, d, dtype=_dh_dtype(dH_dtype), device=dev) if out is None else out
    _ok(lib.hass_topk_distill_bwd(_p(H_d), _p(W), N, d, V, K, _p(topk_idx), _p(topk_q), _p(lse_d), _p(grad_loss),
                                  _p(dH), dH_dtype, _p(ws), ws.numel(), _stream(stream)), "hass_topk_distill_bwd")
    return dH


def topk_distill_fwd_bwd(H_t, H_d, W, K: int, grad_loss=None, dH_dtype: int = HASS_BF16, workspace=None,
                         stream=None, out: Optional[dict] = None) -> dict:
    N, d, V = _dims(H_t, W)
    assert H_d.shape == H_t.shape and H_d.dtype == torch.bfloat16 and H_d.is_contiguous()
    assert grad_loss is None or (grad_loss.dtype == torch.float32 and grad_loss.shape == (N,))
    dev = H_t.device
    ws = _workspace(workspace, topk_distill_workspace_bytes(N, d, V, K), dev)
    if out is None:
        out = dict(loss=torch.empty(N, dtype=torch.float32, device=dev),
                   topk_idx=torch.empty(N, K, dtype=torch.int32, device=dev),
                   topk_q=torch.empty(N, K, dtype=torch.float32, device=dev),
                   lse_t=torch.empty(N, dtype=torch.float32, device=dev),
                   lse_d=torch.empty(N, dtype=torch.float32, device=dev),
                   dH_d=torch.empty(N, d, dtype=_dh_dtype(dH_dtype), device=dev))
    out["workspace"] = ws
    _ok(lib.hass_topk_distill_fwd_bwd(_p(H_t), _p(H_d), _p(W), N, d, V, K, _p(grad_loss), _p(out["loss"]),
                                      _p(out["topk_idx"]), _p(out["topk_q"]), _p(out["lse_t"]), _p(out["lse_d"]),
                                      _p(out["dH_d"]), dH_dtype, _p(ws), ws.numel(), _stream(stream)),
        "hass_topk_distill_fwd_bwd")
    return out


def topk_distill_fwd_bwd_draft(H_d, W, topk_idx, topk_q, grad_loss=None, dH_dtype: int = HASS_BF16, workspace=None,
                               stream=None, out: Optional[dict] = None) -> dict:
    N, d, V = _dims(H_d, W)
    K = topk_idx.shape[1]
    assert topk_idx.dtype == torch.int32 and topk_q.dtype == torch.float32
    assert topk_idx.is_contiguous() and topk_q.is_contiguous() and topk_idx.shape == topk_q.shape == (N, K)
    assert grad_loss is None or (grad_loss.dtype == torch.float32 and grad_loss.shape == (N,))
    dev = H_d.device
    ws = _workspace(workspace, topk_distill_workspace_bytes(N, d, V, K), dev)
    if out is None:
        out = dict(loss=torch.empty(N, dtype=torch.float32, device=dev),
                   lse_d=torch.empty(N, dtype=torch.float32, device=dev),
                   dH_d=torch.empty(N, d, dtype=_dh_dtype(dH_dtype), device=dev))
    out["workspace"] = ws
    _ok(lib.hass_topk_distill_fwd_bwd_draft(_p(H_d), _p(W), N, d, V, K, _p(topk_idx), _p(topk_q), _p(grad_loss),
                                            _p(out["loss"]), _p(out["lse_d"]), _p(out["dH_d"]), dH_dtype, _p(ws),
                                            ws.numel(), _stream(stream)), "hass_topk_distill_fwd_bwd_draft")
    return out


def combined_distill_workspace_bytes(N: int, d: int, V: int, K: int) -> int:
    out = ctypes.c_size_t(0)
    _ok(lib.hass_combined_distill_workspace_bytes(N, d, V, K, ctypes.byref(out)), "hass_combined_distill_workspace_bytes")
    return int(out.value)


def combined_distill_fwd_bwd(H_t, H_d, W, K: int, w_topk: float = 1.0, grad_loss=None, dH_dtype: int = HASS_BF16,
                             workspace=None, stream=None, out: Optional[dict] = None) -> dict:
    """Cross-entropy over the full vocabulary plus w times the Top-K loss, forward and backward."""
    N, d, V = _dims(H_t, W)
    assert H_d.shape == H_t.shape and H_d.dtype == torch.bfloat16 and H_d.is_contiguous()
    assert grad_loss is None or (grad_loss.dtype == torch.float32 and grad_loss.shape == (N,))
    dev = H_t.device
    ws = _workspace(workspace, combined_distill_workspace_bytes(N, d, V, K), dev)
    if out is None:
        out = dict(loss_ce=torch.empty(N, dtype=torch.float32, device=dev),
                   loss=torch.empty(N, dtype=torch.float32, device=dev),
                   topk_idx=torch.empty(N, K, dtype=torch.int32, device=dev),
                   topk_q=torch.empty(N, K, dtype=torch.float32, device=dev),
                   lse_t=torch.empty(N, dtype=torch.float32, device=dev),
                   lse_d=torch.empty(N, dtype=torch.float32, device=dev),
                   dH_d=torch.empty(N, d, dtype=_dh_dtype(dH_dtype), device=dev))
    out["workspace"] = ws
    _ok(lib.hass_combined_distill_fwd_bwd(_p(H_t), _p(H_d), _p(W), N, d, V, K, ctypes.c_float(w_topk), _p(grad_loss),
                                          _p(out["loss_ce"]), _p(out["loss"]), _p(out["topk_idx"]), _p(out["topk_q"]),
                                          _p(out["lse_t"]), _p(out["lse_d"]), _p(out["dH_d"]), dH_dtype, _p(ws),
                                          ws.numel(), _stream(stream)), "hass_combined_distill_fwd_bwd")
    return out


LOSS_TOPK, LOSS_TOP_P, LOSS_NORMED_TOPK, LOSS_BIDIR_TOPK = 0, 1, 2, 3


def variant_distill_fwd_bwd(H_t, H_d, W, K: int, variant: int, param: float = 0.0, grad_loss=None,
                            dH_dtype: int = HASS_BF16, workspace=None, stream=None) -> dict:
    """Top-P / Normed Top-K / Top-K loss, forward and backward. See hass_variant_distill_fwd_bwd."""
    N, d, V = _dims(H_t, W)
    assert H_d.shape == H_t.shape and H_d.dtype == torch.bfloat16 and H_d.is_contiguous()
    assert grad_loss is None or (grad_loss.dtype == torch.float32 and grad_loss.shape == (N,))
    dev = H_t.device
    ws = _workspace(workspace, topk_distill_workspace_bytes(N, d, V, K), dev)
    kk = 2 * K if variant == LOSS_BIDIR_TOPK else K      # the bi-directional set holds up to 2K tokens
    out = dict(loss=torch.empty(N, dtype=torch.float32, device=dev),
               topk_idx=torch.empty(N, kk, dtype=torch.int32, device=dev),
               topk_q=torch.empty(N, kk, dtype=torch.float32, device=dev),
               topk_n=torch.empty(N, dtype=torch.int32, device=dev),
               lse_t=torch.empty(N, dtype=torch.float32, device=dev),
               lse_d=torch.zeros(N, dtype=torch.float32, device=dev),
               dH_d=torch.empty(N, d, dtype=_dh_dtype(dH_dtype), device=dev), workspace=ws)
    _ok(lib.hass_variant_distill_fwd_bwd(_p(H_t), _p(H_d), _p(W), N, d, V, K, int(variant), ctypes.c_float(param),
                                         _p(grad_loss), _p(out["loss"]), _p(out["topk_idx"]), _p(out["topk_q"]),
                                         _p(out["topk_n"]), _p(out["lse_t"]), _p(out["lse_d"]), _p(out["dH_d"]),
                                         dH_dtype, _p(ws), ws.numel(), _stream(stream)), "hass_variant_distill_fwd_bwd")
    return out


def topk_distill_fwd_bwd_host(H_t_host, H_d_host, W, K: int, loss_host, dH_d_host, grad_loss_host=None,
                              topk_idx_host=None, topk_q_host=None, dH_dtype: int = HASS_BF16, workspace=None,
                              stream=None) -> None:
    """H_t_host, H_d_host and the *_host outputs are CPU tensors (pinned for asynchronous copies);
    W and the workspace are CUDA tensors. Returns once the host outputs are valid."""
    assert not H_t_host.is_cuda and not H_d_host.is_cuda and W.is_cuda
    N, d, V = _dims(H_t_host, W)
    assert H_d_host.shape == H_t_host.shape and H_d_host.dtype == torch.bfloat16 and H_d_host.is_contiguous()
    assert loss_host.dtype == torch.float32 and loss_host.shape == (N,) and not loss_host.is_cuda
    assert dH_d_host.dtype == _dh_dtype(dH_dtype) and dH_d_host.shape == (N, d) and dH_d_host.is_contiguous()
    ws = _workspace(workspace, topk_distill_host_workspace_bytes(N, d, V, K, dH_dtype), W.device)
    _ok(lib.hass_topk_distill_fwd_bwd_host(_p(H_t_host), _p(H_d_host), _p(W), N, d, V, K, _p(grad_loss_host),
                                           _p(loss_host), _p(topk_idx_host), _p(topk_q_host), _p(dH_d_host),
                                           dH_dtype, _p(ws), ws.numel(), _stream(stream)),
        "hass_topk_distill_fwd_bwd_host")


HCA_MAX_DRAFTS = 8


def hca_attention_workspace_bytes() -> int:
    n = ctypes.c_size_t(0)
    _ok(lib.hass_hca_attention_workspace_bytes(ctypes.byref(n)), "hass_hca_attention_workspace_bytes")
    return int(n.value)


def hca_attention_fwd(Q, K_t, V_t, K_d=(), V_d=(), scale: Optional[float] = None, want_lse: bool = True,
                      workspace=None, stream=None) -> dict:
    """HCA attention forward. Q [B, T, H, D]; K_t, V_t and every K_d[i], V_d[i] [B, T, Hkv, D], bf16 CUDA
    tensors; entry i of K_d / V_d replaces the i-th sub-diagonal. See hass_hca_attention_fwd."""
    B, T, H, D = Q.shape
    Hkv = K_t.shape[2]
    m = len(K_d)
    assert len(V_d) == m
    for x in (Q, K_t, V_t, *K_d, *V_d):
        assert x.is_cuda and x.dtype == torch.bfloat16 and x.is_contiguous()
    for x in (V_t, *K_d, *V_d):
        assert x.shape == K_t.shape
    assert K_t.shape == (B, T, Hkv, D)
    dev = Q.device
    ws = _workspace(workspace, hca_attention_workspace_bytes(), dev)
    out = dict(O=torch.empty_like(Q), lse=torch.empty(B, H, T, dtype=torch.float32, device=dev) if want_lse else None,
               workspace=ws)
    kd = (ctypes.c_void_p * max(m, 1))(*[x.data_ptr() for x in K_d])
    vd = (ctypes.c_void_p * max(m, 1))(*[x.data_ptr() for x in V_d])
    sc = float(scale) if scale is not None else 1.0 / (D ** 0.5)
    _ok(lib.hass_hca_attention_fwd(_p(Q), _p(K_t), _p(V_t), kd, vd, m, B, T, H, Hkv, D, ctypes.c_float(sc),
                                   _p(out["O"]), _p(out["lse"]), _p(ws), ws.numel(), _stream(stream)),
        "hass_hca_attention_fwd")
    return out


def hca_attention_bwd_workspace_bytes(B: int, T: int, H: int, m: int) -> int:
    n = ctypes.c_size_t(0)
    _ok(lib.hass_hca_attention_bwd_workspace_bytes(B, T, H, m, ctypes.byref(n)), "hass_hca_attention_bwd_workspace_bytes")
    return int(n.value)


def hca_attention_bwd(Q, K_t, V_t, K_d, V_d, O, lse, dO, scale: Optional[float] = None, workspace=None,
                      stream=None) -> dict:
    """HCA attention backward: gradients of every projected input. See hass_hca_attention_bwd."""
    B, T, H, D = Q.shape
    Hkv = K_t.shape[2]
    m = len(K_d)
    assert len(V_d) == m
    for x in (Q, K_t, V_t, O, dO, *K_d, *V_d):
        assert x.is_cuda and x.dtype == torch.bfloat16 and x.is_contiguous()
    assert O.shape == Q.shape and dO.shape == Q.shape and V_t.shape == K_t.shape == (B, T, Hkv, D)
    assert lse.dtype == torch.float32 and lse.shape == (B, H, T) and lse.is_contiguous()
    dev = Q.device
    ws = _workspace(workspace, hca_attention_bwd_workspace_bytes(B, T, H, m), dev)
    out = dict(dQ=torch.empty_like(Q), dK_t=torch.empty_like(K_t), dV_t=torch.empty_like(V_t),
               dK_d=[torch.empty_like(K_t) for _ in range(m)], dV_d=[torch.empty_like(K_t) for _ in range(m)],
               workspace=ws)
    arr = lambda ts: (ctypes.c_void_p * max(m, 1))(*[x.data_ptr() for x in ts])
    sc = float(scale) if scale is not None else 1.0 / (D ** 0.5)
    _ok(lib.hass_hca_attention_bwd(_p(Q), _p(K_t), _p(V_t), arr(K_d), arr(V_d), m, B, T, H, Hkv, D, ctypes.c_float(sc),
                                   _p(O), _p(lse), _p(dO), _p(out["dQ"]), _p(out["dK_t"]), _p(out["dV_t"]),
                                   arr(out["dK_d"]), arr(out["dV_d"]), _p(ws), ws.numel(), _stream(stream)),
        "hass_hca_attention_bwd")
    return out


def check(workspace: torch.Tensor, stream=None) -> None:
    """Synchronises the stream and raises HassError if a kernel recorded a device-side problem."""
    _ok(lib.hass_check(_p(workspace), _stream(stream)), "hass_check")


def selftest_wait_expiry(workspace: torch.Tensor, limit_ns: int = 2_000_000, stream=None) -> None:
    """Enqueues the small kernel whose bounded wait is made to run out; check(workspace) raises
    HASS_ERR_TIMEOUT afterwards. See hass_selftest_wait_expiry."""
    assert workspace.dtype == torch.uint8 and workspace.is_cuda and workspace.is_contiguous()
    _ok(lib.hass_selftest_wait_expiry(_p(workspace), workspace.numel(), int(limit_ns), _stream(stream)),
        "hass_selftest_wait_expiry")


PROFILE_KINDS = ("stats_gemm", "dz_gemm", "dH_gemm", "finalize", "bwd_prep", "exact_route_conditional",
                 "hca_attention", "hca_bwd_dq_convert", "hca_bwd_fused", "hca_bwd_rows", "stats_gemm_draft")


def profile_enable(on: bool) -> None:
    _ok(lib.hass_profile_enable(1 if on else 0), "hass_profile_enable")


def profile_summary() -> dict:
    """{kind: (milliseconds, launches)} since the last summary / enable."""
    n = len(PROFILE_KINDS)
    ms = (ctypes.c_double * n)()
    cnt = (ctypes.c_int64 * n)()
    _ok(lib.hass_profile_summary(ms, cnt, n), "hass_profile_summary")
    return {k: (float(ms[i]), int(cnt[i])) for i, k in enumerate(PROFILE_KINDS)}

"""Host-side checks that need no GPU: the library loads, exports what include/hass.h declares,
rejects bad arguments before touching the device, and sizes its workspace sensibly."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def hass():
    import sys
    sys.path.insert(0, ROOT)
    import __graft_entry__ as entry
    entry.build()
    import paper_2408_15766_b200 as h
    return h


def test_every_declared_symbol_is_exported(hass):
    header = open(os.path.join(ROOT, "include", "hass.h")).read()
    names = set(re.findall(r"\b(hass_[a-z_0-9]+)\s*\(", header))
    assert {"hass_topk_distill_fwd", "hass_topk_distill_bwd", "hass_topk_distill_fwd_bwd"} <= names
    for n in names:
        assert hasattr(hass.lib, n), n


def test_status_strings_and_version(hass):
    assert hass.status_string(0) == "HASS_OK"
    assert hass.status_string(-5) == "HASS_ERR_TIMEOUT"
    assert hass.version() >= 100


def test_workspace_bytes_is_bounded_in_N(hass):
    a = hass.topk_distill_workspace_bytes(8192, 4096, 128256, 10)
    b = hass.topk_distill_workspace_bytes(65536, 4096, 128256, 10)
    scratch = 37 * 128 * 128256 * 2          # one chunk of dz_d rows, independent of N
    assert scratch <= a < scratch + (160 << 20)   # + statistics, lists and the fp32 Omega_hat term of one chunk
    assert b - a < (256 << 20)               # grows only by O(N K) lists and partial statistics
    assert a < 8192 * 128256 * 2             # less than one N x V bf16 matrix


@pytest.mark.parametrize("N,d,V,K", [(0, 64, 64, 1), (4, 12, 64, 1), (4, 64, 64, 65), (4, 64, 64, 0),
                                     (4, 64, 1000, 257), (4, 0, 64, 1)])
def test_bad_sizes_rejected_without_a_device(hass, N, d, V, K):
    out = ctypes.c_size_t(0)
    rc = hass.lib.hass_topk_distill_workspace_bytes(N, d, V, K, ctypes.byref(out))
    assert rc == -1
    buf = ctypes.create_string_buffer(64)
    p = ctypes.cast(buf, ctypes.c_void_p)
    rc = hass.lib.hass_topk_distill_fwd(p, p, p, N, d, V, K, p, p, p, p, p, p, 1 << 20, None)
    assert rc == -1


def test_null_and_misaligned_pointers_rejected(hass):
    buf = ctypes.create_string_buffer(4096)
    base = ctypes.addressof(buf)
    al = ctypes.c_void_p((base + 255) & ~255)
    mis = ctypes.c_void_p(al.value + 2)
    f = hass.lib.hass_topk_distill_fwd
    assert f(None, al, al, 4, 64, 64, 2, al, al, al, al, al, al, 1 << 20, None) == -1
    assert f(mis, al, al, 4, 64, 64, 2, al, al, al, al, al, al, 1 << 20, None) == -1
    assert f(al, al, al, 4, 64, 64, 2, al, al, al, al, al, None, 1 << 20, None) == -3
    assert f(al, al, al, 4, 64, 64, 2, al, al, al, al, al, mis, 1 << 20, None) == -3
    b = hass.lib.hass_topk_distill_bwd
    assert b(al, al, 4, 64, 64, 2, al, al, al, None, al, 7, al, 1 << 20, None) == -1
    assert b(al, al, 4, 64, 64, 2, None, al, al, None, al, 0, al, 1 << 20, None) == -1


def test_no_device_is_an_error_not_a_fallback(hass):
    import torch
    if torch.cuda.is_available():
        pytest.skip("a GPU is present")
    buf = ctypes.create_string_buffer(1 << 16)
    al = ctypes.c_void_p((ctypes.addressof(buf) + 255) & ~255)
    rc = hass.lib.hass_topk_distill_fwd(al, al, al, 4, 64, 64, 2, al, al, al, al, al, al, 1 << 15, None)
    assert rc in (-4, -6)


def test_hca_attention_arguments_rejected_before_the_device(hass):
    buf = ctypes.create_string_buffer(8192)
    al = ctypes.c_void_p((ctypes.addressof(buf) + 255) & ~255)
    mis = ctypes.c_void_p(al.value + 2)
    arr = (ctypes.c_void_p * 9)(*([al.value] * 9))
    f = hass.lib.hass_hca_attention_fwd
    sc = ctypes.c_float(0.088)

    def call(Q=al, m=1, H=2, Hkv=1, D=128, scale=sc, O=al, ws=al, wsz=256, kd=arr):
        return f(Q, al, al, kd, arr, m, 1, 16, H, Hkv, D, scale, O, None, ws, wsz, None)

    assert call(Q=None) == -1                     # null input
    assert call(Q=mis) == -1                      # misaligned input
    assert call(m=9) == -1                        # more draft passes than HASS_HCA_MAX_DRAFTS
    assert call(m=1, kd=None) == -1               # passes announced, no pointers
    assert call(H=3, Hkv=2) == -1                 # query heads not a multiple of key/value heads
    assert call(scale=ctypes.c_float(0.0)) == -1
    assert call(D=64) == -2                       # only head dimension 128
    assert call(ws=None) == -3 and call(wsz=8) == -3
    n = ctypes.c_size_t(0)
    assert hass.lib.hass_hca_attention_workspace_bytes(ctypes.byref(n)) == 0 and n.value == 256
    # backward: the workspace holds the status block, D and the two [B, H, T, m] arrays
    # status block, D [B, H, T] fp32 and the fp32 dQ accumulator [B, T, H, 128], each rounded up to 256 bytes
    rows = 2 * 4 * 100
    need = 256 + rows * 4 + rows * 128 * 4
    assert need <= hass.hca_attention_bwd_workspace_bytes(2, 100, 4, 3) <= need + 2 * 256
    assert hass.hca_attention_bwd_workspace_bytes(2, 100, 4, 0) == hass.hca_attention_bwd_workspace_bytes(2, 100, 4, 3)
    assert hass.lib.hass_hca_attention_bwd_workspace_bytes(2, 100, 4, 9, ctypes.byref(n)) == -1
    g = hass.lib.hass_hca_attention_bwd
    assert g(al, al, al, arr, arr, 1, 1, 16, 2, 1, 128, sc, al, None, al, al, al, al, arr, arr, al, 1 << 20, None) == -1
    assert g(al, al, al, arr, arr, 1, 1, 16, 2, 1, 128, sc, al, al, al, al, al, al, arr, arr, al, 16, None) == -3

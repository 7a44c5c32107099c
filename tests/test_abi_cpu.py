"""Host-side checks of the C ABI that need no GPU: the library loads, exports
every symbol include/ap.h declares, and rejects bad arguments before touching
a device."""
import ctypes
import os
import re

import pytest

from paper_2012_02030_b200 import binding as ap

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
FAKE = 0x10000  # a 16-byte aligned, never dereferenced "pointer"


def _declared():
    text = open(os.path.join(ROOT, "include", "ap.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(ap_[a-z_0-9]+)\s*\(", text)))


def test_every_declared_symbol_is_exported_and_bound():
    names = _declared()
    assert len(names) >= 12
    raw = ctypes.CDLL(ap._LIB_PATH)
    for n in names:
        assert hasattr(raw, n), n
        assert n in ap.EXPORTS, n
        assert hasattr(ap, n), n
    assert sorted(ap.EXPORTS) == names


def test_version_strings_sizes():
    assert ap.ap_version() >= 100
    assert ap.status_string(ap.AP_OK) == "ok"
    for s in range(6):
        assert ap.status_string(s) != "unknown status"
    assert ap.status_string(77) == "unknown status"
    assert ap.ap_tiles_capacity(16, 4096, 4096) == 16 * 32 * 32
    assert ap.ap_tiles_capacity(3, 129, 1) == 6
    assert ap.ap_tiles_capacity(0, 1, 1) == 0
    assert ap.ap_build_mask_workspace_bytes(2, 128, 128) > ap.ap_mask_to_tiles_workspace_bytes(2, 128, 128) > 0
    assert ap.ap_build_mask_workspace_bytes(2, 0, 128) == 0
    assert ap.ap_build_mask_workspace_bytes(1, 1 << 20, 1 << 20) == 0  # index range


def _tiles(H=2, Lq=128, Lk=128, cap=2, ptr=FAKE):
    return ap.ap_tiles(H, Lq, Lk, -(-Lq // 128), -(-Lk // 128), cap, *([ptr] * 9))


def test_forward_rejects_bad_arguments_before_any_device_work():
    t = _tiles()
    f = ap.lib.ap_sparse_attention_fwd
    ok = [FAKE, FAKE, FAKE, ctypes.byref(t), FAKE, 1, 2, 128, 128, 64, ap.AP_BF16, 0.0, None]

    def call(**kw):
        a = list(ok)
        for k, v in kw.items():
            a[int(k[1:])] = v
        return f(*a)

    assert call(a0=None) == ap.AP_ERR_INVALID_ARG
    assert call(a1=FAKE + 2) == ap.AP_ERR_INVALID_ARG        # misaligned
    assert call(a4=None) == ap.AP_ERR_INVALID_ARG
    assert call(a3=None) == ap.AP_ERR_INVALID_ARG
    assert call(a5=0) == ap.AP_ERR_INVALID_ARG               # B
    assert call(a7=129) == ap.AP_ERR_INVALID_ARG             # tiles built for another Lq
    assert call(a9=96) == ap.AP_ERR_UNSUPPORTED              # d
    assert call(a10=7) == ap.AP_ERR_UNSUPPORTED              # dtype
    assert call(a10=3) == ap.AP_ERR_UNSUPPORTED              # the code after AP_F16
    assert (ap.AP_F32, ap.AP_BF16, ap.AP_F16) == (0, 1, 2)
    assert call(a11=-1.0) == ap.AP_ERR_INVALID_ARG           # scale
    assert call(a11=float("nan")) == ap.AP_ERR_INVALID_ARG
    t0 = _tiles(cap=0)
    assert call(a3=ctypes.byref(t0)) == ap.AP_ERR_WORKSPACE
    tn = _tiles(ptr=None)
    assert call(a3=ctypes.byref(tn)) == ap.AP_ERR_INVALID_ARG


def test_backward_rejects_bad_arguments():
    f = ap.lib.ap_sparse_attention_bwd
    t = _tiles()
    ws = ap.ap_sparse_attention_bwd_workspace_bytes(1, 2, 128, 128)
    assert ws == 2 * 4 * 2 * 128 + 4 * 2 and ap.ap_sparse_attention_bwd_workspace_bytes(0, 1, 128, 128) == 0
    ok = [FAKE, FAKE, FAKE, FAKE, FAKE, ctypes.byref(t), FAKE, FAKE, FAKE, 1, 2, 128, 128, 64, 1, 0.0, FAKE, ws, None]
    for idx in (0, 1, 2, 3, 4, 6, 7, 8, 16):
        a = list(ok)
        a[idx] = None
        assert f(*a) == ap.AP_ERR_INVALID_ARG, idx
    a = list(ok); a[14] = 0
    assert f(*a) == ap.AP_ERR_UNSUPPORTED                      # fp32 tensors: no backward
    a = list(ok); a[13] = 96
    assert f(*a) == ap.AP_ERR_UNSUPPORTED
    a = list(ok); a[17] = ws - 1
    assert f(*a) == ap.AP_ERR_WORKSPACE
    a = list(ok); a[11] = 129
    assert f(*a) == ap.AP_ERR_INVALID_ARG                      # tiles built for another Lq


def test_accumulate_and_mask_reject_bad_arguments():
    f = ap.lib.ap_accumulate_attention
    assert f(None, FAKE, FAKE, None, 1, 1, 8, 8, 64, 1, 0, 0.0, None) == ap.AP_ERR_INVALID_ARG
    assert f(FAKE, FAKE, FAKE, FAKE + 4, 1, 1, 8, 8, 64, 1, 0, 0.0, None) == ap.AP_ERR_INVALID_ARG
    assert f(FAKE, FAKE, FAKE, None, 1, 1, 9, 8, 64, 1, 1, 0.0, None) == ap.AP_ERR_INVALID_ARG  # causal, Lk < Lq
    assert f(FAKE, FAKE, FAKE, None, 1, 1, 8, 8, 32, 1, 0, 0.0, None) == ap.AP_ERR_UNSUPPORTED
    f = ap.lib.ap_accumulate_attention_entmax15  # same checks
    assert f(None, FAKE, FAKE, None, 1, 1, 8, 8, 64, 1, 0, 0.0, None) == ap.AP_ERR_INVALID_ARG
    assert f(FAKE, FAKE, FAKE, FAKE + 4, 1, 1, 8, 8, 64, 1, 0, 0.0, None) == ap.AP_ERR_INVALID_ARG
    assert f(FAKE, FAKE, FAKE, None, 1, 1, 9, 8, 64, 1, 1, 0.0, None) == ap.AP_ERR_INVALID_ARG
    assert f(FAKE, FAKE, FAKE, None, 1, 1, 8, 8, 64, 1, 0, -1.0, None) == ap.AP_ERR_INVALID_ARG
    assert f(FAKE, FAKE, FAKE, None, 1, 1, 8, 8, 32, 1, 0, 0.0, None) == ap.AP_ERR_UNSUPPORTED
    assert f(FAKE, FAKE, FAKE, None, 1, 1, 8, 8, 64, 7, 0, 0.0, None) == ap.AP_ERR_UNSUPPORTED  # no such dtype
    t = _tiles(H=1, Lq=8, Lk=8, cap=1)
    ws = ap.ap_build_mask_workspace_bytes(1, 8, 8)
    for g in (ap.lib.ap_build_mask, ap.lib.ap_build_mask_layer):
        base = [FAKE, 1, 8, 8, 0.5, 0, 1, FAKE, ctypes.byref(t), FAKE, FAKE, ws, None]
        for idx, val in ((0, None), (4, 0.0), (4, 1.5), (4, float("nan")), (10, None), (7, FAKE + 1)):
            a = list(base)
            a[idx] = val
            assert g(*a) == ap.AP_ERR_INVALID_ARG, (idx, val)
        a = list(base)
        a[11] = ws - 1
        assert g(*a) == ap.AP_ERR_WORKSPACE
        a = list(base)
        a[2], a[5] = 9, 1  # causal with Lk < Lq
        assert g(*a) == ap.AP_ERR_INVALID_ARG
    ex = ap.lib.ap_build_mask_ex  # flags: per layer = 1, keep ties = 2; anything else is refused
    ok = [FAKE, 1, 8, 8, 0.5, 0, 1, 3, FAKE, ctypes.byref(t), FAKE, FAKE, ws, None]
    for bad in (4, 8, -1):
        a = list(ok); a[7] = bad
        assert ex(*a) == ap.AP_ERR_INVALID_ARG
    a = list(ok); a[12] = ws - 1
    assert ex(*a) == ap.AP_ERR_WORKSPACE
    a = list(ok); a[0] = None
    assert ex(*a) == ap.AP_ERR_INVALID_ARG
    # one selection over the layer ranks ties by a 32-bit index over all heads
    big = [FAKE, 64, 8192, 8192, 0.5, 0, 1, FAKE, None, FAKE, FAKE, ap.ap_build_mask_workspace_bytes(64, 8192, 8192),
           None]
    assert ap.lib.ap_build_mask_layer(*big) == ap.AP_ERR_UNSUPPORTED
    ps, eb = ap.lib.ap_pool_scores, ap.lib.ap_expand_block_mask
    assert ps(None, 1, 128, 128, 16, 0, FAKE, None) == ap.AP_ERR_INVALID_ARG
    assert ps(FAKE, 1, 128, 128, 16, 0, None, None) == ap.AP_ERR_INVALID_ARG
    assert ps(FAKE, 1, 128, 128, 24, 0, FAKE, None) == ap.AP_ERR_UNSUPPORTED   # block size
    assert ps(FAKE, 1, 128, 136, 16, 0, FAKE, None) == ap.AP_ERR_UNSUPPORTED   # Lk not a multiple
    assert ps(FAKE, 1, 256, 128, 16, 1, FAKE, None) == ap.AP_ERR_INVALID_ARG   # causal with Lk < Lq
    assert eb(None, 1, 128, 128, 16, 0, FAKE, None) == ap.AP_ERR_INVALID_ARG
    assert eb(FAKE, 1, 128, 128, 16, 0, FAKE + 4, None) == ap.AP_ERR_INVALID_ARG
    assert eb(FAKE, 1, 120, 128, 16, 0, FAKE, None) == ap.AP_ERR_UNSUPPORTED
    rs = ap.lib.ap_random_scores
    assert rs(None, 1, 8, 8, 1, None) == ap.AP_ERR_INVALID_ARG
    assert rs(FAKE + 4, 1, 8, 8, 1, None) == ap.AP_ERR_INVALID_ARG
    assert rs(FAKE, 1, 0, 8, 1, None) == ap.AP_ERR_INVALID_ARG
    m = ap.lib.ap_mask_to_tiles
    assert m(None, 1, 8, 8, ctypes.byref(t), FAKE, 1 << 20, None) == ap.AP_ERR_INVALID_ARG
    assert m(FAKE, 1, 8, 8, ctypes.byref(t), FAKE, 16, None) == ap.AP_ERR_WORKSPACE
    dt = ap.lib.ap_dense_tiles
    t4 = _tiles(H=1, Lq=256, Lk=256, cap=2)
    assert dt(1, 256, 256, 1, ctypes.byref(t4), None) == ap.AP_ERR_WORKSPACE  # needs 3 tiles
    assert dt(1, 256, 128, 1, ctypes.byref(t4), None) == ap.AP_ERR_INVALID_ARG  # causal with Lk < Lq
    t5 = _tiles(H=1, Lq=256, Lk=300, cap=4)
    assert dt(1, 256, 300, 1, ctypes.byref(t5), None) == ap.AP_ERR_WORKSPACE  # 44 memory keys: 2 + 3 tiles


def test_no_cpu_fallback_without_a_device():
    import torch

    if torch.cuda.is_available():
        pytest.skip("a device is present")
    t = _tiles()
    st = ap.lib.ap_sparse_attention_fwd(FAKE, FAKE, FAKE, ctypes.byref(t), FAKE, 1, 2, 128, 128, 64,
                                        ap.AP_BF16, 0.0, None)
    assert st == ap.AP_ERR_CUDA
    assert ap.lib.ap_device_status(None) == ap.AP_ERR_CUDA
    with pytest.raises(ValueError):
        ap.ap_sparse_attention_fwd(torch.zeros(1, 2, 128, 64), torch.zeros(1, 2, 128, 64),
                                   torch.zeros(1, 2, 128, 64), None)

"""Thin ctypes binding of libap_b200.so: argument marshalling only.

Every function has the name of the C entry point it calls (see include/ap.h)
and takes torch tensors that live on the CUDA device (PyTorch is used for
device memory and streams only).  All arithmetic happens inside the library's
kernels.  If the shared library has not been built the import of this module
fails: there is no fallback path.
"""
from __future__ import annotations

import ctypes
import os

import torch

TILE = 128
AP_OK, AP_ERR_INVALID_ARG, AP_ERR_UNSUPPORTED, AP_ERR_WORKSPACE, AP_ERR_CUDA, AP_ERR_TIMEOUT = range(6)
AP_F32, AP_BF16, AP_F16 = 0, 1, 2
AP_STATIC_MAX_TILES = 1024

# AP_B200_LIB names another build of the same library (e.g. one compiled with development aids)
_LIB_PATH = os.environ.get("AP_B200_LIB") or os.path.join(os.path.dirname(os.path.abspath(__file__)), "libap_b200.so")


class ApError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__("%s: %s (status %d)" % (where, status_string(status), status))


class ap_tiles(ctypes.Structure):
    _fields_ = [
        ("H", ctypes.c_int32), ("Lq", ctypes.c_int32), ("Lk", ctypes.c_int32),
        ("n_qt", ctypes.c_int32), ("n_kt", ctypes.c_int32), ("cap", ctypes.c_int32),
        ("row_ptr", ctypes.c_void_p), ("col_idx", ctypes.c_void_p),
        ("flags", ctypes.c_void_p), ("bitmap", ctypes.c_void_p), ("groups", ctypes.c_void_p),
        ("round_ptr", ctypes.c_void_p), ("round_rows", ctypes.c_void_p), ("round_info", ctypes.c_void_p),
        ("round_bitmap", ctypes.c_void_p),
        ("ground_ptr", ctypes.c_void_p), ("ground_keys", ctypes.c_void_p), ("ground_info", ctypes.c_void_p),
        ("ground_bitmap", ctypes.c_void_p), ("unit_qt", ctypes.c_void_p),
    ]


def _load() -> ctypes.CDLL:
    if not os.path.exists(_LIB_PATH):
        raise ImportError(
            "libap_b200.so is missing: build it with `python -m paper_2012_02030_b200.build` "
            "(there is no fallback implementation)")
    lib = ctypes.CDLL(_LIB_PATH)
    vp, i, f, d, sz, i64 = (ctypes.c_void_p, ctypes.c_int, ctypes.c_float, ctypes.c_double,
                            ctypes.c_size_t, ctypes.c_int64)
    tp = ctypes.POINTER(ap_tiles)
    sig = {
        "ap_version": (i, []),
        "ap_launch_count": (ctypes.c_uint64, []),
        "ap_debug_expire_waits": (None, [i]),
        "ap_debug_schedule": (None, [i]),
        "ap_status_string": (ctypes.c_char_p, [i]),
        "ap_tiles_capacity": (i64, [i, i, i]),
        "ap_build_mask_workspace_bytes": (sz, [i, i, i]),
        "ap_mask_to_tiles_workspace_bytes": (sz, [i, i, i]),
        "ap_accumulate_attention": (i, [vp, vp, vp, vp, i, i, i, i, i, i, i, f, vp]),
        "ap_accumulate_attention_entmax15": (i, [vp, vp, vp, vp, i, i, i, i, i, i, i, f, vp]),
        "ap_build_mask": (i, [vp, i, i, i, d, i, i, vp, tp, vp, vp, sz, vp]),
        "ap_build_mask_layer": (i, [vp, i, i, i, d, i, i, vp, tp, vp, vp, sz, vp]),
        "ap_build_mask_ex": (i, [vp, i, i, i, d, i, i, i, vp, tp, vp, vp, sz, vp]),
        "ap_random_scores": (i, [vp, i, i, i, ctypes.c_uint64, vp]),
        "ap_pool_scores": (i, [vp, i, i, i, i, i, vp, vp]),
        "ap_expand_block_mask": (i, [vp, i, i, i, i, i, vp, vp]),
        "ap_mask_to_tiles": (i, [vp, i, i, i, tp, vp, sz, vp]),
        "ap_dense_tiles": (i, [i, i, i, i, tp, vp]),
        "ap_mask_to_tiles_static": (i, [vp, i, i, i, tp, vp]),
        "ap_sparse_attention_fwd": (i, [vp, vp, vp, tp, vp, i, i, i, i, i, i, f, vp]),
        "ap_sparse_attention_entmax15_fwd": (i, [vp, vp, vp, tp, vp, i, i, i, i, i, i, f, vp]),
        "ap_sparse_attention_fwd_host": (i, [vp, vp, vp, tp, vp, vp, vp, vp, vp, i, i, i, i, i, i, f, vp]),
        "ap_sparse_attention_bwd_workspace_bytes": (sz, [i, i, i, i]),
        "ap_sparse_attention_bwd": (i, [vp, vp, vp, vp, vp, tp, vp, vp, vp, i, i, i, i, i, i, f, vp, sz, vp]),
        "ap_device_status": (i, [vp]),
    }
    for name, (res, args) in sig.items():
        fn = getattr(lib, name)
        fn.restype, fn.argtypes = res, args
    return lib


lib = _load()
EXPORTS = ("ap_version", "ap_launch_count", "ap_debug_expire_waits", "ap_debug_schedule", "ap_status_string", "ap_tiles_capacity", "ap_build_mask_workspace_bytes",
           "ap_mask_to_tiles_workspace_bytes", "ap_accumulate_attention", "ap_accumulate_attention_entmax15", "ap_build_mask", "ap_build_mask_layer", "ap_build_mask_ex", "ap_random_scores", "ap_pool_scores", "ap_expand_block_mask",
           "ap_mask_to_tiles", "ap_mask_to_tiles_static", "ap_dense_tiles", "ap_sparse_attention_fwd", "ap_sparse_attention_entmax15_fwd",
           "ap_sparse_attention_fwd_host", "ap_sparse_attention_bwd_workspace_bytes", "ap_sparse_attention_bwd",
           "ap_device_status")


def status_string(status: int) -> str:
    return lib.ap_status_string(int(status)).decode()


ap_status_string = status_string


def ap_version() -> int:
    return int(lib.ap_version())


def ap_launch_count() -> int:
    return int(lib.ap_launch_count())


def ap_debug_expire_waits(on: bool) -> None:
    lib.ap_debug_expire_waits(1 if on else 0)


def ap_debug_schedule(mode: int) -> None:
    """0: gathered rounds where the builders expect them to pay; 1: the forward follows the rounds only;
    2: the builders give every list row its gathered rounds."""
    lib.ap_debug_schedule(int(mode))


def ap_tiles_capacity(H: int, Lq: int, Lk: int) -> int:
    return int(lib.ap_tiles_capacity(H, Lq, Lk))


def ap_build_mask_workspace_bytes(H: int, Lq: int, Lk: int) -> int:
    return int(lib.ap_build_mask_workspace_bytes(H, Lq, Lk))


def ap_mask_to_tiles_workspace_bytes(H: int, Lq: int, Lk: int) -> int:
    return int(lib.ap_mask_to_tiles_workspace_bytes(H, Lq, Lk))


def _stream(stream) -> int:
    if stream is None:
        stream = torch.cuda.current_stream()
    return int(stream.cuda_stream)


def _ptr(t):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


def _dtype_code(t: torch.Tensor) -> int:
    if t.dtype == torch.float32:
        return AP_F32
    if t.dtype == torch.bfloat16:
        return AP_BF16
    if t.dtype == torch.float16:
        return AP_F16
    raise TypeError("dtype must be float32, bfloat16 or float16, got %s" % t.dtype)


def _check(status: int, where: str) -> None:
    if status != AP_OK:
        raise ApError(status, where)


def _dev(t: torch.Tensor, name: str) -> torch.Tensor:
    if not t.is_cuda or not t.is_contiguous():
        raise ValueError("%s must be a contiguous CUDA tensor" % name)
    return t


class Tiles:
    """Device buffers of a tile list plus the ap_tiles descriptor that points at them."""

    def __init__(self, H: int, Lq: int, Lk: int, device="cuda", cap: int | None = None, gathered: bool = False,
                 paired: bool = False):
        self.H, self.Lq, self.Lk = H, Lq, Lk
        self.n_qt, self.n_kt = -(-Lq // TILE), -(-Lk // TILE)
        self.cap = ap_tiles_capacity(H, Lq, Lk) if cap is None else cap
        self.row_ptr = torch.zeros(H * self.n_qt + 1, dtype=torch.int32, device=device)
        self.col_idx = torch.zeros(max(self.cap, 1), dtype=torch.int32, device=device)
        self.flags = torch.zeros(max(self.cap, 1), dtype=torch.uint8, device=device)
        self.bitmap = torch.zeros((max(self.cap, 1), TILE, 4), dtype=torch.int32, device=device)
        self.groups = torch.zeros(max(self.cap, 1), dtype=torch.uint8, device=device)
        # the forward pass's schedule (rounds of up to eight non-empty 16-column groups)
        self.round_ptr = torch.zeros(H * self.n_qt + 1, dtype=torch.int32, device=device)
        self.round_rows = torch.zeros((max(self.cap, 1), 8), dtype=torch.int32, device=device)
        self.round_info = torch.zeros(max(self.cap, 1), dtype=torch.uint8, device=device)
        self.round_bitmap = torch.zeros((max(self.cap, 1), TILE, 4), dtype=torch.int32, device=device)
        # the optional second schedule (rounds of 128 individually gathered key columns)
        self.gathered = gathered
        g = [None] * 4
        if gathered:
            self.ground_ptr = torch.zeros(H * self.n_qt + 1, dtype=torch.int32, device=device)
            self.ground_keys = torch.zeros((max(self.cap, 1), TILE), dtype=torch.int32, device=device)
            self.ground_info = torch.zeros(max(self.cap, 1), dtype=torch.uint8, device=device)
            self.ground_bitmap = torch.zeros((max(self.cap, 1), TILE, 4), dtype=torch.int32, device=device)
            g = [self.ground_ptr.data_ptr(), self.ground_keys.data_ptr(), self.ground_info.data_ptr(),
                 self.ground_bitmap.data_ptr()]
        # the forward's units of work: pairs of query tiles of a head, balanced by the builders
        self.unit_qt = torch.zeros((H, (self.n_qt + 1) // 2, 2), dtype=torch.int32, device=device) if paired else None
        self.c = ap_tiles(H, Lq, Lk, self.n_qt, self.n_kt, self.cap, self.row_ptr.data_ptr(),
                          self.col_idx.data_ptr(), self.flags.data_ptr(), self.bitmap.data_ptr(),
                          self.groups.data_ptr(), self.round_ptr.data_ptr(), self.round_rows.data_ptr(),
                          self.round_info.data_ptr(), self.round_bitmap.data_ptr(), *g,
                          self.unit_qt.data_ptr() if paired else None)

    def n_tiles(self) -> int:
        """Number of stored tiles (synchronises)."""
        return int(self.row_ptr[-1].item())

    def to_host(self):
        """dict of numpy arrays trimmed to the stored tiles (synchronises)."""
        T = self.n_tiles()
        return dict(row_ptr=self.row_ptr.cpu().numpy(), col_idx=self.col_idx[:T].cpu().numpy(),
                    flags=self.flags[:T].cpu().numpy(), groups=self.groups[:T].cpu().numpy(),
                    bitmap=self.bitmap[:T].cpu().numpy().view("uint32"), n_qt=self.n_qt, n_kt=self.n_kt,
                    **self.rounds_to_host())

    def grounds_to_host(self):
        """The gathered-round arrays trimmed to the stored gathered rounds (synchronises)."""
        R = int(self.ground_ptr[-1].item())
        return dict(ground_ptr=self.ground_ptr.cpu().numpy(), ground_keys=self.ground_keys[:R].cpu().numpy(),
                    ground_info=self.ground_info[:R].cpu().numpy(),
                    ground_bitmap=self.ground_bitmap[:R].cpu().numpy().view("uint32"))

    def rounds_to_host(self):
        """The round arrays trimmed to the stored rounds (synchronises)."""
        R = int(self.round_ptr[-1].item())
        return dict(round_ptr=self.round_ptr.cpu().numpy(), round_rows=self.round_rows[:R].cpu().numpy(),
                    round_info=self.round_info[:R].cpu().numpy(),
                    round_bitmap=self.round_bitmap[:R].cpu().numpy().view("uint32"))


def ap_accumulate_attention(acc, Q, K, bias=None, causal=False, scale=0.0, stream=None) -> None:
    _dev(acc, "acc"), _dev(Q, "Q"), _dev(K, "K")
    B, H, Lq, d = Q.shape
    Lk = K.shape[2]
    if K.shape != (B, H, Lk, d) or acc.shape != (H, Lq, Lk) or acc.dtype != torch.float32 or K.dtype != Q.dtype:
        raise ValueError("shape/dtype mismatch")
    if bias is not None and (_dev(bias, "bias").shape != (H, Lq, Lk) or bias.dtype != torch.float32):
        raise ValueError("bias must be float32 [H,Lq,Lk]")
    _check(lib.ap_accumulate_attention(_ptr(acc), _ptr(Q), _ptr(K), _ptr(bias), B, H, Lq, Lk, d,
                                       _dtype_code(Q), int(bool(causal)), float(scale), _stream(stream)),
           "ap_accumulate_attention")


def ap_accumulate_attention_entmax15(acc, Q, K, bias=None, causal=False, scale=0.0, stream=None) -> None:
    _dev(acc, "acc"), _dev(Q, "Q"), _dev(K, "K")
    B, H, Lq, d = Q.shape
    Lk = K.shape[2]
    if K.shape != (B, H, Lk, d) or acc.shape != (H, Lq, Lk) or acc.dtype != torch.float32 or K.dtype != Q.dtype:
        raise ValueError("shape/dtype mismatch")
    if bias is not None and (_dev(bias, "bias").shape != (H, Lq, Lk) or bias.dtype != torch.float32):
        raise ValueError("bias must be float32 [H,Lq,Lk]")
    _check(lib.ap_accumulate_attention_entmax15(_ptr(acc), _ptr(Q), _ptr(K), _ptr(bias), B, H, Lq, Lk, d,
                                                _dtype_code(Q), int(bool(causal)), float(scale), _stream(stream)),
           "ap_accumulate_attention_entmax15")


def _build_mask(fn, name, acc, keep_frac, causal, keep_diag, mask, tiles, nnz_per_head, workspace, stream) -> None:
    _dev(acc, "acc")
    H, Lq, Lk = acc.shape
    if acc.dtype != torch.float32:
        raise ValueError("acc must be float32")
    if workspace is None:
        workspace = torch.empty(ap_build_mask_workspace_bytes(H, Lq, Lk), dtype=torch.uint8, device=acc.device)
    _check(fn(_ptr(acc), H, Lq, Lk, float(keep_frac), int(bool(causal)), int(bool(keep_diag)),
              _ptr(mask), ctypes.byref(tiles.c) if tiles is not None else None,
              _ptr(nnz_per_head), _ptr(workspace), workspace.numel(), _stream(stream)), name)


def ap_build_mask(acc, keep_frac, causal=False, keep_diag=True, mask=None, tiles: Tiles | None = None,
                  nnz_per_head=None, workspace=None, stream=None) -> None:
    _build_mask(lib.ap_build_mask, "ap_build_mask", acc, keep_frac, causal, keep_diag, mask, tiles, nnz_per_head,
                workspace, stream)


def ap_build_mask_layer(acc, keep_frac, causal=False, keep_diag=True, mask=None, tiles: Tiles | None = None,
                        nnz_per_head=None, workspace=None, stream=None) -> None:
    _build_mask(lib.ap_build_mask_layer, "ap_build_mask_layer", acc, keep_frac, causal, keep_diag, mask, tiles,
                nnz_per_head, workspace, stream)


AP_MASK_PER_LAYER, AP_MASK_KEEP_TIES = 1, 2


def ap_build_mask_ex(acc, keep_frac, causal=False, keep_diag=True, flags=0, mask=None, tiles: Tiles | None = None,
                     nnz_per_head=None, workspace=None, stream=None) -> None:
    _dev(acc, "acc")
    H, Lq, Lk = acc.shape
    if acc.dtype != torch.float32:
        raise ValueError("acc must be float32")
    if workspace is None:
        workspace = torch.empty(ap_build_mask_workspace_bytes(H, Lq, Lk), dtype=torch.uint8, device=acc.device)
    _check(lib.ap_build_mask_ex(_ptr(acc), H, Lq, Lk, float(keep_frac), int(bool(causal)), int(bool(keep_diag)),
                                int(flags), _ptr(mask), ctypes.byref(tiles.c) if tiles is not None else None,
                                _ptr(nnz_per_head), _ptr(workspace), workspace.numel(), _stream(stream)),
           "ap_build_mask_ex")


def ap_pool_scores(acc, block: int, causal=False, pooled=None, stream=None):
    _dev(acc, "acc")
    H, Lq, Lk = acc.shape
    if acc.dtype != torch.float32:
        raise ValueError("acc must be float32")
    if pooled is None:
        pooled = torch.empty((H, max(Lq // max(block, 1), 1), max(Lk // max(block, 1), 1)), dtype=torch.float32,
                             device=acc.device)
    _check(lib.ap_pool_scores(_ptr(acc), H, Lq, Lk, int(block), int(bool(causal)), _ptr(pooled), _stream(stream)),
           "ap_pool_scores")
    return pooled


def ap_expand_block_mask(block_mask, block: int, causal=False, mask=None, stream=None):
    _dev(block_mask, "block_mask")
    H, R, C = block_mask.shape
    if block_mask.dtype != torch.uint8:
        raise ValueError("block_mask must be uint8")
    if mask is None:
        mask = torch.empty((H, R * block, C * block), dtype=torch.uint8, device=block_mask.device)
    _check(lib.ap_expand_block_mask(_ptr(block_mask), H, R * block, C * block, int(block), int(bool(causal)),
                                    _ptr(mask), _stream(stream)), "ap_expand_block_mask")
    return mask


def ap_random_scores(scores, seed: int, stream=None) -> None:
    _dev(scores, "scores")
    H, Lq, Lk = scores.shape
    if scores.dtype != torch.float32:
        raise ValueError("scores must be float32")
    _check(lib.ap_random_scores(_ptr(scores), H, Lq, Lk, int(seed) & ((1 << 64) - 1), _stream(stream)),
           "ap_random_scores")


def ap_mask_to_tiles(mask, tiles: Tiles, workspace=None, stream=None) -> None:
    _dev(mask, "mask")
    H, Lq, Lk = mask.shape
    if mask.dtype != torch.uint8:
        raise ValueError("mask must be uint8")
    if workspace is None:
        workspace = torch.empty(ap_mask_to_tiles_workspace_bytes(H, Lq, Lk), dtype=torch.uint8, device=mask.device)
    _check(lib.ap_mask_to_tiles(_ptr(mask), H, Lq, Lk, ctypes.byref(tiles.c), _ptr(workspace),
                                workspace.numel(), _stream(stream)), "ap_mask_to_tiles")


def ap_mask_to_tiles_static(mask, tiles: Tiles, stream=None) -> None:
    """ap_mask_to_tiles without a workspace: the staging area is the library's built-in
    device array (shapes of at most AP_STATIC_MAX_TILES grid tiles).  The binding passes
    the caller's mask and tile buffers straight through and allocates nothing."""
    _dev(mask, "mask")
    H, Lq, Lk = mask.shape
    if mask.dtype != torch.uint8:
        raise ValueError("mask must be uint8")
    _check(lib.ap_mask_to_tiles_static(_ptr(mask), H, Lq, Lk, ctypes.byref(tiles.c), _stream(stream)),
           "ap_mask_to_tiles_static")


def ap_dense_tiles(tiles: Tiles, causal=False, stream=None) -> None:
    _check(lib.ap_dense_tiles(tiles.H, tiles.Lq, tiles.Lk, int(bool(causal)), ctypes.byref(tiles.c),
                              _stream(stream)), "ap_dense_tiles")


def ap_sparse_attention_fwd(Q, K, V, tiles: Tiles, O=None, scale=0.0, stream=None):
    _dev(Q, "Q"), _dev(K, "K"), _dev(V, "V")
    B, H, Lq, d = Q.shape
    Lk = K.shape[2]
    if K.shape != (B, H, Lk, d) or V.shape != K.shape or K.dtype != Q.dtype or V.dtype != Q.dtype:
        raise ValueError("shape/dtype mismatch")
    if O is None:
        O = torch.empty_like(Q)
    _check(lib.ap_sparse_attention_fwd(_ptr(Q), _ptr(K), _ptr(V), ctypes.byref(tiles.c), _ptr(_dev(O, "O")),
                                       B, H, Lq, Lk, d, _dtype_code(Q), float(scale), _stream(stream)),
           "ap_sparse_attention_fwd")
    return O


def ap_sparse_attention_entmax15_fwd(Q, K, V, tiles: Tiles, O=None, scale=0.0, stream=None):
    _dev(Q, "Q"), _dev(K, "K"), _dev(V, "V")
    B, H, Lq, d = Q.shape
    Lk = K.shape[2]
    if K.shape != (B, H, Lk, d) or V.shape != K.shape or K.dtype != Q.dtype or V.dtype != Q.dtype:
        raise ValueError("shape/dtype mismatch")
    if O is None:
        O = torch.empty_like(Q)
    _check(lib.ap_sparse_attention_entmax15_fwd(_ptr(Q), _ptr(K), _ptr(V), ctypes.byref(tiles.c), _ptr(_dev(O, "O")),
                                                B, H, Lq, Lk, d, _dtype_code(Q), float(scale), _stream(stream)),
           "ap_sparse_attention_entmax15_fwd")
    return O


def ap_sparse_attention_bwd_workspace_bytes(B: int, H: int, Lq: int, Lk: int) -> int:
    return int(lib.ap_sparse_attention_bwd_workspace_bytes(B, H, Lq, Lk))


def ap_sparse_attention_bwd(Q, K, V, O, dO, tiles: Tiles, dQ=None, dK=None, dV=None, scale=0.0, workspace=None,
                            stream=None):
    for t, name in ((Q, "Q"), (K, "K"), (V, "V"), (O, "O"), (dO, "dO")):
        _dev(t, name)
    B, H, Lq, d = Q.shape
    Lk = K.shape[2]
    if (K.shape != (B, H, Lk, d) or V.shape != K.shape or O.shape != Q.shape or dO.shape != Q.shape
            or any(t.dtype != Q.dtype for t in (K, V, O, dO))):
        raise ValueError("shape/dtype mismatch")
    dQ = torch.empty_like(Q) if dQ is None else _dev(dQ, "dQ")
    dK = torch.empty_like(K) if dK is None else _dev(dK, "dK")
    dV = torch.empty_like(V) if dV is None else _dev(dV, "dV")
    if workspace is None:
        workspace = torch.empty(ap_sparse_attention_bwd_workspace_bytes(B, H, Lq, Lk), dtype=torch.uint8,
                                device=Q.device)
    _check(lib.ap_sparse_attention_bwd(_ptr(Q), _ptr(K), _ptr(V), _ptr(O), _ptr(dO), ctypes.byref(tiles.c),
                                       _ptr(dQ), _ptr(dK), _ptr(dV), B, H, Lq, Lk, d, _dtype_code(Q), float(scale),
                                       _ptr(workspace), workspace.numel(), _stream(stream)),
           "ap_sparse_attention_bwd")
    return dQ, dK, dV


def ap_sparse_attention_fwd_host(hQ, hK, hV, tiles: Tiles, hO, dQ, dK, dV, dO, scale=0.0, stream=None):
    """Host tensors in, host tensor out; d* are device staging buffers of the same shapes."""
    B, H, Lq, d = hQ.shape
    Lk = hK.shape[2]
    for t in (hQ, hK, hV, hO):
        if t.is_cuda or not t.is_contiguous():
            raise ValueError("h* must be contiguous host tensors")
    _check(lib.ap_sparse_attention_fwd_host(_ptr(hQ), _ptr(hK), _ptr(hV), ctypes.byref(tiles.c), _ptr(hO),
                                            _ptr(_dev(dQ, "dQ")), _ptr(_dev(dK, "dK")), _ptr(_dev(dV, "dV")),
                                            _ptr(_dev(dO, "dO")), B, H, Lq, Lk, d, _dtype_code(hQ),
                                            float(scale), _stream(stream)), "ap_sparse_attention_fwd_host")
    return hO


def ap_device_status(stream=None) -> int:
    return int(lib.ap_device_status(_stream(stream)))

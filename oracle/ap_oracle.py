"""ctypes front end of the CPU oracle (``ap_oracle.c``).  TEST INFRASTRUCTURE ONLY.

The oracle is the slow fp64 restatement of Attention Pruning's equations that
the CUDA library is checked against.  Only the tests, the smoke check and the
benchmark's CPU-baseline leg may import this module; the CUDA path never does,
and this module imports nothing from the CUDA package.

Arrays are numpy: float32 inputs holding the exact (bf16- or fp32-valued)
numbers the GPU receives, float64 results.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "ap_oracle.c")
_LIB = os.path.join(_HERE, "libap_oracle.so")
TILE = 128


def build(force: bool = False) -> str:
    """Compile ap_oracle.c with gcc (OpenMP, -O2, no fast-math) if stale."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".%d.tmp" % os.getpid()
        subprocess.check_call(
            ["gcc", "-O2", "-std=c99", "-fopenmp", "-shared", "-fPIC", "-o", tmp, _SRC, "-lm"]
        )
        os.replace(tmp, _LIB)
    return _LIB


_lib = None


def _load():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        _lib.oracle_keep_count.restype = ctypes.c_int64
        _lib.oracle_keep_count.argtypes = [ctypes.c_int64, ctypes.c_int64, ctypes.c_double]
        _lib.oracle_mask_to_tiles.restype = ctypes.c_int64
        _lib.oracle_build_mask.restype = ctypes.c_int
        _lib.oracle_num_threads.restype = ctypes.c_int
    return _lib


def _p(a: np.ndarray):
    return a.ctypes.data_as(ctypes.c_void_p)


def _f32(a) -> np.ndarray:
    return np.ascontiguousarray(np.asarray(a, dtype=np.float32))


def num_threads() -> int:
    return int(_load().oracle_num_threads())


def set_num_threads(n: int) -> None:
    _load().oracle_set_num_threads(ctypes.c_int(n))


def keep_count(n_valid: int, n_forced: int, keep_frac: float) -> int:
    """k of Eq. 2's top-k reading: max(n_forced, min(n_valid, floor(keep_frac*n_valid+0.5)))."""
    return int(_load().oracle_keep_count(n_valid, n_forced, float(keep_frac)))


def _check_domain(Lq: int, Lk: int, causal: bool) -> None:
    """Causal: keys j <= i + (Lk - Lq), i.e. Lk - Lq memory keys before the current segment."""
    if causal and Lk < Lq:
        raise ValueError("the causal domain needs Lk >= Lq")


def pool_scores(acc32, block: int, causal: bool = False) -> np.ndarray:
    """Block scores for block-structured pruning: float64 [H, Lq/block, Lk/block], the mean of acc over
    each block's entries inside the domain (0 for blocks outside it)."""
    acc32 = _f32(acc32)
    H, Lq, Lk = acc32.shape
    _check_domain(Lq, Lk, causal)
    if block < 1 or Lq % block or Lk % block:
        raise ValueError("Lq and Lk must be multiples of the block size")
    out = np.zeros((H, Lq // block, Lk // block), dtype=np.float64)
    lib = _load()
    lib.oracle_pool_scores.restype = None
    lib.oracle_pool_scores(_p(acc32), H, Lq, Lk, block, int(bool(causal)), _p(out))
    return out


def expand_block_mask(block_mask, block: int, causal: bool = False) -> np.ndarray:
    """Element mask of a block mask: uint8 [H, R*block, C*block]; a kept block keeps its entries inside the domain."""
    bm = np.ascontiguousarray(np.asarray(block_mask, dtype=np.uint8))
    H, R, C = bm.shape
    Lq, Lk = R * block, C * block
    _check_domain(Lq, Lk, causal)
    out = np.zeros((H, Lq, Lk), dtype=np.uint8)
    lib = _load()
    lib.oracle_expand_block_mask.restype = None
    lib.oracle_expand_block_mask(_p(bm), H, Lq, Lk, block, int(bool(causal)), _p(out))
    return out


def random_scores(H: int, Lq: int, Lk: int, seed: int) -> np.ndarray:
    """Scores of the random-pruning control: float32 [H,Lq,Lk] in [0,1), entry n = (h*Lq+i)*Lk+j from
    the (n+1)-th SplitMix64 output for `seed` (top 24 bits)."""
    out = np.zeros((H, Lq, Lk), dtype=np.float32)
    lib = _load()
    lib.oracle_random_scores.restype = None
    lib.oracle_random_scores(_p(out), ctypes.c_int64(out.size), ctypes.c_uint64(seed & ((1 << 64) - 1)))
    return out


def accumulate(acc: np.ndarray, Q, K, bias=None, causal: bool = False, scale: float | None = None):
    """Eq. 1 as a running sum: acc[H,Lq,Lk] (float64, in place) += sum_b softmax(Q_b K_b^T*scale + bias)."""
    Q, K = _f32(Q), _f32(K)
    B, H, Lq, d = Q.shape
    Lk = K.shape[2]
    assert K.shape == (B, H, Lk, d) and acc.shape == (H, Lq, Lk)
    assert acc.dtype == np.float64 and acc.flags.c_contiguous
    _check_domain(Lq, Lk, causal)
    if bias is not None:
        bias = _f32(bias)
        assert bias.shape == (H, Lq, Lk)
    s = 1.0 / np.sqrt(d) if scale is None else scale
    _load().oracle_accumulate(
        _p(acc), _p(Q), _p(K), _p(bias) if bias is not None else None,
        B, H, Lq, Lk, d, int(bool(causal)), ctypes.c_double(s),
    )
    return acc


def accumulate_rows(rows, Q, K, bias=None, causal: bool = False, scale: float | None = None):
    """Eq. 1's sum for sampled (h, i) rows only; returns float64 [len(rows), Lk]."""
    Q, K = _f32(Q), _f32(K)
    B, H, Lq, d = Q.shape
    Lk = K.shape[2]
    _check_domain(Lq, Lk, causal)
    rows = np.ascontiguousarray(np.asarray(rows, dtype=np.int32).reshape(-1, 2))
    out = np.zeros((rows.shape[0], Lk), dtype=np.float64)
    if bias is not None:
        bias = _f32(bias)
    s = 1.0 / np.sqrt(d) if scale is None else scale
    _load().oracle_accumulate_rows(
        _p(out), _p(rows), rows.shape[0], _p(Q), _p(K), _p(bias) if bias is not None else None,
        B, H, Lq, Lk, d, int(bool(causal)), ctypes.c_double(s),
    )
    return out


def build_mask(acc32, keep_frac: float, causal: bool = False, keep_diag: bool = True):
    """Eq. 2 as exact per-head top-k on fp32 values; returns (mask uint8 [H,Lq,Lk], nnz int64 [H])."""
    acc32 = _f32(acc32)
    H, Lq, Lk = acc32.shape
    _check_domain(Lq, Lk, causal)
    mask = np.zeros((H, Lq, Lk), dtype=np.uint8)
    nnz = np.zeros((H,), dtype=np.int64)
    rc = _load().oracle_build_mask(
        _p(acc32), H, Lq, Lk, ctypes.c_double(keep_frac), int(bool(causal)), int(bool(keep_diag)),
        _p(mask), _p(nnz),
    )
    if rc != 0:
        raise MemoryError("oracle_build_mask")
    return mask, nnz


def build_mask_layer(acc32, keep_frac: float, causal: bool = False, keep_diag: bool = True):
    """Eq. 2 with one threshold for all heads of the layer (the paper's own statement), as an exact
    top-k over the union of the heads' domains; returns (mask uint8 [H,Lq,Lk], nnz int64 [H])."""
    acc32 = _f32(acc32)
    H, Lq, Lk = acc32.shape
    _check_domain(Lq, Lk, causal)
    mask = np.zeros((H, Lq, Lk), dtype=np.uint8)
    nnz = np.zeros((H,), dtype=np.int64)
    lib = _load()
    lib.oracle_build_mask_layer.restype = ctypes.c_int
    rc = lib.oracle_build_mask_layer(
        _p(acc32), H, Lq, Lk, ctypes.c_double(keep_frac), int(bool(causal)), int(bool(keep_diag)),
        _p(mask), _p(nnz),
    )
    if rc != 0:
        raise MemoryError("oracle_build_mask_layer")
    return mask, nnz


def build_mask_ties(acc32, keep_frac: float, causal: bool = False, keep_diag: bool = True, per_layer: bool = False):
    """Eq. 2 with its strict inequality: the threshold is the exact top-k's last kept value and every entry
    equal to it stays; returns (mask uint8 [H,Lq,Lk], nnz int64 [H])."""
    acc32 = _f32(acc32)
    H, Lq, Lk = acc32.shape
    _check_domain(Lq, Lk, causal)
    mask = np.zeros((H, Lq, Lk), dtype=np.uint8)
    nnz = np.zeros((H,), dtype=np.int64)
    lib = _load()
    lib.oracle_build_mask_ties.restype = ctypes.c_int
    rc = lib.oracle_build_mask_ties(
        _p(acc32), H, Lq, Lk, ctypes.c_double(keep_frac), int(bool(causal)), int(bool(keep_diag)),
        int(bool(per_layer)), _p(mask), _p(nnz),
    )
    if rc != 0:
        raise MemoryError("oracle_build_mask_ties")
    return mask, nnz


def mask_to_tiles(mask):
    """Tile list of a mask: dict(row_ptr, col_idx, flags, bitmap) trimmed to the T non-empty tiles."""
    mask = np.ascontiguousarray(np.asarray(mask, dtype=np.uint8))
    H, Lq, Lk = mask.shape
    n_qt, n_kt = -(-Lq // TILE), -(-Lk // TILE)
    cap = H * n_qt * n_kt
    row_ptr = np.zeros((H * n_qt + 1,), dtype=np.int32)
    col_idx = np.zeros((cap,), dtype=np.int32)
    flags = np.zeros((cap,), dtype=np.uint8)
    bitmap = np.zeros((cap, TILE, 4), dtype=np.uint32)
    T = int(_load().oracle_mask_to_tiles(
        _p(mask), H, Lq, Lk, _p(row_ptr), _p(col_idx), _p(flags), _p(bitmap), ctypes.c_int64(cap)))
    assert T >= 0
    return dict(row_ptr=row_ptr, col_idx=col_idx[:T].copy(), flags=flags[:T].copy(),
                bitmap=bitmap[:T].copy(), n_qt=n_qt, n_kt=n_kt)


def attention_fwd(Q, K, V, mask, scale: float | None = None) -> np.ndarray:
    """Masked attention of Section 3.2 in fp64: O[B,H,Lq,d]; rows with no kept key are 0."""
    Q, K, V = _f32(Q), _f32(K), _f32(V)
    mask = np.ascontiguousarray(np.asarray(mask, dtype=np.uint8))
    B, H, Lq, d = Q.shape
    Lk = K.shape[2]
    assert K.shape == (B, H, Lk, d) and V.shape == (B, H, Lk, d) and mask.shape == (H, Lq, Lk)
    O = np.zeros((B, H, Lq, d), dtype=np.float64)
    s = 1.0 / np.sqrt(d) if scale is None else scale
    _load().oracle_attention_fwd(_p(Q), _p(K), _p(V), _p(mask), _p(O), B, H, Lq, Lk, d,
                                 ctypes.c_double(s))
    return O


def attention_bwd(Q, K, V, dO, mask, scale: float | None = None):
    """Derivative of the masked attention of Section 3.2 in fp64: (dQ, dK, dV) for an incoming dO."""
    Q, K, V, dO = _f32(Q), _f32(K), _f32(V), _f32(dO)
    mask = np.ascontiguousarray(np.asarray(mask, dtype=np.uint8))
    B, H, Lq, d = Q.shape
    Lk = K.shape[2]
    assert K.shape == (B, H, Lk, d) and V.shape == (B, H, Lk, d) and dO.shape == Q.shape
    assert mask.shape == (H, Lq, Lk)
    dQ = np.zeros((B, H, Lq, d), dtype=np.float64)
    dK = np.zeros((B, H, Lk, d), dtype=np.float64)
    dV = np.zeros((B, H, Lk, d), dtype=np.float64)
    s = 1.0 / np.sqrt(d) if scale is None else scale
    lib = _load()
    lib.oracle_attention_bwd.restype = None
    lib.oracle_attention_bwd(_p(Q), _p(K), _p(V), _p(dO), _p(mask), _p(dQ), _p(dK), _p(dV), B, H, Lq, Lk, d,
                             ctypes.c_double(s))
    return dQ, dK, dV


def attention_rows(Q, K, V, mask, rows, scale: float | None = None) -> np.ndarray:
    """Masked attention for sampled (b, h, i) rows only; returns float64 [len(rows), d]."""
    Q, K, V = _f32(Q), _f32(K), _f32(V)
    mask = np.ascontiguousarray(np.asarray(mask, dtype=np.uint8))
    B, H, Lq, d = Q.shape
    Lk = K.shape[2]
    rows = np.ascontiguousarray(np.asarray(rows, dtype=np.int32).reshape(-1, 3))
    out = np.zeros((rows.shape[0], d), dtype=np.float64)
    s = 1.0 / np.sqrt(d) if scale is None else scale
    _load().oracle_attention_rows(_p(Q), _p(K), _p(V), _p(mask), _p(out), _p(rows),
                                  rows.shape[0], B, H, Lq, Lk, d, ctypes.c_double(s))
    return out


def entmax15(z) -> np.ndarray:
    """1.5-entmax of a score vector (float64): p_j = max(z_j/2 - tau, 0)^2 with sum p = 1."""
    z = np.ascontiguousarray(np.asarray(z, dtype=np.float64).reshape(-1))
    assert z.size >= 1
    p = np.zeros_like(z)
    lib = _load()
    lib.oracle_entmax15.restype = None
    lib.oracle_entmax15(_p(z), int(z.size), _p(p))
    return p


def accumulate_entmax15(acc: np.ndarray, Q, K, bias=None, causal: bool = False, scale: float | None = None):
    """Eq. 1 as a running sum with the 1.5-entmax attention matrix: acc[H,Lq,Lk] (float64, in place)."""
    Q, K = _f32(Q), _f32(K)
    B, H, Lq, d = Q.shape
    Lk = K.shape[2]
    assert K.shape == (B, H, Lk, d) and acc.shape == (H, Lq, Lk)
    assert acc.dtype == np.float64 and acc.flags.c_contiguous
    _check_domain(Lq, Lk, causal)
    if bias is not None:
        bias = _f32(bias)
        assert bias.shape == (H, Lq, Lk)
    s = 1.0 / np.sqrt(d) if scale is None else scale
    lib = _load()
    lib.oracle_accumulate_entmax15.restype = None
    lib.oracle_accumulate_entmax15(
        _p(acc), _p(Q), _p(K), _p(bias) if bias is not None else None,
        B, H, Lq, Lk, d, int(bool(causal)), ctypes.c_double(s),
    )
    return acc


def accumulate_entmax15_rows(rows, Q, K, bias=None, causal: bool = False, scale: float | None = None):
    """The 1.5-entmax sum for sampled (h, i) rows only; returns float64 [len(rows), Lk]."""
    Q, K = _f32(Q), _f32(K)
    B, H, Lq, d = Q.shape
    Lk = K.shape[2]
    _check_domain(Lq, Lk, causal)
    rows = np.ascontiguousarray(np.asarray(rows, dtype=np.int32).reshape(-1, 2))
    out = np.zeros((rows.shape[0], Lk), dtype=np.float64)
    if bias is not None:
        bias = _f32(bias)
    s = 1.0 / np.sqrt(d) if scale is None else scale
    lib = _load()
    lib.oracle_accumulate_entmax15_rows.restype = None
    lib.oracle_accumulate_entmax15_rows(
        _p(out), _p(rows), rows.shape[0], _p(Q), _p(K), _p(bias) if bias is not None else None,
        B, H, Lq, Lk, d, int(bool(causal)), ctypes.c_double(s),
    )
    return out


def attention_entmax15_fwd(Q, K, V, mask, scale: float | None = None) -> np.ndarray:
    """Masked attention with the 1.5-entmax normaliser in fp64: O[B,H,Lq,d]; rows with no kept key are 0."""
    Q, K, V = _f32(Q), _f32(K), _f32(V)
    mask = np.ascontiguousarray(np.asarray(mask, dtype=np.uint8))
    B, H, Lq, d = Q.shape
    Lk = K.shape[2]
    assert K.shape == (B, H, Lk, d) and V.shape == (B, H, Lk, d) and mask.shape == (H, Lq, Lk)
    O = np.zeros((B, H, Lq, d), dtype=np.float64)
    s = 1.0 / np.sqrt(d) if scale is None else scale
    lib = _load()
    lib.oracle_attention_entmax15_fwd.restype = None
    lib.oracle_attention_entmax15_fwd(_p(Q), _p(K), _p(V), _p(mask), _p(O), B, H, Lq, Lk, d, ctypes.c_double(s))
    return O


def attention_entmax15_rows(Q, K, V, mask, rows, scale: float | None = None) -> np.ndarray:
    """The same for sampled (b, h, i) rows only; returns float64 [len(rows), d]."""
    Q, K, V = _f32(Q), _f32(K), _f32(V)
    mask = np.ascontiguousarray(np.asarray(mask, dtype=np.uint8))
    B, H, Lq, d = Q.shape
    Lk = K.shape[2]
    rows = np.ascontiguousarray(np.asarray(rows, dtype=np.int32).reshape(-1, 3))
    out = np.zeros((rows.shape[0], d), dtype=np.float64)
    s = 1.0 / np.sqrt(d) if scale is None else scale
    lib = _load()
    lib.oracle_attention_entmax15_rows.restype = None
    lib.oracle_attention_entmax15_rows(_p(Q), _p(K), _p(V), _p(mask), _p(out), _p(rows),
                                       rows.shape[0], B, H, Lq, Lk, d, ctypes.c_double(s))
    return out

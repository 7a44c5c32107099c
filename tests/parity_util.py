"""Helpers shared by the GPU parity tests: run a stage on the CUDA library and
on the oracle with the same host-generated inputs, and compare."""
import numpy as np
import torch

from oracle import ap_oracle as orc
from paper_2012_02030_b200 import inputs

# tolerances of the attention output against the fp64 oracle
# bf16 and f32: the stated bounds.  f16 (11 significant bits against bf16's 8): the output's rounding
# to half precision dominates, half an ulp is 2^-11 relative and 2^-10 absolute for |O| in [2, 4).
TOL = {"bf16": dict(max_abs=1e-2, rel_l2=5e-3), "f32": dict(max_abs=1e-5, rel_l2=1e-6),
       "f16": dict(max_abs=2e-3, rel_l2=1e-3)}


def errors(got: np.ndarray, ref: np.ndarray):
    got = got.astype(np.float64)
    diff = got - ref
    return float(np.abs(diff).max()), float(np.linalg.norm(diff.ravel()) / max(np.linalg.norm(ref.ravel()), 1e-300))


def assert_close_attention(got_t: torch.Tensor, ref: np.ndarray, dtype: str, what=""):
    max_abs, rel_l2 = errors(got_t.float().cpu().numpy(), ref)
    tol = TOL[dtype]
    assert max_abs <= tol["max_abs"] and rel_l2 <= tol["rel_l2"], (what, dtype, max_abs, rel_l2)
    return max_abs, rel_l2


def groups_from_bitmap(bitmap: np.ndarray) -> np.ndarray:
    """The tile list's group summary restated from its definition: bit g of a tile's byte is set
    iff some row keeps an entry among the tile's columns [16g, 16g+16).  bitmap: [T,128,4] uint32."""
    T = bitmap.shape[0]
    out = np.zeros(T, dtype=np.uint8)
    if T == 0:
        return out
    bits = np.unpackbits(np.ascontiguousarray(bitmap).view(np.uint8).reshape(T, 128, 16), axis=2, bitorder="little")
    any_col = bits.reshape(T, 128, 128).any(axis=1)          # [T,128]: column holds a kept entry
    any_group = any_col.reshape(T, 8, 16).any(axis=2)        # [T,8]
    for g in range(8):
        out |= (any_group[:, g].astype(np.uint8) << g).astype(np.uint8)
    return out


def rounds_from_tiles(t: dict) -> dict:
    """The forward pass's schedule restated from its definition, slot by slot, from a tile list
    (row_ptr, col_idx, flags, bitmap): the non-empty 16-column groups of a list row in list order
    are its slots, eight slots make a round."""
    row_ptr, col_idx, flags, bitmap = t["row_ptr"], t["col_idx"], t["flags"], t["bitmap"]
    T = len(col_idx)
    bits = np.unpackbits(np.ascontiguousarray(bitmap).view(np.uint8).reshape(T, 128, 16), axis=2,
                         bitorder="little").reshape(T, 128, 8, 16) if T else np.zeros((0, 128, 8, 16), np.uint8)
    round_ptr, rows, info, rbits = [0], [], [], []
    for lr in range(len(row_ptr) - 1):
        slots = []  # (first key row, [128,16] bits, tile fully kept)
        for tt in range(row_ptr[lr], row_ptr[lr + 1]):
            for g in range(8):
                if bits[tt, :, g, :].any():
                    slots.append((int(col_idx[tt]) * 128 + 16 * g, bits[tt, :, g, :], bool(flags[tt] & 1)))
        for k in range(0, len(slots), 8):
            chunk = slots[k:k + 8]
            rows.append([s[0] for s in chunk] + [-1] * (8 - len(chunk)))
            info.append(len(chunk) | (0x80 if len(chunk) == 8 and all(s[2] for s in chunk) else 0))
            b = np.zeros((128, 8, 16), np.uint8)
            for q, s in enumerate(chunk):
                b[:, q, :] = s[1]
            rbits.append(b.reshape(128, 128))
        round_ptr.append(len(rows))
    R = len(rows)
    packed = (np.packbits(np.array(rbits, dtype=np.uint8).reshape(R, 128, 128), axis=2, bitorder="little")
              .view(np.uint32).reshape(R, 128, 4) if R else np.zeros((0, 128, 4), np.uint32))
    return dict(round_ptr=np.array(round_ptr, dtype=np.int32), round_rows=np.array(rows, dtype=np.int32).reshape(R, 8),
                round_info=np.array(info, dtype=np.uint8), round_bitmap=packed)


def assert_tiles_equal(got: dict, want: dict):
    np.testing.assert_array_equal(got["row_ptr"], want["row_ptr"])
    np.testing.assert_array_equal(got["col_idx"], want["col_idx"])
    np.testing.assert_array_equal(got["flags"], want["flags"])
    np.testing.assert_array_equal(got["bitmap"], want["bitmap"])
    if "groups" in got:  # derived data: checked against its definition applied to the oracle's bitmaps
        np.testing.assert_array_equal(got["groups"], groups_from_bitmap(want["bitmap"]))
    if "round_ptr" in got:  # the schedule, likewise, against its definition applied to the oracle's list
        rounds = rounds_from_tiles(want)
        for key in ("round_ptr", "round_rows", "round_info", "round_bitmap"):
            np.testing.assert_array_equal(got[key], rounds[key], err_msg=key)


def gpu_accumulate(ap, w, n_batches, bias_dev):
    acc = torch.zeros((w.H, w.Lq, w.Lk), dtype=torch.float32, device="cuda")
    for t in range(n_batches):
        q, k = inputs.calib_qk(w, t)
        ap.ap_accumulate_attention(acc, q.cuda(), k.cuda(), bias_dev, causal=w.causal)
    return acc


def oracle_accumulate(w, n_batches, bias):
    acc64 = np.zeros((w.H, w.Lq, w.Lk))
    for t in range(n_batches):
        q, k = inputs.calib_qk(w, t)
        orc.accumulate(acc64, inputs.widen(q), inputs.widen(k), None if bias is None else bias.numpy(),
                       causal=w.causal)
    return acc64


def gpu_build_mask(ap, acc_dev, w, want_tiles=True, layer=False):
    H, Lq, Lk = acc_dev.shape
    mask = torch.full((H, Lq, Lk), 7, dtype=torch.uint8, device="cuda")  # poison: every byte must be written
    nnz = torch.full((H,), -1, dtype=torch.int64, device="cuda")
    tiles = ap.Tiles(H, Lq, Lk) if want_tiles else None
    build = ap.ap_build_mask_layer if layer else ap.ap_build_mask
    build(acc_dev, w.keep_frac, w.causal, w.keep_diag, mask, tiles, nnz)
    assert ap.ap_device_status() == ap.AP_OK
    return mask, tiles, nnz


def backward_bounds(q, k, v, d_o, mask, ulp, scale=None, tiny=0.0):
    """Element-wise absolute error bounds for dQ, dK, dV of the tensor-core backward, from a model of
    where it rounds (fp64 numpy, small shapes only).  With P the masked softmax, dP = dO V^T,
    D_i = dO_i . O_i and dS = P o (dP - D):
      * P and dS are each rounded once to the 16-bit type before they enter a product (relative ulp / 2
        each), so every term of dQ = c dS K, dK = c dS^T Q, dV = P^T dO is off by at most ulp times its
        size: the sum of the terms' absolute values bounds the effect;
      * D_i is formed from the rounded output O, an error of at most (ulp / 2) sum_c |dO_ic O_ic|, which
        enters dS_ij as P_ij dD_i and from there dQ_i (times c |K_j|) and dK_j (times c |Q_i|);
      * dV has no D in it.
    ulp = 2^-8 for bf16, 2^-11 for fp16 (one unit in the last place at 1.0); tiny = the absolute
    rounding step at the bottom of the 16-bit type's range (fp16: weights below 2^-24 vanish), 0 where
    that is out of reach (bf16 has fp32's exponent range)."""
    B, H, Lq, d = q.shape
    Lk = k.shape[2]
    c = 1.0 / np.sqrt(d) if scale is None else scale
    keep = mask.astype(bool)[None]                                   # [1, H, Lq, Lk]
    s = np.einsum("bhid,bhjd->bhij", q, k) * c
    s = np.where(keep, s, -np.inf)
    m = s.max(-1, keepdims=True)
    m = np.where(np.isfinite(m), m, 0.0)
    e = np.where(keep, np.exp(s - m), 0.0)
    den = e.sum(-1, keepdims=True)
    p = np.divide(e, den, out=np.zeros_like(e), where=den > 0)
    o = np.einsum("bhij,bhjd->bhid", p, v)
    dp = np.einsum("bhid,bhjd->bhij", d_o, v)
    dd = (d_o * o).sum(-1, keepdims=True)
    ds = p * (dp - dd)
    d_dd = 0.5 * ulp * (np.abs(d_o) * np.abs(o)).sum(-1, keepdims=True)       # [B, H, Lq, 1]
    ads = ulp * np.abs(ds) + p * d_dd + tiny * (1.0 + np.abs(dp - dd))         # per entry of dS
    b_dq = c * np.einsum("bhij,bhjd->bhid", ads, np.abs(k))
    b_dk = c * np.einsum("bhij,bhid->bhjd", ads, np.abs(q))
    b_dv = np.einsum("bhij,bhid->bhjd", ulp * p + tiny, np.abs(d_o))
    return b_dq, b_dk, b_dv

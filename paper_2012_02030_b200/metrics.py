"""Host-side counters used to report throughput (no device work)."""
from __future__ import annotations

import math

TILE = 128


def keep_count(n_valid: int, n_forced: int, keep_frac: float) -> int:
    """Entries kept per head by ap_build_mask: round-half-up of keep_frac*n_valid
    in double, clamped to [n_forced, n_valid]."""
    k = int(math.floor(keep_frac * float(n_valid) + 0.5))
    return max(n_forced, min(n_valid, k))


def attention_macs_fraction(d_model: int, N: int, p: float, credit_qk: bool = False) -> float:
    """Fraction of an attention layer's multiply-accumulates left after pruning a
    fraction p of the attention entries.

    Per token a layer costs 4d (projections) + 2N (Q.K^T and P.V) MACs; Eq. 3
    credits only the P.V product with the saving: (4d + (2-p)N) / (4d + 2N).
    ``credit_qk`` also credits a sampled Q.K^T: (4d + 2(1-p)N) / (4d + 2N).
    """
    kept = (2.0 - p) * N if not credit_qk else 2.0 * (1.0 - p) * N
    return (4.0 * d_model + kept) / (4.0 * d_model + 2.0 * N)


def effective_flops(nnz_total: int, B: int, d: int) -> float:
    """FLOPs of the masked forward counted on kept entries: 4*d per kept entry
    (2*d for q.k, 2*d for p*v), for B sequences sharing the per-head masks."""
    return 4.0 * d * float(nnz_total) * B


def tile_flops(n_tiles: int, B: int, d: int) -> float:
    """FLOPs the tensor cores execute when every listed 128x128 tile is computed densely."""
    return 4.0 * d * TILE * TILE * float(n_tiles) * B


def slot_flops(n_slots: int, B: int, d: int) -> float:
    """FLOPs the tensor cores execute for n_slots slots (one slot = 128 query rows x 16 key columns:
    2*d*128*16 for S = Q K^T and as many for O += P V), per batch element."""
    return 4.0 * d * TILE * 16.0 * float(n_slots) * B


def compulsory_bytes(B: int, H: int, Lq: int, Lk: int, d: int, elem: int) -> float:
    """One read of Q, K, V and one write of O."""
    return float(elem) * B * H * d * (2 * Lq + 2 * Lk)

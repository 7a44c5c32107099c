"""The gathered rounds (the tile list's second schedule): what the builders write, and the forward
under it, against a plain restatement of the definition and against the oracle."""
import numpy as np
import pytest
import torch

from oracle import ap_oracle as orc
from paper_2012_02030_b200 import inputs
from tests.parity_util import assert_close_attention

pytestmark = pytest.mark.gpu


def _column_order(block):
    """Active columns of a 128-row block of the mask: whole 16-column groups first, then the rest."""
    act = block.any(0)
    pad = np.zeros(-(-len(act) // 16) * 16, dtype=bool)
    pad[: len(act)] = act
    whole = np.repeat(pad.reshape(-1, 16).all(1), 16)[: len(act)]
    return np.concatenate([np.nonzero(act & whole)[0], np.nonzero(act & ~whole)[0]]), int(whole.sum()) // 16


def _check_schedule(mask, tiles, forced):
    g, r = tiles.grounds_to_host(), tiles.rounds_to_host()
    gp, rp = g["ground_ptr"], r["round_ptr"]
    m = mask.numpy().astype(bool)
    H, Lq, _ = m.shape
    n_with = 0
    for h in range(H):
        for qt in range(tiles.n_qt):
            block = m[h, qt * 128:(qt + 1) * 128]
            cols, whole = _column_order(block)
            lr = h * tiles.n_qt + qt
            n = gp[lr + 1] - gp[lr]
            want = -(-len(cols) // 128)
            if not forced:  # the builders' rule
                s = -(-(len(cols) - 16 * whole) // 16)
                want = want if 2 * (rp[lr + 1] - rp[lr]) > 4 * want + s else 0
            assert n == want, (h, qt, n, want)
            n_with += n > 0
            for k in range(n):
                cc, rho = cols[128 * k:128 * k + 128], gp[lr] + k
                keys = g["ground_keys"][rho]
                assert np.array_equal(keys[: len(cc)], cc) and np.all(keys[len(cc):] == cc[-1])
                info = int(g["ground_info"][rho])
                assert (info & 15) == -(-len(cc) // 16)
                bits = np.unpackbits(g["ground_bitmap"][rho].view(np.uint8), bitorder="little").reshape(128, 128)
                want_bits = np.zeros((128, 128), dtype=np.uint8)
                want_bits[: block.shape[0], : len(cc)] = block[:, cc]
                assert np.array_equal(bits, want_bits), (h, qt, k)
                assert bool(info & 0x80) == bool(want_bits.all())
    return n_with


def _masks(kind, H, Lq, Lk, causal):
    gen = torch.Generator().manual_seed(hash((kind, H, Lq, Lk)) % (1 << 31))
    n_qt = -(-Lq // 128)
    if kind == "random":
        return inputs.random_mask(H, Lq, Lk, 0.2, seed=9, causal=causal)
    if kind == "columns":      # single key columns shared by the rows of a query tile
        sel = torch.rand((H, n_qt, Lk), generator=gen) < 0.04
    elif kind == "groups":     # whole 16-column groups
        sel = (torch.rand((H, n_qt, -(-Lk // 16)), generator=gen) < 0.2).repeat_interleave(16, dim=2)[:, :, :Lk]
    else:                      # groups and single columns mixed, groups off the 16-column grid as well
        sel = (torch.rand((H, n_qt, -(-Lk // 16)), generator=gen) < 0.1).repeat_interleave(16, dim=2)[:, :, :Lk]
        sel = sel | torch.roll(sel, 5, dims=2) | (torch.rand((H, n_qt, Lk), generator=gen) < 0.02)
    mask = sel.repeat_interleave(128, dim=1)[:, :Lq]
    if causal:
        i = torch.arange(Lq)[:, None]
        mask = mask & (torch.arange(Lk)[None, :] <= i + (Lk - Lq))
    mask[:, :, 0] = True  # no empty rows
    return mask.to(torch.uint8)


@pytest.mark.parametrize("kind", ["random", "columns", "groups", "mixed"])
@pytest.mark.parametrize("H,Lq,Lk,d,causal", [(2, 512, 512, 128, True), (2, 300, 520, 64, False),
                                              (1, 128, 4352, 64, False), (2, 384, 1030, 128, False)])
def test_gathered_rounds_and_forward(kind, H, Lq, Lk, d, causal):
    from paper_2012_02030_b200 import binding as ap

    mask = _masks(kind, H, Lq, Lk, causal)
    tiles = ap.Tiles(H, Lq, Lk, gathered=True)
    ap.ap_debug_schedule(2)  # every list row gets its gathered rounds, whatever the rule says
    try:
        ap.ap_mask_to_tiles(mask.cuda(), tiles)
    finally:
        ap.ap_debug_schedule(0)
    assert ap.ap_device_status() == ap.AP_OK
    assert _check_schedule(mask, tiles, forced=True) > 0
    gen = torch.Generator().manual_seed(31)
    B = 2
    q = torch.randn((B, H, Lq, d), generator=gen).to(torch.bfloat16)
    k, v = (torch.randn((B, H, Lk, d), generator=gen).to(torch.bfloat16) for _ in range(2))
    ref = orc.attention_fwd(inputs.widen(q), inputs.widen(k), inputs.widen(v), mask.numpy())
    out = ap.ap_sparse_attention_fwd(q.cuda(), k.cuda(), v.cuda(), tiles)  # follows the gathered rounds
    assert ap.ap_device_status() == ap.AP_OK
    assert_close_attention(out, ref, "bf16", f"gathered rounds, {kind}")
    ap.ap_debug_schedule(1)  # the same list through the rounds
    try:
        plain = ap.ap_sparse_attention_fwd(q.cuda(), k.cuda(), v.cuda(), tiles)
    finally:
        ap.ap_debug_schedule(0)
    assert_close_attention(plain, ref, "bf16", f"rounds, {kind}")


def test_builders_rule_for_gathered_rounds():
    """Column-sparse list rows get gathered rounds, rows of whole tiles do not; a dense list has none."""
    from paper_2012_02030_b200 import binding as ap

    H, L = 2, 2048
    tiles = ap.Tiles(H, L, L, gathered=True)
    cols = _masks("columns", H, L, L, True)
    ap.ap_mask_to_tiles(cols.cuda(), tiles)
    assert _check_schedule(cols, tiles, forced=False) > 0
    band = inputs.random_mask(H, L, L, 1.0, seed=1, causal=True)
    ap.ap_mask_to_tiles(band.cuda(), tiles)
    assert _check_schedule(band, tiles, forced=False) == 0
    ap.ap_dense_tiles(tiles, causal=True)
    assert int(tiles.ground_ptr.abs().sum().item()) == 0


def test_list_without_gathered_arrays_is_unchanged():
    from paper_2012_02030_b200 import binding as ap

    H, L = 2, 512
    mask = _masks("columns", H, L, L, True)
    a, b = ap.Tiles(H, L, L), ap.Tiles(H, L, L, gathered=True)
    ap.ap_mask_to_tiles(mask.cuda(), a)
    ap.ap_mask_to_tiles(mask.cuda(), b)
    ha, hb = a.to_host(), b.to_host()
    for key in ha:
        assert np.array_equal(ha[key], hb[key]), key


@pytest.mark.parametrize("H,Lq,Lk,d,causal", [(2, 1024, 1024, 128, True), (3, 640, 900, 64, False), (1, 128, 128, 64, True)])
def test_balanced_units_table_and_forward(H, Lq, Lk, d, causal):
    """The optional table of work units: every query tile of a head exactly once, the list row with the
    most rounds paired with the one with the fewest; and the forward under it."""
    from paper_2012_02030_b200 import binding as ap

    mask = _masks("mixed", H, Lq, Lk, causal)
    tiles = ap.Tiles(H, Lq, Lk, paired=True)
    ap.ap_mask_to_tiles(mask.cuda(), tiles)
    n_qt, n_half = tiles.n_qt, (tiles.n_qt + 1) // 2
    units = tiles.unit_qt.cpu().numpy()
    rounds = np.diff(tiles.round_ptr.cpu().numpy()).reshape(H, n_qt)
    for h in range(H):
        order = sorted(range(n_qt), key=lambda qq: (-rounds[h, qq], qq))
        want = [[order[j], order[n_qt - 1 - j] if j != n_qt - 1 - j else -1] for j in range(n_half)]
        assert units[h].tolist() == want
    gen = torch.Generator().manual_seed(5)
    B = 2
    q = torch.randn((B, H, Lq, d), generator=gen).to(torch.bfloat16)
    k, v = (torch.randn((B, H, Lk, d), generator=gen).to(torch.bfloat16) for _ in range(2))
    ref = orc.attention_fwd(inputs.widen(q), inputs.widen(k), inputs.widen(v), mask.numpy())
    out = torch.full_like(q, float("nan")).cuda()
    ap.ap_sparse_attention_fwd(q.cuda(), k.cuda(), v.cuda(), tiles, out)
    assert ap.ap_device_status() == ap.AP_OK
    assert_close_attention(out, ref, "bf16", "balanced units")
    dense = ap.Tiles(H, Lq, Lk, paired=True)
    ap.ap_dense_tiles(dense, causal=causal)
    full = np.ones((H, Lq, Lk), dtype=np.uint8)
    if causal:
        full = np.tril(full, Lk - Lq)
    ref = orc.attention_fwd(inputs.widen(q), inputs.widen(k), inputs.widen(v), full)
    out.fill_(float("nan"))
    ap.ap_sparse_attention_fwd(q.cuda(), k.cuda(), v.cuda(), dense, out)
    assert_close_attention(out, ref, "bf16", "balanced units, dense list")

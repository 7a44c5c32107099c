"""Pins for the CPU oracle: it is checked against things other than itself.

Library routines (torch SDPA / softmax in fp64), closed forms, invariants, brute
force on tiny sizes and a hand-computed 4x4 example.  Chosen so that a dropped
term, a wrong sign or index, or a transposed operand in the oracle fails at
least one test.  No GPU needed.
"""
import itertools
import math
import os
from fractions import Fraction

import numpy as np
import pytest
import torch

from oracle import ap_oracle as orc
from paper_2012_02030_b200 import inputs, metrics

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "hand_4x4.txt")


def _golden():
    out = {}
    for line in open(GOLDEN):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        key, *vals = line.split()
        out[key] = np.array([float(v) for v in vals], dtype=np.float64).reshape(4, 4)
    return out


def _rand(shape, seed, dtype=torch.bfloat16):
    g = torch.Generator().manual_seed(seed)
    return torch.randn(shape, generator=g).to(dtype).to(torch.float32)


# --------------------------------------------------------------------------- forward


@pytest.mark.parametrize("causal", [False, True])
@pytest.mark.parametrize("shape", [(2, 3, 37, 37, 16), (1, 2, 130, 130, 64), (1, 1, 20, 45, 8)])
def test_fwd_all_kept_equals_library_sdpa(shape, causal):
    """Zero mask matrix (nothing pruned) gives the original attention (Section 3.2)."""
    B, H, Lq, Lk, d = shape
    if causal and Lq != Lk:
        pytest.skip("causal needs Lq == Lk")
    q, k, v = _rand((B, H, Lq, d), 1), _rand((B, H, Lk, d), 2), _rand((B, H, Lk, d), 3)
    mask = torch.ones((H, Lq, Lk), dtype=torch.uint8)
    if causal:
        mask = torch.tril(mask)
    got = orc.attention_fwd(q.numpy(), k.numpy(), v.numpy(), mask.numpy())
    ref = torch.nn.functional.scaled_dot_product_attention(
        q.double(), k.double(), v.double(), is_causal=causal)
    np.testing.assert_allclose(got, ref.numpy(), rtol=1e-12, atol=1e-13)


def test_fwd_random_mask_equals_library_masked_softmax():
    """Additive -inf mask inside a library softmax (the paper's own implementation
    route: a large negative value added before the softmax)."""
    B, H, Lq, Lk, d = 2, 2, 50, 70, 16
    q, k, v = _rand((B, H, Lq, d), 4), _rand((B, H, Lk, d), 5), _rand((B, H, Lk, d), 6)
    mask = inputs.random_mask(H, Lq, Lk, 0.3, seed=7)
    mask[:, :, 0] = 1  # no empty rows here
    s = torch.einsum("bhid,bhjd->bhij", q.double(), k.double()) / math.sqrt(d)
    s = s.masked_fill(mask.bool().unsqueeze(0) == 0, float("-inf"))
    ref = torch.softmax(s, dim=-1) @ v.double()
    got = orc.attention_fwd(q.numpy(), k.numpy(), v.numpy(), mask.numpy())
    np.testing.assert_allclose(got, ref.numpy(), rtol=1e-12, atol=1e-13)


def test_fwd_custom_scale_and_rows_sampler():
    B, H, L, d = 2, 2, 33, 8
    q, k, v = _rand((B, H, L, d), 8), _rand((B, H, L, d), 9), _rand((B, H, L, d), 10)
    mask = inputs.random_mask(H, L, L, 0.5, seed=11)
    full = orc.attention_fwd(q.numpy(), k.numpy(), v.numpy(), mask.numpy(), scale=0.37)
    s = torch.einsum("bhid,bhjd->bhij", q.double(), k.double()) * 0.37
    s = s.masked_fill(mask.bool().unsqueeze(0) == 0, float("-inf"))
    ref = torch.nan_to_num(torch.softmax(s, dim=-1), nan=0.0) @ v.double()
    np.testing.assert_allclose(full, ref.numpy(), rtol=1e-12, atol=1e-13)
    rows = [(b, h, i) for b in range(B) for h in range(H) for i in (0, 5, 32)]
    some = orc.attention_rows(q.numpy(), k.numpy(), v.numpy(), mask.numpy(), rows, scale=0.37)
    for r, (b, h, i) in enumerate(rows):
        np.testing.assert_array_equal(some[r], full[b, h, i])


def test_fwd_one_kept_entry_copies_value_row():
    B, H, L, d = 2, 2, 19, 8
    q, k, v = _rand((B, H, L, d), 12), _rand((B, H, L, d), 13), _rand((B, H, L, d), 14)
    g = torch.Generator().manual_seed(15)
    cols = torch.randint(0, L, (H, L), generator=g)
    mask = torch.zeros((H, L, L), dtype=torch.uint8)
    mask.scatter_(2, cols.unsqueeze(-1), 1)
    got = orc.attention_fwd(q.numpy(), k.numpy(), v.numpy(), mask.numpy())
    for h in range(H):
        for i in range(L):
            np.testing.assert_array_equal(got[:, h, i], v[:, h, cols[h, i]].double().numpy())
    eye = torch.eye(L, dtype=torch.uint8).expand(H, L, L)
    got = orc.attention_fwd(q.numpy(), k.numpy(), v.numpy(), eye.numpy())
    np.testing.assert_array_equal(got, v.double().numpy())


def test_fwd_zero_queries_give_plain_mean_and_empty_rows_zero():
    B, H, L, d = 1, 2, 23, 8
    k, v = _rand((B, H, L, d), 16), _rand((B, H, L, d), 17)
    q = torch.zeros((B, H, L, d))
    mask = inputs.random_mask(H, L, L, 0.4, seed=18, empty_rows=(3, 22))
    got = orc.attention_fwd(q.numpy(), k.numpy(), v.numpy(), mask.numpy())
    m = mask.double()
    cnt = m.sum(-1, keepdim=True)
    ref = (m.unsqueeze(0) @ v.double()) / cnt.clamp(min=1)
    np.testing.assert_allclose(got, ref.numpy(), rtol=1e-13, atol=1e-14)
    assert np.all(got[:, :, 3] == 0.0) and np.all(got[:, :, 22] == 0.0)


def test_fwd_key_shift_and_permutation_invariance():
    B, H, L, d = 1, 2, 29, 8
    q, k, v = _rand((B, H, L, d), 19), _rand((B, H, L, d), 20), _rand((B, H, L, d), 21)
    mask = inputs.random_mask(H, L, L, 0.5, seed=22)
    base = orc.attention_fwd(q.numpy(), k.numpy(), v.numpy(), mask.numpy())
    shift = torch.tensor([1.0, -2.0, 0.5, 0.25, -1.0, 2.0, 4.0, -0.5])  # exact in fp32
    got = orc.attention_fwd(q.numpy(), (k + shift).numpy(), v.numpy(), mask.numpy())
    np.testing.assert_allclose(got, base, rtol=1e-10, atol=1e-12)
    perm = torch.randperm(L, generator=torch.Generator().manual_seed(23))
    got = orc.attention_fwd(q.numpy(), k[:, :, perm].numpy(), v[:, :, perm].numpy(),
                            mask[:, :, perm].numpy())
    np.testing.assert_allclose(got, base, rtol=1e-12, atol=1e-13)


def test_fwd_weights_sum_to_one_over_kept_entries():
    """With V = identity the output is the weight matrix itself."""
    H, L = 2, 24
    q, k = _rand((1, H, L, L), 24), _rand((1, H, L, L), 25)
    v = torch.eye(L).expand(1, H, L, L).contiguous()
    mask = inputs.random_mask(H, L, L, 0.3, seed=26, empty_rows=(7,))
    w = orc.attention_fwd(q.numpy(), k.numpy(), v.numpy(), mask.numpy())[0]
    assert np.all(w[mask.numpy() == 0] == 0.0)
    sums = w.sum(-1)
    has = mask.numpy().sum(-1) > 0
    np.testing.assert_allclose(sums[has], 1.0, rtol=0, atol=1e-14)
    assert np.all(sums[~has] == 0.0)
    assert np.all(w >= 0)


# ------------------------------------------------------------------------ accumulate


@pytest.mark.parametrize("causal", [False, True])
@pytest.mark.parametrize("with_bias", [False, True])
def test_acc_equals_library_softmax_sum(causal, with_bias):
    B, H, L, d = 3, 2, 41, 16
    q, k = _rand((B, H, L, d), 30), _rand((B, H, L, d), 31)
    bias = _rand((H, L, L), 32, torch.float32) if with_bias else None
    acc = np.zeros((H, L, L))
    orc.accumulate(acc, q.numpy(), k.numpy(), None if bias is None else bias.numpy(), causal=causal)
    s = torch.einsum("bhid,bhjd->bhij", q.double(), k.double()) / math.sqrt(d)
    if with_bias:
        s = s + bias.double()
    if causal:
        s = s.masked_fill(~torch.tril(torch.ones(L, L, dtype=torch.bool)), float("-inf"))
    ref = torch.softmax(s, dim=-1).sum(0)
    np.testing.assert_allclose(acc, ref.numpy(), rtol=1e-12, atol=1e-14)
    if causal:
        assert np.all(acc[:, ~np.tril(np.ones((L, L), dtype=bool))] == 0.0)
    # calling again continues the running sum (Eq. 1 is a plain sum over samples)
    orc.accumulate(acc, q.numpy(), k.numpy(), None if bias is None else bias.numpy(), causal=causal)
    np.testing.assert_allclose(acc, 2 * ref.numpy(), rtol=1e-12, atol=1e-14)


def test_acc_rows_sum_to_sample_count_and_rect_shapes():
    B, H, Lq, Lk, d = 5, 2, 17, 33, 8
    q, k = _rand((B, H, Lq, d), 33), _rand((B, H, Lk, d), 34)
    acc = np.zeros((H, Lq, Lk))
    orc.accumulate(acc, q.numpy(), k.numpy())
    np.testing.assert_allclose(acc.sum(-1), B, rtol=1e-13)
    s = torch.einsum("bhid,bhjd->bhij", q.double(), k.double()) / math.sqrt(d)
    np.testing.assert_allclose(acc, torch.softmax(s, -1).sum(0).numpy(), rtol=1e-12, atol=1e-14)
    rows = [(0, 0), (1, 16), (1, 3)]
    got = orc.accumulate_rows(rows, q.numpy(), k.numpy())
    for r, (h, i) in enumerate(rows):
        np.testing.assert_array_equal(got[r], acc[h, i])


@pytest.mark.parametrize("with_bias", [False, True])
def test_acc_causal_with_memory_keys_equals_library_softmax_sum(with_bias):
    """Lk = mem + Lq: query i attends to keys 0 .. mem + i (a library softmax over an additive
    -inf mask with the diagonal shifted by mem); entries outside stay untouched."""
    B, H, Lq, mem, d = 3, 2, 23, 18, 16
    Lk = mem + Lq
    q, k = _rand((B, H, Lq, d), 36), _rand((B, H, Lk, d), 37)
    bias = _rand((H, Lq, Lk), 38, torch.float32) if with_bias else None
    acc = np.zeros((H, Lq, Lk))
    orc.accumulate(acc, q.numpy(), k.numpy(), None if bias is None else bias.numpy(), causal=True)
    s = torch.einsum("bhid,bhjd->bhij", q.double(), k.double()) / math.sqrt(d)
    if with_bias:
        s = s + bias.double()
    dom = torch.tril(torch.ones(Lq, Lk, dtype=torch.bool), diagonal=mem)
    ref = torch.softmax(s.masked_fill(~dom, float("-inf")), dim=-1).sum(0)
    np.testing.assert_allclose(acc, ref.numpy(), rtol=1e-12, atol=1e-14)
    assert np.all(acc[:, ~dom.numpy()] == 0.0)
    np.testing.assert_allclose(acc.sum(-1), B, rtol=1e-13)
    rows = [(0, 0), (1, Lq - 1), (1, 7)]
    got = orc.accumulate_rows(rows, q.numpy(), k.numpy(), None if bias is None else bias.numpy(), causal=True)
    for r, (h, i) in enumerate(rows):
        np.testing.assert_array_equal(got[r], acc[h, i])
    with pytest.raises(ValueError):
        orc.accumulate(np.zeros((H, Lk, Lq)), k.numpy(), q.numpy(), causal=True)


def test_acc_zero_queries_closed_form():
    B, H, L, d = 4, 1, 12, 8
    k = _rand((B, H, L, d), 35)
    q = torch.zeros((B, H, L, d))
    acc = np.zeros((H, L, L))
    orc.accumulate(acc, q.numpy(), k.numpy())
    np.testing.assert_allclose(acc, B / L, rtol=1e-15)
    acc = np.zeros((H, L, L))
    orc.accumulate(acc, q.numpy(), k.numpy(), causal=True)
    for i in range(L):
        np.testing.assert_allclose(acc[0, i, : i + 1], B / (i + 1), rtol=1e-15)
        assert np.all(acc[0, i, i + 1:] == 0.0)


# ------------------------------------------------------------------------- build mask


def _domain(Lq, Lk, causal):
    """All (i, j), or under the causal constraint those with j <= i + (Lk - Lq): Lk - Lq memory
    keys that every query sees, then the current segment under its autoregressive mask."""
    return [(i, j) for i in range(Lq) for j in range(Lk) if (not causal or j <= i + (Lk - Lq))]


def _forced(dom, Lq, Lk, causal, keep_diag):
    """Each query's own position, when asked for and defined (square, or causal with memory)."""
    return [(i, j) for (i, j) in dom if keep_diag and (Lq == Lk or causal) and j == i + (Lk - Lq)]


def _brute_force_mask(acc, keep_frac, causal, keep_diag):
    """Among all k-subsets of the domain that contain the forced entries, the one
    with the largest exact sum; among those, the first in index order."""
    Lq, Lk = acc.shape
    dom = _domain(Lq, Lk, causal)
    forced = _forced(dom, Lq, Lk, causal, keep_diag)
    n_valid = len(dom)
    k = max(len(forced), min(n_valid, int(math.floor(keep_frac * n_valid + 0.5))))
    free = [e for e in dom if e not in forced]
    best, best_key = None, None
    for combo in itertools.combinations(free, k - len(forced)):
        chosen = sorted(forced + list(combo), key=lambda e: e[0] * Lk + e[1])
        total = sum(Fraction(float(acc[i, j])) for (i, j) in chosen)
        key = (-total, tuple(i * Lk + j for (i, j) in chosen))
        if best_key is None or key < best_key:
            best, best_key = chosen, key
    mask = np.zeros((Lq, Lk), dtype=np.uint8)
    for (i, j) in best:
        mask[i, j] = 1
    return mask, k


@pytest.mark.parametrize("causal", [False, True])
@pytest.mark.parametrize("keep_diag", [False, True])
def test_mask_brute_force_tiny(causal, keep_diag):
    rng = np.random.default_rng(40)
    for L in (2, 3, 4):
        for keep in (0.2, 0.5, 0.75):
            for trial in range(6):
                # few distinct values => many exact ties, which exercise the index rule
                acc = rng.integers(0, 4, size=(1, L, L)).astype(np.float32) / 4.0
                want, k = _brute_force_mask(acc[0], keep, causal, keep_diag)
                got, nnz = orc.build_mask(acc, keep, causal=causal, keep_diag=keep_diag)
                assert nnz[0] == k
                np.testing.assert_array_equal(got[0], want)


def test_mask_brute_force_rectangular():
    rng = np.random.default_rng(41)
    for (Lq, Lk) in ((2, 4), (3, 2), (4, 3)):
        acc = rng.integers(0, 3, size=(1, Lq, Lk)).astype(np.float32)
        want, k = _brute_force_mask(acc[0], 0.5, False, True)  # keep_diag ignored: Lq != Lk
        got, nnz = orc.build_mask(acc, 0.5, causal=False, keep_diag=True)
        assert nnz[0] == k
        np.testing.assert_array_equal(got[0], want)


@pytest.mark.parametrize("keep_diag", [False, True])
def test_mask_brute_force_causal_with_memory_keys(keep_diag):
    """Lk = mem + Lq: the memory keys are visible to every query, the current segment is causal
    (the Transformer-XL masks of the language-modelling section); the forced entry of query i is
    its own position mem + i."""
    rng = np.random.default_rng(47)
    for (Lq, Lk) in ((2, 3), (2, 5), (3, 4), (3, 5)):
        for keep in (0.3, 0.6):
            for trial in range(4):
                acc = rng.integers(0, 4, size=(1, Lq, Lk)).astype(np.float32) / 4.0
                want, k = _brute_force_mask(acc[0], keep, True, keep_diag)
                got, nnz = orc.build_mask(acc, keep, causal=True, keep_diag=keep_diag)
                assert nnz[0] == k
                np.testing.assert_array_equal(got[0], want)
                if keep_diag:
                    assert all(got[0, i, Lk - Lq + i] == 1 for i in range(Lq))
                assert not got[0][~np.tril(np.ones((Lq, Lk), dtype=bool), Lk - Lq)].any()
    with pytest.raises(ValueError):
        orc.build_mask(np.zeros((1, 3, 2), dtype=np.float32), 0.5, causal=True)


def test_mask_causal_with_memory_equals_last_rows_of_the_square_problem():
    """The domain of (Lq, mem + Lq) is the last Lq rows of the square causal domain of size
    mem + Lq.  With the upper rows of the square problem far below every other value they are the
    last to be kept, so with a count chosen accordingly the square problem's mask restricted to
    the last rows is the rectangular problem's mask."""
    rng = np.random.default_rng(48)
    Lq, mem = 29, 35
    Lk = mem + Lq
    rect = rng.random((2, Lq, Lk), dtype=np.float32)
    rect[1] = np.round(rect[1] * 6) / 6                    # ties
    square = np.full((2, Lk, Lk), -1.0, dtype=np.float32)
    square[:, mem:, :] = rect
    n_rect = Lq * (Lq + 1) // 2 + Lq * mem
    n_square = Lk * (Lk + 1) // 2
    k = 300
    got, nnz = orc.build_mask(rect, k / n_rect, causal=True, keep_diag=False)
    want, _ = orc.build_mask(square, k / n_square, causal=True, keep_diag=False)
    assert nnz.tolist() == [k, k]
    np.testing.assert_array_equal(got, want[:, mem:, :])
    assert not want[:, :mem, :].any()


@pytest.mark.parametrize("causal", [False, True])
def test_mask_invariants(causal):
    rng = np.random.default_rng(42)
    H, L = 3, 67
    acc = rng.random((H, L, L), dtype=np.float32)
    acc[0].flat[::3] = 0.5  # plant ties
    dom = np.tril(np.ones((L, L), dtype=bool)) if causal else np.ones((L, L), dtype=bool)
    n_valid = int(dom.sum())
    prev = None
    for keep in (0.05, 0.1, 0.33, 0.5, 0.9, 1.0):
        mask, nnz = orc.build_mask(acc, keep, causal=causal, keep_diag=True)
        k = max(L, min(n_valid, int(math.floor(keep * n_valid + 0.5))))
        assert metrics.keep_count(n_valid, L, keep) == k == orc.keep_count(n_valid, L, keep)
        for h in range(H):
            m = mask[h].astype(bool)
            assert nnz[h] == k and m.sum() == k          # kept fraction exact
            assert not m[~dom].any()                     # never outside the domain
            assert m[np.arange(L), np.arange(L)].all()   # diagonal forced
            off = ~np.eye(L, dtype=bool)
            kept_free, pruned = acc[h][m & off], acc[h][~m & dom]
            if kept_free.size and pruned.size:
                assert kept_free.min() >= pruned.max()
        if prev is not None:
            assert np.all(prev <= mask)                  # nesting
        prev = mask
    np.testing.assert_array_equal(prev, np.broadcast_to(dom, (H, L, L)).astype(np.uint8))


# --- the per-layer threshold (one selection over all heads, as Eq. 2 is stated in the paper)


def _brute_force_layer(acc, keep_frac, causal, keep_diag):
    """Among all k-subsets of the union of the heads' domains that contain every head's forced
    entries, the one with the largest exact sum; among those, the first in global index order."""
    H, Lq, Lk = acc.shape
    dom = [(h, i, j) for h in range(H) for (i, j) in _domain(Lq, Lk, causal)]
    forced = [e for e in dom if keep_diag and (Lq == Lk or causal) and e[2] == e[1] + (Lk - Lq)]
    N = len(dom)
    k = max(len(forced), min(N, int(math.floor(keep_frac * N + 0.5))))
    free = [e for e in dom if e not in forced]
    gidx = lambda e: (e[0] * Lq + e[1]) * Lk + e[2]
    best, best_key = None, None
    for combo in itertools.combinations(free, k - len(forced)):
        chosen = sorted(forced + list(combo), key=gidx)
        total = sum(Fraction(float(acc[e])) for e in chosen)
        key = (-total, tuple(gidx(e) for e in chosen))
        if best_key is None or key < best_key:
            best, best_key = chosen, key
    mask = np.zeros((H, Lq, Lk), dtype=np.uint8)
    for e in best:
        mask[e] = 1
    return mask, k


@pytest.mark.parametrize("causal", [False, True])
@pytest.mark.parametrize("keep_diag", [False, True])
def test_layer_mask_brute_force_tiny(causal, keep_diag):
    rng = np.random.default_rng(44)
    for (H, L) in ((2, 2), (3, 2), (2, 3)):
        for keep in (0.25, 0.5, 0.7):
            for trial in range(4):
                acc = rng.integers(0, 4, size=(H, L, L)).astype(np.float32) / 4.0  # many exact ties
                want, k = _brute_force_layer(acc, keep, causal, keep_diag)
                got, nnz = orc.build_mask_layer(acc, keep, causal=causal, keep_diag=keep_diag)
                np.testing.assert_array_equal(got, want)
                assert nnz.sum() == k and list(nnz) == [int(want[h].sum()) for h in range(H)]


def test_layer_mask_is_the_per_head_selection_of_the_stacked_heads():
    """Without causal or diagonal structure, one threshold over H heads of [Lq, Lk] is the per-head
    rule applied to a single head of [H*Lq, Lk] (same population, same index order); with one
    head the two rules coincide whatever the structure."""
    rng = np.random.default_rng(45)
    H, Lq, Lk = 3, 17, 23
    acc = rng.random((H, Lq, Lk), dtype=np.float32)
    acc.flat[::5] = 0.25  # ties
    for keep in (0.1, 0.5, 0.93):
        got, nnz = orc.build_mask_layer(acc, keep, causal=False, keep_diag=False)
        want, k = orc.build_mask(acc.reshape(1, H * Lq, Lk), keep, causal=False, keep_diag=False)
        np.testing.assert_array_equal(got.reshape(1, H * Lq, Lk), want)
        assert nnz.sum() == k[0]
    one = rng.random((1, 19, 19), dtype=np.float32)
    for causal in (False, True):
        a, na = orc.build_mask_layer(one, 0.3, causal=causal, keep_diag=True)
        b, nb = orc.build_mask(one, 0.3, causal=causal, keep_diag=True)
        np.testing.assert_array_equal(a, b)
        assert list(na) == list(nb)


@pytest.mark.parametrize("causal", [False, True])
def test_layer_mask_invariants(causal):
    rng = np.random.default_rng(46)
    H, L = 4, 41
    acc = rng.random((H, L, L), dtype=np.float32) * np.array([1.0, 2.0, 0.5, 1.5], dtype=np.float32)[:, None, None]
    dom = np.tril(np.ones((L, L), dtype=bool)) if causal else np.ones((L, L), dtype=bool)
    N = int(dom.sum()) * H
    off = ~np.eye(L, dtype=bool)
    prev = None
    for keep in (0.05, 0.2, 0.5, 0.9, 1.0):
        mask, nnz = orc.build_mask_layer(acc, keep, causal=causal, keep_diag=True)
        k = max(H * L, min(N, int(math.floor(keep * N + 0.5))))
        m = mask.astype(bool)
        assert m.sum() == k == nnz.sum()                      # the kept fraction of the LAYER is exact
        assert [int(m[h].sum()) for h in range(H)] == list(nnz)
        assert not m[:, ~dom].any()                           # never outside the domain
        assert m[:, np.arange(L), np.arange(L)].all()         # every head's diagonal forced
        kept_free, pruned = acc[m & off[None]], acc[~m & dom[None]]
        if kept_free.size and pruned.size:
            assert kept_free.min() >= pruned.max()            # one threshold across all heads
        if keep < 1.0:
            assert nnz[1] > nnz[2]                            # the head with larger values keeps more
        if prev is not None:
            assert np.all(prev <= mask)
        prev = mask


def test_mask_constant_acc_keeps_forced_then_first_indices():
    L = 6
    acc = np.full((1, L, L), 0.125, dtype=np.float32)
    mask, nnz = orc.build_mask(acc, 0.5, causal=False, keep_diag=True)
    want = np.eye(L, dtype=np.uint8)
    need = 18 - L
    for idx in range(L * L):
        i, j = divmod(idx, L)
        if need and i != j:
            want[i, j] = 1
            need -= 1
    np.testing.assert_array_equal(mask[0], want)
    assert nnz[0] == 18


def test_mask_k_smaller_than_forced_keeps_diagonal_only():
    rng = np.random.default_rng(43)
    acc = rng.random((2, 9, 9), dtype=np.float32)
    mask, nnz = orc.build_mask(acc, 0.01, causal=False, keep_diag=True)
    np.testing.assert_array_equal(mask, np.broadcast_to(np.eye(9, dtype=np.uint8), (2, 9, 9)))
    assert list(nnz) == [9, 9]


def test_mask_in_domain_zero_beats_nothing_outside_domain():
    """Causal domain is by index, not by value: in-domain zeros can be kept, out-of-domain never."""
    L = 4
    acc = np.zeros((1, L, L), dtype=np.float32)
    acc[0, 0, 3] = 9.0  # outside the causal domain
    mask, nnz = orc.build_mask(acc, 1.0, causal=True, keep_diag=True)
    np.testing.assert_array_equal(mask[0], np.tril(np.ones((L, L), dtype=np.uint8)))


def test_rounding_of_k_matches_the_workloads():
    want = {"tiny": 1638, "bert": 8192, "lm": 13133, "s2s_self": 16448, "s2s_cross": 32768,
            "long": 419533, "txl": 22138, "llama": 419533}  # txl: 0.1 * (384*385/2 + 384*384) = 22137.6
    for name, w in inputs.WORKLOADS.items():
        assert orc.keep_count(w.n_valid, w.n_forced, w.keep_frac) == want[name]
        assert metrics.keep_count(w.n_valid, w.n_forced, w.keep_frac) == want[name]


# ------------------------------------------------------------------------------ tiles


def _numpy_tiles(mask):
    """Independent re-statement with numpy.packbits (LSB-first)."""
    H, Lq, Lk = mask.shape
    n_qt, n_kt = -(-Lq // 128), -(-Lk // 128)
    pad = np.zeros((H, n_qt * 128, n_kt * 128), dtype=np.uint8)
    pad[:, :Lq, :Lk] = mask
    row_ptr, col_idx, flags, bitmaps = [0], [], [], []
    for h in range(H):
        for qt in range(n_qt):
            for kt in range(n_kt):
                t = pad[h, qt * 128:(qt + 1) * 128, kt * 128:(kt + 1) * 128]
                if t.any():
                    col_idx.append(kt)
                    flags.append(1 if t.all() else 0)
                    bitmaps.append(np.packbits(t, axis=1, bitorder="little").view("<u4"))
            row_ptr.append(len(col_idx))
    return np.array(row_ptr), np.array(col_idx), np.array(flags), np.array(bitmaps).reshape(-1, 128, 4)


@pytest.mark.parametrize("shape", [(2, 128, 128), (2, 300, 200), (1, 130, 515), (3, 5, 7)])
def test_tiles_roundtrip_and_structure(shape):
    H, Lq, Lk = shape
    mask = inputs.random_mask(H, Lq, Lk, 0.02, seed=50).numpy()
    mask[0, : min(128, Lq), : min(128, Lk)] = 1         # a full (or edge-full) tile
    if Lk > 256:
        mask[:, :, 128:256] = 0                          # an empty tile column
    t = orc.mask_to_tiles(mask)
    rp, ci, fl, bm = _numpy_tiles(mask)
    np.testing.assert_array_equal(t["row_ptr"], rp)
    np.testing.assert_array_equal(t["col_idx"], ci)
    np.testing.assert_array_equal(t["flags"], fl)
    np.testing.assert_array_equal(t["bitmap"], bm)
    # structure
    assert t["row_ptr"][0] == 0 and np.all(np.diff(t["row_ptr"]) >= 0)
    n_qt = t["n_qt"]
    back = np.zeros_like(mask)
    pop = 0
    for row in range(H * n_qt):
        cols = t["col_idx"][t["row_ptr"][row]:t["row_ptr"][row + 1]]
        assert np.all(np.diff(cols) > 0)
        h, qt = divmod(row, n_qt)
        for s in range(t["row_ptr"][row], t["row_ptr"][row + 1]):
            bits = np.unpackbits(t["bitmap"][s].view(np.uint8), axis=1, bitorder="little")
            c = int(bits.sum())
            assert c > 0 and (t["flags"][s] == 1) == (c == 128 * 128)
            pop += c
            kt = t["col_idx"][s]
            r1, c1 = min(128, Lq - qt * 128), min(128, Lk - kt * 128)
            assert bits[r1:].sum() == 0 and bits[:, c1:].sum() == 0
            back[h, qt * 128:qt * 128 + r1, kt * 128:kt * 128 + c1] = bits[:r1, :c1]
    np.testing.assert_array_equal(back, mask)
    assert pop == int(mask.sum())


# ------------------------------------------------------------------------ hand example


def test_hand_example_4x4():
    g = _golden()
    e = math.e
    a, b, D2 = e / (2 * e + 2), 1 / (2 * e + 2), 2 * e + e * e + 1
    dense = np.array([[a, b, a, b], [b, a, a, b], [e / D2, e / D2, e * e / D2, 1 / D2], [.25] * 4])
    c2 = 2 * e + e * e
    causal = np.array([[1, 0, 0, 0], [1 / (1 + e), e / (1 + e), 0, 0],
                       [e / c2, e / c2, e * e / c2, 0], [.25] * 4])
    np.testing.assert_allclose(g["dense_attention"], dense, atol=5e-7)
    np.testing.assert_allclose(g["causal_attention"], causal, atol=5e-7)
    Q, K, V = (g[x].astype(np.float32).reshape(1, 1, 4, 4) for x in "QKV")
    np.testing.assert_array_equal((Q[0, 0] @ K[0, 0].T) / 2, g["logits"])

    for is_causal, want in ((False, dense), (True, causal)):
        acc = np.zeros((1, 4, 4))
        orc.accumulate(acc, Q, K, causal=is_causal)
        np.testing.assert_allclose(acc[0], want, rtol=1e-14, atol=1e-16)
        dom = np.tril(np.ones((4, 4), np.uint8)) if is_causal else np.ones((4, 4), np.uint8)
        O = orc.attention_fwd(Q, K, V, dom.reshape(1, 4, 4))
        np.testing.assert_allclose(O[0, 0], want, rtol=1e-14, atol=1e-16)

        key = "causal" if is_causal else "noncausal"
        mask, nnz = orc.build_mask(acc.astype(np.float32), 0.5, causal=is_causal, keep_diag=True)
        np.testing.assert_array_equal(mask[0], g[f"mask_{key}_keep50"].astype(np.uint8))
        assert nnz[0] == (5 if is_causal else 8)
        O = orc.attention_fwd(Q, K, V, mask)
        np.testing.assert_allclose(O[0, 0], g[f"out_{key}_keep50"], atol=5e-7)

    third = 1.0 / 3.0
    mask = g["mask_noncausal_keep50"].astype(np.uint8).reshape(1, 4, 4)
    O = orc.attention_fwd(Q, K, V, mask)
    exact = np.array([[.5, 0, .5, 0], [0, .5, .5, 0], [0, 0, 1, 0], [third, third, 0, third]])
    np.testing.assert_allclose(O[0, 0], exact, rtol=1e-15, atol=0)
    mask[0, 2, :] = 0
    O = orc.attention_fwd(Q, K, V, mask)
    assert np.all(O[0, 0, 2] == 0.0)
    np.testing.assert_allclose(O[0, 0, [0, 1, 3]], exact[[0, 1, 3]], rtol=1e-15, atol=0)


# ------------------------------------------------------------------- MAC model (Eq. 3)


def test_mac_fraction_closed_form():
    """Eq. 3 and its derivation: per token 3d + d projection MACs (per unit of d)
    and N + N attention MACs, of which a fraction p of the P.V product is saved."""
    for d, N, p in ((768, 384, 0.9), (512, 128, 0.5), (4096, 4096, 0.6)):
        B = 3
        proj, qk, pv, outp = 3 * B * N * d * d, B * N * N * d, B * N * N * d, B * N * d * d
        frac = (proj + qk + (1 - p) * pv + outp) / (proj + qk + pv + outp)
        assert metrics.attention_macs_fraction(d, N, p) == pytest.approx(frac, rel=1e-14)
        frac2 = (proj + (1 - p) * (qk + pv) + outp) / (proj + qk + pv + outp)
        assert metrics.attention_macs_fraction(d, N, p, credit_qk=True) == pytest.approx(frac2, rel=1e-14)
    assert metrics.attention_macs_fraction(768, 384, 0.9) == pytest.approx(3494.4 / 3840)
    assert metrics.effective_flops(10, 2, 64) == 4 * 64 * 10 * 2
    assert metrics.tile_flops(3, 2, 64) == 4 * 64 * 128 * 128 * 3 * 2


# --------------------------------------------------------------- random-pruning control


def test_random_scores_follow_the_published_generator_outputs():
    """Score n is the top 24 bits of SplitMix64 output n + 1: checked against the generator's
    published first outputs (tests/golden/splitmix64.txt)."""
    path = os.path.join(os.path.dirname(__file__), "golden", "splitmix64.txt")
    for line in open(path):
        if line.startswith("#") or not line.strip():
            continue
        seed, *outs = [int(t) for t in line.split()]
        got = orc.random_scores(1, 1, len(outs), seed)[0, 0]
        want = np.array([(z >> 40) / 16777216.0 for z in outs], dtype=np.float32)
        np.testing.assert_array_equal(got, want)
        # the value of entry n does not depend on the shape it is asked in
        np.testing.assert_array_equal(orc.random_scores(len(outs), 1, 1, seed).ravel(), want)


def test_random_scores_are_uniform_and_give_a_mask_of_the_exact_count():
    H, L = 2, 256
    u = orc.random_scores(H, L, L, seed=99)
    assert u.min() >= 0.0 and u.max() < 1.0
    assert abs(u.mean() - 0.5) < 4 * (1 / 12 / u.size) ** 0.5
    assert abs(u.var() - 1 / 12) < 2e-3
    hist = np.histogram(u, bins=64, range=(0, 1))[0]
    expect = u.size / 64
    assert ((hist - expect) ** 2 / expect).sum() < 64 + 5 * (2 * 64) ** 0.5      # chi-square, 63 d.o.f.
    assert abs(np.corrcoef(u.ravel()[:-1], u.ravel()[1:])[0, 1]) < 0.01          # neighbours uncorrelated
    assert not np.array_equal(u, orc.random_scores(H, L, L, seed=100))
    # pruning random entries = Eq. 2's selection applied to the scores: same count as a tailored mask
    mask, nnz = orc.build_mask(u, 0.2, causal=True, keep_diag=True)
    k = orc.keep_count(L * (L + 1) // 2, L, 0.2)
    assert nnz.tolist() == [k, k] and mask[:, np.arange(L), np.arange(L)].all()
    rows = mask[0].sum(1) / (np.arange(L) + 1)                                    # kept share per row
    assert abs(rows[64:].mean() - 0.2) < 0.02                                     # spread evenly over rows


# ------------------------------------------------------------- block-structured pruning


@pytest.mark.parametrize("block", [4, 16])
def test_pool_scores_equal_a_reshaped_mean_and_expansion_equals_a_kronecker_product(block):
    """Away from the causal boundary the block mean is a reshape + mean, and the expansion of a
    block mask is its Kronecker product with a block of ones (library routines)."""
    rng = np.random.default_rng(60)
    H, R, C = 2, 5, 7
    acc = rng.random((H, R * block, C * block), dtype=np.float32)
    got = orc.pool_scores(acc, block)
    want = acc.astype(np.float64).reshape(H, R, block, C, block).mean(axis=(2, 4))
    np.testing.assert_allclose(got, want, rtol=1e-14)
    bm = (rng.random((H, R, C)) < 0.4).astype(np.uint8)
    np.testing.assert_array_equal(orc.expand_block_mask(bm, block), np.kron(bm, np.ones((block, block), dtype=np.uint8)))


@pytest.mark.parametrize("mem_blocks", [0, 2])
def test_pool_scores_and_expansion_respect_the_causal_domain(mem_blocks):
    rng = np.random.default_rng(61)
    H, R, block = 2, 6, 8
    Lq, Lk = R * block, (R + mem_blocks) * block
    acc = rng.random((H, Lq, Lk), dtype=np.float32)
    dom = np.tril(np.ones((Lq, Lk), dtype=bool), Lk - Lq)
    got = orc.pool_scores(acc, block, causal=True)
    a = np.where(dom, acc.astype(np.float64), 0.0).reshape(H, R, block, R + mem_blocks, block).sum(axis=(2, 4))
    n = dom.reshape(R, block, R + mem_blocks, block).sum(axis=(1, 3))
    np.testing.assert_allclose(got, np.where(n > 0, a / np.maximum(n, 1), 0.0), rtol=1e-14)
    assert n[0, mem_blocks] == block * (block + 1) // 2          # a diagonal block holds a triangle
    assert np.all(got[:, n == 0] == 0.0)
    bm = np.ones((H, R, R + mem_blocks), dtype=np.uint8)
    np.testing.assert_array_equal(orc.expand_block_mask(bm, block, causal=True), np.broadcast_to(dom, (H, Lq, Lk)))
    # the whole route: pooled scores -> Eq. 2 over blocks -> element mask made of whole blocks
    bmask, nnz = orc.build_mask(got.astype(np.float32), 0.5, causal=True, keep_diag=True)
    mask = orc.expand_block_mask(bmask, block, causal=True)
    n_blocks = R * (R + 1) // 2 + R * mem_blocks
    assert nnz.tolist() == [orc.keep_count(n_blocks, R, 0.5)] * H
    for h in range(H):
        blocks = mask[h].reshape(R, block, R + mem_blocks, block).sum(axis=(1, 3))
        assert np.all((blocks == 0) | (blocks == n))               # a block is kept whole or not at all
        assert np.all(mask[h][np.arange(Lq), np.arange(Lq) + Lk - Lq] == 1)
    with pytest.raises(ValueError):
        orc.pool_scores(acc[:, :-1], block, causal=False)


# ------------------------------------------------------------------------------ backward


@pytest.mark.parametrize("shape", [(2, 2, 37, 37, 16), (1, 2, 20, 45, 8)])
def test_bwd_equals_library_autograd(shape):
    """Gradients of a library softmax over an additive -inf mask, by reverse-mode differentiation
    in fp64 (rows without kept entries are left out of the library graph: they output 0)."""
    B, H, Lq, Lk, d = shape
    q, k, v, g = (_rand(s, 70 + n) for n, s in enumerate(((B, H, Lq, d), (B, H, Lk, d), (B, H, Lk, d), (B, H, Lq, d))))
    mask = inputs.random_mask(H, Lq, Lk, 0.3, seed=74, empty_rows=(3,))
    qd, kd, vd = (t.double().requires_grad_(True) for t in (q, k, v))
    s = torch.einsum("bhid,bhjd->bhij", qd, kd) * 0.31
    s = s.masked_fill(mask.bool().unsqueeze(0) == 0, float("-inf"))
    has = (mask.sum(-1) > 0)
    p = torch.where(has.unsqueeze(0).unsqueeze(-1), torch.softmax(torch.where(has.unsqueeze(0).unsqueeze(-1), s, torch.zeros_like(s)), -1), torch.zeros_like(s))
    p = p * mask.bool().unsqueeze(0)
    out = p @ vd
    (out * g.double()).sum().backward()
    dq, dk, dv = orc.attention_bwd(q.numpy(), k.numpy(), v.numpy(), g.numpy(), mask.numpy(), scale=0.31)
    np.testing.assert_allclose(out.detach().numpy(), orc.attention_fwd(q.numpy(), k.numpy(), v.numpy(), mask.numpy(), scale=0.31), rtol=1e-12, atol=1e-13)
    np.testing.assert_allclose(dq, qd.grad.numpy(), rtol=1e-10, atol=1e-12)
    np.testing.assert_allclose(dk, kd.grad.numpy(), rtol=1e-10, atol=1e-12)
    np.testing.assert_allclose(dv, vd.grad.numpy(), rtol=1e-10, atol=1e-12)
    assert np.all(dq[:, :, 3] == 0.0)                        # the row without kept entries passes no gradient


def test_bwd_matches_central_differences_of_the_forward():
    """Independent of any formula for the derivative: (L(x + e) - L(x - e)) / 2e of the oracle's own
    forward (pinned above), for a few coordinates of Q, K and V."""
    B, H, L, d = 1, 2, 9, 4
    rng = np.random.default_rng(75)
    q, k, v, g = (rng.standard_normal((B, H, L, d)).astype(np.float32) for _ in range(4))
    mask = inputs.random_mask(H, L, L, 0.5, seed=76).numpy()
    mask[:, :, 0] = 1
    dq, dk, dv = orc.attention_bwd(q, k, v, g, mask)
    loss = lambda a, b, c: float((orc.attention_fwd(a, b, c, mask) * g).sum())
    eps = 2.0 ** -10                                          # exact in fp32 next to values of order 1
    for arr, grad, which in ((q, dq, 0), (k, dk, 1), (v, dv, 2)):
        for idx in ((0, 0, 2, 1), (0, 1, 7, 3), (0, 1, 0, 0)):
            hi, lo = arr.copy(), arr.copy()
            hi[idx] += eps
            lo[idx] -= eps
            args_hi = [q, k, v]; args_lo = [q, k, v]
            args_hi[which], args_lo[which] = hi, lo
            fd = (loss(*args_hi) - loss(*args_lo)) / (float(hi[idx]) - float(lo[idx]))
            assert abs(fd - grad[idx]) <= 1e-5 * max(1.0, abs(fd)), (which, idx, fd, grad[idx])


def test_bwd_closed_forms():
    """One kept entry per row: p = 1, so dV is the scattered dO, and dQ = dK = 0.  Q = 0 with all
    entries kept: uniform weights, dV_j = mean-weighted sum of dO."""
    B, H, L, d = 1, 1, 6, 4
    rng = np.random.default_rng(77)
    q, k, v, g = (rng.standard_normal((B, H, L, d)).astype(np.float32) for _ in range(4))
    cols = np.array([2, 0, 5, 5, 1, 3])
    mask = np.zeros((H, L, L), dtype=np.uint8)
    mask[0, np.arange(L), cols] = 1
    dq, dk, dv = orc.attention_bwd(q, k, v, g, mask)
    assert np.all(dq == 0.0) and np.all(dk == 0.0)
    want = np.zeros((L, d))
    for i, j in enumerate(cols):
        want[j] += g[0, 0, i]
    np.testing.assert_allclose(dv[0, 0], want, rtol=1e-15)
    ones = np.ones((H, L, L), dtype=np.uint8)
    dq, dk, dv = orc.attention_bwd(np.zeros_like(q), k, v, g, ones)
    np.testing.assert_allclose(dv[0, 0], np.broadcast_to(g[0, 0].astype(np.float64).sum(0) / L, (L, d)), rtol=1e-13)


# --------------------------------------------------------------------------- 1.5-entmax (sparse normalisation)


def _entmax15_by_bisection(z):
    """Independent route to the same vector: tau is the root of the decreasing function
    sum_j max(z_j/2 - tau, 0)^2 - 1, bracketed by [max/2 - 1, max/2] and found by bisection."""
    x = np.asarray(z, dtype=np.float64) / 2.0
    lo, hi = x.max() - 1.0, x.max()
    for _ in range(200):
        mid = 0.5 * (lo + hi)
        if (np.maximum(x - mid, 0.0) ** 2).sum() >= 1.0:
            lo = mid
        else:
            hi = mid
    return np.maximum(x - 0.5 * (lo + hi), 0.0) ** 2


def test_entmax15_two_scores_closed_form():
    """Two scores a >= b with g = (a - b)/2: u^2 + (u - g)^2 = 1 gives u = (g + sqrt(2 - g^2))/2 while
    g < 1; from g = 1 on the whole mass sits on the larger score."""
    for a, b in ((0.0, 0.0), (0.3, -0.4), (1.0, 0.0), (2.5, 0.9), (-1.0, -2.99), (4.0, 2.0), (5.0, 1.0)):
        g = (a - b) / 2.0
        if g < 1.0:
            u = (g + math.sqrt(2.0 - g * g)) / 2.0
            want = np.array([u * u, (u - g) ** 2])
        else:
            want = np.array([1.0, 0.0])
        np.testing.assert_allclose(orc.entmax15([a, b]), want, rtol=0, atol=1e-15)
        np.testing.assert_allclose(orc.entmax15([b, a]), want[::-1], rtol=0, atol=1e-15)


@pytest.mark.parametrize("n", [1, 2, 3, 7, 64, 1000, 4096])
@pytest.mark.parametrize("spread", [0.05, 1.0, 4.0])
def test_entmax15_against_bisection(n, spread):
    rng = np.random.default_rng(1000 * n + int(100 * spread))
    z = rng.standard_normal(n) * spread + rng.uniform(-30, 30)
    if n >= 7:
        z[3] = z[5] = z.max()                     # ties at the top
    p = orc.entmax15(z)
    assert abs(p.sum() - 1.0) <= 1e-12 and np.all(p >= 0.0)
    np.testing.assert_allclose(p, _entmax15_by_bisection(z), rtol=0, atol=1e-12)


def test_entmax15_invariants_and_special_cases():
    rng = np.random.default_rng(5)
    z = rng.standard_normal(50) * 2.0
    p = orc.entmax15(z)
    np.testing.assert_allclose(orc.entmax15(z + 17.25), p, rtol=0, atol=1e-13)      # shift invariance
    perm = rng.permutation(50)
    np.testing.assert_allclose(orc.entmax15(z[perm]), p[perm], rtol=0, atol=1e-15)   # no dependence on position
    assert np.all(np.diff(p[np.argsort(z)]) >= 0.0)                                 # order preserving
    assert 0 < np.count_nonzero(p) < 50                                             # sparse, unlike a softmax
    np.testing.assert_allclose(orc.entmax15(np.full(9, -3.5)), np.full(9, 1.0 / 9.0), rtol=1e-15)
    np.testing.assert_array_equal(orc.entmax15([1.0, 3.0, -2.0, 0.999]), [0.0, 1.0, 0.0, 0.0])  # gap of 2
    np.testing.assert_allclose(orc.entmax15([0.0, 0.0, -5.0]), [0.5, 0.5, 0.0], rtol=1e-15)
    # every score outside the support lies at or below the threshold: z_j / 2 <= tau
    x = z / 2.0
    tau = x[p > 0].min() - math.sqrt(p[p > 0].min())
    assert np.all(x[p == 0] <= tau + 1e-15)


def test_entmax15_maximises_its_objective():
    """The defining property: p maximises p.z + H(p) over the simplex, H the Tsallis entropy of order 1.5,
    sum_j (p_j - p_j^1.5) / 0.75.  The objective is concave, so it is enough that no move towards another
    point of the simplex raises it."""
    rng = np.random.default_rng(6)

    def objective(p, z):
        return float(p @ z + (p - p ** 1.5).sum() / 0.75)

    for n in (3, 10, 40):
        z = rng.standard_normal(n) * 1.5
        p = orc.entmax15(z)
        best = objective(p, z)
        for _ in range(200):
            q = rng.dirichlet(np.full(n, 0.3))
            for eps in (1e-3, 0.05, 1.0):
                assert objective((1 - eps) * p + eps * q, z) <= best + 1e-12
        # and a wrong exponent, a missing 1/2 or a wrong normalisation would not pass:
        soft = np.exp(z - z.max()); soft /= soft.sum()
        assert objective(soft, z) < best - 1e-6


def _entmax15_rows_np(s, valid):
    """Row-wise 1.5-entmax over the entries marked valid (numpy + the bisection above)."""
    out = np.zeros_like(s)
    for idx in np.ndindex(s.shape[:-1]):
        keep = valid[idx]
        if keep.any():
            out[idx][keep] = _entmax15_by_bisection(s[idx][keep])
    return out


@pytest.mark.parametrize("causal,Lq,Lk", [(False, 9, 14), (True, 11, 11), (True, 6, 13)])
def test_accumulate_entmax15_equals_row_wise_composition(causal, Lq, Lk):
    B, H, d = 3, 2, 8
    q, k = _rand((B, H, Lq, d), 21).numpy(), _rand((B, H, Lk, d), 22).numpy()
    bias = np.random.default_rng(23).standard_normal((H, Lq, Lk)).astype(np.float32)
    scale = 0.7
    s = np.einsum("bhid,bhjd->bhij", q.astype(np.float64), k.astype(np.float64)) * scale + bias[None].astype(np.float64)
    valid = np.ones((Lq, Lk), dtype=bool)
    if causal:
        valid = np.tril(valid, k=Lk - Lq)
    want = _entmax15_rows_np(s, np.broadcast_to(valid, s.shape)).sum(0)
    acc = np.full((H, Lq, Lk), 0.25, dtype=np.float64)        # the call adds to what is there
    orc.accumulate_entmax15(acc, q, k, bias, causal=causal, scale=scale)
    np.testing.assert_allclose(acc - 0.25, want, rtol=0, atol=1e-12)
    assert np.all((acc == 0.25) | np.broadcast_to(valid, acc.shape))   # nothing outside the domain is touched
    rows = [(0, 0), (1, Lq - 1), (1, 3)]
    got = orc.accumulate_entmax15_rows(rows, q, k, bias, causal=causal, scale=scale)
    for r, (h, i) in enumerate(rows):
        np.testing.assert_allclose(got[r], want[h, i], rtol=0, atol=1e-12)


def test_attention_entmax15_equals_row_wise_composition():
    B, H, Lq, Lk, d = 2, 2, 10, 17, 8
    q, k, v = _rand((B, H, Lq, d), 31).numpy(), _rand((B, H, Lk, d), 32).numpy(), _rand((B, H, Lk, d), 33).numpy()
    rng = np.random.default_rng(34)
    mask = (rng.random((H, Lq, Lk)) < 0.4).astype(np.uint8)
    mask[0, 2] = 0                                             # a row with nothing kept
    mask[1, 4] = 0; mask[1, 4, 9] = 1                          # a row with a single kept key
    s = np.einsum("bhid,bhjd->bhij", q.astype(np.float64), k.astype(np.float64)) / math.sqrt(d)
    p = _entmax15_rows_np(s, np.broadcast_to(mask.astype(bool), s.shape))
    want = np.einsum("bhij,bhjd->bhid", p, v.astype(np.float64))
    got = orc.attention_entmax15_fwd(q, k, v, mask)
    np.testing.assert_allclose(got, want, rtol=0, atol=1e-12)
    assert np.all(got[:, 0, 2] == 0.0)
    np.testing.assert_array_equal(got[:, 1, 4], v[:, 1, 9].astype(np.float64))
    rows = [(0, 0, 0), (1, 1, 4), (1, 0, 9)]
    sub = orc.attention_entmax15_rows(q, k, v, mask, rows)
    for r, (b, h, i) in enumerate(rows):
        np.testing.assert_allclose(sub[r], want[b, h, i], rtol=0, atol=1e-12)


# --------------------------------------------------------------------------- Eq. 2 with ties kept


@pytest.mark.parametrize("per_layer", [False, True])
def test_ties_mask_is_a_threshold_on_the_kth_largest_value(per_layer):
    """Without a domain restriction or forced entries the rule is one line of numpy: tau = the k-th largest
    value of the population, mask = (acc >= tau).  Values on a coarse grid, so ties at tau are the rule."""
    rng = np.random.default_rng(41)
    H, Lq, Lk = 3, 9, 14
    acc = (rng.integers(0, 12, size=(H, Lq, Lk)) / 8.0).astype(np.float32)
    for keep in (0.1, 0.37, 0.8, 1.0):
        mask, nnz = orc.build_mask_ties(acc, keep, causal=False, keep_diag=False, per_layer=per_layer)
        pops = [acc] if per_layer else [acc[h:h + 1] for h in range(H)]
        want = []
        for pop in pops:
            k = orc.keep_count(pop.size, 0, keep)
            tau = np.partition(pop.reshape(-1), pop.size - k)[pop.size - k]
            want.append(pop >= tau)
        want = np.concatenate(want, axis=0)
        np.testing.assert_array_equal(mask.astype(bool), want)
        np.testing.assert_array_equal(nnz, want.reshape(H, -1).sum(1))
        assert nnz.sum() >= (orc.keep_count(acc.size, 0, keep) if per_layer else H * orc.keep_count(Lq * Lk, 0, keep))


@pytest.mark.parametrize("causal,Lq,Lk", [(True, 11, 11), (True, 6, 13), (False, 8, 8)])
@pytest.mark.parametrize("per_layer", [False, True])
def test_ties_mask_against_the_exact_count_mask(causal, Lq, Lk, per_layer):
    """With a domain and forced entries: the exact-count mask (pinned above) fixes tau as its smallest kept
    value that is not forced; the ties rule keeps the forced entries and everything in the domain >= tau.
    Distinct values: the two masks coincide."""
    rng = np.random.default_rng(43)
    H = 2
    exact = orc.build_mask_layer if per_layer else orc.build_mask
    dom = np.tril(np.ones((Lq, Lk), dtype=bool), Lk - Lq) if causal else np.ones((Lq, Lk), dtype=bool)
    forced = np.zeros((Lq, Lk), dtype=bool)
    forced[np.arange(Lq), np.arange(Lq) + Lk - Lq] = True
    acc = (rng.integers(0, 6, size=(H, Lq, Lk)) / 4.0).astype(np.float32)
    for keep in (0.15, 0.5, 0.9):
        base, _ = exact(acc, keep, causal=causal, keep_diag=True)
        mask, nnz = orc.build_mask_ties(acc, keep, causal=causal, keep_diag=True, per_layer=per_layer)
        want = np.zeros_like(base, dtype=bool)
        groups = [slice(0, H)] if per_layer else [slice(h, h + 1) for h in range(H)]
        for g in groups:
            kept_free = base[g].astype(bool) & ~forced[None]
            w = np.broadcast_to(forced[None], base[g].shape).copy()
            if kept_free.any():
                w |= (acc[g] >= acc[g][kept_free].min()) & dom[None]
            want[g] = w
        np.testing.assert_array_equal(mask.astype(bool), want)
        np.testing.assert_array_equal(nnz, want.reshape(H, -1).sum(1))
        assert np.all(mask >= base)                                   # a superset of the exact-count mask
    distinct = rng.permutation(H * Lq * Lk).reshape(H, Lq, Lk).astype(np.float32)
    for keep in (0.2, 0.6):
        base, n0 = exact(distinct, keep, causal=causal, keep_diag=True)
        mask, n1 = orc.build_mask_ties(distinct, keep, causal=causal, keep_diag=True, per_layer=per_layer)
        np.testing.assert_array_equal(mask, base)
        np.testing.assert_array_equal(n0, n1)
    flat = np.full((H, Lq, Lk), 0.5, dtype=np.float32)                # all equal: nothing is strictly below
    mask, _ = orc.build_mask_ties(flat, 0.3, causal=causal, keep_diag=True, per_layer=per_layer)
    np.testing.assert_array_equal(mask.astype(bool), np.broadcast_to(dom, mask.shape))

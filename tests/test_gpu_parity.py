"""GPU parity: the CUDA library (through its C ABI) against the CPU oracle on
the same seeded inputs.  Integer outputs (masks, tile lists, counts) must be
bit-exact; attention outputs within max-abs 1e-2 / rel-L2 5e-3 (bf16) and
1e-5 / 1e-6 (fp32)."""
import numpy as np
import pytest
import torch

from oracle import ap_oracle as orc
from paper_2012_02030_b200 import inputs, metrics
from tests import parity_util as pu

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ap():
    from paper_2012_02030_b200 import binding

    assert torch.cuda.is_available()
    return binding


W = inputs.WORKLOADS

# ------------------------------------------------------------------------------ tile lists


@pytest.mark.parametrize("shape", [(2, 128, 128), (2, 300, 200), (1, 130, 515), (3, 5, 7), (1, 1024, 1024)])
def test_mask_to_tiles_bit_exact(ap, shape):
    H, Lq, Lk = shape
    mask = inputs.random_mask(H, Lq, Lk, 0.01, seed=60)
    mask[0, : min(128, Lq), : min(128, Lk)] = 1
    if Lk > 256:
        mask[:, :, 128:256] = 0
    tiles = ap.Tiles(H, Lq, Lk)
    ap.ap_mask_to_tiles(mask.cuda(), tiles)
    assert ap.ap_device_status() == ap.AP_OK
    pu.assert_tiles_equal(tiles.to_host(), orc.mask_to_tiles(mask.numpy()))


def test_mask_to_tiles_all_zero_and_capacity_overflow(ap):
    H, Lq, Lk = 2, 256, 384
    tiles = ap.Tiles(H, Lq, Lk)
    ap.ap_mask_to_tiles(torch.zeros((H, Lq, Lk), dtype=torch.uint8, device="cuda"), tiles)
    assert ap.ap_device_status() == ap.AP_OK
    assert tiles.n_tiles() == 0 and int(tiles.row_ptr.abs().sum()) == 0
    small = ap.Tiles(H, Lq, Lk, cap=3)
    ap.ap_mask_to_tiles(torch.ones((H, Lq, Lk), dtype=torch.uint8, device="cuda"), small)
    assert ap.ap_device_status() == ap.AP_ERR_WORKSPACE   # reported ...
    assert ap.ap_device_status() == ap.AP_OK              # ... and cleared
    assert int(small.row_ptr.max()) == 3                  # truncated, never past the capacity


@pytest.mark.parametrize("causal", [False, True])
@pytest.mark.parametrize("L", [(128, 128), (200, 200), (512, 512), (130, 300), (384, 768), (256, 257), (300, 1000)])
def test_dense_tiles_equal_tiles_of_the_full_domain(ap, L, causal):
    Lq, Lk = L
    H = 2
    dom = torch.ones((H, Lq, Lk), dtype=torch.uint8)
    if causal:  # with Lk > Lq: Lk - Lq memory keys before the causal segment
        dom = torch.tril(dom, diagonal=Lk - Lq)
    tiles = ap.Tiles(H, Lq, Lk)
    ap.ap_dense_tiles(tiles, causal=causal)
    assert ap.ap_device_status() == ap.AP_OK
    pu.assert_tiles_equal(tiles.to_host(), orc.mask_to_tiles(dom.numpy()))


# ------------------------------------------------------------------------------ build mask


def _check_build_mask(ap, acc32: np.ndarray, w, layer=False):
    acc_dev = torch.from_numpy(acc32).cuda()
    mask, tiles, nnz = pu.gpu_build_mask(ap, acc_dev, w, layer=layer)
    want = orc.build_mask_layer if layer else orc.build_mask
    want_mask, want_nnz = want(acc32, w.keep_frac, w.causal, w.keep_diag)
    np.testing.assert_array_equal(nnz.cpu().numpy(), want_nnz)
    np.testing.assert_array_equal(mask.cpu().numpy(), want_mask)
    pu.assert_tiles_equal(tiles.to_host(), orc.mask_to_tiles(want_mask))
    return want_mask


@pytest.mark.parametrize("causal", [False, True])
@pytest.mark.parametrize("keep_diag", [False, True])
@pytest.mark.parametrize("shape", [(3, 67, 67), (2, 128, 128), (2, 300, 300), (1, 5, 5)])
def test_build_mask_random_values_with_ties(ap, shape, causal, keep_diag):
    H, Lq, Lk = shape
    rng = np.random.default_rng(70)
    acc = rng.random((H, Lq, Lk), dtype=np.float32)
    acc[0].flat[::3] = 0.5                      # a third of head 0 ties at one value
    acc[-1] = np.round(acc[-1] * 8) / 8         # 9 distinct values: the threshold is always tied
    acc[0, 0, :3] = [-1.0, -0.0, 0.0]           # negatives and signed zeros
    for keep in (0.1, 0.5, 1.0):
        _check_build_mask(ap, acc, W["tiny"].scaled(H=H, Lq=Lq, Lk=Lk, causal=causal, keep_diag=keep_diag,
                                                     keep_frac=keep))


def _check_build_mask_ties(ap, acc32: np.ndarray, w, layer):
    H, Lq, Lk = acc32.shape
    mask = torch.full((H, Lq, Lk), 7, dtype=torch.uint8, device="cuda")  # poison: every byte must be written
    nnz = torch.full((H,), -1, dtype=torch.int64, device="cuda")
    tiles = ap.Tiles(H, Lq, Lk)
    flags = ap.AP_MASK_KEEP_TIES | (ap.AP_MASK_PER_LAYER if layer else 0)
    ap.ap_build_mask_ex(torch.from_numpy(acc32).cuda(), w.keep_frac, w.causal, w.keep_diag, flags, mask, tiles, nnz)
    assert ap.ap_device_status() == ap.AP_OK
    want_mask, want_nnz = orc.build_mask_ties(acc32, w.keep_frac, w.causal, w.keep_diag, per_layer=layer)
    np.testing.assert_array_equal(nnz.cpu().numpy(), want_nnz)
    np.testing.assert_array_equal(mask.cpu().numpy(), want_mask)
    pu.assert_tiles_equal(tiles.to_host(), orc.mask_to_tiles(want_mask))
    return want_nnz


@pytest.mark.parametrize("layer", [False, True])
@pytest.mark.parametrize("causal,keep_diag", [(False, False), (True, True), (False, True)])
@pytest.mark.parametrize("shape", [(3, 67, 67), (2, 300, 300), (2, 100, 260), (1, 5, 5)])
def test_build_mask_keeping_all_ties(ap, shape, causal, keep_diag, layer):
    """Eq. 2 with its strict inequality: entries equal to the threshold all stay."""
    H, Lq, Lk = shape
    if causal and Lk < Lq:
        pytest.skip("the causal domain needs Lk >= Lq")
    rng = np.random.default_rng(72)
    acc = rng.random((H, Lq, Lk), dtype=np.float32)
    acc[0].flat[::3] = 0.5                      # a third of head 0 ties at one value
    acc[-1] = np.round(acc[-1] * 8) / 8         # 9 distinct values: the threshold is always tied
    acc[0, 0, :3] = [-1.0, -0.0, 0.0]
    more = 0
    for keep in (1e-6, 0.1, 0.5, 1.0):
        w = W["tiny"].scaled(H=H, Lq=Lq, Lk=Lk, causal=causal, keep_diag=keep_diag, keep_frac=keep)
        nnz = _check_build_mask_ties(ap, acc, w, layer)
        k = metrics.keep_count(w.n_valid * (H if layer else 1), w.n_forced * (H if layer else 1), keep)
        more += int(nnz.sum() > (k if layer else k * H))
    assert more > 0 or Lq < 8                   # the case is exercised: ties pushed the count past k
    flags = ap.AP_MASK_KEEP_TIES | (ap.AP_MASK_PER_LAYER if layer else 0)
    assert flags  # with flags = 0 the entry point is ap_build_mask: checked below


def test_build_mask_ex_without_flags_is_build_mask(ap):
    acc = np.random.default_rng(73).random((2, 130, 130), dtype=np.float32)
    acc[1] = np.round(acc[1] * 4) / 4
    dev = torch.from_numpy(acc).cuda()
    for flags, want in ((0, orc.build_mask), (ap.AP_MASK_PER_LAYER, orc.build_mask_layer)):
        mask = torch.empty((2, 130, 130), dtype=torch.uint8, device="cuda")
        nnz = torch.empty((2,), dtype=torch.int64, device="cuda")
        ap.ap_build_mask_ex(dev, 0.3, True, True, flags, mask, None, nnz)
        want_mask, want_nnz = want(acc, 0.3, True, True)
        np.testing.assert_array_equal(mask.cpu().numpy(), want_mask)
        np.testing.assert_array_equal(nnz.cpu().numpy(), want_nnz)


@pytest.mark.parametrize("shape", [(2, 100, 260), (1, 257, 31)])
def test_build_mask_rectangular(ap, shape):
    H, Lq, Lk = shape
    acc = np.random.default_rng(71).random((H, Lq, Lk), dtype=np.float32)
    acc[0] = np.round(acc[0] * 4) / 4
    _check_build_mask(ap, acc, W["s2s_cross"].scaled(H=H, Lq=Lq, Lk=Lk, keep_frac=0.3))


def test_build_mask_constant_and_tiny_fraction(ap):
    acc = np.full((2, 130, 130), 0.25, dtype=np.float32)
    _check_build_mask(ap, acc, W["tiny"].scaled(H=2, Lq=130, Lk=130, keep_frac=0.37))
    _check_build_mask(ap, acc, W["tiny"].scaled(H=2, Lq=130, Lk=130, keep_frac=1e-6))       # forced entries only
    _check_build_mask(ap, acc, W["tiny"].scaled(H=2, Lq=130, Lk=130, keep_frac=1e-6, keep_diag=False))


@pytest.mark.parametrize("causal,L", [(False, 1100), (True, 1536)])
def test_build_mask_large_heads_take_the_one_pass_shortcut(ap, causal, L):
    """Heads of more than 2^20 selectable entries first try to bracket the threshold with a sample
    and select among the keys collected in one pass.  Head 0: distinct values (the shortcut holds);
    head 1: heavily quantised values, so the threshold key is tied thousands of times; head 2:
    skewed values (most mass near zero); head 3: constant, every key falls into the bracket and
    the collected keys overflow their buffer, so the head falls back to the three-pass select."""
    H = 4
    rng = np.random.default_rng(73 + L)
    acc = rng.random((H, L, L), dtype=np.float32)
    acc[1] = np.round(acc[1] * 32) / 32
    acc[2] = acc[2] ** 8
    acc[3] = 0.75
    # head 0: a handful of exact copies of the value at the 5 % threshold, scattered over the head, so
    # that the threshold key is tied a few times and only the copies with the lowest indices are kept
    dom = np.tril(np.ones((L, L), dtype=bool)) if causal else np.ones((L, L), dtype=bool)
    vals = acc[0][dom]
    k = int(0.05 * vals.size)
    v_thr = np.partition(vals, vals.size - k)[vals.size - k]
    rows = rng.integers(L // 2, L, size=9)
    cols = rng.integers(0, L // 2, size=9)
    acc[0, rows, cols] = v_thr
    for keep, keep_diag in ((0.05, True), (0.05, False), (0.5, False), (0.999, True)):
        _check_build_mask(ap, acc, W["tiny"].scaled(H=H, Lq=L, Lk=L, causal=causal, keep_diag=keep_diag,
                                                     keep_frac=keep))


def test_build_mask_optional_outputs(ap):
    acc = np.random.default_rng(72).random((2, 140, 140), dtype=np.float32)
    acc_dev = torch.from_numpy(acc).cuda()
    want_mask, _ = orc.build_mask(acc, 0.2, True, True)
    mask = torch.empty((2, 140, 140), dtype=torch.uint8, device="cuda")
    ap.ap_build_mask(acc_dev, 0.2, True, True, mask=mask)
    np.testing.assert_array_equal(mask.cpu().numpy(), want_mask)
    tiles = ap.Tiles(2, 140, 140)
    ap.ap_build_mask(acc_dev, 0.2, True, True, tiles=tiles)
    pu.assert_tiles_equal(tiles.to_host(), orc.mask_to_tiles(want_mask))
    assert ap.ap_device_status() == ap.AP_OK


@pytest.mark.parametrize("layer", [False, True])
@pytest.mark.parametrize("keep_diag", [False, True])
@pytest.mark.parametrize("shape", [(2, 100, 260), (3, 67, 200), (2, 384, 768), (2, 128, 129), (1, 5, 9)])
def test_build_mask_causal_with_memory_keys(ap, shape, keep_diag, layer):
    """Lk = mem + Lq: query i sees the keys j <= i + mem; its own position mem + i is the forced entry."""
    H, Lq, Lk = shape
    rng = np.random.default_rng(75)
    acc = rng.random((H, Lq, Lk), dtype=np.float32)
    acc[0].flat[::3] = 0.5
    acc[-1] = np.round(acc[-1] * 8) / 8
    for keep in (0.1, 0.5, 1.0):
        want = _check_build_mask(ap, acc, W["tiny"].scaled(H=H, Lq=Lq, Lk=Lk, causal=True, keep_diag=keep_diag,
                                                            keep_frac=keep), layer=layer)
        assert not want[:, ~np.tril(np.ones((Lq, Lk), dtype=bool), Lk - Lq)].any()
        if keep_diag:
            assert all(want[:, i, Lk - Lq + i].all() for i in range(Lq))


@pytest.mark.parametrize("layer", [False, True])
def test_build_mask_causal_with_memory_keys_large(ap, layer):
    """Large enough for the sampled shortcut (more than 2^20 selectable entries per head)."""
    H, Lq, Lk = 2, 1100, 1500
    rng = np.random.default_rng(76)
    acc = rng.random((H, Lq, Lk), dtype=np.float32)
    acc[1] = np.round(acc[1] * 64) / 64
    for keep, keep_diag in ((0.05, True), (0.4, False)):
        _check_build_mask(ap, acc, W["tiny"].scaled(H=H, Lq=Lq, Lk=Lk, causal=True, keep_diag=keep_diag,
                                                     keep_frac=keep), layer=layer)


# ------------------------------------------------------------- build mask, one threshold per layer


@pytest.mark.parametrize("causal", [False, True])
@pytest.mark.parametrize("keep_diag", [False, True])
@pytest.mark.parametrize("shape", [(3, 67, 67), (2, 128, 128), (4, 300, 300), (1, 5, 5)])
def test_build_mask_layer_random_values_with_ties(ap, shape, causal, keep_diag):
    H, Lq, Lk = shape
    rng = np.random.default_rng(80)
    acc = rng.random((H, Lq, Lk), dtype=np.float32)
    acc[0].flat[::3] = 0.5                      # ties inside head 0 and with the last head's values
    acc[-1] = np.round(acc[-1] * 8) / 8
    acc[0, 0, :3] = [-1.0, -0.0, 0.0]
    if H > 2:
        acc[1] *= 0.25                          # a head that loses almost everything at small fractions
    for keep in (0.1, 0.5, 1.0):
        _check_build_mask(ap, acc, W["tiny"].scaled(H=H, Lq=Lq, Lk=Lk, causal=causal, keep_diag=keep_diag,
                                                     keep_frac=keep), layer=True)


def test_build_mask_layer_rectangular_constant_and_tiny_fraction(ap):
    acc = np.random.default_rng(81).random((3, 100, 260), dtype=np.float32)
    acc[0] = np.round(acc[0] * 4) / 4
    _check_build_mask(ap, acc, W["s2s_cross"].scaled(H=3, Lq=100, Lk=260, keep_frac=0.3), layer=True)
    acc = np.full((2, 130, 130), 0.25, dtype=np.float32)    # every entry ties: the lowest global indices win
    _check_build_mask(ap, acc, W["tiny"].scaled(H=2, Lq=130, Lk=130, keep_frac=0.37), layer=True)
    _check_build_mask(ap, acc, W["tiny"].scaled(H=2, Lq=130, Lk=130, keep_frac=0.37, causal=True), layer=True)
    _check_build_mask(ap, acc, W["tiny"].scaled(H=2, Lq=130, Lk=130, keep_frac=1e-6), layer=True)
    _check_build_mask(ap, acc, W["tiny"].scaled(H=2, Lq=130, Lk=130, keep_frac=1e-6, keep_diag=False), layer=True)


def _domain(H, L, causal):
    dom = np.tril(np.ones((L, L), dtype=bool)) if causal else np.ones((L, L), dtype=bool)
    return np.broadcast_to(dom, (H, L, L))


@pytest.mark.parametrize("causal,L", [(False, 1100), (True, 1536)])
def test_build_mask_layer_large_takes_the_one_pass_shortcut(ap, causal, L):
    """More than 2^20 selectable entries in the layer: the threshold is bracketed with a sample and
    selected among the collected keys with grid-wide passes.  Head 1 is quantised to 32 levels, head
    2 skewed towards zero, head 3 constant.  Covered: a threshold tied a few times across heads (the
    copies with the lowest global indices are kept), a threshold on one of head 1's levels (tens of
    thousands of ties: tie counts and a prefix sum), a threshold on head 3's constant (the bracket
    overflows its buffer: three full passes), and thresholds in between."""
    H = 4
    rng = np.random.default_rng(83 + L)
    acc = rng.random((H, L, L), dtype=np.float32)
    acc[1] = np.round(acc[1] * 32) / 32
    acc[2] = acc[2] ** 8
    acc[3] = 0.75
    dom = _domain(H, L, causal)
    vals = acc[dom]
    n = vals.size
    k = int(0.05 * n)
    v_thr = np.partition(vals, n - k)[n - k]
    for h in (0, 2, 0, 2, 0, 2, 0, 2, 0):       # copies of the 5 % threshold in the lower left of two heads
        acc[h, rng.integers(L // 2, L), rng.integers(0, L // 2)] = v_thr
    vals = acc[dom]
    level = np.float32(0.5)                      # one of head 1's levels, cut in the middle of its ties
    k_level = int((vals > level).sum() + (vals == level).sum() // 2)
    for keep, keep_diag in ((0.05, True), (0.05, False), (k_level / n, False), (0.25, False), (0.5, True),
                            (0.999, True)):
        _check_build_mask(ap, acc, W["tiny"].scaled(H=H, Lq=L, Lk=L, causal=causal, keep_diag=keep_diag,
                                                     keep_frac=keep), layer=True)


def test_build_mask_layer_many_small_heads(ap):
    """Each head is far below the size at which the shortcut is tried, the layer is above it."""
    H, L = 16, 300
    acc = np.random.default_rng(84).random((H, L, L), dtype=np.float32)
    acc *= np.linspace(0.2, 1.0, H, dtype=np.float32)[:, None, None]
    for keep in (0.1, 0.6):
        want = _check_build_mask(ap, acc, W["tiny"].scaled(H=H, Lq=L, Lk=L, causal=True, keep_frac=keep), layer=True)
        per_head = want.reshape(H, -1).sum(1)
        assert per_head[0] < per_head[-1]        # unlike the per-head rule, heads keep unequal shares


def test_build_mask_layer_full_size_long(ap):
    """The long workload's layer at full size, on the accumulator the calibration kernel wrote.
    The first four heads as a layer of their own are compared with the oracle entry by entry; for
    all sixteen, the properties that define the result: k entries kept in all, every forced entry
    kept, no pruned entry larger than a kept one, and among the entries equal to the smallest kept
    value the kept ones come first in global index order."""
    w = W["long"]
    acc = pu.gpu_accumulate(ap, w, 1, None)
    _check_build_mask(ap, acc[:4].cpu().numpy(), w.scaled(H=4), layer=True)

    mask, tiles, nnz = pu.gpu_build_mask(ap, acc, w, layer=True)
    k = orc.keep_count(w.H * w.n_valid, w.H * w.n_forced, w.keep_frac)
    assert int(nnz.sum()) == k
    assert torch.equal(mask.view(w.H, -1).sum(-1, dtype=torch.int64), nnz)
    assert int(nnz.min()) < int(nnz.max())
    pop = np.unpackbits(tiles.to_host()["bitmap"].view(np.uint8)).sum()
    assert pop == k
    eye = torch.eye(w.Lq, dtype=torch.bool, device="cuda")
    dom = torch.tril(torch.ones((w.Lq, w.Lk), dtype=torch.bool, device="cuda"))
    assert bool(mask[:, eye].all()) and not bool(mask[:, ~dom].any())
    free = (dom & ~eye).expand(w.H, -1, -1)
    kept, pruned = free & (mask != 0), free & (mask == 0)
    v_kept, v_pruned = acc[kept].min(), acc[pruned].max()
    assert v_kept >= v_pruned
    if v_kept == v_pruned:
        tie = (acc == v_kept).view(-1)
        first_pruned = torch.nonzero(tie & pruned.reshape(-1))[0]
        last_kept = torch.nonzero(tie & kept.reshape(-1))[-1]
        assert int(last_kept) < int(first_pruned)


# ------------------------------------------------------------------ block-structured pruning


@pytest.mark.parametrize("causal,shape", [(False, (2, 256, 384)), (True, (2, 384, 384)), (True, (3, 256, 640)),
                                          (False, (1, 128, 128)), (True, (2, 1024, 1024))])
@pytest.mark.parametrize("block", [16, 32, 128])
def test_block_structured_pruning(ap, shape, causal, block):
    """Pooled block scores against the oracle (fp32 sums against fp64: relative 1e-5); Eq. 2 over the
    blocks on the GPU's own pooled bits, the expansion and the tile list bit for bit; every block kept
    whole or not at all; and the forward pass under the block mask."""
    H, Lq, Lk = shape
    rng = np.random.default_rng(77 + block)
    acc = rng.random((H, Lq, Lk), dtype=np.float32)
    acc[0] *= np.linspace(0.1, 2.0, Lk, dtype=np.float32)[None, :]
    acc_dev = torch.from_numpy(acc).cuda()
    pooled = ap.ap_pool_scores(acc_dev, block, causal)
    np.testing.assert_allclose(pooled.cpu().numpy(), orc.pool_scores(acc, block, causal), rtol=1e-5, atol=1e-7)
    R, C = Lq // block, Lk // block
    bmask = torch.full((H, R, C), 7, dtype=torch.uint8, device="cuda")
    keep_diag = Lq == Lk or causal
    ap.ap_build_mask(pooled, 0.3, causal, keep_diag, mask=bmask)
    want_b, _ = orc.build_mask(pooled.cpu().numpy(), 0.3, causal, keep_diag)
    np.testing.assert_array_equal(bmask.cpu().numpy(), want_b)
    mask = torch.full((H, Lq, Lk), 7, dtype=torch.uint8, device="cuda")
    ap.ap_expand_block_mask(bmask, block, causal, mask=mask)
    want = orc.expand_block_mask(want_b, block, causal)
    np.testing.assert_array_equal(mask.cpu().numpy(), want)
    tiles = ap.Tiles(H, Lq, Lk)
    ap.ap_mask_to_tiles(mask, tiles)
    assert ap.ap_device_status() == ap.AP_OK
    host = tiles.to_host()
    pu.assert_tiles_equal(host, orc.mask_to_tiles(want))
    if block == 128 and not causal:
        assert host["flags"].all()                       # every stored tile is fully kept
    w = W["tiny"].scaled(B=2, H=H, Lq=Lq, Lk=Lk, d=64, dtype="bf16")
    q, k, v = inputs.eval_qkv(w)
    out = ap.ap_sparse_attention_fwd(q.cuda(), k.cuda(), v.cuda(), tiles)
    ref = orc.attention_fwd(inputs.widen(q), inputs.widen(k), inputs.widen(v), want)
    pu.assert_close_attention(out, ref, "bf16", "block mask")


# ------------------------------------------------------------------- random-pruning control


@pytest.mark.parametrize("shape", [(2, 128, 128), (3, 67, 201), (1, 1, 5), (2, 1024, 1024)])
def test_random_scores_bit_exact_and_mask_of_exact_count(ap, shape):
    H, Lq, Lk = shape
    for seed in (0, 1234567, 2**63 + 5):
        got = torch.full((H, Lq, Lk), -1.0, dtype=torch.float32, device="cuda")
        ap.ap_random_scores(got, seed)
        np.testing.assert_array_equal(got.cpu().numpy(), orc.random_scores(H, Lq, Lk, seed))
    if Lq == Lk:  # pruning random entries: Eq. 2's selection on the scores
        w = W["tiny"].scaled(H=H, Lq=Lq, Lk=Lk, causal=True, keep_frac=0.2)
        _check_build_mask(ap, got.cpu().numpy(), w)


# ------------------------------------------------------------------------------ accumulate


def _acc_tolerance(dtype):
    # fp32 FMA dot products + fp32 exp against fp64: relative error of an entry
    return dict(rtol=2e-5, atol=1e-7)


@pytest.mark.parametrize("name,over,n_batches", [
    ("tiny", {}, 3),
    ("tiny", dict(Lq=77, Lk=77, B=3), 2),
    ("tiny", dict(Lq=50, Lk=300, d=128), 2),
    ("bert", dict(B=4, H=3), 2),
    ("lm", dict(B=2, H=2, Lq=300, Lk=300), 2),
    ("long", dict(B=1, H=2, Lq=640, Lk=640), 2),
    # causal with memory keys (Lk = mem + Lq): tile-aligned, ragged, and on the CUDA-core path
    ("txl", dict(B=2, H=2), 2),
    ("txl", dict(B=2, H=2, Lq=200, Lk=333), 2),
    ("long", dict(B=1, H=2, Lq=256, Lk=700), 1),
    ("tiny", dict(Lq=77, Lk=130, causal=True), 2),
    # half precision (the precision of the paper's translation experiments)
    ("s2s_cross", dict(B=3, H=2, dtype="f16"), 2),
    ("long", dict(B=1, H=2, Lq=384, Lk=384, dtype="f16"), 1),
])
def test_accumulate_matches_oracle(ap, name, over, n_batches):
    w = W[name].scaled(**over)
    bias = inputs.calib_bias(w)
    acc = pu.gpu_accumulate(ap, w, n_batches, bias.cuda())
    again = pu.gpu_accumulate(ap, w, n_batches, bias.cuda())
    assert torch.equal(acc, again)  # fixed summation order: bit-reproducible
    want = pu.oracle_accumulate(w, n_batches, bias)
    got = acc.cpu().numpy()
    tol = _acc_tolerance(w.dtype)
    np.testing.assert_allclose(got, want, rtol=tol["rtol"], atol=tol["atol"] * n_batches * w.B)
    if w.causal:
        assert np.all(got[:, ~np.tril(np.ones((w.Lq, w.Lk), dtype=bool), w.Lk - w.Lq)] == 0.0)
    np.testing.assert_allclose(got.sum(-1), n_batches * w.B, rtol=1e-5)


def test_accumulate_without_bias_and_custom_scale(ap):
    w = W["tiny"].scaled(Lq=40, Lk=90)
    q, k = inputs.calib_qk(w, 0)
    acc = torch.zeros((w.H, w.Lq, w.Lk), device="cuda")
    ap.ap_accumulate_attention(acc, q.cuda(), k.cuda(), None, causal=False, scale=0.2)
    want = np.zeros((w.H, w.Lq, w.Lk))
    orc.accumulate(want, inputs.widen(q), inputs.widen(k), None, causal=False, scale=0.2)
    np.testing.assert_allclose(acc.cpu().numpy(), want, rtol=2e-5, atol=1e-7)


# ------------------------------------------------------------------------------ accumulate, 1.5-entmax


def _entmax_acc(ap, w, n_batches, bias_dev, scale=0.0):
    acc = torch.zeros((w.H, w.Lq, w.Lk), dtype=torch.float32, device="cuda")
    for t in range(n_batches):
        q, k = inputs.calib_qk(w, t)
        ap.ap_accumulate_attention_entmax15(acc, q.cuda(), k.cuda(), bias_dev, causal=w.causal, scale=scale)
    assert ap.ap_device_status() == ap.AP_OK
    return acc


def _entmax_want(w, n_batches, bias, scale=None):
    acc64 = np.zeros((w.H, w.Lq, w.Lk))
    for t in range(n_batches):
        q, k = inputs.calib_qk(w, t)
        orc.accumulate_entmax15(acc64, inputs.widen(q), inputs.widen(k), None if bias is None else bias.numpy(),
                                causal=w.causal, scale=scale)
    return acc64


# A weight is p = u^2 with u = x - tau; the fp32 threshold is off by at most a few 1e-6 (the stopping rule of
# the iteration plus the rounding of x, |x| of order 10), so p is off by 2 u dtau <= 2e-5 per sample
# whatever its size: an absolute bound per sample, plus the relative error of the fp32 square.
ENTMAX_ATOL, ENTMAX_RTOL = 2e-5, 1e-4


@pytest.mark.parametrize("name,over,n_batches", [
    ("tiny", {}, 3),
    ("tiny", dict(Lq=77, Lk=77, B=3), 2),            # ragged, bias through direct loads (Lk % 4 != 0)
    ("tiny", dict(Lq=50, Lk=300, d=128), 2),
    ("tiny", dict(B=18, H=2), 1),                    # more samples than one launch holds (8)
    ("bert", dict(B=4, H=3), 2),
    ("lm", dict(B=2, H=2, Lq=300, Lk=300), 2),       # causal
    ("long", dict(B=1, H=2, Lq=640, Lk=640), 2),
    ("txl", dict(B=2, H=2, Lq=200, Lk=333), 2),      # causal with memory keys
    ("s2s_cross", dict(B=3, H=2, dtype="f16"), 2),
    # fp32 tensors: CUDA cores, the row's scores in shared memory
    ("tiny", dict(dtype="f32"), 2),
    ("tiny", dict(dtype="f32", Lq=77, Lk=130, causal=True, d=128), 2),
])
def test_accumulate_entmax15_matches_oracle(ap, name, over, n_batches):
    w = W[name].scaled(**over)
    if w.dtype == "f32" and "dtype" not in over:
        w = w.scaled(dtype="bf16")
    bias = inputs.calib_bias(w)
    acc = _entmax_acc(ap, w, n_batches, bias.cuda())
    assert torch.equal(acc, _entmax_acc(ap, w, n_batches, bias.cuda()))  # fixed order: bit-reproducible
    got, want = acc.cpu().numpy(), _entmax_want(w, n_batches, bias)
    total = n_batches * w.B
    np.testing.assert_allclose(got, want, rtol=ENTMAX_RTOL, atol=ENTMAX_ATOL * total)
    if w.causal:
        assert np.all(got[:, ~np.tril(np.ones((w.Lq, w.Lk), dtype=bool), w.Lk - w.Lq)] == 0.0)
    np.testing.assert_allclose(got.sum(-1), total, rtol=2e-5)
    # sparse, unlike the softmax average: entries no sample gives weight stay exactly zero
    clear = want == 0.0
    assert clear.any() and np.count_nonzero(got[clear]) <= 1e-3 * clear.sum()


def test_accumulate_entmax15_special_rows(ap):
    """Closed forms through the kernel: equal scores give the uniform row (the longest Newton run: the
    threshold has to travel from max - 1 to max - 1/sqrt(n)); a gap of 2 between the best and the second
    best score gives a one-hot row."""
    H, L, d = 1, 1024, 64
    q = torch.zeros((1, H, L, d), dtype=torch.bfloat16, device="cuda")
    k = torch.randn((1, H, L, d), generator=torch.Generator().manual_seed(3)).to(torch.bfloat16).cuda()
    acc = torch.zeros((H, L, L), device="cuda")
    ap.ap_accumulate_attention_entmax15(acc, q, k, None, causal=True)
    rows = torch.arange(1, L + 1, dtype=torch.float32, device="cuda")[:, None]
    want = torch.tril(torch.ones((L, L), device="cuda")) / rows
    assert torch.allclose(acc[0], want, rtol=2e-4, atol=1e-8)
    # one-hot: q_i = k_i = 8 e_(i mod d) ... use a bias instead: +4 on the diagonal, 0 elsewhere, q = 0
    bias = torch.zeros((H, L, L), device="cuda")
    bias[0].fill_diagonal_(4.0)
    acc.zero_()
    ap.ap_accumulate_attention_entmax15(acc, q, k, bias, causal=False)
    assert torch.equal(acc[0], torch.eye(L, device="cuda"))
    assert ap.ap_device_status() == ap.AP_OK


def test_accumulate_entmax15_large_scores(ap):
    """Scores in the hundreds: fp32 resolves x = z/2 to about 1e-5 there, so the threshold and with it
    the weights are coarser (2 u dtau with dtau of that order), but the iteration still ends, rows still sum
    to 1 and almost every row is one-hot or close to it."""
    w = W["tiny"].scaled(Lq=200, Lk=333, dtype="bf16", B=2)
    got = _entmax_acc(ap, w, 1, None, scale=25.0).cpu().numpy()
    want = _entmax_want(w, 1, None, scale=25.0)
    assert np.isfinite(got).all()
    np.testing.assert_allclose(got.sum(-1), w.B, rtol=1e-4)
    np.testing.assert_allclose(got, want, rtol=1e-3, atol=2e-3)


def test_accumulate_entmax15_sharp_scores_custom_scale(ap):
    w = W["tiny"].scaled(Lq=40, Lk=90, dtype="bf16")
    for scale in (0.05, 1.5):
        got = _entmax_acc(ap, w, 1, None, scale=scale).cpu().numpy()
        want = _entmax_want(w, 1, None, scale=scale)
        np.testing.assert_allclose(got, want, rtol=ENTMAX_RTOL, atol=ENTMAX_ATOL * w.B)


# ------------------------------------------------------------------------------ forward


def _fwd_case(ap, w, mask: torch.Tensor, scale=0.0):
    q, k, v = inputs.eval_qkv(w)
    tiles = ap.Tiles(w.H, w.Lq, w.Lk)
    ap.ap_mask_to_tiles(mask.cuda(), tiles)
    out = ap.ap_sparse_attention_fwd(q.cuda(), k.cuda(), v.cuda(), tiles, scale=scale)
    assert ap.ap_device_status() == ap.AP_OK
    ref = orc.attention_fwd(inputs.widen(q), inputs.widen(k), inputs.widen(v), mask.numpy(),
                            scale=None if scale == 0.0 else scale)
    pu.assert_close_attention(out, ref, w.dtype, w.name)
    return out, ref


@pytest.mark.parametrize("dtype", ["f32", "bf16", "f16"])
@pytest.mark.parametrize("d", [64, 128])
@pytest.mark.parametrize("shape", [(2, 2, 128, 128), (1, 2, 200, 333), (2, 1, 513, 130), (1, 1, 5, 7)])
def test_forward_random_masks_ragged_shapes(ap, shape, d, dtype):
    B, H, Lq, Lk = shape
    w = W["tiny"].scaled(B=B, H=H, Lq=Lq, Lk=Lk, d=d, dtype=dtype)
    mask = inputs.random_mask(H, Lq, Lk, 0.15, seed=80, empty_rows=(0, Lq - 1) if Lq > 2 else ())
    mask[0, : min(128, Lq), : min(128, Lk)] = 1   # a FULL (or edge-full) tile next to partial ones
    out, _ = _fwd_case(ap, w, mask)
    o = out.float().cpu().numpy()
    empty = mask.numpy().sum(-1) == 0                  # rows with no kept entry output exact zeros
    if H > 1 or Lq > 128:
        assert empty.any()
    assert np.all(o[:, empty] == 0.0)


@pytest.mark.parametrize("d", [64, 128])
def test_forward_many_one_round_items_per_cta_poisoned_output(ap, d):
    """Far more items than four per SM, each of one round (one query tile, one key tile): the softmax
    warps run ahead of the epilogue warps as far as the hand-over ring lets them, and the end of a
    CTA's work follows a row of very short items.  Every output element must have been written."""
    B, H, L = 64, 16, 128  # 1024 items of one round on 148 CTAs
    w = W["tiny"].scaled(B=B, H=H, Lq=L, Lk=L, d=d, dtype="bf16")
    q, k, v = inputs.eval_qkv(w)
    mask = inputs.random_mask(H, L, L, 0.8, seed=91, causal=True)  # (dense rows: the fixed absolute tolerance applies)
    tiles = ap.Tiles(H, L, L)
    ap.ap_mask_to_tiles(mask.cuda(), tiles)
    out = torch.full_like(q, float("nan")).cuda()
    for _ in range(3):  # the race, if there were one, would not show on every launch
        out.fill_(float("nan"))
        ap.ap_sparse_attention_fwd(q.cuda(), k.cuda(), v.cuda(), tiles, out)
        assert ap.ap_device_status() == ap.AP_OK
        assert not torch.isnan(out).any()
    ref = orc.attention_fwd(inputs.widen(q), inputs.widen(k), inputs.widen(v), mask.numpy())
    # (a million rows, the first of each head with one or two kept entries: |O| reaches the largest single
    # values of V, whose bf16 rounding alone exceeds the fixed absolute bound; so bound by value as well)
    got = out.float().cpu().numpy()
    np.testing.assert_allclose(got, ref, rtol=2.0 ** -8, atol=6e-3)
    assert np.linalg.norm(got - ref) / np.linalg.norm(ref) <= pu.TOL["bf16"]["rel_l2"]


# ---- the same attention with the 1.5-entmax normaliser


def _entmax_fwd_case(ap, w, mask: torch.Tensor, scale=0.0):
    q, k, v = inputs.eval_qkv(w)
    tiles = ap.Tiles(w.H, w.Lq, w.Lk)
    ap.ap_mask_to_tiles(mask.cuda(), tiles)
    out = torch.full_like(q, 3.0).cuda()          # poison: every element must be written
    ap.ap_sparse_attention_entmax15_fwd(q.cuda(), k.cuda(), v.cuda(), tiles, out, scale=scale)
    assert ap.ap_device_status() == ap.AP_OK
    ref = orc.attention_entmax15_fwd(inputs.widen(q), inputs.widen(k), inputs.widen(v), mask.numpy(),
                                     scale=None if scale == 0.0 else scale)
    # Sparse rows average few rows of V, so |O| reaches the size of single values of V (up to 4 and more):
    # the output's own rounding (half an ulp: 2^-9 |O| in bf16, 2^-12 |O| in fp16) no longer fits under a fixed
    # absolute bound.  Bound: that rounding plus the absolute part of the softmax path's tolerance.
    got = out.float().cpu().numpy()
    # fp32 tensors: no rounding of weights or output; the threshold is within 5e-7 max(1, |tau|) of the root
    # and a row's weights move by 2 S1 dtau in total, S1 a few units: 2e-5 absolute
    rtol, atol = {"bf16": (2.0 ** -8, 6e-3), "f16": (2.0 ** -11, 1.5e-3), "f32": (1e-5, 2e-5)}[w.dtype]
    np.testing.assert_allclose(got, ref, rtol=rtol, atol=atol)
    rel_l2 = float(np.linalg.norm(got - ref) / max(np.linalg.norm(ref), 1e-30))
    assert rel_l2 <= (1e-5 if w.dtype == "f32" else pu.TOL[w.dtype]["rel_l2"]), (w.name, rel_l2)
    return out, ref


@pytest.mark.parametrize("dtype", ["bf16", "f16", "f32"])
@pytest.mark.parametrize("d", [64, 128])
@pytest.mark.parametrize("shape", [(2, 2, 128, 128), (1, 2, 200, 333), (2, 1, 513, 130), (1, 1, 5, 7),
                                   (1, 2, 384, 1200)])
def test_entmax_forward_random_masks_ragged_shapes(ap, shape, d, dtype):
    B, H, Lq, Lk = shape
    w = W["tiny"].scaled(B=B, H=H, Lq=Lq, Lk=Lk, d=d, dtype=dtype)
    mask = inputs.random_mask(H, Lq, Lk, 0.15, seed=81, empty_rows=(0, Lq - 1) if Lq > 2 else ())
    mask[0, : min(128, Lq), : min(128, Lk)] = 1   # a fully kept (or edge-full) tile next to partial ones
    if Lq > 256:
        mask[H - 1, 128:256] = 0                   # a query tile with no kept tile at all
    out, _ = _entmax_fwd_case(ap, w, mask)
    o = out.float().cpu().numpy()
    empty = mask.numpy().sum(-1) == 0
    assert np.all(o[:, empty] == 0.0)


def test_entmax_forward_closed_forms_and_scale(ap):
    """One kept entry per row: the output is that row of V, bit for bit.  Everything kept and Q = 0: the mean of
    V.  A sharp custom scale: rows close to one-hot."""
    w = W["tiny"].scaled(B=1, H=2, Lq=256, Lk=256, d=64, dtype="bf16")
    q, k, v = inputs.eval_qkv(w)
    cols = torch.randint(0, w.Lk, (w.H, w.Lq), generator=torch.Generator().manual_seed(9))
    mask = torch.zeros((w.H, w.Lq, w.Lk), dtype=torch.uint8)
    mask.scatter_(2, cols[..., None], 1)
    tiles = ap.Tiles(w.H, w.Lq, w.Lk)
    ap.ap_mask_to_tiles(mask.cuda(), tiles)
    out = ap.ap_sparse_attention_entmax15_fwd(q.cuda(), k.cuda(), v.cuda(), tiles).cpu()
    want = torch.gather(v, 2, cols[None, ..., None].expand(1, w.H, w.Lq, w.d))
    assert torch.equal(out, want)
    ones = torch.ones_like(mask)
    ap.ap_mask_to_tiles(ones.cuda(), tiles)
    out = ap.ap_sparse_attention_entmax15_fwd(torch.zeros_like(q).cuda(), k.cuda(), v.cuda(), tiles).float().cpu()
    mean = v.float().mean(2, keepdim=True).expand_as(out)
    assert float((out - mean).abs().max()) <= 1e-2
    for scale in (0.02, 2.0):
        _entmax_fwd_case(ap, w, inputs.random_mask(w.H, w.Lq, w.Lk, 0.3, seed=5), scale=scale)


@pytest.mark.parametrize("d", [64, 128])
@pytest.mark.parametrize("case", [
    # (B, H, Lq, Lk, group_frac, fill, full_tile_frac, causal)
    (2, 2, 256, 1024, 0.10, 0.30, 0.00, False),   # few active groups per tile: lists pack 8 tiles into ~1
    (1, 2, 300, 1000, 0.25, 0.05, 0.10, False),   # partial tiles mixed with fully kept ones; Lk % 128 != 0
    (1, 2, 640, 640, 0.30, 0.50, 0.00, True),     # causal: lists of 1..5 tiles, packed and tile by tile
    (1, 1, 128, 2052, 0.05, 0.90, 0.00, False),   # 17 key tiles, a last tile of 4 columns; Lk % 8 != 0
    (2, 1, 200, 777, 0.50, 0.02, 0.20, False),    # odd sizes; rows >= Lq in the last query tile
    (1, 1, 128, 1536, 1.00, 0.02, 0.00, False),   # every group active (nothing to pack away)
])
def test_forward_group_sparse_masks(ap, case, d):
    """Masks whose tiles hold few non-empty 16-column groups: the forward packs the groups of
    several key tiles into one tile; runs of neighbouring groups, lone groups, fully kept tiles
    and ragged edges all occur."""
    B, H, Lq, Lk, group_frac, fill, full_frac, causal = case
    w = W["tiny"].scaled(B=B, H=H, Lq=Lq, Lk=Lk, d=d, dtype="bf16")
    mask = inputs.group_sparse_mask(H, Lq, Lk, group_frac, fill, seed=90 + Lk, full_tile_frac=full_frac,
                                    causal=causal)
    assert mask.any()
    out, _ = _fwd_case(ap, w, mask)
    empty = mask.numpy().sum(-1) == 0
    assert np.all(out.float().cpu().numpy()[:, empty] == 0.0)


def test_forward_long_list_beyond_the_packing_plan(ap):
    """A list of more key tiles than the packing plan holds (128) is processed tile by tile."""
    H, Lq, Lk = 1, 128, 129 * 128 + 40
    w = W["tiny"].scaled(B=1, H=H, Lq=Lq, Lk=Lk, d=64, dtype="bf16")
    mask = inputs.group_sparse_mask(H, Lq, Lk, 0.2, 0.2, seed=93)
    mask[:, :, ::128] = 1  # every key tile is in the list
    _fwd_case(ap, w, mask)


def test_forward_custom_scale(ap):
    w = W["tiny"].scaled(B=1, H=2, Lq=150, Lk=150, dtype="bf16")
    _fwd_case(ap, w, inputs.random_mask(2, 150, 150, 0.3, seed=81), scale=0.31)


@pytest.mark.parametrize("dtype", ["f32", "bf16", "f16"])
@pytest.mark.parametrize("causal", [False, True])
@pytest.mark.parametrize("L", [(300, 300), (200, 456)])
def test_forward_dense_tiles_equal_unpruned_attention(ap, dtype, causal, L):
    w = W["tiny"].scaled(B=2, H=2, Lq=L[0], Lk=L[1], dtype=dtype)
    q, k, v = inputs.eval_qkv(w)
    tiles = ap.Tiles(w.H, w.Lq, w.Lk)
    ap.ap_dense_tiles(tiles, causal=causal)
    out = ap.ap_sparse_attention_fwd(q.cuda(), k.cuda(), v.cuda(), tiles)
    dom = torch.ones((w.H, w.Lq, w.Lk), dtype=torch.uint8)
    if causal:
        dom = torch.tril(dom, diagonal=w.Lk - w.Lq)
    ref = orc.attention_fwd(inputs.widen(q), inputs.widen(k), inputs.widen(v), dom.numpy())
    pu.assert_close_attention(out, ref, dtype)


def test_forward_single_kept_entry_copies_value_rows_exactly(ap):
    w = W["bert"].scaled(B=2, H=2, Lq=260, Lk=260)
    q, k, v = inputs.eval_qkv(w)
    eye = torch.eye(260, dtype=torch.uint8).expand(2, 260, 260).contiguous()
    tiles = ap.Tiles(2, 260, 260)
    ap.ap_mask_to_tiles(eye.cuda(), tiles)
    out = ap.ap_sparse_attention_fwd(q.cuda(), k.cuda(), v.cuda(), tiles)
    assert torch.equal(out.cpu(), v)


# ------------------------------------------------------------------------------ backward


def _rel_l2(got, ref):
    return float(np.linalg.norm(got.astype(np.float64) - ref) / max(np.linalg.norm(ref), 1e-300))


def _bwd_case(ap, w, mask: torch.Tensor, tol):
    """dQ, dK, dV of the masked attention against the oracle's derivative, for dO ~ N(0,1)."""
    q, k, v = inputs.eval_qkv(w)
    g = torch.Generator().manual_seed(w.seed0 + 77)
    d_o = torch.randn(q.shape, generator=g).to(q.dtype)
    tiles = ap.Tiles(w.H, w.Lq, w.Lk)
    ap.ap_mask_to_tiles(mask.cuda(), tiles)
    out = ap.ap_sparse_attention_fwd(q.cuda(), k.cuda(), v.cuda(), tiles)
    poison = [torch.full_like(t, float("nan"), device="cuda") for t in (q, k, v)]
    dq, dk, dv = ap.ap_sparse_attention_bwd(q.cuda(), k.cuda(), v.cuda(), out, d_o.cuda(), tiles, *poison)
    assert ap.ap_device_status() == ap.AP_OK
    again = ap.ap_sparse_attention_bwd(q.cuda(), k.cuda(), v.cuda(), out, d_o.cuda(), tiles)
    assert all(torch.equal(a, b) for a, b in zip((dq, dk, dv), again))      # no atomics: bit-reproducible
    want = orc.attention_bwd(inputs.widen(q), inputs.widen(k), inputs.widen(v), inputs.widen(d_o), mask.numpy())
    # element by element: |got - ref| <= rtol |ref| + atol, atol from the rounding model of the kernel
    ulp = 2.0 ** -8 if tol >= 1e-2 else 2.0 ** -11
    bounds = pu.backward_bounds(inputs.widen(q), inputs.widen(k), inputs.widen(v), inputs.widen(d_o), mask.numpy(), ulp,
                                tiny=0.0 if tol >= 1e-2 else 2.0 ** -24)
    dense_rows = mask.numpy().sum(-1) >= 8            # [H, Lq]: rows that keep at least eight entries
    for name, got, ref, atol in zip(("dQ", "dK", "dV"), (dq, dk, dv), want, bounds):
        got = got.float().cpu().numpy()
        assert np.isfinite(got).all(), name
        excess = np.abs(got.astype(np.float64) - ref) - (2.0 * ulp * np.abs(ref) + 2.0 * atol)
        assert excess.max() <= 0.0, (name, float(excess.max()), np.unravel_index(int(excess.argmax()), excess.shape))
        if name == "dQ" and dense_rows.any():
            # rows whose weight is spread need no floor: plain relative error in the L2 norm
            sel = np.broadcast_to(dense_rows[None, :, :, None], ref.shape)
            err = np.linalg.norm((got.astype(np.float64) - ref)[sel]) / max(np.linalg.norm(ref[sel]), 1e-300)
            assert err <= tol, (name, "rows with >= 8 kept entries", float(err))
        if name == "dV":
            # no D in dV: plain relative error in the L2 norm over everything
            err = _rel_l2(got, ref)
            assert err <= tol, (name, float(err))
    return dq, dk, dv


@pytest.mark.parametrize("dtype,tol", [("bf16", 1e-2), ("f16", 2e-3)])
@pytest.mark.parametrize("d", [64, 128])
@pytest.mark.parametrize("shape", [(2, 2, 128, 128), (1, 2, 200, 333), (2, 1, 513, 130), (1, 1, 5, 7)])
def test_backward_random_masks_ragged_shapes(ap, shape, d, dtype, tol):
    B, H, Lq, Lk = shape
    w = W["tiny"].scaled(B=B, H=H, Lq=Lq, Lk=Lk, d=d, dtype=dtype)
    mask = inputs.random_mask(H, Lq, Lk, 0.3, seed=95, empty_rows=(1,) if Lq > 1 else ())
    dq, _, _ = _bwd_case(ap, w, mask, tol)
    if Lq > 1:
        assert torch.all(dq[:, :, 1] == 0)               # a row without kept entries passes no gradient


def test_backward_causal_band_and_absent_tiles(ap):
    """A causal band: most (query tile, key tile) pairs are not in the list; key tiles that no
    query tile keeps get zero gradients."""
    H, L = 2, 640
    i = torch.arange(L)[:, None]
    j = torch.arange(L)[None, :]
    mask = ((j <= i) & (i - j < 100)).to(torch.uint8).expand(H, L, L).contiguous().clone()
    mask[1, :, 512:] = 0                                 # head 1 never looks at the last key tile
    w = W["tiny"].scaled(B=2, H=H, Lq=L, Lk=L, d=128, dtype="bf16")
    _, dk, dv = _bwd_case(ap, w, mask, 1e-2)
    assert torch.all(dk[:, 1, 512:] == 0) and torch.all(dv[:, 1, 512:] == 0)


def test_backward_more_query_tiles_than_the_staged_lookup_holds(ap):
    """A key tile's column of the (query tile, key tile) table is staged for 256 query tiles; beyond
    that the columns kernel reads the table directly."""
    H, Lq, Lk = 1, 260 * 128 + 17, 200
    w = W["tiny"].scaled(B=1, H=H, Lq=Lq, Lk=Lk, d=64, dtype="bf16")
    mask = inputs.random_mask(H, Lq, Lk, 0.05, seed=96)
    mask[:, 258 * 128:, :] = 0
    mask[:, 259 * 128 + 3, 150] = 1            # a lone stored tile far beyond the staged part
    _bwd_case(ap, w, mask, 1e-2)


def test_backward_long_full_size(ap):
    """The long workload at full size under its own calibrated mask (the configuration the benchmark
    times): all of dQ, dK, dV against the oracle's derivative."""
    w = W["long"]
    bias = inputs.calib_bias(w).cuda()
    acc = pu.gpu_accumulate(ap, w, 2, bias)
    del bias
    mask, tiles, _ = pu.gpu_build_mask(ap, acc, w)
    del acc
    q, k, v = inputs.eval_qkv(w)
    g = torch.Generator().manual_seed(w.seed0 + 77)
    d_o = torch.randn(q.shape, generator=g).to(q.dtype)
    out = ap.ap_sparse_attention_fwd(q.cuda(), k.cuda(), v.cuda(), tiles)
    dq, dk, dv = ap.ap_sparse_attention_bwd(q.cuda(), k.cuda(), v.cuda(), out, d_o.cuda(), tiles)
    assert ap.ap_device_status() == ap.AP_OK
    want = orc.attention_bwd(inputs.widen(q), inputs.widen(k), inputs.widen(v), inputs.widen(d_o),
                             mask.cpu().numpy())
    for name, got, ref in zip(("dQ", "dK", "dV"), (dq, dk, dv), want):
        err = _rel_l2(got.float().cpu().numpy(), ref)
        assert err <= 1e-2, (name, err)


# -------------------------------------------------------------------------- seeded sweeps


def test_seeded_sweep_of_small_shapes(ap):
    """Forty seeded random configurations (shape, domain, fraction, value distribution, dtype, density):
    mask builders bit for bit, forward and backward within their tolerances.  Shapes stay small so
    that the oracle finishes at once; they straddle tile edges (1..300 rows and columns)."""
    rng = np.random.default_rng(2024)
    for case in range(40):
        H = int(rng.integers(1, 4))
        Lq = int(rng.integers(1, 301))
        causal = bool(rng.integers(0, 2))
        Lk = Lq + int(rng.integers(0, 200)) * int(rng.integers(0, 2)) if causal else int(rng.integers(1, 301))
        keep_diag = bool(rng.integers(0, 2))
        keep = float(rng.choice([0.01, 0.07, 0.3, 0.5, 0.93, 1.0]))
        acc = rng.random((H, Lq, Lk), dtype=np.float32)
        kind = int(rng.integers(0, 3))
        if kind == 1:
            acc = np.round(acc * 5) / 5                      # six distinct values
        elif kind == 2:
            acc[:] = 0.5                                     # one value
        w = W["tiny"].scaled(H=H, Lq=Lq, Lk=Lk, causal=causal, keep_diag=keep_diag, keep_frac=keep)
        want = _check_build_mask(ap, acc, w, layer=bool(rng.integers(0, 2)))
        d = int(rng.choice([64, 128]))
        dtype = str(rng.choice(["bf16", "f16"]))
        B = int(rng.integers(1, 3))
        wf = w.scaled(B=B, d=d, dtype=dtype, seed0=w.seed0 + case)
        mask = torch.from_numpy(want.copy())
        _fwd_case(ap, wf, mask)
        _bwd_case(ap, wf, mask, 1e-2 if dtype == "bf16" else 2e-3)


def test_seeded_sweep_of_accumulate_and_tile_lists(ap):
    """Thirty seeded random configurations of the calibration sum (shape, domain, dtype, bias or not,
    one to nine samples) and of the tile-list builders on random masks of random density."""
    rng = np.random.default_rng(2025)
    for case in range(30):
        H = int(rng.integers(1, 4))
        Lq = int(rng.integers(1, 301))
        causal = bool(rng.integers(0, 2))
        Lk = Lq + int(rng.integers(0, 200)) * int(rng.integers(0, 2)) if causal else int(rng.integers(1, 301))
        d = int(rng.choice([64, 128]))
        dtype = str(rng.choice(["bf16", "f16", "f32"]))
        B = int(rng.integers(1, 10))
        w = W["tiny"].scaled(B=B, H=H, Lq=Lq, Lk=Lk, d=d, dtype=dtype, causal=causal, seed0=7000 + case)
        bias = None
        if rng.integers(0, 2):
            g = torch.Generator().manual_seed(7100 + case)
            bias = torch.randn((H, Lq, Lk), generator=g)
        acc = pu.gpu_accumulate(ap, w, 1, None if bias is None else bias.cuda())
        want = pu.oracle_accumulate(w, 1, bias)
        np.testing.assert_allclose(acc.cpu().numpy(), want, rtol=2e-5, atol=1e-7 * B, err_msg=str(w))
        density = float(rng.choice([0.0, 0.02, 0.3, 0.9, 1.0]))
        mask = inputs.random_mask(H, Lq, Lk, density, seed=7200 + case, causal=causal)
        tiles = ap.Tiles(H, Lq, Lk)
        ap.ap_mask_to_tiles(mask.cuda(), tiles)
        assert ap.ap_device_status() == ap.AP_OK
        pu.assert_tiles_equal(tiles.to_host(), orc.mask_to_tiles(mask.numpy()))
        dense = ap.Tiles(H, Lq, Lk)
        ap.ap_dense_tiles(dense, causal=causal)
        dom = torch.ones((H, Lq, Lk), dtype=torch.uint8)
        if causal:
            dom = torch.tril(dom, diagonal=Lk - Lq)
        pu.assert_tiles_equal(dense.to_host(), orc.mask_to_tiles(dom.numpy()))


# ------------------------------------------------------------------- the five workloads


def _pipeline(ap, w, n_batches, oracle_acc=True):
    """accumulate -> build mask -> forward on the GPU; stage-exact mask check on the
    GPU's own accumulator bits; forward against the oracle under the GPU-built mask."""
    bias = inputs.calib_bias(w)
    acc = pu.gpu_accumulate(ap, w, n_batches, bias.cuda())
    acc_host = acc.cpu().numpy()
    if oracle_acc:
        want_acc = pu.oracle_accumulate(w, n_batches, bias)
        np.testing.assert_allclose(acc_host, want_acc, rtol=2e-5, atol=1e-7 * n_batches * w.B)
    mask, tiles, nnz = pu.gpu_build_mask(ap, acc, w)
    want_mask, want_nnz = orc.build_mask(acc_host, w.keep_frac, w.causal, w.keep_diag)
    np.testing.assert_array_equal(mask.cpu().numpy(), want_mask)
    np.testing.assert_array_equal(nnz.cpu().numpy(), want_nnz)
    pu.assert_tiles_equal(tiles.to_host(), orc.mask_to_tiles(want_mask))
    k = orc.keep_count(w.n_valid, w.n_forced, w.keep_frac)
    assert np.all(want_nnz == k)                       # kept fraction exact per head
    if oracle_acc:
        # pure-oracle pipeline: masks may differ only where the average sits at the threshold
        pure_mask, _ = orc.build_mask(want_acc.astype(np.float32), w.keep_frac, w.causal, w.keep_diag)
        differ = pure_mask != want_mask
        if differ.any():
            for h in range(w.H):
                forced = np.eye(w.Lq, w.Lk, dtype=bool) if w.n_forced else np.zeros((w.Lq, w.Lk), dtype=bool)
                kept = want_acc[h][pure_mask[h].astype(bool) & ~forced]
                tau = kept.min()
                assert np.all(np.abs(want_acc[h][differ[h]] - tau) <= 4e-5 * tau), h
    q, kk, v = inputs.eval_qkv(w)
    out = ap.ap_sparse_attention_fwd(q.cuda(), kk.cuda(), v.cuda(), tiles)
    assert ap.ap_device_status() == ap.AP_OK
    ref = orc.attention_fwd(inputs.widen(q), inputs.widen(kk), inputs.widen(v), want_mask)
    return pu.assert_close_attention(out, ref, w.dtype, w.name)


def _pipeline_entmax(ap, w, n_batches):
    """The procedure for a model normalised by 1.5-entmax: entmax average -> Eq. 2 on the GPU's own
    accumulator bits (stage-exact; the average is sparse, so zeros tie in great numbers and the
    threshold may be 0) -> entmax forward under that mask against the oracle."""
    bias = inputs.calib_bias(w)
    acc = _entmax_acc(ap, w, n_batches, bias.cuda())
    acc_host = acc.cpu().numpy()
    np.testing.assert_allclose(acc_host, _entmax_want(w, n_batches, bias), rtol=ENTMAX_RTOL,
                               atol=ENTMAX_ATOL * n_batches * w.B)
    for layer in (False, True):
        mask, tiles, nnz = pu.gpu_build_mask(ap, acc, w, layer=layer)
        want_mask, want_nnz = (orc.build_mask_layer if layer else orc.build_mask)(acc_host, w.keep_frac, w.causal,
                                                                                   w.keep_diag)
        np.testing.assert_array_equal(mask.cpu().numpy(), want_mask)
        np.testing.assert_array_equal(nnz.cpu().numpy(), want_nnz)
        pu.assert_tiles_equal(tiles.to_host(), orc.mask_to_tiles(want_mask))
    return _entmax_fwd_case(ap, w, torch.from_numpy(want_mask))


@pytest.mark.parametrize("name,over,n_batches", [
    ("bert", dict(B=4, H=3), 2),
    ("lm", dict(B=2, H=2, Lq=300, Lk=300), 2),
    ("s2s_cross", dict(B=3, H=2, dtype="f16"), 2),
    ("tiny", dict(keep_frac=0.6), 2),            # fp32; keeps more than the average's support: the threshold is 0
    ("long", dict(B=1, H=2, Lq=640, Lk=640), 2),
])
def test_workload_with_entmax_normaliser(ap, name, over, n_batches):
    _pipeline_entmax(ap, W[name].scaled(**over), n_batches)


def test_workload_tiny_full(ap):
    _pipeline(ap, W["tiny"], W["tiny"].calib_batches)


@pytest.mark.parametrize("name", ["bert", "lm", "s2s_self", "s2s_cross", "txl"])
def test_workload_full_shape_configured_calibration(ap, name):
    """Full evaluation shape and the workload's own number of calibration batches (64, 64, 64, 64,
    16): the fp32 sum of up to 4096 samples per entry against the oracle's fp64 sum, the mask on
    the GPU's own accumulator bits, the end-to-end band rule, the forward."""
    _pipeline(ap, W[name], W[name].calib_batches)


@pytest.mark.parametrize("name", ["s2s_self", "s2s_cross"])
def test_workload_seq2seq_in_half_precision(ap, name):
    """The translation experiments run in fp16: the same recipe with fp16 tensors, end to end."""
    _pipeline(ap, W[name].scaled(B=8, dtype="f16"), 2)


def test_workload_long_reduced(ap):
    """The long-context recipe at L = 1024 (8x8 tiles, causal, d = 128), end to end."""
    _pipeline(ap, W["long"].scaled(B=2, H=4, Lq=1024, Lk=1024), 2)


@pytest.mark.parametrize("name", ["long", "llama"])
def test_workload_long_full_size_two_calibration_batches(ap, name):
    """Full size (long: B4 H16 L4096 d128; llama: the same context with B1 H32), calibrated on 2 of
    the 16 batches (the oracle's fp64 average of all 16 would take minutes): sampled accumulator rows,
    then EVERY head's mask bit for bit, the tile list, and EVERY output row against the oracle."""
    w = W[name]
    n_batches = 2
    bias = inputs.calib_bias(w)
    bias_dev = bias.cuda()
    acc = pu.gpu_accumulate(ap, w, n_batches, bias_dev)
    rng = np.random.default_rng(90)
    rows = [(int(h), int(i)) for h, i in zip(rng.integers(0, w.H, 48), rng.integers(0, w.Lq, 48))]
    rows += [(0, 0), (w.H - 1, w.Lq - 1), (3, 127), (3, 128)]
    want_rows = np.zeros((len(rows), w.Lk))
    for t in range(n_batches):
        q, k = inputs.calib_qk(w, t)
        want_rows += orc.accumulate_rows(rows, inputs.widen(q), inputs.widen(k), bias.numpy(), causal=True)
    got_rows = np.stack([acc[h, i].cpu().numpy() for h, i in rows])
    np.testing.assert_allclose(got_rows, want_rows, rtol=2e-5, atol=1e-7 * n_batches * w.B)
    del bias_dev

    mask, tiles, nnz = pu.gpu_build_mask(ap, acc, w)
    k = orc.keep_count(w.n_valid, w.n_forced, w.keep_frac)
    assert k == 419533 and torch.all(nnz == k)
    assert torch.all(mask.view(w.H, -1).sum(-1, dtype=torch.int64) == k)
    host_tiles = tiles.to_host()
    pop = np.unpackbits(host_tiles["bitmap"].view(np.uint8)).sum()
    assert pop == k * w.H
    mask_host = mask.cpu().numpy()
    for h0 in range(0, w.H, 4):       # four heads at a time keeps the host copies small
        want_mask, want_nnz = orc.build_mask(acc[h0:h0 + 4].cpu().numpy(), w.keep_frac, True, True)
        np.testing.assert_array_equal(mask_host[h0:h0 + 4], want_mask, err_msg="heads %d.." % h0)
        assert np.all(want_nnz == k)
    del acc
    pu.assert_tiles_equal(host_tiles, orc.mask_to_tiles(mask_host))

    q, kk, v = inputs.eval_qkv(w)
    out = ap.ap_sparse_attention_fwd(q.cuda(), kk.cuda(), v.cuda(), tiles)
    assert ap.ap_device_status() == ap.AP_OK
    ref = orc.attention_fwd(inputs.widen(q), inputs.widen(kk), inputs.widen(v), mask_host)
    pu.assert_close_attention(out, ref, "bf16", name + "/every row")


def test_host_buffer_entry_point(ap):
    w = W["bert"].scaled(B=2, H=2)
    q, k, v = (t.pin_memory() for t in inputs.eval_qkv(w))
    mask = inputs.random_mask(w.H, w.Lq, w.Lk, 0.5, seed=91)
    tiles = ap.Tiles(w.H, w.Lq, w.Lk)
    ap.ap_mask_to_tiles(mask.cuda(), tiles)
    ho = torch.empty_like(q).pin_memory()
    dq, dk, dv, do = (torch.empty_like(t, device="cuda") for t in (q, k, v, q))
    ap.ap_sparse_attention_fwd_host(q, k, v, tiles, ho, dq, dk, dv, do)
    assert ap.ap_device_status() == ap.AP_OK
    ref = orc.attention_fwd(inputs.widen(q), inputs.widen(k), inputs.widen(v), mask.numpy())
    pu.assert_close_attention(ho, ref, "bf16")


def test_host_buffer_entry_point_pipelines_batch_chunks(ap):
    """More batch elements than chunks (11 -> 6 chunks of 2, the last of 1), two calls back to back on the
    same staging buffers: each result equals the device-tensor call bit for bit (batch elements are
    independent), and the second call's input copies wait for the first call's kernels."""
    w = W["bert"].scaled(B=11, H=2, Lq=200, Lk=200)
    mask = inputs.random_mask(w.H, w.Lq, w.Lk, 0.3, seed=92)
    tiles = ap.Tiles(w.H, w.Lq, w.Lk)
    ap.ap_mask_to_tiles(mask.cuda(), tiles)
    q, k, v = (t.pin_memory() for t in inputs.eval_qkv(w))
    q2, k2, v2 = (t.pin_memory() for t in inputs.eval_qkv(w.scaled(seed0=w.seed0 + 5)))
    ho, ho2 = torch.empty_like(q).pin_memory(), torch.empty_like(q).pin_memory()
    dq, dk, dv, do = (torch.empty_like(t, device="cuda") for t in (q, k, v, q))
    ap.ap_sparse_attention_fwd_host(q, k, v, tiles, ho, dq, dk, dv, do)
    ap.ap_sparse_attention_fwd_host(q2, k2, v2, tiles, ho2, dq, dk, dv, do)
    torch.cuda.current_stream().synchronize()      # the caller's stream is all there is to wait for
    assert ap.ap_device_status() == ap.AP_OK
    want = ap.ap_sparse_attention_fwd(q.cuda(), k.cuda(), v.cuda(), tiles).cpu()
    want2 = ap.ap_sparse_attention_fwd(q2.cuda(), k2.cuda(), v2.cuda(), tiles).cpu()
    assert torch.equal(ho, want) and torch.equal(ho2, want2)
    assert not torch.equal(ho, ho2)

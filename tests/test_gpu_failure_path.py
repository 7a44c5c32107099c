"""The bounded waits of the tensor-core kernels, exercised without faulting or hanging anything.

ap_debug_expire_waits(1) makes the next launches run on one thread block with a short poll limit
and leave out one producer arrival: a wait runs out, the kernel must return by itself with the
device status word raised, and the library must work normally afterwards.
"""
import numpy as np
import pytest
import torch

from oracle import ap_oracle as orc
from paper_2012_02030_b200 import inputs
from tests.parity_util import assert_close_attention


@pytest.mark.gpu
@pytest.mark.parametrize("d", [64, 128])
def test_forward_expired_wait_returns_timeout_once_and_the_next_call_is_correct(d):
    from paper_2012_02030_b200 import binding as ap

    B, H, L = 1, 2, 256
    gen = torch.Generator().manual_seed(4100 + d)
    q, k, v = (torch.randn((B, H, L, d), generator=gen).to(torch.bfloat16) for _ in range(3))
    mask = inputs.random_mask(H, L, L, 0.3, seed=77, causal=True)
    tiles = ap.Tiles(H, L, L)
    ap.ap_mask_to_tiles(mask.cuda(), tiles)
    assert ap.ap_device_status() == ap.AP_OK
    qd, kd, vd = q.cuda(), k.cuda(), v.cuda()
    ap.ap_debug_expire_waits(True)
    try:
        ap.ap_sparse_attention_fwd(qd, kd, vd, tiles)          # returns by itself: every wait is bounded
        assert ap.ap_device_status() == ap.AP_ERR_TIMEOUT      # raised once ...
    finally:
        ap.ap_debug_expire_waits(False)
    assert ap.ap_device_status() == ap.AP_OK                   # ... and cleared by the read
    out = ap.ap_sparse_attention_fwd(qd, kd, vd, tiles)        # tensor memory was freed, barriers are fresh
    assert ap.ap_device_status() == ap.AP_OK
    ref = orc.attention_fwd(inputs.widen(q), inputs.widen(k), inputs.widen(v), mask.numpy())
    assert_close_attention(out, ref, "bf16", "after an expired wait")


@pytest.mark.gpu
@pytest.mark.parametrize("d", [64, 128])
def test_accumulate_expired_wait_returns_timeout_once_and_the_next_call_is_correct(d):
    from paper_2012_02030_b200 import binding as ap

    B, H, L = 2, 2, 256
    gen = torch.Generator().manual_seed(4200 + d)
    q, k = (torch.randn((B, H, L, d), generator=gen).to(torch.bfloat16) for _ in range(2))
    bias = 0.5 * torch.randn((H, L, L), generator=gen)
    qd, kd, bd = q.cuda(), k.cuda(), bias.cuda()
    scratch = torch.zeros((H, L, L), device="cuda")
    assert ap.ap_device_status() == ap.AP_OK
    ap.ap_debug_expire_waits(True)
    try:
        ap.ap_accumulate_attention(scratch, qd, kd, bd, causal=True)   # the first visit's operands never arrive
        assert ap.ap_device_status() == ap.AP_ERR_TIMEOUT
    finally:
        ap.ap_debug_expire_waits(False)
    assert ap.ap_device_status() == ap.AP_OK
    acc = torch.zeros((H, L, L), device="cuda")
    ap.ap_accumulate_attention(acc, qd, kd, bd, causal=True)
    assert ap.ap_device_status() == ap.AP_OK
    want = np.zeros((H, L, L))
    orc.accumulate(want, inputs.widen(q), inputs.widen(k), bias.numpy(), causal=True)
    np.testing.assert_allclose(acc.cpu().numpy(), want, rtol=2e-5, atol=1e-7 * B)


@pytest.mark.gpu
@pytest.mark.parametrize("d", [64, 128])
def test_backward_expired_wait_returns_timeout_once_and_the_next_call_is_correct(d):
    from paper_2012_02030_b200 import binding as ap
    from tests import parity_util as pu

    B, H, L = 1, 2, 256
    gen = torch.Generator().manual_seed(4300 + d)
    q, k, v, d_o = (torch.randn((B, H, L, d), generator=gen).to(torch.bfloat16) for _ in range(4))
    mask = inputs.random_mask(H, L, L, 0.3, seed=78, causal=True)
    tiles = ap.Tiles(H, L, L)
    ap.ap_mask_to_tiles(mask.cuda(), tiles)
    qd, kd, vd, dod = q.cuda(), k.cuda(), v.cuda(), d_o.cuda()
    out = ap.ap_sparse_attention_fwd(qd, kd, vd, tiles)
    assert ap.ap_device_status() == ap.AP_OK
    ap.ap_debug_expire_waits(True)
    try:
        ap.ap_sparse_attention_bwd(qd, kd, vd, out, dod, tiles)    # both kernels' first waits run out
        assert ap.ap_device_status() == ap.AP_ERR_TIMEOUT
    finally:
        ap.ap_debug_expire_waits(False)
    assert ap.ap_device_status() == ap.AP_OK
    dq, dk, dv = ap.ap_sparse_attention_bwd(qd, kd, vd, out, dod, tiles)
    assert ap.ap_device_status() == ap.AP_OK
    ref = orc.attention_bwd(inputs.widen(q), inputs.widen(k), inputs.widen(v), inputs.widen(d_o), mask.numpy())
    for got, want, name in zip((dq, dk, dv), ref, ("dQ", "dK", "dV")):
        err = np.linalg.norm(got.float().cpu().numpy() - want) / np.linalg.norm(want)
        assert err < 1e-2, (name, err)

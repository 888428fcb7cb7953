"""Boundary behaviour on the device: recovery from a failed stage, many workers, and the bounded
wait of the bulk-copy kernels running out (flagged in the status word, no fault, no hang)."""
import numpy as np
import pytest
import torch

import oracle
from gpu_helpers import Pair, f32, u32, widen
from liec_synth import make_gradients, ragged_layout, random_subsets, topk_counts
from paper_2402_11857_b200 import liec

pytestmark = pytest.mark.gpu

SIGN, IDENT, TOPK, RANDK = liec.COMP_SCALED_SIGN, liec.COMP_IDENTITY, liec.COMP_TOPK, liec.COMP_RANDK


def test_failed_stage_inside_step_leaves_the_context_usable():
    """A random-k downlink without a subset fails in the third stage of liec_step; the context must
    return to idle, and a later iteration (state restored, subset given) matches the oracle."""
    lay = ragged_layout()
    k = topk_counts(lay, 1, 50)
    P = Pair(2, lay.seg_offsets, SIGN, RANDK, k=k)
    G = make_gradients("normal", 1.0, 2, lay.dim, 0, base_seed=71)
    Gd = G.cuda()
    with pytest.raises(liec.LiecError) as err:
        P.ctx.liec_step(Gd, 0.1)
    assert err.value.status == 4 and "subset" in str(err.value)
    torch.cuda.synchronize()
    # the uplink and the server pass did run: the error buffer holds v.  Restore and go on.
    P.ed.zero_()
    sets = random_subsets(lay.seg_offsets, k, 1, 0, 71)
    P.step(G, 0.1, down_set=sets[0])
    P.step(G, 0.1, down_set=sets[0], check_messages=False)


def test_abort_step_and_out_of_order_calls():
    lay = ragged_layout()
    P = Pair(2, lay.seg_offsets, SIGN, SIGN)
    G = make_gradients("normal", 1.0, 2, lay.dim, 0, base_seed=72)
    Gd = G.cuda()
    ctx = P.ctx
    ctx.liec_uplink_compress(Gd)
    for call in (lambda: ctx.liec_step(Gd, 0.1), lambda: ctx.liec_downlink_compress(),
                 lambda: ctx.liec_average_step(Gd, 0.1)):
        with pytest.raises(liec.LiecError) as err:
            call()
        assert err.value.status == 4
    # a host-fed step in the middle of an iteration is refused before any copy is enqueued
    Gh = torch.full_like(G, 7.0).pin_memory()
    with pytest.raises(liec.LiecError) as err:
        ctx.liec_step_host(Gh, Gd, 0.1)
    assert err.value.status == 4
    torch.cuda.synchronize()
    assert torch.equal(Gd.cpu(), G)
    ctx.liec_abort_step()
    torch.cuda.synchronize()
    P.step(G, 0.1)     # uplink only had run: params and error are untouched, the oracle still agrees


def test_three_thousand_workers_sign():
    """More workers than one staging chunk of scales in the server pass (1024)."""
    off = [0, 40, 40 + 8192 + 3]
    N = 3000
    P = Pair(N, off, SIGN, SIGN)
    for step in range(2):
        G = make_gradients("normal", 1.0, N, off[-1], step, base_seed=73)
        P.step(G, 0.1)


def _flagged_then_recovers(make_pair, G, lr):
    P = make_pair()
    ctx = P.ctx
    Gd = G.cuda()
    before = {k: (None if v is None or not torch.is_tensor(v) else v.clone()) for k, v in ctx.liec_get_messages().items()}
    ctx.liec_set_copy_wait(poll_limit=1000, expect_extra_bytes=16)
    ctx.liec_uplink_compress(Gd)
    torch.cuda.synchronize()
    status = ctx.liec_device_status()
    assert status & 8, status
    after = ctx.liec_get_messages()
    for name in ("up_words", "up_idx", "up_val"):
        if before[name] is not None:
            assert torch.equal(before[name], after[name]), name   # the flagged kernel left its outputs alone
    ctx.liec_abort_step()
    ctx.liec_set_copy_wait()          # defaults
    ctx.liec_clear_status()
    assert ctx.liec_device_status() == 0
    for step in range(2):
        P.step(G, lr)


def test_bulk_copy_wait_runs_out_sign_bf16():
    """One CTA (one full tile, one worker): the barrier is told to expect 16 bytes more than the copy
    delivers, so the bounded wait runs out; bit 8 is set, nothing is written, service resumes."""
    G = make_gradients("bf16_outliers", 1e-2, 1, 8192, 0, base_seed=74)
    _flagged_then_recovers(lambda: Pair(1, [0, 8192], SIGN, SIGN, grad_dtype=liec.BF16), G, 0.01)


def test_bulk_copy_wait_runs_out_sign_server_pass():
    """The sign server pass stages its tile of e by a bulk copy: when that wait runs out the pass sets
    bit 8 and leaves e and the downlink words alone; after abort + clear the next steps match the oracle."""
    off = [0, 2 * 8192, 2 * 8192 + 100]      # two full tiles (bulk copies) and a ragged one (guarded loads)
    P = Pair(2, off, SIGN, SIGN)
    P.step(make_gradients("normal", 1.0, 2, off[-1], 0, base_seed=79), 0.1)
    ctx = P.ctx
    G = make_gradients("normal", 1.0, 2, off[-1], 1, base_seed=79)
    Gd = G.cuda()
    ctx.liec_uplink_compress(Gd)
    torch.cuda.synchronize()
    e_before, words_before = P.ed.clone(), ctx.liec_get_messages()["down_words"].clone()
    ctx.liec_set_copy_wait(poll_limit=1000, expect_extra_bytes=16)
    ctx.liec_server_aggregate()
    torch.cuda.synchronize()
    assert ctx.liec_device_status() & 8
    assert torch.equal(P.ed[: 2 * 8192], e_before[: 2 * 8192])      # (the ragged tile has no bulk copy and is done)
    assert torch.equal(ctx.liec_get_messages()["down_words"][: 2 * 256], words_before[: 2 * 256])
    P.ed.copy_(e_before)                     # the state after a flagged iteration is the caller's to restore
    ctx.liec_abort_step()
    ctx.liec_set_copy_wait()
    ctx.liec_clear_status()
    assert ctx.liec_device_status() == 0
    for step in (1, 2):
        P.step(make_gradients("normal", 1.0, 2, off[-1], step, base_seed=79), 0.1)


def test_bulk_copy_wait_runs_out_topk_filter():
    """Two full tiles of one segment (a single-tile segment would be selected without any bulk copy)."""
    G = make_gradients("normal", 1.0, 1, 16384, 0, base_seed=75)
    _flagged_then_recovers(lambda: Pair(1, [0, 16384], TOPK, TOPK, k=[163]), G, 0.1)

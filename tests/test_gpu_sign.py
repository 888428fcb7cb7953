"""Scaled-sign and identity paths of the CUDA library against the CPU oracle (needs a B200)."""
import numpy as np
import pytest
import torch

import oracle
from liec_synth import (flat_layout, make_gradients, ragged_layout, resnet18_layout, scaled_layout,
                        gpt2_small_layout)
from paper_2402_11857_b200 import liec

pytestmark = pytest.mark.gpu

SIGN, IDENT = liec.COMP_SCALED_SIGN, liec.COMP_IDENTITY


def _pair(*a, **kw):
    from gpu_helpers import Pair
    return Pair(*a, **kw)


def test_config1_flat_sign_20_steps():
    """N=4, d=65,536, per-vector scaled sign both ways, lr 0.1, 20 steps."""
    lay = flat_layout(65536)
    P = _pair(4, lay.seg_offsets, SIGN, SIGN)
    for step in range(20):
        G = make_gradients("normal", 1.0, 4, lay.dim, step, base_seed=1)
        P.step(G, 0.1)


def test_ragged_segments_sign():
    """Tiles with tails, one-element and sub-word segments, several tiles per segment."""
    lay = ragged_layout()
    rng = np.random.default_rng(0)
    P = _pair(3, lay.seg_offsets, SIGN, SIGN, x0=rng.standard_normal(lay.dim), e0=0.1 * rng.standard_normal(lay.dim))
    for step in range(4):
        G = make_gradients("normal", 0.01, 3, lay.dim, step, base_seed=2)
        G[0, ::7] = 0.0
        G[1, 3::11] = -0.0
        P.step(G, 0.05)


def test_unaligned_rows_sign():
    """d odd: rows of workers 1.. start at addresses that are not 16-byte aligned."""
    off = [0, 5, 8192 + 5, 8192 + 5 + 33, 3 * 8192 + 1]
    P = _pair(3, off, SIGN, SIGN)
    for step in range(3):
        G = make_gradients("normal", 1.0, 3, off[-1], step, base_seed=3)
        P.step(G, 0.1)


def test_resnet18_scaled_layout_sign_many_steps():
    """ResNet-18 tensor list shrunk 16x (62 segments, N=8), per-tensor scales, 50 steps."""
    lay = scaled_layout(resnet18_layout(), 16)
    P = _pair(8, lay.seg_offsets, SIGN, SIGN)
    for step in range(50):
        G = make_gradients("normal", 0.01, 8, lay.dim, step, base_seed=4)
        P.step(G, 0.05, check_messages=(step % 10 == 0))


@pytest.mark.parametrize("blocks", [10, 18, 14])
def test_blockwise_equal_blocks(blocks):
    """Blockwise-SignSGD with the block counts of the paper's runs (10, 18, 14 equal blocks); the
    block boundaries fall at arbitrary offsets, not at multiples of 32 or of the tile."""
    from liec_synth import equal_blocks_layout
    lay = equal_blocks_layout(200_003, blocks)
    P = _pair(4, lay.seg_offsets, SIGN, SIGN)
    for step in range(3):
        G = make_gradients("normal", 0.01, 4, lay.dim, step, base_seed=40 + blocks)
        P.step(G, 0.1)


def test_step_from_host_memory_matches_device_step():
    """liec_step_host (gradients copied from pinned host memory, downlink message copied back)
    leaves the same state as liec_step and returns the message bytes that sit in the workspace."""
    lay = ragged_layout()
    N = 3
    outs = []
    for mode in ("device", "host"):
        X = torch.zeros(N, lay.dim, device="cuda"); e = torch.zeros(lay.dim, device="cuda")
        ctx = liec.Context(X, e, lay.seg_offsets, SIGN, SIGN)
        msg = torch.zeros(liec.down_message_bytes(ctx.cfg), dtype=torch.uint8).pin_memory()
        for step in range(3):
            G = make_gradients("normal", 1.0, N, lay.dim, step, base_seed=41)
            if mode == "device":
                ctx.liec_step(G.cuda(), 0.1)
            else:
                ctx.liec_step_host(G.pin_memory(), torch.empty_like(G, device="cuda"), 0.1, msg)
        torch.cuda.synchronize()
        m = ctx.liec_get_messages()
        outs.append((X.cpu(), e.cpu(), m["down_words"].cpu(), m["down_scales"].cpu(), msg.clone()))
    for a, b in zip(outs[0][:4], outs[1][:4]):
        assert torch.equal(a, b)
    words, scales, msg = outs[1][2], outs[1][3], outs[1][4]
    assert torch.equal(msg[: 4 * words.numel()].view(torch.int32), words)
    assert torch.equal(msg[4 * words.numel():].view(torch.float32), scales)


def test_bf16_gradients_sign():
    """bf16 gradients with sparse +-0.1 outliers, GPT-2 tensor list shrunk 64x, N=5 (not a power of two)."""
    lay = scaled_layout(gpt2_small_layout(), 64)
    P = _pair(5, lay.seg_offsets, SIGN, SIGN, grad_dtype=liec.BF16)
    for step in range(5):
        G = make_gradients("bf16_outliers", 1e-2, 5, lay.dim, step, base_seed=5)
        P.step(G, 1e-3)


def test_bf16_special_values_sign():
    """Signed zeros, subnormals of both signs, the largest finite values: the sign bit is x < 0, so -0 packs as 0
    and a negative subnormal as 1; magnitudes enter the L1 sum exactly."""
    off = [0, 8192 * 3 + 8, 8192 * 3 + 8 + 777]
    P = _pair(4, off, SIGN, SIGN, grad_dtype=liec.BF16)
    special = torch.tensor([0x0000, 0x8000, 0x0001, 0x8001, 0x007F, 0x807F, 0x0080, 0x8080, 0x7F7F, 0xFF7F, 0x3F80, 0xBF80],
                           dtype=torch.int32).to(torch.int16)
    gen = torch.Generator().manual_seed(77)
    for step in range(3):
        G = make_gradients("bf16_outliers", 1e-2, 4, off[-1], step, base_seed=77)
        bits = G.view(torch.int16)
        where = torch.randint(0, off[-1], (4, 4000), generator=gen)
        what = special[torch.randint(0, special.numel(), (4, 4000), generator=gen)]
        bits.scatter_(1, where, what)
        if step == 2:  # one whole tile of negative zeros and one of negative subnormals
            bits[0, :8192] = special[1]
            bits[1, 8192:16384] = special[3]
        P.step(G, 1e-3)


@pytest.mark.parametrize("up,down", [(IDENT, IDENT), (SIGN, IDENT), (IDENT, SIGN)])
def test_identity_combinations(up, down):
    lay = ragged_layout()
    P = _pair(3, lay.seg_offsets, up, down)
    for step in range(3):
        G = make_gradients("normal", 1.0, 3, lay.dim, step, base_seed=6)
        P.step(G, 0.1)


def test_identity_one_worker_is_sgd():
    """Algorithm 1 with C = identity and N = 1 reduces to x <- x - eta g, bit for bit."""
    d = 20000
    x0 = torch.randn(d, generator=torch.Generator().manual_seed(7))
    X = x0.clone().view(1, d).cuda()
    e = torch.zeros(d, device="cuda")
    ctx = liec.Context(X, e, [0, 12345, d], IDENT, IDENT)
    ref = x0.clone()
    for step in range(5):
        G = make_gradients("normal", 1.0, 1, d, step, base_seed=7)
        ctx.liec_step(G.cuda(), 0.05)
        ref = ref - torch.tensor(0.05, dtype=torch.float32) * G[0]
    torch.cuda.synchronize()
    assert torch.equal(X[0].cpu(), ref) and torch.all(e == 0)


def test_staged_calls_equal_fused_step_and_are_deterministic():
    lay = ragged_layout()
    outs = []
    for mode in ("step", "staged", "step"):
        X = torch.zeros(4, lay.dim, device="cuda")
        e = torch.zeros(lay.dim, device="cuda")
        ctx = liec.Context(X, e, lay.seg_offsets, SIGN, SIGN)
        for step in range(3):
            G = make_gradients("normal", 1.0, 4, lay.dim, step, base_seed=8).cuda()
            if mode == "step":
                ctx.liec_step(G, 0.1)
            else:
                ctx.liec_uplink_compress(G); ctx.liec_server_aggregate(); ctx.liec_downlink_compress(); ctx.liec_worker_update(G, 0.1)
        torch.cuda.synchronize()
        m = ctx.liec_get_messages()
        outs.append((X.cpu(), e.cpu(), m["down_words"].cpu(), m["up_words"].cpu()))
    for a, b in zip(outs[0], outs[1]):
        assert torch.equal(a, b)
    for a, b in zip(outs[0], outs[2]):
        assert torch.equal(a, b)


def test_stage_order_and_argument_errors():
    lay = flat_layout(1000)
    X = torch.zeros(2, 1000, device="cuda")
    e = torch.zeros(1000, device="cuda")
    ctx = liec.Context(X, e, lay.seg_offsets, SIGN, SIGN)
    G = torch.zeros(2, 1000, device="cuda")
    with pytest.raises(liec.LiecError) as ei:
        ctx.liec_server_aggregate()
    assert ei.value.status == 4
    ctx.liec_uplink_compress(G)
    with pytest.raises(liec.LiecError) as ei:
        ctx.liec_worker_update(G, 0.1)
    assert ei.value.status == 4
    ctx.liec_server_aggregate(); ctx.liec_downlink_compress()
    with pytest.raises(liec.LiecError) as ei:
        ctx.liec_worker_update(G.clone(), 0.1)      # a different gradient buffer than the uplink saw
    assert ei.value.status == 1
    ctx.liec_worker_update(G, 0.1)
    assert ctx.liec_device_status() == 0 and ctx.liec_launch_count() == 6


def test_resume_from_saved_state():
    """Checkpoint = (X, e): re-creating a context on copies continues identically."""
    lay = scaled_layout(resnet18_layout(), 64)
    N = 4
    grads = [make_gradients("normal", 0.01, N, lay.dim, s, base_seed=9).cuda() for s in range(6)]
    X1 = torch.zeros(N, lay.dim, device="cuda"); e1 = torch.zeros(lay.dim, device="cuda")
    c1 = liec.Context(X1, e1, lay.seg_offsets, SIGN, SIGN)
    for s in range(6):
        c1.liec_step(grads[s], 0.05)
    X2 = torch.zeros(N, lay.dim, device="cuda"); e2 = torch.zeros(lay.dim, device="cuda")
    c2 = liec.Context(X2, e2, lay.seg_offsets, SIGN, SIGN)
    for s in range(3):
        c2.liec_step(grads[s], 0.05)
    torch.cuda.synchronize()
    X3, e3 = X2.clone(), e2.clone()
    c3 = liec.Context(X3, e3, lay.seg_offsets, SIGN, SIGN)
    for s in range(3, 6):
        c3.liec_step(grads[s], 0.05)
    torch.cuda.synchronize()
    assert torch.equal(X1, X3) and torch.equal(e1, e3)

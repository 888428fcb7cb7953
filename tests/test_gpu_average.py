"""Model-averaging iteration and mean model of the CUDA library against the CPU oracle."""
import numpy as np
import pytest
import torch

import oracle
from gpu_helpers import Pair, assert_close, f32, widen
from liec_synth import make_gradients, ragged_layout, resnet18_layout, scaled_layout, topk_counts, gpt2_small_layout
from paper_2402_11857_b200 import liec

pytestmark = pytest.mark.gpu


def _average(P, G, lr):
    Gd = G.to("cuda").contiguous()
    v, xbar = oracle.average_step(P.Xh, P.eh, widen(G), lr)
    P.ctx.liec_average_step(Gd, lr)
    torch.cuda.synchronize()
    assert_close(f32(P.ed), P.eh, "error after averaging")
    assert_close(f32(P.Xd), P.Xh, "params after averaging")
    assert np.all(f32(P.ed) == 0.0)


@pytest.mark.parametrize("comp", [liec.COMP_SCALED_SIGN, liec.COMP_TOPK])
def test_averaging_every_third_step(comp):
    """Algorithm 1 as a whole: compressed iterations with an averaging iteration every 3rd step."""
    lay = ragged_layout()
    k = topk_counts(lay, 1, 100) if comp == liec.COMP_TOPK else None
    rng = np.random.default_rng(3)
    P = Pair(5, lay.seg_offsets, comp, comp, k=k, x0=rng.standard_normal(lay.dim))
    for step in range(7):
        G = make_gradients("normal", 1.0, 5, lay.dim, step, base_seed=31)
        if (step + 1) % 3 == 0:
            _average(P, G, 0.1)
        else:
            P.step(G, 0.1, check_messages=False)
    out = torch.empty(lay.dim, device="cuda")
    P.ctx.liec_mean_params(out)
    torch.cuda.synchronize()
    assert_close(f32(out), oracle.mean_params(P.Xh), "mean model")


def test_averaging_bf16_gradients_and_scaled_layouts():
    lay = scaled_layout(gpt2_small_layout(), 64)
    P = Pair(6, lay.seg_offsets, liec.COMP_SCALED_SIGN, liec.COMP_SCALED_SIGN, grad_dtype=liec.BF16)
    for step in range(4):
        G = make_gradients("bf16_outliers", 1e-2, 6, lay.dim, step, base_seed=32)
        if step % 2 == 1:
            _average(P, G, 1e-3)
        else:
            P.step(G, 1e-3, check_messages=False)


def test_averaging_unaligned_rows_and_stage_order():
    off = [0, 5, 8192 + 5, 3 * 8192 + 1]
    P = Pair(3, off, liec.COMP_SCALED_SIGN, liec.COMP_SCALED_SIGN, e0=np.linspace(-1, 1, off[-1]))
    G = make_gradients("normal", 1.0, 3, off[-1], 0, base_seed=33)
    _average(P, G, 0.2)
    Gd = G.cuda()
    P.ctx.liec_uplink_compress(Gd)
    with pytest.raises(liec.LiecError) as ei:
        P.ctx.liec_average_step(Gd, 0.1)       # in the middle of a compressed iteration
    assert ei.value.status == 4


@pytest.mark.parametrize("N,gdt", [(8, liec.F32), (16, liec.F32), (32, liec.BF16), (40, liec.F32), (300, liec.F32)])
def test_averaging_staged_in_shared_memory(N, gdt):
    """Full aligned tiles take the variant that keeps the workers' gradients of a slice in shared memory
    between the two sweeps (2048-element slices for N = 8 float rows, 1024-element slices for 16 float
    or 32 bfloat16 rows); 40 and 300 float rows of a slice exceed the shared-memory budget and take the
    re-reading variant; the ragged tail and the 8-element segment take the guarded path inside the
    same launch."""
    off = [0, 3 * 8192, 3 * 8192 + 8, 5 * 8192 + 8 + 77]
    dist = ("bf16_outliers", 1e-2) if gdt == liec.BF16 else ("normal", 1.0)
    rng = np.random.default_rng(4)
    P = Pair(N, off, liec.COMP_SCALED_SIGN, liec.COMP_SCALED_SIGN, grad_dtype=gdt,
             x0=rng.standard_normal(off[-1]), e0=rng.standard_normal(off[-1]) * 0.1)
    for step in range(2):
        G = make_gradients(dist[0], dist[1], N, off[-1], step, base_seed=34)
        P.step(G, 0.05, check_messages=False)      # rows drift apart
        _average(P, G, 0.05)


def test_averaging_bulk_copy_wait_runs_out():
    """The staged variant waits for its bulk copies with a bound: told to expect 16 bytes more than they
    deliver, the wait runs out, bit 8 of the status word is set and the CTA writes nothing."""
    off = [0, 8192]
    N = 2
    X0 = torch.randn(N, 8192, device="cuda")
    X = X0.clone()
    e = torch.randn(8192, device="cuda")
    e0 = e.clone()
    ctx = liec.Context(X, e, off, liec.COMP_SCALED_SIGN, liec.COMP_SCALED_SIGN)
    G = make_gradients("normal", 1.0, N, 8192, 0, base_seed=35).cuda()
    ctx.liec_set_copy_wait(poll_limit=1000, expect_extra_bytes=16)
    ctx.liec_average_step(G, 0.1)
    torch.cuda.synchronize()
    assert ctx.liec_device_status() & 8
    assert torch.equal(X, X0) and torch.equal(e, e0)
    ctx.liec_set_copy_wait()
    ctx.liec_clear_status()
    ctx.liec_average_step(G, 0.1)
    torch.cuda.synchronize()
    assert ctx.liec_device_status() == 0
    Xh, eh = X0.cpu().numpy().copy(), e0.cpu().numpy().copy()
    oracle.average_step(Xh, eh, G.cpu().numpy(), 0.1)
    assert_close(f32(X), Xh, "params after averaging")
    assert np.all(f32(e) == 0.0)

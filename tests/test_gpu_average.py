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

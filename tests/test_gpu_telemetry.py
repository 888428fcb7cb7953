"""Squared norms from the CUDA library against the oracle's, and the quantities the paper reports
from them: the error norm and the measured contraction delta of Def. 1 on both sides."""
import math

import numpy as np
import pytest
import torch

import oracle
from gpu_helpers import Pair, f32
from liec_synth import make_gradients, ragged_layout, topk_counts
from paper_2402_11857_b200 import liec

pytestmark = pytest.mark.gpu


def _oracle_sumsq(rows, off):
    return np.asarray([[oracle.tree_sumsq(r[off[t]:off[t + 1]]) for t in range(len(off) - 1)] for r in rows])


@pytest.mark.parametrize("gdt", [liec.F32, liec.BF16])
def test_sumsq_is_bit_exact_and_gives_delta(gdt):
    lay = ragged_layout()
    off, N, T = lay.seg_offsets, 3, lay.num_segments
    P = Pair(N, off, liec.COMP_SCALED_SIGN, liec.COMP_SCALED_SIGN, grad_dtype=gdt)
    dist = ("bf16_outliers", 1e-2) if gdt == liec.BF16 else ("normal", 1.0)
    for step in range(3):
        G = make_gradients(dist[0], dist[1], N, lay.dim, step, base_seed=51)
        r = P.step(G, 0.1)
    Gd = G.cuda()
    out_g = torch.empty(N, T, dtype=torch.float64, device="cuda")
    out_e = torch.empty(1, T, dtype=torch.float64, device="cuda")
    out_x = torch.empty(N, T, dtype=torch.float64, device="cuda")
    P.ctx.liec_sumsq(liec.SUMSQ_GRADS, out_g, grads=Gd)
    P.ctx.liec_sumsq(liec.SUMSQ_ERROR, out_e)
    P.ctx.liec_sumsq(liec.SUMSQ_PARAMS, out_x)
    torch.cuda.synchronize()
    from gpu_helpers import widen
    assert np.array_equal(out_g.cpu().numpy(), _oracle_sumsq(widen(G), off))
    assert np.array_equal(out_e.cpu().numpy(), _oracle_sumsq(P.eh[None, :], off))
    assert np.array_equal(out_x.cpu().numpy(), _oracle_sumsq(P.Xh, off))
    # measured delta (Def. 1) of the last step, per segment: worker side n s^2 / ||g||^2,
    # server side n s^2 / (||e'||^2 + n s^2); on Gaussian gradients both are near 2/pi
    n = np.diff(off).astype(np.float64)
    delta_w = n * r.up_scales.astype(np.float64) ** 2 / out_g.cpu().numpy()
    delta_s = n * r.down_scales.astype(np.float64) ** 2 / (out_e.cpu().numpy()[0] + n * r.down_scales.astype(np.float64) ** 2)
    big = n > 5000
    assert np.all(delta_w[:, big] > 0) and np.all(delta_w <= 1 + 1e-12) and np.all(delta_s <= 1 + 1e-12)
    if gdt == liec.F32:
        assert np.all(np.abs(delta_w[:, big] - 2 / math.pi) < 0.05)
    # the error norm of the paper's error-norm figure
    assert abs(math.sqrt(out_e.sum().item()) - float(np.linalg.norm(P.eh.astype(np.float64)))) < 1e-9 * (1 + np.linalg.norm(P.eh))


def test_topk_delta_from_kept_values():
    lay = ragged_layout()
    off, N, T = lay.seg_offsets, 2, lay.num_segments
    k = topk_counts(lay, 1, 100)
    P = Pair(N, off, liec.COMP_TOPK, liec.COMP_TOPK, k=k)
    G = make_gradients("normal", 1.0, N, lay.dim, 0, base_seed=52)
    r = P.step(G, 0.1)
    out_g = torch.empty(N, T, dtype=torch.float64, device="cuda")
    P.ctx.liec_sumsq(liec.SUMSQ_GRADS, out_g, grads=G.cuda())
    torch.cuda.synchronize()
    koff = np.concatenate([[0], np.cumsum(k)])
    for t in range(T):
        kept = r.up_val[0, koff[t]:koff[t + 1]].astype(np.float64)
        delta = float(np.sum(kept ** 2)) / out_g[0, t].item()
        assert k[t] / (off[t + 1] - off[t]) - 1e-12 <= delta <= 1 + 1e-12     # top-k contracts with delta >= k/d

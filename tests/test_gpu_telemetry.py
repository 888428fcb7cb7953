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


# ---------------------------------------------------------------------------------------------
# Telemetry fused into the iteration's own passes (liec_set_telemetry / liec_get_telemetry)
# ---------------------------------------------------------------------------------------------

def _check_fused(P, e_before, G, r, k):
    """Every number liec_get_telemetry returns against the oracle's tree, bit for bit."""
    off = P.off
    T = len(off) - 1
    tel = P.ctx.liec_get_telemetry()
    torch.cuda.synchronize()
    host = {name: (None if t is None else t.cpu().numpy()) for name, t in tel.items()}
    from gpu_helpers import widen
    assert np.array_equal(host["e_sumsq"], _oracle_sumsq(e_before[None, :], off)[0]), "||e_t||^2 (entering the iteration)"
    assert np.array_equal(host["v_sumsq"], _oracle_sumsq(r.v[None, :], off)[0]), "||v_t||^2"
    assert np.array_equal(host["g_sumsq"], _oracle_sumsq(widen(G), off)), "||g^i_t||^2"
    if k is not None:
        koff = np.concatenate([[0], np.cumsum(k)])
        if r.up_val is not None:
            assert np.array_equal(host["up_kept_sumsq"], _oracle_sumsq(r.up_val, koff)), "uplink kept values"
        if r.down_val is not None:
            assert np.array_equal(host["down_kept_sumsq"], _oracle_sumsq(r.down_val[None, :], koff)[0]), "downlink kept values"
    return host


SPARSE = (liec.COMP_TOPK, liec.COMP_RANDK)


@pytest.mark.parametrize("up,down,gdt", [
    (liec.COMP_SCALED_SIGN, liec.COMP_SCALED_SIGN, liec.F32),
    (liec.COMP_SCALED_SIGN, liec.COMP_SCALED_SIGN, liec.BF16),
    (liec.COMP_TOPK, liec.COMP_TOPK, liec.F32),
    (liec.COMP_TOPK, liec.COMP_SCALED_SIGN, liec.BF16),
    (liec.COMP_SCALED_SIGN, liec.COMP_TOPK, liec.F32),
    (liec.COMP_RANDK, liec.COMP_RANDK, liec.F32),
    (liec.COMP_IDENTITY, liec.COMP_SCALED_SIGN, liec.F32),
    (liec.COMP_TOPK, liec.COMP_IDENTITY, liec.F32),
])
def test_fused_telemetry_is_bit_exact_on_the_ragged_layout(up, down, gdt):
    from liec_synth import random_subsets
    lay = ragged_layout()
    off, N = lay.seg_offsets, 5     # (five workers: the sparse-downlink update serves four per CTA)
    k = topk_counts(lay, 1, 50) if (up in SPARSE or down in SPARSE) else None
    P = Pair(N, off, up, down, k=k, grad_dtype=gdt)
    P.ctx.liec_set_telemetry(True)
    with pytest.raises(liec.LiecError):     # nothing has run yet with the telemetry on
        P.ctx.liec_get_telemetry()
    dist = ("bf16_outliers", 1e-2) if gdt == liec.BF16 else ("normal", 1.0)
    for step in range(3):
        G = make_gradients(dist[0], dist[1], N, lay.dim, step, base_seed=53)
        sets = random_subsets(off, k, N + 1, step, 53) if liec.COMP_RANDK in (up, down) else None
        e_before = P.eh.copy()
        r = P.step(G, 0.1, up_sets=None if sets is None or up != liec.COMP_RANDK else sets[:N],
                   down_set=None if sets is None or down != liec.COMP_RANDK else sets[N])   # also: same bits as the oracle with the telemetry on
        host = _check_fused(P, e_before, G, r, k)
    # the paper's quantities from these sums: measured delta of Def. 1 against its definition
    # evaluated directly in binary64 on the oracle's decoded messages
    n = np.diff(off).astype(np.float64)
    from gpu_helpers import widen
    Gf = widen(G).astype(np.float64)
    for t in range(len(off) - 1):
        x = Gf[0, off[t]:off[t + 1]]
        if up == liec.COMP_SCALED_SIGN:
            cx = np.where(x < 0, -1.0, 1.0) * float(r.up_scales[0, t])
            got = n[t] * float(r.up_scales[0, t]) ** 2 / host["g_sumsq"][0, t]
        elif up in SPARSE:
            koff = np.concatenate([[0], np.cumsum(k)])
            cx = np.zeros_like(x)
            cx[r.up_idx[0, koff[t]:koff[t + 1]].astype(np.int64) - off[t]] = r.up_val[0, koff[t]:koff[t + 1]]
            got = host["up_kept_sumsq"][0, t] / host["g_sumsq"][0, t]
        else:
            continue
        want = 1.0 - float(np.sum((x - cx) ** 2)) / float(np.sum(x ** 2))
        assert abs(got - want) <= 1e-6, (t, got, want)     # (the sign scale is rounded to binary32: 2^-24 relative)
    P.ctx.liec_set_telemetry(False)
    with pytest.raises(liec.LiecError):
        P.ctx.liec_get_telemetry()


def test_fused_telemetry_on_a_segment_of_more_than_2048_tiles():
    BIG = 2049 * 8192 + 5
    off = np.asarray([0, BIG, BIG + 1000], np.int64)
    N = 2
    P = Pair(N, off, liec.COMP_SCALED_SIGN, liec.COMP_SCALED_SIGN)
    P.ctx.liec_set_telemetry(True)
    for step in range(2):
        G = make_gradients("normal", 0.01, N, int(off[-1]), step, base_seed=54)
        e_before = P.eh.copy()
        r = P.step(G, 0.05)
        _check_fused(P, e_before, G, r, None)


def test_fused_telemetry_topk_many_kept_values():
    """k_t above one tile of message values (several tiles and a ragged tail in the message's own tiling)."""
    off = np.asarray([0, 40 * 8192 + 77, 40 * 8192 + 77 + 9000], np.int64)
    k = np.asarray([2 * 8192 + 301, 8192], np.int64)
    N = 3
    P = Pair(N, off, liec.COMP_TOPK, liec.COMP_TOPK, k=k)
    P.ctx.liec_set_telemetry(True)
    for step in range(2):
        G = make_gradients("normal", 1.0, N, int(off[-1]), step, base_seed=55)
        e_before = P.eh.copy()
        r = P.step(G, 0.1)
        _check_fused(P, e_before, G, r, k)

"""Top-k paths of the CUDA library against the CPU oracle (needs a B200)."""
import numpy as np
import pytest
import torch

from liec_synth import (flat_layout, make_gradients, ragged_layout, resnet50_layout, scaled_layout, topk_counts,
                        Layout)
from paper_2402_11857_b200 import liec

pytestmark = pytest.mark.gpu

SIGN, IDENT, TOPK = liec.COMP_SCALED_SIGN, liec.COMP_IDENTITY, liec.COMP_TOPK


def _pair(*a, **kw):
    from gpu_helpers import Pair
    return Pair(*a, **kw)


def test_ragged_topk_one_percent():
    lay = ragged_layout()
    k = topk_counts(lay, 1, 100)
    P = _pair(3, lay.seg_offsets, TOPK, TOPK, k=k)
    for step in range(4):
        G = make_gradients("normal", 1.0, 3, lay.dim, step, base_seed=11)
        P.step(G, 0.1)


def test_k_extremes():
    """k_t = 1 and k_t = n_t (everything kept: e' = 0 everywhere, x <- x - eta*mean-like update)."""
    lay = ragged_layout()
    for k in (np.ones(lay.num_segments, np.int64), np.asarray(lay.sizes, np.int64)):
        P = _pair(2, lay.seg_offsets, TOPK, TOPK, k=k)
        for step in range(2):
            G = make_gradients("normal", 1.0, 2, lay.dim, step, base_seed=12)
            P.step(G, 0.1)


def test_heavy_ties_take_lower_index():
    """Small-integer gradients: a handful of distinct magnitudes, so almost every selection is
    decided by the index rule, and the groups of equal keys overflow the candidate buffer."""
    lay = Layout("ties", (100, 5000, 3 * 8192 + 5, 40000))
    k = np.asarray([7, 50, 245, 333], np.int64)
    P = _pair(3, lay.seg_offsets, TOPK, TOPK, k=k)
    g = torch.Generator().manual_seed(13)
    for step in range(3):
        G = torch.randint(-3, 4, (3, lay.dim), generator=g).float()
        P.step(G, 0.25)


def test_mostly_zero_segments_with_k_above_the_nonzero_count():
    """Rows of which one entry in a hundred is non-zero (an embedding gradient that saw a few tokens)
    with k_t = 5 %: the threshold is the key of zero and millions of entries tie at it, so the dense
    one-CTA path does the selection (both the one-launch-per-problem form and, for the segment of
    more than 1024 tiles, the wide form); its rounds span several tiles and a ragged tail."""
    lay = Layout("sparse", (37 * 8192 + 11, 1030 * 8192 + 3, 9000))
    k = topk_counts(lay, 5, 100)
    N = 2
    P = _pair(N, lay.seg_offsets, TOPK, TOPK, k=k)
    g = torch.Generator().manual_seed(15)
    for step in range(2):
        G = make_gradients("normal", 1.0, N, lay.dim, step, base_seed=15)
        G = torch.where(torch.rand(G.shape, generator=g) < 0.01, G, torch.zeros_like(G))
        P.step(G, 0.1)
    up = P.ctx.liec_topk_route_counts(True)
    assert up["slow"] >= N            # (the 9000-element segment may or may not need it)


def test_quantised_values_ties_at_threshold():
    """Gaussians rounded to multiples of 1/64: ties at the threshold, candidates within the buffer."""
    lay = Layout("quant", (30000, 8192, 70000))
    k = topk_counts(lay, 1, 100)
    P = _pair(4, lay.seg_offsets, TOPK, TOPK, k=k)
    for step in range(3):
        G = make_gradients("normal", 1.0, 4, lay.dim, step, base_seed=14)
        G = torch.round(G * 64) / 64
        P.step(G, 0.1)


def test_crowded_threshold_bin_uses_second_digit():
    """Many entries just around the threshold (what error feedback produces in v): more of them share
    the threshold's first key digit than the candidate buffer holds, yet their keys are distinct."""
    lay = Layout("crowded", (50000, 9000, 3 * 8192))
    k = np.asarray([500, 90, 245], np.int64)
    P = _pair(3, lay.seg_offsets, TOPK, TOPK, k=k)
    g = torch.Generator().manual_seed(22)
    for step in range(3):
        G = torch.randn(3, lay.dim, generator=g) * 0.01
        crowd = torch.rand(3, lay.dim, generator=g) < 0.2
        G = torch.where(crowd, 1.0 + 0.03 * torch.rand(3, lay.dim, generator=g), G)
        G = G * torch.where(torch.rand(3, lay.dim, generator=g) < 0.5, -1.0, 1.0)
        P.step(G, 0.1)


def test_guess_from_previous_step_can_be_wrong():
    """The uplink first tries last step's threshold as a lower bound.  Gradients whose scale jumps
    down (too few candidates) or up (too many) between steps must fall back to the full selection
    and still give the oracle's result; steady scales take the short route."""
    lay = Layout("jumps", (40000, 8192, 3 * 8192 + 17, 500))
    k = topk_counts(lay, 1, 100)
    P = _pair(3, lay.seg_offsets, TOPK, TOPK, k=k)
    scales = [1.0, 1.0, 1e-3, 1e-3, 50.0, 50.0, 1.0, 0.0, 1.0, 1.0]
    for step, sc in enumerate(scales):
        G = make_gradients("normal", 1.0, 3, lay.dim, step, base_seed=23) * sc
        if step == 5:
            G[1] *= 1e-4          # one worker alone changes scale
        P.step(G, 0.1)


def test_all_zero_and_mostly_zero_gradients():
    lay = Layout("zeros", (5000, 20000))
    k = np.asarray([50, 200], np.int64)
    P = _pair(2, lay.seg_offsets, TOPK, TOPK, k=k)
    G = torch.zeros(2, lay.dim)
    P.step(G, 0.1)
    G[0, 17] = -2.0; G[1, 6000] = 1e-30; G[1, 24999] = -0.0
    P.step(G, 0.1)
    G = make_gradients("normal", 1.0, 2, lay.dim, 0, base_seed=15)
    G[:, ::2] = 0.0           # fewer non-zeros than... no: half zero, k small: regular path
    G[:, 5000:24000] = 0.0    # segment 1 mostly zero: threshold falls on the zeros
    P.step(G, 0.1)


def test_resnet50_scaled_student_t_many_steps():
    """ResNet-50 tensor list shrunk 32x (161 segments), N=16, heavy-tailed gradients, k = 1 %."""
    lay = scaled_layout(resnet50_layout(), 32)
    k = topk_counts(lay, 1, 100)
    P = _pair(16, lay.seg_offsets, TOPK, TOPK, k=k)
    for step in range(12):
        G = make_gradients("student_t3", 1e-3, 16, lay.dim, step, base_seed=16)
        P.step(G, 0.1, check_messages=(step % 4 == 0))


def test_large_single_segment_topk():
    """One 2.36 M-element tensor (the largest ResNet conv): several hundred tiles per problem."""
    lay = flat_layout(2359296)
    for num, den in ((1, 100), (1, 1000)):
        k = topk_counts(lay, num, den)
        P = _pair(3, lay.seg_offsets, TOPK, TOPK, k=k)
        for step in range(2):
            G = make_gradients("student_t3", 1e-3, 3, lay.dim, step, base_seed=17)
            P.step(G, 0.1)


def test_many_candidates_take_the_wide_finish():
    """k = 10 % of a 700 k-element tensor: more candidates than one CTA is given to finish, so the
    threshold is found by the wide (multi-CTA) form of the finish step; a small tensor rides along."""
    lay = Layout("wide", (700_000, 5000))
    k = np.asarray([70_000, 50], np.int64)
    P = _pair(2, lay.seg_offsets, TOPK, TOPK, k=k)
    for step in range(3):
        G = make_gradients("normal", 1.0, 2, lay.dim, step, base_seed=24)
        P.step(G, 0.1)


def test_segment_of_more_than_1024_tiles_gathers_candidate_histograms():
    """A 9 M-element tensor (1099 tiles) with k = 1 %: the wide finish step, with the candidate
    histograms taken over the segment's whole candidate region (the long-segment form)."""
    lay = Layout("huge", (9_000_000, 3000))
    k = np.asarray([90_000, 30], np.int64)
    P = _pair(2, lay.seg_offsets, TOPK, TOPK, k=k)
    for step in range(2):
        G = make_gradients("normal", 1.0, 2, lay.dim, step, base_seed=25)
        P.step(G, 0.1)


def test_long_segment_whose_candidate_region_starts_off_a_16_byte_boundary():
    """A 9 M-element tensor behind a small one whose candidate capacity (2 k + 2048 with k = 201) is not
    a multiple of four: the long segment's candidate histograms read its region with 128-bit loads
    from the boundary before it, and must count neither the neighbour's slots nor anything twice."""
    lay = Layout("offset", (20_000, 9_000_000))
    k = np.asarray([201, 90_001], np.int64)
    P = _pair(2, lay.seg_offsets, TOPK, TOPK, k=k)
    for step in range(3):
        G = make_gradients("normal", 1.0, 2, lay.dim, step, base_seed=27)
        P.step(G, 0.1)
    assert P.ctx.liec_topk_route_counts(True)["single_pass"] >= 2     # (the guess route, with its first-digit candidate histogram, ran)


def test_segment_of_more_than_4096_tiles_between_others():
    """A 33.6 M-element tensor (4101 tiles: two runs of the tile scan, whose second run starts from the
    sums of the first) between a mid-size and a small one, k = 0.5 %; the second step runs on the
    guess route."""
    lay = Layout("runs", (300_000, 4100 * 8192 + 7, 5000))
    k = topk_counts(lay, 1, 200)
    P = _pair(2, lay.seg_offsets, TOPK, TOPK, k=k)
    for step in range(2):
        G = make_gradients("normal", 1.0, 2, lay.dim, step, base_seed=28)
        P.step(G, 0.1)


@pytest.mark.parametrize("k0", [1, 2, 3, 4, 5])
def test_all_equal_magnitudes_keep_the_first_indices_of_the_vector(k0):
    """Every entry of the first segments has the same magnitude, so the threshold ties everywhere and the
    cut (last accepted tie) is flat index k - 1 = 0 ... 4, inside the first quad of the vector: the
    worker update must drop the quad's other entries although they equal the threshold."""
    lay = Layout("equal", (9000, 300, 20000))
    k = np.asarray([k0, k0, 200], np.int64)
    P = _pair(2, lay.seg_offsets, TOPK, TOPK, k=k)
    for step in range(2):
        G = make_gradients("normal", 1.0, 2, lay.dim, step, base_seed=29)
        G[:, :9300] = torch.where(G[:, :9300] < 0, -0.5, 0.5)
        P.step(G, 0.1)


def test_bf16_topk():
    lay = ragged_layout()
    k = topk_counts(lay, 1, 50)
    P = _pair(3, lay.seg_offsets, TOPK, TOPK, k=k, grad_dtype=liec.BF16)
    for step in range(3):
        G = make_gradients("bf16_outliers", 1e-2, 3, lay.dim, step, base_seed=18)   # bf16: many equal magnitudes
        P.step(G, 0.01)


@pytest.mark.parametrize("up,down", [(TOPK, SIGN), (SIGN, TOPK), (TOPK, IDENT), (IDENT, TOPK)])
def test_mixed_compressors(up, down):
    lay = ragged_layout()
    k = topk_counts(lay, 1, 100)
    P = _pair(3, lay.seg_offsets, up, down, k=k)
    for step in range(3):
        G = make_gradients("normal", 1.0, 3, lay.dim, step, base_seed=19)
        P.step(G, 0.1)


def test_unaligned_rows_topk():
    off = [0, 5, 8192 + 5, 8192 + 5 + 33, 3 * 8192 + 1]
    k = [1, 80, 3, 160]
    P = _pair(3, off, TOPK, TOPK, k=k)
    for step in range(3):
        G = make_gradients("normal", 1.0, 3, off[-1], step, base_seed=20)
        P.step(G, 0.1)


def test_topk_staged_equals_step_and_deterministic():
    lay = ragged_layout()
    k = topk_counts(lay, 1, 100)
    outs = []
    for mode in ("step", "staged", "step"):
        X = torch.zeros(4, lay.dim, device="cuda")
        e = torch.zeros(lay.dim, device="cuda")
        ctx = liec.Context(X, e, lay.seg_offsets, TOPK, TOPK, k)
        for step in range(3):
            G = make_gradients("normal", 1.0, 4, lay.dim, step, base_seed=21).cuda()
            if mode == "step":
                ctx.liec_step(G, 0.1)
            else:
                ctx.liec_uplink_compress(G); ctx.liec_server_aggregate(); ctx.liec_downlink_compress(); ctx.liec_worker_update(G, 0.1)
        torch.cuda.synchronize()
        assert ctx.liec_device_status() == 0
        m = ctx.liec_get_messages()
        outs.append((X.cpu(), e.cpu(), m["down_idx"].cpu(), m["up_idx"].cpu(), m["up_val"].cpu()))
    for a, b in zip(outs[0], outs[1]):
        assert torch.equal(a, b)
    for a, b in zip(outs[0], outs[2]):
        assert torch.equal(a, b)


def test_guess_overflow_on_a_segment_of_hundreds_of_tiles():
    """The gradient scale rises 50-fold step after step (what a learning-rate warm-up does), so each
    step's guess, last step's threshold, lets far more through than the candidate buffer holds.  With
    288 tiles per problem many CTAs are in flight when the first one finds the buffer full; the problem
    must fall back to the regular route as a whole, with a clean status word."""
    lay = flat_layout(2359296)
    k = topk_counts(lay, 1, 100)
    P = _pair(3, lay.seg_offsets, TOPK, TOPK, k=k)
    scale = 1e-6
    for step in range(7):
        G = make_gradients("normal", 1.0, 3, lay.dim, step, base_seed=26) * scale
        P.step(G, 0.1, check_messages=(step in (0, 3, 6)))
        routes = P.ctx.liec_topk_route_counts(True)
        assert routes["single_pass"] == 0, (step, routes)   # first step: no guess; later: every guess overflows
        scale *= 50.0
    # steady scale again: the guess holds
    for step in range(7, 9):
        G = make_gradients("normal", 1.0, 3, lay.dim, step, base_seed=26) * scale
        P.step(G, 0.1)
    assert P.ctx.liec_topk_route_counts(True)["single_pass"] == 3

"""The largest dimension the library accepts (d just below 2^32, one worker, one segment): flat
indices use the whole unsigned 32-bit range and the row has half a million tiles.  The oracle
cannot run at this size, so the step is checked through what holds at any size: every
element-wise stage recomputed with the same binary32 operations in the same order (exact), sign
words against the gradient's sign (exact), scales against a binary64 sum (one unit in the last
place), the top-k message against the magnitude order of the whole vector."""
import numpy as np
import pytest
import torch

from paper_2402_11857_b200 import liec

pytestmark = pytest.mark.gpu

D = (1 << 32) - 8192 - 24      # ragged last tile, rows stay 16-byte aligned
CH = 1 << 28                   # elements per checking chunk


def _need(gib):
    import gc
    gc.collect()
    torch.cuda.empty_cache()   # blocks cached by earlier tests count as used otherwise
    free, _ = torch.cuda.mem_get_info()
    if free < gib * (1 << 30):
        pytest.skip(f"needs {gib} GiB of free device memory")


def _chunks():
    for a in range(0, D, CH):
        yield a, min(D, a + CH)


def _fill(t, seed, scale):
    gen = torch.Generator(device="cuda").manual_seed(seed)
    for a, b in _chunks():
        t[a:b].normal_(0.0, scale, generator=gen)


def _bits_of(words, a, b):
    """Sign bits of elements a..b-1 (a, b multiples of 32) unpacked from int32 words, as bool."""
    w = words[a // 32:b // 32]
    shifts = torch.arange(32, device="cuda", dtype=torch.int32)
    return ((w[:, None] >> shifts[None, :]) & 1).bool().reshape(-1)


def test_sign_step_at_the_largest_dimension():
    _need(125)
    X = torch.zeros(1, D, device="cuda")
    e = torch.empty(D, device="cuda")
    G = torch.empty(1, D, device="cuda")
    _fill(X[0], 1, 1.0)
    _fill(e, 2, 1e-3)
    _fill(G[0], 3, 1e-2)
    X0, e0 = X.clone(), e.clone()
    ctx = liec.Context(X, e, [0, D], liec.COMP_SCALED_SIGN, liec.COMP_SCALED_SIGN)
    lr = 0.05
    ctx.liec_uplink_compress(G)
    ctx.liec_server_aggregate()
    torch.cuda.synchronize()
    m = ctx.liec_get_messages()
    su = m["up_scales"][0, 0].clone()
    l1 = sum(float(G[0, a:b].abs().double().sum()) for a, b in _chunks())
    want = np.float32(l1 / D)
    assert abs(float(su) - float(want)) <= float(np.spacing(want)), "uplink scale"
    Dw = D - D % 32
    for a, b in _chunks():
        b32 = min(b, Dw)
        assert torch.equal(_bits_of(m["up_words"][0], a, b32), G[0, a:b32] < 0), "uplink sign words"
        p_i = torch.where(G[0, a:b] < 0, -su, su)
        assert torch.equal(e[a:b], e0[a:b] + p_i / 1.0), "v = e + mean of the messages"   # N = 1
    tail = int(m["up_words"][0, -1].item()) & 0xffffffff     # the ragged last word: 8 valid bits, padding 0
    assert tail == int(sum(int(G[0, Dw + q] < 0) << q for q in range(D - Dw)))
    v = e.clone()
    ctx.liec_downlink_compress()
    ctx.liec_worker_update(G, lr)
    torch.cuda.synchronize()
    assert ctx.liec_device_status() == 0
    sd = m["down_scales"][0].clone()
    l1 = sum(float(v[a:b].abs().double().sum()) for a, b in _chunks())
    want = np.float32(l1 / D)
    assert abs(float(sd) - float(want)) <= float(np.spacing(want)), "downlink scale"
    for a, b in _chunks():
        b32 = min(b, Dw)
        assert torch.equal(_bits_of(m["down_words"], a, b32), v[a:b32] < 0), "downlink sign words"
        p = torch.where(v[a:b] < 0, -sd, sd)
        assert torch.equal(e[a:b], v[a:b] - p), "e' = v - p"
        p_i = torch.where(G[0, a:b] < 0, -su, su)
        assert torch.equal(X[0, a:b], X0[0, a:b] - lr * ((p - p_i) + G[0, a:b])), "local update"


def test_topk_step_at_the_largest_dimension():
    _need(125)
    k = 100_000
    X = torch.zeros(1, D, device="cuda")
    e = torch.zeros(D, device="cuda")
    G = torch.empty(1, D, device="cuda")
    _fill(G[0], 4, 1.0)
    ctx = liec.Context(X, e, [0, D], liec.COMP_TOPK, liec.COMP_TOPK, [k])
    lr = 0.05
    for step in range(2):                  # the second step takes the single-pass route
        X0, e0 = X.clone(), e.clone()
        if step == 1:
            G[0, -5:] = torch.tensor([9.0, -9.0, 9.5, -9.5, 10.0], device="cuda")   # winners at the very end of the range
        ctx.liec_uplink_compress(G)
        ctx.liec_server_aggregate()
        torch.cuda.synchronize()
        m = ctx.liec_get_messages()
        idx = torch.from_numpy(m["up_idx"][0].cpu().numpy().view(np.uint32).astype(np.int64)).cuda()
        val = m["up_val"][0].clone()
        assert idx.numel() == k and bool((idx[1:] > idx[:-1]).all()) and int(idx[-1]) < D, "ascending, in range"
        assert torch.equal(val, G[0][idx]), "values are the gradient's"
        thr = float(val.abs().min())
        above = sum(int((G[0, a:b].abs() > thr).sum()) for a, b in _chunks())
        at_least = sum(int((G[0, a:b].abs() >= thr).sum()) for a, b in _chunks())
        assert above <= k <= at_least, "the kept set is a top-k set"
        if step == 1:
            assert int(idx[-1]) == D - 1 and int(idx[-5]) == D - 5
        # v = e + p^1 (N = 1): e0 everywhere, plus the kept values (e0 is not needed afterwards)
        e0[idx] = e0[idx] + val / 1.0
        assert torch.equal(e, e0), "v"
        del e0
        v = e.clone()
        ctx.liec_downlink_compress()
        ctx.liec_worker_update(G, lr)
        torch.cuda.synchronize()
        assert ctx.liec_device_status() == 0
        didx = torch.from_numpy(m["down_idx"].cpu().numpy().view(np.uint32).astype(np.int64)).cuda()
        dval = m["down_val"].clone()
        assert bool((didx[1:] > didx[:-1]).all()) and torch.equal(dval, v[didx])
        thr = float(dval.abs().min())
        above = sum(int((v[a:b].abs() > thr).sum()) for a, b in _chunks())
        at_least = sum(int((v[a:b].abs() >= thr).sum()) for a, b in _chunks())
        assert above <= k <= at_least
        v[didx] = 0.0
        assert torch.equal(e, v), "e' = v - p"
        del v
        for a, b in _chunks():
            p = torch.zeros(b - a, device="cuda")
            p_i = torch.zeros(b - a, device="cuda")
            lo, hi = torch.searchsorted(didx, torch.tensor([a, b], device="cuda")).tolist()
            p[didx[lo:hi] - a] = dval[lo:hi]
            lo, hi = torch.searchsorted(idx, torch.tensor([a, b], device="cuda")).tolist()
            p_i[idx[lo:hi] - a] = val[lo:hi]
            assert torch.equal(X[0, a:b], X0[0, a:b] - lr * ((p - p_i) + G[0, a:b])), "local update"
        del X0

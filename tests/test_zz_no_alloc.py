"""The allocation-free scaled-sign entry point against the regular uplink compressor.

Collected last on purpose (file name), so that a run stopping at the first failure has already
run every other test.  Some users of the library cannot give it a workspace or let it allocate
one (a gradient hook in the middle of a backward pass, a process whose allocator owns all GPU
memory); for them `liec_sign_compress_noalloc` keeps its scratch in a fixed array inside the
library.  The check: two calls in a row (the array is shared and keeps old contents) give the
same words and the same scale, bit for bit, as `liec_uplink_compress` with one worker and one
segment, and a vector beyond the fixed limit is refused with a clear message.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2402_11857_b200 import liec

pytestmark = pytest.mark.gpu


def _regular(x):
    n = x.numel()
    X = torch.zeros(1, n, device="cuda")
    e = torch.zeros(n, device="cuda")
    gdt = liec.BF16 if x.dtype == torch.bfloat16 else liec.F32
    ctx = liec.Context(X, e, [0, n], liec.COMP_SCALED_SIGN, liec.COMP_SCALED_SIGN, grad_dtype=gdt)
    ctx.liec_uplink_compress(x.view(1, n))
    torch.cuda.synchronize()
    m = ctx.liec_get_messages()
    return m["up_words"][0].clone(), m["up_scales"][0].clone()


def test_noalloc_matches_uplink_compress_on_two_calls_in_a_row():
    gen = torch.Generator(device="cuda").manual_seed(5)
    # the second call is shorter than the first: stale partials of the first must not leak in
    cases = [(3 * 8192 * 2048 // 1024 + 77, torch.float32), (8192 * 5 + 13, torch.float32), (100003, torch.bfloat16)]
    for n, dtype in cases:
        x = (torch.randn(n, generator=gen, device="cuda") * 0.01).to(dtype)
        x[::97] = 0.0
        words = torch.full(((n + 31) // 32,), -1, dtype=torch.int32, device="cuda")
        scale = torch.full((1,), float("nan"), device="cuda")
        liec.liec_sign_compress_noalloc(x, words, scale)
        torch.cuda.synchronize()
        ref_words, ref_scale = _regular(x)
        assert torch.equal(words, ref_words)
        assert scale.view(torch.int32).item() == ref_scale.view(torch.int32).item()


def test_noalloc_rejects_oversized_vectors():
    x = torch.zeros(16, device="cuda")
    lib = liec.load_library()
    st = lib.liec_sign_compress_noalloc(x.data_ptr(), liec.F32, liec.NOALLOC_MAX_ELEMENTS + 1, x.data_ptr(),
                                        x.data_ptr(), None)
    assert st == 2
    msg = lib.liec_noalloc_last_error().decode()
    assert "LIEC_NOALLOC_MAX_ELEMENTS" in msg


@pytest.mark.parametrize("n", [3 * 2048 * 8192 + 77, liec.NOALLOC_MAX_ELEMENTS])
def test_noalloc_entry_point_over_several_chunks(n):
    """The allocation-free variant with 3 and 4 chunks of tile partials (n at its documented limit
    uses the last entry of the built-in array): same words and scale as the regular uplink pass,
    and the scale of the oracle."""
    gen = torch.Generator(device="cuda").manual_seed(63)
    x = torch.randn(n, generator=gen, device="cuda") * 0.01
    x[::101] = 0.0
    words = torch.full(((n + 31) // 32,), -1, dtype=torch.int32, device="cuda")
    scale = torch.full((1,), float("nan"), device="cuda")
    for _ in range(2):
        liec.liec_sign_compress_noalloc(x, words, scale)
    torch.cuda.synchronize()
    ref_words, ref_scale = _regular(x)
    assert torch.equal(words, ref_words)
    assert scale.view(torch.int32).item() == ref_scale.view(torch.int32).item()
    want = oracle.scale(x.cpu().numpy())
    assert np.float32(scale.item()).view(np.uint32) == np.float32(want).view(np.uint32)
    # words against the definition: bit b of word w is set iff x[32w+b] < 0
    neg = torch.zeros(((n + 31) // 32) * 32, dtype=torch.bool, device="cuda")
    neg[:n] = x < 0
    packed = (neg.view(-1, 32).to(torch.int64) << torch.arange(32, device="cuda")).sum(dim=1)
    assert torch.equal(packed, words.to(torch.int64) & 0xFFFFFFFF)

"""Host-side checks of the C ABI that need no GPU: the library loads, exports every symbol
that include/liec.h declares, sizes workspaces and rejects bad configurations."""
import ctypes as C
import os
import re

import numpy as np
import pytest

from liec_synth import gpt2_small_layout, ragged_layout, resnet18_layout, resnet50_layout, topk_counts
from paper_2402_11857_b200 import build as cuda_build
from paper_2402_11857_b200 import liec

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    cuda_build.build()
    return liec.load_library()


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "liec.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(liec_[a-z_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    names = declared_symbols()
    assert len(names) >= 14 and "liec_step" in names and "liec_init" in names
    for name in names:
        assert hasattr(lib, name), f"{name} declared in liec.h but not exported"


def test_binding_has_the_same_names():
    for name in declared_symbols():
        if name in ("liec_workspace_bytes", "liec_down_message_bytes", "liec_init", "liec_destroy", "liec_last_error",
                    "liec_noalloc_last_error"):
            continue
        assert hasattr(liec.Context, name) or hasattr(liec, name), f"binding lacks {name}"


def test_workspace_sizes(lib):
    lay = resnet18_layout()
    cfg, keep = liec.make_config(8, lay.seg_offsets, liec.COMP_SCALED_SIGN, liec.COMP_SCALED_SIGN)
    W = int(((np.diff(lay.seg_offsets) + 31) // 32).sum())
    need = liec.workspace_bytes(cfg)
    assert need >= 4 * (8 * W + W) and need < 64 << 20
    assert liec.down_message_bytes(cfg) == 4 * (W + lay.num_segments)
    lay = resnet50_layout()
    k = topk_counts(lay, 1, 100)
    cfg, keep = liec.make_config(16, lay.seg_offsets, liec.COMP_TOPK, liec.COMP_TOPK, k)
    assert liec.down_message_bytes(cfg) == 8 * int(k.sum())
    assert liec.workspace_bytes(cfg) > 8 * 17 * int(k.sum())
    cfg, keep = liec.make_config(32, gpt2_small_layout().seg_offsets, 1, 1, None, liec.BF16)
    assert 0 < liec.workspace_bytes(cfg) < 1 << 30


@pytest.mark.parametrize("mutate,status", [
    (lambda c: setattr(c, "num_workers", 0), 1),
    (lambda c: setattr(c, "num_workers", 70000), 2),
    (lambda c: setattr(c, "dim", 5), 1),
    (lambda c: setattr(c, "uplink", 7), 1),
    (lambda c: setattr(c, "grad_dtype", 3), 1),
    (lambda c: setattr(c, "downlink", liec.COMP_TOPK), 1),   # top-k without k
])
def test_bad_configs_are_rejected_before_any_cuda_call(lib, mutate, status):
    lay = ragged_layout()
    cfg, keep = liec.make_config(4, lay.seg_offsets, 1, 1)
    mutate(cfg)
    assert lib.liec_workspace_bytes(C.byref(cfg)) == 0
    ctx = C.c_void_p()
    st = lib.liec_init(C.byref(cfg), 256, 256, 256, 1 << 40, C.byref(ctx))
    assert st == status and not ctx.value
    assert lib.liec_last_error(None)


def test_bad_tables_and_pointers(lib):
    ctx = C.c_void_p()
    cfg, keep = liec.make_config(2, [0, 10, 10, 20], 1, 1)         # empty segment
    assert lib.liec_init(C.byref(cfg), 256, 256, 256, 1 << 40, C.byref(ctx)) == 1
    cfg, keep = liec.make_config(2, [0, 10, 20], 2, 2, [3, 11])     # k > n
    assert lib.liec_init(C.byref(cfg), 256, 256, 256, 1 << 40, C.byref(ctx)) == 1
    cfg, keep = liec.make_config(2, [0, 2 ** 32], 1, 1)             # d too large for 32-bit indices
    assert lib.liec_init(C.byref(cfg), 256, 256, 256, 1 << 40, C.byref(ctx)) == 2
    cfg, keep = liec.make_config(2, [0, 10, 20], 1, 1)
    assert lib.liec_init(C.byref(cfg), 0, 256, 256, 1 << 40, C.byref(ctx)) == 1        # NULL params
    assert lib.liec_init(C.byref(cfg), 260, 256, 256, 1 << 40, C.byref(ctx)) == 1      # misaligned params
    assert lib.liec_init(C.byref(cfg), 256, 256, 264, 1 << 40, C.byref(ctx)) == 1      # misaligned workspace
    assert lib.liec_init(C.byref(cfg), 256, 256, 256, 16, C.byref(ctx)) == 3           # workspace too small
    assert b"workspace" in lib.liec_last_error(None)

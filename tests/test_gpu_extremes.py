"""Corner configurations against the oracle: the smallest problem, one worker, many workers
(more than a CTA has threads, and not a multiple of any group size used by the kernels)."""
import numpy as np
import pytest

import oracle
from liec_synth import make_gradients, random_subsets
from gpu_helpers import Pair

pytestmark = pytest.mark.gpu

IDENT, SIGN, TOPK, RANDK = oracle.IDENTITY, oracle.SIGN, oracle.TOPK, oracle.RANDK


def _run(N, off, up, down, k=None, steps=3, seed=401):
    off = np.asarray(off, np.int64)
    P = Pair(N, off, up, down, k=None if k is None else np.asarray(k, np.int64))
    for step in range(steps):
        G = make_gradients("normal", 1.0, N, int(off[-1]), step, base_seed=seed)
        kw = {}
        if up == RANDK:
            kw["up_sets"] = random_subsets(off, k, N, step, seed)
        if down == RANDK:
            kw["down_set"] = random_subsets(off, k, 1, step, seed + 1)[0]
        P.step(G, 0.1, **kw)


@pytest.mark.parametrize("comp", [SIGN, TOPK, RANDK, IDENT])
def test_one_worker_one_element(comp):
    _run(1, [0, 1], comp, comp, k=[1] if comp in (TOPK, RANDK) else None)


@pytest.mark.parametrize("comp", [SIGN, TOPK, RANDK])
def test_one_worker_several_tiles(comp):
    off = [0, 3, 3 + 2 * 8192 + 100]
    _run(1, off, comp, comp, k=[1, 200] if comp in (TOPK, RANDK) else None)


@pytest.mark.parametrize("N", [33, 300])
@pytest.mark.parametrize("comp", [SIGN, TOPK, RANDK])
def test_many_workers(N, comp):
    off = [0, 257, 257 + 8192 + 31]
    _run(N, off, comp, comp, k=[5, 90] if comp in (TOPK, RANDK) else None, steps=2)

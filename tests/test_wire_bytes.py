"""Wire-byte accounting of the library against the communication-cost column the paper prints
(tests/golden/comm_cost_table.txt).  CPU only: liec_wire_bytes is host arithmetic."""
import pytest

from oracle_pins import read_golden
from paper_2402_11857_b200 import build as cuda_build
from paper_2402_11857_b200 import liec

MIB = float(1 << 20)
N = 8


@pytest.fixture(scope="module", autouse=True)
def _lib():
    cuda_build.build()


@pytest.mark.parametrize("dataset", ["cifar10", "cifar100"])
def test_comm_cost_column_is_reproduced(dataset):
    g = {k: v[0] for k, v in read_golden("comm_cost_table.txt").items()}
    # d from the P-SGD entry: every worker sends and receives one fp32 vector per iteration
    d = round(g[f"{dataset}.psgd"] * MIB / (2 * N * 4))
    cfg, keep = liec.make_config(N, [0, d], liec.COMP_SCALED_SIGN, liec.COMP_SCALED_SIGN)
    up, down, full = liec.liec_wire_bytes(cfg)
    assert full == 4 * d and up == down == 4 * ((d + 31) // 32 + 1)
    psgd = N * 2 * full / MIB
    both = N * (up + down) / MIB                 # 1-bit both ways
    uplink_only = N * (up + full) / MIB          # compressed uplink, full-precision downlink
    liec_avg = lambda H: (1 - 1 / H) * both + (1 / H) * psgd   # every H-th iteration is sent uncompressed
    tol = 0.011                                  # the table keeps two decimals
    assert abs(psgd - g[f"{dataset}.psgd"]) < tol
    assert abs(both - g[f"{dataset}.doublesqueeze"]) < tol
    assert abs(2 * both - g[f"{dataset}.neolithic"]) < tol
    assert abs(uplink_only - g[f"{dataset}.memsgd"]) < tol
    assert abs(liec_avg(32) - g[f"{dataset}.liec32"]) < tol
    assert abs(liec_avg(100) - g[f"{dataset}.liec100"]) < tol


def test_wire_bytes_of_the_other_messages():
    off = [0, 100, 164, 1000]
    cfg, keep = liec.make_config(4, off, liec.COMP_TOPK, liec.COMP_IDENTITY, [1, 5, 80])
    up, down, full = liec.liec_wire_bytes(cfg)
    assert up == 8 * 86 and down == 4000 and full == 4000
    cfg, keep = liec.make_config(4, off, liec.COMP_SCALED_SIGN, liec.COMP_TOPK, [1, 5, 80])
    up, down, full = liec.liec_wire_bytes(cfg)
    assert up == 4 * ((4 + 2 + 27) + 3) and down == 8 * 86
    cfg, keep = liec.make_config(4, off, liec.COMP_RANDK, liec.COMP_RANDK, [1, 5, 80])   # (index, value) like top-k
    up, down, full = liec.liec_wire_bytes(cfg)
    assert up == down == 8 * 86 and liec.down_message_bytes(cfg) == 8 * 86
    cfg, keep = liec.make_config(4, off, liec.COMP_RANDK, liec.COMP_RANDK)                # k is required
    with pytest.raises(liec.LiecError):
        liec.liec_wire_bytes(cfg)
    cfg, keep = liec.make_config(0, off, 1, 1)
    with pytest.raises(liec.LiecError):
        liec.liec_wire_bytes(cfg)


def test_wire_bytes_with_a_shared_seed():
    """Sender and receiver draw the same random-k subsets from a seed: values only on the wire."""
    off = [0, 100, 164, 1000]
    cfg, keep = liec.make_config(4, off, liec.COMP_RANDK, liec.COMP_RANDK, [1, 5, 80])
    assert liec.liec_wire_bytes_seeded(cfg) == (4 * 86, 4 * 86, 4000)
    cfg, keep = liec.make_config(4, off, liec.COMP_RANDK, liec.COMP_TOPK, [1, 5, 80])     # top-k still sends its indices
    assert liec.liec_wire_bytes_seeded(cfg) == (4 * 86, 8 * 86, 4000)
    cfg, keep = liec.make_config(4, off, liec.COMP_SCALED_SIGN, liec.COMP_SCALED_SIGN)
    assert liec.liec_wire_bytes_seeded(cfg) == liec.liec_wire_bytes(cfg)

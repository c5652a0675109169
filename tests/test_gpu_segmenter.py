"""GPU segmenter (through the C ABI) against the oracle segmenter: integer work, bit-exact."""
import os

import numpy as np
import pytest

from oracle import ltri_oracle as orc
from paper_2412_04757_b200 import binding

pytestmark = pytest.mark.gpu
GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


@pytest.fixture(scope="module")
def lt():
    p = binding.make_params(1, 8, 2, 4096, 512, 1024, 64, 4, max_spans_per_region=16)
    ctx = binding.Ltri(p)
    yield ctx
    ctx.close()


def block_map(c, lens):
    m = sum(lens)
    Mq = np.zeros((m, m), dtype=np.int32)
    p = 0
    for ln in lens:
        for i in range(p, p + ln):
            Mq[i, p:i + 1] = c
        p += ln
    return Mq


def test_golden_block_maps(lt):
    with open(os.path.join(GOLDEN, "block_maps.txt")) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            left, right = line.split("|")
            c, thq, C = (int(v) for v in left.split())
            lens = [int(v) for v in right.split()]
            got = lt.ltri_debug_segment_map(block_map(c, lens), theta_mode=2, theta_q=thq, max_spans=C)
            assert got[:, 1].tolist() == lens and got[0, 0] == 0


@pytest.mark.parametrize("m,seed", [(1, 0), (2, 1), (31, 2), (32, 3), (33, 4), (100, 5), (257, 6), (512, 7)])
def test_random_maps_match_oracle_exactly(lt, m, seed):
    rng = np.random.default_rng(seed)
    Mq = np.tril(rng.integers(0, 2**22, size=(m, m)) * (rng.random((m, m)) < 0.3)).astype(np.int32)
    for C in (1, 5, 16):
        for q in (0.5, 0.9):
            thq = int(np.quantile(Mq[np.tril_indices(m)], q))
            ref, _ = orc.segment_map(Mq, thq, C)
            got = lt.ltri_debug_segment_map(Mq, theta_mode=2, theta_q=thq, max_spans=C)
            assert got.tolist() == ref.tolist()


@pytest.mark.parametrize("m,theta", [(17, 0.0), (64, 0.5), (200, 0.9), (512, 0.95), (300, 1.0)])
def test_quantile_theta_matches_oracle(lt, m, theta):
    rng = np.random.default_rng(m)
    Mq = np.tril(rng.integers(0, 2**25, size=(m, m)) * (rng.random((m, m)) < 0.2)).astype(np.int32)
    thq = orc.theta_q(Mq, 1, theta, 8)
    ref, _ = orc.segment_map(Mq, thq, 16)
    got = lt.ltri_debug_segment_map(Mq, theta_mode=1, theta=theta)
    assert got.tolist() == ref.tolist()
    assert int(lt.ltri_debug_read(binding.BUF_THETA, 0, 0)[0]) == thq


def test_planted_blocks_with_noise(lt):
    rng = np.random.default_rng(42)
    lens = [40, 7, 90, 33, 120, 64, 18, 140]
    Mq = block_map(100000, lens) + np.tril(rng.integers(0, 2000, size=(512, 512))).astype(np.int32)
    thq = 50000
    ref, _ = orc.segment_map(Mq, thq, 16)
    got = lt.ltri_debug_segment_map(Mq, theta_mode=2, theta_q=thq, max_spans=16)
    assert got.tolist() == ref.tolist()
    assert set(np.cumsum(lens)[:-1]) <= set(got[:, 0].tolist())


def test_bad_arguments(lt):
    Mq = np.zeros((8, 8), dtype=np.int32)
    with pytest.raises(binding.LtriError):
        lt.ltri_debug_segment_map(Mq, theta_mode=5)
    with pytest.raises(binding.LtriError):
        lt.ltri_debug_segment_map(np.zeros((1024, 1024), dtype=np.int32), theta_mode=2)   # m > chunk
    with pytest.raises(binding.LtriError):
        lt.ltri_debug_segment_map(Mq, theta_mode=2, max_spans=64)                       # > context's C


@pytest.mark.parametrize("phi_milli", [100, 300, 600])
def test_nms_with_iou_threshold_matches_oracle_exactly(phi_milli):
    # kept spans may overlap once the IoU threshold is above zero; integer rule, so bit-exact on the same map
    p = binding.make_params(1, 8, 2, 4096, 512, 1024, 64, 4, max_spans_per_region=16, nms_iou_milli=phi_milli)
    lt = binding.Ltri(p)
    rng = np.random.default_rng(900 + phi_milli)
    overlaps = 0
    for m in (17, 64, 200, 512):
        for _ in range(3):
            Mq = np.tril(rng.integers(0, 2**20, size=(m, m))).astype(np.int32)
            thq = int(np.quantile(Mq[np.tril_indices(m)], 0.85))
            for C in (3, 16):
                ref, _ = orc.segment_map(Mq, thq, C, phi_milli)
                got = lt.ltri_debug_segment_map(Mq, theta_mode=2, theta_q=thq, max_spans=C)
                assert got.tolist() == ref.tolist()
                overlaps += sum(a[0] + a[1] > b[0] for a, b in zip(ref, ref[1:]))
    assert overlaps > 0 or phi_milli < 300      # (a low threshold rarely lets two of these random spans overlap)
    lt.close()

"""Pins for the oracle's span segmenter (Eq. 4-5, App. "NMS Input Filtration").

Every check compares the oracle with something other than itself: a brute-force triple
loop, closed forms on hand-built maps, numpy's quantile, and torchvision's NMS.
"""
import os

import numpy as np
import pytest
import torch

from oracle import ltri_oracle as orc

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def brute_S(Mq, thq):
    """Eq. 5 as printed: sum over the triangle x<=j<=i<=y of (Mq - theta)."""
    m = Mq.shape[0]
    S = np.zeros((m, m), dtype=object)
    for x in range(m):
        for y in range(x, m):
            tot = 0
            for i in range(x, y + 1):
                for j in range(x, i + 1):
                    tot += int(Mq[i, j]) - thq
            S[x, y] = tot
    return S


def block_map(c, lens):
    m = sum(lens)
    Mq = np.zeros((m, m), dtype=np.int32)
    p = 0
    for ln in lens:
        for i in range(p, p + ln):
            Mq[i, p:i + 1] = c
        p += ln
    return Mq


def spans_of(lens):
    out, p = [], 0
    for ln in lens:
        out.append([p, ln])
        p += ln
    return np.array(out, dtype=np.int32)


@pytest.mark.parametrize("m,seed", [(1, 0), (2, 1), (7, 2), (23, 3), (40, 4)])
def test_two_cumsums_equal_triangle_sum(m, seed):
    rng = np.random.default_rng(seed)
    Mq = np.tril(rng.integers(0, 2**25, size=(m, m))).astype(np.int32)
    thq = int(rng.integers(0, 2**24))
    S = orc.ta_scores(Mq, thq)
    B = brute_S(Mq, thq)
    for x in range(m):
        for y in range(x, m):
            assert int(S[x, y]) == B[x, y]


def test_upper_triangle_of_input_is_ignored():
    rng = np.random.default_rng(5)
    full = rng.integers(0, 1000, size=(12, 12)).astype(np.int32)
    assert np.array_equal(orc.ta_scores(full, 17), orc.ta_scores(np.tril(full), 17))


def test_theta_zero_positive_map_gives_one_span():
    # Sec. 3.2: with positive entries and no threshold the largest score is the whole range.
    rng = np.random.default_rng(6)
    m = 19
    Mq = np.tril(rng.integers(1, 1000, size=(m, m))).astype(np.int32)
    S = orc.ta_scores(Mq, 0)
    iu = np.triu_indices(m)
    best = np.argmax(S[iu])
    assert (iu[0][best], iu[1][best]) == (0, m - 1)
    spans, _ = orc.segment_map(Mq, 0, 8)
    assert spans.tolist() == [[0, m]]


def _golden_cases():
    cases = []
    with open(os.path.join(GOLDEN, "block_maps.txt")) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            left, right = line.split("|")
            c, thq, C = (int(v) for v in left.split())
            cases.append((c, thq, C, [int(v) for v in right.split()]))
    return cases


@pytest.mark.parametrize("c,thq,C,lens", _golden_cases())
def test_block_maps_are_recovered_exactly(c, thq, C, lens):
    assert c / 2 <= thq < c and C >= len(lens)
    spans, _ = orc.segment_map(block_map(c, lens), thq, C)
    assert spans.tolist() == spans_of(lens).tolist()


def test_block_scores_match_closed_form():
    c, thq, lens = 1000, 600, [6, 10, 4]
    S = orc.ta_scores(block_map(c, lens), thq)
    p = 0
    for ln in lens:
        assert S[p, p + ln - 1] == (c - thq) * ln * (ln + 1) // 2
        p += ln
    tot = sum(lens)
    assert S[0, tot - 1] == c * sum(l * (l + 1) // 2 for l in lens) - thq * tot * (tot + 1) // 2


def test_small_theta_merges_adjacent_blocks():
    # two whole blocks l1,l2 merged outscore block 1 alone iff theta < c (l2+1) / (2 l1 + l2 + 1)
    c, l1, l2 = 1200, 8, 6
    bound = c * (l2 + 1) / (2 * l1 + l2 + 1)
    Mq = block_map(c, [l1, l2])
    for thq, merged in [(int(bound) - 5, True), (int(bound) + 5, False)]:
        S = orc.ta_scores(Mq, thq)
        assert (S[0, l1 + l2 - 1] > S[0, l1 - 1]) == merged
    spans, _ = orc.segment_map(Mq, 100, 4)
    assert spans.tolist() == [[0, l1 + l2]]          # well below the bound: one merged span
    spans, _ = orc.segment_map(Mq, c // 2, 4)
    assert spans.tolist() == [[0, l1], [l1, l2]]


def test_centred_intervals_rise_then_fall():
    # App. "NMS Input Filtration": around an isolated dense triangle [p,q] the centred
    # intervals' scores increase up to [p,q] and decrease afterwards.
    c, thq = 1000, 500
    lens = [9, 11, 9]                       # the middle block is [9,19], centred in the map
    S = orc.ta_scores(block_map(c, lens), thq)
    p, q = 9, 19
    mid = (p + q) // 2
    vals = [int(S[mid - r, mid + r]) for r in range(0, mid + 1)]
    peak = int(np.argmax(vals))
    assert (mid - peak, mid + peak) == (p, q)
    assert all(vals[i] < vals[i + 1] for i in range(peak))
    assert all(vals[i] > vals[i + 1] for i in range(peak, len(vals) - 1))


def test_gap_fill_partitions_region_and_respects_cap():
    rng = np.random.default_rng(7)
    for m in (5, 17, 33):
        Mq = np.tril(rng.integers(0, 5000, size=(m, m))).astype(np.int32)
        for C in (1, 2, 5):
            spans, _ = orc.segment_map(Mq, 2500, C)
            assert spans[0, 0] == 0 and spans[-1, 0] + spans[-1, 1] == m
            assert np.all(spans[1:, 0] == spans[:-1, 0] + spans[:-1, 1])
            assert np.all(spans[:, 1] >= 1)
            assert len(spans) <= 2 * C + 1


@pytest.mark.parametrize("phi_milli", [0, 100, 300])
@pytest.mark.parametrize("seed", range(6))
def test_greedy_nms_matches_torchvision(seed, phi_milli):
    tv = pytest.importorskip("torchvision")
    rng = np.random.default_rng(100 + seed)
    m = int(rng.integers(8, 40))
    Mq = np.tril(rng.integers(0, 2**20, size=(m, m))).astype(np.int32)
    thq = int(np.quantile(Mq[np.tril_indices(m)], 0.8))
    S = brute_S(Mq, thq)
    # anti-diagonal filter, written independently of the oracle
    cands = []
    for cdiag in range(2 * m - 1):
        pts = [(x, cdiag - x) for x in range(m) if 0 <= cdiag - x < m and x <= cdiag - x]
        best = max(pts, key=lambda p: (S[p[0], p[1]], -(p[1] - p[0])))
        if S[best[0], best[1]] > 0:
            cands.append(best)
    scores = [S[x, y] for x, y in cands]
    if len(set(scores)) != len(scores):
        pytest.skip("non-distinct scores; library tie order is unspecified")
    C = 5
    boxes = torch.tensor([[x, x, y + 1, y + 1] for x, y in cands], dtype=torch.float64).reshape(-1, 4)
    keep = tv.ops.nms(boxes, torch.tensor([float(s) for s in scores], dtype=torch.float64), phi_milli / 1000.0)[:C]
    kept = sorted(cands[i] for i in keep.tolist())
    expect, pos = [], 0
    for x, y in kept:
        if x > pos:
            expect.append([pos, x - pos])
        expect.append([x, y - x + 1])
        pos = max(pos, y + 1)          # with phi > 0 kept spans may overlap
    if pos < m:
        expect.append([pos, m - pos])
    spans, _ = orc.segment_map(Mq, thq, C, phi_milli)
    assert spans.tolist() == expect
    if phi_milli == 0:                  # a partition
        assert all(a[0] + a[1] == b[0] for a, b in zip(expect, expect[1:]))


def test_anti_diagonal_tie_prefers_shorter_span():
    # all-zero map with theta 0: every score is 0, nothing is a candidate -> one gap span
    spans, _ = orc.segment_map(np.zeros((6, 6), dtype=np.int32), 0, 4)
    assert spans.tolist() == [[0, 6]]
    # a map where [2,2] and [1,3] tie on anti-diagonal 4: the shorter one is the candidate
    Mq = np.zeros((5, 5), dtype=np.int32)
    Mq[2, 2] = 10
    thq = 0
    S = orc.ta_scores(Mq, thq)
    assert S[2, 2] == S[1, 3] == 10
    spans, _ = orc.segment_map(Mq, thq, 1)
    assert [2, 1] in spans.tolist()


@pytest.mark.parametrize("theta", [0.0, 0.5, 0.9, 0.95, 1.0])
def test_quantile_threshold_is_lower_nearest_rank(theta):
    rng = np.random.default_rng(11)
    m = 29
    Mq = rng.integers(0, 2**25, size=(m, m)).astype(np.int32)     # upper triangle must be ignored
    vals = Mq[np.tril_indices(m)]
    got = orc.theta_q(Mq, 1, theta, 32)
    assert got == int(np.quantile(vals, np.float32(theta).astype(np.float64), method="lower"))


def test_absolute_threshold_is_head_mean_probability():
    assert orc.theta_q(np.zeros((3, 3), np.int32), 0, 0.25, 8) == 8 * 2**18
    assert orc.theta_q(np.zeros((3, 3), np.int32), 0, 0.0, 8) == 0


def test_top_k_matches_stable_sort():
    rng = np.random.default_rng(12)
    for n, k in [(1, 4), (5, 5), (50, 7), (200, 32)]:
        sc = rng.integers(0, 20, size=n).astype(np.float32)        # many ties
        ids, _ = orc.top_k(sc, k)
        ref = np.argsort(-sc, kind="stable")[:k]
        assert ids[:len(ref)].tolist() == ref.tolist()
        assert np.all(ids[len(ref):] == -1)


def test_bf16_rounding_matches_torch():
    rng = np.random.default_rng(13)
    xs = np.concatenate([rng.standard_normal(500).astype(np.float32) * 100,
                         np.array([0.0, -0.0, 1.0, 1.00390625, 1.01171875, 3.3895314e38], dtype=np.float32)])
    for x in xs:
        ref = torch.tensor(float(x), dtype=torch.float32).to(torch.bfloat16).view(torch.int16).item() & 0xFFFF
        assert orc.f32_to_bf16(float(x)) == ref

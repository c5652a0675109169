"""Pins of the oracle's dynamic span index vectors (Sec. 3.3.2, Eq. r_v).

The area ratio is this build's reading of the paper's three metrics (span triangle against its row neighbours, its
column neighbours, or both); what the paper fixes is the shape of Eq. r_v -- r_v = 1 at r_a = 1 for every lambda,
r_v = e^(-lambda) at r_a = 0, a larger lambda keeps fewer vectors -- and that the count is span length x r_v within a
minimal and a maximal number.  The pins use maps whose sums have closed forms, worked out here by hand and with
exact rationals, never by calling the oracle.
"""
import math
from fractions import Fraction

import numpy as np
import pytest

from oracle import ltri_oracle as orc
from paper_2412_04757_b200 import inputs


def expected(L, ra: Fraction, lam, lo, hi):
    rv = 1.0 / math.exp(lam * (1.0 - float(ra)))
    x = L * rv
    # round half to even, like the oracle's nearbyint
    r = int(np.rint(x))
    return max(1, min(max(r, lo), hi, L))


@pytest.mark.parametrize("kind", [0, 1, 2])
@pytest.mark.parametrize("lam", [0.0, 0.7, 2.0, 6.0])
def test_uniform_map_closed_form(kind, lam):
    # every causal entry equals c: T = c L(L+1)/2, row neighbours c L x, column neighbours c L (m-1-y)
    m, c = 48, 1000
    M = np.tril(np.full((m, m), c, dtype=np.int32))
    for x, y in [(0, 0), (0, 9), (5, 5), (7, 30), (20, 47), (40, 47), (0, 47)]:
        L = y - x + 1
        T = Fraction(c * L * (L + 1), 2)
        R, Cn = Fraction(c * L * x), Fraction(c * L * (m - 1 - y))
        nb = [R, Cn, R + Cn][kind]
        ra = T / (T + nb)
        assert orc.dynamic_rep_count(M, x, y, kind, lam, 1, 8) == expected(L, ra, lam, 1, 8), (x, y)


def test_block_diagonal_map_keeps_every_token_up_to_the_maximum():
    # no mass outside the blocks: no neighbour knows the span, r_a = 1, r_v = 1 for any lambda (Eq. r_v)
    m = 40
    M = np.zeros((m, m), dtype=np.int32)
    blocks = [(0, 6), (7, 7), (8, 25), (26, 39)]
    for a, b in blocks:
        M[a:b + 1, a:b + 1] = 777
    M = np.tril(M)
    for lam in (0.5, 3.0, 50.0):
        for kind in (0, 1, 2):
            for a, b in blocks:
                assert orc.dynamic_rep_count(M, a, b, kind, lam, 1, 8) == min(b - a + 1, 8)
                assert orc.dynamic_rep_count(M, a, b, kind, lam, 1, 3) == min(b - a + 1, 3)


def test_span_without_own_mass_gets_exp_minus_lambda():
    # T = 0 with positive neighbours: r_a = 0, r_v = e^-lambda
    m = 32
    M = np.zeros((m, m), dtype=np.int32)
    M[10:20, 0:10] = 5     # rows of the span attend only to earlier tokens
    M[20:, 10:20] = 9      # later rows attend to the span's columns
    L = 10
    for lam in (0.0, 0.25, 1.0, 2.5):
        want = max(1, min(int(np.rint(L * math.exp(-lam))), 8))
        for kind in (0, 1, 2):
            assert orc.dynamic_rep_count(M, 10, 19, kind, lam, 1, 8) == want
    # an all-zero map has no neighbours either: r_a = 1 by convention
    assert orc.dynamic_rep_count(np.zeros((8, 8), np.int32), 2, 5, 2, 3.0, 1, 8) == 4


def test_row_and_column_neighbours_are_not_mixed_up():
    m = 24
    M = np.zeros((m, m), dtype=np.int32)
    x, y = 8, 15
    M[x:y + 1, x:y + 1] = np.tril(np.full((8, 8), 100, np.int32))   # T = 100 * 36
    M[x:y + 1, 0:x] = 450                                           # R = 450 * 64 = 8 T
    L, T = 8, 3600
    lam = 2.0
    row = expected(L, Fraction(T, T + 450 * 64), lam, 1, 8)
    assert orc.dynamic_rep_count(M, x, y, 0, lam, 1, 8) == row
    assert orc.dynamic_rep_count(M, x, y, 1, lam, 1, 8) == 8          # no column neighbours at all
    assert orc.dynamic_rep_count(M, x, y, 2, lam, 1, 8) == row
    M2 = M.copy()
    M2[x:y + 1, 0:x] = 0
    M2[y + 1:, x:y + 1] = 450                                         # the same mass, now below the span
    assert orc.dynamic_rep_count(M2, x, y, 0, lam, 1, 8) == 8
    assert orc.dynamic_rep_count(M2, x, y, 1, lam, 1, 8) == expected(L, Fraction(T, T + 450 * 8 * 8), lam, 1, 8)


def test_monotone_in_lambda_and_clamped():
    r = np.random.default_rng(5)
    M = np.tril(r.integers(0, 5000, size=(64, 64)).astype(np.int32))
    for x, y in [(0, 20), (10, 40), (33, 63)]:
        prev = None
        for lam in (0.0, 0.5, 1.0, 2.0, 4.0, 8.0, 30.0):
            c = orc.dynamic_rep_count(M, x, y, 2, lam, 2, 6)
            assert 2 <= c <= 6
            assert prev is None or c <= prev
            prev = c
        assert orc.dynamic_rep_count(M, x, y, 2, 0.0, 2, 6) == 6       # r_v = 1: span length, clamped
        assert orc.dynamic_rep_count(M, x, y, 2, 30.0, 2, 6) == 2      # r_v ~ 0: the minimal number


def test_stream_index_vectors_use_the_counts_decided_when_the_region_was_current():
    cfg = inputs.StreamConfig("dyn", 1, 4, 2, 128, 1024, 128, 0, 16, 256, 4, 4, 16, 64, seed=77, rep_mode=1,
                              ratio_kind=2, min_reps=1, max_reps=4, rep_lambda=1.0)
    st = inputs.SyntheticStream(cfg)
    o = orc.OracleStream(cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim, cfg.chunk, cfg.window, cfg.n_sink, cfg.top_k,
                         cfg.max_tokens, max_spans_per_region=cfg.max_spans_per_region, rep_mode=1, ratio_kind=2,
                         min_reps=1, max_reps=4, rep_lambda=1.0)
    counts, keys = {}, []
    for t0, n in st.prefill_chunks():
        q, k, v = st.tokens(t0, n)
        keys.append(k[0])
        o.prefill_local(q[0], k[0], v[0])
        rs, m = o.region()
        if m > 0:
            spans = o.pending()[-1][2]
            M = o.map()
            got = o.newest_rep_counts()
            for (s0, ln), c in zip(spans, got):
                # restated from the definition with numpy slices of the oracle's own integer map
                x, y = s0 - rs, s0 - rs + ln - 1
                T = int(np.tril(M[x:y + 1, x:y + 1]).sum())
                nb = int(M[x:y + 1, :x].sum()) + int(M[y + 1:, x:y + 1].sum())
                ra = Fraction(T, T + nb) if T + nb else Fraction(1)
                assert c == expected(ln, ra, 1.0, 1, 4)
                counts[int(s0)] = int(c)
        o.prefill_retrieve()
    K = np.concatenate([inputs.bf16_bits(x) for x in keys]).astype(np.uint32) << 16
    K = K.view(np.float32)                                   # [tokens][Hkv][d]
    spans, idx = o.spans(), o.index()
    assert len(spans) > 8 and len(set(counts.values())) > 1  # the counts really vary
    votes = o.votes(0, o.tokens)
    for s, (s0, ln) in enumerate(spans):
        c = counts[int(s0)]
        order = sorted(range(s0, s0 + ln), key=lambda t: (-int(votes[t]), t))[:c]
        want = K[sorted(order)].astype(np.float64).sum(0)    # [Hkv][d]
        got = (idx[s].astype(np.uint32) << 16).view(np.float32).astype(np.float64)
        assert np.all(np.abs(got - want) <= 2.0 ** -7 * np.maximum(np.abs(want), 1e-3)), s

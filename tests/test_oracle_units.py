"""Pins of the oracle's unit-granular retrieval (Eq. 8 as printed: fixed units of tokens are ranked by the maximum
score over their spans and fetched whole)."""
import numpy as np
import pytest

from oracle import ltri_oracle as orc
from paper_2412_04757_b200 import inputs


def f32(t):
    return (inputs.bf16_bits(t).astype(np.uint32) << 16).view(np.float32).astype(np.float64)


def make(cfg, top_k, unit):
    return orc.OracleStream(cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim, cfg.chunk, cfg.window, cfg.n_sink, top_k,
                            cfg.max_tokens, max_spans_per_region=cfg.max_spans_per_region, unit_tokens=unit)


def attention_fp64(q, K, V, tokens, scale):
    """q [d], K, V [T][d]: softmax attention over the given token list, in fp64."""
    s = K[tokens] @ q * scale
    p = np.exp(s - s.max())
    return (p / p.sum()) @ V[tokens]


@pytest.mark.parametrize("U", [32, 48, 128])
def test_unit_scores_selection_and_attended_tokens(U):
    cfg = inputs.StreamConfig("u", 1, 4, 2, 128, 1280, 128, 4, 16, 256, 3, 4, 16, 64, seed=41)
    st = inputs.SyntheticStream(cfg)
    o = make(cfg, 3, U)
    Ks, Vs = [], []
    G, scale = cfg.n_q_heads // cfg.n_kv_heads, 1.0 / np.sqrt(cfg.head_dim)
    checked = 0

    def check(q_rows, rows_abs, out, local_end_of_row):
        nonlocal checked
        K, V = np.concatenate(Ks), np.concatenate(Vs)          # [T][Hkv][d]
        spans, sc, E = o.spans(), o.scores(), o.evicted_end
        u0 = cfg.n_sink // U
        nu = (E + U - 1) // U - u0 if E > cfg.n_sink else 0
        sel, _ = o.selected()
        for g in range(cfg.n_kv_heads):
            # Eq. 8 restated: unit score = max over the spans that meet the unit; then the k best, ties to lower ids
            us = np.full(nu, -np.inf)
            for (s0, ln), v in zip(spans, sc[g]):
                for u in range(s0 // U, (s0 + ln - 1) // U + 1):
                    us[u - u0] = max(us[u - u0], v)
            assert np.array_equal(us.astype(np.float32), o.unit_scores()[g])
            want = sorted(np.argsort(-us, kind="stable")[:min(3, nu)] + u0)
            got = sorted(int(x) for x in sel[g] if x >= 0)
            assert got == [int(x) for x in want]
            toks_sel = [t for u in got for t in range(max(u * U, cfg.n_sink), min((u + 1) * U, E))]
            for r, (qrow, pos) in enumerate(zip(q_rows, rows_abs)):
                toks = list(range(0, min(cfg.n_sink, pos + 1))) + toks_sel + list(range(min(E, pos + 1), local_end_of_row(r)))
                assert len(set(toks)) == len(toks)
                for h in range(g * G, (g + 1) * G):
                    ref = attention_fp64(qrow[h], K[:, g], V[:, g], toks, scale)
                    assert np.abs(out[r, h] - ref).max() < 1e-4
                    checked += 1

    for t0, n in st.prefill_chunks():
        q, k, v = st.tokens(t0, n)
        Ks.append(f32(k[0]))
        Vs.append(f32(v[0]))
        out = o.prefill_chunk(q[0], k[0], v[0])
        if len(o.spans()) and t0 >= 768:
            rows = [0, n // 2, n - 1]
            check(f32(q[0])[rows], [t0 + r for r in rows], out[rows], lambda r: t0 + rows[r] + 1)
    for s in range(cfg.decode_steps):
        q, k, v = st.tokens(cfg.context + s, 1, kind=1)
        Ks.append(f32(k[0]))
        Vs.append(f32(v[0]))
        out = o.decode_step(q[0, 0], k[0, 0], v[0, 0])
        check(f32(q[0]), [cfg.context + s], out[None], lambda r: cfg.context + s + 1)
    assert checked > 50


def test_covering_every_unit_equals_full_attention():
    cfg = inputs.StreamConfig("u", 1, 4, 2, 128, 900, 128, 2, 16, 256, 64, 4, 16, 64, seed=42)
    st = inputs.SyntheticStream(cfg)
    o = make(cfg, 64, 64)
    for t0, n in st.prefill_chunks():
        q, k, v = st.tokens(t0, n)
        out = o.prefill_chunk(q[0], k[0], v[0])
        full = o.full_attention(list(range(t0, t0 + n)), q[0])
        assert np.abs(out - full).max() < 5e-6        # fp32 sums in a different key order
    for s in range(cfg.decode_steps):
        q, k, v = st.tokens(cfg.context + s, 1, kind=1)
        out = o.decode_step(q[0, 0], k[0, 0], v[0, 0])
        assert np.abs(out - o.full_attention([cfg.context + s], q[0])[0]).max() < 5e-6


@pytest.mark.parametrize("U", [0, 64])
def test_overlapping_spans_are_attended_once_per_token(U):
    # NMS with an IoU threshold above zero keeps overlapping spans; selecting all of them must still give plain
    # causal attention (every token once), span-granular and unit-granular
    cfg = inputs.StreamConfig("o", 1, 4, 2, 128, 1000, 128, 2, 16, 256, 64, 8, 16, 64, seed=43)
    st = inputs.SyntheticStream(cfg)
    o = orc.OracleStream(cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim, cfg.chunk, cfg.window, cfg.n_sink, 64,
                         cfg.max_tokens, max_spans_per_region=8, nms_iou_milli=500, unit_tokens=U)
    for t0, n in st.prefill_chunks():
        q, k, v = st.tokens(t0, n)
        out = o.prefill_chunk(q[0], k[0], v[0])
        assert np.abs(out - o.full_attention(list(range(t0, t0 + n)), q[0])).max() < 5e-6
    sp = o.spans()
    assert sum(a[0] + a[1] > b[0] for a, b in zip(sp, sp[1:])) > 3      # the spans really overlap
    assert sp[0][0] == cfg.n_sink and max(a[0] + a[1] for a in sp) == o.evicted_end
    for s in range(cfg.decode_steps):
        q, k, v = st.tokens(cfg.context + s, 1, kind=1)
        out = o.decode_step(q[0, 0], k[0, 0], v[0, 0])
        assert np.abs(out - o.full_attention([cfg.context + s], q[0])[0]).max() < 5e-6


# ---- segmentation per memory unit (Sec. 3.3: every unit is divided into spans on its own) ---------------------------
def block_map(m, blocks, inside=4000, outside=0):
    M = np.full((m, m), outside, dtype=np.int32)
    for a, b in blocks:
        M[a:b + 1, a:b + 1] = inside
    return np.tril(M)


@pytest.mark.parametrize("origin", [0, 64, 100, 37])
def test_per_unit_segmentation_of_block_maps_cuts_blocks_at_unit_boundaries(origin):
    # blocks of strong mutual attention; the expected spans are the blocks cut at the unit boundaries (closed form)
    U, m = 64, 200
    blocks = [(0, 29), (30, 79), (80, 139), (140, 199)]
    M = block_map(m, blocks)
    spans, _ = orc.segment_map(M, 2000, 8, 0, unit=U, origin=origin)   # inside +2000, outside -2000 per entry
    cuts = sorted({0, m} | {a for a, _ in blocks} | {u * U - origin for u in range(1, 8) if 0 < u * U - origin < m})
    want = [[a, b - a] for a, b in zip(cuts[:-1], cuts[1:])]
    assert spans.tolist() == want
    # one piece: the plain segmenter returns the blocks themselves
    plain, _ = orc.segment_map(M, 2000, 8, 0)
    assert plain.tolist() == [[a, b - a + 1] for a, b in blocks]


def test_per_unit_segmentation_properties_on_random_maps():
    r = np.random.default_rng(3)
    for trial in range(20):
        m, U, C = int(r.integers(40, 160)), int(r.choice([16, 32, 48])), int(r.integers(1, 5))
        origin = int(r.integers(0, 200))
        M = np.tril(r.integers(0, 3000, size=(m, m)).astype(np.int32))
        for a in range(0, m, 11):     # some structure
            M[a:a + 9, a:a + 9] += 5000
        M = np.tril(M)
        th = int(np.quantile(M[np.tril_indices(m)], 0.8))
        spans, _ = orc.segment_map(M, th, C, 0, unit=U, origin=origin)
        # a partition of the region whose spans never cross a unit boundary; at most 2C+1 spans per unit; a unit
        # that lies wholly inside the region is segmented exactly like a region made of that unit alone
        assert spans[0, 0] == 0 and (spans[1:, 0] == spans[:-1, 0] + spans[:-1, 1]).all()
        assert spans[-1, 0] + spans[-1, 1] == m
        per_unit = {}
        for s0, ln in spans:
            assert (origin + s0) // U == (origin + s0 + ln - 1) // U
            per_unit.setdefault((origin + s0) // U, []).append([int(s0), int(ln)])
        for u, sp in per_unit.items():
            assert len(sp) <= 2 * C + 1
            a, b = max(u * U - origin, 0), min((u + 1) * U - origin, m)
            alone, _ = orc.segment_map(M[a:b, a:b], th, C, 0)
            assert [[s0 - a, ln] for s0, ln in sp] == alone.tolist()
    # a region inside one unit is one piece
    M = np.tril(r.integers(0, 3000, size=(30, 30)).astype(np.int32))
    assert orc.segment_map(M, 1500, 3, 0, unit=64, origin=70)[0].tolist() == orc.segment_map(M, 1500, 3, 0)[0].tolist()


def test_per_unit_stream_spans_stay_inside_units_and_cover_the_context():
    cfg = inputs.StreamConfig("pu", 1, 4, 2, 128, 1100, 200, 0, 24, 256, 4, 2, 16, 64, seed=43)
    st = inputs.SyntheticStream(cfg)
    U = 64
    o = orc.OracleStream(cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim, cfg.chunk, cfg.window, cfg.n_sink, cfg.top_k,
                         cfg.max_tokens, max_spans_per_region=2, unit_tokens=U, segment_per_unit=1)
    for t0, n in st.prefill_chunks():
        q, k, v = st.tokens(t0, n)
        o.prefill_chunk(q[0], k[0], v[0])
    sp = o.spans()
    assert len(sp) > 10 and sp[0, 0] == cfg.n_sink and (sp[1:, 0] == sp[:-1, 0] + sp[:-1, 1]).all()
    assert ((sp[:, 0] // U) == ((sp[:, 0] + sp[:, 1] - 1) // U)).all()
    # (calls of 200 tokens: a unit that straddles two calls is segmented in two parts, each with its own cap)
    counts = np.bincount(sp[:, 0] // U)
    assert counts.max() <= 2 * (2 * 2 + 1)
    with pytest.raises(ValueError):
        orc.OracleStream(4, 2, 128, 128, 256, 16, 4, 1024, segment_per_unit=1)     # needs unit_tokens

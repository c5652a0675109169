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

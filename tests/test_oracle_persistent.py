"""Pins of the oracle's persistent mechanism (Sec. 3.5): during decode the spans retrieved by the last prefill call
stay in the attention next to the spans each step retrieves itself."""
import numpy as np

from oracle import ltri_oracle as orc
from paper_2412_04757_b200 import inputs


def make(cfg, top_k, persist):
    return orc.OracleStream(cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim, cfg.chunk, cfg.window, cfg.n_sink, top_k,
                            cfg.max_tokens, max_spans_per_region=cfg.max_spans_per_region, persist_decode=persist)


def test_decode_attends_over_the_union_every_span_once():
    cfg = inputs.StreamConfig("p", 1, 4, 2, 128, 1024, 128, 6, 16, 256, 3, 4, 16, 64, seed=31)
    st = inputs.SyntheticStream(cfg)
    a = make(cfg, 3, 1)          # persistent mechanism on
    b = make(cfg, 3, 0)          # off: the plain per-step retrieval
    c = make(cfg, 6, 0)          # a wider oracle that is handed the union explicitly
    for t0, n in st.prefill_chunks():
        q, k, v = st.tokens(t0, n)
        for o in (a, b, c):
            o.prefill_local(q[0], k[0], v[0])
            o.prefill_retrieve()
    last_sel, _ = a.selected()
    assert (last_sel >= 0).all()
    assert (a.persistent() == -1).all()                      # nothing is kept before the first decode step
    differs = 0
    for s in range(cfg.decode_steps):
        q, k, v = st.tokens(cfg.context + s, 1, kind=1)
        for o in (a, b, c):
            o.decode_retrieve(q[0, 0], k[0, 0], v[0, 0])
        assert np.array_equal(a.persistent(), last_sel)      # kept unchanged through decode
        step_sel, _ = a.selected()
        assert np.array_equal(step_sel, b.selected()[0])     # the step's own retrieval is not affected
        union = np.full((cfg.n_kv_heads, 6), -1, dtype=np.int32)
        for g in range(cfg.n_kv_heads):
            ids = [int(x) for x in step_sel[g] if x >= 0]
            ids += [int(x) for x in last_sel[g] if x >= 0 and int(x) not in ids]
            union[g, :len(ids)] = ids
            differs += len(ids) > 3
        c.set_selected(union)
        out_a, out_b, out_c = a.decode_attend(), b.decode_attend(), c.decode_attend()
        assert np.array_equal(out_a, out_c)                  # same keys, same order: the same arithmetic
        if (union[:, 3:] >= 0).any():
            assert not np.array_equal(out_a, out_b)
    assert differs > 0                                       # the case is not vacuous


def test_covering_everything_still_equals_full_attention():
    cfg = inputs.StreamConfig("p", 1, 4, 2, 128, 768, 128, 3, 16, 256, 64, 4, 16, 64, seed=32)
    st = inputs.SyntheticStream(cfg)
    o = make(cfg, 64, 1)
    for t0, n in st.prefill_chunks():
        q, k, v = st.tokens(t0, n)
        o.prefill_chunk(q[0], k[0], v[0])
    for s in range(cfg.decode_steps):
        q, k, v = st.tokens(cfg.context + s, 1, kind=1)
        out = o.decode_step(q[0, 0], k[0, 0], v[0, 0])
        full = o.full_attention([cfg.context + s], q[0])
        assert np.abs(out - full[0]).max() < 2e-6

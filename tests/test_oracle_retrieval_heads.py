"""Pins of the oracle's retrieval heads and collaborative voting (Sec. 3.5).

A layer with a retrieval head locates evidence with that head alone.  The pin: on the head's own data the layer must
behave exactly like a one-head model made of that head and its KV head -- same map, threshold, spans, votes, index
vectors, scores, selection and attention output -- and the selection must serve the layer's other KV heads too.
Voting is pinned by restating the ranking with numpy on hand-made ballots, by its degenerate cases (no ballots, zero
weights) and by the full-attention identity.
"""
import numpy as np
import pytest

from oracle import ltri_oracle as orc
from paper_2412_04757_b200 import inputs


def f32(t):
    return (inputs.bf16_bits(t).astype(np.uint32) << 16).view(np.float32).astype(np.float64)


def make(cfg, Hq=None, Hkv=None, **kw):
    return orc.OracleStream(Hq or cfg.n_q_heads, Hkv or cfg.n_kv_heads, cfg.head_dim, cfg.chunk, cfg.window,
                            cfg.n_sink, cfg.top_k, cfg.max_tokens, max_spans_per_region=cfg.max_spans_per_region,
                            theta_mode=cfg.theta_mode, theta=cfg.theta, **kw)


@pytest.mark.parametrize("head,theta_mode,unit", [(5, 1, 0), (2, 0, 0), (7, 1, 64)])
def test_retrieval_head_layer_equals_the_one_head_model_of_that_head(head, theta_mode, unit):
    cfg = inputs.StreamConfig("rh", 1, 8, 2, 128, 1536, 128, 3, 16, 256, 3, 4, 16, 64, seed=11 + head,
                              theta_mode=theta_mode, theta=0.90 if theta_mode else 0.004)
    G = cfg.n_q_heads // cfg.n_kv_heads
    g = head // G
    st = inputs.SyntheticStream(cfg)
    a = make(cfg, ret_head=head, head_weight=0.5, unit_tokens=unit)
    b = make(cfg, Hq=1, Hkv=1, unit_tokens=unit)
    scale = 1.0 / np.sqrt(cfg.head_dim)
    Ks, Vs = [], []
    n_sel = 0

    def same_retrieval():
        nonlocal n_sel
        assert a.spans().tolist() == b.spans().tolist()
        assert a.evicted_end == b.evicted_end
        if len(a.spans()):
            assert np.array_equal(a.index()[:, g], b.index()[:, 0])
            sa, sb = a.scores(), b.scores()
            for gg in range(cfg.n_kv_heads):                   # one selection for the layer
                assert np.array_equal(sa[gg], sb[0])
                assert a.selected()[0][gg].tolist() == b.selected()[0][0].tolist()
            n_sel += 1

    for t0, n in st.prefill_chunks():
        q, k, v = st.tokens(t0, n)
        Ks.append(f32(k[0]))
        Vs.append(f32(v[0]))
        a.prefill_local(q[0], k[0], v[0])
        b.prefill_local(q[0][:, head:head + 1], k[0][:, g:g + 1], v[0][:, g:g + 1])
        assert np.array_equal(a.map(), b.map())
        assert a.theta_q() == b.theta_q()
        assert a.pending()[-1][2].tolist() == b.pending()[-1][2].tolist() if a.region()[1] else True
        assert np.array_equal(a.votes(0, a.tokens), b.votes(0, b.tokens))
        a.prefill_retrieve()
        b.prefill_retrieve()
        same_retrieval()
        oa, ob = a.prefill_attend(), b.prefill_attend()
        assert np.array_equal(oa[:, head], ob[:, 0])
        # the other heads attend over the same tokens: check one head of another KV head against plain softmax
        if len(a.spans()) and t0 >= 1024:
            K, V = np.concatenate(Ks), np.concatenate(Vs)
            sel = [int(x) for x in a.selected()[0][0] if x >= 0]
            E = a.evicted_end
            if unit:
                toks_sel = [t for u in sel for t in range(max(u * unit, cfg.n_sink), min((u + 1) * unit, E))]
            else:
                sp = a.spans()
                toks_sel = [t for s in sel for t in range(sp[s, 0], sp[s, 0] + sp[s, 1])]
            h2 = (head + G) % cfg.n_q_heads
            g2 = h2 // G
            r = n - 1
            toks = list(range(cfg.n_sink)) + toks_sel + list(range(E, t0 + r + 1))
            s = K[toks][:, g2] @ f32(q[0])[r, h2] * scale
            p = np.exp(s - s.max())
            ref = (p / p.sum()) @ V[toks][:, g2]
            assert np.abs(oa[r, h2] - ref).max() < 1e-4
    for s in range(cfg.decode_steps):
        q, k, v = st.tokens(cfg.context + s, 1, kind=1)
        oa = a.decode_step(q[0, 0], k[0, 0], v[0, 0])
        ob = b.decode_step(q[0, 0][head:head + 1], k[0, 0][g:g + 1], v[0, 0][g:g + 1])
        same_retrieval()
        assert np.array_equal(oa[head], ob[0])
    assert n_sel >= 8


def vote_cfg(**kw):
    return inputs.StreamConfig("cv", 1, 4, 2, 128, 1792, 128, 2, 16, 256, 3, 4, 16, 64, seed=23, **kw)


def run_to_last_chunk(o, cfg, layer=0):
    st = inputs.SyntheticStream(cfg)
    chunks = list(st.prefill_chunks())
    for t0, n in chunks[:-1]:
        q, k, v = st.tokens(t0, n)
        o.prefill_chunk(q[layer], k[layer], v[layer])
    t0, n = chunks[-1]
    q, k, v = st.tokens(t0, n)
    o.prefill_local(q[layer], k[layer], v[layer])
    return st


def ranking(us, tally, k):
    """The voting order restated with numpy: tally first, own score next, lower id last."""
    idx = np.lexsort((np.arange(len(us)), -us.astype(np.float64), -tally.astype(np.float64)))
    return idx[:min(k, len(us))]


def test_no_ballots_or_zero_weights_leave_the_selection_alone():
    cfg = vote_cfg()
    U = 64
    plain = make(cfg, unit_tokens=U)
    run_to_last_chunk(plain, cfg)
    plain.prefill_retrieve()
    want = plain.selected()[0]
    for kw, ballots in [(dict(), []), (dict(ret_head=1, head_weight=0.0), [(0.0, [3, 5, 7])]),
                        (dict(), [(0.0, [2, 4, -1])])]:
        o = make(cfg, unit_tokens=U, collab_vote=1, **kw)
        run_to_last_chunk(o, cfg)
        o.set_ballots(ballots)
        o.prefill_retrieve()
        if "ret_head" in kw:
            ref = make(cfg, unit_tokens=U, **kw)
            run_to_last_chunk(ref, cfg)
            ref.prefill_retrieve()
            assert o.selected()[0].tolist() == ref.selected()[0].tolist()
            assert o.ballot().tolist() == ref.selected()[0][0].tolist()
        else:
            assert o.selected()[0].tolist() == want.tolist()
            assert o.ballot().tolist() == [-1] * cfg.top_k      # no retrieval head: no ballot
        assert not o.tally().any()


@pytest.mark.parametrize("ret_head,hw", [(-1, 0.0), (2, 0.25), (0, 1.5)])
def test_ranking_by_tally_then_own_score(ret_head, hw):
    cfg = vote_cfg()
    U = 64
    o = make(cfg, unit_tokens=U, collab_vote=1, ret_head=ret_head, head_weight=hw)
    run_to_last_chunk(o, cfg)
    u0 = cfg.n_sink // U
    nu = (o.evicted_end + U - 1) // U - u0
    assert nu > 12
    # 0.3 + 0.3 beats 0.5; a unit outside the indexed range and the -1 padding are ignored; equal tallies fall back
    # to the own scores
    ballots = [(0.3, [u0 + 1, u0 + 9, u0 + 4]), (0.5, [u0 + 2, u0 + 4, -1]), (0.3, [u0 + 1, u0 + nu + 3, u0 + 6])]
    o.set_ballots(ballots)
    o.prefill_retrieve()
    us = o.unit_scores()
    own = o.ballot()
    tally = np.zeros(nu, dtype=np.float32)
    for w, ids in ballots:
        for i in ids:
            if 0 <= i - u0 < nu:
                tally[i - u0] += np.float32(w)
    if ret_head >= 0:
        # the own ballot is the own top-k of the retrieval head's scores, and it votes too
        assert sorted(own.tolist()) == sorted((np.argsort(-us[0], kind="stable")[:cfg.top_k] + u0).tolist())
        for i in own:
            tally[i - u0] += np.float32(hw)
    else:
        assert own.tolist() == [-1] * cfg.top_k
    assert np.array_equal(o.tally(), tally)
    sel = o.selected()[0]
    for g in range(cfg.n_kv_heads):
        assert sel[g].tolist() == (ranking(us[g], tally, cfg.top_k) + u0).tolist()
    # with these weights the two-ballot unit leads and the 0.5 unit comes before the single 0.3 ones
    if ret_head < 0:
        assert sel[0][0] in (u0 + 1, u0 + 4) and set(sel[0][:2].tolist()) == {u0 + 1, u0 + 4}
        assert sel[0][2] == u0 + 2


def test_votes_only_reorder_when_every_unit_is_fetched():
    # top_k >= number of units: whatever the ballots, every unit is fetched and the output is full causal attention
    cfg = inputs.StreamConfig("cv", 1, 4, 2, 128, 1024, 128, 2, 16, 256, 64, 4, 16, 64, seed=29)
    U = 32
    st = inputs.SyntheticStream(cfg)
    o = make(cfg, unit_tokens=U, collab_vote=1, ret_head=3, head_weight=0.7)
    qs, pos = [], []
    for t0, n in st.prefill_chunks():
        q, k, v = st.tokens(t0, n)
        o.prefill_local(q[0], k[0], v[0])
        o.set_ballots([(0.4, list(range(t0 % 7, t0 % 7 + 5)) + [-1] * 59)])
        o.prefill_retrieve()
        out = o.prefill_attend()
        ref = o.full_attention(np.arange(t0, t0 + n), q[0])
        assert np.abs(out - ref).max() < 5e-6
    for s in range(cfg.decode_steps):
        q, k, v = st.tokens(cfg.context + s, 1, kind=1)
        out = o.decode_step(q[0, 0], k[0, 0], v[0, 0])
        ref = o.full_attention(np.array([cfg.context + s]), q[0])
        assert np.abs(out - ref[0]).max() < 5e-6


def test_bad_parameters():
    cfg = vote_cfg()
    with pytest.raises(ValueError):
        make(cfg, collab_vote=1)                      # voting needs units: span ids differ between layers
    with pytest.raises(ValueError):
        make(cfg, ret_head=cfg.n_q_heads)
    with pytest.raises(ValueError):
        make(cfg, ret_head=0, head_weight=-0.1)

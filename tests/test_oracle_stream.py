"""Pins for the oracle's streaming state, retrieval and attention (Sec. 3.3-3.4, Eq. 6-8).

References used: torch's scaled_dot_product_attention in fp64 (a library routine), fp64
numpy restatements written from the definitions, brute-force double sums, and the
full-attention equivalence (when top-k covers every indexed span the streamed output is
plain causal attention).
"""
import numpy as np
import pytest
import torch

from oracle import ltri_oracle as orc
from paper_2412_04757_b200 import inputs


def f32(t):
    return t.to(torch.float32).numpy().astype(np.float64)


def sdpa_causal(q, k, v, positions, G):
    """fp64 causal attention of rows q[r] (at absolute positions[r]) over k,v[0..pos]."""
    q64, k64, v64 = (torch.from_numpy(f32(x)) for x in (q, k, v))
    out = np.zeros((len(positions), q.shape[1], q.shape[2]))
    for r, pos in enumerate(positions):
        for h in range(q.shape[1]):
            g = h // G
            o = torch.nn.functional.scaled_dot_product_attention(
                q64[r, h][None, None, None, :], k64[: pos + 1, g][None, None], v64[: pos + 1, g][None, None])
            out[r, h] = o[0, 0, 0].numpy()
    return out


def make(Hq=4, Hkv=2, d=16, chunk=16, window=32, sink=4, top_k=3, T=160, **kw):
    return orc.OracleStream(Hq, Hkv, d, chunk, window, sink, top_k, T, **kw)


def run_prefill(o, q, k, v, chunk, upto=None):
    outs = []
    T = q.shape[0] if upto is None else upto
    for t0 in range(0, T, chunk):
        n = min(chunk, T - t0)
        outs.append(o.prefill_chunk(q[t0:t0 + n], k[t0:t0 + n], v[t0:t0 + n]))
    return np.concatenate(outs)


def test_full_attention_matches_library_sdpa():
    q, k, v = inputs.random_stream(1, 40, 4, 2, 16)
    o = make(T=64, chunk=64, window=64)
    o.prefill_local(q, k, v)
    pos = [0, 1, 7, 39]
    got = o.full_attention(pos, q[pos])
    ref = sdpa_causal(q[pos], k, v, pos, 2)
    assert np.abs(got - ref).max() < 2e-5


@pytest.mark.parametrize("seed,window,chunk", [(2, 32, 16), (3, 48, 16), (4, 20, 8)])
def test_topk_covering_all_spans_equals_full_attention(seed, window, chunk):
    T = 150
    q, k, v = inputs.random_stream(seed, T, 4, 2, 16, sharp=2.0)
    o = make(T=T + 8, chunk=chunk, window=window, top_k=64, max_spans_per_region=3)
    out = run_prefill(o, q, k, v, chunk)
    assert o.spans().shape[0] > 0                       # something was evicted and indexed
    ref = sdpa_causal(q, k, v, list(range(T)), 2)
    assert np.abs(out - ref).max() < 3e-5
    # decode on top: still full attention
    qd, kd, vd = inputs.random_stream(seed + 50, 4, 4, 2, 16)
    kall, vall = torch.cat([k, kd]), torch.cat([v, vd])
    for s in range(4):
        got = o.decode_step(qd[s], kd[s], vd[s])
        ref = sdpa_causal(qd[s:s + 1], kall, vall, [T + s], 2)[0]
        assert np.abs(got - ref).max() < 3e-5


def test_rows_of_ones_values_give_ones():
    # softmax rows sum to 1: with V == 1 every output element is 1
    T = 96
    q, k, v = inputs.random_stream(5, T, 4, 2, 16)
    v = torch.ones_like(v)
    o = make(T=T, top_k=2)
    out = run_prefill(o, q, k, v, 16)
    assert np.abs(out - 1.0).max() < 1e-5


def local_map_fp64(q, k, t0, n, sink_end, loc_begin, G, scale):
    """A_loc[h][r][j] over absolute key index j (0 where the key is not visible)."""
    Hq = q.shape[1]
    A = np.zeros((Hq, n, t0 + n))
    qf, kf = f32(q), f32(k)
    for h in range(Hq):
        g = h // G
        for r in range(n):
            i = t0 + r
            keys = list(range(0, sink_end)) + list(range(loc_begin, i + 1))
            s = kf[keys, g] @ qf[i, h] * scale
            p = np.exp(s - s.max())
            A[h, r, keys] = p / p.sum()
    return A


def test_votes_map_and_index_follow_eq6():
    Hq, Hkv, d, chunk, W, Ls, T = 4, 2, 16, 16, 32, 4, 128
    G = Hq // Hkv
    q, k, v = inputs.random_stream(6, T, Hq, Hkv, d, sharp=2.0)
    o = make(Hq, Hkv, d, chunk, W, Ls, 2, T, max_spans_per_region=3)
    votes = np.zeros(T)
    E = Ls
    scale = 1.0 / np.sqrt(d)
    regions = []
    for t0 in range(0, T, chunk):
        # eviction happens first
        while regions and regions[0][1] <= t0 - W:
            E = regions.pop(0)[1]
        o.prefill_local(q[t0:t0 + chunk], k[t0:t0 + chunk], v[t0:t0 + chunk])
        assert o.evicted_end == E
        sink_end, loc_begin = min(Ls, t0), min(E, t0)
        A = local_map_fp64(q, k, t0, chunk, sink_end, loc_begin, G, scale) * 2**20
        lo = max(loc_begin, Ls)
        votes[lo:t0 + chunk] += A[:, :, lo:].sum(axis=(0, 1))
        got = o.votes(0, t0 + chunk).astype(np.float64)
        # every entry is rounded once per (head,row): |error| <= 0.5 each, plus fp32 noise
        assert np.abs(got - votes[:t0 + chunk]).max() <= 0.5 * Hq * chunk * (t0 // chunk + 1) * 0.2 + 8
        rs, m = o.region()
        assert rs == max(Ls, t0) and m == t0 + chunk - rs
        M = A[:, rs - t0:, rs:].sum(axis=0)
        assert np.abs(o.map() - np.tril(M)).max() <= Hq * 0.5 + 2
        assert np.all(np.triu(o.map(), 1) == 0)
        regions.append((rs, t0 + chunk))
        o.prefill_retrieve()
    # index vectors (one representative): the key of the most voted token of each span
    spans, idx = o.spans(), o.index()
    assert len(spans) > 3
    kb = inputs.bf16_bits(k)
    final_votes = o.votes(0, T)
    for s, (st, ln) in enumerate(spans):
        tok = st + int(np.argmax(final_votes[st:st + ln]))        # first maximum = lower index
        assert np.array_equal(idx[s], kb[tok])


def test_state_tiles_the_stream_after_every_call():
    T, chunk, W, Ls = 200, 24, 40, 10
    q, k, v = inputs.random_stream(7, T, 4, 2, 16, sharp=2.0)
    o = make(T=T, chunk=chunk, window=W, sink=Ls, top_k=2, max_spans_per_region=2)
    t0 = 0
    sizes = [24, 7, 24, 1, 24, 24, 13, 24, 24, 24, 11]
    for n in sizes:
        o.prefill_chunk(q[t0:t0 + n], k[t0:t0 + n], v[t0:t0 + n])
        t0 += n
        pos = Ls
        for st, ln in o.spans():
            assert st == pos and ln >= 1
            pos += ln
        assert pos == o.evicted_end
        for rs, re, sp in o.pending():
            assert rs == pos and len(sp) <= 2 * 2 + 1
            for st, ln in sp:
                assert st == pos and ln >= 1
                pos += ln
            assert pos == re
        assert pos == max(t0, Ls)
        # the local set never holds fewer than `window` tokens once the stream is long enough
        if t0 - n - Ls >= W + chunk:
            assert (t0 - n) - o.evicted_end >= W


def test_eq7_is_bilinear_and_scores_take_max_over_query_spans():
    Hq, Hkv, d, chunk, W, Ls, T, reps = 4, 2, 16, 16, 16, 4, 96, 3
    G = Hq // Hkv
    q, k, v = inputs.random_stream(8, T, Hq, Hkv, d, sharp=2.0)
    o = make(Hq, Hkv, d, chunk, W, Ls, 2, T, reps_per_span=reps, max_spans_per_region=2)
    qf, kf = f32(q), f32(k)
    evict_votes = {}
    for t0 in range(0, T, chunk):
        o.prefill_local(q[t0:t0 + chunk], k[t0:t0 + chunk], v[t0:t0 + chunk])
        for st, ln in o.spans():
            evict_votes.setdefault((int(st), int(ln)), o.votes(st, st + ln))   # votes are final once evicted
        o.prefill_retrieve()
    spans = o.spans()
    assert len(spans) >= 3
    # key representatives from the votes, by the stated rule (largest votes, ties -> lower index)
    def top_tokens(st, votes):
        order = sorted(range(len(votes)), key=lambda i: (-int(votes[i]), i))[:reps]
        return [st + i for i in sorted(order)]
    qtok = o.query_rep_tokens()
    rs, m = o.region()
    pend = o.pending()[-1][2]
    cur_votes = o.votes(rs, rs + m)
    for j, (st, ln) in enumerate(pend):
        assert [t for t in qtok[j] if t >= 0] == top_tokens(st, cur_votes[st - rs:st - rs + ln])
    sc = o.scores()
    idx = o.index()
    for g in range(Hkv):
        for s, (st, ln) in enumerate(spans):
            ktoks = top_tokens(int(st), evict_votes[(int(st), int(ln))])
            best = -np.inf
            for j in range(len(pend)):
                toks = [t for t in qtok[j] if t >= 0]
                # Eq. 7 as printed: the double sum over every (query rep, key rep) pair
                dbl = sum(float(qf[tq, h] @ kf[tk, g]) for h in range(g * G, (g + 1) * G) for tq in toks for tk in ktoks)
                best = max(best, dbl)
            # the stored index vector is the bf16-rounded sum of keys: allow that rounding
            assert abs(sc[g, s] - best) <= 2e-2 * (1 + abs(best))
            if len(ktoks) == 1:
                assert np.array_equal(idx[s, g], inputs.bf16_bits(k)[ktoks[0], g])
    ids, _ = o.selected()
    for g in range(Hkv):
        ref = np.argsort(-sc[g], kind="stable")[:2]
        assert ids[g].tolist() == ref.tolist()


def test_retrieval_finds_the_planted_segment():
    # planted-segment stream: queries aimed at an evicted segment must retrieve spans inside it
    cfg = inputs.config(0)
    st = inputs.SyntheticStream(cfg)
    o = orc.OracleStream(cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim, cfg.chunk, cfg.window, cfg.n_sink,
                         cfg.top_k, cfg.max_tokens, max_spans_per_region=cfg.max_spans_per_region)
    for t0, n in st.prefill_chunks():
        q, k, v = st.tokens(t0, n)
        out = o.prefill_chunk(q[0], k[0], v[0])
        assert np.isfinite(out).all()
    spans = o.spans()
    assert len(spans) > 0 and spans[:, 0][0] == cfg.n_sink
    hits = tot = 0
    for s in range(cfg.decode_steps):
        q, k, v = st.tokens(cfg.context + s, 1, kind=1)
        o.decode_retrieve(q[0], k[0], v[0])
        tgt = st.target[0, cfg.context + s]
        lo, hi = st.bounds[tgt], st.bounds[tgt + 1]
        if hi <= o.evicted_end and lo >= cfg.n_sink:
            ids, _ = o.selected()
            for g in range(cfg.n_kv_heads):
                tot += 1
                sel = [tuple(spans[i]) for i in ids[g] if i >= 0]
                hits += any(a < hi and a + ln > lo for a, ln in sel)
        o.decode_attend()
    assert tot > 0 and hits / tot > 0.7


def test_continuing_from_a_loaded_state_reproduces_the_stream():
    # the state hooks (used by the full-size GPU checks) must not change what the oracle computes
    Hq, Hkv, d, chunk, W, Ls, T = 4, 2, 16, 16, 32, 4, 160
    q, k, v = inputs.random_stream(21, T, Hq, Hkv, d, sharp=2.0)
    a = make(Hq, Hkv, d, chunk, W, Ls, 3, T, max_spans_per_region=3)
    outs, states = [], []
    for t0 in range(0, T, chunk):
        states.append((a.evicted_end, a.spans().copy(), a.index().copy(), a.pending()))
        outs.append(a.prefill_chunk(q[t0:t0 + chunk], k[t0:t0 + chunk], v[t0:t0 + chunk]))
    for c in (5, 8):
        t0 = c * chunk
        b = make(Hq, Hkv, d, chunk, W, Ls, 3, T, max_spans_per_region=3)
        b.append_only(k[:t0], v[:t0])
        # state at the START of call c is the state after eviction: take it from the original after the call
        E_after, spans_after, idx_after = states[c + 1][0], states[c + 1][1], states[c + 1][2]
        b.load_state(E_after, spans_after, idx_after)
        for (rs, re, sp) in states[c + 1][3][:-1]:          # regions still pending, without call c's own region
            b.add_pending(rs, re, sp)
        got = b.prefill_chunk(q[t0:t0 + chunk], k[t0:t0 + chunk], v[t0:t0 + chunk])
        assert np.array_equal(got, outs[c])
        assert b.pending()[-1][2].tolist() == a_pending_of(states, c)


def a_pending_of(states, c):
    return states[c + 1][3][-1][2].tolist()


def test_state_errors():
    q, k, v = inputs.random_stream(9, 40, 4, 2, 16)
    o = make(T=40)
    o.prefill_chunk(q[:16], k[:16], v[:16])
    o.decode_step(q[16], k[16], v[16])
    with pytest.raises(RuntimeError):
        o.prefill_local(q[17:33], k[17:33], v[17:33])          # prefill after decode
    o2 = make(T=20)
    o2.prefill_chunk(q[:16], k[:16], v[:16])
    with pytest.raises(RuntimeError):
        o2.prefill_local(q[16:32], k[16:32], v[16:32])          # capacity

"""Parity at the benchmark's full sizes (configs 1-4 as bench.py runs them: 32K and 128K x 32 layers, 1M x 8 layers,
16 sequences x 128K x 4 layers).

The oracle cannot stream these, so outputs are sampled: for two layers the oracle is brought to the
GPU's state at the start of a call (cache contents, span table, index, pending regions) and then computes that
call itself -- local map, threshold, segmentation, query representatives, scores, top-k, attention rows -- which
are compared with what the GPU produced for the same call: the last call of every config, and on the headline
config also the first call with an index, a mid-stream call and the call before the last.  A second check rebuilds
the votes of one region over the nine calls it spends in the window and compares the index vectors it gets at
eviction; a third continues into decode (the first three steps; on the headline config also the last of its 256).
Every upstream quantity the oracle is seeded with is itself covered by one of these samples.
"""
import numpy as np
import pytest
import torch

from oracle import ltri_oracle as orc
from paper_2412_04757_b200 import binding, inputs
from tests import parity_harness as ph

pytestmark = pytest.mark.gpu


def regions_from_table(spans, lo, hi, chunk):
    """Split the span table rows covering [lo,hi) into chunk-aligned regions."""
    out = []
    for rs in range(lo, hi, chunk):
        sp = spans[(spans[:, 0] >= rs) & (spans[:, 0] < rs + chunk)]
        assert sp[0, 0] == rs and sp[-1, 0] + sp[-1, 1] == rs + chunk
        out.append((rs, rs + chunk, sp))
    return out


# (config, sampled layers, sampled sequence): the 1M-token config keeps one layer on the host (4 GB of K/V).  The
# headline config (2) samples its first and last layer and, besides the last call, the first call that has an
# index to retrieve from, one mid-stream call, the call before the last, and the last decode step as well
CASES = [(1, [0, 31], 0), (2, [0, 31], 0), (3, [5], 0), (4, [2], 11)]


def check_call(lt, cfg, l, SEQ, t0, Kall, Vall, q_call, out_call, rep, rows, what):
    """Right after the GPU has run the prefill call that starts at t0: bring an oracle to the GPU's state behind that
    call's eviction step (cache, span table, index, pending regions), let it compute the call itself, compare the
    region map, threshold, segmentation, scores, selection and sampled output rows.  Returns the oracle."""
    n, W = cfg.chunk, cfg.window
    spans_g = lt.ltri_get_spans(SEQ, l)
    idx_g = lt.ltri_debug_read(binding.BUF_INDEX, SEQ, l)[:, :len(spans_g)].transpose(1, 0, 2).copy()
    E = int(lt.ltri_get_stats(SEQ, l).evicted_end)
    assert E == t0 - W and spans_g[-1, 0] + spans_g[-1, 1] == E
    pend_g = lt.ltri_get_pending_spans(SEQ, l)
    o = ph.oracle_of(cfg)
    o.append_only(Kall[:t0], Vall[:t0])
    o.load_state(E, spans_g, idx_g)
    for (rs, re, sp) in regions_from_table(pend_g, E, t0, n):
        o.add_pending(rs, re, sp)
    o.prefill_local(q_call, Kall[t0:], Vall[t0:])
    rs, m = o.region()
    Mg = np.tril(lt.ltri_debug_read(binding.BUF_MAP, SEQ, l)[:m, :m])
    md = int(np.abs(Mg.astype(np.int64) - o.map()).max())
    rep.max_map_diff = max(rep.max_map_diff, md)
    assert md <= 4 + cfg.n_q_heads, f"{what}: region map differs by {md}"
    thg = int(lt.ltri_debug_read(binding.BUF_THETA, SEQ, l)[0])
    assert abs(thg - o.theta_q()) <= 4 + cfg.n_q_heads
    newest_g = pend_g[pend_g[:, 0] >= rs]
    ref_spans, _ = orc.segment_map(Mg, thg, cfg.max_spans_per_region)
    ref_spans[:, 0] += rs
    assert newest_g.tolist() == ref_spans.tolist(), f"{what}: segmenter on its own map"
    if newest_g.tolist() != o.pending()[-1][2].tolist():
        assert o.seg_gap() < ph.NEAR_TIE, f"{what}: spans differ without a near tie"
        o.set_newest_spans(newest_g)
        rep.span_flips += 1
    o.prefill_retrieve()
    sg = lt.ltri_debug_read(binding.BUF_SCORES, SEQ, l)[:, :len(spans_g)]
    so = o.scores()
    assert np.abs(sg - so).max() / np.abs(so).max() <= 2e-5, f"{what}: scores"
    ph.check_selection(lt.ltri_get_selected(SEQ, l), o, rep, what)
    for r in rows:
        ph.check_output(out_call[l, r:r + 1], o.prefill_attend(r, r + 1), rep, f"{what} row {r}")
    return o, spans_g, idx_g, pend_g


@pytest.mark.parametrize("cfg_idx,LAYERS,SEQ", CASES, ids=[f"cfg{c[0]}" for c in CASES])
def test_sampled_calls_match_the_oracle(cfg_idx, LAYERS, SEQ):
    cfg = inputs.config(cfg_idx)
    dev = torch.device("cuda:0")
    lt = binding.Ltri(ph.params_of(cfg), device=dev)
    L, n, W = cfg.n_layers, cfg.chunk, cfg.window
    ROWS = [0, 1, n // 2 - 1, n // 2, n - 2, n - 1]
    # the other sequences of a batched config are streamed first (they only have to be there for the decode batch)
    others = [s for s in range(cfg.n_seqs) if s != SEQ]
    for s in others:
        so = inputs.SyntheticStream(cfg, seq=s, device=dev)
        for (t0, cnt) in so.prefill_chunks():
            lt.ltri_prefill_chunk(s, 0, L, *so.tokens(t0, cnt))
    st = inputs.SyntheticStream(cfg, seq=SEQ, device=dev)
    chunks = list(st.prefill_chunks())
    last = len(chunks) - 1
    first_indexed = (W + n - 1) // n + 1          # first call whose eviction step leaves a non-empty index
    sampled = {last} if cfg_idx != 2 else {first_indexed, len(chunks) // 2, last - 1, last}
    K = {l: [] for l in LAYERS}
    V = {l: [] for l in LAYERS}
    Q = {l: {} for l in LAYERS}
    probe_call = len(chunks) - 14          # region whose index vectors are rebuilt (evicted 9 calls later)
    snap, state = {}, {}
    rep = ph.Report()
    for ci, (t0, cnt) in enumerate(chunks):
        q, k, v = st.tokens(t0, cnt)
        out = lt.ltri_prefill_chunk(SEQ, 0, L, q, k, v)
        for l in LAYERS:
            K[l].append(k[l].cpu())
            V[l].append(v[l].cpu())
            if ci >= probe_call:
                Q[l][ci] = q[l].cpu()
        if ci in sampled:
            torch.cuda.synchronize()
            assert lt.ltri_sync_status() == 0
            for l in LAYERS:
                Kall, Vall = torch.cat(K[l]), torch.cat(V[l])
                rows = ROWS if ci == last else [0, n - 1]
                snap[l], *state[l] = check_call(lt, cfg, l, SEQ, t0, Kall, Vall, q[l].cpu(), out, rep, rows,
                                               f"layer {l} call {ci} of {len(chunks)}")
    torch.cuda.synchronize()
    assert lt.ltri_sync_status() == 0
    for l in LAYERS:
        Kall, Vall = torch.cat(K[l]), torch.cat(V[l])
        spans_g, idx_g, pend_g = state[l]
        # ---- index vectors of one region: its votes over the nine calls it spends in the window ------------
        c0 = probe_call
        t0c = chunks[c0][0]
        Ec = t0c - W
        o2 = ph.oracle_of(cfg)
        o2.append_only(Kall[:t0c], Vall[:t0c])
        keep = spans_g[:, 0] + spans_g[:, 1] <= Ec
        o2.load_state(Ec, spans_g[keep], idx_g[keep])
        for (rs2, re2, sp2) in regions_from_table(np.concatenate([spans_g, pend_g]), Ec, t0c, n):
            o2.add_pending(rs2, re2, sp2)
        for ci in range(c0, c0 + W // n + 2):
            tt = chunks[ci][0]
            o2.prefill_local(Q[l][ci], Kall[tt:tt + n], Vall[tt:tt + n])
            if ci == c0:
                reg_g = spans_g[(spans_g[:, 0] >= t0c) & (spans_g[:, 0] < t0c + n)]
                if o2.pending()[-1][2].tolist() != reg_g.tolist():
                    assert o2.seg_gap() < ph.NEAR_TIE, f"layer {l}: probe region spans differ without a near tie"
                    o2.set_newest_spans(reg_g)
            if o2.evicted_end >= t0c + n:
                break
        assert o2.evicted_end >= t0c + n, "probe region was not evicted"
        sp2, idx2 = o2.spans(), o2.index()
        sel_rows = np.where((sp2[:, 0] >= t0c) & (sp2[:, 0] < t0c + n))[0]
        assert len(sel_rows) > 0
        for s in sel_rows:
            gs = np.where(spans_g[:, 0] == sp2[s, 0])[0][0]
            assert spans_g[gs, 1] == sp2[s, 1]
            rep.index_rows += 1
            if not np.array_equal(idx_g[gs], idx2[s]):
                vo = np.sort(o2.votes(int(sp2[s, 0]), int(sp2[s, 0] + sp2[s, 1])).astype(np.float64))[::-1]
                assert len(vo) > 1 and (vo[0] - vo[1]) <= ph.NEAR_TIE * max(vo[0], 1.0), \
                    f"layer {l}: index vector of span {gs} differs"
                rep.index_flips += 1
    # ---- decode continues from the same state (all sequences of the config in one batch) --------------------
    if cfg.decode_steps < 3:
        lt.close()
        return
    streams = {s: inputs.SyntheticStream(cfg, seq=s, device=dev) for s in others}
    streams[SEQ] = st
    ids = list(range(cfg.n_seqs))
    pos = ids.index(SEQ)
    # the headline config decodes all its steps and also checks the last one; the others their first three
    n_steps = cfg.decode_steps if cfg_idx == 2 else 3
    checked = {0, 1, 2, n_steps - 1}
    for s in range(n_steps):
        parts = [streams[i].tokens(cfg.context + s, 1, kind=1) for i in ids]
        qd, kd, vd = (torch.cat([pp[j].permute(1, 0, 2, 3) for pp in parts]).contiguous() for j in range(3))
        out = lt.ltri_decode_step(ids, 0, L, qd, kd, vd)
        torch.cuda.synchronize()
        for l in LAYERS:
            o = snap[l]
            o.decode_retrieve(qd[pos, l].cpu(), kd[pos, l].cpu(), vd[pos, l].cpu())   # (appends the step's token)
            if s in checked:
                ph.check_selection(lt.ltri_get_selected(SEQ, l), o, rep, f"layer {l} decode {s}")
                ph.check_output(out[pos, l], o.decode_attend(), rep, f"layer {l} decode {s}")
    assert lt.ltri_sync_status() == 0
    assert rep.span_flips <= 2 and rep.sel_flips <= 6 and rep.index_flips <= 2
    print(rep)
    lt.close()

"""GPU-vs-oracle parity harness used by the ``-m gpu`` tests and the smoke check.

Drives the CUDA library (through the C ABI binding) and one CPU oracle per checked layer over
the same seeded inputs, comparing after every call:

* the Q20 region map and theta (floating point decides an integer: a few units of tolerance);
* the segmenter, bit-exact, on the GPU's own map (oracle segmenter fed the GPU's integers);
* the region's spans against the oracle's own run (bit-exact unless the oracle reports a
  decisive relative gap below 1e-4, in which case the oracle adopts the GPU's pick);
* votes, the span table and the index vectors; scores and the selected span sets (a pick may
  differ only among candidates within 1e-4 relative of the cut; the oracle then adopts it);
* attention outputs: max-abs <= 2e-2 and relative Frobenius error <= 1e-2.
"""
from __future__ import annotations

import dataclasses

import numpy as np
import torch

from oracle import ltri_oracle as orc
from paper_2412_04757_b200 import binding, inputs

MAX_ABS = 2e-2
REL_FRO = 1e-2
NEAR_TIE = 1e-4


@dataclasses.dataclass
class Report:
    calls: int = 0
    regions: int = 0
    span_flips: int = 0
    sel_checks: int = 0
    sel_flips: int = 0
    index_rows: int = 0
    index_flips: int = 0
    max_abs: float = 0.0
    max_rel_fro: float = 0.0
    max_map_diff: int = 0
    max_theta_diff: int = 0
    max_score_rel: float = 0.0
    rep_counts: int = 0
    rep_count_flips: int = 0
    vote_changes: int = 0   # selections that the ballots of other layers changed (collaborative voting)
    cache_hits: int = 0     # host-memory pager: units found in / fetched into the unit caches (last checked layer)
    cache_misses: int = 0


def params_of(cfg: inputs.StreamConfig, max_seqs=None) -> binding.LtriParams:
    return binding.make_params(cfg.n_layers, cfg.n_q_heads, cfg.n_kv_heads, cfg.max_tokens, cfg.chunk, cfg.window,
                               cfg.n_sink, cfg.top_k, head_dim=cfg.head_dim, max_seqs=max_seqs or cfg.n_seqs,
                               reps_per_span=cfg.reps_per_span, max_spans_per_region=cfg.max_spans_per_region,
                               theta_mode=cfg.theta_mode, theta=cfg.theta, rep_mode=cfg.rep_mode,
                               ratio_kind=cfg.ratio_kind, min_reps=cfg.min_reps, max_reps=cfg.max_reps,
                               rep_lambda=cfg.rep_lambda,
                               flags=(binding.FLAG_PERSIST_DECODE if cfg.persist_decode else 0) |
                                     (binding.FLAG_COLLAB_VOTE if cfg.collab_vote else 0) |
                                     (binding.FLAG_SEGMENT_PER_UNIT if cfg.segment_per_unit else 0) |
                                     (binding.FLAG_HOST_KV if cfg.host_kv else 0),
                               cache_units=cfg.cache_units, score_decay=cfg.score_decay,
                               unit_tokens=cfg.unit_tokens, nms_iou_milli=cfg.nms_iou_milli,
                               retrieval_head=cfg.retrieval_head, retrieval_head_score=cfg.retrieval_head_score,
                               layer_theta=cfg.layer_theta, layer_nms_iou_milli=cfg.layer_nms_iou_milli,
                               layer_rep_lambda=cfg.layer_rep_lambda)


def ret_head_of(cfg: inputs.StreamConfig, layer: int):
    """(retrieval head or -1, its weight) of a layer."""
    if cfg.retrieval_head is None:
        return -1, 0.0
    w = 1.0 if cfg.retrieval_head_score is None else float(cfg.retrieval_head_score[layer])
    return int(cfg.retrieval_head[layer]), w


def layer_values(cfg: inputs.StreamConfig, layer: int):
    """(theta, nms_iou_milli, rep_lambda) of a layer: its table entry, else the scalar."""
    return (float(np.float32(cfg.layer_theta[layer])) if cfg.layer_theta else cfg.theta,
            int(cfg.layer_nms_iou_milli[layer]) if cfg.layer_nms_iou_milli else cfg.nms_iou_milli,
            float(np.float32(cfg.layer_rep_lambda[layer])) if cfg.layer_rep_lambda else cfg.rep_lambda)


def oracle_of(cfg: inputs.StreamConfig, layer: int = 0) -> orc.OracleStream:
    rh, w = ret_head_of(cfg, layer)
    theta, phi, lam = layer_values(cfg, layer)
    return orc.OracleStream(cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim, cfg.chunk, cfg.window, cfg.n_sink, cfg.top_k,
                            cfg.max_tokens, reps_per_span=cfg.reps_per_span,
                            max_spans_per_region=cfg.max_spans_per_region, theta_mode=cfg.theta_mode, theta=theta,
                            rep_mode=cfg.rep_mode, ratio_kind=cfg.ratio_kind, min_reps=cfg.min_reps,
                            max_reps=cfg.max_reps, rep_lambda=lam, persist_decode=int(cfg.persist_decode),
                            unit_tokens=cfg.unit_tokens, nms_iou_milli=phi, ret_head=rh, head_weight=w,
                            collab_vote=int(cfg.collab_vote), segment_per_unit=int(cfg.segment_per_unit))


def check_output(got_bf16: torch.Tensor, ref: np.ndarray, rep: Report, what: str):
    got = got_bf16.to(torch.float32).cpu().numpy().astype(np.float64)
    ref = ref.astype(np.float64)
    assert np.isfinite(got).all(), f"{what}: non-finite output"
    ma = float(np.abs(got - ref).max())
    rf = float(np.linalg.norm(got - ref) / max(np.linalg.norm(ref), 1e-30))
    rep.max_abs = max(rep.max_abs, ma)
    rep.max_rel_fro = max(rep.max_rel_fro, rf)
    assert ma <= MAX_ABS, f"{what}: max-abs {ma:.4g} > {MAX_ABS}"
    assert rf <= REL_FRO, f"{what}: relative Frobenius {rf:.4g} > {REL_FRO}"


def check_selection(sel_gpu: np.ndarray, o: orc.OracleStream, rep: Report, what: str, voted=False):
    """sel_gpu [Hkv][k] ascending ids (-1 padded) against the oracle's scores; adopts tolerated picks.

    voted: the units were ranked by the tally of the layers' ballots first (Sec. 3.5, collaborative voting); a pick
    may then differ only among units with the tally of the last unit the oracle took.
    """
    sel_o, _ = o.selected()
    tally = o.tally() if voted else None
    if o.unit_tokens > 0:
        # unit mode: the ids are absolute unit numbers, the scores those of the units that meet the indexed range
        us = o.unit_scores()
        u0 = o.n_sink // o.unit_tokens
        sc = [{u0 + i: us[g][i] for i in range(us.shape[1])} for g in range(us.shape[0])]
    else:
        sc = o.scores()
    adopt = False
    for g in range(sel_gpu.shape[0]):
        a = set(int(x) for x in sel_gpu[g] if x >= 0)
        b = set(int(x) for x in sel_o[g] if x >= 0)
        rep.sel_checks += 1
        assert len(a) == len(b), f"{what}: KV head {g} selected {len(a)} spans, oracle {len(b)}"
        if a == b:
            continue
        # the sets may differ only among spans whose oracle scores are within the near-tie band of the cut
        if voted:
            u0 = o.n_sink // o.unit_tokens
            last = [int(x) for x in sel_o[g] if x >= 0][-1]        # the oracle lists its picks in rank order
            cut = sc[g][last]
            for i in a ^ b:
                assert tally[i - u0] == tally[last - u0], f"{what}: KV head {g} unit {i}: tally differs from the cut's"
        else:
            cut = min(sc[g][i] for i in b)
        band = NEAR_TIE * max(abs(cut), 1e-30)
        for i in a ^ b:
            assert abs(sc[g][i] - cut) <= band, (
                f"{what}: KV head {g} span {i} score {sc[g][i]} vs cut {cut}: not a near tie")
        rep.sel_flips += 1
        adopt = True
    if adopt:
        ids = np.full_like(sel_o, -1)
        for g in range(sel_gpu.shape[0]):
            row = [int(x) for x in sel_gpu[g] if x >= 0]
            ids[g, :len(row)] = row
        o.set_selected(ids)


class StreamPair:
    """The library context plus oracles for the checked (seq, layer) pairs of one workload."""

    def __init__(self, cfg: inputs.StreamConfig, layers, seqs=(0,), device="cuda:0", deep=True):
        self.cfg, self.layers, self.seqs, self.deep = cfg, list(layers), list(seqs), deep
        self.dev = torch.device(device)
        self.lt = binding.Ltri(params_of(cfg), device=device)
        self.orc = {(s, l): oracle_of(cfg, l) for s in self.seqs for l in self.layers}
        if cfg.collab_vote:   # a layer needs the ballots of every layer before it
            assert self.layers == list(range(cfg.n_layers)), "collaborative voting: check every layer"
        self.rep = Report()
        self.n_indexed = {(s, l): 0 for s in self.seqs for l in self.layers}
        self.count_of = {}   # (seq, layer, span start) -> representative count decided when its region was current
        # host-memory pager: the oracle's model of every (seq, layer, KV head) unit cache
        self.cache = {(s, l, g): orc.UnitCachePolicy(cfg.cache_units, cfg.score_decay)
                      for s in self.seqs for l in self.layers for g in range(cfg.n_kv_heads)} if cfg.host_kv else {}

    # ---- one prefill call -------------------------------------------------------------------
    def prefill(self, seq, q, k, v, check_out=True):
        """q [L][n][Hq][d], k, v [L][n][Hkv][d] bf16 on the CPU."""
        cfg, lt, rep = self.cfg, self.lt, self.rep
        L = cfg.n_layers
        out = lt.ltri_prefill_chunk(seq, 0, L, q.to(self.dev), k.to(self.dev), v.to(self.dev))
        torch.cuda.synchronize(self.dev)
        assert lt.ltri_sync_status() == 0
        rep.calls += 1
        ballots = []   # collaborative voting: (weight, units) of the layers handled so far
        for layer in self.layers:
            if (seq, layer) not in self.orc:
                continue
            o = self.orc[(seq, layer)]
            what = f"seq {seq} layer {layer} call@{o.tokens}"
            rh, _ = ret_head_of(cfg, layer)
            gk = slice(None) if rh < 0 else slice(rh // (cfg.n_q_heads // cfg.n_kv_heads),
                                                  rh // (cfg.n_q_heads // cfg.n_kv_heads) + 1)
            nh = cfg.n_q_heads if rh < 0 else 1    # heads summed into the layer's map
            theta_l, phi_l, lambda_l = layer_values(cfg, layer)
            o.prefill_local(q[layer], k[layer], v[layer])
            rs, m = o.region()
            t1 = o.tokens
            if m > 0:
                rep.regions += 1
                pend_g = lt.ltri_get_pending_spans(seq, layer)
                newest_g = pend_g[pend_g[:, 0] >= rs]
                spans_o = o.pending()[-1][2]
                if self.deep:
                    Mg = np.tril(lt.ltri_debug_read(binding.BUF_MAP, seq, layer)[:m, :m])
                    Mo = o.map()
                    md = int(np.abs(Mg.astype(np.int64) - Mo).max())
                    rep.max_map_diff = max(rep.max_map_diff, md)
                    assert md <= 4 + nh, f"{what}: region map differs by {md} Q20 units"
                    thg = int(lt.ltri_debug_read(binding.BUF_THETA, seq, layer)[0])
                    rep.max_theta_diff = max(rep.max_theta_diff, abs(thg - o.theta_q()))
                    assert abs(thg - o.theta_q()) <= 4 + nh, f"{what}: theta {thg} vs {o.theta_q()}"
                    if cfg.theta_mode == 1:
                        assert thg == orc.theta_q(Mg, 1, theta_l, cfg.n_q_heads), f"{what}: theta rank select"
                    # integer pipeline: bit-exact on identical integer input
                    ref_spans, _ = orc.segment_map(Mg, thg, cfg.max_spans_per_region, phi_l,
                                                   unit=cfg.unit_tokens if cfg.segment_per_unit else 0, origin=rs)
                    ref_spans[:, 0] += rs
                    assert newest_g.tolist() == ref_spans.tolist(), f"{what}: segmenter differs on its own map"
                if newest_g.tolist() != spans_o.tolist():
                    assert o.seg_gap() < NEAR_TIE, (
                        f"{what}: spans differ and the oracle's smallest decisive gap is {o.seg_gap():.3g}")
                    rep.span_flips += 1
                    o.set_newest_spans(newest_g)
                # representative counts of the region's spans (Sec. 3.3.2 when rep_mode = 1)
                J = len(newest_g)
                ng = lt.ltri_debug_read(binding.BUF_NREPS, seq, layer)[:J]
                no = o.newest_rep_counts()
                rep.rep_counts += J
                if cfg.rep_mode == 1 and self.deep:
                    # integer sums, one division, one exponential, one rounding: the same on the GPU's own map
                    ref = [orc.dynamic_rep_count(Mg, int(st - rs), int(st - rs + ln - 1), cfg.ratio_kind, lambda_l,
                                                 cfg.min_reps, cfg.max_reps) for st, ln in newest_g]
                    assert ng.tolist() == ref, f"{what}: representative counts differ on the GPU's own map"
                if ng.tolist() != no.tolist():
                    # the two maps differ by a few Q20 units: a count may flip by one where len * r_v is near .5
                    assert cfg.rep_mode == 1 and int(np.abs(ng - no).max()) <= 1, (
                        f"{what}: representative counts {ng.tolist()} vs {no.tolist()}")
                    rep.rep_count_flips += int((ng != no).sum())
                    o.set_newest_rep_counts(ng)
                for (st, ln), c in zip(newest_g, ng):
                    self.count_of[(seq, layer, int(st))] = int(c)
            if self.deep:
                vg = lt.ltri_debug_read(binding.BUF_VOTES, seq, layer)[:t1].astype(np.float64)
                vo = o.votes(0, t1).astype(np.float64)
                lo = cfg.n_sink
                dv = np.abs(vg[lo:] - vo[lo:])
                assert np.all(dv <= 64 + 2e-5 * np.abs(vo[lo:])), f"{what}: votes differ by up to {dv.max()}"
            self._check_index(seq, layer, o, k, what)
            if cfg.collab_vote:
                o.set_ballots(ballots)
            o.prefill_retrieve()
            if len(o.spans()):
                if self.deep and m > 0:
                    # (under a retrieval head only the rows of its KV head mean anything on the GPU side)
                    J = len(o.pending()[-1][2])
                    ug = lt.ltri_debug_read(binding.BUF_QREPS, seq, layer)[:, :J]
                    assert np.allclose(ug[gk], o.query_reps()[gk], rtol=0, atol=1e-4), f"{what}: query representatives"
                    ns = len(o.spans())
                    sg = lt.ltri_debug_read(binding.BUF_SCORES, seq, layer)[:, :ns]
                    so = o.scores()
                    rel = float(np.abs(sg[gk] - so[gk]).max() / max(np.abs(so[gk]).max(), 1e-30))
                    rep.max_score_rel = max(rep.max_score_rel, rel)
                    assert rel <= 2e-5, f"{what}: scores differ by {rel:.3g} relative"
                if cfg.collab_vote:
                    self._vote(seq, layer, o, ballots, what)
                    self._count_vote_changes(o)
                check_selection(lt.ltri_get_selected(seq, layer), o, rep, what, voted=cfg.collab_vote)
                if cfg.host_kv:
                    self._check_cache(seq, layer, o, what)
            if check_out:
                check_output(out[layer], o.prefill_attend(), rep, what)
        return out

    def _check_cache(self, seq, layer, o, what, decode=False):
        """Host-memory pager: the unit cache of every KV head holds what the policy model says after this retrieval,
        fed with the units the call attends over.  Prefill: the unit the indexed range ends in is cached only once it
        is whole.  Decode: the range no longer grows, every named unit is cached, the persistent ones included."""
        cfg, lt = self.cfg, self.lt
        U, E = cfg.unit_tokens, o.evicted_end
        sel = o.selected()[0]          # equal to the GPU's as a set (adopted where a near tie flipped a pick)
        pers = o.persistent() if decode and cfg.persist_decode else np.full_like(sel, -1)
        tags = lt.ltri_debug_read(binding.BUF_CACHE_TAGS, seq, layer)
        scores = lt.ltri_debug_read(binding.BUF_CACHE_SCORES, seq, layer)
        hits = misses = 0
        for g in range(cfg.n_kv_heads):
            pol = self.cache[(seq, layer, g)]
            named = set(int(u) for u in sel[g] if u >= 0) | set(int(u) for u in pers[g] if u >= 0)
            pol.access(sorted(u for u in named if decode or (u + 1) * U <= E))
            assert tags[g].tolist() == pol.tags.tolist(), f"{what}: unit cache of KV head {g} holds other units"
            assert np.array_equal(scores[g], pol.scores), f"{what}: usage scores of KV head {g}"
            hits += pol.hits
            misses += pol.misses
        st = lt.ltri_debug_read(binding.BUF_CACHE_STATS, seq, layer)
        assert (int(st[0]), int(st[1])) == (hits, misses), f"{what}: cache hits/misses {st.tolist()} vs {(hits, misses)}"
        self.rep.cache_hits, self.rep.cache_misses = hits, misses

    def _vote(self, seq, layer, o, ballots, what):
        """Collaborative voting (Sec. 3.5): compare the layer's own ballot, let the oracle adopt a tolerated pick and
        count again, and add the ballot to those the later layers read."""
        cfg, rep = self.cfg, self.rep
        rh, w = ret_head_of(cfg, layer)
        bg = self.lt.ltri_debug_read(binding.BUF_BALLOT, seq, layer)
        bo = o.ballot()
        if rh < 0:
            assert (bg < 0).all() and (bo < 0).all(), f"{what}: a layer without a retrieval head cast a ballot"
            return
        a, b = set(int(x) for x in bg if x >= 0), set(int(x) for x in bo if x >= 0)
        assert len(a) == len(b), f"{what}: ballot of {len(a)} units, oracle {len(b)}"
        if a != b:
            us = o.unit_scores()[0]
            u0 = cfg.n_sink // cfg.unit_tokens
            cut = min(us[i - u0] for i in b)
            for i in a ^ b:
                assert abs(us[i - u0] - cut) <= NEAR_TIE * max(abs(cut), 1e-30), f"{what}: ballot unit {i}: no near tie"
            rep.sel_flips += 1
            o.set_ballot(bg)
        ballots.append((w, o.ballot()))

    def _count_vote_changes(self, o):
        us, sel = o.unit_scores(), o.selected()[0]
        u0 = self.cfg.n_sink // self.cfg.unit_tokens
        for g in range(us.shape[0]):
            own = set((np.argsort(-us[g], kind="stable")[:self.cfg.top_k] + u0).tolist())
            self.rep.vote_changes += own != set(int(x) for x in sel[g] if x >= 0)

    def _check_index(self, seq, layer, o, k, what):
        spans_o = o.spans()
        done = self.n_indexed[(seq, layer)]
        if len(spans_o) == done:
            return
        spans_g = self.lt.ltri_get_spans(seq, layer)
        assert spans_g.tolist() == spans_o.tolist(), f"{what}: span tables differ"
        stats = self.lt.ltri_get_stats(seq, layer)
        assert stats.n_spans == len(spans_o) and stats.evicted_end == o.evicted_end
        assert stats.index_bytes == len(spans_o) * self.cfg.n_kv_heads * self.cfg.head_dim * 2, f"{what}: index size"
        idx_g = self.lt.ltri_debug_read(binding.BUF_INDEX, seq, layer)
        idx_o = o.index()
        for s in range(done, len(spans_o)):
            self.rep.index_rows += 1
            if np.array_equal(idx_g[:, s, :], idx_o[s]):
                continue
            # a different representative token is tolerated only as a near tie in the oracle's votes
            st, ln = spans_o[s]
            vo = o.votes(int(st), int(st + ln)).astype(np.float64)
            top = np.sort(vo)[::-1]
            cnt = self.count_of.get((seq, layer, int(st)), self.cfg.reps_per_span)
            assert cnt < ln and (top[cnt - 1] - top[cnt]) <= \
                NEAR_TIE * max(top[0], 1.0), f"{what}: index vector of span {s} differs"
            self.rep.index_flips += 1
        self.n_indexed[(seq, layer)] = len(spans_o)

    # ---- one decode step ---------------------------------------------------------------------
    def decode(self, seq_ids, q, k, v):
        """q [n_seqs][L][Hq][d], k, v [n_seqs][L][Hkv][d] bf16 on the CPU."""
        cfg, lt, rep = self.cfg, self.lt, self.rep
        L = cfg.n_layers
        out = lt.ltri_decode_step(seq_ids, 0, L, q.to(self.dev), k.to(self.dev), v.to(self.dev))
        torch.cuda.synchronize(self.dev)
        assert lt.ltri_sync_status() == 0
        rep.calls += 1
        for i, seq in enumerate(seq_ids):
            ballots = []
            for layer in self.layers:
                if (seq, layer) not in self.orc:
                    continue
                o = self.orc[(seq, layer)]
                what = f"seq {seq} layer {layer} decode@{o.tokens}"
                if cfg.collab_vote:
                    o.set_ballots(ballots)
                o.decode_retrieve(q[i, layer], k[i, layer], v[i, layer])
                if len(o.spans()):
                    if cfg.collab_vote:
                        self._vote(seq, layer, o, ballots, what)
                        self._count_vote_changes(o)
                    check_selection(lt.ltri_get_selected(seq, layer), o, rep, what, voted=cfg.collab_vote)
                    if cfg.host_kv:
                        self._check_cache(seq, layer, o, what, decode=True)
                    # tokens the step attends over besides sink and local: this step's spans united, under the
                    # persistent mechanism, with those of the last prefill call (every span once)
                    sel_o, _ = o.selected()
                    pers = o.persistent() if cfg.persist_decode else np.full_like(sel_o, -1)
                    sp = o.spans()
                    U, E = cfg.unit_tokens, o.evicted_end
                    want = 0
                    for g in range(sel_o.shape[0]):
                        ids = set(int(x) for x in sel_o[g] if x >= 0) | set(int(x) for x in pers[g] if x >= 0)
                        if U > 0:
                            want += sum(min((j + 1) * U, E) - max(j * U, cfg.n_sink) for j in ids)
                        else:
                            want += sum(int(sp[j, 1]) for j in ids)
                    got = int(lt.ltri_get_stats(seq, layer).retrieved_tokens)
                    assert got == want, f"{what}: attends over {got} retrieved tokens, oracle {want}"
                check_output(out[i, layer], o.decode_attend(), rep, what)
        return out


def run_stream(cfg: inputs.StreamConfig, layers, max_calls=None, decode_steps=None, deep=True, device="cuda:0"):
    """Stream the workload of `cfg` (sequence 0) through both sides; returns the Report."""
    sp = StreamPair(cfg, layers, device=device, deep=deep)
    st = inputs.SyntheticStream(cfg)
    for ci, (t0, n) in enumerate(st.prefill_chunks()):
        if max_calls is not None and ci >= max_calls:
            break
        q, k, v = st.tokens(t0, n)
        sp.prefill(0, q, k, v)
    steps = cfg.decode_steps if decode_steps is None else decode_steps
    if max_calls is None:
        for s in range(steps):
            q, k, v = st.tokens(cfg.context + s, 1, kind=1)
            sp.decode([0], q.permute(1, 0, 2, 3).contiguous(), k.permute(1, 0, 2, 3).contiguous(),
                      v.permute(1, 0, 2, 3).contiguous())
    sp.lt.close()
    return sp.rep

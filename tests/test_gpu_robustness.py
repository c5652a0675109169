"""GPU paths that ordinary streams never reach: keys of very large norm (the attention kernel's second pass),
an expiring device-side wait, a span index loaded from outside, and host-side limits that must leave the context
unchanged.  Everything here is finite input and bounded waiting: nothing is expected to fault, trap or hang."""
import dataclasses

import numpy as np
import pytest
import torch

from paper_2412_04757_b200 import binding, inputs
from tests import parity_harness as ph
from tests.test_gpu_parity import small_cfg

pytestmark = pytest.mark.gpu


def _decode_inputs(st, pos):
    q, k, v = st.tokens(pos, 1, kind=1)
    return (q.permute(1, 0, 2, 3).contiguous(), k.permute(1, 0, 2, 3).contiguous(), v.permute(1, 0, 2, 3).contiguous())


@pytest.mark.parametrize("gain,max_ctas", [(30.0, None), (12.0, "3"), (1.4, None)])
def test_keys_of_very_large_norm_give_the_exact_softmax(gain, max_ctas, monkeypatch):
    # Sec. 3.4 step 3: exact softmax over sink | retrieved | local | current for ANY finite input.  Two keys of
    # KV head 0 are scaled up so that the logits of the queries that point at their segment exceed every earlier
    # tile's maximum by hundreds of log2 units (gain 30 and 12: the kernel's first pass, whose softmax reference
    # moves one tile late, notices and a second pass with the true maximum on every tile redoes the CTA's items) or
    # by an amount the late reference still absorbs (gain 1.4).  The keys sit in a later tile of the local window
    # while they are local and in the packed slab of the retrieved spans afterwards (their own votes make them their
    # spans' representatives, so the spans are retrieved).  KV head 1 keeps ordinary keys, so one launch has CTAs
    # that take the second pass and CTAs that do not; with three CTAs every CTA walks many items in both passes.
    # The map comparison is left to the ordinary tests: with logits of this size the fp32 rounding of a logit (on
    # both sides) is worth dozens of Q20 units at a probability near one, beyond the tolerance that is meant for
    # bf16-sized inputs; spans (with the oracle's tie rule), index, selections and outputs are compared as always.
    if max_ctas:
        monkeypatch.setenv("LTRI_TC_MAX_CTAS", max_ctas)
    cfg = small_cfg(n_layers=2, context=1536, top_k=12, decode_steps=3)
    big = {300, 700}
    retrieved = {(layer, tok): 0 for layer in (0, 1) for tok in big}
    sp = ph.StreamPair(cfg, [0, 1], deep=False)
    st = inputs.SyntheticStream(cfg)
    for t0, n in st.prefill_chunks():
        q, k, v = st.tokens(t0, n)
        for tok in big:
            if t0 <= tok < t0 + n:
                k[:, tok - t0, 0, :] = (k[:, tok - t0, 0, :].float() * gain).to(torch.bfloat16)
        sp.prefill(0, q, k, v)
        for layer in (0, 1):     # prefill calls whose retrieved spans (KV head 0) hold a scaled key
            spans = sp.lt.ltri_get_spans(0, layer)
            sel = sp.lt.ltri_get_selected(0, layer)[0]
            for tok in big:
                retrieved[(layer, tok)] += any(spans[i, 0] <= tok < spans[i, 0] + spans[i, 1] for i in sel[sel >= 0])
    for s in range(cfg.decode_steps):
        sp.decode([0], *_decode_inputs(st, cfg.context + s))
    if gain >= 12.0:   # the continuation over the retrieved spans met the scaled keys too, not only the local part
        assert all(cnt > 0 for cnt in retrieved.values()), retrieved
    assert sp.lt.ltri_sync_status() == 0
    sp.lt.close()
    print(sp.rep)


def test_a_device_side_wait_that_expires_reports_a_timeout_and_the_context_stays_usable():
    # failure detection: every device-side wait is bounded.  The test kernel waits 10^5 cycles on a barrier that
    # nothing completes; the wait expires, the CTA's abort flag releases the second waiter at once (not after its
    # own limit of about a second), the status word reports LTRI_ETIMEOUT once, and the stream that continues on the
    # same context stays bit-identical to one on a context that never saw the time-out.
    cfg = small_cfg(n_layers=2, context=1024, decode_steps=2)
    st = inputs.SyntheticStream(cfg)
    a, b = binding.Ltri(ph.params_of(cfg)), binding.Ltri(ph.params_of(cfg))
    chunks = list(st.prefill_chunks())
    for ci, (t0, n) in enumerate(chunks):
        q, k, v = (x.cuda() for x in st.tokens(t0, n))
        if ci == 4:
            waited = a.ltri_debug_wait_timeout(100_000)
            assert 100_000 <= waited[0] < 5_000_000, waited       # gave up at its limit
            assert 0 <= waited[1] < 50_000_000, waited            # released by the abort flag, long before 2e9
            assert a.ltri_sync_status() == binding.LTRI_ETIMEOUT
            assert a.ltri_sync_status() == 0                      # reported once, then cleared
        assert torch.equal(a.ltri_prefill_chunk(0, 0, 2, q, k, v), b.ltri_prefill_chunk(0, 0, 2, q, k, v))
    for s in range(cfg.decode_steps):
        q, k, v = (x.cuda() for x in _decode_inputs(st, cfg.context + s))
        assert torch.equal(a.ltri_decode_step([0], 0, 2, q, k, v), b.ltri_decode_step([0], 0, 2, q, k, v))
    for layer in range(2):
        assert a.ltri_get_spans(0, layer).tolist() == b.ltri_get_spans(0, layer).tolist()
    assert a.ltri_sync_status() == 0 and b.ltri_sync_status() == 0
    with pytest.raises(binding.LtriError):
        a.ltri_debug_wait_timeout(0)
    a.close()
    b.close()


@pytest.mark.parametrize("unit_tokens", [0, 64])
def test_retrieval_and_attention_from_a_loaded_span_index(unit_tokens):
    # Sec. 3.4 steps 2-3 (Eq. 7-8) driven from a state the GPU did not produce: after a few calls in lockstep the
    # span table is coarsened (neighbouring spans merged in pairs) and every index vector is replaced -- most by
    # random vectors, some by keys of the stream so that the ranking is not arbitrary -- on both sides; scores,
    # selections and outputs of the following calls and decode steps must then match the oracle as usual.
    cfg = small_cfg(n_layers=2, context=1536, decode_steps=3, top_k=5, unit_tokens=unit_tokens)
    sp = ph.StreamPair(cfg, [0, 1])
    st = inputs.SyntheticStream(cfg)
    sizes = [128] * 8 + [16, 112] + [128] * 3          # the call after the 16-token one evicts nothing
    assert sum(sizes) == cfg.context
    rng = np.random.default_rng(5)
    t0, keys = 0, []
    for ci, n in enumerate(sizes):
        q, k, v = st.tokens(t0, n)
        keys.append(k)
        sp.prefill(0, q, k, v)
        t0 += n
        if ci == 8:
            kall = torch.cat(keys, dim=1)                # [L][tokens][Hkv][d]
            for layer in (0, 1):
                o = sp.orc[(0, layer)]
                old = o.spans()
                assert len(old) >= 8
                new = [[int(old[i, 0]), int(old[i, 1] + (old[i + 1, 1] if i + 1 < len(old) else 0))]
                       for i in range(0, len(old), 2)]
                new = np.asarray(new, dtype=np.int32)
                idx = inputs.bf16_bits(torch.from_numpy(rng.standard_normal((len(new), cfg.n_kv_heads, 128)))
                                       .to(torch.bfloat16))
                for s in range(0, len(new), 3):          # every third span: the key of its last token
                    tok = int(new[s, 0] + new[s, 1] - 1)
                    idx[s] = inputs.bf16_bits(kall[layer, tok])
                o.replace_index(new, idx)
                E = sp.lt.ltri_get_stats(0, layer).evicted_end
                assert E == o.evicted_end
                sp.lt.ltri_debug_load_index(0, layer, E, new, idx.transpose(1, 0, 2))
                sp.n_indexed[(0, layer)] = len(new)
                assert sp.lt.ltri_get_spans(0, layer).tolist() == new.tolist()
                got = sp.lt.ltri_debug_read(binding.BUF_INDEX, 0, layer)[:, :len(new)]
                assert np.array_equal(got, idx.transpose(1, 0, 2))
    for s in range(cfg.decode_steps):
        sp.decode([0], *_decode_inputs(st, cfg.context + s))
    assert sp.rep.sel_checks > 10
    # what the loader refuses, on the host, leaving the state alone
    lt = sp.lt
    spans = lt.ltri_get_spans(0, 0)
    idx = lt.ltri_debug_read(binding.BUF_INDEX, 0, 0)[:, :len(spans)].copy()
    E = lt.ltri_get_stats(0, 0).evicted_end
    for bad_E, bad_spans in [(E - 1, spans), (E, spans[:-1]), (E, spans[1:]),
                             (E, np.concatenate([spans[:1], spans[:1], spans[1:]]))]:
        with pytest.raises((binding.LtriError, ValueError)):
            lt.ltri_debug_load_index(0, 0, bad_E, bad_spans, idx[:, :len(bad_spans)])
    assert lt.ltri_get_spans(0, 0).tolist() == spans.tolist()
    lt.close()
    print(sp.rep)


@pytest.mark.parametrize("fused", ["0", "1", "2"])
def test_equal_scores_at_the_cut_go_to_the_lower_span(fused, monkeypatch):
    # Eq. 8 with ties: the loaded index holds only three distinct vectors per KV head (span s gets vector s mod 3),
    # so the scores of a call take three values among the loaded spans and the top-k cut falls inside a group of
    # exactly equal scores; the picks among them must be the lowest span ids, in the prefill retriever and in each
    # of the three decode retrieval paths.  The harness tolerates a different pick among near-equal scores and
    # counts it: here the count must stay zero.
    monkeypatch.setenv("LTRI_DEC_FUSED", fused)
    cfg = small_cfg(n_layers=2, context=1536, decode_steps=3, top_k=5)
    sp = ph.StreamPair(cfg, [0, 1])
    st = inputs.SyntheticStream(cfg)
    rng = np.random.default_rng(11)
    t0, ties_at_cut = 0, 0
    for ci, n in enumerate([128] * 12):
        q, k, v = st.tokens(t0, n)
        sp.prefill(0, q, k, v)
        t0 += n
        if ci > 8:    # how often the cut really fell inside a group of equal scores
            for layer in (0, 1):
                o = sp.orc[(0, layer)]
                sel_o, sc = o.selected()[0], o.scores()
                for g in range(cfg.n_kv_heads):
                    picked = [int(x) for x in sel_o[g] if x >= 0]
                    cut = min(sc[g][i] for i in picked)
                    ties_at_cut += sum(1 for i in range(len(sc[g])) if sc[g][i] == cut) > sum(1 for i in picked if sc[g][i] == cut)
        if ci == 8:
            for layer in (0, 1):
                o = sp.orc[(0, layer)]
                spans = np.asarray(o.spans(), dtype=np.int32)
                assert len(spans) >= 8
                pool = inputs.bf16_bits(torch.from_numpy(rng.standard_normal((3, cfg.n_kv_heads, 128))).to(torch.bfloat16))
                idx = np.stack([pool[s % 3] for s in range(len(spans))])
                o.replace_index(spans, idx)
                sp.lt.ltri_debug_load_index(0, layer, o.evicted_end, spans, idx.transpose(1, 0, 2))
    for s in range(cfg.decode_steps):
        sp.decode([0], *_decode_inputs(st, cfg.context + s))
    assert ties_at_cut > 0
    assert sp.rep.sel_checks >= 16 and sp.rep.sel_flips == 0, sp.rep
    sp.lt.close()
    print(sp.rep)


@pytest.mark.parametrize("fused", ["1", "2"])
def test_hundreds_of_equal_scores_fall_back_to_the_radix_passes(fused, monkeypatch):
    # Eq. 8 with a whole index of equal scores: every loaded span gets the same vector, so several hundred scores are
    # exactly equal and the short cut of the select (which ranks at most 256 keys near the maximum against each
    # other) has to hand over to the radix passes and their id-ordered tie pass; picks = the lowest span ids.
    # (both one-launch decode retrievers: one CTA per KV head, and the cluster of eight)
    monkeypatch.setenv("LTRI_DEC_FUSED", fused)
    cfg = small_cfg(n_layers=1, context=12288, decode_steps=2, top_k=6, max_spans_per_region=8, seg_min=8, seg_max=24)
    sp = ph.StreamPair(cfg, [0], deep=False)
    st = inputs.SyntheticStream(cfg)
    rng = np.random.default_rng(3)
    chunks = list(st.prefill_chunks())
    loaded = 0
    for ci, (t0, n) in enumerate(chunks):
        q, k, v = st.tokens(t0, n)
        sp.prefill(0, q, k, v)
        if ci == len(chunks) - 3:
            o = sp.orc[(0, 0)]
            spans = np.asarray(o.spans(), dtype=np.int32)
            loaded = len(spans)
            one = inputs.bf16_bits(torch.from_numpy(rng.standard_normal((1, cfg.n_kv_heads, 128))).to(torch.bfloat16))
            idx = np.repeat(one, loaded, axis=0)
            o.replace_index(spans, idx)
            sp.lt.ltri_debug_load_index(0, 0, o.evicted_end, spans, idx.transpose(1, 0, 2))
    assert loaded > 256 + 16, loaded      # more equal keys than the short cut ranks
    for s in range(cfg.decode_steps):
        sp.decode([0], *_decode_inputs(st, cfg.context + s))
    assert sp.rep.sel_flips == 0, sp.rep
    sel = sp.lt.ltri_get_selected(0, 0)
    assert sel.shape[1] == cfg.top_k
    sp.lt.close()
    print(sp.rep)


def test_host_entry_with_calls_of_different_sizes_and_layer_ranges():
    # the host-buffer entry pipelines layer groups over staging slices that calls reuse: a short call followed by
    # full ones, and calls over part of the layers, must give what the device entry gives, bit for bit
    cfg = small_cfg(n_layers=6, context=1184, decode_steps=0)
    dev = torch.device("cuda:0")
    st = inputs.SyntheticStream(cfg)
    lt_d = binding.Ltri(ph.params_of(cfg), device=dev)
    p = ph.params_of(cfg)
    p.flags |= binding.FLAG_HOST_STAGING
    lt_h = binding.Ltri(p, device=dev)
    sizes = [128, 32, 128, 128, 8, 128, 120, 128, 128, 128, 128]
    assert sum(sizes) == cfg.context
    keep, t0 = [], 0
    for ci, n in enumerate(sizes):
        q, k, v = st.tokens(t0, n)
        ref = lt_d.ltri_prefill_chunk(0, 0, 6, q.to(dev), k.to(dev), v.to(dev))
        ho = torch.empty_like(q).pin_memory()
        parts = [(0, 6)] if ci % 3 else [(0, 2), (2, 3), (5, 1)]     # every third call: three layer ranges
        for lb, lc in parts:
            hq, hk, hv = (x[lb:lb + lc].contiguous().pin_memory() for x in (q, k, v))
            hpart = torch.empty_like(hq).pin_memory()
            lt_h.ltri_prefill_chunk_host(0, lb, lc, hq, hk, hv, hpart)
            keep.append((ref, lb, lc, hpart, (hq, hk, hv)))
        t0 += n
    lt_h.ltri_host_outputs_ready()
    torch.cuda.synchronize(dev)
    for ref, lb, lc, hpart, _ in keep:
        assert torch.equal(ref[lb:lb + lc].cpu(), hpart)
    for layer in range(6):
        assert lt_d.ltri_get_spans(0, layer).tolist() == lt_h.ltri_get_spans(0, layer).tolist()
    # a call that fails its host-side checks changes nothing: the layers are out of step after a partial call
    q, k, v = st.tokens(0, 16)
    hq, hk, hv = (x[:2].contiguous().pin_memory() for x in (q, k, v))
    before = [lt_h.ltri_get_stats(0, l).tokens for l in range(6)]
    with pytest.raises(binding.LtriError) as e:
        lt_h.ltri_prefill_chunk_host(0, 0, 2, hq, hk, hv, torch.empty_like(hq).pin_memory())   # beyond max_tokens
    assert e.value.code == binding.LTRI_ECAPACITY
    assert [lt_h.ltri_get_stats(0, l).tokens for l in range(6)] == before
    assert lt_d.ltri_sync_status() == 0 and lt_h.ltri_sync_status() == 0
    lt_d.close()
    lt_h.close()


def test_many_short_calls_run_out_of_pending_slots_without_changing_the_context():
    # every call is a region of its own until it leaves the window, and a context keeps window/chunk + 8 of them:
    # calls far shorter than the chunk hit that limit as LTRI_ECAPACITY (documented beside ltri_prefill_chunk), the
    # refused call changes nothing, and a reset makes the sequence usable again
    cfg = small_cfg(n_layers=1, context=1024, decode_steps=0)      # window 384, chunk 128: 3 + 8 slots
    lt = binding.Ltri(ph.params_of(cfg))
    st = inputs.SyntheticStream(cfg)
    t0, refused = 0, None
    for ci in range(40):
        q, k, v = (x.cuda() for x in st.tokens(t0, 16))
        try:
            lt.ltri_prefill_chunk(0, 0, 1, q, k, v)
        except binding.LtriError as e:
            assert e.code == binding.LTRI_ECAPACITY
            refused = ci
            break
        t0 += 16
    # the first two calls lie inside the 32-token sink and make no region; the next 11 fill the slots
    assert refused == 13
    s = lt.ltri_get_stats(0, 0)
    assert s.tokens == t0 and s.n_pending_regions == 11
    lt.ltri_reset_sequence(0)
    q, k, v = (x.cuda() for x in st.tokens(0, 128))
    lt.ltri_prefill_chunk(0, 0, 1, q, k, v)
    torch.cuda.synchronize()
    assert lt.ltri_sync_status() == 0
    lt.close()


def test_retrieved_attention_merge_equals_the_continuation(monkeypatch):
    # the retrieved part of a prefill call is accumulated from scratch and merged with the stored local state at the
    # end of every work item; the variant that loads the state first and continues from it must agree to rounding
    # (both are within the oracle's tolerance in the other tests; here they are compared with each other)
    cfg = small_cfg(n_layers=2, context=1280, decode_steps=0, top_k=8)
    st = inputs.SyntheticStream(cfg)
    a = binding.Ltri(ph.params_of(cfg))
    monkeypatch.setenv("LTRI_ATTN_CONT", "1")
    b = binding.Ltri(ph.params_of(cfg))
    worst = 0.0
    for t0, n in st.prefill_chunks():
        q, k, v = (x.cuda() for x in st.tokens(t0, n))
        oa, ob = a.ltri_prefill_chunk(0, 0, 2, q, k, v), b.ltri_prefill_chunk(0, 0, 2, q, k, v)
        worst = max(worst, float((oa.float() - ob.float()).abs().max()))
    assert worst <= 2e-2
    a.close()
    b.close()

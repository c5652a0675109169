"""GPU path (through the C ABI) against the CPU oracle on the same seeded inputs."""
import dataclasses

import numpy as np
import pytest
import torch

from paper_2412_04757_b200 import binding, inputs
from tests import parity_harness as ph

pytestmark = pytest.mark.gpu


def small_cfg(**kw):
    base = dict(name="small", n_layers=2, n_q_heads=8, n_kv_heads=2, head_dim=128, context=1536, chunk=128,
                decode_steps=6, n_sink=32, window=384, top_k=4, max_spans_per_region=4, seg_min=16, seg_max=128,
                seed=777)
    base.update(kw)
    return inputs.StreamConfig(**base)


def test_cfg0_full_stream_and_decode():
    cfg = inputs.config(0)
    rep = ph.run_stream(cfg, layers=[0])
    assert rep.regions == 8 and rep.calls == 8 + 16
    assert rep.span_flips <= 1 and rep.sel_flips <= 2
    print(rep)


def test_two_layers_gqa4_ragged_tail():
    # context not a multiple of the chunk: the last call is short; window not a multiple either
    cfg = small_cfg(context=1500, window=300)
    rep = ph.run_stream(cfg, layers=[0, 1])
    assert rep.regions >= 20
    print(rep)


@pytest.mark.parametrize("Hq,Hkv", [(4, 4), (4, 2), (16, 2)])
def test_group_sizes(Hq, Hkv):
    cfg = small_cfg(n_layers=1, n_q_heads=Hq, n_kv_heads=Hkv, context=1024, decode_steps=3)
    rep = ph.run_stream(cfg, layers=[0])
    print(rep)


def test_three_representatives_per_span_and_absolute_theta():
    cfg = small_cfg(n_layers=1, reps_per_span=3, theta_mode=0, theta=0.02, context=1024, decode_steps=3)
    rep = ph.run_stream(cfg, layers=[0])
    print(rep)


@pytest.mark.parametrize("kind,lam,lo,hi", [(0, 1.0, 1, 4), (1, 2.0, 1, 8), (2, 0.7, 2, 6)])
def test_dynamic_representative_counts(kind, lam, lo, hi):
    # Sec. 3.3.2: the number of index vectors of a span follows its area ratio; checked per region against the oracle
    # (counts, then the query representatives, index vectors, scores, selections and outputs that depend on them)
    cfg = small_cfg(n_layers=2, context=1280, decode_steps=3, rep_mode=1, ratio_kind=kind, rep_lambda=lam,
                    min_reps=lo, max_reps=hi)
    rep = ph.run_stream(cfg, layers=[0, 1])
    assert rep.rep_counts > 50 and rep.rep_count_flips <= 2
    print(rep)


@pytest.mark.parametrize("fused", ["0", "1", "2"])
def test_persistent_mechanism_in_decode(fused, monkeypatch):
    # Sec. 3.5: the spans the last prefill call retrieved stay in the attention of every decode step (both
    # decode retrieval paths); the harness checks the united token count exactly and the outputs
    monkeypatch.setenv("LTRI_DEC_FUSED", fused)
    cfg = small_cfg(n_layers=2, context=1280, decode_steps=8, persist_decode=True)
    rep = ph.run_stream(cfg, layers=[0, 1])
    print(rep)


def test_maximum_sizes():
    # the largest chunk (1024), top-k (64), spans per region (64 -> room for 129 query spans, more than the tcgen05
    # score kernel takes, so the scores run on the warp-MMA kernel), representatives per span (8) and group size
    # (8 query heads on one KV head) the library accepts; an absolute threshold keeps the planted segments apart
    cfg = small_cfg(n_layers=1, n_q_heads=8, n_kv_heads=1, context=5 * 1024 + 200, chunk=1024, window=1024, n_sink=1024,
                    top_k=64, max_spans_per_region=64, reps_per_span=8, decode_steps=2, seg_min=4, seg_max=24,
                    theta_mode=0, theta=0.01)
    rep = ph.run_stream(cfg, layers=[0])
    assert rep.regions == 5
    print(rep)


@pytest.mark.parametrize("U,persist", [(64, False), (128, False), (40, True)])
def test_unit_granular_retrieval(U, persist):
    # Eq. 8 as printed: fixed units of U tokens ranked by the maximum over their spans and fetched whole; unit
    # selections, the token count of every decode step and the outputs are checked against the oracle
    cfg = small_cfg(n_layers=2, context=1536, decode_steps=4, unit_tokens=U, persist_decode=persist, top_k=3)
    rep = ph.run_stream(cfg, layers=[0, 1])
    assert rep.sel_checks > 20
    print(rep)


@pytest.mark.parametrize("phi_milli,U", [(300, 0), (500, 0), (300, 64)])
def test_overlapping_spans_from_nms_with_iou_threshold(phi_milli, U):
    # NMS with an IoU threshold above zero: spans overlap, selected overlapping spans are attended once per token
    cfg = small_cfg(n_layers=2, context=1536, decode_steps=4, nms_iou_milli=phi_milli, unit_tokens=U, top_k=6,
                    max_spans_per_region=8)
    rep = ph.run_stream(cfg, layers=[0, 1])
    assert rep.sel_checks > 20
    print(rep)


@pytest.mark.parametrize("fused,theta_mode", [("0", 1), ("1", 0), ("2", 1)])
def test_retrieval_heads(fused, theta_mode, monkeypatch):
    # Sec. 3.5: a layer with a retrieval head draws its map, threshold, votes, query representatives and scores from
    # that head alone and fetches one selection for all its KV heads; layers without one keep the default path.  All
    # decode retrieval paths, span-granular retrieval.
    monkeypatch.setenv("LTRI_DEC_FUSED", fused)
    cfg = small_cfg(n_layers=3, context=1408, decode_steps=5, retrieval_head=(5, -1, 2),
                    theta_mode=theta_mode, theta=0.90 if theta_mode else 0.004)
    rep = ph.run_stream(cfg, layers=[0, 1, 2])
    assert rep.sel_checks > 30
    print(rep)


@pytest.mark.parametrize("U,persist,heads,weights", [
    (64, False, (1, -1, 6, 3), (0.5, 0.0, 0.25, 0.25)),
    (32, True, (-1, 4, 4, -1), (0.0, 0.3, 0.3, 0.0)),
    (128, False, (0, 7, 2, 5), None),
])
def test_collaborative_voting(U, persist, heads, weights):
    # Sec. 3.5: every layer with a retrieval head casts its own top-k units as a ballot weighted by the head's score;
    # a layer ranks its units by the tally of the ballots up to its own, then by its own scores.  Ballots, tallied
    # selections, decode token counts and outputs are checked layer by layer.
    cfg = small_cfg(n_layers=4, context=1536, decode_steps=4, unit_tokens=U, persist_decode=persist, top_k=3,
                    retrieval_head=heads, retrieval_head_score=weights, collab_vote=True)
    rep = ph.run_stream(cfg, layers=[0, 1, 2, 3])
    assert rep.sel_checks > 40 and rep.vote_changes > 5   # the other layers' ballots did change selections
    print(rep)


@pytest.mark.parametrize("theta_mode,thetas", [(1, (0.88, 0.93, 0.95)), (0, (0.003, 0.006, 0.0045))])
def test_per_layer_theta_phi_lambda_tables(theta_mode, thetas):
    # the paper's configuration gives theta and phi per layer and a larger lambda to the first layers: every layer of
    # the call must use its own entry (oracle streams are built with the layer's values)
    cfg = small_cfg(n_layers=3, context=1408, decode_steps=3, theta_mode=theta_mode, layer_theta=thetas,
                    layer_nms_iou_milli=(0, 100, 10), layer_rep_lambda=(20.0, 3.0, 0.5), rep_mode=1, ratio_kind=0,
                    min_reps=1, max_reps=4, retrieval_head=(-1, 3, -1))
    rep = ph.run_stream(cfg, layers=[0, 1, 2])
    assert rep.regions >= 30 and rep.rep_counts > 50
    print(rep)


@pytest.mark.parametrize("U,C,chunk,phi", [(64, 3, 128, 0), (32, 2, 128, 0), (48, 2, 96, 0), (64, 3, 128, 300)])
def test_segmentation_per_memory_unit(U, C, chunk, phi):
    # Sec. 3.3: every memory unit is divided into spans on its own -- candidates inside one unit, C spans kept per
    # unit, gaps cut at the unit boundaries; units on the absolute grid (the first region starts at the sink's end,
    # U = 48 does not divide the calls).  The segmenter is compared bit for bit on the GPU's own map.
    cfg = small_cfg(n_layers=2, context=1536 if chunk == 128 else 1152, chunk=chunk, decode_steps=3, unit_tokens=U,
                    max_spans_per_region=C, segment_per_unit=True, top_k=3, nms_iou_milli=phi)
    rep = ph.run_stream(cfg, layers=[0, 1])
    assert rep.regions >= 20
    print(rep)


@pytest.mark.parametrize("cache_units,decay,extra", [
    (4, 0.1, dict(unit_tokens=48, window=256)), (9, 0.5, dict(segment_per_unit=True, max_spans_per_region=3, persist_decode=True)),
    (6, 1.0, dict(retrieval_head=(2, -1), retrieval_head_score=(0.5, 0.0), collab_vote=True)),
])
def test_host_memory_pager(cache_units, decay, extra):
    # Sec. 3.4: evicted rows are mirrored in host memory, the retrieved units of a prefill call come from a unit
    # cache in device memory or, when missing, over the bus from the mirror; decode steps read their units from the
    # cache slots as well (with the persistent mechanism: both sets).  The harness checks the usual parity and, after
    # every call and step, the cache's tags, usage scores and hit/miss counters against the policy model.  The context
    # length leaves the last unit of the indexed range partial.
    kw = dict(n_layers=2, context=2048 - 40, decode_steps=6, unit_tokens=64, top_k=4, host_kv=True,
              cache_units=cache_units, score_decay=decay)
    kw.update(extra)    # (units of 48 tokens with a window of 256: the indexed range ends inside a unit during decode)
    cfg = small_cfg(**kw)
    rep = ph.run_stream(cfg, layers=[0, 1])
    assert rep.cache_misses > 10 and rep.cache_hits > 10
    print(rep)


@pytest.mark.parametrize("groups", ["1", "2"])
def test_host_memory_pager_is_bit_identical_to_the_resident_path(groups, monkeypatch):
    # the same stream through a paged and a resident context: every output bit and every selection equal, also
    # with irregular call sizes (units that are still growing bypass the cache) and after a sequence reset; the
    # paged call issued as one group of layers or as two whose pulls run under the other group's kernels
    monkeypatch.setenv("LTRI_PAGER_GROUPS", groups)
    cfg = small_cfg(n_layers=2, context=1800, decode_steps=4, unit_tokens=48, top_k=5)
    paged = dataclasses.replace(cfg, host_kv=True, cache_units=7, score_decay=0.1)
    st = inputs.SyntheticStream(cfg)
    a, b = binding.Ltri(ph.params_of(cfg)), binding.Ltri(ph.params_of(paged))
    sizes = [128, 100, 128, 7, 128, 128, 61, 128, 128, 128, 128, 128, 96, 128, 128]
    for rnd in range(2):
        t0 = 0
        for n in sizes:
            q, k, v = (x.cuda() for x in st.tokens(t0, n))
            oa = a.ltri_prefill_chunk(0, 0, 2, q, k, v)
            ob = b.ltri_prefill_chunk(0, 0, 2, q, k, v)
            assert torch.equal(oa, ob), f"pass {rnd} call at {t0}"
            for l in range(2):
                assert np.array_equal(a.ltri_get_selected(0, l), b.ltri_get_selected(0, l))
            t0 += n
        assert b.ltri_debug_read(binding.BUF_CACHE_STATS, 0, 1)[1] > 0
        # the paged context keeps sink + a sliding window in device memory: by now the live rows have been moved once
        assert b.ltri_get_stats(0, 0).slab_slides == 1 and a.ltri_get_stats(0, 0).slab_slides == 0
        for step in range(3):      # decode steps read their units from the cache slots
            q, k, v = (x.permute(1, 0, 2, 3).contiguous().cuda() for x in st.tokens(t0 + step, 1, kind=1))
            assert torch.equal(a.ltri_decode_step([0], 0, 2, q, k, v), b.ltri_decode_step([0], 0, 2, q, k, v))
        a.ltri_reset_sequence(0)
        b.ltri_reset_sequence(0)
        assert (b.ltri_debug_read(binding.BUF_CACHE_TAGS, 0, 0) == -1).all()
    assert a.ltri_sync_status() == 0 and b.ltri_sync_status() == 0
    a.close()
    b.close()


def test_sliding_slabs_through_long_decode_and_their_capacity():
    # a paged context holds sink + window in device memory (2 x (window + 2 chunks) + slack rows): a long decode
    # slides the slabs once more, stays bit-identical to the resident path, and ends with a capacity error -- not a
    # fault -- when the tokens since the last eviction no longer fit
    cfg = small_cfg(n_layers=1, context=640, chunk=64, window=128, n_sink=16, decode_steps=900, unit_tokens=32, top_k=3,
                    max_spans_per_region=2)
    paged = dataclasses.replace(cfg, host_kv=True, cache_units=4, score_decay=0.1)
    pa, pb = ph.params_of(cfg), ph.params_of(paged)
    assert binding.ltri_arena_bytes(pb) < binding.ltri_arena_bytes(pa)
    st = inputs.SyntheticStream(cfg)
    a, b = binding.Ltri(pa), binding.Ltri(pb)
    for t0, n in st.prefill_chunks():
        q, k, v = (x.cuda() for x in st.tokens(t0, n))
        assert torch.equal(a.ltri_prefill_chunk(0, 0, 1, q, k, v), b.ltri_prefill_chunk(0, 0, 1, q, k, v))
    slides0 = b.ltri_get_stats(0, 0).slab_slides
    failed_at = None
    for step in range(cfg.decode_steps):
        q, k, v = (x.permute(1, 0, 2, 3).contiguous().cuda() for x in st.tokens(cfg.context + step, 1, kind=1))
        oa = a.ltri_decode_step([0], 0, 1, q, k, v)
        try:
            ob = b.ltri_decode_step([0], 0, 1, q, k, v)
        except binding.LtriError as e:
            assert e.code == binding.LTRI_ECAPACITY
            failed_at = step
            break
        assert torch.equal(oa, ob), f"decode step {step}"
    # window region: 2 * (128 + 128) + 256 = 768 rows
    assert failed_at is not None and failed_at > 256
    assert b.ltri_get_stats(0, 0).slab_slides == slides0 + 1
    assert a.ltri_sync_status() == 0 and b.ltri_sync_status() == 0
    a.close()
    b.close()


def test_voting_layer_by_layer_calls_match_one_call():
    # a real model submits one layer at a time: the ballots of the earlier layers of the same chunk are read from the
    # context's state and the selections must equal those of the all-layers call
    cfg = small_cfg(n_layers=3, context=1024, decode_steps=0, unit_tokens=64, top_k=3, retrieval_head=(2, 5, -1),
                    retrieval_head_score=(0.4, 0.6, 0.0), collab_vote=True)
    st = inputs.SyntheticStream(cfg)
    a, b = binding.Ltri(ph.params_of(cfg)), binding.Ltri(ph.params_of(cfg))
    for t0, n in st.prefill_chunks():
        q, k, v = (x.cuda() for x in st.tokens(t0, n))
        oa = a.ltri_prefill_chunk(0, 0, 3, q, k, v)
        for l in range(3):
            ob = b.ltri_prefill_chunk(0, l, 1, q[l:l + 1].contiguous(), k[l:l + 1].contiguous(), v[l:l + 1].contiguous())
            assert torch.equal(oa[l], ob[0])
            assert np.array_equal(a.ltri_get_selected(0, l), b.ltri_get_selected(0, l))
    assert a.ltri_sync_status() == 0 and b.ltri_sync_status() == 0
    assert (a.ltri_get_selected(0, 2) >= 0).any()
    a.close()
    b.close()


def test_top_k_covering_everything_equals_full_attention():
    # with top_k >= number of spans the streamed output is plain causal attention (oracle O12)
    cfg = small_cfg(n_layers=1, context=640, chunk=64, window=128, top_k=64, max_spans_per_region=2, decode_steps=2)
    sp = ph.StreamPair(cfg, [0])
    st = inputs.SyntheticStream(cfg)
    outs, qs = [], []
    for t0, n in st.prefill_chunks():
        q, k, v = st.tokens(t0, n)
        outs.append(sp.prefill(0, q, k, v)[0])
        qs.append(q[0])
    assert sp.lt.ltri_get_stats(0, 0).n_spans <= 64
    o = sp.orc[(0, 0)]
    pos = [70, 300, 639]
    qall = torch.cat(qs)
    ref = o.full_attention(pos, qall[pos])
    got = torch.cat(outs)[pos].float().cpu().numpy()
    assert np.abs(got - ref).max() <= ph.MAX_ABS
    sp.lt.close()


def test_irregular_call_sizes_and_single_token_calls():
    cfg = small_cfg(n_layers=1, context=900, chunk=128, window=256)
    sp = ph.StreamPair(cfg, [0])
    st = inputs.SyntheticStream(cfg)
    t0 = 0
    for n in [128, 1, 37, 128, 128, 16, 128, 128, 5, 128, 73]:
        q, k, v = st.tokens(t0, n)
        sp.prefill(0, q, k, v)
        t0 += n
    s = sp.lt.ltri_get_stats(0, 0)
    assert s.tokens == t0 and s.n_spans > 0
    for step in range(3):
        q, k, v = st.tokens(t0 + step, 1, kind=1)
        sp.decode([0], q.permute(1, 0, 2, 3).contiguous(), k.permute(1, 0, 2, 3).contiguous(),
                  v.permute(1, 0, 2, 3).contiguous())
    sp.lt.close()
    print(sp.rep)


@pytest.mark.parametrize("paged", [False, True])
def test_batched_decode_independent_sequences(paged):
    # paged: every sequence has its own unit caches and its own sliding slabs (sequence 0 is long enough to slide once,
    # the others are not), and a batched decode step carries one row shift per sequence
    kw = dict(unit_tokens=32, host_kv=True, cache_units=5, window=128, chunk=64, context=1024) if paged else {}
    cfg = small_cfg(**{**dict(n_layers=2, n_seqs=3, context=768, decode_steps=4), **kw})
    sp = ph.StreamPair(cfg, layers=[0, 1], seqs=[0, 1, 2])
    streams = [inputs.SyntheticStream(cfg, seq=s) for s in range(3)]
    for s, st in enumerate(streams):
        upto = cfg.context - (128 if not paged else 320) * s          # different lengths per sequence
        for t0, n in st.prefill_chunks():
            if t0 >= upto:
                break
            q, k, v = st.tokens(t0, n)
            sp.prefill(s, q, k, v, check_out=(t0 + n >= upto))
    lens = [cfg.context - (128 if not paged else 320) * s for s in range(3)]
    if paged:
        assert [sp.lt.ltri_get_stats(s, 0).slab_slides for s in range(3)] == [1, 0, 0]
    for step in range(cfg.decode_steps):
        qs, ks, vs = [], [], []
        for s, st in enumerate(streams):
            q, k, v = st.tokens(lens[s] + step, 1, kind=1)
            qs.append(q[:, 0]); ks.append(k[:, 0]); vs.append(v[:, 0])
        order = [2, 0, 1] if step % 2 else [0, 1, 2]
        sp.decode(order, torch.stack([qs[i] for i in order]), torch.stack([ks[i] for i in order]),
                  torch.stack([vs[i] for i in order]))
    sp.lt.close()
    print(sp.rep)


@pytest.mark.parametrize("fused", ["0", "1", "2"])
def test_decode_retrieval_paths(fused, monkeypatch):
    # decode retrieval has a one-launch path (scores in shared memory) and a two-launch path; check both
    monkeypatch.setenv("LTRI_DEC_FUSED", fused)
    cfg = small_cfg(n_layers=2, context=1280, decode_steps=5, top_k=6)
    rep = ph.run_stream(cfg, layers=[0, 1], deep=False)
    assert rep.sel_checks > 0
    print(rep)


def test_persistent_ctas_walk_several_work_items(monkeypatch):
    # the tensor-core attention kernel is persistent (one CTA per SM); with the CTA count capped every CTA has to
    # process several (token block, KV head, layer) items back to back, including one-tile items
    monkeypatch.setenv("LTRI_TC_MAX_CTAS", "3")
    cfg = small_cfg(n_layers=2, context=1024, decode_steps=0)
    rep = ph.run_stream(cfg, layers=[0, 1], deep=False)
    assert rep.calls == 8
    print(rep)


def test_warp_mma_fallback_path(monkeypatch):
    # the warp-MMA kernels remain selectable; they must match the oracle as well
    monkeypatch.setenv("LTRI_ATTN_IMPL", "mma")
    cfg = small_cfg(n_layers=1, context=768, decode_steps=2)
    rep = ph.run_stream(cfg, layers=[0])
    print(rep)


def test_layer_ranges_are_independent_streams():
    cfg = small_cfg(n_layers=2, context=512, decode_steps=0)
    lt = binding.Ltri(ph.params_of(cfg))
    st = inputs.SyntheticStream(cfg)
    outs_all, outs_split = [], []
    for t0, n in st.prefill_chunks():
        q, k, v = (x.cuda() for x in st.tokens(t0, n))
        outs_all.append(lt.ltri_prefill_chunk(0, 0, 2, q, k, v))
    lt.ltri_reset_sequence(0)
    for t0, n in st.prefill_chunks():
        q, k, v = (x.cuda() for x in st.tokens(t0, n))
        o0 = lt.ltri_prefill_chunk(0, 0, 1, q[:1].contiguous(), k[:1].contiguous(), v[:1].contiguous())
        o1 = lt.ltri_prefill_chunk(0, 1, 1, q[1:].contiguous(), k[1:].contiguous(), v[1:].contiguous())
        outs_split.append(torch.cat([o0, o1]))
    torch.cuda.synchronize()
    for a, b in zip(outs_all, outs_split):
        assert torch.equal(a, b)
    lt.close()


def test_state_and_capacity_errors():
    cfg = small_cfg(n_layers=2, context=256, decode_steps=2)
    lt = binding.Ltri(ph.params_of(cfg))
    st = inputs.SyntheticStream(cfg)
    q, k, v = (x.cuda() for x in st.tokens(0, 128))
    with pytest.raises(binding.LtriError) as e:
        lt.ltri_decode_step([0], 0, 2, q[:, 0][None], k[:, 0][None], v[:, 0][None])   # nothing prefilled yet
    assert e.value.code == binding.LTRI_ESTATE
    lt.ltri_prefill_chunk(0, 0, 2, q, k, v)
    with pytest.raises(binding.LtriError) as e:
        lt.ltri_prefill_chunk(0, 1, 1, q[1:].contiguous(), k[1:].contiguous(), v[1:].contiguous())
        lt.ltri_prefill_chunk(0, 0, 2, q, k, v)                                       # layers out of step
    assert e.value.code == binding.LTRI_ESTATE
    lt.ltri_reset_sequence(0)
    lt.ltri_prefill_chunk(0, 0, 2, q, k, v)
    lt.ltri_prefill_chunk(0, 0, 2, q, k, v)
    with pytest.raises(binding.LtriError) as e:
        lt.ltri_prefill_chunk(0, 0, 2, q, k, v)                                       # beyond max_tokens - decode room
    assert e.value.code == binding.LTRI_ECAPACITY
    qd, kd, vd = q[:, 0][None].contiguous(), k[:, 0][None].contiguous(), v[:, 0][None].contiguous()
    lt.ltri_decode_step([0], 0, 2, qd, kd, vd)
    with pytest.raises(binding.LtriError) as e:
        lt.ltri_prefill_chunk(0, 0, 2, q[:, :1].contiguous(), k[:, :1].contiguous(), v[:, :1].contiguous())
    assert e.value.code == binding.LTRI_ESTATE                                       # prefill after decode
    with pytest.raises(binding.LtriError) as e:
        lt.ltri_decode_step([0, 0], 0, 2, torch.cat([qd, qd]), torch.cat([kd, kd]), torch.cat([vd, vd]))
    assert e.value.code == binding.LTRI_EINVAL                                       # duplicate / too many seqs
    with pytest.raises(binding.LtriError) as e:
        lt.ltri_prefill_chunk(0, 0, 3, q, k, v)
    assert e.value.code == binding.LTRI_EINVAL
    torch.cuda.synchronize()
    assert lt.ltri_sync_status() == 0
    lt.close()


@pytest.mark.parametrize("paged", [False, True])
def test_host_buffer_entry_matches_the_device_entry(paged):
    # the same stream once through ltri_prefill_chunk (device tensors) and once through ltri_prefill_chunk_host
    # (pinned host tensors, layer groups pipelined over internal copy streams): identical outputs and state.
    # paged: the host-entry context also runs the host-memory pager (each layer group spills, slides its slabs and
    # pulls units on its own), against a resident context on the device entry
    cfg = small_cfg(n_layers=6, context=1152 if not paged else 1920, decode_steps=0, unit_tokens=64 if paged else 0)
    dev = torch.device("cuda:0")
    st = inputs.SyntheticStream(cfg)
    lt_d = binding.Ltri(ph.params_of(cfg), device=dev)
    p = ph.params_of(dataclasses.replace(cfg, host_kv=True, cache_units=5) if paged else cfg)
    p.flags |= binding.FLAG_HOST_STAGING
    lt_h = binding.Ltri(p, device=dev)
    outs_h = []
    for t0, n in st.prefill_chunks():
        q, k, v = st.tokens(t0, n)
        ref = lt_d.ltri_prefill_chunk(0, 0, cfg.n_layers, q.to(dev), k.to(dev), v.to(dev))
        hq, hk, hv = (x.contiguous().pin_memory() for x in (q, k, v))
        ho = torch.empty_like(hq).pin_memory()
        lt_h.ltri_prefill_chunk_host(0, 0, cfg.n_layers, hq, hk, hv, ho)
        outs_h.append((ref, ho, (hq, hk, hv)))       # keep the host inputs alive until the work is done
    lt_h.ltri_host_outputs_ready()
    torch.cuda.synchronize(dev)
    assert lt_d.ltri_sync_status() == 0 and lt_h.ltri_sync_status() == 0
    for ref, ho, _ in outs_h:
        assert torch.equal(ref.cpu(), ho)
    for layer in range(cfg.n_layers):
        assert lt_d.ltri_get_spans(0, layer).tolist() == lt_h.ltri_get_spans(0, layer).tolist()
        assert np.array_equal(lt_d.ltri_get_selected(0, layer), lt_h.ltri_get_selected(0, layer))
        assert lt_h.ltri_get_stats(0, layer).slab_slides == (1 if paged else 0)
    # a context created without the staging flag refuses the host entry
    q, k, v = st.tokens(0, cfg.chunk)
    with pytest.raises(binding.LtriError):
        lt_d.ltri_prefill_chunk_host(0, 0, cfg.n_layers, q.contiguous(), k.contiguous(), v.contiguous(), torch.empty_like(q))
    lt_d.close()
    lt_h.close()

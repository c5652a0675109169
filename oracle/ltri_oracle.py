"""ctypes wrapper around the CPU oracle (``ltri_oracle.cpp``).

TEST INFRASTRUCTURE.  Only the tests, the smoke check and the benchmark's CPU-baseline
leg may import this module; the CUDA path never does.  Arrays are numpy; bf16 tensors
are passed as their raw 16-bit patterns (``uint16``).
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "ltri_oracle.cpp")
_LIB = os.path.join(_HERE, "libltri_oracle.so")


def build(force: bool = False) -> str:
    """Compile the oracle with g++ if the shared object is missing or stale."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".tmp{os.getpid()}"
        subprocess.check_call(["g++", "-O2", "-std=c++17", "-shared", "-fPIC", "-pthread", _SRC, "-o", tmp])
        os.replace(tmp, _LIB)
    return _LIB


class _Params(C.Structure):
    _fields_ = [
        ("n_q_heads", C.c_int32), ("n_kv_heads", C.c_int32), ("head_dim", C.c_int32),
        ("chunk", C.c_int32), ("window", C.c_int32), ("n_sink", C.c_int32), ("top_k", C.c_int32),
        ("reps_per_span", C.c_int32), ("max_spans_per_region", C.c_int32),
        ("theta_mode", C.c_int32), ("theta", C.c_float), ("softmax_scale", C.c_float),
        ("max_tokens", C.c_int64),
        ("rep_mode", C.c_int32), ("ratio_kind", C.c_int32), ("min_reps", C.c_int32), ("max_reps", C.c_int32),
        ("rep_lambda", C.c_float), ("persist_decode", C.c_int32), ("unit_tokens", C.c_int32), ("nms_iou_milli", C.c_int32),
        ("segment_per_unit", C.c_int32), ("ret_head", C.c_int32), ("head_weight", C.c_float), ("collab_vote", C.c_int32),
    ]


_lib = None


def lib():
    global _lib
    if _lib is None:
        L = C.CDLL(build())
        vp, ip, i64 = C.c_void_p, C.c_int, C.c_int64
        L.orc_create.restype = vp
        L.orc_create.argtypes = [C.POINTER(_Params)]
        L.orc_destroy.argtypes = [vp]
        L.orc_prefill_local.argtypes = [vp, ip, vp, vp, vp]
        L.orc_prefill_retrieve.argtypes = [vp]
        L.orc_prefill_attend.argtypes = [vp, ip, ip, vp]
        L.orc_append_only.argtypes = [vp, ip, vp, vp]
        L.orc_load_state.argtypes = [vp, ip, ip, vp, vp]
        L.orc_begin_call.argtypes = [vp, ip, vp]
        L.orc_add_pending.argtypes = [vp, ip, ip, ip, vp]
        L.orc_replace_index.argtypes = [vp, ip, vp, vp]
        L.orc_decode_retrieve.argtypes = [vp, vp, vp, vp]
        L.orc_decode_attend.argtypes = [vp, vp]
        L.orc_full_attention.argtypes = [vp, ip, vp, vp, vp]
        for name in ("orc_tokens", "orc_evicted_end", "orc_num_spans", "orc_num_pending_regions",
                     "orc_region_len", "orc_region_start", "orc_num_query_reps"):
            getattr(L, name).argtypes = [vp]
        L.orc_get_spans.argtypes = [vp, vp]
        L.orc_get_index.argtypes = [vp, vp]
        L.orc_get_pending.argtypes = [vp, ip, vp, vp, ip]
        L.orc_set_newest_spans.argtypes = [vp, vp, ip]
        L.orc_get_votes.argtypes = [vp, ip, ip, vp]
        L.orc_get_map.argtypes = [vp, vp]
        L.orc_get_theta_q.argtypes = [vp]
        L.orc_get_theta_q.restype = i64
        L.orc_get_seg_gap.argtypes = [vp]
        L.orc_get_seg_gap.restype = C.c_double
        L.orc_get_query_reps.argtypes = [vp, vp]
        L.orc_get_query_rep_tokens.argtypes = [vp, vp]
        L.orc_get_scores.argtypes = [vp, vp]
        L.orc_get_selected.argtypes = [vp, vp, vp]
        L.orc_set_selected.argtypes = [vp, vp]
        L.orc_theta_q.argtypes = [vp, ip, ip, C.c_float, ip]
        L.orc_theta_q.restype = i64
        L.orc_ta_scores.argtypes = [vp, ip, i64, vp]
        L.orc_segment_map.argtypes = [vp, ip, i64, ip, ip, ip, ip, vp, ip, vp]
        L.orc_top_k.argtypes = [vp, ip, ip, vp, vp]
        L.orc_get_newest_rep_counts.argtypes = [vp, vp, ip]
        L.orc_get_newest_rep_counts.restype = ip
        L.orc_get_persistent.argtypes = [vp, vp]
        L.orc_num_units.argtypes = [vp]
        L.orc_num_units.restype = ip
        L.orc_get_unit_scores.argtypes = [vp, vp]
        L.orc_set_ballots.argtypes = [vp, ip, vp, vp]
        L.orc_get_ballot.argtypes = [vp, vp]
        L.orc_set_ballot.argtypes = [vp, vp]
        L.orc_get_tally.argtypes = [vp, vp]
        L.orc_set_newest_rep_counts.argtypes = [vp, vp, ip]
        L.orc_set_newest_rep_counts.restype = ip
        L.orc_rep_stride.argtypes = [vp]
        L.orc_rep_stride.restype = ip
        L.orc_dynamic_rep_count.argtypes = [vp, ip, ip, ip, ip, C.c_double, ip, ip]
        L.orc_dynamic_rep_count.restype = ip
        L.orc_f32_to_bf16.argtypes = [C.c_float]
        L.orc_f32_to_bf16.restype = C.c_uint16
        _lib = L
    return _lib


def _ptr(a: np.ndarray):
    assert a.flags["C_CONTIGUOUS"]
    return a.ctypes.data_as(C.c_void_p)


def _u16(a) -> np.ndarray:
    """Accept a uint16 numpy array or a torch bf16 tensor (CPU or CUDA)."""
    if isinstance(a, np.ndarray):
        assert a.dtype == np.uint16
        return np.ascontiguousarray(a)
    import torch  # local: torch is only needed for the convenience conversion

    return a.detach().to("cpu").contiguous().view(torch.int16).numpy().view(np.uint16)


class OracleStream:
    """The oracle for one (sequence, layer) stream."""

    def __init__(self, n_q_heads, n_kv_heads, head_dim, chunk, window, n_sink, top_k, max_tokens,
                 reps_per_span=1, max_spans_per_region=None, theta_mode=1, theta=0.90, softmax_scale=0.0,
                 rep_mode=0, ratio_kind=2, min_reps=1, max_reps=4, rep_lambda=2.0, persist_decode=0,
                 unit_tokens=0, nms_iou_milli=0, ret_head=-1, head_weight=0.0, collab_vote=0,
                 segment_per_unit=0):
        if max_spans_per_region is None:
            max_spans_per_region = max(1, chunk // 32)
        self.Hq, self.Hkv, self.d = n_q_heads, n_kv_heads, head_dim
        self.top_k, self.reps = top_k, reps_per_span
        self.chunk, self.window, self.n_sink = chunk, window, n_sink
        self._p = _Params(n_q_heads, n_kv_heads, head_dim, chunk, window, n_sink, top_k, reps_per_span,
                          max_spans_per_region, theta_mode, theta, softmax_scale, max_tokens,
                          rep_mode, ratio_kind, min_reps, max_reps, rep_lambda, persist_decode, unit_tokens, nms_iou_milli,
                          segment_per_unit, ret_head, head_weight, collab_vote)
        self.unit_tokens = unit_tokens
        self.ret_head, self.head_weight = ret_head, head_weight
        self._h = lib().orc_create(C.byref(self._p))
        if not self._h:
            raise ValueError("bad oracle parameters")
        self._n = 0

    def __del__(self):
        try:
            if getattr(self, "_h", None):
                lib().orc_destroy(self._h)
                self._h = None
        except Exception:   # interpreter shutdown: the module globals may be gone already
            pass

    # --- prefill ---------------------------------------------------------
    def prefill_local(self, q, k, v):
        """O1-O6 for one call. q [n][Hq][d], k, v [n][Hkv][d]."""
        q, k, v = _u16(q), _u16(k), _u16(v)
        n = q.shape[0]
        assert q.shape == (n, self.Hq, self.d) and k.shape == (n, self.Hkv, self.d) and v.shape == k.shape
        rc = lib().orc_prefill_local(self._h, n, _ptr(q), _ptr(k), _ptr(v))
        if rc:
            raise RuntimeError(f"oracle prefill_local failed: {rc}")
        self._n = n

    def prefill_retrieve(self):
        lib().orc_prefill_retrieve(self._h)

    def prefill_attend(self, r0=0, r1=None) -> np.ndarray:
        r1 = self._n if r1 is None else r1
        out = np.empty((r1 - r0, self.Hq, self.d), dtype=np.float32)
        lib().orc_prefill_attend(self._h, r0, r1, _ptr(out))
        return out

    def prefill_chunk(self, q, k, v) -> np.ndarray:
        self.prefill_local(q, k, v)
        self.prefill_retrieve()
        return self.prefill_attend()

    # --- test hooks: continue a stream from a given state (no method arithmetic) --------
    def append_only(self, k, v):
        k, v = _u16(k), _u16(v)
        if lib().orc_append_only(self._h, k.shape[0], _ptr(k), _ptr(v)):
            raise RuntimeError("oracle append_only failed")

    def load_state(self, evicted_end, spans, index=None):
        sp = np.ascontiguousarray(np.asarray(spans, dtype=np.int32).reshape(-1, 2))
        kr = None if index is None else np.ascontiguousarray(index, dtype=np.uint16)
        if lib().orc_load_state(self._h, int(evicted_end), len(sp), _ptr(sp), None if kr is None else _ptr(kr)):
            raise ValueError("inconsistent oracle state")

    def replace_index(self, spans, index):
        """Swap the span table and the index vectors ([span][Hkv][d] bf16 bits) of the indexed prefix for given
        ones; the evicted end, the pending regions and the votes stay."""
        sp = np.ascontiguousarray(np.asarray(spans, dtype=np.int32).reshape(-1, 2))
        kr = np.ascontiguousarray(index, dtype=np.uint16)
        assert kr.shape == (len(sp), self.Hkv, self.d)
        if lib().orc_replace_index(self._h, len(sp), _ptr(sp), _ptr(kr)):
            raise ValueError("spans do not tile the indexed prefix")

    def add_pending(self, start, end, spans):
        sp = np.ascontiguousarray(np.asarray(spans, dtype=np.int32).reshape(-1, 2))
        if lib().orc_add_pending(self._h, int(start), int(end), len(sp), _ptr(sp)):
            raise ValueError("inconsistent pending region")

    def begin_call(self, q):
        q = _u16(q)
        if lib().orc_begin_call(self._h, q.shape[0], _ptr(q)):
            raise ValueError("bad call")
        self._n = q.shape[0]

    # --- decode ----------------------------------------------------------
    def decode_retrieve(self, q, k, v):
        q, k, v = _u16(q).reshape(self.Hq, self.d), _u16(k).reshape(self.Hkv, self.d), _u16(v).reshape(self.Hkv, self.d)
        rc = lib().orc_decode_retrieve(self._h, _ptr(q), _ptr(k), _ptr(v))
        if rc:
            raise RuntimeError(f"oracle decode failed: {rc}")

    def decode_attend(self) -> np.ndarray:
        out = np.empty((self.Hq, self.d), dtype=np.float32)
        lib().orc_decode_attend(self._h, _ptr(out))
        return out

    def decode_step(self, q, k, v) -> np.ndarray:
        self.decode_retrieve(q, k, v)
        return self.decode_attend()

    def full_attention(self, positions, q) -> np.ndarray:
        """O12: causal attention of query rows q [cnt][Hq][d] sitting at absolute `positions`."""
        q = _u16(q)
        pos = np.ascontiguousarray(np.asarray(positions, dtype=np.int32))
        out = np.empty((len(pos), self.Hq, self.d), dtype=np.float32)
        lib().orc_full_attention(self._h, len(pos), _ptr(pos), _ptr(q), _ptr(out))
        return out

    # --- state -----------------------------------------------------------
    @property
    def tokens(self):
        return lib().orc_tokens(self._h)

    @property
    def evicted_end(self):
        return lib().orc_evicted_end(self._h)

    def spans(self) -> np.ndarray:
        n = lib().orc_num_spans(self._h)
        a = np.zeros((n, 2), dtype=np.int32)
        if n:
            lib().orc_get_spans(self._h, _ptr(a))
        return a

    def index(self) -> np.ndarray:
        """bf16 bit patterns [span][Hkv][d]."""
        n = lib().orc_num_spans(self._h)
        a = np.zeros((n, self.Hkv, self.d), dtype=np.uint16)
        if n:
            lib().orc_get_index(self._h, _ptr(a))
        return a

    def pending(self):
        """List of (start, end, spans[n][2]) for regions still inside the window."""
        out = []
        cap = 4 * self.chunk
        for r in range(lib().orc_num_pending_regions(self._h)):
            se = np.zeros(2, dtype=np.int32)
            sl = np.zeros((cap, 2), dtype=np.int32)
            c = lib().orc_get_pending(self._h, r, _ptr(se), _ptr(sl), cap)
            out.append((int(se[0]), int(se[1]), sl[:c].copy()))
        return out

    def set_newest_spans(self, spans):
        a = np.ascontiguousarray(np.asarray(spans, dtype=np.int32).reshape(-1, 2))
        if lib().orc_set_newest_spans(self._h, _ptr(a), len(a)):
            raise ValueError("spans do not partition the newest region")

    def votes(self, lo, hi) -> np.ndarray:
        a = np.zeros(hi - lo, dtype=np.int64)
        lib().orc_get_votes(self._h, lo, hi, _ptr(a))
        return a

    def region(self):
        return lib().orc_region_start(self._h), lib().orc_region_len(self._h)

    def map(self) -> np.ndarray:
        m = lib().orc_region_len(self._h)
        a = np.zeros((m, m), dtype=np.int32)
        if m:
            lib().orc_get_map(self._h, _ptr(a))
        return a

    def theta_q(self) -> int:
        return int(lib().orc_get_theta_q(self._h))

    def seg_gap(self) -> float:
        return float(lib().orc_get_seg_gap(self._h))

    def query_reps(self) -> np.ndarray:
        J = lib().orc_num_query_reps(self._h)
        a = np.zeros((self.Hkv, J, self.d), dtype=np.float32)
        if J:
            lib().orc_get_query_reps(self._h, _ptr(a))
        return a

    def query_rep_tokens(self) -> np.ndarray:
        J = lib().orc_num_query_reps(self._h)
        a = np.full((J, lib().orc_rep_stride(self._h)), -1, dtype=np.int32)
        if J and lib().orc_region_len(self._h) > 0:
            lib().orc_get_query_rep_tokens(self._h, _ptr(a))
        return a

    def newest_rep_counts(self) -> np.ndarray:
        """Representative counts of the newest pending region's spans (Sec. 3.3.2 when rep_mode = 1)."""
        a = np.zeros(4096, dtype=np.int32)
        n = lib().orc_get_newest_rep_counts(self._h, _ptr(a), len(a))
        return a[:n].copy()

    def set_newest_rep_counts(self, counts):
        a = np.ascontiguousarray(np.asarray(counts, dtype=np.int32))
        if lib().orc_set_newest_rep_counts(self._h, _ptr(a), len(a)):
            raise ValueError("representative counts do not fit the newest region")

    def scores(self) -> np.ndarray:
        n = lib().orc_num_spans(self._h)
        a = np.zeros((self.Hkv, n), dtype=np.float32)
        if n:
            lib().orc_get_scores(self._h, _ptr(a))
        return a

    def selected(self):
        ids = np.zeros((self.Hkv, self.top_k), dtype=np.int32)
        gaps = np.zeros(self.Hkv, dtype=np.float64)
        lib().orc_get_selected(self._h, _ptr(ids), _ptr(gaps))
        return ids, gaps

    def unit_scores(self) -> np.ndarray:
        """Unit mode: score of every unit that meets the indexed range, [Hkv][units]; unit i is the absolute unit
        n_sink // unit_tokens + i (Eq. 8: the maximum over the unit's spans)."""
        n = lib().orc_num_units(self._h)
        a = np.zeros((self.Hkv, n), dtype=np.float32)
        if n:
            lib().orc_get_unit_scores(self._h, _ptr(a))
        return a

    # --- collaborative voting (Sec. 3.5) ----------------------------------------------
    def set_ballots(self, ballots):
        """Ballots of the preceding layers for the next retrieval, in ascending layer order: a list of
        (weight, unit ids [top_k], -1 padded)."""
        w = np.ascontiguousarray([b[0] for b in ballots], dtype=np.float32)
        ids = np.full((max(len(ballots), 1), self.top_k), -1, dtype=np.int32)
        for i, b in enumerate(ballots):
            ids[i] = np.asarray(b[1], dtype=np.int32)
        lib().orc_set_ballots(self._h, len(ballots), _ptr(w) if len(ballots) else None, _ptr(ids))

    def ballot(self) -> np.ndarray:
        """This layer's own ballot of the last retrieval: absolute unit ids [top_k], -1 padded (all -1 for a layer
        without a retrieval head)."""
        ids = np.zeros(self.top_k, dtype=np.int32)
        lib().orc_get_ballot(self._h, _ptr(ids))
        return ids

    def set_ballot(self, ids):
        a = np.ascontiguousarray(np.asarray(ids, dtype=np.int32).reshape(self.top_k))
        lib().orc_set_ballot(self._h, _ptr(a))

    def tally(self) -> np.ndarray:
        """Summed ballot weights of every unit that meets the indexed range, [units]."""
        a = np.zeros(lib().orc_num_units(self._h), dtype=np.float32)
        if a.size:
            lib().orc_get_tally(self._h, _ptr(a))
        return a

    def persistent(self) -> np.ndarray:
        """Span ids [Hkv][top_k] kept through decode by the persistent mechanism (-1 padded)."""
        ids = np.zeros((self.Hkv, self.top_k), dtype=np.int32)
        lib().orc_get_persistent(self._h, _ptr(ids))
        return ids

    def set_selected(self, ids):
        a = np.ascontiguousarray(np.asarray(ids, dtype=np.int32).reshape(self.Hkv, self.top_k))
        lib().orc_set_selected(self._h, _ptr(a))


# --- stateless pieces ---------------------------------------------------------
def dynamic_rep_count(Mq: np.ndarray, x: int, y: int, kind: int, lam: float, min_reps: int, max_reps: int) -> int:
    """Representative count of the span [x, y] of a region map (Sec. 3.3.2, Eq. r_v)."""
    Mq = np.ascontiguousarray(Mq, dtype=np.int32)
    return int(lib().orc_dynamic_rep_count(_ptr(Mq), Mq.shape[0], x, y, kind, float(lam), min_reps, max_reps))


def theta_q(Mq: np.ndarray, mode: int, theta: float, n_q_heads: int) -> int:
    Mq = np.ascontiguousarray(Mq, dtype=np.int32)
    return int(lib().orc_theta_q(_ptr(Mq), Mq.shape[0], mode, theta, n_q_heads))


def ta_scores(Mq: np.ndarray, thq: int) -> np.ndarray:
    """S[x][y] (x<=y) of Eq. 5 for a square int32 map; entries with x>y are 0."""
    Mq = np.ascontiguousarray(Mq, dtype=np.int32)
    m = Mq.shape[0]
    S = np.zeros((m, m), dtype=np.int64)
    lib().orc_ta_scores(_ptr(Mq), m, int(thq), _ptr(S))
    return S


def segment_map(Mq: np.ndarray, thq: int, max_spans: int, phi_milli: int = 0, unit: int = 0, origin: int = 0):
    """Spans [[start,len],...] covering [0,m) (a partition when phi = 0) and the smallest decisive relative gap.

    unit > 0: the region starts at absolute token `origin` and every unit of `unit` tokens (absolute grid) is
    segmented on its own, `max_spans` kept per unit."""
    Mq = np.ascontiguousarray(Mq, dtype=np.int32)
    m = Mq.shape[0]
    out = np.zeros((2 * m + 1, 2), dtype=np.int32)
    gap = C.c_double(1.0)
    c = lib().orc_segment_map(_ptr(Mq), m, int(thq), max_spans, int(phi_milli), int(unit), int(origin), _ptr(out),
                              len(out), C.byref(gap))
    return out[:c].copy(), gap.value


def top_k(score: np.ndarray, k: int):
    score = np.ascontiguousarray(score, dtype=np.float32)
    ids = np.zeros(k, dtype=np.int32)
    gap = C.c_double(1.0)
    lib().orc_top_k(_ptr(score), len(score), k, _ptr(ids), C.byref(gap))
    return ids, gap.value


def f32_to_bf16(x: float) -> int:
    return int(lib().orc_f32_to_bf16(C.c_float(x)))


class UnitCachePolicy:
    """Which memory units a device-side cache of `capacity` units holds (Sec. 3.4; "GPU cache size" and "score decay
    coefficient" of the implementation details), as this build reads it: at every retrieval the usage score of every
    slot is multiplied by `decay`; a unit the retrieval names that is in the cache gains 1; a named unit that is not
    takes the slot with the lowest score among the slots not named by this retrieval (lowest slot among equals) and
    starts at 1.  Scores are fp32, one rounding per operation.  Results of attention never depend on it.
    """

    def __init__(self, capacity: int, decay: float):
        self.decay = np.float32(decay)
        self.tags = np.full(capacity, -1, dtype=np.int32)
        self.scores = np.zeros(capacity, dtype=np.float32)
        self.hits = 0
        self.misses = 0

    def access(self, units):
        """One retrieval naming `units` (distinct, ascending).  Returns the units that had to be fetched."""
        self.scores = (self.scores * self.decay).astype(np.float32)
        named = np.zeros(len(self.tags), dtype=bool)
        missing = []
        for u in units:
            where = np.nonzero(self.tags == u)[0]
            if len(where):
                named[where[0]] = True
                self.scores[where[0]] = np.float32(self.scores[where[0]] + np.float32(1.0))
                self.hits += 1
            else:
                missing.append(int(u))
        for u in missing:
            free = np.nonzero(~named)[0]
            if len(free) == 0:
                raise ValueError("more units named at once than the cache holds")
            victim = free[np.argmin(self.scores[free])]      # the first minimum: lowest slot among equals
            self.tags[victim] = u
            self.scores[victim] = np.float32(1.0)
            named[victim] = True
            self.misses += 1
        return missing

"""Thin ctypes binding of the C ABI declared in ``include/ltri.h``.

Argument marshalling only: every step of the path runs in the CUDA library.  PyTorch
supplies device memory (the arena, inputs, outputs) and the stream.  There is no CPU
fallback: if the shared library is missing or no CUDA device is present, calls fail.
"""
from __future__ import annotations

import ctypes as C
import os

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libltri.so")

LTRI_OK, LTRI_EINVAL, LTRI_ECAPACITY, LTRI_ESTATE, LTRI_ECUDA, LTRI_EDEVICE, LTRI_ETIMEOUT = 0, -1, -2, -3, -4, -5, -6
FLAG_PERSIST_DECODE = 1
FLAG_HOST_STAGING = 2
FLAG_COLLAB_VOTE = 4
FLAG_SEGMENT_PER_UNIT = 8
FLAG_HOST_KV = 16
BUF_MAP, BUF_VOTES, BUF_INDEX, BUF_THETA, BUF_SCORES, BUF_QREPS, BUF_ROWSTAT, BUF_NREPS = 1, 2, 3, 4, 5, 6, 7, 8
BUF_BALLOT = 9
BUF_CACHE_TAGS, BUF_CACHE_SCORES, BUF_CACHE_STATS = 10, 11, 12

EXPORTS = [
    "ltri_arena_bytes", "ltri_create", "ltri_destroy", "ltri_reset_sequence", "ltri_prefill_chunk",
    "ltri_decode_step", "ltri_get_spans", "ltri_get_pending_spans", "ltri_get_selected", "ltri_get_stats",
    "ltri_sync_status", "ltri_last_cuda_error", "ltri_strerror", "ltri_debug_read", "ltri_span_capacity",
    "ltri_debug_segment_map", "ltri_launch_count", "ltri_profile_enable", "ltri_profile_read",
    "ltri_segment_map_static", "ltri_prefill_chunk_host", "ltri_host_outputs_ready", "ltri_host_kv_bytes",
    "ltri_debug_load_index", "ltri_debug_wait_timeout",
]
KERNEL_CLASSES = ["append", "evict_index", "attn_local", "map_pass", "segment", "score_topk", "attn_retrieved",
                  "decode_retrieve", "decode_attn", "pager_pull"]


class LtriParams(C.Structure):
    _fields_ = [
        ("n_layers", C.c_int32), ("n_q_heads", C.c_int32), ("n_kv_heads", C.c_int32), ("head_dim", C.c_int32),
        ("max_seqs", C.c_int32), ("max_tokens", C.c_int64),
        ("chunk", C.c_int32), ("window", C.c_int32), ("n_sink", C.c_int32), ("top_k", C.c_int32),
        ("reps_per_span", C.c_int32), ("max_spans_per_region", C.c_int32),
        ("theta_mode", C.c_int32), ("theta", C.c_float), ("softmax_scale", C.c_float), ("flags", C.c_uint32),
        ("rep_mode", C.c_int32), ("ratio_kind", C.c_int32), ("min_reps", C.c_int32), ("max_reps", C.c_int32),
        ("rep_lambda", C.c_float), ("unit_tokens", C.c_int32), ("nms_iou_milli", C.c_int32),
        ("retrieval_head", C.POINTER(C.c_int32)), ("retrieval_head_score", C.POINTER(C.c_float)),
        ("layer_theta", C.POINTER(C.c_float)), ("layer_nms_iou_milli", C.POINTER(C.c_int32)),
        ("layer_rep_lambda", C.POINTER(C.c_float)),
        ("host_kv", C.c_void_p), ("host_kv_bytes", C.c_size_t), ("cache_units", C.c_int32), ("score_decay", C.c_float),
        ("arena", C.c_void_p), ("arena_bytes", C.c_size_t),
    ]


class LtriStats(C.Structure):
    _fields_ = [
        ("tokens", C.c_int64), ("evicted_end", C.c_int64), ("n_spans", C.c_int32), ("n_pending_regions", C.c_int32),
        ("index_bytes", C.c_int64), ("retrieved_tokens", C.c_int64), ("last_call_spans", C.c_int32),
        ("slab_slides", C.c_int32),
    ]


class LtriError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__(f"{where}: {strerror(code)} ({code})")


_lib = None


def load():
    """Load libltri.so (must have been built in-tree); raises if it is missing."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise FileNotFoundError(f"{LIB_PATH} not built; run paper_2412_04757_b200/build.py")
        L = C.CDLL(LIB_PATH)
        vp, ip = C.c_void_p, C.c_int
        L.ltri_arena_bytes.restype = C.c_size_t
        L.ltri_arena_bytes.argtypes = [C.POINTER(LtriParams)]
        L.ltri_host_kv_bytes.restype = C.c_size_t
        L.ltri_host_kv_bytes.argtypes = [C.POINTER(LtriParams)]
        L.ltri_create.argtypes = [C.POINTER(LtriParams), vp, C.POINTER(vp)]
        L.ltri_destroy.argtypes = [vp]
        L.ltri_reset_sequence.argtypes = [vp, ip, vp]
        L.ltri_prefill_chunk.argtypes = [vp, ip, ip, ip, ip, vp, vp, vp, vp, vp]
        L.ltri_decode_step.argtypes = [vp, vp, ip, ip, ip, vp, vp, vp, vp, vp]
        L.ltri_prefill_chunk_host.argtypes = [vp, ip, ip, ip, ip, vp, vp, vp, vp, vp]
        L.ltri_host_outputs_ready.argtypes = [vp, vp]
        L.ltri_get_spans.argtypes = [vp, ip, ip, vp, ip, C.POINTER(ip), vp]
        L.ltri_get_pending_spans.argtypes = [vp, ip, ip, vp, ip, C.POINTER(ip), vp]
        L.ltri_get_selected.argtypes = [vp, ip, ip, vp, vp]
        L.ltri_get_stats.argtypes = [vp, ip, ip, C.POINTER(LtriStats), vp]
        L.ltri_sync_status.argtypes = [vp, vp]
        L.ltri_last_cuda_error.argtypes = [vp]
        L.ltri_strerror.restype = C.c_char_p
        L.ltri_strerror.argtypes = [ip]
        L.ltri_debug_read.argtypes = [vp, ip, ip, ip, vp, C.c_size_t, C.POINTER(C.c_size_t), vp]
        L.ltri_span_capacity.argtypes = [vp]
        L.ltri_debug_segment_map.argtypes = [vp, vp, ip, ip, C.c_float, C.c_int64, ip, vp, ip, C.POINTER(ip), vp]
        L.ltri_launch_count.restype = C.c_int64
        L.ltri_launch_count.argtypes = [vp]
        L.ltri_profile_enable.argtypes = [vp, ip]
        L.ltri_profile_read.argtypes = [vp, vp, vp, vp]
        L.ltri_segment_map_static.argtypes = [vp, ip, C.c_int64, ip, vp, ip, vp, vp]
        L.ltri_debug_load_index.argtypes = [vp, ip, ip, C.c_int64, vp, ip, vp, vp]
        L.ltri_debug_wait_timeout.argtypes = [vp, C.c_int64, vp, vp]
        _lib = L
    return _lib


def strerror(code: int) -> str:
    return load().ltri_strerror(code).decode()


def make_params(n_layers, n_q_heads, n_kv_heads, max_tokens, chunk, window, n_sink, top_k, head_dim=128, max_seqs=1,
                reps_per_span=1, max_spans_per_region=0, theta_mode=1, theta=0.90, softmax_scale=0.0,
                rep_mode=0, ratio_kind=2, min_reps=1, max_reps=4, rep_lambda=2.0, flags=0, unit_tokens=0, nms_iou_milli=0,
                retrieval_head=None, retrieval_head_score=None, layer_theta=None, layer_nms_iou_milli=None,
                layer_rep_lambda=None, cache_units=0, score_decay=0.1) -> LtriParams:
    """retrieval_head / retrieval_head_score (head or -1; weight) and layer_theta / layer_nms_iou_milli /
    layer_rep_lambda: per-layer sequences, marshalled into host arrays that live as long as the returned struct."""
    p = LtriParams(n_layers, n_q_heads, n_kv_heads, head_dim, max_seqs, max_tokens, chunk, window, n_sink, top_k,
                   reps_per_span, max_spans_per_region, theta_mode, theta, softmax_scale, flags,
                   rep_mode, ratio_kind, min_reps, max_reps, rep_lambda, unit_tokens, nms_iou_milli, None, None, None, None,
                   None, None, 0, cache_units, score_decay, None, 0)
    if retrieval_head is not None:
        if len(retrieval_head) != n_layers:
            raise ValueError("retrieval_head needs one entry per layer")
        p._rh = (C.c_int32 * n_layers)(*[int(h) for h in retrieval_head])
        p.retrieval_head = C.cast(p._rh, C.POINTER(C.c_int32))
        if retrieval_head_score is not None:
            if len(retrieval_head_score) != n_layers:
                raise ValueError("retrieval_head_score needs one entry per layer")
            p._rw = (C.c_float * n_layers)(*[float(w) for w in retrieval_head_score])
            p.retrieval_head_score = C.cast(p._rw, C.POINTER(C.c_float))
    p._tables = []
    for name, vals, ct in (("layer_theta", layer_theta, C.c_float), ("layer_nms_iou_milli", layer_nms_iou_milli, C.c_int32),
                           ("layer_rep_lambda", layer_rep_lambda, C.c_float)):
        if vals is not None:
            if len(vals) != n_layers:
                raise ValueError(f"{name} needs one entry per layer")
            arr = (ct * n_layers)(*[ct(v).value for v in vals])
            p._tables.append(arr)
            setattr(p, name, C.cast(arr, C.POINTER(ct)))
    return p


def ltri_arena_bytes(params: LtriParams) -> int:
    return int(load().ltri_arena_bytes(C.byref(params)))


def ltri_host_kv_bytes(params: LtriParams) -> int:
    return int(load().ltri_host_kv_bytes(C.byref(params)))


def _check(rc: int, where: str):
    if rc != LTRI_OK:
        raise LtriError(rc, where)


def _dptr(t):
    return C.c_void_p(t.data_ptr())


STATIC_SEGMENT_MAX_M = 256


def ltri_segment_map_static(Mq, theta_q: int, max_spans: int, pairs, n_out, stream=None) -> int:
    """Allocation-free segmenter for callers that cannot allocate device memory where they need it.

    Mq: device int32 tensor [m][m]; pairs: device int32 tensor [cap][2]; n_out: device int32 tensor [1].
    The scratch is a fixed array inside the library, so no context is needed; returns the C status code.
    """
    import torch

    s = stream if stream is not None else torch.cuda.current_stream(Mq.device)
    return int(load().ltri_segment_map_static(_dptr(Mq), Mq.shape[0], int(theta_q), max_spans, _dptr(pairs),
                                              pairs.shape[0], _dptr(n_out), C.c_void_p(s.cuda_stream)))


class Ltri:
    """One library context over a torch-allocated arena.  Methods mirror the C entry points."""

    def __init__(self, params: LtriParams, device="cuda:0", stream=None):
        import torch

        self.torch = torch
        self.lib = load()
        self.device = torch.device(device)
        if self.device.type != "cuda":
            raise ValueError("the ltri library runs on CUDA devices only")
        nbytes = ltri_arena_bytes(params)
        if nbytes == 0:
            raise LtriError(LTRI_EINVAL, "ltri_arena_bytes")
        self.arena = torch.empty(nbytes + 256, dtype=torch.uint8, device=self.device)
        base = (self.arena.data_ptr() + 255) // 256 * 256
        self.params = LtriParams.from_buffer_copy(params)
        self._params_src = params   # owns the host arrays the copy points to
        self.params.arena = base
        self.params.arena_bytes = nbytes
        if params.flags & FLAG_HOST_KV and not params.host_kv:
            # the host mirror of the pager: pinned (page-locked, device-mapped) memory from torch
            hb = ltri_host_kv_bytes(params)
            self.host_kv = torch.empty(hb + 256, dtype=torch.uint8, pin_memory=True)
            self.params.host_kv = (self.host_kv.data_ptr() + 255) // 256 * 256
            self.params.host_kv_bytes = hb
        self.arena_bytes = nbytes
        self._h = C.c_void_p()
        with torch.cuda.device(self.device):
            _check(self.lib.ltri_create(C.byref(self.params), self._stream(stream), C.byref(self._h)), "ltri_create")

    def _stream(self, stream=None):
        s = stream if stream is not None else self.torch.cuda.current_stream(self.device)
        return C.c_void_p(s.cuda_stream)

    def close(self):
        if getattr(self, "_h", None) is not None and self._h.value:
            self.lib.ltri_destroy(self._h)
            self._h = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # --- hot path -----------------------------------------------------------
    def ltri_prefill_chunk(self, seq, layer_begin, layer_count, q, k, v, out=None, stream=None):
        """q [layers][n][Hq][d], k, v [layers][n][Hkv][d] (bf16, device).  Returns out."""
        n = q.shape[1]
        if out is None:
            out = self.torch.empty_like(q)
        rc = self.lib.ltri_prefill_chunk(self._h, seq, layer_begin, layer_count, n, _dptr(q), _dptr(k), _dptr(v),
                                         _dptr(out), self._stream(stream))
        if rc == LTRI_ECUDA:
            raise LtriError(rc, f"ltri_prefill_chunk (cudaError {self.ltri_last_cuda_error()})")
        _check(rc, "ltri_prefill_chunk")
        return out

    def ltri_prefill_chunk_host(self, seq, layer_begin, layer_count, q, k, v, out, stream=None):
        """Same as ltri_prefill_chunk with q, k, v, out in (pinned) host memory.  Returns out, which is complete
        only after ltri_host_outputs_ready(stream) + a synchronisation of that stream."""
        for t in (q, k, v, out):
            if t.device.type != "cpu" or not t.is_contiguous() or t.dtype != self.torch.bfloat16:
                raise ValueError("host entry takes contiguous bf16 CPU tensors")
        rc = self.lib.ltri_prefill_chunk_host(self._h, seq, layer_begin, layer_count, q.shape[1], C.c_void_p(q.data_ptr()),
                                              C.c_void_p(k.data_ptr()), C.c_void_p(v.data_ptr()),
                                              C.c_void_p(out.data_ptr()), self._stream(stream))
        if rc == LTRI_ECUDA:
            raise LtriError(rc, f"ltri_prefill_chunk_host (cudaError {self.ltri_last_cuda_error()})")
        _check(rc, "ltri_prefill_chunk_host")
        return out

    def ltri_host_outputs_ready(self, stream=None):
        _check(self.lib.ltri_host_outputs_ready(self._h, self._stream(stream)), "ltri_host_outputs_ready")

    def ltri_decode_step(self, seq_ids, layer_begin, layer_count, q, k, v, out=None, stream=None):
        """q [n_seqs][layers][Hq][d], k, v [n_seqs][layers][Hkv][d].  Returns out."""
        ids = np.ascontiguousarray(np.asarray(seq_ids, dtype=np.int32))
        if out is None:
            out = self.torch.empty_like(q)
        rc = self.lib.ltri_decode_step(self._h, ids.ctypes.data_as(C.c_void_p), len(ids), layer_begin, layer_count,
                                       _dptr(q), _dptr(k), _dptr(v), _dptr(out), self._stream(stream))
        _check(rc, "ltri_decode_step")
        return out

    def ltri_reset_sequence(self, seq, stream=None):
        _check(self.lib.ltri_reset_sequence(self._h, seq, self._stream(stream)), "ltri_reset_sequence")

    # --- introspection --------------------------------------------------------
    def ltri_get_spans(self, seq, layer, stream=None) -> np.ndarray:
        cap = self.ltri_span_capacity()
        buf = np.zeros((cap, 2), dtype=np.int32)
        n = C.c_int(0)
        _check(self.lib.ltri_get_spans(self._h, seq, layer, buf.ctypes.data_as(C.c_void_p), cap, C.byref(n),
                                       self._stream(stream)), "ltri_get_spans")
        return buf[: n.value].copy()

    def ltri_get_pending_spans(self, seq, layer, stream=None) -> np.ndarray:
        cap = 8 * 1024
        buf = np.zeros((cap, 2), dtype=np.int32)
        n = C.c_int(0)
        _check(self.lib.ltri_get_pending_spans(self._h, seq, layer, buf.ctypes.data_as(C.c_void_p), cap, C.byref(n),
                                               self._stream(stream)), "ltri_get_pending_spans")
        return buf[: n.value].copy()

    def ltri_get_selected(self, seq, layer, stream=None) -> np.ndarray:
        ids = np.zeros((self.params.n_kv_heads, self.params.top_k), dtype=np.int32)
        _check(self.lib.ltri_get_selected(self._h, seq, layer, ids.ctypes.data_as(C.c_void_p), self._stream(stream)),
               "ltri_get_selected")
        return ids

    def ltri_get_stats(self, seq, layer, stream=None) -> LtriStats:
        st = LtriStats()
        _check(self.lib.ltri_get_stats(self._h, seq, layer, C.byref(st), self._stream(stream)), "ltri_get_stats")
        return st

    def ltri_sync_status(self, stream=None) -> int:
        return int(self.lib.ltri_sync_status(self._h, self._stream(stream)))

    def ltri_last_cuda_error(self) -> int:
        return int(self.lib.ltri_last_cuda_error(self._h))

    def ltri_launch_count(self) -> int:
        return int(self.lib.ltri_launch_count(self._h))

    def ltri_profile_enable(self, on: bool):
        _check(self.lib.ltri_profile_enable(self._h, 1 if on else 0), "ltri_profile_enable")

    def ltri_profile_read(self, stream=None):
        """{class name: (ms, launches)} since the previous read."""
        n = len(KERNEL_CLASSES)
        ms = np.zeros(n, dtype=np.float32)
        cnt = np.zeros(n, dtype=np.int64)
        _check(self.lib.ltri_profile_read(self._h, ms.ctypes.data_as(C.c_void_p), cnt.ctypes.data_as(C.c_void_p),
                                          self._stream(stream)), "ltri_profile_read")
        return {KERNEL_CLASSES[i]: (float(ms[i]), int(cnt[i])) for i in range(n)}

    def ltri_span_capacity(self) -> int:
        return int(self.lib.ltri_span_capacity(self._h))

    def ltri_debug_read(self, what, seq, layer, stream=None) -> np.ndarray:
        size = C.c_size_t(0)
        _check(self.lib.ltri_debug_read(self._h, what, seq, layer, None, 0, C.byref(size), self._stream(stream)),
               "ltri_debug_read")
        raw = np.zeros(size.value, dtype=np.uint8)
        _check(self.lib.ltri_debug_read(self._h, what, seq, layer, raw.ctypes.data_as(C.c_void_p), size.value,
                                        C.byref(size), self._stream(stream)), "ltri_debug_read")
        p = self.params
        cap = self.ltri_span_capacity()
        C_ = p.max_spans_per_region if p.max_spans_per_region > 0 else max(1, p.chunk // 32)
        if what == BUF_MAP:
            return raw.view(np.int32).reshape(p.chunk, p.chunk)
        if what == BUF_VOTES:
            return raw.view(np.int64)
        if what == BUF_INDEX:
            return raw.view(np.uint16).reshape(p.n_kv_heads, cap, p.head_dim)
        if what == BUF_THETA:
            return raw.view(np.int64)
        if what == BUF_SCORES:
            return raw.view(np.float32).reshape(p.n_kv_heads, cap)
        if what == BUF_QREPS:
            return raw.view(np.float32).reshape(p.n_kv_heads, -1, p.head_dim)
        if what in (BUF_NREPS, BUF_BALLOT):
            return raw.view(np.int32)
        if what == BUF_CACHE_TAGS:
            return raw.view(np.int32).reshape(p.n_kv_heads, -1)
        if what == BUF_CACHE_SCORES:
            return raw.view(np.float32).reshape(p.n_kv_heads, -1)
        if what == BUF_CACHE_STATS:
            return raw.view(np.int64)
        if what == BUF_ROWSTAT:
            return raw.view(np.float32).reshape(p.chunk, p.n_q_heads, 2)
        return raw

    def ltri_debug_load_index(self, seq, layer, evicted_end, spans: np.ndarray, index_bits: np.ndarray, stream=None):
        """spans int32 [n][2]; index_bits uint16 [Hkv][n][d] (bf16 bit patterns), both on the host."""
        spans = np.ascontiguousarray(spans, dtype=np.int32).reshape(-1, 2)
        index_bits = np.ascontiguousarray(index_bits, dtype=np.uint16)
        n = len(spans)
        if index_bits.shape != (self.params.n_kv_heads, n, self.params.head_dim):
            raise ValueError("index_bits must be [n_kv_heads][n_spans][head_dim]")
        _check(self.lib.ltri_debug_load_index(self._h, seq, layer, int(evicted_end), spans.ctypes.data_as(C.c_void_p), n,
                                              index_bits.ctypes.data_as(C.c_void_p), self._stream(stream)),
               "ltri_debug_load_index")

    def ltri_debug_wait_timeout(self, limit_cycles: int, stream=None) -> np.ndarray:
        """Runs the bounded-wait test kernel; returns the cycles its two waits lasted."""
        waited = np.zeros(2, dtype=np.int64)
        _check(self.lib.ltri_debug_wait_timeout(self._h, int(limit_cycles), waited.ctypes.data_as(C.c_void_p),
                                                self._stream(stream)), "ltri_debug_wait_timeout")
        return waited

    def ltri_debug_segment_map(self, Mq: np.ndarray, theta_mode=2, theta=0.0, theta_q=0, max_spans=None, stream=None):
        Mq = np.ascontiguousarray(Mq, dtype=np.int32)
        m = Mq.shape[0]
        if max_spans is None:
            p = self.params
            max_spans = p.max_spans_per_region if p.max_spans_per_region > 0 else max(1, p.chunk // 32)
        out = np.zeros((2 * m + 2, 2), dtype=np.int32)
        n = C.c_int(0)
        rc = self.lib.ltri_debug_segment_map(self._h, Mq.ctypes.data_as(C.c_void_p), m, theta_mode, theta, int(theta_q),
                                             max_spans, out.ctypes.data_as(C.c_void_p), len(out), C.byref(n),
                                             self._stream(stream))
        _check(rc, "ltri_debug_segment_map")
        return out[: n.value].copy()

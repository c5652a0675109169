"""Seeded synthetic inputs (planted-segment and needle streams).

This module only draws random tensors; it holds none of the method's arithmetic and is
the one piece that both the CUDA path's callers and the CPU oracle's callers may use.

Recipe (stands in for the long-context retrieval workloads the paper evaluates on; only
their shapes are taken: Llama-3-8B attention geometry, 32K-1M token contexts, a needle
at a seeded depth):

* The context of a sequence is cut into segments whose lengths are iid uniform integers
  in ``[seg_min, seg_max]``; the last one is truncated.  Segments are shared by all layers
  and heads of the sequence.
* Keys: every (layer, KV head, segment) has a mean ``mu ~ N(0, I_d)``;
  ``k_t = mu[segment(t)] + 0.3 * eps``.  Values are iid ``N(0, 1)``.
* Queries: every (layer, token) has a target segment shared by the layer's heads;
  ``q_h[t] = mu[g(h)][target] + 0.5 * eps``.  A prefill token targets its own segment with
  probability ``p_self`` and otherwise a uniformly chosen strictly earlier segment (tokens
  of the first segment always target it); a decode token targets a uniformly chosen
  segment that ended before the decode position.
* Needle variant: one extra 64-token segment is inserted at a seeded depth (snapped to a
  segment boundary).  Every (layer, KV head) has a unit direction ``uhat`` and an
  orthogonal unit ``what``; needle keys are ``sqrt(d) * (0.8 uhat + 0.6 what) + 0.3 eps``
  and the queries of the final prefill chunk and of all decode steps are
  ``sqrt(d) * uhat + 0.5 eps`` (cosine 0.8 between the key mean and the query direction).

All tensors are bf16; chunks are generated independently from ``(seed, chunk index)`` so
that a long stream never has to be held in memory at once.
"""
from __future__ import annotations

import dataclasses
import math

import numpy as np
import torch


@dataclasses.dataclass
class StreamConfig:
    """Geometry + method parameters + generator parameters of one workload."""

    name: str
    n_layers: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    context: int          # prefill tokens per sequence
    chunk: int
    decode_steps: int
    n_sink: int
    window: int
    top_k: int
    max_spans_per_region: int
    seg_min: int
    seg_max: int
    n_seqs: int = 1
    needle: bool = False
    p_self: float = 0.5
    reps_per_span: int = 1
    theta_mode: int = 1
    theta: float = 0.90
    seed: int = 2412047570
    rep_mode: int = 0      # 1: dynamic representative counts (Sec. 3.3.2)
    ratio_kind: int = 2
    min_reps: int = 1
    max_reps: int = 4
    rep_lambda: float = 2.0
    nms_iou_milli: int = 0         # NMS IoU threshold in thousandths (0: spans never overlap)
    unit_tokens: int = 0           # retrieval granularity: 0 = spans, U = fixed units of U tokens (Eq. 8 as printed)
    persist_decode: bool = False   # decode keeps the spans selected by the last prefill call (Sec. 3.5)
    retrieval_head: tuple = None   # per layer: retrieval head or -1 (Sec. 3.5); None: no layer has one
    retrieval_head_score: tuple = None   # per layer: the head's score, its voting weight
    collab_vote: bool = False      # collaborative voting over the layers' ballots (Sec. 3.5; needs unit_tokens)
    segment_per_unit: bool = False # every unit of unit_tokens tokens is segmented on its own (Sec. 3.3)
    host_kv: bool = False          # host-memory pager for retrieved units (Sec. 3.4), with a unit cache of
    cache_units: int = 0           # this many units per (seq, layer, KV head) and
    score_decay: float = 0.1       # this decay of the usage scores
    layer_theta: tuple = None          # per-layer tables (None: the scalar holds for every layer)
    layer_nms_iou_milli: tuple = None
    layer_rep_lambda: tuple = None

    @property
    def max_tokens(self) -> int:
        return self.context + self.decode_steps


def config(idx: int) -> StreamConfig:
    """The five benchmark workloads (0 = tiny ... 4 = batched decode)."""
    base = 2412047570
    if idx == 0:
        return StreamConfig("cfg0-tiny", 1, 8, 2, 128, 2048, 256, 16, 64, 512, 4, 8, 32, 256, seed=base)
    if idx == 1:
        return StreamConfig("cfg1-llama8b-32k", 32, 32, 8, 128, 32768, 512, 128, 64, 4096, 32, 16, 32, 512,
                            seed=base + 1)
    if idx == 2:
        return StreamConfig("cfg2-llama8b-128k-needle", 32, 32, 8, 128, 131072, 512, 256, 64, 4096, 32, 16, 32,
                            512, needle=True, seed=base + 2)
    if idx == 3:
        return StreamConfig("cfg3-8layer-1m", 8, 32, 8, 128, 1048576, 1024, 16, 64, 4096, 64, 32, 32, 1024,
                            seed=base + 3)
    if idx == 4:
        return StreamConfig("cfg4-batched-decode-16x128k", 4, 32, 8, 128, 131072, 512, 256, 64, 4096, 32, 16, 32,
                            512, n_seqs=16, seed=base + 4)
    raise ValueError(idx)


class SyntheticStream:
    """Chunk-by-chunk generator for one sequence of a workload."""

    def __init__(self, cfg: StreamConfig, seq: int = 0, device: str | torch.device = "cpu"):
        self.cfg = cfg
        self.seq = seq
        self.device = torch.device(device)
        rng = np.random.default_rng([cfg.seed, seq, 0])
        total = cfg.max_tokens
        lens = []
        covered = 0
        while covered < total:
            ln = int(rng.integers(cfg.seg_min, cfg.seg_max + 1))
            lens.append(ln)
            covered += ln
        self.needle_segment = -1
        if cfg.needle:
            depth = float(rng.random()) * cfg.context
            bounds = np.concatenate([[0], np.cumsum(lens)])
            # snap to a boundary that leaves the needle inside the prefill context
            cand = np.where(bounds <= max(0, cfg.context - 64))[0]
            at = int(cand[np.argmin(np.abs(bounds[cand] - depth))])
            lens.insert(at, 64)
            self.needle_segment = at
        bounds = np.concatenate([[0], np.cumsum(lens)])
        keep = int(np.searchsorted(bounds, total, side="left"))
        self.bounds = bounds[: keep + 1].copy()
        self.bounds[-1] = max(self.bounds[-1], total)
        self.n_segments = len(self.bounds) - 1
        self.seg_of_token = (np.searchsorted(self.bounds, np.arange(total), side="right") - 1).astype(np.int64)

        # per (layer, token) target segment; -1 = the needle query direction
        L = cfg.n_layers
        tgt = np.empty((L, total), dtype=np.int64)
        own = self.seg_of_token
        for layer in range(L):
            r = np.random.default_rng([cfg.seed, seq, 1, layer])
            self_pick = r.random(total) < cfg.p_self
            earlier = np.floor(r.random(total) * np.maximum(own, 1)).astype(np.int64)
            earlier = np.minimum(earlier, np.maximum(own - 1, 0))
            t = np.where(self_pick | (own == 0), own, earlier)
            # decode tokens: a segment that ended before the decode position
            t[cfg.context:] = earlier[cfg.context:]
            tgt[layer] = t
        if cfg.needle:
            final_chunk_start = ((cfg.context - 1) // cfg.chunk) * cfg.chunk
            tgt[:, final_chunk_start:] = -1
        self.target = tgt

        g = torch.Generator(device="cpu")
        g.manual_seed(int(np.random.default_rng([cfg.seed, seq, 2]).integers(0, 2**62)))
        d = cfg.head_dim
        mu = torch.randn(L, cfg.n_kv_heads, self.n_segments, d, generator=g)
        uhat = torch.randn(L, cfg.n_kv_heads, d, generator=g)
        uhat = uhat / uhat.norm(dim=-1, keepdim=True)
        what = torch.randn(L, cfg.n_kv_heads, d, generator=g)
        what = what - (what * uhat).sum(-1, keepdim=True) * uhat
        what = what / what.norm(dim=-1, keepdim=True)
        if cfg.needle:
            mu[:, :, self.needle_segment, :] = math.sqrt(d) * (0.8 * uhat + 0.6 * what)
        self.mu = mu.to(self.device)
        self.qdir = (math.sqrt(d) * uhat).to(self.device)

    def _noise_gen(self, kind: int, idx: int) -> torch.Generator:
        g = torch.Generator(device=self.device)
        g.manual_seed(int(np.random.default_rng([self.cfg.seed, self.seq, 3, kind, idx]).integers(0, 2**62)))
        return g

    def tokens(self, t0: int, n: int, kind: int = 0):
        """q [L][n][Hq][d], k, v [L][n][Hkv][d] (bf16) for tokens [t0, t0+n)."""
        cfg = self.cfg
        L, Hq, Hkv, d = cfg.n_layers, cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim
        G = Hq // Hkv
        dev = self.device
        g = self._noise_gen(kind, t0)
        seg = torch.from_numpy(self.seg_of_token[t0:t0 + n]).to(dev)
        kmean = self.mu[:, :, seg, :].permute(0, 2, 1, 3)               # [L][n][Hkv][d]
        k = kmean + 0.3 * torch.randn(L, n, Hkv, d, generator=g, device=dev)
        v = torch.randn(L, n, Hkv, d, generator=g, device=dev)
        tgt = torch.from_numpy(self.target[:, t0:t0 + n]).to(dev)      # [L][n]
        li = torch.arange(L, device=dev)[:, None].expand(L, n)
        qmean = self.mu[li, :, tgt.clamp(min=0), :]                     # [L][n][Hkv][d]
        if (tgt < 0).any():
            qd = self.qdir[:, None, :, :].expand(L, n, Hkv, d)
            qmean = torch.where((tgt < 0)[:, :, None, None], qd, qmean)
        q = qmean.repeat_interleave(G, dim=2) + 0.5 * torch.randn(L, n, Hq, d, generator=g, device=dev)
        return (q.to(torch.bfloat16).contiguous(), k.to(torch.bfloat16).contiguous(),
                v.to(torch.bfloat16).contiguous())

    def prefill_chunks(self):
        """Yield (t0, n) of the prefill calls."""
        return prefill_calls(self.cfg)

    def needle_range(self):
        if self.needle_segment < 0:
            return None
        return int(self.bounds[self.needle_segment]), int(self.bounds[self.needle_segment + 1])


def prefill_calls(cfg: StreamConfig):
    """Yield (t0, n) of the prefill calls that stream `cfg.context` tokens in chunks."""
    t0 = 0
    while t0 < cfg.context:
        n = min(cfg.chunk, cfg.context - t0)
        yield t0, n
        t0 += n


def random_stream(seed: int, n_tokens: int, n_q_heads: int, n_kv_heads: int, head_dim: int, sharp: float = 1.0):
    """Unstructured iid inputs for small property tests: q [n][Hq][d], k, v [n][Hkv][d] bf16 (CPU)."""
    g = torch.Generator(device="cpu")
    g.manual_seed(seed)
    q = sharp * torch.randn(n_tokens, n_q_heads, head_dim, generator=g)
    k = torch.randn(n_tokens, n_kv_heads, head_dim, generator=g)
    v = torch.randn(n_tokens, n_kv_heads, head_dim, generator=g)
    return q.to(torch.bfloat16), k.to(torch.bfloat16), v.to(torch.bfloat16)


def bf16_bits(t: torch.Tensor) -> np.ndarray:
    """The raw 16-bit patterns of a bf16 tensor as a uint16 numpy array (host copy)."""
    return t.detach().to("cpu").contiguous().view(torch.int16).numpy().view(np.uint16)

"""The allocation-free segmenter entry point against the context-based one.

Some users of the library cannot allocate device memory where they need a segmentation (they run inside a
fully committed memory pool, or under a host that forbids allocation after start-up).  For them the library
keeps the segmenter's scratch in a fixed array of its own.  This test calls that entry point through the C ABI
twice in a row, on different maps, and checks each result against the regular entry point and against the CPU
oracle's segmenter; integer work, so the comparisons are exact.  It is collected last so that a failure here cannot hide another test.
"""
import numpy as np
import pytest
import torch

from oracle import ltri_oracle as orc
from paper_2412_04757_b200 import binding

pytestmark = pytest.mark.gpu


def random_map(m, seed):
    rng = np.random.default_rng(seed)
    return np.tril(rng.integers(0, 2**22, size=(m, m)) * (rng.random((m, m)) < 0.3)).astype(np.int32)


def test_static_scratch_segmenter_matches_context_segmenter_on_two_calls_in_a_row():
    ctx = binding.Ltri(binding.make_params(1, 8, 2, 2048, 256, 512, 64, 4, max_spans_per_region=16))
    dev = torch.device("cuda:0")
    pairs = torch.zeros((64, 2), dtype=torch.int32, device=dev)
    n_out = torch.zeros(1, dtype=torch.int32, device=dev)
    alloc_before = None
    for call, (m, seed, C) in enumerate([(256, 1, 16), (97, 2, 5)]):
        Mq = random_map(m, seed)
        thq = int(np.quantile(Mq[np.tril_indices(m)], 0.9))
        ref = ctx.ltri_debug_segment_map(Mq, theta_mode=2, theta_q=thq, max_spans=C)
        Md = torch.from_numpy(Mq).to(dev)
        torch.cuda.synchronize()
        alloc_before = torch.cuda.memory_allocated(dev)
        rc = binding.ltri_segment_map_static(Md, thq, C, pairs, n_out)
        torch.cuda.synchronize()
        assert rc == binding.LTRI_OK
        assert torch.cuda.memory_allocated(dev) == alloc_before      # nothing came from torch's allocator
        n = int(n_out.item())
        assert n == len(ref), f"call {call}: {n} spans, expected {len(ref)}"
        assert pairs[:n].cpu().numpy().tolist() == ref.tolist(), f"call {call}"
        ref_o, _ = orc.segment_map(Mq, thq, C)
        assert pairs[:n].cpu().numpy().tolist() == ref_o.tolist(), f"call {call}: differs from the oracle's segmenter"
    ctx.close()


def test_static_scratch_segmenter_rejects_sizes_beyond_its_scratch():
    dev = torch.device("cuda:0")
    pairs = torch.zeros((8, 2), dtype=torch.int32, device=dev)
    n_out = torch.zeros(1, dtype=torch.int32, device=dev)
    big = torch.zeros((binding.STATIC_SEGMENT_MAX_M + 1, binding.STATIC_SEGMENT_MAX_M + 1), dtype=torch.int32,
                      device=dev)
    assert binding.ltri_segment_map_static(big, 1, 4, pairs, n_out) == binding.LTRI_ECAPACITY
    ok = torch.zeros((8, 8), dtype=torch.int32, device=dev)
    assert binding.ltri_segment_map_static(ok, 1, 65, pairs, n_out) == binding.LTRI_ECAPACITY
    assert binding.ltri_segment_map_static(ok, 1, 0, pairs, n_out) == binding.LTRI_EINVAL


def test_static_scratch_segmenter_reports_the_full_count_when_the_output_is_short():
    # fewer output pairs than spans: the pairs that fit are written, *n_out still holds the full count
    dev = torch.device("cuda:0")
    Mq = random_map(64, 3)
    thq = int(np.quantile(Mq[np.tril_indices(64)], 0.9))
    ref_o, _ = orc.segment_map(Mq, thq, 6)
    assert len(ref_o) > 2
    pairs = torch.full((2, 2), -7, dtype=torch.int32, device=dev)
    n_out = torch.zeros(1, dtype=torch.int32, device=dev)
    assert binding.ltri_segment_map_static(torch.from_numpy(Mq).to(dev), thq, 6, pairs, n_out) == binding.LTRI_OK
    torch.cuda.synchronize()
    assert int(n_out.item()) == len(ref_o)
    assert pairs.cpu().numpy().tolist() == ref_o[:2].tolist()

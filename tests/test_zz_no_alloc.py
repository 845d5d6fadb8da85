"""mukv_score_frames_noalloc against mukv_compress_chunk.

The entry point under test serves callers that cannot allocate device memory (everything was given
to another pool at start-up, or the allocator is off limits while they run): its scratch is a
fixed array inside the library.  The array is shared by all calls and keeps the previous call's
contents, so the check runs two different calls back to back and both must agree with the regular
entry point: kept token ids bit-exact, scores within the tolerance of the parity tests.
This file is collected last on purpose, so that a failure here cannot hide any other test.
"""
import numpy as np
import pytest
import torch

from paper_2605_22269_b200 import binding as B
from tests import harness as H

pytestmark = pytest.mark.gpu


def _both_ways(name, n_frames, first):
    run = H.GpuRun(name, n_frames=first + n_frames)
    c = run.cfg
    dev = run.device
    q, k, v = run.gs.chunk(first, n_frames)
    kept_ref = torch.full((n_frames, c.keep_per_frame), -1, dtype=torch.int32, device=dev)
    sc_ref = torch.zeros((3, n_frames, c.tokens_per_frame), dtype=torch.float32, device=dev)
    # the regular entry point: frames must continue the stream, so store `first` frames before them
    if first:
        q0, k0, v0 = run.gs.chunk(0, first)
        run.ctx.mukv_compress_chunk(q0, k0, v0, first, 0)
    run.ctx.mukv_compress_chunk(q, k, v, n_frames, first, kept_ref, sc_ref)
    kept = torch.full_like(kept_ref, -2)
    sc = torch.full_like(sc_ref, -2.0)
    B.mukv_score_frames_noalloc(c, q, k[c.n_layers - 1], n_frames, kept, sc)
    torch.cuda.synchronize()
    assert kept.cpu().numpy().tolist() == kept_ref.cpu().numpy().tolist(), f"{name}: kept ids differ"
    H.close(sc.cpu().numpy(), sc_ref.cpu().numpy(), f"{name}: scores")


def test_noalloc_matches_compress_chunk_twice_in_a_row():
    _both_ways("chunk7b", 5, 0)          # bf16, 28 query heads over 4 key heads
    _both_ways("chunk7b", 3, 2)          # fewer frames than the call before: stale scratch must not matter
    _both_ways("tiny", 8, 0)             # fp32


def test_noalloc_rejects_what_does_not_fit():
    wl = H.workload("chunk7b")
    cfg = H.spec_config(wl["spec"], wl)
    x = torch.zeros(64, dtype=torch.bfloat16, device="cuda:0")
    out = torch.zeros(64, dtype=torch.int32, device="cuda:0")
    with pytest.raises(B.MukvError) as e:
        B.mukv_score_frames_noalloc(cfg, x, x, B.NOALLOC_MAX_FRAMES + 1, out, None)
    assert e.value.status == -5 and "static scratch" in str(e.value)
    with pytest.raises(B.MukvError) as e:
        B.mukv_score_frames_noalloc(cfg, x, x, 1, None, None)
    assert e.value.status == -1

"""mukv_score_frames_noalloc against mukv_compress_chunk and against the CPU oracle.

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

from oracle import mukv_oracle as O
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


def test_noalloc_against_the_oracle_with_another_context_created_in_between():
    # the oracle decides, not the other entry point; and a context of a smaller shape created
    # between two calls must not take the scoring kernels' shared memory away
    wl = H.workload("chunk7b")
    spec = wl["spec"]
    cfg = H.spec_config(spec, wl)
    n = 5
    from paper_2605_22269_b200.synth.gpu import GpuStream
    gs = GpuStream(spec, "cuda:0")
    q, k, v = gs.chunk(0, n)
    st = O.Store(dict(H.oracle_cfg(cfg), n_layers=1))
    O.compress_chunk(st, H.to_numpy_bits(q), H.to_numpy_bits(k[-1:]), H.to_numpy_bits(v[-1:]))
    for round_ in range(2):
        kept = torch.full((n, cfg.keep_per_frame), -2, dtype=torch.int32, device="cuda:0")
        sc = torch.full((3, n, cfg.tokens_per_frame), -2.0, dtype=torch.float32, device="cuda:0")
        B.mukv_score_frames_noalloc(cfg, q, k[cfg.n_layers - 1], n, kept, sc)
        torch.cuda.synchronize()
        for f in range(n):
            assert kept[f].cpu().numpy().tolist() == st.kept[f].tolist(), f"round {round_}: kept ids differ at frame {f}"
            for i in range(3):
                H.close(sc[i, f].cpu().numpy(), st.scores[f][i], f"round {round_}: score[{i}] frame {f}")
        if round_ == 0:
            small = H.GpuRun("tiny")                 # fp32, P = 64, D = 64: the smallest shared-memory need
            small.compress()
            B.MukvContext(H.spec_config(H.StreamSpec(seed=5, n_layers=1, n_q_heads=4, n_kv_heads=4, head_dim=64,
                                                     tokens_per_frame=196, bf16=True, n_outlier=0, n_frames=2),
                                        dict(keep=9, fseg=2, chunk=2, alpha=0.7)), "cuda:0").close()


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

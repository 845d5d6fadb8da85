"""Variants beyond the default path, through the C ABI against the CPU oracle: ranking by
caller-supplied scores (the random-drop row of the paper's compression ablation) and moving a
store between buffers (export / import)."""
import ctypes as C

import numpy as np
import pytest
import torch

from oracle import mukv_oracle as O
from paper_2605_22269_b200 import binding as B
from paper_2605_22269_b200.synth.cpu import workload
from tests import harness as H
from tests.test_parity_gpu import full_compress_check, retrieval_check

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("name,n,keep", [("chunk7b", 5, 98), ("tiny", 8, 32), ("chunk7b", 3, 49)])
def test_random_drop_fixture(name, n, keep):
    # "Rand(50%)": uniform random scores from the seeded generator, half of the tokens kept
    run = H.GpuRun(name, n_frames=n, keep_per_frame=keep)
    c = run.cfg
    P = c.tokens_per_frame
    r = run.spec.select_scores(n)                               # [n][P] float32, seeded
    if name == "tiny":
        r[1, 5] = r[1, 9]                                       # an exact tie and a near-tie inside the band
        r[2, 7] = np.float32(r[2, 11] + 4e-7)
    q, k, v = run.gs.chunk(0, n)
    kept = torch.full((n, c.keep_per_frame), -1, dtype=torch.int32, device=run.device)
    run.ctx.mukv_compress_chunk_scored(torch.from_numpy(r).to(run.device), k, v, n, 0, kept)
    torch.cuda.synchronize()
    st = O.Store(H.oracle_cfg(c))
    O.compress_chunk(st, None, H.to_numpy_bits(k), H.to_numpy_bits(v), select_scores=r)
    run.kept = kept.cpu().numpy()
    run.scores = None
    H.check_frames_against_oracle(run, st, range(n), full_layers=True)
    seg = run.ctx.region(3).cpu().numpy()
    for u in range(st.n_segments):
        sk, sv = st.segment_entry(u)
        H.close(seg[u][:, 0], sk, f"segment entry K {u}")
    assert run.ctx.mukv_get_stats().device_status == 0 and run.ctx.mukv_get_stats().refined_frames == 0


def test_export_import_continues_the_stream():
    # 11 frames: 6 stored, store copied to a new buffer, imported, the other 5 appended there;
    # the result must equal the oracle's uninterrupted stream, and retrieval must work on the copy
    wl = dict(workload("chunk7b"))
    wl["fseg"] = 4
    a = H.GpuRun(wl, n_frames=11, max_frames=11)
    c = a.cfg
    q, k, v = a.gs.chunk(0, 6)
    a.ctx.mukv_compress_chunk(q, k, v, 6, 0)
    torch.cuda.synchronize()
    hdr = a.ctx.mukv_export_header()
    assert hdr.frames == 6 and hdr.store_bytes == a.store_bytes()
    b_ctx = B.MukvContext.from_copy(hdr, a.ctx.store.clone())
    a.ctx.close()
    kept = torch.full((11, c.keep_per_frame), -1, dtype=torch.int32, device=a.device)
    q2, k2, v2 = a.gs.chunk(6, 5)
    b_ctx.mukv_compress_chunk(q2, k2, v2, 5, 6, kept[6:])
    torch.cuda.synchronize()
    run = a
    run.ctx = b_ctx
    st = H.oracle_stream(run.spec, H.oracle_cfg(c), range(11), last_only=False, workers=1)
    kept[:6] = b_ctx.region(1)[:6]
    run.kept = kept.cpu().numpy()
    run.scores = None
    H.check_frames_against_oracle(run, st, range(11), full_layers=True)
    seg = b_ctx.region(3).cpu().numpy()
    for u in range(st.n_segments):
        sk, sv = st.segment_entry(u)
        H.close(seg[u][:, 0], sk, f"segment entry K {u}")
        H.close(seg[u][:, 1], sv, f"segment entry V {u}")
        assert b_ctx.region(5)[u].cpu().numpy().tobytes() == st.segment_key(u).tobytes()
    qtok, offs, _ = run.spec.questions(3, 4, 9)
    retrieval_check(run, st, qtok, offs, 2, 3, 0.3, B.RETR_SEMI)
    # a header that does not belong to the buffer is refused on the host
    bad = B.MukvStoreHeader.from_buffer_copy(hdr)
    bad.magic = 1
    with pytest.raises(B.MukvError):
        B.MukvContext.from_copy(bad, b_ctx.store)


def _layered_inputs(spec, n, Ls):
    """Q for Ls scoring layers: layer l of the stack comes from the seeded stream of seed + 100 * l."""
    import copy
    qs = []
    for l in range(Ls):
        sp = copy.copy(spec)
        sp.seed = spec.seed + 100 * l
        qs.append(np.stack([sp.frame_q(t) for t in range(n)]))
    q = np.stack(qs)                                            # [Ls][n][P][Hq][D]
    kv = [spec.frame_kv(t) for t in range(n)]
    k = np.stack([x[0] for x in kv], axis=1)                    # [L][n][P][Hkv][D]
    v = np.stack([x[1] for x in kv], axis=1)
    return q, k, v


@pytest.mark.parametrize("name,Ls,off,opts", [("chunk7b", 5, 0, None), ("chunk7b", 1, 1, None), ("chunk7b", 1, 14, None),
                                              ("chunk7b", 2, 3, {B.OPT_FLAG_MARGIN: 1.0}),
                                              ("chunk7b", 3, 0, {B.OPT_SCORE_PATH: 1})])
def test_scoring_layer_choice_bf16(name, Ls, off, opts):
    # the layer-choice ablation: last-5 fusion, penultimate, middle; also through the double-precision
    # pass (every frame flagged) and on the multiply-add kernel
    n = 4
    run = H.GpuRun(name, n_frames=n, n_score_layers=Ls, score_layer_offset=off, options=opts)
    c = run.cfg
    q, k, v = _layered_inputs(run.spec, n, Ls)
    dq = H.to_device(q if Ls > 1 else q[0], True, run.device)
    dk, dv = H.to_device(k, True, run.device), H.to_device(v, True, run.device)
    kept = torch.full((n, c.keep_per_frame), -1, dtype=torch.int32, device=run.device)
    sc = torch.zeros((3, n, c.tokens_per_frame), dtype=torch.float32, device=run.device)
    run.ctx.mukv_compress_chunk(dq, dk, dv, n, 0, kept, sc)
    torch.cuda.synchronize()
    st = O.Store(H.oracle_cfg(c))
    O.compress_chunk(st, q if Ls > 1 else q[0], k, v)
    run.kept, run.scores = kept.cpu().numpy(), sc.cpu().numpy()
    H.check_frames_against_oracle(run, st, range(n), full_layers=True)
    stats = run.ctx.mukv_get_stats()
    assert stats.device_status == 0
    if opts and B.OPT_FLAG_MARGIN in opts:
        assert stats.refined_frames == n


def test_scoring_layer_choice_fp32():
    spec = H.StreamSpec(seed=51, n_layers=4, n_q_heads=4, n_kv_heads=2, head_dim=64, tokens_per_frame=40, bf16=False,
                        n_outlier=1, n_frames=3, scene_sigma=1.0, frame_sigma=0.5, scene_min=2, scene_max=3)
    wl = dict(spec=spec, keep=11, fseg=2, chunk=3, alpha=0.7)
    run = H.GpuRun(wl, n_score_layers=3, score_layer_offset=1)
    q, k, v = _layered_inputs(spec, 3, 3)
    dq, dk, dv = (H.to_device(x, False, run.device) for x in (q, k, v))
    kept = torch.full((3, 11), -1, dtype=torch.int32, device=run.device)
    sc = torch.zeros((3, 3, 40), dtype=torch.float32, device=run.device)
    run.ctx.mukv_compress_chunk(dq, dk, dv, 3, 0, kept, sc)
    torch.cuda.synchronize()
    st = O.Store(H.oracle_cfg(run.cfg))
    O.compress_chunk(st, q, k, v)
    run.kept, run.scores = kept.cpu().numpy(), sc.cpu().numpy()
    H.check_frames_against_oracle(run, st, range(3), full_layers=True)


def _small_bf16_spec(T):
    return H.StreamSpec(seed=71, n_layers=3, n_q_heads=8, n_kv_heads=2, head_dim=64, tokens_per_frame=100, bf16=True,
                        n_outlier=1, n_frames=T, scene_sigma=1.0, frame_sigma=0.5, scene_min=2, scene_max=4)


def test_past_keys_with_two_scoring_layers_bf16():
    # cached keys of the matching layer for each scoring layer (planes of the stored pages)
    import copy
    T, chunk, W = 7, 2, 3
    spec = _small_bf16_spec(T)
    run = H.GpuRun(dict(spec=spec, keep=25, fseg=2, chunk=chunk, alpha=0.7), past_frames=W, n_score_layers=2,
                   score_layer_offset=0)
    c = run.cfg
    sp2 = copy.copy(spec)
    sp2.seed = spec.seed + 100
    st = O.Store(H.oracle_cfg(c))
    kept = torch.full((T, c.keep_per_frame), -1, dtype=torch.int32, device=run.device)
    scores = torch.zeros((3, T, c.tokens_per_frame), dtype=torch.float32, device=run.device)
    for t0 in range(0, T, chunk):
        n = min(chunk, T - t0)
        q, k, v = spec.chunk(t0, n)
        q = np.stack([q, np.stack([sp2.frame_q(t) for t in range(t0, t0 + n)])])
        O.compress_chunk(st, q, k, v)
        dq, dk, dv = (H.to_device(x, True, run.device) for x in (q, k, v))
        sc = torch.empty((3, n, c.tokens_per_frame), dtype=torch.float32, device=run.device)
        run.ctx.mukv_compress_chunk(dq, dk, dv, n, t0, kept[t0:t0 + n], sc)
        scores[:, t0:t0 + n] = sc
    torch.cuda.synchronize()
    run.kept, run.scores = kept.cpu().numpy(), scores.cpu().numpy()
    H.check_frames_against_oracle(run, st, range(T), full_layers=True)
    assert st.scores[T - 1][0].sum() < 0.999 and run.ctx.mukv_get_stats().device_status == 0


def _oracle_chunked(spec, ocfg, T, chunk):
    st = O.Store(ocfg)
    for t0 in range(0, T, chunk):
        q, k, v = spec.chunk(t0, min(chunk, T - t0))
        O.compress_chunk(st, q, k, v)
    return st


@pytest.mark.parametrize("name,T,chunk,W,over,opts", [
    ("tiny", 8, 3, 3, dict(), None),
    ("tiny", 8, 2, 2, dict(attn_causal=1), None),
    ("chunk7b", 6, 2, 1, dict(), None),
    ("chunk7b", 5, 2, 1, dict(attn_causal=1), {B.OPT_FLAG_MARGIN: 1.0}),
    ("chunk7b", 4, 2, 1, dict(), {B.OPT_SCORE_PATH: 1}),
    ("chunk7b", 37, 16, 1, dict(), None),
    ("small_bf16", 9, 2, 3, dict(), None),
    ("small_bf16", 7, 3, 2, dict(attn_causal=1, keep_low_freq=1), None),
])
def test_past_keys_in_the_attention(name, T, chunk, W, over, opts):
    # Sec. 3.2: the queries of a chunk also attend to the kept keys of the W frames stored before it.
    # bf16 chunks go through the tensor-core kernel (the cached keys are rows of its key tile) unless
    # the multiply-add path is asked for; "small_bf16" has room for three past frames in the tile
    if name == "small_bf16":
        name = dict(spec=_small_bf16_spec(T), keep=25, fseg=2, chunk=chunk, alpha=0.7)
    run = H.GpuRun(name, n_frames=T, past_frames=W, options=opts, **over)
    run.compress(chunk)
    st = _oracle_chunked(run.spec, H.oracle_cfg(run.cfg), T, chunk)
    H.check_frames_against_oracle(run, st, range(T), full_layers=True)
    # the past really takes attention mass away from the frame's own tokens (not in the first chunk)
    assert abs(st.scores[0][0].sum() - 1.0) < 1e-9 and st.scores[T - 1][0].sum() < 0.999
    stats = run.ctx.mukv_get_stats()
    assert stats.device_status == 0
    if opts and B.OPT_FLAG_MARGIN in opts:
        assert stats.refined_frames == T
    if not opts and run.spec.bf16:
        # tensor-core path with cached keys in the tile: the headroom the single-precision selection rests on
        worst = max(float(np.max(np.abs(run.scores[2, t] - st.scores[t][2]))) for t in range(T))
        assert worst < H.FLAG_MARGIN / 2 and stats.refined_frames <= max(1, T // 8), (worst, stats.refined_frames)

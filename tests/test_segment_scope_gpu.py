"""Segment-level dual-signal selection (Sec. 3.3: indicator over the O = F*P tokens of a segment,
kappa_v = floor(rho_v * O) kept, a variable number per frame) with pages of different lengths,
CUDA path against the oracle."""
import numpy as np
import pytest
import torch

from oracle import mukv_oracle as O
from paper_2605_22269_b200 import binding as B
from paper_2605_22269_b200.synth.cpu import StreamSpec, workload
from tests import harness as H
from tests.test_granularities_gpu import retrieve3_check

pytestmark = pytest.mark.gpu


def compress_segment_scope(run, chunk):
    c = run.cfg
    T, P = run.n_frames, c.tokens_per_frame
    kept = torch.full((T, P), -7, dtype=torch.int32, device=run.device)
    scores = torch.zeros((3, T, P), dtype=torch.float32, device=run.device)
    for t0 in range(0, T, chunk):
        n = min(chunk, T - t0)
        q, k, v = run.gs.chunk(t0, n)
        sc = torch.empty((3, n, P), dtype=torch.float32, device=run.device)
        run.ctx.mukv_compress_chunk(q, k, v, n, t0, kept[t0:t0 + n], sc)
        scores[:, t0:t0 + n] = sc
    torch.cuda.synchronize()
    return kept.cpu().numpy(), scores.cpu().numpy()


def check_store(run, st, kept, scores):
    c = run.cfg
    T, P, L = run.n_frames, c.tokens_per_frame, c.n_layers
    cnt = run.ctx.region(10).cpu().numpy()
    ids = run.ctx.region(1).cpu().numpy()
    pt = run.ctx.region(7).cpu().numpy()
    raw = run.ctx.store.cpu().numpy()
    es = 2 if run.spec.bf16 else 4
    row = run.ctx.C * es
    fent = run.ctx.region(2).cpu().numpy()
    for t in range(T):
        n_t = len(st.kept[t])
        assert cnt[t] == n_t, f"frame {t}: {cnt[t]} tokens kept, oracle {n_t}"
        assert kept[t, :n_t].tolist() == st.kept[t].tolist() and np.all(kept[t, n_t:] == -1), f"kept ids frame {t}"
        assert ids[t, :n_t].tolist() == st.kept[t].tolist()
        for s in range(3):
            H.close(scores[s, t], st.scores[t][s], f"score[{s}] frame {t}")
        page = raw[pt[t]:pt[t] + L * 2 * n_t * row].reshape(L, 2, n_t * row)
        assert page[:, 0].tobytes() == st.page_k[t].tobytes(), f"K page bytes differ at frame {t}"
        assert page[:, 1].tobytes() == st.page_v[t].tobytes(), f"V page bytes differ at frame {t}"
        ek, ev = st.frame_entry(t)
        H.close(fent[t][:, 0], ek, f"frame entry K {t}")
        H.close(fent[t][:, 1], ev, f"frame entry V {t}")
        assert run.ctx.region(4)[t].cpu().numpy().tobytes() == st.frame_key(t).tobytes(), f"frame key {t}"
    seg = run.ctx.region(3).cpu().numpy()
    for u in range(st.n_segments):
        sk, sv = st.segment_entry(u)
        H.close(seg[u][:, 0], sk, f"segment entry K {u}")
        H.close(seg[u][:, 1], sv, f"segment entry V {u}")
        assert run.ctx.region(5)[u].cpu().numpy().tobytes() == st.segment_key(u).tobytes(), f"segment key {u}"
    stats = run.ctx.mukv_get_stats()
    assert stats.kept_tokens == sum(len(k) for k in st.kept) and stats.device_status == 0


@pytest.mark.parametrize("opts,refined", [(None, None), ({B.OPT_FLAG_MARGIN: 1.0}, 10), ({B.OPT_SCORE_PATH: 1}, 0)])
def test_segment_scope_bf16(opts, refined):
    # the 7B layout, segments of 4 frames, rho_v = 0.25 over the 784 tokens of a segment; the stream
    # ends with a segment of two frames.  Scored on the tensor cores and ranked in single precision
    # where that is safe; with a margin nothing passes, every segment through the double-precision
    # pass behind it; on the multiply-add path, double precision from the start
    wl = dict(workload("chunk7b"))
    wl["fseg"] = 4
    kv = O.keep_count(0.25, 4 * 196)
    run = H.GpuRun(wl, n_frames=10, max_frames=12, keep_per_segment=kv, options=opts)
    kept, scores = compress_segment_scope(run, 8)
    st = oracle_stream_chunked(run.spec, H.oracle_cfg(run.cfg), 10, 8)
    counts = [len(k) for k in st.kept]
    assert sum(counts[:4]) == kv and sum(counts[8:]) == kv // 2 and len(set(counts)) > 1
    check_store(run, st, kept, scores)
    n_ref = run.ctx.mukv_get_stats().refined_frames
    assert n_ref <= 4 if refined is None else n_ref == refined, n_ref
    if opts:
        return
    qtok, offs, _ = run.spec.questions(4, 3, 9)
    for mode in (B.RETR_SEMI, B.RETR_PARALLEL, B.RETR_HIER):
        retrieve3_check(run, st, qtok, offs, (0, 3, 2), (0.0, 0.3, 0.0), mode)
    # what a store of this kind does not do
    dec = torch.zeros(1 << 20, dtype=torch.uint8, device=run.device)
    idx = torch.zeros((1, 2), dtype=torch.int32, device=run.device)
    with pytest.raises(B.MukvError) as e:
        run.ctx.mukv_gather(idx, idx, 1, 2, dec, 1 << 20)
    assert e.value.status == -8
    with pytest.raises(B.MukvError) as e:                  # the stream has ended with a short segment
        q, k, v = run.gs.chunk(10, 1)
        run.ctx.mukv_compress_chunk(q, k, v, 1, 10)
    assert e.value.status == -6


@pytest.mark.parametrize("over", [dict(), dict(alpha=0.0), dict(alpha=1.0), dict(keep_low_freq=1, attn_causal=1),
                                  dict(n_score_layers=2, score_layer_offset=1)])
def test_segment_scope_sixteen_frame_segments(over):
    # segments of 16 frames (3,136 tokens ranked at once), two full segments and one of five frames,
    # chunks of 16 frames; Eq. 4 variants and two scoring layers on the tensor-core path
    wl = dict(workload("chunk7b"))
    wl["fseg"] = 16
    kv = O.keep_count(0.25, 16 * 196)
    T = 37
    run = H.GpuRun(wl, n_frames=T, max_frames=48, keep_per_segment=kv, **over)
    c = run.cfg
    Ls = max(1, c.n_score_layers)
    P = c.tokens_per_frame
    kept = torch.full((T, P), -7, dtype=torch.int32, device=run.device)
    scores = torch.zeros((3, T, P), dtype=torch.float32, device=run.device)
    st = O.Store(H.oracle_cfg(c))
    for t0 in range(0, T, 16):
        n = min(16, T - t0)
        q, k, v = run.spec.chunk(t0, n)
        if Ls > 1:                                            # a second scoring layer from another seeded stream
            import copy
            sp2 = copy.copy(run.spec)
            sp2.seed = run.spec.seed + 100
            q = np.stack([q, np.stack([sp2.frame_q(t) for t in range(t0, t0 + n)])])
        O.compress_chunk(st, q, k, v)
        dq, dk, dv = (H.to_device(x, True, run.device) for x in (q, k, v))
        sc = torch.empty((3, n, P), dtype=torch.float32, device=run.device)
        run.ctx.mukv_compress_chunk(dq, dk, dv, n, t0, kept[t0:t0 + n], sc)
        scores[:, t0:t0 + n] = sc
    torch.cuda.synchronize()
    sc_np = scores.cpu().numpy()
    check_store(run, st, kept.cpu().numpy(), sc_np)
    assert run.ctx.mukv_get_stats().refined_frames <= 16
    # the headroom the single-precision ranking rests on: fused scores within half the safety margin
    worst = max(float(np.max(np.abs(sc_np[2, t] - st.scores[t][2]))) for t in range(T))
    assert worst < H.FLAG_MARGIN / 2, worst


def test_segment_scope_bf16_odd_token_count():
    # P = 77 (not a multiple of four: the scalar loads of the single-precision ranking), G = 3, D = 64,
    # segments of four frames in chunks of eight, a last segment of three frames
    spec = StreamSpec(seed=13, n_layers=3, n_q_heads=6, n_kv_heads=2, head_dim=64, tokens_per_frame=77, bf16=True,
                      n_outlier=2, n_frames=11, scene_sigma=1.0, frame_sigma=0.5, scene_min=3, scene_max=5)
    wl = dict(spec=spec, keep=19, fseg=4, chunk=8, alpha=0.7)
    run = H.GpuRun(wl, keep_per_segment=O.keep_count(0.3, 4 * 77))
    kept, scores = compress_segment_scope(run, 8)
    st = oracle_stream_chunked(spec, H.oracle_cfg(run.cfg), 11, 8)
    check_store(run, st, kept, scores)
    assert run.ctx.mukv_get_stats().refined_frames <= 4


def oracle_stream_chunked(spec, ocfg, T, chunk):
    st = O.Store(ocfg)
    for t0 in range(0, T, chunk):
        n = min(chunk, T - t0)
        q, k, v = spec.chunk(t0, n)
        O.compress_chunk(st, q, k, v)
    return st


@pytest.mark.parametrize("over", [dict(), dict(alpha=0.0), dict(keep_low_freq=1, attn_causal=1)])
def test_segment_scope_fp32(over):
    spec = StreamSpec(seed=61, n_layers=3, n_q_heads=4, n_kv_heads=2, head_dim=64, tokens_per_frame=50, bf16=False,
                      n_outlier=1, n_frames=11, scene_sigma=1.0, frame_sigma=0.5, scene_min=2, scene_max=4)
    wl = dict(spec=spec, keep=10, fseg=3, chunk=6, alpha=0.8)
    run = H.GpuRun(wl, keep_per_segment=O.keep_count(0.8, 150), **over)
    kept, scores = compress_segment_scope(run, 6)
    st = oracle_stream_chunked(spec, H.oracle_cfg(run.cfg), 11, 6)
    check_store(run, st, kept, scores)
    qtok, offs, _ = spec.questions(3, 2, 6)
    retrieve3_check(run, st, qtok, offs, (0, 4, 2), (0.0, 0.3, 0.0), B.RETR_SEMI, t_limit=np.array([11, 5, 7]))

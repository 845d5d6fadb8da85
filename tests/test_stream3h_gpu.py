"""Full-size workloads (three-hour stream and the 64-question retrieval stress) in the launch
configuration the benchmark times.  The compression of all 10,800 frames runs on the GPU; the
oracle checks every frame's selection on the last layer (all that scoring reads), sampled frames
on all layers, and every question of the retrieval stress."""
import numpy as np
import pytest

from oracle import mukv_oracle as O
from paper_2605_22269_b200 import binding as B
from tests import harness as H

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def stream3h():
    run = H.GpuRun("stream_3h", want_scores=True).compress()
    st = H.oracle_stream(run.spec, H.oracle_cfg(run.cfg), range(run.n_frames), last_only=True)
    return run, st


def test_stream_3h_selection_and_keys(stream3h):
    run, st = stream3h
    T = run.n_frames
    stats = run.ctx.mukv_get_stats()
    assert T == 10800 and stats.frames == T and stats.segments == 675
    assert stats.store_bytes_used == T * 2_809_856                       # ~30.35 GB of kept KV
    worst = H.check_frames_against_oracle(run, st, range(T), full_layers=False)
    print(f"stream_3h: max |fused score - oracle| = {worst:.3e}; refined frames = {stats.refined_frames}")
    # index exactness rests on these two: the single-precision score error stays below half the
    # safety margin, and the double-precision pass stays the exception (0.14 % of the frames when
    # this was written)
    assert worst < H.FLAG_MARGIN / 2
    assert stats.refined_frames <= T // 200
    assert run.ctx.region(4).cpu().numpy()[:T].tobytes() == st.frame_keys().tobytes()
    assert run.ctx.region(5).cpu().numpy()[:675].tobytes() == st.segment_keys().tobytes()


def test_stream_3h_sampled_pages(stream3h):
    run, st = stream3h
    rng = np.random.default_rng(4)
    sample = sorted(set([0, 15, 16, 10799] + rng.integers(0, run.n_frames, size=12).tolist()))
    full = H.oracle_stream(run.spec, H.oracle_cfg(run.cfg), sample, last_only=False, workers=1)
    H.check_frames_against_oracle(run, full, sample, full_layers=True)
    # one whole segment on all layers
    u = 337
    seg = H.oracle_stream(run.spec, H.oracle_cfg(run.cfg), range(16 * u, 16 * u + 16), last_only=False, workers=1)
    sk = np.sum(seg.sum_k, axis=0) / (16.0 * run.cfg.keep_per_frame)
    sv = np.sum(seg.sum_v, axis=0) / (16.0 * run.cfg.keep_per_frame)
    got = run.ctx.region(3)[u].cpu().numpy()
    H.close(got[:, 0], sk.astype(np.float32), "segment entry K")
    H.close(got[:, 1], sv.astype(np.float32), "segment entry V")


def test_retrieval_stress(stream3h):
    run, st = stream3h
    wl = run.wl
    qtok, offs, scenes = run.spec.questions(wl["n_questions"], *wl["q_len"])
    nq, k_seg, k_frm = wl["n_questions"], wl["k_seg"], wl["k_frm"]
    ret = run.retrieve(qtok, offs, k_seg, k_frm, 0, wl["lam"], B.RETR_SEMI)
    dec, meta = run.gather(ret, k_frm)
    frm = ret["frm_idx"].cpu().numpy()
    seg = ret["seg_idx"].cpu().numpy()
    fsc = ret["frm_score"].cpu().numpy()
    hits = 0
    sc_of = run.spec.scene_of_frame()
    for i in range(nq):
        r = O.retrieve(st, qtok[offs[i]:offs[i + 1]], k_seg, k_frm, 0, wl["lam"], O.MODE_SEMI)
        assert seg[i].tolist() == r["seg_idx"].tolist(), f"question {i}: segments differ"
        assert frm[i].tolist() == r["frm_idx"].tolist(), f"question {i}: frames differ"
        H.close(fsc[i], r["frm_score"], f"question {i} scores")
        hits += int(np.sum(sc_of[frm[i]] == scenes[i]))
    print(f"retrieval stress: {hits} of {nq * k_frm} retrieved frames lie in the question's scene")
    # gathered bytes: all 28 layers of three questions against an all-layer oracle of their frames
    kap = run.cfg.keep_per_frame
    dec_np = H.to_numpy_bits(dec[:3])
    meta_np = meta.cpu().numpy()
    for i in range(3):
        stq = H.oracle_stream(run.spec, H.oracle_cfg(run.cfg), frm[i].tolist(), last_only=False, workers=1)
        ref_dec, ref_meta = O.gather(stq, range(k_frm))
        assert dec_np[i].tobytes() == ref_dec.tobytes(), f"question {i}: gathered bytes differ"
        assert meta_np[i][:, 1].tolist() == ref_meta[:, 1].tolist()
        assert meta_np[i][:, 0].tolist() == np.repeat(frm[i], kap).tolist()
    # every other question: the decode buffer equals the pages it names (property at full size)
    pages = run.ctx.region(0)
    for i in range(3, nq, 7):
        for s, t in enumerate(frm[i]):
            got = dec[i][:, :, s * kap:(s + 1) * kap]
            assert bool((got.reshape(-1) == pages[int(t)].reshape(-1)).all())


def test_stream_3h_segment_level_selection(stream3h):
    # The same stream with segment-level selection (kappa_v = 16 * 49 over the 3,136 tokens of a segment), in
    # the launch configuration of the benchmark's variant: kept ids and per-frame counts of all 675 segments.
    # The indicators of a frame do not depend on the scope of the selection, so the oracle's frame-level run
    # above supplies them; Eq. 4 over the segment and the ranking are the oracle's functions.
    import torch
    run0, st = stream3h
    wl = dict(run0.wl)
    fseg, chunk = wl["fseg"], wl["chunk"]
    kv = wl["keep"] * fseg
    run = H.GpuRun(wl, keep_per_segment=kv, want_scores=False)
    c, T = run.cfg, run.n_frames
    P = c.tokens_per_frame
    kept = torch.full((T, P), -7, dtype=torch.int32, device=run.device)
    q, k, v = run.gs.alloc(chunk)
    for t0 in range(0, T, chunk):
        run.gs.fill(t0, chunk, q, k, v)
        run.ctx.mukv_compress_chunk(q, k, v, chunk, t0, kept[t0:t0 + chunk])
    torch.cuda.synchronize()
    kept = kept.cpu().numpy()
    cnt = run.ctx.region(10).cpu().numpy()
    ocfg = H.oracle_cfg(c)
    uneven = 0
    for u in range(T // fseg):
        frames = range(u * fseg, (u + 1) * fseg)
        ia = np.concatenate([st.scores[t][0] for t in frames])
        ifr = np.concatenate([st.scores[t][1] for t in frames])
        fused = O.fuse(ia, ifr, ocfg["alpha"], False)
        sel = O.select_tokens(fused, O.segment_keep_count(kv, fseg, fseg), ocfg["tie_eps"])
        assert len(sel) == kv
        for i, t in enumerate(frames):
            ref = sel[(sel >= i * P) & (sel < (i + 1) * P)] - i * P
            assert cnt[t] == len(ref), f"frame {t}: {cnt[t]} tokens kept, oracle {len(ref)}"
            assert kept[t, :len(ref)].tolist() == ref.tolist() and np.all(kept[t, len(ref):] == -1), f"frame {t}"
            uneven += int(len(ref) != wl["keep"])
    stats = run.ctx.mukv_get_stats()
    print(f"segment-level selection: {uneven} of {T} frames keep another number of tokens than 49; "
          f"{stats.refined_frames} frames went through the double-precision pass")
    assert uneven > T // 2 and stats.device_status == 0 and stats.kept_tokens == (T // fseg) * kv
    assert stats.refined_frames <= T // 25

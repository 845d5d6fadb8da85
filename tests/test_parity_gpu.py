"""CUDA path vs CPU oracle, through the C ABI, on the same seeded inputs.

Bar: kept-token / segment / frame indices and gathered bytes bit-exact; scores and pooled
entries within 1e-3 relative + 1e-5 absolute.
"""
import numpy as np
import pytest
import torch

from oracle import mukv_oracle as O
from paper_2605_22269_b200 import binding as B
from paper_2605_22269_b200.synth.cpu import StreamSpec, workload
from tests import harness as H

pytestmark = pytest.mark.gpu


def full_compress_check(run: H.GpuRun, chunk=None):
    """Whole (small) stream: every frame, every layer, segment entries, keys, timestamps."""
    run.compress(chunk)
    spec, cfg = run.spec, run.cfg
    T = run.n_frames
    st = H.oracle_stream(spec, H.oracle_cfg(cfg), range(T), last_only=False, workers=1)
    H.check_frames_against_oracle(run, st, range(T), full_layers=True)
    seg = run.ctx.region(3).cpu().numpy()
    fkey = run.ctx.region(4).cpu().numpy()
    skey = run.ctx.region(5).cpu().numpy()
    for t in range(T):
        assert fkey[t].tobytes() == st.frame_key(t).tobytes(), f"frame key {t} not bit-exact"
    assert st.n_segments == (T + cfg.frames_per_segment - 1) // cfg.frames_per_segment
    for u in range(st.n_segments):
        sk, sv = st.segment_entry(u)
        H.close(seg[u][:, 0], sk, f"segment entry K {u}")
        H.close(seg[u][:, 1], sv, f"segment entry V {u}")
        assert skey[u].tobytes() == st.segment_key(u).tobytes(), f"segment key {u} not bit-exact"
    ts = run.ctx.region(6).cpu().numpy()[:T]
    assert ts.tolist() == list(range(T))
    stats = run.ctx.mukv_get_stats()
    assert stats.frames == T and stats.segments == st.n_segments and stats.kept_tokens == T * cfg.keep_per_frame
    return st


def retrieval_check(run: H.GpuRun, st: O.Store, qtok, offs, k_seg, k_frm, lam, mode, t_limit=None, top_n=0):
    nq = len(offs) - 1
    ret = run.retrieve(qtok, offs, k_seg, k_frm, top_n, lam, mode, t_limit)
    dec, meta = run.gather(ret, k_frm)
    seg_idx, frm_idx = ret["seg_idx"].cpu().numpy(), ret["frm_idx"].cpu().numpy()
    seg_sc, frm_sc = ret["seg_score"].cpu().numpy(), ret["frm_score"].cpu().numpy()
    counts = ret["counts"].cpu().numpy()
    kap = run.cfg.keep_per_frame
    dec_np = H.to_numpy_bits(dec)
    meta_np = meta.cpu().numpy()
    for i in range(nq):
        r = O.retrieve(st, qtok[offs[i]:offs[i + 1]], k_seg, k_frm, top_n, lam, mode,
                       None if t_limit is None else int(t_limit[i]))
        ns, nf = len(r["seg_idx"]), len(r["frm_idx"])
        assert counts[i].tolist() == [ns, nf], f"question {i}: counts {counts[i]} vs {(ns, nf)}"
        assert seg_idx[i, :ns].tolist() == r["seg_idx"].tolist(), f"question {i}: segments differ"
        assert frm_idx[i, :nf].tolist() == r["frm_idx"].tolist(), f"question {i}: frames differ"
        assert np.all(seg_idx[i, ns:] == -1) and np.all(frm_idx[i, nf:] == -1)
        H.close(seg_sc[i, :ns], r["seg_score"], f"question {i} segment scores")
        H.close(frm_sc[i, :nf], r["frm_score"], f"question {i} frame scores")
        if st.cfg["n_layers"] == run.cfg.n_layers and nf > 0:
            ref_dec, ref_meta = O.gather(st, r["frm_idx"])
            assert dec_np[i][:, :, :nf * kap].tobytes() == ref_dec.tobytes(), f"question {i}: gathered bytes differ"
            assert meta_np[i, :nf * kap].tolist() == ref_meta.tolist()
    return ret


def questions(run, n_q=None, q_len=None):
    wl = run.wl
    n_q = n_q or wl["n_questions"]
    lo, hi = q_len or wl["q_len"]
    return run.spec.questions(n_q, lo, hi)


# ------------------------------------------------------------------------------- config 1
def test_tiny_fp32_full_parity():
    run = H.GpuRun("tiny")
    st = full_compress_check(run)
    qtok, offs, _ = questions(run)
    wl = run.wl
    for mode in (B.RETR_SEMI, B.RETR_PARALLEL, B.RETR_HIER):
        retrieval_check(run, st, qtok, offs, wl["k_seg"], wl["k_frm"], wl["lam"], mode)


def test_tiny_chunking_and_partial_segment():
    # 7 frames in chunks of 3 with segments of 4: segments straddle chunks, the last one is partial
    wl = dict(workload("tiny"))
    run = H.GpuRun(wl, n_frames=7)
    st = full_compress_check(run, chunk=3)
    qtok, offs, _ = run.spec.questions(3, 1, 9)
    retrieval_check(run, st, qtok, offs, 2, 3, 0.3, B.RETR_SEMI)
    retrieval_check(run, st, qtok, offs, 2, 3, 0.3, B.RETR_SEMI, t_limit=np.array([5, 4, 7]))
    retrieval_check(run, st, qtok, offs, 50, 50, 0.5, B.RETR_SEMI)          # k larger than what exists


@pytest.mark.parametrize("name,T,chunk", [("tiny", 7, 3), ("chunk7b", 6, 4)])
def test_segment_entries_owed_by_a_call_reach_every_reader(name, T, chunk):
    # A compress call leaves the segment entries of its chunk to whoever comes next.  Here: calls on a side
    # stream and a view of the store right behind the last call, with no synchronisation by the caller;
    # the same after a reset in the middle of a segment; and a retrieval as the first reader.
    wl = dict(workload(name))
    run = H.GpuRun(wl, n_frames=T)
    side = torch.cuda.Stream()

    def compress(frames):
        with torch.cuda.stream(side):
            for t0 in range(0, frames, chunk):
                n = min(chunk, frames - t0)
                q, k, v = run.gs.chunk(t0, n)
                run.ctx.mukv_compress_chunk(q, k, v, n, t0, stream=side)

    def check_segments(st):
        seg = run.ctx.region(3).cpu().numpy()                  # pools what is owed and waits for `side`
        key = run.ctx.region(5).cpu().numpy()
        for u in range(st.n_segments):
            sk, sv = st.segment_entry(u)
            H.close(seg[u][:, 0], sk, f"segment entry K {u}")
            H.close(seg[u][:, 1], sv, f"segment entry V {u}")
            assert key[u].tobytes() == st.segment_key(u).tobytes(), f"segment key {u}"

    compress(T)
    check_segments(H.oracle_stream(run.spec, H.oracle_cfg(run.cfg), range(T), last_only=False, workers=1))
    with torch.cuda.stream(side):
        run.ctx.mukv_reset(stream=side)
    compress(T - 1)                                            # what the dropped call owed must not come back
    st = H.oracle_stream(run.spec, H.oracle_cfg(run.cfg), range(T - 1), last_only=False, workers=1)
    torch.cuda.synchronize()
    qtok, offs, _ = run.spec.questions(3, 1, 9)
    retrieval_check(run, st, qtok, offs, 2, 3, 0.3, B.RETR_SEMI)   # the retrieval is the first reader
    check_segments(st)


@pytest.mark.parametrize("over", [dict(attn_causal=1), dict(keep_low_freq=1), dict(alpha=0.0), dict(alpha=1.0),
                                  dict(alpha=0.5), dict(keep_per_frame=1), dict(keep_per_frame=64)])
def test_tiny_variants(over):
    run = H.GpuRun("tiny", **over)
    full_compress_check(run)


def test_odd_shapes_bf16():
    # P not a multiple of 32 or 4, GQA with G = 3, D = 64, ragged chunks
    spec = StreamSpec(seed=11, n_layers=3, n_q_heads=6, n_kv_heads=2, head_dim=64, tokens_per_frame=77,
                      bf16=True, n_outlier=2, n_frames=11, scene_sigma=1.0, frame_sigma=0.5, scene_min=3, scene_max=5)
    wl = dict(spec=spec, keep=19, fseg=4, chunk=5, alpha=0.7, n_questions=4, q_len=(1, 7), k_seg=2, k_frm=3, lam=0.3)
    run = H.GpuRun(wl)
    st = full_compress_check(run)
    qtok, offs, _ = questions(run)
    for mode in (B.RETR_SEMI, B.RETR_PARALLEL, B.RETR_HIER):
        retrieval_check(run, st, qtok, offs, 2, 3, 0.3, mode)


def test_degenerate_inputs():
    # constant keys and zero queries: both signals flat, every score 0, lowest indices kept
    run = H.GpuRun("tiny")
    c = run.cfg
    P, L = c.tokens_per_frame, c.n_layers
    q = torch.zeros((2, P, c.n_q_heads, c.head_dim), device="cuda:0")
    k = torch.full((L, 2, P, c.n_kv_heads, c.head_dim), 0.5, device="cuda:0")
    v = torch.ones_like(k)
    kept = torch.zeros((2, c.keep_per_frame), dtype=torch.int32, device="cuda:0")
    run.ctx.mukv_compress_chunk(q, k, v, 2, 0, kept, None)
    torch.cuda.synchronize()
    assert kept.cpu().numpy().tolist() == [list(range(c.keep_per_frame))] * 2
    st = O.Store(H.oracle_cfg(c))
    O.compress_chunk(st, q.cpu().numpy(), k.cpu().numpy(), v.cpu().numpy())
    assert st.kept[0].tolist() == list(range(c.keep_per_frame))
    assert torch.all(run.ctx.region(2)[0, :, 0] == 0.5) and torch.all(run.ctx.region(2)[1, :, 1] == 1.0)


# ------------------------------------------------------------------------------- config 2
def test_chunk7b_full_parity():
    run = H.GpuRun("chunk7b")
    st = full_compress_check(run)
    worst = np.abs(run.scores[2] - np.stack([s[2] for s in st.scores])).max()
    print(f"chunk7b: max |fused score - oracle| = {worst:.3e}; refined frames = "
          f"{run.ctx.mukv_get_stats().refined_frames}")
    # what keeps the single-precision selection exact: the score error stays below half the safety margin
    assert worst < H.FLAG_MARGIN / 2
    qtok, offs, _ = questions(run)
    wl = run.wl
    retrieval_check(run, st, qtok, offs, wl["k_seg"], wl["k_frm"], wl["lam"], B.RETR_SEMI)


def test_chunk7b_causal():
    run = H.GpuRun("chunk7b", n_frames=4, attn_causal=1)
    full_compress_check(run)


@pytest.mark.parametrize("chunk", [1, 3])
def test_chunk7b_small_chunks(chunk):
    # a one-frame chunk spreads a frame over 52 scoring blocks (more partial sums than the selection
    # loads in one batch); three-frame chunks leave block shares that straddle frames
    run = H.GpuRun("chunk7b", n_frames=4)
    full_compress_check(run, chunk=chunk)
    assert run.ctx.mukv_get_stats().device_status == 0


def test_chunk7b_every_frame_through_the_double_pass():
    # a huge safety margin flags every frame: the double-precision pass has to walk a list longer than its grid
    run = H.GpuRun("chunk7b", n_frames=5, options={B.OPT_FLAG_MARGIN: 1.0})
    full_compress_check(run)
    assert run.ctx.mukv_get_stats().refined_frames == 5


@pytest.mark.parametrize("fseg,chunk,opts,over", [(4, 4, None, dict(patch_split=2, grid_width=14)),
                                                  (2, 2, None, dict()),
                                                  (16, 16, {B.OPT_FLAG_MARGIN: 1.0}, dict()),
                                                  (4, 4, {B.OPT_FLAG_MARGIN: 2e-4}, dict())])
def test_chunk_equal_to_a_segment(fseg, chunk, opts, over):
    # chunks that are exactly one segment, with and without a patch level; flagged frames (all of them,
    # or a few with the wider margin) leave the segment entries to the tail kernel
    wl = dict(workload("chunk7b"))
    wl["fseg"] = fseg
    run = H.GpuRun(wl, n_frames=16 if fseg > 2 else 6, options=opts, **over)
    full_compress_check(run, chunk=chunk)
    assert run.ctx.mukv_get_stats().device_status == 0


def test_chunk7b_cuda_core_scoring():
    # bf16 inputs scored by the plain multiply-add kernel (the one fp32 inputs always use)
    run = H.GpuRun("chunk7b", n_frames=3, options={B.OPT_SCORE_PATH: 1})
    full_compress_check(run)


def test_safety_margin_can_only_be_raised():
    run = H.GpuRun("tiny")
    with pytest.raises(B.MukvError) as e:
        run.ctx.mukv_set_option(B.OPT_FLAG_MARGIN, 0.0)
    assert e.value.status == -1
    with pytest.raises(B.MukvError):
        run.ctx.mukv_set_option(99, 1.0)


# The production path for bf16 chunks selects inside compact_kernel from the tensor-core kernel's
# partial sums, in single precision: every variant of Eq. 4 and of the top-kappa rule has to hold
# there too (paper: the low / high frequency ablation, the attention-only and frequency-only rows of
# the compression ablation, alpha per granularity).
@pytest.mark.parametrize("over", [dict(keep_low_freq=1), dict(alpha=0.0), dict(alpha=1.0), dict(alpha=0.5),
                                  dict(alpha=0.8), dict(keep_per_frame=1), dict(keep_per_frame=196),
                                  dict(keep_per_frame=19), dict(keep_low_freq=1, alpha=0.0, attn_causal=1)])
def test_chunk7b_variants_on_the_tensor_core_path(over):
    run = H.GpuRun("chunk7b", n_frames=5, **over)
    full_compress_check(run, chunk=3)
    st = run.ctx.mukv_get_stats()
    assert st.device_status == 0 and st.refined_frames <= 1


def _flat_chunk(run, n, q_val, k_mode):
    """A hand-made bf16 chunk: zero or constant queries; keys constant over tokens ("const"), or
    constant except for one token ("spike")."""
    c = run.cfg
    P, L = c.tokens_per_frame, c.n_layers
    dev = run.device
    q = torch.full((n, P, c.n_q_heads, c.head_dim), q_val, dtype=torch.bfloat16, device=dev)
    k = torch.full((L, n, P, c.n_kv_heads, c.head_dim), 0.5, dtype=torch.bfloat16, device=dev)
    if k_mode == "spike":
        k[:, :, 100] = 2.0
    v = torch.arange(P, dtype=torch.float32, device=dev).to(torch.bfloat16).view(1, 1, P, 1, 1).expand_as(k).contiguous()
    return q, k, v


@pytest.mark.parametrize("k_mode,alpha", [("const", 0.7), ("const", 0.0), ("const", 1.0), ("spike", 0.7),
                                          ("spike", 1.0)])
def test_flat_signals_on_the_tensor_core_path(k_mode, alpha):
    # zero queries and constant keys: both signals flat, every fused score equal (all of them land
    # in one histogram bin), the lowest ids are kept.  With one different key the frequency signal
    # has a single peak and the attention signal stays flat.
    run = H.GpuRun("chunk7b", n_frames=3, alpha=alpha)
    c = run.cfg
    q, k, v = _flat_chunk(run, 3, 0.0, k_mode)
    kept = torch.zeros((3, c.keep_per_frame), dtype=torch.int32, device=run.device)
    sc = torch.zeros((3, 3, c.tokens_per_frame), dtype=torch.float32, device=run.device)
    run.ctx.mukv_compress_chunk(q, k, v, 3, 0, kept, sc)
    torch.cuda.synchronize()
    st = O.Store(H.oracle_cfg(c))
    O.compress_chunk(st, H.to_numpy_bits(q), H.to_numpy_bits(k), H.to_numpy_bits(v))
    got = kept.cpu().numpy()
    for f in range(3):
        assert got[f].tolist() == st.kept[f].tolist(), f"kept ids differ at frame {f}"
        for i in range(3):
            H.close(sc[i, f].cpu().numpy(), st.scores[f][i], f"score[{i}] frame {f}")
    pages = H.to_numpy_bits(run.ctx.region(0)[:3])
    for f in range(3):
        assert pages[f][:, 0].tobytes() == st.page_k[f].tobytes() and pages[f][:, 1].tobytes() == st.page_v[f].tobytes()
    assert run.ctx.mukv_get_stats().device_status == 0


def test_non_finite_inputs_keep_the_lowest_ids():
    # one Inf key: every fused score of that frame is NaN; the frame keeps ids 0..kappa-1, the event
    # is recorded, the neighbouring frames are not disturbed
    run = H.GpuRun("chunk7b", n_frames=3)
    c = run.cfg
    q, k, v = run.gs.chunk(0, 3)
    k[c.n_layers - 1, 1, 5, 0, 3] = float("inf")
    kept = torch.zeros((3, c.keep_per_frame), dtype=torch.int32, device=run.device)
    run.ctx.mukv_compress_chunk(q, k, v, 3, 0, kept, None)
    torch.cuda.synchronize()
    st = O.Store(H.oracle_cfg(c))
    with np.errstate(all="ignore"):
        O.compress_chunk(st, H.to_numpy_bits(q), H.to_numpy_bits(k), H.to_numpy_bits(v))
    got = kept.cpu().numpy()
    assert got[1].tolist() == list(range(c.keep_per_frame)) == st.kept[1].tolist()
    assert got[0].tolist() == st.kept[0].tolist() and got[2].tolist() == st.kept[2].tolist()
    pages = H.to_numpy_bits(run.ctx.region(0)[:3])
    for f in range(3):
        assert pages[f][:, 0].tobytes() == st.page_k[f].tobytes()
    assert run.ctx.mukv_get_stats().device_status == 7
    run.ctx.mukv_reset()
    assert run.ctx.mukv_get_stats().device_status == 0 and run.ctx.mukv_get_stats().frames == 0


def test_two_contexts_of_different_shape():
    # kernel attributes belong to the kernel, not to a context: a second, smaller context must not
    # take shared memory away from the first one's launches (the double-precision pass included)
    big = H.GpuRun("chunk7b", n_frames=4, options={B.OPT_FLAG_MARGIN: 1.0})
    spec = StreamSpec(seed=31, n_layers=2, n_q_heads=8, n_kv_heads=4, head_dim=64, tokens_per_frame=130, bf16=True,
                      n_outlier=2, n_frames=3, scene_sigma=1.0, frame_sigma=0.5, scene_min=2, scene_max=3)
    small = H.GpuRun(dict(spec=spec, keep=33, fseg=2, chunk=3, alpha=0.7), options={B.OPT_FLAG_MARGIN: 1.0})
    full_compress_check(small)
    full_compress_check(big)
    assert big.ctx.mukv_get_stats().refined_frames == 4
    spec32 = StreamSpec(seed=32, n_layers=1, n_q_heads=2, n_kv_heads=2, head_dim=64, tokens_per_frame=40, bf16=False,
                        n_outlier=0, n_frames=2, scene_sigma=1.0, frame_sigma=0.5, scene_min=2, scene_max=3)
    tiny = H.GpuRun(dict(spec=spec32, keep=7, fseg=2, chunk=2, alpha=0.7))
    full_compress_check(tiny)
    full_compress_check(H.GpuRun("tiny"))


@pytest.mark.parametrize("shape", [dict(n_q_heads=8, n_kv_heads=8, head_dim=64, tokens_per_frame=130, keep=33),
                                   dict(n_q_heads=16, n_kv_heads=2, head_dim=128, tokens_per_frame=256, keep=64),
                                   dict(n_q_heads=12, n_kv_heads=4, head_dim=64, tokens_per_frame=16, keep=5)])
def test_tensor_core_tilings(shape):
    # G = 1, 8, 3; P below, at and above one 128-row tile; both head sizes
    keep = shape.pop("keep")
    spec = StreamSpec(seed=21, n_layers=2, bf16=True, n_outlier=2, n_frames=5, scene_sigma=1.0, frame_sigma=0.5,
                      scene_min=2, scene_max=3, **shape)
    wl = dict(spec=spec, keep=keep, fseg=2, chunk=3, alpha=0.7, n_questions=2, q_len=(2, 5), k_seg=1, k_frm=2,
              lam=0.3)
    run = H.GpuRun(wl)
    full_compress_check(run)
    assert run.ctx.mukv_get_stats().device_status == 0


# ------------------------------------------------------------------------------- config 3
def test_stream_1h():
    run = H.GpuRun("stream_1h").compress()
    spec, cfg = run.spec, run.cfg
    T = run.n_frames
    assert T == 1800 and run.ctx.mukv_get_stats().segments == 113
    # every frame: kept ids and scores (oracle on the last layer, which is all that scoring reads)
    st = H.oracle_stream(spec, H.oracle_cfg(cfg), range(T), last_only=True)
    worst = H.check_frames_against_oracle(run, st, range(T), full_layers=False)
    print(f"stream_1h: max |fused score - oracle| = {worst:.3e}; refined = {run.ctx.mukv_get_stats().refined_frames}")
    assert worst < H.FLAG_MARGIN / 2 and run.ctx.mukv_get_stats().refined_frames <= T // 200
    fkey = run.ctx.region(4).cpu().numpy()[:T]
    assert fkey.tobytes() == st.frame_keys().tobytes()
    skey = run.ctx.region(5).cpu().numpy()[:113]
    assert skey.tobytes() == st.segment_keys().tobytes()
    # sampled frames: all layers (pages, frame entries)
    sample = [0, 1, 15, 16, 799, 1234, 1792, 1799]
    st_full = H.oracle_stream(spec, H.oracle_cfg(cfg), sample, last_only=False, workers=1)
    for i, t in enumerate(sample):
        assert st_full.kept[i].tolist() == st.kept[t].tolist()
    H.check_frames_against_oracle(run, st_full, sample, full_layers=True)
    # the last segment is partial (8 frames)
    seg = run.ctx.region(3)[112].cpu().numpy()
    last = H.oracle_stream(spec, H.oracle_cfg(cfg), range(1792, 1800), last_only=False, workers=1)
    sk = np.sum(last.sum_k, axis=0) / (8.0 * cfg.keep_per_frame)
    H.close(seg[:, 0], sk.astype(np.float32), "partial segment entry")
    # retrieval
    qtok, offs, _ = questions(run)
    wl = run.wl
    ret = retrieval_check(run, st, qtok, offs, wl["k_seg"], wl["k_frm"], wl["lam"], B.RETR_SEMI)
    retrieval_check(run, st, qtok, offs, wl["k_seg"], wl["k_frm"], wl["lam"], B.RETR_SEMI,
                    t_limit=np.array([900, 1, 17, 1799, 1800, 16, 450, 1000]))
    # gathered bytes of the first question against an all-layer oracle of its frames
    frm = ret["frm_idx"].cpu().numpy()[0]
    stq = H.oracle_stream(spec, H.oracle_cfg(cfg), frm.tolist(), last_only=False, workers=1)
    ref_dec, ref_meta = O.gather(stq, range(len(frm)))
    dec, meta = run.gather(ret, wl["k_frm"])
    assert H.to_numpy_bits(dec)[0].tobytes() == ref_dec.tobytes()
    assert meta.cpu().numpy()[0][:, 1].tolist() == ref_meta[:, 1].tolist()
    assert meta.cpu().numpy()[0][:, 0].tolist() == np.repeat(frm, cfg.keep_per_frame).tolist()

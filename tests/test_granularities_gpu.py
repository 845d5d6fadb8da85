"""Retrieval over all three granularities (Sec. 3.4: patch-, frame- and segment-level blocks with
their own k_g and lambda_g) and the decode context built from them (summary tokens of the selected
segments, kept tokens of the selected frames and patch-level blocks), CUDA path against the oracle."""
import numpy as np
import pytest
import torch

from oracle import mukv_oracle as O
from paper_2605_22269_b200 import binding as B
from paper_2605_22269_b200.synth.cpu import StreamSpec, workload
from tests import harness as H

pytestmark = pytest.mark.gpu

MODES = {B.RETR_SEMI: O.MODE_SEMI, B.RETR_PARALLEL: O.MODE_PARALLEL, B.RETR_HIER: O.MODE_HIER}


def check_patch_level(run, st, T):
    S = st.n_patches()
    pk = run.ctx.region(8).cpu().numpy()
    pc = run.ctx.region(9).cpu().numpy()
    for t in range(T):
        for sp in range(S):
            assert pc[t, sp] == st.patch_count(t, sp), f"patch count frame {t} super patch {sp}"
            assert pk[t, sp].tobytes() == st.patch_key(t, sp).tobytes(), f"patch key frame {t} super patch {sp}"


def retrieve3_check(run, st, qtok, offs, k_g, lam_g, mode, t_limit=None, top_n=0, full_layers=True):
    """k_g, lam_g in the paper's order (patch, frame, segment)."""
    nq = len(offs) - 1
    dev = run.device
    k_pat, k_frm, k_seg = k_g
    prm = B.MukvRetrParams(k_pat, k_frm, k_seg, lam_g[0], lam_g[1], lam_g[2], top_n, mode)
    q_dev = H.to_device(qtok, run.spec.bf16, dev)
    seg = torch.full((nq, k_seg), -9, dtype=torch.int32, device=dev)
    frm = torch.full((nq, k_frm), -9, dtype=torch.int32, device=dev)
    pat = torch.full((nq, max(k_pat, 1)), -9, dtype=torch.int32, device=dev)
    ssc = torch.zeros((nq, k_seg), dtype=torch.float32, device=dev)
    fsc = torch.zeros((nq, k_frm), dtype=torch.float32, device=dev)
    psc = torch.zeros((nq, max(k_pat, 1)), dtype=torch.float32, device=dev)
    counts = torch.zeros((nq, 3), dtype=torch.int32, device=dev)
    run.ctx.mukv_retrieve3(q_dev, offs, t_limit, prm, seg, frm, pat, ssc, fsc, psc, counts)
    c = run.cfg
    cap = run.ctx.mukv_decode3_tokens(k_seg, k_frm, k_pat)
    es = 2 if run.spec.bf16 else 4
    row = run.ctx.C * es
    stride = c.n_layers * 2 * cap * row
    dec = torch.zeros((nq, stride), dtype=torch.uint8, device=dev)
    ntok = torch.full((nq,), -1, dtype=torch.int32, device=dev)
    meta = torch.full((nq, cap, 2), -5, dtype=torch.int32, device=dev)
    run.ctx.mukv_gather3(seg, frm, pat, counts, nq, k_seg, k_frm, k_pat, dec, stride, ntok, meta)
    torch.cuda.synchronize()
    seg_n, frm_n, pat_n, cnt = seg.cpu().numpy(), frm.cpu().numpy(), pat.cpu().numpy(), counts.cpu().numpy()
    dec_n = dec.cpu().numpy().reshape(nq, c.n_layers, 2, cap, row)
    meta_n, ntok_n = meta.cpu().numpy(), ntok.cpu().numpy()
    for i in range(nq):
        r = O.retrieve3(st, qtok[offs[i]:offs[i + 1]], k_g, lam_g, top_n, MODES[mode],
                        None if t_limit is None else int(t_limit[i]))
        ns, nf, npb = len(r["seg_idx"]), len(r["frm_idx"]), len(r["patch_idx"])
        assert cnt[i].tolist() == [ns, nf, npb], f"question {i}: counts {cnt[i]} vs {(ns, nf, npb)}"
        assert seg_n[i, :ns].tolist() == r["seg_idx"].tolist(), f"question {i}: segments differ"
        assert frm_n[i, :nf].tolist() == r["frm_idx"].tolist(), f"question {i}: frames differ"
        assert pat_n[i, :npb].tolist() == r["patch_idx"].tolist(), f"question {i}: patch blocks differ"
        assert np.all(seg_n[i, ns:] == -1) and np.all(frm_n[i, nf:] == -1)
        if k_pat:
            assert np.all(pat_n[i, npb:] == -1)
            H.close(psc.cpu().numpy()[i, :npb], r["patch_score"], f"question {i} patch scores")
        H.close(ssc.cpu().numpy()[i, :ns], r["seg_score"], f"question {i} segment scores")
        H.close(fsc.cpu().numpy()[i, :nf], r["frm_score"], f"question {i} frame scores")
        if not full_layers:
            continue
        ref, ref_meta = O.gather3(st, r["seg_idx"], r["frm_idx"], r["patch_idx"])
        n = ref_meta.shape[0]
        assert ntok_n[i] == n, f"question {i}: {ntok_n[i]} token slots, oracle {n}"
        assert meta_n[i, :n].tolist() == ref_meta.tolist(), f"question {i}: token meta differs"
        ref_b = ref.reshape(c.n_layers, 2, n, -1).view(np.uint8)
        # frame and patch tokens: bytes; summary tokens: the pooled entry in the storage type, one unit in
        # the last place allowed (the pooled means themselves agree to 1e-3)
        assert dec_n[i][:, :, ns:n].tobytes() == ref_b[:, :, ns:].tobytes(), f"question {i}: gathered bytes differ"
        if ns == 0:
            continue
        if run.spec.bf16:
            got = O.as_f64(dec_n[i][:, :, :ns].copy().view(np.uint16))
            want = O.as_f64(ref[:, :, :ns].reshape(c.n_layers, 2, ns, -1))
            err = np.abs(got - want) - (np.abs(want) * 2.0 ** -7 + 1e-5)
        else:
            got = dec_n[i][:, :, :ns].copy().view(np.float32).astype(np.float64)
            want = ref[:, :, :ns].reshape(c.n_layers, 2, ns, -1).astype(np.float64)
            err = np.abs(got - want) - (np.abs(want) * H.RTOL + H.ATOL)
        assert np.all(err <= 0), f"question {i}: summary tokens differ"


def test_three_granularities_bf16():
    # the 7B layout with the paper's S = 4 super patches on the 14 x 14 grid; segments of 4 frames
    wl = dict(workload("chunk7b"))
    wl["fseg"] = 4
    run = H.GpuRun(wl, n_frames=14, patch_split=2, grid_width=14).compress(chunk=5)
    st = H.oracle_stream(run.spec, H.oracle_cfg(run.cfg), range(14), last_only=False, workers=1)
    H.check_frames_against_oracle(run, st, range(14), full_layers=True)
    check_patch_level(run, st, 14)
    qtok, offs, _ = run.spec.questions(5, 3, 9)
    for mode in MODES:
        retrieve3_check(run, st, qtok, offs, (6, 4, 2), (0.3, 0.3, 0.0), mode)
    retrieve3_check(run, st, qtok, offs, (6, 4, 2), (0.5, 0.2, 0.4), B.RETR_SEMI, top_n=1)
    retrieve3_check(run, st, qtok, offs, (6, 4, 2), (0.3, 0.3, 0.0), B.RETR_SEMI, t_limit=np.array([9, 1, 14, 4, 5]))
    retrieve3_check(run, st, qtok, offs, (200, 30, 9), (0.3, 0.3, 0.0), B.RETR_SEMI)       # k beyond what exists
    retrieve3_check(run, st, qtok, offs, (0, 4, 2), (0.0, 0.3, 0.0), B.RETR_SEMI)          # no patch level asked for


def test_many_patch_rows_and_k_beyond_the_store():
    # one super patch per frame with 98 kept tokens: a question's patch-level rows (12 blocks x 98 rows) do not
    # fit the gather kernel's row list at once; k beyond what exists in the two modes that rank without rerank
    wl = dict(workload("chunk7b"))
    wl["fseg"] = 4
    run = H.GpuRun(wl, n_frames=12, keep_per_frame=98, patch_split=1, grid_width=14).compress(chunk=5)
    st = H.oracle_stream(run.spec, H.oracle_cfg(run.cfg), range(12), last_only=False, workers=1)
    H.check_frames_against_oracle(run, st, range(12), full_layers=True)
    check_patch_level(run, st, 12)
    qtok, offs, _ = run.spec.questions(3, 3, 9)
    retrieve3_check(run, st, qtok, offs, (12, 3, 2), (0.3, 0.3, 0.0), B.RETR_SEMI)
    for mode in (B.RETR_HIER, B.RETR_PARALLEL):
        retrieve3_check(run, st, qtok, offs, (200, 30, 9), (0.3, 0.3, 0.0), mode)


def test_three_granularities_fp32_every_frame_flagged():
    # small fp32 stream; the flagged frames' patch-level keys are written by the tail kernel
    spec = StreamSpec(seed=41, n_layers=2, n_q_heads=4, n_kv_heads=2, head_dim=64, tokens_per_frame=36, bf16=False,
                      n_outlier=1, n_frames=9, scene_sigma=1.0, frame_sigma=0.5, scene_min=2, scene_max=4)
    wl = dict(spec=spec, keep=13, fseg=3, chunk=4, alpha=0.7)
    for options in (None, {B.OPT_FLAG_MARGIN: 1.0}):
        run = H.GpuRun(wl, patch_split=4, grid_width=6, options=options).compress()
        st = H.oracle_stream(spec, H.oracle_cfg(run.cfg), range(9), last_only=False, workers=1)
        H.check_frames_against_oracle(run, st, range(9), full_layers=True)
        check_patch_level(run, st, 9)
        qtok, offs, _ = spec.questions(3, 2, 6)
        for mode in MODES:
            retrieve3_check(run, st, qtok, offs, (7, 3, 2), (0.3, 0.3, 0.0), mode)


def test_paper_k_and_lambda_on_the_one_hour_stream():
    # k_g = {20, 32, 12}, lambda_g = {0.3, 0.3, 0} (the paper's configuration) in all three modes at
    # the size of the one-hour stream; the oracle holds the last layer only (indices and scores)
    wl = dict(workload("stream_1h"))
    run = H.GpuRun(wl, patch_split=2, grid_width=14, want_scores=False).compress()
    st = H.oracle_stream(run.spec, H.oracle_cfg(run.cfg), range(run.n_frames), last_only=True)
    assert run.kept.tolist() == [k.tolist() for k in st.kept]
    check_patch_level(run, st, run.n_frames)
    qtok, offs, _ = run.spec.questions(wl["n_questions"], *wl["q_len"])
    for mode in MODES:
        retrieve3_check(run, st, qtok, offs, (20, 32, 12), (0.3, 0.3, 0.0), mode, full_layers=False)
    retrieve3_check(run, st, qtok, offs, (20, 32, 12), (0.3, 0.3, 0.0), B.RETR_SEMI, full_layers=False,
                    t_limit=np.array([900, 1, 17, 1799, 1800, 16, 450, 1000]))

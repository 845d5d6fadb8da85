"""Pins for the CPU oracle: library routines, closed forms, invariants and brute force.

Each test is chosen so that a plausible mistake in the oracle (a transposed operand, a
softmax over the wrong axis, a wrong head mapping, a dropped normalisation, an off-by-one in
the budget or the tie rule) makes it fail.
"""
import math
import os

import numpy as np
import pytest
import torch

from oracle import mukv_oracle as O

RNG = np.random.default_rng(1234)


def rand(*shape):
    return RNG.standard_normal(shape).astype(np.float32)


# --------------------------------------------------------------------------- Eq. 1
def test_attention_importance_matches_torch_softmax_gqa():
    P, Hq, Hkv, D = 13, 6, 2, 8
    Q, K = rand(P, Hq, D), rand(P, Hkv, D)
    got = O.attention_importance(Q, K)
    q = torch.from_numpy(Q).double().permute(1, 0, 2)                       # [Hq][P][D]
    k = torch.from_numpy(K).double().permute(1, 0, 2).repeat_interleave(Hq // Hkv, dim=0)
    A = torch.softmax(q @ k.transpose(1, 2) / math.sqrt(D), dim=-1)         # [Hq][i][j]
    ref = A.mean(dim=(0, 1)).numpy()
    np.testing.assert_allclose(got, ref, rtol=1e-12, atol=1e-15)


def test_attention_importance_python_loops():
    P, H, D = 5, 2, 4
    Q, K = rand(P, H, D), rand(P, H, D)
    ref = [0.0] * P
    for h in range(H):
        for i in range(P):
            z = [sum(float(Q[i, h, d]) * float(K[j, h, d]) for d in range(D)) / math.sqrt(D) for j in range(P)]
            m = max(z)
            e = [math.exp(v - m) for v in z]
            s = sum(e)
            for j in range(P):
                ref[j] += e[j] / s
    ref = [v / (H * P) for v in ref]
    np.testing.assert_allclose(O.attention_importance(Q, K), ref, rtol=1e-12)


@pytest.mark.parametrize("causal", [False, True])
def test_attention_importance_sums_to_one(causal):
    Q, K = rand(17, 4, 16), rand(17, 2, 16)
    assert abs(O.attention_importance(Q, K, causal).sum() - 1.0) < 1e-12


def test_attention_importance_zero_query_closed_forms():
    P = 11
    Q, K = np.zeros((P, 2, 8), np.float32), rand(P, 2, 8)
    np.testing.assert_allclose(O.attention_importance(Q, K), np.full(P, 1.0 / P), rtol=1e-13)
    # causal, uniform rows: row i spreads 1/(i+1) over keys 0..i
    ref = [sum(1.0 / (i + 1) for i in range(j, P)) / P for j in range(P)]
    np.testing.assert_allclose(O.attention_importance(Q, K, causal=True), ref, rtol=1e-13)


def test_attention_importance_dominant_column():
    P, D = 9, 4
    K = np.zeros((P, 1, D), np.float32)
    K[3, 0, 0] = 1.0
    Q = np.zeros((P, 1, D), np.float32)
    Q[:, 0, 0] = 200.0                       # every query attends to key 3 only
    I = O.attention_importance(Q, K)
    assert abs(I[3] - 1.0) < 1e-12 and np.abs(np.delete(I, 3)).max() < 1e-12


def test_attention_importance_causal_matches_torch_mask():
    P, H, D = 10, 2, 8
    Q, K = rand(P, H, D), rand(P, H, D)
    q = torch.from_numpy(Q).double().permute(1, 0, 2)
    k = torch.from_numpy(K).double().permute(1, 0, 2)
    z = q @ k.transpose(1, 2) / math.sqrt(D)
    z = z.masked_fill(~torch.tril(torch.ones(P, P, dtype=torch.bool)), float("-inf"))
    ref = torch.softmax(z, -1).mean(dim=(0, 1)).numpy()
    np.testing.assert_allclose(O.attention_importance(Q, K, causal=True), ref, rtol=1e-12)


# --------------------------------------------------------------------------- Eq. 2-3
def test_frequency_importance_matches_numpy_fft():
    K = rand(7, 3, 16)
    ref = np.abs(np.fft.fft(K.astype(np.float64), axis=-1)).mean(axis=(1, 2))
    np.testing.assert_allclose(O.frequency_importance(K), ref, rtol=1e-12)


def test_frequency_importance_closed_forms():
    D = 32
    K = np.zeros((4, 1, D), np.float32)
    K[0, 0, 5] = 1.0                                   # impulse: |Z| = 1 in every bin
    K[1, 0, :] = 0.75                                  # constant c: only bin 0, |Z0| = D*c
    K[2, 0, :] = 2.0 * np.cos(2 * np.pi * 3 * np.arange(D) / D)     # cosine: bins 3 and D-3, D*a/2 each
    I = O.frequency_importance(K)
    np.testing.assert_allclose(I[:3], [1.0, 0.75, 2.0], rtol=1e-6)
    assert I[3] == 0.0


def test_dft_parseval_and_symmetry():
    D = 64
    k = rand(D).astype(np.float64)
    Z = O.dft_matrix(D) @ k
    assert abs((np.abs(Z) ** 2).sum() - D * (k ** 2).sum()) < 1e-9
    np.testing.assert_allclose(np.abs(Z[1:]), np.abs(Z[1:][::-1]), rtol=1e-10)
    # sign of the exponent: a delayed impulse has phase -2*pi*b*d/D
    e = np.zeros(D)
    e[1] = 1.0
    np.testing.assert_allclose(O.dft_matrix(D) @ e, np.exp(-2j * np.pi * np.arange(D) / D), atol=1e-12)


def test_frequency_importance_is_per_token_not_per_sequence():
    # scaling one token scales only that token's score
    K = rand(6, 2, 16)
    a = O.frequency_importance(K)
    K2 = K.copy()
    K2[4] *= 3.0
    b = O.frequency_importance(K2)
    np.testing.assert_allclose(b[4], 3 * a[4], rtol=1e-6)
    np.testing.assert_allclose(np.delete(b, 4), np.delete(a, 4), rtol=1e-12)


# --------------------------------------------------------------------------- Eq. 4
def test_minmax_and_fuse():
    x = np.array([3.0, -1.0, 7.0, 2.0])
    n = O.minmax(x)
    assert n[1] == 0.0 and n[2] == 1.0 and np.all((n >= 0) & (n <= 1))
    np.testing.assert_allclose(O.minmax(5 * x + 11), n, rtol=1e-12)      # affine invariance
    assert np.all(O.minmax(np.full(5, 2.5)) == 0.0)
    a, f = np.array([0.1, 0.4, 0.2]), np.array([9.0, 3.0, 6.0])
    np.testing.assert_allclose(O.fuse(a, f, 1.0), O.minmax(a))
    np.testing.assert_allclose(O.fuse(a, f, 0.0), O.minmax(f))
    np.testing.assert_allclose(O.fuse(a, f, 0.7), 0.7 * O.minmax(a) + 0.3 * O.minmax(f))
    np.testing.assert_allclose(O.fuse(a, f, 0.0, keep_low_freq=True), 1.0 - O.minmax(f))


# --------------------------------------------------------------------------- top-k
def brute_topk(s, k, delta):
    """Definition written with plain loops."""
    n = len(s)
    if k >= n:
        return list(range(n))
    order = sorted(range(n), key=lambda i: (-s[i], i))
    tau = s[order[k - 1]]
    sure = [i for i in range(n) if s[i] > tau + delta]
    band = [i for i in range(n) if abs(s[i] - tau) <= delta]
    return sorted(sure + band[: k - len(sure)])


def test_topk_set_equals_stable_sort_without_band():
    for trial in range(200):
        n = int(RNG.integers(1, 12))
        s = RNG.integers(0, 4, size=n).astype(np.float64)          # many exact ties
        k = int(RNG.integers(1, n + 1))
        ref = sorted(sorted(range(n), key=lambda i: (-s[i], i))[:k])
        assert O.topk_set(s, k, 0.0).tolist() == ref


def test_topk_set_band_rule():
    s = np.array([0.5, 0.5 + 5e-7, 0.9, 0.1])
    assert O.topk_set(s, 2, 1e-6).tolist() == [0, 2]        # 0 and 1 tie within the band: lowest index
    assert O.topk_set(s, 2, 0.0).tolist() == [1, 2]
    assert O.topk_set(s, 2, 1e-7).tolist() == [1, 2]
    for trial in range(300):
        n = int(RNG.integers(2, 14))
        s = np.round(RNG.random(n), 1) + RNG.integers(-3, 4, size=n) * 4e-7
        k = int(RNG.integers(1, n))
        assert O.topk_set(s, k, 1e-6).tolist() == brute_topk(s.tolist(), k, 1e-6)


def test_topk_set_budget_and_shape():
    s = RNG.random(196)
    for k in (1, 19, 49, 98, 147, 196):
        idx = O.topk_set(s, k)
        assert idx.shape[0] == k and np.all(np.diff(idx) > 0) and idx.min() >= 0 and idx.max() < 196
    assert O.topk_set(s, 196).tolist() == list(range(196))
    assert O.topk_set(np.zeros(8), 3).tolist() == [0, 1, 2]


def test_select_tokens_non_finite_rule():
    # finite scores: the top-kappa rule; any Inf or NaN: no ranking, the first kappa tokens
    rng = np.random.default_rng(8)
    s = rng.random(40)
    assert O.select_tokens(s, 7).tolist() == O.topk_set(s, 7).tolist()
    for bad in (np.nan, np.inf, -np.inf):
        t = s.copy()
        t[33] = bad
        assert O.select_tokens(t, 7).tolist() == list(range(7))
    # through the whole frame path: one infinite key makes the frame's scores NaN
    Q = rng.standard_normal((1, 12, 2, 8)).astype(np.float32)
    K = rng.standard_normal((1, 1, 12, 2, 8)).astype(np.float32)
    K[0, 0, 4, 1, 2] = np.inf
    st = O.Store(dict(n_layers=1, n_q_heads=2, n_kv_heads=2, head_dim=8, tokens_per_frame=12, keep_per_frame=5,
                      frames_per_segment=2, alpha=0.7))
    with np.errstate(all="ignore"):
        O.compress_chunk(st, Q, K, K)
    assert st.kept[0].tolist() == [0, 1, 2, 3, 4]
    assert not np.all(np.isfinite(st.scores[0][2]))


def test_budget_matches_paper_token_counts():
    path = os.path.join(os.path.dirname(__file__), "golden", "paper_token_counts.txt")
    rows = [l.split() for l in open(path) if l.strip() and not l.startswith("#")]
    assert len(rows) == 5
    for P, drop, blocks, frames, inf_k, mem_k in rows:
        kappa = O.keep_count(1.0 - float(drop), int(P))
        # printed values are rounded (and the ratios are applied without the floor in places)
        assert abs(int(blocks) * kappa / 1000.0 - float(inf_k)) <= 0.1
        assert abs(int(frames) * kappa / 1000.0 - float(mem_k)) <= 1.0
    assert O.keep_count(0.25, 196) == 49 and O.keep_count(0.25, 64) == 16 and O.keep_count(0.1, 196) == 19


# --------------------------------------------------------------------------- compaction, pooling
CFG = dict(n_layers=3, n_q_heads=4, n_kv_heads=2, head_dim=8, tokens_per_frame=12, keep_per_frame=5,
           frames_per_segment=2, alpha=0.7)


def make_store(n_frames=5, cfg=CFG, chunk=2):
    st = O.Store(cfg)
    L, Hq, Hkv, D, P = (cfg[k] for k in ("n_layers", "n_q_heads", "n_kv_heads", "head_dim", "tokens_per_frame"))
    Q, K, V = rand(n_frames, P, Hq, D), rand(L, n_frames, P, Hkv, D), rand(L, n_frames, P, Hkv, D)
    for t0 in range(0, n_frames, chunk):
        O.compress_chunk(st, Q[t0:t0 + chunk], K[:, t0:t0 + chunk], V[:, t0:t0 + chunk])
    return st, Q, K, V


def test_compress_keeps_budget_and_copies_bytes():
    st, Q, K, V = make_store()
    assert st.n_frames == 5 and st.n_segments == 3
    for t in range(5):
        kept = st.kept[t]
        assert kept.shape[0] == CFG["keep_per_frame"] and np.all(np.diff(kept) > 0)
        # the kept tokens are the best under the fused score of that frame
        I = O.fuse(O.attention_importance(Q[t], K[-1, t]), O.frequency_importance(K[-1, t]), CFG["alpha"])
        assert set(kept.tolist()) == set(np.argsort(-I, kind="stable")[: CFG["keep_per_frame"]].tolist())
        for l in range(CFG["n_layers"]):
            for r, j in enumerate(kept):
                assert st.page_k[t][l, r].tobytes() == K[l, t, j].tobytes()
                assert st.page_v[t][l, r].tobytes() == V[l, t, j].tobytes()


def test_random_drop_fixture():
    # the "Rand(50%)" row of the compression ablation: selection by caller-given random scores
    cfg = dict(CFG, keep_per_frame=O.keep_count(0.5, CFG["tokens_per_frame"]))
    L, Hkv, D, P = cfg["n_layers"], cfg["n_kv_heads"], cfg["head_dim"], cfg["tokens_per_frame"]
    K, V = rand(L, 4, P, Hkv, D), rand(L, 4, P, Hkv, D)
    r = np.random.default_rng(3).random((4, P)).astype(np.float32)
    st = O.Store(cfg)
    O.compress_chunk(st, None, K, V, select_scores=r)
    for t in range(4):
        want = np.sort(np.argsort(-r[t].astype(np.float64), kind="stable")[:P // 2])
        assert st.kept[t].tolist() == want.tolist() and len(want) == P // 2
        assert st.page_k[t].tobytes() == K[:, t][:, want].tobytes()
    # half of the memory tokens, as the table prints: 59K -> 29K
    assert abs(300 * O.keep_count(0.5, 196) / 1000.0 - 29) <= 1.0


def test_chunking_does_not_change_the_store():
    a, Q, K, V = make_store(5, chunk=2)
    b = O.Store(CFG)
    O.compress_chunk(b, Q, K, V)
    for t in range(5):
        assert a.kept[t].tolist() == b.kept[t].tolist()
        np.testing.assert_array_equal(a.frame_entry(t)[0], b.frame_entry(t)[0])


def test_pooling_invariants():
    cfg = dict(CFG, keep_per_frame=CFG["tokens_per_frame"])            # kappa = P: plain mean
    st, Q, K, V = make_store(4, cfg)
    for t in range(4):
        ek, ev = st.frame_entry(t)
        np.testing.assert_allclose(ek, K[:, t].astype(np.float64).mean(axis=1).reshape(3, 16), rtol=1e-6, atol=1e-7)
        np.testing.assert_allclose(ev, V[:, t].astype(np.float64).mean(axis=1).reshape(3, 16), rtol=1e-6, atol=1e-7)
        np.testing.assert_array_equal(st.frame_key(t), ek[-1])
    # segment entry = mean of its frames' entries when kappa is uniform
    for u in range(2):
        sk, sv = st.segment_entry(u)
        fr = [st.frame_entry(t) for t in (2 * u, 2 * u + 1)]
        np.testing.assert_allclose(sk, (fr[0][0].astype(np.float64) + fr[1][0]) / 2, rtol=1e-6, atol=1e-7)
        np.testing.assert_allclose(sv, (fr[0][1].astype(np.float64) + fr[1][1]) / 2, rtol=1e-6, atol=1e-7)
    # constant input pools to itself; partial last segment pools over the frames present
    c = O.Store(CFG)
    L, Hq, Hkv, D, P = 3, 4, 2, 8, 12
    Kc = np.full((L, 3, P, Hkv, D), 0.625, np.float32)
    O.compress_chunk(c, rand(3, P, Hq, D), Kc, 2 * Kc)
    assert c.n_segments == 2
    assert np.all(c.frame_entry(1)[0] == np.float32(0.625)) and np.all(c.frame_entry(1)[1] == np.float32(1.25))
    assert np.all(c.segment_entry(1)[0] == np.float32(0.625))
    # constant keys: both signals are flat, every score is 0, the lowest indices are kept
    assert c.kept[0].tolist() != [] and O.topk_set(np.zeros(P), 5).tolist() == [0, 1, 2, 3, 4]


def test_bf16_inputs_are_decoded_exactly():
    x = rand(4, 2, 8)
    bits = (x.view(np.uint32) >> 16).astype(np.uint16)             # truncate to bf16
    exact = (bits.astype(np.uint32) << 16).view(np.float32)
    np.testing.assert_array_equal(O.as_f64(bits), exact.astype(np.float64))
    np.testing.assert_allclose(O.frequency_importance(bits), O.frequency_importance(exact), rtol=0)


# --------------------------------------------------------------------------- Eq. 6-8
def test_pool_question():
    Qq = rand(5, 6, 4)
    q = O.pool_question(Qq, 2)                                       # G = 3
    ref = np.zeros(8)
    for n in range(5):
        for h in range(6):
            for d in range(4):
                ref[(h // 3) * 4 + d] += float(Qq[n, h, d]) / (5 * 3)
    np.testing.assert_allclose(q, ref, rtol=1e-12)
    one = rand(1, 2, 4)
    np.testing.assert_allclose(O.pool_question(one, 2), one.reshape(8).astype(np.float64))


def test_cosine_matches_torch_and_bounds():
    q, keys = rand(16).astype(np.float64), rand(9, 16).astype(np.float64)
    ref = torch.nn.functional.cosine_similarity(torch.from_numpy(keys), torch.from_numpy(q)[None, :], dim=1).numpy()
    got = O.cosine(q, keys)
    np.testing.assert_allclose(got, ref, rtol=1e-12)
    assert np.all(np.abs(got) <= 1 + 1e-12)
    np.testing.assert_allclose(O.cosine(3.0 * q, 0.5 * keys), got, rtol=1e-12)      # scale invariance
    assert abs(O.cosine(q, 2.5 * q[None, :])[0] - 1.0) < 1e-12
    assert O.cosine(q, np.zeros((1, 16)))[0] == 0.0


def manual_store(frame_keys, fseg, n_kv_heads=1):
    """A store whose retrieval keys are given directly (one layer, kappa = 1)."""
    frame_keys = np.asarray(frame_keys, dtype=np.float64)
    T, C = frame_keys.shape
    st = O.Store(dict(n_layers=1, n_q_heads=n_kv_heads, n_kv_heads=n_kv_heads, head_dim=C // n_kv_heads,
                      tokens_per_frame=1, keep_per_frame=1, frames_per_segment=fseg, alpha=0.7))
    for t in range(T):
        st.kept.append(np.array([0]))
        st.sum_k.append(frame_keys[t][None, :].copy())
        st.sum_v.append(frame_keys[t][None, :].copy())
        st.page_k.append(frame_keys[t].astype(np.float32).reshape(1, 1, n_kv_heads, -1))
        st.page_v.append(frame_keys[t].astype(np.float32).reshape(1, 1, n_kv_heads, -1))
    return st


def unit(deg):
    return [math.cos(math.radians(deg)), math.sin(math.radians(deg))]


def test_retrieve_rerank_changes_the_choice():
    # 2-d keys on the unit circle.  Segment 0 = frames at 10 and 55 deg, segment 1 = frames at
    # -12 and -120 deg.  A question at 0 deg ranks frame 0 first in stage 1.
    keys = np.array([unit(10), unit(55), unit(-12), unit(-120)])
    st = manual_store(keys, fseg=2)
    Qq = np.array(unit(0), dtype=np.float32).reshape(1, 1, 2)
    par = O.retrieve(st, Qq, k_seg=1, k_frm=1, mode=O.MODE_PARALLEL)
    assert par["frm_idx"].tolist() == [0] and par["seg_idx"].tolist() == [0]
    np.testing.assert_allclose(par["s_frm"], [math.cos(math.radians(a)) for a in (10, 55, 12, 120)], rtol=1e-6)
    # candidates (top-2): frames 0 (10 deg) and 2 (-12 deg).  Global query = mean of unit(10), unit(55)
    # -> direction 32.5 deg.  gamma_0 = cos(22.5), gamma_2 = cos(44.5).
    lam = 0.3
    semi = O.retrieve(st, Qq, k_seg=1, k_frm=1, lam=lam, mode=O.MODE_SEMI)
    s0 = (1 - lam) * math.cos(math.radians(10)) + lam * math.cos(math.radians(22.5))
    assert semi["frm_idx"].tolist() == [0]
    np.testing.assert_allclose(semi["frm_score"], [s0], rtol=1e-6)
    # a question at -2 deg prefers frame 2 (-12 deg, 10 away) over frame 0 (12 away) in stage 1,
    # but the rerank pulls frame 0 (inside the best segment) back on top
    Qq2 = np.array(unit(-2), dtype=np.float32).reshape(1, 1, 2)
    assert O.retrieve(st, Qq2, 1, 1, mode=O.MODE_PARALLEL)["frm_idx"].tolist() == [2]
    r = O.retrieve(st, Qq2, 1, 1, lam=0.3, mode=O.MODE_SEMI)
    assert r["seg_idx"].tolist() == [0] and r["frm_idx"].tolist() == [0]
    s_new = 0.7 * math.cos(math.radians(12)) + 0.3 * math.cos(math.radians(22.5))
    np.testing.assert_allclose(r["frm_score"], [s_new], rtol=1e-6)
    # hierarchical mode only looks inside the selected segment
    assert O.retrieve(st, Qq2, 1, 1, mode=O.MODE_HIER)["frm_idx"].tolist() == [0]


def test_retrieve_invariants():
    st, Q, K, V = make_store(9, dict(CFG, frames_per_segment=3), chunk=4)
    Qq = rand(6, 4, 8)
    par = O.retrieve(st, Qq, 2, 3, mode=O.MODE_PARALLEL)
    semi0 = O.retrieve(st, Qq, 2, 3, lam=0.0, mode=O.MODE_SEMI)
    assert par["frm_idx"].tolist() == semi0["frm_idx"].tolist()          # lambda = 0: stage 2 changes nothing
    np.testing.assert_allclose(par["frm_score"], semi0["frm_score"])
    big = O.retrieve(st, Qq, 50, 50, mode=O.MODE_SEMI)
    assert big["frm_idx"].tolist() == list(range(9)) and big["seg_idx"].tolist() == [0, 1, 2]
    hier = O.retrieve(st, Qq, 1, 2, mode=O.MODE_HIER)
    assert all(t // 3 == hier["seg_idx"][0] for t in hier["frm_idx"])
    # scores are the cosines of the pooled question with the stored keys
    q = O.pool_question(Qq, 2)
    ref = torch.nn.functional.cosine_similarity(torch.from_numpy(st.frame_keys().astype(np.float64)),
                                                torch.from_numpy(q)[None, :], dim=1).numpy()
    np.testing.assert_allclose(par["s_frm"], ref, rtol=1e-12)
    # visibility: t_limit hides later frames and segments that are not complete before it
    lim = O.retrieve(st, Qq, 50, 50, t_limit=5, mode=O.MODE_SEMI)
    assert lim["frm_idx"].tolist() == [0, 1, 2, 3, 4] and lim["seg_idx"].tolist() == [0]
    # self query: a question equal to a frame key scores 1 there and wins
    key = st.frame_key(4).astype(np.float32).reshape(1, 2, 8)
    self_q = np.repeat(key, 2, axis=1)                                     # both query heads of a group
    r = O.retrieve(st, self_q, 1, 1, mode=O.MODE_PARALLEL)
    assert r["frm_idx"].tolist() == [4] and abs(r["frm_score"][0] - 1.0) < 1e-12


def test_semi_gamma_is_one_for_single_frame_segments():
    keys = RNG.standard_normal((4, 6))
    st = manual_store(keys, fseg=1)
    Qq = keys[2].astype(np.float32).reshape(1, 1, 6)
    r = O.retrieve(st, Qq, k_seg=1, k_frm=1, top_n=1, lam=0.5, mode=O.MODE_SEMI)
    assert r["frm_idx"].tolist() == [2]
    np.testing.assert_allclose(r["frm_score"], [1.0], rtol=1e-6)            # 0.5 * 1 + 0.5 * 1


# --------------------------------------------------------------------------- Eq. 9
def test_gather_layout_and_token_count():
    st, Q, K, V = make_store(6)
    sel = [1, 4, 5]
    dec, meta = O.gather(st, sel)
    kap = CFG["keep_per_frame"]
    assert dec.shape == (3, 2, len(sel) * kap, 2, 8) and meta.shape == (len(sel) * kap, 2)
    for l in range(3):
        for s, t in enumerate(sel):
            for r, j in enumerate(st.kept[t]):
                assert dec[l, 0, s * kap + r].tobytes() == K[l, t, j].tobytes()
                assert dec[l, 1, s * kap + r].tobytes() == V[l, t, j].tobytes()
                assert meta[s * kap + r].tolist() == [t, int(j)]
    # the retrieved context has (blocks x kappa) tokens: 64 x 49 = 3,136 and 64 x 196 = 12,544
    assert 64 * O.keep_count(0.25, 196) == 3136 and 64 * O.keep_count(1.0, 196) == 12544


# --------------------------------------------------------------------------- three granularities
CFG3 = dict(n_layers=2, n_q_heads=4, n_kv_heads=2, head_dim=8, tokens_per_frame=36, keep_per_frame=13,
            frames_per_segment=3, alpha=0.7, patch_split=2, grid_width=6)


def test_context_tokens_match_the_paper():
    path = os.path.join(os.path.dirname(__file__), "golden", "paper_context_tokens.txt")
    rows = [l.split() for l in open(path) if l.strip() and not l.startswith("#")]
    blocks = [(int(k), float(rho), int(n)) for name, k, rho, n in rows[:3]]
    printed = float(rows[3][1])
    with_floor = sum(k * O.keep_count(rho, n) for k, rho, n in blocks)
    assert with_floor == 20 * 4 + 32 * 19 + 12 * 627
    assert abs(with_floor / 1000.0 - printed) <= 0.1
    assert abs(sum(k * rho * n for k, rho, n in blocks) / 1000.0 - printed) <= 0.05


def test_super_patch_of_is_the_quadrant():
    # 14 x 14 grid, 2 x 2 super patches of 7 x 7 = 49 tokens (the paper's S = 4, P = 196)
    ids = np.arange(196)
    sp = O.super_patch_of(ids, 196, 14, 2)
    for j in ids:
        assert sp[j] == (0 if j // 14 < 7 else 2) + (0 if j % 14 < 7 else 1)
    assert np.bincount(sp).tolist() == [49, 49, 49, 49]
    # a grid that does not divide evenly: 6 x 6 cut in 4 x 4 -> rectangles of 2 x 2, only 3 x 3 of them occupied
    sp = O.super_patch_of(np.arange(36), 36, 6, 4)
    assert sorted(set(sp.tolist())) == [0, 1, 2, 4, 5, 6, 8, 9, 10]


def test_patch_blocks_partition_the_frame():
    st, Q, K, V = make_store(5, CFG3)
    S = st.n_patches()
    assert S == 4
    for t in range(5):
        pos = np.concatenate([st.patch_tokens(t, sp) for sp in range(S)])
        assert sorted(pos.tolist()) == list(range(CFG3["keep_per_frame"]))
        # the count-weighted mean of the patch-level keys is the frame-level key (Eq. 5 both ways)
        w = np.array([st.patch_count(t, sp) for sp in range(S)], dtype=np.float64)
        keys = np.stack([st.patch_key(t, sp) for sp in range(S)]).astype(np.float64)
        np.testing.assert_allclose((w[:, None] * keys).sum(0) / w.sum(), st.frame_key(t), rtol=1e-5, atol=1e-6)
        for sp in range(S):
            toks = st.kept[t][st.patch_tokens(t, sp)]
            want = K[-1, t, toks].astype(np.float64).reshape(len(toks), -1).mean(0) if len(toks) else np.zeros(16)
            np.testing.assert_allclose(st.patch_key(t, sp), want, rtol=1e-6, atol=1e-7)


def test_retrieve3_reduces_to_retrieve_and_to_brute_force():
    st, Q, K, V = make_store(11, CFG3, chunk=4)
    S = st.n_patches()
    Qq = rand(5, 4, 8)
    for mode in (O.MODE_SEMI, O.MODE_PARALLEL, O.MODE_HIER):
        for tl in (None, 7):
            a = O.retrieve(st, Qq, 2, 3, 0, 0.3, mode, tl)
            b = O.retrieve3(st, Qq, (4, 3, 2), (0.3, 0.3, 0.0), 0, mode, tl)
            assert a["seg_idx"].tolist() == b["seg_idx"].tolist() and a["frm_idx"].tolist() == b["frm_idx"].tolist()
            np.testing.assert_allclose(a["frm_score"], b["frm_score"], rtol=1e-12)
    # patch level, stage 1 only: the k best existing blocks by cosine, by a plain sort
    r = O.retrieve3(st, Qq, (5, 3, 2), (0.0, 0.0, 0.0), 0, O.MODE_PARALLEL)
    q = O.pool_question(Qq, 2)
    sc = []
    for t in range(11):
        for sp in range(S):
            if st.patch_count(t, sp):
                k = st.patch_key(t, sp).astype(np.float64)
                sc.append((-(k @ q) / (np.linalg.norm(k) * np.linalg.norm(q)), t * S + sp))
    want = sorted(b for _, b in sorted(sc)[:5])
    assert r["patch_idx"].tolist() == want
    # lambda = 0 makes the semi-hierarchical result equal the parallel one at every granularity
    z = O.retrieve3(st, Qq, (5, 3, 2), (0.0, 0.0, 0.0), 0, O.MODE_SEMI)
    assert z["patch_idx"].tolist() == want and z["frm_idx"].tolist() == r["frm_idx"].tolist()
    # HIER: every frame and patch block lies inside a selected segment
    h = O.retrieve3(st, Qq, (6, 4, 2), (0.3, 0.3, 0.0), 0, O.MODE_HIER)
    inside = set(h["seg_idx"].tolist())
    assert all(t // 3 in inside for t in h["frm_idx"]) and all((b // S) // 3 in inside for b in h["patch_idx"])
    # a segment-level lambda > 0 picks among the 2k stage-1 candidates
    s2 = O.retrieve3(st, Qq, (1, 1, 2), (0.3, 0.3, 0.5), 1, O.MODE_SEMI)
    cand = O.topk_set(O.cosine(q, st.segment_keys().astype(np.float64)), 4)
    assert set(s2["seg_idx"].tolist()) <= set(cand.tolist()) and len(s2["seg_idx"]) == 2


def test_gather3_layout():
    import torch
    st, Q, K, V = make_store(7, CFG3, chunk=3)
    S = st.n_patches()
    seg, frm, pat = [0, 2], [1, 5], [2 * S + 1, 6 * S + 3]
    dec, meta = O.gather3(st, seg, frm, pat)
    kap = CFG3["keep_per_frame"]
    n_pat = sum(st.patch_count(b // S, b % S) for b in pat)
    assert dec.shape[2] == len(seg) + len(frm) * kap + n_pat == meta.shape[0]
    # summary tokens: the segment entry in the storage type (float32 here: unchanged)
    for i, u in enumerate(seg):
        ek, ev = st.segment_entry(u)
        assert dec[:, 0, i].reshape(2, -1).tobytes() == ek.tobytes() and dec[:, 1, i].reshape(2, -1).tobytes() == ev.tobytes()
        assert meta[i].tolist() == [-1 - u, -1]
    ref, ref_meta = O.gather(st, frm)
    assert dec[:, :, len(seg):len(seg) + len(frm) * kap].tobytes() == ref.tobytes()
    row = len(seg) + len(frm) * kap
    for b in pat:
        t, sp = b // S, b % S
        for j in st.kept[t]:
            if O.super_patch_of([j], 36, 6, 2)[0] == sp:
                assert dec[1, 0, row].tobytes() == K[1, t, j].tobytes() and meta[row].tolist() == [t, int(j)]
                row += 1
    assert row == dec.shape[2]
    # rounding to bfloat16 storage equals the library's round-to-nearest-even conversion
    x = RNG.standard_normal(1000).astype(np.float32)
    got = O.round_to_dtype(x, np.zeros(1, dtype=np.uint16))
    want = torch.from_numpy(x).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert got.tobytes() == want.tobytes()


# --------------------------------------------------------------------------- layer choice
def test_scoring_layers():
    # which layers: last (default), penultimate, middle, last-5 fusion of a 28-layer model
    assert list(O.score_layers(dict(n_layers=28))) == [27]
    assert list(O.score_layers(dict(n_layers=28, n_score_layers=1, score_layer_offset=1))) == [26]
    assert list(O.score_layers(dict(n_layers=28, n_score_layers=1, score_layer_offset=14))) == [13]
    assert list(O.score_layers(dict(n_layers=28, n_score_layers=5))) == [23, 24, 25, 26, 27]
    # fusion = mean of the per-layer indicators; one layer given as a stack of one equals the plain call
    Q, K = rand(3, 10, 4, 8), rand(3, 10, 2, 8)
    ia, ifr, I = O.score_frame(Q, K, 0.7)
    np.testing.assert_allclose(ia, np.mean([O.attention_importance(Q[l], K[l]) for l in range(3)], axis=0), rtol=1e-14)
    np.testing.assert_allclose(ifr, np.mean([O.frequency_importance(K[l]) for l in range(3)], axis=0), rtol=1e-14)
    assert abs(ia.sum() - 1.0) < 1e-12
    a1 = O.score_frame(Q[:1], K[:1], 0.7)
    a0 = O.score_frame(Q[0], K[0], 0.7)
    for x, y in zip(a1, a0):
        np.testing.assert_allclose(x, y, rtol=1e-14)
    # through compress_chunk: a penultimate-layer configuration ranks by that layer's keys and queries
    cfg = dict(CFG, n_score_layers=1, score_layer_offset=1)
    st = O.Store(cfg)
    L, Hq, Hkv, D, P = 3, 4, 2, 8, 12
    Qc, Kc, Vc = rand(2, P, Hq, D), rand(L, 2, P, Hkv, D), rand(L, 2, P, Hkv, D)
    O.compress_chunk(st, Qc, Kc, Vc)
    for f in range(2):
        want = O.topk_set(O.score_frame(Qc[f], Kc[1, f], 0.7)[2], 5)
        assert st.kept[f].tolist() == want.tolist()


# --------------------------------------------------------------------------- segment-level DCP
def test_segment_scope_selection():
    fs, P = 3, 12
    cfg = dict(CFG, frames_per_segment=fs, keep_per_segment=O.keep_count(0.8, fs * P))
    kv = cfg["keep_per_segment"]
    assert kv == 28                                                     # floor(0.8 * 36)
    L, Hq, Hkv, D = 3, 4, 2, 8
    n = 8                                                               # two whole segments and one of two frames
    Q, K, V = rand(n, P, Hq, D), rand(L, n, P, Hkv, D), rand(L, n, P, Hkv, D)
    st = O.Store(cfg)
    O.compress_chunk(st, Q[:6], K[:, :6], V[:, :6])
    O.compress_chunk(st, Q[6:], K[:, 6:], V[:, 6:])
    counts = [len(k) for k in st.kept]
    assert sum(counts[0:3]) == kv and sum(counts[3:6]) == kv and sum(counts[6:8]) == (kv * 2) // 3
    assert len(set(counts)) > 1                                         # the frames really keep different numbers
    # by hand for the first segment: min-max over all O tokens, then the kappa_v best
    ia = np.concatenate([O.attention_importance(Q[f], K[-1, f]) for f in range(3)])
    ifr = np.concatenate([O.frequency_importance(K[-1, f]) for f in range(3)])
    I = 0.7 * (ia - ia.min()) / (ia.max() - ia.min()) + 0.3 * (ifr - ifr.min()) / (ifr.max() - ifr.min())
    want = np.sort(np.argsort(-I, kind="stable")[:kv])
    got = np.concatenate([st.kept[f] + f * P for f in range(3)])
    assert got.tolist() == want.tolist()
    for f in range(3):
        assert st.page_k[f].tobytes() == K[:, f][:, st.kept[f]].tobytes()
    # the segment entry is the mean over all kept tokens of the segment
    rows = np.concatenate([K[-1, f][st.kept[f]].astype(np.float64).reshape(len(st.kept[f]), -1) for f in range(3)])
    np.testing.assert_allclose(st.segment_key(0), rows.mean(0), rtol=1e-6, atol=1e-7)
    # rho = 1 keeps everything; identical frames keep the same token ids in each
    st1 = O.Store(dict(cfg, keep_per_segment=fs * P))
    O.compress_chunk(st1, Q[:3], K[:, :3], V[:, :3])
    assert all(k.tolist() == list(range(P)) for k in st1.kept)
    Qs, Ks = np.repeat(Q[:1], 3, axis=0), np.repeat(K[:, :1], 3, axis=1)
    st2 = O.Store(dict(cfg, keep_per_segment=3 * 4))
    O.compress_chunk(st2, Qs, Ks, Ks)
    assert st2.kept[0].tolist() == st2.kept[1].tolist() == st2.kept[2].tolist() and len(st2.kept[0]) == 4
    # a frame that keeps nothing has a zero entry and is still retrievable around
    st3 = O.Store(dict(cfg, keep_per_segment=1))
    O.compress_chunk(st3, Q[:3], K[:, :3], V[:, :3])
    assert sorted(len(k) for k in st3.kept) == [0, 0, 1]
    empty = [t for t in range(3) if len(st3.kept[t]) == 0][0]
    assert not st3.frame_entry(empty)[0].any()
    r = O.retrieve(st3, rand(2, Hq, D), 1, 2)
    assert len(r["frm_idx"]) == 2


# --------------------------------------------------------------------------- past keys in the softmax
def test_attention_with_past_keys():
    import torch
    P, Hq, Hkv, D, n_past = 9, 4, 2, 8, 5
    Q, K, Kp = rand(P, Hq, D), rand(P, Hkv, D), rand(n_past, Hkv, D)
    for causal in (False, True):
        got = O.attention_importance(Q, K, causal, Kp)
        # library softmax over the concatenated keys, own columns summed
        kk = torch.from_numpy(np.concatenate([Kp, K]).astype(np.float64)).repeat_interleave(Hq // Hkv, dim=1)
        z = torch.einsum("ihd,jhd->hij", torch.from_numpy(Q.astype(np.float64)), kk) / np.sqrt(D)
        if causal:
            vis = torch.cat([torch.ones(P, n_past, dtype=torch.bool), torch.tril(torch.ones(P, P, dtype=torch.bool))], 1)
            z = z.masked_fill(~vis, float("-inf"))
        a = torch.softmax(z, dim=-1)
        np.testing.assert_allclose(got, a[:, :, n_past:].sum(dim=(0, 1)).numpy() / (Hq * P), rtol=1e-12)
        assert got.sum() < 1.0                                     # the past takes part of the attention mass
    assert np.allclose(O.attention_importance(Q, K, False, Kp[:0]), O.attention_importance(Q, K))
    # a past key far more similar to every query than any own key takes nearly all the mass
    big = np.zeros((1, Hkv, D), dtype=np.float32)
    Qc = np.ones((P, Hq, D), dtype=np.float32)
    big[:] = 50.0
    assert O.attention_importance(Qc, K, False, big).sum() < 1e-6
    # through the store: the second chunk sees the kept keys of the last W frames before it, not its own frames
    cfg = dict(CFG, past_frames=2)
    st = O.Store(cfg)
    L, P2 = 3, 12
    Qs, Ks, Vs = rand(5, P2, 4, 8), rand(L, 5, P2, 2, 8), rand(L, 5, P2, 2, 8)
    O.compress_chunk(st, Qs[:3], Ks[:, :3], Vs[:, :3])
    O.compress_chunk(st, Qs[3:], Ks[:, 3:], Vs[:, 3:])
    past = np.concatenate([st.page_k[1][-1], st.page_k[2][-1]], axis=0)
    for f in (3, 4):
        want = O.topk_set(O.score_frame(Qs[f], Ks[-1, f], 0.7, K_past=past)[2], 5)
        assert st.kept[f].tolist() == want.tolist()
    assert st.kept[0].tolist() == O.topk_set(O.score_frame(Qs[0], Ks[-1, 0], 0.7)[2], 5).tolist()

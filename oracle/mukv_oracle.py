"""CPU oracle for the MuKV compression + retrieval path (test infrastructure only).

This module is the slow, plain statement of what the CUDA library must compute.
It is written from the paper's equations (Sec. 3.3 - 3.5), step by step, in
float64, with numpy only.  It shares no code with the CUDA path and must never
be imported by the product package: only the tests, the smoke check and the
benchmark's CPU-baseline leg may use it.

Notation follows the paper: P tokens per frame, D head dimension, H heads,
L layers, kappa kept tokens per block, C = H*D concatenated feature size,
k_g retrieved blocks per granularity, lambda_g coherence factor.

Layouts (token-major):
    Q  [P][Hq][D]      last-layer queries of one frame
    K  [L][P][Hkv][D]  keys of one frame for all layers (last layer = K[L-1])
    V  [L][P][Hkv][D]
Grouped-query attention: query head h attends with key head h // (Hq // Hkv).

Pins: every function here is checked in tests/test_oracle_pins.py against
library routines, closed forms, invariants or brute force.  The one part that
has no pin is whether the heuristic keeps the tokens that matter for answer
accuracy ("parity unpinned": only the paper's accuracy tables speak to that and
they need its datasets and model weights).
"""
from __future__ import annotations

import numpy as np

TIE_EPS = 1e-6
NORM_FLOOR = 1e-12


# --------------------------------------------------------------------------
# input decoding
# --------------------------------------------------------------------------
def as_f64(x: np.ndarray) -> np.ndarray:
    """Widen an input tensor exactly to float64.

    uint16 arrays hold bfloat16 bit patterns (the upper half of a float32);
    float32 arrays are taken as they are.
    """
    x = np.asarray(x)
    if x.dtype == np.uint16:
        return (x.astype(np.uint32) << np.uint32(16)).view(np.float32).astype(np.float64)
    if x.dtype in (np.float32, np.float64):
        return x.astype(np.float64)
    raise TypeError(f"unsupported input dtype {x.dtype}")


# --------------------------------------------------------------------------
# Sec. 3.3, Eq. 1: attention-based indicator
# --------------------------------------------------------------------------
def attention_importance(Q, K_last, causal: bool = False, K_past=None) -> np.ndarray:
    """I_att[j] = 1/(H*P) * sum_h sum_i A_h[i, j]   (Eq. 1).

    A_h = row-softmax(Q_h K_g^T / sqrt(D)) over the P tokens of the frame,
    g = h // (Hq/Hkv).  With causal=True query i only sees keys j <= i.

    K_past [n_past][Hkv][D] (Sec. 3.2: the prefill of a time step also sees the cached keys of the same
    granularity): the softmax of every query then runs over the past keys and the frame's own tokens
    (past keys are visible to every query, causal or not); the importance is still that of the
    frame's own P tokens, so it sums to less than 1 by the attention mass the past takes.
    """
    Q = as_f64(Q)
    K = as_f64(K_last)
    P, Hq, D = Q.shape
    Hkv = K.shape[1]
    G = Hq // Hkv
    n_past = 0
    if K_past is not None and np.asarray(K_past).shape[0] > 0:
        Kp = as_f64(K_past)
        n_past = Kp.shape[0]
        K = np.concatenate([Kp, K], axis=0)
    col = np.zeros(P, dtype=np.float64)
    for h in range(Hq):
        g = h // G
        z = (Q[:, h, :] @ K[:, g, :].T) / np.sqrt(float(D))       # [i][past ++ own j]
        if causal:
            vis = np.concatenate([np.ones((P, n_past), dtype=bool), np.tril(np.ones((P, P), dtype=bool))], axis=1)
            z = np.where(vis, z, -np.inf)
        m = z.max(axis=1, keepdims=True)
        e = np.exp(z - m)
        a = e / e.sum(axis=1, keepdims=True)
        col += a[:, n_past:].sum(axis=0)
    return col / float(Hq * P)


# --------------------------------------------------------------------------
# Sec. 3.3, Eq. 2-3: frequency-based indicator
# --------------------------------------------------------------------------
def dft_matrix(D: int) -> np.ndarray:
    """W[b, d] = exp(-2*pi*i*b*d/D): the discrete Fourier transform written out."""
    b = np.arange(D, dtype=np.float64).reshape(D, 1)
    d = np.arange(D, dtype=np.float64).reshape(1, D)
    ang = -2.0 * np.pi * np.mod(b * d, float(D)) / float(D)
    return np.cos(ang) + 1j * np.sin(ang)


def frequency_importance(K_last) -> np.ndarray:
    """I_fft[j] = mean over heads and over the D bins of |DFT_D(k_j,head)|  (Eq. 2-3).

    The transform runs along the feature axis of each token's key vector, per
    key head; magnitudes of all D complex bins are averaged.
    """
    K = as_f64(K_last)
    P, Hkv, D = K.shape
    W = dft_matrix(D)
    Z = K.reshape(P * Hkv, D).astype(np.complex128) @ W.T          # [token*head][bin]
    mag = np.abs(Z).reshape(P, Hkv, D)
    return mag.sum(axis=(1, 2)) / float(Hkv * D)


# --------------------------------------------------------------------------
# Sec. 3.3, Eq. 4: dual-signal fusion
# --------------------------------------------------------------------------
def minmax(x: np.ndarray) -> np.ndarray:
    """Min-max normalisation to [0, 1]; a constant vector maps to all zeros."""
    x = np.asarray(x, dtype=np.float64)
    lo, hi = x.min(), x.max()
    if hi == lo:
        return np.zeros_like(x)
    return (x - lo) / (hi - lo)


def fuse(I_att, I_fft, alpha: float, keep_low_freq: bool = False) -> np.ndarray:
    """I = alpha * minmax(I_att) + (1 - alpha) * minmax(I_fft)   (Eq. 4)."""
    a = minmax(I_att)
    f = minmax(I_fft)
    if keep_low_freq:
        f = 1.0 - f
    return float(alpha) * a + (1.0 - float(alpha)) * f


# --------------------------------------------------------------------------
# top-k selection with the tie band
# --------------------------------------------------------------------------
def topk_set(s, k: int, delta: float = TIE_EPS) -> np.ndarray:
    """Indices of the k highest scores, ascending by index.

    tau is the k-th largest score.  Every score above tau + delta is taken;
    the scores within delta of tau are treated as tied and the remaining
    places go to the lowest indices among them.
    """
    s = np.asarray(s, dtype=np.float64)
    n = s.shape[0]
    k = int(k)
    if k <= 0 or n == 0:
        return np.zeros(0, dtype=np.int64)
    if k >= n:
        return np.arange(n, dtype=np.int64)
    tau = np.sort(s)[n - k]
    sure = np.nonzero(s > tau + delta)[0]
    band = np.nonzero(np.abs(s - tau) <= delta)[0]
    need = k - sure.shape[0]
    out = np.concatenate([sure, band[:need]])
    return np.sort(out).astype(np.int64)


# --------------------------------------------------------------------------
# Sec. 3.3 "Granularity Adaptive Compression" + Sec. 3.4 Eq. 5: one frame
# --------------------------------------------------------------------------
def keep_count(rho: float, n_tokens: int) -> int:
    """kappa = floor(rho * |block|)."""
    return int(np.floor(rho * n_tokens + 1e-9))


def select_tokens(I, kappa: int, delta: float = TIE_EPS) -> np.ndarray:
    """Kept token ids of one block from its fused scores (Sec. 3.3, "Granularity Adaptive
    Compression": the kappa highest scores stay), ascending.

    The paper does not say what happens when a score is not a number (Inf or NaN among the
    inputs).  Reading: such a block has no ranking, and its first kappa tokens are kept.
    """
    I = np.asarray(I, dtype=np.float64)
    if not np.all(np.isfinite(I)):
        return np.arange(min(int(kappa), I.shape[0]), dtype=np.int64)
    return topk_set(I, kappa, delta)


def score_frame(Q, K_last, alpha, causal=False, keep_low_freq=False, K_past=None):
    """(I_att, I_fft, I) for one frame.

    Q[P][Hq][D], K_last[P][Hkv][D]: one scoring layer (the paper's default: the last layer).
    Q[Ls][P][Hq][D], K_last[Ls][P][Hkv][D]: several scoring layers (the layer-choice ablation's
    "last-5 fusion"); both indicators are then the means of the per-layer indicators.
    """
    Q = np.asarray(Q)
    K_last = np.asarray(K_last)
    if Q.ndim == 4:
        ia = np.mean([attention_importance(Q[l], K_last[l], causal, None if K_past is None else K_past[l])
                      for l in range(Q.shape[0])], axis=0)
        ifr = np.mean([frequency_importance(K_last[l]) for l in range(Q.shape[0])], axis=0)
    else:
        ia = attention_importance(Q, K_last, causal, K_past)
        ifr = frequency_importance(K_last)
    return ia, ifr, fuse(ia, ifr, alpha, keep_low_freq)


def past_keys(store, t_chunk: int, cfg: dict):
    """Cached keys the chunk's queries also attend to (past_frames = W > 0): the kept keys, in the
    scoring layers, of the W most recent frames stored before the chunk (a chunk is one time step:
    its frames do not see one another's cache).  [Ls][n_past][Hkv][D] in storage form, or None."""
    W = int(cfg.get("past_frames", 0))
    t0 = max(0, t_chunk - W)
    if W <= 0 or t0 == t_chunk:
        return None
    lay = score_layers(cfg)
    return np.stack([np.concatenate([store.page_k[t][l] for t in range(t0, t_chunk)], axis=0) for l in lay])


def score_layers(cfg: dict) -> range:
    """Indices of the layers whose attention and keys give the indicators: n_score_layers layers
    ending score_layer_offset layers before the end of the model (defaults: the last layer alone)."""
    L = cfg["n_layers"]
    Ls = max(int(cfg.get("n_score_layers", 1)), 1)
    off = int(cfg.get("score_layer_offset", 0))
    return range(L - off - Ls, L - off)


def super_patch_of(token_ids, P: int, grid_width: int, split: int) -> np.ndarray:
    """Super patch (0 .. split*split-1, row-major) of each token id of a frame whose P tokens are a
    grid of grid_width columns, cut into split x split rectangles of ceil(rows/split) x
    ceil(grid_width/split) tokens."""
    ids = np.asarray(token_ids, dtype=np.int64)
    rows = P // grid_width
    rh = -(-rows // split)
    cw = -(-grid_width // split)
    return (ids // grid_width) // rh * split + (ids % grid_width) // cw


def compact_rows(X, kept):
    """X[L][P][Hkv][D] -> X[L][kappa][Hkv][D] in ascending token order (bytes untouched)."""
    return np.ascontiguousarray(np.asarray(X)[:, kept, :, :])


def pool_rows(Xc):
    """Sum over the kept tokens of a compacted block: [L][kappa][Hkv][D] -> float64 [L][C]."""
    X = as_f64(Xc)
    L, kap, Hkv, D = X.shape
    return X.sum(axis=1).reshape(L, Hkv * D)


class Store:
    """The compressed cache the oracle builds: one entry per frame, pooled entries per segment."""

    def __init__(self, cfg: dict):
        self.cfg = dict(cfg)
        self.kept = []          # per frame: int64 [kappa], ascending
        self.page_k = []        # per frame: raw-dtype [L][kappa][Hkv][D]
        self.page_v = []
        self.sum_k = []         # per frame: float64 [L][C] sums over kept tokens
        self.sum_v = []
        self.scores = []        # per frame: (I_att, I_fft, I)

    @property
    def n_frames(self) -> int:
        return len(self.kept)

    @property
    def n_segments(self) -> int:
        fs = self.cfg["frames_per_segment"]
        return (self.n_frames + fs - 1) // fs

    # Eq. 5 applied to every layer, K and V: float32 means over the kept tokens
    def frame_entry(self, t: int):
        kap = float(self.kept[t].shape[0])
        if kap == 0.0:                      # segment-scope selection may leave a frame without tokens
            z = np.zeros(self.sum_k[t].shape, dtype=np.float32)
            return z, z.copy()
        return ((self.sum_k[t] / kap).astype(np.float32),
                (self.sum_v[t] / kap).astype(np.float32))

    def frame_key(self, t: int) -> np.ndarray:
        """Retrieval key of frame t: mean of the last-layer kept keys, heads concatenated."""
        return self.frame_entry(t)[0][-1]

    # Sec. 3.2 / Eq. 5 "similarly k_{p_ft}": patch-level blocks.  The frame's P tokens form a grid of
    # grid_width columns; the grid is cut into patch_split x patch_split super patches, and the kept
    # tokens of a frame that fall into one super patch are one patch-level block.  Its key is the
    # mean of their last-layer keys (heads concatenated); a super patch that kept no token has no block.
    def n_patches(self) -> int:
        return int(self.cfg.get("patch_split", 0)) ** 2

    def patch_tokens(self, t: int, sp: int) -> np.ndarray:
        """Positions (in the frame's kept list) of the kept tokens inside super patch sp."""
        ids = self.kept[t]
        return np.nonzero(super_patch_of(ids, self.cfg["tokens_per_frame"], self.cfg["grid_width"],
                                         self.cfg["patch_split"]) == sp)[0]

    def patch_count(self, t: int, sp: int) -> int:
        return int(self.patch_tokens(t, sp).shape[0])

    def patch_key(self, t: int, sp: int) -> np.ndarray:
        pos = self.patch_tokens(t, sp)
        C = self.sum_k[t].shape[1]
        if pos.shape[0] == 0:
            return np.zeros(C, dtype=np.float32)
        rows = as_f64(self.page_k[t][-1][pos]).reshape(pos.shape[0], C)
        return (rows.sum(axis=0) / float(pos.shape[0])).astype(np.float32)

    def patch_keys(self, n_frm: int) -> np.ndarray:
        S = self.n_patches()
        C = self.sum_k[0].shape[1]
        out = np.zeros((n_frm * S, C), dtype=np.float32)
        for t in range(n_frm):
            for sp in range(S):
                out[t * S + sp] = self.patch_key(t, sp)
        return out

    def segment_frames(self, u: int):
        fs = self.cfg["frames_per_segment"]
        return range(u * fs, min((u + 1) * fs, self.n_frames))

    def segment_entry(self, u: int):
        """Mean over all kept tokens of the frames of segment u that are present."""
        fr = list(self.segment_frames(u))
        n_tok = float(sum(self.kept[t].shape[0] for t in fr))
        sk = np.sum([self.sum_k[t] for t in fr], axis=0)
        sv = np.sum([self.sum_v[t] for t in fr], axis=0)
        return (sk / n_tok).astype(np.float32), (sv / n_tok).astype(np.float32)

    def segment_key(self, u: int) -> np.ndarray:
        return self.segment_entry(u)[0][-1]

    def frame_keys(self) -> np.ndarray:
        return np.stack([self.frame_key(t) for t in range(self.n_frames)])

    def segment_keys(self) -> np.ndarray:
        return np.stack([self.segment_key(u) for u in range(self.n_segments)])


def compress_chunk(store: Store, Q, K, V, select_scores=None) -> None:
    """Append one chunk.  Q[n][P][Hq][D] (queries of the scoring layer; [Ls][n][P][Hq][D] with
    several scoring layers, see score_layers), K,V[L][n][P][Hkv][D].

    With select_scores[n][P] the tokens are ranked by those numbers instead of the dual signal:
    the "Rand(50%)" row of the paper's compression ablation (tokens dropped at random) is this
    with uniform random scores and kappa = P/2; Q is not used then.
    """
    cfg = store.cfg
    n = np.asarray(K).shape[1]
    if int(cfg.get("keep_per_segment", 0)) > 0:
        return _compress_chunk_segment_scope(store, Q, K, V)
    t_chunk = store.n_frames                        # frames stored before this chunk
    for f in range(n):
        Kf = np.asarray(K)[:, f]
        Vf = np.asarray(V)[:, f]
        if select_scores is not None:
            I = np.asarray(select_scores, dtype=np.float64)[f]
            ia = ifr = np.zeros_like(I)
        else:
            lay = score_layers(cfg)
            Qa = np.asarray(Q)
            past = past_keys(store, t_chunk, cfg)
            if Qa.ndim == 5:
                ia, ifr, I = score_frame(Qa[:, f], Kf[lay.start:lay.stop], cfg["alpha"],
                                         cfg.get("attn_causal", False), cfg.get("keep_low_freq", False), past)
            else:
                ia, ifr, I = score_frame(Qa[f], Kf[lay.stop - 1], cfg["alpha"],
                                         cfg.get("attn_causal", False), cfg.get("keep_low_freq", False),
                                         None if past is None else past[-1])
        kept = select_tokens(I, cfg["keep_per_frame"], cfg.get("tie_eps", TIE_EPS))
        pk = compact_rows(Kf, kept)
        pv = compact_rows(Vf, kept)
        store.kept.append(kept)
        store.page_k.append(pk)
        store.page_v.append(pv)
        store.sum_k.append(pool_rows(pk))
        store.sum_v.append(pool_rows(pv))
        store.scores.append((ia, ifr, I))


def segment_keep_count(kappa_v: int, frames_present: int, frames_per_segment: int) -> int:
    """Tokens kept in a segment of which only frames_present frames exist (the last one of a stream):
    the budget kappa_v = floor(rho_v * O) of a full segment, scaled to the tokens present."""
    return (int(kappa_v) * int(frames_present)) // int(frames_per_segment)


def _compress_chunk_segment_scope(store: Store, Q, K, V) -> None:
    """Segment-level DCP (Sec. 3.3: "similarly ... I_v in R^O", kappa_v = floor(rho_v * |v_t|)): the
    indicators of every frame of a segment are computed as for a frame (attention inside the frame),
    but the min-max normalisation of Eq. 4 and the top-kappa_v selection run over all O = F * P tokens
    of the segment.  A frame then keeps a variable number of tokens.  The chunk must start on a
    segment boundary and hold whole segments (the last segment of a stream may be short)."""
    cfg = store.cfg
    fs = cfg["frames_per_segment"]
    P = cfg["tokens_per_frame"]
    n = np.asarray(K).shape[1]
    assert store.n_frames % fs == 0, "a chunk must start on a segment boundary"
    lay = score_layers(cfg)
    Qa = np.asarray(Q)
    for s0 in range(0, n, fs):
        m = min(fs, n - s0)
        ia, ifr = [], []
        for f in range(s0, s0 + m):
            Kf = np.asarray(K)[:, f]
            if Qa.ndim == 5:
                a = np.mean([attention_importance(Qa[l, f], Kf[lay.start + l], cfg.get("attn_causal", False))
                             for l in range(len(lay))], axis=0)
                b = np.mean([frequency_importance(Kf[lay.start + l]) for l in range(len(lay))], axis=0)
            else:
                a = attention_importance(Qa[f], Kf[lay.stop - 1], cfg.get("attn_causal", False))
                b = frequency_importance(Kf[lay.stop - 1])
            ia.append(a)
            ifr.append(b)
        ia, ifr = np.concatenate(ia), np.concatenate(ifr)                  # [O]
        I = fuse(ia, ifr, cfg["alpha"], cfg.get("keep_low_freq", False))
        kept_all = select_tokens(I, segment_keep_count(cfg["keep_per_segment"], m, fs), cfg.get("tie_eps", TIE_EPS))
        for i, f in enumerate(range(s0, s0 + m)):
            kept = kept_all[(kept_all >= i * P) & (kept_all < (i + 1) * P)] - i * P
            pk = compact_rows(np.asarray(K)[:, f], kept)
            pv = compact_rows(np.asarray(V)[:, f], kept)
            store.kept.append(kept)
            store.page_k.append(pk)
            store.page_v.append(pv)
            store.sum_k.append(pool_rows(pk))
            store.sum_v.append(pool_rows(pv))
            store.scores.append((ia[i * P:(i + 1) * P], ifr[i * P:(i + 1) * P], I[i * P:(i + 1) * P]))


# --------------------------------------------------------------------------
# Sec. 3.4: semi-hierarchical retrieval
# --------------------------------------------------------------------------
def pool_question(Qq, n_kv_heads: int) -> np.ndarray:
    """q = mean over the question's query tokens (Eq. 6), heads concatenated.

    With grouped-query attention the Hq/Hkv query heads that share a key head
    are averaged, so that q has the same C = Hkv*D features as the block keys.
    """
    X = as_f64(Qq)
    Nq, Hq, D = X.shape
    G = Hq // n_kv_heads
    return X.reshape(Nq, n_kv_heads, G, D).sum(axis=(0, 2)).reshape(n_kv_heads * D) / float(Nq * G)


def cosine(q, keys) -> np.ndarray:
    """cos(q, keys[t]) for every row (Eq. 7); a zero-norm pair scores 0."""
    q = np.asarray(q, dtype=np.float64)
    keys = np.asarray(keys, dtype=np.float64)
    if keys.shape[0] == 0:
        return np.zeros(0, dtype=np.float64)
    num = keys @ q
    den = np.sqrt((keys * keys).sum(axis=1)) * np.sqrt((q * q).sum())
    return num / np.maximum(den, NORM_FLOOR)


MODE_PARALLEL, MODE_HIER, MODE_SEMI = 0, 1, 2


def retrieve(store: Store, Qq, k_seg: int, k_frm: int, top_n: int = 0, lam: float = 0.3,
             mode: int = MODE_SEMI, t_limit=None, delta: float = TIE_EPS):
    """One question.  Returns dict with ascending seg_idx / frm_idx and their scores.

    Visible frames have id < t_limit; a segment is visible when its last stored
    frame is.  Stage 1 ranks every visible block by cosine with q and keeps
    top-2k candidates per granularity; stage 2 (Eq. 8) re-scores the frame
    candidates with their cosine to the mean of the top-N segment keys.
    """
    cfg = store.cfg
    T = store.n_frames
    t_limit = T if t_limit is None else min(int(t_limit), T)
    fs = cfg["frames_per_segment"]
    n_frm = max(t_limit, 0)
    n_seg = sum(1 for u in range(store.n_segments) if min((u + 1) * fs, T) <= t_limit)

    q = pool_question(Qq, cfg["n_kv_heads"])
    key_f = store.frame_keys()[:n_frm].astype(np.float64) if n_frm else np.zeros((0, q.shape[0]))
    key_s = store.segment_keys()[:n_seg].astype(np.float64) if n_seg else np.zeros((0, q.shape[0]))
    s_frm = cosine(q, key_f)
    s_seg = cosine(q, key_s)

    sel_seg = topk_set(s_seg, min(k_seg, n_seg), delta)
    if mode == MODE_PARALLEL:
        sel_frm = topk_set(s_frm, min(k_frm, n_frm), delta)
        final = s_frm[sel_frm]
    elif mode == MODE_HIER:
        inside = np.array([t for t in range(n_frm) if (t // fs) in set(sel_seg.tolist())], dtype=np.int64)
        pick = topk_set(s_frm[inside], min(k_frm, inside.shape[0]), delta)
        sel_frm = inside[pick]
        final = s_frm[sel_frm]
    else:
        cand = topk_set(s_frm, min(2 * k_frm, n_frm), delta)
        N = k_seg if top_n <= 0 else top_n
        top = topk_set(s_seg, min(N, n_seg), delta)
        if top.shape[0] > 0:
            g = key_s[top].sum(axis=0) / float(top.shape[0])
            gamma = cosine(g, key_f[cand])
        else:
            gamma = np.zeros(cand.shape[0])
        s_new = (1.0 - lam) * s_frm[cand] + lam * gamma
        pick = topk_set(s_new, min(k_frm, cand.shape[0]), delta)
        sel_frm = cand[pick]
        final = s_new[pick]
    return {
        "q": q, "s_frm": s_frm, "s_seg": s_seg,
        "seg_idx": sel_seg, "seg_score": s_seg[sel_seg],
        "frm_idx": sel_frm, "frm_score": final,
    }


def _rerank(s_stage1, keys, cand, g, lam, k, delta):
    """Eq. 8 on one granularity's candidates: returns (positions in cand, their calibrated scores)."""
    gamma = cosine(g, keys[cand]) if g is not None else np.zeros(cand.shape[0])
    s_new = (1.0 - lam) * s_stage1[cand] + lam * gamma
    pick = topk_set(s_new, min(k, cand.shape[0]), delta)
    return pick, s_new[pick]


def retrieve3(store: Store, Qq, k_g, lambda_g, top_n: int = 0, mode: int = MODE_SEMI, t_limit=None,
              delta: float = TIE_EPS):
    """Sec. 3.4 over all three granularities.  k_g = (k_patch, k_frm, k_seg) and lambda_g =
    (lambda_patch, lambda_frm, lambda_seg) in the paper's order (patch-, frame-, segment-level); the
    paper's values are k_g = {20, 32, 12}, lambda_g = {0.3, 0.3, 0}.

    Stage 1: cosine of the pooled question with every visible block key of each granularity (Eq. 7),
    top-2k_g candidates per granularity.  Stage 2: the global query is the mean of the top-N
    segment-level keys; every candidate of a granularity with lambda_g > 0 gets Eq. 8 and the best
    k_g are kept (lambda_g = 0: the best k_g by cosine).  PARALLEL keeps the best k_g by cosine at every
    granularity; HIER looks for frame- and patch-level blocks only inside the selected segments.
    Patch-level block ids are frame * S + super patch; a super patch that kept no token is no block.
    """
    cfg = store.cfg
    T = store.n_frames
    t_limit = T if t_limit is None else min(int(t_limit), T)
    fs = cfg["frames_per_segment"]
    S = store.n_patches()
    k_pat, k_frm, k_seg = (int(x) for x in k_g)
    lam_pat, lam_frm, lam_seg = (float(x) for x in lambda_g)
    n_frm = max(t_limit, 0)
    n_seg = sum(1 for u in range(store.n_segments) if min((u + 1) * fs, T) <= t_limit)
    q = pool_question(Qq, cfg["n_kv_heads"])
    C = q.shape[0]
    key_f = store.frame_keys()[:n_frm].astype(np.float64) if n_frm else np.zeros((0, C))
    key_s = store.segment_keys()[:n_seg].astype(np.float64) if n_seg else np.zeros((0, C))
    key_p = store.patch_keys(n_frm).astype(np.float64) if n_frm and S else np.zeros((0, C))
    s_frm, s_seg, s_pat = cosine(q, key_f), cosine(q, key_s), cosine(q, key_p)
    exists = np.array([store.patch_count(b // S, b % S) > 0 for b in range(n_frm * S)], dtype=bool) \
        if S else np.zeros(0, dtype=bool)

    # segment level; its own lambda is applied too (the paper sets it to 0: the global query comes from them)
    N = k_seg if top_n <= 0 else top_n
    top = topk_set(s_seg, min(N, n_seg), delta)
    g = key_s[top].sum(axis=0) / float(top.shape[0]) if top.shape[0] > 0 else None
    if mode == MODE_SEMI and lam_seg > 0.0:
        cand = topk_set(s_seg, min(2 * k_seg, n_seg), delta)
        pick, sc = _rerank(s_seg, key_s, cand, g, lam_seg, k_seg, delta)
        sel_seg, seg_sc = cand[pick], sc
    else:
        sel_seg = topk_set(s_seg, min(k_seg, n_seg), delta)
        seg_sc = s_seg[sel_seg]

    def lower(s1, keys, member, k, lam):
        ids = np.nonzero(member)[0]
        if mode == MODE_HIER:
            inside = set(sel_seg.tolist())
            ids = np.array([b for b in ids if (owner(b) // fs) in inside], dtype=np.int64)
        if mode == MODE_SEMI:
            cand = ids[topk_set(s1[ids], min(2 * k, ids.shape[0]), delta)]
            pick, sc = _rerank(s1, keys, cand, g, lam, k, delta)
            return cand[pick], sc
        pick = topk_set(s1[ids], min(k, ids.shape[0]), delta)
        return ids[pick], s1[ids[pick]]

    owner = lambda b: b
    sel_frm, frm_sc = lower(s_frm, key_f, np.ones(n_frm, dtype=bool), k_frm, lam_frm)
    owner = lambda b: b // S
    if S:
        sel_pat, pat_sc = lower(s_pat, key_p, exists, k_pat, lam_pat)
    else:
        sel_pat, pat_sc = np.zeros(0, dtype=np.int64), np.zeros(0)
    return {"q": q, "seg_idx": sel_seg, "seg_score": seg_sc, "frm_idx": sel_frm, "frm_score": frm_sc,
            "patch_idx": sel_pat, "patch_score": pat_sc}


# --------------------------------------------------------------------------
# Sec. 3.5, Eq. 9: the retrieved context R_k, R_v
# --------------------------------------------------------------------------
def gather(store: Store, frm_idx):
    """decode[l][K then V][slot*kappa + r][Hkv][D] for the selected frames in ascending order,
    and token meta (frame id, token id) per slot."""
    frm_idx = [int(t) for t in frm_idx]
    if not frm_idx:
        return None, np.zeros((0, 2), dtype=np.int32)
    Rk = np.concatenate([store.page_k[t] for t in frm_idx], axis=1)     # [L][n*kappa][Hkv][D]
    Rv = np.concatenate([store.page_v[t] for t in frm_idx], axis=1)
    dec = np.stack([Rk, Rv], axis=1)                                     # [L][2][n*kappa][Hkv][D]
    meta = np.array([(t, int(j)) for t in frm_idx for j in store.kept[t]], dtype=np.int32)
    return dec, meta


def round_to_dtype(x: np.ndarray, like: np.ndarray) -> np.ndarray:
    """float32 values in the storage type of `like`: bfloat16 bit patterns (round to nearest even)
    or float32."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    if like.dtype == np.uint16:
        b = x.view(np.uint32)
        return ((b + np.uint32(0x7FFF) + ((b >> np.uint32(16)) & np.uint32(1))) >> np.uint32(16)).astype(np.uint16)
    return x


def gather3(store: Store, seg_idx, frm_idx, patch_idx):
    """The decode context when the selected blocks of all three granularities are loaded
    (Sec. 3.4, first paragraph; Sec. 3.5).  Per layer, K then V, token slots in this order:
    one summary token per selected segment (its pooled entry, Eq. 5, rounded to the cache's storage
    type), the kept tokens of the selected frames, the kept tokens of the selected patch-level
    blocks; every group ascending by block id, tokens ascending inside a block.
    Returns (decode [L][2][n_tok][Hkv][D], meta [n_tok][2]): meta is (frame, token id), and
    (-1 - segment, -1) for a summary token."""
    S = store.n_patches()
    L = store.page_k[0].shape[0]
    Hkv, D = store.page_k[0].shape[2], store.page_k[0].shape[3]
    ks, vs, meta = [], [], []
    for u in [int(u) for u in seg_idx]:
        ek, ev = store.segment_entry(u)
        ks.append(round_to_dtype(ek, store.page_k[0]).reshape(L, 1, Hkv, D))
        vs.append(round_to_dtype(ev, store.page_v[0]).reshape(L, 1, Hkv, D))
        meta.append((-1 - u, -1))
    for t in [int(t) for t in frm_idx]:
        ks.append(store.page_k[t])
        vs.append(store.page_v[t])
        meta += [(t, int(j)) for j in store.kept[t]]
    for b in [int(b) for b in patch_idx]:
        t, sp = b // S, b % S
        pos = store.patch_tokens(t, sp)
        ks.append(store.page_k[t][:, pos])
        vs.append(store.page_v[t][:, pos])
        meta += [(t, int(store.kept[t][r])) for r in pos]
    if not ks:
        return None, np.zeros((0, 2), dtype=np.int32)
    dec = np.stack([np.concatenate(ks, axis=1), np.concatenate(vs, axis=1)], axis=1)
    return dec, np.array(meta, dtype=np.int32).reshape(-1, 2)

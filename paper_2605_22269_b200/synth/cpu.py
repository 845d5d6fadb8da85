"""Seeded synthetic K/V/Q streams, CPU side (numpy).

The generator holds none of the method's arithmetic: it only produces inputs.
Every value comes from integer hashing plus a handful of IEEE float32
multiplies and adds in a fixed order, so the CUDA generator in ``synth.cu``
produces the same bytes; tests check that.  Frames are generated from their
absolute index in the stream, so any chunking yields the same stream.

Recipe (shapes follow a 7B grouped-query video LLM; see ``StreamSpec``):
  token noise   n ~ N(0,1) per element (quantile table lookup, 65,536 levels)
  outliers      per (layer, key head) ``n_outlier`` channels scaled by ``outlier_scale`` in K and V
  scenes        frames of a scene share a mean mu_c ~ N(0,1) per (layer, head, channel);
                each frame adds nu_t ~ N(0, frame_sigma^2)
  K = (n * scale + scene_sigma * mu_c) + frame_sigma * nu_t,   V = n * scale,   Q = n
Values are rounded to bfloat16 (round to nearest even) or kept float32.
"""
from __future__ import annotations

from dataclasses import dataclass, field

import numpy as np

MASK = (1 << 64) - 1
GOLD = 0x9E3779B97F4A7C15
M1 = 0xBF58476D1CE4E5B9
M2 = 0x94D049BB133111EB

TAG_K, TAG_V, TAG_Q, TAG_OUT, TAG_MU, TAG_NU, TAG_SCENE, TAG_QUEST, TAG_RAND = 1, 2, 3, 4, 5, 6, 7, 8, 9

TABLE_BITS = 16


def mix64(x: int) -> int:
    x &= MASK
    x ^= x >> 30
    x = (x * M1) & MASK
    x ^= x >> 27
    x = (x * M2) & MASK
    x ^= x >> 31
    return x


def stream_key(seed: int, tag: int, sub: int = 0) -> int:
    """Key of one random stream: (seed, tensor tag, sub-stream such as the frame index)."""
    return mix64(mix64((seed * GOLD + tag) & MASK) + ((sub + 1) * GOLD & MASK))


def _mix64_np(x: np.ndarray) -> np.ndarray:
    with np.errstate(over="ignore"):
        x = x ^ (x >> np.uint64(30))
        x = x * np.uint64(M1)
        x = x ^ (x >> np.uint64(27))
        x = x * np.uint64(M2)
        x = x ^ (x >> np.uint64(31))
    return x


_TABLE = None


def normal_table() -> np.ndarray:
    """float32 standard-normal quantiles at (i + 0.5) / 65536."""
    global _TABLE
    if _TABLE is None:
        from scipy.special import ndtri
        n = 1 << TABLE_BITS
        _TABLE = ndtri((np.arange(n, dtype=np.float64) + 0.5) / n).astype(np.float32)
    return _TABLE


def normals(key: int, count: int, start: int = 0) -> np.ndarray:
    """float32 N(0,1) values for element indices start..start+count-1 of stream ``key``.

    Element e uses 16 bits of hash word e >> 2 (four elements per 64-bit word).
    """
    if count <= 0:
        return np.zeros(0, dtype=np.float32)
    w0, w1 = start >> 2, (start + count + 3) >> 2
    words = np.arange(w0, w1, dtype=np.uint64)
    with np.errstate(over="ignore"):
        h = _mix64_np(np.uint64(key) + (words + np.uint64(1)) * np.uint64(GOLD))
    shifts = np.array([0, 16, 32, 48], dtype=np.uint64)
    idx = ((h[:, None] >> shifts[None, :]) & np.uint64(0xFFFF)).reshape(-1).astype(np.int64)
    lo = start - (w0 << 2)
    return normal_table()[idx[lo:lo + count]]


def to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """float32 -> bfloat16 bit patterns (uint16), round to nearest even."""
    b = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    r = b + np.uint32(0x7FFF) + ((b >> np.uint32(16)) & np.uint32(1))
    return (r >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (b.astype(np.uint32) << np.uint32(16)).view(np.float32)


@dataclass
class StreamSpec:
    seed: int
    n_layers: int = 28
    n_q_heads: int = 28
    n_kv_heads: int = 4
    head_dim: int = 128
    tokens_per_frame: int = 196
    bf16: bool = True
    n_outlier: int = 4
    outlier_scale: float = 8.0
    scene_sigma: float = 0.0          # 0 = no scene structure
    frame_sigma: float = 0.0
    scene_min: int = 20               # scene length range, inclusive
    scene_max: int = 20
    n_frames: int = 16                # stream length (for the scene table)
    _scene: np.ndarray | None = field(default=None, repr=False)
    _scale: np.ndarray | None = field(default=None, repr=False)

    # ---- host-side tables handed to both generators -----------------------
    def out_scale(self) -> np.ndarray:
        """float32 [L][Hkv][D]: 1 everywhere, ``outlier_scale`` on the chosen channels."""
        if self._scale is None:
            L, H, D = self.n_layers, self.n_kv_heads, self.head_dim
            s = np.ones((L, H, D), dtype=np.float32)
            for l in range(L):
                for g in range(H):
                    chosen, i = [], 0
                    while len(chosen) < min(self.n_outlier, D):
                        c = mix64(stream_key(self.seed, TAG_OUT, l * H + g) + i) % D
                        i += 1
                        if c not in chosen:
                            chosen.append(c)
                    s[l, g, chosen] = np.float32(self.outlier_scale)
            self._scale = s
        return self._scale

    def scene_of_frame(self) -> np.ndarray:
        """int32 [n_frames]: scene id of every frame (lengths hashed in [scene_min, scene_max])."""
        if self._scene is None:
            out = np.zeros(self.n_frames, dtype=np.int32)
            t, c = 0, 0
            span = self.scene_max - self.scene_min + 1
            while t < self.n_frames:
                ln = self.scene_min + mix64(stream_key(self.seed, TAG_SCENE, c)) % span
                out[t:t + ln] = c
                t += ln
                c += 1
            self._scene = out
        return self._scene

    @property
    def has_scenes(self) -> bool:
        return self.scene_sigma != 0.0 or self.frame_sigma != 0.0

    # ---- tensors -----------------------------------------------------------
    def _finish(self, x: np.ndarray) -> np.ndarray:
        return to_bf16_bits(x) if self.bf16 else np.ascontiguousarray(x, dtype=np.float32)

    def scene_mean(self, c: int) -> np.ndarray:
        """mu_c as float32 [L][Hkv][D]."""
        L, H, D = self.n_layers, self.n_kv_heads, self.head_dim
        return normals(stream_key(self.seed, TAG_MU, int(c)), L * H * D).reshape(L, H, D)

    def frame_kv(self, t: int, last_layer_only: bool = False):
        """K, V of absolute frame t: [L][P][Hkv][D] each ([1][P][Hkv][D] with last_layer_only)."""
        L, H, D, P = self.n_layers, self.n_kv_heads, self.head_dim, self.tokens_per_frame
        l0 = L - 1 if last_layer_only else 0
        n_l = L - l0
        start, cnt = l0 * P * H * D, n_l * P * H * D
        scale = self.out_scale()[l0:, None, :, :]
        k = normals(stream_key(self.seed, TAG_K, t), cnt, start).reshape(n_l, P, H, D) * scale
        v = normals(stream_key(self.seed, TAG_V, t), cnt, start).reshape(n_l, P, H, D) * scale
        if self.has_scenes:
            c = int(self.scene_of_frame()[t])
            mu = self.scene_mean(c)[l0:] * np.float32(self.scene_sigma)
            nu = normals(stream_key(self.seed, TAG_NU, t), n_l * H * D, l0 * H * D).reshape(n_l, H, D) \
                * np.float32(self.frame_sigma)
            k = (k + mu[:, None, :, :]) + nu[:, None, :, :]
        return self._finish(k), self._finish(v)

    def frame_q(self, t: int) -> np.ndarray:
        """Last-layer queries of absolute frame t: [P][Hq][D]."""
        P, Hq, D = self.tokens_per_frame, self.n_q_heads, self.head_dim
        return self._finish(normals(stream_key(self.seed, TAG_Q, t), P * Hq * D).reshape(P, Hq, D))

    def chunk(self, t0: int, n: int, last_layer_only: bool = False):
        """Q[n][P][Hq][D], K[L][n][P][Hkv][D], V[L][n][P][Hkv][D] for frames t0..t0+n-1."""
        qs, ks, vs = [], [], []
        for t in range(t0, t0 + n):
            k, v = self.frame_kv(t, last_layer_only)
            qs.append(self.frame_q(t))
            ks.append(k)
            vs.append(v)
        return np.stack(qs, 0), np.stack(ks, 1), np.stack(vs, 1)

    def select_scores(self, n: int, t0: int = 0) -> np.ndarray:
        """Uniform [0, 1) float32 numbers [n][P] (24 random bits each), one per token of frames
        t0..t0+n-1: the random ranking of a random-drop baseline."""
        P = self.tokens_per_frame
        out = np.empty((n, P), dtype=np.float32)
        for i in range(n):
            words = np.arange(P, dtype=np.uint64)
            with np.errstate(over="ignore"):
                h = _mix64_np(np.uint64(stream_key(self.seed, TAG_RAND, t0 + i)) + (words + np.uint64(1)) * np.uint64(GOLD))
            out[i] = ((h >> np.uint64(40)).astype(np.float64) / float(1 << 24)).astype(np.float32)
        return out

    def questions(self, n_q: int, len_min: int, len_max: int, noise: float = 0.5):
        """Ragged question query tokens near random scene means.

        Returns (tokens [sum Nq][Hq][D], offsets int32 [n_q+1], scene ids int32 [n_q]).
        Token n of question i, head h: mu_c[L-1, h // G, :] * scene_sigma + noise * N(0,1).
        Without scene structure the tokens are plain N(0,1).
        """
        Hq, Hkv, D = self.n_q_heads, self.n_kv_heads, self.head_dim
        G = Hq // Hkv
        span = len_max - len_min + 1
        toks, offs, scenes = [], [0], []
        n_scenes = int(self.scene_of_frame().max()) + 1 if self.has_scenes else 1
        for i in range(n_q):
            kq = stream_key(self.seed, TAG_QUEST, i)
            nq = len_min + mix64(kq + 1) % span
            c = mix64(kq + 2) % n_scenes
            x = normals(kq, nq * Hq * D).reshape(nq, Hq, D)
            if self.has_scenes:
                mu = self.scene_mean(c)[-1] * np.float32(self.scene_sigma)        # [Hkv][D]
                x = np.repeat(mu, G, axis=0)[None, :, :] + np.float32(noise) * x
            toks.append(self._finish(x))
            offs.append(offs[-1] + nq)
            scenes.append(c)
        return np.concatenate(toks, 0), np.asarray(offs, dtype=np.int32), np.asarray(scenes, dtype=np.int32)


# The five workloads, by name.
def workload(name: str) -> dict:
    """Spec + method parameters of a named workload."""
    if name == "tiny":
        spec = StreamSpec(seed=1, n_layers=1, n_q_heads=2, n_kv_heads=2, head_dim=64, tokens_per_frame=64,
                          bf16=False, n_outlier=0, n_frames=8)
        return dict(spec=spec, keep=16, fseg=4, chunk=8, alpha=0.7,
                    n_questions=1, q_len=(16, 16), k_seg=1, k_frm=2, lam=0.3)
    if name == "chunk7b":
        spec = StreamSpec(seed=2, n_frames=16)
        return dict(spec=spec, keep=49, fseg=16, chunk=16, alpha=0.7,
                    n_questions=1, q_len=(32, 32), k_seg=1, k_frm=4, lam=0.3)
    if name == "stream_1h":
        spec = StreamSpec(seed=3, n_frames=1800, scene_sigma=1.0, frame_sigma=0.5, scene_min=20, scene_max=20)
        return dict(spec=spec, keep=49, fseg=16, chunk=16, alpha=0.7,
                    n_questions=8, q_len=(32, 32), k_seg=4, k_frm=8, lam=0.3)
    if name in ("stream_3h", "retrieval_stress"):
        spec = StreamSpec(seed=4, n_frames=10800, scene_sigma=1.0, frame_sigma=0.5, scene_min=10, scene_max=60)
        return dict(spec=spec, keep=49, fseg=16, chunk=16, alpha=0.7,
                    n_questions=64, q_len=(16, 64), k_seg=8, k_frm=16, lam=0.3)
    raise KeyError(name)

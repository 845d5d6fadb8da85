"""Shared helpers of the GPU parity tests: run the CUDA path through the C ABI and the CPU oracle
on the same seeded inputs.  The oracle never sees anything the CUDA path produced."""
from __future__ import annotations

import os
from concurrent.futures import ProcessPoolExecutor

import numpy as np
import torch

from oracle import mukv_oracle as O
from paper_2605_22269_b200 import binding as B
from paper_2605_22269_b200.synth.cpu import StreamSpec, workload

RTOL, ATOL = 1e-3, 1e-5          # floating-point tolerance of the parity tests
FLAG_MARGIN = 3e-6               # the library's built-in safety margin of the single-precision selection


def spec_config(spec: StreamSpec, wl: dict, max_frames: int | None = None, **over) -> B.MukvConfig:
    kw = dict(n_layers=spec.n_layers, n_q_heads=spec.n_q_heads, n_kv_heads=spec.n_kv_heads,
              head_dim=spec.head_dim, tokens_per_frame=spec.tokens_per_frame, keep_per_frame=wl["keep"],
              frames_per_segment=wl["fseg"], max_frames_per_chunk=wl["chunk"],
              max_frames=max_frames or spec.n_frames, dtype=B.BF16 if spec.bf16 else B.FP32, alpha=wl["alpha"])
    kw.update(over)
    return B.make_config(**kw)


def oracle_cfg(cfg: B.MukvConfig) -> dict:
    return dict(n_layers=cfg.n_layers, n_q_heads=cfg.n_q_heads, n_kv_heads=cfg.n_kv_heads, head_dim=cfg.head_dim,
                tokens_per_frame=cfg.tokens_per_frame, keep_per_frame=cfg.keep_per_frame,
                frames_per_segment=cfg.frames_per_segment, alpha=float(cfg.alpha),
                attn_causal=bool(cfg.attn_causal), keep_low_freq=bool(cfg.keep_low_freq), tie_eps=float(cfg.tie_eps),
                patch_split=int(cfg.patch_split), grid_width=int(cfg.grid_width),
                n_score_layers=int(cfg.n_score_layers), score_layer_offset=int(cfg.score_layer_offset),
                keep_per_segment=int(cfg.keep_per_segment), past_frames=int(cfg.past_frames))


def to_device(x: np.ndarray, bf16: bool, device="cuda:0") -> torch.Tensor:
    """numpy input (uint16 bf16 bits or float32) -> device tensor of the matching torch dtype."""
    t = torch.from_numpy(np.ascontiguousarray(x))
    if bf16:
        return t.view(torch.int16).to(device).view(torch.bfloat16)
    return t.to(device)


def to_numpy_bits(t: torch.Tensor) -> np.ndarray:
    """device tensor -> numpy; bf16 comes back as uint16 bit patterns."""
    if t.dtype == torch.bfloat16:
        return t.contiguous().view(torch.int16).cpu().numpy().view(np.uint16)
    return t.cpu().numpy()


def close(got, ref, what=""):
    got = np.asarray(got, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    err = np.abs(got - ref) - (ATOL + RTOL * np.abs(ref))
    assert got.shape == ref.shape, f"{what}: shape {got.shape} vs {ref.shape}"
    assert np.all(err <= 0), f"{what}: max violation {err.max():.3e} (max abs diff {np.abs(got - ref).max():.3e})"


# ---------------------------------------------------------------------------- oracle over many frames
def _oracle_frames(args):
    spec, ocfg, frames, last_only, single_thread = args
    st = O.Store(dict(ocfg, n_layers=1) if last_only else ocfg)

    def work():
        for t in frames:
            q = spec.frame_q(t)
            k, v = spec.frame_kv(t, last_only)
            O.compress_chunk(st, q[None], k[:, None], v[:, None])
    if single_thread:
        from threadpoolctl import threadpool_limits
        with threadpool_limits(limits=1):      # one BLAS thread per worker process
            work()
    else:
        work()
    return st


def oracle_stream(spec: StreamSpec, ocfg: dict, frames, last_only: bool, workers: int | None = None) -> O.Store:
    """Oracle store over `frames` (consecutive from 0 when used for retrieval).  With last_only the
    store holds the last layer only: scores, kept ids and retrieval keys are unchanged by that."""
    frames = list(frames)
    workers = workers or min(len(os.sched_getaffinity(0)), 32)
    spec.out_scale()
    spec.scene_of_frame()
    if workers <= 1 or len(frames) < 4 * workers:
        return _oracle_frames((spec, ocfg, frames, last_only, False))
    parts = np.array_split(np.asarray(frames), workers * 4)
    with ProcessPoolExecutor(max_workers=workers) as ex:
        stores = list(ex.map(_oracle_frames, [(spec, ocfg, p.tolist(), last_only, True) for p in parts if len(p)]))
    out = O.Store(dict(ocfg, n_layers=1) if last_only else ocfg)
    for s in stores:
        for name in ("kept", "page_k", "page_v", "sum_k", "sum_v", "scores"):
            getattr(out, name).extend(getattr(s, name))
    return out


# ---------------------------------------------------------------------------- CUDA path over a stream
class GpuRun:
    """Compresses a whole synthetic stream on the GPU, chunk by chunk, through the C ABI."""

    def __init__(self, name_or_wl, max_frames=None, n_frames=None, device="cuda:0", want_scores=True, options=None,
                 **cfg_over):
        from paper_2605_22269_b200.synth.gpu import GpuStream
        self.wl = workload(name_or_wl) if isinstance(name_or_wl, str) else name_or_wl
        self.spec = self.wl["spec"]
        self.n_frames = n_frames or self.spec.n_frames
        self.cfg = spec_config(self.spec, self.wl, max_frames or self.n_frames, **cfg_over)
        self.ctx = B.MukvContext(self.cfg, device)
        for opt, val in (options or {}).items():
            self.ctx.mukv_set_option(opt, val)
        self.gs = GpuStream(self.spec, device)
        self.device = device
        self.want_scores = want_scores
        self.kept = None
        self.scores = None

    def store_bytes(self) -> int:
        return self.ctx.store.numel()

    def compress(self, chunk=None):
        chunk = chunk or self.wl["chunk"]
        c = self.cfg
        T = self.n_frames
        kept = torch.full((T, c.keep_per_frame), -7, dtype=torch.int32, device=self.device)
        scores = torch.zeros((3, T, c.tokens_per_frame), dtype=torch.float32, device=self.device) \
            if self.want_scores else None
        bufs = {}
        for t0 in range(0, T, chunk):
            n = min(chunk, T - t0)
            if n not in bufs:
                bufs[n] = self.gs.alloc(n)
            q, k, v = bufs[n]
            self.gs.fill(t0, n, q, k, v)
            sc = torch.empty((3, n, c.tokens_per_frame), dtype=torch.float32, device=self.device) \
                if self.want_scores else None
            self.ctx.mukv_compress_chunk(q, k, v, n, t0, kept[t0:t0 + n], sc)
            if self.want_scores:
                scores[:, t0:t0 + n] = sc
        torch.cuda.synchronize()
        self.kept = kept.cpu().numpy()
        self.scores = scores.cpu().numpy() if self.want_scores else None
        return self

    def retrieve(self, qtok_np, offsets, k_seg, k_frm, top_n=0, lam=0.3, mode=B.RETR_SEMI, t_limit=None):
        nq = len(offsets) - 1
        dev = self.device
        qtok = to_device(qtok_np, self.spec.bf16, dev)
        out = dict(seg_idx=torch.full((nq, k_seg), -9, dtype=torch.int32, device=dev),
                   frm_idx=torch.full((nq, k_frm), -9, dtype=torch.int32, device=dev),
                   seg_score=torch.zeros((nq, k_seg), dtype=torch.float32, device=dev),
                   frm_score=torch.zeros((nq, k_frm), dtype=torch.float32, device=dev),
                   counts=torch.zeros((nq, 2), dtype=torch.int32, device=dev))
        self.ctx.mukv_retrieve(qtok, offsets, t_limit, k_seg, k_frm, top_n, lam, mode, out["seg_idx"],
                               out["frm_idx"], out["seg_score"], out["frm_score"], out["counts"])
        return out

    def gather(self, ret, k_frm, with_meta=True):
        nq = ret["frm_idx"].shape[0]
        c = self.cfg
        stride = self.ctx.decode_stride_bytes(k_frm)
        dec = torch.zeros((nq, stride), dtype=torch.uint8, device=self.device)
        meta = torch.full((nq, k_frm * c.keep_per_frame, 2), -5, dtype=torch.int32, device=self.device) \
            if with_meta else None
        self.ctx.mukv_gather(ret["frm_idx"], ret["counts"], nq, k_frm, dec, stride, meta)
        torch.cuda.synchronize()
        shape = (nq, c.n_layers, 2, k_frm * c.keep_per_frame, c.n_kv_heads, c.head_dim)
        dec = dec.view(torch.bfloat16 if self.spec.bf16 else torch.float32).view(shape)
        return dec, meta


def check_frames_against_oracle(run: GpuRun, st: O.Store, frames, full_layers: bool):
    """Kept ids bit-exact, scores within tolerance; with full_layers also page bytes and frame entries."""
    pages = run.ctx.region(0)
    fent = run.ctx.region(2)
    worst = 0.0
    for i, t in enumerate(frames):
        assert run.kept[t].tolist() == st.kept[i].tolist(), f"kept ids differ at frame {t}"
        if run.scores is not None:
            for s in range(3):
                close(run.scores[s, t], st.scores[i][s], f"score[{s}] frame {t}")
            worst = max(worst, float(np.abs(run.scores[2, t] - st.scores[i][2]).max()))
        if full_layers:
            pg = to_numpy_bits(pages[t])                                      # [L][2][kappa][Hkv][D]
            assert pg[:, 0].tobytes() == st.page_k[i].tobytes(), f"K page bytes differ at frame {t}"
            assert pg[:, 1].tobytes() == st.page_v[i].tobytes(), f"V page bytes differ at frame {t}"
            ek, ev = st.frame_entry(i)
            fe = fent[t].cpu().numpy()
            close(fe[:, 0], ek, f"frame entry K {t}")
            close(fe[:, 1], ev, f"frame entry V {t}")
    return worst

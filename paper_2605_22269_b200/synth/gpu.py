"""Device-side generator: same bytes as ``synth.cpu`` (binding of ``synth.cu``)."""
from __future__ import annotations

import ctypes as C
import os

import torch

from .. import build as _build
from .cpu import StreamSpec, normal_table

_LIB = None


def _lib() -> C.CDLL:
    global _LIB
    if _LIB is None:
        path = _build.lib_path("libmukv_synth.so")
        if not os.path.exists(path):
            raise RuntimeError(f"{path} not found: run paper_2605_22269_b200.build.build() first")
        lib = C.CDLL(path)
        vp = C.c_void_p
        lib.mukv_synth_chunk.restype = C.c_int
        lib.mukv_synth_chunk.argtypes = [C.c_uint64, C.c_int, C.c_int, C.c_int, C.c_int, C.c_int, C.c_int,
                                         C.c_float, C.c_float, vp, vp, vp, C.c_longlong, C.c_int, vp, vp, vp, vp]
        _LIB = lib
    return _LIB


class GpuStream:
    """Generates chunks of a ``StreamSpec`` stream directly in device memory."""

    def __init__(self, spec: StreamSpec, device="cuda:0"):
        self.spec = spec
        self.device = torch.device(device)
        self.table = torch.from_numpy(normal_table()).to(self.device)
        self.scale = torch.from_numpy(spec.out_scale()).to(self.device)
        self.scene = torch.from_numpy(spec.scene_of_frame()).to(self.device) if spec.has_scenes else None
        self.dtype = torch.bfloat16 if spec.bf16 else torch.float32

    def alloc(self, n: int):
        s = self.spec
        q = torch.empty((n, s.tokens_per_frame, s.n_q_heads, s.head_dim), dtype=self.dtype, device=self.device)
        k = torch.empty((s.n_layers, n, s.tokens_per_frame, s.n_kv_heads, s.head_dim), dtype=self.dtype,
                        device=self.device)
        v = torch.empty_like(k)
        return q, k, v

    def fill(self, t0: int, n: int, q, k, v, stream=None):
        """Writes frames t0..t0+n-1 into q[:n], k[:, :n] (buffers must have exactly n frames)."""
        s = self.spec
        assert q.shape[0] == n and k.shape[1] == n
        st = (torch.cuda.current_stream() if stream is None else stream).cuda_stream
        rc = _lib().mukv_synth_chunk(s.seed, s.n_layers, s.n_q_heads, s.n_kv_heads, s.head_dim, s.tokens_per_frame,
                                     1 if s.bf16 else 0, s.scene_sigma, s.frame_sigma, self.table.data_ptr(),
                                     self.scale.data_ptr(), None if self.scene is None else self.scene.data_ptr(),
                                     t0, n, q.data_ptr(), k.data_ptr(), v.data_ptr(), st)
        if rc != 0:
            raise RuntimeError(f"mukv_synth_chunk failed with CUDA error {rc}")

    def chunk(self, t0: int, n: int):
        q, k, v = self.alloc(n)
        self.fill(t0, n, q, k, v)
        return q, k, v

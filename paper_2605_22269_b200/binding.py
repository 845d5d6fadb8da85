"""ctypes binding of the C ABI in ``include/mukv.h``.

Argument marshalling only: every step of the path runs in the CUDA library.  PyTorch is used
for device memory (``data_ptr()``) and for the current stream.  If the compiled library is
missing the import of this module still works, but the first use raises ``MukvError``: there
is no CPU fallback.
"""
from __future__ import annotations

import ctypes as C
import os

import numpy as np
import torch

from . import build as _build

BF16, FP32 = 0, 1
RETR_PARALLEL, RETR_HIER, RETR_SEMI = 0, 1, 2
OPT_FLAG_MARGIN, OPT_SCORE_PATH = 0, 1
MAX_QUESTIONS, MAX_TOPK, MAX_TOKENS = 128, 256, 256
NOALLOC_MAX_FRAMES, NOALLOC_MAX_Q_HEADS, NOALLOC_MAX_KV_HEADS = 16, 32, 8

STATUS_NAMES = {0: "MUKV_OK", -1: "MUKV_E_INVALID", -2: "MUKV_E_SHAPE", -3: "MUKV_E_DTYPE", -4: "MUKV_E_ALIGN",
                -5: "MUKV_E_CAPACITY", -6: "MUKV_E_STATE", -7: "MUKV_E_CUDA", -8: "MUKV_E_UNSUPPORTED"}

EXPORTS = ["mukv_store_bytes", "mukv_workspace_bytes", "mukv_create", "mukv_destroy", "mukv_reset", "mukv_set_option",
           "mukv_compress_chunk", "mukv_compress_chunk_scored", "mukv_export_header", "mukv_import",
           "mukv_retrieve3", "mukv_gather3", "mukv_decode3_tokens", "mukv_retrieve", "mukv_gather", "mukv_store_region", "mukv_get_stats",
           "mukv_last_error", "mukv_profile_enable", "mukv_profile_read", "mukv_score_frames_noalloc"]
PROF_KINDS = ["score", "tail", "compact", "segment", "qpool", "scan", "rank", "gather"]


class MukvError(RuntimeError):
    def __init__(self, status: int, message: str):
        super().__init__(f"{STATUS_NAMES.get(status, status)}: {message}")
        self.status = status


class MukvConfig(C.Structure):
    _fields_ = [("n_layers", C.c_int32), ("n_q_heads", C.c_int32), ("n_kv_heads", C.c_int32),
                ("head_dim", C.c_int32), ("tokens_per_frame", C.c_int32), ("keep_per_frame", C.c_int32),
                ("frames_per_segment", C.c_int32), ("max_frames_per_chunk", C.c_int32),
                ("attn_causal", C.c_int32), ("keep_low_freq", C.c_int32),
                ("alpha", C.c_float), ("tie_eps", C.c_float),
                ("dtype", C.c_int32), ("patch_split", C.c_int32), ("grid_width", C.c_int32),
                ("n_score_layers", C.c_int32), ("score_layer_offset", C.c_int32), ("keep_per_segment", C.c_int32),
                ("max_frames", C.c_int64), ("past_frames", C.c_int32), ("reserved", C.c_int32)]


class MukvRetrParams(C.Structure):
    _fields_ = [("k_patch", C.c_int32), ("k_frm", C.c_int32), ("k_seg", C.c_int32),
                ("lambda_patch", C.c_float), ("lambda_frm", C.c_float), ("lambda_seg", C.c_float),
                ("top_n", C.c_int32), ("mode", C.c_int32)]


class MukvStats(C.Structure):
    _fields_ = [("frames", C.c_int64), ("segments", C.c_int64), ("kept_tokens", C.c_int64),
                ("page_bytes", C.c_int64), ("store_bytes_used", C.c_int64), ("refined_frames", C.c_int64),
                ("refined_questions", C.c_int64), ("kernel_launches", C.c_int64),
                ("device_status", C.c_int32), ("reserved", C.c_int32)]


class MukvStoreHeader(C.Structure):
    _fields_ = [("magic", C.c_uint32), ("version", C.c_uint32), ("cfg", MukvConfig), ("frames", C.c_int64),
                ("store_bytes", C.c_uint64)]


_LIB = None


def load_library(path: str | None = None) -> C.CDLL:
    """Loads libmukv.so (built in-tree by ``build.build()``) and declares the prototypes."""
    global _LIB
    if _LIB is not None and path is None:
        return _LIB
    path = path or _build.lib_path("libmukv.so")
    if not os.path.exists(path):
        raise MukvError(-8, f"{path} not found: run paper_2605_22269_b200.build.build() (nvcc, sm_100a) first")
    lib = C.CDLL(path)
    vp, i32, i64, f32 = C.c_void_p, C.c_int32, C.c_int64, C.c_float
    cfgp = C.POINTER(MukvConfig)
    lib.mukv_store_bytes.restype = C.c_size_t
    lib.mukv_store_bytes.argtypes = [cfgp]
    lib.mukv_workspace_bytes.restype = C.c_size_t
    lib.mukv_workspace_bytes.argtypes = [cfgp]
    lib.mukv_create.restype = i32
    lib.mukv_create.argtypes = [cfgp, vp, C.c_size_t, vp, C.c_size_t, C.POINTER(vp)]
    lib.mukv_destroy.restype = None
    lib.mukv_destroy.argtypes = [vp]
    lib.mukv_reset.restype = i32
    lib.mukv_reset.argtypes = [vp, vp]
    lib.mukv_set_option.restype = i32
    lib.mukv_set_option.argtypes = [vp, i32, C.c_double]
    lib.mukv_compress_chunk.restype = i32
    lib.mukv_compress_chunk.argtypes = [vp, vp, vp, vp, i32, i64, vp, vp, vp]
    lib.mukv_compress_chunk_scored.restype = i32
    lib.mukv_compress_chunk_scored.argtypes = [vp, vp, vp, vp, i32, i64, vp, vp]
    lib.mukv_export_header.restype = i32
    lib.mukv_export_header.argtypes = [vp, C.POINTER(MukvStoreHeader)]
    lib.mukv_import.restype = i32
    lib.mukv_import.argtypes = [C.POINTER(MukvStoreHeader), vp, C.c_size_t, vp, C.c_size_t, C.POINTER(vp)]
    lib.mukv_retrieve.restype = i32
    lib.mukv_retrieve.argtypes = [vp, vp, C.POINTER(i32), C.POINTER(i64), i32, i32, i32, i32, f32, i32,
                                  vp, vp, vp, vp, vp, vp]
    lib.mukv_retrieve3.restype = i32
    lib.mukv_retrieve3.argtypes = [vp, vp, C.POINTER(i32), C.POINTER(i64), i32, C.POINTER(MukvRetrParams),
                                   vp, vp, vp, vp, vp, vp, vp, vp]
    lib.mukv_decode3_tokens.restype = i64
    lib.mukv_decode3_tokens.argtypes = [vp, i32, i32, i32]
    lib.mukv_gather3.restype = i32
    lib.mukv_gather3.argtypes = [vp, vp, vp, vp, vp, i32, i32, i32, i32, vp, i64, vp, vp, vp]
    lib.mukv_gather.restype = i32
    lib.mukv_gather.argtypes = [vp, vp, vp, i32, i32, vp, i64, vp, vp]
    lib.mukv_store_region.restype = vp
    lib.mukv_store_region.argtypes = [vp, i32, C.POINTER(C.c_size_t)]
    lib.mukv_get_stats.restype = i32
    lib.mukv_get_stats.argtypes = [vp, C.POINTER(MukvStats), vp]
    lib.mukv_profile_enable.restype = i32
    lib.mukv_profile_enable.argtypes = [vp, i32]
    lib.mukv_profile_read.restype = i32
    lib.mukv_profile_read.argtypes = [vp, C.POINTER(C.c_double), C.POINTER(i64)]
    lib.mukv_score_frames_noalloc.restype = i32
    lib.mukv_score_frames_noalloc.argtypes = [cfgp, vp, vp, i32, vp, vp, vp]
    lib.mukv_last_error.restype = C.c_char_p
    lib.mukv_last_error.argtypes = [vp]
    if path == _build.lib_path("libmukv.so"):
        _LIB = lib
    return lib


def _ptr(t) -> int | None:
    return None if t is None else t.data_ptr()


def _stream(stream) -> int:
    s = torch.cuda.current_stream() if stream is None else stream
    return s.cuda_stream


def make_config(*, n_layers, n_q_heads, n_kv_heads, head_dim, tokens_per_frame, keep_per_frame,
                frames_per_segment, max_frames_per_chunk, max_frames, dtype=BF16, alpha=0.7, tie_eps=1e-6,
                attn_causal=0, keep_low_freq=0, patch_split=0, grid_width=0, n_score_layers=0,
                score_layer_offset=0, keep_per_segment=0, past_frames=0) -> MukvConfig:
    return MukvConfig(n_layers, n_q_heads, n_kv_heads, head_dim, tokens_per_frame, keep_per_frame,
                      frames_per_segment, max_frames_per_chunk, attn_causal, keep_low_freq,
                      alpha, tie_eps, dtype, patch_split, grid_width, n_score_layers, score_layer_offset, keep_per_segment, max_frames, past_frames, 0)


def mukv_score_frames_noalloc(cfg: MukvConfig, q, k_last, n_frames: int, kept_out=None, scores_out=None,
                              stream=None) -> None:
    """Scores ``n_frames`` frames with the library's built-in scratch: no context, no workspace and no
    device allocation (see include/mukv.h).  For callers that cannot allocate device memory."""
    lib = load_library()
    st = lib.mukv_score_frames_noalloc(C.byref(cfg), _ptr(q), _ptr(k_last), n_frames, _ptr(kept_out),
                                       _ptr(scores_out), _stream(stream))
    if st != 0:
        raise MukvError(st, (lib.mukv_last_error(None) or b"").decode())


class MukvContext:
    """Owns the torch buffers behind one ``mukv_ctx`` and forwards calls to the C ABI."""

    def __init__(self, cfg: MukvConfig, device="cuda:0", _header=None, _store=None):
        self.lib = load_library()
        self.cfg = cfg
        self.device = torch.device(device)
        sb = self.lib.mukv_store_bytes(C.byref(cfg))
        wb = self.lib.mukv_workspace_bytes(C.byref(cfg))
        if sb == 0 or wb == 0:
            # let mukv_create produce the message
            sb = wb = 256
        with torch.cuda.device(self.device):
            self.store = torch.empty(sb, dtype=torch.uint8, device=self.device) if _store is None else _store
            self.workspace = torch.empty(wb, dtype=torch.uint8, device=self.device)
            h = C.c_void_p()
            if _header is None:
                st = self.lib.mukv_create(C.byref(cfg), self.store.data_ptr(), sb, self.workspace.data_ptr(), wb,
                                          C.byref(h))
            else:
                st = self.lib.mukv_import(C.byref(_header), self.store.data_ptr(), self.store.numel(),
                                          self.workspace.data_ptr(), wb, C.byref(h))
        if st != 0:
            raise MukvError(st, (self.lib.mukv_last_error(None) or b"").decode())
        self.handle = h
        self.C = cfg.n_kv_heads * cfg.head_dim
        self.torch_dtype = torch.bfloat16 if cfg.dtype == BF16 else torch.float32

    @classmethod
    def from_copy(cls, header: MukvStoreHeader, store: torch.Tensor) -> "MukvContext":
        """mukv_import: a context over `store`, a uint8 device tensor holding a copy of an exported store."""
        cfg = MukvConfig.from_buffer_copy(header.cfg)
        return cls(cfg, store.device, _header=header, _store=store)

    def mukv_export_header(self) -> MukvStoreHeader:
        h = MukvStoreHeader()
        self._check(self.lib.mukv_export_header(self.handle, C.byref(h)))
        return h

    def mukv_compress_chunk_scored(self, select_scores, k, v, n_frames: int, first_frame: int, kept_out=None,
                                   stream=None):
        self._check(self.lib.mukv_compress_chunk_scored(self.handle, _ptr(select_scores), _ptr(k), _ptr(v), n_frames,
                                                        first_frame, _ptr(kept_out), _stream(stream)))

    def close(self):
        if getattr(self, "handle", None):
            self.lib.mukv_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def _check(self, st: int):
        if st != 0:
            raise MukvError(st, (self.lib.mukv_last_error(self.handle) or b"").decode())

    # ---- the calls of include/mukv.h --------------------------------------------------------
    def mukv_reset(self, stream=None):
        self._check(self.lib.mukv_reset(self.handle, _stream(stream)))

    def mukv_set_option(self, option: int, value: float):
        self._check(self.lib.mukv_set_option(self.handle, option, float(value)))

    def mukv_compress_chunk(self, q, k, v, n_frames: int, first_frame: int, kept_out=None, scores_out=None,
                            stream=None):
        self._check(self.lib.mukv_compress_chunk(self.handle, _ptr(q), _ptr(k), _ptr(v), n_frames, first_frame,
                                                 _ptr(kept_out), _ptr(scores_out), _stream(stream)))

    def mukv_retrieve(self, qtok, q_offsets, t_limit, k_seg: int, k_frm: int, top_n: int, lambda_frm: float,
                      mode: int, seg_idx, frm_idx, seg_score, frm_score, counts, stream=None):
        offs = np.ascontiguousarray(q_offsets, dtype=np.int32)
        nq = offs.shape[0] - 1
        tl = None if t_limit is None else np.ascontiguousarray(t_limit, dtype=np.int64)
        self._check(self.lib.mukv_retrieve(
            self.handle, _ptr(qtok), offs.ctypes.data_as(C.POINTER(C.c_int32)),
            None if tl is None else tl.ctypes.data_as(C.POINTER(C.c_int64)),
            nq, k_seg, k_frm, top_n, lambda_frm, mode, _ptr(seg_idx), _ptr(frm_idx), _ptr(seg_score),
            _ptr(frm_score), _ptr(counts), _stream(stream)))

    def mukv_retrieve3(self, qtok, q_offsets, t_limit, params: MukvRetrParams, seg_idx, frm_idx, patch_idx,
                       seg_score, frm_score, patch_score, counts, stream=None):
        offs = np.ascontiguousarray(q_offsets, dtype=np.int32)
        nq = offs.shape[0] - 1
        tl = None if t_limit is None else np.ascontiguousarray(t_limit, dtype=np.int64)
        self._check(self.lib.mukv_retrieve3(
            self.handle, _ptr(qtok), offs.ctypes.data_as(C.POINTER(C.c_int32)),
            None if tl is None else tl.ctypes.data_as(C.POINTER(C.c_int64)), nq, C.byref(params),
            _ptr(seg_idx), _ptr(frm_idx), _ptr(patch_idx), _ptr(seg_score), _ptr(frm_score), _ptr(patch_score),
            _ptr(counts), _stream(stream)))

    def mukv_decode3_tokens(self, k_seg: int, k_frm: int, k_patch: int) -> int:
        return int(self.lib.mukv_decode3_tokens(self.handle, k_seg, k_frm, k_patch))

    def mukv_gather3(self, seg_idx, frm_idx, patch_idx, counts, nq: int, k_seg: int, k_frm: int, k_patch: int, decode,
                     decode_stride_bytes: int, ntok, tok_meta=None, stream=None):
        self._check(self.lib.mukv_gather3(self.handle, _ptr(seg_idx), _ptr(frm_idx), _ptr(patch_idx), _ptr(counts), nq,
                                          k_seg, k_frm, k_patch, _ptr(decode), decode_stride_bytes, _ptr(ntok),
                                          _ptr(tok_meta), _stream(stream)))

    def mukv_gather(self, frm_idx, counts, nq: int, k_frm: int, decode, decode_stride_bytes: int, tok_meta=None,
                    stream=None):
        self._check(self.lib.mukv_gather(self.handle, _ptr(frm_idx), _ptr(counts), nq, k_frm, _ptr(decode),
                                         decode_stride_bytes, _ptr(tok_meta), _stream(stream)))

    def mukv_get_stats(self, stream=None) -> MukvStats:
        s = MukvStats()
        self._check(self.lib.mukv_get_stats(self.handle, C.byref(s), _stream(stream)))
        return s

    def mukv_profile_enable(self, on: bool):
        self._check(self.lib.mukv_profile_enable(self.handle, 1 if on else 0))

    def mukv_profile_read(self) -> dict:
        """{kind: (milliseconds, launches)} since the last read."""
        ms = (C.c_double * len(PROF_KINDS))()
        n = (C.c_int64 * len(PROF_KINDS))()
        self._check(self.lib.mukv_profile_read(self.handle, ms, n))
        return {k: (ms[i], n[i]) for i, k in enumerate(PROF_KINDS)}

    # ---- views into the store (tests, inspection) ---------------------------------------------
    def region(self, which: int) -> torch.Tensor:
        """A torch view of one store region (see mukv_store_region)."""
        n = C.c_size_t()
        p = self.lib.mukv_store_region(self.handle, which, C.byref(n))
        if not p:
            raise MukvError(-1, f"unknown region {which}")
        off = p - self.store.data_ptr()
        raw = self.store[off:off + n.value]
        c = self.cfg
        T = c.max_frames
        segs = (T + c.frames_per_segment - 1) // c.frames_per_segment
        if which == 0 and c.keep_per_segment > 0:
            return raw.view(self.torch_dtype)              # packed pages of different lengths: see the page table
        if which == 0:
            return raw.view(self.torch_dtype).view(T, c.n_layers, 2, c.keep_per_frame, c.n_kv_heads, c.head_dim)
        if which == 1:
            return raw.view(torch.int32).view(T, c.tokens_per_frame if c.keep_per_segment > 0 else c.keep_per_frame)
        if which == 10:
            return raw.view(torch.int32).view(T)
        if which == 2:
            return raw.view(torch.float32).view(T, c.n_layers, 2, self.C)
        if which == 3:
            return raw.view(torch.float32).view(segs, c.n_layers, 2, self.C)
        if which == 4:
            return raw.view(torch.float32).view(T, self.C)
        if which == 5:
            return raw.view(torch.float32).view(segs, self.C)
        if which == 8:
            return raw.view(torch.float32).view(T, c.patch_split ** 2, self.C)
        if which == 9:
            return raw.view(torch.int32).view(T, c.patch_split ** 2)
        return raw.view(torch.int64).view(T)

    def decode_stride_bytes(self, k_frm: int) -> int:
        c = self.cfg
        es = 2 if c.dtype == BF16 else 4
        return c.n_layers * 2 * k_frm * c.keep_per_frame * self.C * es

"""The C ABI: the library loads, exports what include/mukv.h declares, and its host-side checks
work without a GPU (no kernel is launched here)."""
import ctypes as C
import os
import re

import pytest

from paper_2605_22269_b200 import binding as B
from paper_2605_22269_b200 import build as BUILD

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    BUILD.build()
    return B.load_library()


def good_config(**over):
    kw = dict(n_layers=28, n_q_heads=28, n_kv_heads=4, head_dim=128, tokens_per_frame=196, keep_per_frame=49,
              frames_per_segment=16, max_frames_per_chunk=16, max_frames=10800)
    kw.update(over)
    return B.make_config(**kw)


def test_exports_match_header(lib):
    text = open(os.path.join(ROOT, "include", "mukv.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    declared = sorted(set(re.findall(r"\b(mukv_[a-z_0-9]+)\s*\(", text)))
    assert declared == sorted(B.EXPORTS)
    for name in declared:
        assert hasattr(lib, name), f"{name} is declared but not exported"
    synth = C.CDLL(BUILD.lib_path("libmukv_synth.so"))
    assert hasattr(synth, "mukv_synth_chunk")


def test_struct_sizes_match_header():
    assert C.sizeof(B.MukvConfig) == 88 and C.sizeof(B.MukvStats) == 72 and C.sizeof(B.MukvStoreHeader) == 112
    assert C.sizeof(B.MukvRetrParams) == 32


def test_store_size_of_the_three_hour_stream(lib):
    cfg = good_config()
    sb = lib.mukv_store_bytes(C.byref(cfg))
    page = 28 * 2 * 49 * 4 * 128 * 2
    assert page == 2_809_856
    pooled = 10800 * 28 * 2 * 512 * 4
    assert 10800 * page + pooled < sb < 10800 * page + pooled + 200e6       # ~30.35 GB of pages + 1.24 GB pooled
    assert lib.mukv_workspace_bytes(C.byref(cfg)) < 64e6


@pytest.mark.parametrize("over", [dict(head_dim=96), dict(n_q_heads=30), dict(tokens_per_frame=300),
                                  dict(keep_per_frame=0), dict(keep_per_frame=197), dict(alpha=1.5),
                                  dict(dtype=7), dict(max_frames=0), dict(n_kv_heads=3, n_q_heads=27),
                                  dict(frames_per_segment=0), dict(patch_split=5, grid_width=14),
                                  dict(patch_split=2, grid_width=13), dict(patch_split=2, grid_width=0), dict(past_frames=2), dict(past_frames=-1),
                                  dict(keep_per_segment=100000), dict(n_score_layers=20, score_layer_offset=9)])
def test_bad_configs_are_rejected_on_the_host(lib, over):
    cfg = good_config(**over)
    assert lib.mukv_store_bytes(C.byref(cfg)) == 0
    h = C.c_void_p()
    st = lib.mukv_create(C.byref(cfg), 4096, 1 << 20, 8192, 1 << 20, C.byref(h))
    assert st in (-2, -3) and not h.value
    assert len(lib.mukv_last_error(None)) > 0


def test_create_argument_errors(lib):
    cfg = good_config()
    h = C.c_void_p()
    assert lib.mukv_create(C.byref(cfg), None, 0, None, 0, C.byref(h)) == -1
    assert lib.mukv_create(C.byref(cfg), 4096 + 8, 1 << 40, 8192, 1 << 40, C.byref(h)) == -4      # misaligned
    assert lib.mukv_create(C.byref(cfg), 4096, 1024, 8192, 1024, C.byref(h)) == -5                 # too small
    assert b"store needs" in lib.mukv_last_error(None)
    assert lib.mukv_compress_chunk(None, None, None, None, 1, 0, None, None, None) == -1
    assert lib.mukv_gather(None, None, None, 1, 1, None, 0, None, None) == -1


def test_missing_library_fails_loudly(tmp_path):
    with pytest.raises(B.MukvError):
        B.load_library(str(tmp_path / "libmukv.so"))

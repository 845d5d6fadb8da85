"""The seeded input generators: CPU properties, and CPU == GPU bytes."""
import numpy as np
import pytest

from paper_2605_22269_b200.synth import cpu
from paper_2605_22269_b200.synth.cpu import StreamSpec, workload


def test_normals_are_standard_normal():
    x = cpu.normals(cpu.stream_key(7, 1, 3), 400_000).astype(np.float64)
    assert abs(x.mean()) < 0.01 and abs(x.std() - 1.0) < 0.01
    assert abs(np.mean(x ** 4) - 3.0) < 0.1 and np.abs(x).max() > 3.5
    # a sub-range equals the same elements of the full range
    assert np.array_equal(cpu.normals(cpu.stream_key(7, 1, 3), 1000, 4 * 50), x[200:1200].astype(np.float32))


def test_bf16_rounding_is_nearest_even():
    x = np.array([1.0, 1.0 + 2 ** -8, 1.0 + 2 ** -7, 1.0 + 3 * 2 ** -8, -2.5, 0.0], dtype=np.float32)
    got = cpu.bf16_bits_to_f32(cpu.to_bf16_bits(x))
    assert got.tolist() == [1.0, 1.0, 1.0 + 2 ** -7, 1.0 + 2 ** -6, -2.5, 0.0]


def test_stream_structure():
    wl = workload("stream_3h")
    spec = wl["spec"]
    sc = spec.scene_of_frame()
    lens = np.bincount(sc)
    assert sc[0] == 0 and np.all(np.diff(sc) >= 0) and lens[:-1].min() >= 10 and lens.max() <= 60
    scale = spec.out_scale()
    assert scale.shape == (28, 4, 128) and np.all((scale == 8.0).sum(axis=2) == 4)
    k, v = spec.frame_kv(123, last_layer_only=True)
    k_full, v_full = StreamSpec(seed=4, n_layers=2, n_frames=10800, scene_sigma=1.0, frame_sigma=0.5,
                                scene_min=10, scene_max=60).frame_kv(123)
    assert k.shape == (1, 196, 4, 128) and k.dtype == np.uint16 and k_full.shape == (2, 196, 4, 128)
    # frames of one scene share their mean: the token-mean of K correlates within a scene, not across
    def mean_key(t):
        return cpu.bf16_bits_to_f32(spec.frame_kv(t, True)[0]).mean(axis=1).ravel()
    a, b = mean_key(0), mean_key(1)
    far = mean_key(int(np.nonzero(sc == 5)[0][0]))
    assert np.corrcoef(a, b)[0, 1] > 0.5 and abs(np.corrcoef(a, far)[0, 1]) < 0.3


def test_chunking_is_irrelevant_and_questions_are_ragged():
    spec = workload("tiny")["spec"]
    q, k, v = spec.chunk(0, 8)
    q2, k2, v2 = spec.chunk(3, 2)
    assert np.array_equal(k[:, 3:5], k2) and np.array_equal(q[3:5], q2) and q.dtype == np.float32
    toks, offs, scenes = workload("stream_3h")["spec"].questions(64, 16, 64)
    n = np.diff(offs)
    assert n.min() >= 16 and n.max() <= 64 and len(set(n.tolist())) > 10 and toks.shape == (offs[-1], 28, 128)


@pytest.mark.gpu
@pytest.mark.parametrize("name,frames", [("tiny", [0, 5]), ("chunk7b", [3]), ("stream_3h", [0, 4321])])
def test_gpu_generator_matches_cpu(name, frames):
    import torch
    from paper_2605_22269_b200.synth.gpu import GpuStream
    from tests.harness import to_numpy_bits
    spec = workload(name)["spec"]
    gs = GpuStream(spec)
    for t in frames:
        q, k, v = gs.chunk(t, 2)
        torch.cuda.synchronize()
        cq, ck, cv = spec.chunk(t, 2)
        assert to_numpy_bits(q).tobytes() == cq.tobytes()
        assert to_numpy_bits(k).tobytes() == ck.tobytes()
        assert to_numpy_bits(v).tobytes() == cv.tobytes()

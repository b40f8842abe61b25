"""The seeded input generators: deterministic, right shapes, and the structure the workloads promise."""
import numpy as np

from paper_2602_14236_b200 import synth


def test_hash_is_deterministic_and_uniform():
    a = synth.uniform01(1, 2, np.arange(100000))
    assert np.array_equal(a, synth.uniform01(1, 2, np.arange(100000)))
    assert abs(a.mean() - 0.5) < 0.01 and a.min() >= 0 and a.max() < 1
    assert not np.array_equal(a, synth.uniform01(1, 3, np.arange(100000)))
    n = synth.normal(4, 0, 200000)
    assert abs(n.mean()) < 0.01 and abs(n.std() - 1) < 0.01


def test_workload_shapes():
    for i, wl in synth.WORKLOADS.items():
        fr = synth.frames(i, T=2)
        assert fr.shape == (2, wl.H, wl.W, 3) and fr.dtype == np.uint8
    assert synth.WORKLOADS[4].n_tok == 2880 and synth.WORKLOADS[3].n_tok == 576


def test_pan_is_an_exact_window_shift_and_static_frames_repeat():
    fr = synth.frames(3, T=3, t0=10)
    assert np.array_equal(fr[0][:, 3:], fr[1][:, :-3])
    fr5 = synth.frames(5, T=2, t0=5)
    assert np.array_equal(fr5[0], fr5[1])                 # segment 0 is static
    fr5 = synth.frames(5, T=2, t0=305)
    assert np.array_equal(fr5[0][:, 1:], fr5[1][:, :-1])  # segment 1 pans 1 px/frame
    fr5 = synth.frames(5, T=2, t0=605)
    assert np.array_equal(fr5[0][:, 8:], fr5[1][:, :-8])  # segment 2 pans 8 px/frame


def test_frames_are_reproducible_from_any_offset():
    assert np.array_equal(synth.frames(1, T=3)[2], synth.frames(1, T=1, t0=2)[0])
    assert np.array_equal(synth.frames(2, T=3)[2], synth.frames(2, T=1, t0=2)[0])


def test_kv_statistics_and_outliers():
    K, V = synth.kv_numpy(1, 0, L=1, n_tok=64)
    assert K.shape == (1, 64, 4096) and K.dtype == np.float16
    assert abs(float(K.astype(np.float64).std()) - 1.0) < 0.02
    assert not np.array_equal(K, V)
    K2, _ = synth.kv_numpy(2, 0, L=1, n_tok=64)
    assert 1.25 < float(K2.astype(np.float64).std()) < 1.35   # sqrt(0.99 + 0.01*64)

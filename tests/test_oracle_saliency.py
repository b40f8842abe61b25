"""Pins of the oracle's spatial branch (Sec. III-B, Eq. 7): Canny edges, LAB colour variance, patch means."""
import os

import numpy as np
import pytest
from scipy import ndimage

import oracle
from paper_2602_14236_b200 import synth

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _golden(name):
    rows = {}
    with open(os.path.join(GOLD, name)) as f:
        for line in f:
            if line.startswith("#") or not line.strip():
                continue
            parts = line.split()
            rows[parts[0]] = [float(v) for v in parts[1:]]
    return rows


def test_canny_constant_image_has_no_edges():
    assert not oracle.canny(np.full((32, 40), 93, np.uint8)).any()


def test_canny_vertical_step_is_one_line_left_of_the_step():
    gold = _golden("canny_step_profile.txt")
    c = 20
    g = np.zeros((32, 48), np.uint8)
    g[:, c:] = 96
    E, cls = oracle.canny(g, 50, 150, want_cls=True)
    expect = np.zeros_like(E)
    expect[:, c + int(gold["edge_column_offset"][0])] = 1
    assert np.array_equal(E, expect)
    assert np.all(cls[:, c - 1] == 2)
    # the blurred profile and Sobel response of the worked example, by library routines
    k = np.array([1, 4, 6, 4, 1])
    blur = (ndimage.correlate(g.astype(np.int64), np.outer(k, k), mode="nearest") + 128) >> 8
    assert list(blur[10, c - 3:c + 3]) == gold["blur"]
    gx = ndimage.correlate(blur, np.array([[-1, 0, 1], [-2, 0, 2], [-1, 0, 1]]), mode="nearest")
    assert list(gx[10, c - 3:c + 3]) == gold["gx"]


def test_canny_horizontal_step_is_one_line_above_the_step():
    g = np.zeros((40, 32), np.uint8)
    g[17:, :] = 96
    expect = np.zeros((40, 32), np.uint8)
    expect[16, :] = 1
    assert np.array_equal(oracle.canny(g), expect)


def test_canny_thresholds():
    g = np.zeros((32, 48), np.uint8)
    g[:, 20:] = 16                       # gx peaks at 40 < lo
    assert not oracle.canny(g).any()
    g[:, 20:] = 32                       # gx peaks at 80: weak only, no strong pixel to attach to
    E, cls = oracle.canny(g, want_cls=True)
    assert not E.any() and np.all(cls[:, 19] == 1)
    assert oracle.canny(g, 50, 80).any()  # hi = 80 makes the same line strong (m >= hi^2 inclusive)
    assert not oracle.canny(g, 50, 81).any()
    assert np.all(oracle.canny(g, 80, 81, want_cls=True)[1][:, 19] == 1)   # m >= lo^2 inclusive
    assert not oracle.canny(g, 81, 200, want_cls=True)[1].any()


def test_canny_hysteresis_attaches_touching_weak_segments_only():
    g = np.zeros((64, 64), np.uint8)
    amp = np.clip(96 - 2 * (np.arange(64) - 20), 32, 96)      # step height fades from 96 to 32 down the rows
    g[:, 20:40] = amp[:, None]
    g[:, 40:] = amp[:, None]
    g[44:, 50:] += 32                    # a separate weak-only step, nowhere near a strong pixel
    E, cls = oracle.canny(g, want_cls=True)
    line = cls[:, 19:21].max(axis=1)      # rounding in the blur moves the ridge between columns 19 and 20
    assert (line == 2).any() and (line == 1).any() and (line > 0).all()
    assert (E[:, 19] | E[:, 20]).all()   # the weak tail of the line hangs on its strong head
    weak_far = (cls == 1) & (np.arange(64)[None, :] > 40)
    assert weak_far.any() and not E[weak_far].any()


def _propagate(cls):
    """Iterative 8-neighbour dilation restricted to kept pixels, to the fixed point."""
    E = cls == 2
    kept = cls > 0
    while True:
        grown = ndimage.binary_dilation(E, structure=np.ones((3, 3), bool)) & kept
        if np.array_equal(grown, E):
            return E.astype(np.uint8)
        E = grown


@pytest.mark.parametrize("seed", [1, 2, 3])
def test_canny_flood_fill_equals_iterative_propagation(seed):
    rng = np.random.default_rng(seed)
    g = ndimage.uniform_filter(rng.integers(0, 256, (48, 56)).astype(np.float64), 3)
    g = np.clip(g * 1.5 - 60, 0, 255).astype(np.uint8)
    E, cls = oracle.canny(g, 30, 110, want_cls=True)
    assert (cls == 1).any() and (cls == 2).any()
    assert np.array_equal(E, _propagate(cls))


def _canny_cls_numpy(g, lo, hi):
    """Steps (i)-(v) restated with library correlations and whole-array operations."""
    k = np.array([1, 4, 6, 4, 1])
    B = (ndimage.correlate(g.astype(np.int64), np.outer(k, k), mode="nearest") + 128) >> 8
    gx = ndimage.correlate(B, np.array([[-1, 0, 1], [-2, 0, 2], [-1, 0, 1]]), mode="nearest")
    gy = ndimage.correlate(B, np.array([[-1, -2, -1], [0, 0, 0], [1, 2, 1]]), mode="nearest")
    m = gx * gx + gy * gy
    mp = np.pad(m, 1)
    h, w = g.shape

    def nb(dy, dx):
        return mp[1 + dy:1 + dy + h, 1 + dx:1 + dx + w]

    ax, ay = np.abs(gx), np.abs(gy)
    horiz = 32768 * ay <= 13573 * ax
    vert = ~horiz & (32768 * ax <= 13573 * ay)
    diag = ~horiz & ~vert & ((gx > 0) == (gy > 0))
    anti = ~horiz & ~vert & ~diag
    mneg = np.select([horiz, vert, diag, anti], [nb(0, -1), nb(-1, 0), nb(-1, -1), nb(-1, 1)])
    mpos = np.select([horiz, vert, diag, anti], [nb(0, 1), nb(1, 0), nb(1, 1), nb(1, -1)])
    keep = (m > mneg) & (m >= mpos)
    return np.where(keep & (m >= hi * hi), 2, np.where(keep & (m >= lo * lo), 1, 0)).astype(np.uint8)


def test_canny_classes_match_library_restatement_on_a_workload_frame():
    g = oracle.gray(synth.frames(2, T=1)[0][:112, :140])
    _, cls = oracle.canny(g, 50, 150, want_cls=True)
    assert np.array_equal(cls, _canny_cls_numpy(g, 50, 150))
    assert (cls == 2).any() and (cls == 1).any()


def test_canny_diagonal_sectors():
    """A 45-degree step keeps a thin staircase (the two cells of each stair tie and are not compared with
    each other by the diagonal test), the same on either diagonal orientation."""
    y, x = np.mgrid[0:48, 0:48]
    for img in (np.where(x + y >= 48, 120, 0), np.where(x - y >= 0, 120, 0)):
        E = oracle.canny(img.astype(np.uint8))
        assert np.all(E[6:-6].sum(axis=1) == 2)
        assert np.all(E[:, 8:-8].sum(axis=0) == 2)


def test_lab_reference_colours():
    path = os.path.join(GOLD, "lab_reference.txt")
    rows = [l.split() for l in open(path) if not l.startswith("#") and l.strip()]
    for r in rows:
        rgb = np.array([[int(v) for v in r[:3]]], np.uint8)
        lab = oracle.rgb_to_lab(rgb)[0]
        assert np.allclose(lab, [float(v) for v in r[3:]], atol=2e-3), r


def test_lab_neutral_axis_and_monotone_lightness():
    grey = np.repeat(np.arange(256, dtype=np.uint8)[:, None], 3, axis=1)
    lab = oracle.rgb_to_lab(grey)
    assert np.all(np.abs(lab[:, 1:]) < 1e-4)
    assert np.all(np.diff(lab[:, 0]) > 0)
    # both branches of the transfer curve and of f(t): dark values are on the linear pieces
    assert lab[1, 0] == pytest.approx(903.3 * (1 / 255 / 12.92), rel=1e-3)


def test_color_contrast_constant_and_two_valued_windows():
    img = np.empty((24, 30, 3), np.uint8)
    img[:] = (90, 140, 60)
    assert np.all(oracle.color_contrast(img) < 1e-12)     # rounding of the 49-sample mean only
    img[:, 15:] = (100, 150, 80)
    labs = oracle.rgb_to_lab(np.array([[90, 140, 60], [100, 150, 80]], np.uint8))
    d2 = float(((labs[0] - labs[1]) ** 2).sum())
    C = oracle.color_contrast(img, 3, 16.0)
    for x in range(30):
        k = np.clip(x + 3 - 15 + 1, 0, 7)          # window columns on the right-hand colour
        p = k / 7.0
        assert np.allclose(C[:, x], min(1.0, np.sqrt(p * (1 - p) * d2) / 16.0), atol=1e-12)


def test_color_contrast_saturates():
    y, x = np.mgrid[0:28, 0:28]
    img = np.where(((x + y) % 2)[:, :, None] == 0, np.array([255, 0, 0]), np.array([0, 0, 255])).astype(np.uint8)
    assert np.all(oracle.color_contrast(img) == 1.0)


def test_patch_scores_closed_forms():
    p = oracle.Params()
    # (a) edge term only: one full-height edge line -> k = 14 edge pixels per touched patch, s = w_e * 14/196
    g = np.zeros((42, 56), np.uint8)
    g[:, 20:] = 96
    rgb = np.repeat(g[:, :, None], 3, axis=2)
    pe = oracle.Params(w_edge=0.5, w_color=0.0)
    s = oracle.saliency(rgb, pe).reshape(3, 4)
    expect = np.zeros((3, 4))
    expect[:, 1] = 0.5 * 14 / 196.0                # column 19 lies in patch column 1
    assert np.allclose(s, expect, atol=1e-15)
    # (b) everything saturates -> S = 1 everywhere -> s = 1
    y, x = np.mgrid[0:28, 0:28]
    img = np.where(((x + y) % 2)[:, :, None] == 0, np.array([255, 0, 0]), np.array([0, 0, 255])).astype(np.uint8)
    assert np.allclose(oracle.saliency(img, oracle.Params(w_edge=1.0, w_color=1.0)), 1.0)
    # (c) the map is the clamped blend and the score its patch mean
    fr = synth.frames(2, T=1)[0][:56, :70]
    s, S = oracle.saliency(fr, p, want_map=True)
    E = oracle.canny(oracle.gray(fr), p.canny_lo, p.canny_hi)
    C = oracle.color_contrast(fr, p.var_radius, p.sigma_ref)
    assert np.allclose(S, np.clip(0.5 * E + 0.5 * C, 0, 1), atol=1e-15)
    assert np.allclose(s.reshape(4, 5), S.reshape(4, 14, 5, 14).mean(axis=(1, 3)), atol=1e-14)


def test_box_down2_rounds_half_up():
    img = np.zeros((2, 2, 3), np.uint8)
    img[0, 0] = (1, 2, 255)
    img[0, 1] = (0, 0, 255)
    img[1, 0] = (0, 0, 255)
    img[1, 1] = (0, 0, 254)
    assert list(oracle.box_down2(img)[0, 0]) == [0, 1, 255]


def test_saliency_batch_matches_single_frames():
    fr = synth.frames(2, T=2)[:, :56, :56]
    s = oracle.saliency(fr)
    for b in range(2):
        assert np.array_equal(s[b], oracle.saliency(fr[b]))


# ----------------------------------------------------------------------------- frame-adaptive colour term
def test_color_variance_is_what_the_fixed_reading_normalises():
    fr = synth.frames(2, T=1)[0][40:110, 30:120]
    V = oracle.color_variance(fr)
    assert np.array_equal(oracle.color_contrast(fr, sigma_ref=16.0), np.minimum(1.0, np.sqrt(V) / 16.0))
    # library restatement of V: uniform filters over the clamp-extended LAB planes
    lab = oracle.rgb_to_lab(fr).reshape(fr.shape[0], fr.shape[1], 3)
    want = np.zeros(fr.shape[:2])
    for c in range(3):
        m1 = ndimage.uniform_filter(lab[:, :, c], 7, mode="nearest")
        m2 = ndimage.uniform_filter(lab[:, :, c] ** 2, 7, mode="nearest")
        want += m2 - m1 * m1
    assert np.allclose(V, want, rtol=0, atol=1e-9)


def test_global_colour_term_constant_frame_and_numpy_restatement():
    flat = np.full((28, 42, 3), 77, np.uint8)
    assert oracle.color_contrast_global(flat).max() < 1e-12                  # below sigma_min: rounding noise stays noise
    assert oracle.color_normalise_global(np.zeros((4, 5)), 1.0, 0.0).max() == 0.0      # no floor, no contrast: C = 0
    fr = synth.frames(3, T=1, t0=150)[0][:84, :112]
    V = oracle.color_variance(fr)
    for kappa in (0.5, 1.0, 3.0):
        want = np.minimum(1.0, np.sqrt(V) / (kappa * np.sqrt(V.mean())))
        assert np.sqrt(V.mean()) > 0.5
        assert np.allclose(oracle.color_contrast_global(fr, kappa=kappa), want, rtol=1e-13, atol=0)
        assert np.allclose(oracle.color_normalise_global(V, kappa), want, rtol=1e-13, atol=0)
    # a frame whose contrast level lies under the floor is measured against the floor
    dim = 1e-4 * V
    assert np.allclose(oracle.color_normalise_global(dim, 1.0, 0.5), np.minimum(1.0, np.sqrt(dim) / 0.5), rtol=1e-13, atol=0)


def test_global_colour_term_is_invariant_to_the_contrast_scale_and_reduces_to_the_fixed_reading():
    fr = synth.frames(2, T=1)[0][100:184, 60:172]
    V = oracle.color_variance(fr)
    C = oracle.color_normalise_global(V, 1.7)
    for a in (0.01, 9.0):                                                    # V -> a^2 V: every contrast scaled by a
        assert np.allclose(oracle.color_normalise_global(a * a * V, 1.7, 0.0), C, rtol=1e-13, atol=0)
    kappa = 16.0 / np.sqrt(V.mean())                                         # kappa sigma_frame = sigma_ref
    assert np.allclose(oracle.color_contrast_global(fr, kappa=kappa), oracle.color_contrast(fr, sigma_ref=16.0), rtol=1e-12, atol=0)


def test_global_colour_term_two_valued_frame_closed_form():
    """Left half one colour, right half another (width W): a pixel whose 7-wide window holds k columns of the other
    colour has V = (k/7)(1 - k/7) dE^2; the frame mean of V is (8/7) dE^2 / W, so C = sqrt(k (7 - k)) / 7 /
    (kappa sqrt(8 / (7 W))) whatever the two colours are."""
    H, W, kappa = 20, 56, 4.0
    maps = []
    for ca, cb in (((200, 40, 40), (30, 160, 220)), ((90, 90, 90), (96, 90, 84))):
        fr = np.empty((H, W, 3), np.uint8)
        fr[:, :W // 2] = ca
        fr[:, W // 2:] = cb
        maps.append(oracle.color_contrast_global(fr, kappa=kappa))
    want = np.zeros(W)
    for d, k in ((1, 3), (2, 2), (3, 1)):
        c = np.sqrt(k * (7 - k)) / 7 / (kappa * np.sqrt(8 / (7 * W)))
        want[W // 2 - d] = want[W // 2 + d - 1] = c
    assert want.max() < 1.0
    for C in maps:
        assert np.allclose(C, want[None, :], rtol=1e-9, atol=1e-12)


def test_saliency_with_the_global_colour_term_is_the_blend_of_its_parts():
    fr = synth.frames(2, T=1)[0][:112, :140]
    p = oracle.Params(color_norm=1, color_kappa=1.3)
    s, S = oracle.saliency(fr, p, want_map=True)
    E = oracle.canny(oracle.gray(fr))
    want = np.clip(0.5 * E + 0.5 * oracle.color_contrast_global(fr, kappa=1.3), 0, 1)
    assert np.allclose(S, want, rtol=0, atol=1e-15)
    assert np.allclose(s, want.reshape(8, 14, 10, 14).mean(axis=(1, 3)).ravel(), rtol=1e-13, atol=0)
    assert not np.allclose(s, oracle.saliency(fr, oracle.Params()))           # and it is not the fixed reading

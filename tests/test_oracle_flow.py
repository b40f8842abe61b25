"""Pins of the oracle's temporal branch (Sec. III-A, Eq. 5; Farneback flow, Sec. IV-B).

Each test checks the oracle against something fixed outside it: a brute-force
least-squares solve, a closed form, an invariance or a special case.
"""
import numpy as np
import pytest

import oracle
from paper_2602_14236_b200 import synth


def _quadratic(h, w, A, b, c, dx=0.0, dy=0.0):
    y, x = np.mgrid[0:h, 0:w].astype(np.float64)
    x = x - dx
    y = y - dy
    return A[0][0] * x * x + 2 * A[0][1] * x * y + A[1][1] * y * y + b[0] * x + b[1] * y + c


def test_pyr_down_constant_ramp_and_impulse():
    const = np.full((16, 20), 7.25)
    assert np.array_equal(oracle.pyr_down(const), np.full((8, 10), 7.25))
    y, x = np.mgrid[0:16, 0:20].astype(np.float64)
    out = oracle.pyr_down(3 * x - 2 * y)
    # the binomial kernel is symmetric, so a linear ramp is sampled at (2y, 2x) unchanged
    assert np.allclose(out[1:-1, 1:-1], (3 * 2 * x[:8, :10] - 2 * 2 * y[:8, :10])[1:-1, 1:-1], atol=1e-12)
    imp = np.zeros((16, 20))
    imp[8, 10] = 256.0
    k = np.array([1, 4, 6, 4, 1.0])
    out = oracle.pyr_down(imp)
    # output (y,x) reads source (2y+a, 2x+b): impulse at (8,10) reaches outputs 3..5 with taps k[0], k[2], k[4]
    expect = np.zeros((8, 10))
    for oy, ky in ((3, 4), (4, 2), (5, 0)):
        for ox, kx in ((4, 4), (5, 2), (6, 0)):
            expect[oy, ox] = k[ky] * k[kx]
    assert np.allclose(out, expect, atol=1e-12)


def test_pyr_down_clamps_at_border():
    y, x = np.mgrid[0:8, 0:8].astype(np.float64)
    out = oracle.pyr_down(x)
    # at x=0 the taps -2,-1 clamp to column 0: (1*0 + 4*0 + 6*0 + 4*1 + 1*2)/16
    assert out[2, 0] == pytest.approx(6.0 / 16.0, abs=1e-15)


def test_poly_exp_equals_weighted_least_squares():
    """Brute force: solve the 6x6 weighted normal equations at every pixel with numpy."""
    rng = np.random.default_rng(3)
    img = rng.uniform(0, 255, (16, 16))
    r = oracle.poly_exp(img, 2, 1.2)
    g = np.exp(-np.arange(-2, 3) ** 2 / (2 * 1.2 ** 2))
    g /= g.sum()
    pad = np.pad(img, 2, mode="edge")
    dy, dx = np.mgrid[-2:3, -2:3]
    wts = np.sqrt(np.outer(g, g)).ravel()
    basis = np.stack([np.ones(25), dx.ravel(), dy.ravel(), dx.ravel() ** 2, dy.ravel() ** 2, (dx * dy).ravel()], 1)
    for y in range(16):
        for x in range(16):
            f = pad[y:y + 5, x:x + 5].ravel()
            sol = np.linalg.lstsq(basis * wts[:, None], f * wts, rcond=None)[0]
            assert np.allclose(r[:, y, x], sol[1:], atol=1e-9), (y, x)


def test_poly_exp_recovers_a_quadratic_exactly():
    A = [[0.7, -0.2], [-0.2, 0.4]]
    b = [1.5, -0.5]
    img = _quadratic(24, 28, A, b, 3.0)
    r = oracle.poly_exp(img, 2, 1.2)
    y, x = np.mgrid[0:24, 0:28].astype(np.float64)
    inner = (slice(2, -2), slice(2, -2))
    assert np.allclose(r[0][inner], (2 * A[0][0] * x + 2 * A[0][1] * y + b[0])[inner], atol=1e-9)
    assert np.allclose(r[1][inner], (2 * A[0][1] * x + 2 * A[1][1] * y + b[1])[inner], atol=1e-9)
    assert np.allclose(r[2][inner], A[0][0], atol=1e-9)
    assert np.allclose(r[3][inner], A[1][1], atol=1e-9)
    assert np.allclose(r[4][inner], 2 * A[0][1], atol=1e-9)


@pytest.mark.parametrize("d", [(2.0, 0.0), (-1.0, 3.0), (0.37, -1.62)])
def test_flow_iter_recovers_translation_of_a_quadratic(d):
    """f2(x) = f1(x - d) gives b2(x~) - b1(x) = 2A(d~ - d), hence the update returns d for any prior."""
    A = [[1.3, 0.4], [0.4, 0.9]]
    b = [0.2, -0.1]
    h, w = 40, 44
    c1 = oracle.poly_exp(_quadratic(h, w, A, b, 1.0), 2, 1.2)
    c2 = oracle.poly_exp(_quadratic(h, w, A, b, 1.0, dx=d[0], dy=d[1]), 2, 1.2)
    for prior in ((0.0, 0.0), (1.0, -0.5)):
        d_in = np.empty((2, h, w))
        d_in[0], d_in[1] = prior
        out = oracle.flow_iter(c1, c2, d_in, 15, 1e-3)
        inner = (slice(12, -12), slice(12, -12))
        assert np.allclose(out[0][inner], d[0], atol=1e-6)
        assert np.allclose(out[1][inner], d[1], atol=1e-6)


def test_flow_iter_window_extent_border_and_regulariser():
    """A = I everywhere, one pixel with db = (1, 0): d_u = n/(n^2 + eps) where the 15x15 box covers
    that pixel, n = number of in-image pixels of the box; zero elsewhere."""
    h, w = 30, 34
    c1 = np.zeros((5, h, w))
    c2 = np.zeros((5, h, w))
    for c in (c1, c2):
        c[2] = 1.0
        c[3] = 1.0
    y0, x0 = 4, 20
    c2[0, y0, x0] = -2.0          # -(b2 - b1)/2 = +1 along x at that pixel
    eps = 0.5
    out = oracle.flow_iter(c1, c2, np.zeros((2, h, w)), 15, eps)
    for y in range(h):
        for x in range(w):
            n = (min(y + 7, h - 1) - max(y - 7, 0) + 1) * (min(x + 7, w - 1) - max(x - 7, 0) + 1)
            inside = abs(y - y0) <= 7 and abs(x - x0) <= 7
            assert out[0, y, x] == pytest.approx(n / (n * n + eps) if inside else 0.0, abs=1e-14)
            assert out[1, y, x] == 0.0


def test_flow_iter_uses_prior_for_the_fetch_position():
    """With prior d~ = (3, 0) the frame-2 coefficients are read at x + 3 (convention I_cur(x+d) ~ I_prev(x))."""
    h, w = 20, 40
    c1 = np.zeros((5, h, w))
    c2 = np.zeros((5, h, w))
    c1[2] = c1[3] = 1.0
    c2[2] = c2[3] = 1.0
    c2[0, 10, 23] = -2.0
    d_in = np.zeros((2, h, w))
    d_in[0] = 3.0
    out = oracle.flow_iter(c1, c2, d_in, 1, 0.0)     # window 1: purely local solve
    # db = -(b2(x~)-b1)/2 + A d~ = (1,0)*[x~ == (23,10)] + (3,0); d = db
    expect = np.full((h, w), 3.0)
    expect[10, 20] = 4.0
    assert np.allclose(out[0], expect, atol=1e-12)
    assert np.allclose(out[1], 0.0, atol=1e-12)


def test_flow_upsample_uniform_and_ramp():
    dc = np.empty((2, 6, 8))
    dc[0], dc[1] = 1.5, -0.25
    up = oracle.flow_upsample(dc, 12, 16)
    assert np.allclose(up[0], 3.0) and np.allclose(up[1], -0.5)
    y, x = np.mgrid[0:6, 0:8].astype(np.float64)
    dc[0], dc[1] = x, y
    up = oracle.flow_upsample(dc, 12, 16)
    yf, xf = np.mgrid[0:12, 0:16].astype(np.float64)
    inner = (slice(1, -1), slice(1, -1))
    assert np.allclose(up[0][inner], (2 * ((xf + 0.5) / 2 - 0.5))[inner], atol=1e-12)
    assert np.allclose(up[1][inner], (2 * ((yf + 0.5) / 2 - 0.5))[inner], atol=1e-12)
    assert up[0][0, 0] == 0.0      # sample position -0.25 clamps to 0


def test_delta_p_uniform_field_is_its_magnitude():
    f = np.empty((2, 28, 42))
    f[0], f[1] = 3.0, -4.0
    assert np.allclose(oracle.delta_p(f, 14), 5.0, atol=1e-14)
    f[0, :14, :14] = 0.0
    f[1, :14, :14] = 0.0
    dp = oracle.delta_p(f, 14)
    assert dp[0] == 0.0 and np.allclose(dp[1:], 5.0)


def test_delta_p_patch_order_is_row_major():
    f = np.zeros((2, 28, 42))
    f[0, 14:, 28:] = 2.0        # patch row 1, patch column 2 -> index 1*3+2
    dp = oracle.delta_p(f, 14)
    assert dp[5] == pytest.approx(2.0) and dp.sum() == pytest.approx(2.0)


def test_identical_frames_give_exactly_zero_flow():
    fr = synth.texture(5, 56, 56)
    fl = oracle.flow(fr, fr)
    assert np.all(fl == 0.0)
    assert np.all(oracle.delta_p(fl, 14) == 0.0)


def test_full_flow_is_the_stated_composition():
    """oracle.flow == gray -> pyramid -> expansion -> coarse-to-fine (3 updates per level) -> level 0."""
    a = synth.texture(7, 56, 84)
    b = np.roll(a, 1, axis=1)
    p = oracle.Params()
    fl = oracle.flow(a, b, p)
    pyr = [[oracle.gray(f).astype(np.float64)] for f in (a, b)]
    for k in range(2):
        for _ in range(2):
            pyr[k].append(oracle.pyr_down(pyr[k][-1]))
    d = None
    for lvl in (2, 1, 0):
        h, w = pyr[0][lvl].shape
        c1, c2 = oracle.poly_exp(pyr[0][lvl]), oracle.poly_exp(pyr[1][lvl])
        d = np.zeros((2, h, w)) if d is None else oracle.flow_upsample(d, h, w)
        for _ in range(3):
            d = oracle.flow_iter(c1, c2, d)
    assert np.array_equal(fl, d)


def test_integer_translation_of_a_smooth_texture():
    """Accuracy pin (loose by the nature of the method): a pure 2 px shift reads as dP ~ 2 px."""
    canvas = synth.texture(11, 112, 116)
    prev, cur = canvas[:, 0:112], canvas[:, 2:114]        # content moves 2 px to the left
    fl = oracle.flow(prev, cur)
    dp = oracle.delta_p(fl, 14).reshape(8, 8)
    assert np.all(np.abs(dp[1:-1, 1:-1] - 2.0) < 0.05)
    assert np.median(fl[0][14:-14, 14:-14]) == pytest.approx(-2.0, abs=0.02)
    assert abs(np.median(fl[1][14:-14, 14:-14])) < 0.02


def test_brightness_offset_leaves_flow_unchanged():
    """The constant term of the expansion is unused, so a uniform offset (no clipping) changes nothing."""
    canvas = synth.texture(13, 56, 60)
    prev, cur = canvas[:, 0:56], canvas[:, 1:57]
    fl0 = oracle.flow(prev, cur)
    fl1 = oracle.flow(prev, (cur.astype(np.int32) + 9).astype(np.uint8))
    # gray of (c+9) is gray(c)+9 exactly: (77+150+29)*9 = 256*9
    assert np.allclose(fl0, fl1, atol=1e-9)


def test_gray_is_the_integer_luma():
    rgb = np.array([[[255, 255, 255], [0, 0, 0], [255, 0, 0], [0, 255, 0], [0, 0, 255], [10, 200, 77]]], np.uint8)
    g = oracle.gray(rgb)[0]
    assert list(g) == [255, 0, (77 * 255 + 128) >> 8, (150 * 255 + 128) >> 8, (29 * 255 + 128) >> 8,
                       (770 + 30000 + 29 * 77 + 128) >> 8]


def test_flow_score_batch_matches_single_calls():
    fr = synth.frames(1, T=3)[:, :56, :56]
    dP = oracle.flow_score(fr[:-1], fr[1:])
    for b in range(2):
        assert np.array_equal(dP[b], oracle.delta_p(oracle.flow(fr[b], fr[b + 1]), 14))


def test_literal_eq5_frame_difference_score():
    """Eq. 5 as printed: closed forms and the library norm."""
    rng = np.random.default_rng(2)
    a = rng.integers(0, 256, (1, 28, 42, 3)).astype(np.uint8)
    assert np.array_equal(oracle.diff_score(a, a), np.zeros((1, 6)))
    b = np.clip(a.astype(int), 0, 250).astype(np.uint8)
    assert np.allclose(oracle.diff_score(b, b + 5), 5.0, atol=1e-12)                 # uniform offset k -> k
    c = a.copy()
    c[0, 3, 20, 1] = np.uint8((int(a[0, 3, 20, 1]) + 100) % 256)                     # one value in patch (0, 1)
    d = abs(int(c[0, 3, 20, 1]) - int(a[0, 3, 20, 1]))
    got = oracle.diff_score(a, c)[0]
    assert got[1] == pytest.approx(d / np.sqrt(588.0), abs=1e-12) and got[[0, 2, 3, 4, 5]].max() == 0.0
    e = rng.integers(0, 256, (1, 28, 42, 3)).astype(np.uint8)
    diff = e.astype(np.float64) - a.astype(np.float64)
    want = [np.linalg.norm(diff[0, 14 * py:14 * py + 14, 14 * px:14 * px + 14]) / np.sqrt(588.0)
            for py in range(2) for px in range(3)]
    assert np.allclose(oracle.diff_score(a, e)[0], want, rtol=1e-13)
    assert np.allclose(oracle.diff_score(e, a), oracle.diff_score(a, e))             # symmetric

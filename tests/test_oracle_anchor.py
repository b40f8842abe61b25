"""Pins of the oracle's anchor-frame mode (a variant of the temporal test: every token is compared with the patch
its cache entry was computed from, not with the previous frame).  The paper has no worked example for it, so the
pins are closed forms (a uniform fade, a block that enters and leaves), the special case that reduces to the
consecutive-frame routines, the invariant that ties the anchor image to the source-frame table, and a brute-force
scan written out in numpy on a tiny video."""
import dataclasses

import numpy as np
import pytest

import oracle

P = oracle.Params(patch=2, tau_t=4.0, theta_R=0.9, tau_high=0.40, tau_med=0.36, tau_low=0.25, patch_reuse=1)


def _run(frames, s, first_has_no_prev=True, anchor=None, p=P):
    anchor = np.zeros(frames.shape[1:], np.uint8) if anchor is None else anchor
    return oracle.select_anchored(frames, s, first_has_no_prev, anchor, p) + (anchor,)


def test_slow_fade_is_stored_again_once_the_drift_reaches_tau():
    """Every frame is one grey level brighter than the one before: consecutive frames differ by 1 < tau_t in every
    patch, so the consecutive-frame test reuses frame 0 forever.  Against the anchor the difference after k frames is
    exactly k: frames 0, 4, 8, ... are stored (tau_t = 4: static means dP < 4), the others are wholly redundant."""
    T, h, w = 13, 8, 6
    base = np.random.default_rng(0).integers(0, 200, (h, w, 3), dtype=np.uint8)
    frames = np.stack([base + np.uint8(t) for t in range(T)])
    n = (h // 2) * (w // 2)
    s = np.full((T, n), 0.5, np.float32)            # salient: FP16 when stored
    dP, dec, idx, counts, red, anchor = _run(frames, s)
    for t in range(T):
        k = t % 4
        drift = 0.0 if t == 0 else (4.0 if k == 0 else float(k))      # a stored frame is scored against the old anchor
        assert np.array_equal(dP[t], np.full(n, drift, np.float32)), t
        assert (dec[t] == (oracle.FP16 if k == 0 else oracle.REUSE)).all(), t
        assert red[t] == (1 if k else 0)
        assert counts[t].tolist() == ([n, 0, 0, 0, 0] if k else [0, 0, 0, 0, n])
    assert np.array_equal(anchor, frames[12])
    # the consecutive-frame reading on the same video: everything after frame 0 is reused
    consecutive = oracle.diff_score(frames[:-1], frames[1:], patch=2)
    assert (consecutive == 1.0).all()
    for t in range(1, T):
        d, *_ = oracle.select(consecutive[t - 1].astype(np.float32), s[t], True, P)
        assert (d == oracle.REUSE).all()


def test_block_that_enters_and_leaves_reanchors_only_its_patches():
    """A bright 2x2 block covers patch 4 during frames 2..4 of an otherwise constant video.  Patch 4 is stored when
    the block arrives (frame 2) and again when it leaves (frame 5: the anchor then holds the block); every other
    patch, and patch 4 at all other times, is reused from frame 0."""
    T, h, w = 8, 6, 6
    bg = np.full((h, w, 3), 50, np.uint8)
    frames = np.stack([bg] * T)
    frames[2:5, 2:4, 2:4] = 250                      # patch row 1, column 1 -> token 1 * 3 + 1 = 4
    n = 9
    s = np.full((T, n), 0.3, np.float32)            # INT4 when stored
    p = dataclasses.replace(P, theta_R=0.95)        # 8 of 9 static patches (0.889) do not make a frame redundant
    dP, dec, idx, counts, red, anchor = _run(frames, s, p=p)
    want = np.full((T, n), oracle.REUSE, np.uint8)
    want[0] = oracle.INT4
    want[2, 4] = want[5, 4] = oracle.INT4
    assert np.array_equal(dec, want)
    assert dP[2, 4] == dP[5, 4] == np.float32(200.0) and dP[3, 4] == dP[4, 4] == 0.0
    assert idx[2, 2, 0] == 4 and idx[2, 2, 1] == -1
    src = oracle.source_frames(dec)
    assert src[:, 4].tolist() == [0, 0, 2, 2, 2, 5, 5, 5] and (np.delete(src, 4, axis=1) == 0).all()


def test_anchor_image_is_the_composite_named_by_the_source_table():
    """Invariant: after any prefix of the video, patch i of the anchor image is patch i of frame src[t][i], where src
    is the oracle's source-frame table of the decisions (Alg. 1's pointers resolved)."""
    rng = np.random.default_rng(3)
    T, h, w = 12, 8, 10
    frames = rng.integers(0, 256, (1, h, w, 3)).repeat(T, axis=0).astype(np.int16)
    frames += rng.integers(-6, 7, frames.shape) * (rng.random((T, h // 2, w // 2)) < 0.5).repeat(2, 1).repeat(2, 2)[..., None]
    frames = np.clip(frames, 0, 255).astype(np.uint8)
    n = (h // 2) * (w // 2)
    s = rng.uniform(0.2, 0.6, (T, n)).astype(np.float32)
    for upto in (1, 5, T):
        dP, dec, idx, counts, red, anchor = _run(frames[:upto], s[:upto])
        assert 0 < (dec == oracle.REUSE).mean() < 1 or upto == 1
        src = oracle.source_frames(dec)[-1]
        for i in range(n):
            py, px = divmod(i, w // 2)
            sl = (slice(2 * py, 2 * py + 2), slice(2 * px, 2 * px + 2))
            assert np.array_equal(anchor[sl], frames[src[i]][sl]), (upto, i)
    # a second call that carries the anchor continues the scan exactly
    a1 = np.zeros((h, w, 3), np.uint8)
    first = oracle.select_anchored(frames[:5], s[:5], True, a1, P)
    second = oracle.select_anchored(frames[5:], s[5:], False, a1, P)
    for whole, x, y in zip((dP, dec, idx, counts, red), first, second):
        assert np.array_equal(whole, np.concatenate([x, y]))
    assert np.array_equal(a1, anchor)


def test_without_reuse_the_anchor_is_the_previous_frame():
    """tau_t = 0 makes no patch static, so every token is stored in every frame and the anchor is always the previous
    frame: the scores are the consecutive-frame Eq. 5 scores and the decisions those of the per-frame rule."""
    rng = np.random.default_rng(5)
    T, h, w = 6, 6, 8
    frames = rng.integers(0, 256, (T, h, w, 3), dtype=np.uint8)
    n = 12
    s = rng.uniform(0.0, 0.6, (T, n)).astype(np.float32)
    p = dataclasses.replace(P, tau_t=0.0)
    dP, dec, idx, counts, red, anchor = _run(frames, s, p=p)
    assert (dP[0] == 0).all() and np.array_equal(dP[1:], oracle.diff_score(frames[:-1], frames[1:], patch=2).astype(np.float32))
    for t in range(T):
        d, ix, c, r, _ = oracle.select(dP[t], s[t], t > 0, p)
        assert np.array_equal(dec[t], d) and np.array_equal(idx[t], ix) and np.array_equal(counts[t], c) and red[t] == r == 0
    assert np.array_equal(anchor, frames[-1])


@pytest.mark.parametrize("patch_reuse", [0, 1])
def test_scan_written_out_in_numpy(patch_reuse):
    """The whole scan again, in plain numpy on a tiny video with small random changes (so that static and moving
    patches mix and some frames are redundant)."""
    rng = np.random.default_rng(7 + patch_reuse)
    T, h, w, pt = 16, 6, 6, 2
    frames = np.empty((T, h, w, 3), np.uint8)
    frames[0] = rng.integers(0, 256, (h, w, 3))
    for t in range(1, T):
        step = rng.integers(-3, 4, (h, w, 3)) * (rng.random((h // pt, w // pt)) < rng.choice([0.1, 0.6])).repeat(pt, 0).repeat(pt, 1)[..., None]
        frames[t] = np.clip(frames[t - 1].astype(np.int16) + step, 0, 255)
    n = 9
    s = rng.uniform(0.2, 0.5, (T, n)).astype(np.float32)
    p = dataclasses.replace(P, tau_t=2.0, theta_R=0.7, patch_reuse=patch_reuse)
    dP, dec, idx, counts, red, anchor = _run(frames, s, p=p)
    a = np.zeros((h, w, 3), np.int64)
    seen_reuse = seen_red = False
    for t in range(T):
        f = frames[t].astype(np.int64)
        sq = ((f - a) ** 2).reshape(h // pt, pt, w // pt, pt, 3).sum(axis=(1, 3, 4)).reshape(n)
        d = np.sqrt(sq / (3.0 * pt * pt)).astype(np.float32) if t else np.zeros(n, np.float32)
        static = (d < np.float32(p.tau_t)) & (t > 0)
        redundant = t > 0 and np.float32(static.sum()) / np.float32(n) > np.float32(p.theta_R)
        tier = np.where(s[t] > p.tau_high, oracle.FP16, np.where(s[t] > p.tau_med, oracle.INT8, np.where(s[t] > p.tau_low, oracle.INT4, oracle.PRUNE)))
        want = np.where(redundant | (static & bool(patch_reuse)), oracle.REUSE, tier).astype(np.uint8)
        assert np.array_equal(dP[t], d) and np.array_equal(dec[t], want) and red[t] == int(redundant), t
        keep = (want != oracle.REUSE).reshape(h // pt, w // pt).repeat(pt, 0).repeat(pt, 1)[..., None]
        a = np.where(keep, f, a)
        seen_reuse |= bool((want == oracle.REUSE).any() and not redundant)
        seen_red |= bool(redundant)
    assert np.array_equal(anchor, a.astype(np.uint8)) and seen_red and (seen_reuse or not patch_reuse)

"""GPU parity of the anchor-frame mode (salicache_select_anchored) against the oracle, through the C ABI.
Everything it produces is integer work or a correctly rounded square root of an exact integer sum, so every
output is compared bit for bit: scores, decisions, index lists, counts, redundancy flags, row offsets, the running
fill and the anchor image."""
import numpy as np
import pytest

import oracle
from paper_2602_14236_b200 import binding as sc
from paper_2602_14236_b200 import synth

import gpu_util as gu

pytestmark = pytest.mark.gpu


def _video(rng, T, H, W, p_move=0.4, amp=9):
    """A fixed random image plus, per frame, small changes on a random subset of the patches of the frame before."""
    fr = np.empty((T, H, W, 3), np.uint8)
    fr[0] = rng.integers(0, 256, (H, W, 3))
    for t in range(1, T):
        moving = (rng.random((H // 14, W // 14)) < rng.choice([0.05, p_move])).repeat(14, 0).repeat(14, 1)[..., None]
        fr[t] = np.clip(fr[t - 1].astype(np.int16) + rng.integers(-amp, amp + 1, (H, W, 3)) * moving, 0, 255)
    return fr


def _run_gpu(ctx, frames, s, first, anchor, fill0=(0, 0, 0)):
    import torch
    T, n = s.shape
    d = dict(
        dP=torch.full((T, n), -1.0, dtype=torch.float32, device="cuda"),
        decision=torch.full((T, n), 255, dtype=torch.uint8, device="cuda"),
        idx=torch.full((T, 3, n), -7, dtype=torch.int32, device="cuda"),
        counts=torch.full((T, 5), -1, dtype=torch.int32, device="cuda"),
        redundant=torch.full((T,), 255, dtype=torch.uint8, device="cuda"),
        row_offset=torch.full((T, 3), -1, dtype=torch.int64, device="cuda"),
        fill=torch.tensor(list(fill0), dtype=torch.int64, device="cuda"),
    )
    sc.salicache_select_anchored(ctx, torch.from_numpy(frames).cuda(), torch.from_numpy(s).cuda(), T, first, anchor, d["dP"],
                                 d["decision"], d["idx"], d["counts"], d["redundant"], d["row_offset"], d["fill"])
    torch.cuda.synchronize()
    return {k: v.cpu().numpy() for k, v in d.items()}


def _compare(got, ref, fill0=(0, 0, 0)):
    dP, dec, idx, counts, red = ref
    assert np.array_equal(got["dP"], dP)
    assert np.array_equal(got["decision"], dec)
    assert np.array_equal(got["idx"], idx)
    assert np.array_equal(got["counts"], counts)
    assert np.array_equal(got["redundant"], red)
    off, fill = oracle.row_offsets(counts, np.asarray(fill0, np.int64))
    assert np.array_equal(got["row_offset"], off)
    assert np.array_equal(got["fill"], fill)


@pytest.mark.parametrize("H,W,patch_reuse", [(336, 336, 1), (336, 336, 0), (224, 448, 1), (112, 672, 1), (672, 672, 1)])
def test_anchored_scan_matches_the_oracle(H, W, patch_reuse):
    """336 x 336: three bands of patch rows per CTA; 224 x 448: two; 112 x 672: one band of 48 patches; 672 x 672: six
    bands of 48, the most a CTA may own.  Two calls in a row carry the anchor image and the fill."""
    import torch
    rng = np.random.default_rng(H + W + patch_reuse)
    T = 14
    frames = _video(rng, T, H, W)
    kw = dict(synth.thresholds("four"), tau_t=2.5, theta_R=0.8, patch_reuse=patch_reuse)
    ctx = sc.Context(sc.salicache_default_params(H=H, W=W, max_batch=16, chunk_frames=2, L=1, **kw))
    n = ctx.n_tok
    s = rng.uniform(0.15, 0.6, (T, n)).astype(np.float32)
    p = gu.oracle_params(ctx.params)
    ref_anchor = rng.integers(0, 256, (H, W, 3), dtype=np.uint8)           # ignored: the first frame has no predecessor
    d_anchor = torch.from_numpy(ref_anchor.copy()).cuda()
    ref = oracle.select_anchored(frames, s, True, ref_anchor, p)
    dec = ref[1]
    assert ref[4].any() and not ref[4].all(), "the case should mix redundant and stored frames"
    if patch_reuse:
        mixed = [(dec[t] == oracle.REUSE).any() and not ref[4][t] for t in range(T)]
        assert any(mixed), "the case should reuse single patches of a stored frame"
    # first call: frames 0..8, second call continues with 9..13
    g1 = _run_gpu(ctx, frames[:9], s[:9], True, d_anchor)
    _compare(g1, tuple(x[:9] for x in ref))
    g2 = _run_gpu(ctx, frames[9:], s[9:], False, d_anchor, fill0=tuple(g1["fill"]))
    _compare(g2, tuple(x[9:] for x in ref), fill0=tuple(g1["fill"]))
    assert np.array_equal(d_anchor.cpu().numpy(), ref_anchor)
    assert sc.salicache_poll_status(ctx) == 0


def test_anchored_mode_stops_the_drift_of_a_slow_fade():
    """A video that gets one grey level brighter per frame: the consecutive-frame score (salicache_diff_score) is 1
    everywhere, below tau_t = 4, so every frame after the first is reused; against the anchor the frames 0, 4, 8, ...
    are stored."""
    import torch
    T, H, W = 10, 336, 336
    base = np.random.default_rng(1).integers(0, 200, (H, W, 3), dtype=np.uint8)
    frames = np.stack([base + np.uint8(t) for t in range(T)])
    ctx = sc.Context(sc.salicache_default_params(max_batch=16, chunk_frames=2, L=1, tau_t=4.0, **synth.thresholds("int4")))
    s = np.full((T, ctx.n_tok), 0.5, np.float32)
    d_anchor = torch.zeros((H, W, 3), dtype=torch.uint8, device="cuda")
    g = _run_gpu(ctx, frames, s, True, d_anchor)
    assert g["redundant"].tolist() == [0 if t % 4 == 0 else 1 for t in range(T)]
    assert np.array_equal(d_anchor.cpu().numpy(), frames[8])
    d = torch.from_numpy(frames).cuda()
    dP = torch.zeros((T, ctx.n_tok), dtype=torch.float32, device="cuda")
    sc.salicache_diff_score(ctx, d[:-1], d[1:], T - 1, dP[1:])
    out = gu.gpu_select(ctx, dP.cpu().numpy(), s, first_has_no_prev=True)
    assert out["redundant"].cpu().numpy().tolist() == [0] + [1] * (T - 1)


def test_anchored_mode_argument_checks():
    import ctypes
    import torch
    lib = sc.lib()
    ctx = sc.Context(sc.salicache_default_params(max_batch=4, chunk_frames=2, L=1))
    n = ctx.n_tok
    fr = torch.zeros((2, 336, 336, 3), dtype=torch.uint8, device="cuda")
    s = torch.zeros((2, n), dtype=torch.float32, device="cuda")
    anchor = torch.zeros((336 * 336 * 3 + 16,), dtype=torch.uint8, device="cuda")
    dP = torch.zeros((2, n), dtype=torch.float32, device="cuda")
    dec = torch.zeros((2, n), dtype=torch.uint8, device="cuda")
    idx = torch.zeros((2, 3, n), dtype=torch.int32, device="cuda")
    cnt = torch.zeros((2, 5), dtype=torch.int32, device="cuda")
    red = torch.zeros((2,), dtype=torch.uint8, device="cuda")
    off = torch.zeros((2, 3), dtype=torch.int64, device="cuda")
    fill = torch.zeros((3,), dtype=torch.int64, device="cuda")
    args = lambda c, a, B: (c.handle, fr.data_ptr(), s.data_ptr(), B, 1, a, dP.data_ptr(), dec.data_ptr(), idx.data_ptr(),
                            cnt.data_ptr(), red.data_ptr(), off.data_ptr(), fill.data_ptr(), None)
    assert lib.salicache_select_anchored(*args(ctx, None, 2)) == sc.E_NULL
    assert lib.salicache_select_anchored(*args(ctx, anchor.data_ptr() + 4, 2)) == sc.E_ALIGN
    assert lib.salicache_select_anchored(*args(ctx, anchor.data_ptr(), 5)) == sc.E_SHAPE
    assert lib.salicache_select_anchored(*args(ctx, anchor.data_ptr(), 0)) == 0
    wl = synth.WORKLOADS[4]
    anyres = sc.Context(sc.salicache_default_params(H=wl.H, W=wl.W, n_images=wl.n_images, max_batch=4, chunk_frames=2, L=1))
    assert lib.salicache_select_anchored(*args(anyres, anchor.data_ptr(), 1)) == sc.E_PARAM


def test_several_videos_in_one_launch_match_one_video_at_a_time():
    """Five videos of different content, one cluster each, against the oracle video by video; the videos keep their own
    anchor images and fills."""
    import torch
    H = W = 336
    V, T = 5, 9
    rng = np.random.default_rng(77)
    frames = np.stack([_video(rng, T, H, W, p_move=0.2 + 0.15 * v) for v in range(V)])
    kw = dict(synth.thresholds("four"), tau_t=2.5, theta_R=0.8)
    ctx = sc.Context(sc.salicache_default_params(max_batch=16, chunk_frames=2, L=1, **kw))
    n = ctx.n_tok
    s = rng.uniform(0.15, 0.6, (V, T, n)).astype(np.float32)
    p = gu.oracle_params(ctx.params)
    fill0 = np.arange(3 * V, dtype=np.int64).reshape(V, 3)
    d = dict(
        dP=torch.full((V, T, n), -1.0, dtype=torch.float32, device="cuda"),
        decision=torch.full((V, T, n), 255, dtype=torch.uint8, device="cuda"),
        idx=torch.full((V, T, 3, n), -7, dtype=torch.int32, device="cuda"),
        counts=torch.full((V, T, 5), -1, dtype=torch.int32, device="cuda"),
        redundant=torch.full((V, T), 255, dtype=torch.uint8, device="cuda"),
        row_offset=torch.full((V, T, 3), -1, dtype=torch.int64, device="cuda"),
        fill=torch.from_numpy(fill0.copy()).cuda(),
    )
    anchors = torch.zeros((V, H, W, 3), dtype=torch.uint8, device="cuda")
    sc.salicache_select_anchored_batch(ctx, torch.from_numpy(frames).cuda(), torch.from_numpy(s).cuda(), V, T, True, anchors, d["dP"],
                                       d["decision"], d["idx"], d["counts"], d["redundant"], d["row_offset"], d["fill"])
    torch.cuda.synchronize()
    got = {k: v.cpu().numpy() for k, v in d.items()}
    for v in range(V):
        a = np.zeros((H, W, 3), np.uint8)
        ref = oracle.select_anchored(frames[v], s[v], True, a, p)
        _compare({k: x[v] for k, x in got.items()}, ref, fill0=tuple(fill0[v]))
        assert np.array_equal(anchors[v].cpu().numpy(), a)

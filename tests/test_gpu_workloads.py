"""GPU parity on the workloads' own shapes: the anyres layout of workload 4, the streamed segments of
workload 5 with a ring budget, and workload 3 at the full K/V shape (32 layers): an 8-frame store launch
checked on every pool byte, and the 40-frame store launch the benchmark times checked on sampled slabs."""
import numpy as np
import pytest

import oracle
from paper_2602_14236_b200 import binding as sc
from paper_2602_14236_b200 import synth

import gpu_util as gu

pytestmark = pytest.mark.gpu


def _anyres_tokens(full48: np.ndarray, base24: np.ndarray) -> np.ndarray:
    """Per-patch values of the whole frame and of the base image in the token order of the anyres layout."""
    return oracle.anyres_tokens(full48, base24)


def test_anyres_scores_follow_the_token_layout_and_match_the_oracle():
    fr = synth.frames(4, T=3, t0=28)                       # frames 28, 29 | 30: a scene cut between 29 and 30
    ctx = sc.Context(sc.salicache_default_params(H=672, W=672, n_images=5, max_batch=4, chunk_frames=2, L=1))
    assert ctx.n_tok == 2880
    dP, s = gu.gpu_scores(ctx, fr)
    base = np.stack([oracle.box_down2(f) for f in fr])
    rdP_full = oracle.flow_score(fr[:-1], fr[1:])
    rdP_base = oracle.flow_score(base[:-1], base[1:])
    rs_full, rs_base = oracle.saliency(fr), oracle.saliency(base)
    want_dP = np.stack([_anyres_tokens(rdP_full[t], rdP_base[t]) for t in range(2)])
    want_s = np.stack([_anyres_tokens(rs_full[t], rs_base[t]) for t in range(3)])
    gu.assert_scores_close(dP[1:], want_dP, "anyres dP")
    gu.assert_scores_close(s, want_s, "anyres s")
    # brightness jitter alone leaves the flow at zero (frame 28 -> 29); the cut (29 -> 30) does not
    p = gu.oracle_params(ctx.params)
    out = gu.gpu_select(ctx, dP, s)
    red = out["redundant"].cpu().numpy()
    assert red.tolist() == [0, 1, 0]
    dec, idx, counts, rred, _ = gu.oracle_select_all(np.concatenate([np.zeros((1, 2880)), want_dP]).astype(np.float32),
                                                     want_s.astype(np.float32), p)
    near = gu.near_threshold(None, want_s.astype(np.float32), p)
    assert not ((out["decision"].cpu().numpy() != dec) & ~near).any()
    assert (out["counts"].cpu().numpy().sum(axis=1) == 2880).all()


def test_streamed_segments_and_ring_budget_of_workload_5():
    """Frames across the static -> 1 px pan boundary, stored into ring pools smaller than the stream:
    the oldest rows are overwritten, exactly as on the oracle's ring."""
    import torch
    L, T, n_tok, HD = 2, 6, 576, 4096
    fr = synth.frames(5, T=T, t0=297)                      # 297..299 static, 300.. pan 1 px/frame
    th = synth.thresholds("int4")
    ctx = sc.Context(sc.salicache_default_params(max_batch=8, chunk_frames=4, L=L, **th))
    dP, s = gu.gpu_scores(ctx, fr)
    out = gu.gpu_select(ctx, dP, s)
    p = gu.oracle_params(ctx.params)
    rdP = np.zeros((T, n_tok))
    rdP[1:] = oracle.flow_score(fr[:-1], fr[1:])
    rs = oracle.saliency(fr)
    gu.assert_scores_close(dP[1:], rdP[1:], "dP workload 5")
    g_dec, g_idx, g_counts = (out[k].cpu().numpy() for k in ("decision", "idx", "counts"))
    g_off = out["row_offset"].cpu().numpy()
    assert out["redundant"].cpu().numpy().tolist()[:3] == [0, 1, 1]          # static frames point at their predecessor
    assert (g_counts[1:3, 0] == n_tok).all()
    # decisions from the GPU's own scores are the oracle's, bit for bit
    for t in range(T):
        d, i, c, r, _ = oracle.select(dP[t], s[t], t > 0, p)
        assert np.array_equal(d, g_dec[t]) and np.array_equal(i, g_idx[t]) and np.array_equal(c, g_counts[t])
    stored4 = int(g_counts[:, 2].sum())
    cap4 = max(stored4 // 2, 1)                                              # budget: half of what the stream stores
    assert stored4 > 600
    KV = [synth.kv_numpy(5, t, L=L) for t in range(T)]
    K = np.stack([k for k, _ in KV]).view(np.uint16)
    V = np.stack([v for _, v in KV]).view(np.uint16)
    ref = oracle.Pools(L, HD, 128, 64, 1, cap4, ring=1)
    for t in range(T):
        oracle.pack_frame(K[t], V[t], g_idx[t], g_counts[t], g_off[t], ref)
    pools = sc.PoolSet(L, HD, 64, 1, cap4, ring=True)
    sc.salicache_pack_kv(ctx, torch.from_numpy(K.view(np.float16)).cuda(), torch.from_numpy(V.view(np.float16)).cuda(),
                         L * n_tok * HD, out["idx"], out["counts"], out["row_offset"], T, pools.c)
    torch.cuda.synchronize()
    # one call stores more than cap rows: the rows a later row of the call lands on are skipped, so the pool holds
    # the newest cap rows, as on the oracle's ring
    assert stored4 > cap4
    assert np.array_equal(pools.int4_codes.cpu().numpy(), ref.int4_codes)
    assert np.array_equal(pools.int4_sz.cpu().numpy().view(np.uint16), ref.int4_sz)
    assert sc.salicache_poll_status(ctx) == 0


def test_ring_budget_frame_by_frame_matches_the_oracle_ring():
    """The streaming use: one store call per frame into ring pools; the oldest rows are evicted first."""
    import torch
    L, T, n_tok, HD = 1, 5, 576, 4096
    fr = synth.frames(5, T=T, t0=600)                      # 8 px/frame pan: every frame is stored
    ctx = sc.Context(sc.salicache_default_params(max_batch=8, chunk_frames=4, L=L, **synth.thresholds("int4")))
    dP, s = gu.gpu_scores(ctx, fr)
    out = gu.gpu_select(ctx, dP, s)
    g_idx, g_counts, g_off = (out[k].cpu().numpy() for k in ("idx", "counts", "row_offset"))
    cap16, cap4 = 8, 1000                                   # less than two frames of INT4 rows
    KV = [synth.kv_numpy(5, t, L=L) for t in range(T)]
    ref = oracle.Pools(L, HD, 128, cap16, 1, cap4, ring=1)
    pools = sc.PoolSet(L, HD, cap16, 1, cap4, ring=True)
    for t in range(T):
        Kt, Vt = KV[t]
        oracle.pack_frame(Kt.view(np.uint16), Vt.view(np.uint16), g_idx[t], g_counts[t], g_off[t], ref)
        sc.salicache_pack_kv(ctx, torch.from_numpy(Kt).cuda(), torch.from_numpy(Vt).cuda(), L * n_tok * HD,
                             out["idx"][t:], out["counts"][t:], out["row_offset"][t:], 1, pools.c)
    torch.cuda.synchronize()
    assert g_counts[:, 2].sum() > 2 * cap4
    assert np.array_equal(pools.int4_codes.cpu().numpy(), ref.int4_codes)
    assert np.array_equal(pools.int4_sz.cpu().numpy().view(np.uint16), ref.int4_sz)
    assert np.array_equal(pools.fp16_pool.cpu().numpy().view(np.uint16), ref.fp16_pool)


def test_workload_3_full_shape_every_pool_byte():
    """32 layers x 32 heads x 128, one store launch of eight frames around the pan -> hold transition."""
    import torch
    wl = synth.WORKLOADS[3]
    T, L, n_tok, HD = 8, wl.L, wl.n_tok, wl.HD
    t0 = 116
    fr = synth.frames(3, T=T + 1, t0=t0 - 1)
    th = synth.thresholds(wl.background)
    ctx = sc.Context(sc.salicache_default_params(max_batch=16, chunk_frames=16, L=L, **th))
    d_fr = torch.from_numpy(fr).cuda()
    dP = torch.zeros((T, n_tok), dtype=torch.float32, device="cuda")
    s = torch.zeros((T, n_tok), dtype=torch.float32, device="cuda")
    red = torch.zeros((T,), dtype=torch.uint8, device="cuda")
    dec = torch.zeros((T, n_tok), dtype=torch.uint8, device="cuda")
    idx = torch.zeros((T, 3, n_tok), dtype=torch.int32, device="cuda")
    counts = torch.zeros((T, 5), dtype=torch.int32, device="cuda")
    off = torch.zeros((T, 3), dtype=torch.int64, device="cuda")
    fill = torch.zeros((3,), dtype=torch.int64, device="cuda")
    sc.salicache_flow_score(ctx, d_fr[:-1], d_fr[1:], T, dP)
    sc.salicache_frame_redundancy(ctx, dP, T, False, red)
    sc.salicache_saliency(ctx, d_fr[1:], T, s, red)
    sc.salicache_select(ctx, dP, s, T, False, dec, idx, counts, red, off, fill)
    K = torch.empty((T, L, n_tok, HD), dtype=torch.float16, device="cuda")
    V = torch.empty_like(K)
    for t in range(T):
        k, v = synth.kv_torch(3, t, "cuda")
        K[t].copy_(k)
        V[t].copy_(v)
    h_counts = counts.cpu().numpy()
    tot = h_counts[:, [4, 3, 2]].sum(axis=0)
    pools = sc.PoolSet(L, HD, int(tot[0]) + 1, 1, int(tot[2]) + 1)
    sc.salicache_pack_kv(ctx, K, V, L * n_tok * HD, idx, counts, off, T, pools.c)
    torch.cuda.synchronize()
    assert sc.salicache_poll_status(ctx) == 0
    # scores and decisions
    p = gu.oracle_params(ctx.params)
    rdP = oracle.flow_score(fr[:-1], fr[1:])
    gu.assert_scores_close(dP.cpu().numpy(), rdP, "dP workload 3")
    h_red = red.cpu().numpy()
    rs = oracle.saliency(fr[1:])
    gu.assert_scores_close(s.cpu().numpy()[h_red == 0], rs[h_red == 0], "s workload 3")
    assert 0 < h_red.sum() < T                                             # the hold begins inside the window
    h_dP, h_s, h_idx, h_off = dP.cpu().numpy(), s.cpu().numpy(), idx.cpu().numpy(), off.cpu().numpy()
    for t in range(T):
        d, i, c, r, _ = oracle.select(h_dP[t], h_s[t], True, p)
        assert r == h_red[t] and np.array_equal(c, h_counts[t]) and np.array_equal(i, h_idx[t])
    # the store: every pool byte of every layer against the oracle
    ref = oracle.Pools(L, HD, 128, int(tot[0]) + 1, 1, int(tot[2]) + 1)
    hK, hV = K.cpu().numpy().view(np.uint16), V.cpu().numpy().view(np.uint16)
    for t in range(T):
        oracle.pack_frame(hK[t], hV[t], h_idx[t], h_counts[t], h_off[t], ref)
    assert tot[2] > 1000 and tot[0] > 0
    assert np.array_equal(pools.int4_codes.cpu().numpy(), ref.int4_codes)
    assert np.array_equal(pools.int4_sz.cpu().numpy().view(np.uint16), ref.int4_sz)
    assert np.array_equal(pools.fp16_pool.cpu().numpy().view(np.uint16), ref.fp16_pool)

def test_workload_3_store_launch_of_40_frames_as_the_benchmark_times_it():
    """The benchmark stores 40 frames per launch at 32 layers: 40 panning frames of workload 3, every token INT4 or
    FP16, 40 x 576 x 64 = 1.47 million token rows in one launch.  Decisions and row offsets are compared whole; the
    pools on sampled (frame, layer) slabs, K and V, against the oracle's store of the same slab."""
    import torch
    wl = synth.WORKLOADS[3]
    T, L, n_tok, HD = 40, wl.L, wl.n_tok, wl.HD
    fr = synth.frames(3, T=T + 1, t0=79)                        # pairs (79, 80) .. (118, 119): the 3 px/frame pan
    ctx = sc.Context(sc.salicache_default_params(max_batch=T, chunk_frames=T, L=L, **synth.thresholds(wl.background)))
    d_fr = torch.from_numpy(fr).cuda()
    dP = torch.zeros((T, n_tok), dtype=torch.float32, device="cuda")
    s = torch.zeros((T, n_tok), dtype=torch.float32, device="cuda")
    red = torch.zeros((T,), dtype=torch.uint8, device="cuda")
    dec = torch.zeros((T, n_tok), dtype=torch.uint8, device="cuda")
    idx = torch.zeros((T, 3, n_tok), dtype=torch.int32, device="cuda")
    counts = torch.zeros((T, 5), dtype=torch.int32, device="cuda")
    off = torch.zeros((T, 3), dtype=torch.int64, device="cuda")
    fill = torch.zeros((3,), dtype=torch.int64, device="cuda")
    sc.salicache_flow_score(ctx, d_fr[:-1], d_fr[1:], T, dP)
    sc.salicache_frame_redundancy(ctx, dP, T, False, red)
    sc.salicache_saliency(ctx, d_fr[1:], T, s, red)
    sc.salicache_select(ctx, dP, s, T, False, dec, idx, counts, red, off, fill)
    K = torch.empty((T, L, n_tok, HD), dtype=torch.float16, device="cuda")
    V = torch.empty_like(K)
    for t in range(T):
        k, v = synth.kv_torch(3, t, "cuda")
        K[t].copy_(k)
        V[t].copy_(v)
    del k, v
    h_counts, h_idx, h_off = counts.cpu().numpy(), idx.cpu().numpy(), off.cpu().numpy()
    tot = h_counts[:, [4, 3, 2]].sum(axis=0)
    assert tot.sum() * 2 * L > 1_400_000                        # (nearly) every token of every frame is stored
    pools = sc.PoolSet(L, HD, int(tot[0]) + 1, 1, int(tot[2]) + 1)
    sc.salicache_pack_kv(ctx, K, V, L * n_tok * HD, idx, counts, off, T, pools.c)
    torch.cuda.synchronize()
    assert sc.salicache_poll_status(ctx) == 0
    p = gu.oracle_params(ctx.params)
    h_dP, h_s, h_red = dP.cpu().numpy(), s.cpu().numpy(), red.cpu().numpy()
    for t in range(T):
        d, i, c, r, _ = oracle.select(h_dP[t], h_s[t], True, p)
        assert r == h_red[t] and np.array_equal(c, h_counts[t]) and np.array_equal(i, h_idx[t])
    want_off, want_fill = oracle.row_offsets(h_counts)
    assert np.array_equal(h_off, want_off) and np.array_equal(fill.cpu().numpy(), want_fill)
    for t, l in ((0, 0), (0, 31), (13, 17), (27, 5), (39, 0), (39, 31)):
        ref = oracle.Pools(1, HD, 128, int(tot[0]) + 1, 1, int(tot[2]) + 1)
        hK = K[t, l:l + 1].cpu().numpy().view(np.uint16)
        hV = V[t, l:l + 1].cpu().numpy().view(np.uint16)
        assert oracle.pack_frame(hK, hV, h_idx[t], h_counts[t], h_off[t], ref) == 0
        n16, n4 = int(h_counts[t, 4]), int(h_counts[t, 2])
        r16, r4 = slice(int(h_off[t, 0]), int(h_off[t, 0]) + n16), slice(int(h_off[t, 2]), int(h_off[t, 2]) + n4)
        assert n4 > 300
        assert np.array_equal(pools.int4_codes[l, :, r4].cpu().numpy(), ref.int4_codes[0, :, r4]), (t, l)
        assert np.array_equal(pools.int4_sz[l, :, r4].cpu().numpy().view(np.uint16), ref.int4_sz[0, :, r4]), (t, l)
        assert np.array_equal(pools.fp16_pool[l, :, r16].cpu().numpy().view(np.uint16), ref.fp16_pool[0, :, r16]), (t, l)


def test_literal_eq5_difference_score_matches_the_oracle():
    """The frame-difference reading of Eq. 5: exact integer sums, so the float32 scores are the oracle's, rounded."""
    import torch
    for wl, kw in ((1, {}), (3, {}), (4, dict(H=672, W=672, n_images=5))):
        fr = synth.frames(wl, T=4, t0=118 if wl == 3 else 1)
        ctx = sc.Context(sc.salicache_default_params(max_batch=4, chunk_frames=2, L=1, **kw))
        d = torch.from_numpy(fr).cuda()
        dP = torch.full((3, ctx.n_tok), -1.0, dtype=torch.float32, device="cuda")
        sc.salicache_diff_score(ctx, d[:-1], d[1:], 3, dP)
        torch.cuda.synchronize()
        want = oracle.diff_score(fr[:-1], fr[1:])
        if wl == 4:
            base = np.stack([oracle.box_down2(f) for f in fr])
            wb = oracle.diff_score(base[:-1], base[1:])
            want = np.stack([_anyres_tokens(want[t], wb[t]) for t in range(3)])
        assert np.array_equal(dP.cpu().numpy(), want.astype(np.float32)), wl


@pytest.mark.parametrize("wl_index,T,L", [(2, 2, 32), (4, 1, 2)])
def test_store_on_the_other_workloads_kv(wl_index, T, L):
    """Workload 2 (32 layers, 1 % of the elements x8: the scale follows the outlier) and workload 4
    (2880 tokens per frame), INT8 background: pools bit-exact, dequantised values within the target's 1e-3
    of the oracle's (they are equal) and the INT8 error bound s/2 against the input."""
    import torch
    wl = synth.WORKLOADS[wl_index]
    n_tok, HD = wl.n_tok, wl.HD
    th = synth.thresholds(wl.background)
    ctx = sc.Context(sc.salicache_default_params(H=wl.H, W=wl.W, n_images=wl.n_images, max_batch=4, chunk_frames=2, L=L, **th))
    rng = np.random.default_rng(wl_index)
    s = rng.uniform(0.2, 0.6, (T, n_tok)).astype(np.float32)
    out = gu.gpu_select(ctx, None, s, first_has_no_prev=False)
    counts, idx, off, dec = (out[k].cpu().numpy() for k in ("counts", "idx", "row_offset", "decision"))
    K = torch.empty((T, L, n_tok, HD), dtype=torch.float16, device="cuda")
    V = torch.empty_like(K)
    for t in range(T):
        k, v = synth.kv_torch(wl_index, t, "cuda", L=L)
        K[t].copy_(k)
        V[t].copy_(v)
    caps = tuple(int(c) + 1 for c in counts[:, [4, 3, 2]].sum(axis=0))
    pools = sc.PoolSet(L, HD, *caps)
    sc.salicache_pack_kv(ctx, K, V, L * n_tok * HD, out["idx"], out["counts"], out["row_offset"], T, pools.c)
    gK = torch.zeros_like(K)
    gV = torch.zeros_like(V)
    sc.salicache_unpack_kv(ctx, pools.c, out["idx"], out["counts"], out["decision"], out["row_offset"], T, True, gK, gV,
                           L * n_tok * HD)
    torch.cuda.synchronize()
    assert sc.salicache_poll_status(ctx) == 0
    hK, hV = K.cpu().numpy(), V.cpu().numpy()
    ref = oracle.Pools(L, HD, 128, *caps)
    Ko = np.zeros(hK.shape, np.uint16)
    Vo = np.zeros(hK.shape, np.uint16)
    for t in range(T):
        oracle.pack_frame(hK[t].view(np.uint16), hV[t].view(np.uint16), idx[t], counts[t], off[t], ref)
        oracle.unpack_frame(n_tok, idx[t], counts[t], dec[t], off[t], ref, True, Ko[t], Vo[t])
    assert counts[:, 3].sum() > 100 and counts[:, 4].sum() > 100
    assert np.array_equal(pools.int8_codes.cpu().numpy(), ref.int8_codes)
    assert np.array_equal(pools.int8_scale.cpu().numpy().view(np.uint16), ref.int8_scale)
    assert np.array_equal(pools.fp16_pool.cpu().numpy().view(np.uint16), ref.fp16_pool)
    g = gK.cpu().numpy()
    assert np.array_equal(g.view(np.uint16), Ko) and np.array_equal(gV.cpu().numpy().view(np.uint16), Vo)
    # error bound of the symmetric quantiser on the INT8 rows of frame 0, layer 0: |x^ - x| <= s/2 + half an fp16 ulp of x^
    rows = idx[0, 1, :counts[0, 3]]
    x = hK[0, 0, rows].astype(np.float64).reshape(len(rows), HD // 128, 128)
    xh = g[0, 0, rows].astype(np.float64).reshape(x.shape)
    sc8 = ref.int8_scale[0, 0, off[0, 1]:off[0, 1] + len(rows)].view(np.float16).astype(np.float64)
    assert (np.abs(xh - x) <= sc8[..., None] * (0.5 + 2.0 ** -11) + np.abs(xh) * 2.0 ** -11).all()
    if wl.outlier_frac:
        assert np.abs(x).max() > 12.0                      # the x8 outliers are there

"""GPU parity: every stage of the CUDA path against the oracle on the same seeded bytes, through the C ABI."""
import numpy as np
import pytest

import oracle
from paper_2602_14236_b200 import binding as sc
from paper_2602_14236_b200 import synth

import gpu_util as gu

pytestmark = pytest.mark.gpu


def _ctx(**kw):
    base = dict(max_batch=16, chunk_frames=4, L=1)
    base.update(kw)
    return sc.Context(sc.salicache_default_params(**base))


@pytest.fixture(scope="module")
def wl1_frames():
    return synth.frames(1)


@pytest.fixture(scope="module")
def wl1_oracle_scores(wl1_frames):
    fr = wl1_frames
    dP = np.zeros((fr.shape[0], 576))
    dP[1:], fl = oracle.flow_score(fr[:-1], fr[1:], want_flow=True)
    s = oracle.saliency(fr)
    return dP, s, fl


# ------------------------------------------------------------------------------------- scores
def test_flow_score_matches_oracle_on_workload_1(wl1_frames, wl1_oracle_scores):
    ctx = _ctx()
    dP, s, fl = gu.gpu_scores(ctx, wl1_frames, want_flow=True)
    rdP, rs, rfl = wl1_oracle_scores
    # dense field (px): an auxiliary check beside the contract's tolerance on dP.  Single-precision terms, window sums
    # of 225 terms and a compensated 2x2 solve leave about 5e-6 px on fields of up to 3 px; the bound is twice that.
    assert np.abs(fl - rfl).max() < 1e-5
    gu.assert_scores_close(dP[1:], rdP[1:], "dP")
    gu.assert_scores_close(s, rs, "s")


def test_flow_score_independent_pairs_and_chunk_tail(wl1_frames, wl1_oracle_scores):
    """prev/cur given as separate buffers (no frame sharing), B = 7 over chunks of 4 + ragged 3."""
    import torch
    ctx = _ctx()
    prev = torch.from_numpy(wl1_frames[:-1].copy()).cuda()
    cur = torch.from_numpy(wl1_frames[1:].copy()).cuda()
    dP = torch.zeros((7, 576), dtype=torch.float32, device="cuda")
    sc.salicache_flow_score(ctx, prev, cur, 7, dP)
    torch.cuda.synchronize()
    gu.assert_scores_close(dP.cpu().numpy(), wl1_oracle_scores[0][1:], "dP (independent pairs)")


def test_identical_frames_score_exactly_zero():
    import torch
    ctx = _ctx()
    fr = synth.frames(2, T=1)
    both = torch.from_numpy(np.concatenate([fr, fr])).cuda()
    dP = torch.ones((1, 576), dtype=torch.float32, device="cuda")
    sc.salicache_flow_score(ctx, both[:1], both[1:], 1, dP)
    torch.cuda.synchronize()
    assert float(dP.abs().max()) == 0.0


def test_saliency_matches_oracle_on_sprites_and_pan():
    ctx = _ctx()
    for wl, t0 in ((2, 0), (3, 118), (5, 0)):
        fr = synth.frames(wl, T=3, t0=t0)
        _, s = gu.gpu_scores(ctx, fr)
        gu.assert_scores_close(s, oracle.saliency(fr), f"s workload {wl}")


def test_saliency_other_weights_clamp_per_pixel():
    ctx = _ctx(w_edge=1.0, w_color=1.0, canny_lo=30, canny_hi=90, sigma_ref=6.0)
    fr = synth.frames(2, T=2)
    _, s = gu.gpu_scores(ctx, fr)
    gu.assert_scores_close(s, oracle.saliency(fr, gu.oracle_params(ctx.params)), "s (clamped blend)")


def test_saliency_with_the_frame_adaptive_colour_term_matches_the_oracle():
    """The colour term measured against the frame's own contrast level (a second pass over the image): vivid frames,
    a nearly flat frame whose contrast lies under sigma_min, an entirely flat frame, and the anyres layout, where the
    frame and its base image are each normalised by their own statistic."""
    for kw in (dict(color_kappa=1.0), dict(color_kappa=1.7, w_edge=0.8, w_color=0.6)):
        ctx = _ctx(color_norm=1, **kw)
        p = gu.oracle_params(ctx.params)
        fr = np.concatenate([synth.frames(2, T=2), synth.frames(1, T=2, t0=2)])
        dim = (118 + (fr[0].astype(np.int32) - 118) // 64).astype(np.uint8)          # grey levels 116..119 only
        flat = np.full_like(fr[0], 90)
        fr = np.concatenate([fr, dim[None], flat[None]])
        _, s = gu.gpu_scores(ctx, fr)
        want = oracle.saliency(fr, p)
        gu.assert_scores_close(s, want, "s, frame-adaptive colour term")
        assert want[:4].max() > 0.3 and not s[5].any()
        assert not np.allclose(want[:4], oracle.saliency(fr[:4]), atol=1e-3)          # it is not the fixed reading
    ctx = sc.Context(sc.salicache_default_params(H=672, W=672, n_images=5, max_batch=2, chunk_frames=2, L=1, color_norm=1))
    p = gu.oracle_params(ctx.params)
    fr = synth.frames(4, T=2, t0=29)
    _, s = gu.gpu_scores(ctx, fr)
    base = np.stack([oracle.box_down2(f) for f in fr])
    rs_full, rs_base = oracle.saliency(fr, p), oracle.saliency(base, p)
    want = np.stack([oracle.anyres_tokens(rs_full[t], rs_base[t]) for t in range(2)])
    gu.assert_scores_close(s, want, "s anyres, frame-adaptive colour term")


def test_small_frame_and_single_frame_batches():
    ctx = _ctx(H=112, W=112)
    fr = synth.frames(1, T=3)[:, 100:212, 60:172].copy()
    dP, s = gu.gpu_scores(ctx, fr)
    gu.assert_scores_close(dP[1:], oracle.flow_score(fr[:-1], fr[1:]), "dP 112x112")
    gu.assert_scores_close(s, oracle.saliency(fr), "s 112x112")
    assert ctx.n_tok == 64


def test_hysteresis_iteration_cap_is_reported_not_hung():
    ctx = _ctx(hyst_max_iters=1, canny_lo=20, canny_hi=200)
    import torch
    fr = torch.from_numpy(synth.frames(2, T=1)).cuda()
    s = torch.zeros((1, 576), dtype=torch.float32, device="cuda")
    sc.salicache_saliency(ctx, fr, 1, s)
    assert sc.salicache_poll_status(ctx) == sc.E_NOCONVERGE
    assert sc.salicache_poll_status(ctx) == 0          # cleared by the poll


def test_redundant_frames_skip_the_spatial_branch(wl1_frames, wl1_oracle_scores):
    """Alg. 1: a frame with R_frame > theta_R is a pointer to its predecessor and is not scored."""
    import torch
    ctx = _ctx()
    rdP, rs, _ = wl1_oracle_scores
    dP32 = torch.from_numpy(rdP.astype(np.float32)).cuda()
    red = torch.full((8,), 7, dtype=torch.uint8, device="cuda")
    sc.salicache_frame_redundancy(ctx, dP32, 8, True, red)
    p = gu.oracle_params(ctx.params)
    want = np.array([oracle.select(rdP[t].astype(np.float32), rs[t].astype(np.float32), t > 0, p)[3] for t in range(8)])
    assert np.array_equal(red.cpu().numpy(), want) and want[0] == 0 and 0 < want.sum() < 8
    fr = torch.from_numpy(wl1_frames).cuda()
    s = torch.full((8, 576), -3.0, dtype=torch.float32, device="cuda")
    sc.salicache_saliency(ctx, fr, 8, s, red)
    torch.cuda.synchronize()
    got = s.cpu().numpy()
    assert (got[want == 1] == -3.0).all()                       # untouched
    gu.assert_scores_close(got[want == 0], rs[want == 0], "s of the scored frames")
    # and the decisions do not depend on the rows that were skipped
    out = gu.gpu_select(ctx, rdP.astype(np.float32), got)
    dec, idx, counts, r2, _ = gu.oracle_select_all(rdP.astype(np.float32), rs.astype(np.float32), p)
    near = gu.near_threshold(None, rs.astype(np.float32), p)
    assert np.array_equal(out["redundant"].cpu().numpy(), want)
    assert not ((out["decision"].cpu().numpy() != dec) & ~near).any()


# ------------------------------------------------------------------------------------- select
@pytest.mark.parametrize("background", ["int8", "int4", "four"])
def test_select_is_bit_exact_given_the_same_scores(wl1_oracle_scores, background):
    ctx = _ctx(**synth.thresholds(background))
    rdP, rs, _ = wl1_oracle_scores
    dP32, s32 = rdP.astype(np.float32), rs.astype(np.float32)
    s32[2, :3] = [ctx.params.tau_high, ctx.params.tau_med, ctx.params.tau_low]      # exactly on the thresholds
    dP32[2, 5] = ctx.params.tau_t
    out = gu.gpu_select(ctx, dP32, s32, fill0=(5, 0, 7))
    dec, idx, counts, red, off = gu.oracle_select_all(dP32, s32, gu.oracle_params(ctx.params))
    assert np.array_equal(out["decision"].cpu().numpy(), dec)
    assert np.array_equal(out["idx"].cpu().numpy(), idx)
    assert np.array_equal(out["counts"].cpu().numpy(), counts)
    assert np.array_equal(out["redundant"].cpu().numpy(), red)
    assert np.array_equal(out["row_offset"].cpu().numpy(), off + np.array([5, 0, 7]))
    tot = counts[:, [4, 3, 2]].sum(axis=0)
    assert np.array_equal(out["fill"].cpu().numpy(), tot + np.array([5, 0, 7]))
    assert (counts.sum(axis=1) == 576).all()
    assert counts[0, 0] == 0                          # the first frame never reuses


def test_row_offsets_of_a_batch_longer_than_one_sweep_of_the_scan():
    # 2500 frames: the device scans 1024 frames per sweep, so this batch takes three, the last one ragged
    ctx = _ctx(max_batch=2500, **synth.thresholds("four"))
    rng = np.random.default_rng(31)
    T = 2500
    dP = rng.uniform(0.0, 2.0 * ctx.params.tau_t, size=(T, 576)).astype(np.float32)
    s = rng.uniform(0.0, 1.0, size=(T, 576)).astype(np.float32)
    dP[700:720] = 0.0                                # a run of redundant frames: zero counts inside the scan
    fill0 = (3, (1 << 33) + 1, 11)                   # a running fill beyond 32 bits
    out = gu.gpu_select(ctx, dP, s, fill0=fill0)
    dec, idx, counts, red, off = gu.oracle_select_all(dP, s, gu.oracle_params(ctx.params))
    assert np.array_equal(out["counts"].cpu().numpy(), counts)
    assert np.array_equal(out["row_offset"].cpu().numpy(), off + np.array(fill0, np.int64))
    assert np.array_equal(out["fill"].cpu().numpy(), counts[:, [4, 3, 2]].sum(axis=0) + np.array(fill0, np.int64))
    assert red[700:720].all() and counts[:, 2:].sum() > 0


def test_pipeline_decisions_match_oracle_up_to_near_threshold_tokens(wl1_frames, wl1_oracle_scores):
    ctx = _ctx(**synth.thresholds("four"))
    dP, s = gu.gpu_scores(ctx, wl1_frames)
    out = gu.gpu_select(ctx, dP, s)
    rdP, rs, _ = wl1_oracle_scores
    rdP32, rs32 = rdP.astype(np.float32), rs.astype(np.float32)
    p = gu.oracle_params(ctx.params)
    dec, _, counts, red, _ = gu.oracle_select_all(rdP32, rs32, p)
    g_dec = out["decision"].cpu().numpy()
    near = gu.near_threshold(rdP32, rs32, p)
    diff = g_dec != dec
    print(f"near-threshold tokens: {int(near.sum())}, differing decisions: {int(diff.sum())}")
    frame_flip = out["redundant"].cpu().numpy() != red
    assert not frame_flip.any()
    assert not (diff & ~near).any()
    assert len(set(np.unique(dec))) >= 4              # the case exercises several categories


def test_source_frames_table_in_two_batches():
    import torch
    ctx = _ctx()
    rng = np.random.default_rng(9)
    dec = rng.integers(0, 5, (12, 576)).astype(np.uint8)
    dec[0][dec[0] == 0] = 1
    want = oracle.source_frames(dec)
    d_dec = torch.from_numpy(dec).cuda()
    carry = torch.full((576,), -1, dtype=torch.int32, device="cuda")
    src = torch.full((12, 576), -9, dtype=torch.int32, device="cuda")
    sc.salicache_source_frames(ctx, d_dec, 7, 0, carry, src)
    sc.salicache_source_frames(ctx, d_dec[7:], 5, 7, carry, src[7:])
    torch.cuda.synchronize()
    assert np.array_equal(src.cpu().numpy(), want)
    assert np.array_equal(carry.cpu().numpy(), want[-1])


def test_select_without_temporal_scores_and_empty_batch():
    ctx = _ctx()
    s = np.random.default_rng(0).uniform(0, 0.6, (3, 576)).astype(np.float32)
    out = gu.gpu_select(ctx, None, s, first_has_no_prev=False)
    dec, idx, counts, red, off = gu.oracle_select_all(None, s, gu.oracle_params(ctx.params))
    assert np.array_equal(out["decision"].cpu().numpy(), dec) and np.array_equal(out["idx"].cpu().numpy(), idx)
    assert not out["redundant"].cpu().numpy().any()
    import torch
    z = torch.zeros(1, device="cuda")
    sc.salicache_select(ctx, None, z, 0, True, z, z, z, z, z, z)      # B = 0: no launch, no error


# ------------------------------------------------------------------------------------- pack / unpack
def _pack_case(background, L=2, T=3, n_tok=576, ring=False, caps=None, seed=0, fill0=(0, 0, 0)):
    """Random scores -> oracle decisions; K/V from the workload generator; pools on both sides."""
    import torch
    ctx = _ctx(L=L, **synth.thresholds(background))
    rng = np.random.default_rng(seed)
    s = rng.uniform(0.0, 0.6, (T, n_tok)).astype(np.float32)
    dP = rng.uniform(0.0, 1.2, (T, n_tok)).astype(np.float32)
    if T > 2:
        dP[2] = 0.0                                    # a fully redundant frame stores nothing
    p = gu.oracle_params(ctx.params)
    dec, idx, counts, red, off = gu.oracle_select_all(dP, s, p)
    off = off + np.array(fill0, np.int64)
    KV = [synth.kv_numpy(2, t, L=L, n_tok=n_tok) for t in range(T)]
    K = np.stack([k for k, _ in KV]).view(np.uint16)
    V = np.stack([v for _, v in KV]).view(np.uint16)
    tot = counts[:, [4, 3, 2]].sum(axis=0)
    caps = caps or tuple(int(c) + 2 for c in tot)
    ref = oracle.Pools(L, 4096, 128, *caps, ring=int(ring))
    for t in range(T):
        oracle.pack_frame(K[t], V[t], idx[t], counts[t], off[t], ref)
    out = gu.gpu_select(ctx, dP, s, fill0=fill0)
    pools = sc.PoolSet(L, 4096, *caps, ring=ring)
    dK = torch.from_numpy(K.view(np.float16)).cuda()
    dV = torch.from_numpy(V.view(np.float16)).cuda()
    sc.salicache_pack_kv(ctx, dK, dV, L * n_tok * 4096, out["idx"], out["counts"], out["row_offset"], T, pools.c)
    torch.cuda.synchronize()
    return ctx, (K, V, dec, idx, counts, off, ref), (out, pools, dK, dV)


def _assert_pools_equal(pools, ref, caps):
    g = lambda t: t.cpu().numpy()
    if caps[0]:
        assert np.array_equal(g(pools.fp16_pool).view(np.uint16), ref.fp16_pool)
    if caps[1]:
        assert np.array_equal(g(pools.int8_codes), ref.int8_codes)
        assert np.array_equal(g(pools.int8_scale).view(np.uint16), ref.int8_scale)
    if caps[2]:
        assert np.array_equal(g(pools.int4_codes), ref.int4_codes)
        assert np.array_equal(g(pools.int4_sz).view(np.uint16), ref.int4_sz)


@pytest.mark.parametrize("background", ["int8", "int4", "four"])
def test_pack_codes_scales_and_layout_are_bit_exact(background):
    import torch
    ctx, (K, V, dec, idx, counts, off, ref), (out, pools, dK, dV) = _pack_case(background)
    assert sc.salicache_poll_status(ctx) == 0
    assert counts[2].sum() == counts[2][0] == 576      # the redundant frame is all REUSE
    _assert_pools_equal(pools, ref, pools.cap)
    # unpack: dense fp16, bit-exact against the oracle's dequantisation
    T, L, n_tok = K.shape[0], K.shape[1], K.shape[2]
    Ko = np.full(K.shape, 0x7E00, np.uint16)
    Vo = np.full(K.shape, 0x7E00, np.uint16)
    for t in range(T):
        oracle.unpack_frame(n_tok, idx[t], counts[t], dec[t], off[t], ref, True, Ko[t], Vo[t])
    gK = torch.from_numpy(np.full(K.shape, 0x7E00, np.uint16).view(np.float16)).cuda()
    gV = gK.clone()
    sc.salicache_unpack_kv(ctx, pools.c, out["idx"], out["counts"], out["decision"], out["row_offset"], T, True, gK, gV,
                           L * n_tok * 4096)
    torch.cuda.synchronize()
    assert np.array_equal(gK.cpu().numpy().view(np.uint16), Ko)
    assert np.array_equal(gV.cpu().numpy().view(np.uint16), Vo)
    # and the stated absolute bound against the input itself for the quantised tiers
    Kf = K.view(np.float16).astype(np.float32)
    Kg = gK.cpu().numpy().astype(np.float32)
    fp16_rows = dec == oracle.FP16
    assert np.array_equal(Kg.transpose(0, 2, 1, 3)[fp16_rows], Kf.transpose(0, 2, 1, 3)[fp16_rows])


def test_unpack_without_zero_fill_leaves_pruned_and_reused_rows_untouched():
    import torch
    ctx, (K, V, dec, idx, counts, off, ref), (out, pools, dK, dV) = _pack_case("four", L=1, T=2)
    gK = torch.full(K.shape, 3.0, dtype=torch.float16, device="cuda")
    gV = gK.clone()
    sc.salicache_unpack_kv(ctx, pools.c, out["idx"], out["counts"], None, out["row_offset"], 2, False, gK, gV,
                           576 * 4096)
    torch.cuda.synchronize()
    rows = gK.cpu().numpy()[:, 0]
    untouched = (dec == oracle.PRUNE) | (dec == oracle.REUSE)
    assert (rows[untouched] == 3.0).all() and untouched.any()
    assert not (rows[~untouched] == 3.0).all(axis=1).any()


def test_pack_ring_wraps_and_linear_pool_reports_overflow():
    # ring: the batch starts near the end of each pool and wraps to row 0 (no row is written twice)
    ctx, (K, V, dec, idx, counts, off, ref), (out, pools, dK, dV) = _pack_case(
        "int8", L=1, T=2, ring=True, caps=(700, 700, 0), fill0=(690, 1350, 0))
    assert sc.salicache_poll_status(ctx) == 0
    assert counts[:, 4].sum() > 10 and counts[:, 3].sum() > 50
    _assert_pools_equal(pools, ref, (700, 700, 0))
    ctx, (K, V, dec, idx, counts, off, ref), (out, pools, dK, dV) = _pack_case("int8", L=1, T=2, ring=False, caps=(40, 300, 0))
    assert sc.salicache_poll_status(ctx) == sc.E_CAPACITY
    _assert_pools_equal(pools, ref, (40, 300, 0))      # rows past the capacity are dropped on both sides


def test_pack_special_values():
    """All-zero rows, constant rows, tiny and huge magnitudes, negative zero."""
    import torch
    L, n_tok = 1, 576
    ctx = _ctx(L=L, **synth.thresholds("four"))
    rng = np.random.default_rng(4)
    K = rng.standard_normal((1, L, n_tok, 4096)).astype(np.float16)
    K[0, 0, 0] = 0.0
    K[0, 0, 1] = -0.0
    K[0, 0, 2] = 2.5
    K[0, 0, 3] *= np.float16(1e-4)
    K[0, 0, 4] *= np.float16(2000.0)
    K[0, 0, 5, :128] = 0.0
    K[0, 0, 5, 7] = -0.0
    K[0, 0, 6] = np.float16(6e-8)          # subnormal
    K[0, 0, 7, ::2] = 65504.0
    K[0, 0, 7, 1::2] = -65504.0
    V = K[:, :, ::-1].copy()
    for tier_s in (0.38, 0.30):            # all tokens INT8, then all INT4
        s = np.full((1, n_tok), tier_s, np.float32)
        dec, idx, counts, red, off = gu.oracle_select_all(None, s, gu.oracle_params(ctx.params))
        ref = oracle.Pools(L, 4096, 128, 1, 576, 576)
        oracle.pack_frame(K[0].view(np.uint16), V[0].view(np.uint16), idx[0], counts[0], off[0], ref)
        out = gu.gpu_select(ctx, None, s)
        pools = sc.PoolSet(L, 4096, 1, 576, 576)
        sc.salicache_pack_kv(ctx, torch.from_numpy(K).cuda(), torch.from_numpy(V).cuda(), n_tok * 4096, out["idx"],
                             out["counts"], out["row_offset"], 1, pools.c)
        torch.cuda.synchronize()
        _assert_pools_equal(pools, ref, (0, 576, 576))


@pytest.mark.parametrize("heads", [8, 2])
def test_pack_other_row_lengths(heads):
    """8 KV heads x 128 (the grouped-query shape of the paper's model) and a 256-element row."""
    import torch
    L, n_tok, HD = 2, 576, heads * 128
    ctx = _ctx(L=L, heads=heads, **synth.thresholds("four"))
    rng = np.random.default_rng(7)
    s = rng.uniform(0.0, 0.6, (2, n_tok)).astype(np.float32)
    K = rng.standard_normal((2, L, n_tok, HD)).astype(np.float16)
    V = rng.standard_normal((2, L, n_tok, HD)).astype(np.float16)
    dec, idx, counts, red, off = gu.oracle_select_all(None, s, gu.oracle_params(ctx.params))
    caps = tuple(int(c) + 1 for c in counts[:, [4, 3, 2]].sum(axis=0))
    ref = oracle.Pools(L, HD, 128, *caps)
    for t in range(2):
        oracle.pack_frame(K[t].view(np.uint16), V[t].view(np.uint16), idx[t], counts[t], off[t], ref)
    out = gu.gpu_select(ctx, None, s)
    pools = sc.PoolSet(L, HD, *caps)
    sc.salicache_pack_kv(ctx, torch.from_numpy(K).cuda(), torch.from_numpy(V).cuda(), L * n_tok * HD, out["idx"],
                         out["counts"], out["row_offset"], 2, pools.c)
    torch.cuda.synchronize()
    _assert_pools_equal(pools, ref, caps)
    Ko = np.zeros(K.shape, np.uint16)
    Vo = np.zeros(K.shape, np.uint16)
    for t in range(2):
        oracle.unpack_frame(n_tok, idx[t], counts[t], dec[t], off[t], ref, True, Ko[t], Vo[t])
    gK = torch.zeros(K.shape, dtype=torch.float16, device="cuda")
    gV = gK.clone()
    sc.salicache_unpack_kv(ctx, pools.c, out["idx"], out["counts"], out["decision"], out["row_offset"], 2, True, gK, gV,
                           L * n_tok * HD)
    torch.cuda.synchronize()
    assert np.array_equal(gK.cpu().numpy().view(np.uint16), Ko) and np.array_equal(gV.cpu().numpy().view(np.uint16), Vo)


def test_pack_with_one_group_per_token_row():
    """group = heads * head_dim: a single scale (and zero) per token row."""
    import torch
    L, n_tok, HD = 1, 576, 4096
    ctx = _ctx(L=L, group=HD, **synth.thresholds("four"))
    rng = np.random.default_rng(11)
    s = rng.uniform(0.0, 0.6, (2, n_tok)).astype(np.float32)
    KV = [synth.kv_numpy(2, t, L=L) for t in range(2)]
    K = np.stack([k for k, _ in KV])
    V = np.stack([v for _, v in KV])
    K[0, 0, 3] = 0.0                                   # an all-zero row: scale 1, codes 0
    dec, idx, counts, red, off = gu.oracle_select_all(None, s, gu.oracle_params(ctx.params))
    caps = tuple(int(c) + 1 for c in counts[:, [4, 3, 2]].sum(axis=0))
    ref = oracle.Pools(L, HD, HD, *caps)
    for t in range(2):
        oracle.pack_frame(K[t].view(np.uint16), V[t].view(np.uint16), idx[t], counts[t], off[t], ref)
    out = gu.gpu_select(ctx, None, s)
    pools = sc.PoolSet(L, HD, *caps, G=HD)
    assert pools.int8_scale.shape[-1] == 1 and pools.int4_sz.shape[-2] == 1
    sc.salicache_pack_kv(ctx, torch.from_numpy(K).cuda(), torch.from_numpy(V).cuda(), L * n_tok * HD, out["idx"],
                         out["counts"], out["row_offset"], 2, pools.c)
    torch.cuda.synchronize()
    _assert_pools_equal(pools, ref, caps)
    Ko = np.zeros(K.shape, np.uint16)
    Vo = np.zeros(K.shape, np.uint16)
    for t in range(2):
        oracle.unpack_frame(n_tok, idx[t], counts[t], dec[t], off[t], ref, True, Ko[t], Vo[t])
    gK = torch.zeros(K.shape, dtype=torch.float16, device="cuda")
    gV = gK.clone()
    sc.salicache_unpack_kv(ctx, pools.c, out["idx"], out["counts"], out["decision"], out["row_offset"], 2, True, gK, gV,
                           L * n_tok * HD)
    torch.cuda.synchronize()
    assert np.array_equal(gK.cpu().numpy().view(np.uint16), Ko) and np.array_equal(gV.cpu().numpy().view(np.uint16), Vo)


def test_dequantised_values_within_the_stated_bound_of_the_oracle():
    import torch
    ctx, (K, V, dec, idx, counts, off, ref), (out, pools, dK, dV) = _pack_case("four", L=1, T=1, seed=3)
    Ko = np.zeros(K.shape, np.uint16)
    Vo = np.zeros(K.shape, np.uint16)
    oracle.unpack_frame(576, idx[0], counts[0], dec[0], off[0], ref, True, Ko[0], Vo[0])
    gK = torch.zeros(K.shape, dtype=torch.float16, device="cuda")
    gV = gK.clone()
    sc.salicache_unpack_kv(ctx, pools.c, out["idx"], out["counts"], out["decision"], out["row_offset"], 1, True, gK, gV,
                           576 * 4096)
    torch.cuda.synchronize()
    d = np.abs(gK.cpu().numpy().astype(np.float64) - Ko.view(np.float16).astype(np.float64))
    assert d.max() <= 1e-3


# ------------------------------------------------------------------------------------- argument errors
def test_argument_errors_are_returned_not_raised_on_the_device():
    import torch
    ctx = _ctx()
    lib = sc.lib()
    fr = torch.zeros((2, 336, 336, 3), dtype=torch.uint8, device="cuda")
    dP = torch.zeros((2, 576), dtype=torch.float32, device="cuda")
    h = ctx.handle
    assert lib.salicache_flow_score(h, None, fr.data_ptr(), 1, dP.data_ptr(), None, None) == sc.E_NULL
    assert lib.salicache_flow_score(h, fr.data_ptr(), fr.data_ptr(), 17, dP.data_ptr(), None, None) == sc.E_SHAPE
    assert lib.salicache_flow_score(h, fr.data_ptr() + 3, fr.data_ptr(), 1, dP.data_ptr(), None, None) == sc.E_ALIGN
    assert lib.salicache_saliency(h, fr.data_ptr(), -1, dP.data_ptr(), None, None) == sc.E_SHAPE
    assert lib.salicache_saliency(h, fr.data_ptr(), 1, None, None, None) == sc.E_NULL
    assert lib.salicache_frame_redundancy(h, dP.data_ptr(), 1, 1, None, None) == sc.E_NULL
    pools = sc.PoolSet(1, 4096, 4, 4, 4)
    bad = sc.Pools(None, pools.int8_codes.data_ptr(), pools.int8_scale.data_ptr(), pools.int4_codes.data_ptr(),
                   pools.int4_sz.data_ptr(), 4, 4, 4, 0)
    import ctypes
    kv = torch.zeros((1, 576, 4096), dtype=torch.float16, device="cuda")
    i32 = torch.zeros((3, 576), dtype=torch.int32, device="cuda")
    i64 = torch.zeros((3,), dtype=torch.int64, device="cuda")
    assert lib.salicache_pack_kv(h, kv.data_ptr(), kv.data_ptr(), 576 * 4096, i32.data_ptr(), i32.data_ptr(),
                                 i64.data_ptr(), 1, ctypes.byref(bad), None) == sc.E_NULL
    assert lib.salicache_pack_kv(h, kv.data_ptr() + 2, kv.data_ptr(), 576 * 4096, i32.data_ptr(), i32.data_ptr(),
                                 i64.data_ptr(), 1, ctypes.byref(pools.c), None) == sc.E_ALIGN
    assert lib.salicache_pack_kv(h, kv.data_ptr(), kv.data_ptr(), 100, i32.data_ptr(), i32.data_ptr(),
                                 i64.data_ptr(), 2, ctypes.byref(pools.c), None) == sc.E_SHAPE
    # budget bookkeeping: ring pools need the running fill; counts and flags must be there
    u8 = torch.zeros((4,), dtype=torch.uint8, device="cuda")
    ring = sc.PoolSet(1, 4096, 4, 4, 4, ring=True)              # no fill attached
    assert lib.salicache_frames_resident(h, i32.data_ptr(), i64.data_ptr(), 1, ctypes.byref(ring.c), u8.data_ptr(), None) == sc.E_NULL
    assert lib.salicache_frames_resident(h, None, i64.data_ptr(), 1, ctypes.byref(pools.c), u8.data_ptr(), None) == sc.E_NULL
    assert lib.salicache_frames_resident(h, i32.data_ptr(), i64.data_ptr(), -1, ctypes.byref(pools.c), u8.data_ptr(), None) == sc.E_SHAPE
    assert lib.salicache_tokens_live(h, i32.data_ptr(), 1, 0, None, 1, u8.data_ptr(), None) == sc.E_NULL
    assert lib.salicache_tokens_live(h, i32.data_ptr(), 1, -2, u8.data_ptr(), 1, u8.data_ptr(), None) == sc.E_SHAPE
    # parameters of the frame-adaptive colour term
    import pytest as _pt
    for kw in (dict(color_norm=2), dict(color_norm=1, color_kappa=0.0), dict(color_norm=1, color_sigma_min=-1.0)):
        with _pt.raises(sc.SalicacheError) as e:
            _ctx(**kw)
        assert e.value.status == sc.E_PARAM
    noal = sc.salicache_default_params(L=1, color_norm=1)
    assert lib.salicache_saliency_noalloc(ctypes.byref(noal), fr.data_ptr(), 1, dP.data_ptr(), None, None) == sc.E_PARAM
    torch.cuda.synchronize()
    assert sc.salicache_poll_status(ctx) == 0

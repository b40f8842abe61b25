"""GPU parity of the budget bookkeeping: ring pools smaller than the stream, residency of frames and tokens, and
unpacking that returns zeros (never a newer frame's rows) for what has been evicted.  Through the C ABI."""
import numpy as np
import pytest

import oracle
from paper_2602_14236_b200 import binding as sc
from paper_2602_14236_b200 import synth

import gpu_util as gu

pytestmark = pytest.mark.gpu


def test_ring_budget_residency_and_eviction_safe_unpack():
    import torch
    L, T, n_tok, HD = 2, 7, 576, 4096
    fr = np.concatenate([synth.frames(5, T=4, t0=600), synth.frames(5, T=3, t0=297)])      # 8 px pan, then static frames
    ctx = sc.Context(sc.salicache_default_params(max_batch=8, chunk_frames=4, L=L, **synth.thresholds("int4")))
    dP, s = gu.gpu_scores(ctx, fr)
    dP[4] = 5.0                                              # the cut between the two clips: every patch moved
    out = gu.gpu_select(ctx, dP, s)
    g_idx, g_counts, g_off, g_dec = (out[k].cpu().numpy() for k in ("idx", "counts", "row_offset", "decision"))
    fill = out["fill"]
    h_fill = fill.cpu().numpy()
    assert g_counts[5:, 0].min() == n_tok                    # the static frames are reused entirely
    cap16, cap4 = 8, 1300                                    # a little over two frames of INT4 rows
    KV = [synth.kv_numpy(5, t, L=L) for t in range(T)]
    ref = oracle.Pools(L, HD, 128, cap16, 1, cap4, ring=1)
    pools = sc.PoolSet(L, HD, cap16, 1, cap4, ring=True, fill=fill)
    for t in range(T):
        Kt, Vt = KV[t]
        oracle.pack_frame(Kt.view(np.uint16), Vt.view(np.uint16), g_idx[t], g_counts[t], g_off[t], ref)
        sc.salicache_pack_kv(ctx, torch.from_numpy(Kt).cuda(), torch.from_numpy(Vt).cuda(), L * n_tok * HD,
                             out["idx"][t:], out["counts"][t:], out["row_offset"][t:], 1, pools.c)
    torch.cuda.synchronize()
    assert sc.salicache_poll_status(ctx) == 0
    assert np.array_equal(pools.int4_codes.cpu().numpy(), ref.int4_codes)
    # residency of the frames
    caps = np.array([cap16, 1, cap4], np.int64)
    want_res = oracle.frames_resident(g_counts, g_off, caps, True, h_fill)
    d_res = torch.full((T,), 7, dtype=torch.uint8, device="cuda")
    sc.salicache_frames_resident(ctx, out["counts"], out["row_offset"], T, pools.c, d_res)
    assert np.array_equal(d_res.cpu().numpy(), want_res)
    assert want_res.tolist() == [0, 0, 1, 1, 1, 1, 1] or (want_res[0] == 0 and want_res[4] == 1)
    # tokens: the static frames reuse frame 4's entries; had frame 4 been evicted they would be dead with it
    carry = torch.full((n_tok,), -1, dtype=torch.int32, device="cuda")
    src = torch.zeros((T, n_tok), dtype=torch.int32, device="cuda")
    sc.salicache_source_frames(ctx, out["decision"], T, 0, carry, src)
    live = torch.full((T, n_tok), 9, dtype=torch.uint8, device="cuda")
    sc.salicache_tokens_live(ctx, src, T, 0, d_res, T, live)
    want_src = oracle.source_frames(g_dec)
    assert np.array_equal(src.cpu().numpy(), want_src)
    assert np.array_equal(live.cpu().numpy(), oracle.tokens_live(want_src, 0, want_res))
    fake = want_res.copy()
    fake[4] = 0
    sc.salicache_tokens_live(ctx, src, T, 0, torch.from_numpy(fake).cuda(), T, live)
    torch.cuda.synchronize()
    assert not live.cpu().numpy()[5:].any()
    # unpack: evicted rows come back as zeros with E_EVICTED, surviving frames bit-equal, on both sides
    for t in range(T):
        Ko = torch.full((L, n_tok, HD), 1.5, dtype=torch.float16, device="cuda")
        Vo = torch.full((L, n_tok, HD), 1.5, dtype=torch.float16, device="cuda")
        sc.salicache_unpack_kv(ctx, pools.c, out["idx"][t:], out["counts"][t:], out["decision"][t:], out["row_offset"][t:], 1,
                               False, Ko, Vo, L * n_tok * HD)
        torch.cuda.synchronize()
        status = sc.salicache_poll_status(ctx)
        rK = np.full((L, n_tok, HD), 0x3E00, np.uint16)
        rV = np.full((L, n_tok, HD), 0x3E00, np.uint16)
        rst = oracle.unpack_frame(n_tok, g_idx[t], g_counts[t], g_dec[t], g_off[t], ref, False, rK, rV, fill=h_fill)
        assert np.array_equal(Ko.cpu().numpy().view(np.uint16), rK) and np.array_equal(Vo.cpu().numpy().view(np.uint16), rV), t
        stored = int(g_counts[t, 2:5].sum())
        assert status == (sc.E_EVICTED if rst == -9 else 0), t
        if stored and not want_res[t]:
            assert rst == -9
    # without the fill the library cannot know: the caller is then responsible (documented); with linear pools the flag is ignored
    assert want_res[:2].tolist() == [0, 0]


def test_one_call_that_overruns_the_ring_keeps_the_newest_rows():
    """A single store call with more rows than a ring holds: the rows a later row of the same call lands on are
    skipped, so the pool ends up with the newest rows, exactly as the oracle's frame-by-frame ring."""
    import torch
    L, T, n_tok, HD = 1, 5, 576, 4096
    fr = synth.frames(5, T=T, t0=600)
    ctx = sc.Context(sc.salicache_default_params(max_batch=8, chunk_frames=4, L=L, **synth.thresholds("int4")))
    dP, s = gu.gpu_scores(ctx, fr)
    out = gu.gpu_select(ctx, dP, s)
    g_idx, g_counts, g_off = (out[k].cpu().numpy() for k in ("idx", "counts", "row_offset"))
    cap16, cap4 = 5, 777
    assert g_counts[:, 2].sum() > 3 * cap4
    KV = [synth.kv_numpy(5, t, L=L) for t in range(T)]
    K = np.stack([k for k, _ in KV])
    V = np.stack([v for _, v in KV])
    ref = oracle.Pools(L, HD, 128, cap16, 1, cap4, ring=1)
    for t in range(T):
        oracle.pack_frame(K[t].view(np.uint16), V[t].view(np.uint16), g_idx[t], g_counts[t], g_off[t], ref)
    for trial in range(3):                                   # the outcome does not depend on scheduling
        pools = sc.PoolSet(L, HD, cap16, 1, cap4, ring=True)
        sc.salicache_pack_kv(ctx, torch.from_numpy(K).cuda(), torch.from_numpy(V).cuda(), L * n_tok * HD, out["idx"],
                             out["counts"], out["row_offset"], T, pools.c)
        torch.cuda.synchronize()
        assert sc.salicache_poll_status(ctx) == 0
        assert np.array_equal(pools.int4_codes.cpu().numpy(), ref.int4_codes)
        assert np.array_equal(pools.int4_sz.cpu().numpy().view(np.uint16), ref.int4_sz)
        assert np.array_equal(pools.fp16_pool.cpu().numpy().view(np.uint16), ref.fp16_pool)

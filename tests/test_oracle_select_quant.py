"""Pins of the oracle's decision rule (Eq. 6, Eq. 8, Alg. 1), quantisers (Sec. IV-B) and accounting (Eq. 3)."""
import numpy as np
import pytest

import oracle
from oracle import FP16, INT4, INT8, PRUNE, REUSE


# ----------------------------------------------------------------------------- select
def _select_brute(dP, s, has_prev, p):
    """Alg. 1 written token by token in plain Python."""
    n = len(s)
    f32 = np.float32
    static = [has_prev and f32(dP[i]) < f32(p.tau_t) for i in range(n)]
    R = f32(sum(static)) / f32(n) if has_prev else f32(0)
    redundant = bool(has_prev and R > f32(p.theta_R))
    dec = []
    for i in range(n):
        if redundant or (p.patch_reuse and static[i]):
            dec.append(REUSE)
        elif f32(s[i]) > f32(p.tau_high):
            dec.append(FP16)
        elif f32(s[i]) > f32(p.tau_med):
            dec.append(INT8)
        elif f32(s[i]) > f32(p.tau_low):
            dec.append(INT4)
        else:
            dec.append(PRUNE)
    return dec, redundant


@pytest.mark.parametrize("has_prev", [False, True])
@pytest.mark.parametrize("patch_reuse", [0, 1])
def test_select_brute_force_with_values_on_the_thresholds(has_prev, patch_reuse):
    p = oracle.Params(patch_reuse=patch_reuse)
    rng = np.random.default_rng(5)
    n = 576
    s = rng.uniform(0, 0.6, n).astype(np.float32)
    dP = rng.uniform(0, 1.0, n).astype(np.float32)
    s[:6] = [p.tau_high, p.tau_med, p.tau_low, np.nextafter(np.float32(p.tau_high), np.float32(1)),
             np.nextafter(np.float32(p.tau_med), np.float32(1)), np.nextafter(np.float32(p.tau_low), np.float32(1))]
    dP[:8] = 2.0
    dP[8] = p.tau_t                      # not static: the test is strict
    dP[9] = np.nextafter(np.float32(p.tau_t), np.float32(0))
    dec, idx, counts, red, R = oracle.select(dP, s, has_prev, p)
    ref, ref_red = _select_brute(dP, s, has_prev, p)
    assert list(dec) == ref and red == int(ref_red)
    assert list(dec[:6]) == [INT8, INT4, PRUNE, FP16, INT8, INT4]
    if has_prev and patch_reuse:
        assert dec[9] == REUSE and dec[8] != REUSE
    assert counts.sum() == n
    for tier, code in enumerate((FP16, INT8, INT4)):
        lst = idx[tier][:counts[code]]
        assert list(lst) == [i for i in range(n) if dec[i] == code]
        assert np.all(idx[tier][counts[code]:] == -1)


def test_select_frame_redundancy_is_strict_and_first_frame_never_reuses():
    n = 100
    s = np.full(n, 0.5, np.float32)
    for n_static, expect in ((90, 0), (91, 1)):           # theta_R = 0.90: R must exceed it
        dP = np.concatenate([np.zeros(n_static), np.ones(n - n_static)]).astype(np.float32)
        dec, idx, counts, red, R = oracle.select(dP, s, True, oracle.Params())
        assert red == expect and R == np.float32(n_static) / np.float32(n)
        if expect:
            assert np.all(dec == REUSE) and counts[REUSE] == n and counts[1:].sum() == 0
    dec, _, counts, red, _ = oracle.select(np.zeros(n, np.float32), s, False, oracle.Params())
    assert red == 0 and counts[REUSE] == 0 and np.all(dec == FP16)


def test_identical_frames_reuse_everything():
    from paper_2602_14236_b200 import synth
    fr = synth.texture(3, 56, 56)
    dP = oracle.flow_score(fr[None], fr[None])[0].astype(np.float32)
    s = oracle.saliency(fr).astype(np.float32)
    dec, _, counts, red, R = oracle.select(dP, s, True, oracle.Params())
    assert R == 1.0 and red == 1 and counts[REUSE] == 16 and np.all(dec == REUSE)


# ----------------------------------------------------------------------------- fp16 conversion
def test_half_to_float_matches_numpy_on_every_bit_pattern():
    bits = np.arange(65536, dtype=np.uint16)
    ours = oracle.half_to_float(bits)
    ref = bits.view(np.float16).astype(np.float32)
    both_nan = np.isnan(ours) & np.isnan(ref)
    assert np.array_equal(ours[~both_nan].view(np.uint32), ref[~both_nan].view(np.uint32))


def test_float_to_half_matches_numpy():
    rng = np.random.default_rng(0)
    x = np.concatenate([
        rng.standard_normal(20000).astype(np.float32) * 3,
        (rng.standard_normal(5000) * 1e-6).astype(np.float32),           # subnormal halves
        np.array([0.0, -0.0, 65504, 65519.99, 65520, 1e6, 2.0 ** -24, 2.0 ** -25, np.nextafter(np.float32(2.0 ** -25), np.float32(1)),
                  2.0 ** -14, np.nextafter(np.float32(2.0 ** -14), np.float32(0)), np.inf, -np.inf], np.float32),
        # exact ties between neighbouring halves
        (np.arange(1024, 3072, dtype=np.float32) + 0.5) / 1024.0,
        np.arange(0, 200, dtype=np.float32) * np.float32(2.0 ** -25),
    ])
    with np.errstate(over="ignore"):
        ref = x.astype(np.float16).view(np.uint16)
    assert np.array_equal(oracle.float_to_half(x), ref)


# ----------------------------------------------------------------------------- quantisers
def _h(x):
    return np.asarray(x, np.float16).view(np.uint16)


def _f(bits):
    return np.asarray(bits, np.uint16).view(np.float16).astype(np.float64)


def test_int8_hand_example_pins_rounding_and_scale():
    x = np.zeros(128, np.float16)
    x[:8] = [127, -127, 63.5, 0.5, 1.5, 2.5, -0.5, -2.5]     # amax 127 -> s = 1
    q, s16 = oracle.quant_int8_group(_h(x))
    assert s16 == 0x3C00
    assert list(q[:8]) == [127, -127, 64, 0, 2, 2, 0, -2]    # round half to even
    assert np.all(q[8:] == 0)


def test_int4_hand_example_pins_nibble_order_zero_point_and_rounding():
    x = (np.arange(128) % 16).astype(np.float16) + 3           # min 3, max 18 -> s = 1, z = 3
    packed, s16, z16 = oracle.quant_int4_group(_h(x))
    assert s16 == 0x3C00 and z16 == int(_h([3.0])[0])
    assert list(packed[:8]) == [(2 * j) | ((2 * j + 1) << 4) for j in range(8)]
    x2 = np.zeros(128, np.float16)
    x2[:6] = [15, 0.5, 1.5, 2.5, 14.5, 13.5]
    packed, s16, z16 = oracle.quant_int4_group(_h(x2))
    codes = np.stack([packed & 15, packed >> 4], 1).ravel()
    assert s16 == 0x3C00 and z16 == 0 and list(codes[:6]) == [15, 0, 2, 2, 14, 14]


@pytest.mark.parametrize("G", [128, 4096])
def test_quantiser_error_bounds_and_extremes(G):
    rng = np.random.default_rng(G)
    for trial in range(20):
        scale = 10.0 ** rng.uniform(-3, 2)
        x = (rng.standard_normal(G) * scale).astype(np.float16)
        xf = x.astype(np.float64)
        q, s16 = oracle.quant_int8_group(_h(x))
        s = float(_f([s16])[0])
        assert np.all(np.abs(xf - q.astype(np.float64) * s) <= s / 2 * (1 + 2.0 ** -10) + 1e-12)
        i = int(np.argmax(np.abs(xf)))
        assert abs(int(q[i])) == 127 and np.sign(q[i]) == np.sign(xf[i])
        xh = _f(oracle.dequant_int8_group(q, s16))
        ulp = np.spacing(np.abs(xh).astype(np.float16)).astype(np.float64)
        assert np.all(np.abs(xh - xf) <= s / 2 * (1 + 2.0 ** -10) + ulp / 2 + 1e-12)

        packed, s16, z16 = oracle.quant_int4_group(_h(x))
        s, z = float(_f([s16])[0]), float(_f([z16])[0])
        codes = np.stack([packed & 15, packed >> 4], 1).ravel().astype(np.float64)
        assert z == xf.min()
        assert codes[int(np.argmin(xf))] == 0 and codes[int(np.argmax(xf))] == 15
        # the stored scale is (max-min)/15 rounded to fp16, so the top of the range may be clamped by up to
        # 15 * (half an fp16 ulp of s); inside the range the error is at most s/2
        slack = 15 * np.spacing(np.float16(s)).astype(np.float64) / 2
        assert np.all(np.abs(xf - (codes * s + z)) <= s / 2 * (1 + 2.0 ** -10) + slack + 1e-12)
        xh = _f(oracle.dequant_int4_group(packed, s16, z16))
        ulp = np.spacing(np.abs(xh).astype(np.float16)).astype(np.float64)
        assert np.all(np.abs(xh - xf) <= s / 2 * (1 + 2.0 ** -10) + slack + ulp / 2 + 1e-12)


def test_quantiser_special_groups():
    zero = np.zeros(128, np.float16)
    q, s16 = oracle.quant_int8_group(_h(zero))
    assert s16 == 0x3C00 and not q.any()
    packed, s16, z16 = oracle.quant_int4_group(_h(zero))
    assert s16 == 0x3C00 and z16 == 0 and not packed.any()
    const = np.full(128, -2.75, np.float16)
    packed, s16, z16 = oracle.quant_int4_group(_h(const))
    assert not packed.any() and np.array_equal(oracle.dequant_int4_group(packed, s16, z16), _h(const))
    negz = np.zeros(128, np.float16)
    negz[0] = -0.0
    negz[1] = 4.0
    assert oracle.quant_int4_group(_h(negz))[2] == 0        # a zero minimum is stored as +0
    # values already on the grid reproduce exactly
    grid = (np.arange(128) % 255 - 127).astype(np.float16) * np.float16(0.25)
    grid[0] = 127 * 0.25
    q, s16 = oracle.quant_int8_group(_h(grid))
    assert np.array_equal(oracle.dequant_int8_group(q, s16), _h(grid))
    grid4 = (np.arange(128) % 16).astype(np.float16) * np.float16(0.5) - 1
    packed, s16, z16 = oracle.quant_int4_group(_h(grid4))
    assert np.array_equal(oracle.dequant_int4_group(packed, s16, z16), _h(grid4))


def test_int8_is_odd_symmetric():
    rng = np.random.default_rng(9)
    x = rng.standard_normal(128).astype(np.float16)
    q1, s1 = oracle.quant_int8_group(_h(x))
    q2, s2 = oracle.quant_int8_group(_h(-x))
    assert s1 == s2 and np.array_equal(q1, -q2)


# ----------------------------------------------------------------------------- pack / unpack
def _frame_case(L=2, n_tok=24, HD=256, G=128, seed=1):
    rng = np.random.default_rng(seed)
    K = rng.standard_normal((L, n_tok, HD)).astype(np.float16).view(np.uint16)
    V = rng.standard_normal((L, n_tok, HD)).astype(np.float16).view(np.uint16)
    s = rng.uniform(0, 0.6, n_tok).astype(np.float32)
    dP = rng.uniform(0, 1, n_tok).astype(np.float32)
    dec, idx, counts, _, _ = oracle.select(dP, s, True, oracle.Params())
    return K, V, dec, idx, counts


@pytest.mark.parametrize("ring", [0, 1])
def test_pack_layout_and_unpack_roundtrip(ring):
    L, n_tok, HD, G = 2, 24, 256, 128
    K, V, dec, idx, counts = _frame_case(L, n_tok, HD, G)
    assert min(counts) > 0
    caps = (counts[FP16] + 3, counts[INT8] + 2, max(counts[INT4] - 1, 1) if ring else counts[INT4] + 1)
    pools = oracle.Pools(L, HD, G, *[int(c) for c in caps], ring=ring)
    off = np.array([2, 1, 0], np.int64)
    assert oracle.pack_frame(K, V, idx, counts, off, pools) == 0
    for l in range(L):
        for kv, src in enumerate((K, V)):
            for j in range(counts[FP16]):
                assert np.array_equal(pools.fp16_pool[l, kv, 2 + j], src[l, idx[0, j]])
            for j in range(counts[INT8]):
                tok = idx[1, j]
                for g in range(HD // G):
                    q, s16 = oracle.quant_int8_group(src[l, tok, g * G:(g + 1) * G])
                    assert np.array_equal(pools.int8_codes[l, kv, 1 + j, g * G:(g + 1) * G], q)
                    assert pools.int8_scale[l, kv, 1 + j, g] == s16
            j = counts[INT4] - 1                     # with ring=1 the last int4 row wraps to row 0
            row = (j % caps[2]) if ring else j
            tok = idx[2, j]
            pk, s16, z16 = oracle.quant_int4_group(src[l, tok, :G])
            assert np.array_equal(pools.int4_codes[l, kv, row, :G // 2], pk)
            assert tuple(pools.int4_sz[l, kv, row, 0]) == (s16, z16)
    Ko = np.full((L, n_tok, HD), 0x7E00, np.uint16)
    Vo = np.full((L, n_tok, HD), 0x7E00, np.uint16)
    assert oracle.unpack_frame(n_tok, idx, counts, dec, off, pools, True, Ko, Vo) == 0
    Kf, Kof = K.view(np.float16).astype(np.float64), Ko.view(np.float16).astype(np.float64)
    for i in range(n_tok):
        if dec[i] == FP16:
            assert np.array_equal(Ko[:, i], K[:, i])
        elif dec[i] == PRUNE:
            assert not Ko[:, i].any()
        elif dec[i] == REUSE:
            assert np.all(Ko[:, i] == 0x7E00)
    # quantised rows, bit for bit: every group of every row of both tensors is the group dequantiser applied to
    # the codes and the scale / zero found at the pool row that this test locates itself, (off + j) mod cap
    for kv, (out, src) in enumerate(((Ko, K), (Vo, V))):
        for l in range(L):
            for j in range(counts[INT8]):
                tok, row = idx[1, j], 1 + j
                for g in range(HD // G):
                    want = oracle.dequant_int8_group(pools.int8_codes[l, kv, row, g * G:(g + 1) * G], int(pools.int8_scale[l, kv, row, g]))
                    assert np.array_equal(out[l, tok, g * G:(g + 1) * G], want)
            for j in range(counts[INT4]):
                tok, row = idx[2, j], (j % caps[2]) if ring else j
                if ring and j + caps[2] < counts[INT4]:
                    continue                                  # this row was overwritten by a later row of the same frame
                for g in range(HD // G):
                    want = oracle.dequant_int4_group(pools.int4_codes[l, kv, row, g * G // 2:(g + 1) * G // 2],
                                                     int(pools.int4_sz[l, kv, row, g, 0]), int(pools.int4_sz[l, kv, row, g, 1]))
                    assert np.array_equal(out[l, tok, g * G:(g + 1) * G], want)
                    x = src[l, tok, g * G:(g + 1) * G].view(np.float16).astype(np.float64)
                    sc = float(np.array(pools.int4_sz[l, kv, row, g, 0], np.uint16).view(np.float16))
                    assert np.max(np.abs(want.view(np.float16).astype(np.float64) - x)) <= sc * (0.5 + 2.0 ** -9) + 2.0 ** -10 * np.abs(x).max()


def test_unpack_uses_the_scale_of_its_own_group_and_plane():
    """Groups, layers and tensors with very different ranges: a scale taken from the wrong group, layer or tensor
    would be off by a factor of 2 or more, far outside the quantiser's error bound."""
    L, n_tok, HD, G = 3, 16, 512, 128
    rng = np.random.default_rng(21)
    K = rng.standard_normal((L, n_tok, HD))
    V = rng.standard_normal((L, n_tok, HD))
    for l in range(L):
        for g in range(HD // G):
            K[l, :, g * G:(g + 1) * G] *= 2.0 ** (g + 4 * l - 6)
            V[l, :, g * G:(g + 1) * G] *= 2.0 ** (3 - g - 2 * l)
    K, V = K.astype(np.float16).view(np.uint16), V.astype(np.float16).view(np.uint16)
    dec = (np.arange(n_tok) % 3 + 2).astype(np.uint8)             # INT4, INT8, FP16 in turn
    idx = np.full((3, n_tok), -1, np.int32)
    counts = np.zeros(5, np.int32)
    for tier, code in enumerate((FP16, INT8, INT4)):
        toks = np.nonzero(dec == code)[0]
        idx[tier, :len(toks)] = toks
        counts[code] = len(toks)
    pools = oracle.Pools(L, HD, G, 8, 8, 8)
    off = np.zeros(3, np.int64)
    assert oracle.pack_frame(K, V, idx, counts, off, pools) == 0
    Ko, Vo = np.zeros_like(K), np.zeros_like(V)
    assert oracle.unpack_frame(n_tok, idx, counts, dec, off, pools, False, Ko, Vo) == 0
    for out, src in ((Ko, K), (Vo, V)):
        x = src.view(np.float16).astype(np.float64).reshape(L, n_tok, HD // G, G)
        y = out.view(np.float16).astype(np.float64).reshape(L, n_tok, HD // G, G)
        rng_ = x.max(axis=-1) - x.min(axis=-1)
        amax = np.abs(x).max(axis=-1)
        err = np.abs(y - x).max(axis=-1)
        is8, is4 = (dec == INT8)[None, :, None], (dec == INT4)[None, :, None]
        assert np.all(err[np.broadcast_to(is8, err.shape)] <= (amax / 127 * 0.5 * (1 + 2.0 ** -8) + amax * 2.0 ** -10)[np.broadcast_to(is8, err.shape)])
        assert np.all(err[np.broadcast_to(is4, err.shape)] <= (rng_ / 15 * 0.5 * (1 + 2.0 ** -8) + amax * 2.0 ** -10)[np.broadcast_to(is4, err.shape)])
        assert np.array_equal(out[:, dec == FP16], src[:, dec == FP16])


def test_anyres_token_order_on_hand_written_grids():
    """Base image first, then tiles (0,0), (0,1), (1,0), (1,1), each row-major."""
    assert oracle.anyres_tokens([1, 2, 3, 4], [9], tg=1).tolist() == [9, 1, 2, 3, 4]
    full = np.arange(16).reshape(4, 4)          # rows 0 1 2 3 / 4 5 6 7 / 8 9 10 11 / 12 13 14 15
    want = [100, 101, 102, 103, 0, 1, 4, 5, 2, 3, 6, 7, 8, 9, 12, 13, 10, 11, 14, 15]
    assert oracle.anyres_tokens(full, [100, 101, 102, 103], tg=2).tolist() == want
    # the frame of workload 4: token 576 is the top-left patch of the frame, 576 + 24 starts its second patch row,
    # 2 * 576 is patch (0, 24), 3 * 576 is patch (24, 0), the last token is patch (47, 47)
    full = np.arange(48 * 48)
    t = oracle.anyres_tokens(full, -np.arange(576) - 1)
    assert t[0] == -1 and t[575] == -576
    assert (t[576], t[576 + 24], t[2 * 576], t[3 * 576], t[-1]) == (0, 48, 24, 24 * 48, 48 * 48 - 1)
    assert sorted(t[576:].tolist()) == list(range(48 * 48))


def test_row_offsets_are_the_exclusive_scan_of_the_tier_counts():
    rng = np.random.default_rng(4)
    counts = rng.integers(0, 50, (9, 5)).astype(np.int32)
    fill0 = np.array([7, 0, 123456789012], np.int64)
    off, fill = oracle.row_offsets(counts, fill0)
    for k, code in enumerate((FP16, INT8, INT4)):
        acc = int(fill0[k])
        for t in range(9):                      # brute force: every frame starts where the earlier ones end
            assert off[t, k] == acc
            acc += int(counts[t, code])
        assert fill[k] == acc
    # stored with these offsets, the frames' rows tile the pool without gap or overlap
    L, n_tok, HD, G = 1, 24, 256, 128
    frames = [_frame_case(L, n_tok, HD, G, seed=s) for s in (1, 2, 3)]
    cs = np.stack([f[4] for f in frames])
    off, fill = oracle.row_offsets(cs)
    pools = oracle.Pools(L, HD, G, *[int(x) for x in fill])
    pools.int8_scale[:] = 0xFFFF
    pools.int4_sz[:] = 0xFFFF
    for (K, V, dec, idx, counts), o in zip(frames, off):
        assert oracle.pack_frame(K, V, idx, counts, o, pools) == 0
    assert not (pools.int8_scale == 0xFFFF).any() and not (pools.int4_sz == 0xFFFF).any()      # every row written
    K2 = frames[2][0]
    assert np.array_equal(pools.fp16_pool[0, 0, off[2, 0]], K2[0, frames[2][3][0, 0]])


def test_pack_without_ring_reports_overflow_and_drops_the_rows():
    L, n_tok, HD, G = 1, 24, 256, 128
    K, V, dec, idx, counts = _frame_case(L, n_tok, HD, G)
    pools = oracle.Pools(L, HD, G, int(counts[FP16]) - 1, int(counts[INT8]), int(counts[INT4]), ring=0)
    assert oracle.pack_frame(K, V, idx, counts, np.zeros(3, np.int64), pools) == -1


# ----------------------------------------------------------------------------- accounting
def test_accounting_closed_form_and_the_paper_tier_mix():
    L, HD, G, n_tok = 32, 4096, 128, 576
    counts = np.array([[100, 50, 200, 26, 200]])
    ng = HD // G
    payload = L * 2 * (200 * 8192 + 26 * (4096 + 2 * ng) + 200 * (2048 + 4 * ng))
    assert oracle.stored_bytes(counts, L, HD, G, n_tok) - payload == n_tok + 52 + 4 * 426
    assert oracle.raw_bytes(1, L, HD, n_tok) == 301_989_888
    # Fig. 3 proportions (26.7 / 13.1 / 21.4 / 7.1 / 31.7 %) over 100 frames -> about 2.44x with G = 128
    tot = 100 * n_tok
    mix = np.array([[round(tot * f) for f in (0.267, 0.131, 0.214, 0.071, 0.317)]])
    ratio = oracle.raw_bytes(100, L, HD, n_tok) / oracle.stored_bytes(mix, L, HD, G, n_tok)
    assert ratio == pytest.approx(1 / (0.317 + 0.071 * (0.5 + 1 / 128) + 0.214 * (0.25 + 1 / 64)), rel=2e-4)
    assert 2.40 < ratio < 2.48


def test_source_frames_resolve_reuse_chains():
    """Alg. 1 line 7: a chain of reused entries ends at the last frame that stored (or pruned) the token."""
    dec = np.array([[4, 1, 2, 3],      # frame 0: nothing can be reused
                    [0, 0, 4, 0],
                    [0, 2, 0, 0],
                    [4, 0, 0, 0]], np.uint8)
    src = oracle.source_frames(dec)
    assert src.tolist() == [[0, 0, 0, 0], [0, 0, 1, 0], [0, 2, 1, 0], [3, 2, 1, 0]]
    # brute force on random decisions: walk back until a non-reuse entry
    rng = np.random.default_rng(5)
    dec = rng.integers(0, 5, (40, 64)).astype(np.uint8)
    dec[0][dec[0] == 0] = 1
    src = oracle.source_frames(dec)
    for t in range(40):
        for i in range(64):
            k = t
            while dec[k, i] == 0:
                k -= 1
            assert src[t, i] == k
    # a stream cut in two continues through the carried row
    a = oracle.source_frames(dec[:17])
    b = oracle.source_frames(dec[17:], first=17, prev=a[-1])
    assert np.array_equal(np.concatenate([a, b]), src)

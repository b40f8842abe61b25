"""CPU oracle of the Sali-Cache pre-attention filter and K/V store (test infrastructure).

Thin ctypes binding over ``salicache_oracle.c``: argument marshalling only, all of
the arithmetic (the accounting of Eq. 3 included) is in the C file.  Only tests, the smoke check and the benchmark's
CPU-baseline leg may import this package; the CUDA library never does.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from dataclasses import dataclass

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "salicache_oracle.c")
_LIB = os.path.join(_HERE, "liboracle.so")

REUSE, PRUNE, INT4, INT8, FP16 = 0, 1, 2, 3, 4


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (strict IEEE: no contraction, no fast-math)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".tmp{os.getpid()}"
        subprocess.check_call(
            ["gcc", "-O2", "-std=gnu11", "-ffp-contract=off", "-fno-fast-math", "-fopenmp", "-fPIC", "-shared",
             "-fvisibility=hidden", "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


_lib = None


def lib():
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
        _lib.oracle_half_to_float.restype = C.c_float
        _lib.oracle_half_to_float.argtypes = [C.c_uint16]
        _lib.oracle_float_to_half.restype = C.c_uint16
        _lib.oracle_float_to_half.argtypes = [C.c_float]
        _lib.oracle_num_threads.restype = C.c_int
    return _lib


def _p(a, t=None):
    return a.ctypes.data_as(C.c_void_p)


def _c(a, dtype):
    a = np.ascontiguousarray(a, dtype=dtype)
    return a


@dataclass
class Params:
    """Parameters of the path; defaults are the readings stated in the oracle source."""
    patch: int = 14
    pyr_levels: int = 3
    poly_n: int = 5
    poly_sigma: float = 1.2
    win: int = 15
    iters: int = 3
    eps_det: float = 1e-3
    canny_lo: int = 50
    canny_hi: int = 150
    var_radius: int = 3
    sigma_ref: float = 16.0
    w_edge: float = 0.5
    w_color: float = 0.5
    tau_t: float = 0.5
    theta_R: float = 0.90
    tau_high: float = 0.40
    tau_med: float = 0.36
    tau_low: float = 0.25
    patch_reuse: int = 1
    color_norm: int = 0          # 0: fixed sigma_ref; 1: frame-adaptive (kappa x the frame's RMS local contrast)
    color_kappa: float = 1.0
    color_sigma_min: float = 0.5


def num_threads() -> int:
    return int(lib().oracle_num_threads())


def gray(rgb: np.ndarray) -> np.ndarray:
    rgb = _c(rgb, np.uint8)
    h, w, _ = rgb.shape
    g = np.empty((h, w), np.uint8)
    lib().oracle_gray(_p(rgb), C.c_int(h), C.c_int(w), _p(g))
    return g


def box_down2(rgb: np.ndarray) -> np.ndarray:
    rgb = _c(rgb, np.uint8)
    h, w, _ = rgb.shape
    out = np.empty((h // 2, w // 2, 3), np.uint8)
    lib().oracle_box_down2(_p(rgb), C.c_int(h), C.c_int(w), _p(out))
    return out


def pyr_down(img: np.ndarray) -> np.ndarray:
    img = _c(img, np.float64)
    h, w = img.shape
    out = np.empty((h // 2, w // 2), np.float64)
    lib().oracle_pyr_down(_p(img), C.c_int(h), C.c_int(w), _p(out))
    return out


def poly_exp(img: np.ndarray, n: int = 2, sigma: float = 1.2) -> np.ndarray:
    """Returns planes [5][h][w]: r2 (b_x), r3 (b_y), r4 (A_xx), r5 (A_yy), r6 (2 A_xy)."""
    img = _c(img, np.float64)
    h, w = img.shape
    r = np.empty((5, h, w), np.float64)
    lib().oracle_poly_exp(_p(img), C.c_int(h), C.c_int(w), C.c_int(n), C.c_double(sigma), _p(r))
    return r


def flow_iter(c1: np.ndarray, c2: np.ndarray, d_in: np.ndarray, win: int = 15, eps: float = 1e-3) -> np.ndarray:
    c1, c2, d_in = _c(c1, np.float64), _c(c2, np.float64), _c(d_in, np.float64)
    _, h, w = c1.shape
    out = np.empty((2, h, w), np.float64)
    lib().oracle_flow_iter(_p(c1), _p(c2), C.c_int(h), C.c_int(w), _p(d_in), C.c_int(win), C.c_double(eps), _p(out))
    return out


def flow_upsample(dc: np.ndarray, hf: int, wf: int) -> np.ndarray:
    dc = _c(dc, np.float64)
    _, hc, wc = dc.shape
    out = np.empty((2, hf, wf), np.float64)
    lib().oracle_flow_upsample(_p(dc), C.c_int(hc), C.c_int(wc), _p(out), C.c_int(hf), C.c_int(wf))
    return out


def flow(prev: np.ndarray, cur: np.ndarray, p: Params = Params()) -> np.ndarray:
    prev, cur = _c(prev, np.uint8), _c(cur, np.uint8)
    h, w, _ = prev.shape
    out = np.empty((2, h, w), np.float64)
    lib().oracle_flow(_p(prev), _p(cur), C.c_int(h), C.c_int(w), C.c_int(p.pyr_levels), C.c_int(p.poly_n),
                      C.c_double(p.poly_sigma), C.c_int(p.win), C.c_int(p.iters), C.c_double(p.eps_det), _p(out))
    return out


def delta_p(flw: np.ndarray, patch: int = 14) -> np.ndarray:
    flw = _c(flw, np.float64)
    _, h, w = flw.shape
    out = np.empty(((h // patch) * (w // patch),), np.float64)
    lib().oracle_delta_p(_p(flw), C.c_int(h), C.c_int(w), C.c_int(patch), _p(out))
    return out


def flow_score(prev: np.ndarray, cur: np.ndarray, p: Params = Params(), want_flow: bool = False):
    """prev, cur: [B][h][w][3] uint8.  Returns dP [B][n_patches] float64 (and the flow fields)."""
    prev, cur = _c(prev, np.uint8), _c(cur, np.uint8)
    B, h, w, _ = prev.shape
    np_ = (h // p.patch) * (w // p.patch)
    dP = np.empty((B, np_), np.float64)
    fl = np.empty((B, 2, h, w), np.float64) if want_flow else None
    lib().oracle_flow_score_batch(_p(prev), _p(cur), C.c_int(B), C.c_int(h), C.c_int(w), C.c_int(p.patch),
                                  C.c_int(p.pyr_levels), C.c_int(p.poly_n), C.c_double(p.poly_sigma), C.c_int(p.win),
                                  C.c_int(p.iters), C.c_double(p.eps_det), _p(dP),
                                  _p(fl) if want_flow else C.c_void_p(None))
    return (dP, fl) if want_flow else dP


def diff_score(prev: np.ndarray, cur: np.ndarray, patch: int = 14) -> np.ndarray:
    """Eq. 5 read literally.  prev, cur: [B][h][w][3] uint8 -> dP [B][n_patches] float64 (RMS grey-level difference)."""
    prev, cur = _c(prev, np.uint8), _c(cur, np.uint8)
    B, h, w, _ = prev.shape
    out = np.empty((B, (h // patch) * (w // patch)), np.float64)
    for b in range(B):
        lib().oracle_diff_score(_p(prev[b]), _p(cur[b]), C.c_int(h), C.c_int(w), C.c_int(patch), _p(out[b]))
    return out


def canny(g: np.ndarray, lo: int = 50, hi: int = 150, want_cls: bool = False):
    g = _c(g, np.uint8)
    h, w = g.shape
    E = np.empty((h, w), np.uint8)
    cls = np.empty((h, w), np.uint8) if want_cls else None
    lib().oracle_canny(_p(g), C.c_int(h), C.c_int(w), C.c_int(lo), C.c_int(hi), _p(E),
                       _p(cls) if want_cls else C.c_void_p(None))
    return (E, cls) if want_cls else E


def rgb_to_lab(rgb: np.ndarray) -> np.ndarray:
    rgb = _c(rgb, np.uint8).reshape(-1, 3)
    out = np.empty((rgb.shape[0], 3), np.float64)
    lib().oracle_rgb_to_lab(_p(rgb), C.c_int(rgb.shape[0]), _p(out))
    return out


def color_contrast(rgb: np.ndarray, radius: int = 3, sigma_ref: float = 16.0) -> np.ndarray:
    rgb = _c(rgb, np.uint8)
    h, w, _ = rgb.shape
    out = np.empty((h, w), np.float64)
    lib().oracle_color_contrast(_p(rgb), C.c_int(h), C.c_int(w), C.c_int(radius), C.c_double(sigma_ref), _p(out))
    return out


def color_variance(rgb: np.ndarray, radius: int = 3) -> np.ndarray:
    """V [h][w]: summed population variance of L, a, b in the (2 radius + 1)^2 window."""
    rgb = _c(rgb, np.uint8)
    h, w, _ = rgb.shape
    out = np.empty((h, w), np.float64)
    lib().oracle_color_variance(_p(rgb), C.c_int(h), C.c_int(w), C.c_int(radius), _p(out))
    return out


def color_normalise_global(V: np.ndarray, kappa: float = 1.0, sigma_min: float = 0.5) -> np.ndarray:
    """Frame-adaptive colour term from a V map: min(1, sqrt(V) / (kappa max(sqrt(mean V), sigma_min)))."""
    V = _c(V, np.float64)
    out = np.empty(V.shape, np.float64)
    lib().oracle_color_normalise_global(_p(V), C.c_size_t(V.size), C.c_double(kappa), C.c_double(sigma_min), _p(out))
    return out


def color_contrast_global(rgb: np.ndarray, radius: int = 3, kappa: float = 1.0, sigma_min: float = 0.5) -> np.ndarray:
    rgb = _c(rgb, np.uint8)
    h, w, _ = rgb.shape
    out = np.empty((h, w), np.float64)
    lib().oracle_color_contrast_global(_p(rgb), C.c_int(h), C.c_int(w), C.c_int(radius), C.c_double(kappa),
                                       C.c_double(sigma_min), _p(out))
    return out


def saliency(frames: np.ndarray, p: Params = Params(), want_map: bool = False):
    """frames: [B][h][w][3] uint8 (or one frame).  Returns s [B][n_patches] float64.
    p.color_norm = 1 selects the frame-adaptive colour term (p.color_kappa in place of p.sigma_ref)."""
    frames = _c(frames, np.uint8)
    one = frames.ndim == 3
    if one:
        frames = frames[None]
    B, h, w, _ = frames.shape
    def one_frame(b, s_b, S_b):
        head = (_p(frames[b]), C.c_int(h), C.c_int(w), C.c_int(p.patch), C.c_int(p.canny_lo), C.c_int(p.canny_hi),
                C.c_int(p.var_radius))
        tail = (C.c_double(p.w_edge), C.c_double(p.w_color), _p(s_b), _p(S_b) if S_b is not None else C.c_void_p(None))
        if p.color_norm:
            lib().oracle_saliency_global(*head, C.c_double(p.color_kappa), C.c_double(p.color_sigma_min), *tail)
        else:
            lib().oracle_saliency(*head, C.c_double(p.sigma_ref), *tail)

    s = np.empty((B, (h // p.patch) * (w // p.patch)), np.float64)
    if one or want_map or p.color_norm:
        S = np.empty((B, h, w), np.float64) if want_map else None
        for b in range(B):
            one_frame(b, s[b], S[b] if want_map else None)
        if one:
            return (s[0], S[0]) if want_map else s[0]
        return (s, S) if want_map else s
    lib().oracle_saliency_batch(_p(frames), C.c_int(B), C.c_int(h), C.c_int(w), C.c_int(p.patch),
                                C.c_int(p.canny_lo), C.c_int(p.canny_hi), C.c_int(p.var_radius),
                                C.c_double(p.sigma_ref), C.c_double(p.w_edge), C.c_double(p.w_color), _p(s))
    return s


def select(dP, s, has_prev: bool, p: Params = Params()):
    """One frame.  dP, s: float32 [n_tok].  Returns decision u8, idx i32 [3][n_tok], counts i32 [5], redundant, R."""
    s = _c(s, np.float32)
    n = s.shape[0]
    dP = _c(dP if dP is not None else np.zeros(n, np.float32), np.float32)
    dec = np.empty(n, np.uint8)
    idx = np.empty((3, n), np.int32)
    counts = np.empty(5, np.int32)
    red = np.zeros(1, np.uint8)
    R = np.zeros(1, np.float32)
    lib().oracle_select(_p(dP), _p(s), C.c_int(n), C.c_int(int(has_prev)), C.c_int(p.patch_reuse),
                        C.c_float(p.tau_t), C.c_float(p.theta_R), C.c_float(p.tau_high), C.c_float(p.tau_med),
                        C.c_float(p.tau_low), _p(dec), _p(idx), _p(counts), _p(red), _p(R))
    return dec, idx, counts, int(red[0]), float(R[0])


def select_ranked(dP, s, has_prev: bool, shares_permille, p: Params = Params()):
    """One frame, tiers by rank of s among the tokens that are not reused.  shares_permille = (FP16, INT8, INT4) shares
    of those tokens in thousandths.  Returns decision u8, idx i32 [3][n_tok], counts i32 [5], redundant."""
    s = _c(s, np.float32)
    n = s.shape[0]
    dP = _c(dP if dP is not None else np.zeros(n, np.float32), np.float32)
    dec = np.empty(n, np.uint8)
    idx = np.empty((3, n), np.int32)
    counts = np.empty(5, np.int32)
    red = np.zeros(1, np.uint8)
    pm16, pm8, pm4 = (int(x) for x in shares_permille)
    lib().oracle_select_ranked(_p(dP), _p(s), C.c_int(n), C.c_int(int(has_prev)), C.c_int(p.patch_reuse), C.c_float(p.tau_t),
                               C.c_float(p.theta_R), C.c_int(pm16), C.c_int(pm8), C.c_int(pm4), _p(dec), _p(idx), _p(counts),
                               _p(red))
    return dec, idx, counts, int(red[0])


def select_anchored(frames: np.ndarray, s: np.ndarray, first_has_no_prev: bool, anchor: np.ndarray, p: Params = Params()):
    """Anchor-frame mode: every token is compared (Eq. 5 read literally) with the patch its cache entry came from.
    frames u8 [T][h][w][3], s f32 [T][n_tok], anchor u8 [h][w][3] (updated in place).
    Returns dP f32 [T][n_tok], decision u8 [T][n_tok], idx i32 [T][3][n_tok], counts i32 [T][5], redundant u8 [T]."""
    frames, s = _c(frames, np.uint8), _c(s, np.float32)
    assert anchor.dtype == np.uint8 and anchor.flags["C_CONTIGUOUS"]
    T, h, w, _ = frames.shape
    n = (h // p.patch) * (w // p.patch)
    assert s.shape == (T, n) and anchor.shape == (h, w, 3)
    dP = np.empty((T, n), np.float32)
    dec = np.empty((T, n), np.uint8)
    idx = np.empty((T, 3, n), np.int32)
    counts = np.empty((T, 5), np.int32)
    red = np.zeros(T, np.uint8)
    lib().oracle_select_anchored(_p(frames), _p(s), C.c_int(T), C.c_int(h), C.c_int(w), C.c_int(p.patch),
                                 C.c_int(int(first_has_no_prev)), C.c_int(p.patch_reuse), C.c_float(p.tau_t),
                                 C.c_float(p.theta_R), C.c_float(p.tau_high), C.c_float(p.tau_med), C.c_float(p.tau_low),
                                 _p(anchor), _p(dP), _p(dec), _p(idx), _p(counts), _p(red))
    return dP, dec, idx, counts, red


def source_frames(decision: np.ndarray, first: int = 0, prev=None) -> np.ndarray:
    """decision u8 [T][n_tok] -> int32 [T][n_tok]: the frame whose entry each token uses (reuse chains resolved)."""
    decision = _c(decision, np.uint8)
    T, n = decision.shape
    prev = _c(prev if prev is not None else np.full(n, -1, np.int32), np.int32)
    src = np.empty((T, n), np.int32)
    lib().oracle_source_frames(_p(decision), C.c_int(T), C.c_int(n), C.c_int(first), _p(prev), _p(src))
    return src


def half_to_float(bits: np.ndarray) -> np.ndarray:
    bits = _c(bits, np.uint16).ravel()
    f = lib().oracle_half_to_float
    return np.array([f(int(b)) for b in bits], np.float32)


def float_to_half(x: np.ndarray) -> np.ndarray:
    x = _c(x, np.float32).ravel()
    f = lib().oracle_float_to_half
    return np.array([f(float(v)) for v in x], np.uint16)


def quant_int8_group(x16: np.ndarray):
    x16 = _c(x16, np.uint16)
    G = x16.shape[0]
    q = np.empty(G, np.int8)
    s = np.zeros(1, np.uint16)
    lib().oracle_quant_int8_group(_p(x16), C.c_int(G), _p(q), _p(s))
    return q, int(s[0])


def dequant_int8_group(q: np.ndarray, s16: int) -> np.ndarray:
    q = _c(q, np.int8)
    out = np.empty(q.shape[0], np.uint16)
    lib().oracle_dequant_int8_group(_p(q), C.c_int(q.shape[0]), C.c_uint16(s16), _p(out))
    return out


def quant_int4_group(x16: np.ndarray):
    x16 = _c(x16, np.uint16)
    G = x16.shape[0]
    packed = np.empty(G // 2, np.uint8)
    s = np.zeros(1, np.uint16)
    z = np.zeros(1, np.uint16)
    lib().oracle_quant_int4_group(_p(x16), C.c_int(G), _p(packed), _p(s), _p(z))
    return packed, int(s[0]), int(z[0])


def dequant_int4_group(packed: np.ndarray, s16: int, z16: int) -> np.ndarray:
    packed = _c(packed, np.uint8)
    G = packed.shape[0] * 2
    out = np.empty(G, np.uint16)
    lib().oracle_dequant_int4_group(_p(packed), C.c_int(G), C.c_uint16(s16), C.c_uint16(z16), _p(out))
    return out


@dataclass
class Pools:
    """Host-side per-tier pools with the same layout as the device pools."""
    L: int
    HD: int
    G: int
    cap16: int
    cap8: int
    cap4: int
    ring: int = 0

    def __post_init__(self):
        ng = self.HD // self.G
        self.fp16_pool = np.zeros((self.L, 2, self.cap16, self.HD), np.uint16)
        self.int8_codes = np.zeros((self.L, 2, self.cap8, self.HD), np.int8)
        self.int8_scale = np.zeros((self.L, 2, self.cap8, ng), np.uint16)
        self.int4_codes = np.zeros((self.L, 2, self.cap4, self.HD // 2), np.uint8)
        self.int4_sz = np.zeros((self.L, 2, self.cap4, ng, 2), np.uint16)


def pack_frame(K16: np.ndarray, V16: np.ndarray, idx, counts, off, pools: Pools) -> int:
    """K16, V16: uint16 (fp16 bits) [L][n_tok][HD]; off: int64 [3] (FP16, INT8, INT4 row offsets)."""
    K16, V16 = _c(K16, np.uint16), _c(V16, np.uint16)
    L, n_tok, HD = K16.shape
    idx, counts, off = _c(idx, np.int32), _c(counts, np.int32), _c(off, np.int64)
    return int(lib().oracle_pack_frame(
        _p(K16), _p(V16), C.c_int(L), C.c_int(n_tok), C.c_int(HD), C.c_int(pools.G), _p(idx), _p(counts), _p(off),
        C.c_int(pools.ring), _p(pools.fp16_pool), C.c_int64(pools.cap16), _p(pools.int8_codes), _p(pools.int8_scale),
        C.c_int64(pools.cap8), _p(pools.int4_codes), _p(pools.int4_sz), C.c_int64(pools.cap4)))


def unpack_frame(n_tok: int, idx, counts, decision, off, pools: Pools, zero_fill_pruned: bool, K_out, V_out, fill=None) -> int:
    """`fill` (running fill per tier, int64 [3]): with ring pools, rows overwritten since are zeroed and -9 returned."""
    idx, counts, off = _c(idx, np.int32), _c(counts, np.int32), _c(off, np.int64)
    decision = _c(decision, np.uint8)
    assert K_out.dtype == np.uint16 and K_out.flags.c_contiguous and V_out.flags.c_contiguous
    fill = None if fill is None else _c(fill, np.int64)
    return int(lib().oracle_unpack_frame(
        C.c_int(pools.L), C.c_int(n_tok), C.c_int(pools.HD), C.c_int(pools.G), _p(idx), _p(counts), _p(decision),
        _p(off), C.c_int(pools.ring), _p(pools.fp16_pool), C.c_int64(pools.cap16), _p(pools.int8_codes),
        _p(pools.int8_scale), C.c_int64(pools.cap8), _p(pools.int4_codes), _p(pools.int4_sz), C.c_int64(pools.cap4),
        C.c_int(int(zero_fill_pruned)), _p(fill) if fill is not None else C.c_void_p(None), _p(K_out), _p(V_out)))


def frames_resident(counts_all, off_all, caps, ring: bool, fill) -> np.ndarray:
    """resident u8 [T]: 1 when every row frame t stored is still in the (ring) pools at running fill `fill`."""
    c = _c(np.asarray(counts_all).reshape(-1, 5), np.int32)
    o = _c(np.asarray(off_all).reshape(-1, 3), np.int64)
    caps, fill = _c(caps, np.int64), _c(fill, np.int64)
    out = np.empty(c.shape[0], np.uint8)
    lib().oracle_frames_resident(_p(c), _p(o), C.c_int(c.shape[0]), _p(caps), C.c_int(int(ring)), _p(fill), _p(out))
    return out


def tokens_live(src: np.ndarray, first: int, resident: np.ndarray) -> np.ndarray:
    """live u8 [T][n_tok]: 1 when the frame that holds the token's entry (src, reuse chains resolved) is resident;
    resident[k] describes frame first + k."""
    src, resident = _c(src, np.int32), _c(resident, np.uint8)
    T, n = src.shape
    out = np.empty((T, n), np.uint8)
    lib().oracle_tokens_live(_p(src), C.c_int(T), C.c_int(n), C.c_int(first), _p(resident), C.c_int(resident.shape[0]), _p(out))
    return out


def attend(q16: np.ndarray, pools: "Pools", n_rows) -> np.ndarray:
    """Decode attention over the rows the pools hold (n_rows = rows used in the FP16, INT8, INT4 pool).
    q16: fp16 bits [L][H][D].  Returns float64 [L][H][D]."""
    q16 = _c(q16, np.uint16)
    L, H, D = q16.shape
    out = np.empty((L, H, D), np.float64)
    n16, n8, n4 = (int(x) for x in n_rows)
    lib().oracle_attend(_p(q16), C.c_int(L), C.c_int(H), C.c_int(D), C.c_int(pools.G), _p(pools.fp16_pool),
                        C.c_int64(pools.cap16), C.c_int64(n16), _p(pools.int8_codes), _p(pools.int8_scale),
                        C.c_int64(pools.cap8), C.c_int64(n8), _p(pools.int4_codes), _p(pools.int4_sz),
                        C.c_int64(pools.cap4), C.c_int64(n4), _p(out))
    return out


def attend_gqa(q16: np.ndarray, pools: "Pools", n_rows, q_per_kv: int) -> np.ndarray:
    """Grouped-query decode attention: query head hq uses the rows of key/value head hq // q_per_kv.
    q16: fp16 bits [L][H * q_per_kv][D], H the pools' heads.  Returns float64 of the same shape."""
    q16 = _c(q16, np.uint16)
    L, HQ, D = q16.shape
    assert HQ % q_per_kv == 0 and (HQ // q_per_kv) * D == pools.HD
    out = np.empty((L, HQ, D), np.float64)
    n16, n8, n4 = (int(x) for x in n_rows)
    lib().oracle_attend_gqa(_p(q16), C.c_int(L), C.c_int(HQ // q_per_kv), C.c_int(q_per_kv), C.c_int(D), C.c_int(pools.G),
                            _p(pools.fp16_pool), C.c_int64(pools.cap16), C.c_int64(n16), _p(pools.int8_codes),
                            _p(pools.int8_scale), C.c_int64(pools.cap8), C.c_int64(n8), _p(pools.int4_codes),
                            _p(pools.int4_sz), C.c_int64(pools.cap4), C.c_int64(n4), _p(out))
    return out


def stored_bytes(counts_all: np.ndarray, L: int, HD: int, G: int, n_tok: int) -> int:
    """Bytes the mixed-precision store holds for frames with the given per-code counts [T][5]
    (Eq. 3 applied per tier, plus all metadata: scales/zeros, index lists, decision bytes,
    an 8-byte pointer-table entry and three 8-byte row offsets per frame)."""
    c = _c(np.asarray(counts_all).reshape(-1, 5), np.int64)
    f = lib().oracle_stored_bytes
    f.restype = C.c_int64
    return int(f(_p(c), C.c_int64(c.shape[0]), C.c_int(L), C.c_int(HD), C.c_int(G), C.c_int(n_tok)))


def raw_bytes(T: int, L: int, HD: int, n_tok: int) -> int:
    """Eq. 3 for T frames of n_tok tokens, fp16, K and V."""
    f = lib().oracle_raw_bytes
    f.restype = C.c_int64
    return int(f(C.c_int64(T), C.c_int(L), C.c_int(HD), C.c_int(n_tok)))


def anyres_tokens(full: np.ndarray, base: np.ndarray, tg: int = 24) -> np.ndarray:
    """Per-patch values of the whole frame ((2 tg)^2, row-major) and of the base image (tg^2) in token order:
    base, tile (0,0), (0,1), (1,0), (1,1), each row-major."""
    full, base = _c(full, np.float64).ravel(), _c(base, np.float64).ravel()
    assert full.size == 4 * tg * tg and base.size == tg * tg
    out = np.empty(5 * tg * tg, np.float64)
    lib().oracle_anyres_tokens(_p(full), _p(base), C.c_int(tg), _p(out))
    return out


def row_offsets(counts_all: np.ndarray, fill=None):
    """First pool row of every frame per tier (FP16, INT8, INT4) for per-code counts [T][5], continuing from
    the running fill [3].  Returns (off int64 [T][3], fill after the last frame int64 [3])."""
    c = _c(np.asarray(counts_all).reshape(-1, 5), np.int32)
    fill = np.zeros(3, np.int64) if fill is None else _c(fill, np.int64).copy()
    off = np.empty((c.shape[0], 3), np.int64)
    lib().oracle_row_offsets(_p(c), C.c_int(c.shape[0]), _p(fill), _p(off))
    return off, fill

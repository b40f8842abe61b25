"""ctypes binding over libsalicache.so: argument marshalling only.

Every function below has the name of the C entry point it calls and passes device pointers of
torch tensors plus the current CUDA stream.  Nothing is computed in Python and there is no CPU
fallback: a missing or unloadable library raises at import of this module's `lib()`.
"""
from __future__ import annotations

import ctypes as C
import os

from . import build as _build

REUSE, PRUNE, INT4, INT8, FP16 = 0, 1, 2, 3, 4

E_NULL, E_SHAPE, E_ALIGN, E_PARAM, E_CUDA, E_CAPACITY, E_NOCONVERGE, E_NOMEM, E_EVICTED = -1, -2, -3, -4, -5, -6, -7, -8, -9


class SalicacheError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {lib().salicache_strerror(status).decode()} ({status})")


class Params(C.Structure):
    _fields_ = [
        ("H", C.c_int32), ("W", C.c_int32), ("patch", C.c_int32), ("n_images", C.c_int32),
        ("max_batch", C.c_int32), ("chunk_frames", C.c_int32),
        ("pyr_levels", C.c_int32), ("poly_n", C.c_int32), ("poly_sigma", C.c_double),
        ("win", C.c_int32), ("iters", C.c_int32), ("eps_det", C.c_double),
        ("canny_lo", C.c_int32), ("canny_hi", C.c_int32), ("var_radius", C.c_int32),
        ("sigma_ref", C.c_double), ("w_edge", C.c_double), ("w_color", C.c_double),
        ("hyst_max_iters", C.c_int32),
        ("tau_t", C.c_float), ("theta_R", C.c_float), ("tau_high", C.c_float), ("tau_med", C.c_float),
        ("tau_low", C.c_float), ("patch_reuse", C.c_int32),
        ("L", C.c_int32), ("heads", C.c_int32), ("head_dim", C.c_int32), ("group", C.c_int32),
        ("color_norm", C.c_int32), ("color_kappa", C.c_double), ("color_sigma_min", C.c_double),
    ]


class Pools(C.Structure):
    _fields_ = [
        ("fp16_pool", C.c_void_p), ("int8_codes", C.c_void_p), ("int8_scale", C.c_void_p),
        ("int4_codes", C.c_void_p), ("int4_sz", C.c_void_p),
        ("cap_fp16", C.c_int64), ("cap_int8", C.c_int64), ("cap_int4", C.c_int64), ("ring", C.c_int32),
        ("d_fill", C.c_void_p),
    ]


EXPORTS = [
    "salicache_default_params", "salicache_create", "salicache_destroy", "salicache_strerror",
    "salicache_tokens_per_frame", "salicache_launch_count", "salicache_flow_score", "salicache_saliency", "salicache_select",
    "salicache_pack_kv", "salicache_unpack_kv", "salicache_poll_status", "salicache_saliency_noalloc",
    "salicache_frame_redundancy", "salicache_source_frames", "salicache_diff_score", "salicache_attend",
    "salicache_select_anchored", "salicache_select_ranked", "salicache_attend_gqa", "salicache_select_anchored_batch",
    "salicache_frames_resident", "salicache_tokens_live",
]

_lib = None


def lib():
    """Loads (building first if the sources are newer) the CUDA library.  Fails loudly if it cannot."""
    global _lib
    if _lib is None:
        path = _build.LIB
        if os.path.exists(os.path.join(_build.CSRC, "api.cu")) and _build.nvcc_path() is not None:
            path = _build.build()
        if not os.path.exists(path):
            raise ImportError(f"{path} is missing: build it with `python -m paper_2602_14236_b200.build`; "
                              "there is no CPU fallback")
        _lib = C.CDLL(path)
        _lib.salicache_strerror.restype = C.c_char_p
        _lib.salicache_strerror.argtypes = [C.c_int]
        _lib.salicache_create.argtypes = [C.POINTER(C.c_void_p), C.POINTER(Params)]
        _lib.salicache_destroy.argtypes = [C.c_void_p]
        _lib.salicache_tokens_per_frame.argtypes = [C.c_void_p]
        _lib.salicache_default_params.argtypes = [C.POINTER(Params)]
        _lib.salicache_launch_count.argtypes = [C.c_void_p]
        _lib.salicache_launch_count.restype = C.c_int64
        vp, i32, i64 = C.c_void_p, C.c_int, C.c_int64
        _lib.salicache_flow_score.argtypes = [vp, vp, vp, i32, vp, vp, vp]
        _lib.salicache_saliency.argtypes = [vp, vp, i32, vp, vp, vp]
        _lib.salicache_diff_score.argtypes = [vp, vp, vp, i32, vp, vp]
        _lib.salicache_frame_redundancy.argtypes = [vp, vp, i32, i32, vp, vp]
        _lib.salicache_source_frames.argtypes = [vp, vp, i32, i32, vp, vp, vp]
        _lib.salicache_select.argtypes = [vp, vp, vp, i32, i32, vp, vp, vp, vp, vp, vp, vp]
        _lib.salicache_select_ranked.argtypes = [vp, vp, vp, i32, i32, i32, i32, i32, vp, vp, vp, vp, vp, vp, vp]
        _lib.salicache_select_anchored_batch.argtypes = [vp, vp, vp, i32, i32, i32, vp, vp, vp, vp, vp, vp, vp, vp, vp]
        _lib.salicache_select_anchored.argtypes = [vp, vp, vp, i32, i32, vp, vp, vp, vp, vp, vp, vp, vp, vp]
        _lib.salicache_pack_kv.argtypes = [vp, vp, vp, i64, vp, vp, vp, i32, C.POINTER(Pools), vp]
        _lib.salicache_unpack_kv.argtypes = [vp, C.POINTER(Pools), vp, vp, vp, vp, i32, i32, vp, vp, i64, vp]
        _lib.salicache_poll_status.argtypes = [vp, vp]
        _lib.salicache_attend.argtypes = [vp, vp, C.POINTER(Pools), vp, vp, vp]
        _lib.salicache_attend_gqa.argtypes = [vp, vp, i32, C.POINTER(Pools), vp, vp, vp]
        _lib.salicache_saliency_noalloc.argtypes = [C.POINTER(Params), vp, i32, vp, vp, vp]
        _lib.salicache_frames_resident.argtypes = [vp, vp, vp, i32, C.POINTER(Pools), vp, vp]
        _lib.salicache_tokens_live.argtypes = [vp, vp, i32, i32, vp, i32, vp, vp]
    return _lib


def _ptr(t):
    return None if t is None else C.c_void_p(t.data_ptr())


def _stream(stream=None):
    import torch
    s = torch.cuda.current_stream() if stream is None else stream
    return C.c_void_p(s.cuda_stream)


def _check(status: int, where: str):
    if status != 0:
        raise SalicacheError(status, where)


def salicache_default_params(**overrides) -> Params:
    p = Params()
    _check(lib().salicache_default_params(C.byref(p)), "salicache_default_params")
    for k, v in overrides.items():
        if not hasattr(p, k):
            raise AttributeError(k)
        setattr(p, k, v)
    return p


class Context:
    """Owns a salicache_ctx (scratch only).  Create it with the wanted device current."""

    def __init__(self, params: Params):
        self.params = params
        self._h = C.c_void_p()
        _check(lib().salicache_create(C.byref(self._h), C.byref(params)), "salicache_create")
        self.n_tok = int(lib().salicache_tokens_per_frame(self._h))
        self.HD = params.heads * params.head_dim

    def close(self):
        if self._h:
            lib().salicache_destroy(self._h)
            self._h = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def launch_count(self) -> int:
        return int(lib().salicache_launch_count(self._h))

    @property
    def handle(self):
        return self._h


def salicache_flow_score(ctx: Context, d_prev, d_cur, B: int, d_deltaP, d_flow=None, stream=None):
    _check(lib().salicache_flow_score(ctx.handle, _ptr(d_prev), _ptr(d_cur), B, _ptr(d_deltaP), _ptr(d_flow),
                                      _stream(stream)), "salicache_flow_score")


def salicache_diff_score(ctx: Context, d_prev, d_cur, B: int, d_deltaP, stream=None):
    _check(lib().salicache_diff_score(ctx.handle, _ptr(d_prev), _ptr(d_cur), B, _ptr(d_deltaP), _stream(stream)),
           "salicache_diff_score")


def salicache_saliency(ctx: Context, d_frames, B: int, d_s, d_skip=None, stream=None):
    _check(lib().salicache_saliency(ctx.handle, _ptr(d_frames), B, _ptr(d_s), _ptr(d_skip), _stream(stream)),
           "salicache_saliency")


def salicache_frame_redundancy(ctx: Context, d_deltaP, B: int, first_has_no_prev: bool, d_frame_redundant, stream=None):
    _check(lib().salicache_frame_redundancy(ctx.handle, _ptr(d_deltaP), B, int(first_has_no_prev),
                                            _ptr(d_frame_redundant), _stream(stream)), "salicache_frame_redundancy")


def salicache_saliency_noalloc(params: Params, d_frames, B: int, d_s, d_status=None, stream=None):
    """Spatial score for hosts that cannot allocate device memory (no context needed): at most
    NOALLOC_MAX_FRAMES frames of at most NOALLOC_MAX_SIDE pixels a side per call.  Calls on one
    device share a fixed scratch array inside the library, so they must not overlap on the GPU."""
    _check(lib().salicache_saliency_noalloc(C.byref(params), _ptr(d_frames), B, _ptr(d_s), _ptr(d_status),
                                            _stream(stream)), "salicache_saliency_noalloc")


NOALLOC_MAX_FRAMES, NOALLOC_MAX_SIDE = 8, 336


def salicache_source_frames(ctx: Context, d_decision, B: int, first_frame: int, d_carry, d_src, stream=None):
    _check(lib().salicache_source_frames(ctx.handle, _ptr(d_decision), B, first_frame, _ptr(d_carry), _ptr(d_src),
                                         _stream(stream)), "salicache_source_frames")


def salicache_select(ctx: Context, d_deltaP, d_s, B: int, first_has_no_prev: bool, d_decision, d_idx, d_counts,
                     d_frame_redundant, d_row_offset, d_fill, stream=None):
    _check(lib().salicache_select(ctx.handle, _ptr(d_deltaP), _ptr(d_s), B, int(first_has_no_prev), _ptr(d_decision),
                                  _ptr(d_idx), _ptr(d_counts), _ptr(d_frame_redundant), _ptr(d_row_offset),
                                  _ptr(d_fill), _stream(stream)), "salicache_select")


def salicache_select_ranked(ctx: Context, d_deltaP, d_s, B: int, first_has_no_prev: bool, shares_permille, d_decision, d_idx,
                            d_counts, d_frame_redundant, d_row_offset, d_fill, stream=None):
    pm16, pm8, pm4 = (int(x) for x in shares_permille)
    _check(lib().salicache_select_ranked(ctx.handle, _ptr(d_deltaP), _ptr(d_s), B, int(first_has_no_prev), pm16, pm8, pm4,
                                         _ptr(d_decision), _ptr(d_idx), _ptr(d_counts), _ptr(d_frame_redundant),
                                         _ptr(d_row_offset), _ptr(d_fill), _stream(stream)), "salicache_select_ranked")


def salicache_select_anchored(ctx: Context, d_frames, d_s, B: int, first_has_no_prev: bool, d_anchor, d_deltaP, d_decision,
                              d_idx, d_counts, d_frame_redundant, d_row_offset, d_fill, stream=None):
    _check(lib().salicache_select_anchored(ctx.handle, _ptr(d_frames), _ptr(d_s), B, int(first_has_no_prev), _ptr(d_anchor),
                                           _ptr(d_deltaP), _ptr(d_decision), _ptr(d_idx), _ptr(d_counts),
                                           _ptr(d_frame_redundant), _ptr(d_row_offset), _ptr(d_fill), _stream(stream)),
           "salicache_select_anchored")


def salicache_select_anchored_batch(ctx: Context, d_frames, d_s, n_videos: int, B: int, first_has_no_prev: bool, d_anchor, d_deltaP,
                                    d_decision, d_idx, d_counts, d_frame_redundant, d_row_offset, d_fill, stream=None):
    _check(lib().salicache_select_anchored_batch(ctx.handle, _ptr(d_frames), _ptr(d_s), n_videos, B, int(first_has_no_prev),
                                                 _ptr(d_anchor), _ptr(d_deltaP), _ptr(d_decision), _ptr(d_idx), _ptr(d_counts),
                                                 _ptr(d_frame_redundant), _ptr(d_row_offset), _ptr(d_fill), _stream(stream)),
           "salicache_select_anchored_batch")


def salicache_pack_kv(ctx: Context, d_K, d_V, frame_stride: int, d_idx, d_counts, d_row_offset, B: int, pools: Pools,
                      stream=None):
    _check(lib().salicache_pack_kv(ctx.handle, _ptr(d_K), _ptr(d_V), frame_stride, _ptr(d_idx), _ptr(d_counts),
                                   _ptr(d_row_offset), B, C.byref(pools), _stream(stream)), "salicache_pack_kv")


def salicache_unpack_kv(ctx: Context, pools: Pools, d_idx, d_counts, d_decision, d_row_offset, B: int,
                        zero_fill_pruned: bool, d_K_out, d_V_out, frame_stride: int, stream=None):
    _check(lib().salicache_unpack_kv(ctx.handle, C.byref(pools), _ptr(d_idx), _ptr(d_counts), _ptr(d_decision),
                                     _ptr(d_row_offset), B, int(zero_fill_pruned), _ptr(d_K_out), _ptr(d_V_out),
                                     frame_stride, _stream(stream)), "salicache_unpack_kv")


def salicache_attend(ctx: Context, d_q, pools: Pools, d_fill, d_out, stream=None):
    _check(lib().salicache_attend(ctx.handle, _ptr(d_q), C.byref(pools), _ptr(d_fill), _ptr(d_out), _stream(stream)),
           "salicache_attend")


def salicache_attend_gqa(ctx: Context, d_q, q_per_kv: int, pools: Pools, d_fill, d_out, stream=None):
    _check(lib().salicache_attend_gqa(ctx.handle, _ptr(d_q), int(q_per_kv), C.byref(pools), _ptr(d_fill), _ptr(d_out),
                                      _stream(stream)), "salicache_attend_gqa")


def salicache_frames_resident(ctx: Context, d_counts, d_row_offset, B: int, pools: Pools, d_resident, stream=None):
    _check(lib().salicache_frames_resident(ctx.handle, _ptr(d_counts), _ptr(d_row_offset), B, C.byref(pools), _ptr(d_resident),
                                           _stream(stream)), "salicache_frames_resident")


def salicache_tokens_live(ctx: Context, d_src, B: int, first_frame: int, d_resident_table, n_table: int, d_live, stream=None):
    _check(lib().salicache_tokens_live(ctx.handle, _ptr(d_src), B, first_frame, _ptr(d_resident_table), n_table, _ptr(d_live),
                                       _stream(stream)), "salicache_tokens_live")


def salicache_poll_status(ctx: Context, stream=None) -> int:
    return int(lib().salicache_poll_status(ctx.handle, _stream(stream)))


class PoolSet:
    """Device pools as torch tensors (memory only) plus the C struct that points at them."""

    def __init__(self, L: int, HD: int, cap16: int, cap8: int, cap4: int, ring: bool = False, device="cuda", G: int = 128,
                 fill=None):
        import torch
        ng = HD // G
        self.L, self.HD, self.G = L, HD, G
        self.cap = (cap16, cap8, cap4)
        z = lambda shape, dt: torch.zeros(shape, dtype=dt, device=device)
        self.fp16_pool = z((L, 2, max(cap16, 1), HD), torch.float16)
        self.int8_codes = z((L, 2, max(cap8, 1), HD), torch.int8)
        self.int8_scale = z((L, 2, max(cap8, 1), ng), torch.float16)
        self.int4_codes = z((L, 2, max(cap4, 1), HD // 2), torch.uint8)
        self.int4_sz = z((L, 2, max(cap4, 1), ng, 2), torch.float16)
        self.c = Pools(self.fp16_pool.data_ptr(), self.int8_codes.data_ptr(), self.int8_scale.data_ptr(),
                       self.int4_codes.data_ptr(), self.int4_sz.data_ptr(), cap16, cap8, cap4, int(ring),
                       None if fill is None else fill.data_ptr())
        self.fill = fill              # keeps the tensor alive

    def nbytes(self) -> int:
        return sum(t.numel() * t.element_size() for t in
                   (self.fp16_pool, self.int8_codes, self.int8_scale, self.int4_codes, self.int4_sz))

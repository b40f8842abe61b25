"""salicache_saliency_noalloc against salicache_saliency, through the C ABI.

The allocation-free entry point serves hosts that cannot call cudaMalloc while they run (their own
pool owns the GPU, or they sit under an allocator lock), so it keeps its scratch in a fixed array
inside the library that every call on the device shares and that remembers the previous call.  The
test therefore makes two calls in a row on different inputs and checks each against the
context-based entry point and against the CPU oracle: leftovers of the first call must not leak
into the second.  This file
sorts after the other test files on purpose, so a run that stops at the first failure has already
finished them."""
import ctypes

import numpy as np
import pytest

import oracle
from paper_2602_14236_b200 import binding as sc
from paper_2602_14236_b200 import synth

pytestmark = pytest.mark.gpu


def _reference(params, frames):
    import torch
    ctx = sc.Context(params)
    s = torch.zeros((frames.shape[0], ctx.n_tok), dtype=torch.float32, device="cuda")
    sc.salicache_saliency(ctx, frames, frames.shape[0], s)
    torch.cuda.synchronize()
    assert sc.salicache_poll_status(ctx) == 0
    return s.cpu().numpy()


def test_two_calls_in_a_row_match_the_context_entry_point():
    import torch
    params = sc.salicache_default_params(max_batch=8, chunk_frames=8, L=1)
    busy = torch.from_numpy(synth.frames(2, T=sc.NOALLOC_MAX_FRAMES)).cuda()        # sprites: many edges
    calm = torch.from_numpy(synth.frames(3, T=3, t0=200)).cuda()                      # fewer frames, other content
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    side = torch.cuda.Stream()            # not the default stream: the one-time set-up must be visible to any stream
    torch.cuda.synchronize()
    for frames in (busy, calm):
        B = frames.shape[0]
        s = torch.full((B, 576), -1.0, dtype=torch.float32, device="cuda")
        torch.cuda.synchronize()
        with torch.cuda.stream(side):
            sc.salicache_saliency_noalloc(params, frames, B, s, status)
        torch.cuda.synchronize()
        got = s.cpu().numpy()
        ref = _reference(params, frames)
        assert np.all(np.abs(got - ref) <= 1e-6 + 1e-4 * np.abs(ref))      # the tolerance of the score tests
        assert np.array_equal(got, ref)                                     # same kernels: same bits
        want = oracle.saliency(frames.cpu().numpy())                        # and both are the oracle's score
        assert np.all(np.abs(got - want) <= 1e-6 + 1e-4 * np.abs(want))
    assert int(status.item()) == 0


def test_smaller_frames_status_word_and_limits():
    import torch
    small = sc.salicache_default_params(H=112, W=224, max_batch=4, chunk_frames=4, L=1)
    fr = torch.from_numpy(synth.frames(2, T=2)[:, 60:172, 40:264].copy()).cuda()
    s = torch.zeros((2, 8 * 16), dtype=torch.float32, device="cuda")
    sc.salicache_saliency_noalloc(small, fr, 2, s)                          # NULL status word
    torch.cuda.synchronize()
    assert np.array_equal(s.cpu().numpy(), _reference(small, fr))
    capped = sc.salicache_default_params(L=1, hyst_max_iters=1, canny_lo=20, canny_hi=200)
    full = torch.from_numpy(synth.frames(2, T=1)).cuda()
    s1 = torch.zeros((1, 576), dtype=torch.float32, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    sc.salicache_saliency_noalloc(capped, full, 1, s1, status)              # one sweep cannot finish the edges
    torch.cuda.synchronize()
    assert int(status.item()) == sc.E_NOCONVERGE
    lib = sc.lib()
    ok = sc.salicache_default_params(L=1)
    big = sc.salicache_default_params(H=672, W=672, L=1)
    f336 = torch.zeros((1, 336, 336, 3), dtype=torch.uint8, device="cuda")
    out = torch.zeros((9, 576), dtype=torch.float32, device="cuda")
    call = lambda p, f, B, o: lib.salicache_saliency_noalloc(ctypes.byref(p), f, B, o, None, None)
    assert call(ok, f336.data_ptr(), sc.NOALLOC_MAX_FRAMES + 1, out.data_ptr()) == sc.E_SHAPE
    assert call(big, f336.data_ptr(), 1, out.data_ptr()) == sc.E_SHAPE
    assert call(ok, None, 1, out.data_ptr()) == sc.E_NULL
    assert call(ok, f336.data_ptr() + 1, 1, out.data_ptr()) == sc.E_ALIGN
    assert call(ok, f336.data_ptr(), 0, out.data_ptr()) == 0
    torch.cuda.synchronize()

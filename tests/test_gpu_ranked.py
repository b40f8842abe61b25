"""GPU parity of the adaptive tier rule (salicache_select_ranked) against the oracle, through the C ABI: integer work on
the same float32 scores, so decisions, index lists, counts, flags, row offsets and the running fill are compared bit
for bit."""
import numpy as np
import pytest

import oracle
from paper_2602_14236_b200 import binding as sc
from paper_2602_14236_b200 import synth

import gpu_util as gu

pytestmark = pytest.mark.gpu


def _run(ctx, dP, s, first, shares, fill0=(0, 0, 0)):
    import torch
    T, n = s.shape
    d = dict(
        decision=torch.full((T, n), 255, dtype=torch.uint8, device="cuda"),
        idx=torch.full((T, 3, n), -7, dtype=torch.int32, device="cuda"),
        counts=torch.full((T, 5), -1, dtype=torch.int32, device="cuda"),
        redundant=torch.full((T,), 255, dtype=torch.uint8, device="cuda"),
        row_offset=torch.full((T, 3), -1, dtype=torch.int64, device="cuda"),
        fill=torch.tensor(list(fill0), dtype=torch.int64, device="cuda"),
    )
    d_dP = torch.from_numpy(dP).cuda() if dP is not None else None
    sc.salicache_select_ranked(ctx, d_dP, torch.from_numpy(s).cuda(), T, first, shares, d["decision"], d["idx"], d["counts"],
                               d["redundant"], d["row_offset"], d["fill"])
    torch.cuda.synchronize()
    return {k: v.cpu().numpy() for k, v in d.items()}


@pytest.mark.parametrize("anyres,patch_reuse,shares", [(False, 1, (432, 97, 292)), (False, 0, (250, 250, 250)),
                                                       (True, 1, (317, 71, 214)), (False, 1, (1000, 1000, 0))])
def test_ranked_select_matches_the_oracle(anyres, patch_reuse, shares):
    rng = np.random.default_rng(17 + anyres + patch_reuse)
    T = 6
    kw = dict(H=672, W=672, n_images=5) if anyres else {}
    ctx = sc.Context(sc.salicache_default_params(max_batch=8, chunk_frames=2, L=1, patch_reuse=patch_reuse, **kw))
    n = ctx.n_tok
    assert n == (2880 if anyres else 576)
    s = rng.uniform(0.0, 0.7, (T, n)).astype(np.float32)
    s[2] = np.round(s[2] * 8) / 8                           # a frame full of ties
    s[3] = 0.01 * s[3]                                      # a frame that fixed thresholds would prune wholly
    dP = rng.uniform(0.0, 1.2, (T, n)).astype(np.float32)
    dP[4] = 0.1                                             # a redundant frame
    dP[5, : n // 2] = 0.2                                   # half the patches static
    p = gu.oracle_params(ctx.params)
    fill0 = (5, 0, 11)
    got = _run(ctx, dP, s, True, shares, fill0)
    fill = np.asarray(fill0, np.int64)
    for t in range(T):
        dec, idx, counts, red = oracle.select_ranked(dP[t], s[t], t > 0, shares, p)
        assert np.array_equal(got["decision"][t], dec), t
        assert np.array_equal(got["idx"][t], idx), t
        assert np.array_equal(got["counts"][t], counts), t
        assert got["redundant"][t] == red
        assert np.array_equal(got["row_offset"][t], fill)
        fill = fill + counts[[oracle.FP16, oracle.INT8, oracle.INT4]]
    assert np.array_equal(got["fill"], fill)
    assert got["redundant"].tolist() == [0, 0, 0, 0, 1, 0]
    if patch_reuse:
        assert got["counts"][5, 0] >= n // 2
    # without temporal scores every frame ranks all its tokens
    got = _run(ctx, None, s, False, shares)
    for t in range(T):
        dec, idx, counts, red = oracle.select_ranked(None, s[t], False, shares, p)
        assert np.array_equal(got["decision"][t], dec) and np.array_equal(got["idx"][t], idx) and red == 0


def test_ranked_select_argument_checks():
    import torch
    lib = sc.lib()
    ctx = sc.Context(sc.salicache_default_params(max_batch=4, chunk_frames=2, L=1))
    n = ctx.n_tok
    s = torch.zeros((2, n), dtype=torch.float32, device="cuda")
    dec = torch.zeros((2, n), dtype=torch.uint8, device="cuda")
    idx = torch.zeros((2, 3, n), dtype=torch.int32, device="cuda")
    cnt = torch.zeros((2, 5), dtype=torch.int32, device="cuda")
    red = torch.zeros((2,), dtype=torch.uint8, device="cuda")
    off = torch.zeros((2, 3), dtype=torch.int64, device="cuda")
    fill = torch.zeros((3,), dtype=torch.int64, device="cuda")
    call = lambda sp, B, pm: lib.salicache_select_ranked(ctx.handle, None, sp, B, 1, pm, 100, 100, dec.data_ptr(), idx.data_ptr(),
                                                         cnt.data_ptr(), red.data_ptr(), off.data_ptr(), fill.data_ptr(), None)
    assert call(None, 2, 100) == sc.E_NULL
    assert call(s.data_ptr(), 5, 100) == sc.E_SHAPE
    assert call(s.data_ptr(), 2, 1001) == sc.E_PARAM and call(s.data_ptr(), 2, -1) == sc.E_PARAM
    assert call(s.data_ptr(), 0, 100) == 0

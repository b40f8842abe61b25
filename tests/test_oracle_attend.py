"""Pins of the oracle's decode attention over the mixed-precision store (Eq. 2 with the just-in-time
dequantisation of Sec. III-C): special cases with closed forms, and the textbook softmax-attention
written with library routines on the dequantised cache."""
import numpy as np
import pytest

import oracle


def _filled_pools(rng, L=2, H=3, D=128, n=(5, 7, 6)):
    HD = H * D
    K = rng.standard_normal((L, sum(n), HD)).astype(np.float16)
    V = rng.standard_normal((L, sum(n), HD)).astype(np.float16)
    pools = oracle.Pools(L, HD, 128, n[0] + 2, n[1] + 1, n[2] + 3)
    idx = np.full((3, sum(n)), -1, np.int32)
    idx[0, :n[0]] = np.arange(0, n[0])
    idx[1, :n[1]] = np.arange(n[0], n[0] + n[1])
    idx[2, :n[2]] = np.arange(n[0] + n[1], sum(n))
    counts = np.array([0, 0, n[2], n[1], n[0]], np.int32)
    oracle.pack_frame(K.view(np.uint16), V.view(np.uint16), idx, counts, np.zeros(3, np.int64), pools)
    return pools, n


def _dense(pools, n, L, H, D):
    """The cache the pools hold, dequantised in exact arithmetic: [L][2][rows][H][D] float64."""
    HD = H * D
    hf = lambda a: a.view(np.float16).astype(np.float64)
    k16 = hf(pools.fp16_pool[:, :, :n[0]])
    s8 = hf(pools.int8_scale[:, :, :n[1]])
    k8 = pools.int8_codes[:, :, :n[1]].astype(np.float64).reshape(L, 2, n[1], HD // 128, 128) * s8[..., None]
    sz = hf(pools.int4_sz[:, :, :n[2]])
    c4 = pools.int4_codes[:, :, :n[2]]
    nib = np.stack([c4 & 15, c4 >> 4], axis=-1).reshape(L, 2, n[2], HD).astype(np.float64)
    k4 = nib.reshape(L, 2, n[2], HD // 128, 128) * sz[..., 0:1] + sz[..., 1:2]
    return np.concatenate([k16, k8.reshape(L, 2, n[1], HD), k4.reshape(L, 2, n[2], HD)], axis=2).reshape(L, 2, sum(n), H, D)


def test_attention_equals_softmax_attention_on_the_dequantised_cache():
    from scipy.special import softmax
    rng = np.random.default_rng(0)
    L, H, D = 2, 3, 128
    pools, n = _filled_pools(rng, L, H, D)
    q = rng.standard_normal((L, H, D)).astype(np.float16)
    got = oracle.attend(q.view(np.uint16), pools, n)
    dense = _dense(pools, n, L, H, D)
    scores = np.einsum("lhd,ljhd->lhj", q.astype(np.float64), dense[:, 0]) / np.sqrt(D)
    want = np.einsum("lhj,ljhd->lhd", softmax(scores, axis=-1), dense[:, 1])
    assert np.allclose(got, want, rtol=1e-12, atol=1e-13)


def test_single_row_returns_its_value_and_equal_keys_average_the_values():
    rng = np.random.default_rng(1)
    L, H, D = 1, 2, 128
    pools, n = _filled_pools(rng, L, H, D, n=(1, 0, 0))
    q = rng.standard_normal((L, H, D)).astype(np.float16)
    got = oracle.attend(q.view(np.uint16), pools, n)
    assert np.array_equal(got, _dense(pools, n, L, H, D)[:, 1, 0])            # softmax of one score is 1
    # equal keys in every tier: uniform weights, the output is the mean of the dequantised values
    pools, n = _filled_pools(rng, L, H, D, n=(3, 3, 3))
    pools.fp16_pool[:, 0] = pools.fp16_pool[:, 0, :1]
    pools.int8_codes[:, 0] = 0
    pools.int4_codes[:, 0] = 0
    pools.int4_sz[:, 0, :, :, 1] = 0
    pools.fp16_pool[:, 0] = 0                                                  # all keys are the zero vector
    got = oracle.attend(q.view(np.uint16), pools, n)
    assert np.allclose(got, _dense(pools, n, L, H, D)[:, 1].mean(axis=1), rtol=1e-13, atol=1e-14)


def test_empty_store_row_order_and_query_scale():
    rng = np.random.default_rng(2)
    L, H, D = 1, 2, 128
    pools, n = _filled_pools(rng, L, H, D, n=(4, 4, 4))
    q = rng.standard_normal((L, H, D)).astype(np.float16)
    assert np.array_equal(oracle.attend(q.view(np.uint16), pools, (0, 0, 0)), np.zeros((L, H, D)))
    full = oracle.attend(q.view(np.uint16), pools, n)
    # attention is a set function of the rows: swapping two rows of a pool (keys and values together) changes nothing
    for arr in (pools.int8_codes, pools.int8_scale):
        arr[:, :, [0, 2]] = arr[:, :, [2, 0]]
    assert np.allclose(oracle.attend(q.view(np.uint16), pools, n), full, rtol=1e-12, atol=1e-14)
    # a zero query weighs every row equally
    z = np.zeros((L, H, D), np.float16)
    assert np.allclose(oracle.attend(z.view(np.uint16), pools, n), _dense(pools, n, L, H, D)[:, 1].mean(axis=1), rtol=1e-13)
    # rows beyond n are ignored
    part = oracle.attend(q.view(np.uint16), pools, (4, 2, 0))
    dense = _dense(pools, (4, 2, 0), L, H, D)
    from scipy.special import softmax
    sc = np.einsum("lhd,ljhd->lhj", q.astype(np.float64), dense[:, 0]) / np.sqrt(D)
    assert np.allclose(part, np.einsum("lhj,ljhd->lhd", softmax(sc, axis=-1), dense[:, 1]), rtol=1e-12, atol=1e-13)


def test_grouped_query_attention_against_library_softmax_and_the_one_query_per_head_routine():
    """Query head hq reads key/value head hq // q_per_kv.  Pinned by the textbook expression with library routines on
    the dequantised cache, by q_per_kv = 1 (the plain routine), and by feeding the plain routine the queries of one
    slot of every group (it must return that slot's rows of the grouped result)."""
    from scipy.special import softmax
    rng = np.random.default_rng(4)
    L, H, D, G = 2, 3, 128, 4
    pools, n = _filled_pools(rng, L, H, D)
    q = rng.standard_normal((L, H * G, D)).astype(np.float16)
    got = oracle.attend_gqa(q.view(np.uint16), pools, n, G)
    dense = _dense(pools, n, L, H, D)                                            # [L][2][rows][H][D]
    kv = np.repeat(dense, G, axis=3)                                             # key/value head of every query head
    scores = np.einsum("lhd,ljhd->lhj", q.astype(np.float64), kv[:, 0]) / np.sqrt(D)
    want = np.einsum("lhj,ljhd->lhd", softmax(scores, axis=-1), kv[:, 1])
    assert np.allclose(got, want, rtol=1e-12, atol=1e-13)
    for slot in range(G):
        plain = oracle.attend(np.ascontiguousarray(q[:, slot::G]).view(np.uint16), pools, n)
        assert np.array_equal(plain, got[:, slot::G])
    q1 = rng.standard_normal((L, H, D)).astype(np.float16)
    assert np.array_equal(oracle.attend_gqa(q1.view(np.uint16), pools, n, 1), oracle.attend(q1.view(np.uint16), pools, n))
    # a transposed head mapping (hq % H instead of hq // q_per_kv) would fail the slot test above; check it does differ
    wrong = np.einsum("lhj,ljhd->lhd", softmax(np.einsum("lhd,ljhd->lhj", q.astype(np.float64), np.tile(dense, (1, 1, 1, G, 1))[:, 0]) / np.sqrt(D), axis=-1),
                      np.tile(dense, (1, 1, 1, G, 1))[:, 1])
    assert not np.allclose(got, wrong, rtol=1e-6, atol=1e-8)

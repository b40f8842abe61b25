"""Pins of the oracle's budget bookkeeping: which frames a ring of pool rows still holds after oldest-first
eviction, that a reused token dies with the frame holding its entry, and that unpacking never returns another
frame's rows."""
import numpy as np

import oracle

FP16, INT8, INT4 = oracle.FP16, oracle.INT8, oracle.INT4
CODE = (FP16, INT8, INT4)


def _last_writer_residency(counts, off, caps, upto):
    """Brute force: replay every row write of frames 0..upto into slot tables; a frame is resident when it still
    owns every slot it wrote."""
    T = counts.shape[0]
    owner = [dict() for _ in range(3)]
    for t in range(upto + 1):
        for k in range(3):
            for j in range(int(counts[t, CODE[k]])):
                owner[k][(int(off[t, k]) + j) % int(caps[k])] = (t, j)
    res = np.zeros(upto + 1, np.uint8)
    for t in range(upto + 1):
        res[t] = all(owner[k].get((int(off[t, k]) + j) % int(caps[k])) == (t, j)
                     for k in range(3) for j in range(int(counts[t, CODE[k]])))
    return res


def test_ring_residency_equals_the_last_writer_of_every_slot():
    rng = np.random.default_rng(12)
    for trial in range(6):
        T = 30
        counts = np.zeros((T, 5), np.int32)
        counts[:, FP16] = rng.integers(0, 9, T)
        counts[:, INT8] = rng.integers(0, 30, T) * (rng.random(T) < 0.7)
        counts[:, INT4] = rng.integers(0, 60, T)
        counts[10, INT4] = 400                                   # one frame larger than its ring
        caps = np.array([17 + trial, 64, 150 + 10 * trial], np.int64)
        fill0 = np.array([5, 0, 1000], np.int64)
        off, _ = oracle.row_offsets(counts, fill0)
        for upto in (0, 7, 18, T - 1):
            fill = off[upto] + counts[upto, list(CODE)]
            want = _last_writer_residency(counts, off, caps, upto)
            got = oracle.frames_resident(counts[:upto + 1], off[:upto + 1], caps, True, fill)
            assert np.array_equal(got, want), (trial, upto)
        assert 0 < got.sum() < T


def test_linear_pools_hold_what_fits_and_nothing_else():
    counts = np.zeros((4, 5), np.int32)
    counts[:, INT4] = [10, 10, 10, 0]
    counts[:, FP16] = [1, 0, 0, 0]
    off, fill = oracle.row_offsets(counts)
    caps = np.array([1, 0, 25], np.int64)
    assert oracle.frames_resident(counts, off, caps, False, fill).tolist() == [1, 1, 0, 1]
    assert oracle.frames_resident(counts, off, np.array([0, 0, 25], np.int64), False, fill).tolist() == [0, 1, 0, 1]


def test_tokens_live_follow_their_source_frame():
    dec = np.array([[4, 2, 1],
                    [0, 4, 0],
                    [0, 0, 2],
                    [4, 0, 0]], np.uint8)
    src = oracle.source_frames(dec)                      # [[0,0,0],[0,1,0],[0,1,2],[3,1,2]]
    resident = np.array([0, 1, 1, 1], np.uint8)          # frame 0 has been evicted
    live = oracle.tokens_live(src, 0, resident)
    assert live.tolist() == [[0, 0, 0], [0, 1, 0], [0, 1, 1], [1, 1, 1]]
    # a table that starts at frame 2: sources before it count as evicted
    assert oracle.tokens_live(src[2:], 2, resident[2:]).tolist() == [[0, 0, 1], [1, 0, 1]]
    rng = np.random.default_rng(3)
    dec = rng.integers(0, 5, (25, 40)).astype(np.uint8)
    dec[0][dec[0] == 0] = 2
    src = oracle.source_frames(dec)
    resident = (rng.random(25) < 0.6).astype(np.uint8)
    live = oracle.tokens_live(src, 0, resident)
    for t in range(25):
        for i in range(40):
            k = t
            while dec[k, i] == 0:                        # walk the reuse chain by hand
                k -= 1
            assert live[t, i] == resident[k]


def test_unpack_never_returns_rows_of_a_newer_frame():
    """Five frames into a ring that holds about two: unpacking with the running fill zeroes exactly the rows that
    have been overwritten (whole evicted frames, and the older part of the frame at the boundary) and returns the
    others unchanged."""
    L, n_tok, HD, G = 2, 24, 256, 128
    rng = np.random.default_rng(8)
    frames, decs = [], []
    for t in range(5):
        K = rng.standard_normal((L, n_tok, HD)).astype(np.float16).view(np.uint16)
        V = rng.standard_normal((L, n_tok, HD)).astype(np.float16).view(np.uint16)
        s = rng.uniform(0.2, 0.6, n_tok).astype(np.float32)
        dec, idx, counts, _, _ = oracle.select(np.ones(n_tok, np.float32), s, True, oracle.Params())
        frames.append((K, V, idx, counts))
        decs.append(dec)
    counts_all = np.stack([f[3] for f in frames])
    off, fill = oracle.row_offsets(counts_all)
    caps = np.array([int(1.6 * counts_all[:, c].mean()) + 1 for c in CODE], np.int64)
    pools = oracle.Pools(L, HD, G, *[int(c) for c in caps], ring=1)
    fresh = []
    for t, (K, V, idx, counts) in enumerate(frames):
        assert oracle.pack_frame(K, V, idx, counts, off[t], pools) == 0
        Ko, Vo = np.zeros_like(K), np.zeros_like(V)
        assert oracle.unpack_frame(n_tok, idx, counts, decs[t], off[t], pools, False, Ko, Vo) == 0
        fresh.append((Ko, Vo))                               # what the frame reads right after its own store
    resident = oracle.frames_resident(counts_all, off, caps, True, fill)
    assert resident.tolist()[0] == 0 and resident.tolist()[-1] == 1
    saw_partial = False
    for t, (K, V, idx, counts) in enumerate(frames):
        Ko, Vo = np.full_like(K, 0x7E00), np.full_like(V, 0x7E00)
        st = oracle.unpack_frame(n_tok, idx, counts, decs[t], off[t], pools, False, Ko, Vo, fill=fill)
        assert (st == 0) == bool(resident[t])
        n_zero = 0
        for k, code in enumerate(CODE):
            for j in range(int(counts[code])):
                tok = idx[k, j]
                gone = off[t, k] + j < fill[k] - caps[k]
                want = 0 if gone else fresh[t][0][:, tok]
                assert np.array_equal(Ko[:, tok], np.zeros_like(Ko[:, tok]) if gone else want)
                assert np.array_equal(Vo[:, tok], np.zeros_like(Vo[:, tok]) if gone else fresh[t][1][:, tok])
                n_zero += int(gone)
        stored = int(counts[list(CODE)].sum())
        saw_partial |= 0 < n_zero < stored
    assert saw_partial

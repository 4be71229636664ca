"""Pins of the oracle's incremental path (oracle.append) against facts that do not come from it.

The reading: generated tokens are chunked by Eq. 1 as a stream that starts afresh behind the
prompt, and a finished chunk is clustered and pooled like a prompt chunk.  What fixes the result:
  * a stream that ends on a chunk boundary must leave exactly the cores the one-shot compress
    stage (chunk -> gsc -> merge, pinned elsewhere) produces for the same tokens;
  * a stream that stops inside a chunk leaves those cores for the finished part and the open
    tokens untouched behind them;
  * a case small enough to work by hand.
"""
import numpy as np
import pytest

import oracle

DELIM = [13, 29889]


def _stream(seed, B, Hkv, m, d, p_delim, n_centroids=4, sigma=0.05, dtype=np.float32):
    rng = np.random.default_rng(seed)
    ids = rng.integers(100, 30000, size=(B, m)).astype(np.int32)
    ids[np.isin(ids, DELIM)] = 99
    ids[rng.random((B, m)) < p_delim] = DELIM[0]
    cent = rng.normal(size=(n_centroids, d))
    cent /= np.linalg.norm(cent, axis=1, keepdims=True)
    pick = rng.integers(0, n_centroids, size=(B, Hkv, m))
    K = cent[pick] + sigma / np.sqrt(d) * rng.normal(size=(B, Hkv, m, d))
    V = rng.normal(size=(B, Hkv, m, d))
    if dtype == np.uint16:   # any bf16 bit patterns will do: keep the top half of the fp32 bits
        K = (K.astype(np.float32).view(np.uint32) >> 16).astype(np.uint16)
        V = (V.astype(np.float32).view(np.uint32) >> 16).astype(np.uint16)
    else:
        K, V = K.astype(np.float32), V.astype(np.float32)
    return ids, K, V


def _empty_state(B, Hkv, cap, d, dtype):
    return dict(core_k=np.zeros((B, Hkv, cap, d), dtype), core_v=np.zeros((B, Hkv, cap, d), dtype),
                count=np.zeros((B, Hkv, cap), np.int32), core_len=np.zeros((B, Hkv), np.int32),
                tail_len=np.zeros((B, Hkv), np.int32))


def _run(ids, K, V, tau, max_len, upto=None):
    B, Hkv, m, d = K.shape
    st = _empty_state(B, Hkv, m, d, K.dtype)
    for t in range(m if upto is None else upto):
        oracle.append(st, ids[:, t], K[:, :, t], V[:, :, t], DELIM, tau, max_len)
    return st


@pytest.mark.parametrize("dtype", [np.float32, np.uint16])
@pytest.mark.parametrize("seed,max_len,p_delim", [(0, 256, 0.08), (1, 8, 0.05), (2, 5, 0.0), (3, 256, 0.5)])
def test_stream_ending_on_a_boundary_equals_one_shot_compress(dtype, seed, max_len, p_delim):
    B, Hkv, m, d = 3, 2, 120, 16
    ids, K, V = _stream(seed, B, Hkv, m, d, p_delim, dtype=dtype)
    ids[:, -1] = DELIM[1]   # every sequence ends by closing its chunk
    ref = oracle.compress(ids, DELIM, K, V, 0.7, max_len)
    st = _run(ids, K, V, 0.7, max_len)
    assert np.array_equal(st["core_len"], ref["core_len"]) and not st["tail_len"].any()
    for b in range(B):
        for h in range(Hkv):
            L = ref["core_len"][b, h]
            assert np.array_equal(st["count"][b, h, :L], ref["count"][b, h, :L])
            assert np.array_equal(st["core_k"][b, h, :L], ref["core_k"][b, h, :L])
            assert np.array_equal(st["core_v"][b, h, :L], ref["core_v"][b, h, :L])
    if p_delim < 0.5:
        assert st["margin"] == ref["margin"]


def test_stream_stopping_inside_a_chunk_keeps_the_open_tokens_as_they_came():
    B, Hkv, m, d = 2, 3, 90, 8
    ids, K, V = _stream(7, B, Hkv, m, d, 0.07)
    ids[:, 70] = DELIM[0]
    ids[:, 71:] = 500          # 19 open tokens behind the last delimiter
    st = _run(ids, K, V, 0.7, 64)
    ref = oracle.compress(ids[:, :71], DELIM, K[:, :, :71], V[:, :, :71], 0.7, 64)
    assert np.array_equal(st["core_len"], ref["core_len"])
    assert (st["tail_len"] == 19).all()
    for b in range(B):
        for h in range(Hkv):
            L = ref["core_len"][b, h]
            assert np.array_equal(st["core_k"][b, h, :L], ref["core_k"][b, h, :L])
            assert np.array_equal(st["core_k"][b, h, L:L + 19], K[b, h, 71:])
            assert np.array_equal(st["core_v"][b, h, L:L + 19], V[b, h, 71:])
            assert (st["count"][b, h, L:L + 19] == 1).all()


def test_hand_worked_stream():
    """Keys in the plane, tau = 0.7.  Tokens: a = (1, 0), b = (1, 0.1), c = (0, 1), a delimiter, e = (0, 2).
    cos(a, b) = 1 / sqrt(1.01) = 0.995 > 0.7 and cos(a, c) = 0: the first chunk is {a, b}, {c}.  The
    delimiter closes it and stays a core of its own.  e is an open tail of one token."""
    ids = np.array([[100, 101, 102, 13, 103]], np.int32)
    K = np.array([[1, 0], [1, 0.1], [0, 1], [5, 5], [0, 2]], np.float32)[None, None]
    V = np.array([[2, 0], [4, 2], [7, 7], [9, 9], [1, 1]], np.float32)[None, None]
    st = _empty_state(1, 1, 5, 2, np.float32)
    lens = []
    for t in range(5):
        oracle.append(st, ids[:, t], K[:, :, t], V[:, :, t], DELIM, 0.7, 256)
        lens.append((int(st["core_len"][0, 0]), int(st["tail_len"][0, 0])))
    assert lens == [(0, 1), (0, 2), (0, 3), (3, 0), (3, 1)]
    assert st["count"][0, 0].tolist() == [2, 1, 1, 1, 0]
    np.testing.assert_allclose(st["core_k"][0, 0, :4], [[1, 0.05], [0, 1], [5, 5], [0, 2]], rtol=1e-7)
    np.testing.assert_allclose(st["core_v"][0, 0, :4], [[3, 1], [7, 7], [9, 9], [1, 1]], rtol=1e-7)


def test_length_cut_and_neighbouring_delimiters():
    # max_chunk_len 3, no merging (tau above every similarity): cuts after every third ordinary token
    ids = np.array([[1, 2, 3, 4, 13, 13, 5, 6, 7, 8]], np.int32)
    K = np.eye(10, dtype=np.float32)[None, None]
    st = _empty_state(1, 1, 10, 10, np.float32)
    lens = []
    for t in range(10):
        oracle.append(st, ids[:, t], K[:, :, t], K[:, :, t], DELIM, 2.0, 3)
        lens.append((int(st["core_len"][0, 0]), int(st["tail_len"][0, 0])))
    assert lens == [(0, 1), (0, 2), (3, 0), (3, 1), (5, 0), (6, 0), (6, 1), (6, 2), (9, 0), (9, 1)]
    assert np.array_equal(st["core_k"][0, 0], K[0, 0])   # nothing merged, nothing moved


def test_a_full_cache_is_refused():
    st = _empty_state(1, 1, 2, 4, np.float32)
    k = np.ones((1, 1, 4), np.float32)
    oracle.append(st, [1], k, k, DELIM, 0.7)
    oracle.append(st, [2], k, k, DELIM, 0.7)
    with pytest.raises(OverflowError):
        oracle.append(st, [3], k, k, DELIM, 0.7)

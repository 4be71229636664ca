"""Pins for the oracle's multi-query Proportional Attention (Eq. 4 with Q in R^{m x d}) and for the
"no chunking" ablation arm (Algorithm 1 over a whole sequence, Table 4a)."""
import itertools

import numpy as np
import pytest

import oracle


def _cache(rng, B=2, Hkv=2, cap=37, d=16):
    ck = rng.normal(size=(B, Hkv, cap, d)).astype(np.float32)
    cv = rng.normal(size=(B, Hkv, cap, d)).astype(np.float32)
    cnt = rng.integers(1, 9, size=(B, Hkv, cap)).astype(np.int32)
    clen = rng.integers(cap // 2, cap + 1, size=(B, Hkv)).astype(np.int32)
    return ck, cv, cnt, clen


def test_one_query_is_the_decode_step():
    rng = np.random.default_rng(0)
    ck, cv, cnt, clen = _cache(rng)
    q = rng.normal(size=(2, 6, 1, 16)).astype(np.float32)
    a = oracle.attn_multi(q, ck, cv, cnt, clen)
    b = oracle.attn(q[:, :, 0], ck, cv, cnt, clen)
    assert np.array_equal(a[:, :, 0], b)
    assert np.array_equal(oracle.attn_multi(q, ck, cv, cnt, clen, causal=True), a)   # m = 1: the mask is empty


@pytest.mark.parametrize("causal", [False, True])
def test_counts_of_one_give_textbook_attention(causal):
    """All counts 1 (no merging): softmax(Q K^T / sqrt(d) [+ causal mask over the last m rows]) V, written
    with numpy for one head at a time."""
    rng = np.random.default_rng(1)
    B, Hkv, G, m, d, cap = 1, 2, 3, 5, 8, 19
    ck, cv, _, clen = _cache(rng, B, Hkv, cap, d)
    clen[:] = [[cap, 11]]
    q = rng.normal(size=(B, Hkv * G, m, d)).astype(np.float32)
    got = oracle.attn_multi(q, ck, cv, None, clen, causal=causal)
    for hq in range(Hkv * G):
        h, L = hq // G, int(clen[0, hq // G])
        S = q[0, hq].astype(np.float64) @ ck[0, h, :L].astype(np.float64).T / np.sqrt(d)      # [m, L]
        if causal:
            t = np.arange(L)[None, :]
            i = np.arange(m)[:, None]
            S = np.where(t < L - (m - 1 - i), S, -np.inf)
        P = np.exp(S - S.max(axis=1, keepdims=True))
        want = (P / P.sum(axis=1, keepdims=True)) @ cv[0, h, :L].astype(np.float64)
        assert np.allclose(got[0, hq], want, rtol=1e-12, atol=1e-14)


def test_clusters_of_identical_tokens_reproduce_uncompressed_attention_for_every_query():
    """The paper's remark under Eq. 4: adding log s multiplies the post-exponential score by s.  Cores that
    stand for s identical (k, v) tokens must give every one of the m queries exactly what attention over
    the expanded cache gives."""
    rng = np.random.default_rng(2)
    d, m = 8, 4
    sizes = [3, 1, 5, 2]
    ck = rng.normal(size=(1, 1, len(sizes), d)).astype(np.float32)
    cv = rng.normal(size=(1, 1, len(sizes), d)).astype(np.float32)
    cnt = np.array([[sizes]], dtype=np.int32)
    q = rng.normal(size=(1, 2, m, d)).astype(np.float32)
    comp = oracle.attn_multi(q, ck, cv, cnt, np.array([[len(sizes)]], dtype=np.int32))
    rep = np.repeat(np.arange(len(sizes)), sizes)
    full = oracle.attn_multi(q, ck[:, :, rep], cv[:, :, rep], None, np.array([[len(rep)]], dtype=np.int32))
    assert np.allclose(comp, full, rtol=1e-12, atol=1e-14)
    plain = oracle.attn_multi(q, ck, cv, None, np.array([[len(sizes)]], dtype=np.int32))
    assert not np.allclose(plain, full, rtol=1e-3)      # the pin bites without log s


def test_causal_query_i_is_a_decode_step_over_a_shorter_cache():
    rng = np.random.default_rng(3)
    ck, cv, cnt, clen = _cache(rng, B=1, Hkv=2, cap=23, d=8)
    m = 6
    clen[:] = [[23, 4]]      # the second head is shorter than m: its first queries see nothing
    q = rng.normal(size=(1, 4, m, 8)).astype(np.float32)
    got = oracle.attn_multi(q, ck, cv, cnt, clen, causal=True)
    for i in range(m):
        want = oracle.attn(q[:, :, i], ck, cv, cnt, np.maximum(clen - (m - 1 - i), 0).astype(np.int32))
        assert np.allclose(got[:, :, i], want, rtol=1e-13, atol=1e-15)
    assert np.all(got[0, 2:, 0] == 0) and np.all(got[0, 2:, 1] == 0)      # 4 - (5 - i) <= 0 for i = 0, 1


# ------------------------------------------------------------------ global clustering (no chunking)


def test_global_clustering_is_algorithm_1_with_one_chunk_per_sequence():
    """Brute force: the seeds are the lexicographically first maximal independent set of the graph
    Sim > tau over the WHOLE sequence, every other token joins its lowest adjacent seed; a delimiter-like
    token in the middle does not stop a cluster."""
    rng = np.random.default_rng(4)
    n, d, tau = 11, 6, 0.5
    cent = rng.normal(size=(3, d))
    K = (cent[rng.integers(0, 3, size=(1, 1, n))] + 0.3 * rng.normal(size=(1, 1, n, d))).astype(np.float32)
    V = rng.normal(size=K.shape).astype(np.float32)
    r = oracle.compress_global(K, V, tau)
    assert r["margin"] > 1e-6
    sim = np.array([[oracle.sim(K[0, 0], i, j) for j in range(n)] for i in range(n)])
    adj = sim > tau
    best = None
    for k in range(1, n + 1):
        for sub in itertools.combinations(range(n), k):
            indep = all(not adj[a, b] for a, b in itertools.combinations(sub, 2))
            maximal = all(any(adj[t, s_] for s_ in sub) for t in range(n) if t not in sub)
            if indep and maximal and (best is None or list(sub) < list(best)):
                best = sub
    seeds = [t for t in range(n) if r["assign"][0, 0, t] == t]
    assert seeds == list(best)
    for t in range(n):
        if t not in seeds:
            assert r["assign"][0, 0, t] == min(s_ for s_ in seeds if adj[s_, t])
    assert int(r["core_len"][0, 0]) == len(seeds) and int(r["count"][0, 0, :len(seeds)].sum()) == n


def test_global_clustering_merges_across_what_chunking_would_separate():
    """Two identical tokens on either side of a delimiter: chunked compression keeps both, global merges them."""
    d = 8
    k = np.zeros((1, 1, 3, d), dtype=np.float32)
    k[0, 0, 0, 0] = k[0, 0, 2, 0] = 1.0
    k[0, 0, 1, 1] = 1.0                      # the delimiter's key, orthogonal
    v = np.arange(3 * d, dtype=np.float32).reshape(1, 1, 3, d)
    ids = np.array([[5, 7, 5]], dtype=np.int32)
    chunked = oracle.compress(ids, (7,), k, v, 0.5)
    glob = oracle.compress_global(k, v, 0.5)
    assert int(chunked["core_len"][0, 0]) == 3 and int(glob["core_len"][0, 0]) == 2
    assert glob["assign"][0, 0].tolist() == [0, 1, 0] and glob["count"][0, 0, :2].tolist() == [2, 1]
    assert np.array_equal(glob["core_v"][0, 0, 0], (v[0, 0, 0] + v[0, 0, 2]) / 2)

"""Pins for the oracle's merge (Eq. 3), bf16 rounding and proportional attention (Eq. 4).

Reference values come from hand arithmetic, torch's own float->bf16 conversion and a
textbook softmax attention written with numpy / scipy; never from the oracle itself.
"""
import math

import numpy as np
import pytest
import torch
from scipy.special import softmax

import oracle

DELIMS = (13, 29889, 29892)


def _bits(x):
    return torch.as_tensor(np.asarray(x, dtype=np.float32)).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)


def _textbook_attention(q, K, V, G, scale=None):
    """softmax(q K^T / sqrt(d)) V per query head, KV head = hq // G (float64 numpy)."""
    B, Hq, d = q.shape
    scale = 1.0 / math.sqrt(d) if scale is None else scale
    out = np.zeros((B, Hq, d))
    for b in range(B):
        for hq in range(Hq):
            s = (K[b, hq // G] @ q[b, hq]) * scale
            out[b, hq] = softmax(s) @ V[b, hq // G]
    return out


# ------------------------------------------------------------ bf16 rounding


def test_bf16_rounding_matches_torch_and_ties_to_even():
    rng = np.random.default_rng(0)
    x = np.concatenate([rng.normal(size=4000), rng.normal(size=2000) * 1e-3, rng.normal(size=2000) * 1e4,
                        [0.0, -0.0, 1.0, -1.0, 3.3e38, -3.3e38, 1e-40, 65504.0]]).astype(np.float32)
    want = _bits(x)
    got = np.array([oracle.f64_to_bf16_bits(float(v)) for v in x], dtype=np.uint16)
    assert np.array_equal(got, want)
    # exact ties, worked by hand: spacing at 1.0 is 2^-7
    assert oracle.f64_to_bf16_bits(1.0 + 2.0 ** -8) == 0x3F80          # tie -> even mantissa 0
    assert oracle.f64_to_bf16_bits(1.0 + 3 * 2.0 ** -8) == 0x3F82      # tie -> even mantissa 2
    assert oracle.f64_to_bf16_bits(1.0 + 2.0 ** -8 + 2.0 ** -40) == 0x3F81  # just above a tie (a double
    # rounded through float32 first would lose the 2^-40 and give 0x3F80)
    assert oracle.f64_to_bf16_bits(-(1.0 + 3 * 2.0 ** -8)) == 0xBF82


# -------------------------------------------------------------------- Eq. 3


def test_merge_hand_worked_means_counts_and_order():
    # one head, 7 tokens, d = 2; tokens 0,2,6 form a cluster, 1,4 another, 3,5 another
    K = np.array([[1, 10], [2, 20], [3, 30], [4, 40], [6, 60], [8, 80], [5, 50]], dtype=np.float32)
    V = -2.0 * K + 1.0
    assign = np.array([0, 1, 0, 3, 1, 3, 0], dtype=np.int32)
    ck, cv, cnt, clen = oracle.merge(K.reshape(1, 1, 7, 2), V.reshape(1, 1, 7, 2), assign.reshape(1, 1, 7))
    assert clen.tolist() == [[3]]
    assert cnt[0, 0, :3].tolist() == [3, 2, 2]
    assert ck[0, 0, :3].tolist() == [[3.0, 30.0], [4.0, 40.0], [6.0, 60.0]]
    assert cv[0, 0, :3].tolist() == [[-5.0, -59.0], [-7.0, -79.0], [-11.0, -119.0]]


def test_merge_bf16_mean_is_rounded_once_and_singletons_are_bit_exact():
    # members 1.0 and 1.0 + 2^-7 average to the tie 1 + 2^-8 -> rounds to even (1.0)
    K = np.array([[0x3F80], [0x3F81], [0x4049], [0x3F81], [0x3F82]], dtype=np.uint16).reshape(1, 1, 5, 1)
    V = K.copy()
    assign = np.array([0, 0, 2, 3, 3], dtype=np.int32).reshape(1, 1, 5)
    ck, cv, cnt, clen = oracle.merge(K, V, assign)
    assert clen[0, 0] == 3 and cnt[0, 0, :3].tolist() == [2, 1, 2]
    assert ck[0, 0, :3, 0].tolist() == [0x3F80, 0x4049, 0x3F82]  # (1+2^-7 + 1+2^-6)/2 = tie -> 0x3F82
    assert np.array_equal(ck, cv)


def _case(seed, dtype="f32", B=2, Hkv=2, n=120, d=16):
    rng = np.random.default_rng(seed)
    ids = rng.integers(100, 200, size=(B, n)).astype(np.int32)
    ids[rng.random((B, n)) < 0.1] = 13
    cent = rng.normal(size=(B, Hkv, 9, d))
    pick = rng.integers(0, 9, size=(B, Hkv, n))
    K = (np.take_along_axis(cent, pick[..., None], axis=2) + 0.05 * rng.normal(size=(B, Hkv, n, d))).astype(np.float32)
    V = rng.normal(size=(B, Hkv, n, d)).astype(np.float32)
    if dtype == "bf16":
        K, V = _bits(K), _bits(V)
    return ids, K, V


def _dec(a):
    return oracle.bf16_bits_to_f64(a) if a.dtype == np.uint16 else a.astype(np.float64)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_merge_conserves_sums_and_both_routines_agree(dtype):
    ids, K, V = _case(1, dtype)
    B, Hkv, n, d = K.shape
    r = oracle.compress(ids, DELIMS, K, V, 0.7, max_chunk_len=32)
    ck2, cv2, cnt2, clen2 = oracle.merge(K, V, r["assign"])
    for name, other in (("core_k", ck2), ("core_v", cv2), ("count", cnt2), ("core_len", clen2)):
        assert np.array_equal(r[name], other), name
    tol = 1e-6 if dtype == "f32" else 1e-2
    for b in range(B):
        for h in range(Hkv):
            L = r["core_len"][b, h]
            c = r["count"][b, h, :L].astype(np.float64)
            assert c.min() >= 1 and int(c.sum()) == n
            assert np.all(r["count"][b, h, L:] == 0)
            for X, C in ((K, r["core_k"]), (V, r["core_v"])):
                tot = _dec(X[b, h]).sum(axis=0)
                rec = (c[:, None] * _dec(C[b, h, :L])).sum(axis=0)
                assert np.allclose(rec, tot, atol=tol * np.abs(_dec(X[b, h])).sum(axis=0).max())
            # singleton clusters carry their token's bits unchanged, in position order
            a = r["assign"][b, h]
            seeds = np.flatnonzero(a == np.arange(n))
            assert len(seeds) == L
            single = np.flatnonzero(r["count"][b, h, :L] == 1)
            assert np.array_equal(r["core_k"][b, h, single], K[b, h, seeds[single]])
            assert np.array_equal(r["core_v"][b, h, single], V[b, h, seeds[single]])


def test_merge_capacity_clamps_writes_but_reports_needed_length():
    ids, K, V = _case(2)
    full = oracle.compress(ids, DELIMS, K, V, 0.7)
    cap = int(full["core_len"].min()) - 3
    r = oracle.compress(ids, DELIMS, K, V, 0.7, cap=cap)
    assert np.array_equal(r["core_len"], full["core_len"])
    assert np.array_equal(r["core_k"], full["core_k"][:, :, :cap])
    assert np.array_equal(r["count"], full["count"][:, :, :cap])


# -------------------------------------------------------------------- Eq. 4


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_no_merge_threshold_reduces_to_textbook_attention(dtype):
    ids, K, V = _case(3, dtype, Hkv=2)
    B, Hkv, n, d = K.shape
    G = 3
    rng = np.random.default_rng(30)
    q = rng.normal(size=(B, Hkv * G, d)).astype(np.float32)
    if dtype == "bf16":
        q = _bits(q)
    r = oracle.compress(ids, DELIMS, K, V, 2.0)
    assert np.all(r["core_len"] == n) and np.all(r["count"] == 1)
    got = oracle.attn(q, r["core_k"], r["core_v"], r["count"], r["core_len"])
    want = _textbook_attention(_dec(q), _dec(K), _dec(V), G)
    assert np.allclose(got, want, rtol=0, atol=1e-12)
    # count=None means plain attention as well
    assert np.allclose(oracle.attn(q, r["core_k"], r["core_v"], None, r["core_len"]), want, atol=1e-12)


def test_identical_members_reproduce_uncompressed_attention():
    """Eq. 4's log s term: a core standing for s identical tokens weighs as s tokens."""
    rng = np.random.default_rng(4)
    B, Hkv, G, d, n_proto = 1, 2, 2, 8, 5
    reps = [3, 1, 4, 2, 6]
    protoK = rng.normal(size=(B, Hkv, n_proto, d)).astype(np.float32)
    protoV = rng.normal(size=(B, Hkv, n_proto, d)).astype(np.float32)
    # one chunk: prototypes interleaved so clusters are not contiguous
    order = [0, 1, 2, 0, 3, 2, 4, 4, 2, 0, 4, 3, 4, 2, 4, 4]
    assert [order.count(i) for i in range(n_proto)] == reps
    K = np.ascontiguousarray(protoK[:, :, order])
    V = np.ascontiguousarray(protoV[:, :, order])
    ids = np.full((B, len(order)), 500, dtype=np.int32)
    r = oracle.compress(ids, DELIMS, K, V, 0.999)
    assert np.all(r["core_len"] == n_proto), "test premise: prototypes are not near-parallel"
    assert r["count"][0, 0, :n_proto].tolist() == reps
    q = rng.normal(size=(B, Hkv * G, d)).astype(np.float32)
    got = oracle.attn(q, r["core_k"], r["core_v"], r["count"], r["core_len"])
    want = _textbook_attention(q.astype(np.float64), K.astype(np.float64), V.astype(np.float64), G)
    assert np.allclose(got, want, atol=1e-12)
    # and without the size term the answer is visibly different (the pin bites)
    plain = oracle.attn(q, r["core_k"], r["core_v"], None, r["core_len"])
    assert np.abs(plain - want).max() > 1e-3


def test_attention_closed_form_two_cores():
    # d = 1, q = 1, scale = 1: k = (ln 2, 0), counts (1, 3), v = (10, 20)
    # weights ~ 1*e^{ln 2} = 2 and 3*e^0 = 3  ->  o = (2*10 + 3*20) / 5 = 16
    q = np.array([[[1.0]]], dtype=np.float32)
    ck = np.array([[[[math.log(2.0)], [0.0]]]], dtype=np.float32)
    cv = np.array([[[[10.0], [20.0]]]], dtype=np.float32)
    cnt = np.array([[[1, 3]]], dtype=np.int32)
    out = oracle.attn(q, ck, cv, cnt, np.array([[2]], dtype=np.int32), scale=1.0)
    assert out[0, 0, 0] == pytest.approx(16.0, abs=1e-6)
    # default scale is 1/sqrt(d) = 1 here as well
    assert oracle.attn(q, ck, cv, cnt, np.array([[2]], dtype=np.int32))[0, 0, 0] == pytest.approx(16.0, abs=1e-6)
    # only the first core_len rows take part
    assert oracle.attn(q, ck, cv, cnt, np.array([[1]], dtype=np.int32), scale=1.0)[0, 0, 0] == pytest.approx(10.0)
    # an empty head yields zeros
    assert oracle.attn(q, ck, cv, cnt, np.array([[0]], dtype=np.int32), scale=1.0)[0, 0, 0] == 0.0


def test_attention_scale_gqa_mapping_and_permutation_invariance():
    rng = np.random.default_rng(5)
    B, Hkv, G, d, cap = 2, 3, 4, 16, 40
    ck = rng.normal(size=(B, Hkv, cap, d)).astype(np.float32)
    cv = rng.normal(size=(B, Hkv, cap, d)).astype(np.float32)
    cnt = rng.integers(1, 9, size=(B, Hkv, cap)).astype(np.int32)
    clen = rng.integers(1, cap + 1, size=(B, Hkv)).astype(np.int32)
    q = rng.normal(size=(B, Hkv * G, d)).astype(np.float32)
    got = oracle.attn(q, ck, cv, cnt, clen)
    # expand every core into `count` copies and run textbook attention per (b, head)
    for b in range(B):
        for hq in range(Hkv * G):
            h = hq // G
            L = clen[b, h]
            Kx = np.repeat(ck[b, h, :L].astype(np.float64), cnt[b, h, :L], axis=0)
            Vx = np.repeat(cv[b, h, :L].astype(np.float64), cnt[b, h, :L], axis=0)
            w = softmax(Kx @ q[b, hq].astype(np.float64) / math.sqrt(d))
            assert np.allclose(got[b, hq], w @ Vx, atol=1e-12)
    # shuffling the valid rows of every head leaves the output unchanged
    ck2, cv2, cnt2 = ck.copy(), cv.copy(), cnt.copy()
    for b in range(B):
        for h in range(Hkv):
            p = rng.permutation(clen[b, h])
            ck2[b, h, :clen[b, h]] = ck[b, h, p]
            cv2[b, h, :clen[b, h]] = cv[b, h, p]
            cnt2[b, h, :clen[b, h]] = cnt[b, h, p]
    assert np.allclose(oracle.attn(q, ck2, cv2, cnt2, clen), got, atol=1e-12)
    # large logits do not overflow (max-subtracted softmax)
    big = oracle.attn(q * 300, ck, cv, cnt, clen)
    assert np.all(np.isfinite(big))

"""Pins for the oracle's chunking (Eq. 1) and GSC (Eq. 2, Algorithm 1).

None of these re-type the oracle's loops: they use hand-worked fixtures, closed-form
cosines of planar angles, brute force over all subsets, and structural invariants.
"""
import itertools
import math
import os

import numpy as np
import pytest

import oracle

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")
DELIMS = (13, 29889, 29892)


def _rows(name):
    with open(os.path.join(GOLDEN, name)) as f:
        for line in f:
            line = line.strip()
            if line and not line.startswith("#"):
                yield [part.split() for part in line.split(";")]


# ------------------------------------------------------------------ chunking


@pytest.mark.parametrize("row", list(_rows("chunk_cases.txt")))
def test_chunk_hand_worked(row):
    ids, max_len, expect = row
    ids = np.array([[int(x) for x in ids]], dtype=np.int32)
    seg_off, seq_seg_off = oracle.chunk(ids, DELIMS, int(max_len[0]))
    assert seg_off.tolist() == [int(x) for x in expect]
    assert seq_seg_off.tolist() == [0, len(expect) - 1]


def _check_chunk_properties(ids, seg_off, seq_seg_off, max_len):
    B, n = ids.shape
    isd = np.isin(ids, DELIMS).reshape(-1)
    assert seg_off[0] == 0 and seg_off[-1] == B * n
    assert np.all(np.diff(seg_off) >= 1), "segments tile the axis, none empty"
    assert seq_seg_off[0] == 0 and seq_seg_off[-1] == len(seg_off) - 1
    for b in range(B):
        assert seg_off[seq_seg_off[b]] == b * n, "no segment spans two sequences"
    for s in range(len(seg_off) - 1):
        a, e = seg_off[s], seg_off[s + 1]
        if isd[a]:
            assert e - a == 1, "a delimiter is alone in its segment"
            continue
        assert not isd[a:e].any(), "no delimiter inside a chunk"
        assert e - a <= max_len
        at_seq_start = a % n == 0
        # the chunk opens a run (left neighbour is a delimiter / sequence start) or follows a cut
        if not (at_seq_start or isd[a - 1]):
            prev = seg_off[s] - seg_off[s - 1]
            assert prev == max_len and not isd[a - 1]
        at_seq_end = e % n == 0
        if not (at_seq_end or isd[e]):
            assert e - a == max_len, "a chunk ends early only at a hard cut"


@pytest.mark.parametrize("seed", range(6))
def test_chunk_properties_random(seed):
    rng = np.random.default_rng(seed)
    B, n = int(rng.integers(1, 4)), int(rng.integers(1, 400))
    p_delim = [0.0, 0.05, 0.3, 0.9, 1.0, 0.1][seed]
    ids = rng.integers(100, 200, size=(B, n)).astype(np.int32)
    mask = rng.random((B, n)) < p_delim
    ids[mask] = rng.choice(DELIMS, size=int(mask.sum()))
    max_len = [256, 256, 4, 7, 3, 1][seed]
    seg_off, seq_seg_off = oracle.chunk(ids, DELIMS, max_len)
    _check_chunk_properties(ids, seg_off, seq_seg_off, max_len)


def test_chunk_batch_equals_per_sequence():
    rng = np.random.default_rng(11)
    ids = rng.integers(0, 40, size=(3, 97)).astype(np.int32)
    ids[rng.random(ids.shape) < 0.2] = 13
    seg_off, seq_seg_off = oracle.chunk(ids, DELIMS, 5)
    for b in range(3):
        so, _ = oracle.chunk(ids[b:b + 1], DELIMS, 5)
        got = seg_off[seq_seg_off[b]:seq_seg_off[b + 1] + 1] - b * 97
        assert got.tolist() == so.tolist()


# --------------------------------------------------------------------- Eq. 2


def _planar_keys(angles_deg, d=8, radius=None, dtype=np.float32):
    a = np.deg2rad(np.asarray(angles_deg, dtype=np.float64))
    r = np.ones_like(a) if radius is None else np.asarray(radius, dtype=np.float64)
    K = np.zeros((len(a), d), dtype=np.float64)
    K[:, 2] = r * np.cos(a)   # put the plane on axes 2 and 5: catches a dropped component
    K[:, 5] = r * np.sin(a)
    return K.astype(dtype)


def test_sim_is_cosine_of_angle_and_scale_invariant():
    angles = [0, 30, 45, 60, 90, 120, 180, 275]
    K = _planar_keys(angles, radius=[1, 2, 0.5, 3, 1, 7, 0.25, 4])
    for i, j in itertools.combinations(range(len(angles)), 2):
        want = math.cos(math.radians(angles[i] - angles[j]))
        assert oracle.sim(K, i, j) == pytest.approx(want, abs=2e-7)
        assert oracle.sim(K, j, i) == pytest.approx(want, abs=2e-7)


def test_sim_zero_norm_is_zero_and_bf16_bits_are_decoded():
    K = np.zeros((2, 4), dtype=np.float32)
    K[1] = [1, 2, 3, 4]
    assert oracle.sim(K, 0, 1) == 0.0
    # bf16 bits: 0x3f80 = 1.0, 0x4000 = 2.0, 0xbf80 = -1.0
    Kb = np.array([[0x3f80, 0x0000, 0x4000, 0x0000], [0x3f80, 0x4000, 0x0000, 0xbf80]], dtype=np.uint16)
    # rows (1,0,2,0) and (1,2,0,-1): dot 1, norms sqrt5, sqrt6
    assert oracle.sim(Kb, 0, 1) == pytest.approx(1.0 / math.sqrt(30.0), abs=1e-15)


# --------------------------------------------------------------- Algorithm 1


def _gsc_one_chunk(K2d, tau):
    l = K2d.shape[0]
    K = np.ascontiguousarray(K2d).reshape(1, 1, l, -1)
    assign, margin = oracle.gsc(K, np.array([0, l], dtype=np.int32), np.array([0, 1], dtype=np.int32), tau)
    return assign[0, 0], margin


@pytest.mark.parametrize("row", list(_rows("gsc_angle_cases.txt")))
def test_gsc_hand_worked(row):
    angles, tau_deg, expect = row
    K = _planar_keys([float(x) for x in angles], d=16)
    assign, _ = _gsc_one_chunk(K, math.cos(math.radians(float(tau_deg[0]))))
    assert assign.tolist() == [int(x) for x in expect]


def test_gsc_threshold_is_strict():
    K = np.zeros((3, 4), dtype=np.float32)
    K[:, 1] = 1.0  # three identical unit keys: Sim is exactly 1.0
    assert _gsc_one_chunk(K, 1.0)[0].tolist() == [0, 1, 2]      # 1.0 > 1.0 is false
    assert _gsc_one_chunk(K, float(np.nextafter(np.float32(1.0), np.float32(0.0))))[0].tolist() == [0, 0, 0]
    # orthogonal keys have Sim exactly 0: tau = 0 does not merge, tau < 0 does
    E = np.eye(3, 4, dtype=np.float32)
    assert _gsc_one_chunk(E, 0.0)[0].tolist() == [0, 1, 2]
    assert _gsc_one_chunk(E, -1e-6)[0].tolist() == [0, 0, 0]


def _brute_force_lfmis(adj):
    """Seeds = lexicographically first maximal independent set; members -> lowest adjacent seed."""
    l = adj.shape[0]
    best = None
    for bits in range(1 << l):
        S = [i for i in range(l) if bits >> i & 1]
        if any(adj[a, b] for a, b in itertools.combinations(S, 2)):
            continue  # not independent
        if any(not any(adj[i, s] for s in S) for i in range(l) if i not in S):
            continue  # not maximal
        key = tuple(S)
        if best is None or key < best:
            best = key
    assign = []
    for i in range(l):
        assign.append(i if i in best else min(s for s in best if adj[i, s]))
    return assign


@pytest.mark.parametrize("seed", range(12))
def test_gsc_equals_first_maximal_independent_set(seed):
    rng = np.random.default_rng(100 + seed)
    l, d = int(rng.integers(2, 11)), int(rng.integers(2, 5))
    K = rng.normal(size=(l, d)).astype(np.float32)
    tau = float(rng.choice([0.2, 0.5, 0.7, 0.9]))
    Kd = K.astype(np.float64)
    Kn = Kd / np.linalg.norm(Kd, axis=1, keepdims=True)
    C = Kn @ Kn.T
    assert np.abs(C - tau)[~np.eye(l, dtype=bool)].min() > 1e-9
    adj = (C > tau) & ~np.eye(l, dtype=bool)
    # a non-seed may be adjacent to a LATER seed only; "lowest adjacent seed" must also be earlier
    got, _ = _gsc_one_chunk(K, tau)
    assert got.tolist() == _brute_force_lfmis(adj)


def _random_case(seed, dtype):
    rng = np.random.default_rng(seed)
    B, Hkv, n, d = 2, 3, 160, 16
    ids = rng.integers(100, 200, size=(B, n)).astype(np.int32)
    ids[rng.random((B, n)) < 0.12] = 29889
    cent = rng.normal(size=(B, Hkv, 12, d))
    pick = rng.integers(0, 12, size=(B, Hkv, n))
    K = np.take_along_axis(cent, pick[..., None], axis=2) + 0.05 * rng.normal(size=(B, Hkv, n, d))
    K = K.astype(np.float32)
    if dtype == "bf16":
        import torch
        K = torch.from_numpy(K).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    return ids, K


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("tau", [0.3, 0.7, 0.9])
def test_gsc_partition_invariants(dtype, tau):
    ids, K = _random_case(5, dtype)
    B, Hkv, n, _ = K.shape
    seg_off, seq_seg_off = oracle.chunk(ids, DELIMS, 16)
    assign, margin = oracle.gsc(K, seg_off, seq_seg_off, tau)
    assert margin > 0
    seg_of = np.repeat(np.arange(len(seg_off) - 1), np.diff(seg_off)).reshape(B, n)
    for b in range(B):
        for h in range(Hkv):
            a = assign[b, h]
            assert np.all(a >= 0) and np.all(a <= np.arange(n)), "seed index <= member index"
            assert np.all(a[a] == a), "a seed is its own seed; members point at seeds only"
            assert np.all(seg_of[b][a] == seg_of[b]), "no cluster crosses a segment"
            # counts per segment sum to the segment length
            seeds = np.flatnonzero(a == np.arange(n))
            sizes = np.bincount(a, minlength=n)[seeds]
            per_seg = np.bincount(seg_of[b][seeds] - seg_of[b][0], weights=sizes,
                                  minlength=seq_seg_off[b + 1] - seq_seg_off[b])
            want = np.diff(seg_off)[seq_seg_off[b]:seq_seg_off[b + 1]]
            assert per_seg.astype(int).tolist() == want.tolist()
            # delimiters stay alone
            isd = np.isin(ids[b], DELIMS)
            assert np.all(a[isd] == np.flatnonzero(isd))
            assert np.all(np.bincount(a, minlength=n)[isd] == 1)


def test_gsc_threshold_extremes_and_identical_keys():
    ids, K = _random_case(6, "f32")
    B, Hkv, n, _ = K.shape
    seg_off, seq_seg_off = oracle.chunk(ids, DELIMS, 256)
    a_hi, _ = oracle.gsc(K, seg_off, seq_seg_off, 2.0)
    assert np.all(a_hi == np.arange(n)), "tau >= 1 forbids every merge"
    a_lo, _ = oracle.gsc(K, seg_off, seq_seg_off, -2.0)
    first = np.repeat(seg_off[:-1], np.diff(seg_off)).reshape(B, n) - (np.arange(B) * n)[:, None]
    assert np.all(a_lo == first[:, None, :]), "tau < -1 merges each segment into one cluster"
    Ksame = np.broadcast_to(K[:, :, :1, :], K.shape).copy()
    a_same, _ = oracle.gsc(Ksame, seg_off, seq_seg_off, 0.99)
    assert np.all(a_same == first[:, None, :])


def test_gsc_lower_tau_compresses_more_on_clustered_keys():
    ids, K = _random_case(7, "f32")
    seg_off, seq_seg_off = oracle.chunk(ids, DELIMS, 256)
    n = K.shape[2]
    kept = [np.mean(oracle.gsc(K, seg_off, seq_seg_off, t)[0] == np.arange(n)) for t in (0.5, 0.9, 0.999)]
    assert kept[0] <= kept[1] <= kept[2] and kept[0] < kept[2]


def test_gsc_honours_strides():
    ids, K = _random_case(8, "f32")
    seg_off, seq_seg_off = oracle.chunk(ids, DELIMS, 256)
    base, _ = oracle.gsc(K, seg_off, seq_seg_off, 0.7)
    Kt = np.ascontiguousarray(K.transpose(0, 2, 1, 3)).transpose(0, 2, 1, 3)  # [B,n,Hkv,d] storage
    assert not Kt.flags["C_CONTIGUOUS"]
    got, _ = oracle.gsc(Kt, seg_off, seq_seg_off, 0.7)
    assert np.array_equal(base, got)

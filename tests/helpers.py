"""Shared pieces of the GPU parity tests: run both sides on the same bytes and compare."""
import numpy as np
import torch

import oracle
from paper_2603_14303_b200 import binding, synth

# Floating-point acceptance: |gpu - ref| <= tol * max(|ref|, rms(ref vector)) element by element
# (relative error with the vector's RMS as the floor for near-zero elements), tol = 1e-2 for bf16
# storage and 1e-5 for fp32.  Integer products (offsets, assignments, counts, lengths): bit-exact.
TOL = {torch.bfloat16: 1e-2, torch.float32: 1e-5}


def decode_bits(a: np.ndarray) -> np.ndarray:
    return oracle.bf16_bits_to_f64(a) if a.dtype == np.uint16 else a.astype(np.float64)


def to_f64(t: torch.Tensor) -> np.ndarray:
    return t.detach().cpu().to(torch.float64).numpy()


def assert_close_vectors(got: np.ndarray, ref: np.ndarray, tol: float, what: str):
    """got, ref: [..., d] float64."""
    assert got.shape == ref.shape, (what, got.shape, ref.shape)
    if got.size == 0:
        return
    rms = np.sqrt((ref ** 2).mean(axis=-1, keepdims=True))
    floor = np.maximum(np.abs(ref), rms)
    err = np.abs(got - ref)
    bad = err > tol * floor + 1e-30
    if bad.any():
        idx = np.unravel_index(np.argmax(err / (floor + 1e-30)), err.shape)
        raise AssertionError(f"{what}: {int(bad.sum())} elements off, worst at {idx}: got {got[idx]} ref {ref[idx]} "
                             f"(rel {err[idx] / floor[idx]:.3e} > {tol})")


def oracle_compress(ids: torch.Tensor, K: torch.Tensor, V: torch.Tensor, delims, tau, max_chunk_len=256, cap=None):
    return oracle.compress(ids.cpu().numpy(), delims, synth.to_numpy_bits(K), synth.to_numpy_bits(V), tau,
                           max_chunk_len, cap)


def compare_plan(plan: binding.ChunkPlan, seg_off: np.ndarray, seq_seg_off: np.ndarray):
    binding.check_status(plan.status, "sc_chunk")
    n_seg = int(plan.n_seg.item())
    assert n_seg == len(seg_off) - 1
    assert np.array_equal(plan.seg_off[: n_seg + 1].cpu().numpy(), seg_off)
    assert np.array_equal(plan.seq_seg_off.cpu().numpy(), seq_seg_off)
    # tiles: greedy packing of whole segments into <= SC_TILE_ROWS tokens, re-derived here
    tile_seg = plan.tile_seg.cpu().numpy()
    cnt = plan.seq_tile_cnt.cpu().numpy()
    for b in range(plan.B):
        s, s1, want = int(seq_seg_off[b]), int(seq_seg_off[b + 1]), []
        while s < s1:
            want.append(s)
            e = s + 1
            while e < s1 and seg_off[e + 1] - seg_off[s] <= binding.SC_TILE_ROWS:
                e += 1
            s = e
        want.append(s1)
        assert cnt[b] == len(want) - 1
        assert tile_seg[b, : len(want)].tolist() == want


def compare_compressed(got: binding.CompressedLayer, ref: dict, dtype, check_assign=True):
    tol = TOL[dtype]
    core_len = got.core_len.cpu().numpy()
    assert np.array_equal(core_len, ref["core_len"]), "core_len"
    if check_assign and got.assign is not None:
        assert np.array_equal(got.assign.cpu().numpy(), ref["assign"]), "assign"
    B, Hkv = core_len.shape
    cap = got.core_k.shape[2]
    cnt = got.count.cpu().numpy()
    gk, gv = to_f64(got.core_k), to_f64(got.core_v)
    for b in range(B):
        for h in range(Hkv):
            L = min(int(core_len[b, h]), cap)
            assert np.array_equal(cnt[b, h, :L], ref["count"][b, h, :L]), f"count[{b},{h}]"
            assert_close_vectors(gk[b, h, :L], decode_bits(ref["core_k"][b, h, :L]), tol, f"core_k[{b},{h}]")
            assert_close_vectors(gv[b, h, :L], decode_bits(ref["core_v"][b, h, :L]), tol, f"core_v[{b},{h}]")
            # singleton cores are exact copies
            single = np.flatnonzero(ref["count"][b, h, :L] == 1)
            assert np.array_equal(gk[b, h, single], decode_bits(ref["core_k"][b, h, single]))


def layer_from_oracle(ref: dict, dtype, device) -> binding.CompressedLayer:
    def dev(a):
        if a.dtype == np.uint16:
            return torch.from_numpy(a.view(np.int16)).view(torch.bfloat16).to(device)
        return torch.from_numpy(a).to(device)
    return binding.CompressedLayer(dev(ref["core_k"]), dev(ref["core_v"]), dev(ref["count"]), dev(ref["core_len"]))


def assert_valid_run_of_algorithm1(assign: np.ndarray, Kb: np.ndarray, seg_off, tau: float, clear: float = 1e-5):
    """Where similarities come within rounding of tau, fp32 (GPU) and fp64 (oracle) may decide differently
    and both partitions are valid runs of Algorithm 1.  What is unique is checked exactly: replaying
    Algorithm 1 along the given partition (assign[b, h, t] = seed position), every comparison whose
    similarity is clear of tau by `clear` must have been decided as Eq. 2 says, the lowest unassigned token
    of a chunk must be a seed, and every token must end up assigned.  seg_off is over the flattened [B*n] axis."""
    B, Hkv, n = assign.shape
    for s in range(len(seg_off) - 1):
        a, e = int(seg_off[s]), int(seg_off[s + 1])
        b, a, e = a // n, a - (a // n) * n, e - (a // n) * n
        for h in range(Hkv):
            taken = np.zeros(e - a, dtype=bool)
            for i in range(a, e):
                if taken[i - a]:
                    continue
                assert assign[b, h, i] == i, "the lowest unassigned token must be a seed"
                taken[i - a] = True
                for j in range(i + 1, e):
                    if taken[j - a]:
                        continue
                    joined = assign[b, h, j] == i
                    sim = oracle.sim(Kb[b, h], i, j)
                    if abs(sim - tau) > clear:
                        assert joined == (sim > tau), (b, h, i, j, sim)
                    taken[j - a] |= joined
            assert taken.all()

"""GPU parity: every product of the CUDA path against the CPU oracle on the same seeded bytes.

All calls go through the C-ABI library (via the ctypes binding).  Offsets, assignments, counts
and lengths are compared bit-exactly; merged K/V and attention outputs with the tolerance in
helpers.py.
"""
import os

import numpy as np
import pytest
import torch

import oracle
from helpers import (TOL, assert_close_vectors, compare_compressed, compare_plan, layer_from_oracle,
                     oracle_compress, to_f64)
from paper_2603_14303_b200 import binding, synth

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
DELIMS = synth.DELIMS
GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


# ---------------------------------------------------------------------------------- sc_chunk


def _chunk_both(ids_np, max_len):
    ids = torch.from_numpy(ids_np).to(DEV)
    plan = binding.chunk(ids, DELIMS, max_len)
    seg_off, seq_seg_off = oracle.chunk(ids_np, DELIMS, max_len)
    compare_plan(plan, seg_off, seq_seg_off)
    return plan


def test_chunk_hand_worked_cases():
    for line in open(os.path.join(GOLDEN, "chunk_cases.txt")):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        ids, max_len, expect = [p.split() for p in line.split(";")]
        plan = _chunk_both(np.array([[int(x) for x in ids]], dtype=np.int32), int(max_len[0]))
        n_seg = int(plan.n_seg.item())
        assert plan.seg_off[: n_seg + 1].tolist() == [int(x) for x in expect]


@pytest.mark.parametrize("B,n,p_delim,max_len", [
    (1, 1, 0.0, 256), (1, 1, 1.0, 256), (1, 2047, 0.05, 256), (1, 2048, 0.05, 256), (2, 2049, 0.05, 256),
    (3, 5000, 0.0, 256), (3, 5000, 1.0, 256), (2, 6000, 0.0, 7), (2, 4500, 0.3, 3), (1, 10000, 0.002, 100),
    (4, 4096, 0.04, 1), (1, 70000, 0.045, 256), (1, 9000, 0.0005, 256)])
def test_chunk_matches_oracle(B, n, p_delim, max_len):
    rng = np.random.default_rng(B * 1000 + n)
    ids = rng.integers(100, 30000, size=(B, n)).astype(np.int32)
    mask = rng.random((B, n)) < p_delim
    ids[mask] = rng.choice(DELIMS, size=int(mask.sum()))
    _chunk_both(ids, max_len)


def test_chunk_empty_input_and_capacity_error():
    ids = torch.zeros((2, 0), dtype=torch.int32, device=DEV)
    plan = binding.chunk(ids, DELIMS, 256)
    assert int(plan.n_seg.item()) == 0 and plan.seq_seg_off.tolist() == [0, 0, 0] and plan.seq_tile_cnt.tolist() == [0, 0]
    # too-small segment capacity: status says so, n_seg still reports the need, nothing out of bounds
    ids_np = np.full((1, 300), 13, dtype=np.int32)
    t = torch.from_numpy(ids_np).to(DEV)
    i32 = dict(dtype=torch.int32, device=DEV)
    canary = 0x5A5A5A5A
    seg_off = torch.full((100 + 1 + 8,), canary, **i32)
    tile_seg = torch.full((1, 7 + 8), canary, **i32)
    st = torch.zeros(1, **i32)
    ws = torch.empty(binding.lib().sc_chunk_workspace_bytes(1, 300), dtype=torch.uint8, device=DEV)
    n_seg, sso, stc = torch.zeros(1, **i32), torch.zeros(2, **i32), torch.zeros(1, **i32)
    binding.sc_chunk(t, DELIMS, 256, seg_off[:101], sso, n_seg, tile_seg[:, :7], stc, ws, st)
    assert int(st.item()) == binding.SC_ERR_CAPACITY and int(n_seg.item()) == 300
    assert torch.all(seg_off[101:] == canary) and torch.all(tile_seg[:, 7:] == canary)
    assert seg_off[:100].tolist() == list(range(100))


# ------------------------------------------------------------------------------- sc_compress


def _compress_both(w, layer=0, flags=0, cap=None, strided=False, tau=None):
    tau = w.tau if tau is None else tau
    ids, run_id, run_lens = synth.token_ids(w)
    K, V = synth.layer_kv(w, layer, run_id, run_lens)          # CPU bytes, shared by both sides
    ref = oracle_compress(ids, K, V, w.delims, tau, w.max_chunk_len, cap)
    Kd, Vd = K.to(DEV), V.to(DEV)
    if strided:  # [B, n, Hkv, d] storage viewed as [B, Hkv, n, d]
        Kd = Kd.transpose(1, 2).contiguous().transpose(1, 2)
        Vd = Vd.transpose(1, 2).contiguous().transpose(1, 2)
    plan = binding.chunk(ids.to(DEV), w.delims, w.max_chunk_len)
    got = binding.compress(Kd, Vd, plan, tau, cap=cap, want_assign=True, flags=flags)
    return ref, got, plan, (K, V)


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
@pytest.mark.parametrize("flags", [0, binding.SC_FLAG_GENERIC, binding.SC_FLAG_TWO_PASS])
def test_compress_cfg0_matches_oracle(dtype, flags):
    w = synth.config(0, dtype=dtype)
    ref, got, plan, _ = _compress_both(w, flags=flags)
    assert ref["margin"] > 1e-3
    binding.check_status(plan.status)
    compare_compressed(got, ref, torch.bfloat16 if dtype == "bf16" else torch.float32)
    kept = ref["core_len"].sum() / (w.Hkv * w.n)
    assert 0.1 < kept < 0.5


@pytest.mark.parametrize("flags", [0, binding.SC_FLAG_GENERIC, binding.SC_FLAG_TWO_PASS])
@pytest.mark.parametrize("length", [1, 2, 31, 32, 33, 47, 48, 49, 63, 64, 65, 127, 128, 129, 200, 255, 256])
def test_compress_fixed_chunk_lengths(length, flags):
    w = synth.config(0, n=3000, Hkv=2, Hq=8, gap=("fixed", length), centroids=("uniform", 5), seed=length)
    ref, got, plan, _ = _compress_both(w, flags=flags)
    assert ref["margin"] > 1e-4
    binding.check_status(plan.status)
    compare_compressed(got, ref, torch.bfloat16)


@pytest.mark.parametrize("flags", [0, binding.SC_FLAG_GENERIC])
def test_compress_ragged_lognormal_batch(flags):
    w = synth.config(2, B=3, n=5000, Hkv=2, Hq=8, L=1)
    ref, got, plan, _ = _compress_both(w, flags=flags)
    assert ref["margin"] > 1e-4
    compare_compressed(got, ref, torch.bfloat16)


@pytest.mark.parametrize("flags", [0, binding.SC_FLAG_GENERIC])
@pytest.mark.parametrize("max_len", [256, 16, 5])
def test_compress_hard_cut_and_no_delimiters(flags, max_len):
    w = synth.config(0, n=1500, Hkv=2, Hq=8, gap=("fixed", 100000), max_chunk_len=max_len, centroids=("uniform", 3))
    ref, got, plan, _ = _compress_both(w, flags=flags)
    compare_compressed(got, ref, torch.bfloat16)


@pytest.mark.parametrize("flags", [0, binding.SC_FLAG_GENERIC])
def test_compress_threshold_extremes(flags):
    w = synth.config(0, n=1024, Hkv=2, Hq=8)
    for tau in (2.0, -2.0, 1.0):
        ref, got, plan, (K, V) = _compress_both(w, flags=flags, tau=tau)
        compare_compressed(got, ref, torch.bfloat16)
        if tau >= 1.0:  # nothing merges: the compressed cache is the cache, bit for bit
            assert torch.equal(got.core_k.cpu(), K) and torch.equal(got.core_v.cpu(), V)
            assert torch.all(got.count == 1) and torch.all(got.core_len == w.n)


@pytest.mark.parametrize("flags", [0, binding.SC_FLAG_GENERIC])
def test_compress_all_identical_and_zero_keys(flags):
    w = synth.config(0, n=700, Hkv=2, Hq=8)
    ids, run_id, run_lens = synth.token_ids(w)
    K, V = synth.layer_kv(w, 0, run_id, run_lens)
    K[:, 0] = K[:, 0, :1]            # head 0: every key identical -> one cluster per segment
    K[:, 1, 100:140] = 0             # head 1: a stretch of zero-norm keys (Sim := 0 < tau)
    ref = oracle_compress(ids, K, V, w.delims, 0.7)
    plan = binding.chunk(ids.to(DEV), w.delims)
    got = binding.compress(K.to(DEV), V.to(DEV), plan, 0.7, want_assign=True, flags=flags)
    compare_compressed(got, ref, torch.bfloat16)
    n_seg = int(plan.n_seg.item())
    assert int(got.core_len[0, 0]) == n_seg
    # zero keys with a negative threshold: Sim = 0 > tau merges them
    ref = oracle_compress(ids, K, V, w.delims, -0.5)
    got = binding.compress(K.to(DEV), V.to(DEV), plan, -0.5, want_assign=True, flags=flags)
    compare_compressed(got, ref, torch.bfloat16)


@pytest.mark.parametrize("flags", [0, binding.SC_FLAG_GENERIC])
def test_compress_strided_layout_and_determinism(flags):
    w = synth.config(0, n=2048, B=2)
    ref, got, plan, (K, V) = _compress_both(w, flags=flags, strided=True)
    compare_compressed(got, ref, torch.bfloat16)
    again = binding.compress(K.to(DEV), V.to(DEV), plan, w.tau, want_assign=True, flags=flags)
    L = got.core_len.cpu().numpy()
    assert torch.equal(again.core_len, got.core_len) and torch.equal(again.assign, got.assign)
    for b in range(w.B):
        for h in range(w.Hkv):
            assert torch.equal(again.core_k[b, h, : L[b, h]], got.core_k[b, h, : L[b, h]])
            assert torch.equal(again.core_v[b, h, : L[b, h]], got.core_v[b, h, : L[b, h]])
            assert torch.equal(again.count[b, h, : L[b, h]], got.count[b, h, : L[b, h]])


@pytest.mark.parametrize("flags", [0, binding.SC_FLAG_GENERIC])
def test_compress_capacity_overflow_is_reported_not_written(flags):
    w = synth.config(0, n=1024, Hkv=2, Hq=8)
    ids, run_id, run_lens = synth.token_ids(w)
    K, V = synth.layer_kv(w, 0, run_id, run_lens)
    full = oracle_compress(ids, K, V, w.delims, w.tau)
    cap = int(full["core_len"].min()) - 5
    plan = binding.chunk(ids.to(DEV), w.delims)
    canary = 12345
    # carve the [1, 2, cap, *] outputs out of larger buffers whose tails hold a canary
    flat_k = torch.full((2 * cap * 128 + 4096,), 7.0, dtype=torch.bfloat16, device=DEV)
    flat_v = torch.full((2 * cap * 128 + 4096,), 7.0, dtype=torch.bfloat16, device=DEV)
    flat_c = torch.full((2 * cap + 4096,), canary, dtype=torch.int32, device=DEV)
    view = binding.CompressedLayer(flat_k[: 2 * cap * 128].view(1, 2, cap, 128), flat_v[: 2 * cap * 128].view(1, 2, cap, 128),
                                   flat_c[: 2 * cap].view(1, 2, cap), torch.zeros((1, 2), dtype=torch.int32, device=DEV))
    binding.compress(K.to(DEV), V.to(DEV), plan, w.tau, cap=cap, out=view, flags=flags)
    assert int(plan.status.item()) == binding.SC_ERR_CAPACITY
    assert np.array_equal(view.core_len.cpu().numpy(), full["core_len"])
    assert np.array_equal(view.count.cpu().numpy(), full["count"][:, :, :cap])
    assert torch.all(flat_c[2 * cap:] == canary)
    assert torch.all(flat_k[2 * cap * 128:] == 7.0) and torch.all(flat_v[2 * cap * 128:] == 7.0)
    # head 0 overflowed too: its surplus rows must not have spilled into head 1's first rows
    ref_cap = oracle_compress(ids, K, V, w.delims, w.tau, cap=cap)
    compare_compressed(view, ref_cap, torch.bfloat16)


@pytest.mark.parametrize("cfg,kw", [(1, {}), (2, {}), (3, dict(tau=0.9, sigma=0.15)), (4, dict(B=1, gap=("poisson", 128.0))),
                                    (4, dict(B=2, n=32768, gap=("poisson", 8.0), centroids=("ratio", 2.0)))])
def test_compress_full_size_layer_of_the_benchmark_shapes(cfg, kw):
    """One whole layer at the benchmark's sizes (every block walks many tiles; cfg4 with mean chunk
    length 128 is mostly tiles longer than SC_TILE_ROWS), compared in full with the oracle."""
    w = synth.config(cfg, L=1, **kw)
    ref, got, plan, _ = _compress_both(w, layer=0)
    binding.check_status(plan.status)
    assert ref["margin"] > 1e-4
    compare_compressed(got, ref, torch.bfloat16)


def test_compress_near_ties_are_decided_consistently():
    """Noise 0.3 at tau = 0.9 puts similarities on both sides of the threshold, some within rounding of
    it, where fp32 (GPU) and fp64 (oracle) may decide differently and both partitions are valid runs of
    Algorithm 1.  What is unique is checked exactly: replaying Algorithm 1 along the GPU's partition,
    every comparison whose similarity is clear of tau (by 1e-5) must have been decided as Eq. 2 says;
    the merged cores must then equal Eq. 3 applied to the GPU's own partition."""
    w = synth.config(3, L=1, n=8192, Hkv=2, Hq=14, tau=0.9, sigma=0.3)
    ids, run_id, run_lens = synth.token_ids(w)
    K, V = synth.layer_kv(w, 0, run_id, run_lens)
    Kb, Vb = synth.to_numpy_bits(K), synth.to_numpy_bits(V)
    seg_off, seq_seg_off = oracle.chunk(ids.numpy(), w.delims, w.max_chunk_len)
    assert oracle.gsc(Kb, seg_off, seq_seg_off, w.tau)[1] < 1e-4      # the oracle does meet near-ties here
    plan = binding.chunk(ids.to(DEV), w.delims, w.max_chunk_len)
    got = binding.compress(K.to(DEV), V.to(DEV), plan, w.tau, want_assign=True)
    binding.check_status(plan.status)
    assign = got.assign.cpu().numpy()
    for h in range(w.Hkv):
        for s in range(len(seg_off) - 1):
            a, e = int(seg_off[s]), int(seg_off[s + 1])
            taken = np.zeros(e - a, dtype=bool)
            for i in range(a, e):
                if taken[i - a]:
                    continue
                assert assign[0, h, i] == i, "the lowest unassigned token must be a seed"
                taken[i - a] = True
                for j in range(i + 1, e):
                    if taken[j - a]:
                        continue
                    joined = assign[0, h, j] == i
                    sim = oracle.sim(Kb[0, h], i, j)
                    if abs(sim - w.tau) > 1e-5:
                        assert joined == (sim > w.tau), (h, i, j, sim)
                    taken[j - a] |= joined
            assert taken.all()
    ck, cv, cnt, clen = oracle.merge(Kb, Vb, assign, None, seg_off, seq_seg_off)
    compare_compressed(got, dict(core_k=ck, core_v=cv, count=cnt, core_len=clen, assign=assign), torch.bfloat16)


@pytest.mark.parametrize("flags", [0, binding.SC_FLAG_GENERIC])
def test_compress_chain_similarity_in_long_segments(flags):
    """Keys built from random sign vectors L_t: k_t = L_t + L_{t+1} is similar to its neighbours in the sequence
    only (cos about 1/2 against about 0), k_t = L_t + L_{t+1} + L_{t+2} to the two on either side.  Along such a
    chain whether a token is a seed depends on the token before it, all the way down the segment: the opposite
    of chunks that are unions of cliques, and the deepest case for any scheme that settles Algorithm 1 for many
    tokens at once.  Segments of 33..256 tokens (several in a tile, alone in a tile, across two 128-row blocks)."""
    rng = np.random.default_rng(77)
    delim, plain = synth.DELIMS[0], max(synth.DELIMS) + 1
    lengths = [200, 256, 40, 100, 33, 129, 64, 20, 255, 128, 90, 37, 5, 161]
    ids = []
    for l in lengths:
        ids += [plain] * l + [delim]
    n, d = len(ids), 128
    ids = torch.tensor([ids], dtype=torch.int32)
    L = rng.choice([-1.0, 1.0], size=(2, n + 2, d))
    K = torch.empty((1, 2, n, d), dtype=torch.bfloat16)
    K[0, 0] = torch.from_numpy(L[0, :n] + L[0, 1:n + 1])                       # entries 0, +-2, +-3: exact in bf16
    K[0, 1] = torch.from_numpy(L[1, :n] + L[1, 1:n + 1] + L[1, 2:n + 2])
    V = torch.empty((1, 2, n, d), dtype=torch.bfloat16)
    V[:] = torch.from_numpy(rng.normal(size=(1, 2, n, d)))
    tau = 0.26
    ref = oracle_compress(ids, K, V, synth.DELIMS, tau)
    assert oracle.gsc(synth.to_numpy_bits(K), *oracle.chunk(ids.numpy(), synth.DELIMS, 256), tau)[1] > 2e-6   # no similarity within fp32 rounding of tau
    # the structure is what the docstring says: about every other token of a plain chain is a seed
    seeds = (ref["assign"][0, 0] == np.arange(n)).sum()
    assert 0.4 * n < seeds < 0.7 * n
    plan = binding.chunk(ids.to(DEV), synth.DELIMS)
    got = binding.compress(K.to(DEV), V.to(DEV), plan, tau, want_assign=True, flags=flags)
    compare_compressed(got, ref, torch.bfloat16)


@pytest.mark.parametrize("n", [1, 5, 31, 33, 130])
def test_compress_tiny_contexts(n):
    """Contexts shorter than a TMA box / a tile, two sequences and heads."""
    w = synth.config(0, B=2, n=n, Hkv=2, Hq=8, gap=("poisson", 6.0), centroids=("uniform", 3), seed=n)
    ref, got, plan, _ = _compress_both(w)
    binding.check_status(plan.status)
    compare_compressed(got, ref, torch.bfloat16)


def test_compress_workspace_is_left_clean_and_can_be_shared_by_consecutive_calls():
    w = synth.config(0, n=6000, L=3, gap=("poisson", 40.0))
    ids, run_id, run_lens = synth.token_ids(w)
    plan = binding.chunk(ids.to(DEV), w.delims)
    ws = binding.compress_workspace(w.B, w.Hkv, w.n, DEV)
    for rep in range(2):
        for layer, flags in enumerate((0, binding.SC_FLAG_GENERIC, binding.SC_FLAG_TWO_PASS, 0)):
            K, V = synth.layer_kv(w, layer % w.L, run_id, run_lens)
            ref = oracle_compress(ids, K, V, w.delims, w.tau)
            got = binding.compress(K.to(DEV), V.to(DEV), plan, w.tau, want_assign=True, workspace=ws, flags=flags)
            binding.check_status(plan.status)
            compare_compressed(got, ref, torch.bfloat16)
            n_words = 64 + w.B * w.Hkv * plan.n_tile_cap
            assert int(ws.view(torch.int32)[:n_words].abs().max()) == 0, "status words and counters are zero again"


def test_compress_overlapped_independent_layer_launches_match_ordinary_ones():
    """SC_FLAG_OVERLAP_PREV on sc_compress: layers with their own K/V, cores, workspace and status, launched
    back to back so that one layer's tail overlaps the next layer's start."""
    w = synth.config(1, n=8192, L=4)
    ids, run_id, run_lens = synth.token_ids(w)
    plan = binding.chunk(ids.to(DEV), w.delims)
    KV = [tuple(x.to(DEV) for x in synth.layer_kv(w, l, run_id, run_lens)) for l in range(w.L)]
    refs = [oracle_compress(ids, KV[l][0].cpu(), KV[l][1].cpu(), w.delims, w.tau) for l in range(w.L)]
    ws = [binding.compress_workspace(w.B, w.Hkv, w.n, DEV) for _ in range(w.L)]
    st = torch.zeros((w.L, 1), dtype=torch.int32, device=DEV)
    outs = [None] * w.L
    torch.cuda.synchronize()
    for rep in range(3):
        for l in range(w.L):
            if outs[l] is None:
                outs[l] = binding.compress(KV[l][0], KV[l][1], plan, w.tau, workspace=ws[l])   # allocates once
                continue
            o = outs[l]
            o.core_k.zero_(); o.core_len.zero_()
        torch.cuda.synchronize()
        for l in range(w.L):
            o = outs[l]
            binding.sc_compress(KV[l][0], KV[l][1], plan, w.tau, o.core_k, o.core_v, o.count, o.core_len, None, ws[l], st[l],
                                binding.SC_FLAG_OVERLAP_PREV if l > 0 else 0)
        torch.cuda.synchronize()
        assert int(st.abs().max()) == 0
        for l in range(w.L):
            compare_compressed(outs[l], refs[l], torch.bfloat16, check_assign=False)
            n_words = 64 + w.B * w.Hkv * plan.n_tile_cap
            assert int(ws[l].view(torch.int32)[:n_words].abs().max()) == 0


def test_compress_bounded_wait_reports_timeout_and_leaves_the_context_usable():
    """The look-back's wait is bounded: if a predecessor never reports (here: the ticket counter starts one
    round in, so the first tile of every head is never processed), the waiting tiles give up after the
    limit, the status word says SC_ERR_TIMEOUT, the kernel ends, and the next call works."""
    w = synth.config(0, n=4096)
    ids, run_id, run_lens = synth.token_ids(w)
    K, V = synth.layer_kv(w, 0, run_id, run_lens)
    plan = binding.chunk(ids.to(DEV), w.delims)
    ws = binding.compress_workspace(w.B, w.Hkv, w.n, DEV)
    ws.view(torch.int32)[0] = w.B * w.Hkv          # first ticket handed out = tile 1 of head 0
    out = binding.compress(K.to(DEV), V.to(DEV), plan, w.tau, workspace=ws)    # allocates the outputs
    torch.cuda.synchronize()
    assert int(plan.status.item()) == binding.SC_ERR_TIMEOUT
    # as the header says: zero the workspace after a timeout, then carry on
    ws.zero_(); plan.status.zero_()
    ref = oracle_compress(ids, K, V, w.delims, w.tau)
    got = binding.compress(K.to(DEV), V.to(DEV), plan, w.tau, workspace=ws, out=out)
    binding.check_status(plan.status)
    compare_compressed(got, ref, torch.bfloat16, check_assign=False)


# ---------------------------------------------------------------------------- sc_decode_attn


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
@pytest.mark.parametrize("flags", [0, binding.SC_FLAG_GENERIC])
def test_decode_cfg0_end_to_end_and_on_oracle_cores(dtype, flags):
    w = synth.config(0, dtype=dtype)
    tdt = torch.bfloat16 if dtype == "bf16" else torch.float32
    ref, got, plan, _ = _compress_both(w)
    ref_layer = layer_from_oracle(ref, tdt, DEV)
    ws = binding.decode_workspace(w.B, w.Hq, w.Hkv, w.d, w.n, DEV)
    for step in range(w.decode_steps):
        q = synth.queries(w, step, 0)
        want = oracle.attn(synth.to_numpy_bits(q), ref["core_k"], ref["core_v"], ref["count"], ref["core_len"])
        out_e2e = binding.decode_attn(q.to(DEV), got, workspace=ws, flags=flags)
        out_iso = binding.decode_attn(q.to(DEV), ref_layer, workspace=ws, flags=flags)
        assert_close_vectors(to_f64(out_iso), want, TOL[tdt], f"decode on oracle cores, step {step}")
        assert_close_vectors(to_f64(out_e2e), want, TOL[tdt], f"decode end to end, step {step}")


@pytest.mark.parametrize("flags", [0, binding.SC_FLAG_GENERIC])
@pytest.mark.parametrize("Hkv,G", [(4, 7), (2, 1), (2, 8), (3, 2)])
def test_decode_gqa_shapes_ragged_lengths_and_plain_attention(Hkv, G, flags):
    rng = np.random.default_rng(Hkv * 10 + G)
    B, d, cap = 3, 128, 1500
    ck = torch.from_numpy(rng.normal(size=(B, Hkv, cap, d)).astype(np.float32)).to(torch.bfloat16)
    cv = torch.from_numpy(rng.normal(size=(B, Hkv, cap, d)).astype(np.float32)).to(torch.bfloat16)
    cnt = torch.from_numpy(rng.integers(1, 40, size=(B, Hkv, cap)).astype(np.int32))
    clen = torch.from_numpy(rng.integers(0, cap + 1, size=(B, Hkv)).astype(np.int32))
    clen[0, 0], clen[1, 0], clen[2, Hkv - 1] = 0, 1, cap           # empty, single row, full
    if Hkv > 1:
        clen[0, 1] = 17
    q = torch.from_numpy(rng.normal(size=(B, Hkv * G, d)).astype(np.float32)).to(torch.bfloat16)
    layer = binding.CompressedLayer(ck.to(DEV), cv.to(DEV), cnt.to(DEV), clen.to(DEV))
    for use_count in (True, False):
        want = oracle.attn(synth.to_numpy_bits(q), synth.to_numpy_bits(ck), synth.to_numpy_bits(cv),
                           cnt.numpy() if use_count else None, clen.numpy())
        out = binding.decode_attn(q.to(DEV), layer, flags=flags, use_count=use_count)
        assert_close_vectors(to_f64(out), want, 1e-2, f"decode G={G} count={use_count}")
        assert torch.all(out[0, :G] == 0), "a head without cores yields zeros"


def test_decode_many_heads_of_very_different_lengths_in_one_launch():
    """A launch of several waves of blocks (many heads, a long capacity): the split count comes from the
    capacity, and each head uses as many of its blocks as its own length warrants -- from none (empty head)
    and one (a few rows) to all of them (a full head); the blocks left over only take their ticket, and any of
    them may be the one that merges.  Two calls in a row on one workspace."""
    rng = np.random.default_rng(4242)
    B, Hkv, G, d, cap = 6, 8, 4, 128, 12000
    g = torch.Generator(device=DEV)
    g.manual_seed(99)
    ck = torch.randn((B, Hkv, cap, d), generator=g, device=DEV).to(torch.bfloat16)
    cv = torch.randn((B, Hkv, cap, d), generator=g, device=DEV).to(torch.bfloat16)
    cnt = torch.randint(1, 40, (B, Hkv, cap), generator=g, device=DEV, dtype=torch.int32)
    clen = torch.from_numpy(rng.integers(0, cap + 1, size=(B, Hkv)).astype(np.int32))
    clen[0, 0], clen[0, 1], clen[0, 2], clen[1, 0], clen[5, 7] = 0, 1, 17, 1025, cap
    clen[2] = torch.tensor([300, 700, 1024, 2048, 2049, 5000, 11999, 64], dtype=torch.int32)
    q = torch.from_numpy(rng.normal(size=(B, Hkv * G, d)).astype(np.float32)).to(torch.bfloat16).to(DEV)
    layer = binding.CompressedLayer(ck, cv, cnt, clen.to(DEV))
    ws = binding.decode_workspace(B, Hkv * G, Hkv, d, cap, DEV)
    want = oracle.attn(synth.to_numpy_bits(q), synth.to_numpy_bits(ck), synth.to_numpy_bits(cv), cnt.cpu().numpy(),
                       clen.numpy())
    first = binding.decode_attn(q, layer, workspace=ws)
    again = binding.decode_attn(q, layer, workspace=ws)
    assert_close_vectors(to_f64(first), want, 1e-2, "decode, heads of very different lengths")
    assert torch.equal(first, again)
    assert torch.all(first[0, :G] == 0), "a head without cores yields zeros"


@pytest.mark.parametrize("flags", [0, binding.SC_FLAG_GENERIC])
def test_decode_is_deterministic_and_scale_is_honoured(flags):
    w = synth.config(0, n=4096)
    ref, got, plan, _ = _compress_both(w)
    q = synth.queries(w, 0, 0).to(DEV)
    ws = binding.decode_workspace(w.B, w.Hq, w.Hkv, w.d, w.n, DEV)
    a = binding.decode_attn(q, got, workspace=ws, flags=flags)
    b = binding.decode_attn(q, got, workspace=ws, flags=flags)
    assert torch.equal(a, b)
    c = binding.decode_attn(q, got, workspace=ws, flags=flags, scale=0.05)
    want = oracle.attn(synth.to_numpy_bits(q), ref["core_k"], ref["core_v"], ref["count"], ref["core_len"], scale=0.05)
    assert_close_vectors(to_f64(c), want, 1e-2, "custom scale")


@pytest.mark.parametrize("cfg", [1, 2, 3, 4])
def test_decode_full_size_layer_in_the_benchmark_launch_shape(cfg):
    """One layer of each benchmark workload at full size, cores compressed on the GPU into buffers of the
    benchmark's capacity (n / 2, which sets the number of splits), three decode steps against the oracle."""
    w = synth.config(cfg, L=1)
    ids, run_id, run_lens = synth.token_ids(w)
    K, V = synth.layer_kv(w, 0, run_id, run_lens)
    ref = oracle_compress(ids, K, V, w.delims, w.tau, w.max_chunk_len, w.n // 2)
    plan = binding.chunk(ids.to(DEV), w.delims, w.max_chunk_len)
    got = binding.compress(K.to(DEV), V.to(DEV), plan, w.tau, cap=w.n // 2)
    binding.check_status(plan.status)
    assert np.array_equal(got.core_len.cpu().numpy(), ref["core_len"])
    ws = binding.decode_workspace(w.B, w.Hq, w.Hkv, w.d, w.n // 2, DEV)
    for step in range(3):
        q = synth.queries(w, step, 0)
        want = oracle.attn(synth.to_numpy_bits(q), ref["core_k"], ref["core_v"], ref["count"], ref["core_len"])
        out = binding.decode_attn(q.to(DEV), got, workspace=ws)
        assert_close_vectors(to_f64(out), want, 1e-2, f"cfg{cfg} step {step}")


def test_no_merge_compress_then_decode_equals_exact_attention():
    """tau >= 1: the whole path must reproduce exact softmax attention over the raw cache."""
    w = synth.config(0, n=1536)
    ref, got, plan, (K, V) = _compress_both(w, tau=2.0)
    q = synth.queries(w, 0, 0)
    out = binding.decode_attn(q.to(DEV), got)
    Kf, Vf, qf = K.double(), V.double(), q.double()
    G = w.G
    for hq in range(w.Hq):
        s = (Kf[0, hq // G] @ qf[0, hq]) / np.sqrt(w.d)
        want = torch.softmax(s, 0) @ Vf[0, hq // G]
        assert_close_vectors(to_f64(out[0, hq]), want.numpy(), 1e-2, f"exact attention head {hq}")


def test_overlapped_independent_layer_launches_match_ordinary_ones():
    """SC_FLAG_OVERLAP_PREV: layers with their own q/out/workspace launched back to back."""
    w = synth.config(0, n=4096, L=4)
    ids, run_id, run_lens = synth.token_ids(w)
    plan = binding.chunk(ids.to(DEV), w.delims)
    layers, refs = [], []
    for l in range(w.L):
        K, V = synth.layer_kv(w, l, run_id, run_lens)
        refs.append(oracle_compress(ids, K, V, w.delims, w.tau))
        layers.append(binding.compress(K.to(DEV), V.to(DEV), plan, w.tau))
    steps = 6
    q = torch.stack([torch.stack([synth.queries(w, s, l) for l in range(w.L)]) for s in range(steps)]).to(DEV)
    plain, fast = torch.empty_like(q), torch.empty_like(q)
    ws = [binding.decode_workspace(w.B, w.Hq, w.Hkv, w.d, w.n, DEV) for _ in range(w.L)]
    st = torch.zeros((w.L, 1), dtype=torch.int32, device=DEV)
    for s in range(steps):
        for l in range(w.L):
            binding.decode_attn(q[s, l], layers[l], out=plain[s, l], workspace=ws[l], status=st[l])
    torch.cuda.synchronize()
    for rep in range(3):
        for s in range(steps):
            for l in range(w.L):
                binding.decode_attn(q[s, l], layers[l], out=fast[s, l], workspace=ws[l], status=st[l],
                                    flags=binding.SC_FLAG_OVERLAP_PREV if l > 0 else 0)
        torch.cuda.synchronize()
        assert torch.equal(plain, fast)
        fast.zero_()
    assert int(st.abs().max()) == 0
    for l in range(w.L):
        want = oracle.attn(synth.to_numpy_bits(q[2, l].cpu()), refs[l]["core_k"], refs[l]["core_v"], refs[l]["count"],
                           refs[l]["core_len"])
        assert_close_vectors(to_f64(plain[2, l]), want, 1e-2, f"layer {l}")
    for x in ws:
        assert int(x.view(torch.int32)[:64].abs().max()) == 0, "arrival counters are left at zero"


def _bf16_bits(x64: np.ndarray) -> np.ndarray:
    """float64 -> bf16 bit patterns (uint16), via torch's round-to-nearest-even conversion."""
    return torch.from_numpy(x64).to(torch.float32).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)


@pytest.mark.parametrize("share_workspace", [False, True])
def test_chained_layer_launches_where_each_query_is_the_previous_output(share_workspace):
    """SC_FLAG_OVERLAP_CHAIN: layer l+1's query IS layer l's output (same shape), the launches go back to
    back.  The chained launches must equal ordinary stream-ordered launches bit for bit, and the oracle run
    as the same chain (its output rounded to bf16 between layers) within the bf16 tolerance.  Along a run
    of overlapped launches every write is ordered behind the preceding kernel's completion, so the calls
    may also share one workspace."""
    w = synth.config(0, n=8192, L=6)
    ids, run_id, run_lens = synth.token_ids(w)
    plan = binding.chunk(ids.to(DEV), w.delims)
    layers, refs = [], []
    for l in range(w.L):
        K, V = synth.layer_kv(w, l, run_id, run_lens)
        refs.append(oracle_compress(ids, K, V, w.delims, w.tau, cap=w.n // 2))
        layers.append(binding.compress(K.to(DEV), V.to(DEV), plan, w.tau, cap=w.n // 2))
    n_ws = 1 if share_workspace else w.L
    ws = [binding.decode_workspace(w.B, w.Hq, w.Hkv, w.d, w.n // 2, DEV) for _ in range(n_ws)]
    st = torch.zeros(1, dtype=torch.int32, device=DEV)
    q0 = (4.0 * synth.queries(w, 0, 0)).to(DEV)     # sharper softmax than N(0,1) queries give
    # x[0] = q0, x[l + 1] = attention of layer l on x[l]
    plain = torch.zeros((w.L + 1, w.B, w.Hq, w.d), dtype=q0.dtype, device=DEV)
    plain[0] = q0
    for l in range(w.L):
        binding.decode_attn(plain[l], layers[l], out=plain[l + 1], workspace=ws[l % n_ws], status=st)
    torch.cuda.synchronize()
    for rep in range(4):
        chain = torch.zeros_like(plain)
        chain[0] = q0
        torch.cuda.synchronize()
        for l in range(w.L):
            binding.decode_attn(chain[l], layers[l], out=chain[l + 1], workspace=ws[l % n_ws], status=st,
                                flags=binding.SC_FLAG_OVERLAP_CHAIN if l > 0 else 0)
        torch.cuda.synchronize()
        assert torch.equal(plain, chain), f"repeat {rep}"
    assert int(st.item()) == 0
    x = synth.to_numpy_bits(q0.cpu())
    for l in range(w.L):
        r = refs[l]
        want = oracle.attn(x, r["core_k"], r["core_v"], r["count"], r["core_len"])
        assert_close_vectors(to_f64(plain[l + 1]), want, 1e-2, f"chain, layer {l}")
        x = _bf16_bits(want)
    for x in ws:
        assert int(x.view(torch.int32)[:64].abs().max()) == 0, "arrival counters are left at zero"


def test_overlapped_launches_two_apart_may_share_a_workspace():
    """Two workspaces used alternately by a run of SC_FLAG_OVERLAP_PREV launches: launch l and launch l+2
    write the same scratch, which is safe because a kernel's writes wait for its predecessor's completion
    and that one waited for its own predecessor."""
    w = synth.config(0, n=4096, L=6)
    ids, run_id, run_lens = synth.token_ids(w)
    plan = binding.chunk(ids.to(DEV), w.delims)
    layers = []
    for l in range(w.L):
        K, V = synth.layer_kv(w, l, run_id, run_lens)
        layers.append(binding.compress(K.to(DEV), V.to(DEV), plan, w.tau))
    q = torch.stack([synth.queries(w, 1, l) for l in range(w.L)]).to(DEV)
    ws = [binding.decode_workspace(w.B, w.Hq, w.Hkv, w.d, w.n, DEV) for _ in range(2)]
    plain, fast = torch.empty_like(q), torch.empty_like(q)
    for l in range(w.L):
        binding.decode_attn(q[l], layers[l], out=plain[l], workspace=ws[l % 2])
    torch.cuda.synchronize()
    for rep in range(5):
        fast.zero_()
        for l in range(w.L):
            binding.decode_attn(q[l], layers[l], out=fast[l], workspace=ws[l % 2],
                                flags=binding.SC_FLAG_OVERLAP_PREV if l > 0 else 0)
        torch.cuda.synchronize()
        assert torch.equal(plain, fast), f"repeat {rep}"


@pytest.mark.parametrize("L,n,flags,dtype", [(5, 3000, 0, "bf16"), (33, 700, 0, "bf16"), (3, 1500, binding.SC_FLAG_GENERIC, "bf16"),
                                             (2, 900, 0, "f32")])
def test_all_layers_in_one_launch_equal_one_launch_per_layer(L, n, flags, dtype):
    """sc_compress_layers: every layer has its own K and V (so it clusters differently), all share the chunk
    plan; the products must equal sc_compress layer by layer, bit for bit, and layer 0 the oracle."""
    w = synth.config(0, n=n, L=L, B=2, Hkv=2, Hq=8, dtype=dtype)
    ids, run_id, run_lens = synth.token_ids(w)
    plan = binding.chunk(ids.to(DEV), w.delims, w.max_chunk_len)
    Ks, Vs, single = [], [], []
    for l in range(L):
        K, V = synth.layer_kv(w, l, run_id, run_lens)
        Ks.append(K.to(DEV)); Vs.append(V.to(DEV))
        single.append(binding.compress(Ks[l], Vs[l], plan, w.tau, want_assign=True, flags=flags))
    i32 = dict(dtype=torch.int32, device=DEV)
    outs = [binding.CompressedLayer(torch.zeros_like(s.core_k), torch.zeros_like(s.core_v), torch.zeros_like(s.count),
                                    torch.zeros_like(s.core_len), torch.full_like(s.assign, -1)) for s in single]
    ws = binding.compress_layers_workspace(L, w.B, w.Hkv, n, DEV)
    for rep in range(2):   # the workspace is left ready for the next call
        binding.sc_compress_layers(Ks, Vs, plan, w.tau, outs, ws, plan.status, flags)
        binding.check_status(plan.status)
        for l in range(L):
            a, b = single[l], outs[l]
            assert torch.equal(a.core_len, b.core_len) and torch.equal(a.assign, b.assign), f"layer {l}"
            for bb in range(w.B):
                for h in range(w.Hkv):
                    m = int(a.core_len[bb, h])
                    assert torch.equal(a.count[bb, h, :m], b.count[bb, h, :m])
                    assert torch.equal(a.core_k[bb, h, :m], b.core_k[bb, h, :m]) and torch.equal(a.core_v[bb, h, :m], b.core_v[bb, h, :m])
    K0, V0 = synth.layer_kv(w, 0, run_id, run_lens)
    compare_compressed(outs[0], oracle_compress(ids, K0, V0, w.delims, w.tau), K0.dtype)
    fused_words = binding.lib().sc_compress_layers_workspace_bytes(L, w.B, w.Hkv, n) - binding.lib().sc_compress_workspace_bytes(w.B, w.Hkv, n)
    assert int(ws[: max(fused_words, 256)].view(torch.int32).abs().max()) == 0, "status words and counters are left at zero"

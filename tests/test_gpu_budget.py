"""sc_compress_budget on the GPU against the oracle's budget search, and the fixed-size chunking mode."""
import numpy as np
import pytest
import torch

import oracle
from helpers import assert_valid_run_of_algorithm1, compare_compressed, compare_plan, oracle_compress
from paper_2603_14303_b200 import binding, synth

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _spread_workload(dtype="bf16", n=3072, B=2):
    # noise large enough that same-centroid similarities straddle the whole grid [0.5, 0.9]: the kept
    # fraction then really depends on the threshold (the benchmark workloads are flat over that range)
    return synth.config(0, n=n, B=B, Hkv=2, Hq=8, sigma=0.6, dtype=dtype)


@pytest.mark.parametrize("dtype,flags", [("bf16", 0), ("bf16", binding.SC_FLAG_GENERIC), ("f32", 0)])
@pytest.mark.parametrize("target", [0.45, 0.6, 0.75])
def test_budget_search_picks_the_oracles_threshold(dtype, flags, target):
    w = _spread_workload(dtype)
    ids, run_id, run_lens = synth.token_ids(w)
    K, V = synth.layer_kv(w, 0, run_id, run_lens)
    Kb, Vb = synth.to_numpy_bits(K), synth.to_numpy_bits(V)
    T = 17
    ref = oracle.budget(ids.numpy(), w.delims, Kb, Vb, target, 0.5, 0.9, T)
    tc = ref["target_cores"]
    # the test is only meaningful if no decision of the search hangs on a handful of near-tie pairs
    assert all(abs(c - tc) > 16 for _, c in ref["visited"]), ref["visited"]
    assert 0 < ref["index"] < T - 1, "the target should fall inside the grid"
    plan = binding.chunk(ids.to(DEV), w.delims, w.max_chunk_len)
    got, tau, search = binding.compress_to_budget(K.to(DEV), V.to(DEV), plan, target, 0.5, 0.9, T, want_assign=True,
                                                  flags=flags)
    binding.check_status(plan.status)
    assert int(search[0]) == ref["index"]
    assert float(tau.item()) == ref["tau"] == float(oracle.tau_grid(0.5, 0.9, T)[ref["index"]])
    assert 3 <= int(search[1]) <= len(ref["visited"])
    # at the chosen threshold: a valid run of Algorithm 1 (similarities do come near tau here), its count
    # within a few near-tie pairs of the oracle's, and Eq. 3 on the GPU's own partition
    assign = got.assign.cpu().numpy()
    seg_off, seq_seg_off = ref["seg_off"], ref["seq_seg_off"]
    assert_valid_run_of_algorithm1(assign, Kb, seg_off, ref["tau"])
    assert abs(int(got.core_len.sum()) - int(ref["core_len"].sum())) <= 4
    ck, cv, cnt, clen = oracle.merge(Kb, Vb, assign, None, seg_off, seq_seg_off)
    compare_compressed(got, dict(core_k=ck, core_v=cv, count=cnt, core_len=clen, assign=assign), K.dtype)


def test_budget_end_cases_and_workspace_reuse():
    """Targets outside what the grid can reach pick its ends after one or two counting passes; the same
    workspace serves call after call (it is left as it was found)."""
    w = _spread_workload(n=2048, B=1)
    ids, run_id, run_lens = synth.token_ids(w)
    K, V = synth.layer_kv(w, 0, run_id, run_lens)
    Kd, Vd = K.to(DEV), V.to(DEV)
    plan = binding.chunk(ids.to(DEV), w.delims, w.max_chunk_len)
    B, Hkv, n, d = K.shape
    ws = torch.zeros(binding.lib().sc_compress_budget_workspace_bytes(B, Hkv, n), dtype=torch.uint8, device=DEV)
    tau = torch.zeros(1, dtype=torch.float32, device=DEV)
    search = torch.zeros(2, dtype=torch.int32, device=DEV)
    out = binding.compress(Kd, Vd, plan, 0.7)      # buffers of the right shape
    # (target, upper end of the grid): nothing to keep -> lowest threshold after one pass; everything to keep
    # but even 0.6 still merges -> highest threshold after two
    for target, tau_hi, want_index, want_passes in ((0.0, 0.9, 0, 1), (1.0, 0.6, 8, 2), (0.0, 0.9, 0, 1)):
        grid = oracle.tau_grid(0.5, tau_hi, 9)
        binding.sc_compress_budget(Kd, Vd, plan, target, 0.5, tau_hi, 9, out.core_k, out.core_v, out.count,
                                   out.core_len, tau, search, ws, status=plan.status)
        binding.check_status(plan.status)
        assert search.tolist() == [want_index, want_passes]
        assert float(tau.item()) == float(grid[want_index])
        ref = oracle_compress(ids, K, V, w.delims, float(grid[want_index]))
        assert abs(int(out.core_len.sum()) - int(ref["core_len"].sum())) <= 4
    # an ordinary sc_compress on the compress part of the same workspace still works afterwards
    again = binding.compress(Kd, Vd, plan, 2.0, workspace=ws[256:])
    assert int(again.core_len.sum()) == Hkv * n


def test_budget_argument_validation():
    w = _spread_workload(n=512, B=1)
    ids, run_id, run_lens = synth.token_ids(w)
    K, V = synth.layer_kv(w, 0, run_id, run_lens)
    Kd, Vd = K.to(DEV), V.to(DEV)
    plan = binding.chunk(ids.to(DEV), w.delims, w.max_chunk_len)
    out = binding.compress(Kd, Vd, plan, 0.7)
    ws = torch.zeros(binding.lib().sc_compress_budget_workspace_bytes(1, 2, 512), dtype=torch.uint8, device=DEV)
    tau = torch.zeros(1, dtype=torch.float32, device=DEV)
    search = torch.zeros(2, dtype=torch.int32, device=DEV)
    call = lambda *a, **k: binding.sc_compress_budget(Kd, Vd, plan, *a, out.core_k, out.core_v, out.count,
                                                      out.core_len, tau, search, ws, **k)
    for bad in ((0.5, 0.9, 0.5, 9), (0.5, 0.5, 0.9, 1), (0.5, 0.5, 0.9, 66), (1.5, 0.5, 0.9, 9), (-0.1, 0.5, 0.9, 9)):
        with pytest.raises(binding.ScError) as err:
            call(*bad)
        assert err.value.code == binding.SC_ERR_INVALID_ARG
    with pytest.raises(binding.ScError):
        call(0.5, 0.5, 0.9, 9, flags=binding.SC_FLAG_TWO_PASS)
    with pytest.raises(binding.ScError):
        binding.sc_compress_budget(Kd, Vd, plan, 0.5, 0.5, 0.9, 9, out.core_k, out.core_v, out.count, out.core_len,
                                   tau, search, ws[:1024])


# ------------------------------------------------------------------------- fixed-size chunking


@pytest.mark.parametrize("size", [64, 48])
def test_fixed_size_chunking_mode(size):
    """The paper's fixed-size ablation arm (Table 4a, 64-token chunks): chunk_fixed cuts every `size`
    tokens and gives delimiters no special role; the whole compress path then runs on those chunks."""
    w = synth.config(0, n=4000)
    ids, run_id, run_lens = synth.token_ids(w)
    K, V = synth.layer_kv(w, 0, run_id, run_lens)
    plan = binding.chunk_fixed(ids.to(DEV), size)
    seg_off, seq_seg_off = oracle.chunk(ids.numpy(), (), size)
    compare_plan(plan, seg_off, seq_seg_off)
    lens = np.diff(seg_off)
    assert (lens[:-1] == size).all() and lens[-1] == 4000 - size * (len(lens) - 1)
    ref = oracle_compress(ids, K, V, (), w.tau, size)
    assert ref["margin"] > 1e-4
    got = binding.compress(K.to(DEV), V.to(DEV), plan, w.tau, want_assign=True)
    binding.check_status(plan.status)
    compare_compressed(got, ref, torch.bfloat16)
    # tokens of different delimiter-bounded chunks do merge here: this is not the semantic chunking
    sem = oracle_compress(ids, K, V, w.delims, w.tau)
    assert not np.array_equal(sem["core_len"], ref["core_len"])

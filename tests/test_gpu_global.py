"""sc_compress_global (Algorithm 1 over whole sequences, the "no chunking" ablation arm of Table 4a)
against the oracle's compress_global on the same bytes."""
import numpy as np
import pytest
import torch

import oracle
from helpers import compare_compressed
from paper_2603_14303_b200 import binding, synth

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _both(K, V, tau, flags=0, cap=None):
    ref = oracle.compress_global(synth.to_numpy_bits(K), synth.to_numpy_bits(V), tau, cap)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    got = binding.compress_global(K.to(DEV), V.to(DEV), tau, cap=cap, want_assign=True, flags=flags, status=status)
    torch.cuda.synchronize()
    return ref, got, int(status.item())


@pytest.mark.parametrize("n,B,flags,dtype", [
    (1000, 2, 0, "bf16"), (1000, 2, binding.SC_FLAG_GENERIC, "bf16"), (700, 1, 0, "bf16"), (128, 1, 0, "bf16"),
    (129, 2, 0, "bf16"), (50, 1, 0, "bf16"), (1, 2, 0, "bf16"), (2, 1, 0, "bf16"), (600, 2, 0, "f32"), (4096, 1, 0, "bf16")])
def test_global_clustering_matches_oracle(n, B, flags, dtype):
    w = synth.config(0, n=n, B=B, Hkv=2, Hq=8, dtype=dtype)
    ids, run_id, run_lens = synth.token_ids(w)
    K, V = synth.layer_kv(w, 0, run_id, run_lens)
    ref, got, status = _both(K, V, w.tau, flags)
    assert status == 0
    assert ref["margin"] > 1e-4, "the workload keeps similarities clear of the threshold"
    compare_compressed(got, ref, K.dtype)
    # clusters do reach across delimiters here, which chunked compression never allows
    if n >= 600:
        chunked = oracle.compress(ids.numpy(), w.delims, synth.to_numpy_bits(K), synth.to_numpy_bits(V), w.tau)
        assert int(ref["core_len"].sum()) <= int(chunked["core_len"].sum())


def test_global_clustering_fp32_other_head_size_and_strided_layout():
    w = synth.config(0, n=520, B=2, Hkv=3, Hq=6, d=72, dtype="f32")
    ids, run_id, run_lens = synth.token_ids(w)
    K, V = synth.layer_kv(w, 0, run_id, run_lens)
    ref = oracle.compress_global(synth.to_numpy_bits(K), synth.to_numpy_bits(V), w.tau)
    # [B, n, Hkv, d] storage viewed head-major
    Ks = K.permute(0, 2, 1, 3).contiguous().to(DEV).permute(0, 2, 1, 3)
    Vs = V.permute(0, 2, 1, 3).contiguous().to(DEV).permute(0, 2, 1, 3)
    got = binding.compress_global(Ks, Vs, w.tau, want_assign=True)
    compare_compressed(got, ref, K.dtype)


@pytest.mark.parametrize("dtype,d,n", [("bf16", 128, 127), ("f32", 256, 255)])
def test_long_dependence_chain_needs_the_finishing_kernel(dtype, d, n):
    """Keys (e_i + e_{i+1}) / sqrt(2): token i is similar (cos 1/2) to its two neighbours only -- a path graph.
    Algorithm 1 gives seeds 0, 2, 4, ... each absorbing the next token, and deciding token i needs token i-1
    decided first: far more dependent steps than the rounds that are enqueued up front."""
    K = torch.zeros((1, 1, n, d))
    for i in range(n):
        K[0, 0, i, i] = 1.0
        K[0, 0, i, i + 1] = 1.0
    V = torch.arange(n * d, dtype=torch.float32).reshape(1, 1, n, d) / (n * d)
    dt = torch.bfloat16 if dtype == "bf16" else torch.float32
    ref, got, status = _both(K.to(dt), V.to(dt), 0.4)
    assert status == 0
    want = np.arange(n) - (np.arange(n) % 2)
    assert ref["assign"][0, 0].tolist() == want.tolist()
    compare_compressed(got, ref, dt)


def test_global_clustering_extremes_and_capacity():
    w = synth.config(0, n=300, B=1, Hkv=2, Hq=8)
    ids, run_id, run_lens = synth.token_ids(w)
    K, V = synth.layer_kv(w, 0, run_id, run_lens)
    ref, got, status = _both(K, V, 2.0)            # nothing merges
    assert status == 0 and got.core_len.tolist() == [[300, 300]]
    assert torch.equal(got.core_k.cpu(), K) and torch.equal(got.core_v.cpu(), V)
    ref, got, status = _both(K, V, -2.0)           # everything joins token 0
    assert status == 0 and got.core_len.tolist() == [[1, 1]] and got.count[0, :, 0].tolist() == [300, 300]
    compare_compressed(got, ref, K.dtype)
    Kz = K.clone()
    Kz[0, 0, 5] = 0                                # a zero-norm key: similarity 0 to everything
    ref, got, status = _both(Kz, V, w.tau)
    compare_compressed(got, ref, K.dtype)
    ref, got, status = _both(Kz, V, -0.5)          # ... which is above a negative threshold
    compare_compressed(got, ref, K.dtype)
    # too small a capacity: reported, core_len still says what is needed, nothing written past the end
    need = int(ref["core_len"].max())
    ref, got, status = _both(K, V, w.tau, cap=8)
    assert status == binding.SC_ERR_CAPACITY
    assert np.array_equal(got.core_len.cpu().numpy(), ref["core_len"]) and need >= 1
    compare_compressed(got, ref, K.dtype, check_assign=True)


@pytest.mark.parametrize("n", [40, 700, 1500])
def test_cluster_sizes_across_the_pooling_paths(n):
    """Clusters of up to 32 members are ordered in registers, up to 1024 by repeated selection, larger ones by
    walking the assignment array: one big cluster (everything similar to token 0 except a few strangers that
    found their own) exercises each in turn, in both dtypes."""
    rng = np.random.default_rng(n)
    for dt in (torch.bfloat16, torch.float32):
        base = rng.normal(size=128)
        K = torch.from_numpy(base + 0.05 * rng.normal(size=(1, 2, n, 128))).float()
        strangers = rng.choice(np.arange(1, n), size=5, replace=False)
        K[0, :, strangers] = torch.from_numpy(rng.normal(size=(2, 5, 128))).float()
        V = torch.from_numpy(rng.normal(size=(1, 2, n, 128))).float()
        ref, got, status = _both(K.to(dt), V.to(dt), 0.8)
        assert status == 0 and ref["margin"] > 1e-4
        assert int(ref["count"][0, 0, 0]) >= n - 6
        compare_compressed(got, ref, dt)


def test_decode_over_globally_clustered_cores():
    w = synth.config(0, n=1500, B=1)
    ids, run_id, run_lens = synth.token_ids(w)
    K, V = synth.layer_kv(w, 0, run_id, run_lens)
    ref, got, status = _both(K, V, w.tau)
    q = synth.queries(w, 0, 0)
    want = oracle.attn(synth.to_numpy_bits(q), ref["core_k"], ref["core_v"], ref["count"], ref["core_len"])
    out = binding.decode_attn(q.to(DEV), got)
    from helpers import assert_close_vectors, to_f64
    assert_close_vectors(to_f64(out), want, 1e-2, "decode over global cores")

"""sc_prefill_attn (Eq. 4 with a block of m queries per head) against the oracle's attn_multi."""
import numpy as np
import pytest
import torch

import oracle
from helpers import TOL, assert_close_vectors, layer_from_oracle, oracle_compress, to_f64
from paper_2603_14303_b200 import binding, synth

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _random_cache(rng, B, Hkv, cap, d, dtype, lens=None):
    tdt = torch.bfloat16 if dtype == "bf16" else torch.float32
    ck = torch.from_numpy(rng.normal(size=(B, Hkv, cap, d)).astype(np.float32)).to(tdt)
    cv = torch.from_numpy(rng.normal(size=(B, Hkv, cap, d)).astype(np.float32)).to(tdt)
    cnt = torch.from_numpy(rng.integers(1, 40, size=(B, Hkv, cap)).astype(np.int32))
    if lens is None:
        lens = rng.integers(0, cap + 1, size=(B, Hkv))
    clen = torch.from_numpy(np.asarray(lens, dtype=np.int32).reshape(B, Hkv))
    return ck, cv, cnt, clen


def _check(q, ck, cv, cnt, clen, causal, flags=0, use_count=True, poison=True):
    want = oracle.attn_multi(synth.to_numpy_bits(q), synth.to_numpy_bits(ck), synth.to_numpy_bits(cv),
                             cnt.numpy() if use_count else None, clen.numpy(), causal=causal)
    ckd, cvd = ck.to(DEV).clone(), cv.to(DEV).clone()
    if poison:   # rows past a head's length hold garbage in real use (NaN included): they must not leak
        for b in range(ck.shape[0]):
            for h in range(ck.shape[1]):
                ckd[b, h, int(clen[b, h]):] = float("nan")
                cvd[b, h, int(clen[b, h]):] = float("nan")
    layer = binding.CompressedLayer(ckd, cvd, cnt.to(DEV), clen.to(DEV))
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    out = torch.full(q.shape, float("nan"), dtype=q.dtype, device=DEV)
    binding.prefill_attn(q.to(DEV), layer, out=out, status=status, causal=causal, flags=flags, use_count=use_count)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    assert_close_vectors(to_f64(out), want, TOL[q.dtype], f"prefill causal={causal} flags={flags}")
    return out


@pytest.mark.parametrize("G,m", [(4, 32), (4, 48), (4, 1), (7, 5), (8, 40), (1, 130), (4, 256)])
@pytest.mark.parametrize("causal", [False, True])
def test_prefill_tensor_core_path_shapes(G, m, causal):
    rng = np.random.default_rng(G * 1000 + m)
    B, Hkv, cap, d = 2, 2, 700, 128
    lens = [[700, 0], [129, 333]] if not causal else [[700, 3], [128, 333]]
    ck, cv, cnt, clen = _random_cache(rng, B, Hkv, cap, d, "bf16", lens)
    q = torch.from_numpy(rng.normal(size=(B, Hkv * G, m, d)).astype(np.float32)).to(torch.bfloat16)
    _check(q, ck, cv, cnt, clen, causal)


@pytest.mark.parametrize("m,causal", [(1, False), (8, True), (33, False), (128, True)])
def test_prefill_few_queries_split_the_keys_over_a_cluster(m, causal):
    """Few query rows and a long cache: the keys of a head are shared out among the CTAs of a cluster (up to
    eight), whose partial results are folded through distributed shared memory.  Heads that are empty, shorter
    than one CTA's share, and full to capacity."""
    rng = np.random.default_rng(500 + m)
    B, Hkv, G, cap, d = 1, 3, 4, 4500, 128
    ck, cv, cnt, clen = _random_cache(rng, B, Hkv, cap, d, "bf16", [[4500, 0 if not causal else m, 300]])
    q = torch.from_numpy(rng.normal(size=(B, Hkv * G, m, d)).astype(np.float32)).to(torch.bfloat16)
    _check(q, ck, cv, cnt, clen, causal)


def test_prefill_sharp_scores_and_no_counts():
    """Large query norms make the softmax pick out few rows (the running maximum is raised many times);
    count = NULL is plain attention."""
    rng = np.random.default_rng(11)
    ck, cv, cnt, clen = _random_cache(rng, 1, 2, 1500, 128, "bf16", [[1500, 1111]])
    q = torch.from_numpy(6.0 * rng.normal(size=(1, 8, 64, 128)).astype(np.float32)).to(torch.bfloat16)
    _check(q, ck, cv, cnt, clen, False)
    _check(q, ck, cv, cnt, clen, True, use_count=False)


@pytest.mark.parametrize("dtype,d,flags", [("f32", 64, 0), ("f32", 128, 0), ("bf16", 128, binding.SC_FLAG_GENERIC), ("bf16", 72, 0)])
def test_prefill_generic_path(dtype, d, flags):
    rng = np.random.default_rng(5)
    ck, cv, cnt, clen = _random_cache(rng, 2, 2, 300, d, dtype)
    tdt = torch.bfloat16 if dtype == "bf16" else torch.float32
    q = torch.from_numpy(rng.normal(size=(2, 6, 9, d)).astype(np.float32)).to(tdt)
    for causal in (False, True):
        _check(q, ck, cv, cnt, clen, causal, flags=flags)


def test_prefill_one_query_equals_decode_and_whole_path():
    """On cores the GPU compressed itself: m = 1 is the decode step; a block of queries matches the oracle
    run on the oracle's cores; the tensor-core and CUDA-core kernels agree."""
    w = synth.config(0, n=4096)
    ids, run_id, run_lens = synth.token_ids(w)
    K, V = synth.layer_kv(w, 0, run_id, run_lens)
    ref = oracle_compress(ids, K, V, w.delims, w.tau)
    plan = binding.chunk(ids.to(DEV), w.delims, w.max_chunk_len)
    got = binding.compress(K.to(DEV), V.to(DEV), plan, w.tau)
    q1 = synth.queries(w, 0, 0).to(DEV)
    dec = binding.decode_attn(q1, got)
    pre = binding.prefill_attn(q1.unsqueeze(2).contiguous(), got)
    assert_close_vectors(to_f64(pre[:, :, 0]), to_f64(dec), 1e-2, "m = 1 against the decode kernel")
    m = 96
    q = torch.stack([synth.queries(w, s, 0) for s in range(m)], dim=2).contiguous()      # [B, Hq, m, d]
    want = oracle.attn_multi(synth.to_numpy_bits(q), ref["core_k"], ref["core_v"], ref["count"], ref["core_len"])
    a = binding.prefill_attn(q.to(DEV), got)
    assert_close_vectors(to_f64(a), want, 1e-2, "whole path, tensor cores")
    bq = binding.prefill_attn(q.to(DEV), got, flags=binding.SC_FLAG_GENERIC)
    assert_close_vectors(to_f64(bq), want, 1e-2, "whole path, CUDA cores")
    # causal tail: the cache's last m rows stand for the queries' own tokens
    wc = oracle.attn_multi(synth.to_numpy_bits(q), ref["core_k"], ref["core_v"], ref["count"], ref["core_len"], causal=True)
    c = binding.prefill_attn(q.to(DEV), got, causal=True)
    assert_close_vectors(to_f64(c), wc, 1e-2, "whole path, causal tail")


def test_prefill_argument_validation():
    q = torch.zeros((1, 8, 4, 128), dtype=torch.bfloat16, device=DEV)
    ck = torch.zeros((1, 2, 16, 128), dtype=torch.bfloat16, device=DEV)
    clen = torch.zeros((1, 2), dtype=torch.int32, device=DEV)
    raw = lambda Hq, Hkv, m, d, flags=0, dt=binding.SC_BF16: binding.lib().sc_prefill_attn(
        q.data_ptr(), dt, 1, Hq, Hkv, m, d, ck.data_ptr(), ck.data_ptr(), None, 16, clen.data_ptr(), 0.0, flags,
        q.data_ptr(), None, None)
    assert raw(8, 3, 4, 128) == binding.SC_ERR_INVALID_ARG
    assert raw(8, 2, 4, 100) == binding.SC_ERR_UNSUPPORTED
    assert raw(8, 2, 4, 128, dt=5) == binding.SC_ERR_UNSUPPORTED
    assert raw(8, 2, 4, 128, flags=binding.SC_FLAG_OVERLAP_PREV) == binding.SC_ERR_INVALID_ARG
    assert raw(8, 2, 0, 128) == binding.SC_OK
    out = binding.prefill_attn(q, binding.CompressedLayer(ck, ck, None, clen), use_count=False)
    assert torch.all(out == 0), "heads without cores yield zeros"

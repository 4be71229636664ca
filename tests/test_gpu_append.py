"""sc_append against the oracle's incremental path, through the C ABI, on the same bytes."""
import numpy as np
import pytest
import torch

import oracle
from helpers import TOL, assert_close_vectors, decode_bits, oracle_compress, to_f64
from paper_2603_14303_b200 import binding, synth

pytestmark = pytest.mark.gpu
DEV = torch.device("cuda:0")
DELIM = [13, 29889, 29892]


def _stream(seed, B, Hkv, m, d, p_delim, dtype, n_centroids=5, sigma=0.1):
    """Seeded generated stream: token ids with delimiters at rate p_delim, keys = unit centroid + noise of
    RMS norm sigma (same-centroid cosine ~ 1 / (1 + sigma^2), cross-centroid ~ 0), values N(0, 1)."""
    rng = np.random.default_rng(seed)
    ids = rng.integers(100, 29000, size=(B, m)).astype(np.int32)
    ids[rng.random((B, m)) < p_delim] = DELIM[seed % 3]
    cent = rng.normal(size=(n_centroids, d))
    cent /= np.linalg.norm(cent, axis=1, keepdims=True)
    K = cent[rng.integers(0, n_centroids, size=(B, Hkv, m))] + sigma / np.sqrt(d) * rng.normal(size=(B, Hkv, m, d))
    V = rng.normal(size=(B, Hkv, m, d))
    return torch.from_numpy(ids), torch.from_numpy(K).to(dtype), torch.from_numpy(V).to(dtype)


class Both:
    """The same cache on both sides: oracle state (numpy) and device buffers."""

    def __init__(self, B, Hkv, cap, d, dtype, prefill=None):
        npdt = np.uint16 if dtype == torch.bfloat16 else np.float32
        self.dtype = dtype
        if prefill is None:
            self.st = dict(core_k=np.zeros((B, Hkv, cap, d), npdt), core_v=np.zeros((B, Hkv, cap, d), npdt),
                           count=np.zeros((B, Hkv, cap), np.int32), core_len=np.zeros((B, Hkv), np.int32))
            self.ck = torch.zeros((B, Hkv, cap, d), dtype=dtype, device=DEV)
            self.cv = torch.zeros_like(self.ck)
            self.cnt = torch.zeros((B, Hkv, cap), dtype=torch.int32, device=DEV)
            self.clen = torch.zeros((B, Hkv), dtype=torch.int32, device=DEV)
        else:
            ref, got = prefill
            self.st = {k: ref[k].copy() for k in ("core_k", "core_v", "count", "core_len")}
            self.ck, self.cv, self.cnt, self.clen = got.core_k, got.core_v, got.count, got.core_len
        self.st["tail_len"] = np.zeros((B, Hkv), np.int32)
        self.tlen = torch.zeros((B, Hkv), dtype=torch.int32, device=DEV)
        self.alen = torch.full((B, Hkv), -1, dtype=torch.int32, device=DEV)
        self.status = torch.zeros(1, dtype=torch.int32, device=DEV)

    def step(self, ids_t, k_t, v_t, tau, max_len):
        ids_t, k_t, v_t = ids_t.contiguous(), k_t.contiguous(), v_t.contiguous()
        oracle.append(self.st, ids_t.numpy(), synth.to_numpy_bits(k_t), synth.to_numpy_bits(v_t), DELIM, tau, max_len)
        binding.sc_append(k_t.to(DEV), v_t.to(DEV), ids_t.to(DEV), DELIM, max_len, tau,
                          self.ck, self.cv, self.cnt, self.clen, self.tlen, self.alen, self.status)

    def compare(self, what):
        binding.check_status(self.status, what)
        st = self.st
        assert np.array_equal(self.clen.cpu().numpy(), st["core_len"]), f"{what}: core_len"
        assert np.array_equal(self.tlen.cpu().numpy(), st["tail_len"]), f"{what}: tail_len"
        assert np.array_equal(self.alen.cpu().numpy(), st["core_len"] + st["tail_len"]), f"{what}: attn_len"
        gk, gv, cnt = to_f64(self.ck), to_f64(self.cv), self.cnt.cpu().numpy()
        B, Hkv = st["core_len"].shape
        for b in range(B):
            for h in range(Hkv):
                L = int(st["core_len"][b, h] + st["tail_len"][b, h])
                assert np.array_equal(cnt[b, h, :L], st["count"][b, h, :L]), f"{what}: count[{b},{h}]"
                rk, rv = decode_bits(st["core_k"][b, h, :L]), decode_bits(st["core_v"][b, h, :L])
                assert_close_vectors(gk[b, h, :L], rk, TOL[self.dtype], f"{what}: core_k[{b},{h}]")
                assert_close_vectors(gv[b, h, :L], rv, TOL[self.dtype], f"{what}: core_v[{b},{h}]")
                single = np.flatnonzero(st["count"][b, h, :L] == 1)   # untouched rows are exact copies
                assert np.array_equal(gk[b, h, single], rk[single]) and np.array_equal(gv[b, h, single], rv[single])


@pytest.mark.parametrize("dtype,d", [(torch.bfloat16, 128), (torch.float32, 64), (torch.float32, 40)])
@pytest.mark.parametrize("max_len,p_delim", [(256, 0.06), (32, 0.02), (7, 0.0)])
def test_append_from_an_empty_cache_matches_the_oracle_step_by_step(dtype, d, max_len, p_delim):
    B, Hkv, m = 3, 2, 300
    ids, K, V = _stream(11 + max_len, B, Hkv, m, d, p_delim, dtype)
    both = Both(B, Hkv, m, d, dtype)
    for t in range(m):
        both.step(ids[:, t], K[:, :, t], V[:, :, t], 0.7, max_len)
        if t % 37 == 0 or t == m - 1:
            both.compare(f"step {t}")
    assert both.st["margin"] > 1e-4


def test_append_behind_a_compressed_prompt_then_decode():
    """Prompt compressed by sc_compress, 150 generated tokens appended, and each step's attention over
    cores + open tail compared with Eq. 4 on the oracle's state."""
    w = synth.config(0)
    tdt = torch.bfloat16
    ids, run_id, run_lens = synth.token_ids(w)
    K, V = synth.layer_kv(w, 0, run_id, run_lens)
    m = 150
    cap = w.n + m
    ref = oracle_compress(ids, K, V, w.delims, w.tau, w.max_chunk_len, cap)
    plan = binding.chunk(ids.to(DEV), w.delims, w.max_chunk_len)
    got = binding.compress(K.to(DEV), V.to(DEV), plan, w.tau, cap=cap)
    binding.check_status(plan.status)
    both = Both(w.B, w.Hkv, cap, w.d, tdt, prefill=(ref, got))
    gids, gK, gV = _stream(5, w.B, w.Hkv, m, w.d, 0.05, tdt)
    ws = binding.decode_workspace(w.B, w.Hq, w.Hkv, w.d, cap, DEV)
    for t in range(m):
        both.step(gids[:, t], gK[:, :, t], gV[:, :, t], w.tau, w.max_chunk_len)
        if t % 10 == 0 or t == m - 1:
            q = synth.queries(w, t, 0)
            st = both.st
            want = oracle.attn(synth.to_numpy_bits(q), st["core_k"], st["core_v"], st["count"],
                               st["core_len"] + st["tail_len"])
            layer = binding.CompressedLayer(both.ck, both.cv, both.cnt, both.alen)
            out = binding.decode_attn(q.to(DEV), layer, workspace=ws)
            assert_close_vectors(to_f64(out), want, 1e-2, f"decode after {t + 1} appended tokens")
    both.compare("end")
    assert int(both.clen.sum()) < int(torch.from_numpy(ref["core_len"]).sum()) + w.B * w.Hkv * m   # something merged


@pytest.mark.parametrize("kind", ["identical", "distinct", "zero"])
def test_append_longest_chunk_degenerate_keys(kind):
    """A 256-token chunk closed by its length: all keys equal (one cluster), all orthogonal (256 clusters),
    all zero (similarity 0 to everything: no merging at tau = 0.7)."""
    B, Hkv, d, m = 1, 2, 256, 256
    rng = np.random.default_rng(3)
    if kind == "identical":
        K = np.broadcast_to(rng.normal(size=(1, 1, 1, d)), (B, Hkv, m, d)).copy()
    elif kind == "distinct":
        K = np.broadcast_to(np.eye(m, d)[None, None], (B, Hkv, m, d)).copy()
    else:
        K = np.zeros((B, Hkv, m, d))
    K, V = torch.from_numpy(K).float(), torch.from_numpy(rng.normal(size=(B, Hkv, m, d))).float()
    ids = torch.full((B, m), 500, dtype=torch.int32)
    both = Both(B, Hkv, m, d, torch.float32)
    for t in range(m):
        both.step(ids[:, t], K[:, :, t], V[:, :, t], 0.7, 256)
    both.compare(kind)
    assert (both.st["core_len"] == (1 if kind == "identical" else 256)).all() and not both.st["tail_len"].any()


def test_append_full_cache_is_reported_and_left_alone():
    B, Hkv, d, cap = 2, 2, 128, 4
    ids, K, V = _stream(1, B, Hkv, 6, d, 0.0, torch.bfloat16)
    both = Both(B, Hkv, cap, d, torch.bfloat16)
    for t in range(4):
        both.step(ids[:, t], K[:, :, t], V[:, :, t], 0.7, 256)
    both.compare("full")
    before = (both.ck.clone(), both.cnt.clone(), both.clen.clone(), both.tlen.clone())
    binding.sc_append(K[:, :, 4].contiguous().to(DEV), V[:, :, 4].contiguous().to(DEV), ids[:, 4].to(DEV), DELIM, 256, 0.7,
                      both.ck, both.cv, both.cnt, both.clen, both.tlen, both.alen, both.status)
    assert int(both.status.item()) == binding.SC_ERR_CAPACITY
    assert torch.equal(both.ck, before[0]) and torch.equal(both.cnt, before[1])
    assert torch.equal(both.clen, before[2]) and torch.equal(both.tlen, before[3])
    assert (both.alen.cpu().numpy() == 4).all()


def test_append_refuses_lengths_that_cannot_be_its_own_state():
    B, Hkv, d, cap = 1, 2, 128, 16
    ids, K, V = _stream(2, B, Hkv, 1, d, 0.0, torch.bfloat16)
    both = Both(B, Hkv, cap, d, torch.bfloat16)
    both.tlen.fill_(5)            # an open chunk of 5 tokens cannot exist with max_chunk_len = 4
    binding.sc_append(K[:, :, 0].contiguous().to(DEV), V[:, :, 0].contiguous().to(DEV), ids[:, 0].contiguous().to(DEV), DELIM, 4,
                      0.7, both.ck, both.cv, both.cnt, both.clen, both.tlen, both.alen, both.status)
    assert int(both.status.item()) == binding.SC_ERR_INVALID_ARG
    assert int(both.clen.abs().max()) == 0 and (both.tlen == 5).all() and int(both.cnt.abs().max()) == 0


@pytest.mark.parametrize("dtype,d", [(torch.bfloat16, 128), (torch.float32, 64)])
def test_all_layers_in_one_launch_equal_one_launch_per_layer(dtype, d):
    """sc_append_layers: every layer of a generated token in one launch.  Each layer has its own keys and
    values (so chunks cluster differently per layer); after every token the batched caches must equal, bit
    for bit, caches maintained by one sc_append per layer, and layer 0 must match the oracle's state."""
    B, Hkv, m, L, max_len = 2, 2, 160, 3, 24
    streams = [_stream(40 + l, B, Hkv, m, d, 0.07, dtype) for l in range(L)]
    ids = streams[0][0]                       # the token ids are the model's, the same for every layer
    single = [Both(B, Hkv, m, d, dtype) for _ in range(L)]
    batched = [Both(B, Hkv, m, d, dtype) for _ in range(L)]
    k_new = [torch.zeros((B, Hkv, d), dtype=dtype, device=DEV) for _ in range(L)]
    v_new = [torch.zeros((B, Hkv, d), dtype=dtype, device=DEV) for _ in range(L)]
    table = binding.append_table([(k_new[l], v_new[l], x.ck, x.cv, x.cnt, x.clen, x.tlen, x.alen)
                                  for l, x in enumerate(batched)])
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    tok = torch.zeros(B, dtype=torch.int32, device=DEV)
    for t in range(m):
        for l in range(L):
            single[l].step(ids[:, t], streams[l][1][:, :, t], streams[l][2][:, :, t], 0.7, max_len)
            k_new[l].copy_(streams[l][1][:, :, t])
            v_new[l].copy_(streams[l][2][:, :, t])
        tok.copy_(ids[:, t])
        binding.sc_append_layers(table, k_new[0], tok, DELIM, max_len, 0.7, m, status)
        if t % 40 == 39 or t == m - 1:
            binding.check_status(status, "sc_append_layers")
            for l in range(L):
                a, b = single[l], batched[l]
                for x, y in ((a.clen, b.clen), (a.tlen, b.tlen), (a.alen, b.alen), (a.cnt, b.cnt), (a.ck, b.ck), (a.cv, b.cv)):
                    assert torch.equal(x, y), f"layer {l}, token {t}"
    single[0].compare("layer 0 after the stream")
    # a full cache in one layer is reported and leaves that layer alone
    batched[1].clen.fill_(m)
    batched[1].tlen.zero_()
    before = batched[1].ck.clone()
    binding.sc_append_layers(table, k_new[0], tok, DELIM, max_len, 0.7, m, status)
    assert int(status.item()) == binding.SC_ERR_CAPACITY and torch.equal(before, batched[1].ck)

"""sc_decode_attn_static against sc_decode_attn (collected last on purpose).

Some users of the library reach the decode loop with no way left to allocate device memory: a
server whose KV-cache pool took all free HBM at start-up, a plug-in whose host forbids
allocation in its step callback, a loop that cannot afford the synchronisation an allocation
may cause.  sc_decode_attn_static serves them with the split partials and arrival counters in a
fixed array inside the library image instead of a caller-provided workspace.  It must give what
sc_decode_attn gives, on the first call and again on the next one, when the shared array still
holds the first call's leftovers.
"""
import numpy as np
import pytest
import torch

from helpers import TOL, assert_close_vectors, to_f64
from paper_2603_14303_b200 import binding

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _cores(rng, B, Hkv, cap, d, dtype):
    ck = torch.from_numpy(rng.normal(size=(B, Hkv, cap, d)).astype(np.float32)).to(dtype).to(DEV)
    cv = torch.from_numpy(rng.normal(size=(B, Hkv, cap, d)).astype(np.float32)).to(dtype).to(DEV)
    cnt = torch.from_numpy(rng.integers(1, 30, size=(B, Hkv, cap)).astype(np.int32)).to(DEV)
    clen = torch.from_numpy(rng.integers(cap // 3, cap + 1, size=(B, Hkv)).astype(np.int32))
    clen[0, 0] = 0          # a head without cores
    clen[-1, -1] = cap      # a full head
    return binding.CompressedLayer(ck, cv, cnt, clen.to(DEV))


@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32])
def test_static_scratch_decode_matches_workspace_decode_twice_in_a_row(dtype):
    rng = np.random.default_rng(20260314)
    B, Hkv, G, d, cap = 2, 4, 4, 128, 3000
    layer = _cores(rng, B, Hkv, cap, d, dtype)
    ws = binding.decode_workspace(B, Hkv * G, Hkv, d, cap, DEV)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    # two different problems back to back: the second call meets the first one's leftovers
    for call, use_count in enumerate((True, False)):
        q = torch.from_numpy(rng.normal(size=(B, Hkv * G, d)).astype(np.float32)).to(dtype).to(DEV)
        want = binding.decode_attn(q, layer, workspace=ws, use_count=use_count)
        got = torch.full_like(q, float("nan"))
        binding.sc_decode_attn_static(q, layer.core_k, layer.core_v, layer.count if use_count else None,
                                      layer.core_len, got, status=status)
        torch.cuda.synchronize()
        assert int(status.item()) == binding.SC_OK
        assert_close_vectors(to_f64(got), to_f64(want), TOL[dtype], f"static scratch, call {call}")
        assert torch.all(got[0, :G] == 0), "a head without cores yields zeros"


def test_static_scratch_rejects_oversized_and_overlapped_calls():
    rng = np.random.default_rng(7)
    layer = _cores(rng, 1, 2, 64, 128, torch.bfloat16)
    q = torch.zeros((1, 8, 128), dtype=torch.bfloat16, device=DEV)
    out = torch.empty_like(q)
    # the workspace this shape would need is far beyond the fixed array: refused, nothing enqueued
    B, Hq, Hkv, d, cap = 64, 64, 8, 128, 65536
    assert binding.lib().sc_decode_workspace_bytes(B, Hq, Hkv, d, cap) > binding.SC_STATIC_SCRATCH_BYTES
    code = binding.lib().sc_decode_attn_static(q.data_ptr(), binding.SC_BF16, B, Hq, Hkv, d, layer.core_k.data_ptr(),
                                               layer.core_v.data_ptr(), None, cap, layer.core_len.data_ptr(), 0.0, 0,
                                               out.data_ptr(), None, None)
    assert code == binding.SC_ERR_CAPACITY
    with pytest.raises(binding.ScError) as err:
        binding.sc_decode_attn_static(q, layer.core_k, layer.core_v, layer.count, layer.core_len, out,
                                      flags=binding.SC_FLAG_OVERLAP_PREV)
    assert err.value.code == binding.SC_ERR_INVALID_ARG

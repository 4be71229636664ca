"""sc_decode_attn_static against sc_decode_attn and the oracle (collected last on purpose).

Some users of the library reach the decode loop with no way left to allocate device memory: a
server whose KV-cache pool took all free HBM at start-up, a plug-in whose host forbids
allocation in its step callback, a loop that cannot afford the synchronisation an allocation
may cause.  sc_decode_attn_static serves them with the split partials and arrival counters in a
fixed array inside the library image instead of a caller-provided workspace.  It must give what
sc_decode_attn gives (the same kernels run, so bit for bit) and what Eq. 4 says, on the first
call and again on the next one, when the shared array still holds an earlier call's leftovers;
it must allocate nothing; and it must refuse, before anything is enqueued, a shape whose scratch
would not fit the fixed array.
"""
import numpy as np
import pytest
import torch

import oracle
from helpers import TOL, assert_close_vectors, to_f64
from paper_2603_14303_b200 import binding, synth

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _cores(rng, B, Hkv, cap, d, dtype, max_len=None):
    g = torch.Generator(device=DEV)
    g.manual_seed(int(rng.integers(1 << 30)))
    ck = torch.randn((B, Hkv, cap, d), generator=g, device=DEV).to(dtype)
    cv = torch.randn((B, Hkv, cap, d), generator=g, device=DEV).to(dtype)
    cnt = torch.randint(1, 30, (B, Hkv, cap), generator=g, device=DEV, dtype=torch.int32)
    top = cap if max_len is None else min(max_len, cap)
    clen = torch.from_numpy(rng.integers(top // 3, top + 1, size=(B, Hkv)).astype(np.int32))
    clen[0, 0] = 0          # a head without cores
    clen[-1, -1] = top      # the longest head
    return binding.CompressedLayer(ck, cv, cnt, clen.to(DEV))


def _oracle_attn(q, layer, use_count, rows):
    """Eq. 4 by the oracle on the first `rows` rows of every head (all that core_len reaches)."""
    bits = lambda t: synth.to_numpy_bits(t[:, :, :rows].contiguous())
    cnt = layer.count[:, :, :rows].contiguous().cpu().numpy() if use_count else None
    return oracle.attn(synth.to_numpy_bits(q), bits(layer.core_k), bits(layer.core_v), cnt,
                       layer.core_len.cpu().numpy())


@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32])
def test_static_scratch_decode_matches_workspace_decode_twice_in_a_row(dtype):
    rng = np.random.default_rng(20260314)
    B, Hkv, G, d, cap = 2, 4, 4, 128, 3000
    layer = _cores(rng, B, Hkv, cap, d, dtype)
    ws = binding.decode_workspace(B, Hkv * G, Hkv, d, cap, DEV)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    # leftovers from a problem with another number of heads and another split count
    other = _cores(rng, 3, 2, 700, d, dtype)
    binding.sc_decode_attn_static(torch.ones((3, 4, d), dtype=dtype, device=DEV), other.core_k, other.core_v,
                                  other.count, other.core_len, torch.empty((3, 4, d), dtype=dtype, device=DEV))
    # two different problems back to back: the second call meets the first one's leftovers
    for call, use_count in enumerate((True, False)):
        q = torch.from_numpy(rng.normal(size=(B, Hkv * G, d)).astype(np.float32)).to(dtype).to(DEV)
        same = binding.decode_attn(q, layer, workspace=ws, use_count=use_count)
        got = torch.full_like(q, float("nan"))
        torch.cuda.synchronize()
        held, free = torch.cuda.memory_allocated(), torch.cuda.mem_get_info()[0]
        binding.sc_decode_attn_static(q, layer.core_k, layer.core_v, layer.count if use_count else None,
                                      layer.core_len, got, status=status)
        torch.cuda.synchronize()
        assert torch.cuda.memory_allocated() == held and torch.cuda.mem_get_info()[0] == free, "the call allocated"
        assert int(status.item()) == binding.SC_OK
        assert torch.equal(got, same), f"call {call}: differs from sc_decode_attn"
        want = _oracle_attn(q, layer, use_count, cap)
        assert_close_vectors(to_f64(got), want, TOL[dtype], f"static scratch vs oracle, call {call}")
        assert torch.all(got[0, :G] == 0), "a head without cores yields zeros"


def test_static_scratch_at_its_size_limit():
    """The largest batch whose scratch still fits the fixed array runs and is right; one sequence more is
    refused with SC_ERR_CAPACITY before anything is enqueued."""
    rng = np.random.default_rng(5)
    Hkv, G, d, cap = 2, 4, 128, 32768
    need = lambda B: binding.lib().sc_decode_workspace_bytes(B, Hkv * G, Hkv, d, cap)
    B = 1
    while need(B + 1) <= binding.SC_STATIC_SCRATCH_BYTES:
        B += 1
    assert need(B) <= binding.SC_STATIC_SCRATCH_BYTES < need(B + 1)
    assert need(B) > 0.9 * binding.SC_STATIC_SCRATCH_BYTES, "the probe shape should come close to the limit"
    layer = _cores(rng, B, Hkv, cap, d, torch.bfloat16, max_len=1200)
    q = torch.from_numpy(rng.normal(size=(B, Hkv * G, d)).astype(np.float32)).to(torch.bfloat16).to(DEV)
    same = binding.decode_attn(q, layer)
    for call in range(2):
        got = torch.full_like(q, float("nan"))
        binding.sc_decode_attn_static(q, layer.core_k, layer.core_v, layer.count, layer.core_len, got)
        torch.cuda.synchronize()
        assert torch.equal(got, same), f"call {call}"
    assert_close_vectors(to_f64(got), _oracle_attn(q, layer, True, 1200), 1e-2, "at the size limit")
    # one sequence more: same pointers are fine, nothing may be launched
    before = binding.launch_counter()
    code = binding.lib().sc_decode_attn_static(q.data_ptr(), binding.SC_BF16, B + 1, Hkv * G, Hkv, d,
                                               layer.core_k.data_ptr(), layer.core_v.data_ptr(), None, cap,
                                               layer.core_len.data_ptr(), 0.0, 0, got.data_ptr(), None, None)
    assert code == binding.SC_ERR_CAPACITY and binding.launch_counter() == before


def test_static_scratch_rejects_oversized_and_overlapped_calls_like_sc_decode_attn():
    rng = np.random.default_rng(7)
    layer = _cores(rng, 1, 2, 64, 128, torch.bfloat16)
    q = torch.zeros((1, 8, 128), dtype=torch.bfloat16, device=DEV)
    out = torch.empty_like(q)
    raw = lambda B, Hq, Hkv, d, cap, flags=0, dt=binding.SC_BF16: binding.lib().sc_decode_attn_static(
        q.data_ptr(), dt, B, Hq, Hkv, d, layer.core_k.data_ptr(), layer.core_v.data_ptr(), None, cap,
        layer.core_len.data_ptr(), 0.0, flags, out.data_ptr(), None, None)
    # the workspace this shape would need is far beyond the fixed array: refused, nothing enqueued
    assert binding.lib().sc_decode_workspace_bytes(64, 64, 8, 128, 65536) > binding.SC_STATIC_SCRATCH_BYTES
    assert raw(64, 64, 8, 128, 65536) == binding.SC_ERR_CAPACITY
    # argument errors are reported as sc_decode_attn reports them, ahead of the size check
    assert raw(64, 64, 8, 0, 65536) == binding.SC_ERR_UNSUPPORTED
    assert raw(64, 64, 8, 100, 65536) == binding.SC_ERR_UNSUPPORTED
    assert raw(64, 63, 8, 128, 65536) == binding.SC_ERR_INVALID_ARG
    assert raw(64, 64, 8, 128, 65536, dt=7) == binding.SC_ERR_UNSUPPORTED
    for flag in (binding.SC_FLAG_OVERLAP_PREV, binding.SC_FLAG_OVERLAP_CHAIN):
        with pytest.raises(binding.ScError) as err:
            binding.sc_decode_attn_static(q, layer.core_k, layer.core_v, layer.count, layer.core_len, out, flags=flag)
        assert err.value.code == binding.SC_ERR_INVALID_ARG

"""ctypes binding of the C-ABI library (``include/semanticache.h``).

Argument marshalling only: torch provides device memory and the current stream, every step
of the path runs in the library's CUDA kernels.  There is no fallback: if the library has not
been built, or a call reports an error, an exception is raised.
"""
from __future__ import annotations

import ctypes
import dataclasses
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libsemanticache.so")

SC_OK, SC_ERR_INVALID_ARG, SC_ERR_UNSUPPORTED, SC_ERR_CAPACITY, SC_ERR_CUDA, SC_ERR_TIMEOUT = range(6)
SC_BF16, SC_F32 = 0, 1
SC_FLAG_GENERIC, SC_FLAG_TWO_PASS, SC_FLAG_OVERLAP_PREV, SC_FLAG_OVERLAP_CHAIN, SC_FLAG_CAUSAL_TAIL = 1, 2, 4, 8, 16
SC_MAX_CHUNK_LEN, SC_MAX_DELIMS, SC_TILE_ROWS = 256, 64, 128
_STATUS_NAMES = ["SC_OK", "SC_ERR_INVALID_ARG", "SC_ERR_UNSUPPORTED", "SC_ERR_CAPACITY", "SC_ERR_CUDA",
                 "SC_ERR_TIMEOUT"]

EXPORTS = ["sc_version", "sc_launch_counter", "sc_chunk_bounds", "sc_chunk_workspace_bytes", "sc_chunk",
           "sc_compress_workspace_bytes", "sc_compress", "sc_decode_workspace_bytes", "sc_decode_attn",
           "sc_decode_attn_static", "sc_append", "sc_compress_budget_workspace_bytes", "sc_compress_budget",
           "sc_compress_global_workspace_bytes", "sc_compress_global", "sc_prefill_attn", "sc_append_layers",
           "sc_compress_layers_workspace_bytes", "sc_compress_layers"]
SC_MAX_LAYERS_PER_CALL = 64
SC_BUDGET_MAX_GRID = 65
SC_STATIC_SCRATCH_BYTES = 8 << 20


class ScError(RuntimeError):
    def __init__(self, where: str, code: int):
        self.code = code
        super().__init__(f"{where}: {_STATUS_NAMES[code] if 0 <= code < 6 else code}")


class _GscParams(ctypes.Structure):
    _fields_ = [("tau", ctypes.c_float), ("max_chunk_len", ctypes.c_int32), ("flags", ctypes.c_uint32)]


class _Budget(ctypes.Structure):
    _fields_ = [("target_kept", ctypes.c_float), ("tau_lo", ctypes.c_float), ("tau_hi", ctypes.c_float),
                ("n_grid", ctypes.c_int32)]


class _CompressLayer(ctypes.Structure):
    _fields_ = [(k, ctypes.c_void_p) for k in ("K", "V", "core_k", "core_v", "count", "core_len", "assign")]


class _Strides(ctypes.Structure):
    _fields_ = [("b", ctypes.c_int64), ("h", ctypes.c_int64), ("n", ctypes.c_int64)]


_lib = None
_i32, _vp, _sz = ctypes.c_int32, ctypes.c_void_p, ctypes.c_size_t


def lib() -> ctypes.CDLL:
    """The loaded C-ABI library; raises if it was never built (no CPU fallback exists)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: run `python -m paper_2603_14303_b200.build` "
                               "(there is no fallback implementation)")
        L = ctypes.CDLL(LIB_PATH)
        L.sc_version.restype = ctypes.c_char_p
        L.sc_launch_counter.restype = ctypes.c_uint64
        L.sc_chunk_bounds.restype = _i32
        L.sc_chunk_bounds.argtypes = [_i32, _i32, ctypes.POINTER(_i32), ctypes.POINTER(_i32)]
        for f in (L.sc_chunk_workspace_bytes, L.sc_compress_workspace_bytes, L.sc_decode_workspace_bytes):
            f.restype = _sz
        L.sc_chunk_workspace_bytes.argtypes = [_i32, _i32]
        L.sc_compress_workspace_bytes.argtypes = [_i32, _i32, _i32]
        L.sc_decode_workspace_bytes.argtypes = [_i32] * 5
        L.sc_chunk.restype = _i32
        L.sc_chunk.argtypes = [_vp, _i32, _i32, ctypes.POINTER(_i32), _i32, _i32, _vp, _i32, _vp, _vp, _vp, _i32,
                               _vp, _vp, _sz, _vp, _vp]
        L.sc_compress.restype = _i32
        L.sc_compress.argtypes = [_vp, _vp, _Strides, _i32, _i32, _i32, _i32, _i32, _vp, _vp, _vp, _vp, _vp, _i32,
                                  ctypes.POINTER(_GscParams), _vp, _vp, _vp, _i32, _vp, _vp, _vp, _sz, _vp, _vp]
        L.sc_compress_layers_workspace_bytes.restype = _sz
        L.sc_compress_layers_workspace_bytes.argtypes = [_i32, _i32, _i32, _i32]
        L.sc_compress_layers.restype = _i32
        L.sc_compress_layers.argtypes = [ctypes.POINTER(_CompressLayer), _i32, _Strides, _i32, _i32, _i32, _i32, _i32,
                                         _vp, _vp, _vp, _vp, _vp, _i32, ctypes.POINTER(_GscParams), _i32, _vp, _sz, _vp, _vp]
        L.sc_compress_budget_workspace_bytes.restype = _sz
        L.sc_compress_budget_workspace_bytes.argtypes = [_i32, _i32, _i32]
        L.sc_compress_budget.restype = _i32
        L.sc_compress_budget.argtypes = [_vp, _vp, _Strides, _i32, _i32, _i32, _i32, _i32, _vp, _vp, _vp, _vp, _vp, _i32,
                                         ctypes.POINTER(_GscParams), ctypes.POINTER(_Budget), _vp, _vp, _vp, _i32, _vp,
                                         _vp, _vp, _vp, _vp, _sz, _vp, _vp]
        L.sc_compress_global_workspace_bytes.restype = _sz
        L.sc_compress_global_workspace_bytes.argtypes = [_i32, _i32, _i32]
        L.sc_compress_global.restype = _i32
        L.sc_compress_global.argtypes = [_vp, _vp, _Strides, _i32, _i32, _i32, _i32, _i32, ctypes.c_float, ctypes.c_uint32,
                                         _vp, _vp, _vp, _i32, _vp, _vp, _vp, _sz, _vp, _vp]
        L.sc_decode_attn.restype = _i32
        L.sc_decode_attn.argtypes = [_vp, _i32, _i32, _i32, _i32, _i32, _vp, _vp, _vp, _i32, _vp, ctypes.c_float,
                                     ctypes.c_uint32, _vp, _vp, _sz, _vp, _vp]
        L.sc_append_layers.restype = _i32
        L.sc_append_layers.argtypes = [_vp, _i32, _i32, _i32, _i32, _i32, _vp, ctypes.POINTER(_i32), _i32, _i32,
                                       ctypes.c_float, _i32, _vp, _vp]
        L.sc_prefill_attn.restype = _i32
        L.sc_prefill_attn.argtypes = [_vp, _i32, _i32, _i32, _i32, _i32, _i32, _vp, _vp, _vp, _i32, _vp, ctypes.c_float,
                                      ctypes.c_uint32, _vp, _vp, _vp]
        L.sc_decode_attn_static.restype = _i32
        L.sc_decode_attn_static.argtypes = [_vp, _i32, _i32, _i32, _i32, _i32, _vp, _vp, _vp, _i32, _vp,
                                            ctypes.c_float, ctypes.c_uint32, _vp, _vp, _vp]
        L.sc_append.restype = _i32
        L.sc_append.argtypes = [_vp, _vp, _i32, _i32, _i32, _i32, _vp, ctypes.POINTER(_i32), _i32, _i32, ctypes.c_float,
                                _vp, _vp, _vp, _i32, _vp, _vp, _vp, _vp, _vp]
        _lib = L
    return _lib


def _ptr(t):
    return None if t is None else t.data_ptr()


def _stream(t: torch.Tensor):
    return torch.cuda.current_stream(t.device).cuda_stream


def _dt(t: torch.Tensor) -> int:
    if t.dtype == torch.bfloat16:
        return SC_BF16
    if t.dtype == torch.float32:
        return SC_F32
    raise TypeError(f"unsupported dtype {t.dtype}")


def _check(where: str, code: int):
    if code != SC_OK:
        raise ScError(where, code)


def _need_cuda(*ts):
    for t in ts:
        if t is not None and not t.is_cuda:
            raise ValueError("device tensors required")


def launch_counter() -> int:
    """Kernels launched (or captured into a graph) by the library since it was loaded."""
    return int(lib().sc_launch_counter())


def chunk_bounds(B: int, n: int):
    a, b = _i32(0), _i32(0)
    _check("sc_chunk_bounds", lib().sc_chunk_bounds(B, n, ctypes.byref(a), ctypes.byref(b)))
    return a.value, b.value


# ------------------------------------------------------------------------------------ raw calls


def sc_chunk(token_ids, delim_ids, max_chunk_len, seg_off, seq_seg_off, n_seg, tile_seg, seq_tile_cnt,
             workspace, status=None):
    """Raw sc_chunk on caller-provided device buffers (see the header for shapes)."""
    _need_cuda(token_ids, seg_off, seq_seg_off, n_seg, tile_seg, seq_tile_cnt, workspace)
    B, n = token_ids.shape
    assert token_ids.dtype == torch.int32 and token_ids.is_contiguous()
    dl = (_i32 * max(len(delim_ids), 1))(*[int(x) for x in delim_ids])
    n_tile_cap = tile_seg.shape[1] - 1 if tile_seg.dim() == 2 else tile_seg.numel() // max(B, 1) - 1
    code = lib().sc_chunk(_ptr(token_ids), B, n, dl, len(delim_ids), max_chunk_len, _ptr(seg_off),
                          seg_off.numel() - 1, _ptr(seq_seg_off), _ptr(n_seg), _ptr(tile_seg), n_tile_cap,
                          _ptr(seq_tile_cnt), _ptr(workspace), workspace.numel() * workspace.element_size(),
                          _ptr(status), _stream(seg_off))
    _check("sc_chunk", code)


def sc_compress(K, V, plan: "ChunkPlan", tau, core_k, core_v, count, core_len, assign=None, workspace=None,
                status=None, flags=0):
    """Raw sc_compress for one layer on caller-provided buffers."""
    _need_cuda(K, V, core_k, core_v, count, core_len, assign, workspace)
    B, Hkv, n, d = K.shape
    assert V.shape == K.shape and V.stride() == K.stride() and V.dtype == K.dtype and K.stride(3) == 1
    assert core_k.is_contiguous() and core_v.is_contiguous() and count.is_contiguous()
    cap = core_k.shape[2]
    prm = _GscParams(float(tau), int(plan.max_chunk_len), int(flags))
    st = _Strides(K.stride(0), K.stride(1), K.stride(2))
    code = lib().sc_compress(_ptr(K), _ptr(V), st, _dt(K), B, Hkv, n, d, _ptr(plan.seg_off), _ptr(plan.seq_seg_off),
                             _ptr(plan.n_seg), _ptr(plan.tile_seg), _ptr(plan.seq_tile_cnt), plan.n_tile_cap,
                             ctypes.byref(prm), _ptr(core_k), _ptr(core_v), _ptr(count), cap, _ptr(core_len),
                             _ptr(assign), _ptr(workspace), workspace.numel() * workspace.element_size(),
                             _ptr(status), _stream(K))
    _check("sc_compress", code)


def compress_layers_workspace(L, B, Hkv, n, device) -> torch.Tensor:
    """Zero-initialised workspace for sc_compress_layers."""
    return torch.zeros(lib().sc_compress_layers_workspace_bytes(L, B, Hkv, n), dtype=torch.uint8, device=device)


def sc_compress_layers(Ks, Vs, plan: "ChunkPlan", tau, outs, workspace, status=None, flags=0):
    """Raw sc_compress_layers: ``Ks``/``Vs`` lists of [B, Hkv, n, d] tensors (same shape, dtype and strides),
    ``outs`` a list of CompressedLayer (same capacity), one per layer; every layer in one launch."""
    L = len(Ks)
    K0 = Ks[0]
    B, Hkv, n, d = K0.shape
    cap = outs[0].core_k.shape[2]
    rows = (_CompressLayer * L)()
    for l in range(L):
        K, V, o = Ks[l], Vs[l], outs[l]
        _need_cuda(K, V, o.core_k, o.core_v, o.count, o.core_len, o.assign)
        assert K.shape == K0.shape and V.shape == K0.shape and K.stride() == K0.stride() and V.stride() == K0.stride()
        assert K.dtype == K0.dtype and V.dtype == K0.dtype and K.stride(3) == 1 and o.core_k.shape[2] == cap
        assert o.core_k.is_contiguous() and o.core_v.is_contiguous() and o.count.is_contiguous()
        rows[l] = _CompressLayer(_ptr(K), _ptr(V), _ptr(o.core_k), _ptr(o.core_v), _ptr(o.count), _ptr(o.core_len),
                                 _ptr(o.assign))
    prm = _GscParams(float(tau), int(plan.max_chunk_len), int(flags))
    st = _Strides(K0.stride(0), K0.stride(1), K0.stride(2))
    code = lib().sc_compress_layers(rows, L, st, _dt(K0), B, Hkv, n, d, _ptr(plan.seg_off), _ptr(plan.seq_seg_off),
                                    _ptr(plan.n_seg), _ptr(plan.tile_seg), _ptr(plan.seq_tile_cnt), plan.n_tile_cap,
                                    ctypes.byref(prm), cap, _ptr(workspace),
                                    workspace.numel() * workspace.element_size(), _ptr(status), _stream(K0))
    _check("sc_compress_layers", code)


def sc_compress_budget(K, V, plan: "ChunkPlan", target_kept, tau_lo, tau_hi, n_grid, core_k, core_v, count, core_len,
                       tau_out, search_out, workspace, assign=None, status=None, flags=0):
    """Raw sc_compress_budget for one layer: the threshold is searched on the device for the kept fraction."""
    _need_cuda(K, V, core_k, core_v, count, core_len, assign, workspace, tau_out, search_out)
    B, Hkv, n, d = K.shape
    assert V.shape == K.shape and V.stride() == K.stride() and V.dtype == K.dtype and K.stride(3) == 1
    assert core_k.is_contiguous() and core_v.is_contiguous() and count.is_contiguous()
    assert tau_out is None or tau_out.dtype == torch.float32
    assert search_out is None or (search_out.dtype == torch.int32 and search_out.numel() >= 2)
    cap = core_k.shape[2]
    prm = _GscParams(0.0, int(plan.max_chunk_len), int(flags))
    bud = _Budget(float(target_kept), float(tau_lo), float(tau_hi), int(n_grid))
    st = _Strides(K.stride(0), K.stride(1), K.stride(2))
    code = lib().sc_compress_budget(_ptr(K), _ptr(V), st, _dt(K), B, Hkv, n, d, _ptr(plan.seg_off),
                                    _ptr(plan.seq_seg_off), _ptr(plan.n_seg), _ptr(plan.tile_seg),
                                    _ptr(plan.seq_tile_cnt), plan.n_tile_cap, ctypes.byref(prm), ctypes.byref(bud),
                                    _ptr(core_k), _ptr(core_v), _ptr(count), cap, _ptr(core_len), _ptr(assign),
                                    _ptr(tau_out), _ptr(search_out), _ptr(workspace),
                                    workspace.numel() * workspace.element_size(), _ptr(status), _stream(K))
    _check("sc_compress_budget", code)


def sc_compress_global(K, V, tau, core_k, core_v, count, core_len, workspace, assign=None, status=None, flags=0):
    """Raw sc_compress_global for one layer: Algorithm 1 over whole sequences (no chunking), then Eq. 3."""
    _need_cuda(K, V, core_k, core_v, count, core_len, assign, workspace)
    B, Hkv, n, d = K.shape
    assert V.shape == K.shape and V.stride() == K.stride() and V.dtype == K.dtype and K.stride(3) == 1
    assert core_k.is_contiguous() and core_v.is_contiguous() and count.is_contiguous()
    st = _Strides(K.stride(0), K.stride(1), K.stride(2))
    code = lib().sc_compress_global(_ptr(K), _ptr(V), st, _dt(K), B, Hkv, n, d, float(tau), int(flags), _ptr(core_k),
                                    _ptr(core_v), _ptr(count), core_k.shape[2], _ptr(core_len), _ptr(assign),
                                    _ptr(workspace), workspace.numel() * workspace.element_size(), _ptr(status),
                                    _stream(K))
    _check("sc_compress_global", code)


def sc_decode_attn(q, core_k, core_v, count, core_len, out, workspace, scale=0.0, status=None, flags=0):
    """Raw sc_decode_attn for one layer and one decode step."""
    _need_cuda(q, core_k, core_v, count, core_len, out, workspace)
    B, Hq, d = q.shape
    _, Hkv, cap, _ = core_k.shape
    assert q.is_contiguous() and out.is_contiguous() and core_k.is_contiguous() and core_v.is_contiguous()
    code = lib().sc_decode_attn(_ptr(q), _dt(q), B, Hq, Hkv, d, _ptr(core_k), _ptr(core_v), _ptr(count), cap,
                                _ptr(core_len), float(scale), int(flags), _ptr(out), _ptr(workspace),
                                workspace.numel() * workspace.element_size(), _ptr(status), _stream(q))
    _check("sc_decode_attn", code)


def sc_prefill_attn(q, core_k, core_v, count, core_len, out, scale=0.0, status=None, flags=0):
    """Raw sc_prefill_attn: Proportional Attention for a block of m queries per head, q/out [B, Hq, m, d]."""
    _need_cuda(q, core_k, core_v, count, core_len, out)
    B, Hq, m, d = q.shape
    _, Hkv, cap, _ = core_k.shape
    assert q.is_contiguous() and out.is_contiguous() and core_k.is_contiguous() and core_v.is_contiguous()
    assert out.shape == q.shape and out.dtype == q.dtype
    code = lib().sc_prefill_attn(_ptr(q), _dt(q), B, Hq, Hkv, m, d, _ptr(core_k), _ptr(core_v), _ptr(count), cap,
                                 _ptr(core_len), float(scale), int(flags), _ptr(out), _ptr(status), _stream(q))
    _check("sc_prefill_attn", code)


def sc_decode_attn_static(q, core_k, core_v, count, core_len, out, scale=0.0, status=None, flags=0):
    """Raw sc_decode_attn_static: one decode step with the scratch inside the library image.

    For callers that cannot allocate device memory (see the header); nothing is allocated here
    either -- every buffer, ``out`` included, is the caller's.  Calls on one GPU share the
    library's scratch array, so keep them on one stream.
    """
    _need_cuda(q, core_k, core_v, count, core_len, out)
    B, Hq, d = q.shape
    _, Hkv, cap, _ = core_k.shape
    assert q.is_contiguous() and out.is_contiguous() and core_k.is_contiguous() and core_v.is_contiguous()
    code = lib().sc_decode_attn_static(_ptr(q), _dt(q), B, Hq, Hkv, d, _ptr(core_k), _ptr(core_v), _ptr(count),
                                       cap, _ptr(core_len), float(scale), int(flags), _ptr(out), _ptr(status),
                                       _stream(q))
    _check("sc_decode_attn_static", code)


def sc_append(k_new, v_new, token_ids, delim_ids, max_chunk_len, tau, core_k, core_v, count, core_len, tail_len,
              attn_len, status=None):
    """Raw sc_append: one generated token per sequence joins one layer's cache (see the header)."""
    _need_cuda(k_new, v_new, token_ids, core_k, core_v, count, core_len, tail_len, attn_len, status)
    B, Hkv, d = k_new.shape
    cap = core_k.shape[2]
    assert k_new.is_contiguous() and v_new.is_contiguous() and core_k.is_contiguous() and core_v.is_contiguous()
    assert core_k.shape == (B, Hkv, cap, d) and token_ids.dtype == torch.int32 and token_ids.numel() == B
    delims = (_i32 * max(len(delim_ids), 1))(*[int(x) for x in delim_ids])
    code = lib().sc_append(_ptr(k_new), _ptr(v_new), _dt(k_new), B, Hkv, d, _ptr(token_ids), delims, len(delim_ids),
                           int(max_chunk_len), float(tau), _ptr(core_k), _ptr(core_v), _ptr(count), cap,
                           _ptr(core_len), _ptr(tail_len), _ptr(attn_len), _ptr(status), _stream(k_new))
    _check("sc_append", code)


def append_table(layers) -> torch.Tensor:
    """Device table for sc_append_layers: ``layers`` is a list of (k_new, v_new, core_k, core_v, count, core_len,
    tail_len, attn_len) tensor tuples, one per layer.  Returns an int64 tensor [L, 8] of their addresses;
    keep the tensors alive (and where they are) for as long as the table is used."""
    rows = [[t.data_ptr() for t in row] for row in layers]
    dev = layers[0][2].device
    return torch.tensor(rows, dtype=torch.int64).to(dev)


def sc_append_layers(table, k_new0, token_ids, delim_ids, max_chunk_len, tau, cap, status=None):
    """Raw sc_append_layers: one generated token per sequence joins every layer's cache in one launch.
    ``table`` from append_table; ``k_new0`` any one layer's k_new (for dtype and shape [B, Hkv, d])."""
    _need_cuda(table, k_new0, token_ids, status)
    B, Hkv, d = k_new0.shape
    assert table.dtype == torch.int64 and table.dim() == 2 and table.shape[1] == 8 and table.is_contiguous()
    delims = (_i32 * max(len(delim_ids), 1))(*[int(x) for x in delim_ids])
    code = lib().sc_append_layers(_ptr(table), table.shape[0], _dt(k_new0), B, Hkv, d, _ptr(token_ids), delims,
                                  len(delim_ids), int(max_chunk_len), float(tau), int(cap), _ptr(status),
                                  _stream(k_new0))
    _check("sc_append_layers", code)


# ------------------------------------------------------------------------- convenience wrappers


@dataclasses.dataclass
class ChunkPlan:
    """Device-resident result of sc_chunk, shared by every layer and KV head."""
    B: int
    n: int
    max_chunk_len: int
    seg_off: torch.Tensor
    seq_seg_off: torch.Tensor
    n_seg: torch.Tensor
    tile_seg: torch.Tensor
    seq_tile_cnt: torch.Tensor
    n_tile_cap: int
    status: torch.Tensor


@dataclasses.dataclass
class CompressedLayer:
    """Semantic cores of one layer: rows < core_len[b, h] of each head are valid."""
    core_k: torch.Tensor
    core_v: torch.Tensor
    count: torch.Tensor
    core_len: torch.Tensor
    assign: torch.Tensor | None = None


def check_status(status: torch.Tensor, where: str = "device status"):
    """Synchronising read of a device status word; raises on a device-reported error."""
    code = int(status.item())
    if code != SC_OK:
        raise ScError(where, code)


def chunk(token_ids: torch.Tensor, delim_ids, max_chunk_len: int = SC_MAX_CHUNK_LEN) -> ChunkPlan:
    """Allocate worst-case outputs and run sc_chunk.  Does not synchronise."""
    dev = token_ids.device
    B, n = token_ids.shape
    n_seg_cap, n_tile_cap = chunk_bounds(B, n)
    i32 = dict(dtype=torch.int32, device=dev)
    plan = ChunkPlan(B, n, max_chunk_len, torch.empty(n_seg_cap + 1, **i32), torch.empty(B + 1, **i32),
                     torch.empty(1, **i32), torch.empty((B, n_tile_cap + 1), **i32), torch.empty(max(B, 1), **i32),
                     n_tile_cap, torch.zeros(1, **i32))
    ws = torch.empty(lib().sc_chunk_workspace_bytes(B, n), dtype=torch.uint8, device=dev)
    sc_chunk(token_ids, delim_ids, max_chunk_len, plan.seg_off, plan.seq_seg_off, plan.n_seg, plan.tile_seg,
             plan.seq_tile_cnt, ws, plan.status)
    return plan


def chunk_fixed(token_ids: torch.Tensor, size: int = 64) -> ChunkPlan:
    """Fixed-size chunking, the paper's ablation arm (Table 4a compares semantic chunks with chunks of 64
    tokens): every `size` tokens form a chunk and delimiters play no role -- sc_chunk with an empty
    delimiter set and max_chunk_len = size.  The plan is used like any other."""
    if not 1 <= size <= SC_MAX_CHUNK_LEN:
        raise ValueError(f"chunk size must be in 1..{SC_MAX_CHUNK_LEN}")
    return chunk(token_ids, (), size)


def compress_workspace(B, Hkv, n, device) -> torch.Tensor:
    """Zero-initialised workspace for sc_compress (its status words and counters must start at zero)."""
    return torch.zeros(lib().sc_compress_workspace_bytes(B, Hkv, n), dtype=torch.uint8, device=device)


def compress(K, V, plan: ChunkPlan, tau: float, cap: int | None = None, want_assign: bool = False,
             workspace: torch.Tensor | None = None, flags: int = 0, out: CompressedLayer | None = None):
    """Allocate (or reuse ``out``) the core buffers and run sc_compress for one layer."""
    B, Hkv, n, d = K.shape
    dev = K.device
    cap = n if cap is None else cap
    if out is None:
        out = CompressedLayer(torch.empty((B, Hkv, cap, d), dtype=K.dtype, device=dev),
                              torch.empty((B, Hkv, cap, d), dtype=K.dtype, device=dev),
                              torch.zeros((B, Hkv, cap), dtype=torch.int32, device=dev),
                              torch.zeros((B, Hkv), dtype=torch.int32, device=dev),
                              torch.empty((B, Hkv, n), dtype=torch.int32, device=dev) if want_assign else None)
    if workspace is None:
        workspace = compress_workspace(B, Hkv, n, dev)
    sc_compress(K, V, plan, tau, out.core_k, out.core_v, out.count, out.core_len, out.assign, workspace,
                plan.status, flags)
    return out


def compress_to_budget(K, V, plan: ChunkPlan, target_kept: float, tau_lo: float = 0.5, tau_hi: float = 0.9,
                       n_grid: int = 17, cap: int | None = None, want_assign: bool = False, flags: int = 0):
    """Allocate the outputs and run sc_compress_budget.  Returns (CompressedLayer, tau [1] float32,
    search [2] int32: grid index, counting passes) -- all on the device, nothing synchronises."""
    B, Hkv, n, d = K.shape
    dev = K.device
    cap = n if cap is None else cap
    out = CompressedLayer(torch.empty((B, Hkv, cap, d), dtype=K.dtype, device=dev),
                          torch.empty((B, Hkv, cap, d), dtype=K.dtype, device=dev),
                          torch.zeros((B, Hkv, cap), dtype=torch.int32, device=dev),
                          torch.zeros((B, Hkv), dtype=torch.int32, device=dev),
                          torch.empty((B, Hkv, n), dtype=torch.int32, device=dev) if want_assign else None)
    ws = torch.zeros(lib().sc_compress_budget_workspace_bytes(B, Hkv, n), dtype=torch.uint8, device=dev)
    tau = torch.zeros(1, dtype=torch.float32, device=dev)
    search = torch.zeros(2, dtype=torch.int32, device=dev)
    sc_compress_budget(K, V, plan, target_kept, tau_lo, tau_hi, n_grid, out.core_k, out.core_v, out.count, out.core_len,
                       tau, search, ws, out.assign, plan.status, flags)
    return out, tau, search


def compress_global(K, V, tau: float, cap: int | None = None, want_assign: bool = False, flags: int = 0,
                    status: torch.Tensor | None = None, workspace: torch.Tensor | None = None):
    """Allocate the outputs (and the workspace) and run sc_compress_global for one layer."""
    B, Hkv, n, d = K.shape
    dev = K.device
    cap = n if cap is None else cap
    out = CompressedLayer(torch.empty((B, Hkv, cap, d), dtype=K.dtype, device=dev),
                          torch.empty((B, Hkv, cap, d), dtype=K.dtype, device=dev),
                          torch.zeros((B, Hkv, cap), dtype=torch.int32, device=dev),
                          torch.zeros((B, Hkv), dtype=torch.int32, device=dev),
                          torch.empty((B, Hkv, n), dtype=torch.int32, device=dev) if want_assign else None)
    if workspace is None:
        workspace = torch.empty(lib().sc_compress_global_workspace_bytes(B, Hkv, n), dtype=torch.uint8, device=dev)
    sc_compress_global(K, V, tau, out.core_k, out.core_v, out.count, out.core_len, workspace, out.assign, status, flags)
    return out


def prefill_attn(q, layer: CompressedLayer, out=None, scale: float = 0.0, status=None, causal: bool = False,
                 flags: int = 0, use_count: bool = True):
    """Proportional Attention of a block of queries q [B, Hq, m, d] over one layer's cores."""
    if out is None:
        out = torch.empty_like(q)
    sc_prefill_attn(q, layer.core_k, layer.core_v, layer.count if use_count else None, layer.core_len, out, scale,
                    status, flags | (SC_FLAG_CAUSAL_TAIL if causal else 0))
    return out


def decode_workspace(B, Hq, Hkv, d, cap, device) -> torch.Tensor:
    """Zero-initialised workspace for sc_decode_attn (its arrival counters must start at zero)."""
    return torch.zeros(lib().sc_decode_workspace_bytes(B, Hq, Hkv, d, cap), dtype=torch.uint8, device=device)


def decode_attn(q, layer: CompressedLayer, out=None, workspace=None, scale: float = 0.0, status=None, flags=0,
                use_count: bool = True):
    """One decode step of Proportional Attention over one layer's cores."""
    B, Hq, d = q.shape
    _, Hkv, cap, _ = layer.core_k.shape
    if out is None:
        out = torch.empty_like(q)
    if workspace is None:
        workspace = decode_workspace(B, Hq, Hkv, d, cap, q.device)
    sc_decode_attn(q, layer.core_k, layer.core_v, layer.count if use_count else None, layer.core_len, out,
                   workspace, scale, status, flags)
    return out

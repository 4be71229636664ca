"""SemantiCache oracle -- TEST INFRASTRUCTURE, not the product.

Thin numpy front end of ``semanticache_oracle.c`` (plain C, double accumulators,
written from the paper's Eq. 1-4 and Algorithm 1).  It shares nothing with the CUDA
path and must only be used by tests, the smoke check and the benchmark's
cpu-baseline leg.

Array conventions: bf16 tensors are numpy ``uint16`` arrays holding the raw bits,
fp32 tensors are ``float32``; K, V are ``[B, Hkv, n, d]`` (any strides with the last
axis contiguous), cores ``[B, Hkv, cap, d]``, counts ``[B, Hkv, cap]`` int32.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "semanticache_oracle.c")
_SO = os.path.join(_HERE, "libsemanticache_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the C oracle with gcc (OpenMP over the outer (b, head) loops only)."""
    if force or not os.path.exists(_SO) or os.path.getmtime(_SO) < os.path.getmtime(_SRC):
        cmd = ["gcc", "-O2", "-std=c11", "-ffp-contract=off", "-fopenmp", "-fPIC", "-shared",
               _SRC, "-o", _SO, "-lm"]
        subprocess.run(cmd, check=True)
    return _SO


def _load():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        _lib.oracle_chunk.restype = ctypes.c_int64
        _lib.oracle_sim.restype = ctypes.c_double
        _lib.oracle_f64_to_bf16.restype = ctypes.c_uint16
        _lib.oracle_f64_to_bf16.argtypes = [ctypes.c_double]
    return _lib


def _p(a):
    return ctypes.c_void_p(a.ctypes.data) if a is not None else ctypes.c_void_p(0)


def _dtype_code(a: np.ndarray) -> int:
    if a.dtype == np.uint16:
        return 0
    if a.dtype == np.float32:
        return 1
    raise TypeError(f"oracle takes uint16 (bf16 bits) or float32, got {a.dtype}")


def _kv_strides(K: np.ndarray):
    assert K.ndim == 4 and K.strides[3] == K.itemsize, "last axis must be contiguous"
    return tuple(ctypes.c_int64(s // K.itemsize) for s in K.strides[:3])


def bf16_bits_to_f64(a: np.ndarray) -> np.ndarray:
    """Decode raw bf16 bits (uint16) exactly."""
    return (a.astype(np.uint32) << 16).view(np.float32).astype(np.float64)


def f64_to_bf16_bits(x: float) -> int:
    return int(_load().oracle_f64_to_bf16(float(x)))


def num_threads() -> int:
    """Threads the OpenMP loops will use (the benchmark reports this as 'cores')."""
    env = os.environ.get("OMP_NUM_THREADS")
    if env:
        return int(env)
    return len(os.sched_getaffinity(0))


def chunk(token_ids: np.ndarray, delim_ids, max_chunk_len: int = 256):
    """Eq. 1.  Returns (seg_off[n_seg+1], seq_seg_off[B+1]) over the flattened token axis."""
    ids = np.ascontiguousarray(token_ids, dtype=np.int32)
    assert ids.ndim == 2
    B, n = ids.shape
    delim = np.ascontiguousarray(np.asarray(list(delim_ids), dtype=np.int32))
    seg_off = np.zeros(B * n + 1, dtype=np.int32)
    seq_seg_off = np.zeros(B + 1, dtype=np.int32)
    n_seg = _load().oracle_chunk(_p(ids), ctypes.c_int32(B), ctypes.c_int32(n), _p(delim),
                                 ctypes.c_int32(len(delim)), ctypes.c_int32(max_chunk_len),
                                 _p(seg_off), _p(seq_seg_off))
    return seg_off[: n_seg + 1].copy(), seq_seg_off


def sim(K2d: np.ndarray, a: int, b: int) -> float:
    """Eq. 2 between rows a and b of a contiguous [rows, d] array."""
    K2d = np.ascontiguousarray(K2d)
    return float(_load().oracle_sim(_p(K2d), ctypes.c_int32(_dtype_code(K2d)), ctypes.c_int64(a),
                                    ctypes.c_int64(b), ctypes.c_int32(K2d.shape[1])))


def gsc(K: np.ndarray, seg_off: np.ndarray, seq_seg_off: np.ndarray, tau: float):
    """Algorithm 1 per (b, head, segment).  Returns (assign[B,Hkv,n] int32, min |Sim-tau|)."""
    B, Hkv, n, d = K.shape
    sb, sh, sn = _kv_strides(K)
    assign = np.full((B, Hkv, n), -1, dtype=np.int32)
    margin = ctypes.c_double(0.0)
    seg_off = np.ascontiguousarray(seg_off, dtype=np.int32)
    seq_seg_off = np.ascontiguousarray(seq_seg_off, dtype=np.int32)
    _load().oracle_gsc(_p(K), ctypes.c_int32(_dtype_code(K)), sb, sh, sn, ctypes.c_int32(B),
                       ctypes.c_int32(Hkv), ctypes.c_int32(n), ctypes.c_int32(d), _p(seg_off),
                       _p(seq_seg_off), ctypes.c_float(tau), _p(assign), ctypes.byref(margin))
    return assign, margin.value


def merge(K: np.ndarray, V: np.ndarray, assign: np.ndarray, cap: int | None = None,
          seg_off: np.ndarray | None = None, seq_seg_off: np.ndarray | None = None):
    """Eq. 3.  Returns (core_k, core_v, count, core_len).

    With seg_off/seq_seg_off given, members of a seed are looked for inside the seed's
    segment only (same result, far fewer comparisons; used for timing)."""
    B, Hkv, n, d = K.shape
    assert V.shape == K.shape and V.dtype == K.dtype and V.strides == K.strides
    cap = n if cap is None else cap
    sb, sh, sn = _kv_strides(K)
    core_k = np.zeros((B, Hkv, cap, d), dtype=K.dtype)
    core_v = np.zeros((B, Hkv, cap, d), dtype=K.dtype)
    count = np.zeros((B, Hkv, cap), dtype=np.int32)
    core_len = np.zeros((B, Hkv), dtype=np.int32)
    assign = np.ascontiguousarray(assign, dtype=np.int32)
    common = (_p(K), _p(V), ctypes.c_int32(_dtype_code(K)), sb, sh, sn, ctypes.c_int32(B),
              ctypes.c_int32(Hkv), ctypes.c_int32(n), ctypes.c_int32(d))
    tail = (_p(assign), _p(core_k), _p(core_v), _p(count), ctypes.c_int32(cap), _p(core_len))
    if seg_off is None:
        _load().oracle_merge(*common, *tail)
    else:
        seg_off = np.ascontiguousarray(seg_off, dtype=np.int32)
        seq_seg_off = np.ascontiguousarray(seq_seg_off, dtype=np.int32)
        _load().oracle_merge_seg(*common, _p(seg_off), _p(seq_seg_off), *tail)
    return core_k, core_v, count, core_len


def attn(q: np.ndarray, core_k: np.ndarray, core_v: np.ndarray, count: np.ndarray | None,
         core_len: np.ndarray, scale: float | None = None) -> np.ndarray:
    """Eq. 4 for one decode step.  q: [B, Hq, d].  Returns float64 [B, Hq, d]."""
    q = np.ascontiguousarray(q)
    core_k = np.ascontiguousarray(core_k)
    core_v = np.ascontiguousarray(core_v)
    B, Hq, d = q.shape
    _, Hkv, cap, _ = core_k.shape
    assert Hq % Hkv == 0 and q.dtype == core_k.dtype == core_v.dtype
    if count is not None:
        count = np.ascontiguousarray(count, dtype=np.int32)
    core_len = np.ascontiguousarray(core_len, dtype=np.int32)
    scale = 1.0 / np.sqrt(d) if scale is None else scale
    out = np.zeros((B, Hq, d), dtype=np.float64)
    _load().oracle_attn(_p(q), ctypes.c_int32(_dtype_code(q)), ctypes.c_int32(B), ctypes.c_int32(Hq),
                        ctypes.c_int32(Hkv), ctypes.c_int32(d), _p(core_k), _p(core_v), _p(count),
                        ctypes.c_int32(cap), _p(core_len), ctypes.c_double(scale), _p(out))
    return out


def attn_multi(q: np.ndarray, core_k: np.ndarray, core_v: np.ndarray, count: np.ndarray | None,
               core_len: np.ndarray, scale: float | None = None, causal: bool = False) -> np.ndarray:
    """Eq. 4 with a block of m queries per head.  q: [B, Hq, m, d].  Returns float64 [B, Hq, m, d].

    causal: the last m rows of the cache are the queries' own tokens; query i sees rows
    t < core_len - (m - 1 - i)."""
    q = np.ascontiguousarray(q)
    core_k = np.ascontiguousarray(core_k)
    core_v = np.ascontiguousarray(core_v)
    B, Hq, m, d = q.shape
    _, Hkv, cap, _ = core_k.shape
    assert Hq % Hkv == 0 and q.dtype == core_k.dtype == core_v.dtype
    if count is not None:
        count = np.ascontiguousarray(count, dtype=np.int32)
    core_len = np.ascontiguousarray(core_len, dtype=np.int32)
    scale = 1.0 / np.sqrt(d) if scale is None else scale
    out = np.zeros((B, Hq, m, d), dtype=np.float64)
    _load().oracle_attn_multi(_p(q), ctypes.c_int32(_dtype_code(q)), ctypes.c_int32(B), ctypes.c_int32(Hq),
                              ctypes.c_int32(Hkv), ctypes.c_int32(m), ctypes.c_int32(d), _p(core_k), _p(core_v),
                              _p(count), ctypes.c_int32(cap), _p(core_len), ctypes.c_double(scale),
                              ctypes.c_int32(1 if causal else 0), _p(out))
    return out


def compress_global(K, V, tau, cap=None):
    """The paper's "no chunking" ablation arm (Table 4a): Algorithm 1 over each whole sequence as one
    chunk (delimiters get no special treatment), then Eq. 3.  Same products as ``compress``."""
    B, Hkv, n, _ = K.shape
    seg_off = (np.arange(B + 1, dtype=np.int64) * n).astype(np.int32)
    seq_seg_off = np.arange(B + 1, dtype=np.int32)
    assign, margin = gsc(K, seg_off, seq_seg_off, tau)
    core_k, core_v, count, core_len = merge(K, V, assign, cap)
    return dict(seg_off=seg_off, seq_seg_off=seq_seg_off, assign=assign, margin=margin,
                core_k=core_k, core_v=core_v, count=count, core_len=core_len)


def compress(token_ids, delim_ids, K, V, tau, max_chunk_len=256, cap=None):
    """chunk -> gsc -> merge, the whole compress stage.  Returns a dict of every product."""
    seg_off, seq_seg_off = chunk(token_ids, delim_ids, max_chunk_len)
    assign, margin = gsc(K, seg_off, seq_seg_off, tau)
    core_k, core_v, count, core_len = merge(K, V, assign, cap, seg_off, seq_seg_off)
    return dict(seg_off=seg_off, seq_seg_off=seq_seg_off, assign=assign, margin=margin,
                core_k=core_k, core_v=core_v, count=count, core_len=core_len)


def append(state: dict, token_ids_new, k_new: np.ndarray, v_new: np.ndarray, delim_ids, tau: float,
           max_chunk_len: int = 256) -> None:
    """One generated token per sequence joins one layer's cache, in place (the incremental reading).

    The paper compresses the prompt once and does not say what happens to generated tokens.  The
    reading taken: Eq. 1 keeps running over the generated stream, starting afresh behind the prompt.
    ``state`` holds ``core_k``/``core_v`` [B, Hkv, cap, d], ``count`` [B, Hkv, cap], ``core_len`` and
    ``tail_len`` [B, Hkv], and ``margin`` (the smallest |Sim - tau| met so far).  Rows
    [core_len, core_len + tail_len) are the tokens of the chunk that is still open, as they came.
    A token that is not a delimiter is stored behind them; a chunk is finished by reaching
    ``max_chunk_len`` tokens or by a delimiter, which then becomes a core of its own.  A finished
    chunk goes through ``gsc`` and ``merge`` as one segment and its cores replace its first rows.
    """
    ck, cv, cnt, clen, tlen = (state[k] for k in ("core_k", "core_v", "count", "core_len", "tail_len"))
    B, Hkv, cap, d = ck.shape
    delims = set(int(x) for x in delim_ids)

    def finish(b, h):
        cl, tl = int(clen[b, h]), int(tlen[b, h])
        if tl >= 2:
            Kt = np.ascontiguousarray(ck[b:b + 1, h:h + 1, cl:cl + tl])
            Vt = np.ascontiguousarray(cv[b:b + 1, h:h + 1, cl:cl + tl])
            seg_off, seq_seg_off = np.array([0, tl], dtype=np.int32), np.array([0, 1], dtype=np.int32)
            assign, margin = gsc(Kt, seg_off, seq_seg_off, tau)
            pk, pv, pc, pl = merge(Kt, Vt, assign, tl, seg_off, seq_seg_off)
            p = int(pl[0, 0])
            ck[b, h, cl:cl + p], cv[b, h, cl:cl + p], cnt[b, h, cl:cl + p] = pk[0, 0, :p], pv[0, 0, :p], pc[0, 0, :p]
            state["margin"] = min(state.get("margin", np.inf), margin)
            tl = p
        clen[b, h], tlen[b, h] = cl + tl, 0

    for b in range(B):
        is_delim = int(token_ids_new[b]) in delims
        for h in range(Hkv):
            if int(clen[b, h]) + int(tlen[b, h]) >= cap:
                raise OverflowError(f"no free row in sequence {b}, head {h}")
            if is_delim:
                if tlen[b, h] > 0:
                    finish(b, h)
                row = int(clen[b, h])
                ck[b, h, row], cv[b, h, row], cnt[b, h, row] = k_new[b, h], v_new[b, h], 1
                clen[b, h] = row + 1
            else:
                row = int(clen[b, h]) + int(tlen[b, h])
                ck[b, h, row], cv[b, h, row], cnt[b, h, row] = k_new[b, h], v_new[b, h], 1
                tlen[b, h] += 1
                if tlen[b, h] == max_chunk_len:
                    finish(b, h)


def tau_grid(tau_lo: float, tau_hi: float, n_grid: int) -> np.ndarray:
    """The thresholds a budget search may choose from: tau_i = tau_lo + i * ((tau_hi - tau_lo) / (n_grid - 1)),
    every operation rounded to float32 (the threshold of Algorithm 1 is a float32 parameter)."""
    lo, hi = np.float32(tau_lo), np.float32(tau_hi)
    step = np.float32(hi - lo) / np.float32(n_grid - 1)
    return np.array([np.float32(lo + np.float32(np.float32(i) * step)) for i in range(n_grid)], dtype=np.float32)


def budget(token_ids, delim_ids, K, V, target_kept: float, tau_lo: float, tau_hi: float, n_grid: int,
           max_chunk_len: int = 256, cap=None):
    """Compress one layer to a KV budget (the kept fractions of Table 1; Table 4b: a lower threshold keeps less).

    The paper states budgets and a threshold but not how one is turned into the other.  The reading
    taken: the threshold is searched on a grid of ``n_grid`` values between ``tau_lo`` and ``tau_hi``
    for the one whose number of cores (all sequences and heads of the layer together) comes nearest
    to ``target_kept`` times the number of tokens, assuming that the count does not fall as the
    threshold rises:
      1. the two ends are evaluated; if even the lowest threshold keeps at least the target, it is
         chosen; if even the highest keeps less than the target, that one is;
      2. otherwise the interval is halved (middle index, rounded down) until its ends are adjacent,
         keeping "fewer than the target" at the lower end and "at least the target" at the upper;
      3. of the two ends the one whose count is nearer the target is chosen, the lower on a tie.
    Returns the compress products at the chosen threshold plus ``tau``, ``index``, ``target_cores``
    and ``visited`` (list of (index, cores) in evaluation order)."""
    seg_off, seq_seg_off = chunk(token_ids, delim_ids, max_chunk_len)
    B, Hkv, n, _ = K.shape
    grid = tau_grid(tau_lo, tau_hi, n_grid)
    target = int(np.floor(float(target_kept) * (B * Hkv * n) + 0.5))
    pos = np.arange(n, dtype=np.int32)
    visited, margins = [], []

    def cores(i):
        assign, margin = gsc(K, seg_off, seq_seg_off, float(grid[i]))
        c = int((assign == pos).sum())
        visited.append((i, c))
        margins.append(margin)
        return c

    lo, hi = 0, n_grid - 1
    k_lo, k_hi = cores(lo), cores(hi)
    if k_lo >= target:
        pick = lo
    elif k_hi < target:
        pick = hi
    else:
        while hi - lo > 1:
            mid = (lo + hi) // 2
            k = cores(mid)
            if k >= target:
                hi, k_hi = mid, k
            else:
                lo, k_lo = mid, k
        pick = hi if (k_hi - target) < (target - k_lo) else lo
    out = compress(token_ids, delim_ids, K, V, float(grid[pick]), max_chunk_len, cap)
    out.update(tau=float(grid[pick]), index=pick, target_cores=target, visited=visited,
               search_margin=min(margins))
    return out

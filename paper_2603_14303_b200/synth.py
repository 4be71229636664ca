"""Seeded synthetic workloads shaped like Llama / Mistral / Qwen2 KV caches.

This module only draws random inputs (token ids with delimiters, clustered keys,
Gaussian values and queries).  It contains none of the method's arithmetic and is the
one piece of code that both the CUDA path's callers and the test oracle's callers use.

Recipe (per workload):
  * token ids: runs of non-delimiter tokens whose lengths follow the workload's gap law
    (Poisson(mean) or a clipped lognormal), each run followed by one delimiter id drawn
    uniformly from the delimiter set; non-delimiter ids are uniform over the rest of the
    vocabulary; every sequence has exactly n tokens.
  * keys: per (layer, sequence, KV head, run) a few unit-norm centroids; each token of the
    run picks one and adds isotropic Gaussian noise whose expected norm is ``sigma``
    (per-component std sigma/sqrt(d)); with noise_reading="literal" the per-component std
    is sigma itself.  Delimiter tokens get their own random unit key.
  * values and queries: N(0, 1) per component.
Everything is rounded once to the storage dtype; those bytes are the input of both sides.
"""
from __future__ import annotations

import dataclasses
import math

import numpy as np
import torch

DELIMS = (13, 29889, 29892)


@dataclasses.dataclass(frozen=True)
class Workload:
    name: str
    B: int
    n: int
    L: int
    Hkv: int
    Hq: int
    d: int = 128
    vocab: int = 32000
    delims: tuple = DELIMS
    gap: tuple = ("poisson", 24.0)          # or ("lognormal", median, sigma_ln, max_len)
    centroids: tuple = ("uniform", 6)       # or ("ratio", r): max(1, round((l+1)/r) - 1)
    sigma: float = 0.15
    noise_reading: str = "norm"             # "norm" | "literal"
    tau: float = 0.7
    max_chunk_len: int = 256
    decode_steps: int = 32
    seed: int = 0
    dtype: str = "bf16"                     # "bf16" | "f32"

    @property
    def G(self) -> int:
        return self.Hq // self.Hkv

    def replace(self, **kw) -> "Workload":
        return dataclasses.replace(self, **kw)


def config(i: int, **kw) -> Workload:
    """The five benchmark configurations (0 = toy ... 4 = ratio / chunk-size sweep base)."""
    if i == 0:
        w = Workload("cfg0-toy", B=1, n=2048, L=1, Hkv=8, Hq=32, gap=("poisson", 24.0),
                     centroids=("uniform", 6), decode_steps=32, seed=0)
    elif i == 1:
        w = Workload("cfg1-llama3-8b-32k", B=1, n=32768, L=32, Hkv=8, Hq=32, gap=("poisson", 20.0),
                     centroids=("uniform", 8), decode_steps=256, seed=1)
    elif i == 2:
        w = Workload("cfg2-mistral-7b-16x16k", B=16, n=16384, L=32, Hkv=8, Hq=32,
                     gap=("lognormal", 18.0, 0.8, 256), centroids=("uniform", 8),
                     decode_steps=128, seed=2)
    elif i == 3:
        w = Workload("cfg3-qwen2-7b-128k", B=1, n=131072, L=28, Hkv=4, Hq=28, gap=("poisson", 30.0),
                     centroids=("uniform", 8), decode_steps=512, seed=3)
    elif i == 4:
        w = Workload("cfg4-llama3-8b-4x64k", B=4, n=65536, L=32, Hkv=8, Hq=32, gap=("poisson", 32.0),
                     centroids=("ratio", 4.0), decode_steps=64, seed=4)
    else:
        raise ValueError(i)
    return w.replace(**kw) if kw else w


def _draw_gap(rng: np.random.Generator, gap: tuple) -> int:
    if gap[0] == "poisson":
        return int(rng.poisson(gap[1]))
    if gap[0] == "lognormal":
        _, median, sig, mx = gap
        return int(min(max(round(math.exp(rng.normal(math.log(median), sig))), 1), mx))
    if gap[0] == "fixed":
        return int(gap[1])
    raise ValueError(gap)


def token_ids(w: Workload):
    """Token ids and the generator's own record of the runs it drew.

    Returns (ids int32 [B, n], run_id int64 [B, n], run_len list[np.ndarray]); run_id is
    -1 at delimiter tokens, else the index of the run inside its sequence.  Always on CPU.
    """
    ids = np.empty((w.B, w.n), dtype=np.int32)
    run_id = np.empty((w.B, w.n), dtype=np.int64)
    run_lens = []
    delims = np.asarray(w.delims, dtype=np.int32)
    # non-delimiter ids: draw from [0, vocab - n_delim) and step over the delimiter ids
    sorted_delims = np.sort(delims)
    for b in range(w.B):
        rng = np.random.default_rng([w.seed, 7919, b])
        t, r, lens = 0, 0, []
        while t < w.n:
            g = min(_draw_gap(rng, w.gap), w.n - t)
            if g > 0:
                raw = rng.integers(0, w.vocab - len(delims), size=g, dtype=np.int64)
                for dl in sorted_delims:
                    raw = raw + (raw >= dl)
                ids[b, t:t + g] = raw
                run_id[b, t:t + g] = r
                lens.append(g)
                r += 1
                t += g
            if t < w.n:
                ids[b, t] = delims[rng.integers(0, len(delims))]
                run_id[b, t] = -1
                t += 1
        run_lens.append(np.asarray(lens, dtype=np.int64))
    return torch.from_numpy(ids), torch.from_numpy(run_id), run_lens


def _torch_dtype(w: Workload):
    return torch.bfloat16 if w.dtype == "bf16" else torch.float32


def layer_kv(w: Workload, layer: int, run_id: torch.Tensor, run_lens, device="cpu"):
    """K, V of one layer: [B, Hkv, n, d] in the workload's dtype, on ``device``.

    The random stream depends on (seed, layer, b) and on the device type, so a caller
    that needs the same bytes on both sides generates once and copies.
    """
    dev = torch.device(device)
    dt = _torch_dtype(w)
    K = torch.empty((w.B, w.Hkv, w.n, w.d), dtype=dt, device=dev)
    V = torch.empty_like(K)
    comp_std = w.sigma / math.sqrt(w.d) if w.noise_reading == "norm" else w.sigma
    for b in range(w.B):
        g = torch.Generator(device=dev)
        g.manual_seed((w.seed * 1000003 + layer * 10007 + b * 101 + 17) & 0x7FFFFFFFFFFFFFFF)
        rid = run_id[b].to(dev)
        is_delim = rid < 0
        lens = torch.as_tensor(run_lens[b], device=dev)
        n_runs = max(int(lens.numel()), 1)
        if w.centroids[0] == "uniform":
            cmax = int(w.centroids[1])
            c_run = torch.randint(1, cmax + 1, (w.Hkv, n_runs), generator=g, device=dev)
        else:
            r = float(w.centroids[1])
            c1 = torch.clamp(torch.round((lens.double() + 1.0) / r) - 1.0, min=1.0).long()
            if c1.numel() == 0:
                c1 = torch.ones(1, dtype=torch.long, device=dev)
            cmax = int(c1.max().item())
            c_run = c1.unsqueeze(0).expand(w.Hkv, n_runs).contiguous()
        cent = torch.randn((w.Hkv, n_runs, cmax, w.d), generator=g, device=dev)
        cent = cent / cent.norm(dim=-1, keepdim=True)
        rid_c = rid.clamp(min=0)
        u = torch.rand((w.Hkv, w.n), generator=g, device=dev)
        cidx = torch.minimum((u * c_run[:, rid_c]).long(), c_run[:, rid_c] - 1)
        h_ix = torch.arange(w.Hkv, device=dev).unsqueeze(1).expand(w.Hkv, w.n)
        k = cent[h_ix, rid_c.unsqueeze(0).expand(w.Hkv, w.n), cidx]          # [Hkv, n, d]
        k = k + comp_std * torch.randn((w.Hkv, w.n, w.d), generator=g, device=dev)
        kd = torch.randn((w.Hkv, w.n, w.d), generator=g, device=dev)
        kd = kd / kd.norm(dim=-1, keepdim=True)
        k = torch.where(is_delim.view(1, w.n, 1), kd, k)
        K[b] = k.to(dt)
        V[b] = torch.randn((w.Hkv, w.n, w.d), generator=g, device=dev).to(dt)
    return K, V


def queries(w: Workload, step: int, layer: int, device="cpu") -> torch.Tensor:
    """Decode-step queries [B, Hq, d] ~ N(0, 1) in the workload's dtype."""
    dev = torch.device(device)
    g = torch.Generator(device=dev)
    g.manual_seed((w.seed * 7368787 + step * 65537 + layer * 257 + 3) & 0x7FFFFFFFFFFFFFFF)
    return torch.randn((w.B, w.Hq, w.d), generator=g, device=dev).to(_torch_dtype(w))


def generated_stream(w: Workload, m: int, layer: int = 0, mean_gap: float = 20.0, n_centroids: int = 5):
    """A seeded stand-in for m generated tokens per sequence: ids [B, m] int32 with a delimiter after
    Poisson(mean_gap) ordinary tokens, and this layer's K, V [B, Hkv, m, d] in the workload's dtype
    (keys: one of n_centroids unit directions per head plus noise of RMS norm w.sigma; values N(0, 1))."""
    rng = np.random.default_rng((w.seed * 1000003 + layer * 9176 + 77) & 0x7FFFFFFF)
    ids = rng.integers(1000, w.vocab, size=(w.B, m)).astype(np.int32)
    ids[np.isin(ids, np.array(w.delims))] = 999
    for b in range(w.B):
        t = int(rng.poisson(mean_gap))
        while t < m:
            ids[b, t] = w.delims[int(rng.integers(len(w.delims)))]
            t += 1 + int(rng.poisson(mean_gap))
    cent = rng.normal(size=(w.Hkv, n_centroids, w.d))
    cent /= np.linalg.norm(cent, axis=-1, keepdims=True)
    pick = rng.integers(0, n_centroids, size=(w.B, w.Hkv, m))
    K = cent[np.arange(w.Hkv)[None, :, None], pick] + w.sigma / math.sqrt(w.d) * rng.normal(size=(w.B, w.Hkv, m, w.d))
    V = rng.normal(size=(w.B, w.Hkv, m, w.d))
    dt = _torch_dtype(w)
    return torch.from_numpy(ids), torch.from_numpy(K).to(dt), torch.from_numpy(V).to(dt)


def to_numpy_bits(t: torch.Tensor) -> np.ndarray:
    """CPU numpy view for the test oracle: bf16 -> uint16 raw bits, others unchanged."""
    t = t.detach().cpu()
    if t.dtype == torch.bfloat16:
        return t.contiguous().view(torch.int16).numpy().view(np.uint16)
    return t.contiguous().numpy()

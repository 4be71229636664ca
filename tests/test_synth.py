"""The synthetic workloads have the structure the recipe promises (CPU only)."""
import numpy as np
import pytest
import torch

import oracle
from paper_2603_14303_b200 import synth


def test_token_ids_shape_delimiters_and_runs():
    w = synth.config(0)
    ids, run_id, run_lens = synth.token_ids(w)
    assert ids.shape == (1, 2048) and ids.dtype == torch.int32
    isd = np.isin(ids.numpy(), w.delims)
    assert np.array_equal(isd, run_id.numpy() < 0)
    assert 60 <= isd.sum() <= 110                      # ~2048/25 delimiters
    assert int(run_lens[0].sum()) + int(isd.sum()) == w.n
    assert ids.min() >= 0 and ids.max() < w.vocab
    again, _, _ = synth.token_ids(w)
    assert torch.equal(ids, again)


def test_lognormal_gaps_are_clipped():
    w = synth.config(2, B=2, n=4096)
    _, _, run_lens = synth.token_ids(w)
    allr = np.concatenate(run_lens)
    assert allr.min() >= 1 and allr.max() <= 256
    assert 12 <= np.median(allr) <= 26


@pytest.mark.parametrize("reading,lo,hi", [("norm", 0.15, 0.40), ("literal", 0.97, 1.0)])
def test_cfg0_kept_fraction_and_threshold_margin(reading, lo, hi):
    w = synth.config(0, noise_reading=reading)
    ids, run_id, run_lens = synth.token_ids(w)
    K, V = synth.layer_kv(w, 0, run_id, run_lens)
    assert K.dtype == torch.bfloat16 and K.shape == (1, 8, 2048, 128)
    r = oracle.compress(ids.numpy(), w.delims, synth.to_numpy_bits(K), synth.to_numpy_bits(V), w.tau)
    kept = r["core_len"].sum() / (w.Hkv * w.n)
    assert lo <= kept <= hi
    assert r["margin"] > 1e-3, "similarities sit clear of the threshold"


def test_layers_and_steps_differ_and_are_reproducible():
    w = synth.config(0, n=256)
    ids, run_id, run_lens = synth.token_ids(w)
    K0, _ = synth.layer_kv(w, 0, run_id, run_lens)
    K0b, _ = synth.layer_kv(w, 0, run_id, run_lens)
    K1, _ = synth.layer_kv(w, 1, run_id, run_lens)
    assert torch.equal(K0, K0b) and not torch.equal(K0, K1)
    assert not torch.equal(synth.queries(w, 0, 0), synth.queries(w, 1, 0))
    assert torch.equal(synth.queries(w, 3, 0), synth.queries(w, 3, 0))


def test_ratio_centroids_hit_target_reduction():
    w = synth.config(4, B=1, n=4096, gap=("poisson", 32.0), centroids=("ratio", 4.0))
    ids, run_id, run_lens = synth.token_ids(w)
    K, V = synth.layer_kv(w, 0, run_id, run_lens)
    r = oracle.compress(ids.numpy(), w.delims, synth.to_numpy_bits(K[:, :2]), synth.to_numpy_bits(V[:, :2]), w.tau)
    kept = r["core_len"].sum() / (2 * w.n)
    assert 0.2 <= kept <= 0.3

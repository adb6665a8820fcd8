"""The seeded input generators: determinism, formats, distributions."""
import numpy as np
import torch

from paper_2510_18239_b200 import synth


def test_bf16_round_trip_matches_torch():
    x = np.random.default_rng(0).normal(size=4096).astype(np.float32) * 3
    x[:4] = [0.0, -0.0, 1.0, 65504.0]
    bits = synth.f32_to_bf16_bits(x)
    ref = torch.from_numpy(x).to(torch.bfloat16)
    assert np.array_equal(bits.view(np.int16), ref.view(torch.int16).numpy())
    assert np.array_equal(synth.bf16_bits_to_f32(bits), ref.float().numpy())


def test_streams_are_deterministic_and_independent():
    wl = synth.named_workloads()["tiny_fp32"]
    a, b = synth.make_inputs(wl, seed=0), synth.make_inputs(wl, seed=0)
    for k in a:
        assert np.array_equal(a[k], b[k]), k
    c = synth.make_inputs(wl, seed=1)
    assert not np.array_equal(a["table"], c["table"])
    assert a["table"].dtype == np.float32 and a["table"].shape == (768, 64)
    assert abs(a["table"].var() - 1 / 64) < 2e-3
    # one row per use
    ids = np.concatenate([a["hist_ids"], a["cand_ids"]])
    assert ids.size == 768 and np.unique(ids).size == 768
    assert a["lengths"].tolist() == [64] * 4


def test_zipf_skew_and_range():
    ids = synth.zipf_ids(0, "hist_ids", 200_000, 100_000, 1.1)
    assert ids.dtype == np.int32 and ids.min() >= 0 and ids.max() < 100_000
    _, counts = np.unique(ids, return_counts=True)
    top = np.sort(counts)[::-1]
    # P(rank 1) / P(rank 2) = 2^1.1 ~ 2.14 ; top-1000 ranks carry most of the mass
    assert 1.8 < top[0] / top[1] < 2.6
    assert top[:1000].sum() / ids.size > 0.6


def test_ragged_lengths_and_bf16_workload():
    wl = synth.named_workloads()["production_ragged"].replace(B=64, V=5000, C=16)
    inp = synth.make_inputs(wl, seed=3)
    ln = inp["lengths"]
    assert ln.min() >= 1024 and ln.max() <= 4096 and ln.dtype == np.int32
    assert inp["hist_ids"].size == int(ln.sum()) and inp["cand_ids"].size == 64 * 16
    assert inp["table"].dtype == np.uint16 and inp["Wq"].shape == (4, 256, 256)
    w = synth.storage_to_f64(inp["Wg"], wl.dtype)
    assert abs(w.var() - 1 / 256) < 1e-4
    assert abs(synth.storage_to_f64(inp["links"], wl.dtype).std() - 1.0) < 0.05

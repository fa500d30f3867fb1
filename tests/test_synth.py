"""Host-side checks of the seeded input generator (storage formats, laws, sharding)."""

import numpy as np
import pytest
import torch

from paper_2607_13332_b200 import synth


def test_bf16_rounding_matches_torch():
    rng = np.random.default_rng(0)
    x = np.concatenate([rng.standard_normal(20000).astype(np.float32) * 3,
                        np.array([0.0, -0.0, 1.0, 1.00390625, 1.01171875, 3.3895314e38, 1e-40],
                                 dtype=np.float32)])
    bits = synth.f32_to_bf16_bits(x)
    ref = torch.from_numpy(x).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    np.testing.assert_array_equal(bits, ref)
    back = synth.bf16_bits_to_f32(bits)
    np.testing.assert_array_equal(back, torch.from_numpy(x).to(torch.bfloat16).float().numpy())


def test_generator_is_deterministic_and_shaped():
    wl = synth.TINY.scaled(batch=1)
    a = synth.codec_inputs(wl, seed=3)
    b = synth.codec_inputs(wl, seed=3)
    c = synth.codec_inputs(wl, seed=4)
    for name in ("U", "E", "P", "ids", "Z0", "X", "G"):
        np.testing.assert_array_equal(a[name], b[name])
    assert not np.array_equal(a["X"], c["X"])
    assert a["X"].shape == (1024, 512) and a["U"].shape == (512, 8)
    assert a["E"].shape == (1024, 512) and a["P"].shape == (1024, 512)
    assert a["ids"].dtype == np.int32 and a["ids"].min() >= 0 and a["ids"].max() < 1024
    assert abs(float(np.std(a["E"])) - 0.02) < 1e-3
    assert abs(float(np.std(a["G"])) - 1e-2) < 1e-3


def test_zipf_ids_follow_the_law():
    V, n, s = 5000, 200000, 1.1
    ids = synth.zipf_ids(n, V, s, seed=5, scatter=False)
    assert ids.min() >= 0 and ids.max() < V
    harmonic = np.sum(np.arange(1, V + 1, dtype=np.float64) ** -s)
    counts = np.bincount(ids, minlength=V)
    for r in (1, 2, 10):
        expect = n * r ** -s / harmonic
        assert abs(counts[r - 1] - expect) < 5 * np.sqrt(expect)
    scattered = synth.zipf_ids(n, V, s, seed=5, scatter=True)
    assert np.array_equal(np.sort(np.bincount(scattered, minlength=V)), np.sort(counts))


def test_sinusoid_rows():
    P = synth.sinusoidal_positions(8, 6)
    np.testing.assert_allclose(P[0], [0, 1, 0, 1, 0, 1])
    assert abs(P[3, 0] - np.sin(3.0)) < 1e-15 and abs(P[3, 1] - np.cos(3.0)) < 1e-15


@pytest.mark.parametrize("n,world", [(10, 1), (10, 3), (7, 8), (65536, 8)])
def test_shard_tokens_partitions(n, world):
    covered = []
    for r in range(world):
        covered.extend(synth.shard_tokens(n, r, world))
    assert covered == list(range(n))
    sizes = [len(synth.shard_tokens(n, r, world)) for r in range(world)]
    assert max(sizes) - min(sizes) <= 1

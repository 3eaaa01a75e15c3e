"""Host-side checks of the seeded workload generators (no CUDA)."""
import numpy as np
import pytest

from paper_2607_06763_b200 import synth


@pytest.mark.parametrize("T", [1, 2, 16, 64, 200, 256])
def test_geo_tree_shape(T):
    rng = np.random.default_rng(T)
    t = synth.tree_geo(rng, T)
    assert len(t) == T and t[0] == -1 and all(-1 <= t[i] < i for i in range(T))
    d = synth.depths(t)
    assert d.max() <= synth.MAX_DEPTH and np.all(np.diff(d) >= 0)  # BFS numbering: depth never decreases
    assert np.bincount(t[t >= 0], minlength=T).max() <= synth.FANOUT


def test_bestfirst_and_small_trees():
    rng = np.random.default_rng(5)
    t = synth.tree_bestfirst(rng, 64)
    assert len(t) == 64 and all(-1 <= t[i] < i for i in range(64)) and synth.depths(t).max() <= 16
    s = synth.tree_small_uniform(rng, 8, 3, 3)
    assert len(s) == 8 and synth.depths(s).max() == 3 and np.bincount(s[s >= 0]).max() <= 3


def test_bf16_round_trip_matches_torch():
    import torch
    x = np.random.default_rng(0).standard_normal(4096).astype(np.float32) * 37.0
    bits = synth.f32_to_bf16_bits(x)
    want = torch.from_numpy(x).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    np.testing.assert_array_equal(bits, want)
    np.testing.assert_array_equal(synth.f32_to_bf16_bits(synth.bf16_bits_to_f32(bits)), bits)


@pytest.mark.parametrize("idx", [0, 1, 4])
def test_configs_are_seeded_and_consistent(idx):
    a, b = synth.config(idx, 0), synth.config(idx, 0)
    for name in ("S0", "q", "k", "v", "g", "beta", "parent", "node_offsets", "path", "path_offsets"):
        np.testing.assert_array_equal(getattr(a, name), getattr(b, name))
    assert not np.array_equal(a.S0, synth.config(idx, 1).S0)
    assert a.node_offsets[0] == 0 and a.node_offsets[-1] == len(a.parent) == a.q.shape[0]
    qn = np.linalg.norm(a.f64("q"), axis=-1)
    assert np.allclose(qn, 1.0, atol=1e-2)
    assert np.all(a.f64("g") <= 0) and np.all((a.f64("beta") >= 0) & (a.f64("beta") <= 1))
    for s in range(a.n_seq):
        p = a.path[a.path_offsets[s]:a.path_offsets[s + 1]]
        par = a.parent[a.node_offsets[s]:a.node_offsets[s + 1]]
        assert all(par[n] == (-1 if t == 0 else p[t - 1]) for t, n in enumerate(p))


def test_config1_bytes_match_the_stated_figure():
    w = synth.config(1)
    assert w.algorithmic_bytes() == 5775360  # 2*2 MiB state + q,k 0.5 MiB + v 0.5 MiB + o 0.5 MiB + g,beta 8 KiB

"""GPU parity: the CUDA library (through the C ABI) against the fp64 oracle, element by element."""
import numpy as np
import pytest

from paper_2607_06763_b200 import synth

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def tl(cuda_device):
    from tests import gdn_testlib
    return gdn_testlib


def _check_full(tl, w, what, max_depth=16):
    """verify + commit on the GPU, whole-workload oracle comparison."""
    dc = tl.DeviceCase(w, max_depth=max_depth)
    S0_before = dc.S0.clone()
    assert dc.verify() == 0
    assert dc.device_status() == 0
    assert bool((dc.S0 == S0_before).all()), "verify must leave the state bit-identical"
    ref = tl.oracle_verify(w)
    tl.assert_close_per_head(dc.o_host(), ref, w.node_offsets, what + " o", bf16_out=tl.is_bf16_out(w))
    assert dc.commit() == 0
    assert dc.device_status() == 0
    tl.assert_state_close(dc.S0.cpu().numpy().astype(np.float64), tl.oracle_commit(w), what=what + " S_new")
    return dc


def _check_sampled(tl, w, seqs, what):
    """verify + commit on the full workload; the oracle evaluates only the sampled sequences."""
    dc = tl.DeviceCase(w)
    assert dc.verify() == 0
    assert dc.device_status() == 0
    o = dc.o_host()
    assert np.all(np.isfinite(o))
    sub, nodes = tl.sub_workload(w, seqs)
    tl.assert_close_per_head(o[nodes], tl.oracle_verify(sub), sub.node_offsets, what + " o",
                             bf16_out=tl.is_bf16_out(w))
    assert dc.commit() == 0
    assert dc.device_status() == 0
    S = dc.S0.cpu().numpy().astype(np.float64)
    assert np.all(np.isfinite(S))
    tl.assert_state_close(S[list(seqs)], tl.oracle_commit(sub), what=what + " S_new")
    # sequences with an empty accepted path keep their state bit for bit
    for b in range(w.n_seq):
        if w.path_offsets[b + 1] == w.path_offsets[b]:
            np.testing.assert_array_equal(S[b].astype(np.float32), w.S0[b])


@pytest.mark.parametrize("rep", [0, 1, 2])
def test_config0_tiny_fp32(tl, rep):
    _check_full(tl, synth.config(0, rep), f"cfg0 rep{rep}")


@pytest.mark.parametrize("rep", [0, 1, 2])
@pytest.mark.parametrize("out_dtype", [synth.BF16, synth.F32])
def test_config1_single_layer(tl, rep, out_dtype):
    _check_full(tl, synth.config(1, rep, out_dtype=out_dtype), f"cfg1 rep{rep} {out_dtype}")


# The four large configurations, whole: every layer slot / sequence of every repetition goes through the oracle, by
# the separate entry points (verify, then commit) and by the fused one (the same repetition as the previous step,
# the next repetition as the new trees); repetition 0 also with fp32 outputs.
BIG_CONFIGS = {"cfg1x48": 5, "cfg2": 2, "cfg3": 3, "cfg4": 4}


@pytest.mark.parametrize("rep", [0, 1, 2])
@pytest.mark.parametrize("name", sorted(BIG_CONFIGS))
def test_big_config_whole_workload_separate_calls(tl, name, rep):
    _check_full(tl, synth.config(BIG_CONFIGS[name], rep), f"{name} rep{rep}")


@pytest.mark.parametrize("rep", [0, 1, 2])
@pytest.mark.parametrize("name", sorted(BIG_CONFIGS))
def test_big_config_whole_workload_fused_call(tl, name, rep):
    prev, new = synth.config(BIG_CONFIGS[name], rep), synth.config(BIG_CONFIGS[name], (rep + 1) % 3)
    if prev.n_seq != new.n_seq:
        pytest.skip("repetitions differ in batch size")
    _fused_case(tl, prev, new, f"fused {name} rep{rep}")


@pytest.mark.parametrize("name", sorted(BIG_CONFIGS))
def test_big_config_whole_workload_fp32_outputs(tl, name):
    _check_full(tl, synth.config(BIG_CONFIGS[name], 0, out_dtype=synth.F32), f"{name} f32 out")


# ------------------------------------------------------------------ edge shapes
def _edge_trees():
    rng = np.random.default_rng(7)
    deep = synth.tree_chain(16)
    return {
        "single": [np.array([-1], np.int32)],
        "star": [synth.tree_star(37)],
        "chain16": [deep],
        "forest": [np.array([-1, -1, 0, 1, 1, -1, 5, 2], np.int32)],
        "ragged_tail": [synth.tree_geo(rng, 33), synth.tree_geo(rng, 1), synth.tree_geo(rng, 95),
                        synth.tree_geo(rng, 130)],
        "bestfirst": [synth.tree_bestfirst(rng, 64)],
    }


@pytest.mark.parametrize("name", ["single", "star", "chain16", "forest", "ragged_tail", "bestfirst"])
@pytest.mark.parametrize("dims", [(2, 4, 128, 128, synth.BF16, synth.F32), (1, 1, 64, 64, synth.BF16, synth.BF16),
                                  (2, 2, 32, 48, synth.F32, synth.F32), (1, 3, 20, 7, synth.F32, synth.BF16)])
def test_edge_shapes(tl, name, dims):
    h_qk, h_v, d_k, d_v, idt, odt = dims
    w = synth.random_case(100 + len(name), _edge_trees()[name], h_qk, h_v, d_k, d_v, idt, odt, name=name)
    _check_full(tl, w, f"{name} {dims}")


def test_deep_chain_needs_larger_max_depth(tl):
    w = synth.random_case(5, [synth.tree_chain(40)], 1, 2, 64, 64, synth.F32, synth.F32,
                          paths=[np.arange(40, dtype=np.int32)])
    _check_full(tl, w, "chain40", max_depth=40)
    dc = tl.DeviceCase(w, max_depth=16)
    sentinel = 123.0
    dc.o.fill_(sentinel)
    assert dc.verify() == 0
    assert dc.device_status() == -8  # GDN_ERR_DEPTH
    assert bool((dc.o == sentinel).all()), "a rejected tree must produce no output"


def test_empty_inputs(tl):
    import torch
    import paper_2607_06763_b200 as gdn
    w = synth.random_case(1, [np.array([-1], np.int32)], 1, 1, 32, 32)
    dc = tl.DeviceCase(w)
    dc.shape.n_seq = 0
    dc.shape.total_nodes = 0
    assert dc.verify() == 0 and dc.commit() == 0
    # an all-empty accepted path set leaves every state untouched
    w2 = synth.random_case(2, [synth.tree_chain(5), synth.tree_star(4)], 1, 2, 32, 32,
                           paths=[np.zeros(0, np.int32), np.zeros(0, np.int32)])
    dc2 = tl.DeviceCase(w2)
    before = dc2.S0.clone()
    assert dc2.commit() == 0 and dc2.device_status() == 0
    assert bool((dc2.S0 == before).all())
    assert gdn.gdn_status_string(0) == "ok"
    torch.cuda.synchronize()


# ------------------------------------------------------------------ invariants on GPU results
def test_chain_equals_token_by_token_commit(tl):
    """A chain's node t output equals a 1-node verify after committing the first t tokens one by one."""
    T = 6
    w = synth.random_case(9, [synth.tree_chain(T)], 2, 4, 128, 128, synth.BF16, synth.F32)
    dc = tl.DeviceCase(w)
    assert dc.verify() == 0 and dc.device_status() == 0
    o_tree = dc.o_host()
    S = w.S0.copy()
    for t in range(T):
        sl = slice(t, t + 1)
        one = synth.Workload("one", 1, w.h_qk, w.h_v, w.d_k, w.d_v, w.in_dtype, w.out_dtype, w.scale, S.copy(), w.q[sl],
                             w.k[sl], w.v[sl], w.g[sl], w.beta[sl], np.array([-1], np.int32),
                             np.array([0, 1], np.int32), np.array([0], np.int32), np.array([0, 1], np.int32))
        d1 = tl.DeviceCase(one)
        assert d1.verify() == 0 and d1.commit() == 0 and d1.device_status() == 0
        np.testing.assert_allclose(d1.o_host()[0], o_tree[t], rtol=2e-4, atol=2e-5)
        S = d1.S0.cpu().numpy()


def test_sibling_permutation_permutes_outputs(tl):
    rng = np.random.default_rng(3)
    t = synth.tree_geo(rng, 40)
    w = synth.random_case(3, [t], 2, 4, 128, 128, synth.BF16, synth.F32)
    # swap two sibling subtrees by a valid renumbering: reverse the order of nodes within each BFS level
    d = synth.depths(t)
    order = np.concatenate([np.nonzero(d == lev)[0][::-1] for lev in range(1, d.max() + 1)])
    new_id = np.empty(len(t), np.int64)
    new_id[order] = np.arange(len(t))
    w2 = synth.random_case(3, [t], 2, 4, 128, 128, synth.BF16, synth.F32)
    w2.parent = np.asarray([-1 if t[old] < 0 else new_id[t[old]] for old in order], dtype=np.int32)
    for name in ("q", "k", "v", "g", "beta"):
        setattr(w2, name, np.ascontiguousarray(getattr(w, name)[order]))
    a, b = tl.DeviceCase(w), tl.DeviceCase(w2)
    assert a.verify() == 0 and b.verify() == 0 and a.device_status() == 0 and b.device_status() == 0
    np.testing.assert_allclose(b.o_host(), a.o_host()[order], rtol=1e-5, atol=1e-6)


# ------------------------------------------------------------------ error reporting (host-made faults only)
def test_device_side_rejections(tl):
    w = synth.random_case(11, [synth.tree_chain(6), synth.tree_star(5)], 1, 2, 64, 64, synth.F32, synth.F32,
                          paths=[np.array([0, 1, 2], np.int32), np.array([0, 3], np.int32)])
    # (1) parent[] not topological in tree 0: tree 0 yields nothing, tree 1 is still verified
    bad = synth.random_case(11, [synth.tree_chain(6), synth.tree_star(5)], 1, 2, 64, 64, synth.F32, synth.F32,
                            paths=[np.array([0, 1, 2], np.int32), np.array([0, 3], np.int32)])  # same tensors as w
    bad.parent = w.parent.copy()
    bad.parent[2] = 4
    dc = tl.DeviceCase(bad)
    dc.o.fill_(77.0)
    assert dc.verify() == 0
    assert dc.device_status() == -7  # GDN_ERR_TREE
    o = dc.o_host()
    assert np.all(o[:6] == 77.0)
    good = tl.oracle_verify(w)
    tl.assert_close_per_head(o[6:], good[6:], np.array([0, 5]), "tree after a rejected one")
    # (2) accepted path that is not a chain from a root: state unchanged, status set
    wp = synth.random_case(11, [synth.tree_chain(6), synth.tree_star(5)], 1, 2, 64, 64, synth.F32, synth.F32,
                           paths=[np.array([0, 2], np.int32), np.array([0, 3], np.int32)])
    dp = tl.DeviceCase(wp)
    before = dp.S0.clone()
    assert dp.commit() == 0
    assert dp.device_status() == -9  # GDN_ERR_PATH
    assert bool((dp.S0[0] == before[0]).all()), "rejected path must leave the state untouched"
    sub, _ = tl.sub_workload(wp, [1])
    tl.assert_state_close(dp.S0[1:2].cpu().numpy().astype(np.float64), tl.oracle_commit(sub))


def test_host_side_rejections(tl):
    import paper_2607_06763_b200 as gdn
    w = synth.random_case(12, [synth.tree_chain(4)], 1, 2, 64, 64)
    dc = tl.DeviceCase(w)
    args = (dc.S0, dc.q, dc.k, dc.v, dc.g, dc.beta, dc.parent, dc.node_offsets, dc.o, dc.ws, dc.ws_bytes, dc.status)
    assert gdn.gdn_tree_verify(dc.shape, None, *args[1:]) == -1           # NULL
    assert gdn.gdn_tree_verify(dc.shape, dc.S0.data_ptr() + 4, *args[1:]) == -4   # misaligned
    assert gdn.gdn_tree_verify(dc.shape, *args[:9], dc.ws, dc.ws_bytes - 1, dc.status) == -10  # workspace too small
    s = gdn.GdnShape.from_workload(w)
    s.d_k = 130
    assert gdn.gdn_tree_verify(s, *args) == -2
    s = gdn.GdnShape.from_workload(w)
    s.in_dtype = 9
    assert gdn.gdn_tree_verify(s, *args) == -3
    s = gdn.GdnShape.from_workload(w)
    s.h_v = 3
    s.h_qk = 2
    assert gdn.gdn_tree_commit(s, dc.S0, dc.k, dc.v, dc.g, dc.beta, dc.parent, dc.node_offsets, dc.path,
                               dc.path_offsets, dc.status) == -2
    assert dc.device_status() == 0


# ------------------------------------------------------------------ host-buffer entry points
def test_host_buffer_entry_points(tl):
    import torch
    import paper_2607_06763_b200 as gdn
    w = synth.config(1, 0)
    shape = gdn.GdnShape.from_workload(w)
    L = int(w.path_offsets[-1])
    arena_bytes = gdn.gdn_tree_host_arena_bytes(shape, L)
    arena = torch.empty(arena_bytes, dtype=torch.uint8, device="cuda")
    o_h = np.zeros((w.total_nodes, w.h_v, w.d_v), dtype=np.uint16)
    rc = gdn.gdn_tree_verify_host(shape, w.S0, w.q, w.k, w.v, w.g, w.beta, w.parent, w.node_offsets, o_h, arena,
                                  arena_bytes)
    assert rc == 0
    tl.assert_close_per_head(synth.bf16_bits_to_f32(o_h).astype(np.float64), tl.oracle_verify(w), w.node_offsets,
                             "verify_host o", bf16_out=True)
    S_h = w.S0.copy()
    rc = gdn.gdn_tree_commit_host(shape, S_h, w.k, w.v, w.g, w.beta, w.parent, w.node_offsets, w.path,
                                  w.path_offsets, L, arena, arena_bytes)
    assert rc == 0
    tl.assert_state_close(S_h.astype(np.float64), tl.oracle_commit(w), what="commit_host S_new")
    # one decode iteration through host buffers: commit of the previous step's path + verify of a new tree
    new = synth.config(1, 1)
    shape_new = gdn.GdnShape.from_workload(new)
    fb = gdn.gdn_tree_commit_verify_host_arena_bytes(shape_new, w.total_nodes, L)
    assert fb > 0
    arena2 = torch.empty(fb, dtype=torch.uint8, device="cuda")
    S2 = w.S0.copy()
    o2 = np.zeros((new.total_nodes, new.h_v, new.d_v), dtype=np.uint16)
    rc = gdn.gdn_tree_commit_verify_host(shape_new, S2, w.total_nodes, w.k, w.v, w.g, w.beta, w.parent,
                                         w.node_offsets, w.path, w.path_offsets, L, new.q, new.k, new.v, new.g,
                                         new.beta, new.parent, new.node_offsets, o2, arena2, fb)
    assert rc == 0
    S_ref = tl.oracle_commit(w)
    tl.assert_state_close(S2.astype(np.float64), S_ref, what="commit_verify_host S_new")
    from oracle import gdn_oracle as orc
    o_ref = orc.verify(S_ref, new.f64("q"), new.f64("k"), new.f64("v"), new.f64("g"), new.f64("beta"), new.parent,
                       new.node_offsets, new.scale)
    tl.assert_close_per_head(synth.bf16_bits_to_f32(o2).astype(np.float64), o_ref, new.node_offsets,
                             "commit_verify_host o", bf16_out=True)
    assert gdn.gdn_tree_commit_verify_host(shape_new, S2, w.total_nodes, w.k, w.v, w.g, w.beta, w.parent,
                                           w.node_offsets, w.path, w.path_offsets, L, new.q, new.k, new.v, new.g,
                                           new.beta, new.parent, new.node_offsets, o2, arena2, fb - 4096) == -10   # GDN_ERR_WORKSPACE


def _oracle_step(S_ref, prev, new):
    """oracle: commit prev's accepted paths on S_ref, then verify `new` on the result"""
    from oracle import gdn_oracle as orc
    S_new = orc.commit(S_ref, prev.f64("k"), prev.f64("v"), prev.f64("g"), prev.f64("beta"), prev.parent,
                       prev.node_offsets, prev.path, prev.path_offsets)
    o = orc.verify(S_new, new.f64("q"), new.f64("k"), new.f64("v"), new.f64("g"), new.f64("beta"), new.parent,
                   new.node_offsets, new.scale)
    return S_new, o


def test_host_buffer_fused_call_pipelined_over_sequence_groups(tl):
    """More sequences than one: the host-buffer fused call cuts the batch into groups and overlaps copies and kernels
    on helper streams (node and path offsets rebased per group).  13 ragged sequences, empty paths and a rejected one
    among them, against the oracle; a second call on the same arena must give the same."""
    import torch
    import paper_2607_06763_b200 as gdn
    rng = np.random.default_rng(401)
    sizes = [64, 5, 33, 1, 64, 17, 48, 9, 64, 2, 40, 64, 21]
    prev_trees = [synth.tree_geo(rng, T) for T in sizes]
    paths = [synth.root_path(t, int(rng.integers(0, len(t)))) if i % 4 else np.zeros(0, np.int32)
             for i, t in enumerate(prev_trees)]
    prev = synth.random_case(402, prev_trees, 4, 8, 128, 128, synth.BF16, synth.BF16, paths=paths, name="host_prev")
    new = synth.random_case(403, [synth.tree_geo(rng, T) for T in reversed(sizes)], 4, 8, 128, 128, synth.BF16,
                            synth.BF16, name="host_new")
    shape = gdn.GdnShape.from_workload(new)
    L = int(prev.path_offsets[-1])
    fb = gdn.gdn_tree_commit_verify_host_arena_bytes(shape, prev.total_nodes, L)
    arena = torch.empty(fb, dtype=torch.uint8, device="cuda")
    S_ref, o_ref = _oracle_step(prev.S0.astype(np.float64), prev, new)
    for call in range(2):
        S = prev.S0.copy()
        o = np.zeros((new.total_nodes, new.h_v, new.d_v), dtype=np.uint16)
        rc = gdn.gdn_tree_commit_verify_host(shape, S, prev.total_nodes, prev.k, prev.v, prev.g, prev.beta, prev.parent,
                                             prev.node_offsets, prev.path, prev.path_offsets, L, new.q, new.k, new.v,
                                             new.g, new.beta, new.parent, new.node_offsets, o, arena, fb)
        assert rc == 0, gdn.gdn_status_string(rc)
        tl.assert_state_close(S.astype(np.float64), S_ref, what=f"pipelined host call {call}: state")
        tl.assert_close_per_head(synth.bf16_bits_to_f32(o).astype(np.float64), o_ref, new.node_offsets,
                                 f"pipelined host call {call}: o", bf16_out=True)
    # one accepted path that is not a chain: reported, that state kept, everything else as before
    bad_paths = list(paths)
    bad_paths[5] = np.array([0, 0], np.int32)
    bad = synth.random_case(402, prev_trees, 4, 8, 128, 128, synth.BF16, synth.BF16, paths=bad_paths, name="host_bad")
    Lb = int(bad.path_offsets[-1])
    S = bad.S0.copy()
    o = np.zeros((new.total_nodes, new.h_v, new.d_v), dtype=np.uint16)
    fb2 = gdn.gdn_tree_commit_verify_host_arena_bytes(shape, bad.total_nodes, Lb)
    arena2 = torch.empty(fb2, dtype=torch.uint8, device="cuda")
    rc = gdn.gdn_tree_commit_verify_host(shape, S, bad.total_nodes, bad.k, bad.v, bad.g, bad.beta, bad.parent,
                                         bad.node_offsets, bad.path, bad.path_offsets, Lb, new.q, new.k, new.v, new.g,
                                         new.beta, new.parent, new.node_offsets, o, arena2, fb2)
    assert rc == -9
    np.testing.assert_array_equal(S[5], bad.S0[5])


# ------------------------------------------------------------------ fused commit + verify
def _fused_case(tl, prev, new, what):
    """commit(prev.path) + verify(new tree) in one call against: oracle commit, then oracle verify on that state."""
    import paper_2607_06763_b200 as gdn
    assert prev.n_seq == new.n_seq
    dp, dn = tl.DeviceCase(prev), tl.DeviceCase(new)
    S = dp.S0.clone()
    rc = gdn.gdn_tree_commit_verify(dn.shape, S, dp.k, dp.v, dp.g, dp.beta, dp.parent, dp.node_offsets, dp.path,
                                    dp.path_offsets, dn.q, dn.k, dn.v, dn.g, dn.beta, dn.parent, dn.node_offsets,
                                    dn.o, dn.ws, dn.ws_bytes, dn.status)
    assert rc == 0, gdn.gdn_status_string(rc)
    assert dn.device_status() == 0
    S_ref = tl.oracle_commit(prev)
    tl.assert_state_close(S.cpu().numpy().astype(np.float64), S_ref, what=what + " S_new")
    from oracle import gdn_oracle as orc
    o_ref = orc.verify(S_ref, new.f64("q"), new.f64("k"), new.f64("v"), new.f64("g"), new.f64("beta"), new.parent,
                       new.node_offsets, new.scale)
    tl.assert_close_per_head(dn.o_host(), o_ref, new.node_offsets, what + " o", bf16_out=tl.is_bf16_out(new))
    for b in range(prev.n_seq):   # empty accepted paths leave their states bit-identical
        if prev.path_offsets[b + 1] == prev.path_offsets[b]:
            assert bool((S[b] == dp.S0[b]).all())


@pytest.mark.parametrize("out_dtype", [synth.BF16, synth.F32])
def test_fused_commit_verify_tensor_core_path(tl, out_dtype):
    rng = np.random.default_rng(21)
    prev_trees = [synth.tree_geo(rng, 64), synth.tree_chain(16), synth.tree_geo(rng, 40), synth.tree_star(9)]
    paths = [synth.longest_path(prev_trees[0]), np.arange(16, dtype=np.int32), np.zeros(0, np.int32),
             np.array([0, 5], np.int32)]
    prev = synth.random_case(31, prev_trees, 2, 4, 128, 128, synth.BF16, out_dtype, paths=paths, name="prev")
    new_trees = [synth.tree_geo(rng, 64), synth.tree_geo(rng, 17), synth.tree_chain(16), synth.tree_geo(rng, 33)]
    new = synth.random_case(32, new_trees, 2, 4, 128, 128, synth.BF16, out_dtype, name="new")
    _fused_case(tl, prev, new, f"fused {out_dtype}")


def test_fused_commit_verify_general_shapes_and_rejected_path(tl):
    import paper_2607_06763_b200 as gdn
    rng = np.random.default_rng(22)
    prev = synth.random_case(33, [synth.tree_geo(rng, 20), synth.tree_chain(7)], 1, 2, 64, 48, synth.F32, synth.F32)
    new = synth.random_case(34, [synth.tree_geo(rng, 90), synth.tree_geo(rng, 5)], 1, 2, 64, 48, synth.F32, synth.F32)
    _fused_case(tl, prev, new, "fused generic")
    # tensor-core path, one accepted path that is not a chain: that state stays, its tree is verified on it
    prev_trees = [synth.tree_chain(6), synth.tree_chain(6)]
    bad = synth.random_case(35, prev_trees, 1, 2, 128, 128, synth.BF16, synth.F32,
                            paths=[np.array([0, 2], np.int32), np.array([0, 1, 2], np.int32)])
    new2 = synth.random_case(36, [synth.tree_star(8), synth.tree_star(8)], 1, 2, 128, 128, synth.BF16, synth.F32)
    dp, dn = tl.DeviceCase(bad), tl.DeviceCase(new2)
    S = dp.S0.clone()
    rc = gdn.gdn_tree_commit_verify(dn.shape, S, dp.k, dp.v, dp.g, dp.beta, dp.parent, dp.node_offsets, dp.path,
                                    dp.path_offsets, dn.q, dn.k, dn.v, dn.g, dn.beta, dn.parent, dn.node_offsets,
                                    dn.o, dn.ws, dn.ws_bytes, dn.status)
    assert rc == 0 and dn.device_status() == -9
    assert bool((S[0] == dp.S0[0]).all()), "a rejected path must leave its state untouched"
    good = synth.random_case(35, prev_trees, 1, 2, 128, 128, synth.BF16, synth.F32,
                             paths=[np.zeros(0, np.int32), np.array([0, 1, 2], np.int32)])
    S_ref = tl.oracle_commit(good)
    tl.assert_state_close(S.cpu().numpy().astype(np.float64), S_ref, what="fused, rejected path")
    from oracle import gdn_oracle as orc
    o_ref = orc.verify(S_ref, new2.f64("q"), new2.f64("k"), new2.f64("v"), new2.f64("g"), new2.f64("beta"),
                       new2.parent, new2.node_offsets, new2.scale)
    tl.assert_close_per_head(dn.o_host(), o_ref, new2.node_offsets, "fused, rejected path o")


@pytest.mark.parametrize("out_dtype", [synth.BF16, synth.F32])
def test_fused_call_with_nothing_to_commit(tl, out_dtype):
    """Every accepted path empty (the first step of a decode loop, or a step whose drafts were all rejected): the
    fused call is then a plain verification and must leave every state bit-identical; path offsets come from a tensor
    made just before the call.  One unit per CTA and several units per CTA."""
    import torch
    import paper_2607_06763_b200 as gdn
    rng = np.random.default_rng(77)
    for trees, hk, hv in (([synth.tree_geo(rng, 64)], 2, 4),
                          ([synth.tree_geo(rng, T) for T in (64, 16, 37, 9, 64)], 2, 4),
                          ([synth.tree_geo(rng, 64) for _ in range(12)], 16, 32)):
        w = synth.random_case(78 + len(trees), trees, hk, hv, 128, 128, synth.BF16, out_dtype)
        d = tl.DeviceCase(w)
        S = d.S0.clone()
        no_paths = torch.zeros(w.n_seq + 1, dtype=torch.int32, device="cuda")
        rc = gdn.gdn_tree_commit_verify(d.shape, S, d.k, d.v, d.g, d.beta, d.parent, d.node_offsets, d.path, no_paths,
                                        d.q, d.k, d.v, d.g, d.beta, d.parent, d.node_offsets, d.o, d.ws, d.ws_bytes,
                                        d.status)
        assert rc == 0 and d.device_status() == 0
        assert bool((S == d.S0).all())
        tl.assert_close_per_head(d.o_host(), tl.oracle_verify(w), w.node_offsets, f"nothing to commit, {len(trees)} trees",
                                 bf16_out=tl.is_bf16_out(w))


def test_refused_fused_call_launches_nothing(tl):
    """A fused call that is refused on the host (here: workspace too small, then a NULL output) must not have
    committed anything: state bit-identical, device status word untouched -- also on shapes that run as two kernels."""
    import paper_2607_06763_b200 as gdn
    rng = np.random.default_rng(91)
    for trees_prev, trees_new in (([synth.tree_geo(rng, 40)], [synth.tree_geo(rng, 100)]),      # grouped: two kernels
                                  ([synth.tree_geo(rng, 40)], [synth.tree_geo(rng, 50)])):      # one fused kernel
        prev = synth.random_case(92, trees_prev, 2, 4, 128, 128, synth.BF16, synth.F32)
        new = synth.random_case(93, trees_new, 2, 4, 128, 128, synth.BF16, synth.F32)
        dp, dn = tl.DeviceCase(prev), tl.DeviceCase(new)
        S = dp.S0.clone()
        args = (dn.shape, S, dp.k, dp.v, dp.g, dp.beta, dp.parent, dp.node_offsets, dp.path, dp.path_offsets, dn.q,
                dn.k, dn.v, dn.g, dn.beta, dn.parent, dn.node_offsets)
        assert gdn.gdn_tree_commit_verify(*args, dn.o, dn.ws, dn.ws_bytes - 256, dn.status) == -10
        assert gdn.gdn_tree_commit_verify(*args, None, dn.ws, dn.ws_bytes, dn.status) == -1
        assert dn.device_status() == 0
        assert bool((S == dp.S0).all()), "a refused call must leave the state as it was"
        assert gdn.gdn_tree_commit_verify(*args, dn.o, dn.ws, dn.ws_bytes, dn.status) == 0
        assert dn.device_status() == 0
        tl.assert_state_close(S.cpu().numpy().astype(np.float64), tl.oracle_commit(prev), what="after the retry")


def test_path_longer_than_max_depth_is_rejected_by_both_entry_points(tl):
    """max_depth = 8 and an accepted path of 12 nodes: the separate commit and the fused call must agree
    (GDN_ERR_PATH, state unchanged)."""
    import paper_2607_06763_b200 as gdn
    prev = synth.random_case(94, [synth.tree_chain(12)], 2, 4, 128, 128, synth.BF16, synth.F32,
                             paths=[np.arange(12, dtype=np.int32)])
    new = synth.random_case(95, [synth.tree_star(8)], 2, 4, 128, 128, synth.BF16, synth.F32)
    dp16 = tl.DeviceCase(prev)
    dn = tl.DeviceCase(new, max_depth=8)
    S = dp16.S0.clone()
    rc = gdn.gdn_tree_commit(dn.shape, S, dp16.k, dp16.v, dp16.g, dp16.beta, dp16.parent, dp16.node_offsets,
                             dp16.path, dp16.path_offsets, dn.status)
    assert rc == 0 and dn.device_status() == -9
    assert bool((S == dp16.S0).all())
    dn.status.zero_()
    rc = gdn.gdn_tree_commit_verify(dn.shape, S, dp16.k, dp16.v, dp16.g, dp16.beta, dp16.parent, dp16.node_offsets,
                                    dp16.path, dp16.path_offsets, dn.q, dn.k, dn.v, dn.g, dn.beta, dn.parent,
                                    dn.node_offsets, dn.o, dn.ws, dn.ws_bytes, dn.status)
    assert rc == 0 and dn.device_status() == -9
    assert bool((S == dp16.S0).all())
    # the new tree is verified against the unchanged state all the same
    tl.assert_close_per_head(dn.o_host(), tl.oracle_verify(dataclass_replace_S0(new, prev.S0)), new.node_offsets,
                             "verify on the unchanged state")


def dataclass_replace_S0(w, S0):
    import dataclasses
    return dataclasses.replace(w, S0=S0)


# ------------------------------------------------------------------ trees larger than one CTA tile (grouped path)
@pytest.mark.parametrize("case", ["t65", "t1000_bestfirst", "forest200", "deep_narrow", "mixed_batch"])
def test_large_trees_grouped_tensor_core_path(tl, case):
    rng = np.random.default_rng(77)
    if case == "t65":
        trees = [synth.tree_geo(rng, 65)]
    elif case == "t1000_bestfirst":
        trees = [synth.tree_bestfirst(rng, 1000, width=8)]
    elif case == "forest200":
        a, b2 = synth.tree_geo(rng, 120), synth.tree_geo(rng, 80)
        trees = [np.concatenate([a, np.where(b2 < 0, -1, b2 + 120)]).astype(np.int32)]
    elif case == "deep_narrow":   # many chains of 16 hanging off one root: every group starts deep in the tree
        par = [-1]
        for c in range(20):
            prev = 0
            for _ in range(15):
                par.append(prev)
                prev = len(par) - 1
        trees = [np.asarray(par, np.int32)]
    else:
        trees = [synth.tree_geo(rng, 30), synth.tree_geo(rng, 257), synth.tree_chain(16), synth.tree_geo(rng, 64),
                 synth.tree_geo(rng, 129)]
    w = synth.random_case(500 + len(case), trees, 2, 4, 128, 128, synth.BF16, synth.F32, name=case)
    _check_full(tl, w, case)


def test_fused_commit_with_extreme_decay_takes_the_plain_replay(tl):
    """A path whose cumulative decay underflows (g very negative) must still commit correctly: S -> k w terms only."""
    trees = [synth.tree_chain(12), synth.tree_chain(12)]
    paths = [np.arange(12, dtype=np.int32), np.arange(5, dtype=np.int32)]
    prev = synth.random_case(41, trees, 1, 2, 128, 128, synth.BF16, synth.F32, paths=paths, name="prev")
    prev.g = synth.store(np.full(prev.g.shape, -9.0, np.float32), synth.BF16)   # alpha = e^-9 per step, A_12 ~ 1e-47
    new = synth.random_case(42, [synth.tree_star(5), synth.tree_star(5)], 1, 2, 128, 128, synth.BF16, synth.F32)
    _fused_case(tl, prev, new, "fused extreme decay")


def test_rows_of_a_neighbouring_tree_never_leak(tl):
    """The tensor-core path stages 64-row boxes, so a short tree's tile also holds rows of the next tree.  Poison
    that neighbour with NaNs: the short tree's outputs and committed state must be unaffected."""
    trees = [synth.tree_chain(10), synth.tree_star(12)]
    w = synth.random_case(61, trees, 2, 4, 128, 128, synth.BF16, synth.F32,
                          paths=[np.arange(4, dtype=np.int32), np.zeros(0, np.int32)])
    clean = tl.oracle_verify(w)
    nan16 = np.uint16(0x7FC0)
    for name in ("q", "k", "v", "g", "beta"):
        getattr(w, name)[10:] = nan16          # every row of the second tree
    dc = tl.DeviceCase(w)
    assert dc.verify() == 0 and dc.device_status() == 0
    o = dc.o.float().cpu().numpy().astype(np.float64)
    assert np.all(np.isfinite(o[:10]))
    tl.assert_close_per_head(o[:10], clean[:10], np.array([0, 10]), "short tree next to a poisoned one")
    assert dc.commit() == 0 and dc.device_status() == 0
    assert bool(torch_isfinite(dc.S0[0]))


def torch_isfinite(t):
    import torch
    return torch.isfinite(t).all()


def test_calls_are_cuda_graph_capturable(tl):
    """The library allocates nothing, never synchronises and launches only on the given stream, so a decode step
    can be captured once and replayed (Section 3.4.2 runs the verify under CUDA graphs)."""
    import torch
    import paper_2607_06763_b200 as gdn
    rng = np.random.default_rng(91)
    prev_trees = [synth.tree_geo(rng, 64), synth.tree_geo(rng, 30)]
    paths = [synth.longest_path(prev_trees[0]), synth.longest_path(prev_trees[1])]
    prev = synth.random_case(92, prev_trees, 2, 4, 128, 128, synth.BF16, synth.BF16, paths=paths, name="prev")
    new = synth.random_case(93, [synth.tree_geo(rng, 64), synth.tree_geo(rng, 50)], 2, 4, 128, 128, synth.BF16,
                            synth.BF16, name="new")
    dp, dn = tl.DeviceCase(prev), tl.DeviceCase(new)
    S = dp.S0.clone()

    def call(stream):
        return gdn.gdn_tree_commit_verify(dn.shape, S, dp.k, dp.v, dp.g, dp.beta, dp.parent, dp.node_offsets,
                                          dp.path, dp.path_offsets, dn.q, dn.k, dn.v, dn.g, dn.beta, dn.parent,
                                          dn.node_offsets, dn.o, dn.ws, dn.ws_bytes, dn.status, stream)

    assert call(None) == 0 and dn.device_status() == 0   # eager once (also loads the kernels before the capture)
    S_eager, o_eager = S.clone(), dn.o.clone()
    side = torch.cuda.Stream()
    graph = torch.cuda.CUDAGraph()
    S.copy_(dp.S0)
    torch.cuda.synchronize()
    with torch.cuda.graph(graph, stream=side):
        rc = call(torch.cuda.current_stream())
    assert rc == 0
    for _ in range(2):   # the captured step replays on a restored state, bit for bit like the eager call
        S.copy_(dp.S0)
        dn.o.zero_()
        graph.replay()
        assert dn.device_status() == 0
        assert bool((S == S_eager).all()) and bool((dn.o == o_eager).all())
    S_ref = tl.oracle_commit(prev)
    tl.assert_state_close(S.cpu().numpy().astype(np.float64), S_ref, what="graph replay S_new")
    from oracle import gdn_oracle as orc
    o_ref = orc.verify(S_ref, new.f64("q"), new.f64("k"), new.f64("v"), new.f64("g"), new.f64("beta"), new.parent,
                       new.node_offsets, new.scale)
    tl.assert_close_per_head(dn.o_host(), o_ref, new.node_offsets, "graph replay o", bf16_out=True)
    # the separate entry points under one capture as well
    S2 = dn.S0.clone()
    graph2 = torch.cuda.CUDAGraph()
    torch.cuda.synchronize()
    with torch.cuda.graph(graph2, stream=side):
        st = torch.cuda.current_stream()
        rc1 = dn.verify(stream=st)
        rc2 = gdn.gdn_tree_commit(dn.shape, S2, dn.k, dn.v, dn.g, dn.beta, dn.parent, dn.node_offsets, dn.path,
                                  dn.path_offsets, dn.status, st)
    assert rc1 == 0 and rc2 == 0
    dn.o.zero_()
    graph2.replay()
    assert dn.device_status() == 0
    tl.assert_close_per_head(dn.o_host(), tl.oracle_verify(new), new.node_offsets, "graph verify o", bf16_out=True)
    tl.assert_state_close(S2.cpu().numpy().astype(np.float64), tl.oracle_commit(new), what="graph commit")


def test_persistent_pipeline_with_rejected_and_empty_trees(tl):
    """640 units, so that a persistent CTA walks two or three of them: rejected trees, empty trees and rejected
    accepted paths sit at the first, the middle and the last place of a CTA's walk.  Every good tree must come out
    right (the prefetch pipeline and its barrier phases stay consistent across skipped units), every rejected
    tree must write nothing, and a rejected path must leave its state alone."""
    import torch
    import paper_2607_06763_b200 as gdn
    rng = np.random.default_rng(123)
    n_seq = 160
    sizes = rng.integers(1, 65, n_seq)
    bad_tree = {0, 5, 75, 76, 149, 150, 151}       # parent[] made non-topological below
    empty_tree = {2, 77, 152, 9}
    bad_path = {1, 78, 153, 10}
    prev_trees, new_trees, paths = [], [], []
    for b in range(n_seq):
        tp = synth.tree_geo(rng, int(rng.integers(2, 65)))
        prev_trees.append(tp)
        pth = synth.root_path(tp, int(rng.integers(0, len(tp))))
        if b % 7 == 3:
            pth = np.zeros(0, np.int32)             # nothing accepted
        if b in bad_path:
            pth = np.array([0, len(tp) - 1, 1], np.int32) if len(tp) > 2 else np.array([1, 0], np.int32)
        paths.append(pth)
        new_trees.append(np.zeros(0, np.int32) if b in empty_tree else synth.tree_geo(rng, max(int(sizes[b]), 3)))
    prev = synth.random_case(124, prev_trees, 2, 4, 128, 128, synth.BF16, synth.F32, paths=paths, name="prev")
    new = synth.random_case(125, new_trees, 2, 4, 128, 128, synth.BF16, synth.F32, name="new")
    good_new = new.parent.copy()
    for b in bad_tree:
        lo = int(new.node_offsets[b])
        new.parent[lo + 1] = 2                      # parent index >= node index: rejected on the device
    dp, dn = tl.DeviceCase(prev), tl.DeviceCase(new)
    S = dp.S0.clone()
    dn.o.fill_(77.0)
    rc = gdn.gdn_tree_commit_verify(dn.shape, S, dp.k, dp.v, dp.g, dp.beta, dp.parent, dp.node_offsets, dp.path,
                                    dp.path_offsets, dn.q, dn.k, dn.v, dn.g, dn.beta, dn.parent, dn.node_offsets,
                                    dn.o, dn.ws, dn.ws_bytes, dn.status)
    assert rc == 0
    assert dn.device_status() in (-7, -9)           # GDN_ERR_TREE or GDN_ERR_PATH, whichever was seen first
    # reference: rejected paths count as empty, rejected trees are left out of the comparison
    ref_paths = [np.zeros(0, np.int32) if b in bad_path else paths[b] for b in range(n_seq)]
    prev_ref = synth.random_case(124, prev_trees, 2, 4, 128, 128, synth.BF16, synth.F32, paths=ref_paths)
    S_ref = tl.oracle_commit(prev_ref)
    S_host = S.cpu().numpy().astype(np.float64)
    tl.assert_state_close(S_host, S_ref, what="pipeline S_new")
    for b in bad_path:
        assert bool((S[b] == dp.S0[b]).all()), "a rejected path must leave its state untouched"
    from oracle import gdn_oracle as orc
    new.parent = good_new
    o_ref = orc.verify(S_ref, new.f64("q"), new.f64("k"), new.f64("v"), new.f64("g"), new.f64("beta"), new.parent,
                       new.node_offsets, new.scale)
    o = dn.o_host()
    for b in range(n_seq):
        lo, hi = int(new.node_offsets[b]), int(new.node_offsets[b + 1])
        if b in bad_tree:
            assert np.all(o[lo:hi] == 77.0), f"rejected tree {b} wrote outputs"
        elif hi > lo:
            tl.assert_close_per_head(o[lo:hi], o_ref[lo:hi], np.array([0, hi - lo]), f"pipeline o, tree {b}")
    # the plain verify walks the same units and skips the rejected / empty ones altogether
    dn.o.fill_(55.0)
    dn.status.zero_()
    before = dn.S0.clone()
    assert dn.verify() == 0 and dn.device_status() == -7
    assert bool((dn.S0 == before).all()), "verify must not touch the state"
    o_ref = tl.oracle_verify(new)
    o = dn.o_host()
    for b in range(n_seq):
        lo, hi = int(new.node_offsets[b]), int(new.node_offsets[b + 1])
        if b in bad_tree:
            assert np.all(o[lo:hi] == 55.0), f"rejected tree {b} wrote outputs"
        elif hi > lo:
            tl.assert_close_per_head(o[lo:hi], o_ref[lo:hi], np.array([0, hi - lo]), f"pipeline verify o, tree {b}")


def test_commit_tile_kernel_paths(tl):
    """d = 128 / bf16 commit kernel: longest legal path, empty path, and every way a path can be rejected."""
    trees = [synth.tree_chain(16), synth.tree_chain(16), synth.tree_star(9), synth.tree_chain(5), synth.tree_chain(5),
             synth.tree_chain(5), synth.tree_star(6)]
    paths = [np.arange(16, dtype=np.int32),            # 0: all 16 nodes
             np.zeros(0, np.int32),                    # 1: nothing accepted
             np.array([0, 7], np.int32),               # 2: root and one leaf of a star
             np.array([0, 1, 9], np.int32),            # 3: node id outside the tree        -> rejected
             np.array([1, 2], np.int32),               # 4: does not start at a root        -> rejected
             np.array([0, 2], np.int32),               # 5: skips a node                    -> rejected
             np.array([0, 3], np.int32)]               # 6: fine
    w = synth.random_case(41, trees, 2, 4, 128, 128, synth.BF16, synth.BF16, paths=paths)
    rejected = {3, 4, 5}
    ref_paths = [np.zeros(0, np.int32) if b in rejected else paths[b] for b in range(len(trees))]
    w_ref = synth.random_case(41, trees, 2, 4, 128, 128, synth.BF16, synth.BF16, paths=ref_paths)
    dc = tl.DeviceCase(w)
    before = dc.S0.clone()
    assert dc.commit() == 0 and dc.device_status() == -9
    tl.assert_state_close(dc.S0.cpu().numpy().astype(np.float64), tl.oracle_commit(w_ref), what="tile commit")
    for b in rejected | {1}:
        assert bool((dc.S0[b] == before[b]).all())
    # without parent[] only the topological order of the path can be checked: 0,2 passes, 2,1 does not
    w2 = synth.random_case(42, [synth.tree_chain(5), synth.tree_chain(5)], 1, 2, 128, 128, synth.BF16, synth.BF16,
                           paths=[np.array([0, 2], np.int32), np.array([2, 1], np.int32)])
    d2 = tl.DeviceCase(w2)
    before2 = d2.S0.clone()
    assert d2.commit(parent=False) == 0 and d2.device_status() == -9
    assert bool((d2.S0[1] == before2[1]).all()) and not bool((d2.S0[0] == before2[0]).all())
    # a path longer than max_depth is rejected as a whole
    w3 = synth.random_case(43, [synth.tree_chain(12)], 1, 2, 128, 128, synth.BF16, synth.BF16,
                           paths=[np.arange(10, dtype=np.int32)])
    d3 = tl.DeviceCase(w3, max_depth=8)
    before3 = d3.S0.clone()
    assert d3.commit() == 0 and d3.device_status() == -9
    assert bool((d3.S0 == before3).all())


def test_fused_call_on_large_trees(tl):
    """Trees beyond one CTA tile: the fused entry point runs the commit tile kernel and the grouped verify kernel back
    to back; results as for the small-tree kernel."""
    rng = np.random.default_rng(131)
    prev_trees = [synth.tree_geo(rng, 200), synth.tree_geo(rng, 70), synth.tree_chain(16)]
    new_trees = [synth.tree_geo(rng, 256), synth.tree_geo(rng, 20), synth.tree_geo(rng, 130)]
    prev = synth.random_case(132, prev_trees, 2, 4, 128, 128, synth.BF16, synth.BF16, name="prev")
    new = synth.random_case(133, new_trees, 2, 4, 128, 128, synth.BF16, synth.BF16, name="new")
    _fused_case(tl, prev, new, "fused, large trees")


@pytest.mark.parametrize("seed", list(range(10)))
def test_fused_randomized_shapes(tl, seed):
    """Random batches on the tensor-core path: head counts and ratios, tree kinds and sizes from 1 to 64 nodes, root
    paths up to 16 nodes (bushy, chains, stars), accepted paths from empty to 16 nodes, both output types."""
    rng = np.random.default_rng(1000 + seed)
    n_seq = int(rng.integers(1, 41))
    h_qk = int(rng.choice([1, 2, 4]))
    h_v = h_qk * int(rng.choice([1, 2, 4]))
    out_dtype = synth.BF16 if seed % 2 else synth.F32

    def tree():
        kind = int(rng.integers(0, 4))
        n = int(rng.integers(1, 65))
        if kind == 0:
            return synth.tree_geo(rng, n)
        if kind == 1:
            return synth.tree_chain(min(n, 16))
        if kind == 2:
            return synth.tree_star(n)
        return synth.tree_bestfirst(rng, n) if n >= 4 else synth.tree_geo(rng, n)

    prev_trees = [tree() for _ in range(n_seq)]
    new_trees = [tree() for _ in range(n_seq)]
    paths = []
    for t in prev_trees:
        r = int(rng.integers(0, 4))
        if r == 0:
            paths.append(np.zeros(0, np.int32))
        elif r == 1:
            paths.append(synth.longest_path(t))
        else:
            paths.append(synth.root_path(t, int(rng.integers(0, len(t)))))
    prev = synth.random_case(2000 + seed, prev_trees, h_qk, h_v, 128, 128, synth.BF16, out_dtype, paths=paths, name="prev")
    new = synth.random_case(3000 + seed, new_trees, h_qk, h_v, 128, 128, synth.BF16, out_dtype, name="new")
    _fused_case(tl, prev, new, f"randomized {seed}")


@pytest.mark.parametrize("seed", list(range(6)))
def test_verify_and_commit_randomized_shapes(tl, seed):
    """Random batches through the plain entry points: even seeds keep every tree within one CTA tile (persistent
    kernel), odd seeds mix in trees of up to 300 nodes (grouped kernel, groups of 49 to 64 nodes)."""
    rng = np.random.default_rng(5000 + seed)
    n_seq = int(rng.integers(1, 25))
    h_qk = int(rng.choice([1, 2, 4]))
    h_v = h_qk * int(rng.choice([1, 2]))
    big = seed % 2 == 1
    trees = []
    for _ in range(n_seq):
        n = int(rng.integers(1, 301 if big else 65))
        kind = int(rng.integers(0, 3))
        trees.append(synth.tree_geo(rng, n) if kind == 0 else synth.tree_bestfirst(rng, n) if kind == 1 and n >= 4
                     else synth.tree_star(min(n, 200)))
    w = synth.random_case(6000 + seed, trees, h_qk, h_v, 128, 128, synth.BF16, synth.F32)
    dc = tl.DeviceCase(w)
    before = dc.S0.clone()
    assert dc.verify() == 0 and dc.device_status() == 0
    assert bool((dc.S0 == before).all())
    tl.assert_close_per_head(dc.o_host(), tl.oracle_verify(w), w.node_offsets, f"randomized verify {seed}")
    assert dc.commit() == 0 and dc.device_status() == 0
    tl.assert_state_close(dc.S0.cpu().numpy().astype(np.float64), tl.oracle_commit(w), what=f"randomized commit {seed}")


# ------------------------------------------------------------------ per-branch recurrent comparator (Section 5.2, Figure 5)
@pytest.mark.parametrize("cfg", [0, 1])
def test_recurrent_comparator_matches_oracle(tl, cfg):
    import paper_2607_06763_b200 as gdn
    for rep in range(3):
        w = synth.config(cfg, rep, out_dtype=synth.F32)
        dc = tl.DeviceCase(w)
        S_before = dc.S0.clone()
        rc = gdn.gdn_tree_verify_recurrent(dc.shape, dc.S0, dc.q, dc.k, dc.v, dc.g, dc.beta, dc.parent, dc.node_offsets,
                                           dc.o, dc.status)
        assert rc == 0 and dc.device_status() == 0
        assert bool((dc.S0 == S_before).all()), "verify must not write the state"
        tl.assert_close_per_head(dc.o_host(), tl.oracle_verify(w), w.node_offsets, f"recurrent cfg{cfg} rep{rep}")


def test_recurrent_comparator_agrees_with_the_tensor_core_path_on_a_ragged_batch(tl):
    """Two structurally different GPU evaluations (token-by-token replay per branch; triangular form on the tensor
    core) of the same trees, both against the oracle: forests, chains, a 300-node tree, bf16 outputs."""
    import paper_2607_06763_b200 as gdn
    rng = np.random.default_rng(123)
    a, b2 = synth.tree_geo(rng, 30), synth.tree_geo(rng, 20)
    forest = np.concatenate([a, np.where(b2 < 0, -1, b2 + 30)]).astype(np.int32)
    trees = [synth.tree_geo(rng, 64), forest, synth.tree_chain(16), synth.tree_bestfirst(rng, 300, width=4),
             synth.tree_star(9)]
    w = synth.random_case(124, trees, 2, 4, 128, 128, synth.BF16, synth.BF16, name="recurrent_ragged")
    ref = tl.oracle_verify(w)
    dc = tl.DeviceCase(w)
    assert gdn.gdn_tree_verify_recurrent(dc.shape, dc.S0, dc.q, dc.k, dc.v, dc.g, dc.beta, dc.parent, dc.node_offsets,
                                         dc.o, dc.status) == 0
    assert dc.device_status() == 0
    tl.assert_close_per_head(dc.o_host(), ref, w.node_offsets, "recurrent ragged", bf16_out=True)
    dc.o.zero_()
    assert dc.verify() == 0 and dc.device_status() == 0
    tl.assert_close_per_head(dc.o_host(), ref, w.node_offsets, "tensor-core ragged", bf16_out=True)


def test_recurrent_comparator_rejects_a_broken_branch(tl):
    import paper_2607_06763_b200 as gdn
    w = synth.random_case(125, [synth.tree_chain(20)], 1, 2, 64, 64, synth.F32, synth.F32)
    dc = tl.DeviceCase(w)     # max_depth 16 < 20 nodes on the only branch
    dc.o.fill_(7.0)
    assert gdn.gdn_tree_verify_recurrent(dc.shape, dc.S0, dc.q, dc.k, dc.v, dc.g, dc.beta, dc.parent, dc.node_offsets,
                                         dc.o, dc.status) == 0
    assert dc.device_status() == -8 and bool((dc.o == 7.0).all())

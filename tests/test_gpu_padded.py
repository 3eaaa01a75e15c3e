"""Padded, shape-static entry points (Section 3.4.2: dense [N, T, H, d] inputs, the tree shared by every layer slot,
gate activations inside the call) against the oracle's padded front end, through the C ABI."""
import numpy as np
import pytest

from paper_2607_06763_b200 import synth

pytestmark = pytest.mark.gpu


class PaddedDevice:
    def __init__(self, w, max_depth=16):
        import torch
        import paper_2607_06763_b200 as gdn
        from paper_2607_06763_b200.binding import to_device
        self.w = w
        self.shape = gdn.GdnShape(w.n_slots, w.h_qk, w.h_v, w.d, w.d, 1, 1 if w.out_dtype == synth.BF16 else 0, max_depth,
                                  w.n_slots * w.t_pad, w.t_pad, w.scale)
        for n in ("S0", "q", "k", "v", "g_in", "beta_in", "parent", "n_nodes", "path", "path_len"):
            setattr(self, n, to_device(getattr(w, n)))
        odt = torch.bfloat16 if w.out_dtype == synth.BF16 else torch.float32
        self.o = torch.full((w.n_slots, w.t_pad, w.h_v, w.d), 7.0, dtype=odt, device="cuda")
        self.status = torch.zeros(1, dtype=torch.int32, device="cuda")

    def status_value(self):
        import torch
        torch.cuda.synchronize()
        return int(self.status.item())

    def o_host(self):
        return self.o.float().cpu().numpy().astype(np.float64)


def _oracle_verify(w, S0=None):
    from oracle import gdn_oracle as orc
    return orc.verify_padded(w.S0.astype(np.float64) if S0 is None else S0, w.f64("q"), w.f64("k"), w.f64("v"),
                             w.f64("g_in"), w.f64("beta_in"), w.parent, w.n_nodes, w.scale, w.raw_gates)


def _oracle_commit(w, S0):
    from oracle import gdn_oracle as orc
    return orc.commit_padded(S0, w.f64("k"), w.f64("v"), w.f64("g_in"), w.f64("beta_in"), w.parent, w.n_nodes, w.path,
                             w.path_len, w.raw_gates)


def _assert_outputs(tl, d, o_ref, what):
    """rows of each slot's tree against the oracle; rows beyond the node count must still hold the fill value"""
    w = d.w
    o = d.o_host()
    for s in range(w.n_slots):
        n = int(w.n_nodes[s % w.n_trees])
        tl.assert_close_per_head(o[s, :n], o_ref[s, :n], np.array([0, n]), f"{what} slot {s}",
                                 bf16_out=w.out_dtype == synth.BF16)
        assert np.all(o[s, n:] == 7.0), f"{what}: rows beyond the tree of slot {s} were written"


@pytest.fixture(scope="module")
def tl(cuda_device):
    from tests import gdn_testlib
    return gdn_testlib


def _trees(rng, sizes):
    return [synth.tree_geo(rng, T) if T > 1 else np.array([-1], np.int32) for T in sizes]


@pytest.mark.parametrize("raw_gates", [False, True])
@pytest.mark.parametrize("t_pad,sizes,out_dtype", [(64, (64, 37, 64), synth.BF16), (64, (1, 50), synth.F32),
                                                   (32, (32, 9), synth.BF16), (48, (48, 40, 3), synth.F32)])
def test_verify_padded(tl, t_pad, sizes, out_dtype, raw_gates):
    import paper_2607_06763_b200 as gdn
    rng = np.random.default_rng(sum(sizes) + t_pad)
    w = synth.padded_case(700 + t_pad + len(sizes), _trees(rng, sizes), 3, t_pad, raw_gates, out_dtype=out_dtype)
    d = PaddedDevice(w)
    S_before = d.S0.clone()
    rc = gdn.gdn_tree_verify_padded(d.shape, w.n_trees, raw_gates, d.S0, d.q, d.k, d.v, d.g_in, d.beta_in, d.parent,
                                    d.n_nodes, d.o, d.status)
    assert rc == 0, gdn.gdn_status_string(rc)
    assert d.status_value() == 0
    assert bool((d.S0 == S_before).all())
    _assert_outputs(tl, d, _oracle_verify(w), f"verify_padded T{t_pad} raw={raw_gates}")


@pytest.mark.parametrize("raw_gates", [False, True])
def test_commit_verify_padded(tl, raw_gates):
    """Previous step padded to 48 rows, new step to 64; one tree commits nothing (path_len 0)."""
    import paper_2607_06763_b200 as gdn
    rng = np.random.default_rng(801)
    prev_trees = _trees(rng, (48, 20, 33))
    paths = [synth.longest_path(prev_trees[0]), np.zeros(0, np.int32), synth.root_path(prev_trees[2], 17)]
    prev = synth.padded_case(810, prev_trees, 4, 48, raw_gates, paths=paths)
    new = synth.padded_case(811, _trees(rng, (64, 64, 11)), 4, 64, raw_gates)
    dp, dn = PaddedDevice(prev), PaddedDevice(new)
    S = dp.S0.clone()
    rc = gdn.gdn_tree_commit_verify_padded(dn.shape, new.n_trees, raw_gates, S, prev.t_pad, dp.k, dp.v, dp.g_in,
                                           dp.beta_in, dp.parent, dp.n_nodes, dp.path, dp.path_len, dn.q, dn.k, dn.v,
                                           dn.g_in, dn.beta_in, dn.parent, dn.n_nodes, dn.o, dn.status)
    assert rc == 0, gdn.gdn_status_string(rc)
    assert dn.status_value() == 0
    S_ref = _oracle_commit(prev, prev.S0.astype(np.float64))
    tl.assert_state_close(S.cpu().numpy().astype(np.float64), S_ref, what="commit_verify_padded state")
    for s in range(prev.n_slots):
        if prev.path_len[s % prev.n_trees] == 0:
            assert bool((S[s] == dp.S0[s]).all())
    _assert_outputs(tl, dn, _oracle_verify(new, S_ref), f"commit_verify_padded raw={raw_gates}")


def test_commit_verify_padded_with_nothing_to_commit(tl):
    """All path lengths zero: a plain verification, every state untouched."""
    import paper_2607_06763_b200 as gdn
    rng = np.random.default_rng(803)
    prev = synth.padded_case(820, _trees(rng, (64, 30)), 5, 64, True, paths=[np.zeros(0, np.int32)] * 2)
    new = synth.padded_case(821, _trees(rng, (64, 41)), 5, 64, True)
    dp, dn = PaddedDevice(prev), PaddedDevice(new)
    S = dp.S0.clone()
    rc = gdn.gdn_tree_commit_verify_padded(dn.shape, new.n_trees, True, S, prev.t_pad, dp.k, dp.v, dp.g_in, dp.beta_in,
                                           dp.parent, dp.n_nodes, dp.path, dp.path_len, dn.q, dn.k, dn.v, dn.g_in,
                                           dn.beta_in, dn.parent, dn.n_nodes, dn.o, dn.status)
    assert rc == 0 and dn.status_value() == 0
    assert bool((S == dp.S0).all())
    _assert_outputs(tl, dn, _oracle_verify(new, prev.S0.astype(np.float64)), "padded, nothing to commit")


def test_padded_call_captured_once_replayed_with_another_tree(tl):
    """Shapes do not depend on the tree: capture the fused padded call in a CUDA graph, then overwrite the device
    arrays (tree, node counts, accepted path, node tensors, state) in place and replay."""
    import torch
    import paper_2607_06763_b200 as gdn
    rng = np.random.default_rng(901)
    steps = []
    for i, (ps, ns) in enumerate((((64,), (64,)), ((31,), (50,)), ((64,), (7,)))):
        prev = synth.padded_case(910 + i, _trees(rng, ps), 6, 64, True)
        new = synth.padded_case(920 + i, _trees(rng, ns), 6, 64, True)
        steps.append((prev, new))
    dp, dn = PaddedDevice(steps[0][0]), PaddedDevice(steps[0][1])
    S = dp.S0.clone()
    side = torch.cuda.Stream()
    graph = torch.cuda.CUDAGraph()

    def call(stream):
        rc = gdn.gdn_tree_commit_verify_padded(dn.shape, 1, True, S, 64, dp.k, dp.v, dp.g_in, dp.beta_in, dp.parent,
                                               dp.n_nodes, dp.path, dp.path_len, dn.q, dn.k, dn.v, dn.g_in, dn.beta_in,
                                               dn.parent, dn.n_nodes, dn.o, dn.status, stream)
        assert rc == 0, gdn.gdn_status_string(rc)

    call(None)                      # warm-up outside the capture (kernel attributes, tensor-map entry point)
    torch.cuda.synchronize()
    with torch.cuda.graph(graph, stream=side):
        call(torch.cuda.current_stream())
    from paper_2607_06763_b200.binding import to_device
    for prev, new in steps:
        for dev, w in ((dp, prev), (dn, new)):
            for n in ("q", "k", "v", "g_in", "beta_in", "parent", "n_nodes", "path", "path_len"):
                getattr(dev, n).copy_(to_device(getattr(w, n)))
            dev.w = w
        S.copy_(to_device(prev.S0))
        dn.o.fill_(7.0)
        graph.replay()
        assert dn.status_value() == 0
        S_ref = _oracle_commit(prev, prev.S0.astype(np.float64))
        tl.assert_state_close(S.cpu().numpy().astype(np.float64), S_ref, what="graph replay state")
        _assert_outputs(tl, dn, _oracle_verify(new, S_ref), "graph replay")


def test_padded_rejections(tl):
    import paper_2607_06763_b200 as gdn
    rng = np.random.default_rng(5)
    w = synth.padded_case(950, _trees(rng, (20, 30)), 2, 32, True)
    d = PaddedDevice(w)
    args = (d.S0, d.q, d.k, d.v, d.g_in, d.beta_in, d.parent, d.n_nodes, d.o, d.status)
    assert gdn.gdn_tree_verify_padded(d.shape, 3, True, *args) == -2              # 4 slots do not split over 3 trees
    bad = gdn.GdnShape.from_buffer_copy(d.shape)
    bad.total_nodes -= 1
    assert gdn.gdn_tree_verify_padded(bad, 2, True, *args) == -2
    big = gdn.GdnShape.from_buffer_copy(d.shape)
    big.max_tree_nodes, big.total_nodes = 96, 4 * 96
    assert gdn.gdn_tree_verify_padded(big, 2, True, *args) == -5                  # more than 64 rows per slot
    assert gdn.gdn_tree_verify_padded(d.shape, 2, True, None, *args[1:]) == -1
    assert d.status_value() == 0 and bool((d.o == 7.0).all())
    # device-side: a node count beyond the padded size, a parent that points forward
    d.n_nodes[0] = 33
    assert gdn.gdn_tree_verify_padded(d.shape, 2, True, *args) == 0
    assert d.status_value() == -7
    d.status.zero_()
    d.n_nodes[0] = 20
    d.parent[1, 5] = 9
    d.o.fill_(7.0)
    assert gdn.gdn_tree_verify_padded(d.shape, 2, True, *args) == 0
    assert d.status_value() == -7
    o = d.o_host()
    assert np.all(o[1] == 7.0) and np.all(o[3] == 7.0), "slots of the rejected tree must stay untouched"
    ref = _oracle_verify(w)
    for s in (0, 2):
        tl.assert_close_per_head(o[s, :20], ref[s, :20], np.array([0, 20]), f"good tree, slot {s}", bf16_out=True)


# ----------------------------------------------------------------------------- plan as an object of its own (any T)
def _plan(d, w):
    import torch
    import paper_2607_06763_b200 as gdn
    nbytes = gdn.gdn_tree_plan_bytes(d.shape, w.n_trees)
    assert nbytes > 0
    plan = torch.empty(nbytes, dtype=torch.uint8, device="cuda")
    rc = gdn.gdn_tree_plan(d.shape, w.n_trees, d.parent, d.n_nodes, plan, d.status)
    assert rc == 0, gdn.gdn_status_string(rc)
    return plan


@pytest.mark.parametrize("raw_gates", [False, True])
@pytest.mark.parametrize("t_pad,sizes,n_layers,out_dtype", [(64, (64, 37), 3, synth.BF16), (128, (128, 70, 5), 2, synth.F32),
                                                            (256, (256, 131), 2, synth.BF16), (200, (66,), 3, synth.F32),
                                                            (512, (512,), 1, synth.BF16)])
def test_verify_planned(tl, t_pad, sizes, n_layers, out_dtype, raw_gates):
    """Trees of up to 512 rows per slot, several slots per tree, rows beyond the node count poisoned; one plan serves
    two verification calls (the plan is read-only for them)."""
    import paper_2607_06763_b200 as gdn
    rng = np.random.default_rng(sum(sizes) + t_pad)
    w = synth.padded_case(1200 + t_pad + len(sizes), _trees(rng, sizes), n_layers, t_pad, raw_gates, out_dtype=out_dtype)
    d = PaddedDevice(w)
    plan = _plan(d, w)
    S_before = d.S0.clone()
    ref = _oracle_verify(w)
    for rep in range(2):
        d.o.fill_(7.0)
        rc = gdn.gdn_tree_verify_planned(d.shape, w.n_trees, raw_gates, d.S0, d.q, d.k, d.v, d.g_in, d.beta_in, plan, d.o,
                                         d.status)
        assert rc == 0, gdn.gdn_status_string(rc)
        assert d.status_value() == 0
        assert bool((d.S0 == S_before).all())
        _assert_outputs(tl, d, ref, f"verify_planned T{t_pad} raw={raw_gates} call {rep}")


@pytest.mark.parametrize("raw_gates", [False, True])
def test_commit_padded_then_verify_planned(tl, raw_gates):
    """A decode step on 256-row slots: the accepted paths of the previous trees are committed, then the new trees
    are verified against the advanced states; one tree commits nothing."""
    import paper_2607_06763_b200 as gdn
    rng = np.random.default_rng(1301)
    prev_trees = _trees(rng, (256, 90))
    paths = [synth.longest_path(prev_trees[0]), np.zeros(0, np.int32)]
    prev = synth.padded_case(1310, prev_trees, 2, 256, raw_gates, paths=paths)
    new = synth.padded_case(1311, _trees(rng, (200, 256)), 2, 256, raw_gates)
    dp, dn = PaddedDevice(prev), PaddedDevice(new)
    S = dp.S0.clone()
    rc = gdn.gdn_tree_commit_padded(dp.shape, prev.n_trees, raw_gates, S, dp.k, dp.v, dp.g_in, dp.beta_in, dp.parent,
                                    dp.n_nodes, dp.path, dp.path_len, dn.status)
    assert rc == 0, gdn.gdn_status_string(rc)
    plan = _plan(dn, new)
    rc = gdn.gdn_tree_verify_planned(dn.shape, new.n_trees, raw_gates, S, dn.q, dn.k, dn.v, dn.g_in, dn.beta_in, plan,
                                     dn.o, dn.status)
    assert rc == 0, gdn.gdn_status_string(rc)
    assert dn.status_value() == 0
    S_ref = _oracle_commit(prev, prev.S0.astype(np.float64))
    tl.assert_state_close(S.cpu().numpy().astype(np.float64), S_ref, what="commit_padded state")
    for s in range(prev.n_slots):
        if prev.path_len[s % prev.n_trees] == 0:
            assert bool((S[s] == dp.S0[s]).all())
    _assert_outputs(tl, dn, _oracle_verify(new, S_ref), f"commit_padded + verify_planned raw={raw_gates}")


def test_planned_step_captured_once_replayed_with_another_tree(tl):
    """plan + commit + verify of 128-row slots in one CUDA graph; trees, node counts, paths and tensors are then
    overwritten in place and the graph replayed."""
    import torch
    import paper_2607_06763_b200 as gdn
    from paper_2607_06763_b200.binding import to_device
    rng = np.random.default_rng(1401)
    steps = []
    for i, (ps, ns) in enumerate((((128,), (128,)), ((40,), (99,)), ((128,), (65,)))):
        prev = synth.padded_case(1410 + i, _trees(rng, ps), 3, 128, True)
        new = synth.padded_case(1420 + i, _trees(rng, ns), 3, 128, True)
        steps.append((prev, new))
    dp, dn = PaddedDevice(steps[0][0]), PaddedDevice(steps[0][1])
    S = dp.S0.clone()
    plan = torch.empty(gdn.gdn_tree_plan_bytes(dn.shape, 1), dtype=torch.uint8, device="cuda")

    def call(stream):
        assert gdn.gdn_tree_plan(dn.shape, 1, dn.parent, dn.n_nodes, plan, dn.status, stream) == 0
        assert gdn.gdn_tree_commit_padded(dp.shape, 1, True, S, dp.k, dp.v, dp.g_in, dp.beta_in, dp.parent, dp.n_nodes,
                                          dp.path, dp.path_len, dn.status, stream) == 0
        assert gdn.gdn_tree_verify_planned(dn.shape, 1, True, S, dn.q, dn.k, dn.v, dn.g_in, dn.beta_in, plan, dn.o,
                                           dn.status, stream) == 0

    call(None)
    torch.cuda.synchronize()
    side = torch.cuda.Stream()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph, stream=side):
        call(torch.cuda.current_stream())
    for prev, new in steps:
        for dev, w in ((dp, prev), (dn, new)):
            for n in ("q", "k", "v", "g_in", "beta_in", "parent", "n_nodes", "path", "path_len"):
                getattr(dev, n).copy_(to_device(getattr(w, n)))
            dev.w = w
        S.copy_(to_device(prev.S0))
        dn.o.fill_(7.0)
        graph.replay()
        assert dn.status_value() == 0
        S_ref = _oracle_commit(prev, prev.S0.astype(np.float64))
        tl.assert_state_close(S.cpu().numpy().astype(np.float64), S_ref, what="planned graph replay state")
        _assert_outputs(tl, dn, _oracle_verify(new, S_ref), "planned graph replay")


def test_planned_rejections(tl):
    import torch
    import paper_2607_06763_b200 as gdn
    rng = np.random.default_rng(15)
    w = synth.padded_case(1500, _trees(rng, (100, 128)), 2, 128, False)
    d = PaddedDevice(w)
    plan = torch.empty(gdn.gdn_tree_plan_bytes(d.shape, 2), dtype=torch.uint8, device="cuda")
    assert gdn.gdn_tree_plan(d.shape, 3, d.parent, d.n_nodes, plan, d.status) == -2       # 4 slots, 3 trees
    assert gdn.gdn_tree_plan(d.shape, 2, d.parent, d.n_nodes, plan[:1024], d.status) == -10   # plan too small
    assert gdn.gdn_tree_plan(d.shape, 2, None, d.n_nodes, plan, d.status) == -1
    # a plan buffer that no plan was built in, and a plan built for another depth bound: refused on the device
    # (GDN_ERR_WORKSPACE in *status_dev), nothing is written
    blank = torch.zeros_like(plan)
    assert gdn.gdn_tree_verify_planned(d.shape, 2, False, d.S0, d.q, d.k, d.v, d.g_in, d.beta_in, blank, d.o, d.status) == 0
    assert d.status_value() == -10 and bool((d.o == 7.0).all())
    d.status.zero_()
    shallow = gdn.GdnShape.from_buffer_copy(d.shape)
    shallow.max_depth = 12
    plan12 = torch.empty(gdn.gdn_tree_plan_bytes(shallow, 2), dtype=torch.uint8, device="cuda")
    assert gdn.gdn_tree_plan(shallow, 2, d.parent, d.n_nodes, plan12, d.status) == 0
    assert d.status_value() == 0
    if plan12.numel() >= plan.numel():
        assert gdn.gdn_tree_verify_planned(d.shape, 2, False, d.S0, d.q, d.k, d.v, d.g_in, d.beta_in, plan12, d.o,
                                           d.status) == 0
        assert d.status_value() == -10 and bool((d.o == 7.0).all())
        d.status.zero_()
    # device-side: a parent that points forward in tree 1 -> its slots are skipped, tree 0 is verified
    d.parent[1, 70] = 90
    assert gdn.gdn_tree_plan(d.shape, 2, d.parent, d.n_nodes, plan, d.status) == 0
    assert d.status_value() == -7
    d.status.zero_()
    rc = gdn.gdn_tree_verify_planned(d.shape, 2, False, d.S0, d.q, d.k, d.v, d.g_in, d.beta_in, plan, d.o, d.status)
    assert rc == 0 and d.status_value() == 0
    o = d.o_host()
    assert np.all(o[1] == 7.0) and np.all(o[3] == 7.0), "slots of the rejected tree must stay untouched"
    ref = _oracle_verify(w)
    for s in (0, 2):
        tl.assert_close_per_head(o[s, :100], ref[s, :100], np.array([0, 100]), f"good tree, slot {s}", bf16_out=True)
    # a path that does not start at a root: the commit reports it and leaves the states of that tree's slots alone
    S = d.S0.clone()
    d.path[0, :2] = torch.tensor([5, 0], dtype=torch.int32)
    d.path_len[0] = 2
    rc = gdn.gdn_tree_commit_padded(d.shape, 2, False, S, d.k, d.v, d.g_in, d.beta_in, d.parent, d.n_nodes, d.path,
                                    d.path_len, d.status)
    assert rc == 0
    assert d.status_value() == -9
    assert bool((S[0] == d.S0[0]).all()) and bool((S[2] == d.S0[2]).all())
    assert not bool((S[1] == d.S0[1]).all()), "the other tree's path is committed all the same"


# ----------------------------------------------------------------------------- full-size workloads in the padded layout
@pytest.mark.parametrize("cfg", [5, 2])
def test_full_size_stack_through_the_padded_entry_points(tl, cfg):
    """The 48-slot stacks of the benchmark (64- and 256-node trees, every slot carrying the same full-size tree, so
    that their ragged packing already is the padded layout) through the shape-static entry points in the launch
    configuration bench.py --layout padded times: commit of the accepted path, then verification, whole workload
    against the oracle."""
    import torch
    import paper_2607_06763_b200 as gdn
    from paper_2607_06763_b200.binding import to_device
    from oracle import gdn_oracle as orc
    w = synth.config(cfg, 1)
    T = int(w.node_offsets[1])
    assert w.total_nodes == w.n_seq * T
    shape = gdn.GdnShape.from_workload(w)
    d = {n: to_device(getattr(w, n)) for n in ("S0", "q", "k", "v", "g", "beta")}
    plen = int(w.path_offsets[1])
    path1 = np.zeros((1, shape.max_depth), np.int32)
    path1[0, :plen] = w.path[:plen]
    parent1, nodes1 = to_device(w.parent[:T].reshape(1, T).copy()), to_device(np.array([T], np.int32))
    path_d, len_d = to_device(path1), to_device(np.array([plen], np.int32))
    o = torch.zeros((w.total_nodes, w.h_v, w.d_v), dtype=torch.bfloat16, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    S = d["S0"].clone()
    if T <= 64:
        rc = gdn.gdn_tree_commit_verify_padded(shape, 1, False, S, T, d["k"], d["v"], d["g"], d["beta"], parent1, nodes1,
                                               path_d, len_d, d["q"], d["k"], d["v"], d["g"], d["beta"], parent1, nodes1,
                                               o, status)
        assert rc == 0, gdn.gdn_status_string(rc)
    else:
        plan = torch.empty(gdn.gdn_tree_plan_bytes(shape, 1), dtype=torch.uint8, device="cuda")
        assert gdn.gdn_tree_plan(shape, 1, parent1, nodes1, plan, status) == 0
        assert gdn.gdn_tree_commit_padded(shape, 1, False, S, d["k"], d["v"], d["g"], d["beta"], parent1, nodes1, path_d,
                                          len_d, status) == 0
        assert gdn.gdn_tree_verify_planned(shape, 1, False, S, d["q"], d["k"], d["v"], d["g"], d["beta"], plan, o,
                                           status) == 0
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    S_ref = orc.commit(w.S0.astype(np.float64), w.f64("k"), w.f64("v"), w.f64("g"), w.f64("beta"), w.parent,
                       w.node_offsets, w.path, w.path_offsets)
    o_ref = orc.verify(S_ref, w.f64("q"), w.f64("k"), w.f64("v"), w.f64("g"), w.f64("beta"), w.parent, w.node_offsets,
                       w.scale)
    tl.assert_state_close(S.cpu().numpy().astype(np.float64), S_ref, what=f"padded full-size cfg{cfg} state")
    tl.assert_close_per_head(o.float().cpu().numpy().astype(np.float64), o_ref, w.node_offsets,
                             f"padded full-size cfg{cfg}", bf16_out=True)

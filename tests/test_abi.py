"""CPU-side checks of the C-ABI library: it builds, loads, exports every declared symbol, and its host-only logic
(shape checks, tree/path validation, workspace sizing) behaves.  No kernel is launched here."""
import ctypes
import os
import re

import numpy as np
import pytest

import paper_2607_06763_b200 as gdn
from paper_2607_06763_b200 import build, synth

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build.build_library()
    return gdn.load_library()


def _declared_functions():
    text = open(os.path.join(ROOT, "include", "gdn_tree.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(gdn_[a-z_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol(lib):
    names = _declared_functions()
    assert "gdn_tree_verify" in names and "gdn_tree_commit" in names
    for n in names:
        assert hasattr(lib, n), f"{n} is declared in include/gdn_tree.h but not exported"
    from paper_2607_06763_b200 import binding
    assert sorted(binding.EXPORTS) == names, "the Python binding must wrap exactly the declared entry points"


def test_shape_struct_matches_header():
    text = open(os.path.join(ROOT, "include", "gdn_tree.h")).read()
    body = re.search(r"typedef struct gdn_shape \{(.*?)\} gdn_shape_t;", text, flags=re.S).group(1)
    body = re.sub(r"/\*.*?\*/", "", body, flags=re.S)
    fields = re.findall(r"(int32_t|float)\s+(\w+);", body)
    assert [f for _, f in fields] == [f for f, _ in gdn.GdnShape._fields_]
    assert ctypes.sizeof(gdn.GdnShape) == 4 * len(fields)


def test_status_strings(lib):
    seen = set()
    for code in range(0, -12, -1):
        s = gdn.gdn_status_string(code)
        assert s and s != "unknown status" and s not in seen
        seen.add(s)
    assert gdn.gdn_status_string(-99) == "unknown status"


def _shape(w, **kw):
    s = gdn.GdnShape.from_workload(w)
    for k, v in kw.items():
        setattr(s, k, v)
    return s


def test_workspace_bytes(lib):
    w = synth.config(0)
    s = _shape(w)
    n = gdn.gdn_tree_workspace_bytes(s)
    assert n >= w.total_nodes * w.h_v * w.d_v * 4 and n % 256 == 0
    assert gdn.gdn_tree_workspace_bytes(_shape(w, d_k=6)) == 0      # not a multiple of 4
    assert gdn.gdn_tree_workspace_bytes(_shape(w, h_v=3)) == 0      # not a multiple of h_qk
    assert gdn.gdn_tree_workspace_bytes(_shape(w, max_depth=65)) == 0
    assert gdn.gdn_tree_host_arena_bytes(s, 3) > n


def test_plan_bytes_and_padded_entry_points_on_the_host(lib):
    """Size of the shared-tree plan and the host-side refusals of the padded entry points (no CUDA call is made)."""
    def shape(n_seq, t_pad, h_v=32, max_depth=16):
        return gdn.GdnShape(n_seq, 16, h_v, 128, 128, 1, 1, max_depth, n_seq * t_pad, t_pad, 0.0883883)
    base = gdn.gdn_tree_plan_bytes(shape(48, 256), 1)
    assert base > 0 and base % 256 == 0
    # the plan depends on the padded size, the depth bound and the number of trees -- not on slots or heads
    assert gdn.gdn_tree_plan_bytes(shape(96, 256), 1) == base
    assert gdn.gdn_tree_plan_bytes(shape(48, 256, h_v=16), 1) == base
    assert gdn.gdn_tree_plan_bytes(shape(48, 512), 1) > base
    assert gdn.gdn_tree_plan_bytes(shape(48, 256), 2) > base
    assert gdn.gdn_tree_plan_bytes(shape(48, 256, max_depth=8), 1) < base
    assert gdn.gdn_tree_plan_bytes(shape(48, 256), 0) == 0
    s = shape(4, 128)
    assert gdn.gdn_tree_plan(s, 3, 16, 16, _FakeBuf(1 << 20), 16) == -2               # 4 slots, 3 trees
    assert gdn.gdn_tree_plan(s, 2, None, 16, _FakeBuf(1 << 20), 16) == -1
    assert gdn.gdn_tree_plan(s, 2, 16, 16, _FakeBuf(256), 16) == -10                  # plan buffer too small
    assert gdn.gdn_tree_verify_planned(s, 2, 0, 16, 16, 16, 16, 16, 16, _FakeBuf(256), 16, 16) == -10
    assert gdn.gdn_tree_verify_planned(s, 2, 0, None, 16, 16, 16, 16, 16, _FakeBuf(1 << 20), 16, 16) == -1
    far = gdn.GdnShape(4, 16, 32, 128, 128, 1, 1, 16, 4 * 2048, 2048, 0.0883883)
    assert gdn.gdn_tree_verify_planned(far, 2, 0, 16, 16, 16, 16, 16, 16, _FakeBuf(1 << 24), 16, 16) in (-2, -5)
    f32 = gdn.GdnShape(4, 16, 32, 128, 128, 0, 0, 16, 4 * 128, 128, 0.0883883)        # fp32 inputs: general path only
    assert gdn.gdn_tree_commit_padded(f32, 2, 0, 16, 16, 16, 16, 16, 16, 16, 16, 16, 16) == -5
    assert gdn.gdn_tree_commit_padded(s, 2, 0, 16, 16, 16, 16, 16, 16, None, 16, 16, 16) == -1   # n_nodes missing


class _FakeBuf:
    """Stands in for a device buffer in calls that are refused before any CUDA work: an aligned fake address and a
    size, with the two methods the binding asks of a tensor."""
    def __init__(self, nbytes):
        self._n = nbytes

    def data_ptr(self):
        return 1 << 20

    def numel(self):
        return self._n

    def element_size(self):
        return 1


def test_validate_host(lib):
    rng = np.random.default_rng(0)
    trees = [synth.tree_geo(rng, 20), synth.tree_chain(16), synth.tree_star(9)]
    w = synth.random_case(1, trees, 1, 1, 4, 4)
    s = _shape(w)
    assert gdn.gdn_tree_validate_host(s, w.parent, w.node_offsets, w.path, w.path_offsets) == 0
    assert gdn.gdn_tree_validate_host(s, w.parent, w.node_offsets) == 0
    bad = w.parent.copy()
    bad[5] = 7
    assert gdn.gdn_tree_validate_host(s, bad, w.node_offsets) == -7
    assert gdn.gdn_tree_validate_host(_shape(w, max_depth=15), w.parent, w.node_offsets) == -8
    off = w.node_offsets.copy()
    off[1] += 1
    bad_off_parent = w.parent.copy()
    assert gdn.gdn_tree_validate_host(_shape(w, max_tree_nodes=19), w.parent, w.node_offsets) == -7
    off2 = w.node_offsets.copy()
    off2[-1] -= 1
    assert gdn.gdn_tree_validate_host(s, bad_off_parent, off2) == -7
    path = w.path.copy()
    p0 = int(w.path_offsets[1])
    if w.path_offsets[2] - p0 >= 2:
        path[p0 + 1] = path[p0]           # not a child of the previous entry
        assert gdn.gdn_tree_validate_host(s, w.parent, w.node_offsets, path, w.path_offsets) == -9
    po = w.path_offsets.copy()
    po[0] = 1
    assert gdn.gdn_tree_validate_host(s, w.parent, w.node_offsets, w.path, po) == -9
    assert gdn.gdn_tree_validate_host(s, None, w.node_offsets) == -1


def test_entry_points_reject_bad_arguments_before_touching_cuda(lib):
    """These return on the host before any CUDA call, so they are safe without a GPU."""
    w = synth.config(0)
    s = _shape(w)
    assert gdn.gdn_tree_verify(s, None, None, None, None, None, None, None, None, None, None, 0, None) == -1
    assert gdn.gdn_tree_commit(s, None, None, None, None, None, None, None, None, None, None) == -1
    assert gdn.gdn_tree_verify(_shape(w, in_dtype=5), 16, 16, 16, 16, 16, 16, 16, 16, 16, 256, 1 << 30, 16) == -3
    assert gdn.gdn_tree_verify(s, 16, 16, 16, 16, 16, 16, 16, 16, 16, None, 0, 16) == -10
    assert gdn.gdn_tree_verify(s, 16, 16, 24, 16, 16, 16, 16, 16, 16, 256, 1 << 30, 16) == -4
    assert gdn.gdn_tree_verify(s, 16, 16, 16, 16, 16, 16, 16, 16, 16, 256, 8, 16) == -10
    assert gdn.gdn_tree_verify(_shape(w, n_seq=0, total_nodes=0), None, None, None, None, None, None, None, None,
                               None, None, 0, None) == 0


def test_missing_library_fails_loudly(monkeypatch, tmp_path):
    from paper_2607_06763_b200 import binding
    monkeypatch.setattr(binding, "_lib", None)
    monkeypatch.setattr(binding, "_HERE", str(tmp_path))
    with pytest.raises(RuntimeError, match="no CPU fallback"):
        binding.load_library()

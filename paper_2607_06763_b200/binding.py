"""ctypes binding of the C-ABI library declared in ``include/gdn_tree.h``.

Argument marshalling only: every step of verify and commit runs in the CUDA kernels of ``libgdn_tree.so``.
Tensor arguments may be torch tensors (their ``data_ptr()`` is passed), numpy arrays (host entry points) or raw
integer addresses.  There is no fallback of any kind: if the library has not been built, ``load_library`` raises.
"""
from __future__ import annotations

import ctypes
import os

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB_NAME = "libgdn_tree.so"
_lib = None

GDN_F32 = 0
GDN_BF16 = 1
DTYPE_CODES = {"f32": GDN_F32, "bf16": GDN_BF16}

EXPORTS = (
    "gdn_status_string",
    "gdn_tree_workspace_bytes",
    "gdn_tree_validate_host",
    "gdn_tree_verify",
    "gdn_tree_commit",
    "gdn_tree_host_arena_bytes",
    "gdn_tree_verify_host",
    "gdn_tree_commit_host",
    "gdn_tree_commit_verify_host_arena_bytes",
    "gdn_tree_commit_verify_host",
    "gdn_tree_verify_static",
    "gdn_tree_commit_verify",
    "gdn_tree_verify_recurrent",
    "gdn_tree_verify_padded",
    "gdn_tree_commit_verify_padded",
    "gdn_tree_plan_bytes",
    "gdn_tree_plan",
    "gdn_tree_verify_planned",
    "gdn_tree_commit_padded",
)

GDN_STATIC_SCRATCH_BYTES = 4 << 20


class GdnShape(ctypes.Structure):
    """Mirror of ``gdn_shape_t``."""
    _fields_ = [
        ("n_seq", ctypes.c_int32),
        ("h_qk", ctypes.c_int32),
        ("h_v", ctypes.c_int32),
        ("d_k", ctypes.c_int32),
        ("d_v", ctypes.c_int32),
        ("in_dtype", ctypes.c_int32),
        ("out_dtype", ctypes.c_int32),
        ("max_depth", ctypes.c_int32),
        ("total_nodes", ctypes.c_int32),
        ("max_tree_nodes", ctypes.c_int32),
        ("scale", ctypes.c_float),
    ]

    @classmethod
    def from_workload(cls, w, max_depth: int = 16, max_tree_nodes: int | None = None) -> "GdnShape":
        """Shape of a ``synth.Workload``."""
        import numpy as np
        sizes = np.diff(w.node_offsets)
        mt = int(sizes.max()) if len(sizes) else 1
        return cls(w.n_seq, w.h_qk, w.h_v, w.d_k, w.d_v, DTYPE_CODES[w.in_dtype], DTYPE_CODES[w.out_dtype],
                   max_depth, w.total_nodes, max(1, mt if max_tree_nodes is None else max_tree_nodes), w.scale)


def library_path() -> str:
    return os.path.join(_HERE, _LIB_NAME)


def load_library():
    """Load ``libgdn_tree.so`` (built in-tree by ``paper_2607_06763_b200.build``); raises if it is missing."""
    global _lib
    if _lib is None:
        path = library_path()
        if not os.path.exists(path):
            raise RuntimeError(
                f"{path} is missing: the CUDA library has not been built "
                "(run `python -m paper_2607_06763_b200.build`); there is no CPU fallback")
        lib = ctypes.CDLL(path)
        vp, sp = ctypes.c_void_p, ctypes.POINTER(GdnShape)
        lib.gdn_status_string.restype = ctypes.c_char_p
        lib.gdn_status_string.argtypes = [ctypes.c_int]
        lib.gdn_tree_workspace_bytes.restype = ctypes.c_size_t
        lib.gdn_tree_workspace_bytes.argtypes = [sp]
        lib.gdn_tree_validate_host.restype = ctypes.c_int
        lib.gdn_tree_validate_host.argtypes = [sp, vp, vp, vp, vp]
        lib.gdn_tree_verify.restype = ctypes.c_int
        lib.gdn_tree_verify.argtypes = [sp] + [vp] * 10 + [ctypes.c_size_t, vp, vp]
        lib.gdn_tree_commit.restype = ctypes.c_int
        lib.gdn_tree_commit.argtypes = [sp] + [vp] * 11
        lib.gdn_tree_host_arena_bytes.restype = ctypes.c_size_t
        lib.gdn_tree_host_arena_bytes.argtypes = [sp, ctypes.c_int32]
        lib.gdn_tree_verify_host.restype = ctypes.c_int
        lib.gdn_tree_verify_host.argtypes = [sp] + [vp] * 10 + [ctypes.c_size_t, vp]
        lib.gdn_tree_commit_host.restype = ctypes.c_int
        lib.gdn_tree_commit_host.argtypes = [sp] + [vp] * 9 + [ctypes.c_int32, vp, ctypes.c_size_t, vp]
        lib.gdn_tree_commit_verify_host_arena_bytes.restype = ctypes.c_size_t
        lib.gdn_tree_commit_verify_host_arena_bytes.argtypes = [sp, ctypes.c_int32, ctypes.c_int32]
        lib.gdn_tree_commit_verify_host.restype = ctypes.c_int
        lib.gdn_tree_commit_verify_host.argtypes = ([sp, vp, ctypes.c_int32] + [vp] * 8 + [ctypes.c_int32] + [vp] * 8 +
                                                    [vp, ctypes.c_size_t, vp])
        lib.gdn_tree_commit_verify.restype = ctypes.c_int
        lib.gdn_tree_commit_verify.argtypes = [sp] + [vp] * 18 + [ctypes.c_size_t, vp, vp]
        lib.gdn_tree_verify_padded.restype = ctypes.c_int
        lib.gdn_tree_verify_padded.argtypes = [sp, ctypes.c_int32, ctypes.c_int32] + [vp] * 11
        lib.gdn_tree_commit_verify_padded.restype = ctypes.c_int
        lib.gdn_tree_commit_verify_padded.argtypes = ([sp, ctypes.c_int32, ctypes.c_int32, vp, ctypes.c_int32] +
                                                      [vp] * 18)
        lib.gdn_tree_plan_bytes.restype = ctypes.c_size_t
        lib.gdn_tree_plan_bytes.argtypes = [sp, ctypes.c_int32]
        lib.gdn_tree_plan.restype = ctypes.c_int
        lib.gdn_tree_plan.argtypes = [sp, ctypes.c_int32, vp, vp, vp, ctypes.c_size_t, vp, vp]
        lib.gdn_tree_verify_planned.restype = ctypes.c_int
        lib.gdn_tree_verify_planned.argtypes = ([sp, ctypes.c_int32, ctypes.c_int32] + [vp] * 7 +
                                                [ctypes.c_size_t, vp, vp, vp])
        lib.gdn_tree_commit_padded.restype = ctypes.c_int
        lib.gdn_tree_commit_padded.argtypes = [sp, ctypes.c_int32, ctypes.c_int32] + [vp] * 11
        lib.gdn_tree_verify_static.restype = ctypes.c_int
        lib.gdn_tree_verify_static.argtypes = [sp] + [vp] * 11
        lib.gdn_tree_verify_recurrent.restype = ctypes.c_int
        lib.gdn_tree_verify_recurrent.argtypes = [sp] + [vp] * 11
        _lib = lib
    return _lib


def to_device(a, device="cuda"):
    """numpy array -> torch tensor on ``device``; ``uint16`` arrays are bf16 bit patterns and come back as bf16."""
    import numpy as np
    import torch
    a = np.ascontiguousarray(a)
    if a.dtype == np.uint16:
        return torch.from_numpy(a.view(np.int16).copy()).view(torch.bfloat16).to(device)
    return torch.from_numpy(a).to(device)


def _ptr(x):
    """Address of a torch tensor / numpy array / int / None."""
    if x is None:
        return None
    if isinstance(x, int):
        return x
    if hasattr(x, "data_ptr"):
        return x.data_ptr()
    if hasattr(x, "ctypes"):
        return x.ctypes.data
    raise TypeError(f"cannot take the address of {type(x)!r}")


def _stream(stream):
    if stream is None:
        return None
    return stream.cuda_stream if hasattr(stream, "cuda_stream") else int(stream)


def gdn_status_string(status: int) -> str:
    return load_library().gdn_status_string(int(status)).decode()


def gdn_tree_workspace_bytes(shape: GdnShape) -> int:
    return int(load_library().gdn_tree_workspace_bytes(ctypes.byref(shape)))


def gdn_tree_validate_host(shape: GdnShape, parent, node_offsets, path=None, path_offsets=None) -> int:
    return int(load_library().gdn_tree_validate_host(ctypes.byref(shape), _ptr(parent), _ptr(node_offsets),
                                                      _ptr(path), _ptr(path_offsets)))


def gdn_tree_verify(shape: GdnShape, S0, q, k, v, g, beta, parent, node_offsets, o, workspace, workspace_bytes,
                    status_dev, stream=None) -> int:
    return int(load_library().gdn_tree_verify(ctypes.byref(shape), _ptr(S0), _ptr(q), _ptr(k), _ptr(v), _ptr(g),
                                               _ptr(beta), _ptr(parent), _ptr(node_offsets), _ptr(o),
                                               _ptr(workspace), int(workspace_bytes), _ptr(status_dev),
                                               _stream(stream)))


def gdn_tree_commit(shape: GdnShape, S, k, v, g, beta, parent, node_offsets, path, path_offsets, status_dev,
                    stream=None) -> int:
    return int(load_library().gdn_tree_commit(ctypes.byref(shape), _ptr(S), _ptr(k), _ptr(v), _ptr(g), _ptr(beta),
                                               _ptr(parent), _ptr(node_offsets), _ptr(path), _ptr(path_offsets),
                                               _ptr(status_dev), _stream(stream)))


def gdn_tree_host_arena_bytes(shape: GdnShape, total_path_len: int = 0) -> int:
    return int(load_library().gdn_tree_host_arena_bytes(ctypes.byref(shape), int(total_path_len)))


def gdn_tree_verify_host(shape: GdnShape, S0, q, k, v, g, beta, parent, node_offsets, o, dev_arena, arena_bytes,
                         stream=None) -> int:
    return int(load_library().gdn_tree_verify_host(ctypes.byref(shape), _ptr(S0), _ptr(q), _ptr(k), _ptr(v),
                                                    _ptr(g), _ptr(beta), _ptr(parent), _ptr(node_offsets), _ptr(o),
                                                    _ptr(dev_arena), int(arena_bytes), _stream(stream)))


def gdn_tree_commit_host(shape: GdnShape, S, k, v, g, beta, parent, node_offsets, path, path_offsets,
                         total_path_len, dev_arena, arena_bytes, stream=None) -> int:
    return int(load_library().gdn_tree_commit_host(ctypes.byref(shape), _ptr(S), _ptr(k), _ptr(v), _ptr(g),
                                                    _ptr(beta), _ptr(parent), _ptr(node_offsets), _ptr(path),
                                                    _ptr(path_offsets), int(total_path_len), _ptr(dev_arena),
                                                    int(arena_bytes), _stream(stream)))


def gdn_tree_commit_verify_host_arena_bytes(shape: GdnShape, prev_total_nodes: int, total_path_len: int) -> int:
    return int(load_library().gdn_tree_commit_verify_host_arena_bytes(ctypes.byref(shape), int(prev_total_nodes),
                                                                      int(total_path_len)))


def gdn_tree_commit_verify_host(shape: GdnShape, S, prev_total_nodes, k_prev, v_prev, g_prev, beta_prev, parent_prev,
                                node_offsets_prev, path, path_offsets, total_path_len, q, k, v, g, beta, parent,
                                node_offsets, o, dev_arena, arena_bytes, stream=None) -> int:
    return int(load_library().gdn_tree_commit_verify_host(
        ctypes.byref(shape), _ptr(S), int(prev_total_nodes), _ptr(k_prev), _ptr(v_prev), _ptr(g_prev), _ptr(beta_prev),
        _ptr(parent_prev), _ptr(node_offsets_prev), _ptr(path), _ptr(path_offsets), int(total_path_len), _ptr(q),
        _ptr(k), _ptr(v), _ptr(g), _ptr(beta), _ptr(parent), _ptr(node_offsets), _ptr(o), _ptr(dev_arena),
        int(arena_bytes), _stream(stream)))


def gdn_tree_verify_padded(shape, n_trees, raw_gates, S0, q, k, v, g, beta, parent, n_nodes, o, status_dev,
                           stream=None) -> int:
    """``gdn_tree_verify_padded``: dense ``[slots, T, ...]`` inputs, trees shared by slots, optional raw gates."""
    return int(load_library().gdn_tree_verify_padded(
        ctypes.byref(shape), int(n_trees), int(bool(raw_gates)), _ptr(S0), _ptr(q), _ptr(k), _ptr(v), _ptr(g), _ptr(beta),
        _ptr(parent), _ptr(n_nodes), _ptr(o), _ptr(status_dev), _stream(stream)))


def gdn_tree_commit_verify_padded(shape, n_trees, raw_gates, S, prev_t_pad, k_prev, v_prev, g_prev, beta_prev,
                                  parent_prev, n_nodes_prev, path, path_len, q, k, v, g, beta, parent, n_nodes, o,
                                  status_dev, stream=None) -> int:
    """``gdn_tree_commit_verify_padded``: the fused step in the padded layout."""
    return int(load_library().gdn_tree_commit_verify_padded(
        ctypes.byref(shape), int(n_trees), int(bool(raw_gates)), _ptr(S), int(prev_t_pad), _ptr(k_prev), _ptr(v_prev),
        _ptr(g_prev), _ptr(beta_prev), _ptr(parent_prev), _ptr(n_nodes_prev), _ptr(path), _ptr(path_len), _ptr(q),
        _ptr(k), _ptr(v), _ptr(g), _ptr(beta), _ptr(parent), _ptr(n_nodes), _ptr(o), _ptr(status_dev),
        _stream(stream)))


def gdn_tree_plan_bytes(shape, n_trees) -> int:
    """``gdn_tree_plan_bytes``: size of the shared-tree plan of the padded layout."""
    return int(load_library().gdn_tree_plan_bytes(ctypes.byref(shape), int(n_trees)))


def gdn_tree_plan(shape, n_trees, parent, n_nodes, plan, status_dev, stream=None) -> int:
    """``gdn_tree_plan``: build the plan of the ``n_trees`` shared trees (once per decode step)."""
    return int(load_library().gdn_tree_plan(ctypes.byref(shape), int(n_trees), _ptr(parent), _ptr(n_nodes), _ptr(plan),
                                            int(plan.numel() * plan.element_size()), _ptr(status_dev), _stream(stream)))


def gdn_tree_verify_planned(shape, n_trees, raw_gates, S0, q, k, v, g, beta, plan, o, status_dev, stream=None) -> int:
    """``gdn_tree_verify_planned``: verification in the padded layout against a plan built by ``gdn_tree_plan``."""
    return int(load_library().gdn_tree_verify_planned(
        ctypes.byref(shape), int(n_trees), int(bool(raw_gates)), _ptr(S0), _ptr(q), _ptr(k), _ptr(v), _ptr(g),
        _ptr(beta), _ptr(plan), int(plan.numel() * plan.element_size()), _ptr(o), _ptr(status_dev), _stream(stream)))


def gdn_tree_commit_padded(shape, n_trees, raw_gates, S, k, v, g, beta, parent, n_nodes, path, path_len, status_dev,
                           stream=None) -> int:
    """``gdn_tree_commit_padded``: the delayed commit in the padded layout (one accepted path per tree)."""
    return int(load_library().gdn_tree_commit_padded(
        ctypes.byref(shape), int(n_trees), int(bool(raw_gates)), _ptr(S), _ptr(k), _ptr(v), _ptr(g), _ptr(beta),
        _ptr(parent), _ptr(n_nodes), _ptr(path), _ptr(path_len), _ptr(status_dev), _stream(stream)))


def gdn_tree_verify_recurrent(shape, S0, q, k, v, g, beta, parent, node_offsets, o, status_dev, stream=None) -> int:
    """``gdn_tree_verify_recurrent``: the per-branch recurrent baseline (same results as ``gdn_tree_verify``)."""
    return int(load_library().gdn_tree_verify_recurrent(ctypes.byref(shape), _ptr(S0), _ptr(q), _ptr(k), _ptr(v),
                                                         _ptr(g), _ptr(beta), _ptr(parent), _ptr(node_offsets),
                                                         _ptr(o), _ptr(status_dev), _stream(stream)))


def gdn_tree_verify_static(shape: GdnShape, S0, q, k, v, g, beta, parent, node_offsets, o, status_dev,
                           stream=None) -> int:
    """``gdn_tree_verify`` for callers that cannot allocate device memory: the scratch is a fixed array inside the
    library (at most ``GDN_STATIC_SCRATCH_BYTES``), shared by all calls on a device, so overlapping calls race."""
    return int(load_library().gdn_tree_verify_static(ctypes.byref(shape), _ptr(S0), _ptr(q), _ptr(k), _ptr(v),
                                                      _ptr(g), _ptr(beta), _ptr(parent), _ptr(node_offsets),
                                                      _ptr(o), _ptr(status_dev), _stream(stream)))


def gdn_tree_commit_verify(shape: GdnShape, S, k_prev, v_prev, g_prev, beta_prev, parent_prev, node_offsets_prev,
                           path, path_offsets, q, k, v, g, beta, parent, node_offsets, o, workspace,
                           workspace_bytes, status_dev, stream=None) -> int:
    """Commit of the previous step's accepted paths fused with the verification of the new trees."""
    return int(load_library().gdn_tree_commit_verify(
        ctypes.byref(shape), _ptr(S), _ptr(k_prev), _ptr(v_prev), _ptr(g_prev), _ptr(beta_prev), _ptr(parent_prev),
        _ptr(node_offsets_prev), _ptr(path), _ptr(path_offsets), _ptr(q), _ptr(k), _ptr(v), _ptr(g), _ptr(beta),
        _ptr(parent), _ptr(node_offsets), _ptr(o), _ptr(workspace), int(workspace_bytes), _ptr(status_dev),
        _stream(stream)))

"""Shared helpers of the GPU parity tests: device marshalling, oracle calls and the tolerance rule."""
from __future__ import annotations

import numpy as np

import paper_2607_06763_b200 as gdn
from paper_2607_06763_b200 import synth

# Tolerances.  The arithmetic is held to |gpu - ref| <= 1e-4*|ref| + 1e-4*rms(ref over the same tree and head)
# for outputs and for the committed state.  A bf16 output additionally carries its own rounding: round-to-nearest
# with an 8-bit significand is off by at most 2^-8*|ref|, so that much is added elementwise, and the norm-wise
# relative error of a head (about 1.6e-3 for ideally rounded values, a statistical figure, hence only checked
# where a head has at least 1024 output elements) must stay below 2e-3.
TOL_F32 = 1e-4
TOL_STATE = 1e-4
BF16_HALF_ULP = 2.0 ** -8
TOL_BF16_NORMWISE = 2e-3


def _torch():
    import torch
    return torch


def to_dev(a: np.ndarray):
    """numpy -> cuda tensor; uint16 arrays are reinterpreted as bf16."""
    from paper_2607_06763_b200.binding import to_device
    return to_device(a, "cuda")


class DeviceCase:
    """A workload resident on the GPU plus its output / workspace / status buffers."""

    def __init__(self, w: synth.Workload, max_depth: int = 16, max_tree_nodes: int | None = None):
        torch = _torch()
        self.w = w
        self.shape = gdn.GdnShape.from_workload(w, max_depth=max_depth, max_tree_nodes=max_tree_nodes)
        self.S0 = to_dev(w.S0)
        self.q, self.k, self.v, self.g, self.beta = (to_dev(getattr(w, n)) for n in ("q", "k", "v", "g", "beta"))
        self.parent, self.node_offsets = to_dev(w.parent), to_dev(w.node_offsets)
        self.path = to_dev(w.path if w.path.size else np.zeros(1, np.int32))
        self.path_offsets = to_dev(w.path_offsets)
        odt = torch.float32 if w.out_dtype == synth.F32 else torch.bfloat16
        self.o = torch.zeros((max(w.total_nodes, 1), w.h_v, w.d_v), dtype=odt, device="cuda")
        self.ws_bytes = gdn.gdn_tree_workspace_bytes(self.shape)
        self.ws = torch.zeros(max(self.ws_bytes, 256), dtype=torch.uint8, device="cuda")
        self.status = torch.zeros(1, dtype=torch.int32, device="cuda")

    def verify(self, stream=None) -> int:
        return gdn.gdn_tree_verify(self.shape, self.S0, self.q, self.k, self.v, self.g, self.beta, self.parent,
                                   self.node_offsets, self.o, self.ws, self.ws_bytes, self.status, stream)

    def commit(self, S=None, stream=None, parent=True) -> int:
        return gdn.gdn_tree_commit(self.shape, self.S0 if S is None else S, self.k, self.v, self.g, self.beta,
                                   self.parent if parent else None, self.node_offsets, self.path,
                                   self.path_offsets, self.status, stream)

    def device_status(self) -> int:
        _torch().cuda.synchronize()
        return int(self.status.item())

    def o_host(self) -> np.ndarray:
        return self.o.float().cpu().numpy().astype(np.float64)[: self.w.total_nodes]


def oracle_verify(w: synth.Workload, first_seq=0, n_do=None) -> np.ndarray:
    from oracle import gdn_oracle as orc
    return orc.verify(w.f64("S0"), w.f64("q"), w.f64("k"), w.f64("v"), w.f64("g"), w.f64("beta"), w.parent,
                      w.node_offsets, w.scale, first_seq=first_seq, n_do=n_do)


def oracle_commit(w: synth.Workload) -> np.ndarray:
    from oracle import gdn_oracle as orc
    return orc.commit(w.f64("S0"), w.f64("k"), w.f64("v"), w.f64("g"), w.f64("beta"), w.parent, w.node_offsets,
                      w.path, w.path_offsets)


def sub_workload(w: synth.Workload, seqs) -> synth.Workload:
    """The same tensors restricted to a few sequences (for oracle sampling of large configurations)."""
    seqs = list(seqs)
    nodes = np.concatenate([np.arange(w.node_offsets[b], w.node_offsets[b + 1]) for b in seqs]).astype(np.int64)
    trees = [w.parent[w.node_offsets[b]:w.node_offsets[b + 1]] for b in seqs]
    paths = [w.path[w.path_offsets[b]:w.path_offsets[b + 1]] for b in seqs]
    parent, node_offsets = synth._pack(trees)
    path, path_offsets = synth._pack_paths(paths)
    return synth.Workload(w.name + "_sub", len(seqs), w.h_qk, w.h_v, w.d_k, w.d_v, w.in_dtype, w.out_dtype, w.scale,
                          w.S0[seqs], w.q[nodes], w.k[nodes], w.v[nodes], w.g[nodes], w.beta[nodes], parent,
                          node_offsets, path, path_offsets, dict(w.meta)), nodes


def assert_close_per_head(got: np.ndarray, ref: np.ndarray, node_offsets, what: str, bf16_out: bool = False,
                          tol: float = TOL_F32):
    """got/ref: [N, H, d].  Bound per element: tol*|ref| + tol*rms(ref over the tree and head), plus the bf16
    rounding allowance and the norm-wise 2e-3 check when the output was stored as bf16."""
    assert got.shape == ref.shape, (got.shape, ref.shape)
    assert np.all(np.isfinite(got)), f"{what}: non-finite values"
    worst = 0.0
    for b in range(len(node_offsets) - 1):
        lo, hi = int(node_offsets[b]), int(node_offsets[b + 1])
        if hi == lo:
            continue
        r, x = ref[lo:hi], got[lo:hi]
        rms = np.sqrt(np.mean(r * r, axis=(0, 2), keepdims=True))
        bound = tol * np.abs(r) + tol * rms + (BF16_HALF_ULP * np.abs(r) if bf16_out else 0.0)
        ratio = np.abs(x - r) / np.maximum(bound, 1e-300)
        worst = max(worst, float(ratio.max()))
        if bf16_out and r.shape[0] * r.shape[2] >= 1024:
            nw = np.sqrt(np.sum((x - r) ** 2, axis=(0, 2)) / np.maximum(np.sum(r * r, axis=(0, 2)), 1e-300))
            assert float(nw.max()) <= TOL_BF16_NORMWISE, f"{what}: norm-wise relative error {nw.max():.2e}"
    assert worst <= 1.0, f"{what}: worst error is {worst:.3f}x the allowed bound (tol {tol})"
    return worst


def assert_state_close(got: np.ndarray, ref: np.ndarray, tol: float = TOL_STATE, what: str = "state"):
    """got/ref: [B, H, d_v, d_k]; rms over each (sequence, head) tile."""
    assert got.shape == ref.shape
    assert np.all(np.isfinite(got)), f"{what}: non-finite values"
    rms = np.sqrt(np.mean(ref * ref, axis=(2, 3), keepdims=True))
    bound = tol * np.abs(ref) + tol * rms
    worst = float((np.abs(got - ref) / np.maximum(bound, 1e-300)).max())
    assert worst <= 1.0, f"{what}: worst error is {worst:.3f}x the allowed bound (tol {tol})"
    return worst


def is_bf16_out(w: synth.Workload) -> bool:
    return w.out_dtype == synth.BF16

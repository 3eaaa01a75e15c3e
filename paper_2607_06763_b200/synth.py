"""Seeded synthetic workloads for GDN tree verify / commit.

This module only *makes inputs*: draft-tree shapes, accepted paths and random
tensors with the value distributions of the benchmark configurations.  It
contains none of the gated-delta-rule arithmetic and imports neither the CUDA
binding nor the CPU oracle, so both sides can be fed the same bytes.

Tree shapes follow the parameters the paper states for its draft trees: a node
budget of 32-512 (Section 4.3), a per-node fan-out of at most 8 (Algorithm 1),
and at most 16 nodes on a root path (Section 6: the drafter's block of 16
positions).  The paper's trees come from a trained drafter on public benchmark
suites; the seeded random trees here stand in for them.

bf16 tensors are carried as ``numpy.uint16`` bit patterns (numpy has no bf16).
"""
from __future__ import annotations

from dataclasses import dataclass, field

import numpy as np

SEED_BASE = 260706763
MAX_DEPTH = 16  # nodes on a root path
FANOUT = 8

F32 = "f32"
BF16 = "bf16"


# ----------------------------------------------------------------------------- dtype helpers
def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round fp32 to bf16 (round-to-nearest-even) and return the 16-bit patterns."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    bias = ((u >> np.uint32(16)) & np.uint32(1)) + np.uint32(0x7FFF)
    return ((u + bias) >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def store(x: np.ndarray, dtype: str) -> np.ndarray:
    """Round an fp32/fp64 array to the storage dtype (``f32`` array or bf16 bit patterns)."""
    x32 = np.ascontiguousarray(x, dtype=np.float32)
    return x32 if dtype == F32 else f32_to_bf16_bits(x32)


def widen(a: np.ndarray, dtype: str) -> np.ndarray:
    """Stored values as fp64, exactly."""
    return (a if dtype == F32 else bf16_bits_to_f32(a)).astype(np.float64)


# ----------------------------------------------------------------------------- tree shapes
def depths(parent: np.ndarray) -> np.ndarray:
    """Number of nodes on each node's root path (a root has depth 1)."""
    d = np.zeros(len(parent), dtype=np.int32)
    for i, p in enumerate(parent):
        d[i] = 1 if p < 0 else d[p] + 1
    return d


def root_path(parent: np.ndarray, node: int) -> np.ndarray:
    """Node ids from the root down to ``node`` (inclusive)."""
    out = []
    n = int(node)
    while n >= 0:
        out.append(n)
        n = int(parent[n])
    return np.asarray(out[::-1], dtype=np.int32)


def bfs_renumber(parent: np.ndarray) -> np.ndarray:
    """Renumber a tree/forest in breadth-first order (stable in the old ids); returns the new parent[]."""
    T = len(parent)
    d = depths(parent)
    order = np.argsort(d, kind="stable")
    new_id = np.empty(T, dtype=np.int64)
    new_id[order] = np.arange(T)
    out = np.empty(T, dtype=np.int32)
    for old in range(T):
        p = parent[old]
        out[new_id[old]] = -1 if p < 0 else new_id[p]
    return out


def tree_chain(T: int) -> np.ndarray:
    return np.arange(-1, T - 1, dtype=np.int32)


def tree_star(T: int) -> np.ndarray:
    p = np.zeros(T, dtype=np.int32)
    p[0] = -1
    return p


def tree_small_uniform(rng: np.random.Generator, T: int = 8, kmax: int = 3, depth: int = 3) -> np.ndarray:
    """BFS tree with child counts uniform on {0..kmax} (root >= 1), redrawn until exactly T nodes and the given depth."""
    while True:
        parent = [-1]
        dep = [1]
        i = 0
        while i < len(parent) and len(parent) <= T:
            if dep[i] < depth:
                c = int(rng.integers(0, kmax + 1))
                if i == 0:
                    c = max(c, 1)
                for _ in range(c):
                    parent.append(i)
                    dep.append(dep[i] + 1)
            i += 1
        if len(parent) == T and max(dep) == depth:
            return np.asarray(parent, dtype=np.int32)


def tree_geo(rng: np.random.Generator, T: int, max_depth: int = MAX_DEPTH, fanout: int = FANOUT,
             mean_children: float = 2.0) -> np.ndarray:
    """BFS-grown tree: child counts geometric on {0,1,..} with the given mean, clipped to ``fanout``; truncated at T nodes."""
    p = 1.0 / (1.0 + mean_children)
    parent = [-1]
    dep = [1]
    nchild = [0]
    i = 0
    while len(parent) < T:
        if i < len(parent):
            if dep[i] < max_depth:
                c = min(int(rng.geometric(p)) - 1, fanout)
                if i == 0:
                    c = max(c, 1)
                c = min(c, T - len(parent))
                for _ in range(c):
                    parent.append(i)
                    dep.append(dep[i] + 1)
                    nchild.append(0)
                nchild[i] += c
            i += 1
        else:
            # frontier died out: the lowest-index node that may still grow receives one more child
            for j in range(len(parent)):
                if dep[j] < max_depth and nchild[j] < fanout:
                    parent.append(j)
                    dep.append(dep[j] + 1)
                    nchild.append(0)
                    nchild[j] += 1
                    break
            else:
                raise ValueError("tree cannot reach the requested size under the depth/fan-out caps")
    return bfs_renumber(np.asarray(parent, dtype=np.int32))


def tree_bestfirst(rng: np.random.Generator, T: int, width: int = 4, fanout: int = FANOUT,
                   max_depth: int = MAX_DEPTH, concentration: float = 0.25) -> np.ndarray:
    """Shape of a width-``width`` best-first expansion (Algorithm 1) driven by seeded synthetic child probabilities.

    Only the shape is used: every node added to the tree proposes ``fanout`` children whose probabilities are a
    Dirichlet draw sharpened towards one dominant child (the smaller ``concentration``, the sharper, the deeper the tree); a candidate's score is the product along its path, and
    each round moves the ``width`` best candidates into the tree.
    """
    parent_of = [-1]
    dep = [1]
    score = [1.0]
    frontier = []  # (score, parent id) of candidate children not yet in the tree
    batch = [0]
    while len(parent_of) < T:
        for n in batch:
            if dep[n] < max_depth:
                pr = rng.dirichlet(np.full(fanout, concentration))
                frontier.extend((score[n] * float(pc), n) for pc in pr)
        if not frontier:
            raise ValueError("frontier exhausted")
        frontier.sort(key=lambda t: -t[0])
        take = frontier[: min(width, T - len(parent_of))]
        frontier = frontier[len(take):]
        batch = []
        for s, par in take:
            batch.append(len(parent_of))
            parent_of.append(par)
            dep.append(dep[par] + 1)
            score.append(s)
    return bfs_renumber(np.asarray(parent_of, dtype=np.int32))


# ----------------------------------------------------------------------------- tensors
def _softplus(x):
    return np.log1p(np.exp(-np.abs(x))) + np.maximum(x, 0.0)


def random_tensors(rng: np.random.Generator, B: int, N: int, h_qk: int, h_v: int, d_k: int, d_v: int, dtype: str):
    """Stored tensors with the benchmark value distributions.

    S0 ~ N(0, sd 0.1) fp32; q, k ~ N(0,1) L2-normalised per (node, head); v ~ N(0,1);
    g = -softplus(N(0,1)) (so exp(g) in (0,1)); beta = sigmoid(N(0,1)).  q,k,v,g,beta are rounded to ``dtype``.
    """
    S0 = (0.1 * rng.standard_normal((B, h_v, d_v, d_k), dtype=np.float32)).astype(np.float32)

    def unit(shape):
        x = rng.standard_normal(shape, dtype=np.float32)
        x /= np.sqrt(np.sum(x.astype(np.float64) ** 2, axis=-1, keepdims=True)).astype(np.float32)
        return x

    q = unit((N, h_qk, d_k))
    k = unit((N, h_qk, d_k))
    v = rng.standard_normal((N, h_v, d_v), dtype=np.float32)
    g = -_softplus(rng.standard_normal((N, h_v), dtype=np.float32))
    beta = 1.0 / (1.0 + np.exp(-rng.standard_normal((N, h_v), dtype=np.float32)))
    return S0, store(q, dtype), store(k, dtype), store(v, dtype), store(g, dtype), store(beta, dtype)


@dataclass
class Workload:
    """One batch of trees with its tensors (stored dtype) and one accepted path per tree."""
    name: str
    n_seq: int
    h_qk: int
    h_v: int
    d_k: int
    d_v: int
    in_dtype: str
    out_dtype: str
    scale: float
    S0: np.ndarray            # [B,H_v,d_v,d_k] fp32
    q: np.ndarray             # [N,H_k,d_k] stored dtype
    k: np.ndarray
    v: np.ndarray             # [N,H_v,d_v]
    g: np.ndarray             # [N,H_v]
    beta: np.ndarray
    parent: np.ndarray        # [N] int32, local ids
    node_offsets: np.ndarray  # [B+1] int32
    path: np.ndarray          # [sum L_b] int32, local ids root first
    path_offsets: np.ndarray  # [B+1] int32
    meta: dict = field(default_factory=dict)

    @property
    def total_nodes(self) -> int:
        return int(self.node_offsets[-1])

    def f64(self, name: str) -> np.ndarray:
        a = getattr(self, name)
        return a.astype(np.float64) if name == "S0" else widen(a, self.in_dtype)

    def algorithmic_bytes(self) -> int:
        """Bytes one verify+commit pass must move: S0 read + S_new write + q,k,v,g,beta read + o write."""
        isz = 4 if self.in_dtype == F32 else 2
        osz = 4 if self.out_dtype == F32 else 2
        N = self.total_nodes
        state = self.n_seq * self.h_v * self.d_v * self.d_k * 4
        return (2 * state + 2 * N * self.h_qk * self.d_k * isz + N * self.h_v * self.d_v * isz
                + 2 * N * self.h_v * isz + N * self.h_v * self.d_v * osz)


def _pack(trees):
    node_offsets = np.zeros(len(trees) + 1, dtype=np.int32)
    node_offsets[1:] = np.cumsum([len(t) for t in trees])
    parent = np.concatenate(trees).astype(np.int32) if trees else np.zeros(0, np.int32)
    return parent, node_offsets


def _pack_paths(paths):
    path_offsets = np.zeros(len(paths) + 1, dtype=np.int32)
    path_offsets[1:] = np.cumsum([len(p) for p in paths])
    path = np.concatenate(paths).astype(np.int32) if paths and path_offsets[-1] > 0 else np.zeros(0, np.int32)
    return path, path_offsets


def longest_path(parent: np.ndarray) -> np.ndarray:
    d = depths(parent)
    return root_path(parent, int(np.argmax(d)))  # argmax returns the lowest id among ties


def make_workload(name: str, trees, paths, h_qk: int, h_v: int, d_k: int, d_v: int, in_dtype: str, out_dtype: str,
                  rng: np.random.Generator, meta=None) -> Workload:
    parent, node_offsets = _pack(trees)
    path, path_offsets = _pack_paths(paths)
    B, N = len(trees), int(node_offsets[-1])
    S0, q, k, v, g, beta = random_tensors(rng, B, N, h_qk, h_v, d_k, d_v, in_dtype)
    return Workload(name, B, h_qk, h_v, d_k, d_v, in_dtype, out_dtype, float(1.0 / np.sqrt(d_k)), S0, q, k, v, g,
                    beta, parent, node_offsets, path, path_offsets, dict(meta or {}))


CONFIG_NAMES = {0: "cfg0_tiny_f32", 1: "cfg1_layer_T64", 2: "cfg2_stack48_T256", 3: "cfg3_ragged32",
                4: "cfg4_chains64x16", 5: "cfg1x48_stack48_T64"}


def config(idx: int, rep: int = 0, out_dtype: str | None = None, n_layers: int = 48) -> Workload:
    """The benchmark configurations.  0-4 are the five listed configurations; 5 is configuration 1's layer
    replicated over ``n_layers`` layer slots in one launch (all GDN heads of a 48-layer stack, 64-node tree, batch 1).
    """
    rng = np.random.Generator(np.random.PCG64(SEED_BASE + 101 * idx + rep))
    if idx == 0:
        t = tree_small_uniform(rng, 8, 3, 3)
        leaves = np.setdiff1d(np.arange(8), t[t >= 0])
        leaf = int(leaves[rng.integers(0, len(leaves))])
        return make_workload(CONFIG_NAMES[0], [t], [root_path(t, leaf)], 2, 4, 32, 32, F32, out_dtype or F32, rng)
    if idx == 1:
        t = tree_geo(rng, 64)
        return make_workload(CONFIG_NAMES[1], [t], [longest_path(t)], 16, 32, 128, 128, BF16, out_dtype or BF16, rng)
    if idx == 5:
        t = tree_geo(rng, 64)
        p = longest_path(t)
        return make_workload(CONFIG_NAMES[5], [t] * n_layers, [p] * n_layers, 16, 32, 128, 128, BF16,
                             out_dtype or BF16, rng, {"layers": n_layers})
    if idx == 2:
        t = tree_geo(rng, 256)
        d = depths(t)
        L = min(int(rng.integers(1, 17)), int(d.max()))
        cands = np.nonzero(d == L)[0]
        p = root_path(t, int(cands[rng.integers(0, len(cands))]))
        return make_workload(CONFIG_NAMES[2], [t] * n_layers, [p] * n_layers, 16, 32, 128, 128, BF16,
                             out_dtype or BF16, rng, {"layers": n_layers})
    if idx == 3:
        sizes = rng.integers(16, 257, size=32)
        trees = [tree_geo(rng, int(T)) for T in sizes]
        paths = [root_path(t, int(rng.integers(0, len(t)))) for t in trees]
        return make_workload(CONFIG_NAMES[3], trees, paths, 16, 32, 128, 128, BF16, out_dtype or BF16, rng)
    if idx == 4:
        trees = [tree_chain(16) for _ in range(64)]
        paths = [np.arange(int(rng.integers(0, 17)), dtype=np.int32) for _ in trees]
        return make_workload(CONFIG_NAMES[4], trees, paths, 16, 32, 128, 128, BF16, out_dtype or BF16, rng)
    raise ValueError(f"unknown configuration {idx}")


def layer_sweep(T: int, rep: int = 0, out_dtype: str = BF16) -> Workload:
    """One layer with configuration 1's head shapes and a GEO tree of ``T`` nodes (the tree-size sweep of the
    paper's Table 1 / Figure 5: budgets 32..512); accepted path = longest root path."""
    rng = np.random.Generator(np.random.PCG64(SEED_BASE + 101 * 6 + 7 * T + rep))
    t = tree_geo(rng, T)
    return make_workload(f"layer_T{T}", [t], [longest_path(t)], 16, 32, 128, 128, BF16, out_dtype, rng)


def deep_stack(path_len: int, n_layers: int = 48, rep: int = 0, out_dtype: str = BF16) -> Workload:
    """Configuration "1x48" with a 64-node best-first tree that reaches depth 16 and an accepted path of exactly
    ``path_len`` nodes (the first nodes of its deepest root path; 0..16): the accepted-length sweep of the commit."""
    rng = np.random.Generator(np.random.PCG64(SEED_BASE + 101 * 7 + rep))
    # a spine of 16 nodes (one accepted candidate per depth) with the rest of the 64-node budget hanging off its first
    # 15 nodes as rejected siblings, three or four each: the shape of a deep, narrow best-first tree
    t = bfs_renumber(np.asarray([i - 1 for i in range(16)] + [i % 15 for i in range(48)], np.int32))
    p = longest_path(t)[:path_len]
    return make_workload(f"stack{n_layers}_T64_deep_L{path_len}", [t] * n_layers, [p] * n_layers, 16, 32, 128, 128, BF16,
                         out_dtype, rng, {"layers": n_layers})


def bestfirst_stack(n_layers: int = 48, rep: int = 0, out_dtype: str = BF16, T: int = 64) -> Workload:
    """Configuration "1x48" with the tree shape of Algorithm 1 (width-4 best-first expansion, fan-out 8, depth cap
    16, seeded synthetic child probabilities) instead of the geometric one: deeper root paths, the report-only
    second shape of the headline workload.  Accepted path = longest root path."""
    rng = np.random.Generator(np.random.PCG64(SEED_BASE + 101 * 8 + rep))
    t = tree_bestfirst(rng, T, concentration=0.1)   # accepted lengths of 12-14, as the paper reports for 64-node trees
    p = longest_path(t)
    return make_workload(f"stack{n_layers}_T{T}_bestfirst", [t] * n_layers, [p] * n_layers, 16, 32, 128, 128, BF16,
                         out_dtype, rng, {"layers": n_layers})


@dataclass
class PaddedWorkload:
    """A batch in the padded layout of Section 3.4.2: ``n_slots`` slots of ``t_pad`` rows, slot ``s`` carrying tree
    ``s % n_trees``; node tensors ``[n_slots, t_pad, heads, d]`` (bf16 bit patterns), ``g_in / beta_in`` either finished
    gates or raw gate inputs; one accepted path per tree, padded to ``MAX_DEPTH`` entries."""
    n_slots: int
    n_trees: int
    t_pad: int
    h_qk: int
    h_v: int
    d: int
    raw_gates: bool
    out_dtype: str
    scale: float
    S0: np.ndarray
    q: np.ndarray
    k: np.ndarray
    v: np.ndarray
    g_in: np.ndarray
    beta_in: np.ndarray
    parent: np.ndarray
    n_nodes: np.ndarray
    path: np.ndarray
    path_len: np.ndarray

    def f64(self, name: str) -> np.ndarray:
        a = getattr(self, name)
        return a.astype(np.float64) if a.dtype != np.uint16 else bf16_bits_to_f32(a).astype(np.float64)


def padded_case(seed: int, trees, n_layers: int, t_pad: int, raw_gates: bool, h_qk: int = 2, h_v: int = 4,
                out_dtype: str = BF16, paths=None, poison_padding: bool = True) -> PaddedWorkload:
    """Seeded padded batch: ``len(trees)`` trees shared by ``n_layers`` slots each (slot order: layer-major, so slot
    ``s`` carries tree ``s % len(trees)``), every slot with its own state and node tensors.  Rows beyond a tree's node
    count hold NaN in q, k, v, g, beta when ``poison_padding`` (nothing may depend on them) and parent entries there
    are out of range.  Accepted path per tree: ``paths[i]`` or the longest root path."""
    rng = np.random.Generator(np.random.PCG64(SEED_BASE + 7919 * seed))
    n_trees, d = len(trees), 128
    B = n_trees * n_layers
    S0, q, k, v, g, beta = random_tensors(rng, B, B * t_pad, h_qk, h_v, d, d, BF16)
    if raw_gates:   # the layer's gate inputs themselves, N(0,1), in the storage type
        g = store(rng.standard_normal((B * t_pad, h_v), dtype=np.float32), BF16)
        beta = store(rng.standard_normal((B * t_pad, h_v), dtype=np.float32), BF16)
    shape4 = lambda x: x.reshape((B, t_pad) + x.shape[1:])
    q, k, v, g, beta = (shape4(x).copy() for x in (q, k, v, g, beta))
    parent = np.full((n_trees, t_pad), 12345, np.int32)
    n_nodes = np.zeros(n_trees, np.int32)
    path = np.zeros((n_trees, MAX_DEPTH), np.int32)
    path_len = np.zeros(n_trees, np.int32)
    for i, t in enumerate(trees):
        assert len(t) <= t_pad
        parent[i, : len(t)] = t
        n_nodes[i] = len(t)
        pth = longest_path(t) if paths is None else np.asarray(paths[i], np.int32)
        path[i, : len(pth)] = pth
        path_len[i] = len(pth)
    if poison_padding:
        nan_bits = np.uint16(0x7FC0)
        for s_ in range(B):
            n = int(n_nodes[s_ % n_trees])
            for x in (q, k, v, g, beta):
                x[s_, n:] = nan_bits
    return PaddedWorkload(B, n_trees, t_pad, h_qk, h_v, d, raw_gates, out_dtype, 1.0 / np.sqrt(d), S0, q, k, v, g, beta,
                          parent, n_nodes, path, path_len)


def random_case(seed: int, trees, h_qk, h_v, d_k, d_v, in_dtype=F32, out_dtype=F32, paths=None, name="case"):
    """A free-form case for tests: given trees, random accepted root paths unless ``paths`` is given."""
    rng = np.random.Generator(np.random.PCG64(seed))
    if paths is None:
        paths = [root_path(t, int(rng.integers(0, len(t)))) if len(t) else np.zeros(0, np.int32) for t in trees]
    return make_workload(name, list(trees), list(paths), h_qk, h_v, d_k, d_v, in_dtype, out_dtype, rng)

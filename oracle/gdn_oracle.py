"""ctypes front end of the fp64 CPU oracle (``gdn_oracle.c``).

TEST INFRASTRUCTURE ONLY: imported by the tests, the smoke check and the CPU
baseline leg of the benchmark.  It imports nothing from the CUDA package and
the CUDA package imports nothing from here.

The oracle evaluates, for every node of every draft tree, the gated delta rule
of Eq. 7 along the node's root path starting from the committed state, then
Eq. 8 for the output; commit replays Eq. 7 along one accepted root path
(Section 3.4.1 and the end of Section 3.4.2).  All arithmetic is fp64; inputs
are the stored (fp32 or bf16-rounded) values widened exactly.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "gdn_oracle.c")
_LIB = os.path.join(_HERE, "libgdn_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile ``gdn_oracle.c`` with gcc into ``libgdn_oracle.so`` next to it."""
    if not force and os.path.exists(_LIB) and os.path.getmtime(_LIB) >= os.path.getmtime(_SRC):
        return _LIB
    tmp = _LIB + f".{os.getpid()}.tmp"
    subprocess.check_call(
        ["gcc", "-O2", "-std=c99", "-fopenmp", "-fPIC", "-shared", "-o", tmp, _SRC, "-lm"]
    )
    os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        dp = ctypes.POINTER(ctypes.c_double)
        ip = ctypes.POINTER(ctypes.c_int32)
        lib.gdn_oracle_threads.restype = ctypes.c_int
        lib.gdn_oracle_verify.restype = ctypes.c_int
        lib.gdn_oracle_verify.argtypes = [ctypes.c_int] * 5 + [ctypes.c_double] + [dp] * 6 + [ip, ip, dp,
                                                                                            ctypes.c_int, ctypes.c_int]
        lib.gdn_oracle_commit.restype = ctypes.c_int
        lib.gdn_oracle_commit.argtypes = [ctypes.c_int] * 5 + [dp] * 5 + [ip] * 4 + [dp]
        lib.gdn_oracle_gates.restype = None
        lib.gdn_oracle_gates.argtypes = [ctypes.c_int64, dp, dp, dp, dp]
        _lib = lib
    return _lib


def _f64(a, shape):
    a = np.ascontiguousarray(a, dtype=np.float64)
    assert a.shape == tuple(shape), (a.shape, shape)
    return a


def _i32(a, n):
    a = np.ascontiguousarray(a, dtype=np.int32)
    assert a.shape == (n,), (a.shape, n)
    return a


def _dp(a):
    return a.ctypes.data_as(ctypes.POINTER(ctypes.c_double))


def _ip(a):
    return a.ctypes.data_as(ctypes.POINTER(ctypes.c_int32))


def threads() -> int:
    """Number of host threads the oracle's OpenMP loops use."""
    return int(_load().gdn_oracle_threads())


def verify(S0, q, k, v, g, beta, parent, node_offsets, scale, first_seq=0, n_do=None):
    """Per-node outputs ``o [N, H_v, d_v]`` (fp64) by re-running Eq. 7 over each root path, then Eq. 8.

    ``S0 [B,H_v,d_v,d_k]``, ``q,k [N,H_k,d_k]``, ``v [N,H_v,d_v]``, ``g,beta [N,H_v]``,
    ``parent [N]`` (local ids, -1 = root), ``node_offsets [B+1]``.  With ``n_do`` set only
    sequences ``first_seq .. first_seq+n_do-1`` are evaluated (other rows of ``o`` stay zero).
    """
    lib = _load()
    B, h_v, d_v, d_k = np.shape(S0)
    N, h_qk, _ = np.shape(q)
    node_offsets = _i32(node_offsets, B + 1)
    assert int(node_offsets[-1]) == N
    S0 = _f64(S0, (B, h_v, d_v, d_k))
    q = _f64(q, (N, h_qk, d_k))
    k = _f64(k, (N, h_qk, d_k))
    v = _f64(v, (N, h_v, d_v))
    g = _f64(g, (N, h_v))
    beta = _f64(beta, (N, h_v))
    parent = _i32(parent, N)
    o = np.zeros((N, h_v, d_v), dtype=np.float64)
    if n_do is None:
        n_do = B - first_seq
    assert 0 <= first_seq and first_seq + n_do <= B
    rc = lib.gdn_oracle_verify(B, h_qk, h_v, d_k, d_v, float(scale), _dp(S0), _dp(q), _dp(k), _dp(v), _dp(g),
                               _dp(beta), _ip(parent), _ip(node_offsets), _dp(o), first_seq, n_do)
    if rc != 0:
        raise ValueError(f"gdn_oracle_verify failed with code {rc}")
    return o


def commit(S0, k, v, g, beta, parent, node_offsets, path, path_offsets):
    """Post-acceptance state ``S_new [B,H_v,d_v,d_k]`` (fp64): Eq. 7 replayed along each accepted root path."""
    lib = _load()
    B, h_v, d_v, d_k = np.shape(S0)
    N, h_qk, _ = np.shape(k)
    node_offsets = _i32(node_offsets, B + 1)
    path_offsets = _i32(path_offsets, B + 1)
    path = _i32(path, int(path_offsets[-1]))
    S0 = _f64(S0, (B, h_v, d_v, d_k))
    k = _f64(k, (N, h_qk, d_k))
    v = _f64(v, (N, h_v, d_v))
    g = _f64(g, (N, h_v))
    beta = _f64(beta, (N, h_v))
    parent = _i32(parent, N)
    S_new = np.empty_like(S0)
    if path.size == 0:
        path = np.zeros(1, dtype=np.int32)  # keep a valid pointer for an all-empty batch
    rc = lib.gdn_oracle_commit(B, h_qk, h_v, d_k, d_v, _dp(S0), _dp(k), _dp(v), _dp(g), _dp(beta), _ip(parent),
                               _ip(node_offsets), _ip(path), _ip(path_offsets), _dp(S_new))
    if rc != 0:
        raise ValueError(f"gdn_oracle_commit failed with code {rc}")
    return S_new


def gates(a_raw, b_raw):
    """Gate activations of the "scalars" stage (Section 3.4.2): ``g = -softplus(a_raw)``, ``beta = sigmoid(b_raw)``,
    elementwise in fp64.  Returns ``(g, beta)`` with the shape of the inputs."""
    lib = _load()
    a = np.ascontiguousarray(a_raw, dtype=np.float64)
    b = np.ascontiguousarray(b_raw, dtype=np.float64)
    assert a.shape == b.shape
    g, beta = np.empty_like(a), np.empty_like(b)
    lib.gdn_oracle_gates(a.size, _dp(a), _dp(b), _dp(g), _dp(beta))
    return g, beta


def _unpad(n_slots, n_trees, t_pad, n_nodes, parent_pad):
    """Row indices (into the flattened ``[n_slots * t_pad]`` node axis), packed ``parent`` and ``node_offsets`` of the
    padded layout of Section 3.4.2: slot ``s`` carries tree ``s % n_trees`` in its first ``n_nodes[tree]`` rows."""
    n_nodes = np.asarray(n_nodes, dtype=np.int64)
    parent_pad = np.asarray(parent_pad, dtype=np.int32).reshape(n_trees, t_pad)
    rows, parents, offs = [], [], [0]
    for s in range(n_slots):
        tr = s % n_trees
        T = int(n_nodes[tr])
        assert 0 <= T <= t_pad
        rows.append(np.arange(s * t_pad, s * t_pad + T, dtype=np.int64))
        parents.append(parent_pad[tr, :T])
        offs.append(offs[-1] + T)
    return (np.concatenate(rows) if rows else np.zeros(0, np.int64),
            np.concatenate(parents).astype(np.int32) if parents else np.zeros(0, np.int32),
            np.asarray(offs, dtype=np.int32))


def verify_padded(S0, q, k, v, g_in, beta_in, parent_pad, n_nodes, scale, raw_gates):
    """Verification in the padded layout of Section 3.4.2: ``q,k [B,T,H_k,d_k]``, ``v [B,T,H_v,d_v]``, ``g_in, beta_in
    [B,T,H_v]`` (raw gate inputs if ``raw_gates``), ``parent_pad [n_trees,T]``, ``n_nodes [n_trees]``; slot ``s`` carries
    tree ``s % n_trees``.  Returns ``o [B,T,H_v,d_v]`` (rows beyond a tree's node count are zero).  The padded tensors
    are unpacked to the ragged form and handed to :func:`verify`: only indices move here."""
    B, T = np.shape(q)[:2]
    n_trees = len(n_nodes)
    rows, parent, offs = _unpad(B, n_trees, T, n_nodes, parent_pad)
    flat = lambda x: np.asarray(x, dtype=np.float64).reshape((B * T,) + tuple(np.shape(x)[2:]))[rows]
    g, beta = flat(g_in), flat(beta_in)
    if raw_gates:
        g, beta = gates(g, beta)
    o_r = verify(S0, flat(q), flat(k), flat(v), g, beta, parent, offs, scale)
    o = np.zeros((B * T,) + o_r.shape[1:], dtype=np.float64)
    o[rows] = o_r
    return o.reshape((B, T) + o_r.shape[1:])


def commit_padded(S0, k, v, g_in, beta_in, parent_pad, n_nodes, path_pad, path_len, raw_gates):
    """Commit in the padded layout: ``path_pad [n_trees, max_depth]``, ``path_len [n_trees]`` (every slot of a tree
    commits that tree's accepted path).  Returns ``S_new``."""
    B, T = np.shape(k)[:2]
    n_trees = len(n_nodes)
    rows, parent, offs = _unpad(B, n_trees, T, n_nodes, parent_pad)
    flat = lambda x: np.asarray(x, dtype=np.float64).reshape((B * T,) + tuple(np.shape(x)[2:]))[rows]
    g, beta = flat(g_in), flat(beta_in)
    if raw_gates:
        g, beta = gates(g, beta)
    path_pad = np.asarray(path_pad, dtype=np.int32).reshape(n_trees, -1)
    paths = [path_pad[s % n_trees, : int(path_len[s % n_trees])] for s in range(B)]
    poffs = np.concatenate([[0], np.cumsum([len(p) for p in paths])]).astype(np.int32)
    path = np.concatenate(paths).astype(np.int32) if paths else np.zeros(0, np.int32)
    return commit(S0, flat(k), flat(v), g, beta, parent, offs, path, poffs)

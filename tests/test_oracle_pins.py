"""Pins of the fp64 CPU oracle against things other than itself (all CPU, no CUDA).

Each pin is chosen so that a plausible mistake in ``oracle/gdn_oracle.c`` -- a dropped term, a wrong sign, a
transposed operand, a wrong head mapping, an exclusive instead of inclusive decay -- fails at least one of them:

* dense-matrix brute force of Eq. 7/8 with numpy matmul on tiny sizes;
* the triangular ("chunk") form of Eq. 9-11 through a dense linear solve -- an independent formulation;
* the closed-form end state of Eq. 12 restricted to the accepted path;
* a hand-worked scalar tree (tests/golden/scalar_tree_example.json);
* chain tree == token-by-token decoding with a carried state;
* invariance under renumbering of the tree; composition commit-then-verify;
* closed forms: beta = 0, zero state, orthonormal keys (exact recall), norm contraction.
"""
import json
import os

import numpy as np
import pytest

from oracle import gdn_oracle as orc
from paper_2607_06763_b200 import synth

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _case(seed, trees, h_qk=2, h_v=4, d_k=4, d_v=3, paths=None):
    w = synth.random_case(seed, trees, h_qk, h_v, d_k, d_v, paths=paths)
    return w


def _verify(w, **kw):
    return orc.verify(w.f64("S0"), w.f64("q"), w.f64("k"), w.f64("v"), w.f64("g"), w.f64("beta"), w.parent,
                      w.node_offsets, w.scale, **kw)


def _commit(w, path=None, path_offsets=None):
    return orc.commit(w.f64("S0"), w.f64("k"), w.f64("v"), w.f64("g"), w.f64("beta"), w.parent, w.node_offsets,
                      w.path if path is None else path, w.path_offsets if path_offsets is None else path_offsets)


def _trees(seed):
    rng = np.random.default_rng(seed)
    return [synth.tree_small_uniform(rng, 8, 3, 3), synth.tree_geo(rng, 7, max_depth=4), synth.tree_chain(5),
            synth.tree_star(6), np.array([-1, -1, 0, 1, 1], dtype=np.int32)]  # last one is a forest


# ------------------------------------------------------------------ 1. dense-matrix brute force
def _brute_states(w, b, h):
    """S_i (d_k x d_v) for every node of tree b, head h, by explicit matrix products A_n S + B_n."""
    rep = w.h_v // w.h_qk
    base = int(w.node_offsets[b])
    T = int(w.node_offsets[b + 1]) - base
    S0 = w.f64("S0")[b, h].T  # memory [d_v][d_k] -> d_k x d_v
    k, v, g, beta = w.f64("k"), w.f64("v"), w.f64("g"), w.f64("beta")
    eye = np.eye(w.d_k)
    states = []
    for i in range(T):
        p = int(w.parent[base + i])
        Sp = S0 if p < 0 else states[p]
        kk = k[base + i, h // rep][:, None]
        vv = v[base + i, h][None, :]
        A = np.exp(g[base + i, h]) * (eye - beta[base + i, h] * (kk @ kk.T))
        states.append(A @ Sp + beta[base + i, h] * (kk @ vv))
    return states


@pytest.mark.parametrize("seed", [1, 2, 3])
def test_brute_force_dense_matrices(seed):
    w = _case(seed, _trees(seed))
    o = _verify(w)
    rep = w.h_v // w.h_qk
    q = w.f64("q")
    for b in range(w.n_seq):
        base = int(w.node_offsets[b])
        for h in range(w.h_v):
            states = _brute_states(w, b, h)
            for i, S in enumerate(states):
                want = w.scale * (q[base + i, h // rep] @ S)
                np.testing.assert_allclose(o[base + i, h], want, rtol=1e-12, atol=1e-13)
    S_new = _commit(w)
    for b in range(w.n_seq):
        L = int(w.path_offsets[b + 1] - w.path_offsets[b])
        leaf = int(w.path[w.path_offsets[b + 1] - 1]) if L else None
        for h in range(w.h_v):
            want = w.f64("S0")[b, h].T if leaf is None else _brute_states(w, b, h)[leaf]
            np.testing.assert_allclose(S_new[b, h].T, want, rtol=1e-12, atol=1e-13)


# ------------------------------------------------------------------ 2./3. triangular form, Eq. 9-12
def _wy(w, b, h):
    """Eq. 9-11 for tree b, head h via a dense solve; returns (O [T,d_v], Utilde [T,d_v], a [T], anc mask)."""
    rep = w.h_v // w.h_qk
    base = int(w.node_offsets[b])
    T = int(w.node_offsets[b + 1]) - base
    par = w.parent[base:base + T]
    anc = np.zeros((T, T), dtype=bool)  # anc[i, j] : j is a proper ancestor of i
    for i in range(T):
        p = par[i]
        while p >= 0:
            anc[i, p] = True
            p = par[p]
    K = w.f64("k")[base:base + T, h // rep]
    Q = w.f64("q")[base:base + T, h // rep]
    V = w.f64("v")[base:base + T, h]
    g = w.f64("g")[base:base + T, h]
    beta = w.f64("beta")[base:base + T, h]
    S0 = w.f64("S0")[b, h].T
    G = np.array([g[i] + g[anc[i]].sum() for i in range(T)])  # inclusive path sums
    a = np.exp(G)
    ratio = a[:, None] / a[None, :]
    X = anc * ratio * beta[:, None] * (K @ K.T)
    Y = (anc | np.eye(T, dtype=bool)) * ratio * (Q @ K.T)
    IX = np.eye(T) + X
    U = np.linalg.solve(IX, beta[:, None] * V)
    W = np.linalg.solve(IX, (beta * a)[:, None] * K)
    Ut = U - W @ S0
    O = w.scale * (a[:, None] * (Q @ S0) + Y @ Ut)
    return O, Ut, a, anc, K, S0


@pytest.mark.parametrize("seed", [11, 12])
def test_triangular_form_eq9_to_eq11(seed):
    rng = np.random.default_rng(seed)
    trees = _trees(seed) + [synth.tree_geo(rng, 12, max_depth=6)]
    w = _case(seed, trees, h_qk=1, h_v=2, d_k=5, d_v=4)
    o = _verify(w)
    for b in range(w.n_seq):
        base, end = int(w.node_offsets[b]), int(w.node_offsets[b + 1])
        for h in range(w.h_v):
            O = _wy(w, b, h)[0]
            np.testing.assert_allclose(o[base:end, h], O, rtol=1e-11, atol=1e-13)


@pytest.mark.parametrize("seed", [21, 22])
def test_end_state_closed_form_eq12_masked(seed):
    w = _case(seed, _trees(seed), h_qk=2, h_v=2, d_k=4, d_v=5)
    S_new = _commit(w)
    for b in range(w.n_seq):
        L = int(w.path_offsets[b + 1] - w.path_offsets[b])
        if L == 0:
            continue
        n = int(w.path[w.path_offsets[b + 1] - 1])
        for h in range(w.h_v):
            _, Ut, a, anc, K, S0 = _wy(w, b, h)
            on_path = anc[n].copy()
            on_path[n] = True
            want = a[n] * S0 + K.T @ (on_path[:, None] * (a[n] / a)[:, None] * Ut)
            np.testing.assert_allclose(S_new[b, h].T, want, rtol=1e-11, atol=1e-13)


# ------------------------------------------------------------------ hand-worked example
def test_hand_worked_scalar_tree():
    gold = json.load(open(os.path.join(GOLDEN, "scalar_tree_example.json")))
    T = len(gold["parent"])
    col = lambda key: np.asarray(gold[key], dtype=np.float64).reshape(T, 1, 1)
    S0 = np.full((1, 1, 1, 1), gold["S0"])
    g = np.log(np.asarray(gold["alpha"])).reshape(T, 1)
    beta = np.asarray(gold["beta"]).reshape(T, 1)
    parent = np.asarray(gold["parent"], dtype=np.int32)
    off = np.array([0, T], dtype=np.int32)
    o = orc.verify(S0, col("q"), col("k"), col("v"), g, beta, parent, off, 1.0)
    np.testing.assert_allclose(o.ravel(), gold["o"], rtol=0, atol=1e-15)
    for key, want in gold["commit"].items():
        path = np.asarray(json.loads(key), dtype=np.int32)
        S = orc.commit(S0, col("k"), col("v"), g, beta, parent, off, path, np.array([0, len(path)], np.int32))
        assert abs(S.item() - want) < 1e-15, (key, S.item(), want)
    # the solve result printed in the fixture, through the triangular form
    w = synth.random_case(0, [parent], 1, 1, 1, 1)
    w.S0[:] = gold["S0"]
    w.q, w.k, w.v = (np.asarray(gold[n], np.float32).reshape(T, 1, 1) for n in ("q", "k", "v"))
    w.g, w.beta, w.scale = g.astype(np.float32), beta.astype(np.float32), 1.0
    np.testing.assert_allclose(_wy(w, 0, 0)[1].ravel(), gold["u_tilde"], atol=1e-6)


# ------------------------------------------------------------------ chain == sequential decoding
def test_chain_equals_sequential_decoding():
    T = 9
    w = _case(31, [synth.tree_chain(T)], h_qk=2, h_v=4, d_k=6, d_v=5, paths=[np.arange(T, dtype=np.int32)])
    o = _verify(w)
    rep = w.h_v // w.h_qk
    q, k, v, g, beta = (w.f64(n) for n in ("q", "k", "v", "g", "beta"))
    for h in range(w.h_v):
        S = w.f64("S0")[0, h].T.copy()
        for t in range(T):  # one decode step per token, state carried
            kt = k[t, h // rep]
            S = np.exp(g[t, h]) * S
            S = S + beta[t, h] * np.outer(kt, v[t, h] - kt @ S)
            np.testing.assert_allclose(o[t, h], w.scale * (q[t, h // rep] @ S), rtol=1e-12, atol=1e-14)
            Sc = _commit(w, np.arange(t + 1, dtype=np.int32), np.array([0, t + 1], np.int32))
            np.testing.assert_allclose(Sc[0, h].T, S, rtol=1e-12, atol=1e-14)
    S_empty = _commit(w, np.zeros(0, np.int32), np.array([0, 0], np.int32))
    np.testing.assert_array_equal(S_empty, w.f64("S0"))


# ------------------------------------------------------------------ renumbering / sibling order
def test_invariance_under_topological_renumbering():
    rng = np.random.default_rng(41)
    t = synth.tree_geo(rng, 14, max_depth=5)
    w = _case(41, [t], h_qk=1, h_v=2, d_k=4, d_v=4)
    o = _verify(w)
    T = len(t)
    # random valid renumbering: repeatedly pick any node whose parent is already placed
    placed, order = set(), []
    while len(order) < T:
        ready = [i for i in range(T) if i not in placed and (t[i] < 0 or t[i] in placed)]
        pick = ready[rng.integers(0, len(ready))]
        placed.add(pick)
        order.append(pick)
    order = np.asarray(order)
    new_id = np.empty(T, dtype=np.int64)
    new_id[order] = np.arange(T)
    w2 = _case(41, [t], h_qk=1, h_v=2, d_k=4, d_v=4)
    w2.parent = np.asarray([-1 if t[old] < 0 else new_id[t[old]] for old in order], dtype=np.int32)
    for name in ("q", "k", "v", "g", "beta"):
        setattr(w2, name, getattr(w, name)[order])
    assert not np.array_equal(order, np.arange(T))
    o2 = _verify(w2)
    np.testing.assert_allclose(o2, o[order], rtol=1e-13, atol=1e-15)


def test_commit_then_single_node_equals_child_in_tree():
    rng = np.random.default_rng(51)
    t = synth.tree_geo(rng, 10, max_depth=4)
    w = _case(51, [t], h_qk=2, h_v=2, d_k=3, d_v=4)
    o = _verify(w)
    child = int(np.nonzero(t >= 0)[0][-1])
    par_path = synth.root_path(t, int(t[child]))
    S_mid = _commit(w, par_path, np.array([0, len(par_path)], np.int32))
    one = np.array([-1], dtype=np.int32)
    sl = slice(child, child + 1)
    o1 = orc.verify(S_mid, w.f64("q")[sl], w.f64("k")[sl], w.f64("v")[sl], w.f64("g")[sl], w.f64("beta")[sl], one,
                    np.array([0, 1], np.int32), w.scale)
    np.testing.assert_allclose(o1[0], o[child], rtol=1e-12, atol=1e-14)


# ------------------------------------------------------------------ closed forms
def test_beta_zero_is_pure_decay():
    w = _case(61, _trees(61))
    w.beta = np.zeros_like(w.beta)
    o = _verify(w)
    S_new = _commit(w)
    rep = w.h_v // w.h_qk
    g, q = w.f64("g"), w.f64("q")
    for b in range(w.n_seq):
        base = int(w.node_offsets[b])
        T = int(w.node_offsets[b + 1]) - base
        for i in range(T):
            chain = synth.root_path(w.parent[base:base + T], i) + base
            for h in range(w.h_v):
                a = np.exp(g[chain, h].sum())
                want = w.scale * a * (w.f64("S0")[b, h] @ q[base + i, h // rep])
                np.testing.assert_allclose(o[base + i, h], want, rtol=1e-12, atol=1e-14)
        chain = w.path[w.path_offsets[b]:w.path_offsets[b + 1]] + base
        for h in range(w.h_v):
            np.testing.assert_allclose(S_new[b, h], np.exp(g[chain, h].sum()) * w.f64("S0")[b, h], rtol=1e-12)


def test_zero_state_single_node():
    w = _case(71, [np.array([-1], np.int32)], h_qk=2, h_v=4, d_k=4, d_v=3)
    w.S0[:] = 0
    o = _verify(w)
    rep = w.h_v // w.h_qk
    for h in range(w.h_v):
        qk = w.f64("q")[0, h // rep] @ w.f64("k")[0, h // rep]
        np.testing.assert_allclose(o[0, h], w.scale * w.f64("beta")[0, h] * qk * w.f64("v")[0, h], rtol=1e-12)


def test_orthonormal_keys_exact_recall():
    """g = 0, beta = 1, orthonormal keys: the state stores v_j under k_j, so q_i = k_j (j on the root path of i)
    returns scale * v_j whatever S0 was along the other directions."""
    rng = np.random.default_rng(81)
    t = synth.tree_geo(rng, 6, max_depth=4)
    d_k = 6
    w = _case(81, [t], h_qk=1, h_v=2, d_k=d_k, d_v=3)
    Qm, _ = np.linalg.qr(rng.standard_normal((d_k, d_k)))
    w.k = Qm.astype(np.float32)[: len(t), None, :]
    w.g = np.zeros_like(w.g)
    w.beta = np.ones_like(w.beta)
    for i in range(len(t)):
        chain = synth.root_path(t, i)
        for j in chain:
            w.q = w.k.copy()
            w.q[i] = w.k[j]
            o = _verify(w)
            for h in range(w.h_v):
                np.testing.assert_allclose(o[i, h], w.scale * w.f64("v")[j, h], rtol=1e-6, atol=1e-7)


def test_state_norm_contracts_without_writes():
    w = _case(91, _trees(91), h_qk=2, h_v=2, d_k=5, d_v=4)
    w.v = np.zeros_like(w.v)
    S_new = _commit(w)
    g = w.f64("g")
    for b in range(w.n_seq):
        chain = w.path[w.path_offsets[b]:w.path_offsets[b + 1]] + int(w.node_offsets[b])
        for h in range(w.h_v):
            bound = np.exp(g[chain, h].sum()) * np.linalg.norm(w.f64("S0")[b, h])
            assert np.linalg.norm(S_new[b, h]) <= bound * (1 + 1e-12)


# ------------------------------------------------------------------ argument checks and sampling
def test_rejects_bad_trees_and_paths():
    w = _case(101, [synth.tree_chain(4)])
    bad = w.parent.copy()
    bad[2] = 3
    with pytest.raises(ValueError):
        orc.verify(w.f64("S0"), w.f64("q"), w.f64("k"), w.f64("v"), w.f64("g"), w.f64("beta"), bad, w.node_offsets, 1.0)
    with pytest.raises(ValueError):
        _commit(w, np.array([1, 2], np.int32), np.array([0, 2], np.int32))  # does not start at a root
    with pytest.raises(ValueError):
        _commit(w, np.array([0, 2], np.int32), np.array([0, 2], np.int32))  # 2 is not a child of 0


def test_sequence_sampling_matches_full_run():
    w = _case(111, _trees(111))
    full = _verify(w)
    part = _verify(w, first_seq=1, n_do=2)
    lo, hi = int(w.node_offsets[1]), int(w.node_offsets[3])
    np.testing.assert_array_equal(part[lo:hi], full[lo:hi])
    assert not part[:lo].any() and not part[hi:].any()


# ------------------------------------------------------------------ gate activations and the padded layout
def test_gate_activations_functional_equations_and_limits():
    """g = -softplus(a), beta = sigmoid(b): pinned by what fixes the two functions -- values at 0, the reflection
    identities, the derivative relation softplus' = sigmoid, and the asymptotes for large arguments."""
    x = np.linspace(-30.0, 30.0, 2401)
    g, beta = orc.gates(x, x)
    sp = -g
    g_neg, beta_neg = orc.gates(-x, -x)
    assert orc.gates(np.zeros(1), np.zeros(1))[0][0] == pytest.approx(-np.log(2.0), abs=1e-16)
    assert orc.gates(np.zeros(1), np.zeros(1))[1][0] == 0.5
    np.testing.assert_allclose(beta + beta_neg, 1.0, rtol=0, atol=5e-16)            # sigmoid(-x) = 1 - sigmoid(x)
    np.testing.assert_allclose(sp - (-g_neg), x, rtol=0, atol=1e-13)                # softplus(x) - softplus(-x) = x
    np.testing.assert_allclose(np.exp(-sp), beta_neg, rtol=1e-13, atol=1e-300)      # e^{-softplus(x)} = sigmoid(-x)
    h = x[1] - x[0]
    np.testing.assert_allclose((sp[2:] - sp[:-2]) / (2 * h), beta[1:-1], rtol=0, atol=2e-5)   # d softplus = sigmoid
    big = np.array([50.0, 200.0, 745.0])
    gb, bb = orc.gates(big, big)
    np.testing.assert_allclose(-gb, big, rtol=1e-15)
    assert np.all(bb == 1.0) or np.all(1.0 - bb < 1e-20)
    gs, bs = orc.gates(-big, -big)
    np.testing.assert_allclose(-gs, np.exp(-big), rtol=1e-12, atol=0)
    np.testing.assert_allclose(bs, np.exp(-big), rtol=1e-12, atol=0)
    assert np.all(np.isfinite(orc.gates(np.array([-1e4, 1e4]), np.array([-1e4, 1e4]))[0]))


def test_gate_activations_against_library_routines():
    scipy_special = pytest.importorskip("scipy.special")
    rng = np.random.default_rng(3)
    x = rng.normal(size=4000) * 6.0
    g, beta = orc.gates(x, x)
    np.testing.assert_allclose(-g, np.logaddexp(0.0, x), rtol=1e-14, atol=1e-300)
    np.testing.assert_allclose(beta, scipy_special.expit(x), rtol=1e-14, atol=1e-300)


def test_hand_worked_scalar_tree_through_raw_gates_and_padded_layout():
    """The hand example again, now entering through the raw gate inputs and the padded [slots, T, ...] layout with
    three slots sharing the one tree (T padded to 6).  alpha = .5 <-> a = 0 (softplus(0) = ln 2), alpha = .25 <-> a =
    ln 3, beta = .5 <-> b = 0; alpha = 1 and beta in {0, 1} are reached in the limit, here |raw| = 40 (off by 4e-18)."""
    ex = json.load(open(os.path.join(os.path.dirname(__file__), "golden", "scalar_tree_example.json")))
    a_raw = {0.5: 0.0, 1.0: -40.0, 0.25: np.log(3.0)}
    b_raw = {0.5: 0.0, 1.0: 40.0, 0.0: -40.0}
    T, B = 6, 3
    pad = lambda vals, fill=0.0: np.array(list(vals) + [fill] * (T - len(vals)))
    a = np.tile(pad([a_raw[x] for x in ex["alpha"]], 7.0)[None, :, None], (B, 1, 1))
    b = np.tile(pad([b_raw[x] for x in ex["beta"]], -3.0)[None, :, None], (B, 1, 1))
    k = np.tile(pad(ex["k"], 5.0)[None, :, None, None], (B, 1, 1, 1))
    v = np.tile(pad(ex["v"], 5.0)[None, :, None, None], (B, 1, 1, 1))
    q = np.tile(pad(ex["q"], 5.0)[None, :, None, None], (B, 1, 1, 1))
    parent = np.array([ex["parent"] + [0, 0]], dtype=np.int32)      # the padding rows carry garbage parents
    S0 = np.full((B, 1, 1, 1), ex["S0"])
    o = orc.verify_padded(S0, q, k, v, a, b, parent, [4], 1.0, raw_gates=True)
    for s in range(B):
        np.testing.assert_allclose(o[s, :4, 0, 0], ex["o"], rtol=0, atol=1e-15)
        assert np.all(o[s, 4:] == 0.0)
    for key, want in ex["commit"].items():
        path = json.loads(key)
        S = orc.commit_padded(S0, k, v, a, b, parent, [4], np.array([path + [0] * (16 - len(path))]), [len(path)],
                              raw_gates=True)
        np.testing.assert_allclose(S[:, 0, 0, 0], want, rtol=0, atol=1e-15)


def test_padded_layout_equals_ragged_layout():
    """Two trees shared by five slots, T padded to 24: the padded front end must give exactly what the ragged calls give
    on the unpacked tensors (with the activations applied by hand through independent library routines)."""
    scipy_special = pytest.importorskip("scipy.special")
    rng = np.random.default_rng(11)
    trees = [synth.tree_geo(rng, 17), synth.tree_geo(rng, 24)]
    B, T, hk, hv, d = 5, 24, 2, 4, 8
    parent = np.full((2, T), 99, np.int32)
    for i, t in enumerate(trees):
        parent[i, : len(t)] = t
    q, k = rng.normal(size=(B, T, hk, d)), rng.normal(size=(B, T, hk, d))
    v = rng.normal(size=(B, T, hv, d))
    a, b = rng.normal(size=(B, T, hv)), rng.normal(size=(B, T, hv))
    S0 = rng.normal(size=(B, hv, d, d)) * 0.1
    n_nodes = [17, 24]
    o = orc.verify_padded(S0, q, k, v, a, b, parent, n_nodes, 0.3, raw_gates=True)
    paths = np.zeros((2, 16), np.int32)
    plen = []
    for i, t in enumerate(trees):
        p = synth.longest_path(t)
        paths[i, : len(p)] = p
        plen.append(len(p))
    S_new = orc.commit_padded(S0, k, v, a, b, parent, n_nodes, paths, plen, raw_gates=True)
    for s in range(B):
        tr = s % 2
        n = n_nodes[tr]
        g, beta = -np.logaddexp(0.0, a[s, :n]), scipy_special.expit(b[s, :n])
        offs = np.array([0, n], np.int32)
        o_ref = orc.verify(S0[s:s + 1], q[s, :n], k[s, :n], v[s, :n], g, beta, trees[tr], offs, 0.3)
        np.testing.assert_allclose(o[s, :n], o_ref, rtol=1e-13, atol=1e-14)
        assert np.all(o[s, n:] == 0.0)
        S_ref = orc.commit(S0[s:s + 1], k[s, :n], v[s, :n], g, beta, trees[tr], offs, paths[tr, : plen[tr]],
                           np.array([0, plen[tr]], np.int32))
        np.testing.assert_allclose(S_new[s], S_ref[0], rtol=1e-13, atol=1e-14)

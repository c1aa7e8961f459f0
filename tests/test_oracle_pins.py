"""Pins for the CPU oracle: each test checks an oracle function against something that is not the
oracle itself -- a closed form, an invariant, a library routine, or brute force on a tiny input."""
import itertools
import math
import os

import numpy as np
import pytest
import torch

import oracle
from helpers import check_tree_invariants

RNG = np.random.default_rng(1234)
GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _golden():
    out = {}
    for line in open(os.path.join(GOLD, "paper_constants.txt")):
        line = line.split("#")[0].strip()
        if line:
            k, v = [t.strip() for t in line.split("=")]
            out[k] = float(v)
    return out


# ------------------------------------------------------------------ O0 cached projections
def test_tables_identity_and_matmul():
    V, E = 37, 24
    emb = RNG.standard_normal((V, E)).astype(np.float32)
    eye = np.eye(E, dtype=np.float32)
    assert np.array_equal(oracle.tdes_tables(emb, eye), emb)  # g = identity reproduces e_v
    W = RNG.standard_normal((8, E)).astype(np.float32)
    b = RNG.standard_normal(8).astype(np.float32)
    want = (emb.astype(np.float64) @ W.astype(np.float64).T + b).astype(np.float32)
    got = oracle.tdes_tables(emb, W, b)
    np.testing.assert_allclose(got, want, rtol=0, atol=1e-6)
    # a transposed weight would fail this: W is [m, E]
    assert got.shape == (V, 8)


def test_tables_bf16_embedding():
    emb = torch.randn(11, 16, generator=torch.Generator().manual_seed(3)).to(torch.bfloat16)
    W = RNG.standard_normal((4, 16)).astype(np.float32)
    want = (emb.to(torch.float64).numpy() @ W.astype(np.float64).T).astype(np.float32)
    np.testing.assert_allclose(oracle.tdes_tables(emb, W), want, atol=1e-6)


# ------------------------------------------------------------------ O1 vocab pass
def test_vocab_probabilities_sum_to_one():
    z = (3.0 * RNG.standard_normal((3, 501))).astype(np.float32)
    ids, lp, lse, st = oracle.vocab_pass(z, 501)
    assert (st == 0).all()
    np.testing.assert_allclose(np.exp(lp.astype(np.float64)).sum(1), 1.0, atol=1e-5)
    # lse itself in fp64 against the direct definition
    for r in range(3):
        zz = z[r].astype(np.float64)
        assert abs(lse[r] - math.log(np.exp(zz).sum())) < 1e-12
        assert sorted(ids[r]) == list(range(501))  # a permutation of the vocabulary


def test_vocab_uniform_row_tie_break():
    V, K = 777, 9
    z = np.full((1, V), 1.25, np.float32)
    ids, lp, lse, st = oracle.vocab_pass(z, K)
    assert ids[0].tolist() == list(range(K))  # equal logits: token id ascending
    np.testing.assert_allclose(lp[0], -math.log(V), atol=1e-6)


def test_vocab_dominant_logit():
    z = np.zeros((1, 100), np.float32)
    z[0, 42] = 60.0
    ids, lp, _, _ = oracle.vocab_pass(z, 3)
    assert ids[0, 0] == 42 and abs(lp[0, 0]) < 1e-6
    assert ids[0, 1:].tolist() == [0, 1]
    np.testing.assert_allclose(lp[0, 1:], -60.0, atol=1e-5)


def test_vocab_shift_invariance():
    z = (2.0 * RNG.standard_normal((2, 300))).astype(np.float32)
    z = np.round(z * 64) / 64  # so that adding 8 is exact
    a = oracle.vocab_pass(z.astype(np.float32), 10)
    b = oracle.vocab_pass((z + 8.0).astype(np.float32), 10)
    assert np.array_equal(a[0], b[0])
    np.testing.assert_allclose(a[1], b[1], atol=2e-6)


def test_vocab_against_library_and_brute_force():
    V, K = 4000, 16
    z = (2.0 * RNG.standard_normal((4, V))).astype(np.float32)
    z = np.round(z * 8) / 8  # many exact ties
    ids, lp, lse, _ = oracle.vocab_pass(z.astype(np.float32), K)
    ref = torch.log_softmax(torch.from_numpy(z).double(), dim=1)
    vals, _ = torch.topk(ref, K, dim=1)
    np.testing.assert_allclose(lp, vals.numpy(), atol=1e-6)
    for r in range(4):
        order = sorted(range(V), key=lambda v: (-float(z[r, v]), v))[:K]
        assert ids[r].tolist() == order


def test_vocab_bf16_matches_upconverted():
    zb = (2.0 * torch.randn(3, 999, generator=torch.Generator().manual_seed(5))).to(torch.bfloat16)
    a = oracle.vocab_pass(zb, 8)
    b = oracle.vocab_pass(zb.float().numpy(), 8)
    for x, y in zip(a, b):
        assert np.array_equal(x, y)


def test_vocab_masked_and_bad_rows():
    z = RNG.standard_normal((4, 50)).astype(np.float32)
    z[0, 10:] = -np.inf  # masked tokens are allowed
    z[1, 3] = np.nan
    z[2, 7] = np.inf
    z[3, :] = -np.inf
    ids, lp, lse, st = oracle.vocab_pass(z, 12)
    assert st.tolist() == [0, 1, 1, 1]
    assert set(ids[0, :10].tolist()) == set(range(10))
    assert np.isneginf(lp[0, 10:]).all() and ids[0, 10:].tolist() == [10, 11]
    assert abs(np.exp(lp[0, :10].astype(np.float64)).sum() - 1) < 1e-5


# ------------------------------------------------------------------ O2 SABA
def _saba(lp0, hid, hist=4.0, prefix=100, grid=(32, 512, 16), **kw):
    p = oracle.SabaParams(**kw)
    return oracle.saba(lp0, hid, hist, prefix, p, *grid)


def test_saba_state_closed_forms():
    L, dh = 6, 8
    lp0 = np.log(np.array([0.5, 0.25, 0.125, 0.5, 0.25, 0.125], np.float32))
    same = np.tile(RNG.standard_normal(dh).astype(np.float32), (L, 1))
    st, B, U, s = _saba(lp0, same, phi_bias=50.0)
    assert abs(st[0] - (0.5 + 0.25 + 0.125) * 2 / 6) < 1e-7  # conf is a mean of probabilities
    assert abs(st[1] - 1.0) < 1e-12  # identical rows: every r_d = 1, trend term 0
    ortho = np.eye(L, dh, dtype=np.float32) * 3.0
    st, *_ = _saba(lp0, ortho, phi_bias=50.0)
    assert abs(st[1]) < 1e-12
    # 2-D rows at angles 0, 60, 90, 180 degrees: r = cos 60, cos 30, cos 90
    ang = np.deg2rad([0.0, 60.0, 90.0, 180.0])
    h = np.stack([2 * np.cos(ang), 2 * np.sin(ang)], 1).astype(np.float32)
    st, *_ = _saba(lp0[:4], h, phi_bias=50.0)
    r = [math.cos(math.radians(60)), math.cos(math.radians(30)), math.cos(math.radians(90))]
    assert abs(st[1] - (sum(r) / 3 + (r[2] - r[0]))) < 1e-6
    # zero-norm row: its cosines are taken as 0; single position: degen = 0
    h0 = h.copy()
    h0[1] = 0
    st, *_ = _saba(lp0[:4], h0, phi_bias=50.0)
    assert abs(st[1] - (r[2] / 3 + (r[2] - 0.0))) < 1e-6
    st, *_ = _saba(lp0[:1], h[:1], phi_bias=50.0)
    assert st[1] == 0.0


def test_saba_tau_and_clamp():
    lp0 = np.log(np.full(4, 0.5, np.float32))
    h = np.tile(np.ones(4, np.float32), (4, 1))
    st, B, U, status = _saba(lp0, h, hist=3.0, phi_conf=10.0, phi_degen=2.0, phi_hist=-1.0, phi_bias=7.0)
    assert abs(st[3] - (10 * 0.5 + 2 * 1.0 - 3.0 + 7.0)) < 1e-6 and status == 0  # lp0 is an fp32 log
    st, B, U, status = _saba(lp0, h, hist=3.0, phi_conf=-100.0, tau_min=0.5)
    assert st[3] == 0.5 and status == oracle.ST_TAU_CLAMPED


def test_saba_budget_rules():
    g = _golden()
    grid = (int(g["saba_grid_min"]), int(g["saba_grid_max"]), int(g["saba_grid_step"]))
    lp0 = np.log(np.full(4, 0.3, np.float32))
    h = RNG.standard_normal((4, 16)).astype(np.float32)
    # constant cost: utility is increasing in B -> largest budget; 31 grid points
    st, B, U, _ = _saba(lp0, h, grid=grid, phi_bias=80.0, c0=2.0)
    assert B == 512 and len(U) == int(g["saba_grid_points"]) and np.all(np.diff(U) > 0)
    # tau tiny: gain saturates at 1 -> smallest budget of minimal cost
    st, B, U, _ = _saba(lp0, h, grid=grid, phi_bias=-5.0, tau_min=1e-3, c0=1.0, c1=0.01)
    assert B == 32
    # affine cost with a prefix term, against the definition written out here
    st, B, U, _ = _saba(lp0, h, prefix=1000, grid=grid, phi_bias=90.0, c0=18.0, c1=0.01, c2=1e-5)
    tau = 90.0
    Bs = np.arange(32, 513, 16)
    want = (1 - np.exp(-Bs / tau)) / (18.0 + 0.01 * Bs + 1e-5 * Bs * 1000)
    np.testing.assert_allclose(U, want, rtol=1e-12)
    assert B == int(Bs[np.argmax(want)])
    # quasi-concave utility: the grid argmax brackets the continuous stationary point (bisection on dU/dB)
    c0, c1 = 18.0, 0.02

    def dU(Bc):
        G, dG = 1 - math.exp(-Bc / tau), math.exp(-Bc / tau) / tau
        Cc = c0 + c1 * Bc + 1e-5 * Bc * 1000
        return dG * Cc - G * (c1 + 1e-5 * 1000)

    st, B, U, _ = _saba(lp0, h, prefix=1000, grid=grid, phi_bias=90.0, c0=c0, c1=c1, c2=1e-5)
    lo, hi = 1.0, 5000.0
    for _ in range(200):
        mid = 0.5 * (lo + hi)
        lo, hi = (mid, hi) if dU(mid) > 0 else (lo, mid)
    assert abs(B - lo) <= 16


def test_saba_cost_table_interpolation():
    lp0 = np.log(np.full(4, 0.3, np.float32))
    h = RNG.standard_normal((4, 16)).astype(np.float32)
    st, B, U, _ = _saba(lp0, h, grid=(16, 256, 16), phi_bias=100.0, cost_mode=1, pts_n=[0.0, 64.0, 256.0],
                        pts_t=[18.0, 18.0, 18.0 + 0.02 * 192])
    Bs = np.arange(16, 257, 16)
    cost = 18.0 + 0.02 * np.maximum(0, Bs - 64)
    np.testing.assert_allclose(U, (1 - np.exp(-Bs / 100.0)) / cost, rtol=1e-12)
    assert B == int(Bs[np.argmax((1 - np.exp(-Bs / 100.0)) / cost)])
    # ties -> smallest budget: zero gain slope cannot happen, so force equal utilities with a huge tau_min
    st, B, U, _ = _saba(lp0, h, grid=(16, 64, 16), phi_bias=-1.0, tau_min=1e-9, c0=1.0)
    assert np.all(U == U[0]) and B == 16


# ------------------------------------------------------------------ O3 TDES edges
def _tdes_case(L=3, K=4, m=6, V=30, seed=0):
    g = np.random.default_rng(seed)
    ids = np.stack([g.choice(V, K, replace=False) for _ in range(L)]).astype(np.int32)
    lp = -np.sort(g.uniform(0.1, 5.0, (L, K)).astype(np.float32), axis=1)
    P = g.standard_normal((V, m)).astype(np.float32)
    Cc = g.standard_normal((V, m)).astype(np.float32)
    u = g.standard_normal((L, m)).astype(np.float32)
    return ids, lp, P, Cc, u


def test_tdes_centering_and_neutral_cases():
    ids, lp, P, Cc, u = _tdes_case()
    L, K = ids.shape
    beta = 0.7
    e = oracle.tdes_edges(ids, lp, 5, P, Cc, u, 1.3, beta)
    resid = (e.astype(np.float64) - lp[:, None, :]) / beta
    assert np.abs(resid[0, 0].sum()) < 1e-5 and np.abs(resid[1:].sum(-1)).max() < 1e-5  # rows of f~ sum to 0
    assert np.all(e[0, 1:] == 0)  # depth 1 has a single parent
    e0 = oracle.tdes_edges(ids, lp, 5, P, Cc, u, 1.3, 0.0)  # beta = 0: the DDTree score, exactly
    assert np.array_equal(e0[1:], np.broadcast_to(lp[1:, None, :], (L - 1, K, K)))
    assert np.array_equal(e0[0, 0], lp[0])
    ez = oracle.tdes_edges(ids, lp, 5, P, np.zeros_like(Cc), u, 1.3, beta)  # child tower constant -> f~ = 0
    np.testing.assert_allclose(ez[1:], np.broadcast_to(lp[1:, None, :], (L - 1, K, K)), atol=1e-6)
    e1 = oracle.tdes_edges(ids[:, :1], lp[:, :1], 5, P, Cc, u, 1.3, beta)  # a single child: nothing to centre
    np.testing.assert_allclose(e1[:, 0, 0], lp[:, 0], atol=1e-7)
    er = oracle.tdes_edges(ids, lp, 5, P, Cc, u, 1.3, beta, root_edge=0)
    assert np.array_equal(er[0, 0], lp[0]) and np.array_equal(er[1:], e[1:])


def test_tdes_against_centred_child_restatement():
    ids, lp, P, Cc, u = _tdes_case(L=4, K=5, m=8, V=40, seed=3)
    L, K = ids.shape
    m = P.shape[1]
    s, beta, root = 0.9, 0.2, 17
    e = oracle.tdes_edges(ids, lp, root, P, Cc, u, s, beta)
    P64, C64, u64 = P.astype(np.float64), Cc.astype(np.float64), u.astype(np.float64)
    for j in range(L):
        parents = [root] if j == 0 else ids[j - 1].tolist()
        cbar = C64[ids[j]].mean(0)
        for i, p in enumerate(parents):
            for c in range(K):
                # f~ = s/sqrt(m) (P[p] + u_d) . (C[c] - mean_c C): the u_d.(P+u) terms cancel
                ft = s / math.sqrt(m) * np.dot(P64[p] + u64[j], C64[ids[j, c]] - cbar)
                assert abs(float(e[j, i, c]) - (float(lp[j, c]) + beta * ft)) < 2e-6
    # hand example, m = 1: P = 2, C = (1, 3), u = 0.5, s = 1: f = 2.5*1.5, 2.5*3.5 -> f~ = -2.5, +2.5
    e = oracle.tdes_edges(np.array([[0, 1]], np.int32), np.array([[-1.0, -2.0]], np.float32), 2,
                          np.array([[0.0], [0.0], [2.0]], np.float32), np.array([[1.0], [3.0], [0.0]], np.float32),
                          np.array([[0.5]], np.float32), 1.0, 0.5)
    np.testing.assert_allclose(e[0, 0], [-1.0 - 1.25, -2.0 + 1.25], atol=1e-7)


def test_tdes_depth_embedding_uses_child_depth():
    # u enters through row j (the child's depth); permuting u's rows must change depth j only via row j
    ids, lp, P, Cc, u = _tdes_case(L=3, K=3, m=4, V=12, seed=9)
    e = oracle.tdes_edges(ids, lp, 1, P, Cc, u, 1.0, 1.0)
    u2 = u.copy()
    u2[2] += 1.0
    e2 = oracle.tdes_edges(ids, lp, 1, P, Cc, u2, 1.0, 1.0)
    assert np.array_equal(e[:2], e2[:2]) and not np.array_equal(e[2], e2[2])


# ------------------------------------------------------------------ O4 best-first selection
def _all_prefixes(edge):
    """Every prefix with its fp32 path score (root-to-leaf fp32 adds) and bottleneck key."""
    L, K, _ = edge.shape
    out = {}
    for ln in range(1, L + 1):
        for t in itertools.product(range(K), repeat=ln):
            S = np.float32(0.0)
            key = np.float32(np.inf)
            for d in range(ln):
                S = np.float32(S + edge[d, t[d - 1] if d else 0, t[d]])
                key = min(key, S)
            out[t] = (S, key)
    return out


def _edge_of(edge, t):
    return float(edge[len(t) - 1, t[-2] if len(t) > 1 else 0, t[-1]])


def _best_first_rescan(edge, budget):
    """Independent restatement: rebuild the frontier from the selected set at every step.  Equal scores:
    shorter prefix first, then the lexicographically smaller parent, then under one parent the larger edge
    score, then the lower candidate rank."""
    L, K, _ = edge.shape
    allp = _all_prefixes(edge)
    sel = []
    when = {(): 0}
    for step in range(budget):
        frontier = [t for t in allp if t not in when and t[:-1] in when]
        if not frontier:
            break
        best = min(frontier, key=lambda t: (-float(allp[t][0]), len(t), t[:-1], -_edge_of(edge, t), t[-1]))
        when[best] = step + 1
        sel.append(best)
    return sel


@pytest.mark.parametrize("L,K,budget,mono,seed", [
    (3, 3, 7, True, 0), (4, 3, 20, True, 1), (3, 4, 11, False, 2), (4, 4, 30, False, 3), (4, 2, 9, False, 4),
    (2, 4, 20, False, 5), (4, 3, 13, False, 6), (3, 3, 39, False, 7),
])
def test_select_against_exhaustive_enumeration(L, K, budget, mono, seed):
    g = np.random.default_rng(seed)
    edge = g.normal(-1.0, 1.0, (L, K, K)).astype(np.float32)
    if mono:
        edge = -np.abs(edge)
    edge = np.round(edge * 4) / 4 if seed % 2 else edge  # odd seeds: many exact score ties
    edge = edge.astype(np.float32)
    tup, ln, S = oracle.select(edge, budget)
    got = [tuple(int(x) for x in t[:n]) for t, n in zip(tup, ln)]
    allp = _all_prefixes(edge)
    n_all = len(allp)
    assert len(got) == min(budget, n_all) and len(set(got)) == len(got)
    for t, s in zip(got, S):
        assert allp[t][0] == s  # fp32 path score, accumulated root to leaf
        assert t[:-1] == () or t[:-1] in got[: got.index(t)]  # prefix-closed, parents first
    assert got == _best_first_rescan(edge, budget)  # same sequence as the from-scratch restatement
    # bottleneck-key theorem: every selected key >= every unselected key
    ksel = min(float(allp[t][1]) for t in got)
    krest = max([float(v[1]) for t, v in allp.items() if t not in got], default=-np.inf)
    assert ksel >= krest
    if mono:
        # all edges <= 0: the selection is the global top-B by path score (DDTree's rule),
        # and exp(S) is the product of the edge probabilities
        smin = min(float(allp[t][0]) for t in got)
        smax_rest = max([float(v[0]) for t, v in allp.items() if t not in got], default=-np.inf)
        assert smin >= smax_rest
        assert sorted(float(allp[t][0]) for t in got) == sorted((float(v[0]) for v in allp.values()), reverse=True)[
            : len(got)][::-1]
        for t in got[:5]:
            prod = math.prod(math.exp(float(edge[d, t[d - 1] if d else 0, t[d]])) for d in range(len(t)))
            assert abs(math.exp(float(allp[t][0])) - prod) < 1e-5


def test_select_special_cases():
    L, K = 5, 3
    # sharply peaked rows: a budget of L gives the chain of top-1 tokens (the DFlash draft, Eq. 2)
    edge = np.full((L, K, K), -20.0, np.float32)
    edge[:, :, 0] = -0.01
    tup, ln, S = oracle.select(edge, L)
    assert [tuple(t[:n]) for t, n in zip(tup, ln)] == [(0,) * d for d in range(1, L + 1)]
    # budget beyond the number of prefixes: complete tree (K=2, L=3 -> 2 + 4 + 8 = 14)
    e2 = RNG.normal(size=(3, 2, 2)).astype(np.float32)
    tup, ln, S = oracle.select(e2, 50)
    assert len(ln) == 14
    # budget 1: the best depth-1 node; budget 0: nothing
    tup, ln, S = oracle.select(e2, 1)
    assert ln.tolist() == [1] and tup[0, 0] == int(np.argmax(e2[0, 0])) and S[0] == e2[0, 0].max()
    assert len(oracle.select(e2, 0)[1]) == 0
    # all scores equal: shorter first, then the parent's ranks lexicographically, then candidate rank
    e3 = np.zeros((3, 2, 2), np.float32)
    tup, ln, S = oracle.select(e3, 6)
    assert [tuple(t[:n]) for t, n in zip(tup, ln)] == [(0,), (1,), (0, 0), (0, 1), (1, 0), (1, 1)]
    # equal path scores, different parents: the lexicographically smaller parent goes first, even when it was
    # selected later
    e5 = np.full((2, 2, 2), -9.0, np.float32)
    e5[0, 0] = [-1.0, 0.0]          # (1,) is selected first, then (0,)
    e5[1, 1, 0] = -5.0              # (1,0): 0 - 5
    e5[1, 0, 0] = -4.0              # (0,0): -1 - 4
    tup, ln, S = oracle.select(e5, 3)
    assert [tuple(t[:n]) for t, n in zip(tup, ln)] == [(1,), (0,), (0, 0)] and S[2] == -5.0
    # equal path scores under one parent although the edges differ (4e7 + 1 and 4e7 + 2 both round to 4e7):
    # the larger edge first, here the higher rank
    e6 = np.full((2, 2, 2), -9.0, np.float32)
    e6[0, 0] = [4.0e7, -1.0]
    e6[1, 0] = [1.0, 2.0]
    tup, ln, S = oracle.select(e6, 2)
    assert [tuple(t[:n]) for t, n in zip(tup, ln)] == [(0,), (0, 1)] and S[1] == np.float32(4.0e7)
    # the parent row is the PARENT's candidate index: make child 1 great only under parent 1
    e4 = np.full((2, 2, 2), -5.0, np.float32)
    e4[0, 0] = [-1.0, -2.0]
    e4[1, 1, 1] = 3.0
    tup, ln, S = oracle.select(e4, 3)
    assert [tuple(t[:n]) for t, n in zip(tup, ln)] == [(0,), (1,), (1, 1)] and S[2] == 1.0


# ------------------------------------------------------------------ O5 emission
def test_emit_invariants_and_order():
    L, K, V = 4, 3, 50
    g = np.random.default_rng(11)
    ids = np.stack([g.choice(V, K, replace=False) for _ in range(L)]).astype(np.int32)
    edge = g.normal(-1, 1, (L, K, K)).astype(np.float32)
    for budget in (1, 5, 17, 40):
        tup, ln, S = oracle.select(edge, budget)
        o = oracle.emit(tup, ln, S, ids, 9, 100, 41)
        check_tree_invariants(o, budget, L, ids, 9, 100)
        n = o["n_nodes"]
        assert n == len(ln) + 1
        # rebuild each node's tuple from parent links and check canonical (length, tuple) order + tokens
        tuples = [()]
        for i in range(1, n):
            tuples.append(tuples[o["parent"][i]] + (int(o["cand"][i]),))
            assert o["token"][i] == ids[o["depth"][i] - 1, o["cand"][i]]
        assert tuples == sorted(tuples, key=lambda t: (len(t), t))
        want = {tuple(int(x) for x in t[:k]): s for t, k, s in zip(tup, ln, S)}
        for i in range(1, n):
            assert o["path_score"][i] == want[tuples[i]]
    o = oracle.emit(np.zeros((0, L), np.int32), np.zeros(0, np.int32), np.zeros(0, np.float32), ids, 9, 100, 41)
    assert o["n_nodes"] == 1 and o["token"][0] == 9 and o["position"][0] == 99


def test_emit_mask_spans_words():
    L, K = 6, 8
    g = np.random.default_rng(2)
    ids = np.stack([g.choice(500, K, replace=False) for _ in range(L)]).astype(np.int32)
    edge = g.normal(-1, 0.5, (L, K, K)).astype(np.float32)
    tup, ln, S = oracle.select(edge, 100)
    o = oracle.emit(tup, ln, S, ids, 1, 10, 101)
    assert o["mask"].shape == (101, 4) and o["mask"][:, 1:].any()
    check_tree_invariants(o, 100, L)


# ------------------------------------------------------------------ O6 acceptance walk
def test_accept_hand_built_tree():
    #        0(root, tok 100)
    #      /        \
    #   1(tok 5)    2(tok 6)
    #   /    \         \
    # 3(7)   4(8)      5(7)
    #          \
    #          6(9)
    token = np.array([100, 5, 6, 7, 8, 7, 9, -1], np.int32)
    parent = np.array([-1, 0, 0, 1, 1, 2, 4, -1], np.int32)
    L = 4
    tn = np.array([42, 0, 0, 0, 0, 0, 0, -1], np.int32)  # root wants 42: no child carries it
    assert oracle.accept(7, token, parent, tn, L)[0::2] == (0, 42)
    tn = np.array([6, 0, 7, 0, 0, 11, 0, -1], np.int32)  # 0 -> 2 -> 5, then 11 unmatched
    a, path, bonus = oracle.accept(7, token, parent, tn, L)
    assert (a, path.tolist(), bonus) == (2, [2, 5, -1, -1], 11)
    tn = np.array([5, 8, 0, 0, 9, 0, 77, -1], np.int32)  # 0 -> 1 -> 4 -> 6 (full depth of this branch)
    a, path, bonus = oracle.accept(7, token, parent, tn, L)
    assert (a, path.tolist(), bonus) == (3, [1, 4, 6, -1], 77)
    # token 7 exists under node 2 but not as a child of root->1->... after 8: the walk must respect parents
    tn = np.array([5, 7, 0, 6, 0, 0, 0, -1], np.int32)
    a, path, bonus = oracle.accept(7, token, parent, tn, L)
    assert (a, path.tolist(), bonus) == (2, [1, 3, -1, -1], 6)


def test_accept_chain_reaches_full_depth():
    L = 5
    token = np.array([1, 10, 11, 12, 13, 14], np.int32)
    parent = np.array([-1, 0, 1, 2, 3, 4], np.int32)
    tn = np.array([10, 11, 12, 13, 14, 99], np.int32)
    a, path, bonus = oracle.accept(6, token, parent, tn, L)
    assert (a, path.tolist(), bonus) == (L, [1, 2, 3, 4, 5], 99)


# ------------------------------------------------------------------ replay check (comparison rule)
def test_replay_check_accepts_own_tree_and_rejects_a_worse_one():
    L, K = 4, 4
    g = np.random.default_rng(21)
    ids = np.stack([g.choice(99, K, replace=False) for _ in range(L)]).astype(np.int32)
    edge = g.normal(-1, 1, (L, K, K)).astype(np.float32)
    tup, ln, S = oracle.select(edge, 12)
    o = oracle.emit(tup, ln, S, ids, 0, 10, 13)
    ok, worst = oracle.replay_check(edge, o["n_nodes"], o["parent"], o["cand"], o["depth"], 1e-5)
    assert ok and worst == 0.0
    # replace the last-popped node by the worst depth-1 candidate not in the tree (if any) -> invalid
    tup2, ln2, S2 = tup.copy(), ln.copy(), S.copy()
    have = {tuple(t[:n]) for t, n in zip(tup, ln)}
    # find a leaf to drop and a clearly worse frontier node to add
    allp = _all_prefixes(edge)
    frontier = [t for t in allp if t not in have and (t[:-1] == () or t[:-1] in have)]
    worst_t = min(frontier, key=lambda t: float(allp[t][0]))
    last = tuple(int(x) for x in tup[-1][: ln[-1]])
    if worst_t[:-1] != last and allp[worst_t][0] < S[-1] - 1e-3:
        tup2[-1] = -1
        tup2[-1, : len(worst_t)] = worst_t
        ln2[-1] = len(worst_t)
        S2[-1] = allp[worst_t][0]
        o2 = oracle.emit(tup2, ln2, S2, ids, 0, 10, 13)
        ok, worst = oracle.replay_check(edge, o2["n_nodes"], o2["parent"], o2["cand"], o2["depth"], 1e-5)
        assert not ok


# ------------------------------------------------------------------ whole round
def test_build_trees_round_is_the_steps_in_order():
    import graft_inputs as gi
    w = gi.small(batch=3, L=4, V=400, K=4, budget_min=8, budget_max=24, budget_step=8)
    x = gi.batch_inputs(w)
    tb = gi.tdes_tables(w)
    sp = oracle.SabaParams(**gi.saba_defaults(w))
    o = oracle.build_trees(x["logits"], x["hidden"], x["root_token"], x["hist"], x["prefix_len"], None, sp,
                           (w.budget_min, w.budget_max, w.budget_step), tb["P"], tb["C"], tb["u"], tb["s"], w.beta, w.K)
    for b in range(w.batch):
        ids, lp, lse, st = oracle.vocab_pass(x["logits"][b], w.K)
        assert np.array_equal(ids, o["topk_id"][b]) and np.array_equal(lp, o["topk_lp"][b])
        state, B, U, _ = oracle.saba(lp[:, 0], x["hidden"][b], float(x["hist"][b]), int(x["prefix_len"][b]), sp,
                                     w.budget_min, w.budget_max, w.budget_step)
        assert B == o["budget"][b] and np.array_equal(state, o["state"][b])
        e = oracle.tdes_edges(ids, lp, int(x["root_token"][b]), tb["P"], tb["C"], tb["u"], 1.0, w.beta)
        assert np.array_equal(e, o["edge"][b])
        tup, ln, S = oracle.select(e, B)
        em = oracle.emit(tup, ln, S, ids, int(x["root_token"][b]), int(x["prefix_len"][b]), w.nmax)
        for k in ("token", "parent", "depth", "position", "path_score", "mask"):
            assert np.array_equal(em[k], o[k][b]), k
        check_tree_invariants({k: o[k][b] for k in o}, B, w.L, ids, int(x["root_token"][b]), int(x["prefix_len"][b]))
    # threads > 1 gives the same bytes
    o2 = oracle.build_trees(x["logits"], x["hidden"], x["root_token"], x["hist"], x["prefix_len"], None, sp,
                            (w.budget_min, w.budget_max, w.budget_step), tb["P"], tb["C"], tb["u"], tb["s"], w.beta,
                            w.K, threads=2)
    for k in o:
        assert np.array_equal(o[k], o2[k], equal_nan=True), k


def test_build_trees_bad_row_gives_root_only_tree():
    import graft_inputs as gi
    w = gi.small(batch=2, L=3, V=100, K=4, fixed_budget=8, budget_min=8, budget_max=8)
    x = gi.batch_inputs(w)
    x["logits"][1, 2, 5] = float("nan")
    tb = gi.tdes_tables(w)
    o = oracle.build_trees(x["logits"], None, x["root_token"], None, x["prefix_len"], x["fixed_budget"].numpy(),
                           oracle.SabaParams(), (8, 8, 8), tb["P"], tb["C"], tb["u"], 1.0, 0.2, w.K)
    assert o["status"].tolist() == [0, 1] and o["n_nodes"].tolist() == [9, 1]


# --------------------------------------------------------------------------- O7 acceptance history (Eq. 15)
def test_hist_constant_history_and_empty_history():
    assert oracle.hist_update([], 4) == 0.0
    for w in (1, 3, 8):
        for n in (1, 2, 8, 20):
            assert oracle.hist_update([5] * n, w) == 5.0


def test_hist_step_change_crosses_over_in_w_rounds():
    w = 4
    a = [2] * 10
    vals = []
    for t in range(1, 7):
        a.append(6)
        vals.append(oracle.hist_update(a, w))
    assert vals == [3.0, 4.0, 5.0, 6.0, 6.0, 6.0]  # one more new entry in the window each round, then saturated


def test_hist_is_the_mean_of_the_last_w_entries():
    rng = np.random.default_rng(15)
    a = rng.integers(0, 17, size=40).astype(np.int32)
    for w in (1, 5, 8, 64):
        for n in (1, 3, 8, 40):
            want = float(np.mean(a[:n][-w:].astype(np.float64)))
            assert abs(oracle.hist_update(a[:n], w) - want) < 1e-12

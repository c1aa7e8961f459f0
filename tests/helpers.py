"""Shared test helpers: tree invariants, and the GPU-vs-oracle comparison rule.

Comparison rule: token ids, parents, depths, positions, masks, node counts, budgets, status bits and the
acceptance outputs must match bit for bit, padding included; log-probs, log-sum-exp, edge scores, path
scores and the SABA state must agree within EPS = 1e-5 absolute.  The results are fp32 numbers, so where a
value is so large that a few fp32 spacings exceed EPS (one spacing does beyond |x| = 128) the bound is that many
spacings instead: max(EPS, k ulp), k = 1 for log-probs and log-sum-exp, 2 for path scores, 3 for edge scores.  At
the magnitudes of the configured workloads (|x| < 64) this is plain 1e-5.  tau = phi . s + bias carries the
state's error times phi: it is held to EPS * sum_i |phi_i| |s_i| (or one fp32 spacing of tau if larger).
Infinities must be the same infinity.  A sequence whose tree differs is excused only if
  * its budget is the oracle's runner-up with a relative utility gap below 1e-6 (the oracle's tree is then
    rebuilt at that budget), or
  * its node set is a valid best-first outcome on the ORACLE's scores when every comparison may be off by
    EPS (oracle.replay_check), has the oracle's node count and satisfies every tree invariant.
Top-K membership and order are never excused.
"""
import numpy as np

EPS = 1e-5

def check_tree_invariants(o, budget, L, ids=None, root_token=None, prefix_len=None):
    n = int(o["n_nodes"])
    tok, par, dep, pos, msk = o["token"], o["parent"], o["depth"], o["position"], o["mask"]
    Nmax, W = msk.shape
    assert 1 <= n <= budget + 1 <= Nmax
    assert par[0] == -1 and dep[0] == 0
    kids = {}
    for i in range(1, n):
        p = int(par[i])
        assert 0 <= p < i and dep[i] == dep[p] + 1 and 1 <= dep[i] <= L  # prefix-closed, level order
        kids.setdefault(p, []).append(int(tok[i]))
        row = 0
        for w in range(W):
            row |= int(msk[i, w]) << (32 * w)
        prow = 0
        for w in range(W):
            prow |= int(msk[p, w]) << (32 * w)
        assert row == prow | (1 << i) and bin(row).count("1") == dep[i] + 1 and row & 1
    assert int(msk[0, 0]) == 1 and not msk[0, 1:].any()
    for p, ts in kids.items():
        assert len(set(ts)) == len(ts)  # sibling tokens distinct
    assert list(dep[:n]) == sorted(dep[:n])
    if prefix_len is not None:
        assert np.array_equal(pos[:n], prefix_len - 1 + dep[:n])
    if root_token is not None:
        assert tok[0] == root_token
    assert (tok[n:] == -1).all() and (par[n:] == -1).all() and (dep[n:] == -1).all() and (pos[n:] == -1).all()
    assert (o["path_score"][n:] == 0).all() and not msk[n:].any()




def gpu_round(g, w, x, dev="cuda", debug=True):
    """Run the library on inputs x (CPU tensors) and return numpy outputs."""
    import torch
    cu = lambda t: None if t is None else t.to(dev)  # noqa: E731
    out = g.alloc_out(x["logits"].shape[0], debug=debug)
    g.build_trees(cu(x["logits"]), cu(x["hidden"]), cu(x["root_token"]), cu(x["hist"]), cu(x["prefix_len"]),
                  cu(x["fixed_budget"]), out)
    torch.cuda.synchronize()
    return out, out.cpu()


def oracle_round(oracle, w, x, tb, saba_kw, threads=8):
    sp = oracle.SabaParams(**saba_kw)
    fb = None if x["fixed_budget"] is None else x["fixed_budget"].numpy()
    return oracle.build_trees(x["logits"], x["hidden"], x["root_token"].numpy(), x["hist"].numpy(),
                              x["prefix_len"].numpy(), fb, sp, (w.budget_min, w.budget_max, w.budget_step),
                              tb["P"].numpy(), tb["C"].numpy(), tb["u"].numpy(), tb["s"], w.beta, w.K,
                              threads=threads)


def tolerance(b, tol=EPS, ulps=1):
    """max(tol, ulps * fp32 spacing at |b|) per element (b: the oracle's values)."""
    b = np.asarray(b, np.float64)
    with np.errstate(invalid="ignore", over="ignore"):
        bf = np.where(np.isfinite(b), np.abs(b), 0.0).astype(np.float32)
        return np.maximum(tol, ulps * np.spacing(bf).astype(np.float64))


def max_delta(a, b):
    """Largest |a - b| over the finite entries of b (0 if there are none)."""
    a = np.asarray(a, np.float64)
    b = np.asarray(b, np.float64)
    fin = np.isfinite(b) & np.isfinite(a)
    return float(np.abs(a[fin] - b[fin]).max(initial=0.0))


def _close(a, b, tol, ulps=1):
    """|a - b| <= max(tol, ulps * (fp32 spacing at |b|)), or both the same infinity."""
    a = np.asarray(a, np.float64)
    b = np.asarray(b, np.float64)
    same_inf = np.isinf(a) & np.isinf(b) & (np.sign(a) == np.sign(b))
    with np.errstate(invalid="ignore", over="ignore"):  # inf - inf where both sides are the same infinity
        return bool(np.all(same_inf | (np.abs(a - b) <= tolerance(b, tol, ulps))))


def compare_round(oracle, w, x, tb, saba_kw, gpu, orc):
    """Apply the comparison rule to every sequence.  Returns counts of excused sequences."""
    Bt = gpu["n_nodes"].shape[0]
    L, K = w.L, w.K
    excused_budget = excused_tree = 0
    deltas = dict(topk_lp=0.0, lse=0.0, edge=0.0, path_score=0.0, state=0.0, tau=0.0)  # observed max |delta|

    def seen(key, a, b_):
        deltas[key] = max(deltas[key], max_delta(a, b_))
    for b in range(Bt):
        assert gpu["status"][b] == orc["status"][b], (b, gpu["status"][b], orc["status"][b])
        if orc["status"][b] & 1:
            assert gpu["n_nodes"][b] == 1 and gpu["token"][b, 0] == x["root_token"][b]
            assert (gpu["token"][b, 1:] == -1).all() and not gpu["mask"][b, 1:].any()
            continue
        # candidates: exact ids, log-probs within EPS
        assert np.array_equal(gpu["topk_id"][b], orc["topk_id"][b]), f"seq {b}: top-K ids differ"
        seen("topk_lp", gpu["topk_lp"][b], orc["topk_lp"][b])
        seen("lse", gpu["lse"][b], orc["lse"][b])
        assert _close(gpu["topk_lp"][b], orc["topk_lp"][b], EPS), f"seq {b}: log-probs"
        assert _close(gpu["lse"][b], orc["lse"][b], EPS), f"seq {b}: lse"
        # edges
        # (three spacings where those exceed EPS: an edge score is the rounded sum of a log-probability that may
        # itself be one off, both sides round the sum once, and the fp32 dot product behind beta f has its own error)
        seen("edge", gpu["edge"][b, 0, 0], orc["edge"][b, 0, 0])
        seen("edge", gpu["edge"][b, 1:], orc["edge"][b, 1:])
        assert _close(gpu["edge"][b, 0, 0], orc["edge"][b, 0, 0], EPS, ulps=3), f"seq {b}: depth-1 edges"
        assert _close(gpu["edge"][b, 1:], orc["edge"][b, 1:], EPS, ulps=3), f"seq {b}: edges"
        # SABA
        o_budget = int(orc["budget"][b])
        ref = {k: orc[k][b] for k in ("n_nodes", "token", "parent", "depth", "position", "path_score", "mask")}
        if x["fixed_budget"] is None:
            st_g, st_o = gpu["state"][b].astype(np.float64), orc["state"][b]
            seen("state", st_g[:3], st_o[:3])
            seen("tau", st_g[3], st_o[3])
            assert np.all(np.abs(st_g[:3] - st_o[:3]) <= EPS), (b, st_g, st_o)
            phi = np.abs([saba_kw.get("phi_conf", 0.0), saba_kw.get("phi_degen", 0.0), saba_kw.get("phi_hist", 0.0)])
            tau_tol = max(EPS * float(phi @ np.abs(st_o[:3])), float(np.spacing(np.float32(abs(st_o[3])))))
            assert abs(st_g[3] - st_o[3]) <= tau_tol, (b, st_g, st_o, tau_tol)
        if int(gpu["budget"][b]) != o_budget:
            U = orc["Ugrid"][b]
            order = np.argsort(-U, kind="stable")
            grid = np.arange(w.budget_min, w.budget_max + 1, w.budget_step)
            gap = (U[order[0]] - U[order[1]]) / U[order[0]]
            assert int(gpu["budget"][b]) == int(grid[order[1]]) and gap < 1e-6, \
                f"seq {b}: budget {gpu['budget'][b]} vs {o_budget}, gap {gap}"
            excused_budget += 1
            o_budget = int(gpu["budget"][b])
            tup, ln, S = oracle.select(orc["edge"][b], o_budget)
            ref = oracle.emit(tup, ln, S, orc["topk_id"][b], int(x["root_token"][b]), int(x["prefix_len"][b]), w.nmax)
        tree_g = {k: gpu[k][b] for k in ("n_nodes", "token", "parent", "depth", "position", "path_score", "mask")}
        check_tree_invariants(tree_g, o_budget, L, None, int(x["root_token"][b]), int(x["prefix_len"][b]))
        same = all(np.array_equal(tree_g[k], ref[k]) for k in ("token", "parent", "depth", "position", "mask")) \
            and int(tree_g["n_nodes"]) == int(ref["n_nodes"])
        n = int(tree_g["n_nodes"])
        if same:
            seen("path_score", tree_g["path_score"][:n], ref["path_score"][:n])
            assert _close(tree_g["path_score"][:n], ref["path_score"][:n], EPS, ulps=2), f"seq {b}: path scores"
        else:
            assert n == int(ref["n_nodes"]), f"seq {b}: node count {n} vs {ref['n_nodes']}"
            cand = np.full(n, -1, np.int32)
            for i in range(1, n):
                hit = np.nonzero(orc["topk_id"][b][tree_g["depth"][i] - 1] == tree_g["token"][i])[0]
                assert len(hit) == 1, f"seq {b}: node {i} token is not a candidate of its depth"
                cand[i] = hit[0]
            ok, worst = oracle.replay_check(orc["edge"][b], n, tree_g["parent"][:n], cand, tree_g["depth"][:n], EPS)
            assert ok, f"seq {b}: tree differs and is not a valid best-first outcome (shortfall {worst})"
            # path scores of the library's nodes against the oracle's edges, summed root to leaf in fp32
            S = np.zeros(n, np.float32)
            for i in range(1, n):
                pa = tree_g["parent"][i]
                row = 0 if pa == 0 else cand[pa]
                S[i] = np.float32(S[pa] + orc["edge"][b][tree_g["depth"][i] - 1, row, cand[i]])
            seen("path_score", tree_g["path_score"][:n], S)
            assert _close(tree_g["path_score"][:n], S, EPS, ulps=2), f"seq {b}: path scores"
            excused_tree += 1
    return dict(excused_budget=excused_budget, excused_tree=excused_tree, sequences=Bt, max_delta=deltas)


def compare_accept(oracle, gi, g, w, out, gpu, dev="cuda"):
    """Acceptance walk: library vs oracle on the LIBRARY's trees, exact."""
    import torch
    Bt = gpu["n_nodes"].shape[0]
    tn = np.stack([gi.target_next_from_depth(gi.target_tokens(w, b), gpu["depth"][b]) for b in range(Bt)])
    tn_d = torch.from_numpy(tn).to(dev)
    a_len = torch.empty(Bt, dtype=torch.int32, device=dev)
    a_path = torch.empty((Bt, w.L), dtype=torch.int32, device=dev)
    bonus = torch.empty(Bt, dtype=torch.int32, device=dev)
    g.accept(out, tn_d, a_len, a_path, bonus)
    torch.cuda.synchronize()
    a_len, a_path, bonus = a_len.cpu().numpy(), a_path.cpu().numpy(), bonus.cpu().numpy()
    for b in range(Bt):
        a, path, bo = oracle.accept(int(gpu["n_nodes"][b]), gpu["token"][b], gpu["parent"][b], tn[b], w.L)
        assert a == a_len[b] and np.array_equal(path, a_path[b]) and bo == bonus[b], (b, a, a_len[b])
    return a_len

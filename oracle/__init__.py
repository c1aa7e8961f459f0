"""CPU oracle for the GRAFT draft-tree round -- TEST INFRASTRUCTURE, not product code.

Thin ctypes marshalling around ``graft_oracle.c`` and ``tdes_train_oracle.c`` (plain C, fp64; each C function cites the
passage of the paper it restates).  Only the tests, the smoke check and the benchmark's
CPU-baseline leg may import this package; the CUDA library never does, and this package never
imports the CUDA package.  ``build()`` compiles the C file with gcc next to itself.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from dataclasses import dataclass, field

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "graft_oracle.c")
_SRCS = [_SRC, os.path.join(_HERE, "tdes_train_oracle.c")]
_LIB = os.path.join(_HERE, "libgraft_oracle.so")
_lib = None

F32, BF16 = 0, 1
ST_BAD_LOGITS, ST_TAU_CLAMPED, ST_FRONTIER_EMPTY = 1, 2, 4


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (no fast-math: fp64 semantics must be the plain ones)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < max(os.path.getmtime(f) for f in _SRCS):
        subprocess.check_call(
            ["gcc", "-O2", "-std=c99", "-fPIC", "-shared", "-ffp-contract=off", "-o", _LIB, *_SRCS, "-lm"]
        )
    return _LIB


def lib():
    global _lib
    if _lib is None:
        build()
        _lib = C.CDLL(_LIB)
    return _lib


class _SabaParams(C.Structure):
    _fields_ = [
        ("phi_conf", C.c_double), ("phi_degen", C.c_double), ("phi_hist", C.c_double), ("phi_bias", C.c_double),
        ("tau_min", C.c_double), ("cost_mode", C.c_int32), ("c0", C.c_double), ("c1", C.c_double),
        ("c2", C.c_double), ("n_pts", C.c_int32), ("pts_n", C.POINTER(C.c_double)),
        ("pts_t", C.POINTER(C.c_double)),
    ]


@dataclass
class SabaParams:
    """phi, tau_min and the cost model C_t(B) (affine Eq. 17, or a piecewise-linear table)."""
    phi_conf: float = 0.0
    phi_degen: float = 0.0
    phi_hist: float = 0.0
    phi_bias: float = 0.0
    tau_min: float = 1e-3
    cost_mode: int = 0
    c0: float = 1.0
    c1: float = 0.0
    c2: float = 0.0
    pts_n: list = field(default_factory=list)
    pts_t: list = field(default_factory=list)

    def _c(self):
        n = np.ascontiguousarray(self.pts_n, dtype=np.float64)
        t = np.ascontiguousarray(self.pts_t, dtype=np.float64)
        s = _SabaParams(self.phi_conf, self.phi_degen, self.phi_hist, self.phi_bias, self.tau_min, self.cost_mode,
                        self.c0, self.c1, self.c2, len(n), n.ctypes.data_as(C.POINTER(C.c_double)),
                        t.ctypes.data_as(C.POINTER(C.c_double)))
        s._keep = (n, t)
        return s


def _p(a):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


def _as_bits(x):
    """Accept fp32 ndarray, or bf16 given as uint16 bit patterns (ndarray) / torch.bfloat16 tensor."""
    if hasattr(x, "detach"):  # torch tensor
        import torch
        x = x.detach().cpu().contiguous()
        if x.dtype == torch.bfloat16:
            return x.view(torch.int16).numpy().view(np.uint16), BF16
        return x.to(torch.float32).numpy(), F32
    x = np.ascontiguousarray(x)
    if x.dtype == np.uint16:
        return x, BF16
    if x.dtype == np.float32:
        return x, F32
    raise TypeError(f"unsupported dtype {x.dtype}")


def tdes_tables(emb, W, bias=None):
    emb, dt = _as_bits(emb)
    V, E = emb.shape
    W = np.ascontiguousarray(W, dtype=np.float32)
    m = W.shape[0]
    b = None if bias is None else np.ascontiguousarray(bias, dtype=np.float32)
    out = np.empty((V, m), dtype=np.float32)
    rc = lib().oracle_tdes_tables(_p(emb), dt, V, E, m, _p(W), _p(b), _p(out))
    assert rc == 0
    return out


def vocab_pass(logits, K):
    """logits [rows, V] -> (topk_id [rows,K] int32, topk_lp [rows,K] f32, lse [rows] f64, status [rows])."""
    z, dt = _as_bits(logits)
    rows, V = z.shape
    ids = np.empty((rows, K), dtype=np.int32)
    lp = np.empty((rows, K), dtype=np.float32)
    lse = np.empty(rows, dtype=np.float64)
    st = np.empty(rows, dtype=np.int32)
    rc = lib().oracle_vocab_pass(_p(z), dt, C.c_int64(rows), V, K, _p(ids), _p(lp), _p(lse), _p(st))
    assert rc == 0
    return ids, lp, lse, st


def saba(lp0, hidden, hist, prefix_len, params: SabaParams, bmin, bmax, bstep):
    """One sequence. Returns (state[4] f64 = conf, degen, hist, tau; budget; U over the grid; status)."""
    lp0 = np.ascontiguousarray(lp0, dtype=np.float32)
    h, dt = _as_bits(hidden)
    L, dh = h.shape
    grid = (bmax - bmin) // bstep + 1
    state = np.zeros(4, dtype=np.float64)
    U = np.zeros(grid, dtype=np.float64)
    budget = C.c_int32(0)
    status = C.c_int32(0)
    sp = params._c()
    rc = lib().oracle_saba(_p(lp0), _p(h), dt, L, dh, C.c_double(hist), C.c_int32(prefix_len), C.byref(sp),
                           bmin, bmax, bstep, _p(state), C.byref(budget), _p(U), C.byref(status))
    assert rc == 0
    return state, budget.value, U, status.value


def tdes_edges(topk_id, topk_lp, root_token, P, Ctab, u, s, beta, root_edge=1):
    """One sequence. topk_id/lp [L,K]; returns edge [L,K,K] f32."""
    ids = np.ascontiguousarray(topk_id, dtype=np.int32)
    lp = np.ascontiguousarray(topk_lp, dtype=np.float32)
    L, K = ids.shape
    P = np.ascontiguousarray(P, dtype=np.float32)
    Ctab = np.ascontiguousarray(Ctab, dtype=np.float32)
    u = np.ascontiguousarray(u, dtype=np.float32)
    m = P.shape[1]
    edge = np.empty((L, K, K), dtype=np.float32)
    rc = lib().oracle_tdes_edges(_p(ids), _p(lp), C.c_int32(root_token), _p(P), _p(Ctab), _p(u), C.c_double(s),
                                 C.c_double(beta), int(root_edge), L, K, m, _p(edge))
    assert rc == 0
    return edge


def select(edge, budget):
    """edge [L,K,K] -> (tuples [n,L] int32 (-1 padded), lengths [n], S [n]) in pop order."""
    edge = np.ascontiguousarray(edge, dtype=np.float32)
    L, K, _ = edge.shape
    tup = np.full((max(budget, 1), L), -1, dtype=np.int32)
    ln = np.zeros(max(budget, 1), dtype=np.int32)
    S = np.zeros(max(budget, 1), dtype=np.float32)
    n = C.c_int32(0)
    rc = lib().oracle_select(_p(edge), L, K, int(budget), _p(tup), _p(ln), _p(S), C.byref(n))
    assert rc == 0, rc
    return tup[: n.value], ln[: n.value], S[: n.value]


def emit(tuples, lengths, S, topk_id, root_token, prefix_len, Nmax):
    ids = np.ascontiguousarray(topk_id, dtype=np.int32)
    L, K = ids.shape
    W = (Nmax + 31) // 32
    n_sel = len(lengths)
    tup = np.ascontiguousarray(tuples, dtype=np.int32).reshape(max(n_sel, 0), L) if n_sel else np.zeros((1, L), np.int32)
    ln = np.ascontiguousarray(lengths, dtype=np.int32) if n_sel else np.zeros(1, np.int32)
    Sv = np.ascontiguousarray(S, dtype=np.float32) if n_sel else np.zeros(1, np.float32)
    out = dict(
        token=np.empty(Nmax, np.int32), parent=np.empty(Nmax, np.int32), depth=np.empty(Nmax, np.int32),
        position=np.empty(Nmax, np.int32), path_score=np.empty(Nmax, np.float32),
        mask=np.empty((Nmax, W), np.uint32), cand=np.empty(Nmax, np.int32),
    )
    n_nodes = C.c_int32(0)
    rc = lib().oracle_emit(_p(tup), _p(ln), _p(Sv), n_sel, L, K, _p(ids), C.c_int32(root_token),
                           C.c_int32(prefix_len), Nmax, W, C.byref(n_nodes), _p(out["token"]), _p(out["parent"]),
                           _p(out["depth"]), _p(out["position"]), _p(out["path_score"]), _p(out["mask"]),
                           _p(out["cand"]))
    assert rc == 0
    out["n_nodes"] = n_nodes.value
    return out


def accept(n_nodes, token, parent, target_next, L):
    token = np.ascontiguousarray(token, dtype=np.int32)
    parent = np.ascontiguousarray(parent, dtype=np.int32)
    tn = np.ascontiguousarray(target_next, dtype=np.int32)
    path = np.empty(L, np.int32)
    a = C.c_int32(0)
    bonus = C.c_int32(0)
    rc = lib().oracle_accept(int(n_nodes), _p(token), _p(parent), _p(tn), L, C.byref(a), _p(path), C.byref(bonus))
    assert rc == 0
    return a.value, path, bonus.value


def hist_update(a_hist, w):
    """hist for the next round from all accepted lengths so far, oldest first (Eq. 15)."""
    a = np.ascontiguousarray(a_hist, dtype=np.int32)
    f = lib().oracle_hist_update
    f.restype = C.c_double
    return float(f(_p(a), int(a.size), int(w)))


class _TdesLossCfg(C.Structure):
    _fields_ = [("gamma", C.c_double), ("w1", C.c_double), ("lambda_kl", C.c_double), ("lambda_pair", C.c_double),
                ("lambda_bce", C.c_double)]


def tdes_loss(P, Ctab, u, s, groups, pairs, edges, gamma, w1, lambda_kl, lambda_pair, lambda_bce, grad=True):
    """TDES training objective and its gradients (Eq. 7-12).

    groups: dict(parent [G], depth [G], child [G,K], logq [G,K], ztgt [G,K]); pairs [N,6] = (p+, c+, d+, p-, c-, d-);
    edges [N,4] = (p, c, d, y).  Returns dict(loss [4] = KL, pair, BCE, total; gP, gC, gu, gs in fp64)."""
    P = np.ascontiguousarray(P, dtype=np.float32)
    Ctab = np.ascontiguousarray(Ctab, dtype=np.float32)
    u = np.ascontiguousarray(u, dtype=np.float32)
    V, m = P.shape
    L = u.shape[0]
    gp = np.ascontiguousarray(groups["parent"], dtype=np.int32)
    gd = np.ascontiguousarray(groups["depth"], dtype=np.int32)
    gc = np.ascontiguousarray(groups["child"], dtype=np.int32)
    gc = gc.reshape(gp.size, -1) if gp.size else gc.reshape(0, 1)
    K = gc.shape[1]
    gq = np.ascontiguousarray(groups["logq"], dtype=np.float32)
    gz = np.ascontiguousarray(groups["ztgt"], dtype=np.float32)
    pairs = np.ascontiguousarray(pairs, dtype=np.int32).reshape(-1, 6)
    edges = np.ascontiguousarray(edges, dtype=np.int32).reshape(-1, 4)
    for ids in (gp, gc, pairs[:, [0, 1, 3, 4]], edges[:, :2]):
        if ids.size and (ids.min() < 0 or ids.max() >= V):
            raise ValueError("token id out of range")
    cfg = _TdesLossCfg(gamma, w1, lambda_kl, lambda_pair, lambda_bce)
    loss = np.zeros(4, np.float64)
    out = {"loss": loss}
    if grad:
        out.update(gP=np.zeros((V, m)), gC=np.zeros((V, m)), gu=np.zeros((L, m)), gs=np.zeros(1))
    pp = (lambda k: _p(out[k])) if grad else (lambda k: None)
    rc = lib().oracle_tdes_loss(_p(P), _p(Ctab), _p(u), C.c_double(s), V, L, m, K, int(gp.size), _p(gp), _p(gd), _p(gc),
                                _p(gq), _p(gz), int(pairs.shape[0]), _p(pairs), int(edges.shape[0]), _p(edges),
                                C.byref(cfg), _p(loss), pp("gP"), pp("gC"), pp("gu"), pp("gs"))
    if rc != 0:
        raise ValueError(f"oracle_tdes_loss failed ({rc})")
    return out


def saba_fit(state, budget, gain, prefix_len, latency):
    """Least-squares fit of the SABA gain and cost models to replay logs (Sec. 3.3, Eq. 16-17).

    The paper fits the parameters on held-out prompts by same-prefix budget replay and does not give the procedure;
    the reading restated here is ordinary least squares, in fp64, with numpy's SVD-based solver as the one step:
      gain: 0 < g_i < 1 at budget B_i  =>  tau_i = -B_i / ln(1 - g_i);  (phi, bias) = argmin sum (tau_i - phi.s_i - bias)^2
      cost: (c0, c1, c2) = argmin sum (T_i - c0 - c1 B_i - c2 B_i prefix_i)^2
    Returns dict(phi [4] = conf, degen, hist, bias; c [3]; n_gain; n_cost).
    Pins (tests/test_oracle_saba_fit.py): exact recovery of known parameters from noise-free logs, the normal
    equations' residual orthogonality, invariance under duplication and permutation of the rounds."""
    s = np.asarray(state, dtype=np.float32).astype(np.float64).reshape(-1, 3)
    B = np.asarray(budget, dtype=np.int32).astype(np.float64)
    g = np.asarray(gain, dtype=np.float32).astype(np.float64)
    pre = np.asarray(prefix_len, dtype=np.int32).astype(np.float64)
    T = np.asarray(latency, dtype=np.float32).astype(np.float64)
    use = (g > 0.0) & (g < 1.0)
    tau = -B[use] / np.log1p(-g[use])
    X = np.concatenate([s[use], np.ones((int(use.sum()), 1))], axis=1)
    phi = np.linalg.lstsq(X, tau, rcond=None)[0] if use.sum() >= 4 else np.zeros(4)
    H = np.stack([np.ones_like(B), B, B * pre], axis=1)
    c = np.linalg.lstsq(H, T, rcond=None)[0] if B.size >= 3 else np.zeros(3)
    return dict(phi=phi, c=c, n_gain=int(use.sum()), n_cost=int(B.size))


def replay_check(edge, n_nodes, parent, cand, depth, eps):
    """Is the given node set a valid best-first outcome on the oracle's edge scores up to eps?"""
    edge = np.ascontiguousarray(edge, dtype=np.float32)
    L, K, _ = edge.shape
    parent = np.ascontiguousarray(parent, dtype=np.int32)
    cand = np.ascontiguousarray(cand, dtype=np.int32)
    depth = np.ascontiguousarray(depth, dtype=np.int32)
    worst = C.c_double(0)
    rc = lib().oracle_replay_check(_p(edge), L, K, int(n_nodes), _p(parent), _p(cand), _p(depth), C.c_double(eps),
                                   C.byref(worst))
    return rc == 0, worst.value


def build_trees(logits, hidden, root_token, hist, prefix_len, fixed_budget, saba_params: SabaParams, grid, P, Ctab, u,
                s, beta, K, root_edge=1, threads: int = 1):
    """Whole round for a batch.  logits [B,L,V], hidden [B,L,dh] or None.  ``grid`` = (bmin, bmax, bstep).
    Returns a dict of arrays shaped like the library's outputs (plus cand / Ugrid / lse in fp64).
    ``threads`` > 1 splits the batch over a thread pool (ctypes releases the GIL)."""
    z, zdt = _as_bits(logits)
    Bt, L, V = z.shape
    if hidden is not None:
        h, hdt = _as_bits(hidden)
        dh = h.shape[2]
    else:
        h, hdt, dh = None, F32, 0
    bmin, bmax, bstep = grid
    Nmax = bmax + 1
    W = (Nmax + 31) // 32
    G = (bmax - bmin) // bstep + 1
    P = np.ascontiguousarray(P, dtype=np.float32)
    Ctab = np.ascontiguousarray(Ctab, dtype=np.float32)
    u = np.ascontiguousarray(u, dtype=np.float32)
    m = P.shape[1]
    root_token = np.ascontiguousarray(root_token, dtype=np.int32)
    hist = np.ascontiguousarray(hist if hist is not None else np.zeros(Bt), dtype=np.float64)
    prefix_len = np.ascontiguousarray(prefix_len, dtype=np.int32)
    fb = None if fixed_budget is None else np.ascontiguousarray(fixed_budget, dtype=np.int32)
    o = dict(
        n_nodes=np.zeros(Bt, np.int32), budget=np.zeros(Bt, np.int32), token=np.zeros((Bt, Nmax), np.int32),
        parent=np.zeros((Bt, Nmax), np.int32), depth=np.zeros((Bt, Nmax), np.int32),
        position=np.zeros((Bt, Nmax), np.int32), path_score=np.zeros((Bt, Nmax), np.float32),
        mask=np.zeros((Bt, Nmax, W), np.uint32), status=np.zeros(Bt, np.int32), cand=np.zeros((Bt, Nmax), np.int32),
        topk_id=np.zeros((Bt, L, K), np.int32), topk_lp=np.zeros((Bt, L, K), np.float32),
        lse=np.zeros((Bt, L), np.float64), edge=np.zeros((Bt, L, K, K), np.float32),
        state=np.zeros((Bt, 4), np.float64), Ugrid=np.zeros((Bt, G), np.float64),
    )
    sp = saba_params._c()

    def run(lo, hi):
        if hi <= lo:
            return 0
        sl = slice(lo, hi)
        return lib().oracle_build_trees(
            hi - lo, L, V, K, m, dh, _p(z[sl]), zdt, _p(h[sl]) if h is not None else None, hdt, _p(root_token[sl]),
            _p(hist[sl]), _p(prefix_len[sl]), _p(fb[sl]) if fb is not None else None, C.byref(sp), bmin, bmax, bstep,
            _p(P), _p(Ctab), _p(u), C.c_double(s), C.c_double(beta), int(root_edge), Nmax, W,
            _p(o["n_nodes"][sl]), _p(o["budget"][sl]), _p(o["token"][sl]), _p(o["parent"][sl]), _p(o["depth"][sl]),
            _p(o["position"][sl]), _p(o["path_score"][sl]), _p(o["mask"][sl]), _p(o["status"][sl]),
            _p(o["cand"][sl]), _p(o["topk_id"][sl]), _p(o["topk_lp"][sl]), _p(o["lse"][sl]), _p(o["edge"][sl]),
            _p(o["state"][sl]), _p(o["Ugrid"][sl]))

    if threads <= 1 or Bt == 1:
        assert run(0, Bt) == 0
    else:
        from concurrent.futures import ThreadPoolExecutor
        threads = min(threads, Bt)
        cuts = [Bt * i // threads for i in range(threads + 1)]
        with ThreadPoolExecutor(threads) as ex:
            rcs = list(ex.map(lambda i: run(cuts[i], cuts[i + 1]), range(threads)))
        assert all(r == 0 for r in rcs)
    return o

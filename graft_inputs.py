"""Seeded synthetic inputs for the GRAFT draft-tree round.

This module only *draws* inputs (random numbers, index sets, dtype rounding); it holds none of
the method's arithmetic on the round's path (the one exception is data synthesis for the fitting step:
`saba_replay_logs` evaluates the gain and latency models of Eq. 16-17 forward to fabricate the logs that
the fit is then asked to recover) and is the one piece of code that both the CPU oracle's tests and the
CUDA library's tests / benchmark use.  Every sequence is generated from its own counter-based
stream (Philox keyed by (seed, tensor tag, sequence index)), so sequence b has the same bytes
whatever the batch size or the rank that generates it.

Workload shapes (block length 16; vocabularies 32,000 / 128,256 / 151,936; hidden widths
256 / 2560 / 4096) stand in for a diffusion drafter's one-pass outputs:

* logits[b, j, v] = 2 n + boost, n ~ N(0,1); at position j a seeded set of 64 distinct token ids
  with ranks r = 1..64 gets boost H_{b,j} r^-1.1, H_{b,j} = H_b - 0.4 j;
* hidden[b, j, :]: i.i.d. N(0,1), or an AR(1) chain h_j = rho_j h_{j-1} + sqrt(1-rho_j^2) g_j with
  rho_j rising from 0.2 to 0.8 so that adjacent rows grow more similar at later positions;
* TDES tables: either (emb, W_p, b_p, W_c, b_c, u) for the table-precompute step (small cases)
  or the projected tables P, C ~ N(0,1) directly (large cases), u ~ N(0, 0.25), s = 1;
* SABA: phi = (-160, +20, -5; bias 200), tau_min = 8, cost table t(n) = 18 + 0.02 max(0, n - 64) ms;
* target ids: a continuation y_1..y_{L+1} per sequence, drawn before and independently of any tree.
"""
from __future__ import annotations

from dataclasses import dataclass, replace

import numpy as np
import torch

N_BOOST = 64
ZIPF_S = 1.1


@dataclass(frozen=True)
class Workload:
    name: str
    batch: int
    L: int
    V: int
    K: int
    hidden_dim: int
    logits_dtype: str  # "f32" | "bf16"
    hidden_dtype: str
    budget_min: int
    budget_max: int
    budget_step: int = 16
    fixed_budget: int | None = None  # None -> SABA
    boost_lo: float = 12.0  # H_b ~ U[boost_lo, boost_hi]; equal -> constant
    boost_hi: float = 12.0
    hidden_ar1: bool = True
    m: int = 128
    beta: float = 0.2
    target_mode: str = "sampled"  # "sampled" (from the boosted distribution) | "decay" (match rate 0.9 -> 0.3)
    seed: int = 20375

    @property
    def nmax(self) -> int:
        return self.budget_max + 1

    @property
    def mask_words(self) -> int:
        return (self.nmax + 31) // 32

    def with_batch(self, batch: int) -> "Workload":
        return replace(self, batch=batch)


# The five stated configurations and the headline metric's configuration "M".
C1 = Workload("C1", 1, 16, 32000, 8, 256, "f32", "f32", 64, 64, 16, fixed_budget=64, hidden_ar1=False, seed=20375)
C2 = Workload("C2", 16, 16, 151936, 16, 2560, "bf16", "bf16", 16, 256, target_mode="decay", seed=20376)
C3 = Workload("C3", 64, 16, 128256, 32, 4096, "bf16", "bf16", 16, 512, boost_lo=6.0, boost_hi=14.0,
              target_mode="decay", seed=20377)
C4 = Workload("C4", 256, 16, 151936, 32, 4096, "bf16", "bf16", 16, 512, target_mode="decay", seed=20378)
C5 = Workload("C5", 128, 16, 151936, 32, 4096, "bf16", "bf16", 16, 512, target_mode="decay", seed=20379)
M = Workload("M", 64, 16, 151936, 32, 4096, "bf16", "bf16", 16, 512, target_mode="decay", seed=20380)
WORKLOADS = {w.name: w for w in (C1, C2, C3, C4, C5, M)}

_TAGS = {"logits": 1, "hidden": 2, "boost_ids": 3, "boost_h": 4, "tables": 5, "scalars": 6, "target": 7, "emb": 8, "traces": 9, "replay": 10}


def _rng(seed: int, tag: str, b: int = 0) -> np.random.Generator:
    return np.random.Generator(np.random.Philox(key=[(seed << 8) | _TAGS[tag], b]))


def _to_dtype(x: np.ndarray, dtype: str) -> torch.Tensor:
    t = torch.from_numpy(np.ascontiguousarray(x, dtype=np.float32))
    return t.to(torch.bfloat16) if dtype == "bf16" else t  # round-to-nearest-even


def boost_ids(w: Workload, b: int) -> np.ndarray:
    """[L, 64] distinct token ids per position; column r-1 holds the rank-r boosted token."""
    g = _rng(w.seed, "boost_ids", b)
    n = min(N_BOOST, w.V)
    return np.stack([g.choice(w.V, size=n, replace=False) for _ in range(w.L)]).astype(np.int64)


def boost_height(w: Workload, b: int) -> float:
    if w.boost_hi == w.boost_lo:
        return w.boost_lo
    return float(_rng(w.seed, "boost_h", b).uniform(w.boost_lo, w.boost_hi))


def logits_seq(w: Workload, b: int) -> torch.Tensor:
    """[L, V] logits of sequence b in the workload's dtype."""
    g = _rng(w.seed, "logits", b)
    z = g.standard_normal((w.L, w.V), dtype=np.float32)
    z *= 2.0
    ids = boost_ids(w, b)
    H = boost_height(w, b)
    ranks = np.arange(1, ids.shape[1] + 1, dtype=np.float64) ** (-ZIPF_S)
    for j in range(w.L):
        z[j, ids[j]] += ((H - 0.4 * j) * ranks).astype(np.float32)
    return _to_dtype(z, w.logits_dtype)


def hidden_seq(w: Workload, b: int) -> torch.Tensor:
    g = _rng(w.seed, "hidden", b)
    x = g.standard_normal((w.L, w.hidden_dim), dtype=np.float32)
    if w.hidden_ar1 and w.L > 1:
        for j in range(1, w.L):
            rho = 0.2 + 0.6 * j / (w.L - 1)
            x[j] = rho * x[j - 1] + np.sqrt(1.0 - rho * rho) * x[j]
    return _to_dtype(x, w.hidden_dtype)


def batch_inputs(w: Workload, lo: int = 0, hi: int | None = None) -> dict:
    """Inputs of sequences lo..hi-1 (default: the whole batch) as CPU torch tensors."""
    hi = w.batch if hi is None else hi
    n = hi - lo
    logits = torch.empty((n, w.L, w.V), dtype=torch.bfloat16 if w.logits_dtype == "bf16" else torch.float32)
    hidden = torch.empty((n, w.L, w.hidden_dim), dtype=torch.bfloat16 if w.hidden_dtype == "bf16" else torch.float32)
    root = np.empty(n, np.int32)
    hist = np.empty(n, np.float32)
    prefix = np.empty(n, np.int32)
    for i, b in enumerate(range(lo, hi)):
        logits[i] = logits_seq(w, b)
        hidden[i] = hidden_seq(w, b)
        g = _rng(w.seed, "scalars", b)
        root[i] = g.integers(0, w.V)
        hist[i] = g.uniform(1.0, 9.0)
        prefix[i] = g.integers(128, 4097)
    out = dict(logits=logits, hidden=hidden, root_token=torch.from_numpy(root), hist=torch.from_numpy(hist),
               prefix_len=torch.from_numpy(prefix))
    out["fixed_budget"] = None if w.fixed_budget is None else torch.full((n,), w.fixed_budget, dtype=torch.int32)
    return out


def tdes_tables(w: Workload) -> dict:
    """Projected tables P, C [V, m] ~ N(0,1) (what emb W^T + b looks like for W ~ N(0, 1/E)), u, s."""
    g = _rng(w.seed, "tables")
    P = g.standard_normal((w.V, w.m), dtype=np.float32)
    Cc = g.standard_normal((w.V, w.m), dtype=np.float32)
    u = (0.5 * g.standard_normal((w.L, w.m), dtype=np.float32)).astype(np.float32)
    return dict(P=torch.from_numpy(P), C=torch.from_numpy(Cc), u=torch.from_numpy(u), s=1.0)


def tdes_weights(V: int, E: int, m: int, L: int, seed: int, emb_dtype: str = "f32") -> dict:
    """Raw scorer parameters for the table-precompute step: emb ~ N(0,1), W ~ N(0,1/E), b ~ N(0,0.01)."""
    g = _rng(seed, "emb")
    emb = _to_dtype(g.standard_normal((V, E), dtype=np.float32), emb_dtype)
    sc = np.float32(1.0 / np.sqrt(E))
    Wp = g.standard_normal((m, E), dtype=np.float32) * sc
    Wc = g.standard_normal((m, E), dtype=np.float32) * sc
    bp = (0.1 * g.standard_normal(m, dtype=np.float32)).astype(np.float32)
    bc = (0.1 * g.standard_normal(m, dtype=np.float32)).astype(np.float32)
    u = (0.5 * g.standard_normal((L, m), dtype=np.float32)).astype(np.float32)
    return dict(emb=emb, Wp=torch.from_numpy(Wp), bp=torch.from_numpy(bp), Wc=torch.from_numpy(Wc),
                bc=torch.from_numpy(bc), u=torch.from_numpy(u), s=1.0)


def saba_defaults(w: Workload) -> dict:
    """Synthetic SABA parameters (the fitted ones are not published) and the verification-cost table."""
    return dict(phi_conf=-160.0, phi_degen=20.0, phi_hist=-5.0, phi_bias=200.0, tau_min=8.0, cost_mode=1,
                c0=0.0, c1=0.0, c2=0.0, pts_n=[0.0, 64.0, 1024.0], pts_t=[18.0, 18.0, 18.0 + 0.02 * (1024.0 - 64.0)])


def target_tokens(w: Workload, b: int, logits_b: torch.Tensor | None = None) -> np.ndarray:
    """y_1..y_{L+1} for sequence b (int32 [L+1]); y_{L+1} is a uniform random id.

    "sampled": y_d is a draw from position d's distribution, taken as argmax(logits + Gumbel noise).
    "decay":   with probability 0.9 - 0.6 (d-1)/(L-1), y_d is the boosted token of Zipf(1.1)-distributed
               rank among that position's 64; otherwise a uniform random id.
    """
    g = _rng(w.seed, "target", b)
    y = np.empty(w.L + 1, np.int32)
    if w.target_mode == "sampled":
        z = (logits_b if logits_b is not None else logits_seq(w, b)).to(torch.float32).numpy()
        for j in range(w.L):
            y[j] = int(np.argmax(z[j] + g.gumbel(size=w.V)))
    else:
        ids = boost_ids(w, b)
        pr = np.arange(1, ids.shape[1] + 1, dtype=np.float64) ** (-ZIPF_S)
        pr /= pr.sum()
        for j in range(w.L):
            p_match = 0.9 - 0.6 * j / max(1, w.L - 1)
            if g.uniform() < p_match:
                y[j] = ids[j, g.choice(ids.shape[1], p=pr)]
            else:
                y[j] = g.integers(0, w.V)
    y[w.L] = g.integers(0, w.V)
    return y


def target_next_from_depth(y: np.ndarray, depth: np.ndarray) -> np.ndarray:
    """target_next[i] = y_{depth(i)+1}: the target's next token after node i if the path to i was accepted.
    Padding rows (depth -1) get -1."""
    d = np.asarray(depth)
    out = np.full(d.shape, -1, np.int32)
    ok = d >= 0
    out[ok] = y[d[ok]]
    return out


def tdes_traces(V: int, L: int, K: int, n_groups: int, n_pairs: int, n_edges: int, seed: int,
                pos_rate: float = 0.15) -> dict:
    """Synthetic TDES training traces (the paper's come from target-model runs that are not available).

    Token ids are Zipf-distributed over a random permutation of the vocabulary (a few hot tokens, a long tail), depths
    uniform in 1..L.  groups: a parent, a depth, K distinct children, their draft log-probabilities (descending, as
    top-K candidates are) and target logits ~ N(0, 2^2); pairs: a compatible edge and an alternative that keeps
    either its child (wrong parent) or its parent (competing child), half each; edges: (p, c, d, y) with about
    `pos_rate` positives."""
    g = _rng(seed, "traces")
    perm = g.permutation(V)
    w = 1.0 / np.arange(1, V + 1, dtype=np.float64) ** ZIPF_S
    cdf = np.cumsum(w / w.sum())

    def tokens(shape):
        return perm[np.minimum(np.searchsorted(cdf, g.random(shape)), V - 1)].astype(np.int32)

    child = np.empty((n_groups, K), np.int32)
    for i in range(n_groups):  # K distinct children per group
        got = np.unique(tokens(4 * K))
        while got.size < K:
            got = np.unique(np.concatenate([got, tokens(4 * K)]))
        child[i] = g.permutation(got)[:K]
    gaps = g.exponential(0.7, size=(n_groups, K)).astype(np.float32)
    logq = -np.cumsum(gaps, axis=1, dtype=np.float32)
    groups = dict(parent=tokens(n_groups), depth=g.integers(1, L + 1, n_groups).astype(np.int32), child=child,
                  logq=logq.astype(np.float32), ztgt=(2.0 * g.standard_normal((n_groups, K))).astype(np.float32))
    pos = np.stack([tokens(n_pairs), tokens(n_pairs), g.integers(1, L + 1, n_pairs).astype(np.int32)], axis=1)
    neg = pos.copy()
    swap_parent = g.random(n_pairs) < 0.5
    neg[swap_parent, 0] = tokens(int(swap_parent.sum()))
    neg[~swap_parent, 1] = tokens(int((~swap_parent).sum()))
    pairs = np.concatenate([pos, neg], axis=1).astype(np.int32)
    edges = np.stack([tokens(n_edges), tokens(n_edges), g.integers(1, L + 1, n_edges).astype(np.int32),
                      (g.random(n_edges) < pos_rate).astype(np.int32)], axis=1).astype(np.int32)
    return dict(groups=groups, pairs=pairs, edges=edges)


def saba_replay_logs(n: int, seed: int, phi=(-160.0, 20.0, -5.0, 200.0), c=(6.0, 0.012, 2.0e-6), noise: float = 0.02,
                     bmin: int = 32, bmax: int = 512, bstep: int = 16) -> dict:
    """Synthetic same-prefix budget replay logs (the paper's come from held-out prompts run through the models).

    Per logged round: a decoding state (conf ~ U(0.2, 0.95), degen ~ U(0.5, 1.4), hist ~ U(0, 8)), a budget from the
    paper's grid, a prefix length ~ U{16..4096}; the gain and the latency follow the models of Eq. 16-17 with the
    given parameters, times (1 + noise * N(0,1)) each; gains are clipped to [0, 1]."""
    g = _rng(seed, "replay")
    state = np.stack([g.uniform(0.2, 0.95, n), g.uniform(0.5, 1.4, n), g.uniform(0.0, 8.0, n)], axis=1)
    budget = (bmin + bstep * g.integers(0, (bmax - bmin) // bstep + 1, n)).astype(np.int32)
    prefix = g.integers(16, 4097, n).astype(np.int32)
    tau = state @ np.asarray(phi[:3]) + phi[3]
    gain = (1.0 - np.exp(-budget / np.maximum(tau, 1.0))) * (1.0 + noise * g.standard_normal(n))
    lat = (c[0] + c[1] * budget + c[2] * budget * prefix.astype(np.float64)) * (1.0 + noise * g.standard_normal(n))
    return dict(state=state.astype(np.float32), budget=budget, gain=np.clip(gain, 0.0, 1.0).astype(np.float32),
                prefix_len=prefix, latency=lat.astype(np.float32))


STYLES = ("normal", "quant1", "quant025", "flat", "peaked", "mixed", "huge", "masked", "twopeaks", "ramp")


def styled_logits(z, style, rng, gen, K):
    """Logits of one of ten shapes, from ordinary to degenerate (z: fp32 [batch, L, V] drawn by graft_inputs)."""
    Bt, L, V = z.shape
    if style == "quant1":
        return torch.round(z)
    if style == "quant025":
        return torch.round(z * 4) / 4
    if style == "flat":
        return 1e-3 * torch.randn(z.shape, generator=gen)
    if style == "peaked":       # one token of probability 1 to fp32 precision
        out = torch.zeros_like(z)
        return out.scatter_(2, torch.randint(0, V, (Bt, L), generator=gen)[..., None], 30.0)
    if style == "twopeaks":     # two equal winners (or one, where the draws coincide)
        out = torch.zeros_like(z)
        out.scatter_(2, torch.randint(0, V, (Bt, L), generator=gen)[..., None], 20.0)
        return out.scatter_(2, torch.randint(0, V, (Bt, L), generator=gen)[..., None], 20.0)
    if style == "mixed":
        out = torch.round(z)
        out[:, ::2] = 0.0
        return out
    if style == "huge":         # log-probabilities in the hundreds: one fp32 ulp is above the tolerance
        return z * float(rng.choice([5.0, 10.0, 30.0]))
    if style == "masked":       # between one and 2K finite tokens per row
        keep_n = int(rng.integers(1, max(2, min(V, 2 * K))))
        return z.masked_fill(torch.rand(z.shape, generator=gen).argsort(dim=2) >= keep_n, float("-inf"))
    if style == "ramp":
        return -torch.arange(V, dtype=torch.float32).expand(z.shape).clone() * float(rng.choice([1e-3, 0.1, 1.0]))
    return z


def adversarial_rows(V, gen):
    """Named single rows (fp32 [V]) that defeat a top-K filter built on partitions of a row: sorted rows, blocks of
    large elements, rows of ramps of several periods, bulk and sparse ties, masked halves.  For timing the vocab pass
    on its worst cases; `gen` is a seeded torch.Generator."""
    ar = torch.arange(V, dtype=torch.float32)
    base = 2.0 * torch.randn(V, generator=gen)
    srt = torch.sort(2.0 * torch.randn(V, generator=gen)).values
    low = -1.0 - 7.0 * torch.rand(V, generator=gen)
    rows = [("ordinary", base), ("sorted ascending", srt), ("sorted descending", srt.flip(0))]
    for s in (1e-3, 0.1, 1.0):
        rows.append((f"ramp up, step {s:g} (ties in bf16)", ar * s))
        rows.append((f"ramp down, step {s:g} (ties in bf16)", -ar * s))
    for n in sorted({min(n, V // 2) for n in (1000, 5000, 50000)}):
        at = V // 8
        z = base.clone()
        z[at:at + n] += 20.0
        rows.append((f"block of {n} large elements", z))
        z = base.clone()
        z[at:at + n] = 20.0 + torch.sort(torch.randn(n, generator=gen)).values
        rows.append((f"sorted block of {n} large elements", z))
    for per in (32, 256, 512, 1024, 2048, 4096, 6144, 16384):
        rows.append((f"ramps of period {per}, rising", (ar % per) / per * 8))
        rows.append((f"ramps of period {per}, falling", -(ar % per) / per * 8))
    rows.append(("ramps of period 1024, falling, distinct tops", -(ar % 1024) / 1024 * 8 + (ar // 1024) * 1e-2))
    rows.append(("all equal", torch.zeros(V)))
    rows.append(("alternating +1 / -1", torch.where(ar % 2 == 0, 1.0, -1.0)))
    rows.append(("two values at random", torch.where(torch.rand(V, generator=gen) < 0.5, 1.0, 0.0)))
    rows.append(("coarse grid of 1/8", torch.round(base * 8) / 8))
    z = low.clone()
    z[::1024] = 0.0
    rows.append(("one tied winner in 1024 over a lower rest", z))
    z = low.clone()
    z[::256] = 0.0
    rows.append(("one tied winner in 256 over a lower rest", z))
    rows.append(("forty winners at the end of a flat row", torch.cat([torch.zeros(V - 40), torch.arange(40).float()])))
    rows.append(("2000 rising elements at the end", torch.cat([base[: V - min(2000, V // 2)], 10 + torch.arange(min(2000, V // 2)).float() * 0.01])))
    z = base.clone()
    z[::2] = float("-inf")
    rows.append(("every second element -inf", z))
    z = base.clone()
    z[: V // 2] = float("-inf")
    rows.append(("front half -inf", z))
    rows.append(("heavy tail (cubed)", base ** 3))
    return rows


def small(name: str = "T", **kw) -> Workload:
    """A small workload for tests; override any field."""
    base = dict(name=name, batch=2, L=4, V=1000, K=4, hidden_dim=32, logits_dtype="f32", hidden_dtype="f32",
                budget_min=8, budget_max=24, budget_step=8, fixed_budget=None, m=16, seed=7)
    base.update(kw)
    return Workload(**base)

"""Pins of the oracle's TDES training objective (Eq. 7-12) to things other than itself: library loss routines on
scores from a matrix product, reverse-mode differentiation of the plain definition, finite differences, a
hand-computed example and the cases where a term vanishes."""
import math

import numpy as np
import torch
import torch.nn.functional as F

import graft_inputs as gi
import oracle

CFG = dict(gamma=0.7, w1=3.0, lambda_kl=1.0, lambda_pair=1.0, lambda_bce=0.25)


def _setup(V=60, L=5, K=6, m=8, n_groups=9, n_pairs=11, n_edges=13, seed=5, s=1.3):
    g = np.random.default_rng(seed)
    P = g.standard_normal((V, m)).astype(np.float32)
    Ct = g.standard_normal((V, m)).astype(np.float32)
    u = (0.5 * g.standard_normal((L, m))).astype(np.float32)
    tr = gi.tdes_traces(V, L, K, n_groups, n_pairs, n_edges, seed)
    return P, Ct, u, s, tr


def _torch_losses(P, Ct, u, s, tr, cfg):
    """The three losses from torch's own loss routines; the scores come from batched matrix products."""
    m = P.shape[1]
    gr = tr["groups"]
    d = torch.from_numpy(gr["depth"]).long() - 1
    a = P[torch.from_numpy(gr["parent"]).long()] + u[d]                                    # [G, m]
    b = Ct[torch.from_numpy(gr["child"]).long()] + u[d][:, None, :]                        # [G, K, m]
    f = s * torch.bmm(b, a[:, :, None])[:, :, 0] / math.sqrt(m)                            # [G, K]
    logq = torch.from_numpy(gr["logq"]).double()
    z = torch.from_numpy(gr["ztgt"]).double()
    l_kl = F.kl_div(F.log_softmax(logq + f, dim=1), F.softmax(z, dim=1), reduction="batchmean")

    def score(e):
        e = torch.from_numpy(np.ascontiguousarray(e)).long()
        aa = P[e[:, 0]] + u[e[:, 2] - 1]
        bb = Ct[e[:, 1]] + u[e[:, 2] - 1]
        return s * (aa * bb).sum(1) / math.sqrt(m)

    pr = tr["pairs"]
    l_pair = F.softplus(cfg["gamma"] - score(pr[:, :3]) + score(pr[:, 3:])).mean()
    ed = tr["edges"]
    y = torch.from_numpy(ed[:, 3].astype(np.float64))
    l_bce = F.binary_cross_entropy_with_logits(score(ed[:, :3]), y, pos_weight=torch.tensor(cfg["w1"]).double())
    total = cfg["lambda_kl"] * l_kl + cfg["lambda_pair"] * l_pair + cfg["lambda_bce"] * l_bce
    return l_kl, l_pair, l_bce, total


def test_losses_are_the_library_routines_and_gradients_are_autograd():
    P, Ct, u, s, tr = _setup()
    o = oracle.tdes_loss(P, Ct, u, s, tr["groups"], tr["pairs"], tr["edges"], **CFG)
    tp = torch.from_numpy(P).double().requires_grad_()
    tc = torch.from_numpy(Ct).double().requires_grad_()
    tu = torch.from_numpy(u).double().requires_grad_()
    ts = torch.tensor(s, dtype=torch.float64, requires_grad=True)
    l_kl, l_pair, l_bce, total = _torch_losses(tp, tc, tu, ts, tr, CFG)
    assert np.allclose(o["loss"], [l_kl.item(), l_pair.item(), l_bce.item(), total.item()], rtol=1e-12, atol=1e-13)
    total.backward()
    for name, t in (("gP", tp), ("gC", tc), ("gu", tu)):
        assert np.allclose(o[name], t.grad.numpy(), rtol=1e-10, atol=1e-13), name
        assert np.abs(o[name]).max() > 1e-4
    assert abs(o["gs"][0] - ts.grad.item()) <= 1e-11 * max(1.0, abs(ts.grad.item()))


def test_gradients_against_central_differences():
    P, Ct, u, s, tr = _setup(seed=8)
    o = oracle.tdes_loss(P, Ct, u, s, tr["groups"], tr["pairs"], tr["edges"], **CFG)

    def total(P_, C_, u_, s_):
        return oracle.tdes_loss(P_, C_, u_, s_, tr["groups"], tr["pairs"], tr["edges"], grad=False, **CFG)["loss"][3]

    rng = np.random.default_rng(0)
    h = 2.0 ** -7  # exactly representable steps: the arrays are fp32
    for name, idx in (("gP", 0), ("gC", 1), ("gu", 2)):
        arr = (P, Ct, u)[idx]
        nz = np.argwhere(np.abs(o[name]) > 1e-5)
        assert len(nz) > 10
        for r, k in nz[rng.choice(len(nz), 12, replace=False)]:
            hi, lo = [a.copy() for a in (P, Ct, u)], [a.copy() for a in (P, Ct, u)]
            hi[idx][r, k] = arr[r, k] + np.float32(h)
            lo[idx][r, k] = arr[r, k] - np.float32(h)
            step = float(hi[idx][r, k]) - float(lo[idx][r, k])
            fd = (total(*hi, s) - total(*lo, s)) / step
            assert abs(fd - o[name][r, k]) <= 2e-3 * max(abs(fd), 1e-2), (name, r, k, fd, o[name][r, k])
    fd = (total(P, Ct, u, s + 1e-4) - total(P, Ct, u, s - 1e-4)) / 2e-4
    assert abs(fd - o["gs"][0]) <= 1e-5 * max(1.0, abs(fd))


def test_hand_computed_example():
    # V = 3, m = 1, L = 1, s = 2: a = P[0] + u = 1.5; children 1 and 2: b = -0.5 and 3.5, so f = -1.5 and 10.5
    P = np.array([[1.0], [2.0], [0.0]], np.float32)
    Ct = np.array([[0.5], [-1.0], [3.0]], np.float32)
    u = np.array([[0.5]], np.float32)
    groups = dict(parent=[0], depth=[1], child=[[1, 2]], logq=[[math.log(0.5)] * 2], ztgt=[[0.0, 0.0]])
    pairs = [[0, 1, 1, 0, 2, 1]]
    edges = [[0, 1, 1, 1]]
    o = oracle.tdes_loss(P, Ct, u, 2.0, groups, pairs, edges, gamma=1.0, w1=3.0, lambda_kl=1.0, lambda_pair=0.5,
                         lambda_bce=0.25)
    # pi_theta = softmax(-1.5, 10.5), pi_tgt = (1/2, 1/2): KL = -ln 2 - (ln pi_1 + ln pi_2) / 2 = 6 - ln 2 + ln(1 + e^-12)
    kl = 6.0 - math.log(2.0) + math.log1p(math.exp(-12.0))
    pair = 13.0 + math.log1p(math.exp(-13.0))          # softplus(1 + 1.5 + 10.5)
    bce = 3.0 * (1.5 + math.log1p(math.exp(-1.5)))     # -3 ln sigma(-1.5)
    assert np.allclose(o["loss"], [kl, pair, bce, kl + 0.5 * pair + 0.25 * bce], rtol=1e-14)
    assert abs(kl - 5.306858963) < 1e-8 and abs(pair - 13.00000226) < 1e-8 and abs(bce - 5.104239834) < 1e-8
    # d L / d f1 and d L / d f2, then the chain rule through f = 2 a b by hand
    p1 = 1.0 / (1.0 + math.exp(12.0))
    sig13 = 1.0 / (1.0 + math.exp(-13.0))
    g1 = (p1 - 0.5) - 0.5 * sig13 - 0.25 * 3.0 / (1.0 + math.exp(-1.5))
    g2 = ((1.0 - p1) - 0.5) + 0.5 * sig13
    assert np.allclose(o["gC"][:, 0], [0.0, g1 * 2 * 1.5, g2 * 2 * 1.5], rtol=1e-13)
    assert np.allclose(o["gP"][:, 0], [g1 * 2 * -0.5 + g2 * 2 * 3.5, 0.0, 0.0], rtol=1e-13)
    assert np.allclose(o["gu"][0, 0], g1 * 2 * (1.5 - 0.5) + g2 * 2 * (1.5 + 3.5), rtol=1e-13)
    assert np.allclose(o["gs"][0], g1 * -0.75 + g2 * 5.25, rtol=1e-13)


def test_terms_that_vanish():
    P, Ct, u, s, tr = _setup(seed=12, n_pairs=0, n_edges=0)
    gr = dict(tr["groups"])
    # the parent tower cancels (P[p] = -u_d), so f = 0 for every child, and the target equals the draft up to a shift
    gr["depth"] = np.full_like(gr["depth"], 2)
    P[gr["parent"]] = -u[1]
    gr["ztgt"] = gr["logq"] + np.float32(7.0)
    o = oracle.tdes_loss(P, Ct, u, s, gr, tr["pairs"], tr["edges"], **CFG)
    assert np.all(np.abs(o["loss"]) < 1e-6)  # the shifted fp32 logits differ from the draft's by rounding only
    for k in ("gP", "gC", "gu", "gs"):
        assert np.abs(o[k]).max() < 1e-6
    # a shift of the target logits changes nothing; lambda = 0 switches a term and its gradient off
    P, Ct, u, s, tr = _setup(seed=13)
    a = oracle.tdes_loss(P, Ct, u, s, tr["groups"], tr["pairs"], tr["edges"], **CFG)
    gr = dict(tr["groups"])
    gr["ztgt"] = (gr["ztgt"].astype(np.float64) + 4.0).astype(np.float32)
    b = oracle.tdes_loss(P, Ct, u, s, gr, tr["pairs"], tr["edges"], **CFG)
    assert np.allclose(a["loss"], b["loss"], rtol=0, atol=1e-5)
    only_pair = oracle.tdes_loss(P, Ct, u, s, tr["groups"], tr["pairs"], tr["edges"],
                                 **dict(CFG, lambda_kl=0.0, lambda_bce=0.0))
    no_items = oracle.tdes_loss(P, Ct, u, s, dict(parent=[], depth=[], child=np.zeros((0, 6)), logq=np.zeros((0, 6)),
                                                  ztgt=np.zeros((0, 6))), tr["pairs"], [],
                                **dict(CFG, lambda_kl=1.0, lambda_bce=1.0))
    assert np.allclose(only_pair["gP"], no_items["gP"], rtol=1e-13, atol=0)
    assert no_items["loss"][0] == 0.0 and no_items["loss"][2] == 0.0
    assert abs(only_pair["loss"][3] - only_pair["loss"][1]) < 1e-15

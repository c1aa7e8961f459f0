"""Parity of graft_tdes_loss (TDES training objective and gradients, Eq. 7-12) with the oracle, through the C ABI."""
import numpy as np
import pytest
import torch

import graft_inputs as gi
import oracle

pytestmark = pytest.mark.gpu

CFG = dict(gamma=0.5, w1=4.0, lambda_kl=1.0, lambda_pair=1.0, lambda_bce=0.25)  # the paper's loss weights
LOSS_RTOL = 1e-5    # fp32 scores and softmaxes, fp64 sums
GRAD_TOL = 1e-4     # of the largest gradient entry: fp32 atomic additions in no fixed order


def _ctx(V, L, K, m, seed):
    from paper_2608_20375_b200 import Graft
    g = Graft(V, L, K, m, 32, 1, 8, 16, 8, 0.2, 1, 0, 0)
    rng = np.random.default_rng(seed)
    P = rng.standard_normal((V, m)).astype(np.float32)
    Ct = rng.standard_normal((V, m)).astype(np.float32)
    u = (0.5 * rng.standard_normal((L, m))).astype(np.float32)
    s = 0.8
    keep = [torch.from_numpy(x).cuda() for x in (P, Ct, u)]
    g.set_tdes_tables(keep[0], keep[1], keep[2], s)
    return g, P, Ct, u, s, keep


def _dev(tr):
    groups = {k: torch.from_numpy(np.ascontiguousarray(v)).cuda() for k, v in tr["groups"].items()}
    return groups, torch.from_numpy(tr["pairs"]).cuda(), torch.from_numpy(tr["edges"]).cuda()


def _run(g, V, L, m, tr, grad=True, cfg=CFG):
    groups, pairs, edges = _dev(tr)
    loss = torch.full((4,), 7.0, dtype=torch.float64, device="cuda")  # overwritten
    skipped = torch.full((1,), -1, dtype=torch.int32, device="cuda")
    out = dict(loss=loss, skipped=skipped)
    if grad:
        out.update(gP=torch.zeros((V, m), device="cuda"), gC=torch.zeros((V, m), device="cuda"),
                   gu=torch.zeros((L, m), device="cuda"), gs=torch.zeros(1, device="cuda"))
    g.tdes_loss(groups, pairs, edges, loss=loss, skipped=skipped, gP=out.get("gP"), gC=out.get("gC"),
                gu=out.get("gu"), gs=out.get("gs"), **cfg)
    torch.cuda.synchronize()
    return {k: v.cpu().numpy() for k, v in out.items()}


def _compare(got, ref, grad=True):
    assert np.all(np.abs(got["loss"] - ref["loss"]) <= LOSS_RTOL * np.maximum(1.0, np.abs(ref["loss"]))), \
        (got["loss"], ref["loss"])
    if grad:
        for k in ("gP", "gC", "gu", "gs"):
            scale = max(np.abs(ref[k]).max(), 1e-12)
            err = np.abs(got[k].astype(np.float64) - ref[k]).max()
            assert err <= GRAD_TOL * scale, (k, err, scale)
            # rows nobody touched stay exactly zero
            if k in ("gP", "gC"):
                untouched = ~np.any(ref[k] != 0.0, axis=1)
                assert not np.any(got[k][untouched])


@pytest.mark.parametrize("V,L,K,m,ng,npair,ne", [
    (500, 6, 6, 16, 40, 50, 70),            # less than one CTA's worth of warps
    (3000, 16, 32, 128, 700, 1500, 2501),   # the paper's shapes, several CTAs and a ragged tail
    (2000, 8, 5, 40, 333, 0, 999),          # m not a multiple of 128, no pairs
    (1500, 4, 8, 256, 200, 300, 0),         # two 128-float chunks per row, no edges
    (1200, 3, 7, 384, 150, 150, 150),       # three chunks
    (900, 32, 1, 8, 100, 100, 100),         # K = 1: pi = 1, the distribution term vanishes
])
def test_loss_and_gradients(V, L, K, m, ng, npair, ne):
    g, P, Ct, u, s, keep = _ctx(V, L, K, m, seed=V + m)
    tr = gi.tdes_traces(V, L, K, ng, npair, ne, seed=V + K)
    got = _run(g, V, L, m, tr)
    ref = oracle.tdes_loss(P, Ct, u, s, tr["groups"], tr["pairs"], tr["edges"], **CFG)
    _compare(got, ref)
    assert got["skipped"][0] == 0
    if K == 1:
        assert abs(got["loss"][0]) < 1e-6
    # losses only: the same losses, nothing else written
    lo = _run(g, V, L, m, tr, grad=False)
    assert np.array_equal(lo["loss"], got["loss"]) or np.allclose(lo["loss"], got["loss"], rtol=1e-12)
    g.destroy()


def test_hot_rows_and_many_items():
    """A tiny vocabulary: thousands of atomic additions land on each gradient row."""
    V, L, K, m = 40, 4, 8, 64
    g, P, Ct, u, s, keep = _ctx(V, L, K, m, seed=3)
    tr = gi.tdes_traces(V, L, K, 4000, 9000, 20000, seed=4)
    got = _run(g, V, L, m, tr)
    ref = oracle.tdes_loss(P, Ct, u, s, tr["groups"], tr["pairs"], tr["edges"], **CFG)
    _compare(got, ref)
    g.destroy()


def test_items_with_bad_ids_are_left_out():
    V, L, K, m = 800, 5, 6, 32
    g, P, Ct, u, s, keep = _ctx(V, L, K, m, seed=9)
    tr = gi.tdes_traces(V, L, K, 120, 130, 140, seed=10)
    gr = {k: v.copy() for k, v in tr["groups"].items()}
    pairs, edges = tr["pairs"].copy(), tr["edges"].copy()
    gr["parent"][3] = V          # token past the table
    gr["child"][10, 2] = -1      # negative token
    gr["depth"][20] = 0          # depth below 1
    gr["depth"][21] = L + 1
    pairs[5, 4] = V + 7
    pairs[6, 2] = 0
    edges[7, 0] = -5
    edges[8, 2] = L + 3
    bad_g, bad_p, bad_e = [3, 10, 20, 21], [5, 6], [7, 8]
    got = _run(g, V, L, m, dict(groups=gr, pairs=pairs, edges=edges))
    assert got["skipped"][0] == 8
    keep_g = np.setdiff1d(np.arange(120), bad_g)
    sub = dict(groups={k: v[keep_g] for k, v in gr.items()}, pairs=np.delete(pairs, bad_p, 0),
               edges=np.delete(edges, bad_e, 0))
    # the oracle on the remaining items; its means divide by fewer items, the library's by all of them
    cfg = dict(CFG, lambda_kl=CFG["lambda_kl"] * 116 / 120, lambda_pair=CFG["lambda_pair"] * 128 / 130,
               lambda_bce=CFG["lambda_bce"] * 138 / 140)
    ref = oracle.tdes_loss(P, Ct, u, s, sub["groups"], sub["pairs"], sub["edges"], **cfg)
    ref["loss"][:3] *= np.array([116 / 120, 128 / 130, 138 / 140])
    _compare(got, ref)
    g.destroy()


def test_empty_lists_and_argument_checks():
    from paper_2608_20375_b200 import GraftError
    V, L, K, m = 300, 4, 4, 16
    g, P, Ct, u, s, keep = _ctx(V, L, K, m, seed=1)
    loss = torch.ones(4, dtype=torch.float64, device="cuda")
    gP = torch.zeros((V, m), device="cuda")
    g.tdes_loss(None, None, None, loss=loss, **CFG)
    torch.cuda.synchronize()
    assert loss.cpu().tolist() == [0.0, 0.0, 0.0, 0.0]
    with pytest.raises(GraftError):  # some but not all gradient buffers
        g.tdes_loss(None, None, None, loss=loss, gP=gP, **CFG)
    g.destroy()


def test_full_size_tables():
    """The paper's shapes: V = 151,936, m = 128, L = 16, K = 32; tens of thousands of items."""
    V, L, K, m = 151936, 16, 32, 128
    g, P, Ct, u, s, keep = _ctx(V, L, K, m, seed=21)
    tr = gi.tdes_traces(V, L, K, 8192, 16384, 32768, seed=22)
    got = _run(g, V, L, m, tr)
    ref = oracle.tdes_loss(P, Ct, u, s, tr["groups"], tr["pairs"], tr["edges"], **CFG)
    _compare(got, ref)
    g.destroy()

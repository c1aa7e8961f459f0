"""Parity of graft_saba_fit (least-squares fit of the SABA models, Eq. 16-17) with the oracle, through the C ABI."""
import numpy as np
import pytest
import torch

import graft_inputs as gi
import oracle

pytestmark = pytest.mark.gpu

# both sides work in fp64 on the same fp32 logs; the library solves the normal equations (columns scaled), the oracle
# an SVD: the difference is the conditioning of the scaled normal equations times fp64 rounding
RTOL = 1e-8


def _ctx():
    from paper_2608_20375_b200 import Graft
    return Graft(1000, 4, 4, 16, 8, 1, 8, 8, 8, 0.0, 1, 0, 0)


def _fit(g, lg):
    dev = {k: torch.from_numpy(np.ascontiguousarray(v)).cuda() for k, v in lg.items()}
    out = torch.full((10,), 7.0, dtype=torch.float64, device="cuda")
    g.saba_fit(dev["state"], dev["budget"], dev["gain"], dev["prefix_len"], dev["latency"], out)
    torch.cuda.synchronize()
    return out.cpu().numpy()


@pytest.mark.parametrize("n,seed,noise", [(7, 1, 0.02), (1000, 2, 0.02), (100003, 3, 0.05), (2_000_000, 4, 0.02),
                                          (5000, 5, 0.0)])
def test_fit_matches_the_oracle(n, seed, noise):
    g = _ctx()
    lg = gi.saba_replay_logs(n, seed=seed, noise=noise)
    ref = oracle.saba_fit(**lg)
    for _ in range(2):  # the accumulators clear themselves: a second call gives the same answer
        got = _fit(g, lg)
        assert got[9] == 0.0
        assert got[7] == ref["n_gain"] and got[8] == ref["n_cost"]
        scale_phi = np.abs(ref["phi"]).max()
        assert np.all(np.abs(got[:4] - ref["phi"]) <= RTOL * scale_phi * 10), (got[:4], ref["phi"])
        assert np.all(np.abs(got[4:7] - ref["c"]) <= RTOL * np.maximum(np.abs(ref["c"]), 1e-9) * 100), (got[4:7], ref["c"])
    g.destroy()


def test_degenerate_logs_are_reported():
    g = _ctx()
    lg = gi.saba_replay_logs(50, seed=8)
    lg["gain"][:] = 1.0               # nothing to fit the gain model to
    lg["budget"][:] = 64              # one budget: the cost columns are dependent
    lg["prefix_len"][:] = 100
    got = _fit(g, lg)
    assert int(got[9]) == 3 and not np.any(got[:7])
    assert got[7] == 0 and got[8] == 50
    # a usable call afterwards is not disturbed by the failed one
    lg2 = gi.saba_replay_logs(500, seed=9)
    ref = oracle.saba_fit(**lg2)
    got2 = _fit(g, lg2)
    assert got2[9] == 0.0 and np.allclose(got2[4:7], ref["c"], rtol=1e-6)
    g.destroy()


def test_unaligned_arrays_take_the_scalar_path():
    g = _ctx()
    lg = gi.saba_replay_logs(3001, seed=12)
    dev = {k: torch.from_numpy(np.ascontiguousarray(v)).cuda() for k, v in lg.items()}
    out = torch.zeros(10, dtype=torch.float64, device="cuda")
    # views that start one round in: 4 bytes (12 for the state) past a 16-byte boundary
    g.saba_fit(dev["state"][1:], dev["budget"][1:], dev["gain"][1:], dev["prefix_len"][1:], dev["latency"][1:], out)
    torch.cuda.synchronize()
    ref = oracle.saba_fit(**{k: v[1:] for k, v in lg.items()})
    got = out.cpu().numpy()
    assert got[9] == 0.0 and got[8] == 3000
    assert np.allclose(got[:4], ref["phi"], rtol=1e-7) and np.allclose(got[4:7], ref["c"], rtol=1e-7)
    g.destroy()

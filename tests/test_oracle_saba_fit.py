"""Pins of the oracle's least-squares fit of the SABA models (Eq. 16-17): what the mathematics fixes."""
import numpy as np

import graft_inputs as gi
import oracle


def test_noise_free_logs_give_the_parameters_back():
    phi, c = (-120.0, 35.0, -4.0, 180.0), (5.0, 0.02, 3.0e-6)
    n = 4000
    rng = np.random.default_rng(1)
    state = np.stack([rng.uniform(0.2, 0.95, n), rng.uniform(0.5, 1.4, n), rng.uniform(0, 8, n)], 1).astype(np.float32)
    budget = (32 + 16 * rng.integers(0, 31, n)).astype(np.int32)
    prefix = rng.integers(16, 4097, n).astype(np.int32)
    tau = state.astype(np.float64) @ np.array(phi[:3]) + phi[3]
    # gains and latencies straight from Eq. 16-17 (kept in fp64 -> fp32 rounding is the only noise)
    gain = (-np.expm1(-budget / tau)).astype(np.float32)
    lat = (c[0] + c[1] * budget + c[2] * budget * prefix.astype(np.float64)).astype(np.float32)
    f = oracle.saba_fit(state, budget, gain, prefix, lat)
    assert np.allclose(f["phi"], phi, rtol=2e-3, atol=0.3)     # fp32 gains near 1 carry little of tau
    assert np.allclose(f["c"], c, rtol=1e-4)
    assert f["n_gain"] == int(((gain > 0) & (gain < 1)).sum()) and f["n_cost"] == n


def test_residuals_are_orthogonal_to_the_regressors():
    lg = gi.saba_replay_logs(3000, seed=5)
    f = oracle.saba_fit(**lg)
    g = lg["gain"].astype(np.float64)
    use = (g > 0) & (g < 1)
    B = lg["budget"].astype(np.float64)
    tau = -B[use] / np.log1p(-g[use])
    X = np.concatenate([lg["state"][use].astype(np.float64), np.ones((use.sum(), 1))], 1)
    r = tau - X @ f["phi"]
    assert np.all(np.abs(X.T @ r) <= 1e-7 * np.abs(X.T @ tau))
    H = np.stack([np.ones_like(B), B, B * lg["prefix_len"]], 1)
    r2 = lg["latency"].astype(np.float64) - H @ f["c"]
    assert np.all(np.abs(H.T @ r2) <= 1e-7 * np.abs(H.T @ lg["latency"].astype(np.float64)))
    # and the fit is close to the parameters the logs were drawn from (2 % multiplicative noise)
    assert np.allclose(f["c"], (6.0, 0.012, 2.0e-6), rtol=0.05)


def test_duplicated_and_permuted_rounds_do_not_move_the_fit():
    lg = gi.saba_replay_logs(500, seed=9)
    f = oracle.saba_fit(**lg)
    perm = np.random.default_rng(0).permutation(500)
    twice = {k: np.concatenate([v[perm], v]) for k, v in lg.items()}
    f2 = oracle.saba_fit(**twice)
    assert np.allclose(f["phi"], f2["phi"], rtol=1e-9) and np.allclose(f["c"], f2["c"], rtol=1e-9)
    assert f2["n_cost"] == 1000


def test_gains_of_zero_and_one_are_left_out():
    lg = gi.saba_replay_logs(400, seed=3)
    lg["gain"][:50] = 1.0
    lg["gain"][50:80] = 0.0
    f = oracle.saba_fit(**lg)
    rest = {k: v[80:] for k, v in lg.items()}
    f2 = oracle.saba_fit(**rest)
    assert np.allclose(f["phi"], f2["phi"], rtol=1e-10)
    assert f["n_gain"] == f2["n_gain"] and f["n_cost"] == 400

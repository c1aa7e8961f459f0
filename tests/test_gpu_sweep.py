"""The budget / beta sweep harness of bench.py (`--sweep`): its node counts, budgets and accepted lengths against the
oracle run the same way (same inputs, same beta and budget rule, the oracle's own trees and walk), on a small workload.
The sweep's targets are synthetic; this test checks the harness, not the paper's gains."""
import numpy as np
import pytest
import torch

import bench
import graft_inputs as gi
import oracle
from helpers import oracle_round

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("name,beta,fixed", bench.sweep_arms(48)[:4] + [("beta=0.4 (SABA budget)", 0.4, None)])
def test_sweep_arm_matches_the_oracle(name, beta, fixed):
    w = gi.small(batch=6, L=8, V=20011, K=16, budget_min=16, budget_max=128, budget_step=16, m=32, hidden_dim=64,
                 logits_dtype="bf16", hidden_dtype="bf16", target_mode="decay", seed=4242)
    x = gi.batch_inputs(w)
    x["seq_ids"] = list(range(w.batch))
    got = bench.sweep_arm(w, x, beta, fixed, torch.device("cuda", 0), rounds=2)
    assert got["us_per_round"] > 0
    # the oracle, run the same way
    wb = gi.Workload(**{**w.__dict__, "beta": beta})
    xo = dict(x, fixed_budget=None if fixed is None else torch.full((w.batch,), fixed, dtype=torch.int32))
    tb = gi.tdes_tables(w)
    orc = oracle_round(oracle, wb, xo, tb, gi.saba_defaults(w))
    nodes, acc = [], []
    for b in range(w.batch):
        tn = gi.target_next_from_depth(gi.target_tokens(w, b), orc["depth"][b])
        a, _, _ = oracle.accept(int(orc["n_nodes"][b]), orc["token"][b], orc["parent"][b], tn, w.L)
        nodes.append(int(orc["n_nodes"][b]) - 1)
        acc.append(a)
    assert np.array_equal(got["budget"], orc["budget"])
    assert np.array_equal(got["nodes"], nodes)
    assert np.array_equal(got["accepted"], acc)
    assert got["avg_nodes"] == pytest.approx(np.mean(nodes))
    assert got["mean_accepted"] == pytest.approx(np.mean(acc))
    cost = np.interp(nodes, gi.saba_defaults(w)["pts_n"], gi.saba_defaults(w)["pts_t"])
    assert got["modelled_verify_ms"] == pytest.approx(cost.mean())
    if fixed is not None:
        assert (got["budget"] == fixed).all()

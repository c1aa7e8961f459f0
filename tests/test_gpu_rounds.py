"""Several decoding rounds in a row with the acceptance history kept on the device (Eq. 15), and the round
captured in a CUDA graph."""
import numpy as np
import pytest
import torch

import graft_inputs as gi
import oracle
from helpers import compare_round, gpu_round, oracle_round

pytestmark = pytest.mark.gpu

DT = {"f32": 0, "bf16": 1}


def _graft(w):
    from paper_2608_20375_b200 import Graft
    g = Graft(w.V, w.L, w.K, w.m, w.hidden_dim, w.batch, w.budget_min, w.budget_max, w.budget_step, w.beta, 1,
              DT[w.logits_dtype], DT[w.hidden_dtype])
    tb = gi.tdes_tables(w)
    saba_kw = gi.saba_defaults(w)
    keep = [tb["P"].cuda(), tb["C"].cuda(), tb["u"].cuda()]
    g.set_tdes_tables(keep[0], keep[1], keep[2], tb["s"])
    g.set_saba(**saba_kw)
    return g, tb, saba_kw, keep


def _target_next_from_tree(rng, tree, V, p_follow=0.75):
    """Target next-token ids per node: mostly the token of one of the node's children, so that walks get somewhere."""
    n = int(tree["n_nodes"])
    tn = rng.integers(0, V, size=tree["token"].shape[0]).astype(np.int32)
    children = {}
    for i in range(1, n):
        children.setdefault(int(tree["parent"][i]), []).append(i)
    for i in range(n):
        if i in children and rng.random() < p_follow:
            tn[i] = tree["token"][children[i][int(rng.integers(len(children[i])))]]
    return tn


@pytest.mark.parametrize("hist_w", [1, 3, 8])
def test_rounds_with_device_resident_history(hist_w):
    rounds = 7
    base = dict(batch=5, L=6, V=3000, K=6, budget_min=8, budget_max=40, budget_step=8, m=16, hidden_dim=32)
    w0 = gi.small(**base)
    g, tb, saba_kw, keep = _graft(w0)
    window = torch.zeros((w0.batch, hist_w), dtype=torch.int32, device="cuda")
    count = torch.zeros(w0.batch, dtype=torch.int32, device="cuda")
    hist_dev = torch.zeros(w0.batch, dtype=torch.float32, device="cuda")
    g.set_hist_window(hist_w, window, count, hist_dev)
    rng = np.random.default_rng(77)
    accepted = [[] for _ in range(w0.batch)]  # the oracle's record of a_t per sequence
    a_len = torch.empty(w0.batch, dtype=torch.int32, device="cuda")
    a_path = torch.empty((w0.batch, w0.L), dtype=torch.int32, device="cuda")
    bonus = torch.empty(w0.batch, dtype=torch.int32, device="cuda")
    for r in range(rounds):
        w = gi.small(**base, seed=4100 + r)  # new drafter outputs every round
        x = gi.batch_inputs(w)
        hist_orc = np.array([oracle.hist_update(a, hist_w) for a in accepted], dtype=np.float32)
        assert np.array_equal(hist_dev.cpu().numpy(), hist_orc), f"round {r}: device history differs"
        x["hist"] = torch.from_numpy(hist_orc.copy())
        out = g.alloc_out(w.batch, debug=True)
        g.build_trees(x["logits"].cuda(), x["hidden"].cuda(), x["root_token"].cuda(), hist_dev, x["prefix_len"].cuda(),
                      None, out)
        torch.cuda.synchronize()
        gpu = out.cpu()
        orc = oracle_round(oracle, w, x, tb, saba_kw)
        stats = compare_round(oracle, w, x, tb, saba_kw, gpu, orc)
        assert stats["excused_tree"] == 0 and stats["excused_budget"] == 0, stats
        tn = np.stack([_target_next_from_tree(rng, {k: orc[k][b] for k in ("n_nodes", "token", "parent")}, w.V)
                       for b in range(w.batch)])
        g.accept(out, torch.from_numpy(tn).cuda(), a_len, a_path, bonus)
        torch.cuda.synchronize()
        for b in range(w.batch):
            a, path, bo = oracle.accept(int(orc["n_nodes"][b]), orc["token"][b], orc["parent"][b], tn[b], w.L)
            assert int(a_len[b]) == a and int(bonus[b]) == bo
            accepted[b].append(a)
        assert count.cpu().tolist() == [r + 1] * w.batch
    assert max(max(a) for a in accepted) >= 2  # the walks did get somewhere
    g.set_hist_window(0)
    g.destroy()


def test_round_in_a_cuda_graph():
    """build_trees + accept captured once and replayed: the library calls allocate nothing, synchronise nothing and
    keep no per-launch host state that a replay would miss."""
    w = gi.small(batch=4, L=8, V=6000, K=8, budget_min=16, budget_max=96, budget_step=16, m=32, hidden_dim=64,
                 logits_dtype="bf16", hidden_dtype="bf16")
    g, tb, saba_kw, keep = _graft(w)
    g.set_edge_rows(min(w.L, 8))
    xs = [gi.batch_inputs(gi.small(batch=4, L=8, V=6000, K=8, budget_min=16, budget_max=96, budget_step=16, m=32,
                                   hidden_dim=64, logits_dtype="bf16", hidden_dtype="bf16", seed=900 + i))
          for i in range(2)]
    stat = {k: xs[0][k].cuda().clone() for k in ("logits", "hidden", "root_token", "hist", "prefix_len")}
    out = g.alloc_out(w.batch)
    tn = torch.zeros((w.batch, g.nmax), dtype=torch.int32, device="cuda")
    a_len = torch.empty(w.batch, dtype=torch.int32, device="cuda")
    a_path = torch.empty((w.batch, w.L), dtype=torch.int32, device="cuda")
    bonus = torch.empty(w.batch, dtype=torch.int32, device="cuda")

    def round_():
        g.build_trees(stat["logits"], stat["hidden"], stat["root_token"], stat["hist"], stat["prefix_len"], None, out)
        g.accept(out, tn, a_len, a_path, bonus)

    # eager results for both input sets
    eager = []
    for x in xs:
        for k in stat:
            stat[k].copy_(x[k].cuda())
        round_()
        torch.cuda.synchronize()
        eager.append({k: v.copy() for k, v in out.cpu().items()})
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        round_()  # warm-up on the capture stream
    torch.cuda.current_stream().wait_stream(side)
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph, stream=side):
        round_()
    for rep in range(2):
        for i, x in enumerate(xs):
            for k in stat:
                stat[k].copy_(x[k].cuda())
            graph.replay()
            torch.cuda.synchronize()
            got = out.cpu()
            for k in ("n_nodes", "budget", "status", "token", "parent", "depth", "position", "path_score", "mask"):
                assert np.array_equal(got[k], eager[i][k]), (rep, i, k)
    g.destroy()


def test_micro_batches_on_streams_of_their_own():
    """Two micro-batches, each with its own context and stream, so that one's tree building overlaps the other's
    (stub) verification: every round's results are the sequential schedule's, bit for bit, and the sequential
    schedule's first and last rounds are the oracle's."""
    from paper_2608_20375_b200.pipeline import MicroBatch, join, run_rounds

    rounds, hist_w, n_micro = 5, 3, 2
    base = dict(batch=6, L=8, V=5000, K=8, budget_min=16, budget_max=96, budget_step=16, m=32, hidden_dim=64,
                logits_dtype="bf16", hidden_dtype="bf16")
    w0 = gi.small(**base)
    keys = ("n_nodes", "budget", "status", "token", "parent", "depth", "position", "path_score", "mask", "topk_id",
            "topk_lp", "lse", "edge", "state")
    ctxs = [_graft(w0) for _ in range(n_micro)]
    tb, saba_kw = ctxs[0][1], ctxs[0][2]
    hist_bufs = []
    for g, *_ in ctxs:
        bufs = (torch.zeros((w0.batch, hist_w), dtype=torch.int32, device="cuda"),
                torch.zeros(w0.batch, dtype=torch.int32, device="cuda"),
                torch.zeros(w0.batch, dtype=torch.float32, device="cuda"))
        g.set_hist_window(hist_w, *bufs)
        hist_bufs.append(bufs)
    micro = [MicroBatch(g, w0.batch, w0.L, out=g.alloc_out(w0.batch, debug=True)) for g, *_ in ctxs]
    ws = [[gi.small(**base, seed=5200 + 10 * i + r) for r in range(rounds)] for i in range(n_micro)]
    xs = [[gi.batch_inputs(w) for w in row] for row in ws]
    dev_x = [[{k: x[k].cuda() for k in ("logits", "hidden", "root_token", "prefix_len")} for x in row] for row in xs]
    burn = torch.randn(1024, 1024, device="cuda")
    tn_dev = {}   # (i, r) -> target ids, fixed by the sequential pass
    record = {}   # schedule -> (i, r) -> outputs
    rng = np.random.default_rng(11)

    def draft(i, r):
        return dict(dev_x[i][r], hist=hist_bufs[i][2])

    def run(schedule, overlap):
        for bufs in hist_bufs:
            for t in bufs:
                t.zero_()
        record[schedule] = {}

        def verify(i, r, out):
            y = burn
            for _ in range(4):  # stands in for the target model's forward pass on this stream
                y = torch.mm(y, burn) * 1e-3
            if (i, r) not in tn_dev:  # sequential pass only: choose the target ids from the tree just built
                torch.cuda.current_stream().synchronize()
                t = out.cpu()
                tn = np.stack([_target_next_from_tree(rng, {k: t[k][b] for k in ("n_nodes", "token", "parent")},
                                                      w0.V) for b in range(w0.batch)])
                tn_dev[(i, r)] = torch.from_numpy(tn).cuda()
            return tn_dev[(i, r)]

        def after(i, r, mb):
            snap = {k: getattr(mb.out, k).clone() for k in keys}
            snap["accept_len"] = mb.accept_len.clone()
            snap["hist"] = hist_bufs[i][2].clone()
            record[schedule][(i, r)] = snap

        run_rounds(micro, rounds, draft, verify, overlap=overlap, after_round=after)
        join(micro)
        torch.cuda.synchronize()

    run("sequential", False)
    run("overlapped", True)
    for key, snap in record["sequential"].items():
        for k, v in snap.items():
            assert torch.equal(v, record["overlapped"][key][k]), (key, k)
    assert max(int(s["accept_len"].max()) for s in record["sequential"].values()) >= 2
    # the sequential schedule against the oracle: the first round (no history yet) and the last (hist from the device)
    for i in range(n_micro):
        for r in (0, rounds - 1):
            snap = record["sequential"][(i, r)]
            x = dict(xs[i][r])
            prev = record["sequential"][(i, r - 1)]["hist"] if r > 0 else torch.zeros(w0.batch)
            x["hist"] = prev.cpu().float()
            orc = oracle_round(oracle, ws[i][r], x, tb, saba_kw)
            gpu = {k: snap[k].cpu().numpy() for k in keys}
            gpu["mask"] = gpu["mask"].view("uint32")
            stats = compare_round(oracle, ws[i][r], x, tb, saba_kw, gpu, orc)
            assert stats["excused_tree"] == 0 and stats["excused_budget"] == 0, stats
    for g, *_ in ctxs:
        g.set_hist_window(0)
        g.destroy()

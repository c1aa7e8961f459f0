"""Guard words around every output buffer: nothing may be written outside the bytes a call owns.

Every output of graft_build_trees, graft_accept, graft_vocab_pass, graft_vocab_pass_static, graft_vocab_pass_partial,
graft_vocab_merge and graft_tdes_edges is a view into the middle of a larger device buffer filled with a sentinel
byte; after the call the bytes before and after the view must still be the sentinel.  Shapes are deliberately odd
(odd V, K = 27, the largest node table, batches that are multiples of nothing) so that every ragged path runs.  This
host-side check stands in for a memory checker on the device.
"""
import numpy as np
import pytest
import torch

import graft_inputs as gi

pytestmark = pytest.mark.gpu

GUARD = 4096      # bytes before and after every output
SENTINEL = 0xA5
DT = {"f32": 0, "bf16": 1}


class Guarded:
    """Output tensors carved out of sentinel-filled buffers."""

    def __init__(self):
        self.items = []

    def new(self, shape, dtype):
        n = int(np.prod(shape)) * torch.empty((), dtype=dtype).element_size()
        raw = torch.full((n + 2 * GUARD,), SENTINEL, dtype=torch.uint8, device="cuda")
        view = raw[GUARD:GUARD + n].view(dtype).view(shape)
        self.items.append((raw, n))
        return view

    def check(self, what):
        torch.cuda.synchronize()
        for i, (raw, n) in enumerate(self.items):
            head, tail = raw[:GUARD], raw[GUARD + n:]
            assert bool((head == SENTINEL).all()), f"{what}: bytes before output {i} were overwritten"
            assert bool((tail == SENTINEL).all()), f"{what}: bytes after output {i} were overwritten"


def _graft(w):
    from paper_2608_20375_b200 import Graft
    return Graft(w.V, w.L, w.K, w.m, w.hidden_dim, w.batch, w.budget_min, w.budget_max, w.budget_step, w.beta, 1,
                 DT[w.logits_dtype], DT[w.hidden_dtype])


CASES = [
    dict(batch=7, L=5, V=4099, K=27, budget_min=1, budget_max=1023, budget_step=73, m=20, hidden_dim=33,
         logits_dtype="bf16", hidden_dtype="bf16"),                       # the largest node table, odd everything
    dict(batch=3, L=16, V=30011, K=32, budget_min=16, budget_max=512, budget_step=16, m=128, hidden_dim=256,
         logits_dtype="bf16", hidden_dtype="f32"),
    dict(batch=5, L=3, V=97, K=13, budget_min=4, budget_max=40, budget_step=3, m=4, hidden_dim=1),
    dict(batch=1, L=32, V=1001, K=1, budget_min=32, budget_max=32, budget_step=1, fixed_budget=32, m=8, hidden_dim=7),
]


@pytest.mark.parametrize("kw", CASES)
@pytest.mark.parametrize("debug", [True, False])
def test_round_and_walk_write_only_their_outputs(kw, debug):
    from paper_2608_20375_b200.binding import TreeOut
    w = gi.small(**kw)
    g = _graft(w)
    tb = gi.tdes_tables(w)
    keep = [tb["P"].cuda(), tb["C"].cuda(), tb["u"].cuda()]
    g.set_tdes_tables(keep[0], keep[1], keep[2], tb["s"])
    g.set_saba(**gi.saba_defaults(w))
    x = gi.batch_inputs(w)
    cu = lambda t: None if t is None else t.cuda()  # noqa: E731
    B, N, W, L, K = w.batch, g.nmax, g.mask_words, w.L, w.K
    i32, f32 = torch.int32, torch.float32
    gd = Guarded()
    out = TreeOut(gd.new((B,), i32), gd.new((B,), i32), gd.new((B, N), i32), gd.new((B, N), i32), gd.new((B, N), i32),
                  gd.new((B, N), i32), gd.new((B, N), f32), gd.new((B, N, W), i32), gd.new((B,), i32))
    if debug:
        out.topk_id, out.topk_lp = gd.new((B, L, K), i32), gd.new((B, L, K), f32)
        out.lse, out.edge, out.state = gd.new((B, L), f32), gd.new((B, L, K, K), f32), gd.new((B, 4), f32)
    g.build_trees(cu(x["logits"]), cu(x["hidden"]), cu(x["root_token"]), cu(x["hist"]), cu(x["prefix_len"]),
                  cu(x["fixed_budget"]), out)
    gd.check("graft_build_trees")
    depth = out.depth.cpu().numpy()
    tn = np.stack([gi.target_next_from_depth(gi.target_tokens(w, b), depth[b]) for b in range(B)])
    a_len, a_path, bonus = gd.new((B,), i32), gd.new((B, L), i32), gd.new((B,), i32)
    g.accept(out, torch.from_numpy(tn).cuda(), a_len, a_path, bonus)
    gd.check("graft_accept")
    assert int(out.n_nodes.min()) >= 1 and int(a_len.max()) <= L  # (the outputs themselves were written)
    g.destroy()


@pytest.mark.parametrize("V,K,L,Bt,dtype", [(4099, 27, 3, 5, "bf16"), (151937, 32, 2, 3, "bf16"), (32001, 8, 7, 1, "f32"),
                                           (33, 27, 2, 2, "bf16")])
def test_vocab_pass_entry_points_write_only_their_outputs(V, K, L, Bt, dtype):
    from paper_2608_20375_b200 import Graft, VOCAB_PARTIAL_BYTES, vocab_pass_static, vocab_range
    tdt = torch.bfloat16 if dtype == "bf16" else torch.float32
    z = (2.0 * torch.randn((Bt, L, V), generator=torch.Generator().manual_seed(V))).to(tdt).cuda()
    i32, f32 = torch.int32, torch.float32
    g = Graft(V, L, K, 16, 8, Bt, 8, 8, 8, 0.0, 1, DT[dtype], 0)
    for name, call in (("graft_vocab_pass", lambda o: g.vocab_pass(z, *o)),
                       ("graft_vocab_pass_static", lambda o: vocab_pass_static(z, K, *o))):
        gd = Guarded()
        o = (gd.new((Bt, L, K), i32), gd.new((Bt, L, K), f32), gd.new((Bt, L), f32), gd.new((Bt, L), i32))
        call(o)
        gd.check(name)
        assert int(o[0].min()) >= 0 and int(o[0].max()) < V
    # two shards, their pieces, the merge
    gd = Guarded()
    parts = gd.new((2, Bt * L, VOCAB_PARTIAL_BYTES), torch.uint8)
    offs, keep = [], []
    for r in range(2):
        lo, hi = vocab_range(V, r, 2)
        offs.append(lo)
        gs = Graft(hi - lo, L, min(K, hi - lo), 16, 8, Bt, 8, 8, 8, 0.0, 1, DT[dtype], 0)
        gs.vocab_pass_partial(z[:, :, lo:hi].contiguous(), parts[r])
        keep.append(gs)
    gd.check("graft_vocab_pass_partial")
    o = (gd.new((Bt, L, K), i32), gd.new((Bt, L, K), f32), gd.new((Bt, L), f32), gd.new((Bt, L), i32))
    g.vocab_merge(parts, offs, *o)
    gd.check("graft_vocab_merge")
    assert int(o[0].min()) >= 0 and int(o[0].max()) < V
    for gs in keep + [g]:
        gs.destroy()


def test_edge_scores_write_only_their_output():
    w = gi.small(batch=3, L=5, V=3001, K=27, m=36, beta=0.4)
    g = _graft(w)
    tb = gi.tdes_tables(w)
    keep = [tb["P"].cuda(), tb["C"].cuda(), tb["u"].cuda()]
    g.set_tdes_tables(keep[0], keep[1], keep[2], tb["s"])
    gen = torch.Generator().manual_seed(3)
    ids = torch.stack([torch.randperm(w.V, generator=gen)[:w.K] for _ in range(w.batch * w.L)]).view(w.batch, w.L, w.K)
    lp = -torch.rand((w.batch, w.L, w.K), generator=gen).cumsum(-1)
    gd = Guarded()
    edge = gd.new((w.batch, w.L, w.K, w.K), torch.float32)
    g.tdes_edges(ids.to(torch.int32).cuda(), lp.cuda(), torch.zeros(w.batch, dtype=torch.int32).cuda(), edge)
    gd.check("graft_tdes_edges")
    assert bool(torch.isfinite(edge[:, 1:]).all())
    g.destroy()

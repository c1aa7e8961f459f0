"""GPU parity: the CUDA library (through its C ABI) against the CPU oracle on the same seeded inputs."""
import numpy as np
import pytest
import torch

import graft_inputs as gi
import oracle
from helpers import (EPS, check_tree_invariants, compare_accept, compare_round, gpu_round, oracle_round,
                     tolerance)

pytestmark = pytest.mark.gpu

DT = {"f32": 0, "bf16": 1}


def _graft(w, max_batch=None, beta=None, root_edge=1):
    from paper_2608_20375_b200 import Graft
    g = Graft(w.V, w.L, w.K, w.m, w.hidden_dim, max_batch or w.batch, w.budget_min, w.budget_max, w.budget_step,
              w.beta if beta is None else beta, root_edge, DT[w.logits_dtype], DT[w.hidden_dtype])
    return g


def _setup(w, g):
    tb = gi.tdes_tables(w)
    saba_kw = gi.saba_defaults(w)
    keep = [tb["P"].cuda(), tb["C"].cuda(), tb["u"].cuda()]
    g.set_tdes_tables(keep[0], keep[1], keep[2], tb["s"])
    g.set_saba(**saba_kw)
    return tb, saba_kw, keep


# --------------------------------------------------------------------------- vocab pass
def _vocab_case(z, K, dtype):
    """z: [batch, L, V] CPU tensor in its dtype."""
    from paper_2608_20375_b200 import Graft
    Bt, L, V = z.shape
    g = Graft(V, L, K, 16, 8, Bt, 8, 8, 8, 0.0, 1, DT[dtype], 0)
    ids = torch.empty((Bt, L, K), dtype=torch.int32, device="cuda")
    lp = torch.empty((Bt, L, K), dtype=torch.float32, device="cuda")
    lse = torch.empty((Bt, L), dtype=torch.float32, device="cuda")
    rs = torch.empty((Bt, L), dtype=torch.int32, device="cuda")
    g.vocab_pass(z.cuda(), ids, lp, lse, rs)
    torch.cuda.synchronize()
    o_ids, o_lp, o_lse, o_st = oracle.vocab_pass(z.reshape(Bt * L, V), K)
    ids, lp, lse, rs = (t.cpu().numpy().reshape(Bt * L, -1) for t in (ids, lp, lse, rs))
    assert np.array_equal(rs[:, 0], o_st)
    good = o_st == 0
    assert np.array_equal(ids[good], o_ids[good])
    a, b = lp[good].astype(np.float64), o_lp[good].astype(np.float64)
    fin = np.isfinite(b)
    assert np.array_equal(np.isneginf(a), np.isneginf(b))
    # (an fp32 result cannot be closer than its own spacing: one ulp beyond |x| = 128 already exceeds EPS)
    assert np.all(np.abs(a[fin] - b[fin]) <= tolerance(b[fin]))
    # candidates come in rank order, so their log-probabilities never increase along a row, and equal logits get the
    # same bits (every candidate of a row is measured against one log-sum-exp)
    assert np.all(a[:, 1:] <= a[:, :-1]), "log-probabilities increase along a row"
    zf = z.reshape(Bt * L, V).float().numpy()
    for r in np.nonzero(good)[0][:64]:
        vals = zf[r, ids[r]]
        same = vals[1:] == vals[:-1]
        assert np.array_equal(lp[r, 1:][same], lp[r, :-1][same]), f"row {r}: equal logits, different log-probabilities"
    # lse is returned as an fp32 number: allow its own rounding on top of EPS
    assert np.all(np.abs(lse[good, 0] - o_lse[good]) <= tolerance(o_lse[good]))
    g.destroy()
    return float(np.abs(lse[good, 0] - o_lse[good]).max(initial=0))


@pytest.mark.parametrize("V,K,L,Bt,dtype", [
    (32000, 8, 16, 1, "f32"),      # rows split over many CTAs
    (4099, 32, 3, 5, "bf16"),      # odd V: rows start at 2-byte offsets
    (4097, 16, 4, 3, "f32"),       # odd V in fp32
    (33, 32, 2, 2, "bf16"),        # K almost V, everything through the ragged path
    (8, 8, 1, 1, "f32"),           # K == V
    (151936, 32, 2, 3, "bf16"),    # several tiles and a ragged tail per row
    (20000, 16, 16, 40, "bf16"),   # many rows per CTA
    (70001, 5, 1, 1, "bf16"),      # one row shared by every CTA
])
def test_vocab_pass_shapes(V, K, L, Bt, dtype):
    g = torch.Generator().manual_seed(V + K)
    z = 2.0 * torch.randn((Bt, L, V), generator=g)
    z[:, :, : min(V, 7)] += 6.0
    z = z.to(torch.bfloat16) if dtype == "bf16" else z
    _vocab_case(z, K, dtype)


def test_vocab_pass_ties_uniform_masked_and_bad_rows():
    V, K = 9000, 32
    g = torch.Generator().manual_seed(1)
    z = torch.round(2.0 * torch.randn((1, 8, V), generator=g) * 2) / 2  # heavy ties
    z[0, 1] = 1.25                        # all equal: ids 0..K-1
    z[0, 2, 100:] = float("-inf")         # masked vocabulary
    z[0, 3, 5] = float("nan")
    z[0, 4, 77] = float("inf")
    z[0, 5] = float("-inf")
    z[0, 6] = torch.arange(V, dtype=torch.float32) * 1e-3   # ascending: every element a new maximum
    z[0, 7] = -torch.arange(V, dtype=torch.float32) * 1e-3  # descending
    _vocab_case(z, K, "f32")
    _vocab_case(z.to(torch.bfloat16), K, "bf16")


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
def test_vocab_pass_full_width_rows_with_bulk_ties(dtype):
    """Rows of the full vocabulary width, cut across CTAs, in which almost every element ties with the K-th largest:
    the candidate filter lets everything through, so the exact selection over the whole segment takes over, and the
    ids alone decide across the pieces of a row."""
    V, K, L = 151936, 32, 8
    g = torch.Generator().manual_seed(9)
    z = torch.zeros((2, L, V))
    z[0, 0] = 1.25                                                    # all equal
    z[0, 1] = torch.round(torch.randn(V, generator=g))                # seven or so distinct values
    z[0, 2] = -(torch.arange(V) // 4096).float()                      # descending plateaus of 4096
    z[0, 3] = (torch.arange(V) // 4096).float()                       # ascending plateaus: the best sit at the end
    z[0, 4, :] = float("-inf")
    z[0, 4, V - 40:] = 3.0                                            # forty finite elements at the very end
    z[0, 5, ::2] = 1.0                                                # alternating
    z[0, 6] = torch.randn(V, generator=g)
    z[0, 6, 1000:1000 + K + 5] = 9.0                                  # K + 5 tied winners inside one piece
    z[0, 7] = torch.randn(V, generator=g)
    z[0, 7, torch.arange(0, V, V // 40)] = 9.0                        # forty tied winners spread over every piece
    z[1] = z[0].flip(0)
    _vocab_case(z.to(torch.bfloat16) if dtype == "bf16" else z, K, dtype)


@pytest.mark.parametrize("V", [151936, 40003])
@pytest.mark.parametrize("dtype", ["bf16", "f32"])
def test_vocab_pass_bulk_ties_beside_larger_values(V, dtype):
    """Thousands of elements tie with the K-th largest value while a few lie above it: the top-K are the larger
    ones, wherever they are, then the tied ones of smallest id -- also when tied elements share a chunk with a larger
    one, when only one tied element is wanted, when the tied value is negative, and when the tied elements do not
    start at the front of the row."""
    K, L = 32, 8
    g = torch.Generator().manual_seed(V)
    z = torch.zeros((2, L, V))
    z[0, 0, torch.randint(0, V, (5,), generator=g)] = 4.0            # five winners anywhere, the rest ties at 0
    z[0, 1, 5000] = 5.0                                               # a winner whose chunk is otherwise ties
    z[0, 1, 17] = 2.5                                                 # ... and one among the first tied elements
    idx = torch.randperm(V, generator=g)[:K - 1]
    z[0, 2, idx] = 1.0 + torch.arange(K - 1).float() / 64             # K - 1 distinct winners: one tied element wanted
    z[0, 3] = -7.5                                                    # ties at a negative value
    z[0, 3, V - 3] = -7.0
    z[0, 4, :3000] = -1.0 - torch.rand(3000, generator=g)             # the tied elements start behind 3000 lower ones
    z[0, 4, V // 2] = 2.0
    z[0, 5, torch.arange(0, V, 997)] = 3.0                            # more than K winners above the ties
    z[0, 6, :10] = torch.arange(10).float()                           # winners and ties together at the front
    z[0, 7] = torch.where(torch.rand(V, generator=g) < 0.5, 0.0, -0.5)  # two values, half each
    z[0, 7, V - 1] = 0.25
    z[1] = z[0].flip(0)
    _vocab_case(z.to(torch.bfloat16) if dtype == "bf16" else z, K, dtype)
    # rows of +0 and -0 (one value, two bit patterns) under one winner: the tied elements are the first of either
    zs = torch.zeros((1, L, V))
    zs[0, :, 1::2] = -0.0
    zs[0, :, 700] = 1.0
    _vocab_case(zs.to(torch.bfloat16) if dtype == "bf16" else zs, K, dtype)


@pytest.mark.parametrize("V,dtype", [(151936, "bf16"), (40003, "bf16"), (40003, "f32")])
def test_vocab_pass_sorted_rows(V, dtype):
    """Rows in ascending and descending order (distinct values, values that tie in blocks after rounding to bf16, a
    sorted half beside an ordinary one): the large elements sit side by side, so every chunk that reaches the filter's
    threshold is full of candidates and the selection runs through the exact path with its rising filter."""
    K, L = 32, 8
    g = torch.Generator().manual_seed(V + 1)
    srt = torch.sort(2.0 * torch.randn(V, generator=g)).values
    ar = torch.arange(V, dtype=torch.float32)
    z = torch.empty((2, L, V))
    z[0, 0] = srt
    z[0, 1] = srt.flip(0)
    z[0, 2] = ar * 1e-3
    z[0, 3] = -ar * 1e-3
    z[0, 4] = ar
    z[0, 5] = -ar * 0.1
    z[0, 6] = torch.cat([2.0 * torch.randn(V // 2, generator=g), srt[V // 2:] - 1.0])
    z[0, 7] = torch.roll(srt, V // 3)
    z[1] = z[0].flip(0)
    _vocab_case(z.to(torch.bfloat16) if dtype == "bf16" else z, K, dtype)


@pytest.mark.parametrize("V,dtype", [(151936, "bf16"), (40003, "bf16"), (151936, "f32")])
def test_vocab_pass_rows_of_ramps(V, dtype):
    """Rows made of ramps as long as a chunk, a streaming warp's block, a tile, or three quanta of the partition, rising
    or falling: patterns in step with the kernel's lanes, for which the maxima of its 64 groups of threads bound the
    K-th largest element poorly (more chunks reach that bound than the hit list holds) and the bound is taken from the
    chunk maxima instead."""
    K, L = 32, 8
    ar = torch.arange(V, dtype=torch.float32)
    z = torch.empty((2, L, V))
    for j, per in enumerate((32, 1024, 16384, 6144)):
        z[0, 2 * j] = (ar % per) / per * 8 + ar * 1e-6
        z[0, 2 * j + 1] = -(ar % per) / per * 8
    z[1] = z[0].flip(0).roll(515, 1)
    _vocab_case(z.to(torch.bfloat16) if dtype == "bf16" else z, K, dtype)


@pytest.mark.parametrize("V,dtype", [(151936, "bf16"), (40003, "bf16"), (151936, "f32")])
def test_vocab_pass_sparse_ties(V, dtype):
    """Hundreds of elements tie with the K-th largest value, one in every 256 or 4096 elements, over a lower random
    rest: the tied elements of smallest id are wanted, and they are chunks apart -- at a positive and at a negative
    value, alone, under a few larger elements, and starting far into the row."""
    K, L = 32, 8
    g = torch.Generator().manual_seed(V + 7)
    z = -2.0 - 6.0 * torch.rand((2, L, V), generator=g)
    z[0, 0, ::256] = 1.5
    z[0, 1, ::256] = -1.5
    z[0, 2, 5::4096] = 0.25
    z[0, 2, torch.randint(0, V, (7,), generator=g)] = 3.0
    z[0, 3, 5::4096] = -0.75
    z[0, 3, torch.randint(0, V, (40,), generator=g)] = 3.0   # more winners than K: no tied element is wanted
    z[0, 4, V // 2::256] = 1.0                                # the ties start half-way into the row
    z[0, 5, 3::256] = -1.0
    z[0, 5, 3 + 256 * 9] = -0.5                               # a winner in the place of a tied element
    z[0, 6, ::33] = 0.0                                       # a tie in every chunk but not at a fixed lane
    z[0, 7, 31::32] = -1.25                                   # the last element of every chunk
    z[1] = z[0].flip(0).roll(771, 1)
    _vocab_case(z.to(torch.bfloat16) if dtype == "bf16" else z, K, dtype)


def test_vocab_pass_whole_row_segments_of_rows_that_defeat_the_filter():
    """At the benchmark's width and batch (64 x 16 rows of 151,936 bf16 logits) a CTA's segments are whole rows of ten
    tiles: there the hit list overflows on rows of ramps and on sparse ties (hundreds of chunks reach the bound), the
    bound is taken from the chunk maxima, the tie walk follows the chunk maxima, and sorted rows fill the key buffer.
    Sixteen such shapes, rolled differently for every sequence; sampled rows against the oracle."""
    from paper_2608_20375_b200 import Graft
    V, K, L, Bt = 151936, 32, 16, 64
    g = torch.Generator().manual_seed(77)
    ar = torch.arange(V, dtype=torch.float32)
    low = lambda: -2.0 - 6.0 * torch.rand(V, generator=g)
    srt = torch.sort(2.0 * torch.randn(V, generator=g)).values
    pats = []
    for per in (256, 1024, 6144, 16384):
        pats.append((ar % per) / per * 8)
        pats.append(-(ar % per) / per * 8)
    x = low(); x[::256] = 1.5; pats.append(x)                         # sparse ties, positive
    x = low(); x[::256] = -1.5; pats.append(x)                        # ... negative
    x = low(); x[5::4096] = 0.25; x[torch.randint(0, V, (7,), generator=g)] = 3.0; pats.append(x)
    x = low(); x[V // 2::256] = 1.0; pats.append(x)                   # the ties start half-way into the row
    pats.append(srt)
    pats.append(srt.flip(0))
    # (the rest in [-8, -1] rounds to bf16 -1.0 at its top: most group maxima tie there, below the sparse winners)
    x = -1.0 - 7.0 * torch.rand(V, generator=g); x[::256] = 0.0; pats.append(x)
    x = 2.0 * torch.randn(V, generator=g); x[20000:25000] = 20.0 + torch.sort(torch.randn(5000, generator=g)).values
    pats.append(x)
    assert len(pats) == L
    row = torch.stack(pats).to(torch.bfloat16)
    z = torch.stack([torch.roll(row, 37 * b * (b % 3), 1) for b in range(Bt)])      # [Bt, L, V]
    gr = Graft(V, L, K, 16, 8, Bt, 8, 8, 8, 0.0, 1, DT["bf16"], 0)
    ids = torch.empty((Bt, L, K), dtype=torch.int32, device="cuda")
    lp = torch.empty((Bt, L, K), dtype=torch.float32, device="cuda")
    lse = torch.empty((Bt, L), dtype=torch.float32, device="cuda")
    rs = torch.empty((Bt, L), dtype=torch.int32, device="cuda")
    gr.vocab_pass(z.cuda(), ids, lp, lse, rs)
    torch.cuda.synchronize()
    gr.destroy()
    sample = [b * L + d for b in (0, 1, 2, 7, 30, 63) for d in range(L)]
    o_ids, o_lp, o_lse, o_st = oracle.vocab_pass(z.reshape(Bt * L, V)[sample], K)
    ids, lp, lse, rs = (t.cpu().numpy().reshape(Bt * L, -1)[sample] for t in (ids, lp, lse, rs))
    assert np.array_equal(rs[:, 0], o_st) and not o_st.any()
    assert np.array_equal(ids, o_ids)
    assert np.all(np.abs(lp.astype(np.float64) - o_lp) <= tolerance(o_lp))
    assert np.all(np.abs(lse[:, 0] - o_lse) <= tolerance(o_lse))


@pytest.mark.parametrize("seed,dtype", [(0, "bf16"), (1, "f32"), (2, "bf16"), (3, "bf16")])
def test_vocab_pass_compositions_of_rows_that_defeat_the_filter(seed, dtype):
    """Random compositions of `graft_inputs.adversarial_rows` at the benchmark's batch and width (whole-row segments):
    a row as it is, reversed, negated, scaled, spliced with another, or with a few winners planted on top; every
    sequence rolled by its own offset; 96 sampled rows against the oracle."""
    from paper_2608_20375_b200 import Graft
    V, K, L, Bt = 151936, 32, 16, 64
    g0 = torch.Generator().manual_seed(1000 + seed)
    rng = np.random.default_rng(seed)
    pool = gi.adversarial_rows(V, g0)
    pats = []
    for d in range(L):
        r = pool[int(rng.integers(len(pool)))][1].clone()
        op = int(rng.integers(6))
        if op == 1:
            r = r.flip(0)
        elif op == 2:
            r = -r
        elif op == 3:
            cut = int(rng.integers(1, V - 1))
            r[cut:] = pool[int(rng.integers(len(pool)))][1][cut:]
        elif op == 4:
            r = r * float(rng.choice([0.1, 3.0, 17.0]))
        elif op == 5:
            r[torch.randint(0, V, (int(rng.integers(1, 60)),), generator=g0)] = r[torch.isfinite(r)].max() + 1.0
        pats.append(torch.nan_to_num(r, nan=0.0, posinf=1e4))
    row = torch.stack(pats).to(torch.bfloat16 if dtype == "bf16" else torch.float32)
    z = torch.stack([torch.roll(row, int(rng.integers(V)), 1) for b in range(Bt)])
    gr = Graft(V, L, K, 16, 8, Bt, 8, 8, 8, 0.0, 1, DT[dtype], 0)
    ids = torch.empty((Bt, L, K), dtype=torch.int32, device="cuda")
    lp = torch.empty((Bt, L, K), dtype=torch.float32, device="cuda")
    lse = torch.empty((Bt, L), dtype=torch.float32, device="cuda")
    rs = torch.empty((Bt, L), dtype=torch.int32, device="cuda")
    gr.vocab_pass(z.cuda(), ids, lp, lse, rs)
    torch.cuda.synchronize()
    gr.destroy()
    sample = sorted(set(int(x) for x in rng.integers(0, Bt * L, 96)))
    o_ids, o_lp, o_lse, o_st = oracle.vocab_pass(z.reshape(Bt * L, V)[sample], K)
    ids, lp, lse, rs = (t.cpu().numpy().reshape(Bt * L, -1)[sample] for t in (ids, lp, lse, rs))
    assert np.array_equal(rs[:, 0], o_st)
    good = o_st == 0
    assert good.any() and np.array_equal(ids[good], o_ids[good])
    a, b = lp[good].astype(np.float64), o_lp[good]
    fin = np.isfinite(b)
    assert np.array_equal(np.isneginf(a), np.isneginf(b))
    assert np.all(np.abs(a[fin] - b[fin]) <= tolerance(b[fin]))
    assert np.all(np.abs(lse[good, 0] - o_lse[good]) <= tolerance(o_lse[good]))


@pytest.mark.parametrize("V,dtype", [(3, "bf16"), (6, "f32"), (14, "bf16"), (4099, "bf16"), (4097, "f32")])
def test_vocab_pass_dominant_logit_outside_the_bulk_copies(V, dtype):
    """One logit 30 above the rest, placed where the 16-byte bulk copies do not reach (tiny rows, the ragged first
    and last elements of odd-length rows): the log-probability of that token is a rounding error away from 0, and
    a path of 32 such tokens must stay within the tolerance of 1e-5, so each must be within about 1e-7."""
    from paper_2608_20375_b200 import Graft
    L, K = 8, min(V, 4)
    z = torch.zeros((2, L, V))
    for j in range(L):
        z[0, j, (0, V - 1, 1, V - 2)[j % 4]] = 30.0 + j
        z[1, j, (V - 1, 0)[j % 2]] = 30.0
    zz = z.to(torch.bfloat16) if dtype == "bf16" else z
    _vocab_case(zz, K, dtype)
    g = Graft(V, L, K, 16, 8, 2, 8, 8, 8, 0.0, 1, DT[dtype], 0)
    ids = torch.empty((2, L, K), dtype=torch.int32, device="cuda")
    lp = torch.empty((2, L, K), dtype=torch.float32, device="cuda")
    lse = torch.empty((2, L), dtype=torch.float32, device="cuda")
    g.vocab_pass(zz.cuda(), ids, lp, lse)
    torch.cuda.synchronize()
    o_ids, o_lp, o_lse, o_st = oracle.vocab_pass(zz.reshape(2 * L, V), K)
    top = lp.cpu().numpy().reshape(2 * L, K)[:, 0].astype(np.float64)
    assert np.abs(top - o_lp[:, 0]).max() <= 1.5e-7, (top, o_lp[:, 0])  # 32 of them stay within 1e-5
    g.destroy()


def test_vocab_pass_large_magnitudes_and_negative_zero():
    V, K = 5000, 8
    g = torch.Generator().manual_seed(2)
    z = 30.0 * torch.randn((1, 4, V), generator=g)
    z[0, 0] += 500.0
    z[0, 1] -= 500.0
    z[0, 2, ::2] = 0.0
    z[0, 2, 1::2] = -0.0
    z[0, 3] *= 1e-3
    _vocab_case(z, K, "f32")
    _vocab_case(z.to(torch.bfloat16), K, "bf16")


def test_vocab_pass_is_reproducible_and_counters_reset():
    w = gi.small(batch=3, L=4, V=50000, K=16, logits_dtype="bf16")
    x = gi.batch_inputs(w)
    g = _graft(w, beta=0.0)
    z = x["logits"].cuda()
    outs = []
    for _ in range(3):
        ids = torch.empty((3, 4, 16), dtype=torch.int32, device="cuda")
        lp = torch.empty((3, 4, 16), dtype=torch.float32, device="cuda")
        lse = torch.empty((3, 4), dtype=torch.float32, device="cuda")
        g.vocab_pass(z, ids, lp, lse)
        torch.cuda.synchronize()
        outs.append((ids.cpu(), lp.cpu(), lse.cpu()))
    for o in outs[1:]:
        assert torch.equal(o[0], outs[0][0])
        assert torch.equal(o[1], outs[0][1])


# --------------------------------------------------------------------------- TDES
@pytest.mark.parametrize("V,E,m,emb_dtype", [
    (777, 200, 24, "bf16"),     # tensor-core path, ragged in every dimension
    (4099, 512, 128, "bf16"),   # tensor-core path, several tiles
    (300, 64, 4, "bf16"),       # tensor-core path, the narrowest scorer
    (500, 100, 16, "bf16"),     # E not a multiple of 8: the FMA kernel
    (777, 200, 24, "f32"),      # fp32 embeddings: the FMA kernel
    (70001, 2048, 8, "bf16"),   # tensor-core path at the sizes it runs at: two slabs of rows, two chunks along E
    (66000, 1096, 24, "bf16"),  # a second slab of 464 rows and a last chunk of 72 columns
])
def test_tdes_precompute_against_oracle(V, E, m, emb_dtype):
    L = 4
    wts = gi.tdes_weights(V, E, m, L, seed=5, emb_dtype=emb_dtype)
    w = gi.small(V=V, m=m, L=L)
    g = _graft(w)
    out = torch.empty((V, m), dtype=torch.float32, device="cuda")
    for Wk, bk in (("Wp", "bp"), ("Wc", None)):
        g.tdes_precompute(wts["emb"].cuda(), wts[Wk].cuda(), None if bk is None else wts[bk].cuda(), out)
        torch.cuda.synchronize()
        want = oracle.tdes_tables(wts["emb"], wts[Wk].numpy(), None if bk is None else wts[bk].numpy())
        np.testing.assert_allclose(out.cpu().numpy(), want, rtol=1e-5, atol=1e-5)
    g.destroy()


@pytest.mark.parametrize("K,L,m,beta,root_edge", [(4, 4, 16, 0.2, 1), (32, 16, 128, 0.2, 1), (7, 3, 36, 0.7, 0),
                                                   (16, 5, 128, 0.0, 1)])
def test_tdes_edges_against_oracle(K, L, m, beta, root_edge):
    V, Bt = 3000, 3
    w = gi.small(batch=Bt, V=V, K=K, L=L, m=m, beta=beta)
    g = _graft(w, root_edge=root_edge)
    tb, _, keep = _setup(w, g)
    x = gi.batch_inputs(w)
    ids, lp, _, _ = oracle.vocab_pass(x["logits"].reshape(Bt * L, V), K)
    ids, lp = ids.reshape(Bt, L, K), lp.reshape(Bt, L, K)
    edge = torch.empty((Bt, L, K, K), dtype=torch.float32, device="cuda")
    g.tdes_edges(torch.from_numpy(ids).cuda(), torch.from_numpy(lp).cuda(), x["root_token"].cuda(), edge)
    torch.cuda.synchronize()
    edge = edge.cpu().numpy()
    for b in range(Bt):
        want = oracle.tdes_edges(ids[b], lp[b], int(x["root_token"][b]), tb["P"].numpy(), tb["C"].numpy(),
                                 tb["u"].numpy(), tb["s"], beta, root_edge)
        assert np.abs(edge[b] - want).max() <= EPS
        if beta == 0.0:
            assert np.array_equal(edge[b], want)  # the DDTree score, bit for bit


# --------------------------------------------------------------------------- vocabulary-parallel vocab pass
@pytest.mark.parametrize("V,K,L,Bt,dtype,world", [
    (50000, 16, 4, 3, "bf16", 2), (151936, 32, 2, 2, "bf16", 4), (32000, 8, 3, 2, "f32", 3), (9000, 32, 2, 2, "bf16", 8),
    (70, 16, 2, 2, "f32", 5),  # shards narrower than K
])
def test_vocab_pass_parallel_matches_the_full_row_oracle(V, K, L, Bt, dtype, world):
    """The ranks of a vocabulary-parallel run, emulated one after the other on this device: every shard's pieces,
    then the merge, against the oracle on the full rows."""
    from paper_2608_20375_b200 import Graft, VOCAB_PARTIAL_BYTES, vocab_range
    w = gi.small(batch=Bt, L=L, V=V, K=K, logits_dtype=dtype)
    z = gi.batch_inputs(w)["logits"]
    z[0, 0, 5] = z[0, 0, V - 3] = z[0, 0, 7]  # equal values in different shards: ids decide
    z[1, 1, ::2] = float("-inf")             # masked tokens
    rows = Bt * L
    parts, offs, keep = [], [], []
    for r in range(world):
        lo, hi = vocab_range(V, r, world)
        offs.append(lo)
        gs = Graft(hi - lo, L, min(K, hi - lo), 16, 8, Bt, 8, 8, 8, 0.0, 1, DT[dtype], 0)  # a narrow shard keeps all it has
        p = torch.empty((rows, VOCAB_PARTIAL_BYTES), dtype=torch.uint8, device="cuda")
        gs.vocab_pass_partial(z[:, :, lo:hi].contiguous().cuda(), p)
        parts.append(p)
        keep.append(gs)
    allp = torch.stack(parts).contiguous()
    ids = torch.empty((Bt, L, K), dtype=torch.int32, device="cuda")
    lp = torch.empty((Bt, L, K), dtype=torch.float32, device="cuda")
    lse = torch.empty((Bt, L), dtype=torch.float32, device="cuda")
    rs = torch.empty((Bt, L), dtype=torch.int32, device="cuda")
    gm = Graft(V, L, K, 16, 8, Bt, 8, 8, 8, 0.0, 1, DT[dtype], 0)  # the merge uses K and L of its context
    keep.append(gm)
    gm.vocab_merge(allp, offs, ids, lp, lse, rs)
    torch.cuda.synchronize()
    o_ids, o_lp, o_lse, o_st = oracle.vocab_pass(z.reshape(rows, V), K)
    ids, lp, lse, rs = (t.cpu().numpy().reshape(rows, -1) for t in (ids, lp, lse, rs))
    assert np.array_equal(rs[:, 0], o_st)
    good = o_st == 0
    assert good.all()
    assert np.array_equal(ids[good], o_ids[good])
    a, b = lp[good].astype(np.float64), o_lp[good].astype(np.float64)
    assert np.array_equal(np.isneginf(a), np.isneginf(b))
    fin = np.isfinite(b)
    assert np.abs(a[fin] - b[fin]).max(initial=0) <= EPS
    assert np.all(np.abs(lse[good, 0] - o_lse[good]) <= tolerance(o_lse[good]))
    for gs in keep:
        gs.destroy()


# --------------------------------------------------------------------------- whole round, small
@pytest.mark.parametrize("kw", [
    dict(batch=4, L=4, V=1000, K=4, budget_min=8, budget_max=24, budget_step=8),
    dict(batch=3, L=6, V=5000, K=8, budget_min=16, budget_max=96, budget_step=16, logits_dtype="bf16",
         hidden_dtype="bf16", hidden_dim=64, m=32),
    dict(batch=2, L=16, V=20011, K=32, budget_min=32, budget_max=512, budget_step=16, logits_dtype="bf16", m=128,
         hidden_dim=128, boost_lo=6.0, boost_hi=14.0),
    dict(batch=2, L=3, V=50, K=4, budget_min=200, budget_max=200, fixed_budget=200),  # budget > all prefixes
    dict(batch=2, L=5, V=300, K=1, budget_min=4, budget_max=12, budget_step=4),        # K = 1: a chain
    dict(batch=2, L=1, V=300, K=8, budget_min=4, budget_max=4, fixed_budget=4),        # single position
    dict(batch=3, L=8, V=3000, K=16, budget_min=0, budget_max=64, fixed_budget=0),     # empty budget
    dict(batch=5, L=16, V=32000, K=8, budget_min=64, budget_max=64, fixed_budget=64, hidden_ar1=False),
])
@pytest.mark.parametrize("beta", [0.2, 0.0])
def test_round_small(kw, beta):
    w = gi.small(**kw, beta=beta)
    g = _graft(w)
    tb, saba_kw, keep = _setup(w, g)
    x = gi.batch_inputs(w)
    out, gpu = gpu_round(g, w, x)
    orc = oracle_round(oracle, w, x, tb, saba_kw)
    stats = compare_round(oracle, w, x, tb, saba_kw, gpu, orc)
    assert stats["excused_tree"] + stats["excused_budget"] <= max(1, w.batch // 4), stats
    compare_accept(oracle, gi, g, w, out, gpu)


def test_round_edge_rows_need_the_separate_kernel_when_the_tables_are_wide():
    """m = 512 with K = 32, L = 16: the table rows do not fit in the tree kernel's shared memory, so every depth
    is scored by the separate kernel and the split cannot be changed."""
    from paper_2608_20375_b200 import GraftError
    w = gi.small(batch=3, L=16, V=6000, K=32, budget_min=32, budget_max=512, budget_step=16, m=512, hidden_dim=64,
                 boost_lo=6.0, boost_hi=14.0)
    g = _graft(w)
    assert g.edge_rows() == w.L
    with pytest.raises(GraftError):
        g.set_edge_rows(4)
    tb, saba_kw, keep = _setup(w, g)
    x = gi.batch_inputs(w)
    out, gpu = gpu_round(g, w, x)
    orc = oracle_round(oracle, w, x, tb, saba_kw)
    stats = compare_round(oracle, w, x, tb, saba_kw, gpu, orc)
    assert stats["excused_tree"] + stats["excused_budget"] <= 1, stats


_SPLIT_CASES = [
    dict(batch=4, L=16, V=20011, K=32, budget_min=32, budget_max=512, budget_step=16, logits_dtype="bf16", m=128,
         hidden_dim=128, boost_lo=6.0, boost_hi=14.0),
    dict(batch=3, L=6, V=5000, K=8, budget_min=16, budget_max=96, budget_step=16, m=32),
    dict(batch=2, L=5, V=300, K=1, budget_min=4, budget_max=12, budget_step=4),  # a chain: every depth is reached
    dict(batch=3, L=16, V=32000, K=8, budget_min=64, budget_max=64, fixed_budget=64, hidden_ar1=False, m=36),
    dict(batch=2, L=12, V=900, K=5, budget_min=40, budget_max=40, fixed_budget=40, m=20, boost_lo=14.0,
         boost_hi=14.0),                                                          # peaked: deep and narrow
]


@pytest.mark.parametrize("kw", _SPLIT_CASES)
@pytest.mark.parametrize("rows", [0, 1, 3, None])
def test_round_edge_rows_split(kw, rows):
    """The depths up to `rows` are scored by the separate kernel, the rest on demand inside the tree kernel
    (None: all by the separate kernel).  Every split must give oracle-valid trees."""
    w = gi.small(**kw)
    g = _graft(w)
    g.set_edge_rows(min(w.L, w.L if rows is None else rows))
    tb, saba_kw, keep = _setup(w, g)
    x = gi.batch_inputs(w)
    out, gpu = gpu_round(g, w, x)
    orc = oracle_round(oracle, w, x, tb, saba_kw)
    stats = compare_round(oracle, w, x, tb, saba_kw, gpu, orc)
    assert stats["excused_tree"] + stats["excused_budget"] <= max(1, w.batch // 4), stats
    assert int(gpu["depth"].max()) >= min(w.L, 3)  # the case does reach the depths scored on demand
    g.destroy()


@pytest.mark.parametrize("kw", _SPLIT_CASES)
def test_round_does_not_depend_on_the_edge_rows_split(kw):
    """Both scorers run the same arithmetic in the same order, so the trees are the same bit for bit."""
    w = gi.small(**kw)
    g = _graft(w)
    _setup(w, g)
    x = gi.batch_inputs(w)
    outs = []
    for rows in (0, 2, w.L):
        g.set_edge_rows(min(rows, w.L))
        outs.append(gpu_round(g, w, x, debug=False)[1])
    for other in outs[1:]:
        for k in ("n_nodes", "budget", "status", "token", "parent", "depth", "position", "path_score", "mask"):
            assert np.array_equal(outs[0][k], other[k]), k
    g.destroy()


@pytest.mark.parametrize("kw", _SPLIT_CASES[:3] + [
    dict(batch=3, L=16, V=6000, K=32, budget_min=32, budget_max=512, budget_step=16, m=512, hidden_dim=64)])
@pytest.mark.parametrize("rows", [0, None])
def test_round_without_debug_outputs_gives_the_same_trees(kw, rows):
    """The production call (no candidate / edge / state outputs requested) must give the trees of the call
    that also writes the debug arrays, bit for bit."""
    w = gi.small(**kw)
    g = _graft(w)
    if rows is not None and w.m < 512:  # (m = 512: the split is fixed, every depth by the separate kernel)
        g.set_edge_rows(rows)
    _setup(w, g)
    x = gi.batch_inputs(w)
    _, a = gpu_round(g, w, x, debug=True)
    _, b = gpu_round(g, w, x, debug=False)
    for k in ("n_nodes", "budget", "status", "token", "parent", "depth", "position", "path_score", "mask"):
        assert np.array_equal(a[k], b[k]), k
    g.destroy()


def test_round_bad_rows_and_status_bits():
    w = gi.small(batch=4, L=4, V=2000, K=4, budget_min=8, budget_max=24, budget_step=8)
    g = _graft(w)
    tb, saba_kw, keep = _setup(w, g)
    x = gi.batch_inputs(w)
    x["logits"][1, 2, 17] = float("nan")
    x["logits"][3, 0, :] = float("-inf")
    saba_kw = dict(saba_kw, phi_bias=-1e4)  # tau clamps on every sequence
    g.set_saba(**saba_kw)
    out, gpu = gpu_round(g, w, x)
    orc = oracle_round(oracle, w, x, tb, saba_kw)
    assert gpu["status"].tolist() == [2, 1, 2, 1] == orc["status"].tolist()
    compare_round(oracle, w, x, tb, saba_kw, gpu, orc)


@pytest.mark.parametrize("budget", [40, 600, 1000])
def test_round_with_thousands_of_equal_path_scores(budget):
    """Uniform rows and beta = 0: every prefix of a depth has the same score, so the threshold is decided among
    thousands of equal keys (the exact select's list overflows and the radix passes take over) and the last nodes are
    chosen by the order among equal scores alone.  One sequence has a single raised token per row, so that a few
    hundred distinct scores sit beside the ties."""
    w = gi.small(batch=3, L=5, V=2000, K=32, budget_min=budget, budget_max=budget, fixed_budget=budget, beta=0.0, m=16)
    g = _graft(w)
    tb, saba_kw, keep = _setup(w, g)
    x = gi.batch_inputs(w)
    x["logits"][:] = 0.0
    x["logits"][1, :, 3] = 2.0
    x["logits"][2, 1:, :] = torch.round(x["logits"][2, 1:, :] + torch.arange(w.V) % 3)
    out, gpu = gpu_round(g, w, x)
    orc = oracle_round(oracle, w, x, tb, saba_kw)
    stats = compare_round(oracle, w, x, tb, saba_kw, gpu, orc)
    # the sequences with a raised token add the same few fp32 numbers in different orders along different paths, so
    # their near-ties may fall differently on log-probabilities that differ within the tolerance (checked as valid
    # best-first outcomes by compare_round); the all-uniform sequence has exact ties and must match bit for bit
    assert stats["excused_budget"] == 0 and stats["excused_tree"] <= 2, stats
    for k in ("token", "parent", "depth", "mask"):
        assert np.array_equal(gpu[k][0], orc[k][0]), k
    assert gpu["n_nodes"].tolist() == [budget + 1] * 3
    compare_accept(oracle, gi, g, w, out, gpu)


@pytest.mark.parametrize("beta", [0.0, 0.25])
def test_round_every_cut_through_small_groups_of_tied_prefixes(beta):
    """The same sequence under every fixed budget from 1 to 96: its logits sit on a grid of 1/2 with pairs and triples of
    equal values among the best candidates of every position, and exact powers of two as probabilities' ratios, so
    prefixes tie in twos to tens -- siblings, cousins under different parents, a parent with the chain below it -- and
    every budget cuts such a group somewhere.  A few tied keys at the threshold are resolved among the tied nodes of
    the table (more than 32 by the sequential expansion): either way the tree must be the oracle's, node for node."""
    nb = 96
    w = gi.small(batch=nb, L=5, V=64, K=8, budget_min=1, budget_max=nb, budget_step=1, fixed_budget=1, beta=beta, m=8,
                 seed=5)
    g = _graft(w)
    tb, saba_kw, keep = _setup(w, g)
    if beta != 0.0:  # equal rows for tokens that share a logit, so that their edge scores tie as well
        for t in (tb["P"], tb["C"]):
            t[1::2] = t[0::2][: t[1::2].shape[0]]
        keep = [tb["P"].cuda(), tb["C"].cuda(), tb["u"].cuda()]
        g.set_tdes_tables(keep[0], keep[1], keep[2], tb["s"])
    x = gi.batch_inputs(w)
    row = torch.full((w.L, w.V), -20.0)
    for d in range(w.L):
        vals = [4.0, 4.0, 3.5, 3.5, 3.5, 3.0, 2.5, 2.5][:: 1 if d % 2 == 0 else -1]
        row[d, 2 * d: 2 * d + 8] = torch.tensor(vals)
    x["logits"][:] = row.to(x["logits"].dtype)
    x["root_token"][:] = x["root_token"][0]
    x["hist"][:] = x["hist"][0]
    x["prefix_len"][:] = x["prefix_len"][0]
    x["hidden"][:] = x["hidden"][0]
    x["fixed_budget"] = torch.arange(1, nb + 1, dtype=torch.int32)
    out, gpu = gpu_round(g, w, x)
    orc = oracle_round(oracle, w, x, tb, saba_kw)
    stats = compare_round(oracle, w, x, tb, saba_kw, gpu, orc)
    assert stats["excused_budget"] == 0 and stats["excused_tree"] == 0, stats
    for k in ("n_nodes", "token", "parent", "depth", "mask", "status"):
        assert np.array_equal(gpu[k], orc[k]), k
    assert gpu["n_nodes"].tolist() == [b + 1 for b in range(1, nb + 1)]
    compare_accept(oracle, gi, g, w, out, gpu)


@pytest.mark.parametrize("beta", [0.0, 0.2])
@pytest.mark.parametrize("shape", ["all equal", "16 equal winners", "32 equal winners", "one-hot", "two-hot", "mixed"])
def test_round_every_cut_through_large_groups_of_tied_prefixes(shape, beta):
    """Rows of exactly equal probabilities at the benchmark's K and L: all K candidates of every position equal, 16
    equal winners over 16 equal others, one token of probability 1 (its chain ties with nothing, everything else ties
    in hundreds), two tokens of probability 1/2, and a mix of these along the depth.  Without edge scores (beta = 0)
    hundreds to thousands of prefixes tie with the B-th largest key; 64 fixed budgets from 1 to 512 cut those groups
    everywhere.  The tree must be the oracle's, node for node."""
    nb, K, L, V = 64, 32, 16, 1000
    w = gi.small(batch=nb, L=L, V=V, K=K, budget_min=1, budget_max=512, budget_step=1, fixed_budget=1, beta=beta, m=16,
                 seed=9)
    g = _graft(w)
    tb, saba_kw, keep = _setup(w, g)
    x = gi.batch_inputs(w)
    row = torch.full((L, V), -30.0)
    for d in range(L):
        kind = shape if shape != "mixed" else ("all equal", "one-hot", "16 equal winners", "two-hot")[d % 4]
        at = 3 * d
        if kind == "all equal":
            row[d] = 0.0
        elif kind == "16 equal winners":
            row[d, at:at + 32] = 0.0
            row[d, at:at + 16] = 1.0
        elif kind == "32 equal winners":
            row[d, at:at + 32] = 3.0
        elif kind == "one-hot":
            row[d] = -60.0
            row[d, at] = 0.0
        elif kind == "two-hot":
            row[d] = -60.0
            row[d, at] = 0.0
            row[d, at + 5] = 0.0
    x["logits"][:] = row.to(x["logits"].dtype)
    for k in ("root_token", "hist", "prefix_len", "hidden"):
        x[k][:] = x[k][0]
    x["fixed_budget"] = torch.tensor([1 + (511 * i) // (nb - 1) for i in range(nb)], dtype=torch.int32)
    out, gpu = gpu_round(g, w, x)
    orc = oracle_round(oracle, w, x, tb, saba_kw)
    stats = compare_round(oracle, w, x, tb, saba_kw, gpu, orc)
    assert stats["excused_budget"] == 0 and stats["excused_tree"] == 0, stats
    for k in ("n_nodes", "token", "parent", "depth", "mask", "status"):
        assert np.array_equal(gpu[k], orc[k]), k
    compare_accept(oracle, gi, g, w, out, gpu)


@pytest.mark.parametrize("budget", [20, 50, 150])
def test_round_with_equal_scores_across_depths_and_masked_tokens(budget):
    """Sequence 0: below a uniform first position every later position has one token of probability 1 to fp32
    precision, so a depth-1 prefix and the chain under it have exactly the same path score and the order among equal
    scores (shallower first, then the order of the prefixes) decides across depths.  Sequence 1: only five tokens
    of a K = 8 candidate set are finite at the deeper positions, so three children of every node score -inf.
    Sequence 2: see below."""
    w = gi.small(batch=3, L=5, V=500, K=8, budget_min=budget, budget_max=budget, fixed_budget=budget, beta=0.0, m=16)
    g = _graft(w)
    tb, saba_kw, keep = _setup(w, g)
    x = gi.batch_inputs(w)
    x["logits"][0] = 0.0
    x["logits"][0, 1:, 7] = 40.0
    x["logits"][1, 1:, 5:] = float("-inf")
    # sequence 2: one token of probability 1 at every position, the rest 46 below: the threshold lies far below the
    # best score (beyond the range the threshold search's bins resolve)
    x["logits"][2] = 0.0
    x["logits"][2, :, 7] = 40.0
    out, gpu = gpu_round(g, w, x)
    orc = oracle_round(oracle, w, x, tb, saba_kw)
    stats = compare_round(oracle, w, x, tb, saba_kw, gpu, orc)
    assert stats["excused_budget"] == 0 and stats["excused_tree"] <= 1, stats
    for k in ("n_nodes", "token", "parent", "depth", "mask", "status"):
        assert np.array_equal(gpu[k][0], orc[k][0]), k
    compare_accept(oracle, gi, g, w, out, gpu)


def test_round_affine_cost_and_paper_grid():
    w = gi.small(batch=6, L=8, V=4000, K=8, budget_min=32, budget_max=512, budget_step=16, hidden_dim=96)
    g = _graft(w)
    tb, _, keep = _setup(w, g)
    saba_kw = dict(phi_conf=-120.0, phi_degen=30.0, phi_hist=4.0, phi_bias=150.0, tau_min=8.0, cost_mode=0, c0=18.0,
                   c1=0.02, c2=2e-6)
    g.set_saba(**saba_kw)
    x = gi.batch_inputs(w)
    out, gpu = gpu_round(g, w, x)
    orc = oracle_round(oracle, w, x, tb, saba_kw)
    compare_round(oracle, w, x, tb, saba_kw, gpu, orc)
    assert len(set(gpu["budget"].tolist())) > 1  # budgets actually vary with the state


def test_host_buffer_entry_point_matches_device_entry_point():
    w = gi.small(batch=3, L=6, V=5000, K=8, budget_min=16, budget_max=96, budget_step=16, logits_dtype="bf16")
    g = _graft(w)
    tb, saba_kw, keep = _setup(w, g)
    x = gi.batch_inputs(w)
    out, gpu = gpu_round(g, w, x, debug=False)
    pin = lambda t: None if t is None else t.pin_memory()  # noqa: E731
    h = g.alloc_out(w.batch, device="cpu", pinned=True)
    g.build_trees_host(pin(x["logits"]), pin(x["hidden"]), pin(x["root_token"]), pin(x["hist"]), pin(x["prefix_len"]),
                       None, h)
    for k in ("n_nodes", "budget", "token", "parent", "depth", "position", "path_score", "mask", "status"):
        assert np.array_equal(getattr(h, k).numpy().view(gpu[k].dtype), gpu[k]), k


def test_argument_validation():
    from paper_2608_20375_b200 import Graft, GraftError
    with pytest.raises(GraftError, match="supported"):
        Graft(1000, 4, 64, 16, 8, 1, 8, 8)  # K > 32
    with pytest.raises(GraftError, match="supported"):
        Graft(1000, 4, 4, 18, 8, 1, 8, 8)   # m not a multiple of 4
    with pytest.raises(GraftError, match="supported"):
        Graft(1000, 4, 4, 16, 8, 1, 8, 2000)
    w = gi.small()
    g = _graft(w)
    x = gi.batch_inputs(w)
    out = g.alloc_out(w.batch)
    cu = lambda t: t.cuda()  # noqa: E731
    with pytest.raises(GraftError, match="not set"):  # TDES tables missing with beta != 0
        g.build_trees(cu(x["logits"]), cu(x["hidden"]), cu(x["root_token"]), cu(x["hist"]), cu(x["prefix_len"]), None, out)
    _setup(w, g)
    with pytest.raises(GraftError, match="invalid"):  # SABA without hidden states
        g.build_trees(cu(x["logits"]), None, cu(x["root_token"]), cu(x["hist"]), cu(x["prefix_len"]), None, out)
    big = gi.batch_inputs(w.with_batch(w.batch + 1))
    with pytest.raises(GraftError, match="invalid"):  # batch beyond max_batch
        g.build_trees(cu(big["logits"]), cu(big["hidden"]), cu(big["root_token"]), cu(big["hist"]),
                      cu(big["prefix_len"]), None, g.alloc_out(w.batch + 1))
    assert g.launch_count() == 0


# --------------------------------------------------------------------------- stated configurations
def test_config_C1_full():
    w = gi.C1
    g = _graft(w)
    tb, saba_kw, keep = _setup(w, g)
    x = gi.batch_inputs(w)
    out, gpu = gpu_round(g, w, x)
    orc = oracle_round(oracle, w, x, tb, saba_kw)
    compare_round(oracle, w, x, tb, saba_kw, gpu, orc)
    a = compare_accept(oracle, gi, g, w, out, gpu)
    assert 0 <= a[0] <= w.L
    # beta = 0 reduces to DDTree: product-of-probabilities scores, and the tree is the top-B by path score
    g0 = _graft(w, beta=0.0)
    out0, gpu0 = gpu_round(g0, w, x)
    w0 = gi.Workload(**{**w.__dict__, "beta": 0.0})
    orc0 = oracle_round(oracle, w0, x, tb, saba_kw)
    compare_round(oracle, w0, x, tb, saba_kw, gpu0, orc0)
    n = gpu0["n_nodes"][0]
    assert (gpu0["path_score"][0, 1:n] <= 0).all()


def _report(name, stats):
    """The observed largest differences of a configured workload: printed, and appended as a JSON line to the file
    that GRAFT_PARITY_REPORT names (if any)."""
    import json
    import os
    line = json.dumps(dict(config=name, **{k: v for k, v in stats.items()}))
    print("parity", line)
    if os.environ.get("GRAFT_PARITY_REPORT"):
        with open(os.environ["GRAFT_PARITY_REPORT"], "a") as f:
            f.write(line + "\n")


@pytest.mark.parametrize("name", ["C2", "C3", "M", "C5", "C4"])
def test_config_full_size_every_sequence(name):
    """Full-size launch configuration: EVERY sequence is compared with the oracle under the comparison rule and the
    observed largest differences are reported.  No budget may differ; a tree may differ from the oracle's (as a valid
    best-first outcome on a score gap below the tolerance, which compare_round verifies) in at most 1 % of the
    sequences, i.e. in none below a batch of 100 (observed: one sequence of C4's 256, none elsewhere)."""
    import os
    w = gi.WORKLOADS[name]
    g = _graft(w)
    tb, saba_kw, keep = _setup(w, g)
    x = gi.batch_inputs(w)
    cu = lambda t: t.cuda()  # noqa: E731
    z, h, root, hist, pref = (cu(x[k]) for k in ("logits", "hidden", "root_token", "hist", "prefix_len"))
    out = g.alloc_out(w.batch, debug=True)
    g.build_trees(z, h, root, hist, pref, None, out)
    torch.cuda.synchronize()
    gpu = out.cpu()
    assert (gpu["status"] == 0).all()
    assert np.array_equal(gpu["n_nodes"], gpu["budget"] + 1)
    orc = oracle_round(oracle, w, x, tb, saba_kw, threads=os.cpu_count() or 8)
    stats = compare_round(oracle, w, x, tb, saba_kw, gpu, orc)
    _report(name, stats)
    assert stats["sequences"] == w.batch
    assert stats["excused_budget"] == 0 and stats["excused_tree"] <= w.batch // 100, stats
    # at these magnitudes the rule is plain 1e-5 absolute: check the observed differences against it directly
    for k in ("topk_lp", "lse", "edge", "path_score", "state"):
        assert stats["max_delta"][k] <= EPS, (k, stats["max_delta"])
    compare_accept(oracle, gi, g, w, out, gpu)
    assert len(set(gpu["budget"].tolist())) > 1 or name in ("C2",)
    # the call the benchmark times (no debug outputs: the first depths by the edge-score kernel, deeper ones on
    # demand) gives the same trees as the call checked above, bit for bit, for every sequence
    out_p = g.alloc_out(w.batch, debug=False)
    g.build_trees(z, h, root, hist, pref, None, out_p)
    torch.cuda.synchronize()
    prod = out_p.cpu()
    for k in ("n_nodes", "budget", "status", "token", "parent", "depth", "position", "path_score", "mask"):
        assert np.array_equal(prod[k], gpu[k]), k
    g.destroy()


@pytest.mark.parametrize("K,L,budget", [(1, 5, 5), (1, 16, 16), (4, 8, 40), (32, 16, 512)])
def test_acceptance_walk_reaches_full_depth(K, L, budget):
    """Peaked rows (one token far above the rest at every position) and targets that follow the chain of best tokens:
    the walk accepts all L draft tokens, the path is the chain, and the bonus token is the target's token after the
    deepest node.  A second sequence's targets leave the chain at the last depth (a = L - 1)."""
    w = gi.small(batch=2, L=L, V=2000, K=K, budget_min=budget, budget_max=budget, fixed_budget=budget, beta=0.0, m=16)
    g = _graft(w)
    _setup(w, g)
    x = gi.batch_inputs(w)
    best = torch.randint(0, w.V, (w.batch, L), generator=torch.Generator().manual_seed(11))
    x["logits"].scatter_(2, best[..., None], 25.0)
    out, gpu = gpu_round(g, w, x)
    y = np.concatenate([best.numpy(), [[1234], [77]]], axis=1).astype(np.int32)  # y_1..y_L, then the bonus token
    y[1, L - 1] = next(t for t in range(w.V) if t not in set(gpu["topk_id"][1, L - 1].tolist()))  # no child carries it
    tn = np.stack([gi.target_next_from_depth(y[b], gpu["depth"][b]) for b in range(w.batch)])
    a_len = torch.empty(w.batch, dtype=torch.int32, device="cuda")
    a_path = torch.empty((w.batch, L), dtype=torch.int32, device="cuda")
    bonus = torch.empty(w.batch, dtype=torch.int32, device="cuda")
    g.accept(out, torch.from_numpy(tn).cuda(), a_len, a_path, bonus)
    torch.cuda.synchronize()
    a_len, a_path, bonus = a_len.cpu().numpy(), a_path.cpu().numpy(), bonus.cpu().numpy()
    assert a_len.tolist() == [L, L - 1]
    assert bonus.tolist() == [1234, int(y[1, L - 1])]
    for b in range(w.batch):
        a, path, bo = oracle.accept(int(gpu["n_nodes"][b]), gpu["token"][b], gpu["parent"][b], tn[b], L)
        assert a == a_len[b] and np.array_equal(path, a_path[b]) and bo == bonus[b]
        n = int(a_len[b])
        assert np.array_equal(gpu["token"][b][a_path[b, :n]], y[b, :n])          # the path spells the targets
        assert np.array_equal(gpu["depth"][b][a_path[b, :n]], np.arange(1, n + 1))
        assert (a_path[b, n:] == -1).all()
    g.destroy()


# --------------------------------------------------------------------------- seeded sweep of shapes
def _fuzz_cases():
    rng = np.random.default_rng(20375)
    cases = []
    for i in range(14):
        K = int(rng.choice([1, 2, 3, 5, 8, 13, 16, 27, 32]))
        L = int(rng.choice([1, 2, 3, 7, 16, 24, 32]))
        if L * K * K * 4 > 128 * 1024:
            L = 16
        V = int(rng.choice([K + 1, 97, 1000, 4099, 30011]))
        V = max(V, K)
        bstep = int(rng.choice([1, 3, 8, 16]))
        bmin = int(rng.choice([0, 1, 4, 16]))
        bmax = bmin + bstep * int(rng.integers(0, 30))
        bmax = min(bmax, 1023)
        m = int(rng.choice([4, 8, 20, 64, 132]))
        cases.append(dict(batch=int(rng.integers(1, 6)), L=L, V=V, K=K, budget_min=bmin, budget_max=bmax,
                          budget_step=bstep, m=m, hidden_dim=int(rng.choice([1, 7, 8, 33, 256])),
                          logits_dtype=str(rng.choice(["f32", "bf16"])), hidden_dtype=str(rng.choice(["f32", "bf16"])),
                          beta=float(rng.choice([0.0, 0.2, 1.5])), seed=5000 + i,
                          fixed_budget=(None if rng.random() < 0.6 else int(rng.integers(0, bmax + 1)))))
    return cases


@pytest.mark.parametrize("kw", _fuzz_cases())
@pytest.mark.parametrize("rows", [None, 1])
def test_round_seeded_sweep_of_shapes(kw, rows):
    """Odd sizes (K and L from 1 to 32, tiny vocabularies, m = 4, hidden width 1, budgets from 0 to ~500 on coarse
    and fine grids), every one against the oracle; once with the library's split of the edge scores, once with all
    depths but the first scored inside the tree kernel."""
    w = gi.small(**kw)
    g = _graft(w)
    if rows is not None:
        from paper_2608_20375_b200 import GraftError
        try:
            g.set_edge_rows(min(rows, w.L))
        except GraftError:
            g.destroy()
            pytest.skip("the split is fixed for this shape")
    tb, saba_kw, keep = _setup(w, g)
    x = gi.batch_inputs(w)
    out, gpu = gpu_round(g, w, x)
    orc = oracle_round(oracle, w, x, tb, saba_kw)
    stats = compare_round(oracle, w, x, tb, saba_kw, gpu, orc)
    assert stats["excused_tree"] + stats["excused_budget"] <= 1, stats  # observed: none
    compare_accept(oracle, gi, g, w, out, gpu)
    g.destroy()


@pytest.mark.parametrize("kw", _fuzz_cases()[:10])
@pytest.mark.parametrize("step", [1.0, 0.25])
def test_round_seeded_sweep_with_quantised_logits(kw, step):
    """The same odd shapes with logits rounded to a coarse grid: the candidates of a row hold many equal values, so
    log-probabilities, edge scores and path scores tie in bulk (exactly with beta = 0, up to the fp32 rounding of
    different summation orders otherwise).  Every tree must still be the oracle's or a valid best-first outcome on
    the oracle's scores, and with beta = 0 and exact ties it must be the oracle's."""
    w = gi.small(**kw)
    g = _graft(w)
    tb, saba_kw, keep = _setup(w, g)
    x = gi.batch_inputs(w)
    z = x["logits"].float()
    x["logits"] = (torch.round(z / step) * step).to(x["logits"].dtype)
    out, gpu = gpu_round(g, w, x)
    orc = oracle_round(oracle, w, x, tb, saba_kw)
    stats = compare_round(oracle, w, x, tb, saba_kw, gpu, orc)
    print("excused", stats)
    assert stats["excused_budget"] <= 1 and stats["excused_tree"] <= 1, stats  # observed: none
    compare_accept(oracle, gi, g, w, out, gpu)
    g.destroy()


@pytest.mark.parametrize("noise", [0.0, 1e-3])
@pytest.mark.parametrize("beta", [0.0, 0.2])
def test_round_when_the_node_table_overflows(noise, beta):
    """Flat distributions with K = 20 and a budget of 1000: levels 0..2 hold 421 prefixes, fewer than the budget, so
    level 3 would append 8000 more with no threshold to prune by, which is more than the node table of the parallel
    phase holds; the sequential expansion then builds the whole tree."""
    w = gi.small(batch=2, L=4, V=700, K=20, budget_min=1000, budget_max=1000, fixed_budget=1000, beta=beta, m=16)
    g = _graft(w)
    tb, saba_kw, keep = _setup(w, g)
    x = gi.batch_inputs(w)
    gen = torch.Generator().manual_seed(3)
    x["logits"] = noise * torch.randn(x["logits"].shape, generator=gen)
    out, gpu = gpu_round(g, w, x)
    orc = oracle_round(oracle, w, x, tb, saba_kw)
    stats = compare_round(oracle, w, x, tb, saba_kw, gpu, orc)
    print("excused", stats)
    assert stats["excused_budget"] == 0 and stats["excused_tree"] <= (0 if noise == 0.0 and beta == 0.0 else 1), stats
    assert gpu["n_nodes"].tolist() == [1001, 1001] and gpu["status"].tolist() == [0, 0]
    if noise == 0.0 and beta == 0.0:
        for k in ("token", "parent", "depth", "mask"):
            assert np.array_equal(gpu[k], orc[k]), k
    compare_accept(oracle, gi, g, w, out, gpu)
    g.destroy()


@pytest.mark.parametrize("K,L", [(5, 6), (32, 4)])
def test_round_with_identical_table_rows_and_tied_candidates(K, L):
    """Every token has the same projections, so f is the same for every edge of a depth and the centred score
    vanishes up to rounding: edge scores tie wherever the candidates' log-probabilities tie (logits on a coarse
    grid), and the rows' order falls back on the candidates' rank."""
    w = gi.small(batch=3, L=L, V=900, K=K, budget_min=8, budget_max=200, budget_step=8, beta=0.7, m=24, seed=31)
    from paper_2608_20375_b200 import Graft
    g = Graft(w.V, w.L, w.K, w.m, w.hidden_dim, w.batch, w.budget_min, w.budget_max, w.budget_step, w.beta, 1, 0, 0)
    tb = gi.tdes_tables(w)
    tb["P"][:] = tb["P"][0]
    tb["C"][:] = tb["C"][1]
    saba_kw = gi.saba_defaults(w)
    keep = [tb["P"].cuda(), tb["C"].cuda(), tb["u"].cuda()]
    g.set_tdes_tables(keep[0], keep[1], keep[2], tb["s"])
    g.set_saba(**saba_kw)
    x = gi.batch_inputs(w)
    x["logits"] = torch.round(x["logits"] * 2) / 2
    out, gpu = gpu_round(g, w, x)
    orc = oracle_round(oracle, w, x, tb, saba_kw)
    compare_round(oracle, w, x, tb, saba_kw, gpu, orc)
    compare_accept(oracle, gi, g, w, out, gpu)
    g.destroy()


@pytest.mark.parametrize("beta", [0.0, 0.3])
@pytest.mark.parametrize("rows", [None, 0, 3])
def test_round_deep_trees_with_ties_scored_on_demand(beta, rows):
    """Narrow candidate sets and peaked distributions on a coarse grid give trees sixteen levels deep with ties at
    every level; the deeper edge rows are scored inside the tree kernel.  The call without debug outputs (the one
    the benchmark times) must give the trees of the call that is checked against the oracle, bit for bit."""
    w = gi.small(batch=4, L=16, V=3000, K=3, budget_min=16, budget_max=256, budget_step=16, beta=beta, m=32, seed=77,
                 boost_lo=12.0, boost_hi=16.0)
    g = _graft(w)
    if rows is not None:
        g.set_edge_rows(rows)
    tb, saba_kw, keep = _setup(w, g)
    x = gi.batch_inputs(w)
    x["logits"] = torch.round(x["logits"])
    out, gpu = gpu_round(g, w, x)
    orc = oracle_round(oracle, w, x, tb, saba_kw)
    compare_round(oracle, w, x, tb, saba_kw, gpu, orc)
    assert int(gpu["depth"].max()) >= 10  # beyond the depths the edge-score kernel covers by default
    out_p = g.alloc_out(w.batch, debug=False)
    cu = lambda t: t.cuda()  # noqa: E731
    g.build_trees(cu(x["logits"]), cu(x["hidden"]), cu(x["root_token"]), cu(x["hist"]), cu(x["prefix_len"]), None, out_p)
    torch.cuda.synchronize()
    prod = out_p.cpu()
    for k in ("n_nodes", "budget", "status", "token", "parent", "depth", "position", "path_score", "mask"):
        assert np.array_equal(prod[k], gpu[k]), k
    g.destroy()


# --------------------------------------------------------------------------- random sweep of input styles
_styled_logits = gi.styled_logits


@pytest.mark.parametrize("seed", [101, 102, 103])
def test_round_random_sweep_of_input_styles(seed):
    """Fifty random rounds per seed: shapes from K = 1 to 32 and L = 1 to 32 over vocabularies of K + 1 to 30,011
    tokens, budgets on odd grids, and logits of ten styles (ordinary, on coarse grids, flat, one or two dominant
    tokens, mostly masked, in the hundreds, ramps).  Every round against the oracle under the comparison rule, the
    acceptance walk too, and the call without debug outputs against the checked call, bit for bit."""
    from paper_2608_20375_b200 import Graft, GraftError
    rng = np.random.default_rng(seed)
    styles = ["normal", "quant1", "quant025", "flat", "peaked", "mixed", "huge", "masked", "twopeaks", "ramp"]
    done = seqs = excused = 0
    for ci in range(50):
        K = int(rng.choice([1, 2, 3, 4, 5, 8, 13, 16, 20, 27, 32]))
        L = int(rng.choice([1, 2, 3, 5, 7, 12, 16, 24, 32]))
        if L * K * K * 4 > 128 * 1024:
            L = 16
        V = max(K, int(rng.choice([K + 1, 97, 1000, 4099, 30011])))
        bstep = int(rng.choice([1, 3, 8, 16]))
        bmin = int(rng.choice([0, 1, 4, 16, 64]))
        bmax = min(bmin + bstep * int(rng.integers(0, 64)), 1023)
        kw = dict(batch=int(rng.integers(1, 5)), L=L, V=V, K=K, budget_min=bmin, budget_max=bmax, budget_step=bstep,
                  m=int(rng.choice([4, 8, 20, 64, 128])), hidden_dim=int(rng.choice([1, 8, 33, 256])),
                  logits_dtype=str(rng.choice(["f32", "bf16"])), hidden_dtype=str(rng.choice(["f32", "bf16"])),
                  beta=float(rng.choice([0.0, 0.0, 0.2, 1.5])), seed=int(rng.integers(1, 1 << 30)),
                  fixed_budget=(None if rng.random() < 0.5 else int(rng.integers(0, bmax + 1))))
        style = styles[ci % len(styles)]
        rows = int(rng.choice([-1, 0, 1, 3]))
        w = gi.small(**kw)
        try:
            g = _graft(w)
        except GraftError:
            continue  # a shape beyond the shared-memory limits
        tb, saba_kw, keep = _setup(w, g)
        if rows >= 0:
            try:
                g.set_edge_rows(min(rows, w.L))
            except GraftError:
                pass
        x = gi.batch_inputs(w)
        gen = torch.Generator().manual_seed(kw["seed"])
        x["logits"] = _styled_logits(x["logits"].float(), style, rng, gen, K).to(x["logits"].dtype)
        out, gpu = gpu_round(g, w, x)
        orc = oracle_round(oracle, w, x, tb, saba_kw)
        try:
            st = compare_round(oracle, w, x, tb, saba_kw, gpu, orc)
            seqs += st["sequences"]
            excused += st["excused_tree"] + st["excused_budget"]
            compare_accept(oracle, gi, g, w, out, gpu)
        except AssertionError as e:
            raise AssertionError(f"case {ci} ({style}, edge rows {rows}, {kw}): {e}") from e
        out_p = g.alloc_out(w.batch, debug=False)
        cu = lambda t: None if t is None else t.cuda()  # noqa: E731
        g.build_trees(cu(x["logits"]), cu(x["hidden"]), cu(x["root_token"]), cu(x["hist"]), cu(x["prefix_len"]),
                      cu(x["fixed_budget"]), out_p)
        torch.cuda.synchronize()
        prod = out_p.cpu()
        for k in ("n_nodes", "budget", "status", "token", "parent", "depth", "position", "path_score", "mask"):
            assert np.array_equal(prod[k], gpu[k], equal_nan=prod[k].dtype.kind == "f"), (ci, style, k)
        g.destroy()
        done += 1
    assert done >= 40
    print("excused", excused, "of", seqs)
    # (degenerate styles tie in bulk; the excused trees are valid best-first outcomes on near-ties)
    assert excused <= seqs // 20, (excused, seqs)  # observed: 0 to 3 per hundred

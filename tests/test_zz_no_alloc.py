"""The allocation-free vocab pass (graft_vocab_pass_static) against the context-based one.

Some hosts cannot let a library allocate device memory -- a server whose own pool owns the whole GPU after
start-up, or a latency path that must not touch the driver's allocator -- so this entry point keeps its
scratch in a static device array.  The test calls it through the C ABI twice in a row (the array is shared by
all calls and keeps the previous call's contents) and checks both results against graft_vocab_pass, and against
the CPU oracle on the same rows.  It lives
in a file that pytest collects last, and it must pass both alone in a fresh process and after the other tests.
"""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu


def _reference(z, K):
    from paper_2608_20375_b200 import Graft
    Bt, L, V = z.shape
    g = Graft(V, L, K, 16, 8, Bt, 8, 8, 8, 0.0, 1, 1 if z.dtype == torch.bfloat16 else 0, 0)
    ids = torch.empty((Bt, L, K), dtype=torch.int32, device="cuda")
    lp = torch.empty((Bt, L, K), dtype=torch.float32, device="cuda")
    lse = torch.empty((Bt, L), dtype=torch.float32, device="cuda")
    rs = torch.empty((Bt, L), dtype=torch.int32, device="cuda")
    g.vocab_pass(z, ids, lp, lse, rs)
    torch.cuda.synchronize()
    out = tuple(t.cpu().numpy() for t in (ids, lp, lse, rs))
    g.destroy()
    return out


@pytest.mark.parametrize("shape,K,dtype", [((3, 5, 40003), 16, torch.bfloat16), ((1, 16, 32000), 8, torch.float32)])
def test_static_entry_point_matches_context_entry_point_twice(shape, K, dtype):
    from paper_2608_20375_b200 import vocab_pass_static
    gen = torch.Generator().manual_seed(11)
    inputs = [(2.0 * torch.randn(shape, generator=gen)).to(dtype).cuda() for _ in range(2)]
    inputs[1][0, 1, 7] = float("nan")  # the second call also has a row that must be flagged
    Bt, L, V = shape
    for call, z in enumerate(inputs):  # two calls in a row on the shared static scratch
        want_ids, want_lp, want_lse, want_rs = _reference(z, K)
        ids = torch.full((Bt, L, K), -7, dtype=torch.int32, device="cuda")
        lp = torch.zeros((Bt, L, K), dtype=torch.float32, device="cuda")
        lse = torch.zeros((Bt, L), dtype=torch.float32, device="cuda")
        rs = torch.full((Bt, L), -7, dtype=torch.int32, device="cuda")
        torch.cuda.synchronize()
        free_before = torch.cuda.mem_get_info()[0]
        vocab_pass_static(z, K, ids, lp, lse, rs)
        torch.cuda.synchronize()
        if call == 1:  # (the very first launch may make the driver load the kernel's code)
            assert torch.cuda.mem_get_info()[0] == free_before  # nothing was allocated on the device
        good = want_rs == 0
        assert np.array_equal(rs.cpu().numpy(), want_rs)
        assert np.array_equal(ids.cpu().numpy()[good], want_ids[good])
        assert np.abs(lp.cpu().numpy()[good] - want_lp[good]).max() <= 1e-5
        assert np.abs(lse.cpu().numpy()[good] - want_lse[good]).max() <= 1e-5
        # and against the oracle directly
        import oracle
        o_ids, o_lp, o_lse, o_st = oracle.vocab_pass(z.cpu().reshape(Bt * L, V), K)
        ok = o_st == 0
        assert np.array_equal(rs.cpu().numpy().reshape(-1), o_st)
        assert np.array_equal(ids.cpu().numpy().reshape(Bt * L, K)[ok], o_ids[ok])
        assert np.abs(lp.cpu().numpy().reshape(Bt * L, K)[ok].astype(np.float64) - o_lp[ok]).max() <= 1e-5
        assert np.abs(lse.cpu().numpy().reshape(-1)[ok].astype(np.float64) - o_lse[ok]).max() <= 1e-5


def test_static_entry_point_rejects_sizes_beyond_its_scratch():
    from paper_2608_20375_b200 import GraftError, binding
    lib = binding.load_library()
    z = torch.zeros(64, dtype=torch.float32, device="cuda")
    i32 = torch.empty(8, dtype=torch.int32, device="cuda")
    f32 = torch.empty(8, dtype=torch.float32, device="cuda")
    # 16385 rows > 16384: the size check comes before anything is read or launched
    rc = lib.graft_vocab_pass_static(16385, 1, 64, 4, 0, z.data_ptr(), i32.data_ptr(), f32.data_ptr(), f32.data_ptr(),
                                     i32.data_ptr(), None)
    with pytest.raises(GraftError, match="supported"):
        binding._check(lib, rc, "graft_vocab_pass_static")
    assert lib.graft_vocab_pass_static(1, 1, 64, 4, 0, None, i32.data_ptr(), f32.data_ptr(), f32.data_ptr(),
                                       i32.data_ptr(), None) == 1  # NULL logits: invalid argument

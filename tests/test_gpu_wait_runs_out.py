"""A bounded device-side wait that runs out: the kernel must return, say so in the rows' status words, and leave the
device usable.

The vocab pass waits on shared-memory barriers with an iteration limit; when a wait gives up, the thread block
raises a flag, stops waiting, drains its copies in flight and finishes, and every row it finishes or leaves a piece of
carries GRAFT_ST_INTERNAL.  To make a wait run out without faulting, trapping or hanging anything, this test compiles
a SECOND copy of the vocab pass (one source file, into a temporary folder) with a tiny iteration limit and a build flag
under which thread block 0 never issues the copy of its third tile.  The shipped library is not touched.
"""
import ctypes as C
import os
import subprocess

import numpy as np
import pytest
import torch

import oracle

pytestmark = pytest.mark.gpu

ST_INTERNAL = 8


def _build_test_library(tmp_path):
    from paper_2608_20375_b200 import build as b
    out = os.path.join(str(tmp_path), "libgraft_waittest.so")
    cmd = [os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc"), *b.NVCC_FLAGS, "-DGRAFT_SPIN_LIMIT=512u",
           "-DGRAFT_TEST_WITHHOLD_TILE=2", "-I", os.path.join(b.HERE, "..", "include"), "-shared",
           os.path.join(b.CSRC, "vocab_pass.cu"), "-o", out, "-lcudart"]
    subprocess.check_call(cmd, stderr=subprocess.DEVNULL)
    return out


def test_a_wait_that_runs_out_is_reported_and_the_device_stays_usable(tmp_path):
    lib = C.CDLL(_build_test_library(tmp_path))
    vp = C.c_void_p
    lib.graft_vocab_pass_static.argtypes = [C.c_int32, C.c_int32, C.c_int32, C.c_int32, C.c_int, vp, vp, vp, vp, vp, vp]
    Bt, L, V, K = 8, 16, 151936, 16  # every thread block gets about eight tiles
    g = torch.Generator().manual_seed(5)
    z = (2.0 * torch.randn((Bt, L, V), generator=g)).to(torch.bfloat16)
    zc = z.cuda()
    ids = torch.full((Bt, L, K), -7, dtype=torch.int32, device="cuda")
    lp = torch.zeros((Bt, L, K), dtype=torch.float32, device="cuda")
    lse = torch.zeros((Bt, L), dtype=torch.float32, device="cuda")
    rs = torch.full((Bt, L), -7, dtype=torch.int32, device="cuda")
    stream = C.c_void_p(torch.cuda.current_stream().cuda_stream)
    rc = lib.graft_vocab_pass_static(Bt, L, V, K, 1, zc.data_ptr(), ids.data_ptr(), lp.data_ptr(), lse.data_ptr(),
                                     rs.data_ptr(), stream)
    assert rc == 0                      # the call only enqueues: host-side status
    torch.cuda.synchronize()            # the kernel came back by itself, and without a device error
    st = rs.cpu().numpy().reshape(-1)
    assert (st >= 0).all()              # every row's status word was written
    flagged = (st & ST_INTERNAL) != 0
    assert flagged.any(), "the wait that ran out was not reported"
    assert flagged.sum() <= 4           # only rows of thread block 0 (about two rows; one may be shared)
    # rows that no block with a failed wait touched are correct
    o_ids, o_lp, o_lse, o_st = oracle.vocab_pass(z.reshape(Bt * L, V), K)
    ok = ~flagged
    assert np.array_equal(st[ok], o_st[ok])
    assert np.array_equal(ids.cpu().numpy().reshape(Bt * L, K)[ok], o_ids[ok])
    assert np.abs(lse.cpu().numpy().reshape(-1)[ok] - o_lse[ok]).max() <= 1e-5
    # the device and the shipped library are fine afterwards: an ordinary call gives the oracle's rows
    from paper_2608_20375_b200 import vocab_pass_static
    vocab_pass_static(zc, K, ids, lp, lse, rs)
    torch.cuda.synchronize()
    assert np.array_equal(rs.cpu().numpy().reshape(-1), o_st)
    assert np.array_equal(ids.cpu().numpy().reshape(Bt * L, K), o_ids)
    assert np.abs(lp.cpu().numpy().reshape(Bt * L, K) - o_lp).max() <= 1e-5

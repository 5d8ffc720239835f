"""The no-allocation point evaluation against the CPU oracle and the workspace-based call (GPU, collected last).

Some callers of this library run where device memory cannot be allocated -- inside a serving
engine whose pool owns all of HBM -- so `imm_mle_eval_point_noalloc` keeps its scratch in a fixed
array inside the library.  Calls share that array and it keeps the previous call's contents, so
the check is made on two calls in a row, the second on a smaller matrix than the first.
"""
import ctypes
import random

import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu

P = 0xFFFFFFFF00000001


@pytest.fixture(scope="module")
def imm():
    if not torch.cuda.is_available():
        pytest.fail("a CUDA device is required for -m gpu tests")
    from paper_2602_22700_b200 import imm as binding
    binding.lib()
    return binding


def _case(imm, rng, prng, rows, cols, np_dtype):
    lo, hi = (-128, 127) if np_dtype == np.int8 else (-2**31, 2**31 - 1)
    M = torch.from_numpy(rng.integers(lo, hi, size=(rows, cols), endpoint=True, dtype=np.int64).astype(np_dtype)).cuda()
    r_row = [prng.randrange(P) for _ in range(imm.ceil_log2(rows))]
    r_col = [prng.randrange(P) for _ in range(imm.ceil_log2(cols))]
    return M, imm.eq_table(r_row), imm.eq_table(r_col), r_row, r_col


def test_noalloc_point_eval_matches_oracle_and_workspace_version_twice_in_a_row(imm, oracle):
    rng = np.random.default_rng(2024)
    prng = random.Random(2024)
    out = torch.zeros(1, dtype=torch.int64, device="cuda")
    # first a matrix that fills many slots of the shared array, then smaller ones that reuse them
    for rows, cols, dt in ((3000, 5000, np.int32), (700, 1300, np.int32), (4100, 9000, np.int8), (33, 70, np.int8)):
        M, er, ec, r_row, r_col = _case(imm, rng, prng, rows, cols, dt)
        # expected value: the CPU oracle's plain two-sided evaluation, its own eq tables included
        want_oracle = oracle.mle_eval_point(M.cpu().numpy(), oracle.eq_table(r_row), oracle.eq_table(r_col))
        want = imm.mle_eval_point(M, er, ec)
        assert int(want[0]) & (2**64 - 1) == want_oracle
        out.fill_(-1)
        got = imm.mle_eval_point_noalloc(M, er, ec, out)
        torch.cuda.synchronize()
        assert int(got[0]) & (2**64 - 1) == want_oracle     # integers mod p: equality, as everywhere else
        # and once more on the same input, back to back on the same stream
        out.fill_(-1)
        imm.mle_eval_point_noalloc(M, er, ec, out)
        imm.mle_eval_point_noalloc(M, er, ec, out)
        torch.cuda.synchronize()
        assert int(out[0]) == int(want[0])


def test_noalloc_rejects_what_does_not_fit_before_touching_the_gpu(imm):
    L = imm.lib()
    fake = 0x10000                                   # never dereferenced: the size check comes first
    big = 1 << 20
    assert L.imm_mle_eval_point_noalloc(fake, imm.I32, big, big, big, fake, fake, fake, None) == imm.ERR_LIMIT
    assert L.imm_mle_eval_point_noalloc(fake, imm.I8, big, big, big, fake, fake, fake, None) == imm.ERR_LIMIT
    assert L.imm_mle_eval_point_noalloc(fake, imm.I32, 0, 4, 4, fake, fake, fake, None) == -2
    assert L.imm_mle_eval_point_noalloc(None, imm.I32, 4, 4, 4, fake, fake, fake, None) == -1

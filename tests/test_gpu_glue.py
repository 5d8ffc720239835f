"""GPU parity of the requantisation link check against the CPU oracle (run with -m gpu).

Integers throughout: the count of differing entries and the position of the first must be equal.
"""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu

MAXU = (1 << 64) - 1


@pytest.fixture(scope="module")
def imm():
    if not torch.cuda.is_available():
        pytest.fail("a CUDA device is required for -m gpu tests")
    from paper_2602_22700_b200 import imm as binding
    binding.lib()
    return binding


@pytest.fixture(scope="module")
def synth():
    from paper_2602_22700_b200 import synth as s
    return s


@pytest.fixture(scope="module")
def glue():
    from oracle import glue as g
    return g


def result(t):
    cnt, first = (int(v) for v in t.cpu())
    return cnt, first                      # first is -1 when the device word is UINT64_MAX (int64 view)


def strided(t, pad, offset_elems):
    rows, cols = t.shape
    buf = torch.zeros(rows * (cols + pad) + offset_elems + 64, dtype=t.dtype, device=t.device)
    v = buf[offset_elems:offset_elems + rows * (cols + pad)].view(rows, cols + pad)[:, :cols]
    v.copy_(t)
    return v


def edge_heavy(rng, rows, cols, shift, lo, hi):
    """int32 values clustered at the rounding boundaries, the clamp edges and the type's extremes."""
    step = 1 << shift
    q = rng.integers(lo - 3, hi + 4, size=(rows, cols), dtype=np.int64)
    near = q * step + step // 2 + rng.integers(-2, 3, size=(rows, cols))       # around a tie
    wide = rng.integers(-2**31, 2**31, size=(rows, cols), dtype=np.int64)
    pick = rng.random((rows, cols))
    C = np.where(pick < 0.6, near, np.where(pick < 0.9, rng.integers(-70000, 70000, size=(rows, cols)), wide))
    C = np.clip(C, -2**31, 2**31 - 1)
    C.reshape(-1)[:4] = [2**31 - 1, -2**31, 2**31 - step // 2 - 1, -2**31 + step // 2][:min(4, C.size)]
    return C.astype(np.int32)


SHAPES = [(1, 1), (1, 15), (3, 16), (5, 17), (37, 53), (64, 4096), (129, 4097), (300, 1000), (33, 14336), (2050, 300),
          (7, 70000), (5000, 8)]


@pytest.mark.parametrize("rows,cols", SHAPES)
@pytest.mark.parametrize("layout", ["contiguous", "padded_rows", "unaligned"])
def test_requant_check_matches_oracle(imm, glue, rows, cols, layout):
    rng = np.random.default_rng(rows * 131 + cols)
    shift, rnd, lo, hi = 9, 256, -127, 127
    Ch = edge_heavy(rng, rows, cols, shift, lo, hi)
    Hh = glue.requantize(Ch, shift, rnd, lo, hi)
    C, H = torch.from_numpy(Ch).cuda(), torch.from_numpy(Hh).cuda()
    if layout == "padded_rows":            # aligned rows with a leading dimension beyond the columns
        C, H = strided(C, 8 - cols % 8 + 8, 0), strided(H, 16 - cols % 16 + 16, 0)
    elif layout == "unaligned":
        C, H = strided(C, 3, 1), strided(H, 5, 3)
    assert result(imm.requant_check(C, H)) == (0, -1) == glue.requant_check(Ch, Hh, shift, rnd, lo, hi)
    # planted differences: a few in H, one in C that crosses a boundary
    nbad = min(rows * cols, 5)
    for flat in rng.choice(rows * cols, size=nbad, replace=False):
        i, j = divmod(int(flat), cols)
        Hh[i, j] = np.int8((int(Hh[i, j]) + 1 + 128) % 256 - 128)
        H[i, j] = int(Hh[i, j])
    assert result(imm.requant_check(C, H)) == glue.requant_check(Ch, Hh, shift, rnd, lo, hi)
    assert glue.requant_check(Ch, Hh, shift, rnd, lo, hi)[0] == nbad
    i, j = rows - 1, cols - 1
    Ch[i, j] = np.int32(int(Ch[i, j]) - 4 * 512 if Ch[i, j] > 0 else int(Ch[i, j]) + 4 * 512)
    C[i, j] = int(Ch[i, j])
    assert result(imm.requant_check(C, H)) == glue.requant_check(Ch, Hh, shift, rnd, lo, hi)


@pytest.mark.parametrize("shift,rnd,lo,hi", [(0, 0, -127, 127), (1, 1, -128, 127), (4, 8, 0, 15), (9, 0, -127, 127),
                                             (9, 511, -127, 127), (16, 1 << 15, -127, 127), (30, (1 << 30) - 1, -1, 1),
                                             (12, 7, -3, -3)])
def test_requant_check_other_parameters(imm, glue, shift, rnd, lo, hi):
    rng = np.random.default_rng(shift * 1000 + rnd % 997)
    Ch = edge_heavy(rng, 130, 1040, shift, lo, hi)
    Hh = glue.requantize(Ch, shift, rnd, lo, hi)
    C, H = torch.from_numpy(Ch).cuda(), torch.from_numpy(Hh).cuda()
    assert result(imm.requant_check(C, H, shift, rnd, lo, hi)) == (0, -1)
    # the same H against a neighbouring map differs where the oracle says it does
    other = (shift, (rnd + 1) % (1 << shift) if shift else 0, lo, hi) if shift else (1, 0, lo, hi)
    assert result(imm.requant_check(C, H, *other)) == glue.requant_check(Ch, Hh, *other)
    # every entry wrong: the count is the whole matrix, the first position 0
    H2 = torch.from_numpy(((Hh.astype(np.int16) + 128 + 77) % 256 - 128).astype(np.int8)).cuda()
    assert result(imm.requant_check(C, H2, shift, rnd, lo, hi)) == (130 * 1040, 0)


def test_ffn_pair_link_at_full_size(imm, glue, synth):
    """The hidden activations between the FFN up and down projections: the down proof's A must be the
    requantised C of the up proof.  Honest pair: the link holds; one altered entry on either side is
    found where it is."""
    up, down = synth.ffn_pair(1, device="cuda")
    assert up.C.shape == down.A.shape == (2048, 14336)
    out = torch.empty(2, dtype=torch.int64, device="cuda")
    assert result(imm.requant_check(up.C, down.A, out=out)) == (0, -1)
    Ch, Hh = up.C.cpu().numpy(), down.A.cpu().numpy()
    assert glue.requant_check(Ch, Hh, 9, 256, -127, 127) == (0, -1)
    H = down.A.clone()
    H[1234, 5678] += 1
    assert result(imm.requant_check(up.C, H, out=out)) == (1, 1234 * 14336 + 5678)
    C = up.C.clone()
    C[2047, 14335] += 512
    C[7, 0] -= 512
    want = glue.requant_check(C.cpu().numpy(), Hh, 9, 256, -127, 127)
    assert result(imm.requant_check(C, down.A, out=out)) == want and want[1] == 7 * 14336 and want[0] >= 1
    # a down projection proved over unrelated activations is caught by the link, not by its own proof
    unrelated = synth.gauss_i8(2, synth.tid(0, synth.ROLE_ACT2), 2048, 14336, synth.Q_SIGMA20, "cuda")
    cnt, first = result(imm.requant_check(up.C, unrelated, out=out))
    assert (cnt, first) == glue.requant_check(Ch, unrelated.cpu().numpy(), 9, 256, -127, 127) and cnt > 2048 * 14336 // 2


def test_requant_check_refuses_bad_arguments(imm):
    L = imm.lib()
    C = torch.zeros((4, 8), dtype=torch.int32, device="cuda")
    H = torch.zeros((4, 8), dtype=torch.int8, device="cuda")
    out = torch.zeros(2, dtype=torch.int64, device="cuda")
    ok = (C.data_ptr(), H.data_ptr(), 4, 8, 8, 8)
    assert L.imm_requant_check(*ok, 9, 256, -127, 127, out.data_ptr(), None) == 0
    assert L.imm_requant_check(None, H.data_ptr(), 4, 8, 8, 8, 9, 256, -127, 127, out.data_ptr(), None) == imm.ERR_ARG
    assert L.imm_requant_check(*ok, 9, 256, -127, 127, None, None) == imm.ERR_ARG
    assert L.imm_requant_check(*ok, 31, 0, -127, 127, out.data_ptr(), None) == imm.ERR_ARG
    assert L.imm_requant_check(*ok, 9, 512, -127, 127, out.data_ptr(), None) == imm.ERR_ARG
    assert L.imm_requant_check(*ok, 9, -1, -127, 127, out.data_ptr(), None) == imm.ERR_ARG
    assert L.imm_requant_check(*ok, 9, 256, 5, 4, out.data_ptr(), None) == imm.ERR_ARG
    assert L.imm_requant_check(*ok, 9, 256, -129, 127, out.data_ptr(), None) == imm.ERR_ARG
    assert L.imm_requant_check(C.data_ptr(), H.data_ptr(), 0, 8, 8, 8, 9, 256, -127, 127, out.data_ptr(), None) == imm.ERR_SHAPE
    assert L.imm_requant_check(C.data_ptr(), H.data_ptr(), 4, 8, 7, 8, 9, 256, -127, 127, out.data_ptr(), None) == imm.ERR_SHAPE
    assert L.imm_requant_check(*ok, 9, 256, -127, 127, out.data_ptr() + 4, None) == imm.ERR_ALIGN
    with pytest.raises(ValueError):
        imm.requant_check(C, C)
    with pytest.raises(ValueError):
        imm.requant_check(C.cpu(), H.cpu())


# ---------------------------------------------------------------- activation table and gated product

def act_tables():
    import math
    silu = np.array([int(round(v / (1.0 + math.exp(-v / 16.0)))) for v in range(-128, 128)], dtype=np.int8)
    relu = np.array([max(0, v) for v in range(-128, 128)], dtype=np.int8)
    ident = np.arange(-128, 128, dtype=np.int8)
    rng = np.random.default_rng(5)
    anyt = rng.integers(-128, 128, 256).astype(np.int8)                # any table is a valid input
    return {"silu": silu, "relu": relu, "identity": ident, "random": anyt}


GATED_SHAPES = [(1, 1), (1, 15), (3, 16), (5, 17), (37, 53), (64, 4096), (129, 4097), (33, 14336), (2050, 300), (7, 70000)]


@pytest.mark.parametrize("rows,cols", GATED_SHAPES)
@pytest.mark.parametrize("layout", ["contiguous", "padded_rows", "unaligned"])
@pytest.mark.parametrize("gated", [True, False])
def test_gated_link_check_matches_oracle(imm, glue, rows, cols, layout, gated):
    rng = np.random.default_rng(rows * 77 + cols + (1 if gated else 0))
    act = act_tables()["silu" if (rows + cols) % 2 else "random"]
    par = (9, 256, 7, 64, -127, 127)
    Gh = edge_heavy(rng, rows, cols, 9, -128, 127)
    Uh = edge_heavy(rng, rows, cols, 9, -128, 127) if gated else None
    Hh = glue.gated_link(Gh, Uh, act, *par)
    G, H = torch.from_numpy(Gh).cuda(), torch.from_numpy(Hh).cuda()
    U = torch.from_numpy(Uh).cuda() if gated else None
    if layout == "padded_rows":
        G, H = strided(G, 8 - cols % 8 + 8, 0), strided(H, 16 - cols % 16 + 16, 0)
        U = strided(U, 4 - cols % 4 + 12, 0) if gated else None
    elif layout == "unaligned":
        G, H = strided(G, 3, 1), strided(H, 5, 3)
        U = strided(U, 1, 2) if gated else None
    assert result(imm.gated_link_check(G, U, H, act, *par)) == (0, -1) == glue.gated_link_check(Gh, Uh, Hh, act, *par)
    nbad = min(rows * cols, 5)
    for flat in rng.choice(rows * cols, size=nbad, replace=False):
        i, j = divmod(int(flat), cols)
        Hh[i, j] = np.int8((int(Hh[i, j]) + 1 + 128) % 256 - 128)
        H[i, j] = int(Hh[i, j])
    want = glue.gated_link_check(Gh, Uh, Hh, act, *par)
    assert want[0] == nbad and result(imm.gated_link_check(G, U, H, act, *par)) == want
    # an altered accumulator on either side is found exactly where the oracle finds it (or nowhere)
    Gh[rows - 1, cols - 1] = np.int32(int(Gh[rows - 1, cols - 1]) - 40 * 512 if Gh[rows - 1, cols - 1] > 0 else int(Gh[rows - 1, cols - 1]) + 40 * 512)
    G[rows - 1, cols - 1] = int(Gh[rows - 1, cols - 1])
    if gated:
        Uh[0, 0] = np.int32(int(Uh[0, 0]) - 40 * 512 if Uh[0, 0] > 0 else int(Uh[0, 0]) + 40 * 512)
        U[0, 0] = int(Uh[0, 0])
    assert result(imm.gated_link_check(G, U, H, act, *par)) == glue.gated_link_check(Gh, Uh, Hh, act, *par)


@pytest.mark.parametrize("name", ["silu", "relu", "identity", "random"])
@pytest.mark.parametrize("shift,rnd,shift2,rnd2,lo,hi", [(9, 256, 7, 64, -127, 127), (0, 0, 0, 0, -128, 127), (4, 8, 14, 1 << 13, -1, 1),
                                                         (16, 1 << 15, 6, 0, 0, 100), (30, 5, 7, 127, -128, 127)])
def test_gated_link_other_tables_and_parameters(imm, glue, name, shift, rnd, shift2, rnd2, lo, hi):
    rng = np.random.default_rng(shift * 100 + shift2)
    act = act_tables()[name]
    Gh, Uh = edge_heavy(rng, 130, 1040, shift, -128, 127), edge_heavy(rng, 130, 1040, shift, -128, 127)
    par = (shift, rnd, shift2, rnd2, lo, hi)
    Hh = glue.gated_link(Gh, Uh, act, *par)
    G, U, H = (torch.from_numpy(x).cuda() for x in (Gh, Uh, Hh))
    assert result(imm.gated_link_check(G, U, H, act, *par)) == (0, -1)
    # the same H against another table, and with gate and up swapped: differs where the oracle says
    other = act_tables()["relu" if name != "relu" else "silu"]
    assert result(imm.gated_link_check(G, U, H, other, *par)) == glue.gated_link_check(Gh, Uh, Hh, other, *par)
    assert result(imm.gated_link_check(U, G, H, act, *par)) == glue.gated_link_check(Uh, Gh, Hh, act, *par)
    # the activation alone
    Ah = glue.gated_link(Gh, None, act, *par)
    assert result(imm.gated_link_check(G, None, torch.from_numpy(Ah).cuda(), act, shift, rnd)) == (0, -1)
    assert result(imm.gated_link_check(G, None, H, act, shift, rnd)) == glue.gated_link_check(Gh, None, Hh, act, *par)


def test_gated_ffn_link_at_full_size(imm, glue, synth):
    """Gate and up projections of the FFN at 2048 tokens (two int32 outputs of 2048 x 14336) against the
    hidden activations the oracle derives from them; one altered entry is found where it is."""
    up, down = synth.ffn_pair(1, device="cuda")
    G = up.C
    U = torch.roll(up.C, shifts=(1, 7), dims=(0, 1)).contiguous()      # a second accumulator matrix of the same statistics
    act = act_tables()["silu"]
    par = (9, 256, 7, 64, -127, 127)
    Gh, Uh = G.cpu().numpy(), U.cpu().numpy()
    Hh = glue.gated_link(Gh, Uh, act, *par)
    assert len(np.unique(Hh)) > 50                                     # a real spread of values, not a saturated matrix
    H = torch.from_numpy(Hh).cuda()
    out = torch.empty(2, dtype=torch.int64, device="cuda")
    assert result(imm.gated_link_check(G, U, H, act, *par, out=out)) == (0, -1)
    H[2047, 14335] += 1
    H[100, 3] -= 1
    assert result(imm.gated_link_check(G, U, H, act, *par, out=out)) == (2, 100 * 14336 + 3)


def test_gated_link_check_refuses_bad_arguments(imm):
    L = imm.lib()
    import ctypes
    G = torch.zeros((4, 8), dtype=torch.int32, device="cuda")
    H = torch.zeros((4, 8), dtype=torch.int8, device="cuda")
    out = torch.zeros(2, dtype=torch.int64, device="cuda")
    table = (ctypes.c_int8 * 256)()
    t = ctypes.addressof(table)
    call = L.imm_gated_link_check
    ok = (G.data_ptr(), G.data_ptr(), H.data_ptr(), 4, 8, 8, 8, 8, t)
    assert call(*ok, 9, 256, 7, 64, -127, 127, out.data_ptr(), None) == 0
    assert call(None, G.data_ptr(), H.data_ptr(), 4, 8, 8, 8, 8, t, 9, 256, 7, 64, -127, 127, out.data_ptr(), None) == imm.ERR_ARG
    assert call(G.data_ptr(), G.data_ptr(), H.data_ptr(), 4, 8, 8, 8, 8, None, 9, 256, 7, 64, -127, 127, out.data_ptr(), None) == imm.ERR_ARG
    assert call(*ok, 9, 512, 7, 64, -127, 127, out.data_ptr(), None) == imm.ERR_ARG          # rnd >= 2^shift
    assert call(*ok, 9, 256, 15, 64, -127, 127, out.data_ptr(), None) == imm.ERR_ARG         # shift2 > 14
    assert call(*ok, 9, 256, 7, 128, -127, 127, out.data_ptr(), None) == imm.ERR_ARG         # rnd2 >= 2^shift2
    assert call(*ok, 9, 256, 7, 64, 5, 4, out.data_ptr(), None) == imm.ERR_ARG               # lo > hi
    assert call(G.data_ptr(), G.data_ptr(), H.data_ptr(), 4, 8, 7, 8, 8, t, 9, 256, 7, 64, -127, 127, out.data_ptr(), None) == imm.ERR_SHAPE
    assert call(G.data_ptr(), G.data_ptr(), H.data_ptr(), 0, 8, 8, 8, 8, t, 9, 256, 7, 64, -127, 127, out.data_ptr(), None) == imm.ERR_SHAPE
    assert call(*ok, 9, 256, 7, 64, -127, 127, out.data_ptr() + 4, None) == imm.ERR_ALIGN
    # without U the second stage's parameters are ignored
    assert call(G.data_ptr(), None, H.data_ptr(), 4, 8, 8, 8, 8, t, 9, 256, 99, -5, 7, 3, out.data_ptr(), None) == 0
    torch.cuda.synchronize()

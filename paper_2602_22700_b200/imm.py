"""Thin binding of the C-ABI CUDA library ``libimm.so`` (see ``include/imm.h``).

Argument marshalling only: every function here checks tensor dtypes/devices, takes raw
pointers and calls the library entry point of the same name.  PyTorch supplies device memory
and the current stream, nothing else.  There is no CPU fallback: if the library is missing or
a tensor is not on a CUDA device the call raises.
"""
from __future__ import annotations

import ctypes
import os
from typing import List, Optional, Sequence, Tuple

import torch

P = 0xFFFFFFFF00000001
OK, REJECT = 0, 1
ERR_ARG, ERR_SHAPE, ERR_ALIGN, ERR_WORKSPACE, ERR_NONCANONICAL, ERR_CUDA, ERR_TIMEOUT, ERR_LIMIT = -1, -2, -3, -4, -5, -6, -7, -8
I8, I32 = 0, 1
BIND_ROWS, BIND_COLS = 0, 1
FIELD_ADD, FIELD_SUB, FIELD_MUL = 0, 1, 2
ERRORS = {-8: "IMM_ERR_LIMIT", -7: "IMM_ERR_TIMEOUT", -1: "IMM_ERR_ARG", -2: "IMM_ERR_SHAPE", -3: "IMM_ERR_ALIGN", -4: "IMM_ERR_WORKSPACE",
          -5: "IMM_ERR_NONCANONICAL", -6: "IMM_ERR_CUDA"}

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libimm.so")

EXPORTS = ("imm_version", "imm_last_cuda_error", "imm_challenge", "imm_field_binop", "imm_eq_table",
           "imm_mle_workspace", "imm_mle_partial_eval", "imm_mle_eval_point",
           "imm_sumcheck_matmul_workspace", "imm_sumcheck_matmul_prove",
           "imm_sumcheck_matmul_host_arena", "imm_sumcheck_matmul_prove_host", "imm_sumcheck_verify",
           "imm_profile_enable", "imm_profile_calls", "imm_profile_read", "imm_mle_eval_point_noalloc",
           "imm_ldd_tv_kl", "imm_ldd_topk_workspace", "imm_ldd_topk_distance", "imm_ldd_tail_fraction",
           "imm_sumcheck_batched_transcript_len", "imm_sumcheck_matmul_batched_workspace",
           "imm_sumcheck_matmul_prove_batched", "imm_sumcheck_verify_batched",
           "imm_commit_workspace", "imm_commit", "imm_commit_launches",
           "imm_sumcheck_matmul_fs_workspace", "imm_sumcheck_matmul_prove_fs", "imm_fs_challenges",
           "imm_sumcheck_verify_fs", "imm_sumcheck_expected_workspace", "imm_sumcheck_expected",
           "imm_sumcheck_matmul_fs_batched_workspace", "imm_sumcheck_matmul_prove_fs_batched",
           "imm_fs_batched_challenges", "imm_sumcheck_verify_fs_batched", "imm_requant_check", "imm_sumcheck_matmul_launches",
           "imm_gated_link_check")
FS_BATCH_MAX = 1024
COMMIT_LEAF = 4096
NOALLOC_MAX_TILES = 8192
PROFILE_PHASES = ("eq_tables", "claim_C", "bind_rows_A", "bind_cols_B", "sumcheck_rounds")


class ImmError(RuntimeError):
    def __init__(self, code: int, where: str, detail: str = ""):
        self.code = code
        super().__init__(f"{where}: {ERRORS.get(code, code)}" + (f" ({detail})" if detail else ""))


class CommitDesc(ctypes.Structure):
    _fields_ = [("msg", ctypes.c_void_p), ("nbytes", ctypes.c_uint64), ("r", ctypes.c_uint8 * 32),
                ("r_len", ctypes.c_int32), ("reserved", ctypes.c_int32)]


class MatmulDesc(ctypes.Structure):
    _fields_ = [("A", ctypes.c_void_p), ("B", ctypes.c_void_p), ("C", ctypes.c_void_p),
                ("m", ctypes.c_int64), ("k", ctypes.c_int64), ("n", ctypes.c_int64),
                ("lda", ctypes.c_int64), ("ldb", ctypes.c_int64), ("ldc", ctypes.c_int64),
                ("proof_id", ctypes.c_uint64)]


_lib = None


def lib() -> ctypes.CDLL:
    """Load libimm.so (built in-tree by ``paper_2602_22700_b200.build``); raises if absent."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise ImportError(f"{LIB_PATH} is missing: build it with `python -m paper_2602_22700_b200.build`; "
                          "there is no fallback path")
    L = ctypes.CDLL(LIB_PATH)
    vp, u64, i64, ci, sz = ctypes.c_void_p, ctypes.c_uint64, ctypes.c_int64, ctypes.c_int, ctypes.c_size_t
    L.imm_version.restype = ci
    L.imm_last_cuda_error.restype = ctypes.c_char_p
    L.imm_challenge.restype = u64
    L.imm_challenge.argtypes = [u64, u64, ctypes.c_uint32, ctypes.c_uint32]
    L.imm_field_binop.restype = ci
    L.imm_field_binop.argtypes = [ci, vp, vp, vp, i64, vp]
    L.imm_eq_table.restype = ci
    L.imm_eq_table.argtypes = [vp, ci, vp, vp]
    L.imm_mle_workspace.restype = sz
    L.imm_mle_workspace.argtypes = [ci, i64, i64, ci]
    L.imm_mle_partial_eval.restype = ci
    L.imm_mle_partial_eval.argtypes = [vp, ci, i64, i64, i64, ci, vp, vp, vp, sz, vp]
    L.imm_mle_eval_point.restype = ci
    L.imm_mle_eval_point.argtypes = [vp, ci, i64, i64, i64, vp, vp, vp, vp, sz, vp]
    L.imm_mle_eval_point_noalloc.restype = ci
    L.imm_mle_eval_point_noalloc.argtypes = [vp, ci, i64, i64, i64, vp, vp, vp, vp]
    L.imm_sumcheck_matmul_workspace.restype = sz
    L.imm_sumcheck_matmul_workspace.argtypes = [vp, ci]
    L.imm_sumcheck_matmul_prove.restype = ci
    L.imm_sumcheck_matmul_prove.argtypes = [vp, ci, u64, vp, i64, vp, vp, sz, vp]
    L.imm_sumcheck_matmul_host_arena.restype = sz
    L.imm_sumcheck_matmul_host_arena.argtypes = [vp, ci]
    L.imm_sumcheck_matmul_prove_host.restype = ci
    L.imm_sumcheck_matmul_prove_host.argtypes = [vp, ci, u64, vp, i64, vp, vp, sz, vp]
    L.imm_profile_enable.restype = ci
    L.imm_profile_enable.argtypes = [ci]
    L.imm_profile_calls.restype = i64
    L.imm_profile_calls.argtypes = []
    L.imm_profile_read.restype = ci
    L.imm_profile_read.argtypes = [i64, vp, ci]
    L.imm_ldd_tv_kl.restype = ci
    L.imm_ldd_tv_kl.argtypes = [vp, vp, i64, i64, i64, vp, vp, vp]
    L.imm_ldd_topk_distance.restype = ci
    L.imm_ldd_topk_distance.argtypes = [vp, i64, i64, i64, vp, ci, vp, vp, vp, sz, vp]
    L.imm_ldd_topk_workspace.restype = sz
    L.imm_ldd_topk_workspace.argtypes = [i64, i64, ci]
    L.imm_ldd_tail_fraction.restype = ci
    L.imm_ldd_tail_fraction.argtypes = [vp, vp, i64, ctypes.c_double, ctypes.c_double, vp, vp, vp]
    L.imm_sumcheck_verify.restype = ci
    L.imm_sumcheck_verify.argtypes = [vp, ci, u64, u64, vp, vp, vp, vp]
    L.imm_sumcheck_batched_transcript_len.restype = i64
    L.imm_sumcheck_batched_transcript_len.argtypes = [ci, ci]
    L.imm_sumcheck_matmul_batched_workspace.restype = sz
    L.imm_sumcheck_matmul_batched_workspace.argtypes = [vp, ci]
    L.imm_sumcheck_matmul_prove_batched.restype = ci
    L.imm_sumcheck_matmul_prove_batched.argtypes = [vp, ci, u64, u64, vp, vp, vp, sz, vp]
    L.imm_sumcheck_matmul_fs_workspace.restype = sz
    L.imm_sumcheck_matmul_fs_workspace.argtypes = [vp, ci]
    L.imm_sumcheck_matmul_prove_fs.restype = ci
    L.imm_sumcheck_matmul_prove_fs.argtypes = [vp, ci, vp, vp, i64, vp, vp, sz, vp]
    L.imm_fs_challenges.restype = ci
    L.imm_fs_challenges.argtypes = [vp, ci, vp, i64, i64, i64, u64, vp, vp, vp]
    L.imm_sumcheck_verify_fs.restype = ci
    L.imm_sumcheck_verify_fs.argtypes = [vp, ci, vp, i64, i64, i64, u64, vp, vp, vp, vp]
    L.imm_sumcheck_matmul_fs_batched_workspace.restype = sz
    L.imm_sumcheck_matmul_fs_batched_workspace.argtypes = [vp, ci]
    L.imm_sumcheck_matmul_prove_fs_batched.restype = ci
    L.imm_sumcheck_matmul_prove_fs_batched.argtypes = [vp, ci, vp, u64, vp, vp, vp, sz, vp]
    L.imm_fs_batched_challenges.restype = ci
    L.imm_fs_batched_challenges.argtypes = [vp, ci, vp, ci, vp, u64, vp, vp]
    L.imm_sumcheck_verify_fs_batched.restype = ci
    L.imm_sumcheck_verify_fs_batched.argtypes = [vp, ci, vp, ci, vp, u64, vp, vp]
    L.imm_sumcheck_expected_workspace.restype = sz
    L.imm_sumcheck_expected_workspace.argtypes = [vp, ci, ci]
    L.imm_sumcheck_expected.restype = ci
    L.imm_sumcheck_expected.argtypes = [vp, ci, u64, vp, vp, vp, vp, vp, sz, vp]
    L.imm_commit_launches.restype = ci
    L.imm_commit_launches.argtypes = [vp, ci]
    L.imm_commit_workspace.restype = sz
    L.imm_commit_workspace.argtypes = [vp, ci]
    L.imm_commit.restype = ci
    L.imm_commit.argtypes = [vp, ci, vp, vp, vp, sz, vp]
    L.imm_sumcheck_verify_batched.restype = ci
    L.imm_sumcheck_verify_batched.argtypes = [vp, ci, ci, u64, u64, vp, vp]
    L.imm_sumcheck_matmul_launches.restype = ci
    L.imm_sumcheck_matmul_launches.argtypes = [vp, ci]
    L.imm_requant_check.restype = ci
    L.imm_requant_check.argtypes = [vp, vp, i64, i64, i64, i64, ci, ctypes.c_int32, ctypes.c_int32, ctypes.c_int32, vp, vp]
    L.imm_gated_link_check.restype = ci
    L.imm_gated_link_check.argtypes = [vp, vp, vp, i64, i64, i64, i64, i64, vp, ci, ctypes.c_int32, ci, ctypes.c_int32,
                                       ctypes.c_int32, ctypes.c_int32, vp, vp]
    _lib = L
    return L


def _check(rc: int, where: str):
    if rc < 0:
        detail = lib().imm_last_cuda_error().decode() if rc == -6 else ""
        raise ImmError(rc, where, detail)
    return rc


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


def _cuda(t: torch.Tensor, dtype, what: str) -> torch.Tensor:
    if not isinstance(t, torch.Tensor) or t.device.type != "cuda":
        raise ValueError(f"{what} must be a CUDA tensor (no CPU path exists)")
    if t.dtype != dtype:
        raise ValueError(f"{what} must have dtype {dtype}, got {t.dtype}")
    return t


def _matrix(t: torch.Tensor, what: str, device="cuda") -> Tuple[int, int, int, int, int]:
    """(ptr, dtype code, rows, cols, ld) of a 2-D int8/int32 tensor with contiguous rows."""
    if t.dim() != 2 or t.dtype not in (torch.int8, torch.int32):
        raise ValueError(f"{what} must be a 2-D int8 or int32 tensor")
    if t.device.type != device:
        raise ValueError(f"{what} must live on {device}")
    rows, cols = t.shape
    if cols > 1 and t.stride(1) != 1:
        raise ValueError(f"{what} must have unit column stride")
    ld = t.stride(0) if rows > 1 else max(cols, 1)
    return t.data_ptr(), (I8 if t.dtype == torch.int8 else I32), rows, cols, ld


def ceil_log2(d: int) -> int:
    return max(0, (int(d) - 1).bit_length())


def transcript_len(k: int) -> int:
    return 3 * ceil_log2(k) + 3


def version() -> int:
    return lib().imm_version()


def challenge(seed: int, proof_id: int, domain: int, index: int) -> int:
    return lib().imm_challenge(seed, proof_id, domain, index)


def challenges(seed: int, proof_id: int, domain: int, count: int) -> List[int]:
    return [challenge(seed, proof_id, domain, i) for i in range(count)]


def field_binop(op: int, x: torch.Tensor, y: torch.Tensor) -> torch.Tensor:
    """Element-wise field add/sub/mul of two int64 CUDA tensors holding canonical bit patterns."""
    _cuda(x, torch.int64, "x"); _cuda(y, torch.int64, "y")
    x, y = x.contiguous(), y.contiguous()
    assert x.numel() == y.numel()
    out = torch.empty_like(x)
    _check(lib().imm_field_binop(op, x.data_ptr(), y.data_ptr(), out.data_ptr(), x.numel(), _stream()),
           "imm_field_binop")
    return out


def eq_table(r: Sequence[int], device="cuda") -> torch.Tensor:
    """E[i] = eq(r, i) as an int64 CUDA tensor of 2^len(r) canonical bit patterns."""
    n = len(r)
    arr = (ctypes.c_uint64 * max(n, 1))(*[int(v) for v in r])
    out = torch.empty(1 << min(n, 24), dtype=torch.int64, device=device)
    _check(lib().imm_eq_table(ctypes.addressof(arr), n, out.data_ptr(), _stream()), "imm_eq_table")
    return out


def mle_workspace(dtype_code: int, rows: int, cols: int, bind: int) -> int:
    return lib().imm_mle_workspace(dtype_code, rows, cols, bind)


def mle_partial_eval(mat: torch.Tensor, bind: int, eq: torch.Tensor,
                     ws: Optional[torch.Tensor] = None) -> torch.Tensor:
    ptr, code, rows, cols, ld = _matrix(mat, "mat")
    _cuda(eq, torch.int64, "eq")
    need = mle_workspace(code, rows, cols, bind)
    if ws is None:
        ws = torch.empty(max(need, 16), dtype=torch.uint8, device=mat.device)
    out = torch.empty(cols if bind == BIND_ROWS else rows, dtype=torch.int64, device=mat.device)
    _check(lib().imm_mle_partial_eval(ptr, code, rows, cols, ld, bind, eq.data_ptr(), out.data_ptr(),
                                      ws.data_ptr(), ws.numel(), _stream()), "imm_mle_partial_eval")
    return out


def mle_eval_point(mat: torch.Tensor, eq_row: torch.Tensor, eq_col: torch.Tensor,
                   ws: Optional[torch.Tensor] = None) -> torch.Tensor:
    ptr, code, rows, cols, ld = _matrix(mat, "mat")
    _cuda(eq_row, torch.int64, "eq_row"); _cuda(eq_col, torch.int64, "eq_col")
    need = mle_workspace(code, rows, cols, BIND_ROWS)
    if ws is None:
        ws = torch.empty(max(need, 16), dtype=torch.uint8, device=mat.device)
    out = torch.empty(1, dtype=torch.int64, device=mat.device)
    _check(lib().imm_mle_eval_point(ptr, code, rows, cols, ld, eq_row.data_ptr(), eq_col.data_ptr(),
                                    out.data_ptr(), ws.data_ptr(), ws.numel(), _stream()),
           "imm_mle_eval_point")
    return out


def mle_eval_point_noalloc(mat: torch.Tensor, eq_row: torch.Tensor, eq_col: torch.Tensor,
                           out: torch.Tensor) -> torch.Tensor:
    """Point evaluation for callers that cannot allocate device memory: no workspace, the
    partial sums live in a fixed array inside the library (see imm.h for capacity and the
    sharing rules).  ``out`` is a caller-provided 1-element int64 CUDA tensor."""
    ptr, code, rows, cols, ld = _matrix(mat, "mat")
    _cuda(eq_row, torch.int64, "eq_row"); _cuda(eq_col, torch.int64, "eq_col"); _cuda(out, torch.int64, "out")
    _check(lib().imm_mle_eval_point_noalloc(ptr, code, rows, cols, ld, eq_row.data_ptr(), eq_col.data_ptr(),
                                            out.data_ptr(), _stream()), "imm_mle_eval_point_noalloc")
    return out


def make_descs(problems, device="cuda"):
    """ctypes descriptor array for (A, B, C, proof_id) tuples; tensors must stay alive."""
    arr = (MatmulDesc * len(problems))()
    for i, (A, B, C, pid) in enumerate(problems):
        pa, ca, m, k, lda = _matrix(A, "A", device)
        pb, cb, k2, n, ldb = _matrix(B, "B", device)
        pc, cc, m2, n2, ldc = _matrix(C, "C", device)
        if ca != I8 or cb != I8 or cc != I32 or k != k2 or m != m2 or n != n2:
            raise ValueError("need A int8 m x k, B int8 k x n, C int32 m x n")
        arr[i] = MatmulDesc(pa, pb, pc, m, k, n, lda, ldb, ldc, int(pid))
    return arr


def sumcheck_matmul_workspace(descs) -> int:
    return lib().imm_sumcheck_matmul_workspace(ctypes.addressof(descs), len(descs))


def _launch_counts(descs) -> Tuple[int, int]:
    """(launches of a plain proving pass, launches of its contraction side alone) for this batch: 3 and 1
    when it takes the fused contraction launch, else 5 and 4 (eq tables + three contractions)."""
    plain = lib().imm_sumcheck_matmul_launches(ctypes.addressof(descs), len(descs))
    return plain, (1 if plain == 3 else 4)


class Prover:
    """Holds the descriptor array, workspace and output buffers of one batch so that repeated
    ``prove`` calls do no allocation.  ``problems``: list of (A, B, C, proof_id) CUDA tensors."""

    def __init__(self, problems, device="cuda"):
        self.problems = list(problems)
        self.descs = make_descs(self.problems)
        self.nproofs = len(self.problems)
        self.stride = max(transcript_len(A.shape[1]) for (A, _, _, _) in self.problems)
        need = sumcheck_matmul_workspace(self.descs)
        if need == 0:
            raise ImmError(-2, "imm_sumcheck_matmul_workspace")
        self.ws = torch.empty(need, dtype=torch.uint8, device=device)
        self.transcripts = torch.zeros((self.nproofs, self.stride), dtype=torch.int64, device=device)
        self.status = torch.full((self.nproofs,), -99, dtype=torch.int32, device=device)
        self.launches = _launch_counts(self.descs)[0]

    def prove(self, seed: int) -> torch.Tensor:
        """Enqueue one proving pass on the current stream; returns the device transcript tensor."""
        _check(lib().imm_sumcheck_matmul_prove(ctypes.addressof(self.descs), self.nproofs, seed,
                                               self.transcripts.data_ptr(), self.stride,
                                               self.status.data_ptr(), self.ws.data_ptr(),
                                               self.ws.numel(), _stream()), "imm_sumcheck_matmul_prove")
        return self.transcripts

    def lengths(self) -> List[int]:
        return [transcript_len(A.shape[1]) for (A, _, _, _) in self.problems]


def sumcheck_matmul_prove(problems, seed: int) -> List[List[int]]:
    """Convenience: prove a batch and return each proof's transcript as Python ints (synchronises)."""
    pr = Prover(problems)
    t = pr.prove(seed)
    torch.cuda.synchronize()
    if int(pr.status.abs().max()) != 0:
        raise ImmError(int(pr.status.min()), "device status")
    host = t.cpu()
    return [[int(v) & 0xFFFFFFFFFFFFFFFF for v in host[i, :n]] for i, n in enumerate(pr.lengths())]


class HostProver:
    """End-to-end variant: matrices live in (pinned) HOST tensors; every ``prove`` copies them to a
    device arena, proves, and copies the transcripts back (synchronous)."""

    def __init__(self, problems, device="cuda"):
        self.problems = list(problems)
        self.descs = make_descs(self.problems, device="cpu")
        self.nproofs = len(self.problems)
        self.stride = max(transcript_len(A.shape[1]) for (A, _, _, _) in self.problems)
        need = lib().imm_sumcheck_matmul_host_arena(ctypes.addressof(self.descs), self.nproofs)
        if need == 0:
            raise ImmError(-2, "imm_sumcheck_matmul_host_arena")
        self.arena = torch.empty(need, dtype=torch.uint8, device=device)
        self.transcripts = torch.zeros((self.nproofs, self.stride), dtype=torch.int64).pin_memory()
        self.status = torch.full((self.nproofs,), -99, dtype=torch.int32).pin_memory()
        self.h2d_bytes = sum(A.numel() + B.numel() + 4 * C.numel() for (A, B, C, _) in self.problems)
        self.d2h_bytes = self.transcripts.numel() * 8 + self.status.numel() * 4

    def prove(self, seed: int) -> torch.Tensor:
        _check(lib().imm_sumcheck_matmul_prove_host(ctypes.addressof(self.descs), self.nproofs, seed,
                                                    self.transcripts.data_ptr(), self.stride,
                                                    self.status.data_ptr(), self.arena.data_ptr(),
                                                    self.arena.numel(), _stream()),
               "imm_sumcheck_matmul_prove_host")
        return self.transcripts


def profile_enable(capacity: int) -> None:
    """Create a ring of `capacity` per-call event sets (0 switches phase timing off)."""
    _check(lib().imm_profile_enable(int(capacity)), "imm_profile_enable")


def profile_calls() -> int:
    return lib().imm_profile_calls()


def profile_read(call: int) -> List[float]:
    """Milliseconds per phase (PROFILE_PHASES order) of profiled prove call `call`; waits for it."""
    buf = (ctypes.c_float * len(PROFILE_PHASES))()
    _check(lib().imm_profile_read(int(call), ctypes.addressof(buf), len(PROFILE_PHASES)), "imm_profile_read")
    return [float(v) for v in buf]


def sumcheck_verify(transcript: Sequence[int], nrounds: int, seed: int, proof_id: int,
                    expect_c0: Optional[int] = None, expect_a_fin: Optional[int] = None,
                    expect_b_fin: Optional[int] = None) -> Tuple[int, int]:
    """Host verifier; returns (status, fail_at)."""
    n = 3 * nrounds + 3
    arr = (ctypes.c_uint64 * n)(*[int(v) & 0xFFFFFFFFFFFFFFFF for v in list(transcript)[:n]])
    keep = []

    def opt(v):
        if v is None:
            return None
        box = ctypes.c_uint64(int(v))
        keep.append(box)
        return ctypes.addressof(box)

    fail = ctypes.c_int(-2)
    rc = lib().imm_sumcheck_verify(ctypes.addressof(arr), nrounds, seed, proof_id, opt(expect_c0),
                                   opt(expect_a_fin), opt(expect_b_fin), ctypes.addressof(fail))
    _check(rc, "imm_sumcheck_verify")
    return rc, fail.value


# ------------------------------------------------------------------ batched proof


def batched_transcript_len(nrounds: int, nproofs: int) -> int:
    return lib().imm_sumcheck_batched_transcript_len(nrounds, nproofs)


class BatchedProver:
    """One sumcheck for a random linear combination of product claims (every k padded to the largest
    2^b).  Holds descriptors, workspace and outputs; ``prove`` allocates nothing."""

    def __init__(self, problems, device="cuda"):
        self.problems = list(problems)
        self.descs = make_descs(self.problems)
        self.nproofs = len(self.problems)
        self.nrounds = max(ceil_log2(A.shape[1]) for (A, _, _, _) in self.problems)
        need = lib().imm_sumcheck_matmul_batched_workspace(ctypes.addressof(self.descs), self.nproofs)
        if need == 0:
            raise ImmError(ERR_SHAPE, "imm_sumcheck_matmul_batched_workspace")
        self.ws = torch.empty(need, dtype=torch.uint8, device=device)
        self.length = batched_transcript_len(self.nrounds, self.nproofs)
        self.transcript = torch.zeros((self.length,), dtype=torch.int64, device=device)
        self.status = torch.full((self.nproofs,), -99, dtype=torch.int32, device=device)
        self.launches = _launch_counts(self.descs)[0] + 1        # ... and the combining launch

    def prove(self, seed: int, batch_id: int) -> torch.Tensor:
        """Enqueue one batched proving pass on the current stream; returns the device transcript."""
        _check(lib().imm_sumcheck_matmul_prove_batched(ctypes.addressof(self.descs), self.nproofs, seed,
                                                       batch_id, self.transcript.data_ptr(),
                                                       self.status.data_ptr(), self.ws.data_ptr(),
                                                       self.ws.numel(), _stream()),
               "imm_sumcheck_matmul_prove_batched")
        return self.transcript


def sumcheck_matmul_prove_batched(problems, seed: int, batch_id: int) -> List[int]:
    """Convenience: one batched proof as Python ints (synchronises)."""
    pr = BatchedProver(problems)
    t = pr.prove(seed, batch_id)
    torch.cuda.synchronize()
    if int(pr.status.abs().max()) != 0:
        raise ImmError(int(pr.status.min()), "device status")
    return [int(v) & 0xFFFFFFFFFFFFFFFF for v in t.cpu()]


def sumcheck_verify_batched(transcript: Sequence[int], nrounds: int, nproofs: int, seed: int,
                            batch_id: int, expect: Optional[Sequence[int]] = None) -> Tuple[int, int]:
    """Host verifier of a batched transcript; returns (status, fail_at)."""
    n = 1 + 3 * nrounds + 3 * nproofs
    words = [int(v) & 0xFFFFFFFFFFFFFFFF for v in list(transcript)[:n]]
    if len(words) != n:
        raise ValueError("transcript too short")
    arr = (ctypes.c_uint64 * n)(*words)
    exp = None
    if expect is not None:
        if len(expect) != 3 * nproofs:
            raise ValueError("expect must hold 3 words per proof")
        exp = (ctypes.c_uint64 * (3 * nproofs))(*[int(v) & 0xFFFFFFFFFFFFFFFF for v in expect])
    fail = ctypes.c_int(-2)
    rc = lib().imm_sumcheck_verify_batched(ctypes.addressof(arr), nrounds, nproofs, seed, batch_id,
                                           None if exp is None else ctypes.addressof(exp),
                                           ctypes.addressof(fail))
    _check(rc, "imm_sumcheck_verify_batched")
    return rc, fail.value


# ------------------------------------------------------------------ hash commitments


class Committer:
    """Commitments c = Hash(m || r) to a batch of CUDA tensors (each tensor's bytes, which must be
    contiguous, are one message).  Holds descriptors, workspace and outputs; ``commit`` allocates
    nothing.  ``randomness``: None (no r for any message) or one 32-byte string (or None) per message."""

    def __init__(self, messages, randomness=None, device="cuda"):
        self.messages = list(messages)
        n = len(self.messages)
        if randomness is None:
            randomness = [None] * n
        if len(randomness) != n:
            raise ValueError("one randomness entry per message")
        self.descs = (CommitDesc * max(n, 1))()
        self.nbytes = 0
        for i, (t, r) in enumerate(zip(self.messages, randomness)):
            if not isinstance(t, torch.Tensor) or t.device.type != "cuda":
                raise ValueError("messages must be CUDA tensors (no CPU path exists)")
            if not t.is_contiguous():
                raise ValueError("a message must be contiguous")
            size = t.numel() * t.element_size()
            self.descs[i].msg = t.data_ptr() if size else None
            self.descs[i].nbytes = size
            self.nbytes += size
            if r is not None:
                if len(r) != 32:
                    raise ValueError("randomness must be 32 bytes")
                self.descs[i].r = (ctypes.c_uint8 * 32)(*bytes(r))
                self.descs[i].r_len = 32
        self.n = n
        self.launches = lib().imm_commit_launches(ctypes.addressof(self.descs), n)
        need = lib().imm_commit_workspace(ctypes.addressof(self.descs), n)
        if need == 0:
            raise ImmError(ERR_ARG, "imm_commit_workspace")
        self.ws = torch.empty(need, dtype=torch.uint8, device=device)
        self.digests = torch.zeros((n, 32), dtype=torch.uint8, device=device)
        self.roots = torch.zeros((n, 32), dtype=torch.uint8, device=device)

    def commit(self) -> torch.Tensor:
        """Enqueue the commitments on the current stream; returns the (n, 32) device tensor of digests."""
        _check(lib().imm_commit(ctypes.addressof(self.descs), self.n, self.digests.data_ptr(),
                                self.roots.data_ptr(), self.ws.data_ptr(), self.ws.numel(), _stream()),
               "imm_commit")
        return self.digests


def commit(messages, randomness=None) -> List[bytes]:
    """Convenience: commitments as bytes objects (synchronises)."""
    c = Committer(messages, randomness)
    d = c.commit().cpu().numpy()
    return [bytes(row) for row in d]


# ------------------------------------------------------------------ non-interactive proof


def commit_matrices(problems, randomness=None) -> torch.Tensor:
    """(nproofs, 96) uint8 CUDA tensor: the commitments to A, B and C of every problem, in that order
    (the statement of a non-interactive proof).  ``randomness``: None or one 32-byte string per matrix."""
    msgs = [t for (A, B, C, _) in problems for t in (A, B, C)]
    c = Committer(msgs, randomness)
    return c.commit().view(len(problems), 96)


class FsProver:
    """Non-interactive prover: challenges hashed from the commitments and the transcript."""

    def __init__(self, problems, commitments: torch.Tensor, device="cuda"):
        self.problems = list(problems)
        self.descs = make_descs(self.problems)
        self.nproofs = len(self.problems)
        self.commitments = _cuda(commitments, torch.uint8, "commitments").contiguous()
        if self.commitments.numel() != 96 * self.nproofs:
            raise ValueError("commitments must hold 96 bytes per proof")
        self.stride = max(transcript_len(A.shape[1]) for (A, _, _, _) in self.problems)
        need = lib().imm_sumcheck_matmul_fs_workspace(ctypes.addressof(self.descs), self.nproofs)
        if need == 0:
            raise ImmError(ERR_SHAPE, "imm_sumcheck_matmul_fs_workspace")
        self.ws = torch.empty(need, dtype=torch.uint8, device=device)
        self.transcripts = torch.zeros((self.nproofs, self.stride), dtype=torch.int64, device=device)
        self.status = torch.full((self.nproofs,), -99, dtype=torch.int32, device=device)
        self.launches = _launch_counts(self.descs)[1] + 2        # statements, contractions, hashed rounds

    def prove(self) -> torch.Tensor:
        _check(lib().imm_sumcheck_matmul_prove_fs(ctypes.addressof(self.descs), self.nproofs,
                                                  self.commitments.data_ptr(), self.transcripts.data_ptr(),
                                                  self.stride, self.status.data_ptr(), self.ws.data_ptr(),
                                                  self.ws.numel(), _stream()), "imm_sumcheck_matmul_prove_fs")
        return self.transcripts

    def lengths(self) -> List[int]:
        return [transcript_len(A.shape[1]) for (A, _, _, _) in self.problems]


def sumcheck_matmul_prove_fs(problems, commitments: torch.Tensor) -> List[List[int]]:
    """Convenience: non-interactive transcripts as Python ints (synchronises)."""
    pr = FsProver(problems, commitments)
    t = pr.prove()
    torch.cuda.synchronize()
    if int(pr.status.abs().max()) != 0:
        raise ImmError(int(pr.status.min()), "device status")
    host = t.cpu()
    return [[int(v) & 0xFFFFFFFFFFFFFFFF for v in host[i, :n]] for i, n in enumerate(pr.lengths())]


def _com96(commitments) -> "ctypes.Array":
    data = bytes(commitments)
    if len(data) != 96:
        raise ValueError("the statement's commitments are 96 bytes")
    return (ctypes.c_uint8 * 96)(*data)


def fs_challenges(transcript: Optional[Sequence[int]], nrounds: int, commitments, m: int, k: int, n: int,
                  proof_id: int) -> Tuple[List[int], List[int], List[int]]:
    """(r_row, r_col, r_k) as the verifier of a non-interactive proof derives them (r_k empty when no
    transcript is given)."""
    com = _com96(commitments)
    a, c = ceil_log2(m), ceil_log2(n)
    rr, rc_, rk = (ctypes.c_uint64 * max(a, 1))(), (ctypes.c_uint64 * max(c, 1))(), (ctypes.c_uint64 * max(nrounds, 1))()
    arr = None
    if transcript is not None:
        words = [int(v) & 0xFFFFFFFFFFFFFFFF for v in list(transcript)[:3 * nrounds + 1]]
        arr = (ctypes.c_uint64 * len(words))(*words)
    _check(lib().imm_fs_challenges(None if arr is None else ctypes.addressof(arr), nrounds, ctypes.addressof(com),
                                   m, k, n, proof_id, ctypes.addressof(rr), ctypes.addressof(rc_),
                                   None if arr is None else ctypes.addressof(rk)), "imm_fs_challenges")
    return list(rr)[:a], list(rc_)[:c], (list(rk)[:nrounds] if arr is not None else [])


def sumcheck_verify_fs(transcript: Sequence[int], nrounds: int, commitments, m: int, k: int, n: int, proof_id: int,
                       expect_c0: Optional[int] = None, expect_a_fin: Optional[int] = None,
                       expect_b_fin: Optional[int] = None) -> Tuple[int, int]:
    """Host verifier of a non-interactive proof; returns (status, fail_at)."""
    cnt = 3 * nrounds + 3
    arr = (ctypes.c_uint64 * cnt)(*[int(v) & 0xFFFFFFFFFFFFFFFF for v in list(transcript)[:cnt]])
    com = _com96(commitments)
    keep = []

    def opt(v):
        if v is None:
            return None
        box = ctypes.c_uint64(int(v))
        keep.append(box)
        return ctypes.addressof(box)

    fail = ctypes.c_int(-2)
    rc = lib().imm_sumcheck_verify_fs(ctypes.addressof(arr), nrounds, ctypes.addressof(com), m, k, n, proof_id,
                                      opt(expect_c0), opt(expect_a_fin), opt(expect_b_fin), ctypes.addressof(fail))
    _check(rc, "imm_sumcheck_verify_fs")
    return rc, fail.value


class FsBatchedProver:
    """One non-interactive proof for all products of a batch (at most FS_BATCH_MAX members)."""

    def __init__(self, problems, commitments: torch.Tensor, device="cuda"):
        self.problems = list(problems)
        self.descs = make_descs(self.problems)
        self.nproofs = len(self.problems)
        self.commitments = _cuda(commitments, torch.uint8, "commitments").contiguous()
        if self.commitments.numel() != 96 * self.nproofs:
            raise ValueError("commitments must hold 96 bytes per proof")
        self.nrounds = max(ceil_log2(A.shape[1]) for (A, _, _, _) in self.problems)
        need = lib().imm_sumcheck_matmul_fs_batched_workspace(ctypes.addressof(self.descs), self.nproofs)
        if need == 0:
            raise ImmError(ERR_LIMIT if self.nproofs > FS_BATCH_MAX else ERR_SHAPE,
                           "imm_sumcheck_matmul_fs_batched_workspace")
        self.ws = torch.empty(need, dtype=torch.uint8, device=device)
        self.length = batched_transcript_len(self.nrounds, self.nproofs)
        self.transcript = torch.zeros((self.length,), dtype=torch.int64, device=device)
        self.status = torch.full((self.nproofs,), -99, dtype=torch.int32, device=device)
        self.launches = _launch_counts(self.descs)[1] + 1 + 3 + 2 * self.nrounds     # statements, contractions, the round chain

    def prove(self, batch_id: int) -> torch.Tensor:
        _check(lib().imm_sumcheck_matmul_prove_fs_batched(ctypes.addressof(self.descs), self.nproofs,
                                                          self.commitments.data_ptr(), batch_id,
                                                          self.transcript.data_ptr(), self.status.data_ptr(),
                                                          self.ws.data_ptr(), self.ws.numel(), _stream()),
               "imm_sumcheck_matmul_prove_fs_batched")
        return self.transcript


def sumcheck_matmul_prove_fs_batched(problems, commitments: torch.Tensor, batch_id: int) -> List[int]:
    """Convenience: the batched non-interactive transcript as Python ints (synchronises)."""
    pr = FsBatchedProver(problems, commitments)
    t = pr.prove(batch_id)
    torch.cuda.synchronize()
    if int(pr.status.abs().max()) != 0:
        raise ImmError(int(pr.status.min()), "device status")
    return [int(v) & 0xFFFFFFFFFFFFFFFF for v in t.cpu()]


def _shape_descs(shapes_and_ids):
    """Descriptor array that carries only m, k, n and proof_id (for the host functions)."""
    arr = (MatmulDesc * len(shapes_and_ids))()
    for i, (m, k, n, pid) in enumerate(shapes_and_ids):
        arr[i] = MatmulDesc(None, None, None, m, k, n, k, n, n, pid)
    return arr


def fs_batched_challenges(transcript: Optional[Sequence[int]], nrounds: int, shapes_and_ids, commitments,
                          batch_id: int) -> Tuple[List[int], List[int]]:
    """(rho, r_k) of a batched non-interactive proof; ``shapes_and_ids``: (m, k, n, proof_id) per member,
    ``commitments``: 96 bytes per member."""
    n = len(shapes_and_ids)
    descs = _shape_descs(shapes_and_ids)
    data = bytes(commitments)
    if len(data) != 96 * n:
        raise ValueError("96 commitment bytes per member")
    com = (ctypes.c_uint8 * len(data))(*data)
    rho, rk = (ctypes.c_uint64 * n)(), (ctypes.c_uint64 * max(nrounds, 1))()
    arr = None
    if transcript is not None:
        words = [int(v) & 0xFFFFFFFFFFFFFFFF for v in list(transcript)[:3 * nrounds + 1]]
        arr = (ctypes.c_uint64 * len(words))(*words)
    _check(lib().imm_fs_batched_challenges(None if arr is None else ctypes.addressof(arr), nrounds,
                                           ctypes.addressof(descs), n, ctypes.addressof(com), batch_id,
                                           ctypes.addressof(rho), None if arr is None else ctypes.addressof(rk)),
           "imm_fs_batched_challenges")
    return list(rho), (list(rk)[:nrounds] if arr is not None else [])


def sumcheck_verify_fs_batched(transcript: Sequence[int], nrounds: int, shapes_and_ids, commitments, batch_id: int,
                               expect: Optional[Sequence[int]] = None) -> Tuple[int, int]:
    """Host verifier of a batched non-interactive proof; returns (status, fail_at)."""
    n = len(shapes_and_ids)
    total = 1 + 3 * nrounds + 3 * n
    words = [int(v) & 0xFFFFFFFFFFFFFFFF for v in list(transcript)[:total]]
    if len(words) != total:
        raise ValueError("transcript too short")
    arr = (ctypes.c_uint64 * total)(*words)
    descs = _shape_descs(shapes_and_ids)
    data = bytes(commitments)
    if len(data) != 96 * n:
        raise ValueError("96 commitment bytes per member")
    com = (ctypes.c_uint8 * len(data))(*data)
    exp = None
    if expect is not None:
        if len(expect) != 3 * n:
            raise ValueError("expect must hold 3 words per member")
        exp = (ctypes.c_uint64 * (3 * n))(*[int(v) & 0xFFFFFFFFFFFFFFFF for v in expect])
    fail = ctypes.c_int(-2)
    rc = lib().imm_sumcheck_verify_fs_batched(ctypes.addressof(arr), nrounds, ctypes.addressof(descs), n,
                                              ctypes.addressof(com), batch_id,
                                              None if exp is None else ctypes.addressof(exp), ctypes.addressof(fail))
    _check(rc, "imm_sumcheck_verify_fs_batched")
    return rc, fail.value


# ------------------------------------------------------------------ the verifier's pass


class Verifier:
    """The verifier's own (c0, a_fin, b_fin) of every proof: one pass over the opened matrices.
    ``batched``: the problems are the members of one batched proof."""

    def __init__(self, problems, batched: bool = False, device="cuda"):
        self.problems = list(problems)
        self.descs = make_descs(self.problems)
        self.nproofs = len(self.problems)
        self.batched = bool(batched)
        need = lib().imm_sumcheck_expected_workspace(ctypes.addressof(self.descs), self.nproofs, int(self.batched))
        if need == 0:
            raise ImmError(ERR_SHAPE, "imm_sumcheck_expected_workspace")
        self.ws = torch.empty(need, dtype=torch.uint8, device=device)
        self.values = torch.zeros((self.nproofs, 3), dtype=torch.int64, device=device)
        self.status = torch.full((self.nproofs,), -99, dtype=torch.int32, device=device)
        self.launches = _launch_counts(self.descs)[1] + 2        # E_k tables, contractions, the inner products

    def expected(self, seed: int = 0, batch_id: Optional[int] = None, points=None) -> torch.Tensor:
        """Enqueue the pass on the current stream; returns the (nproofs, 3) device tensor.  ``points``:
        per proof (r_row, r_col, r_k) for hashed challenges, else they come from the generator."""
        if self.batched != (batch_id is not None):
            raise ValueError("batch_id goes with batched=True")
        bid = ctypes.c_uint64(int(batch_id)) if batch_id is not None else None
        arr = None
        if points is not None:
            if len(points) != self.nproofs:
                raise ValueError("one (r_row, r_col, r_k) per proof")
            arr = (ctypes.c_uint64 * (96 * self.nproofs))()
            for i, triple in enumerate(points):
                for j, vals in enumerate(triple):
                    if len(vals) > 32:
                        raise ValueError("at most 32 challenges per point")
                    for t, v in enumerate(vals):
                        arr[96 * i + 32 * j + t] = int(v)
        _check(lib().imm_sumcheck_expected(ctypes.addressof(self.descs), self.nproofs, seed,
                                           None if bid is None else ctypes.addressof(bid),
                                           None if arr is None else ctypes.addressof(arr),
                                           self.values.data_ptr(), self.status.data_ptr(), self.ws.data_ptr(),
                                           self.ws.numel(), _stream()), "imm_sumcheck_expected")
        return self.values


def sumcheck_expected(problems, seed: int = 0, batch_id: Optional[int] = None, points=None) -> List[Tuple[int, int, int]]:
    """Convenience: the verifier's (c0, a_fin, b_fin) per proof as Python ints (synchronises)."""
    v = Verifier(problems, batched=batch_id is not None)
    t = v.expected(seed, batch_id, points)
    torch.cuda.synchronize()
    if int(v.status.abs().max()) != 0:
        raise ImmError(int(v.status.min()), "device status")
    return [tuple(int(x) & 0xFFFFFFFFFFFFFFFF for x in row) for row in t.cpu()]


# ------------------------------------------------------------------ links between products


def requant_check(C: torch.Tensor, H: torch.Tensor, shift: int = 9, rnd: int = 256, lo: int = -127, hi: int = 127,
                  out: Optional[torch.Tensor] = None) -> torch.Tensor:
    """Checks H == clamp(floor((C + rnd) / 2^shift), lo, hi) entry by entry (C int32, H int8, same
    shape).  Returns a 2-element int64 CUDA tensor: the number of differing entries and the row-major
    position of the first (-1 if none).  Enqueued on the current stream; ``out`` to reuse a buffer."""
    pc, cc, rows, cols, ldc = _matrix(C, "C")
    ph, ch, rows2, cols2, ldh = _matrix(H, "H")
    if cc != I32 or ch != I8 or (rows, cols) != (rows2, cols2):
        raise ValueError("need C int32 and H int8 of the same shape")
    if out is None:
        out = torch.empty(2, dtype=torch.int64, device=C.device)
    _cuda(out, torch.int64, "out")
    _check(lib().imm_requant_check(pc, ph, rows, cols, ldc, ldh, int(shift), int(rnd), int(lo), int(hi),
                                   out.data_ptr(), _stream()), "imm_requant_check")
    return out


def gated_link_check(G: torch.Tensor, U: Optional[torch.Tensor], H: torch.Tensor, act, shift: int = 9, rnd: int = 256,
                     shift2: int = 7, rnd2: int = 64, lo: int = -127, hi: int = 127,
                     out: Optional[torch.Tensor] = None) -> torch.Tensor:
    """Checks H == clamp(floor((act[q(G)] * q(U) + rnd2) / 2^shift2), lo, hi) entry by entry, q(X) =
    clamp(floor((X + rnd) / 2^shift), -128, 127); U None: H == act[q(G)].  G, U int32 and H int8 CUDA
    matrices of one shape; ``act``: 256 int8 values (bytes, list or CPU tensor), act[v + 128] answers v.
    Returns a 2-element int64 CUDA tensor: differing entries and the position of the first (-1 if none)."""
    pg, cg, rows, cols, ldg = _matrix(G, "G")
    ph, ch, rows2, cols2, ldh = _matrix(H, "H")
    if cg != I32 or ch != I8 or (rows, cols) != (rows2, cols2):
        raise ValueError("need G int32 and H int8 of the same shape")
    pu, ldu = None, ldg
    if U is not None:
        pu, cu, rows3, cols3, ldu = _matrix(U, "U")
        if cu != I32 or (rows3, cols3) != (rows, cols):
            raise ValueError("need U int32 of the shape of G")
    table = (ctypes.c_int8 * 256)(*[int(v) for v in (act.tolist() if hasattr(act, "tolist") else act)])
    if out is None:
        out = torch.empty(2, dtype=torch.int64, device=G.device)
    _cuda(out, torch.int64, "out")
    _check(lib().imm_gated_link_check(pg, pu, ph, rows, cols, ldg, ldu, ldh, ctypes.addressof(table), int(shift), int(rnd),
                                      int(shift2), int(rnd2), int(lo), int(hi), out.data_ptr(), _stream()),
           "imm_gated_link_check")
    return out


# ------------------------------------------------------------------ logit distance distribution


def _logit_rows(t: torch.Tensor, what: str) -> Tuple[int, int, int]:
    """(steps, n, ld) of a 2-D float32 CUDA tensor whose rows are contiguous."""
    if not t.is_cuda:
        raise ValueError(f"{what}: a CUDA tensor is required (there is no CPU path)")
    if t.dtype != torch.float32 or t.dim() != 2 or (t.shape[1] > 1 and t.stride(1) != 1):
        raise ValueError(f"{what}: expected a 2-D float32 tensor with contiguous rows")
    return int(t.shape[0]), int(t.shape[1]), int(t.stride(0)) if t.shape[0] > 1 else max(int(t.stride(0)), int(t.shape[1]))


def ldd_tv_kl(logits: torch.Tensor, ref_logits: torch.Tensor) -> Tuple[torch.Tensor, torch.Tensor]:
    """TV distance and KL(reference || deployed) per row; returns two float64 tensors of ``steps``."""
    steps, n, ld = _logit_rows(logits, "logits")
    if _logit_rows(ref_logits, "ref_logits") != (steps, n, ld):
        raise ValueError("logits and ref_logits must have the same shape and row stride")
    tv = torch.empty(steps, dtype=torch.float64, device=logits.device)
    kl = torch.empty(steps, dtype=torch.float64, device=logits.device)
    _check(lib().imm_ldd_tv_kl(logits.data_ptr(), ref_logits.data_ptr(), steps, n, ld, tv.data_ptr(), kl.data_ptr(),
                               _stream()), "imm_ldd_tv_kl")
    return tv, kl


def ldd_topk_distance(ref_logits: torch.Tensor, topk: torch.Tensor,
                      workspace: Optional[torch.Tensor] = None) -> Tuple[torch.Tensor, torch.Tensor]:
    """Top-K distance of every row to its claimed index set (int32, steps x K); returns
    (float64 distances, int32 per-row status).  ``workspace``: a uint8 CUDA tensor of at least
    ``imm_ldd_topk_workspace`` bytes to reuse between calls (allocated here when absent)."""
    steps, n, ld = _logit_rows(ref_logits, "ref_logits")
    topk = _cuda(topk, torch.int32, "topk")
    if topk.dim() != 2 or topk.shape[0] != steps or not topk.is_contiguous():
        raise ValueError("topk: expected a contiguous int32 tensor of shape (steps, K)")
    dist = torch.empty(steps, dtype=torch.float64, device=ref_logits.device)
    status = torch.full((steps,), -99, dtype=torch.int32, device=ref_logits.device)
    k = int(topk.shape[1])
    need = lib().imm_ldd_topk_workspace(steps, n, k)
    if workspace is None:
        workspace = torch.empty(max(need, 16), dtype=torch.uint8, device=ref_logits.device)
    _check(lib().imm_ldd_topk_distance(ref_logits.data_ptr(), steps, n, ld, topk.data_ptr(), k,
                                       dist.data_ptr(), status.data_ptr(), workspace.data_ptr(), workspace.numel(),
                                       _stream()), "imm_ldd_topk_distance")
    return dist, status


def ldd_tail_fraction(dist: torch.Tensor, offsets: torch.Tensor, t1: float, t2: float) -> Tuple[torch.Tensor, torch.Tensor]:
    """p(t1) of every request and the flag p(t1) > t2; ``offsets`` is int64 with nrequests + 1 entries."""
    dist = _cuda(dist, torch.float64, "dist")
    offsets = _cuda(offsets, torch.int64, "offsets")
    nreq = int(offsets.numel()) - 1
    p = torch.empty(max(nreq, 0), dtype=torch.float64, device=dist.device)
    flag = torch.empty(max(nreq, 0), dtype=torch.int32, device=dist.device)
    _check(lib().imm_ldd_tail_fraction(dist.data_ptr(), offsets.data_ptr(), nreq, float(t1), float(t2), p.data_ptr(),
                                       flag.data_ptr(), _stream()), "imm_ldd_tail_fraction")
    return p, flag

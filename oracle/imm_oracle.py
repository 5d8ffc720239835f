"""ctypes binding of the plain-C oracle (test infrastructure only; see ``imm_oracle.c``).

Argument marshalling only: every number is computed by the C file.  Matrices are numpy arrays
(int8 / int32, row-major, possibly with a leading dimension larger than the column count);
field elements are Python ints or numpy uint64 arrays of canonical values.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

P = 0xFFFFFFFF00000001
I8, I32 = 0, 1
BIND_ROWS, BIND_COLS = 0, 1
OK, REJECT = 0, 1

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "imm_oracle.c")
_LIB = os.path.join(_HERE, "liboracle.so")

BUILD_FLAGS = ["-O2", "-Wall", "-shared", "-fPIC"]        # how the oracle is compiled (reported beside its timings)

_u64 = ctypes.c_uint64
_i64 = ctypes.c_int64
_vp = ctypes.c_void_p


def build(force: bool = False) -> str:
    """Compile ``imm_oracle.c`` with gcc into ``liboracle.so`` beside it (plain -O2)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".tmp{os.getpid()}"
        subprocess.check_call(["gcc"] + BUILD_FLAGS + ["-o", tmp, _SRC])
        os.replace(tmp, _LIB)
    return _LIB


_lib = None


def lib() -> ctypes.CDLL:
    global _lib
    if _lib is None:
        L = ctypes.CDLL(build())
        for name in ("orc_add", "orc_sub", "orc_mul", "orc_pow"):
            getattr(L, name).restype = _u64
            getattr(L, name).argtypes = [_u64, _u64]
        L.orc_lift.restype = _u64
        L.orc_lift.argtypes = [_i64]
        L.orc_mix64.restype = _u64
        L.orc_mix64.argtypes = [_u64]
        L.orc_stream.restype = _u64
        L.orc_stream.argtypes = [_u64, _u64, _u64]
        L.orc_challenge.restype = _u64
        L.orc_challenge.argtypes = [_u64, _u64, ctypes.c_uint32, ctypes.c_uint32]
        L.orc_ceil_log2.restype = ctypes.c_int
        L.orc_ceil_log2.argtypes = [_i64]
        L.orc_eq_closed.restype = _u64
        L.orc_eq_closed.argtypes = [_vp, ctypes.c_int, _u64]
        L.orc_eq_table.restype = None
        L.orc_eq_table.argtypes = [_vp, ctypes.c_int, _vp]
        L.orc_mle_eval_bruteforce.restype = _u64
        L.orc_mle_eval_bruteforce.argtypes = [_vp, ctypes.c_int, _i64, _i64, _i64, _vp, _vp]
        L.orc_mle_partial_eval.restype = None
        L.orc_mle_partial_eval.argtypes = [_vp, ctypes.c_int, _i64, _i64, _i64, ctypes.c_int, _vp, _vp]
        L.orc_mle_eval_point.restype = _u64
        L.orc_mle_eval_point.argtypes = [_vp, ctypes.c_int, _i64, _i64, _i64, _vp, _vp]
        L.orc_sumcheck_matmul_prove.restype = ctypes.c_int
        L.orc_sumcheck_matmul_prove.argtypes = [_vp, _vp, _vp, _i64, _i64, _i64, _i64, _i64, _i64,
                                                _u64, _u64, _vp]
        L.orc_interp_deg2.restype = _u64
        L.orc_interp_deg2.argtypes = [_u64, _u64, _u64, _u64]
        L.orc_sumcheck_verify.restype = ctypes.c_int
        L.orc_sumcheck_verify.argtypes = [_vp, ctypes.c_int, _u64, _u64, _vp, _vp, _vp, _vp]
        L.orc_sumcheck_matmul_prove_batched.restype = ctypes.c_int
        L.orc_sumcheck_matmul_prove_batched.argtypes = [ctypes.c_int] + [_vp] * 9 + [_u64, _u64, _vp, _vp]
        L.orc_sumcheck_verify_batched.restype = ctypes.c_int
        L.orc_sumcheck_verify_batched.argtypes = [_vp, ctypes.c_int, ctypes.c_int, _u64, _u64, _vp, _vp]
        L.orc_matmul_i8_i32.restype = None
        L.orc_matmul_i8_i32.argtypes = [_vp, _vp, _vp, _i64, _i64, _i64]
        _lib = L
    return _lib


# ------------------------------------------------------------------ marshalling helpers


def _fe_array(values) -> np.ndarray:
    arr = np.ascontiguousarray(np.asarray(values, dtype=np.uint64).reshape(-1))
    return arr


def _mat(mat: np.ndarray):
    """Return (array kept alive, dtype code, rows, cols, ld) for a 2-D int8/int32 array whose
    rows are contiguous (a column slice of a wider row-major array is accepted)."""
    if mat.ndim != 2:
        raise ValueError("matrix must be 2-D")
    if mat.dtype == np.int8:
        code = I8
    elif mat.dtype == np.int32:
        code = I32
    else:
        raise ValueError("matrix dtype must be int8 or int32")
    rows, cols = mat.shape
    if cols > 1 and mat.strides[1] != mat.itemsize:
        mat = np.ascontiguousarray(mat)
    if rows > 1 and (mat.strides[0] % mat.itemsize != 0 or mat.strides[0] < cols * mat.itemsize):
        mat = np.ascontiguousarray(mat)
    ld = mat.strides[0] // mat.itemsize if rows > 1 else max(cols, 1)
    return mat, code, rows, cols, ld


def _ptr(arr: np.ndarray) -> int:
    return arr.ctypes.data


# ------------------------------------------------------------------ field / generator


def add(x: int, y: int) -> int:
    return lib().orc_add(x, y)


def sub(x: int, y: int) -> int:
    return lib().orc_sub(x, y)


def mul(x: int, y: int) -> int:
    return lib().orc_mul(x, y)


def power(x: int, e: int) -> int:
    return lib().orc_pow(x, e)


def lift(v: int) -> int:
    return lib().orc_lift(int(v))


def mix64(z: int) -> int:
    return lib().orc_mix64(z & 0xFFFFFFFFFFFFFFFF)


def stream(seed: int, sid: int, ctr: int) -> int:
    return lib().orc_stream(seed, sid, ctr)


def challenge(seed: int, proof_id: int, domain: int, index: int) -> int:
    return lib().orc_challenge(seed, proof_id, domain, index)


def challenges(seed: int, proof_id: int, domain: int, count: int) -> np.ndarray:
    return np.array([challenge(seed, proof_id, domain, i) for i in range(count)], dtype=np.uint64)


def ceil_log2(d: int) -> int:
    return lib().orc_ceil_log2(d)


# ------------------------------------------------------------------ eq / MLE


def eq_closed(r, i: int) -> int:
    r = _fe_array(r)
    return lib().orc_eq_closed(_ptr(r), len(r), i)


def eq_table(r) -> np.ndarray:
    r = _fe_array(r)
    out = np.empty(1 << len(r), dtype=np.uint64)
    lib().orc_eq_table(_ptr(r), len(r), _ptr(out))
    return out


def mle_eval_bruteforce(mat: np.ndarray, x, y) -> int:
    mat, code, rows, cols, ld = _mat(mat)
    x, y = _fe_array(x), _fe_array(y)
    assert len(x) == ceil_log2(rows) and len(y) == ceil_log2(cols)
    return lib().orc_mle_eval_bruteforce(_ptr(mat), code, rows, cols, ld, _ptr(x), _ptr(y))


def mle_partial_eval(mat: np.ndarray, bind: int, eq) -> np.ndarray:
    mat, code, rows, cols, ld = _mat(mat)
    eq = _fe_array(eq)
    need, outlen = (rows, cols) if bind == BIND_ROWS else (cols, rows)
    assert len(eq) >= need
    out = np.empty(outlen, dtype=np.uint64)
    lib().orc_mle_partial_eval(_ptr(mat), code, rows, cols, ld, bind, _ptr(eq), _ptr(out))
    return out


def mle_eval_point(mat: np.ndarray, eq_row, eq_col) -> int:
    mat, code, rows, cols, ld = _mat(mat)
    eq_row, eq_col = _fe_array(eq_row), _fe_array(eq_col)
    assert len(eq_row) >= rows and len(eq_col) >= cols
    return lib().orc_mle_eval_point(_ptr(mat), code, rows, cols, ld, _ptr(eq_row), _ptr(eq_col))


# ------------------------------------------------------------------ protocol


def matmul_i8_i32(A: np.ndarray, B: np.ndarray) -> np.ndarray:
    A = np.ascontiguousarray(A, dtype=np.int8)
    B = np.ascontiguousarray(B, dtype=np.int8)
    m, k = A.shape
    k2, n = B.shape
    assert k == k2
    C = np.empty((m, n), dtype=np.int32)
    lib().orc_matmul_i8_i32(_ptr(A), _ptr(B), _ptr(C), m, k, n)
    return C


def transcript_len(k: int) -> int:
    return 3 * ceil_log2(k) + 3


def sumcheck_matmul_prove(A: np.ndarray, B: np.ndarray, C: np.ndarray, seed: int,
                          proof_id: int) -> np.ndarray:
    A, ca, m, k, lda = _mat(A)
    B, cb, k2, n, ldb = _mat(B)
    C, cc, m2, n2, ldc = _mat(C)
    assert ca == I8 and cb == I8 and cc == I32 and k == k2 and m == m2 and n == n2
    out = np.empty(transcript_len(k), dtype=np.uint64)
    rc = lib().orc_sumcheck_matmul_prove(_ptr(A), _ptr(B), _ptr(C), m, k, n, lda, ldb, ldc,
                                         seed, proof_id, _ptr(out))
    if rc != OK:
        raise ValueError(f"orc_sumcheck_matmul_prove returned {rc}")
    return out


def interp_deg2(g0: int, g1: int, g2: int, r: int) -> int:
    return lib().orc_interp_deg2(g0, g1, g2, r)


def sumcheck_verify(transcript, nrounds: int, seed: int, proof_id: int, expect_c0=None,
                    expect_a_fin=None, expect_b_fin=None):
    """Return (status, fail_at)."""
    t = _fe_array(transcript)
    assert len(t) >= 3 * nrounds + 3
    keep = []

    def opt(v):
        if v is None:
            return None
        box = _u64(int(v))
        keep.append(box)
        return ctypes.addressof(box)

    fail = ctypes.c_int(-2)
    rc = lib().orc_sumcheck_verify(_ptr(t), nrounds, seed, proof_id, opt(expect_c0),
                                   opt(expect_a_fin), opt(expect_b_fin), ctypes.addressof(fail))
    return rc, fail.value


def batched_transcript_len(k: int, nproofs: int) -> int:
    """k: the largest inner dimension of the batch."""
    return 1 + 3 * ceil_log2(k) + 3 * nproofs


def sumcheck_matmul_prove_batched(problems, seed: int, batch_id: int) -> np.ndarray:
    """``problems`` is a sequence of (A, B, C, proof_id); every k is padded to the largest 2^b."""
    mats, dims, ptrs = [], [], [[], [], []]
    for A, B, C, _ in problems:
        A, ca, m, k, lda = _mat(A)
        B, cb, k2, n, ldb = _mat(B)
        C, cc, m2, n2, ldc = _mat(C)
        assert ca == I8 and cb == I8 and cc == I32 and k == k2 and m == m2 and n == n2
        mats.append((A, B, C))
        dims.append((m, k, n, lda, ldb, ldc))
        for lst, M in zip(ptrs, (A, B, C)):
            lst.append(_ptr(M))
    count = len(problems)
    parr = [np.array(lst, dtype=np.uint64) for lst in ptrs]
    darr = [np.array([d[i] for d in dims], dtype=np.int64) for i in range(6)]
    ids = np.array([int(p[3]) for p in problems], dtype=np.uint64)
    out = np.empty(batched_transcript_len(max(d[1] for d in dims), count) if count else 0, dtype=np.uint64)
    rc = lib().orc_sumcheck_matmul_prove_batched(count, *[_ptr(a) for a in parr],
                                                 *[_ptr(a) for a in darr], seed, batch_id,
                                                 _ptr(ids), _ptr(out))
    if rc != OK:
        raise ValueError(f"orc_sumcheck_matmul_prove_batched returned {rc}")
    return out


def sumcheck_verify_batched(transcript, nrounds: int, nproofs: int, seed: int, batch_id: int,
                            expect=None):
    """Return (status, fail_at); ``expect`` is the verifier's own 3*nproofs tail words."""
    t = _fe_array(transcript)
    assert len(t) >= 1 + 3 * nrounds + 3 * nproofs
    e = None if expect is None else _fe_array(expect)
    assert e is None or len(e) == 3 * nproofs
    fail = ctypes.c_int(-2)
    rc = lib().orc_sumcheck_verify_batched(_ptr(t), nrounds, nproofs, seed, batch_id,
                                           None if e is None else _ptr(e), ctypes.addressof(fail))
    return rc, fail.value

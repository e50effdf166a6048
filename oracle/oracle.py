"""ctypes front end of ``gelo_oracle.c`` (fp64, naive loops) -- TEST INFRASTRUCTURE ONLY.

Every function takes and returns C-contiguous float64 numpy arrays.  The
arithmetic lives in the C file; this module only marshals arguments, builds the
shared object with gcc when it is missing, and derives a few quantities that
are plain definitions (relative Frobenius error, 2-norm condition number).

Paper passages followed: Section 3.2 (Eq. 1-4) for the chain, "Mitigation 1"
for the bounded condition number, "Mitigation 2" (Eq. 7-9) for shield rows.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import threading

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "gelo_oracle.c")
_LIB = os.path.join(_HERE, "libgelo_oracle.so")
_lock = threading.Lock()
_lib = None

ORTHOGONAL = 0
NONORTHOGONAL = 1
DEFAULT_GAMMA = 0.5
COND_BOUND = 100.0

__all__ = [
    "ORTHOGONAL", "NONORTHOGONAL", "DEFAULT_GAMMA", "COND_BOUND", "build", "philox4x32_10",
    "philox_words", "gaussian", "matmul", "rows_times_w", "householder_qr", "lu_inverse",
    "singular_extremes", "cond2", "sample_mixing", "sample_mixing_verified", "median_row_norm",
    "shield_rows", "student_t", "shield_rows_t", "e4m3_decode", "e4m3_encode", "quantize_e4m3", "project_e4m3", "chain", "direct", "rel_fro", "num_threads",
]


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (-O2, OpenMP) if the shared object is missing or stale."""
    with _lock:
        stale = (not os.path.exists(_LIB)) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC)
        if force or stale:
            tmp = _LIB + f".{os.getpid()}.tmp"
            subprocess.check_call(
                ["gcc", "-O2", "-fopenmp", "-shared", "-fPIC", "-std=c11", "-o", tmp, _SRC, "-lm"])
            os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        build()
        lib = ctypes.CDLL(_LIB)
        lib.oracle_median_row_norm.restype = ctypes.c_double
        lib.oracle_e4m3_decode.restype = ctypes.c_double
        lib.oracle_e4m3_decode.argtypes = [ctypes.c_uint8]
        lib.oracle_e4m3_encode.restype = ctypes.c_uint8
        lib.oracle_e4m3_encode.argtypes = [ctypes.c_float]
        lib.oracle_quantize_e4m3.restype = ctypes.c_float
        for name in ("oracle_householder_qr", "oracle_lu_inverse", "oracle_singular_extremes",
                     "oracle_sample_mixing", "oracle_chain"):
            getattr(lib, name).restype = ctypes.c_int
        _lib = lib
    return _lib


def num_threads() -> int:
    """Threads the OpenMP loops will use (OMP_NUM_THREADS or the visible cores)."""
    env = os.environ.get("OMP_NUM_THREADS")
    if env and env.isdigit() and int(env) > 0:
        return int(env)
    try:
        return len(os.sched_getaffinity(0))
    except AttributeError:  # pragma: no cover
        return os.cpu_count() or 1


def _f64(a):
    return np.ascontiguousarray(a, dtype=np.float64)


def _p(a):
    return a.ctypes.data_as(ctypes.c_void_p)


_i64 = ctypes.c_int64
_u64 = ctypes.c_uint64
_u32 = ctypes.c_uint32
_dbl = ctypes.c_double


def philox4x32_10(counter, key):
    """One Philox4x32-10 block: 4 counter words, 2 key words -> 4 output words (uint32)."""
    c = np.ascontiguousarray(counter, dtype=np.uint32)
    k = np.ascontiguousarray(key, dtype=np.uint32)
    out = np.empty(4, dtype=np.uint32)
    _load().oracle_philox4x32_10(_p(c), _p(k), _p(out))
    return out


def philox_words(seed, stream, attempt, first, count):
    """The uint32 word of elements first..first+count-1 of the stream (seed, stream, attempt)."""
    out = np.empty(int(count), dtype=np.uint32)
    _load().oracle_philox_words(_u64(seed), _u32(stream), _u32(attempt), _u64(first), _u64(count), _p(out))
    return out


def gaussian(seed, stream, attempt, rows, cols):
    """rows x cols standard normals; element (i, j) uses stream index i*cols + j."""
    out = np.empty((int(rows), int(cols)), dtype=np.float64)
    _load().oracle_gaussian(_u64(seed), _u32(stream), _u32(attempt), _u64(0), _u64(int(rows) * int(cols)), _p(out))
    return out


def matmul(A, B):
    """Naive triple-loop product of two row-major matrices."""
    A, B = _f64(A), _f64(B)
    M, K = A.shape
    K2, N = B.shape
    assert K == K2
    C = np.empty((M, N), dtype=np.float64)
    _load().oracle_matmul(_i64(M), _i64(N), _i64(K), _p(A), _i64(K), _p(B), _i64(N), _p(C), _i64(N))
    return C


def rows_times_w(H, W, rows):
    """out[r] = H[rows[r]] @ W for the selected rows only (Eq. 4's right-hand side)."""
    H, W = _f64(H), _f64(W)
    rows = np.ascontiguousarray(rows, dtype=np.int64)
    n, d = H.shape
    d2, p = W.shape
    assert d == d2 and (rows.size == 0 or (rows.min() >= 0 and rows.max() < n))
    out = np.empty((rows.size, p), dtype=np.float64)
    _load().oracle_rows_times_w(_i64(rows.size), _p(rows), _i64(d), _i64(p), _p(H), _p(W), _p(out))
    return out


def direct(H, W):
    """The result the method must reproduce: H @ W (Eq. 4)."""
    return matmul(H, W)


def householder_qr(G):
    """G = Q R with diag(R) > 0 by unblocked Householder reflections.  Returns (Q, R)."""
    G = _f64(G)
    m = G.shape[0]
    assert G.shape == (m, m)
    Q = np.empty((m, m)); R = np.empty((m, m))
    rc = _load().oracle_householder_qr(_i64(m), _p(G), _p(Q), _p(R))
    if rc != 0:
        raise MemoryError("oracle_householder_qr")
    return Q, R


def lu_inverse(A):
    """A^-1 by Gaussian elimination with partial pivoting."""
    A = _f64(A)
    m = A.shape[0]
    assert A.shape == (m, m)
    X = np.empty((m, m))
    rc = _load().oracle_lu_inverse(_i64(m), _p(A), _p(X))
    if rc == 1:
        raise ZeroDivisionError("singular matrix")
    if rc != 0:
        raise MemoryError("oracle_lu_inverse")
    return X


def singular_extremes(A):
    """(sigma_max, sigma_min) of a square matrix by one-sided Jacobi."""
    A = _f64(A)
    m = A.shape[0]
    assert A.shape == (m, m)
    hi = _dbl(); lo = _dbl()
    rc = _load().oracle_singular_extremes(_i64(m), _p(A), ctypes.byref(hi), ctypes.byref(lo))
    if rc < 0:
        raise MemoryError("oracle_singular_extremes")
    return hi.value, lo.value


def cond2(A):
    """2-norm condition number sigma_max / sigma_min (Mitigation 1)."""
    hi, lo = singular_extremes(A)
    return float("inf") if lo == 0.0 else hi / lo


def sample_mixing(m, kind, seed, attempt=0, gamma=DEFAULT_GAMMA):
    """(A, Ainv) for one attempt.  kind 0: orthogonal Q, Ainv = A^T; kind 1: Q0 + gamma*G1/sqrt(m)."""
    A = np.empty((m, m)); X = np.empty((m, m))
    rc = _load().oracle_sample_mixing(_i64(m), ctypes.c_int(kind), _u64(seed), _u32(attempt), _dbl(gamma), _p(A), _p(X))
    if rc != 0:
        raise RuntimeError(f"oracle_sample_mixing rc={rc}")
    return A, X


def sample_mixing_verified(m, kind, seed, gamma=DEFAULT_GAMMA, bound=COND_BOUND, max_attempts=8):
    """Sample, verify kappa_2(A) <= bound for non-orthogonal A, resample with the next attempt
    number otherwise (Mitigation 1 asks for a conditioning check on every drawn A).  Returns (A, Ainv, cond, attempt)."""
    for attempt in range(max_attempts):
        A, X = sample_mixing(m, kind, seed, attempt, gamma)
        if kind == ORTHOGONAL:
            return A, X, 1.0, attempt
        c = cond2(A)
        if c <= bound:
            return A, X, c, attempt
    raise ArithmeticError("no well-conditioned A within the attempt limit")


def median_row_norm(H):
    H = _f64(H)
    n, d = H.shape
    return float(_load().oracle_median_row_norm(_i64(n), _i64(d), _p(H)))


def shield_rows(H, k, scale, seed):
    """S (k x d) = (scale * median row norm of H / sqrt(d)) * N(0,1) draws of stream 2."""
    H = _f64(H)
    n, d = H.shape
    S = np.empty((int(k), d), dtype=np.float64)
    _load().oracle_shield_rows(_i64(n), _i64(d), _i64(k), _p(H), _dbl(scale), _u64(seed), _p(S))
    return S


def student_t(seed, nu, count, first=0):
    """Standardised (unit-variance) Student-t draws with nu degrees of freedom, elements first..first+count-1."""
    assert 3 <= int(nu) <= 63
    out = np.empty(int(count), dtype=np.float64)
    _load().oracle_student_t(_u64(seed), _u32(nu), _u64(first), _u64(count), _p(out))
    return out


def shield_rows_t(H, k, scale, seed, nu):
    """S (k x d) = (scale * median row norm of H / sqrt(d)) * standardised Student-t draws (Table 9's other kind)."""
    assert 3 <= int(nu) <= 63
    H = _f64(H)
    n, d = H.shape
    S = np.empty((int(k), d), dtype=np.float64)
    _load().oracle_shield_rows_t(_i64(n), _i64(d), _i64(k), _p(H), _dbl(scale), _u64(seed), _u32(nu), _p(S))
    return S


def e4m3_decode(codes):
    """Values (float64) of an array of E4M3 codes (uint8)."""
    codes = np.ascontiguousarray(codes, dtype=np.uint8)
    table = np.array([_load().oracle_e4m3_decode(c) for c in range(256)], dtype=np.float64)
    return table[codes]


def e4m3_encode(x):
    """Nearest E4M3 code (ties to even, saturating at 448) of every element of a float32 array."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    L = _load()
    return np.array([L.oracle_e4m3_encode(float(v)) for v in x.ravel()], dtype=np.uint8).reshape(x.shape)


def quantize_e4m3(x):
    """Per-tensor quantisation: (codes uint8, scale float32) with scale = max|x| / 448, codes = encode(x / scale)."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    codes = np.empty(x.shape, dtype=np.uint8)
    scale = _load().oracle_quantize_e4m3(_i64(x.size), _p(x), _p(codes))
    return codes, np.float32(scale)


def project_e4m3(u_codes, u_scale, w_codes, w_scale):
    """Y' = (s_U s_W) (U8 W8): the offloaded product of Eq. 2 on E4M3 operands, exact in fp64."""
    return float(u_scale) * float(w_scale) * matmul(e4m3_decode(u_codes), e4m3_decode(w_codes))


def chain(A, Ainv, H, S, W, want_intermediates=False):
    """U = A [H; S], Y' = U W, Y = (Ainv Y')[0:n].  Returns Y, or (U, Y', Y)."""
    A, Ainv, H, W = _f64(A), _f64(Ainv), _f64(H), _f64(W)
    n, d = H.shape
    k = 0 if S is None else int(S.shape[0])
    S = _f64(S) if k else np.zeros((0, d))
    m = n + k
    p = W.shape[1]
    assert A.shape == (m, m) and Ainv.shape == (m, m) and W.shape[0] == d
    Y = np.empty((n, p))
    U = np.empty((m, d)) if want_intermediates else None
    Yp = np.empty((m, p)) if want_intermediates else None
    rc = _load().oracle_chain(_i64(n), _i64(k), _i64(d), _i64(p), _p(A), _p(Ainv), _p(H), _p(S), _p(W),
                              _p(U) if U is not None else None, _p(Yp) if Yp is not None else None, _p(Y))
    if rc != 0:
        raise MemoryError("oracle_chain")
    return (U, Yp, Y) if want_intermediates else Y


def rel_fro(X, ref):
    """||X - ref||_F / ||ref||_F in fp64."""
    X = np.asarray(X, dtype=np.float64); ref = np.asarray(ref, dtype=np.float64)
    den = np.linalg.norm(ref)
    return float(np.linalg.norm(X - ref) / den) if den > 0 else float(np.linalg.norm(X - ref))

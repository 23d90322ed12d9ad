"""ctypes front end of the CPU oracle (oracle/oz_oracle.c).

TEST INFRASTRUCTURE ONLY: imported by tests/, by the smoke check and by the
benchmark's CPU-baseline leg.  The GPU package never imports this module and
this module never imports the GPU package.

`build()` compiles the C file with gcc (OpenMP) into oracle/liboz_oracle.so.
Array conventions are those stated at the top of oz_oracle.c.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "oz_oracle.c")
_LIB = os.path.join(_HERE, "liboz_oracle.so")

SET_S, SET_E, SET_A = 0, 1, 2
QUANT_RN, QUANT_TZ = 0, 1
SCALE_MAXEXP, SCALE_CS, SCALE_ACCURATE = 0, 1, 2
SUB_FP8, SUB_INT8, SUB_INT8_NATIVE = 0, 1, 2
NONFINITE_SHIFT = -(2**31)

_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle if the shared object is missing or older than its source."""
    if (not force and os.path.exists(_LIB)
            and os.path.getmtime(_LIB) >= os.path.getmtime(_SRC)):
        return _LIB
    cmd = ["gcc", "-O2", "-std=c11", "-fopenmp", "-fPIC", "-shared", "-ffp-contract=off",
           "-o", _LIB, _SRC, "-lm"]
    subprocess.run(cmd, check=True)
    return _LIB


def lib() -> C.CDLL:
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
        _lib.ozo_e4m3_value.restype = C.c_double
        _lib.ozo_i128_to_double.restype = C.c_double
        _lib.ozo_i128_to_double.argtypes = [C.c_int64, C.c_int64]
        _lib.ozo_cs_bound.restype = C.c_uint64
        _lib.ozo_cs_bound.argtypes = [C.c_int, C.c_int64]
        _lib.ozo_plane_products.restype = C.c_int64
        _lib.ozo_plane_products_merged.restype = C.c_int64
        _lib.ozo_centred_residue.argtypes = [C.c_int64, C.c_int]
    return _lib


def _p(a: np.ndarray):
    return a.ctypes.data_as(C.c_void_p)


def _i64(v):
    return C.c_int64(int(v))


def num_threads() -> int:
    """Threads the OpenMP loops will use (OMP_NUM_THREADS or the core count)."""
    env = os.environ.get("OMP_NUM_THREADS")
    if env:
        return int(env.split(",")[0])
    return len(os.sched_getaffinity(0))


# ---------------------------------------------------------------- constants
def modset(s: int) -> list[int]:
    buf = (C.c_int * 16)()
    r = lib().ozo_modset(s, buf)
    return [buf[i] for i in range(r)]


def pstore(s: int, substrate: int = 0) -> int:
    return lib().ozo_pstore_sub(s, substrate)


def planes_of(m: int) -> int:
    return lib().ozo_planes_of(m)


def M(s: int) -> int:
    out = (C.c_uint64 * 2)()
    lib().ozo_M(s, out)
    return int(out[0]) | (int(out[1]) << 64)


def budget_maxexp(s: int, k: int) -> tuple[int, int]:
    ta, tb = C.c_int(), C.c_int()
    lib().ozo_budget_maxexp(s, _i64(k), C.byref(ta), C.byref(tb))
    return ta.value, tb.value


def cs_bound(s: int, k: int) -> int:
    return int(lib().ozo_cs_bound(s, k))


def garner_constants(s: int) -> list[int]:
    buf = (C.c_int * 16)()
    lib().ozo_garner_constants(s, buf)
    return [buf[i] for i in range(len(modset(s)))]


def centred_residue(x: int, m: int) -> int:
    return lib().ozo_centred_residue(int(x), m)


def split(d: int, m: int) -> list[int]:
    out = (C.c_int * 3)()
    n = lib().ozo_split(int(d), m, out)
    return [out[i] for i in range(n)]


def e4m3_value(code: int) -> float:
    return lib().ozo_e4m3_value(code)


def e4m3_encode(v: int) -> int:
    return lib().ozo_e4m3_encode(int(v))


def in_e4m3(v: int) -> bool:
    return bool(lib().ozo_in_e4m3(int(v)))


def i128_to_double(x: int) -> float:
    lo = x & (2**64 - 1)
    hi = (x >> 64)
    lo = lo - 2**64 if lo >= 2**63 else lo
    return lib().ozo_i128_to_double(lo, hi)


def crt_single(s: int, residues) -> int:
    c = (C.c_int * 16)(*[int(v) for v in residues])
    out = (C.c_int64 * 2)()
    lib().ozo_crt_single(s, c, out)
    return (int(out[1]) << 64) | (int(out[0]) & (2**64 - 1))


def byteplane_residue(x: int, m: int, nbytes: int = 8):
    u0, u1, mc, mh = C.c_int(), C.c_int(), C.c_int(), C.c_int()
    xs = int(x)
    res = lib().ozo_byteplane_residue(_i64(xs), m, nbytes, C.byref(u0), C.byref(u1),
                                      C.byref(mc), C.byref(mh))
    return res, u0.value, u1.value, mc.value, mh.value


# ---------------------------------------------------------------- stages
def _check_cm(X: np.ndarray):
    assert X.dtype == np.float64 and X.ndim == 2 and X.flags.f_contiguous, \
        "operands are column-major float64"


def shifts(side: int, X: np.ndarray, s: int, rule: int, tbits: int) -> np.ndarray:
    _check_cm(X)
    lines = X.shape[0] if side == 0 else X.shape[1]
    k = X.shape[1] if side == 0 else X.shape[0]
    out = np.zeros(lines, dtype=np.int32)
    lib().ozo_shifts(side, _i64(lines), _i64(k), _p(X), _i64(max(X.shape[0], 1)), s, rule,
                     tbits, _p(out))
    return out


def esc_threshold(s: int) -> int:
    f = lib().ozo_esc_threshold
    f.restype = C.c_uint32
    return int(f(s))


def esc_flatness(side: int, X: np.ndarray) -> int:
    """Smallest flatness code q = floor(2^16 phi^2) over the lines of one operand (exponent-span check)."""
    _check_cm(X)
    lines = X.shape[0] if side == 0 else X.shape[1]
    k = X.shape[1] if side == 0 else X.shape[0]
    f = lib().ozo_esc_flatness
    f.restype = C.c_uint32
    return int(f(side, _i64(lines), _i64(k), _p(X), _i64(max(X.shape[0], 1))))


def esc_check(A: np.ndarray, B: np.ndarray, s: int) -> bool:
    _check_cm(A)
    _check_cm(B)
    m, k = A.shape
    n = B.shape[1]
    return bool(lib().ozo_esc_check(_i64(m), _i64(n), _i64(k), _p(A), _i64(max(m, 1)), _p(B), _i64(max(k, 1)), s))


def esc_rows(A: np.ndarray, B: np.ndarray, s: int) -> np.ndarray:
    """Rows of the product that the exponent-span check sends to the native FP64 path (1 = re-issued)."""
    _check_cm(A)
    _check_cm(B)
    m, k = A.shape
    n = B.shape[1]
    flag = np.zeros(max(m, 1), dtype=np.uint8)
    f = lib().ozo_esc_rows
    f.restype = C.c_int64
    count = f(_i64(m), _i64(n), _i64(k), _p(A), _i64(max(m, 1)), _p(B), _i64(max(k, 1)), s, _p(flag))
    assert count == int(flag[:m].sum())
    return flag[:m]


def native_rows(A: np.ndarray, B: np.ndarray, flag: np.ndarray, alpha: float = 1.0, beta: float = 0.0,
                C0: np.ndarray | None = None) -> np.ndarray:
    """The native FP64 path (compensated inner products) on the flagged rows; other rows keep C0."""
    _check_cm(A)
    _check_cm(B)
    m, k = A.shape
    n = B.shape[1]
    Cm = np.asfortranarray(C0.copy()) if C0 is not None else np.zeros((m, n), dtype=np.float64, order="F")
    flag = np.ascontiguousarray(flag, dtype=np.uint8)
    lib().ozo_native_rows(_i64(m), _i64(n), _i64(k), _p(A), _i64(max(m, 1)), _p(B), _i64(max(k, 1)), _p(flag),
                          C.c_double(alpha), C.c_double(beta), _p(Cm), _i64(max(m, 1)))
    return Cm


def dgemm_fallback(A: np.ndarray, B: np.ndarray, s: int = SET_S, quant: int = QUANT_RN, alpha: float = 1.0,
                   beta: float = 0.0, C0: np.ndarray | None = None):
    """The whole method (norm-based scale rule) with out-of-range rows re-issued on the native path.
    Returns (C, flag)."""
    _check_cm(A)
    _check_cm(B)
    m, k = A.shape
    n = B.shape[1]
    Cm = np.asfortranarray(C0.copy()) if C0 is not None else np.zeros((m, n), dtype=np.float64, order="F")
    flag = np.zeros(max(m, 1), dtype=np.uint8)
    f = lib().ozo_dgemm_fallback
    f.restype = C.c_int64
    rc = f(_i64(m), _i64(n), _i64(k), _p(A), _i64(max(m, 1)), _p(B), _i64(max(k, 1)), _p(Cm), _i64(max(m, 1)), s,
           quant, C.c_double(alpha), C.c_double(beta), _p(flag))
    assert rc >= 0
    return Cm, flag[:m]


def bound_digit(x: float, E: int) -> int:
    return lib().ozo_bound_digit(C.c_double(x), int(E))


def accurate_budget_log2(s: int) -> int:
    return lib().ozo_accurate_budget_log2(s)


def shifts_accurate(A: np.ndarray, B: np.ndarray, s: int):
    """Shifts of both operands by the accurate rule (the extra bound product of Sec. 2 "The FP8
    variant"); returns (shiftA, shiftB, rowmax, colmax)."""
    _check_cm(A)
    _check_cm(B)
    m, k = A.shape
    n = B.shape[1]
    sA, sB = np.zeros(m, dtype=np.int32), np.zeros(n, dtype=np.int32)
    rm, cm = np.zeros(m, dtype=np.uint32), np.zeros(n, dtype=np.uint32)
    rc = lib().ozo_shifts_accurate(_i64(m), _i64(n), _i64(k), _p(A), _i64(max(m, 1)), _p(B), _i64(max(k, 1)), s,
                                   _p(sA), _p(sB), _p(rm), _p(cm))
    assert rc == 0
    return sA, sB, rm, cm


def quantise(side: int, X: np.ndarray, shift: np.ndarray, quant: int) -> np.ndarray:
    _check_cm(X)
    lines = X.shape[0] if side == 0 else X.shape[1]
    k = X.shape[1] if side == 0 else X.shape[0]
    Q = np.zeros((lines, k), dtype=np.int64)
    lib().ozo_quantise(side, _i64(lines), _i64(k), _p(X), _i64(max(X.shape[0], 1)), _p(shift),
                       quant, _p(Q))
    return Q


def residues(Q: np.ndarray, s: int) -> np.ndarray:
    lines, k = Q.shape
    r = len(modset(s))
    D = np.zeros((r, lines, k), dtype=np.int16)
    lib().ozo_residues(_i64(lines), _i64(k), _p(np.ascontiguousarray(Q)), s, _p(D))
    return D


def planes(D: np.ndarray, s: int, substrate: int, row_pitch: int | None = None) -> np.ndarray:
    r, lines, k = D.shape
    pitch = row_pitch if row_pitch is not None else (k + 15) // 16 * 16
    P = np.full((pstore(s, substrate), lines, pitch), 0xAA, dtype=np.uint8)
    rc = lib().ozo_planes(_i64(lines), _i64(k), _p(np.ascontiguousarray(D)), s, substrate, _p(P),
                          _i64(lines * pitch), _i64(pitch))
    assert rc == pstore(s, substrate), "a digit was not representable on the substrate"
    return P


def pstore_merged(s: int, side: int) -> int:
    return lib().ozo_pstore_merged(s, side)


def planes_merged(side: int, D: np.ndarray, s: int, row_pitch: int | None = None,
                  substrate: int = SUB_FP8) -> np.ndarray:
    """Planes of the merged-accumulator layout.  FP8: side 0 stores -16*d1 in place of d1.
    INT8: side 0 stores -d0, 4*d1, d0+d1 and side 1 stores d0, 4*d1, d0+d1."""
    r, lines, k = D.shape
    pitch = row_pitch if row_pitch is not None else (k + 15) // 16 * 16
    P = np.full((pstore_merged(s, side), lines, pitch), 0xAA, dtype=np.uint8)
    rc = lib().ozo_planes_merged_sub(side, _i64(lines), _i64(k), _p(np.ascontiguousarray(D)), s, substrate, _p(P),
                                     _i64(lines * pitch), _i64(pitch))
    assert rc == pstore_merged(s, side), "a digit was not representable on the substrate"
    return P


def plane_products_merged(PA: np.ndarray, PB: np.ndarray, k: int, s: int, substrate: int = SUB_FP8):
    _, m, pa = PA.shape
    _, n, pb = PB.shape
    R = np.zeros((len(modset(s)), n, m), dtype=np.uint16)
    f = lib().ozo_plane_products_merged_sub
    f.restype = C.c_int64
    worst = f(_i64(m), _i64(n), _i64(k), _p(PA), _i64(m * pa), _i64(pa), _p(PB), _i64(n * pb), _i64(pb), s,
              substrate, _p(R))
    return R, int(worst)


def products(DA: np.ndarray, DB: np.ndarray, s: int) -> np.ndarray:
    r, m, k = DA.shape
    n = DB.shape[1]
    R = np.zeros((r, n, m), dtype=np.uint16)
    lib().ozo_products(_i64(m), _i64(n), _i64(k), _p(np.ascontiguousarray(DA)),
                       _p(np.ascontiguousarray(DB)), s, _p(R))
    return R


def plane_products(PA: np.ndarray, PB: np.ndarray, k: int, s: int, substrate: int):
    """Residues recomputed from the stored planes; also the largest |accumulator|."""
    _, m, pa = PA.shape
    _, n, pb = PB.shape
    r = len(modset(s))
    R = np.zeros((r, n, m), dtype=np.uint16)
    worst = lib().ozo_plane_products(_i64(m), _i64(n), _i64(k), _p(PA), _i64(m * pa), _i64(pa),
                                     _p(PB), _i64(n * pb), _i64(pb), s, substrate, _p(R))
    return R, int(worst)


def _ci_to_int(CI: np.ndarray) -> np.ndarray:
    """(n, m, 2) int64 words -> object array (m, n) of Python ints."""
    lo = CI[..., 0].astype(object)
    hi = CI[..., 1].astype(object)
    lo = np.where(lo < 0, lo + 2**64, lo)
    return (hi * 2**64 + lo).T


def crt(R: np.ndarray, s: int, as_int: bool = False):
    r, n, m = R.shape
    CI = np.zeros((n, m, 2), dtype=np.int64)
    lib().ozo_crt(_i64(m), _i64(n), _p(np.ascontiguousarray(R)), s, _p(CI))
    return _ci_to_int(CI) if as_int else CI


def direct(QA: np.ndarray, QB: np.ndarray, as_int: bool = False):
    m, k = QA.shape
    n = QB.shape[0]
    CI = np.zeros((n, m, 2), dtype=np.int64)
    lib().ozo_direct(_i64(m), _i64(n), _i64(k), _p(np.ascontiguousarray(QA)),
                     _p(np.ascontiguousarray(QB)), _p(CI))
    return _ci_to_int(CI) if as_int else CI


def output(CI: np.ndarray, shiftA: np.ndarray, shiftB: np.ndarray, alpha: float = 1.0,
           beta: float = 0.0, C0: np.ndarray | None = None) -> np.ndarray:
    n, m, _ = CI.shape
    Cm = np.zeros((m, n), dtype=np.float64, order="F") if C0 is None else np.array(C0, order="F")
    lib().ozo_output(_i64(m), _i64(n), _p(np.ascontiguousarray(CI)), _p(shiftA), _p(shiftB),
                     C.c_double(alpha), C.c_double(beta), _p(Cm), _i64(max(m, 1)))
    return Cm


def dd_gemm(A: np.ndarray, B: np.ndarray):
    """Double-double reference product: (hi, lo, |A||B|), each m x n column-major."""
    _check_cm(A)
    _check_cm(B)
    m, k = A.shape
    n = B.shape[1]
    hi = np.zeros((m, n), dtype=np.float64, order="F")
    lo = np.zeros((m, n), dtype=np.float64, order="F")
    ab = np.zeros((m, n), dtype=np.float64, order="F")
    lib().ozo_dd_gemm(_i64(m), _i64(n), _i64(k), _p(A), _i64(max(m, 1)), _p(B), _i64(max(k, 1)),
                      _p(hi), _p(lo), _p(ab))
    return hi, lo, ab


def dgemm(A: np.ndarray, B: np.ndarray, s: int = SET_S, quant: int = QUANT_RN,
          rule: int = SCALE_CS, alpha: float = 1.0, beta: float = 0.0,
          C0: np.ndarray | None = None, want_stages: bool = False):
    """The whole method.  Returns C, or (C, shiftA, shiftB, R) with want_stages."""
    _check_cm(A)
    _check_cm(B)
    m, k = A.shape
    n = B.shape[1]
    r = len(modset(s))
    Cm = np.zeros((m, n), dtype=np.float64, order="F") if C0 is None else np.array(C0, order="F")
    sA = np.zeros(m, dtype=np.int32)
    sB = np.zeros(n, dtype=np.int32)
    R = np.zeros((r, n, m), dtype=np.uint16)
    rc = lib().ozo_dgemm(_i64(m), _i64(n), _i64(k), _p(A), _i64(max(m, 1)), _p(B),
                         _i64(max(k, 1)), _p(Cm), _i64(max(m, 1)), s, quant, rule,
                         C.c_double(alpha), C.c_double(beta), _p(sA), _p(sB), _p(R))
    assert rc == 0
    return (Cm, sA, sB, R) if want_stages else Cm

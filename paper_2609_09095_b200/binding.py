"""ctypes binding of include/oz.h -- argument marshalling only.

Names mirror the C entry points.  Tensors are torch CUDA tensors used purely as device buffers;
matrices are column-major, expressed as torch tensors of shape (cols, rows) that are contiguous
(so `t.T` is the m x n matrix), or any tensor for which the caller passes the leading dimension.
The library is required: importing a function when liboz_b200.so is missing raises.
"""
from __future__ import annotations

import ctypes as C
import os

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.environ.get("OZ_B200_LIB") or os.path.join(_HERE, "liboz_b200.so")

OZ_OK = 0
OZ_ERR_INVALID_ARG, OZ_ERR_UNSUPPORTED, OZ_ERR_WORKSPACE, OZ_ERR_CUDA = 1, 2, 3, 4
OZ_ERR_NONFINITE_INPUT, OZ_ERR_RANGE, OZ_ERR_TIMEOUT = 5, 6, 7
OZ_SET_S, OZ_SET_E, OZ_SET_A = 0, 1, 2
OZ_SUB_FP8, OZ_SUB_INT8, OZ_SUB_INT8_NATIVE = 0x001, 0x002, 0x004
OZ_QUANT_RN, OZ_QUANT_TZ = 0x010, 0x020
OZ_SCALE_MAXEXP, OZ_SCALE_CS, OZ_SCALE_ACCURATE = 0x100, 0x200, 0x400
OZ_ACC_MERGED, OZ_ACC_SEPARATE = 0x1000, 0x2000
OZ_RECON_TENSOR = 0x4000
OZ_FALLBACK_FP64 = 0x8000
OZ_STORAGE_FUSED = 0x10000
OZ_K_MAX = 1048576
OZ_NONFINITE_SHIFT = -(2 ** 31)
OZ_STATIC_MAX_LINES = 262144

EXPORTS = ["oz_set_info", "oz_plane_count", "oz_plane_count_side", "oz_row_pitch", "oz_residue_elem_bytes", "oz_workspace_bytes", "oz_set_workspace", "oz_dgemm",
           "oz_dgemm_ex", "oz_dgemm_host", "oz_operand_bytes", "oz_product_workspace_bytes", "oz_prepare_operand",
           "oz_dgemm_prepared", "oz_deconstruct", "oz_deconstruct_static",
           "oz_residue_gemm", "oz_reconstruct",
           "oz_query_status", "oz_query_fallback_rows", "oz_set_stage_events", "oz_launch_count", "oz_status_string"]

__all__ = EXPORTS + ["EXPORTS", "OzError", "load", "check", "LIB_PATH", "OZ_OK", "OZ_ERR_INVALID_ARG",
                     "OZ_ERR_UNSUPPORTED", "OZ_ERR_WORKSPACE", "OZ_ERR_CUDA",
                     "OZ_ERR_NONFINITE_INPUT", "OZ_ERR_RANGE", "OZ_ERR_TIMEOUT", "OZ_SET_S",
                     "OZ_SET_E", "OZ_SET_A", "OZ_SUB_FP8", "OZ_SUB_INT8", "OZ_SUB_INT8_NATIVE", "OZ_QUANT_RN", "OZ_QUANT_TZ",
                     "OZ_SCALE_MAXEXP", "OZ_SCALE_CS", "OZ_SCALE_ACCURATE", "OZ_ACC_MERGED", "OZ_ACC_SEPARATE", "OZ_RECON_TENSOR", "OZ_FALLBACK_FP64", "OZ_STORAGE_FUSED", "OZ_K_MAX", "OZ_NONFINITE_SHIFT", "OZ_STATIC_MAX_LINES"]

_lib = None


class OzError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__(f"{where}: {oz_status_string(code)} (status {code})")


def load() -> C.CDLL:
    """Load liboz_b200.so; there is no fallback implementation."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise ImportError(f"{LIB_PATH} is missing: build it with "
                          "`python -m paper_2609_09095_b200.build` (needs nvcc)")
    lib = C.CDLL(LIB_PATH)
    i64, u32, vp, dbl, i32 = C.c_int64, C.c_uint32, C.c_void_p, C.c_double, C.c_int
    lib.oz_set_info.argtypes = [i32, C.POINTER(i32), C.POINTER(i32), C.POINTER(i32)]
    lib.oz_plane_count.argtypes = [i32, u32]
    lib.oz_plane_count_side.argtypes = [i32, u32, i32]
    lib.oz_row_pitch.argtypes = [i64]
    lib.oz_row_pitch.restype = i64
    lib.oz_residue_elem_bytes.argtypes = [i32]
    lib.oz_residue_elem_bytes.restype = C.c_size_t
    lib.oz_workspace_bytes.argtypes = [i64, i64, i64, i32, u32]
    lib.oz_workspace_bytes.restype = C.c_size_t
    lib.oz_set_workspace.argtypes = [vp, C.c_size_t]
    lib.oz_dgemm.argtypes = [i64, i64, i64, vp, i64, vp, i64, vp, i64, i32, u32, vp]
    lib.oz_dgemm_ex.argtypes = [i64, i64, i64, dbl, vp, i64, vp, i64, dbl, vp, i64, i32, u32, vp]
    lib.oz_dgemm_host.argtypes = lib.oz_dgemm_ex.argtypes
    lib.oz_operand_bytes.argtypes = [i32, i64, i64, i32, u32]
    lib.oz_operand_bytes.restype = C.c_size_t
    lib.oz_product_workspace_bytes.argtypes = [i64, i64, i32]
    lib.oz_product_workspace_bytes.restype = C.c_size_t
    lib.oz_prepare_operand.argtypes = [i32, i64, i64, vp, i64, i32, u32, vp, C.c_size_t, vp]
    lib.oz_dgemm_prepared.argtypes = [i64, i64, i64, dbl, vp, vp, dbl, vp, i64, i32, u32, vp]
    lib.oz_deconstruct.argtypes = [i32, i64, i64, vp, i64, i32, u32, vp, i64, i64, vp, vp, vp]
    lib.oz_deconstruct_static.argtypes = [i32, i64, i64, vp, i64, i32, u32, vp, i64, i64, vp, vp]
    lib.oz_residue_gemm.argtypes = [i64, i64, i64, vp, i64, i64, vp, i64, i64, i32, u32, vp, i64,
                                    i64, vp]
    lib.oz_reconstruct.argtypes = [i64, i64, vp, i64, i64, vp, vp, i32, dbl, dbl, vp, i64, vp]
    lib.oz_query_status.argtypes = [vp]
    lib.oz_query_fallback_rows.argtypes = [vp, C.POINTER(C.c_int64)]
    lib.oz_set_stage_events.argtypes = [C.POINTER(vp)]
    lib.oz_launch_count.restype = C.c_uint64
    lib.oz_status_string.argtypes = [i32]
    lib.oz_status_string.restype = C.c_char_p
    _lib = lib
    return lib


def _ptr(t) -> int:
    """Device (or pinned host) address of a torch tensor, or a raw integer address."""
    if t is None:
        return 0
    if isinstance(t, int):
        return t
    return t.data_ptr()


def _stream(stream) -> int:
    if stream is None:
        import torch
        return torch.cuda.current_stream().cuda_stream
    if isinstance(stream, int):
        return stream
    return stream.cuda_stream


def check(code: int, where: str = "oz") -> None:
    if code != OZ_OK:
        raise OzError(code, where)


def oz_status_string(code: int) -> str:
    return load().oz_status_string(code).decode()


def oz_set_info(modset: int):
    r, p = C.c_int(), C.c_int()
    mod = (C.c_int * 16)()
    check(load().oz_set_info(modset, C.byref(r), C.byref(p), mod), "oz_set_info")
    return r.value, p.value, [mod[i] for i in range(r.value)]


def oz_plane_count(modset: int, route: int = 0) -> int:
    return load().oz_plane_count(modset, route)


def oz_plane_count_side(modset: int, route: int, side: int) -> int:
    return load().oz_plane_count_side(modset, route, side)


def oz_row_pitch(k: int) -> int:
    return load().oz_row_pitch(k)


def oz_residue_elem_bytes(modset: int) -> int:
    return load().oz_residue_elem_bytes(modset)


def oz_workspace_bytes(m, n, k, modset, route=0) -> int:
    return load().oz_workspace_bytes(m, n, k, modset, route)


def oz_set_workspace(workspace, nbytes: int | None = None) -> int:
    if workspace is None:
        return load().oz_set_workspace(None, 0)
    if nbytes is None:
        nbytes = workspace.numel() * workspace.element_size()
    return load().oz_set_workspace(_ptr(workspace), nbytes)


def oz_dgemm(m, n, k, A, lda, B, ldb, Cm, ldc, modset=OZ_SET_S, route=0, stream=None) -> int:
    return load().oz_dgemm(m, n, k, _ptr(A), lda, _ptr(B), ldb, _ptr(Cm), ldc, modset, route,
                           _stream(stream))


def oz_dgemm_ex(m, n, k, alpha, A, lda, B, ldb, beta, Cm, ldc, modset=OZ_SET_S, route=0,
                stream=None) -> int:
    return load().oz_dgemm_ex(m, n, k, alpha, _ptr(A), lda, _ptr(B), ldb, beta, _ptr(Cm), ldc,
                              modset, route, _stream(stream))


def oz_dgemm_host(m, n, k, alpha, A, lda, B, ldb, beta, Cm, ldc, modset=OZ_SET_S, route=0,
                  stream=None) -> int:
    """A, B, Cm are HOST tensors (pinned) or raw host addresses."""
    return load().oz_dgemm_host(m, n, k, alpha, _ptr(A), lda, _ptr(B), ldb, beta, _ptr(Cm), ldc,
                                modset, route, _stream(stream))


def oz_operand_bytes(side, lines, k, modset, route=0) -> int:
    return load().oz_operand_bytes(side, lines, k, modset, route)


def oz_product_workspace_bytes(m, n, modset) -> int:
    return load().oz_product_workspace_bytes(m, n, modset)


def oz_prepare_operand(side, lines, k, X, ldx, modset, route, operand, nbytes=None, stream=None) -> int:
    if nbytes is None:
        nbytes = operand.numel() * operand.element_size()
    return load().oz_prepare_operand(side, lines, k, _ptr(X), ldx, modset, route, _ptr(operand), nbytes,
                                     _stream(stream))


def oz_dgemm_prepared(m, n, k, alpha, operandA, operandB, beta, Cm, ldc, modset=OZ_SET_S, route=0,
                      stream=None) -> int:
    return load().oz_dgemm_prepared(m, n, k, alpha, _ptr(operandA), _ptr(operandB), beta, _ptr(Cm), ldc,
                                    modset, route, _stream(stream))


def oz_deconstruct(side, lines, k, X, ldx, modset, route, planes, plane_stride, row_pitch, shift,
                   scratch, stream=None) -> int:
    return load().oz_deconstruct(side, lines, k, _ptr(X), ldx, modset, route, _ptr(planes),
                                 plane_stride, row_pitch, _ptr(shift), _ptr(scratch),
                                 _stream(stream))


def oz_deconstruct_static(side, lines, k, X, ldx, modset, route, planes, plane_stride, row_pitch,
                          shift, stream=None) -> int:
    """oz_deconstruct with the scan scratch held inside the library: for callers that cannot
    allocate device memory.  At most OZ_STATIC_MAX_LINES lines; calls must not overlap on the GPU."""
    return load().oz_deconstruct_static(side, lines, k, _ptr(X), ldx, modset, route, _ptr(planes),
                                        plane_stride, row_pitch, _ptr(shift), _stream(stream))


def oz_residue_gemm(m, n, k, PA, strideA, pitchA, PB, strideB, pitchB, modset, route, R, ldr,
                    mod_stride, stream=None) -> int:
    return load().oz_residue_gemm(m, n, k, _ptr(PA), strideA, pitchA, _ptr(PB), strideB, pitchB,
                                  modset, route, _ptr(R), ldr, mod_stride, _stream(stream))


def oz_reconstruct(m, n, R, ldr, mod_stride, shiftA, shiftB, modset, alpha, beta, Cm, ldc,
                   stream=None) -> int:
    return load().oz_reconstruct(m, n, _ptr(R), ldr, mod_stride, _ptr(shiftA), _ptr(shiftB), modset,
                                 alpha, beta, _ptr(Cm), ldc, _stream(stream))


def oz_query_status(stream=None) -> int:
    return load().oz_query_status(_stream(stream))


def oz_query_fallback_rows(stream=None) -> int:
    """Rows re-issued on the native FP64 path since the last such query (synchronises the stream)."""
    rows = C.c_int64(0)
    check(load().oz_query_fallback_rows(_stream(stream), C.byref(rows)), "oz_query_fallback_rows")
    return int(rows.value)


def oz_set_stage_events(events) -> int:
    """events: five torch.cuda.Event objects (already recorded once, so their handles exist),
    five raw cudaEvent_t addresses, or None."""
    if events is None:
        return load().oz_set_stage_events(None)
    arr = (C.c_void_p * 5)(*[e if isinstance(e, int) else e.cuda_event for e in events])
    return load().oz_set_stage_events(arr)


def oz_launch_count() -> int:
    return int(load().oz_launch_count())

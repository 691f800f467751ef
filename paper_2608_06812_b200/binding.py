"""ctypes binding of libozk.so: the same names and arguments as include/ozk.h.

Only argument marshalling happens here.  Pointers are plain integers (device
addresses, e.g. torch.Tensor.data_ptr()); `stream` is a cudaStream_t as an
integer (torch.cuda.current_stream().cuda_stream), 0 for the default stream.
The library is loaded on first use and a missing build is an error: there is
no fallback path.
"""
from __future__ import annotations

import ctypes
import os
from ctypes import c_char, c_char_p, c_int, c_int64, c_size_t, c_void_p

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libozk.so")

OZK_OK = 0
OZK_ERR_INVALID_ARG = -1
OZK_ERR_UNSUPPORTED = -2
OZK_ERR_WORKSPACE = -3
OZK_ERR_CUDA = -4
OZK_ERR_NONFINITE = -5
OZK_ERR_DEVICE_TIMEOUT = -6
OZK_MIN_MODULI, OZK_MAX_MODULI, OZK_DEFAULT_MODULI = 2, 27, 19
OZK_CHUNK_K, OZK_MAX_K = 131072, 2097152
OZK_MAX_EXTENDED_BITS = 62

# name -> (restype, argtypes): every symbol include/ozk.h declares
SIGNATURES = {
    "ozk_get_moduli": (c_int, [c_int, c_void_p]),
    "ozk_capacity_bits": (c_int, [c_int64, c_int]),
    "ozk_get_crt_constants": (c_int, [c_int, c_void_p, c_void_p]),
    "ozk_status_string": (c_char_p, [c_int]),
    "ozk_version": (c_char_p, []),
    "ozk_dgemm_workspace_bytes": (c_size_t, [c_int64, c_int64, c_int64, c_int]),
    "ozk_igemm_i8_workspace_bytes": (c_size_t, [c_int64, c_int64, c_int64]),
    "ozk_set_workspace": (c_int, [c_void_p, c_size_t]),
    "ozk_get_async_status": (c_int, [c_void_p]),
    "ozk_dgemm": (c_int, [c_int64, c_int64, c_int64, c_void_p, c_int64, c_void_p, c_int64, c_void_p, c_int64, c_int, c_void_p]),
    "ozk_capacity_bits_ext": (c_int, [c_int64, c_int, c_int]),
    "ozk_dgemm_ext": (c_int, [c_int64, c_int64, c_int64, c_void_p, c_int64, c_void_p, c_int64, c_void_p, c_int64, c_int, c_int, c_void_p]),
    "ozk_igemm_i8": (c_int, [c_int64, c_int64, c_int64, c_void_p, c_int64, c_void_p, c_int64, c_void_p, c_int64, c_void_p]),
    "ozk_dgemm_host_workspace_bytes": (c_size_t, [c_int64, c_int64, c_int64, c_int]),
    "ozk_dgemm_host": (c_int, [c_int64, c_int64, c_int64, c_void_p, c_int64, c_void_p, c_int64, c_void_p, c_int64, c_int, c_void_p]),
    "ozk_dgemm_oz1_workspace_bytes": (c_size_t, [c_int64, c_int64, c_int64]),
    "ozk_dgemm_oz1": (c_int, [c_int64, c_int64, c_int64, c_void_p, c_int64, c_void_p, c_int64, c_void_p, c_int64, c_void_p]),
    "ozk_stage_preprocess": (c_int, [c_int64, c_int64, c_int64, c_void_p, c_int64, c_void_p, c_int64, c_int,
                                     c_void_p, c_void_p, c_void_p, c_void_p, c_void_p]),
    "ozk_stage_read_planes": (c_int, [c_char, c_int64, c_int64, c_int64, c_int, c_int, c_int, c_void_p, c_void_p]),
    "ozk_stage_residue_gemm": (c_int, [c_int64, c_int64, c_int64, c_int, c_void_p, c_void_p]),
    "ozk_stage_crt": (c_int, [c_int64, c_int64, c_int64, c_int, c_void_p, c_void_p, c_void_p, c_void_p, c_int64,
                              c_void_p, c_void_p]),
    "ozk_stage_wait_probe": (c_int, [c_void_p]),
    "ozk_row_shifts_noalloc": (c_int, [c_int64, c_int64, c_void_p, c_int64, c_int, c_void_p, c_void_p]),
    "ozk_stage_timing_enable": (c_int, [c_int]),
    "ozk_stage_gemm_cycles": (c_int, [c_void_p]),
    "ozk_stage_set_karatsuba": (c_int, [c_int]),
    "ozk_stage_timing_read": (c_int, [c_void_p]),
    "ozk_stage_mma_probe": (c_int, [c_void_p, c_void_p, c_int64, c_int, c_void_p, c_void_p]),
}

_lib = None


def lib() -> ctypes.CDLL:
    """The loaded library; raises if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: build it with `python -m paper_2608_06812_b200.build`")
        handle = ctypes.CDLL(LIB_PATH)
        for name, (res, args) in SIGNATURES.items():
            fn = getattr(handle, name)
            fn.restype, fn.argtypes = res, args
        _lib = handle
    return _lib


class OzkError(RuntimeError):
    def __init__(self, status: int, call: str):
        self.status = status
        super().__init__(f"{call}: {ozk_status_string(status)} ({status})")


def check(status: int, call: str) -> None:
    if status != OZK_OK:
        raise OzkError(status, call)


def ozk_status_string(status: int) -> str:
    return lib().ozk_status_string(status).decode()


def ozk_version() -> str:
    return lib().ozk_version().decode()


def ozk_get_moduli(num_moduli: int) -> list[int]:
    buf = (c_int * max(num_moduli, 1))()
    n = lib().ozk_get_moduli(num_moduli, buf)
    if n < 0:
        raise OzkError(n, "ozk_get_moduli")
    return list(buf[:n])


def ozk_capacity_bits(K: int, num_moduli: int) -> int:
    return lib().ozk_capacity_bits(K, num_moduli)


def ozk_capacity_bits_ext(K: int, num_moduli: int, max_bits: int) -> int:
    return lib().ozk_capacity_bits_ext(K, num_moduli, max_bits)


def ozk_get_crt_constants(num_moduli: int) -> tuple[int, list[int]]:
    """P and the weights w_l as Python integers."""
    P = (ctypes.c_uint32 * 6)()
    W = (ctypes.c_uint32 * (6 * num_moduli))()
    check(lib().ozk_get_crt_constants(num_moduli, P, W), "ozk_get_crt_constants")
    join = lambda words: sum(int(w) << (32 * i) for i, w in enumerate(words))
    return join(P), [join(W[6 * l:6 * l + 6]) for l in range(num_moduli)]


def ozk_dgemm_workspace_bytes(M: int, N: int, K: int, num_moduli: int) -> int:
    return lib().ozk_dgemm_workspace_bytes(M, N, K, num_moduli)


def ozk_igemm_i8_workspace_bytes(M: int, N: int, K: int) -> int:
    return lib().ozk_igemm_i8_workspace_bytes(M, N, K)


def ozk_set_workspace(dev_ptr: int, nbytes: int) -> int:
    return lib().ozk_set_workspace(dev_ptr, nbytes)


def ozk_get_async_status(stream: int = 0) -> int:
    return lib().ozk_get_async_status(stream)


def ozk_dgemm(M, N, K, A, lda, B, ldb, C, ldc, num_moduli, stream=0) -> int:
    return lib().ozk_dgemm(M, N, K, A, lda, B, ldb, C, ldc, num_moduli, stream)


def ozk_dgemm_ext(M, N, K, A, lda, B, ldb, C, ldc, num_moduli, max_bits, stream=0) -> int:
    return lib().ozk_dgemm_ext(M, N, K, A, lda, B, ldb, C, ldc, num_moduli, max_bits, stream)


def ozk_igemm_i8(M, N, K, A, lda, B, ldb, C, ldc, stream=0) -> int:
    return lib().ozk_igemm_i8(M, N, K, A, lda, B, ldb, C, ldc, stream)


def ozk_stage_preprocess(M, N, K, A, lda, B, ldb, num_moduli, s_out=None, t_out=None, At_out=None, Bt_out=None, stream=0) -> int:
    return lib().ozk_stage_preprocess(M, N, K, A, lda, B, ldb, num_moduli, s_out, t_out, At_out, Bt_out, stream)


def ozk_stage_read_planes(operand: str, M, N, K, num_moduli, l, limb, out, stream=0) -> int:
    return lib().ozk_stage_read_planes(operand.encode(), M, N, K, num_moduli, l, limb, out, stream)


def ozk_stage_residue_gemm(M, N, K, num_moduli, residues_out=None, stream=0) -> int:
    return lib().ozk_stage_residue_gemm(M, N, K, num_moduli, residues_out, stream)


def ozk_stage_crt(M, N, K, num_moduli, residues_in, s_in, t_in, C, ldc, x_out=None, stream=0) -> int:
    return lib().ozk_stage_crt(M, N, K, num_moduli, residues_in, s_in, t_in, C, ldc, x_out, stream)


def ozk_stage_mma_probe(P, Q, K, scale_byte, D, stream=0) -> int:
    return lib().ozk_stage_mma_probe(P, Q, K, scale_byte, D, stream)


def ozk_stage_timing_enable(enable: bool) -> int:
    return lib().ozk_stage_timing_enable(1 if enable else 0)


def ozk_stage_timing_read() -> tuple[float, float, float]:
    ms = (ctypes.c_float * 3)()
    check(lib().ozk_stage_timing_read(ms), "ozk_stage_timing_read")
    return float(ms[0]), float(ms[1]), float(ms[2])


def ozk_stage_set_karatsuba(enable: bool) -> int:
    return lib().ozk_stage_set_karatsuba(1 if enable else 0)


def ozk_stage_gemm_cycles() -> tuple[int, int, int]:
    """Clocks of the limb GEMM's issuing thread: (whole kernel, waiting for tensor memory, waiting for operands)."""
    clk = (ctypes.c_longlong * 3)()
    check(lib().ozk_stage_gemm_cycles(clk), "ozk_stage_gemm_cycles")
    return int(clk[0]), int(clk[1]), int(clk[2])


def ozk_stage_wait_probe(stream=0) -> int:
    return lib().ozk_stage_wait_probe(stream)


def ozk_row_shifts_noalloc(M, K, A, lda, num_moduli, s_out, stream=0) -> int:
    """Row shifts of A without any workspace: the scratch is a fixed 512 KiB array inside the
    library (at most 65536 rows), for callers that may not allocate device memory."""
    return lib().ozk_row_shifts_noalloc(M, K, A, lda, num_moduli, s_out, stream)


def ozk_dgemm_oz1_workspace_bytes(M: int, N: int, K: int) -> int:
    return lib().ozk_dgemm_oz1_workspace_bytes(M, N, K)


def ozk_dgemm_oz1(M, N, K, A, lda, B, ldb, C, ldc, stream=0) -> int:
    return lib().ozk_dgemm_oz1(M, N, K, A, lda, B, ldb, C, ldc, stream)


def ozk_dgemm_host_workspace_bytes(M: int, N: int, K: int, num_moduli: int) -> int:
    return lib().ozk_dgemm_host_workspace_bytes(M, N, K, num_moduli)


def ozk_dgemm_host(M, N, K, A, lda, B, ldb, C, ldc, num_moduli, stream=0) -> int:
    """A, B, C are HOST addresses (pinned memory for full speed)."""
    return lib().ozk_dgemm_host(M, N, K, A, lda, B, ldb, C, ldc, num_moduli, stream)

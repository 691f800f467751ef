"""Helpers for the GPU tests: device buffers through torch, column-major marshalling."""
from __future__ import annotations

import numpy as np
import torch

from paper_2608_06812_b200 import binding as ozk

_ws = {"buf": None}


def stream() -> int:
    return torch.cuda.current_stream().cuda_stream


def _register(buf: torch.Tensor, nbytes: int) -> None:
    """Registers the buffer from an odd multiple of 256 bytes on: the least alignment the library accepts."""
    offset = (-buf.data_ptr()) % 512 + 256
    ozk.check(ozk.ozk_set_workspace(buf.data_ptr() + offset, nbytes), "ozk_set_workspace")


def ensure_workspace(nbytes: int) -> None:
    """One growing device workspace shared by all tests of a process."""
    nbytes = max(int(nbytes), 1 << 20)
    buf = _ws["buf"]
    if buf is None or buf.numel() < nbytes + 1024:
        torch.cuda.synchronize()
        _ws["buf"] = None
        buf = torch.empty(nbytes + 1024, dtype=torch.uint8, device="cuda")
        _ws["buf"] = buf
        _register(buf, buf.numel() - 1024)


def register_small_workspace(nbytes: int = 1 << 20) -> None:
    """Registers a fresh workspace of exactly nbytes (for tests of the 'workspace too small' error);
    the next ensure_workspace() call replaces it."""
    torch.cuda.synchronize()
    _ws["buf"] = None
    buf = torch.empty(nbytes + 1024, dtype=torch.uint8, device="cuda")
    _register(buf, nbytes)
    _ws["small"] = buf


def to_dev_colmajor(X: np.ndarray, ld: int | None = None) -> torch.Tensor:
    """Uploads X[r, c] as a column-major device buffer with leading dimension ld."""
    rows, cols = X.shape
    ld = rows if ld is None else ld
    host = np.zeros((cols, ld), dtype=X.dtype)
    host[:, :rows] = X.T
    return torch.from_numpy(host).cuda()


def from_dev_colmajor(T: torch.Tensor, rows: int, cols: int) -> np.ndarray:
    """Inverse of to_dev_colmajor for a (cols, ld) device tensor."""
    return T.cpu().numpy()[:cols, :rows].T.copy()


def dgemm(A: np.ndarray, B: np.ndarray, L: int, lda=None, ldb=None, ldc=None, max_bits=None) -> np.ndarray:
    """ozk_dgemm (or ozk_dgemm_ext when max_bits is given) on freshly uploaded column-major copies."""
    M, K = A.shape
    _, N = B.shape
    lda = max(M, 1) if lda is None else lda
    ldb = max(K, 1) if ldb is None else ldb
    ldc = max(M, 1) if ldc is None else ldc
    ensure_workspace(ozk.ozk_dgemm_workspace_bytes(M, N, K, L))
    dA, dB = to_dev_colmajor(A, lda), to_dev_colmajor(B, ldb)
    dC = torch.full((max(N, 1), ldc), float("nan"), dtype=torch.float64, device="cuda")
    if max_bits is None:
        ozk.check(ozk.ozk_dgemm(M, N, K, dA.data_ptr(), lda, dB.data_ptr(), ldb, dC.data_ptr(), ldc, L, stream()), "ozk_dgemm")
    else:
        ozk.check(ozk.ozk_dgemm_ext(M, N, K, dA.data_ptr(), lda, dB.data_ptr(), ldb, dC.data_ptr(), ldc, L, max_bits, stream()),
                  "ozk_dgemm_ext")
    ozk.check(ozk.ozk_get_async_status(stream()), "ozk_get_async_status")
    return from_dev_colmajor(dC, M, N)


def bits_equal(X: np.ndarray, Y: np.ndarray) -> bool:
    return np.array_equal(np.ascontiguousarray(X).view(np.uint64), np.ascontiguousarray(Y).view(np.uint64))

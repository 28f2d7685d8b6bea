"""Python face of the CPU oracle (ctypes over oracle/libubp_oracle.so).

TEST INFRASTRUCTURE ONLY: imported by tests/, by the smoke check and by the
benchmark's CPU-baseline leg. The product package never imports this module
and this module never imports the product package.

Every function forwards to the C function of the same name (see
ubp_oracle.c for what each computes and which passage of the paper it
follows); this file only marshals numpy arrays.
"""
from __future__ import annotations

import ctypes as C
from typing import Optional, Tuple

import numpy as np

from .build import build as _build

_lib = None

OK, E_ARG, E_RAGGED, E_SPACE, E_FORMAT = 0, -1, -2, -3, -4


class OracleError(RuntimeError):
    def __init__(self, code: int, what: str):
        super().__init__(f"{what}: oracle error {code}")
        self.code = code


def lib():
    global _lib
    if _lib is None:
        L = C.CDLL(_build())
        L.orc_block_budget.restype = C.c_int64
        L.orc_block_budget.argtypes = [C.c_int64, C.c_int64, C.c_int, C.c_int]
        L.orc_blob_size.restype = C.c_size_t
        L.orc_blob_size.argtypes = [C.c_int, C.c_int, C.c_int, C.c_int64]
        L.orc_num_threads.restype = C.c_int
        for f in (L.orc_bed_expand, L.orc_greedy_select, L.orc_optimal_select):
            f.restype = C.c_int64
        _lib = L
    return _lib


def _p(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


def _chk(rc: int, what: str):
    if rc != 0:
        raise OracleError(rc, what)


def num_threads() -> int:
    return int(lib().orc_num_threads())


def block_budget(M: int, Cin: int, sparsity_pct: int, Nb: int) -> int:
    return int(lib().orc_block_budget(M, Cin, sparsity_pct, Nb))


def decode_mask(mask: np.ndarray, Nb: int) -> Tuple[np.ndarray, np.ndarray]:
    """Blocks (start row i, input channel j) of a mask, in k = i + M*j order."""
    mask = np.ascontiguousarray(mask, dtype=np.uint8)
    M, Cin = mask.shape
    n = C.c_int64(0)
    _chk(lib().orc_decode_mask(_p(mask), M, Cin, Nb, None, None, C.c_int64(0), C.byref(n)), "decode_mask")
    bi = np.zeros(max(n.value, 1), np.int32)
    bj = np.zeros(max(n.value, 1), np.int32)
    _chk(lib().orc_decode_mask(_p(mask), M, Cin, Nb, _p(bi), _p(bj), C.c_int64(n.value), C.byref(n)),
         "decode_mask")
    return bi[:n.value].copy(), bj[:n.value].copy()


def pack(W: np.ndarray, mask: np.ndarray, Nb: int) -> bytes:
    """Canonical packed blob of (W [M][C][R] or [M][C], mask [M][C])."""
    mask = np.ascontiguousarray(mask, dtype=np.uint8)
    M, Cin = mask.shape
    W = np.ascontiguousarray(W, dtype=np.float32).reshape(M, Cin, -1)
    R = W.shape[2]
    ln = C.c_size_t(0)
    _chk(lib().orc_pack(_p(W), _p(mask), M, Cin, R, Nb, None, C.c_size_t(0), C.byref(ln)), "pack")
    buf = np.zeros(ln.value, np.uint8)
    _chk(lib().orc_pack(_p(W), _p(mask), M, Cin, R, Nb, _p(buf), C.c_size_t(ln.value), C.byref(ln)), "pack")
    return buf.tobytes()


def blob_dims(blob: bytes):
    b = np.frombuffer(blob, np.uint8)
    d = np.zeros(5, np.int32)
    _chk(lib().orc_blob_dims(_p(b), C.c_size_t(b.size), _p(d)), "blob_dims")
    return tuple(int(x) for x in d)  # M, C, R, Nb, m


def unpack(blob: bytes) -> Tuple[np.ndarray, np.ndarray]:
    b = np.frombuffer(blob, np.uint8)
    M, Cin, R, Nb, m = blob_dims(blob)
    W = np.empty((M, Cin, R), np.float32)
    mask = np.empty((M, Cin), np.uint8)
    _chk(lib().orc_unpack(_p(b), C.c_size_t(b.size), _p(W), _p(mask)), "unpack")
    return W, mask


def masked_matmul(W, mask, X, bias=None, relu=False, want_scale=True):
    """Y = act((W*mask) @ X + bias) in double; also the error scale
    A = |W*mask| @ |X| + |bias| when want_scale."""
    mask = np.ascontiguousarray(mask, dtype=np.uint8)
    M, Cin = mask.shape
    W = np.ascontiguousarray(W, dtype=np.float32).reshape(M, Cin)
    X = np.ascontiguousarray(X, dtype=np.float32).reshape(Cin, -1)
    Nc = X.shape[1]
    bias = None if bias is None else np.ascontiguousarray(bias, dtype=np.float32)
    Y = np.empty((M, Nc), np.float64)
    A = np.empty((M, Nc), np.float64) if want_scale else None
    _chk(lib().orc_masked_matmul(_p(W), _p(mask), M, Cin, _p(X), C.c_int64(Nc), C.c_int64(Nc),
                                 _p(bias), int(bool(relu)), _p(Y), _p(A)), "masked_matmul")
    return (Y, A) if want_scale else Y


def masked_matmul_samples(W, mask, X, so, sn, bias=None, relu=False):
    mask = np.ascontiguousarray(mask, dtype=np.uint8)
    M, Cin = mask.shape
    W = np.ascontiguousarray(W, dtype=np.float32).reshape(M, Cin)
    X = np.ascontiguousarray(X, dtype=np.float32).reshape(Cin, -1)
    Nc = X.shape[1]
    so = np.ascontiguousarray(so, dtype=np.int32)
    sn = np.ascontiguousarray(sn, dtype=np.int64)
    bias = None if bias is None else np.ascontiguousarray(bias, dtype=np.float32)
    Y = np.empty(so.size, np.float64)
    A = np.empty(so.size, np.float64)
    _chk(lib().orc_masked_matmul_samples(_p(W), _p(mask), M, Cin, _p(X), C.c_int64(Nc), C.c_int64(Nc),
                                         _p(bias), int(bool(relu)), _p(so), _p(sn), C.c_int64(so.size),
                                         _p(Y), _p(A)), "masked_matmul_samples")
    return Y, A


def masked_conv3x3(W, mask, In, bias=None, relu=False):
    """In: [C][B][H][Wd] (channel-major). Returns Y, A as [M][B][H][Wd] double."""
    mask = np.ascontiguousarray(mask, dtype=np.uint8)
    M, Cin = mask.shape
    W = np.ascontiguousarray(W, dtype=np.float32).reshape(M, Cin, 9)
    In = np.ascontiguousarray(In, dtype=np.float32)
    _, B, H, Wd = In.shape
    bias = None if bias is None else np.ascontiguousarray(bias, dtype=np.float32)
    Y = np.empty((M, B, H, Wd), np.float64)
    A = np.empty((M, B, H, Wd), np.float64)
    hw = H * Wd
    _chk(lib().orc_masked_conv3x3(_p(W), _p(mask), M, Cin, _p(In), B, H, Wd,
                                  C.c_int64(hw), C.c_int64(B * hw), _p(bias), int(bool(relu)),
                                  _p(Y), _p(A), C.c_int64(hw), C.c_int64(B * hw)), "masked_conv3x3")
    return Y, A


def masked_conv3x3_samples(W, mask, In, sb, so, sy, sx, bias=None, relu=False):
    mask = np.ascontiguousarray(mask, dtype=np.uint8)
    M, Cin = mask.shape
    W = np.ascontiguousarray(W, dtype=np.float32).reshape(M, Cin, 9)
    In = np.ascontiguousarray(In, dtype=np.float32)
    _, B, H, Wd = In.shape
    bias = None if bias is None else np.ascontiguousarray(bias, dtype=np.float32)
    sb, so, sy, sx = (np.ascontiguousarray(a, dtype=np.int32) for a in (sb, so, sy, sx))
    Y = np.empty(sb.size, np.float64)
    A = np.empty(sb.size, np.float64)
    hw = H * Wd
    _chk(lib().orc_masked_conv3x3_samples(_p(W), _p(mask), M, Cin, _p(In), B, H, Wd,
                                          C.c_int64(hw), C.c_int64(B * hw), _p(bias), int(bool(relu)),
                                          _p(sb), _p(so), _p(sy), _p(sx), C.c_int64(sb.size),
                                          _p(Y), _p(A)), "masked_conv3x3_samples")
    return Y, A


def wros_spmm(blob: bytes, X, bias=None, relu=False, tile_w: int = 4):
    """The paper's weight-rotating output-stationary walk over the packed blob."""
    b = np.frombuffer(blob, np.uint8)
    M, Cin, R, Nb, m = blob_dims(blob)
    X = np.ascontiguousarray(X, dtype=np.float32).reshape(Cin, -1)
    Nc = X.shape[1]
    bias = None if bias is None else np.ascontiguousarray(bias, dtype=np.float32)
    Y = np.empty((M, Nc), np.float64)
    _chk(lib().orc_wros_spmm(_p(b), C.c_size_t(b.size), _p(X), C.c_int64(Nc), C.c_int64(Nc),
                             _p(bias), int(bool(relu)), int(tile_w), _p(Y)), "wros_spmm")
    return Y


# ---------------------------------------------------------------------------
# Block selection (Section 3.1 Eq. 1, Section 3.2 Eq. 3 and Eq. 4, Section 4.1
# Algorithms 1 and 2). Candidate index k = i + M*j (start row i, input channel j).
# ---------------------------------------------------------------------------

def block_scores(W: np.ndarray, Nb: int) -> np.ndarray:
    """Eq. 1 scores as a float32 vector of length C*M (k = i + M*j); -inf where i + Nb > M."""
    W = np.ascontiguousarray(W, dtype=np.float32)
    M, Cin = W.shape[:2]
    W = W.reshape(M, Cin, -1)
    S = np.empty(M * Cin, np.float32)
    _chk(lib().orc_block_scores(_p(W), M, Cin, W.shape[2], Nb, _p(S)), "block_scores")
    return S


def bed_expand(S: np.ndarray, Nb: int, m: int) -> Tuple[np.ndarray, np.ndarray]:
    """Algorithm 1: the chosen original indices, in the order chosen, and their scores when chosen."""
    S = np.ascontiguousarray(S, dtype=np.float32)
    Ibar = np.zeros(max(m, 1), np.int64)
    sc = np.zeros(max(m, 1), np.float32)
    n = int(lib().orc_bed_expand(_p(S), C.c_int64(S.size), Nb, C.c_int64(m), _p(Ibar), _p(sc)))
    if n < 0:
        raise OracleError(n, "bed_expand")
    return Ibar[:n].copy(), sc[:n].copy()


def bed_divide(Ibar: np.ndarray, Nb: int) -> np.ndarray:
    """Algorithm 2: final block start indices, ascending."""
    Ibar = np.ascontiguousarray(Ibar, dtype=np.int64)
    I = np.zeros(max(Ibar.size, 1), np.int64)
    _chk(lib().orc_bed_divide(_p(Ibar), C.c_int64(Ibar.size), Nb, _p(I)), "bed_divide")
    return I[:Ibar.size].copy()


def greedy_select(S: np.ndarray, Nb: int, m: int) -> np.ndarray:
    """Eq. 3: block start indices in the order chosen."""
    S = np.ascontiguousarray(S, dtype=np.float32)
    I = np.zeros(max(m, 1), np.int64)
    n = int(lib().orc_greedy_select(_p(S), C.c_int64(S.size), Nb, C.c_int64(m), _p(I)))
    if n < 0:
        raise OracleError(n, "greedy_select")
    return I[:n].copy()


def optimal_select(S: np.ndarray, Nb: int, m: int) -> Tuple[Optional[np.ndarray], float]:
    """Eq. 4: (ascending block start indices or None when m blocks do not fit, best total)."""
    S = np.ascontiguousarray(S, dtype=np.float32)
    I = np.zeros(max(m, 1), np.int64)
    tot = C.c_double(0.0)
    n = int(lib().orc_optimal_select(_p(S), C.c_int64(S.size), Nb, C.c_int64(m), _p(I), C.byref(tot)))
    if n < -1:
        raise OracleError(n, "optimal_select")
    return (I[:m].copy() if n == m else None), float(tot.value)


def starts_to_mask(I: np.ndarray, M: int, Cin: int, Nb: int) -> np.ndarray:
    I = np.ascontiguousarray(I, dtype=np.int64)
    mask = np.empty((M, Cin), np.uint8)
    _chk(lib().orc_starts_to_mask(_p(I), C.c_int64(I.size), M, Cin, Nb, _p(mask)), "starts_to_mask")
    return mask


def bed_select(W: np.ndarray, Nb: int, m: int):
    """Scores, expansion, division, mask: returns (mask [M][C] uint8, I ascending, Ibar in the order chosen)."""
    M, Cin = W.shape[:2]
    S = block_scores(W, Nb)
    Ibar, _ = bed_expand(S, Nb, m)
    I = bed_divide(Ibar, Nb)
    return starts_to_mask(I, M, Cin, Nb), I, Ibar

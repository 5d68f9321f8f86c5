"""CPU oracle (fp64) for the codebook-binary linear layer.

TEST INFRASTRUCTURE ONLY: imported by tests/, the smoke check and the
benchmark's CPU-baseline leg.  It shares nothing with the CUDA package and
the CUDA package never imports it.  The arithmetic lives in btc_oracle.c (plain
C, fp64, the paper's definitions written out); this module only builds that
file with gcc, converts fp16/bf16 bit patterns to fp64 exactly and marshals
arrays.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from typing import Optional

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "btc_oracle.c")
_SO = os.path.join(_HERE, "libbtc_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile btc_oracle.c into libbtc_oracle.so (gcc -O2 -fopenmp, no fast-math)."""
    if force or not os.path.exists(_SO) or os.path.getmtime(_SO) < os.path.getmtime(_SRC):
        tmp = _SO + f".tmp{os.getpid()}"
        subprocess.check_call(["gcc", "-O2", "-fopenmp", "-fPIC", "-shared", "-std=c11",
                               "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _SO)
    return _SO


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        lib.btc_oracle_bits_per_weight.restype = ctypes.c_double
        lib.btc_oracle_storage_bits.restype = ctypes.c_double
        lib.btc_oracle_sqdist_pm1.restype = ctypes.c_double
        _lib = lib
    return _lib


def _p(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def threads() -> int:
    return int(_load().btc_oracle_threads())


def to_f64(bits_or_float: np.ndarray, dtype: str) -> np.ndarray:
    """Exact widening of fp16 / bf16 bit patterns (uint16) or float arrays to fp64."""
    a = np.asarray(bits_or_float)
    if dtype == "f16":
        if a.dtype == np.uint16:
            a = a.view(np.float16)
        return np.ascontiguousarray(a.astype(np.float64))
    if dtype == "bf16":
        if a.dtype != np.uint16:
            raise TypeError("bf16 inputs are passed as uint16 bit patterns")
        f32 = (a.astype(np.uint32) << np.uint32(16)).view(np.float32)
        return np.ascontiguousarray(f32.astype(np.float64))
    if dtype in ("f32", "f64"):
        return np.ascontiguousarray(a.astype(np.float64))
    raise ValueError(dtype)


def _check(rc: int):
    if rc == 1:
        raise MemoryError("oracle: out of memory")
    if rc == 2:
        raise ValueError("oracle: bad shape (v must divide K; segment must divide v)")
    if rc == 3:
        raise ValueError("oracle: index >= Kc")


def _common(idx, C_pm1, alpha, mu):
    idx = np.ascontiguousarray(idx, dtype=np.uint16)
    C = np.ascontiguousarray(C_pm1, dtype=np.int8)
    al = np.ascontiguousarray(np.asarray(alpha).astype(np.float64))
    m = None if mu is None else np.ascontiguousarray(np.asarray(mu).astype(np.float64))
    return idx, C, al, m


def decode_pm1(idx, C_pm1) -> np.ndarray:
    """The +-1 matrix B^[N, K] the indices stand for."""
    idx = np.ascontiguousarray(idx, dtype=np.uint16)
    C = np.ascontiguousarray(C_pm1, dtype=np.int8)
    N, Kb = idx.shape
    Kc, v = C.shape
    B = np.empty((N, Kb * v), dtype=np.int8)
    _check(_load().btc_oracle_decode_pm1(_p(idx), _p(C), N, Kb * v, v, Kc, _p(B)))
    return B


def dense_weight(idx, C_pm1, alpha, mu=None) -> np.ndarray:
    """W^ = alpha * B^ + mu as a dense fp64 [N, K] matrix."""
    idx, C, al, m = _common(idx, C_pm1, alpha, mu)
    B = decode_pm1(idx, C)
    W = np.empty(B.shape, dtype=np.float64)
    _load().btc_oracle_dense_weight(_p(B), _p(al), _p(m), B.shape[0], B.shape[1], _p(W))
    return W


def linear(x_f64, idx, C_pm1, alpha, mu=None, return_B: bool = False):
    """y = x * W^T in fp64 via dense decode and the naive triple loop."""
    idx, C, al, m = _common(idx, C_pm1, alpha, mu)
    x = np.ascontiguousarray(x_f64, dtype=np.float64)
    M, K = x.shape
    N, Kb = idx.shape
    Kc, v = C.shape
    if Kb * v != K:
        raise ValueError("x and idx disagree on K")
    y = np.empty((M, N), dtype=np.float64)
    B = np.empty((N, K), dtype=np.int8) if return_B else None
    _check(_load().btc_oracle_linear(_p(x), _p(idx), _p(C), _p(al), _p(m), M, N, K, v, Kc, _p(y), _p(B)))
    return (y, B) if return_B else y


def linear_terms(x_f64, N: int, terms) -> np.ndarray:
    """y = x * W^T for a weight that is a SUM of codebook-binary terms, each covering a column range:
        W^[n, k] = sum over terms t with k0_t <= k < k0_t + K_t of ( alpha_t[n] * B^_t[n, k - k0_t] + mu_t[n] ).
    This is what a binariser with several scale groups per row emits (Eq. 1-2 applied per group of columns after the
    columns are ordered by group: the split-point groups of Section 5's ablation) and what a residual binarisation of
    salient columns emits (two terms over the same range, W ~ alpha_1 B_1 + alpha_2 B_2, Section 3).
    terms: iterable of (k0, idx [N, K_t/v], C_pm1 [Kc, v], alpha [N], mu [N] or None).  Dense fp64 weight, then the naive
    triple loop."""
    x = np.ascontiguousarray(x_f64, dtype=np.float64)
    M, K = x.shape
    W = np.zeros((N, K), dtype=np.float64)
    for (k0, idx, C_pm1, alpha, mu) in terms:
        Wt = dense_weight(idx, C_pm1, alpha, mu)
        if Wt.shape[0] != N or k0 < 0 or k0 + Wt.shape[1] > K:
            raise ValueError("term outside the layer")
        W[:, k0:k0 + Wt.shape[1]] += Wt
    y = np.empty((M, N), dtype=np.float64)
    _load().btc_oracle_matmul_nt(_p(x), _p(np.ascontiguousarray(W)), M, N, K, _p(y))
    return y


def lut_linear(x_f64, idx, C_pm1, alpha, mu=None, seg: int = 4) -> np.ndarray:
    """Same result through the paper's Stage-I / Stage-II lookup tables."""
    idx, C, al, m = _common(idx, C_pm1, alpha, mu)
    x = np.ascontiguousarray(x_f64, dtype=np.float64)
    M, K = x.shape
    N, Kb = idx.shape
    Kc, v = C.shape
    y = np.empty((M, N), dtype=np.float64)
    _check(_load().btc_oracle_lut_linear(_p(x), _p(idx), _p(C), _p(al), _p(m), M, N, K, v, Kc, seg, _p(y)))
    return y


def pack_codebook(C_pm1) -> np.ndarray:
    """uint32 [Kc]: bit t (LSB first) set where C[k][t] >= 0."""
    C = np.ascontiguousarray(C_pm1, dtype=np.int8)
    out = np.empty(C.shape[0], dtype=np.uint32)
    _load().btc_oracle_pack_codebook(_p(C), C.shape[0], C.shape[1], _p(out))
    return out


def index_bits(Kc: int) -> int:
    """ceil(log2 Kc), at least 1: the index width of the paper's storage accounting (Section 4.3)."""
    b = 1
    while (1 << b) < Kc:
        b += 1
    return b


def packed_row_bytes(Kb: int, bits: int, align: int = 16) -> int:
    """Bytes from one packed row to the next: ceil(Kb*bits/8) rounded up to `align`."""
    n = (Kb * bits + 7) // 8
    return (n + align - 1) // align * align


def pack_indices(idx, bits: int, pitch: Optional[int] = None) -> np.ndarray:
    """uint16 [N, Kb] -> uint8 [N, pitch]: each row the little-endian bit string of its indices, `bits` bits each."""
    idx = np.ascontiguousarray(idx, dtype=np.uint16)
    N, Kb = idx.shape
    pitch = packed_row_bytes(Kb, bits) if pitch is None else pitch
    out = np.empty((N, pitch), dtype=np.uint8)
    _check(_load().btc_oracle_pack_indices(_p(idx), N, Kb, bits, ctypes.c_size_t(pitch), _p(out)))
    return out


def unpack_indices(packed, Kb: int, bits: int) -> np.ndarray:
    packed = np.ascontiguousarray(packed, dtype=np.uint8)
    N, pitch = packed.shape
    idx = np.empty((N, Kb), dtype=np.uint16)
    _check(_load().btc_oracle_unpack_indices(_p(packed), N, Kb, bits, ctypes.c_size_t(pitch), _p(idx)))
    return idx


def sqdist_pm1(b, c) -> float:
    b = np.ascontiguousarray(b, dtype=np.int8)
    c = np.ascontiguousarray(c, dtype=np.int8)
    return float(_load().btc_oracle_sqdist_pm1(_p(b), _p(c), b.size))


def storage_bits(N: int, K: int, v: int, Kc: int) -> float:
    return float(_load().btc_oracle_storage_bits(N, K, v, Kc))


def bits_per_weight(N: int, K: int, v: int, Kc: int, scale_bits_per_row: int = 0,
                    mode: str = "container", with_codebook: bool = False) -> float:
    m = {"nominal": 0, "container": 1, "stored": 2}[mode]
    return float(_load().btc_oracle_bits_per_weight(N, K, v, Kc, scale_bits_per_row, m, int(with_codebook)))


def transform(x_f64, sigma_pm1, P1, P2) -> np.ndarray:
    """x' = x * diag(sigma) * (P1 kron P2), dense fp64 (small K only)."""
    x = np.ascontiguousarray(x_f64, dtype=np.float64)
    P1 = np.ascontiguousarray(P1, dtype=np.float64)
    P2 = np.ascontiguousarray(P2, dtype=np.float64)
    s = np.ascontiguousarray(sigma_pm1, dtype=np.int8)
    M, K = x.shape
    k1, k2 = P1.shape[0], P2.shape[0]
    if k1 * k2 != K or s.size != K:
        raise ValueError("transform factor sizes must multiply to K")
    out = np.empty_like(x)
    _check(_load().btc_oracle_transform(_p(x), _p(s), _p(P1), _p(P2), M, k1, k2, _p(out)))
    return out

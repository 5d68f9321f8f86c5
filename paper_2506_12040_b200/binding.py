"""ctypes binding of libbtc_b200.so: argument marshalling only.

Every step of the layer runs in the library's CUDA kernels; torch supplies device memory
and the current stream.  There is no CPU or eager-PyTorch fallback: if the shared library
cannot be loaded, importing this module raises.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional

import torch

from . import build as _build

BTC_F16, BTC_BF16, BTC_F32 = 0, 1, 2
_DT = {torch.float16: BTC_F16, torch.bfloat16: BTC_BF16, torch.float32: BTC_F32}

EXPORTS = (
    "btc_version", "btc_status_string", "btc_last_cuda_error", "btc_codebook_packed_bytes",
    "btc_codebook_pack", "btc_codebook_pack_host", "btc_linear_workspace_bytes", "btc_linear_gemv",
    "btc_linear_gemm", "btc_linear_gemv_batch", "btc_linear_gemm_static_scratch", "btc_decode_pm1", "btc_validate_indices", "btc_bits_per_weight", "btc_device_status", "btc_device_status_reset", "btc_selftest_bounded_wait",
    "btc_codebook_kmeans_workspace_bytes", "btc_codebook_kmeans",
    "btc_index_bits", "btc_index_packed_row_bytes", "btc_index_pack", "btc_index_unpack", "btc_linear_gemv_packed", "btc_linear_gemv_sum",
    "btc_linear_gemv_lut_workspace_bytes", "btc_linear_gemv_lut", "btc_linear_workspace_bytes_ex",
    "btc_activation_transform",
)


class BtcTransform(ctypes.Structure):
    _fields_ = [("sigma_bits", ctypes.c_void_p), ("P1", ctypes.c_void_p), ("P2", ctypes.c_void_p),
                ("k1", ctypes.c_int), ("k2", ctypes.c_int)]


class BtcLinearProblem(ctypes.Structure):
    _fields_ = [("x", ctypes.c_void_p), ("idx", ctypes.c_void_p), ("C_packed", ctypes.c_void_p),
                ("alpha", ctypes.c_void_p), ("mu", ctypes.c_void_p), ("y", ctypes.c_void_p),
                ("x_dtype", ctypes.c_int), ("y_dtype", ctypes.c_int),
                ("M", ctypes.c_int), ("N", ctypes.c_int), ("K", ctypes.c_int), ("v", ctypes.c_int), ("Kc", ctypes.c_int),
                ("idx_bits", ctypes.c_int), ("x_stride", ctypes.c_int), ("idx_stride", ctypes.c_int)]


class BtcError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        msg = lib.btc_status_string(status).decode()
        if status == 6:
            msg += f" [cudaError {lib.btc_last_cuda_error()}]"
        super().__init__(f"{where}: {msg} (status {status})")


def _load() -> ctypes.CDLL:
    path = _build.LIB
    if not os.path.exists(path) or _build.is_stale():
        # The library travels with the source tree; build it in place if it is absent or older
        # than its sources.  No nvcc means no library, and that is an error, not a fallback.
        _build.build_library()
    L = ctypes.CDLL(path)
    vp, ci, sz = ctypes.c_void_p, ctypes.c_int, ctypes.c_size_t
    L.btc_version.restype = ci
    L.btc_status_string.restype = ctypes.c_char_p
    L.btc_status_string.argtypes = [ci]
    L.btc_last_cuda_error.restype = ci
    L.btc_codebook_packed_bytes.restype = sz
    L.btc_codebook_packed_bytes.argtypes = [ci, ci]
    L.btc_codebook_pack.argtypes = [vp, ci, ci, vp, vp]
    L.btc_codebook_pack_host.argtypes = [vp, ci, ci, vp]
    L.btc_linear_workspace_bytes.restype = sz
    L.btc_linear_workspace_bytes.argtypes = [ci] * 5
    L.btc_linear_workspace_bytes_ex.restype = sz
    L.btc_linear_workspace_bytes_ex.argtypes = [ci] * 6
    lin = [vp, ci, vp, vp, vp, vp, ctypes.POINTER(BtcTransform), vp, ci, ci, ci, ci, ci, ci, vp, sz, vp]
    L.btc_linear_gemv.argtypes = lin
    L.btc_linear_gemm.argtypes = lin
    L.btc_linear_gemv_batch.argtypes = [ctypes.POINTER(BtcLinearProblem), ci, vp]
    L.btc_linear_gemv_sum.argtypes = [ctypes.POINTER(BtcLinearProblem), ci, vp]
    L.btc_linear_gemm_static_scratch.argtypes = lin[:14] + [vp]
    L.btc_decode_pm1.argtypes = [vp, vp, ci, ci, ci, ci, vp, vp]
    L.btc_validate_indices.argtypes = [vp, sz, ci, vp, vp]
    L.btc_device_status.argtypes = [ctypes.POINTER(ctypes.c_int)]
    L.btc_selftest_bounded_wait.argtypes = [vp]
    L.btc_codebook_kmeans_workspace_bytes.restype = sz
    L.btc_codebook_kmeans_workspace_bytes.argtypes = [ci, ci]
    L.btc_codebook_kmeans.argtypes = [vp, sz, ci, ci, ci, vp, vp, vp, vp, sz, vp]
    L.btc_index_bits.argtypes = [ci]
    L.btc_index_packed_row_bytes.restype = sz
    L.btc_index_packed_row_bytes.argtypes = [ci, ci]
    L.btc_index_pack.argtypes = [vp, ci, ci, ci, vp, vp]
    L.btc_index_unpack.argtypes = [vp, ci, ci, ci, vp, vp]
    L.btc_linear_gemv_packed.argtypes = [vp, ci, vp, vp, vp, vp, vp, ci, ci, ci, ci, ci, ci, vp]
    L.btc_linear_gemv_lut_workspace_bytes.restype = sz
    L.btc_linear_gemv_lut_workspace_bytes.argtypes = [ci] * 5
    L.btc_linear_gemv_lut.argtypes = [vp, ci, vp, vp, vp, vp, vp, ci, ci, ci, ci, ci, ci, vp, sz, vp]
    L.btc_activation_transform.argtypes = [vp, ci, ctypes.POINTER(BtcTransform), vp, ci, ci, ci, vp]
    L.btc_bits_per_weight.restype = ctypes.c_double
    L.btc_bits_per_weight.argtypes = [ci] * 7
    return L


lib = _load()


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


def _ptr(t: Optional[torch.Tensor]) -> Optional[int]:
    return None if t is None else t.data_ptr()


def _dev(t: torch.Tensor, name: str):
    if not t.is_cuda:
        raise ValueError(f"{name} must be a CUDA tensor")
    if not t.is_contiguous():
        raise ValueError(f"{name} must be contiguous")


def packed_words(Kc: int, v: int) -> int:
    n = int(lib.btc_codebook_packed_bytes(Kc, v))
    if n == 0:
        raise ValueError("invalid codebook shape")
    return n // 4


def codebook_pack(C_pm1: torch.Tensor) -> torch.Tensor:
    """int8 [Kc, v] of +-1 (device) -> packed codebook buffer (int32 words).  The first Kc words are
    the public form (bit t = element t); the rest is kernel-private.  Pass the whole tensor on."""
    _dev(C_pm1, "C_pm1")
    if C_pm1.dtype != torch.int8 or C_pm1.dim() != 2:
        raise ValueError("C_pm1 must be int8 [Kc, v]")
    Kc, v = C_pm1.shape
    out = torch.empty(packed_words(Kc, v), dtype=torch.int32, device=C_pm1.device)
    st = lib.btc_codebook_pack(C_pm1.data_ptr(), Kc, v, out.data_ptr(), _stream())
    if st:
        raise BtcError(st, "btc_codebook_pack")
    return out


def codebook_pack_host(C_pm1: torch.Tensor) -> torch.Tensor:
    """Host-memory variant (CPU tensors in and out); no GPU work."""
    if C_pm1.is_cuda or C_pm1.dtype != torch.int8 or C_pm1.dim() != 2 or not C_pm1.is_contiguous():
        raise ValueError("C_pm1 must be a contiguous CPU int8 [Kc, v] tensor")
    Kc, v = C_pm1.shape
    out = torch.empty(packed_words(Kc, v), dtype=torch.int32)
    st = lib.btc_codebook_pack_host(C_pm1.data_ptr(), Kc, v, out.data_ptr())
    if st:
        raise BtcError(st, "btc_codebook_pack_host")
    return out


def linear_workspace_bytes(M: int, N: int, K: int, v: int, Kc: int) -> int:
    return int(lib.btc_linear_workspace_bytes(M, N, K, v, Kc))


def _linear(fn, name, x, idx, C_packed, alpha, v, Kc, mu, out, out_dtype, workspace, transform):
    for t, n in ((x, "x"), (idx, "idx"), (C_packed, "C_packed"), (alpha, "alpha")):
        _dev(t, n)
    if x.dim() != 2 or idx.dim() != 2:
        raise ValueError("x must be [M, K] and idx [N, K/v]")
    if x.dtype not in (torch.float16, torch.bfloat16):
        raise ValueError("x must be fp16 or bf16")
    if idx.element_size() != 2 or alpha.dtype != torch.float16 or C_packed.element_size() != 4:
        raise ValueError("idx must be 16-bit integers, alpha fp16, C_packed 32-bit words")
    M, K = x.shape
    N, Kb = idx.shape
    if C_packed.numel() != packed_words(Kc, v):
        raise ValueError("C_packed is not the buffer codebook_pack wrote for this (Kc, v)")
    if Kb * v != K or alpha.numel() != N:
        raise ValueError("shape mismatch between x, idx, v and alpha")
    if mu is not None:
        _dev(mu, "mu")
        if mu.dtype != torch.float16 or mu.numel() != N:
            raise ValueError("mu must be fp16 [N]")
    if out is None:
        out = torch.empty((M, N), dtype=out_dtype, device=x.device)
    else:
        _dev(out, "out")
        if tuple(out.shape) != (M, N):
            raise ValueError("out must be [M, N]")
    tr = None
    if transform is not None:
        sig, P1, P2 = transform
        tr = BtcTransform(sig.data_ptr(), P1.data_ptr(), P2.data_ptr(), P1.shape[0], P2.shape[0])
    need = int(lib.btc_linear_workspace_bytes_ex(M, N, K, v, Kc, int(transform is not None)))
    ws_ptr, ws_bytes = None, 0
    if need:
        if workspace is None:
            workspace = torch.empty(need, dtype=torch.uint8, device=x.device)
        ws_ptr, ws_bytes = workspace.data_ptr(), workspace.numel() * workspace.element_size()
    st = fn(x.data_ptr(), _DT[x.dtype], idx.data_ptr(), C_packed.data_ptr(), alpha.data_ptr(), _ptr(mu),
            ctypes.byref(tr) if tr is not None else None, out.data_ptr(), _DT[out.dtype],
            M, N, K, v, Kc, ws_ptr, ws_bytes, _stream())
    if st:
        raise BtcError(st, name)
    return out


def linear_gemv(x, idx, C_packed, alpha, v, Kc, mu=None, out=None, out_dtype=torch.float32, workspace=None,
                transform=None):
    """Decode path (M <= 8): y[M, N] = x * W^T with W^ = alpha * C[idx] (+ mu)."""
    return _linear(lib.btc_linear_gemv, "btc_linear_gemv", x, idx, C_packed, alpha, v, Kc, mu, out, out_dtype,
                   workspace, transform)


def linear_gemm(x, idx, C_packed, alpha, v, Kc, mu=None, out=None, out_dtype=torch.float32, workspace=None,
                transform=None):
    """Tensor-core path (any M, built for large M)."""
    return _linear(lib.btc_linear_gemm, "btc_linear_gemm", x, idx, C_packed, alpha, v, Kc, mu, out, out_dtype,
                   workspace, transform)


class GemvBatch:
    """A fixed list of independent decode-path layers (M <= 8 each) marshalled once, run with one
    btc_linear_gemv_batch call per `run()`: each entry is a dict with x, idx, C_packed, alpha, v, Kc,
    and optionally mu, out (fp32 [M, N] is allocated when absent)."""

    def __init__(self, layers):
        self.layers = []
        arr = (BtcLinearProblem * len(layers))()
        for i, L in enumerate(layers):
            x, idx, Cp, alpha = L["x"], L["idx"], L["C_packed"], L["alpha"]
            for t, n in ((x, "x"), (idx, "idx"), (Cp, "C_packed"), (alpha, "alpha")):
                _dev(t, n)
            M, K = x.shape
            v, Kc = int(L["v"]), int(L["Kc"])
            bits = int(L.get("idx_bits", 0))
            if bits in (0, 16):
                N, Kb = idx.shape
                if idx.element_size() != 2:
                    raise ValueError("idx must be 16-bit")
            else:                       # dense-packed rows (uint8 [N, row bytes]) written by index_pack
                N, Kb = idx.shape[0], K // v
                if idx.dtype != torch.uint8 or idx.shape[1] != int(lib.btc_index_packed_row_bytes(Kb, Kc)):
                    raise ValueError("idx is not the buffer index_pack wrote for this (K/v, Kc)")
            if Kb * v != K or alpha.numel() != N or Cp.numel() != packed_words(Kc, v):
                raise ValueError("shape mismatch between x, idx, v, alpha and C_packed")
            if x.dtype not in (torch.float16, torch.bfloat16, torch.float32) or alpha.dtype != torch.float16:
                raise ValueError("x must be fp16/bf16 (or fp32 from activation_transform), alpha fp16")
            mu = L.get("mu")
            out = L.get("out")
            if out is None:
                out = torch.empty((M, N), dtype=torch.float32, device=x.device)
            arr[i] = BtcLinearProblem(x.data_ptr(), idx.data_ptr(), Cp.data_ptr(), alpha.data_ptr(), _ptr(mu),
                                      out.data_ptr(), _DT[x.dtype], _DT[out.dtype], M, N, K, v, Kc, bits, 0, 0)
            self.layers.append((x, idx, Cp, alpha, mu, out))          # keeps the tensors alive
        self._arr = arr
        self.outs = [t[5] for t in self.layers]

    def run(self):
        st = lib.btc_linear_gemv_batch(self._arr, len(self.layers), _stream())
        if st:
            raise BtcError(st, "btc_linear_gemv_batch")
        return self.outs


def activation_transform(x, transform, out_dtype=torch.float32, out=None):
    """x' = x * diag(sigma) * (P1 kron P2) for the rows of x (fp16 / bf16 [M, K]); transform = (sigma_bits int32
    [ceil(K/32)], P1 fp32 [k1, k1], P2 fp32 [k2, k2]).  out_dtype: torch.float32 or the dtype of x."""
    _dev(x, "x")
    sig, P1, P2 = transform
    for t, n in ((sig, "sigma_bits"), (P1, "P1"), (P2, "P2")):
        _dev(t, n)
    M, K = x.shape
    if out is None:
        out = torch.empty((M, K), dtype=out_dtype, device=x.device)
    T = BtcTransform(sig.data_ptr(), P1.data_ptr(), P2.data_ptr(), P1.shape[0], P2.shape[0])
    st = lib.btc_activation_transform(x.data_ptr(), _DT[x.dtype], ctypes.byref(T), out.data_ptr(), _DT[out.dtype], M, K, _stream())
    if st:
        raise BtcError(st, "btc_activation_transform")
    return out


def linear_gemv_batch(layers):
    """One btc_linear_gemv_batch call over `layers` (see GemvBatch); returns the list of outputs."""
    return GemvBatch(layers).run()


STATIC_SCRATCH_BYTES = 65536


def linear_gemm_static_scratch(x, idx, C_packed, alpha, v, Kc, mu=None, out=None):
    """btc_linear_gemm for callers that cannot allocate device memory: the scratch of the mean term is a
    fixed array inside the library (STATIC_SCRATCH_BYTES, so M <= 16384), shared by all calls on a device.
    `out` must be given by such a caller; when it is None this wrapper allocates it with torch, the
    library itself still allocates nothing.  Calls that may overlap on the GPU race on the array."""
    for t, n in ((x, "x"), (idx, "idx"), (C_packed, "C_packed"), (alpha, "alpha")):
        _dev(t, n)
    M, K = x.shape
    N, Kb = idx.shape
    if Kb * v != K or alpha.numel() != N or C_packed.numel() != packed_words(Kc, v):
        raise ValueError("shape mismatch between x, idx, v, alpha and C_packed")
    if out is None:
        out = torch.empty((M, N), dtype=torch.float32, device=x.device)
    st = lib.btc_linear_gemm_static_scratch(x.data_ptr(), _DT[x.dtype], idx.data_ptr(), C_packed.data_ptr(),
                                            alpha.data_ptr(), _ptr(mu), None, out.data_ptr(), _DT[out.dtype],
                                            M, N, K, v, Kc, _stream())
    if st:
        raise BtcError(st, "btc_linear_gemm_static_scratch")
    return out


def linear_gemv_sum(x, terms, N: int, out=None):
    """btc_linear_gemv_sum: y = sum of codebook-binary terms.  x: [M, K] activations; terms: list of dicts with k0 (first
    column of the term), idx (16-bit [N, K_t/v], may be a column-range view of a wider matrix), C_packed, alpha, v, Kc
    and optionally mu.  Returns fp32 [M, N]."""
    _dev(x, "x")
    M, K = x.shape
    if out is None:
        out = torch.empty((M, N), dtype=torch.float32, device=x.device)
    arr = (BtcLinearProblem * len(terms))()
    keep = []
    for i, T in enumerate(terms):
        idx, Cp, alpha, mu = T["idx"], T["C_packed"], T["alpha"], T.get("mu")
        v, Kc, k0 = int(T["v"]), int(T["Kc"]), int(T["k0"])
        if idx.dim() != 2 or idx.shape[0] != N or idx.stride(1) != 1 or idx.element_size() != 2:
            raise ValueError("idx must be 16-bit [N, K_t/v] with unit column stride")
        Kt = idx.shape[1] * v
        if k0 < 0 or k0 + Kt > K or alpha.numel() != N:
            raise ValueError("term outside the layer")
        xt = x[:, k0:k0 + Kt]
        arr[i] = BtcLinearProblem(xt.data_ptr(), idx.data_ptr(), Cp.data_ptr(), alpha.data_ptr(), _ptr(mu), out.data_ptr(),
                                  _DT[x.dtype], _DT[out.dtype], M, N, Kt, v, Kc, 0,
                                  0 if Kt == K else K, 0 if idx.stride(0) == idx.shape[1] else idx.stride(0))
        keep.append((xt, idx, Cp, alpha, mu))
    st = lib.btc_linear_gemv_sum(arr, len(terms), _stream())
    if st:
        raise BtcError(st, "btc_linear_gemv_sum")
    return out


def linear_gemv_lut(x, idx, C_packed, alpha, v, Kc, mu=None, out=None, workspace=None):
    """btc_linear_gemv_lut: the layer through the paper's two-stage lookup tables (M <= 8)."""
    for t, n in ((x, "x"), (idx, "idx"), (C_packed, "C_packed"), (alpha, "alpha")):
        _dev(t, n)
    M, K = x.shape
    N, Kb = idx.shape
    if Kb * v != K or alpha.numel() != N or C_packed.numel() != packed_words(Kc, v):
        raise ValueError("shape mismatch between x, idx, v, alpha and C_packed")
    if out is None:
        out = torch.empty((M, N), dtype=torch.float32, device=x.device)
    need = int(lib.btc_linear_gemv_lut_workspace_bytes(M, N, K, v, Kc))
    if workspace is None:
        workspace = torch.empty(max(need, 256), dtype=torch.uint8, device=x.device)
    st = lib.btc_linear_gemv_lut(x.data_ptr(), _DT[x.dtype], idx.data_ptr(), C_packed.data_ptr(), alpha.data_ptr(), _ptr(mu),
                                 out.data_ptr(), _DT[out.dtype], M, N, K, v, Kc, workspace.data_ptr(), workspace.numel(), _stream())
    if st:
        raise BtcError(st, "btc_linear_gemv_lut")
    return out


def index_bits(Kc: int) -> int:
    return int(lib.btc_index_bits(Kc))


def index_pack(idx: torch.Tensor, Kc: int) -> torch.Tensor:
    """16-bit indices [N, K/v] (device) -> dense-packed rows, uint8 [N, row bytes] (btc_index_pack)."""
    _dev(idx, "idx")
    if idx.dim() != 2 or idx.element_size() != 2:
        raise ValueError("idx must be 16-bit integers [N, K/v]")
    N, Kb = idx.shape
    out = torch.empty((N, int(lib.btc_index_packed_row_bytes(Kb, Kc))), dtype=torch.uint8, device=idx.device)
    st = lib.btc_index_pack(idx.data_ptr(), N, Kb, Kc, out.data_ptr(), _stream())
    if st:
        raise BtcError(st, "btc_index_pack")
    return out


def index_unpack(packed: torch.Tensor, Kb: int, Kc: int) -> torch.Tensor:
    _dev(packed, "packed")
    N = packed.shape[0]
    out = torch.empty((N, Kb), dtype=torch.int16, device=packed.device)
    st = lib.btc_index_unpack(packed.data_ptr(), N, Kb, Kc, out.data_ptr(), _stream())
    if st:
        raise BtcError(st, "btc_index_unpack")
    return out


def linear_gemv_packed(x, idx_packed, C_packed, alpha, v, Kc, mu=None, out=None, out_dtype=torch.float32):
    """btc_linear_gemv_packed: the decode path (M <= 8) reading dense-packed index rows."""
    for t, n in ((x, "x"), (idx_packed, "idx_packed"), (C_packed, "C_packed"), (alpha, "alpha")):
        _dev(t, n)
    M, K = x.shape
    N = idx_packed.shape[0]
    if idx_packed.dtype != torch.uint8 or idx_packed.shape[1] != int(lib.btc_index_packed_row_bytes(K // v, Kc)):
        raise ValueError("idx_packed is not the buffer index_pack wrote for this (K/v, Kc)")
    if out is None:
        out = torch.empty((M, N), dtype=out_dtype, device=x.device)
    st = lib.btc_linear_gemv_packed(x.data_ptr(), _DT[x.dtype], idx_packed.data_ptr(), C_packed.data_ptr(), alpha.data_ptr(),
                                    _ptr(mu), out.data_ptr(), _DT[out.dtype], M, N, K, v, Kc, _stream())
    if st:
        raise BtcError(st, "btc_linear_gemv_packed")
    return out


def linear(x, idx, C_packed, alpha, v, Kc, **kw):
    """Routes by M the way a caller would: decode path up to 8 rows, tensor-core path above."""
    return (linear_gemv if x.shape[0] <= 8 else linear_gemm)(x, idx, C_packed, alpha, v, Kc, **kw)


def codebook_kmeans(vecs: torch.Tensor, v: int, Kc: int, max_iter: int = 20, workspace: Optional[torch.Tensor] = None):
    """btc_codebook_kmeans on n packed vectors (int32 words on the device, bit t = element t).  Returns
    (C_words int32 [Kc], z int16 [n], info int32 [4] on the device: E-steps run, centroids in use, distinct
    vectors, converged)."""
    _dev(vecs, "vecs")
    if vecs.dtype != torch.int32 or vecs.dim() != 1:
        raise ValueError("vecs must be a 1-D int32 tensor of packed vectors")
    need = int(lib.btc_codebook_kmeans_workspace_bytes(v, Kc))
    if workspace is None:
        workspace = torch.empty(max(need, 256), dtype=torch.uint8, device=vecs.device)
    C = torch.empty(Kc, dtype=torch.int32, device=vecs.device)
    z = torch.empty(vecs.numel(), dtype=torch.int16, device=vecs.device)
    info = torch.empty(4, dtype=torch.int32, device=vecs.device)
    st = lib.btc_codebook_kmeans(vecs.data_ptr(), vecs.numel(), v, Kc, max_iter, C.data_ptr(), z.data_ptr(), info.data_ptr(),
                                 workspace.data_ptr(), workspace.numel(), _stream())
    if st:
        raise BtcError(st, "btc_codebook_kmeans")
    return C, z, info


def decode_pm1(idx, C_packed, v, Kc) -> torch.Tensor:
    """Decoded sign matrix int8 [N, K]."""
    _dev(idx, "idx"); _dev(C_packed, "C_packed")
    N, Kb = idx.shape
    out = torch.empty((N, Kb * v), dtype=torch.int8, device=idx.device)
    st = lib.btc_decode_pm1(idx.data_ptr(), C_packed.data_ptr(), N, Kb * v, v, Kc,
                            out.data_ptr(), _stream())
    if st:
        raise BtcError(st, "btc_decode_pm1")
    return out


def validate_indices(idx, Kc: int) -> int:
    """Number of indices >= Kc (synchronises to read the count back)."""
    _dev(idx, "idx")
    bad = torch.empty(1, dtype=torch.int32, device=idx.device)
    st = lib.btc_validate_indices(idx.data_ptr(), idx.numel(), Kc, bad.data_ptr(), _stream())
    if st:
        raise BtcError(st, "btc_validate_indices")
    return int(bad.item())


def device_status() -> int:
    """Device-side status word (0 = ok, 7 = a bounded wait ran out).  Synchronises the device."""
    out = ctypes.c_int(0)
    st = lib.btc_device_status(ctypes.byref(out))
    if st:
        raise BtcError(st, "btc_device_status")
    return int(out.value)


def device_status_reset() -> None:
    st = lib.btc_device_status_reset()
    if st:
        raise BtcError(st, "btc_device_status_reset")


def selftest_bounded_wait() -> None:
    """Launches the bounded-wait self-test on the current stream (see btc_selftest_bounded_wait)."""
    st = lib.btc_selftest_bounded_wait(_stream())
    if st:
        raise BtcError(st, "btc_selftest_bounded_wait")


def bits_per_weight(N, K, v, Kc, scale_bits_per_row=0, mode="container", with_codebook=False) -> float:
    m = {"nominal": 0, "container": 1, "stored": 2}[mode]
    return float(lib.btc_bits_per_weight(N, K, v, Kc, scale_bits_per_row, m, int(with_codebook)))

"""Shared helpers for the GPU parity tests: run a generated layer through the C ABI (via the
Python binding) and through the CPU oracle, and measure the two error figures the tolerance is
stated in."""
import numpy as np
import torch

import oracle
import paper_2506_12040_b200 as btc

TOL_GEMV = 2e-3    # fp32 accumulate, M <= 8
TOL_GEMM = 1e-2    # bf16 tensor-core path


def to_device(L, device="cuda"):
    """LayerData (numpy) -> dict of device tensors in the layouts the C ABI takes."""
    dt = torch.float16 if L.spec.x_dtype == "f16" else torch.bfloat16
    x = torch.from_numpy(L.x_bits.view(np.int16).copy()).to(device).view(dt)
    idx = torch.from_numpy(L.idx.view(np.int16).copy()).to(device)
    C = torch.from_numpy(L.C_pm1.copy()).to(device)
    alpha = torch.from_numpy(L.alpha.view(np.int16).copy()).to(device).view(torch.float16)
    mu = None if L.mu is None else torch.from_numpy(L.mu.view(np.int16).copy()).to(device).view(torch.float16)
    return {"x": x, "idx": idx, "C_pm1": C, "alpha": alpha, "mu": mu, "Cp": btc.codebook_pack(C)}


def oracle_y(L):
    return oracle.linear(L.x_f64(), L.idx, L.C_pm1, L.alpha, L.mu)


def errors(y_gpu: torch.Tensor, y_ref: np.ndarray, L):
    """(max abs err / max abs ref,  max over outputs of abs err / (|alpha_n| * sum_k |x_mk| + |mu_n| * sum|x|))."""
    y = y_gpu.detach().double().cpu().numpy()
    err = np.abs(y - y_ref)
    rel = err.max() / max(np.abs(y_ref).max(), 1e-300)
    ax = np.abs(L.x_f64()).sum(1)                                   # [M]
    scale = np.outer(ax, np.abs(L.alpha.astype(np.float64)))         # [M, N]
    if L.mu is not None:
        scale = scale + np.outer(ax, np.abs(L.mu.astype(np.float64)))
    fwd = (err / np.maximum(scale, 1e-300)).max()
    return float(rel), float(fwd)


def run_layer(L, path="auto", **kw):
    d = to_device(L)
    fn = {"auto": btc.linear, "gemv": btc.linear_gemv, "gemm": btc.linear_gemm}[path]
    y = fn(d["x"], d["idx"], d["Cp"], d["alpha"], L.spec.v, L.spec.Kc, mu=d["mu"], **kw)
    torch.cuda.synchronize()
    return y, d

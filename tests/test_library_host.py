"""CPU-side checks of the C-ABI library: it loads, exports every declared symbol, and its host
logic (argument validation, host packing, accounting) behaves; no kernel is launched here."""
import ctypes
import os
import re

import numpy as np
import torch

import oracle
import paper_2506_12040_b200 as btc
from paper_2506_12040_b200 import binding
import workloads as wl

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_exports_every_declared_symbol():
    hdr = open(os.path.join(ROOT, "include", "btc.h")).read()
    declared = set(re.findall(r"BTC_API[^;(]*?\b(btc_\w+)\s*\(", hdr))
    assert declared == set(binding.EXPORTS)
    for name in declared:
        assert hasattr(btc.lib, name), name
    assert btc.lib.btc_version() >= 100


def test_status_strings():
    for st in range(0, 8):
        assert btc.lib.btc_status_string(st)
    assert b"unknown" in btc.lib.btc_status_string(99)


def test_host_pack_matches_oracle_convention():
    for v in (1, 4, 13, 16, 20, 32):
        C = wl.make_codebook_pm1(50, v, seed=v, distinct=False)
        got = btc.codebook_pack_host(torch.from_numpy(C.copy())).numpy().view(np.uint32)
        assert got.size * 4 == btc.lib.btc_codebook_packed_bytes(50, v)
        assert np.array_equal(got[:50], oracle.pack_codebook(C))
    z = torch.tensor([[0, -1, 3, -2]], dtype=torch.int8)          # zero counts as +1
    assert btc.codebook_pack_host(z)[0].item() == 0b0101


def _call(fn, **over):
    """Calls a linear entry point with fake (never dereferenced) pointers; validation runs on the host."""
    a = dict(x=0x1000, x_dt=0, idx=0x2000, Cp=0x3000, alpha=0x4000, mu=None, T=None, y=0x5000, y_dt=2,
             M=1, N=64, K=64, v=16, Kc=256, ws=None, ws_bytes=0, stream=None)
    a.update(over)
    return fn(a["x"], a["x_dt"], a["idx"], a["Cp"], a["alpha"], a["mu"], a["T"], a["y"], a["y_dt"],
              a["M"], a["N"], a["K"], a["v"], a["Kc"], a["ws"], a["ws_bytes"], a["stream"])


def test_argument_validation_returns_codes():
    for fn in (btc.lib.btc_linear_gemv, btc.lib.btc_linear_gemm):
        assert _call(fn, x=None) == 1
        assert _call(fn, idx=None) == 1
        assert _call(fn, y=None) == 1
        assert _call(fn, K=60) == 2            # v does not divide K
        assert _call(fn, v=0) == 2
        assert _call(fn, v=33) == 2
        assert _call(fn, Kc=0) == 2
        assert _call(fn, Kc=65537) == 2
        assert _call(fn, M=0) == 2
        assert _call(fn, x=0x1008) == 3        # 16-byte alignment
        assert _call(fn, idx=0x2002) == 3
        assert _call(fn, alpha=0x4001) == 3
        assert _call(fn, x_dt=2) == 4          # fp32 activations are not supported
        assert _call(fn, y_dt=7) == 4
    assert _call(btc.lib.btc_linear_gemv, M=9) == 2
    assert btc.lib.btc_codebook_pack(None, 4, 4, 0x100, None) == 1
    assert btc.lib.btc_codebook_pack(0x100, 4, 40, 0x200, None) == 2
    assert btc.lib.btc_decode_pm1(0x100, 0x200, 4, 10, 4, 4, 0x300, None) == 2
    assert btc.lib.btc_validate_indices(None, 4, 4, 0x100, None) == 1
    # the transform on its own: NULL, factor sizes, dtypes, alignment -- all decided on the host
    import ctypes
    from paper_2506_12040_b200.binding import BtcLinearProblem, BtcTransform
    T = BtcTransform(0x1000, 0x2000, 0x3000, 4, 8)
    at = btc.lib.btc_activation_transform
    assert at(None, 0, ctypes.byref(T), 0x5000, 2, 1, 32, None) == 1
    assert at(0x4000, 0, None, 0x5000, 2, 1, 32, None) == 1
    assert at(0x4000, 0, ctypes.byref(T), 0x5000, 2, 1, 40, None) == 2      # k1 * k2 != K
    assert at(0x4000, 2, ctypes.byref(T), 0x5000, 2, 1, 32, None) == 4      # fp32 input
    assert at(0x4000, 0, ctypes.byref(T), 0x5000, 1, 1, 32, None) == 4      # fp16 in, bf16 out
    assert at(0x4008, 0, ctypes.byref(T), 0x5000, 2, 1, 32, None) == 3
    # fp32 activations in a batch call only where the decode kernel covers the layer (v = 10 is not a multiple of 4)
    P = (BtcLinearProblem * 1)()
    P[0] = BtcLinearProblem(0x4000, 0x6000, 0x7000, 0x8000, None, 0x9000, 2, 2, 1, 16, 80, 10, 64, 0, 0, 0)
    assert btc.lib.btc_linear_gemv_batch(P, 1, None) == 4


def test_accounting_matches_closed_forms():
    assert btc.bits_per_weight(4096, 4096, 16, 4096) == 0.75
    assert btc.bits_per_weight(4096, 4096, 16, 8192) == 0.8125
    assert btc.bits_per_weight(5120, 5120, 20, 65536) == 0.8
    assert btc.bits_per_weight(4096, 4096, 16, 7132, mode="stored") == 1.0
    for (N, K, v, Kc, sb, mode, cb) in [(4096, 11008, 16, 7132, 16, "container", True),
                                        (5120, 5120, 20, 21619, 32, "nominal", False)]:
        assert abs(btc.bits_per_weight(N, K, v, Kc, sb, mode, cb)
                   - oracle.bits_per_weight(N, K, v, Kc, sb, mode, cb)) < 1e-15
    assert btc.lib.btc_bits_per_weight(1, 1, 40, 4, 0, 0, 0) == -1.0
    assert btc.lib.btc_codebook_packed_bytes(8192, 16) == 8192 * 14
    assert btc.lib.btc_codebook_packed_bytes(7133, 16) == 7136 * 14
    assert btc.lib.btc_codebook_packed_bytes(0, 16) == 0
    assert btc.linear_workspace_bytes(1, 4096, 4096, 15, 4096) == 0   # invalid shape: v does not divide K

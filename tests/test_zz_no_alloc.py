"""btc_linear_gemm_static_scratch: the entry point for callers that cannot allocate device memory
(code running where cudaMalloc is off limits, or a host that hands a plugin only its inputs and outputs).
Its scratch is a fixed array inside the library, so there is no workspace argument.  This file is
collected last on purpose; it must pass alone in a fresh process and after all other tests."""
import numpy as np
import pytest
import torch

import paper_2506_12040_b200 as btc
import workloads as wl
from util import TOL_GEMM, errors, oracle_y, to_device


@pytest.mark.gpu
def test_static_scratch_matches_workspace_entry_point_twice():
    """Two calls in a row (different layers, so the shared array is reused with stale contents) must each
    match btc_linear_gemm given a caller workspace, and the oracle, within the tensor-core tolerance."""
    for seed, (N, K, M) in enumerate([(300, 1024, 200), (520, 512, 777)]):
        L = wl.make_layer(wl.LayerSpec("t", N, K, 16, 8192, x_dtype="bf16", with_mu=True), M, seed=900 + seed)
        d = to_device(L)
        want = btc.linear_gemm(d["x"], d["idx"], d["Cp"], d["alpha"], 16, 8192, mu=d["mu"])
        out = torch.full((M, N), float("nan"), dtype=torch.float32, device="cuda")
        got = btc.linear_gemm_static_scratch(d["x"], d["idx"], d["Cp"], d["alpha"], 16, 8192, mu=d["mu"], out=out)
        torch.cuda.synchronize()
        ref = np.abs(want.double().cpu().numpy()).max()
        assert float((got - want).abs().max()) <= TOL_GEMM * ref
        rel, fwd = errors(got, oracle_y(L), L)
        assert rel <= TOL_GEMM and fwd <= TOL_GEMM, (rel, fwd)


@pytest.mark.gpu
def test_static_scratch_rejects_sizes_beyond_its_array():
    M = btc.binding.STATIC_SCRATCH_BYTES // 4 + 1
    st = btc.lib.btc_linear_gemm_static_scratch(0x1000, 1, 0x2000, 0x3000, 0x4000, None, None, 0x5000, 2,
                                                M, 64, 64, 16, 256, None)
    assert st == 5, btc.lib.btc_status_string(st)

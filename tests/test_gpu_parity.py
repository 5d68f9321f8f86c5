"""GPU parity: the CUDA path (through the C ABI) against the fp64 CPU oracle, element by element,
on the same seeded inputs.  Tolerances: decode bit-exact; outputs max-rel-err <= 2e-3 for the
decode path (fp32 accumulate, M <= 8) and <= 1e-2 for the tensor-core path."""
from dataclasses import replace

import numpy as np
import pytest
import torch

import oracle
import paper_2506_12040_b200 as btc
import workloads as wl
from util import TOL_GEMM, TOL_GEMV, errors, oracle_y, run_layer, to_device

pytestmark = pytest.mark.gpu


def _spec(N, K, v, Kc, **kw):
    return wl.LayerSpec("t", N, K, v, Kc, **kw)


# ------------------------------------------------------------------ packing / decode: bit exact

@pytest.mark.parametrize("v,Kc", [(1, 2), (4, 9), (8, 85), (13, 500), (16, 4096), (16, 7132), (20, 65536), (32, 1000)])
def test_pack_and_decode_bit_exact(v, Kc):
    N, Kb = 37, 11
    L = wl.make_layer(_spec(N, Kb * v, v, Kc), 1, seed=100 + v)
    d = to_device(L)
    assert np.array_equal(d["Cp"].cpu().numpy().view(np.uint32)[:Kc], oracle.pack_codebook(L.C_pm1))
    B = btc.decode_pm1(d["idx"], d["Cp"], v, Kc).cpu().numpy()
    assert np.array_equal(B, oracle.decode_pm1(L.idx, L.C_pm1))


def test_validate_indices_counts():
    idx = torch.arange(0, 5000, dtype=torch.int32).to(torch.int16).cuda()
    assert btc.validate_indices(idx, 65536) == 0
    assert btc.validate_indices(idx, 4096) == 5000 - 4096
    assert btc.validate_indices(idx, 1) == 4999


# ------------------------------------------------------------------ one-hot probes: decode through the real kernels

@pytest.mark.parametrize("N,K,v,Kc", [(200, 256, 16, 300), (130, 320, 20, 65536), (64, 96, 12, 777)])
@pytest.mark.parametrize("path", ["gemv", "gemm"])
def test_one_hot_probe_is_exact(N, K, v, Kc, path):
    """x = e_k  =>  y[m, n] = alpha_n * B^[n, k] exactly (one non-zero term), so the production kernels'
    decode is checked bit for bit without materialising the weight."""
    M = 8 if path == "gemv" else 160
    L = wl.make_layer(_spec(N, K, v, Kc), M, seed=7)
    ks = (np.arange(M) * 37 + 5) % K
    xb = np.zeros((M, K), dtype=np.float16)
    xb[np.arange(M), ks] = 1.0
    L.x_bits = xb.view(np.uint16)
    y, _ = run_layer(L, path)
    B = oracle.decode_pm1(L.idx, L.C_pm1)
    want = L.alpha.astype(np.float32)[None, :] * B[:, ks].T.astype(np.float32)
    assert np.array_equal(y.cpu().numpy(), want)


# ------------------------------------------------------------------ decode path parity (M <= 8)

SMALL = [
    # N, K, v, Kc, M, dist, mu
    (1, 16, 16, 1, 1, "uniform", False),
    (5, 64, 16, 7, 3, "uniform", True),
    (257, 1040, 16, 4096, 8, "uniform", False),
    (300, 2000, 20, 65536, 4, "zipf", False),
    (129, 4096, 16, 8192, 1, "uniform", True),
    (150, 2048, 16, 65536, 1, "uniform", True),
    (77, 1024, 16, 50000, 2, "zipf", False),
    (300, 8192, 16, 8192, 8, "uniform", True),      # few row tiles, very long K: the split tensor-core launch
    (1000, 11008, 16, 4096, 5, "uniform", False),
    (70, 11008, 16, 8192, 2, "uniform", False),
    (1000, 640, 20, 21619, 5, "zipf", True),
    (33, 72, 4, 9, 7, "uniform", False),
    (96, 512, 8, 85, 6, "uniform", False),
    (40, 126, 18, 21619, 1, "uniform", False),
    (64, 960, 32, 5000, 8, "uniform", True),
]


@pytest.mark.parametrize("N,K,v,Kc,M,dist,mu", SMALL)
def test_gemv_parity_small(N, K, v, Kc, M, dist, mu):
    L = wl.make_layer(_spec(N, K, v, Kc, idx_dist=dist, with_mu=mu, outlier_frac=0.01), M, seed=N + K + M)
    y, _ = run_layer(L, "gemv")
    rel, fwd = errors(y, oracle_y(L), L)
    assert rel <= TOL_GEMV and fwd <= TOL_GEMV, (rel, fwd)


@pytest.mark.parametrize("config", [1, 2, 3])
def test_gemv_parity_benchmark_configs(config):
    """Full-size layers of the benchmark configs, every output compared (the oracle needs seconds)."""
    cfg = wl.CONFIGS[config]
    seen = set()
    for lid, spec in enumerate(cfg["layers"]):
        if (spec.N, spec.K) in seen:
            continue
        seen.add((spec.N, spec.K))
        for M in cfg["M"]:
            L = wl.make_layer(spec, M, cfg["seed"], lid)
            y, _ = run_layer(L, "gemv")
            rel, fwd = errors(y, oracle_y(L), L)
            assert rel <= TOL_GEMV and fwd <= TOL_GEMV, (spec, M, rel, fwd)


def test_gemv_is_deterministic_and_respects_bounds():
    L = wl.make_layer(_spec(517, 4096, 16, 8192), 8, seed=3)
    d = to_device(L)
    M, N = 8, 517
    guard = torch.full((M * N + 512,), 12345.0, dtype=torch.float32, device="cuda")
    out = guard[256:256 + M * N].view(M, N)
    btc.linear_gemv(d["x"], d["idx"], d["Cp"], d["alpha"], 16, 8192, out=out)
    first = out.clone()
    btc.linear_gemv(d["x"], d["idx"], d["Cp"], d["alpha"], 16, 8192, out=out)
    torch.cuda.synchronize()
    assert torch.equal(first, out)
    assert bool((guard[:256] == 12345.0).all()) and bool((guard[256 + M * N:] == 12345.0).all())


@pytest.mark.parametrize("dt", [torch.float16, torch.bfloat16])
def test_gemv_half_outputs(dt):
    L = wl.make_layer(_spec(300, 1024, 16, 4096), 2, seed=9)
    y32, _ = run_layer(L, "gemv")
    y16, _ = run_layer(L, "gemv", out_dtype=dt)
    assert torch.equal(y16, y32.to(dt))


def test_gemv_bf16_activations():
    L = wl.make_layer(_spec(260, 2048, 16, 8192, x_dtype="bf16"), 4, seed=12)
    y, _ = run_layer(L, "gemv")
    rel, fwd = errors(y, oracle_y(L), L)
    assert rel <= TOL_GEMV and fwd <= TOL_GEMV


# ------------------------------------------------------------------ tensor-core path parity

GEMM_SMALL = [
    # N, K, v, Kc, M, xdt, mu
    (128, 64, 16, 100, 128, "bf16", False),
    (256, 256, 16, 8192, 256, "bf16", False),
    (200, 320, 16, 4096, 130, "bf16", True),
    (384, 1024, 16, 8192, 512, "f16", False),
    (130, 640, 20, 65536, 300, "bf16", False),
    (1000, 512, 8, 85, 9, "bf16", True),
    (512, 2048, 16, 7132, 1024, "bf16", False),
    # v = 20 with K a multiple of 320 (weights through tensor memory): one index tile exactly; a K that ends inside an
    # index tile with the table in shared memory; 256-row x tiles
    (300, 1280, 20, 65536, 130, "f16", True),
    (260, 2240, 20, 5000, 600, "bf16", False),
    (7680, 640, 20, 4096, 512, "bf16", False),
]


@pytest.mark.parametrize("N,K,v,Kc,M,xdt,mu", GEMM_SMALL)
def test_gemm_parity_small(N, K, v, Kc, M, xdt, mu):
    L = wl.make_layer(_spec(N, K, v, Kc, x_dtype=xdt, with_mu=mu), M, seed=N + K + M)
    y, _ = run_layer(L, "gemm")
    rel, fwd = errors(y, oracle_y(L), L)
    assert rel <= TOL_GEMM and fwd <= TOL_GEMM, (rel, fwd)


def test_gemm_parity_benchmark_config_M512_every_output():
    """Config 4 at M = 512 in the launch configuration the bench times: the three full-size layers, every one of the
    M x N outputs against the full fp64 product (seconds per shape on the host cores)."""
    cfg = wl.CONFIGS[4]
    for lid, spec in enumerate(cfg["layers"]):
        L = wl.make_layer(spec, 512, cfg["seed"], lid)
        y, _ = run_layer(L, "gemm")
        rel, fwd = errors(y, oracle_y(L), L)
        assert rel <= TOL_GEMM and fwd <= TOL_GEMM, (spec, rel, fwd)
    assert btc.device_status() == 0


def test_gemm_parity_benchmark_config_M2048():
    """Config 4 at M = 2048: the 4096 x 4096 layer in full; for the two 11008-wide layers the oracle recomputes one
    row of x out of every 128-row tile (a different offset in each tile, so every CTA row of either tile height is
    touched), plus the first and last rows, with all N columns of each -- every CTA of the launch is covered."""
    cfg = wl.CONFIGS[4]
    M = 2048
    for lid, spec in enumerate(cfg["layers"]):
        L = wl.make_layer(spec, M, cfg["seed"], lid)
        y, _ = run_layer(L, "gemm")
        assert bool(torch.isfinite(y).all())
        if spec.N == spec.K:
            rel, fwd = errors(y, oracle_y(L), L)
        else:
            tiles = np.arange(M // 128)
            rows = np.unique(np.concatenate([[0, 1, 127, 128, M - 1], tiles * 128 + (tiles * 37 + 11) % 128]))
            sub = wl.LayerData(spec, len(rows), L.C_pm1, L.idx, L.alpha, L.x_bits[rows].copy(), L.mu)
            rel, fwd = errors(y[torch.from_numpy(rows).cuda()], oracle_y(sub), sub)
        assert rel <= TOL_GEMM and fwd <= TOL_GEMM, (spec, M, rel, fwd)
    assert btc.device_status() == 0


def test_gemm_parity_config3_shapes_v20_M512():
    """The tensor-core path on the config-3 layers (v = 20, 65536 centroids, Zipf indices; K = 5120 = 16 x 320, so the
    weights go through tensor memory in the five-phase expansion) at M = 512, bf16 activations as on that path: one row
    of x out of every 128-row tile plus the first and last rows, all N columns of each, against the oracle."""
    cfg = wl.CONFIGS[3]
    M = 512
    for lid in (0, 4):
        spec = replace(cfg["layers"][lid], x_dtype="bf16")
        L = wl.make_layer(spec, M, cfg["seed"], lid)
        y, _ = run_layer(L, "gemm")
        assert bool(torch.isfinite(y).all())
        tiles = np.arange(M // 128)
        rows = np.unique(np.concatenate([[0, 1, 127, 128, 255, 256, M - 1], tiles * 128 + (tiles * 37 + 11) % 128]))
        sub = wl.LayerData(spec, len(rows), L.C_pm1, L.idx, L.alpha, L.x_bits[rows].copy(), L.mu)
        rel, fwd = errors(y[torch.from_numpy(rows).cuda()], oracle_y(sub), sub)
        assert rel <= TOL_GEMM and fwd <= TOL_GEMM, (spec, rel, fwd)
    assert btc.device_status() == 0


SPLIT_K = [
    # N, K, M, xdt, mu, out dtype   (v = 16, few 128-row tiles, K >= 4096: the tensor-core path splits K over the idle SMs)
    (300, 4096, 16, "bf16", False, torch.float32),
    (200, 11008, 9, "f16", True, torch.float32),
    (1000, 5120, 100, "bf16", True, torch.float16),
    (640, 8192, 300, "bf16", False, torch.bfloat16),
]


@pytest.mark.parametrize("N,K,M,xdt,mu,odt", SPLIT_K)
def test_gemm_split_k_matches_oracle_and_unsplit(N, K, M, xdt, mu, odt):
    """With the full workspace K is split over several CTAs per tile and the partial sums are added in a fixed order;
    with only the minimum workspace (the entry point without allocation) the same call runs unsplit.  Both against
    the oracle; the split result twice, bit for bit."""
    L = wl.make_layer(_spec(N, K, 16, 8192, x_dtype=xdt, with_mu=mu), M, seed=N + K + M)
    d = to_device(L)
    assert btc.linear_workspace_bytes(M, N, K, 16, 8192) > 4 * M * N          # room for at least two partial copies
    y1 = btc.linear_gemm(d["x"], d["idx"], d["Cp"], d["alpha"], 16, 8192, mu=d["mu"], out_dtype=odt)
    y2 = btc.linear_gemm(d["x"], d["idx"], d["Cp"], d["alpha"], 16, 8192, mu=d["mu"], out_dtype=odt)
    y3 = btc.linear_gemm_static_scratch(d["x"], d["idx"], d["Cp"], d["alpha"], 16, 8192, mu=d["mu"])
    torch.cuda.synchronize()
    assert torch.equal(y1, y2)
    want = oracle_y(L)
    tol = TOL_GEMM if odt == torch.float32 else TOL_GEMM + 2.0 ** -8
    for y in (y1, y3):
        rel, fwd = errors(y.float(), want, L)
        assert rel <= tol and fwd <= tol, (N, K, M, rel, fwd)
    assert btc.device_status() == 0


def test_gemm_deterministic_and_bounded():
    L = wl.make_layer(_spec(300, 1024, 16, 8192, x_dtype="bf16"), 200, seed=5)
    d = to_device(L)
    M, N = 200, 300
    guard = torch.full((M * N + 512,), 777.0, dtype=torch.float32, device="cuda")
    out = guard[256:256 + M * N].view(M, N)
    btc.linear_gemm(d["x"], d["idx"], d["Cp"], d["alpha"], 16, 8192, out=out)
    first = out.clone()
    btc.linear_gemm(d["x"], d["idx"], d["Cp"], d["alpha"], 16, 8192, out=out)
    torch.cuda.synchronize()
    assert torch.equal(first, out)
    assert bool((guard[:256] == 777.0).all()) and bool((guard[256 + M * N:] == 777.0).all())


# ------------------------------------------------------------------ several layers in one launch

def test_gemv_batch_matches_oracle_and_single_calls():
    """Seven layers of mixed shape (the decode layer set scaled down, ragged N, one with mu, one bf16) in one
    btc_linear_gemv_batch call: every output against the oracle, and (for M <= 2, where both run the same kernel) bit-identical to the per-layer call."""
    shapes = [(272, 1024, 16, 4096, False, "f16"), (272, 1024, 16, 4096, True, "f16"), (100, 1024, 16, 8192, False, "f16"),
              (1000, 1024, 16, 8192, False, "bf16"), (688, 2752, 16, 8192, False, "f16"), (37, 320, 20, 65536, False, "f16"),
              (513, 640, 20, 21619, True, "f16"), (64, 96, 12, 777, False, "f16"), (300, 2048, 16, 8192, False, "f16")]
    for M in (1, 2, 8):
        Ls = [wl.make_layer(_spec(N, K, v, Kc, with_mu=mu, x_dtype=dt, outlier_frac=0.01), M, seed=50 + i)
              for i, (N, K, v, Kc, mu, dt) in enumerate(shapes)]
        ds = [to_device(L) for L in Ls]
        layers = [dict(x=d["x"], idx=d["idx"], C_packed=d["Cp"], alpha=d["alpha"], mu=d["mu"], v=L.spec.v, Kc=L.spec.Kc)
                  for L, d in zip(Ls, ds)]
        outs = btc.linear_gemv_batch(layers)
        torch.cuda.synchronize()
        for L, d, y in zip(Ls, ds, outs):
            rel, fwd = errors(y, oracle_y(L), L)
            assert rel <= TOL_GEMV and fwd <= TOL_GEMV, (L.spec, M, rel, fwd)
            single = btc.linear_gemv(d["x"], d["idx"], d["Cp"], d["alpha"], L.spec.v, L.spec.Kc, mu=d["mu"])
            if M <= 2:      # same kernel, same arithmetic: identical bits
                assert torch.equal(single, y), (L.spec, M)
            else:           # single calls with M > 2 take the fp16 bit-trick kernel
                rel2, fwd2 = errors(single, oracle_y(L), L)
                assert rel2 <= TOL_GEMV and fwd2 <= TOL_GEMV, (L.spec, M, rel2, fwd2)
    assert btc.device_status() == 0


@pytest.mark.parametrize("M", [1, 2, 4, 8])
def test_fused_decode_step_full_size_every_output(M):
    """The launch the benchmark's headline times: ONE btc_linear_gemv_batch call over the seven full-size layers of
    the LLaMA-2-7B-shaped decode set (config 2), at the M the bench runs it with; every output of every layer against
    the oracle."""
    cfg = wl.CONFIGS[2]
    Ls = [wl.make_layer(s, M, cfg["seed"], i) for i, s in enumerate(cfg["layers"])]
    ds = [to_device(L) for L in Ls]
    outs = btc.GemvBatch([dict(x=d["x"], idx=d["idx"], C_packed=d["Cp"], alpha=d["alpha"], v=L.spec.v, Kc=L.spec.Kc)
                          for L, d in zip(Ls, ds)]).run()
    torch.cuda.synchronize()
    for L, y in zip(Ls, outs):
        rel, fwd = errors(y, oracle_y(L), L)
        assert rel <= TOL_GEMV and fwd <= TOL_GEMV, (L.spec, M, rel, fwd)
    assert btc.device_status() == 0


@pytest.mark.parametrize("M", [1, 2, 4, 8])
def test_gemv_batch_large_codebooks_16bit_table(M):
    """Codebooks too large to sit in shared memory as 32-bit words (v <= 16): the decode kernel keeps them as 16-bit
    halves.  65536 centroids at v = 16 is the codebook of all patterns; 40000 and a v = 12 layer ride in the same launch."""
    shapes = [(200, 4096, 16, 65536, True, "uniform"), (130, 1024, 16, 40000, False, "zipf"), (64, 768, 12, 4096, False, "uniform"),
              (300, 11008, 16, 65536, False, "uniform")]
    Ls = [wl.make_layer(_spec(N, K, v, Kc, idx_dist=dist, with_mu=mu, outlier_frac=0.01), M, seed=900 + i)
          for i, (N, K, v, Kc, mu, dist) in enumerate(shapes)]
    ds = [to_device(L) for L in Ls]
    outs = btc.linear_gemv_batch([dict(x=d["x"], idx=d["idx"], C_packed=d["Cp"], alpha=d["alpha"], mu=d["mu"], v=L.spec.v, Kc=L.spec.Kc)
                                  for L, d in zip(Ls, ds)])
    torch.cuda.synchronize()
    for L, y in zip(Ls, outs):
        rel, fwd = errors(y, oracle_y(L), L)
        assert rel <= TOL_GEMV and fwd <= TOL_GEMV, (L.spec, M, rel, fwd)
    assert btc.device_status() == 0


@pytest.mark.parametrize("Kc", [256, 4096, 65536])
@pytest.mark.parametrize("dist", ["uniform", "zipf"])
def test_chained_decode_blocks_with_teacher_forcing(Kc, dist):
    """The dependent decode chain in the launch grouping the benchmark times ({q,k,v}, o, {gate,up}, down; fp16
    outputs feed the next launch), two blocks at full layer sizes: every layer's output against the oracle evaluated
    on the fp16 activations the chain actually handed to that layer."""
    cfg5 = wl.config_layers(5, Kc=Kc, idx_dist=dist)
    sp = cfg5["layers"]
    Ls = [wl.make_layer(s5, 1, cfg5["seed"], i) for i, s5 in enumerate(sp)]
    ds = [to_device(L) for L in Ls]
    lay = [dict(idx=d["idx"], C_packed=d["Cp"], alpha=d["alpha"], v=L.spec.v, Kc=L.spec.Kc) for L, d in zip(Ls, ds)]
    h = ds[0]["x"][:1].clone()
    f16 = lambda n: torch.empty((1, n), dtype=torch.float16, device="cuda")
    for blk in range(2):
        qkv = [f16(4096) for _ in range(3)]
        o_out, gu, nxt = f16(4096), [f16(11008) for _ in range(2)], f16(4096)
        steps = [([0, 1, 2], h, qkv), ([3], qkv[0], [o_out]), ([4, 5], o_out, gu), ([6], gu[0], [nxt])]
        for ids, xin, outs in steps:
            btc.GemvBatch([dict(x=xin, out=o, **lay[i]) for i, o in zip(ids, outs)]).run()
            torch.cuda.synchronize()
            x64 = xin.double().cpu().numpy()
            assert np.isfinite(x64).all() and np.abs(x64).max() < 1e3      # unit-gain chain: no drift towards overflow
            for i, o in zip(ids, outs):
                want = oracle.linear(x64, Ls[i].idx, Ls[i].C_pm1, Ls[i].alpha, None)
                got = o.double().cpu().numpy()
                # the output is the fp32 result rounded to fp16: half an fp16 ulp on top of the decode tolerance
                tol = TOL_GEMV * np.abs(want).max() + 2.0 ** -11 * np.abs(want)
                assert (np.abs(got - want) <= tol).all(), (Kc, dist, blk, i, float(np.abs(got - want).max()), float(np.abs(want).max()))
        h = nxt
    assert btc.device_status() == 0


# ------------------------------------------------------------------ online activation transform

@pytest.mark.parametrize("path,M,k1,k2", [("gemv", 2, 32, 32), ("gemv", 1, 64, 64), ("gemm", 96, 16, 64), ("gemv", 8, 8, 40), ("gemv", 4, 64, 64), ("gemm", 300, 20, 72),
                                           ("gemm", 200, 64, 64), ("gemm", 130, 48, 96), ("gemm", 64, 100, 32), ("gemm", 70, 40, 48)])
def test_online_transform_prologue(path, M, k1, k2):
    """x' = x * diag(sigma) * (P1 kron P2) before the layer (Section 4.2, applied on the fly): against the oracle's dense
    K x K Kronecker form in fp64.  On the decode path x' stays fp32 up to the layer kernel, so the decode tolerance holds;
    on the tensor-core path x' is rounded to the activation dtype, as any activation is there.  From 64 rows on, with k2 a
    multiple of 16, the two products run on the warp-level tensor cores (tf32): the last four cases, with k1 that is and is
    not a multiple of 16 and of 8, and k2 on both bank phases."""
    K = k1 * k2
    v = 16 if K % 16 == 0 else 20
    L = wl.make_layer(_spec(272, K, v, 4096, x_dtype="f16" if path == "gemv" else "bf16"), M, seed=77 + k1)
    rng = np.random.default_rng(5 + k1)
    sigma = rng.choice(np.array([-1, 1], dtype=np.int8), size=K)
    P1 = np.linalg.qr(rng.standard_normal((k1, k1)))[0].astype(np.float32)
    P2 = np.linalg.qr(rng.standard_normal((k2, k2)))[0].astype(np.float32)
    bits = np.zeros((K + 31) // 32, dtype=np.uint32)
    for i in np.nonzero(sigma < 0)[0]:
        bits[i >> 5] |= np.uint32(1) << np.uint32(i & 31)
    d = to_device(L)
    tr = (torch.from_numpy(bits.view(np.int32)).cuda(), torch.from_numpy(P1).cuda(), torch.from_numpy(P2).cuda())
    fn = btc.linear_gemv if path == "gemv" else btc.linear_gemm
    y = fn(d["x"], d["idx"], d["Cp"], d["alpha"], v, 4096, transform=tr)
    torch.cuda.synchronize()
    xt = oracle.transform(L.x_f64(), sigma, P1.astype(np.float64), P2.astype(np.float64))
    ref = oracle.linear(xt, L.idx, L.C_pm1, L.alpha)
    err = np.abs(y.double().cpu().numpy() - ref)
    tol = TOL_GEMV if path == "gemv" else TOL_GEMM
    assert err.max() / np.abs(ref).max() <= tol
    scale = np.outer(np.abs(xt).sum(1), np.abs(L.alpha.astype(np.float64)))
    assert (err / np.maximum(scale, 1e-300)).max() <= tol


@pytest.mark.parametrize("M,k1,k2,xdt", [(1, 64, 64, "f16"), (2, 32, 40, "bf16"), (4, 64, 64, "f16")])
def test_shared_transform_then_fused_layers(M, k1, k2, xdt):
    """Layers that share their input (q / k / v of a block): btc_activation_transform once, fp32 x' out, then ONE
    btc_linear_gemv_batch call over the three layers on x'.  x' itself against the oracle's dense Kronecker form (fp32
    products of fp32 factors: 1e-5 of the row's largest |x'|; rounded to the 16-bit dtype: half an ulp more), every
    output of every layer against oracle.linear on the oracle's x' at the decode tolerance."""
    K = k1 * k2
    Ls = [wl.make_layer(_spec(N, K, 16, 4096, x_dtype=xdt), M, seed=91 + i, layer_id=i) for i, N in enumerate((272, 520, 272))]
    rng = np.random.default_rng(3 + k1)
    sigma = rng.choice(np.array([-1, 1], dtype=np.int8), size=K)
    P1 = np.linalg.qr(rng.standard_normal((k1, k1)))[0].astype(np.float32)
    P2 = np.linalg.qr(rng.standard_normal((k2, k2)))[0].astype(np.float32)
    bits = np.zeros((K + 31) // 32, dtype=np.uint32)
    for i in np.nonzero(sigma < 0)[0]:
        bits[i >> 5] |= np.uint32(1) << np.uint32(i & 31)
    tr = (torch.from_numpy(bits.view(np.int32)).cuda(), torch.from_numpy(P1).cuda(), torch.from_numpy(P2).cuda())
    ds = [to_device(L) for L in Ls]
    x = ds[0]["x"]                                           # the shared input: layer 0's activations
    x64 = Ls[0].x_f64()
    xt_ref = oracle.transform(x64, sigma, P1.astype(np.float64), P2.astype(np.float64))
    xt = btc.activation_transform(x, tr)
    xt16 = btc.activation_transform(x, tr, out_dtype=x.dtype)
    torch.cuda.synchronize()
    big = np.abs(xt_ref).max(axis=1, keepdims=True)
    assert (np.abs(xt.double().cpu().numpy() - xt_ref) <= 1e-5 * big).all()
    ulp = 2.0 ** -11 if xdt == "f16" else 2.0 ** -8
    assert (np.abs(xt16.double().cpu().numpy() - xt_ref) <= 1e-5 * big + ulp * np.abs(xt_ref)).all()
    outs = btc.linear_gemv_batch([dict(x=xt, idx=d["idx"], C_packed=d["Cp"], alpha=d["alpha"], v=16, Kc=4096) for d in ds])
    torch.cuda.synchronize()
    for L, y in zip(Ls, outs):
        ref = oracle.linear(xt_ref, L.idx, L.C_pm1, L.alpha)
        err = np.abs(y.double().cpu().numpy() - ref)
        assert err.max() / np.abs(ref).max() <= TOL_GEMV
        scale = np.outer(np.abs(xt_ref).sum(1), np.abs(L.alpha.astype(np.float64)))
        assert (err / np.maximum(scale, 1e-300)).max() <= TOL_GEMV
    assert btc.device_status() == 0


@pytest.mark.parametrize("M,k1,k2,xdt", [(96, 48, 96, "f16"), (64, 86, 128, "bf16"), (130, 64, 64, "bf16")])
def test_activation_transform_many_rows(M, k1, k2, xdt):
    """btc_activation_transform from 64 rows on (the tf32 tensor-core form; 86 x 128 and 64 x 64 are the shapes with
    compile-time sizes) against the oracle's dense Kronecker form, on sampled rows where K is large: fp32 output within
    2^-9 of the row's largest |x'| (two tf32 roundings per product term, random signs), 16-bit output half an ulp more."""
    K = k1 * k2
    rng = np.random.default_rng(9 + k1)
    x_bits = wl.make_x(M, K, xdt, 4242, 3)
    x64 = (x_bits.view(np.float16).astype(np.float64) if xdt == "f16"
           else wl.bf16_bits_to_f32(x_bits).astype(np.float64)).reshape(M, K)
    sigma = rng.choice(np.array([-1, 1], dtype=np.int8), size=K)
    P1 = np.linalg.qr(rng.standard_normal((k1, k1)))[0].astype(np.float32)
    P2 = np.linalg.qr(rng.standard_normal((k2, k2)))[0].astype(np.float32)
    bits = np.zeros((K + 31) // 32, dtype=np.uint32)
    for i in np.nonzero(sigma < 0)[0]:
        bits[i >> 5] |= np.uint32(1) << np.uint32(i & 31)
    tr = (torch.from_numpy(bits.view(np.int32)).cuda(), torch.from_numpy(P1).cuda(), torch.from_numpy(P2).cuda())
    dt = torch.float16 if xdt == "f16" else torch.bfloat16
    x = torch.from_numpy(x_bits.view(np.int16).reshape(M, K).copy()).cuda().view(dt)
    xt = btc.activation_transform(x, tr)
    xt16 = btc.activation_transform(x, tr, out_dtype=dt)
    torch.cuda.synchronize()
    rows = np.arange(M) if K <= 4608 else np.array([0, 1, M // 2, M - 1])
    ref = oracle.transform(x64[rows], sigma, P1.astype(np.float64), P2.astype(np.float64))
    big = np.abs(ref).max(axis=1, keepdims=True)
    got = xt[torch.from_numpy(rows).cuda()].double().cpu().numpy()
    assert (np.abs(got - ref) <= 2.0 ** -9 * big).all(), float((np.abs(got - ref) / big).max())
    got16 = xt16[torch.from_numpy(rows).cuda()].double().cpu().numpy()
    ulp = 2.0 ** -11 if xdt == "f16" else 2.0 ** -8
    assert (np.abs(got16 - ref) <= 2.0 ** -9 * big + ulp * np.abs(ref)).all()
    assert btc.device_status() == 0


def test_online_transform_full_size_M512():
    """The transform in front of the 4096 x 4096 config-4 layer at M = 512 (K = 64 x 64: the tensor-core form of the
    transform, then the tensor-core layer kernel), as the benchmark times it: six rows of x spread over the row tiles,
    all N columns of each, against the oracle's dense Kronecker form followed by the oracle layer."""
    cfg = wl.CONFIGS[4]
    spec, M, k1, k2 = cfg["layers"][0], 512, 64, 64
    L = wl.make_layer(spec, M, cfg["seed"], 0)
    rng = np.random.default_rng(11)
    sigma = rng.choice(np.array([-1, 1], dtype=np.int8), size=spec.K)
    P1 = np.linalg.qr(rng.standard_normal((k1, k1)))[0].astype(np.float32)
    P2 = np.linalg.qr(rng.standard_normal((k2, k2)))[0].astype(np.float32)
    bits = np.zeros((spec.K + 31) // 32, dtype=np.uint32)
    for i in np.nonzero(sigma < 0)[0]:
        bits[i >> 5] |= np.uint32(1) << np.uint32(i & 31)
    d = to_device(L)
    tr = (torch.from_numpy(bits.view(np.int32)).cuda(), torch.from_numpy(P1).cuda(), torch.from_numpy(P2).cuda())
    y = btc.linear_gemm(d["x"], d["idx"], d["Cp"], d["alpha"], spec.v, spec.Kc, transform=tr)
    torch.cuda.synchronize()
    assert bool(torch.isfinite(y).all())
    rows = np.array([0, 127, 128, 300, 383, M - 1])
    xt = oracle.transform(L.x_f64()[rows], sigma, P1.astype(np.float64), P2.astype(np.float64))
    ref = oracle.linear(xt, L.idx, L.C_pm1, L.alpha)
    err = np.abs(y[torch.from_numpy(rows).cuda()].double().cpu().numpy() - ref)
    assert err.max() / np.abs(ref).max() <= TOL_GEMM
    scale = np.outer(np.abs(xt).sum(1), np.abs(L.alpha.astype(np.float64)))
    assert (err / np.maximum(scale, 1e-300)).max() <= TOL_GEMM
    assert btc.device_status() == 0


# ------------------------------------------------------------------ invariants through the production kernels

@pytest.mark.parametrize("path,M", [("gemv", 1), ("gemv", 6), ("gemm", 72)])
def test_codebook_permutation_and_negation_invariance(path, M):
    """Relabelling the centroids (codebook rows permuted, indices remapped) must not change y at all, and negating
    every centroid together with every alpha must give the same y: both hold bit for bit, because each kernel sees the
    same weights in the same order."""
    N, K, v, Kc = 304, 1024, 16, 4096
    L = wl.make_layer(_spec(N, K, v, Kc, x_dtype="f16" if path == "gemv" else "bf16"), M, seed=31)
    y0, _ = run_layer(L, path)
    rng = np.random.default_rng(3)
    perm = rng.permutation(Kc)                       # new position of old centroid k is inv[k]
    inv = np.empty(Kc, dtype=np.int64)
    inv[perm] = np.arange(Kc)
    L1 = wl.LayerData(L.spec, M, L.C_pm1[perm].copy(), inv[L.idx].astype(np.uint16), L.alpha, L.x_bits, L.mu)
    y1, _ = run_layer(L1, path)
    assert torch.equal(y0, y1)
    L2 = wl.LayerData(L.spec, M, (-L.C_pm1).astype(np.int8), L.idx, (-L.alpha).astype(np.float16), L.x_bits, L.mu)
    y2, _ = run_layer(L2, path)
    rel, fwd = errors(y2, oracle_y(L), L)
    tol = TOL_GEMV if path == "gemv" else TOL_GEMM
    assert rel <= tol and fwd <= tol
    if path == "gemm":                               # exact +-1 products, same accumulation order
        assert torch.equal(y0, y2)


def test_gemv_is_linear_in_x_for_powers_of_two():
    """Scaling x by a power of two scales y by the same factor exactly (the per-slice block-fixed-point scale follows)."""
    L = wl.make_layer(_spec(272, 2048, 16, 8192), 2, seed=8)
    y0, _ = run_layer(L, "gemv")
    L4 = wl.LayerData(L.spec, 2, L.C_pm1, L.idx, L.alpha, (L.x_bits.view(np.float16) * np.float16(4.0)).view(np.uint16), L.mu)
    y4, _ = run_layer(L4, "gemv")
    assert torch.equal(y4, 4.0 * y0)


def test_rows_of_x_are_independent():
    """Row m of y depends on row m of x only: running rows one at a time gives the same numbers as running them together."""
    L = wl.make_layer(_spec(272, 1024, 16, 4096), 2, seed=21)
    y, d = run_layer(L, "gemv")
    for m in range(2):
        ym = btc.linear_gemv(d["x"][m:m + 1].contiguous(), d["idx"], d["Cp"], d["alpha"], 16, 4096)
        assert torch.equal(ym[0], y[m])


def test_gemm_many_tiles_ragged_shapes():
    """More tiles than SMs, ragged N and M, and a K that ends inside an index tile (17 k steps); 30 sampled rows of y
    (all columns) against the oracle, with mu."""
    N, K, M = 2100, 1088, 2300
    L = wl.make_layer(_spec(N, K, 16, 7132, x_dtype="bf16", with_mu=True), M, seed=123)
    y, _ = run_layer(L, "gemm")
    rows = np.unique(np.concatenate([[0, 127, 128, 255, 256, M - 1], (np.arange(24) * 97 + 13) % M]))
    sub = wl.LayerData(L.spec, len(rows), L.C_pm1, L.idx, L.alpha, L.x_bits[rows].copy(), L.mu)
    rel, fwd = errors(y[torch.from_numpy(rows).cuda()], oracle_y(sub), sub)
    assert rel <= TOL_GEMM and fwd <= TOL_GEMM, (rel, fwd)
    assert bool(torch.isfinite(y).all()) and btc.device_status() == 0


# ------------------------------------------------------------------ failure detection without a GPU fault

def test_bounded_wait_gives_up_and_context_stays_usable():
    """A wait whose partner never arrives must run out (about a millisecond here), raise the status word and return;
    afterwards the status can be cleared and the kernels still work."""
    assert btc.device_status() == 0
    btc.selftest_bounded_wait()
    torch.cuda.synchronize()
    assert btc.device_status() == 7          # BTC_ERR_TIMEOUT
    btc.device_status_reset()
    assert btc.device_status() == 0
    L = wl.make_layer(_spec(272, 1024, 16, 4096), 1, seed=2)
    y, _ = run_layer(L, "gemv")
    rel, fwd = errors(y, oracle_y(L), L)
    assert rel <= TOL_GEMV and fwd <= TOL_GEMV and btc.device_status() == 0


def test_debug_index_check_raises_status_word_only():
    """BTC_DEBUG_CHECK_INDICES=1 (read when the library first needs it, hence a fresh process): every linear call first
    runs a range check of idx on the same stream; an index >= Kc raises the status word (BTC_ERR_INDEX = 8), nothing
    traps, and after a reset the library works as before.  The planted index (Kc + 4 of a 4096-entry table that sits in
    shared memory in front of the index stages) keeps the layer kernel's own lookup inside its shared memory."""
    import os
    import subprocess
    import sys
    code = r'''
import numpy as np, torch, sys
sys.path.insert(0, "tests")
import paper_2506_12040_b200 as btc, workloads as wl
from util import to_device
L = wl.make_layer(wl.LayerSpec("t", 64, 256, 16, 4096), 1, seed=1)
d = to_device(L)
assert btc.device_status() == 0
btc.linear_gemv(d["x"], d["idx"], d["Cp"], d["alpha"], 16, 4096); torch.cuda.synchronize()
assert btc.device_status() == 0
bad = d["idx"].clone(); bad[3, 2] = 4100
btc.linear_gemv(d["x"], bad, d["Cp"], d["alpha"], 16, 4096); torch.cuda.synchronize()
assert btc.device_status() == 8, btc.device_status()
btc.device_status_reset()
y = btc.linear_gemv(d["x"], d["idx"], d["Cp"], d["alpha"], 16, 4096); torch.cuda.synchronize()
assert btc.device_status() == 0 and bool(torch.isfinite(y).all())
print("index check ok")
'''
    env = dict(os.environ, BTC_DEBUG_CHECK_INDICES="1")
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    r = subprocess.run([sys.executable, "-c", code], cwd=root, env=env, capture_output=True, text=True, timeout=600)
    assert r.returncode == 0 and "index check ok" in r.stdout, r.stdout + r.stderr


# ------------------------------------------------------------------ dense-packed indices (Section 4.3 index width)

@pytest.mark.parametrize("Kc,N,Kb", [(2, 5, 16), (256, 33, 24), (4096, 300, 64), (8192, 129, 688), (7132, 17, 40), (21619, 64, 8),
                                     (65536, 9, 16)])
def test_index_pack_and_unpack_bit_exact(Kc, N, Kb):
    """btc_index_pack / btc_index_unpack against the oracle's bit-by-bit packing: every byte, padding included."""
    idx = wl.make_indices(N, Kb, Kc, "uniform", 77 + Kc, 1)
    d = torch.from_numpy(idx.view(np.int16)).cuda()
    packed = btc.index_pack(d, Kc)
    bits = oracle.index_bits(Kc)
    assert btc.index_bits(Kc) == bits and packed.shape[1] == oracle.packed_row_bytes(Kb, bits)
    assert np.array_equal(packed.cpu().numpy(), oracle.pack_indices(idx, bits))
    back = btc.index_unpack(packed, Kb, Kc)
    assert np.array_equal(back.cpu().numpy().view(np.uint16), idx)


@pytest.mark.parametrize("N,K,v,Kc,M,mu", [(300, 2048, 16, 4096, 1, False), (129, 4096, 16, 8192, 2, True), (1000, 11008, 16, 8192, 1, False),
                                           (257, 1152, 16, 7132, 8, False), (77, 1152, 12, 4096, 4, True), (64, 512, 8, 4096, 1, False)])
def test_linear_on_packed_indices_matches_oracle_and_unpacked(N, K, v, Kc, M, mu):
    """The decode kernel reading 12- / 13-bit rows: every output against the oracle, and bit-identical to the same kernel
    reading the uint16 containers (same lookups, same arithmetic)."""
    L = wl.make_layer(_spec(N, K, v, Kc, with_mu=mu, outlier_frac=0.01), M, seed=N + K + M)
    d = to_device(L)
    packed = btc.index_pack(d["idx"], Kc)
    y = btc.linear_gemv_packed(d["x"], packed, d["Cp"], d["alpha"], v, Kc, mu=d["mu"])
    # (a one-term sum runs the same kernel on the uint16 containers; plain calls at M <= 2 take another geometry)
    y16 = btc.linear_gemv_sum(d["x"], [dict(k0=0, idx=d["idx"], C_packed=d["Cp"], alpha=d["alpha"], mu=d["mu"], v=v, Kc=Kc)], N)
    torch.cuda.synchronize()
    rel, fwd = errors(y, oracle_y(L), L)
    assert rel <= TOL_GEMV and fwd <= TOL_GEMV, (rel, fwd)
    assert torch.equal(y, y16)
    assert btc.device_status() == 0


def test_fused_decode_step_on_packed_indices_full_size():
    """The seven full-size layers of config 2 as ONE launch over 13-bit index rows (M = 1): every output against the oracle."""
    cfg = wl.CONFIGS[2]
    Ls = [wl.make_layer(s, 1, cfg["seed"], i) for i, s in enumerate(cfg["layers"])]
    ds = [to_device(L) for L in Ls]
    outs = btc.GemvBatch([dict(x=d["x"], idx=btc.index_pack(d["idx"], L.spec.Kc), idx_bits=13, C_packed=d["Cp"], alpha=d["alpha"],
                               v=L.spec.v, Kc=L.spec.Kc) for L, d in zip(Ls, ds)]).run()
    torch.cuda.synchronize()
    for L, y in zip(Ls, outs):
        rel, fwd = errors(y, oracle_y(L), L)
        assert rel <= TOL_GEMV and fwd <= TOL_GEMV, (L.spec, rel, fwd)
    assert btc.device_status() == 0


# ------------------------------------------------------------------ scale groups per row / residual terms

@pytest.mark.parametrize("M,N,K", [(1, 300, 4096), (2, 129, 2048), (8, 257, 4096)])
def test_linear_sum_of_terms_groups_and_residual(M, N, K):
    """Three column groups with their own (alpha, mu) over ONE index matrix (column-range views), plus a residual term
    with its own codebook and indices over the first group's columns: btc_linear_gemv_sum against the oracle's dense sum."""
    v, Kc = 16, 4096
    L = wl.make_layer(_spec(N, K, v, Kc, with_mu=True, outlier_frac=0.01), M, seed=N + K + M)
    d = to_device(L)
    Kb = K // v
    bounds = [0, Kb // 4, Kb // 4 + Kb // 2, Kb]                  # in blocks; multiples of 8
    assert all(b % 8 == 0 for b in bounds)
    rng = np.random.default_rng(N)
    als = [(np.abs(rng.standard_normal(N)) * 0.02).astype(np.float16) for _ in range(3)]
    mus = [(rng.standard_normal(N) * 0.002).astype(np.float16) for _ in range(3)]
    L2 = wl.make_layer(_spec(N, bounds[1] * v, v, 300), M, seed=5 + N)       # the residual term's codebook / indices / scale
    d2 = to_device(L2)
    al2 = (L2.alpha.astype(np.float32) * 0.25).astype(np.float16)
    dev = lambda a: torch.from_numpy(a.view(np.int16).copy()).cuda().view(torch.float16)
    terms = [dict(k0=bounds[g] * v, idx=d["idx"][:, bounds[g]:bounds[g + 1]], C_packed=d["Cp"], alpha=dev(als[g]), mu=dev(mus[g]), v=v, Kc=Kc)
             for g in range(3)]
    terms.append(dict(k0=0, idx=d2["idx"], C_packed=d2["Cp"], alpha=dev(al2), v=v, Kc=300))
    y = btc.linear_gemv_sum(d["x"], terms, N)
    y2 = btc.linear_gemv_sum(d["x"], terms, N)
    torch.cuda.synchronize()
    assert torch.equal(y, y2)
    oterms = [(bounds[g] * v, L.idx[:, bounds[g]:bounds[g + 1]], L.C_pm1, als[g], mus[g]) for g in range(3)]
    oterms.append((0, L2.idx, L2.C_pm1, al2, None))
    ref = oracle.linear_terms(L.x_f64(), N, oterms)
    err = np.abs(y.double().cpu().numpy() - ref)
    assert err.max() / np.abs(ref).max() <= TOL_GEMV
    scale = np.outer(np.abs(L.x_f64()).sum(1), sum(np.abs(a.astype(np.float64)) for a in als) + np.abs(al2.astype(np.float64))
                     + sum(np.abs(m_.astype(np.float64)) for m_ in mus))
    assert (err / scale).max() <= TOL_GEMV
    assert btc.device_status() == 0


# ------------------------------------------------------------------ the paper's two-stage lookup scheme as a kernel

@pytest.mark.parametrize("N,K,v,Kc,M,mu", [(300, 1024, 16, 4096, 1, False), (4096, 4096, 16, 8192, 1, False), (129, 2048, 16, 300, 3, True),
                                           (513, 640, 20, 5000, 2, True), (64, 768, 12, 777, 8, False), (11008, 4096, 16, 8192, 2, False)])
def test_lut_scheme_kernel_matches_oracle(N, K, v, Kc, M, mu):
    """btc_linear_gemv_lut (Stage-I activation tables, Stage-II codebook table in fp16, gather-accumulate) against the
    oracle's dense product, at the decode tolerance; twice, bit for bit (slices are added in a fixed order)."""
    L = wl.make_layer(_spec(N, K, v, Kc, with_mu=mu, outlier_frac=0.01), M, seed=N + K + M)
    d = to_device(L)
    y = btc.linear_gemv_lut(d["x"], d["idx"], d["Cp"], d["alpha"], v, Kc, mu=d["mu"])
    y2 = btc.linear_gemv_lut(d["x"], d["idx"], d["Cp"], d["alpha"], v, Kc, mu=d["mu"])
    torch.cuda.synchronize()
    rel, fwd = errors(y, oracle_y(L), L)
    assert rel <= TOL_GEMV and fwd <= TOL_GEMV, (rel, fwd)
    assert torch.equal(y, y2)

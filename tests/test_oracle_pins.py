"""Pins for the CPU oracle: things the paper and the mathematics fix, none of which
is the oracle's own formula retyped.  Each test names the mistake it would catch."""
import itertools
import math
import os

import numpy as np
import pytest

import oracle
import workloads as wl

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _read_fixture(name):
    rows = {}
    with open(os.path.join(GOLDEN, name)) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            key, *vals = line.split()
            rows.setdefault(key, []).append([float(t) for t in vals])
    return rows


def _tiny(seed, N=5, K=24, v=6, Kc=7, M=2, with_mu=True, dist="uniform"):
    spec = wl.LayerSpec("tiny", N, K, v, Kc, idx_dist=dist, with_mu=with_mu)
    return wl.make_layer(spec, M, seed)


def _brute(L):
    """Per-element expansion in pure Python: the storage rule and the dot product, no numpy."""
    s = L.spec
    x = L.x_f64()
    mu = None if L.mu is None else L.mu.astype(np.float64)
    y = [[0.0] * s.N for _ in range(L.M)]
    for m in range(L.M):
        for r in range(s.N):
            acc = 0.0
            for j in range(s.Kb):
                cen = L.C_pm1[int(L.idx[r, j])]
                for t in range(s.v):
                    w = float(L.alpha[r]) * (1.0 if cen[t] >= 0 else -1.0)
                    if mu is not None:
                        w += float(mu[r])
                    acc += float(x[m, j * s.v + t]) * w
            y[m][r] = acc
    return np.array(y)


# ---------------------------------------------------------------- hand-expanded fixture

def test_hand_expanded_fixture():
    """Catches: wrong block/row indexing, transposed codebook, dropped alpha or mu, wrong bit order."""
    fx = _read_fixture("tiny_layer.txt")
    C = np.array(fx["C"], dtype=np.int8)
    idx = np.array(fx["idx"], dtype=np.uint16)
    alpha = np.array(fx["alpha"][0])
    mu = np.array(fx["mu"][0])
    x = np.array(fx["x"], dtype=np.float64)
    assert np.array_equal(oracle.decode_pm1(idx, C), np.array(fx["B"], dtype=np.int8))
    assert np.array_equal(oracle.pack_codebook(C), np.array(fx["packed"][0], dtype=np.uint32))
    ones = np.ones(3)
    assert np.array_equal(oracle.linear(x, idx, C, ones)[0], np.array(fx["dots"][0]))
    assert np.array_equal(oracle.linear(x, idx, C, alpha)[0], np.array(fx["y_nomu"][0]))
    assert np.array_equal(oracle.linear(x, idx, C, alpha, mu)[0], np.array(fx["y_mu"][0]))
    for seg in (1, 2, 4):
        assert np.array_equal(oracle.lut_linear(x, idx, C, alpha, mu, seg=seg)[0], np.array(fx["y_mu"][0]))
    W = oracle.dense_weight(idx, C, alpha, mu)
    assert W[1, 2] == 2 * -1 - 0.5 and W[0, 0] == 0.5 + 0.25 and W[2, 7] == 1 + 1


# ---------------------------------------------------------------- brute force on tiny inputs

@pytest.mark.parametrize("seed,N,K,v,Kc,M", [(1, 5, 24, 6, 7, 2), (2, 3, 20, 20, 5, 1),
                                             (3, 7, 32, 16, 40, 3), (4, 4, 36, 9, 3, 2),
                                             (5, 2, 64, 32, 6, 1), (6, 6, 16, 4, 16, 4)])
def test_brute_force(seed, N, K, v, Kc, M):
    """Catches: any indexing slip in decode / dense weight / matmul (non-square, ragged shapes)."""
    L = _tiny(seed, N, K, v, Kc, M)
    y = oracle.linear(L.x_f64(), L.idx, L.C_pm1, L.alpha, L.mu)
    np.testing.assert_allclose(y, _brute(L), rtol=1e-13, atol=1e-15)


def test_dense_weight_through_library_matmul():
    """Third opinion: the oracle's dense W^ fed to numpy's fp64 matmul (catches a transposed operand)."""
    L = _tiny(11, N=9, K=48, v=12, Kc=30, M=5)
    W = oracle.dense_weight(L.idx, L.C_pm1, L.alpha, L.mu)
    y = oracle.linear(L.x_f64(), L.idx, L.C_pm1, L.alpha, L.mu)
    np.testing.assert_allclose(y, L.x_f64() @ W.T, rtol=1e-12, atol=1e-14)
    assert W.shape == (9, 48)


# ---------------------------------------------------------------- the +-1 / bit identities

def test_bit_identity_dot_equals_2_sum_set_minus_sum():
    """<x, c> = 2*sum_{bit=1} x - sum x with bits from the packed word; ties the packing
    convention (bit=1 <=> +1, LSB first) to the decode.  Catches a flipped bit meaning or order."""
    L = _tiny(21, N=6, K=40, v=20, Kc=50, M=1, with_mu=False)
    packed = oracle.pack_codebook(L.C_pm1)
    x = L.x_f64()[0]
    ones = np.ones(L.spec.N)
    y = oracle.linear(L.x_f64(), L.idx, L.C_pm1, ones)[0]
    for r in range(L.spec.N):
        acc = 0.0
        for j in range(L.spec.Kb):
            w = int(packed[L.idx[r, j]])
            xs = x[j * 20:(j + 1) * 20]
            acc += 2.0 * sum(xs[t] for t in range(20) if (w >> t) & 1) - sum(xs)
        assert abs(acc - y[r]) <= 1e-12 * max(1.0, abs(y[r]))


def test_sqdist_is_4_hamming_on_packed_words():
    """||b - c||^2 = 4 * popcount(b xor c)  (Section 4.1, E-step)."""
    C = wl.make_codebook_pm1(64, 13, seed=5)
    packed = oracle.pack_codebook(C)
    for a, b in itertools.combinations(range(0, 64, 7), 2):
        ham = bin(int(packed[a]) ^ int(packed[b])).count("1")
        assert oracle.sqdist_pm1(C[a], C[b]) == 4 * ham
    assert int(packed.max()) < (1 << 13)


def test_pack_roundtrip_all_v():
    """bit t of the packed word <=> element t, for every supported v; zero counts as +1 (sign(0)=+1)."""
    for v in range(1, 33):
        C = wl.make_codebook_pm1(37, v, seed=v, distinct=False)
        packed = oracle.pack_codebook(C)
        t = np.arange(v, dtype=np.uint64)
        bits = (packed.astype(np.uint64)[:, None] >> t[None, :]) & np.uint64(1)
        assert np.array_equal(np.where(bits == 1, 1, -1).astype(np.int8), C)
    Cz = np.array([[0, -1, 5, -7]], dtype=np.int8)
    assert oracle.pack_codebook(Cz)[0] == 0b0101
    assert np.array_equal(oracle.decode_pm1(np.array([[0]], dtype=np.uint16), Cz), [[1, -1, 1, -1]])


def test_ones_probe_counts_minus_bits():
    """alpha = 1 and x = 1  =>  y_n = K - 2 * (number of -1 weights in row n), an integer."""
    L = _tiny(31, N=8, K=64, v=16, Kc=33, M=1, with_mu=False)
    packed = oracle.pack_codebook(L.C_pm1)
    y = oracle.linear(np.ones((1, 64)), L.idx, L.C_pm1, np.ones(8))[0]
    for r in range(8):
        minus = sum(16 - bin(int(packed[k])).count("1") for k in L.idx[r])
        assert y[r] == 64 - 2 * minus


def test_one_hot_probe_reads_back_weight_columns():
    """x = e_k  =>  y[:, n] = W^[n, k] exactly; catches an off-by-one in the block offset j*v + t."""
    L = _tiny(32, N=5, K=30, v=10, Kc=12, M=1)
    W = oracle.dense_weight(L.idx, L.C_pm1, L.alpha, L.mu)
    y = oracle.linear(np.eye(30), L.idx, L.C_pm1, L.alpha, L.mu)   # M = K probes
    assert np.array_equal(y, W.T)
    B = oracle.decode_pm1(L.idx, L.C_pm1)
    a = L.alpha.astype(np.float64)[:, None]
    assert np.array_equal(W, a * B + L.mu.astype(np.float64)[:, None])


# ---------------------------------------------------------------- the paper's LUT formulation

@pytest.mark.parametrize("v,seg", [(16, 4), (16, 8), (20, 4), (20, 10), (12, 6), (8, 8)])
def test_lut_formulation_agrees_with_dense(v, seg):
    """The two-stage lookup scheme (a different algorithm from the appendix) reaches the same number."""
    L = _tiny(40 + v + seg, N=11, K=v * 5, v=v, Kc=23, M=3)
    y = oracle.linear(L.x_f64(), L.idx, L.C_pm1, L.alpha, L.mu)
    z = oracle.lut_linear(L.x_f64(), L.idx, L.C_pm1, L.alpha, L.mu, seg=seg)
    scale = np.abs(y).max()
    assert np.abs(y - z).max() <= 1e-12 * scale
    np.testing.assert_allclose(z, _brute(L), rtol=1e-11, atol=1e-13)


# ---------------------------------------------------------------- special cases = textbook routines

def test_identity_codebook_is_plain_sign_gemm():
    """Kc = 2^v with C[k] = bit pattern of k is the 1-bit (W1A16) layer: a plain sign-matrix product.
    The sign matrix is drawn independently and the indices are derived from it."""
    v, N, K, M = 8, 12, 40, 3
    rng = np.random.default_rng(7)
    S = rng.choice(np.array([-1, 1], dtype=np.int8), size=(N, K))
    C = np.array([[1 if (k >> t) & 1 else -1 for t in range(v)] for k in range(1 << v)], dtype=np.int8)
    bits = (S.reshape(N, K // v, v) > 0).astype(np.int64)
    idx = (bits << np.arange(v)).sum(-1).astype(np.uint16)
    x = rng.standard_normal((M, K))
    y = oracle.linear(x, idx, C, np.ones(N))
    np.testing.assert_allclose(y, x @ S.T.astype(np.float64), rtol=1e-13, atol=1e-13)
    assert np.array_equal(oracle.decode_pm1(idx, C), S)


def test_all_plus_codebook_and_single_centroid():
    """All-(+1) codebook => y_n = alpha_n * sum(x); Kc = 1 likewise with its only centroid."""
    N, K, v = 6, 24, 8
    rng = np.random.default_rng(3)
    x = rng.standard_normal((2, K))
    alpha = rng.random(N) + 0.1
    idx = rng.integers(0, 4, size=(N, K // v)).astype(np.uint16)
    y = oracle.linear(x, idx, np.ones((4, v), dtype=np.int8), alpha)
    np.testing.assert_allclose(y, np.outer(x.sum(1), alpha), rtol=1e-13)
    c = np.array([[1, -1, -1, 1, 1, 1, -1, 1]], dtype=np.int8)
    y1 = oracle.linear(x, np.zeros((N, K // v), dtype=np.uint16), c, alpha)
    base = (x.reshape(2, K // v, v) * c[0]).sum((1, 2))
    np.testing.assert_allclose(y1, np.outer(base, alpha), rtol=1e-13)


# ---------------------------------------------------------------- invariants

def test_invariants():
    L = _tiny(51, N=10, K=60, v=12, Kc=19, M=2, with_mu=False)
    x = L.x_f64()
    y = oracle.linear(x, L.idx, L.C_pm1, L.alpha)
    a64 = L.alpha.astype(np.float64)
    # linearity in x
    x2 = np.random.default_rng(0).standard_normal(x.shape)
    y2 = oracle.linear(x2, L.idx, L.C_pm1, L.alpha)
    np.testing.assert_allclose(oracle.linear(2.0 * x - 3.0 * x2, L.idx, L.C_pm1, L.alpha), 2 * y - 3 * y2,
                               rtol=1e-12, atol=1e-12)
    # permuting the codebook rows with idx remapped leaves y unchanged
    perm = np.random.default_rng(1).permutation(19)          # new position p holds old centroid perm[p]
    inv = np.argsort(perm)
    assert np.array_equal(oracle.linear(x, inv[L.idx].astype(np.uint16), L.C_pm1[perm], L.alpha), y)
    # negating all centroids and all alpha leaves y unchanged
    np.testing.assert_allclose(oracle.linear(x, L.idx, -L.C_pm1, -a64), y, rtol=1e-14)
    # permuting output rows permutes y
    rp = np.random.default_rng(2).permutation(10)
    assert np.array_equal(oracle.linear(x, L.idx[rp], L.C_pm1, L.alpha[rp]), y[:, rp])
    # splitting K into two calls and summing
    h = 3  # blocks in the first part
    ya = oracle.linear(x[:, :h * 12], L.idx[:, :h], L.C_pm1, L.alpha)
    yb = oracle.linear(x[:, h * 12:], L.idx[:, h:], L.C_pm1, L.alpha)
    np.testing.assert_allclose(ya + yb, y, rtol=1e-12, atol=1e-13)


def test_bad_inputs_are_errors():
    C = np.ones((4, 4), dtype=np.int8)
    with pytest.raises(ValueError):
        oracle.linear(np.ones((1, 8)), np.array([[0, 4]], dtype=np.uint16), C, np.ones(1))   # idx >= Kc
    with pytest.raises(ValueError):
        oracle.lut_linear(np.ones((1, 8)), np.array([[0, 1]], dtype=np.uint16), C, np.ones(1), seg=3)


# ---------------------------------------------------------------- accounting closed forms

def test_bits_per_weight_closed_forms():
    assert oracle.bits_per_weight(4096, 4096, 16, 4096) == 0.75
    assert oracle.bits_per_weight(4096, 4096, 16, 8192) == 0.8125
    assert oracle.bits_per_weight(5120, 5120, 20, 65536) == 0.8
    assert oracle.bits_per_weight(4096, 4096, 16, 8192, mode="stored") == 1.0
    assert oracle.bits_per_weight(4096, 4096, 16, 7132, mode="container") == 13 / 16
    assert abs(oracle.bits_per_weight(4096, 4096, 16, 7132, mode="nominal") - math.log2(7132) / 16) < 1e-15
    # (log2 Kc + scale bits per row amortised over the row) / v, written per weight
    got = oracle.bits_per_weight(4096, 11008, 16, 8192, scale_bits_per_row=16)
    assert abs(got - (13 / 16 + 16 / 11008)) < 1e-15
    # codebook term and the Section 4.3 storage formula  v*c + ceil(log2 c) * m*n / v
    assert oracle.storage_bits(4096, 4096, 16, 7132) == 16 * 7132 + 13 * 4096 * 4096 / 16
    full = oracle.bits_per_weight(4096, 4096, 16, 7132, with_codebook=True)
    assert abs(full - oracle.storage_bits(4096, 4096, 16, 7132) / 4096 ** 2) < 1e-15
    # compression ratio 16 v / ceil(log2 c)
    assert 16 / oracle.bits_per_weight(1, 16, 16, 7132) == 16 * 16 / 13


def test_paper_tables():
    fx = _read_fixture("paper_tables.txt")
    for v, c in fx["vc"]:
        assert abs(oracle.bits_per_weight(1, int(v), int(v), int(c), mode="nominal") - 0.8) < 0.011
        assert abs(c - 2 ** (0.8 * v)) < 1.0
    for c, mb in fx["cbmem"]:
        elems = 224 * (oracle.storage_bits(0, 16, 16, int(c)))      # v*c elements per layer, 224 layers
        assert abs(elems / 1e6 - mb) < 0.02                          # one byte per element
    # 2:4 sparsity: 2 sign bits + ceil(log2 6) mask bits over 4 weights
    assert oracle.bits_per_weight(1, 4, 4, 6, mode="container") + 2 / 4 == fx["sparse24"][0][0]


# ---------------------------------------------------------------- transform (identities only)

def test_transform_identities():
    rng = np.random.default_rng(9)
    k1, k2, M = 3, 4, 2
    K = k1 * k2
    x = rng.standard_normal((M, K))
    sig = rng.choice(np.array([-1, 1], dtype=np.int8), size=K)
    P1 = rng.standard_normal((k1, k1)) + 3 * np.eye(k1)
    P2 = rng.standard_normal((k2, k2)) + 3 * np.eye(k2)
    # T = I
    assert np.array_equal(oracle.transform(x, np.ones(K, dtype=np.int8), np.eye(k1), np.eye(k2)), x)
    # dense Kronecker (library) and the two-small-matmul form agree with the oracle
    T = np.diag(sig.astype(np.float64)) @ np.kron(P1, P2)
    xt = oracle.transform(x, sig, P1, P2)
    np.testing.assert_allclose(xt, x @ T, rtol=1e-12, atol=1e-13)
    two = np.stack([(P1.T @ (x[m] * sig).reshape(k1, k2) @ P2).reshape(-1) for m in range(M)])
    np.testing.assert_allclose(xt, two, rtol=1e-12, atol=1e-13)
    # (x T)(T^-1 W^T) = x W^T  (Eq. 4)
    W = rng.standard_normal((5, K))
    np.testing.assert_allclose(xt @ (np.linalg.inv(T) @ W.T), x @ W.T, rtol=1e-10, atol=1e-10)


# ---------------------------------------------------------------- planted mistakes must be caught

def test_pins_catch_planted_mistakes():
    """Mutants of the definition (made here, on the CPU) each disagree with the oracle on the same
    inputs the pins use, i.e. the pins above would fail if the oracle had that mistake."""
    L = _tiny(61, N=6, K=36, v=12, Kc=9, M=2)
    s = L.spec
    x = L.x_f64()
    y = oracle.linear(x, L.idx, L.C_pm1, L.alpha, L.mu)
    a = L.alpha.astype(np.float64)
    mu = L.mu.astype(np.float64)
    B = L.C_pm1[L.idx.astype(np.int64)].reshape(s.N, s.K).astype(np.float64)
    good = x @ (a[:, None] * B + mu[:, None]).T
    np.testing.assert_allclose(y, good, rtol=1e-12, atol=1e-13)
    mutants = {
        "dropped mu": x @ (a[:, None] * B).T,
        "flipped sign": x @ (-a[:, None] * B + mu[:, None]).T,
        "reversed bit order": x @ (a[:, None] * B.reshape(s.N, s.Kb, s.v)[:, :, ::-1].reshape(s.N, s.K) + mu[:, None]).T,
        "blocks transposed": x @ (a[:, None] * L.C_pm1[L.idx.T.reshape(s.N, s.Kb).astype(np.int64)].reshape(s.N, s.K) + mu[:, None]).T,
        "alpha per column": x @ (np.resize(a, s.K)[None, :] * B + mu[:, None]).T,
    }
    for name, bad in mutants.items():
        assert np.abs(bad - y).max() > 1e-3 * np.abs(y).max(), name


# ------------------------------------------------------------------ codebook construction (Section 4.1)

def _read_kmeans_fixture():
    vals = {"vec": [], "init": [], "C1": [], "C2": []}
    with open(os.path.join(GOLDEN, "kmeans_tiny.txt")) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            key, *rest = line.split()
            nums = [int(t) for t in rest]
            if key in vals:
                vals[key].append(nums)
            else:
                vals[key] = nums
    return vals


def test_kmeans_hand_worked_example():
    from oracle import codebook_kmeans as km
    g = _read_kmeans_fixture()
    B = np.array(g["vec"], dtype=np.int8)
    c = g["c"][0]
    C0, n_unique = km.initial_codebook(B, c)
    assert n_unique == 5 and np.array_equal(C0, np.array(g["init"], dtype=np.int8))
    z1 = km.e_step(B, C0)
    assert z1.tolist() == g["z1"]
    C1 = km.m_step(B, z1, C0)
    assert np.array_equal(C1, np.array(g["C1"], dtype=np.int8))
    z2 = km.e_step(B, C1)
    assert z2.tolist() == g["z2"]
    C2 = km.m_step(B, z2, C1)
    assert np.array_equal(C2, np.array(g["C2"], dtype=np.int8))
    C, z, iters, _ = km.optimize_codebook(B, c, max_iter=10)
    assert iters == g["iterations"][0] and z.tolist() == g["z3"] and np.array_equal(C, C2)
    assert km.total_hamming(B, C, z) == g["total_hamming"][0]
    # stopping early by max_iter: one E-step and one M-step
    C_a, z_a, it_a, _ = km.optimize_codebook(B, c, max_iter=1)
    assert it_a == 1 and z_a.tolist() == g["z1"] and np.array_equal(C_a, C1)


def test_kmeans_majority_vote_ties_and_empty_clusters():
    from oracle import codebook_kmeans as km
    B = np.array([[1, -1], [-1, 1]], dtype=np.int8)
    C = km.m_step(B, np.array([0, 0]), np.array([[-1, -1], [1, -1]], dtype=np.int8))
    assert C.tolist() == [[1, 1], [1, -1]]          # element means 0 -> +1; the empty cluster keeps its centroid


def test_kmeans_single_centroid_is_the_bitwise_majority():
    """c = 1 after one M-step: the centroid is the element-wise majority of all vectors (closed form)."""
    from oracle import codebook_kmeans as km
    rng = np.random.default_rng(5)
    B = np.where(rng.random((501, 12)) < 0.4, 1, -1).astype(np.int8)
    C, z, iters, _ = km.optimize_codebook(B, 1, max_iter=5)
    assert np.array_equal(C[0], np.where(B.astype(np.int64).sum(axis=0) >= 0, 1, -1))
    assert not z.any() and iters == 2


def test_kmeans_e_step_equals_hamming_argmin_on_packed_words():
    """||b - c||^2 = 4 d_H(b, c) (Section 4.1): the E-step's Euclidean argmin equals the argmin of
    POPCNT(b xor c) on packed words, first index among equals."""
    from oracle import codebook_kmeans as km
    rng = np.random.default_rng(6)
    v = 11
    B = np.where(rng.random((300, v)) < 0.5, 1, -1).astype(np.int8)
    C = np.where(rng.random((17, v)) < 0.5, 1, -1).astype(np.int8)
    z = km.e_step(B, C)
    bw, cw = km.pack_words(B), km.pack_words(C)
    for i in range(B.shape[0]):
        d = [bin(int(bw[i]) ^ int(cw[k])).count("1") for k in range(C.shape[0])]
        assert z[i] == d.index(min(d))
        assert ((B[i].astype(int) - C[z[i]].astype(int)) ** 2).sum() == 4 * min(d)


def test_kmeans_e_step_per_distinct_vector_equals_the_per_vector_definition():
    """e_step evaluates every distinct vector once; the definition (Section 4.1 (2)) visits every vector.  Inputs with
    many repeated vectors, ties between centroids and duplicated centroids: the two must agree everywhere."""
    from oracle import codebook_kmeans as km
    rng = np.random.default_rng(16)
    for v, n, c in ((6, 500, 9), (12, 800, 40), (3, 200, 8)):
        proto = np.where(rng.random((30, v)) < 0.5, 1, -1).astype(np.int8)
        B = proto[rng.integers(0, 30, n)]
        C = np.where(rng.random((c, v)) < 0.5, 1, -1).astype(np.int8)
        C[c - 1] = C[0]                              # a duplicated centroid: the smaller index must win
        assert np.array_equal(km.e_step(B, C), km.e_step_per_vector(B, C))


def test_kmeans_objective_never_increases_and_few_distinct_vectors_are_kept_exactly():
    from oracle import codebook_kmeans as km
    rng = np.random.default_rng(7)
    v, c = 10, 24
    proto = np.where(rng.random((40, v)) < 0.5, 1, -1).astype(np.int8)
    B = proto[rng.integers(0, 40, 4000)]
    flip = rng.random(B.shape) < 0.03
    B = np.where(flip, -B, B).astype(np.int8)
    C = km.initial_codebook(B, c)[0]
    prev = None
    for _ in range(6):
        z = km.e_step(B, C)
        obj = km.total_hamming(B, C, z)
        assert prev is None or obj <= prev          # the E-step cannot increase it ...
        C = km.m_step(B, z, C)
        obj2 = km.total_hamming(B, C, z)
        assert obj2 <= obj                          # ... nor can the majority vote
        prev = obj2
    # at most c distinct vectors: the codebook is the set of distinct vectors and the loss is zero
    few = proto[:c][rng.integers(0, c, 1000)]
    C2, z2, iters, n_unique = km.optimize_codebook(few, c + 5, max_iter=10)
    assert C2.shape[0] == n_unique <= c and km.total_hamming(few, C2, z2) == 0
    assert len({tuple(r) for r in C2.tolist()}) == n_unique


# ------------------------------------------------------------------ dense index packing (Section 4.3)

def test_index_packing_hand_written_12_bit_example():
    """Two 12-bit indices 0xABC, 0x123 -> bit string LSB first: bytes BC, 3A (low nibble A of the first index's top
    bits, high nibble 3 of the second index's low bits), 12.  Worked by hand."""
    idx = np.array([[0xABC, 0x123]], dtype=np.uint16)
    packed = oracle.pack_indices(idx, 12, pitch=4)
    assert packed.tolist() == [[0xBC, 0x3A, 0x12, 0x00]]
    assert oracle.unpack_indices(packed, 2, 12).tolist() == [[0xABC, 0x123]]
    # 13 bits: 0x1ABC, 0x0123 -> bits 0..12 = 0x1ABC, bits 13..25 = 0x0123: the 26-bit number 0x0123 << 13 | 0x1ABC
    word = (0x0123 << 13) | 0x1ABC
    packed13 = oracle.pack_indices(np.array([[0x1ABC, 0x0123]], dtype=np.uint16), 13, pitch=4)
    assert packed13.tolist() == [[word & 0xFF, (word >> 8) & 0xFF, (word >> 16) & 0xFF, (word >> 24) & 0xFF]]


@pytest.mark.parametrize("bits", [1, 5, 8, 12, 13, 15, 16])
def test_index_packing_against_numpy_bit_strings_and_round_trip(bits):
    """Independent construction: numpy unpackbits / packbits with little-endian bit order over the concatenated fields."""
    rng = np.random.default_rng(bits)
    N, Kb = 7, 37
    idx = rng.integers(0, 1 << bits, size=(N, Kb), dtype=np.uint32).astype(np.uint16)
    packed = oracle.pack_indices(idx, bits)
    fields = ((idx[:, :, None].astype(np.uint32) >> np.arange(bits, dtype=np.uint32)) & 1).astype(np.uint8)   # [N, Kb, bits]
    want = np.packbits(fields.reshape(N, Kb * bits), axis=1, bitorder="little")
    nbytes = (Kb * bits + 7) // 8
    assert packed.shape[1] == oracle.packed_row_bytes(Kb, bits) and packed.shape[1] % 16 == 0
    assert np.array_equal(packed[:, :nbytes], want) and not packed[:, nbytes:].any()
    assert np.array_equal(oracle.unpack_indices(packed, Kb, bits), idx)


def test_index_packing_size_is_the_papers_storage_count():
    """Section 4.3: the indices of an m x n layer take ceil(log2 c) * mn / v bits.  A packed 4096 x 4096 layer at v = 16
    holds exactly that many bits (the row length is a multiple of 16 bytes here, so there is no padding), and the
    index width follows the codebook sizes of Table 3a."""
    for Kc, bits in ((4096, 12), (8192, 13), (7132, 13), (21619, 15), (65536, 16), (256, 8), (2, 1), (1, 1)):
        assert oracle.index_bits(Kc) == bits
    N = K = 4096
    v = 16
    for Kc in (4096, 8192):
        b = oracle.index_bits(Kc)
        assert oracle.packed_row_bytes(K // v, b) * N * 8 == oracle.storage_bits(N, K, v, Kc) - v * Kc
    # rejects an index that does not fit the width, and a pitch shorter than the bit string
    with pytest.raises(ValueError):
        oracle.pack_indices(np.array([[4096]], dtype=np.uint16), 12)
    with pytest.raises(ValueError):
        oracle.pack_indices(np.zeros((1, 9), dtype=np.uint16), 12, pitch=13)


# ------------------------------------------------------------------ several scale groups per row / residual terms

def test_linear_terms_reduces_to_linear_and_adds_up():
    """One term over all columns IS the plain layer; column groups with their own (alpha, mu) equal the sum of the plain
    layer on each column slice; two terms over the same columns (residual binarisation) equal the sum of two layers;
    and a brute-force element-by-element evaluation agrees."""
    rng = np.random.default_rng(11)
    N, K, v, Kc, M = 9, 96, 8, 21, 3
    x = rng.standard_normal((M, K))
    C = rng.choice(np.array([-1, 1], dtype=np.int8), size=(Kc, v))
    idx = rng.integers(0, Kc, size=(N, K // v)).astype(np.uint16)
    al = np.abs(rng.standard_normal(N)) * 0.02
    mu = rng.standard_normal(N) * 0.002
    one = oracle.linear_terms(x, N, [(0, idx, C, al, mu)])
    assert np.allclose(one, oracle.linear(x, idx, C, al, mu), rtol=1e-13, atol=1e-15)
    # three column groups (bounds in blocks), each with its own scales
    bounds = [0, 4, 9, 12]
    als = [np.abs(rng.standard_normal(N)) * 0.02 for _ in range(3)]
    mus = [rng.standard_normal(N) * 0.002 for _ in range(3)]
    terms = [(bounds[g] * v, idx[:, bounds[g]:bounds[g + 1]], C, als[g], mus[g]) for g in range(3)]
    y = oracle.linear_terms(x, N, terms)
    want = sum(oracle.linear(x[:, bounds[g] * v:bounds[g + 1] * v], idx[:, bounds[g]:bounds[g + 1]], C, als[g], mus[g]) for g in range(3))
    assert np.allclose(y, want, rtol=1e-12, atol=1e-14)
    # brute force, element by element
    brute = np.zeros((M, N))
    for m in range(M):
        for n in range(N):
            for k in range(K):
                g = next(i for i in range(3) if bounds[i] * v <= k < bounds[i + 1] * v)
                brute[m, n] += x[m, k] * (als[g][n] * C[idx[n, k // v], k % v] + mus[g][n])
    assert np.allclose(y, brute, rtol=1e-12, atol=1e-14)
    # residual: a second binary term over the first group's columns, with its own codebook and indices
    C2 = rng.choice(np.array([-1, 1], dtype=np.int8), size=(5, v))
    idx2 = rng.integers(0, 5, size=(N, 4)).astype(np.uint16)
    al2 = np.abs(rng.standard_normal(N)) * 0.005
    yr = oracle.linear_terms(x, N, terms + [(0, idx2, C2, al2, None)])
    assert np.allclose(yr, y + oracle.linear(x[:, :4 * v], idx2, C2, al2), rtol=1e-12, atol=1e-14)
    with pytest.raises(ValueError):
        oracle.linear_terms(x, N, [(K - 8, idx, C, al, mu)])

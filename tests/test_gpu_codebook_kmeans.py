"""GPU parity of btc_codebook_kmeans against the numpy oracle (bit-exact: integer work)."""
import os
import sys

import numpy as np
import pytest
import torch

sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.abspath(__file__))))

pytestmark = pytest.mark.gpu

import paper_2506_12040_b200 as btc  # noqa: E402
from oracle import codebook_kmeans as km  # noqa: E402


def _vectors(n, v, kind, seed):
    """Seeded +-1 vectors: 'noisy' = a few prototypes with flipped elements (what binarised weight blocks of a
    trained layer look like: a skewed pattern distribution), 'iid' = independent fair signs, 'few' = at most a
    handful of distinct vectors."""
    rng = np.random.default_rng(seed)
    if kind == "iid":
        return np.where(rng.random((n, v)) < 0.5, 1, -1).astype(np.int8)
    protos = np.where(rng.random((7 if kind == "few" else 60, v)) < 0.5, 1, -1).astype(np.int8)
    B = protos[rng.integers(0, protos.shape[0], n)]
    if kind == "noisy":
        B = np.where(rng.random(B.shape) < 0.08, -B, B).astype(np.int8)
    return B


def _run(B, v, Kc, max_iter):
    words = torch.from_numpy(km.pack_words(B).view(np.int32).copy()).cuda()
    C, z, info = btc.codebook_kmeans(words, v, Kc, max_iter)
    torch.cuda.synchronize()
    return C.cpu().numpy().view(np.uint32), z.cpu().numpy().view(np.uint16), info.cpu().numpy()


CASES = [
    # n, v, Kc, max_iter, kind
    (8, 4, 2, 10, "fixture"),
    (5000, 8, 16, 30, "noisy"),
    (20000, 12, 256, 25, "noisy"),
    (30000, 10, 100, 3, "iid"),          # stops by max_iter
    (4000, 16, 300, 12, "noisy"),
    (3000, 16, 64, 40, "iid"),           # nearly all vectors distinct
    (2000, 9, 50, 10, "few"),            # fewer distinct vectors than centroids
    (1, 5, 3, 4, "iid"),
    (70000, 13, 5000, 6, "noisy"),       # ragged: many tiles of centroids and patterns
    (30000, 20, 700, 8, "noisy"),        # the longest vectors of the paper's range
    (9000, 18, 3000, 5, "iid"),
    (100, 1, 2, 3, "iid"),               # one element per vector: two patterns
    (1000, 6, 1, 5, "noisy"),            # a single centroid: the bitwise majority
    (500, 16, 65536, 3, "iid"),          # the largest codebook, far more slots than vectors
]


@pytest.mark.parametrize("n,v,Kc,max_iter,kind", CASES)
def test_kmeans_matches_oracle_bit_for_bit(n, v, Kc, max_iter, kind):
    if kind == "fixture":
        B = np.array([[1, 1, 1, 1]] * 3 + [[-1, 1, 1, 1]] * 2 + [[-1, -1, -1, 1], [-1, -1, -1, -1], [-1, -1, 1, -1]], dtype=np.int8)
    else:
        B = _vectors(n, v, kind, seed=n + v + Kc)
    C_ref, z_ref, iters_ref, n_unique, converged = km.optimize_codebook(B, Kc, max_iter, with_flag=True)
    C, z, info = _run(B, v, Kc, max_iter)
    k_eff = min(Kc, n_unique)
    assert info[0] == iters_ref and info[1] == k_eff and info[2] == n_unique
    assert np.array_equal(C[:k_eff], km.pack_words(C_ref)) and not C[k_eff:].any()
    assert np.array_equal(z.astype(np.int64), z_ref)
    assert info[3] == int(converged)


def test_kmeans_feeds_the_layer():
    """The construction's outputs are the layer's inputs: centroids -> btc_codebook_pack, z -> idx; decoding them
    gives the nearest-centroid approximation of the sign matrix, whose Hamming error equals the oracle's objective."""
    N, K, v, Kc = 64, 256, 16, 128
    B = _vectors(N * K // v, v, "noisy", seed=3)                        # blocks of a 64 x 256 sign matrix, row-major
    C, z, info = _run(B, v, Kc, 15)
    C_ref, z_ref, _, _ = km.optimize_codebook(B, Kc, 15)
    C_pm1 = km.unpack_words(C[:info[1]], v)
    Cp = btc.codebook_pack(torch.from_numpy(np.ascontiguousarray(C_pm1)).cuda())
    idx = torch.from_numpy(z.view(np.int16).reshape(N, K // v).copy()).cuda()
    Bhat = btc.decode_pm1(idx, Cp, v, int(info[1])).cpu().numpy()
    assert (Bhat.reshape(-1, v) != B).sum() == km.total_hamming(B, C_ref, z_ref)


def test_kmeans_argument_errors():
    w = torch.zeros(16, dtype=torch.int32, device="cuda")
    with pytest.raises(btc.BtcError):
        btc.codebook_kmeans(w, 24, 16, 5)            # v > 20: unsupported
    with pytest.raises(btc.BtcError):
        btc.codebook_kmeans(w, 8, 0, 5)
    with pytest.raises(btc.BtcError):
        btc.codebook_kmeans(w, 8, 4, 0)
    with pytest.raises(btc.BtcError):
        btc.codebook_kmeans(w, 8, 4, 5, workspace=torch.empty(256, dtype=torch.uint8, device="cuda"))

"""CPU oracle for binary codebook construction (Section 4.1 "Flash and Accurate Binary Codebook";
appendix Algorithm "Binary Codebook Optimization").

TEST INFRASTRUCTURE ONLY: imported by tests/ (and nothing else).  It shares nothing with the CUDA
package and the CUDA package never imports it.  Plain numpy on +-1 vectors; slow on purpose.

Input: vectors b_i in {+-1}^v as an int8 array [n, v].  Steps, in the paper's order:

  Initialisation (Section 4.1 (1)): the distinct vectors U with their frequencies.  If there are
      at most c of them the codebook is U itself and every vector maps to its own copy.  Otherwise
      the c most frequent distinct vectors are the initial centroids.
  E-step (Section 4.1 (2), Eq. "||b - c||^2 = 4 d_H(b, c)"): z_i = argmin_k ||b_i - c_k||^2, evaluated
      here literally as a squared Euclidean distance on the +-1 values.  A vector identical to a
      centroid has distance 0, so the paper's "first test for identity" is the same rule.
  M-step (Section 4.1 (3)): c_k = sign(mean of the vectors assigned to k), sign(0) = +1; a cluster
      without vectors keeps its centroid (appendix algorithm: the update runs only "if |B_k| > 0").
  Loop (appendix algorithm): E-step; stop if no assignment changed; M-step; at most max_iter times.
      The returned z is the one of the last E-step that ran and C the one of the last M-step that
      ran (after max_iter iterations the two are one M-step apart, as in the printed algorithm).

Readings where the paper leaves a choice (both sides of a parity test must take the same one):
  * order among equally frequent vectors at initialisation, and the order of U when |U| <= c:
    frequency descending, then the packed word (bit t = (b_t + 1) / 2, LSB first) ascending;
  * nearest centroid among several at the same distance: the smallest index k;
  * the appendix samples the initial centroids at random from U; the main text takes the most
    frequent ones.  The main text is followed (it is deterministic).
"""
from __future__ import annotations

import numpy as np


def pack_words(B_pm1: np.ndarray) -> np.ndarray:
    """[n, v] of +-1 -> uint32 [n], bit t = (b_t + 1) / 2 (values >= 0 count as +1)."""
    B = np.asarray(B_pm1)
    n, v = B.shape
    w = np.zeros(n, dtype=np.uint64)
    for t in range(v):
        w |= (B[:, t] >= 0).astype(np.uint64) << np.uint64(t)
    return w.astype(np.uint32)


def unpack_words(words: np.ndarray, v: int) -> np.ndarray:
    w = np.asarray(words, dtype=np.uint64)
    out = np.empty((w.size, v), dtype=np.int8)
    for t in range(v):
        out[:, t] = np.where((w >> np.uint64(t)) & np.uint64(1), 1, -1)
    return out


def initial_codebook(B_pm1: np.ndarray, c: int):
    """Distinct vectors ordered by (frequency descending, packed word ascending); the first min(c, |U|)."""
    words = pack_words(B_pm1)
    uniq, counts = np.unique(words, return_counts=True)
    order = np.lexsort((uniq, -counts))                 # last key is the primary one
    uniq = uniq[order]
    k = min(c, uniq.size)
    return unpack_words(uniq[:k], B_pm1.shape[1]), uniq.size


def e_step(B_pm1: np.ndarray, C_pm1: np.ndarray) -> np.ndarray:
    """z_i = argmin_k sum_t (b_it - c_kt)^2, smallest k among equals.  Distinct vectors are evaluated once."""
    words = pack_words(B_pm1)
    uniq, inverse = np.unique(words, return_inverse=True)
    U = unpack_words(uniq, B_pm1.shape[1]).astype(np.int32)
    C = np.asarray(C_pm1, dtype=np.int32)
    z_u = np.empty(uniq.size, dtype=np.int64)
    step = max(1, (1 << 22) // max(1, C.shape[0]))
    for s in range(0, uniq.size, step):
        d = ((U[s:s + step, None, :] - C[None, :, :]) ** 2).sum(axis=2)     # squared Euclidean distances
        z_u[s:s + step] = np.argmin(d, axis=1)                              # first minimum = smallest k
    return z_u[inverse]


def e_step_per_vector(B_pm1: np.ndarray, C_pm1: np.ndarray) -> np.ndarray:
    """The E-step exactly as Section 4.1 (2) words it, one vector at a time and every vector on its own:
    z_i = argmin_k ||b_i - c_k||^2, smallest k among equals.  Slow; e_step above must agree with it on every input
    (identical vectors have identical distances, which is all that e_step's evaluation per distinct vector uses)."""
    B = np.asarray(B_pm1, dtype=np.int64)
    C = np.asarray(C_pm1, dtype=np.int64)
    z = np.empty(B.shape[0], dtype=np.int64)
    for i in range(B.shape[0]):
        best, best_d = 0, None
        for k in range(C.shape[0]):
            d = int(((B[i] - C[k]) ** 2).sum())
            if best_d is None or d < best_d:
                best, best_d = k, d
        z[i] = best
    return z


def m_step(B_pm1: np.ndarray, z: np.ndarray, C_pm1: np.ndarray) -> np.ndarray:
    C = np.array(C_pm1, dtype=np.int8, copy=True)
    B = np.asarray(B_pm1, dtype=np.int64)
    for k in range(C.shape[0]):
        members = B[z == k]
        if members.shape[0] > 0:
            mean = members.sum(axis=0) / members.shape[0]
            C[k] = np.where(mean >= 0, 1, -1)                               # sign, with sign(0) = +1
    return C


def optimize_codebook(B_pm1: np.ndarray, c: int, max_iter: int, with_flag: bool = False):
    """Returns (C int8 [c_eff, v], z int64 [n], E-steps run, number of distinct vectors) and, with_flag, whether
    the loop ended because an E-step changed no assignment."""
    B = np.asarray(B_pm1, dtype=np.int8)
    C, n_unique = initial_codebook(B, c)
    z = None
    iters = 0
    converged = False
    for _ in range(max_iter):
        z_new = e_step(B, C)
        iters += 1
        if z is not None and np.array_equal(z_new, z):
            converged = True
            break
        z = z_new
        C = m_step(B, z, C)
    if z is None:
        z = e_step(B, C)
    return (C, z, iters, n_unique, converged) if with_flag else (C, z, iters, n_unique)


def total_hamming(B_pm1: np.ndarray, C_pm1: np.ndarray, z: np.ndarray) -> int:
    """sum_i d_H(b_i, c_{z_i}) (the objective both steps do not increase)."""
    return int((np.asarray(B_pm1) != np.asarray(C_pm1)[z]).sum())

"""Counter-based seeded generators for codebook-binary linear layers.

Every array is a pure function of (seed, stream, position): element i of a
stream is mix(mix(seed, stream) + (i+1)*GOLDEN) with the splitmix64 finaliser,
so any slice can be regenerated without generating what precedes it.

Recipe (shapes follow LLaMA-2-7B / 13B projections; codebook sizes follow the
paper's Table 3a, e.g. v16 with a few thousand centroids, v20 with 65536):

* codebook: Kc *distinct* v-bit sign patterns, the first Kc entries of a
  seeded permutation of all 2^v patterns, emitted as int8 +1/-1 [Kc, v];
* indices:  uint16 [N, K/v]; "uniform" over [0, Kc) or "zipf": centroid rank r
  (1-based) drawn with probability proportional to r^-1.1 by inverse CDF, so
  centroid 0 is the most frequent (the paper initialises its codebook with
  the most frequent patterns first);
* alpha:    |N(0, 0.02^2)| rounded to nearest-even fp16, subnormals kept;
* x:        N(0, 1) rounded to fp16 or bf16 bits; optionally ceil(frac*K)
  seeded channels are multiplied by 20 first (activation outliers), the same
  channels for every row of x.

Seeds: base = 42 + 1000*config (42 is the seed the paper's experiments use),
each layer/tensor adds its own stream id.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field, replace
from typing import Dict, List, Optional

import numpy as np

_GOLDEN = np.uint64(0x9E3779B97F4A7C15)
_M1 = np.uint64(0xBF58476D1CE4E5B9)
_M2 = np.uint64(0x94D049BB133111EB)


def _mix(z: np.ndarray) -> np.ndarray:
    z = np.asarray(z, dtype=np.uint64)
    with np.errstate(over="ignore"):
        z = (z ^ (z >> np.uint64(30))) * _M1
        z = (z ^ (z >> np.uint64(27))) * _M2
    return z ^ (z >> np.uint64(31))


def stream_seed(seed: int, stream: int) -> np.uint64:
    """Key of one stream: two rounds of the finaliser over (seed, stream)."""
    with np.errstate(over="ignore"):
        a = _mix(np.uint64(seed & 0xFFFFFFFFFFFFFFFF) + _GOLDEN)
        b = _mix(a ^ (np.uint64(stream & 0xFFFFFFFFFFFFFFFF) * _GOLDEN + _GOLDEN))
    return np.uint64(b)


def _u64(seed: int, stream: int, n: int, offset: int = 0) -> np.ndarray:
    key = stream_seed(seed, stream)
    ctr = np.arange(offset + 1, offset + n + 1, dtype=np.uint64)
    with np.errstate(over="ignore"):
        return _mix(key + ctr * _GOLDEN)


def _uniform01(seed: int, stream: int, n: int, offset: int = 0) -> np.ndarray:
    """fp64 uniforms in [0, 1) with 53 random bits."""
    return (_u64(seed, stream, n, offset) >> np.uint64(11)).astype(np.float64) * (2.0 ** -53)


def _normal(seed: int, stream: int, n: int) -> np.ndarray:
    """Standard normals in fp64 by Box-Muller over consecutive pairs of a stream."""
    m = (n + 1) // 2
    u = _u64(seed, stream, 2 * m)
    u1 = ((u[0::2] >> np.uint64(11)).astype(np.float64) + 1.0) * (2.0 ** -53)  # (0, 1]
    u2 = (u[1::2] >> np.uint64(11)).astype(np.float64) * (2.0 ** -53)
    r = np.sqrt(-2.0 * np.log(u1))
    out = np.empty(2 * m, dtype=np.float64)
    out[0::2] = r * np.cos(2.0 * np.pi * u2)
    out[1::2] = r * np.sin(2.0 * np.pi * u2)
    return out[:n]


def f32_to_bf16_bits(a: np.ndarray) -> np.ndarray:
    """Round-to-nearest-even float32 -> bfloat16 bit patterns (uint16)."""
    b = np.ascontiguousarray(a, dtype=np.float32).view(np.uint32)
    lsb = (b >> np.uint32(16)) & np.uint32(1)
    r = (b + np.uint32(0x7FFF) + lsb) >> np.uint32(16)
    return r.astype(np.uint16)


def bf16_bits_to_f32(bits: np.ndarray) -> np.ndarray:
    return (np.ascontiguousarray(bits, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


# ----------------------------------------------------------------------------
# tensors
# ----------------------------------------------------------------------------

def make_codebook_pm1(Kc: int, v: int, seed: int, stream: int = 0, distinct: bool = True) -> np.ndarray:
    """int8 [Kc, v] of +1/-1.  Element t of centroid k is +1 where bit t of the
    k-th drawn pattern is set.  Patterns are distinct when Kc <= 2^v."""
    if not (1 <= v <= 32 and Kc >= 1):
        raise ValueError("bad codebook shape")
    if distinct and Kc <= (1 << v) and v <= 22:
        keys = _u64(seed, stream, 1 << v)
        pats = np.argsort(keys, kind="stable")[:Kc].astype(np.uint64)
    elif distinct and Kc <= (1 << v):
        pats = np.empty(0, dtype=np.uint64)
        off = 0
        while pats.size < Kc:
            draw = _u64(seed, stream, 2 * Kc, off) & np.uint64((1 << v) - 1)
            off += 2 * Kc
            allp = np.concatenate([pats, draw])
            _, first = np.unique(allp, return_index=True)
            pats = allp[np.sort(first)]
        pats = pats[:Kc]
    else:
        pats = _u64(seed, stream, Kc) & np.uint64((1 << v) - 1)
    t = np.arange(v, dtype=np.uint64)
    bits = (pats[:, None] >> t[None, :]) & np.uint64(1)
    return np.where(bits == 1, 1, -1).astype(np.int8)


def make_indices(N: int, Kb: int, Kc: int, dist: str, seed: int, stream: int = 1) -> np.ndarray:
    """uint16 [N, Kb] centroid indices, all < Kc."""
    if not 1 <= Kc <= 65536:
        raise ValueError("Kc out of range")
    u = _uniform01(seed, stream, N * Kb)
    if dist == "uniform":
        idx = np.minimum((u * Kc).astype(np.int64), Kc - 1)
    elif dist == "zipf":
        w = np.arange(1, Kc + 1, dtype=np.float64) ** -1.1
        cdf = np.cumsum(w)
        cdf /= cdf[-1]
        idx = np.minimum(np.searchsorted(cdf, u, side="right"), Kc - 1)
    else:
        raise ValueError(f"unknown index distribution {dist!r}")
    return idx.astype(np.uint16).reshape(N, Kb)


def make_sign_words(n: int, v: int, seed: int, stream: int = 7, prototypes: int = 4096, flip: float = 0.06) -> np.ndarray:
    """n packed v-bit sign vectors (uint32, bit t = element t) standing in for the blocks of a binarised weight
    matrix: each is one of `prototypes` seeded patterns (picked with Zipf(1.1) frequencies) with every element
    flipped independently with probability `flip`, which gives the skewed, clustered pattern histogram that a
    codebook is built for.  prototypes = 0: independent fair signs."""
    mask = np.uint64((1 << v) - 1)
    if prototypes <= 0:
        return (_u64(seed, stream, n) & mask).astype(np.uint32)
    protos = _u64(seed, stream + 100, prototypes) & mask
    w = np.arange(1, prototypes + 1, dtype=np.float64) ** -1.1
    cdf = np.cumsum(w) / w.sum()
    pick = np.minimum(np.searchsorted(cdf, _uniform01(seed, stream + 101, n), side="right"), prototypes - 1)
    words = protos[pick]
    for t in range(v):
        f = _uniform01(seed, stream + 200 + t, n) < flip
        words = words ^ (f.astype(np.uint64) << np.uint64(t))
    return words.astype(np.uint32)


def make_alpha_f16(N: int, seed: int, stream: int = 2, sigma: float = 0.02, scale: float = 1.0,
                   signed: bool = False) -> np.ndarray:
    """|N(0, sigma^2)| * scale as fp16; with signed=True the draw keeps its sign."""
    a = _normal(seed, stream, N)
    if not signed:
        a = np.abs(a)
    return (a * sigma * scale).astype(np.float16)


def make_mu_f16(N: int, seed: int, stream: int = 5, sigma: float = 0.002) -> np.ndarray:
    return (_normal(seed, stream, N) * sigma).astype(np.float16)


def make_x(M: int, K: int, dtype: str, seed: int, stream: int = 3,
           outlier_frac: float = 0.0, outlier_gain: float = 20.0) -> np.ndarray:
    """uint16 bit patterns [M, K] of fp16 ("f16") or bfloat16 ("bf16") N(0,1) draws."""
    x = _normal(seed, stream, M * K).reshape(M, K)
    if outlier_frac > 0.0:
        n_out = int(math.ceil(outlier_frac * K))
        order = np.argsort(_u64(seed, stream + 1, K), kind="stable")[:n_out]
        x[:, order] *= outlier_gain
    if dtype == "f16":
        return x.astype(np.float16).view(np.uint16)
    if dtype == "bf16":
        return f32_to_bf16_bits(x.astype(np.float32))
    raise ValueError(f"unknown x dtype {dtype!r}")


# ----------------------------------------------------------------------------
# layers and configs
# ----------------------------------------------------------------------------

@dataclass(frozen=True)
class LayerSpec:
    name: str
    N: int
    K: int
    v: int
    Kc: int
    idx_dist: str = "uniform"
    x_dtype: str = "f16"
    outlier_frac: float = 0.0
    alpha_scale: float = 1.0      # multiplies the 0.02 sigma (unit-gain chains use 1/(0.02*sqrt(K)))
    alpha_signed: bool = False    # N(0, sigma^2) instead of |N(0, sigma^2)| (chains: keeps the activations zero-mean)
    with_mu: bool = False

    @property
    def Kb(self) -> int:
        return self.K // self.v


@dataclass
class LayerData:
    spec: LayerSpec
    M: int
    C_pm1: np.ndarray            # int8  [Kc, v]
    idx: np.ndarray              # uint16 [N, K/v]
    alpha: np.ndarray            # float16 [N]
    x_bits: np.ndarray           # uint16 [M, K], fp16 or bf16 bit patterns
    mu: Optional[np.ndarray] = None   # float16 [N] or None

    def x_f64(self) -> np.ndarray:
        if self.spec.x_dtype == "f16":
            return self.x_bits.view(np.float16).astype(np.float64)
        return bf16_bits_to_f32(self.x_bits).astype(np.float64)


def make_layer(spec: LayerSpec, M: int, seed: int, layer_id: int = 0,
               parts: str = "all") -> LayerData:
    """Draw one layer.  Streams: 16*layer_id + {0: codebook, 1: idx, 2: alpha, 3: x,
    4: outlier channels, 5: mu}."""
    if spec.K % spec.v:
        raise ValueError("v must divide K")
    s0 = 16 * layer_id
    C = make_codebook_pm1(spec.Kc, spec.v, seed, s0 + 0)
    idx = make_indices(spec.N, spec.Kb, spec.Kc, spec.idx_dist, seed, s0 + 1)
    alpha = make_alpha_f16(spec.N, seed, s0 + 2, scale=spec.alpha_scale, signed=spec.alpha_signed)
    x = make_x(M, spec.K, spec.x_dtype, seed, s0 + 3, spec.outlier_frac)
    mu = make_mu_f16(spec.N, seed, s0 + 5) if spec.with_mu else None
    return LayerData(spec, M, C, idx, alpha, x, mu)


def _llama7b(v: int, Kc: int, **kw) -> List[LayerSpec]:
    sq = [LayerSpec(n, 4096, 4096, v, Kc, **kw) for n in ("q_proj", "k_proj", "v_proj", "o_proj")]
    mlp = [LayerSpec("gate_proj", 11008, 4096, v, Kc, **kw),
           LayerSpec("up_proj", 11008, 4096, v, Kc, **kw),
           LayerSpec("down_proj", 4096, 11008, v, Kc, **kw)]
    return sq + mlp


def _llama13b_k5120(v: int, Kc: int, **kw) -> List[LayerSpec]:
    sq = [LayerSpec(n, 5120, 5120, v, Kc, **kw) for n in ("q_proj", "k_proj", "v_proj", "o_proj")]
    mlp = [LayerSpec("gate_proj", 13824, 5120, v, Kc, **kw),
           LayerSpec("up_proj", 13824, 5120, v, Kc, **kw)]
    return sq + mlp


# config id -> {"layers": [...], "M": (...), "seed": base seed}
CONFIGS: Dict[int, dict] = {
    1: {"layers": [LayerSpec("linear", 4096, 4096, 16, 4096)], "M": (1,), "seed": 42 + 1000},
    2: {"layers": _llama7b(16, 8192, outlier_frac=0.001), "M": (1, 8), "seed": 42 + 2000},
    3: {"layers": _llama13b_k5120(20, 65536, idx_dist="zipf"), "M": (1, 4), "seed": 42 + 3000},
    4: {"layers": [LayerSpec("sq", 4096, 4096, 16, 8192, x_dtype="bf16"),
                   LayerSpec("gate_up", 11008, 4096, 16, 8192, x_dtype="bf16"),
                   LayerSpec("down", 4096, 11008, 16, 8192, x_dtype="bf16")],
        "M": (512, 2048), "seed": 42 + 4000},
}


def config_layers(config: int, Kc: Optional[int] = None, idx_dist: Optional[str] = None) -> dict:
    """Layer list of one benchmark config.  Config 5 is the 32-layer decode chain
    (7 projections per layer, v=16); Kc and the index distribution are swept.  So that a
    chain of 224 linears with nothing between them stays inside fp16 range for every
    point of the sweep, its scales have unit RMS gain (sigma = 1/sqrt(K)) and keep the
    sign of their normal draw: with all-positive scales every output carries the same
    multiple of the common component <x, mean centroid>, the next layer's input has a
    non-zero mean, and that mode grows from layer to layer (with few centroids or Zipf
    indices the mean centroid is far from zero); with signed scales the activations stay
    zero-mean and uncorrelated, and the expected gain of a layer is exactly one."""
    if config in CONFIGS:
        return CONFIGS[config]
    if config == 5:
        kc = 4096 if Kc is None else Kc
        dist = idx_dist or "uniform"
        one = _llama7b(16, kc, idx_dist=dist)
        one = [replace(s, alpha_scale=1.0 / (0.02 * math.sqrt(s.K)), alpha_signed=True) for s in one]
        return {"layers": one, "n_blocks": 32, "M": (1,), "seed": 42 + 5000}
    raise KeyError(config)

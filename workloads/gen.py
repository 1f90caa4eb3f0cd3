"""Seeded generators for the indexer top-k workloads.

Every array is drawn on the CPU from a counter-based generator (Philox), so the
bytes depend only on (config name, shape, seed).  The shapes and value
structure follow the five benchmark configurations:

  tiny_f32      fp32, iid Gaussian q/k, Gaussian head weights
  dsa_bf16      bf16 q/k, keys carry a slow positional drift along one direction
  fp8_ar1       e4m3 codes + per-token fp32 absmax scales, AR(1) queries (rho = 0.9)
  fp8_1m        same recipe, 4096 queries at the end of a 1,048,576-key context
  hot_fp8       e4m3, a shared set of high-scoring keys (for the previous-chunk sampler)
  adv_planted   heavy-tailed key norms + 5 % planted keys along query directions
  adv_cluster   all planted keys identical, along a component shared by all queries
  adv_ties      q/k coordinates on 4 levels (continuous head weights)
  adv_ties_exact  same, with +-1/sqrt(H) weights so every sum is exact (mass ties)

Storage formats are produced here (bf16 / e4m3 rounding); decoding is the
consumer's business.  The query's per-token fp8 scale is folded into the head
weights, w[t, h] <- w[t, h] * q_scale[t], which is exact for the score because
ReLU is positively homogeneous.
"""
from __future__ import annotations

import dataclasses
from typing import Optional

import numpy as np

BASE_SEED = 0x260711976


@dataclasses.dataclass
class IndexerInputs:
    """One problem instance.  `q`, `k` hold storage codes: float32 for dtype
    "f32", uint16 bit patterns for "bf16", uint8 codes for "e4m3"."""

    name: str
    dtype: str
    q: np.ndarray  # [T, H, D]
    w: np.ndarray  # [T, H] float32
    k: np.ndarray  # [N, D]
    k_scale: Optional[np.ndarray]  # [N] float32, e4m3 only
    topk: int
    causal_offset: int
    meta: dict = dataclasses.field(default_factory=dict)

    @property
    def T(self) -> int:
        return self.q.shape[0]

    @property
    def H(self) -> int:
        return self.q.shape[1]

    @property
    def D(self) -> int:
        return self.q.shape[2]

    @property
    def N(self) -> int:
        return self.k.shape[0]

    def visible(self, t: int) -> int:
        """Number of keys row t may see: keys 0 .. causal_offset + t, clipped to N."""
        return int(min(self.N, max(0, self.causal_offset + t + 1)))

    def valid_pairs(self) -> int:
        return int(sum(self.visible(t) for t in range(self.T)))


# ----------------------------------------------------------------------------
# storage formats
# ----------------------------------------------------------------------------

def bf16_encode(x: np.ndarray) -> np.ndarray:
    """float32 -> bf16 bit patterns (uint16), round to nearest even."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    bias = ((u >> 16) & 1) + np.uint32(0x7FFF)
    return ((u + bias) >> 16).astype(np.uint16)


def e4m3_encode(x: np.ndarray) -> np.ndarray:
    """float32 -> OCP e4m3 ("fn": no inf, max 448) codes, round to nearest even,
    saturating at +-448."""
    x = np.asarray(x, dtype=np.float32)
    sign = (np.signbit(x)).astype(np.uint8) << 7
    a = np.minimum(np.abs(x).astype(np.float64), 448.0)
    _, e = np.frexp(a)  # a = m * 2**e with m in [0.5, 1)
    ex = np.maximum(e - 1, -6)  # exponent of the leading bit, clamped to the subnormal range
    steps = np.rint(a / np.exp2(ex - 3.0))  # multiples of the local quantum, ties to even
    carry = steps >= 16
    ex = np.where(carry, ex + 1, ex)
    steps = np.where(carry, 8.0, steps)
    normal = steps >= 8
    code = np.where(normal, ((ex + 7).astype(np.int64) << 3) | (steps.astype(np.int64) - 8), steps.astype(np.int64))
    return (code.astype(np.uint8) | sign).astype(np.uint8)


def quantize_e4m3_per_token(x: np.ndarray) -> tuple[np.ndarray, np.ndarray]:
    """Per-token absmax quantisation: one fp32 scale per leading index, taken over all
    trailing axes; scale = absmax / 448 (1 when the token is all zero)."""
    x = np.asarray(x, dtype=np.float32)
    flat = x.reshape(x.shape[0], -1)
    absmax = np.abs(flat).max(axis=1)
    scale = np.where(absmax > 0, absmax / np.float32(448.0), np.float32(1.0)).astype(np.float32)
    codes = e4m3_encode((flat / scale[:, None]).astype(np.float32)).reshape(x.shape)
    return codes, scale


# ----------------------------------------------------------------------------
# random draws
# ----------------------------------------------------------------------------

def _rng(seed: int, stream: int) -> np.random.Generator:
    return np.random.Generator(np.random.Philox(key=[seed & 0xFFFFFFFFFFFFFFFF, stream]))


def _normal(seed: int, stream: int, shape, std: float) -> np.ndarray:
    x = _rng(seed, stream).standard_normal(shape, dtype=np.float32)
    x *= np.float32(std)
    return x


def _ar1_along_rows(eps: np.ndarray, rho: float) -> np.ndarray:
    """x[0] = eps[0]; x[t] = rho x[t-1] + sqrt(1 - rho^2) eps[t] (stationary variance)."""
    out = np.empty_like(eps)
    out[0] = eps[0]
    c = np.float32(np.sqrt(1.0 - rho * rho))
    r = np.float32(rho)
    for t in range(1, eps.shape[0]):
        out[t] = r * out[t - 1] + c * eps[t]
    return out


def _unit(v: np.ndarray) -> np.ndarray:
    n = np.linalg.norm(v.astype(np.float64), axis=-1, keepdims=True)
    n = np.where(n > 0, n, 1.0)
    return (v / n).astype(np.float32)


# ----------------------------------------------------------------------------
# configurations
# ----------------------------------------------------------------------------

CONFIGS = {
    # name: (recipe, dtype, T, N, H, D, topk, config id for the seed)
    "tiny_f32": ("iid", "f32", 64, 4096, 8, 64, 256, 1),
    "dsa_bf16": ("drift", "bf16", 4096, 65536, 64, 128, 2048, 2),
    "fp8_ar1": ("ar1", "e4m3", 8192, 131072, 64, 128, 2048, 3),
    "fp8_1m": ("ar1", "e4m3", 4096, 1048576, 64, 128, 2048, 4),
    "adv_planted": ("planted", "bf16", 4096, 65536, 64, 128, 2048, 5),
    "adv_cluster": ("cluster", "bf16", 4096, 65536, 64, 128, 2048, 6),
    "adv_ties": ("ties", "bf16", 4096, 65536, 64, 128, 2048, 7),
    "adv_ties_exact": ("ties_exact", "bf16", 4096, 65536, 64, 128, 2048, 8),
    # stand-in for the cross-chunk structure the previous-chunk sampler relies on (paper Sec. 3.2 "Sampling")
    "hot_fp8": ("hot", "e4m3", 4096, 1048576, 64, 128, 2048, 9),
}


def _store(x: np.ndarray, dtype: str) -> np.ndarray:
    if dtype == "f32":
        return np.ascontiguousarray(x, dtype=np.float32)
    if dtype == "bf16":
        return bf16_encode(x)
    raise ValueError(dtype)


def make_inputs(recipe: str, dtype: str, T: int, N: int, H: int, D: int, topk: int,
                seed: int, causal_offset: Optional[int] = None, name: str = "custom") -> IndexerInputs:
    """Draw one instance of `recipe` at the given shape."""
    if causal_offset is None:
        causal_offset = N - T  # the chunk sits at the end of the context
    meta: dict = {"recipe": recipe, "seed": seed}
    sd = 1.0 / np.sqrt(D)
    w = _normal(seed, 2, (T, H), 1.0 / np.sqrt(H))

    if recipe == "ar1":
        q = _ar1_along_rows(_normal(seed, 0, (T, H * D), sd), 0.9).reshape(T, H, D)
    elif recipe in ("ties", "ties_exact"):
        q = None
    else:
        q = _normal(seed, 0, (T, H, D), sd)

    if recipe in ("iid", "ar1"):
        k = _normal(seed, 1, (N, D), sd)
    elif recipe == "hot":
        # "adjacent chunks attend to the same prefix tokens": 3k/2 keys at random positions of the first half of the
        # context carry a shared direction c that every query head carries too, and the head weights are
        # positive, so these keys score high for every row of every chunk; which of them make a row's top-k
        # is decided by the independent parts
        k = _normal(seed, 1, (N, D), sd)
        c = _unit(_normal(seed, 6, (D,), 1.0))
        n_hot = min(max(N // 8, 1), (3 * topk) // 2)
        pos = np.sort(_rng(seed, 5).permutation(max(N // 2, n_hot))[:n_hot])
        k[pos] += c[None, :]
        q = q + np.float32(0.5) * c[None, None, :]
        w = np.abs(w)
        meta["hot_pos"] = pos
        meta["hot_dir"] = c
    elif recipe == "drift":
        k = _normal(seed, 1, (N, D), sd)
        u = _unit(_normal(seed, 3, (D,), 1.0))
        s = np.arange(N, dtype=np.float64)
        k += (0.2 * np.sin(s / 4096.0))[:, None].astype(np.float32) * u[None, :]
        meta["drift_dir"] = u
    elif recipe in ("planted", "cluster"):
        # heavy-tailed norms: direction uniform, norm = |t_3| / median|t_3|
        direction = _unit(_normal(seed, 1, (N, D), 1.0))
        t3 = np.abs(_rng(seed, 4).standard_t(3.0, size=N))
        norms = (t3 / np.median(t3)).astype(np.float32)
        k = direction * norms[:, None]
        n_plant = int(round(0.05 * N))
        pos = _rng(seed, 5).permutation(N)[:n_plant]
        if recipe == "planted":
            # each planted key points along one query's positive-weight mean direction, norm 3
            target = _rng(seed, 6).integers(0, T, size=n_plant)
            dirs = _unit(np.einsum("th,thd->td", np.maximum(w, 0.0), q))
            k[pos] = 3.0 * dirs[target]
            meta["planted_target"] = target
        else:
            # one shared direction, present in every query head; all planted keys identical
            c = _unit(_normal(seed, 6, (D,), 1.0))
            q = q + np.float32(0.5) * c[None, None, :]
            k[pos] = 3.0 * c[None, :]
            meta["cluster_dir"] = c
        meta["planted_pos"] = np.sort(pos)
    elif recipe in ("ties", "ties_exact"):
        # coordinates on four levels {+-0.5, +-1.5} * 2^-ceil(log2(D)/2): exactly representable
        step = np.float32(2.0 ** -int(np.ceil(np.log2(D) / 2.0)))

        def four_levels(stream, shape):
            g = _rng(seed, stream).standard_normal(shape, dtype=np.float32)
            mag = np.where(np.abs(g) < 1.0, np.float32(0.5), np.float32(1.5))
            return np.sign(g).astype(np.float32) * mag * step

        q = four_levels(0, (T, H, D))
        k = four_levels(1, (N, D))
        if recipe == "ties_exact":
            w = (np.where(w >= 0, 1.0, -1.0) * 2.0 ** -int(np.ceil(np.log2(H) / 2.0))).astype(np.float32)
    else:
        raise ValueError(f"unknown recipe {recipe!r}")

    k_scale = None
    if dtype == "e4m3":
        q_codes, q_scale = quantize_e4m3_per_token(q)
        k_codes, k_scale = quantize_e4m3_per_token(k)
        w = (w * q_scale[:, None]).astype(np.float32)
        q_st, k_st = q_codes, k_codes
    else:
        q_st, k_st = _store(q, dtype), _store(k, dtype)

    return IndexerInputs(name=name, dtype=dtype, q=q_st, w=np.ascontiguousarray(w, dtype=np.float32),
                         k=k_st, k_scale=k_scale, topk=topk, causal_offset=int(causal_offset), meta=meta)


def make_config(name: str, T: Optional[int] = None, N: Optional[int] = None, H: Optional[int] = None,
                D: Optional[int] = None, topk: Optional[int] = None, dtype: Optional[str] = None,
                seed: Optional[int] = None, causal_offset: Optional[int] = None) -> IndexerInputs:
    """The named configuration, optionally at a reduced shape (same recipe and seed rule)."""
    recipe, dt, T0, N0, H0, D0, k0, cid = CONFIGS[name]
    return make_inputs(recipe, dtype or dt, T or T0, N or N0, H or H0, D or D0, topk or k0,
                       seed if seed is not None else BASE_SEED + cid, causal_offset, name=name)


# ----------------------------------------------------------------------------
# k-NN retrieval variant (inner product over a corpus of embeddings)
# ----------------------------------------------------------------------------

@dataclasses.dataclass
class KnnInputs:
    """A batch of queries and a corpus, both bf16 codes (uint16), row-major [rows, D]."""

    name: str
    q: np.ndarray      # [T, D] uint16
    x: np.ndarray      # [N, D] uint16
    topk: int
    meta: dict

    @property
    def T(self) -> int:
        return int(self.q.shape[0])

    @property
    def N(self) -> int:
        return int(self.x.shape[0])

    @property
    def D(self) -> int:
        return int(self.q.shape[1])

    def valid_pairs(self) -> int:
        return self.T * self.N


KNN_CONFIGS = {
    # name: (T, N, D, topk, config id for the seed).  Stand-in for 768-d passage embeddings: unit vectors drawn
    # around 64 cluster centres (concentrated similarities, no temporal structure), queries drawn like passages.
    "knn_bf16": (64, 1 << 20, 768, 1024, 20),
}


def make_knn(name: str = "knn_bf16", T: Optional[int] = None, N: Optional[int] = None, D: Optional[int] = None,
             topk: Optional[int] = None) -> KnnInputs:
    T0, N0, D0, k0, cid = KNN_CONFIGS[name]
    T, N, D, topk = T or T0, N or N0, D or D0, topk or k0
    seed = BASE_SEED + cid
    n_centres = 64
    centres = _unit(_normal(seed, 0, (n_centres, D), 1.0))

    def draw(stream: int, rows: int) -> np.ndarray:
        which = _rng(seed, stream).integers(0, n_centres, size=rows)
        out = np.empty((rows, D), dtype=np.float32)
        step = 1 << 16
        for r0 in range(0, rows, step):  # in slabs: the corpus can be several GB in fp32
            r1 = min(rows, r0 + step)
            g = _rng(seed, stream + 100 + r0 // step).standard_normal((r1 - r0, D), dtype=np.float32)
            out[r0:r1] = _unit(g / np.float32(np.sqrt(D)) + np.float32(0.7) * centres[which[r0:r1]])
        return out

    x = draw(1, N)
    q = draw(2, T)
    return KnnInputs(name=name, q=bf16_encode(q), x=bf16_encode(x), topk=topk,
                     meta={"recipe": "embed", "seed": seed, "centres": n_centres})


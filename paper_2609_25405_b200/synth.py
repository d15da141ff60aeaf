"""Seeded synthetic inputs: model shapes, weights, token ids, workload draws.

This module holds NO arithmetic of the method.  It only draws random numbers
and lays them out, so that the CUDA path and the CPU checker can be fed the
same bits.  It imports neither of them.

Weights: every matrix (token embedding and LM head included) is N(0, 0.02^2)
drawn in float32 and rounded to bfloat16 (round to nearest, ties to even);
norm gains are 1.  Each tensor has its own generator keyed by
(seed, layer, tensor id), so any tensor can be regenerated alone, in any
order, without holding the whole model.
"""
from dataclasses import dataclass
import numpy as np


@dataclass(frozen=True)
class ModelShape:
    name: str
    L: int
    d: int
    Hq: int
    Hkv: int
    Dh: int
    F: int
    V: int
    rope_theta: float = 1.0e4
    rms_eps: float = 1.0e-5
    page_size: int = 16

    @property
    def n_qkv(self):
        return (self.Hq + 2 * self.Hkv) * self.Dh

    def with_layers(self, L):
        return ModelShape(f"{self.name}-L{L}", L, self.d, self.Hq, self.Hkv, self.Dh,
                          self.F, self.V, self.rope_theta, self.rms_eps, self.page_size)


SHAPES = {
    "tiny": ModelShape("tiny", 2, 256, 4, 4, 64, 1024, 1024),
    "1b": ModelShape("1b", 16, 2048, 32, 8, 64, 8192, 128256),
    "7b": ModelShape("7b", 32, 4096, 32, 8, 128, 14336, 32000),
}


def f32_to_bf16_bits(a):
    """float32 array -> uint16 bfloat16 bit patterns, round-to-nearest-even."""
    u = np.ascontiguousarray(a, dtype=np.float32).view(np.uint32)
    rounded = u + (np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1)))
    return (rounded >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(b):
    return (np.asarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


_TENSOR_IDS = {"attn_norm": 0, "wq": 1, "wk": 2, "wv": 3, "wo": 4, "ffn_norm": 5,
               "wg": 6, "wu": 7, "wd": 8}
_GLOBAL_LAYER = 1 << 20
_GLOBAL_IDS = {"tok_emb": 0, "final_norm": 1, "lm_head": 2}


class Weights:
    """Lazily generated bf16-exact weights, returned as float32 arrays.

    Interface used by the checker: .tok_emb, .final_norm, .lm_head and
    .layer(l) -> dict.  `cache=True` keeps generated tensors (small models)."""

    def __init__(self, shape: ModelShape, seed: int = 0, std: float = 0.02, cache=True):
        """cache: True keeps float32 tensors, "bits" keeps the uint16 bf16 patterns (half the
        memory; converted on access), False regenerates on every access."""
        self.shape = shape
        self.seed = seed
        self.std = std
        self._cache = {} if cache else None
        self._bits = (cache == "bits")

    def _normal_bits(self, key, rows, cols):
        rng = np.random.default_rng([self.seed, key[0], key[1]])
        a = rng.standard_normal((rows, cols), dtype=np.float32)
        a *= np.float32(self.std)
        return f32_to_bf16_bits(a).reshape(rows, cols)

    def _normal_bf16(self, key, rows, cols):
        if self._bits:
            return self._normal_bits(key, rows, cols)
        return bf16_bits_to_f32(self._normal_bits(key, rows, cols)).reshape(rows, cols)

    def _get(self, key, maker):
        if self._cache is None:
            v = maker()
        else:
            if key not in self._cache:
                self._cache[key] = maker()
            v = self._cache[key]
        if v.dtype == np.uint16:
            return bf16_bits_to_f32(v).reshape(v.shape)
        return v

    def prefetch(self, threads=8):
        """Generate every tensor into the cache with a thread pool (numpy releases the GIL)."""
        from concurrent.futures import ThreadPoolExecutor
        jobs = [(l, n) for l in range(self.shape.L) for n in _TENSOR_IDS] + [(None, "tok_emb"), (None, "lm_head")]

        def run(j):
            if j[0] is None:
                getattr(self, j[1])
            else:
                self.tensor(*j)
        with ThreadPoolExecutor(threads) as ex:
            list(ex.map(run, jobs))
        return self

    def tensor(self, layer, name):
        s = self.shape
        dims = {"wq": (s.Hq * s.Dh, s.d), "wk": (s.Hkv * s.Dh, s.d), "wv": (s.Hkv * s.Dh, s.d),
                "wo": (s.d, s.Hq * s.Dh), "wg": (s.F, s.d), "wu": (s.F, s.d), "wd": (s.d, s.F)}
        key = (layer, _TENSOR_IDS[name])
        if name in ("attn_norm", "ffn_norm"):
            return self._get(key, lambda: np.ones(s.d, dtype=np.float32))
        r, c = dims[name]
        return self._get(key, lambda: self._normal_bf16(key, r, c))

    def layer(self, l):
        return {n: self.tensor(l, n) for n in _TENSOR_IDS}

    @property
    def tok_emb(self):
        key = (_GLOBAL_LAYER, _GLOBAL_IDS["tok_emb"])
        return self._get(key, lambda: self._normal_bf16(key, self.shape.V, self.shape.d))

    @property
    def lm_head(self):
        key = (_GLOBAL_LAYER, _GLOBAL_IDS["lm_head"])
        return self._get(key, lambda: self._normal_bf16(key, self.shape.V, self.shape.d))

    @property
    def final_norm(self):
        return np.ones(self.shape.d, dtype=np.float32)



LORA_TARGETS = ("wq", "wk", "wv", "wo", "wg", "wu", "wd")


class LoraAdapters:
    """Seeded random low-rank adapter factors for every projection of every layer (inputs only; how
    they enter the forward pass is for each side to state).  For projection `name` of layer l with
    weight [out, in]: A [rank, in] and B [out, rank], both N(0, std^2) rounded to bf16 and returned
    as float32; `alpha` is the usual scaling numerator (the update is scaled by alpha / rank)."""

    def __init__(self, shape: ModelShape, rank: int, seed: int = 7, std: float = 0.02, alpha=None):
        assert 1 <= rank <= 64
        self.shape, self.rank, self.seed, self.std = shape, int(rank), seed, std
        self.alpha = float(2 * rank if alpha is None else alpha)
        self._cache = {}

    @property
    def scale(self):
        return self.alpha / self.rank

    def _dims(self, name):
        s = self.shape
        return {"wq": (s.Hq * s.Dh, s.d), "wk": (s.Hkv * s.Dh, s.d), "wv": (s.Hkv * s.Dh, s.d),
                "wo": (s.d, s.Hq * s.Dh), "wg": (s.F, s.d), "wu": (s.F, s.d), "wd": (s.d, s.F)}[name]

    def factors(self, layer, name):
        """(A [rank, in], B [out, rank]) of one projection."""
        key = (layer, name)
        if key not in self._cache:
            out, inn = self._dims(name)
            t = LORA_TARGETS.index(name)
            rng = np.random.default_rng([self.seed, 1000 + layer, t])
            a = rng.standard_normal((self.rank, inn), dtype=np.float32) * np.float32(self.std)
            b = rng.standard_normal((out, self.rank), dtype=np.float32) * np.float32(self.std)
            self._cache[key] = (bf16_bits_to_f32(f32_to_bf16_bits(a)).reshape(a.shape),
                                bf16_bits_to_f32(f32_to_bf16_bits(b)).reshape(b.shape))
        return self._cache[key]


def token_ids(rng, n, V):
    """n token ids uniform in [0, V)."""
    return rng.integers(0, V, size=n, dtype=np.int64)


def lognormal_lengths(rng, n, median, lo, hi, sigma=1.0):
    """Lengths exp(N(ln median, sigma^2)), rounded to nearest, clipped to [lo, hi]."""
    x = np.exp(rng.normal(np.log(median), sigma, size=n))
    return np.clip(np.rint(x), lo, hi).astype(np.int64)


def nominal_chunks(n, C):
    """C, C, ..., remainder."""
    sizes = [C] * (n // C)
    if n % C:
        sizes.append(n % C)
    return sizes


def random_partition(rng, n, max_chunk=None):
    """A random ordered partition of n into positive parts (each <= max_chunk)."""
    sizes = []
    left = n
    while left > 0:
        hi = left if max_chunk is None else min(left, max_chunk)
        c = int(rng.integers(1, hi + 1))
        sizes.append(c)
        left -= c
    return sizes


@dataclass
class Cfg1Workload:
    """Tiny mixed workload: 4 generation requests with 64 cached prompt tokens
    decoding 8 greedy steps, plus embedding requests of 100 and 37 tokens in
    chunks of 32, mean pooling."""
    prompts: list          # 4 arrays of 64 token ids
    embed_tokens: list     # arrays of 100 and 37 token ids
    chunk: int = 32
    decode_steps: int = 8
    pool_mode: str = "mean"


def cfg1_workload(seed=1001, V=1024, n_gen=4, ctx=64, embed_lens=(100, 37)):
    rng = np.random.default_rng(seed)
    prompts = [token_ids(rng, ctx, V) for _ in range(n_gen)]
    embeds = [token_ids(rng, n, V) for n in embed_lens]
    return Cfg1Workload(prompts, embeds)

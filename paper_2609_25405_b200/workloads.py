"""Synthetic mixed-batch workloads and the host-side packer that composes each step.

Host glue only (no arithmetic of the forward pass).  The packer is the simple policy the
benchmark configurations need: in-flight decode rows are reserved first, then embedding
requests are admitted first-come-first-served in chunks of at most C tokens until the token
budget is full (the chunk-admission rule of the paper's Section 4.2: a request longer than the
residual budget contributes a chunk instead of leaving the budget unused).
"""
from dataclasses import dataclass

import numpy as np

from . import consts as B
from . import synth


@dataclass
class MixSpec:
    name: str
    shape: str                 # key of synth.SHAPES
    n_decode: int
    ctx_lo: int
    ctx_hi: int
    budget: int
    chunk: int
    emb_dist: str              # "lognormal" | "uniform"
    emb_a: int                 # median | lo
    emb_lo: int
    emb_hi: int
    pool_mode: int
    seed: int


SPECS = {
    # 1B-class shape: 32 decode rows, contexts U[128,1024]; embedding lengths lognormal(median 256,
    # sigma 1) clipped to [16,2048], chunk 256, last-token pooling, 2048-token budget
    "cfg2-1b": MixSpec("cfg2-1b", "1b", 32, 128, 1024, 2048, 256, "lognormal", 256, 16, 2048, B.POOL_LAST, 1002),
    # 7B-class shape: 64 decode rows, contexts U[512,4096]; embedding lengths lognormal(median 512,
    # sigma 1) clipped to [32,4096], chunk 512, last-token pooling, 4096-token budget
    "cfg3-7b": MixSpec("cfg3-7b", "7b", 64, 512, 4096, 4096, 512, "lognormal", 512, 32, 4096, B.POOL_LAST, 1003),
    # small decode-heavy case for profiler captures (use with --layers and --decode-alias)
    # a small decode-heavy step of the 1B shape, the size the trace replay's steps have on average
    "dec-1b": MixSpec("dec-1b", "1b", 400, 128, 1024, 448, 256, "uniform", 128, 16, 256, B.POOL_LAST, 1011),
    "dec-7b": MixSpec("dec-7b", "7b", 256, 2048, 2048, 512, 256, "uniform", 128, 128, 1024, B.POOL_MEAN, 1010),
}


def sweep_spec(frac, seed=1004, cap_decode=0):
    """Embedding-fraction sweep on the 7B shape: 4096-token budget, decode contexts 2048,
    embedding lengths U[128,2048], mean pooling, chunk cap 512.  cap_decode > 0 is the
    capacity-true variant: the decode rows are capped at what one GPU can hold unaliased (268 MB of
    K/V per row), the embedding rows stay, so the step is smaller than 4096 rows."""
    n_emb = int(round(4096 * frac))
    n_dec = 4096 - n_emb
    name = f"cfg4-7b-f{frac:g}"
    if cap_decode and n_dec > cap_decode:
        n_dec = cap_decode
        name += f"-cap{cap_decode}"
    return MixSpec(name, "7b", n_dec, 2048, 2048, n_dec + n_emb, 512, "uniform", 128, 128, 2048, B.POOL_MEAN, seed)


class _Req:
    __slots__ = ("n", "done", "pages", "slot", "kind")

    def __init__(self, kind, n, done=0):
        self.kind, self.n, self.done, self.pages, self.slot = kind, n, done, [], -1


class MixedWorkload:
    """Generates one step's descriptor entries at a time and owns pages / slots.

    `kv` and `pool` are binding.KvCache / binding.Pool (their free lists are host-side, so the
    packer can be advanced without launching anything: `warm` steps bring the embedding queue to
    its steady state; the KV those skipped steps would have written is whatever the arena holds).
    `decode_alias` > 0 makes decode request i read the context pages of request i % decode_alias
    (read-only sharing; every row still appends to a private tail page).
    """

    def __init__(self, spec, kv, pool, max_pos, decode_alias=0, shape=None):
        self.spec = spec
        self.shape = shape if shape is not None else synth.SHAPES[spec.shape]
        self.kv, self.pool = kv, pool
        self.P = self.shape.page_size
        self.max_pos = max_pos
        self.rng = np.random.default_rng(spec.seed)
        self.decodes = []
        self.inflight = []
        self.alias = decode_alias
        ctxs = self.rng.integers(spec.ctx_lo, spec.ctx_hi + 1, size=spec.n_decode)
        for i, c in enumerate(ctxs):
            r = _Req("gen", int(c) + 1, int(c))
            if decode_alias and i >= decode_alias:
                src = self.decodes[i % decode_alias]
                n_shared = int(c) // self.P            # full context pages are shared read-only
                assert int(c) % self.P == 0 and src.done == int(c)
                r.pages = list(src.pages[:n_shared])
            else:
                r.pages = self.kv.alloc((int(c) + self.P - 1) // self.P)
            self.decodes.append(r)

    def _draw_len(self):
        s = self.spec
        if s.emb_dist == "lognormal":
            return int(synth.lognormal_lengths(self.rng, 1, s.emb_a, s.emb_lo, s.emb_hi)[0])
        return int(self.rng.integers(s.emb_lo, s.emb_hi + 1))

    def _grow(self, r, n_tokens):
        need = (n_tokens + self.P - 1) // self.P - len(r.pages)
        if need > 0:
            r.pages.extend(self.kv.alloc(need))

    def next_step(self):
        """Returns (entries, commit).  Call commit() after the step was enqueued (or to skip it)."""
        s = self.spec
        V = self.shape.V
        entries, plan = [], []
        for r in self.decodes:
            if r.done + 1 > self.max_pos:
                raise RuntimeError("decode request reached max_pos")
            self._grow(r, r.done + 1)
            entries.append(dict(kind=B.KIND_DECODE, tokens=self.rng.integers(0, V, 1), pos_start=r.done,
                                pages=r.pages, is_final=True))
            plan.append((r, 1))
        left = s.budget - len(self.decodes)
        queue, idx, nxt = self.inflight, 0, []
        while left > 0:
            if idx < len(queue):
                r = queue[idx]
                idx += 1
            else:
                r = _Req("embed", self._draw_len())
                r.slot = self.pool.alloc()
            q = min(s.chunk, r.n - r.done, left)
            self._grow(r, r.done + q)
            final = (r.done + q == r.n)
            entries.append(dict(kind=B.KIND_EMBED_CHUNK, tokens=self.rng.integers(0, V, q), pos_start=r.done,
                                pages=r.pages, pool_slot=r.slot, pool_mode=s.pool_mode, is_final=final))
            plan.append((r, q))
            if not final:
                nxt.append(r)
            left -= q
        self.inflight = queue[idx:] + nxt        # requests the budget did not reach stay first in line

        def commit(advance_decode=True):
            for r, q in plan:
                if r.kind == "gen" and not advance_decode:
                    continue
                r.done += q
                if r.kind == "embed" and r.done == r.n:
                    self.kv.free(r.pages)
                    self.pool.free(r.slot)
                    r.pages, r.slot = [], -1
                elif r.kind == "gen":
                    r.n += 1
        return entries, commit


def step_work(shape, entries):
    """Algorithmic work of one step: GEMM flops, attention flops, bytes (weights once, KV read,
    KV write).  Counts what the method itself must do, whatever the kernels do."""
    s = shape
    T = sum(len(e["tokens"]) for e in entries)
    n_logit = sum(1 for e in entries if e["kind"] == B.KIND_DECODE or
                  (e["kind"] == B.KIND_PREFILL_CHUNK and e.get("is_final")))
    per_layer = s.d * s.n_qkv + s.Hq * s.Dh * s.d + 3 * s.d * s.F
    gemm = 2.0 * s.L * per_layer * T + 2.0 * s.d * s.V * n_logit
    pairs = 0
    kv_tok_read = 0
    pairs_chunk = 0          # (query, key) pairs of chunk rows: the tensor-bound share of attention
    kv_tok_read_decode = 0   # keys decode rows read: the HBM-bound share
    for e in entries:
        q, p0 = len(e["tokens"]), e["pos_start"]
        pairs += q * p0 + q * (q + 1) // 2
        kv_tok_read += p0 + q
        if e["kind"] == B.KIND_DECODE:
            kv_tok_read_decode += p0 + q
        else:
            pairs_chunk += q * p0 + q * (q + 1) // 2
    attn = 4.0 * s.Dh * s.Hq * s.L * pairs
    kv_tok = s.L * 2 * s.Hkv * s.Dh * 2
    w_bytes = 2.0 * (s.L * per_layer + (s.d * s.V if n_logit else 0)) + 2.0 * s.d * T
    return dict(T=T, n_logit=n_logit, gemm_flops=gemm, attn_flops=attn, weight_bytes=w_bytes,
                kv_read_bytes=float(kv_tok) * kv_tok_read, kv_write_bytes=float(kv_tok) * T,
                attn_flops_chunk=4.0 * s.Dh * s.Hq * s.L * pairs_chunk,
                kv_read_bytes_decode=float(kv_tok) * kv_tok_read_decode)

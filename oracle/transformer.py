"""Plain definition of the result (test infrastructure only; see package doc).

Chunking, incremental pooling, the paged cache and batching are exact
reformulations of a plain computation (Section 3.3, last paragraph: the
incremental and the single-pass pooler are algebraically equal up to
floating-point summation order).  So the oracle computes that plain
computation: one pass over the whole token sequence of ONE request, no cache,
no chunks, no batch.

Model family (the configurations fix it; the paper only names the backbones,
Section 5.1): decoder-only, pre-norm RMSNorm, rotary position embedding in the
"rotate-half" pairing, grouped-query causal attention, SwiGLU feed-forward, no
biases, untied LM head.

`cfg` is any object with integer attributes L, d, Hq, Hkv, Dh, F, V and float
attributes rope_theta, rms_eps.  `W` is any object with
    W.tok_emb [V,d], W.final_norm [d], W.lm_head [V,d], and
    W.layer(l) -> dict(attn_norm[d], wq[Hq*Dh,d], wk[Hkv*Dh,d], wv[Hkv*Dh,d],
                       wo[d,Hq*Dh], ffn_norm[d], wg[F,d], wu[F,d], wd[d,F])
All matrices are [out, in]; y = x @ w.T.
"""
import numpy as np


def rmsnorm(x, g, eps):
    """x * rsqrt(mean(x^2) + eps) * g over the last axis."""
    ms = np.mean(x * x, axis=-1, keepdims=True)
    return x / np.sqrt(ms + eps) * g


def rope_cos_sin(Dh, theta, positions, dtype):
    """Rotary angles: angle[p, i] = p * theta^(-2i/Dh), i in [0, Dh/2).

    Angles are formed in float64; cos/sin are then held in float32 precision
    (that is what any fp32 implementation can hold) and returned in `dtype`.
    """
    i = np.arange(Dh // 2, dtype=np.float64)
    inv_freq = theta ** (-2.0 * i / Dh)
    ang = np.asarray(positions, dtype=np.float64)[:, None] * inv_freq[None, :]
    cos = np.cos(ang).astype(np.float32).astype(dtype)
    sin = np.sin(ang).astype(np.float32).astype(dtype)
    return cos, sin


def apply_rope(x, cos, sin):
    """x [n, H, Dh]; pairs (i, i + Dh/2) are rotated by the angle of (pos, i)."""
    half = x.shape[-1] // 2
    x1 = x[..., :half]
    x2 = x[..., half:]
    c = cos[:, None, :]
    s = sin[:, None, :]
    return np.concatenate([x1 * c - x2 * s, x2 * c + x1 * s], axis=-1)


def silu(x):
    return x / (1.0 + np.exp(-x))


def causal_attention(q, k, v, Hq, Hkv):
    """q [n,Hq,Dh], k,v [n,Hkv,Dh] -> o [n,Hq,Dh].

    Query head a uses KV head a // (Hq/Hkv).  Row t sees keys s <= t only;
    softmax of q.k/sqrt(Dh) with the maximum subtracted.
    """
    n, _, Dh = q.shape
    group = Hq // Hkv
    scale = 1.0 / np.sqrt(np.asarray(Dh, dtype=q.dtype))
    visible = np.tril(np.ones((n, n), dtype=bool))
    o = np.empty_like(q)
    for a in range(Hq):
        b = a // group
        s = (q[:, a, :] @ k[:, b, :].T) * scale
        s = np.where(visible, s, -np.inf)
        s = s - np.max(s, axis=-1, keepdims=True)
        p = np.exp(s)
        p = p / np.sum(p, axis=-1, keepdims=True)
        o[:, a, :] = p @ v[:, b, :]
    return o


def forward(cfg, W, tokens, logit_rows=None, dtype=np.float64, pos_offset=0,
            return_kv=False):
    """Whole-sequence forward of one request.

    Returns (Hhat [n,d], logits [len(logit_rows), V]).  Hhat is the output of
    the final RMSNorm (the hidden states of the last layer that Section 2.1 pools); logits are computed
    for `logit_rows` only (all rows if None, none if empty).  `pos_offset`
    shifts every position by a constant (used by a rotary-invariance pin).
    With return_kv=True also returns per-layer (k_rotated, v) lists.
    """
    tokens = np.asarray(tokens, dtype=np.int64)
    n = tokens.shape[0]
    x = np.asarray(W.tok_emb)[tokens].astype(dtype)
    cos, sin = rope_cos_sin(cfg.Dh, cfg.rope_theta, np.arange(n) + pos_offset, dtype)
    kv = []
    for l in range(cfg.L):
        w = W.layer(l)
        h = rmsnorm(x, w["attn_norm"].astype(dtype), cfg.rms_eps)
        q = (h @ w["wq"].astype(dtype).T).reshape(n, cfg.Hq, cfg.Dh)
        k = (h @ w["wk"].astype(dtype).T).reshape(n, cfg.Hkv, cfg.Dh)
        v = (h @ w["wv"].astype(dtype).T).reshape(n, cfg.Hkv, cfg.Dh)
        q = apply_rope(q, cos, sin)
        k = apply_rope(k, cos, sin)
        if return_kv:
            kv.append((k, v))
        o = causal_attention(q, k, v, cfg.Hq, cfg.Hkv).reshape(n, cfg.Hq * cfg.Dh)
        x = x + o @ w["wo"].astype(dtype).T
        h = rmsnorm(x, w["ffn_norm"].astype(dtype), cfg.rms_eps)
        act = silu(h @ w["wg"].astype(dtype).T) * (h @ w["wu"].astype(dtype).T)
        x = x + act @ w["wd"].astype(dtype).T
    hhat = rmsnorm(x, np.asarray(W.final_norm).astype(dtype), cfg.rms_eps)
    if logit_rows is None:
        logit_rows = np.arange(n)
    logit_rows = np.asarray(logit_rows, dtype=np.int64)
    if logit_rows.size:
        logits = hhat[logit_rows] @ np.asarray(W.lm_head).astype(dtype).T
    else:
        logits = np.zeros((0, cfg.V), dtype=dtype)
    if return_kv:
        return hhat, logits, kv
    return hhat, logits


class MergedLora:
    """Weights of the adapted model in the plain definition: every adapted
    projection W [out, in] becomes W + (alpha / r) B A with A [r, in] and
    B [out, r] (a low-rank update of the shared backbone, Section 2.1
    "Parameter sharing").  The embedding, the norm gains and the LM head are
    shared unchanged.  `adapters.factors(l, name) -> (A, B)`, `adapters.scale`
    = alpha / r.  Requests of the adapted type (embedding) run `forward` /
    `embed` on this object; requests of the other type run them on the base
    weights: that per-request choice is the whole of the row-type dependence.
    """

    TARGETS = ("wq", "wk", "wv", "wo", "wg", "wu", "wd")

    def __init__(self, W, adapters, dtype=np.float64):
        self.W, self.adapters, self.dtype = W, adapters, dtype
        self._layers = {}

    @property
    def tok_emb(self):
        return self.W.tok_emb

    @property
    def final_norm(self):
        return self.W.final_norm

    @property
    def lm_head(self):
        return self.W.lm_head

    def layer(self, l):
        if l not in self._layers:
            w = dict(self.W.layer(l))
            for name in self.TARGETS:
                A, B = self.adapters.factors(l, name)
                w[name] = (np.asarray(w[name]).astype(self.dtype)
                           + self.adapters.scale * (B.astype(self.dtype) @ A.astype(self.dtype)))
            self._layers[l] = w
        return self._layers[l]


def l2_normalise(e, eps=1e-12):
    """e / max(||e||_2, eps); the zero vector maps to zeros."""
    return e / max(float(np.sqrt(np.sum(e * e))), eps)


def embed(cfg, W, tokens, mode, dtype=np.float64):
    """Single-pass embedding of the whole text.

    mode "mean": (1/n) sum_t Hhat_t  (Eq. 1-2 with w = 1 and one chunk);
    mode "wmean": sum_t w_t Hhat_t / sum_t w_t with w_t = t + 1, the 1-based
    position (Eq. 1-2; the paper leaves the weights open, this is the reading
    taken); mode "last": Hhat_{n-1}; mode "cls": Hhat_0 (positional heads,
    Section 3.3); mode "max": the element-wise maximum over all rows of Hhat, the
    example taken here of an "arbitrary deterministic head" that needs every
    row at once (Section 3.3, buffered heads).  The pooled vector is
    L2-normalised.
    """
    hhat, _ = forward(cfg, W, tokens, logit_rows=[], dtype=dtype)
    if mode == "mean":
        e = np.sum(hhat, axis=0) / hhat.shape[0]
    elif mode == "wmean":
        w = np.arange(1, hhat.shape[0] + 1, dtype=hhat.dtype)
        e = np.sum(w[:, None] * hhat, axis=0) / np.sum(w)
    elif mode == "last":
        e = hhat[-1]
    elif mode == "cls":
        e = hhat[0]
    elif mode == "max":
        e = np.max(hhat, axis=0)
    else:
        raise ValueError(mode)
    return l2_normalise(e)


def argmax_lowest(row):
    """Index of the maximum; the lowest index wins ties."""
    return int(np.argmax(row))


def generate(cfg, W, prompt, steps, dtype=np.float64):
    """Greedy generation by full-sequence recompute.

    Every step runs `forward` on the entire current sequence and appends the
    argmax of the last row.  Returns (new_tokens [steps], logits [steps, V]).
    """
    seq = [int(t) for t in prompt]
    out_tokens = []
    out_logits = []
    for _ in range(steps):
        _, lg = forward(cfg, W, seq, logit_rows=[len(seq) - 1], dtype=dtype)
        t = argmax_lowest(lg[0])
        out_tokens.append(t)
        out_logits.append(lg[0])
        seq.append(t)
    return np.asarray(out_tokens, dtype=np.int64), np.stack(out_logits)

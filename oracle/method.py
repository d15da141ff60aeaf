"""The method restated step by step (test infrastructure only; see package doc).

Where `transformer` computes the plain result, this module takes the method's
own steps in the paper's order and notation, so the method's invariants can be
brute-forced on small shapes:

* a request is executed as K chunks of sizes c_1..c_K over successive
  iterations (chunked embedding, Section 3.2; Section 3.3, first paragraph);
  chunk k attends causally over the K/V its request produced in chunks 1..k-1
  plus its own rows;
* the incremental pooler keeps S and W per request and applies
      S^(k) = S^(k-1) + sum_j w_{k,j} H_j^(k),   S^(0) = 0        (Eq. 1)
      W^(k) = W^(k-1) + sum_j w_{k,j},           W^(0) = 0        (Eq. 2)
  emitting S^(K)/W^(K) after the final chunk; mean pooling is w = 1; the
  positional heads keep one row: CLS H_1^(1), last token H_{c_K}^(K); a
  head that needs all rows buffers A^(k) = [A^(k-1); H^(k)] and runs after
  the final chunk (element-wise max is the example used);
* with a shared backbone, rows of embedding requests carry a low-rank
  adapter on every projection and rows of generation requests do not
  (Section 2.1 "Parameter sharing", Section 5.1): taken here as the
  unmerged two-branch product per request;
* a decode token is a chunk of one row whose logits are wanted
  (Section 3.2: a decode step contributes a single token of its request).

GPU results are never compared with this module's floating-point outputs;
they are compared with `transformer`.  The integer helpers at the bottom
(page slot map, pool counters) ARE the expected values for the bit-exact
bookkeeping checks.
"""
import numpy as np

from .transformer import rmsnorm, rope_cos_sin, apply_rope, silu, l2_normalise


class RequestState:
    """What one request carries across iterations: per-layer K/V rows so far,
    and the pooler state (S, W, retained row)."""

    def __init__(self, cfg, dtype=np.float64):
        self.n_cached = 0
        self.k = [np.zeros((0, cfg.Hkv, cfg.Dh), dtype=dtype) for _ in range(cfg.L)]
        self.v = [np.zeros((0, cfg.Hkv, cfg.Dh), dtype=dtype) for _ in range(cfg.L)]
        self.S = np.zeros(cfg.d, dtype=dtype)      # Eq. 1, S^(0) = 0
        self.W = 0.0                               # Eq. 2, W^(0) = 0
        self.count = 0                             # integer token count (mean: equals W)
        self.chunks = 0
        self.retained = None
        self.A = np.zeros((0, cfg.d), dtype=dtype)  # buffered heads: A^(0) is empty


def _proj(h, w, name, lora, l, dtype):
    """One projection of this request's rows.  Base: h W^T.  With an adapter
    (requests of the adapted type only) the low-rank branch is taken as two
    thin products and added, never merged into W:
        y = h W^T + (alpha / r) (h A^T) B^T."""
    y = h @ w[name].astype(dtype).T
    if lora is not None:
        A, B = lora.factors(l, name)
        y = y + lora.scale * ((h @ A.astype(dtype).T) @ B.astype(dtype).T)
    return y


def chunk_forward(cfg, W, st, tokens, dtype=np.float64, lora=None):
    """One iteration's rows of one request: c = len(tokens) new rows at
    positions st.n_cached .. st.n_cached+c-1.  Appends their K/V to the
    request's lists and returns the final-normed hidden states H^(k) [c, d].
    `lora`: adapter factors applied to this request's rows (embedding
    requests in the shared-backbone deployment), None for base-model rows."""
    tokens = np.asarray(tokens, dtype=np.int64)
    c = tokens.shape[0]
    p0 = st.n_cached
    x = np.asarray(W.tok_emb)[tokens].astype(dtype)
    cos, sin = rope_cos_sin(cfg.Dh, cfg.rope_theta, np.arange(p0, p0 + c), dtype)
    group = cfg.Hq // cfg.Hkv
    scale = 1.0 / np.sqrt(np.asarray(cfg.Dh, dtype=dtype))
    for l in range(cfg.L):
        w = W.layer(l)
        h = rmsnorm(x, w["attn_norm"].astype(dtype), cfg.rms_eps)
        q = apply_rope(_proj(h, w, "wq", lora, l, dtype).reshape(c, cfg.Hq, cfg.Dh), cos, sin)
        k = apply_rope(_proj(h, w, "wk", lora, l, dtype).reshape(c, cfg.Hkv, cfg.Dh), cos, sin)
        v = _proj(h, w, "wv", lora, l, dtype).reshape(c, cfg.Hkv, cfg.Dh)
        st.k[l] = np.concatenate([st.k[l], k], axis=0)
        st.v[l] = np.concatenate([st.v[l], v], axis=0)
        o = np.empty((c, cfg.Hq, cfg.Dh), dtype=dtype)
        for j in range(c):
            n_vis = p0 + j + 1                     # keys 0 .. p0+j
            for a in range(cfg.Hq):
                b = a // group
                s = (st.k[l][:n_vis, b, :] @ q[j, a, :]) * scale
                s = s - np.max(s)
                p = np.exp(s)
                p = p / np.sum(p)
                o[j, a, :] = p @ st.v[l][:n_vis, b, :]
        x = x + _proj(o.reshape(c, cfg.Hq * cfg.Dh), w, "wo", lora, l, dtype)
        h = rmsnorm(x, w["ffn_norm"].astype(dtype), cfg.rms_eps)
        act = silu(_proj(h, w, "wg", lora, l, dtype)) * _proj(h, w, "wu", lora, l, dtype)
        x = x + _proj(act, w, "wd", lora, l, dtype)
    st.n_cached = p0 + c
    return rmsnorm(x, np.asarray(W.final_norm).astype(dtype), cfg.rms_eps)


def pool_update(st, H, mode, is_final, weights=None):
    """Incremental pooler for one chunk's hidden states H [c, d].

    Additive heads (Eq. 1-2): form the chunk's weighted partial sum, then add
    it to S once; W grows by the chunk's weight sum.  Positional heads keep
    one row.  Returns the L2-normalised embedding on the final chunk, else
    None."""
    c = H.shape[0]
    first = st.chunks == 0
    st.chunks += 1
    st.count += c
    if mode == "mean" or mode == "wmean":
        w = np.ones(c, dtype=H.dtype) if weights is None else np.asarray(weights, dtype=H.dtype)
        st.S = st.S + np.sum(w[:, None] * H, axis=0)          # Eq. 1
        st.W = st.W + float(np.sum(w))                         # Eq. 2
        if is_final:
            return l2_normalise(st.S / st.W)
    elif mode == "last":
        if is_final:
            st.retained = H[c - 1].copy()                      # H_{c_K}^(K)
            return l2_normalise(st.retained)
    elif mode == "cls":
        if first:
            st.retained = H[0].copy()                          # H_1^(1)
        if is_final:
            return l2_normalise(st.retained)
    elif mode == "max":
        # buffered head: A^(k) = [A^(k-1); H^(k)], the head runs once over all n rows
        st.A = np.concatenate([st.A, H], axis=0)
        if is_final:
            return l2_normalise(np.max(st.A, axis=0))
    else:
        raise ValueError(mode)
    return None


def embed_chunked(cfg, W, tokens, sizes, mode, dtype=np.float64, lora=None):
    """Chunked embedding with incremental pooling: one chunk per iteration."""
    assert sum(sizes) == len(tokens) and all(c > 0 for c in sizes)
    st = RequestState(cfg, dtype)
    at = 0
    out = None
    for k, c in enumerate(sizes):
        H = chunk_forward(cfg, W, st, tokens[at:at + c], dtype, lora)
        # position weights w_{k,j} = 1-based position of row j of chunk k in the whole text
        w = np.arange(at + 1, at + c + 1) if mode == "wmean" else None
        out = pool_update(st, H, mode, is_final=(k == len(sizes) - 1), weights=w)
        at += c
    return out, st


def prefill_then_decode(cfg, W, prompt, sizes, steps, dtype=np.float64, forced=None):
    """Prompt in prefill chunks, then `steps` single-row decode iterations over
    the cached K/V.  Greedy (lowest index on ties) unless `forced` gives the
    tokens to feed.  Returns (tokens [steps], logits [steps, V])."""
    st = RequestState(cfg, dtype)
    at = 0
    H = None
    for c in sizes:
        H = chunk_forward(cfg, W, st, prompt[at:at + c], dtype)
        at += c
    lm = np.asarray(W.lm_head).astype(dtype)
    toks, lgs = [], []
    lg = H[-1] @ lm.T
    for s in range(steps):
        t = int(np.argmax(lg))
        toks.append(t)
        lgs.append(lg)
        if s + 1 < steps:
            feed = t if forced is None else int(forced[s])
            H = chunk_forward(cfg, W, st, [feed], dtype)
            lg = H[-1] @ lm.T
    return np.asarray(toks, dtype=np.int64), np.stack(lgs)


# ---------------------------------------------------------------------------
# Integer bookkeeping (expected values for the bit-exact checks)
# ---------------------------------------------------------------------------

def kv_slot(page_table, pos, page_size):
    """Where the K/V row of position `pos` of a request lives: the request's
    page list maps block pos // page_size to a physical page; the row sits at
    slot pos % page_size of that page."""
    return int(page_table[pos // page_size]), int(pos % page_size)


def pages_needed(n_tokens, page_size):
    return (n_tokens + page_size - 1) // page_size


def pool_counters_after(sizes_done):
    """(count, chunks) of a pool slot after the listed chunk sizes."""
    return int(sum(sizes_done)), len(sizes_done)

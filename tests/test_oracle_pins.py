"""Pins for the CPU oracle: library routines, closed forms, invariants, brute force.

None of these retypes the oracle's own formula; each compares it with
something fixed from outside: a torch / transformers library routine, a
hand-derivable closed form, a mathematical invariant, or the method's own
equivalence claims (Section 3.3: incremental == single-pass pooling;
Section 3.1: the forward is the same for every request type).
"""
import itertools
import types

import numpy as np
import pytest
import torch

from oracle import method as M
from oracle import scalar as S
from oracle import transformer as T
from paper_2609_25405_b200 import synth

TINY = synth.SHAPES["tiny"]
MICRO = synth.ModelShape("micro", 2, 16, 4, 2, 4, 24, 32)       # GQA group 2
MICRO1 = synth.ModelShape("micro1", 1, 8, 2, 2, 4, 8, 16)


def _w(shape, seed=0, std=0.02):
    return synth.Weights(shape, seed, std)


# --------------------------------------------------------------------------
# library-routine pins
# --------------------------------------------------------------------------

def _torch_forward(cfg, W, tokens):
    """The same model assembled from torch library routines only
    (embedding, rms_norm, linear, scaled_dot_product_attention, silu); the
    rotary step uses complex multiplication, a different formulation of the
    same rotation."""
    F = torch.nn.functional
    tt = lambda a: torch.from_numpy(np.asarray(a, dtype=np.float64))
    n = len(tokens)
    x = F.embedding(torch.as_tensor(np.asarray(tokens)), tt(W.tok_emb))
    half = cfg.Dh // 2
    inv = cfg.rope_theta ** (-torch.arange(half, dtype=torch.float64) * 2.0 / cfg.Dh)
    ang = torch.arange(n, dtype=torch.float64)[:, None] * inv[None, :]
    rot = torch.polar(torch.ones_like(ang), ang)                 # e^{i angle}

    def rope(z):                                                 # z [n,H,Dh]
        zc = torch.complex(z[..., :half], z[..., half:]) * rot[:, None, :]
        return torch.cat([zc.real, zc.imag], dim=-1)

    for l in range(cfg.L):
        w = {k: tt(v) for k, v in W.layer(l).items()}
        h = F.rms_norm(x, (cfg.d,), w["attn_norm"], cfg.rms_eps)
        q = rope(F.linear(h, w["wq"]).view(n, cfg.Hq, cfg.Dh))
        k = rope(F.linear(h, w["wk"]).view(n, cfg.Hkv, cfg.Dh))
        v = F.linear(h, w["wv"]).view(n, cfg.Hkv, cfg.Dh)
        o = F.scaled_dot_product_attention(q.transpose(0, 1)[None], k.transpose(0, 1)[None],
                                           v.transpose(0, 1)[None], is_causal=True,
                                           enable_gqa=True)[0]
        x = x + F.linear(o.transpose(0, 1).reshape(n, cfg.Hq * cfg.Dh), w["wo"])
        h = F.rms_norm(x, (cfg.d,), w["ffn_norm"], cfg.rms_eps)
        x = x + F.linear(F.silu(F.linear(h, w["wg"])) * F.linear(h, w["wu"]), w["wd"])
    hh = F.rms_norm(x, (cfg.d,), tt(W.final_norm), cfg.rms_eps)
    return hh.numpy(), F.linear(hh, tt(W.lm_head)).numpy()


@pytest.mark.parametrize("shape,n", [(MICRO, 11), (TINY, 37)])
def test_forward_matches_torch_library_routines(shape, n):
    W = _w(shape, 3, std=0.2 if shape is MICRO else 0.02)
    toks = synth.token_ids(np.random.default_rng(5), n, shape.V)
    hh, lg = T.forward(shape, W, toks)
    hh_t, lg_t = _torch_forward(shape, W, toks)
    # the oracle holds cos/sin at float32 precision (6e-8 relative), torch here in binary64
    assert np.max(np.abs(hh - hh_t)) < 1e-6
    assert np.max(np.abs(lg - lg_t)) < 1e-6


def test_forward_matches_transformers_llama():
    """An independent implementation of the same model family: a randomly
    initialised LlamaForCausalLM from the installed `transformers`, loaded
    with the same weights."""
    tr = pytest.importorskip("transformers")
    cfg = synth.ModelShape("hf", 2, 64, 4, 2, 16, 96, 50)
    W = _w(cfg, 7, std=0.1)
    hf_cfg = tr.LlamaConfig(vocab_size=cfg.V, hidden_size=cfg.d, intermediate_size=cfg.F,
                            num_hidden_layers=cfg.L, num_attention_heads=cfg.Hq,
                            num_key_value_heads=cfg.Hkv, head_dim=cfg.Dh,
                            rms_norm_eps=cfg.rms_eps, rope_theta=cfg.rope_theta,
                            attention_bias=False, mlp_bias=False, tie_word_embeddings=False,
                            max_position_embeddings=128, attn_implementation="eager")
    model = tr.LlamaForCausalLM(hf_cfg).double().eval()
    tt = lambda a: torch.from_numpy(np.asarray(a, dtype=np.float64))
    sd = {"model.embed_tokens.weight": tt(W.tok_emb), "model.norm.weight": tt(W.final_norm),
          "lm_head.weight": tt(W.lm_head)}
    names = {"attn_norm": "input_layernorm", "ffn_norm": "post_attention_layernorm",
             "wq": "self_attn.q_proj", "wk": "self_attn.k_proj", "wv": "self_attn.v_proj",
             "wo": "self_attn.o_proj", "wg": "mlp.gate_proj", "wu": "mlp.up_proj",
             "wd": "mlp.down_proj"}
    for l in range(cfg.L):
        for k, v in W.layer(l).items():
            sd[f"model.layers.{l}.{names[k]}.weight"] = tt(v)
    missing = model.load_state_dict(sd, strict=False)
    assert not [m for m in missing.missing_keys if "rotary" not in m]
    toks = synth.token_ids(np.random.default_rng(11), 23, cfg.V)
    with torch.no_grad():
        out = model(torch.as_tensor(toks)[None], output_hidden_states=True)
    _, lg = T.forward(cfg, W, toks)
    assert np.max(np.abs(lg - out.logits[0].numpy())) < 1e-6


def test_l2_normalise_matches_torch_and_zero_vector():
    e = np.random.default_rng(0).standard_normal(33)
    ref = torch.nn.functional.normalize(torch.from_numpy(e), dim=0, eps=1e-12).numpy()
    assert np.allclose(T.l2_normalise(e), ref, atol=1e-15)
    assert np.all(T.l2_normalise(np.zeros(5)) == 0.0)


# --------------------------------------------------------------------------
# brute force with scalar loops
# --------------------------------------------------------------------------

@pytest.mark.parametrize("shape,n", [(MICRO1, 5), (MICRO, 6)])
def test_forward_matches_scalar_loops(shape, n):
    W = _w(shape, 1, std=0.3)
    toks = synth.token_ids(np.random.default_rng(2), n, shape.V)
    hh, lg = T.forward(shape, W, toks)
    hh_s, lg_s = S.forward_loops(shape, W, toks)
    # the array code keeps cos/sin at float32 precision; the loops use binary64
    assert np.max(np.abs(hh - np.array(hh_s))) < 5e-6
    assert np.max(np.abs(lg - np.array(lg_s))) < 5e-6


# --------------------------------------------------------------------------
# closed forms and invariants of the building blocks
# --------------------------------------------------------------------------

class _HandWeights:
    """Wq = Wk = 0 (uniform attention), Wv = Wo = I, FFN off (Wd = 0)."""

    def __init__(self, cfg, emb):
        self.cfg = cfg
        self.tok_emb = emb
        self.final_norm = np.ones(cfg.d)
        self.lm_head = np.eye(cfg.V, cfg.d)

    def layer(self, l):
        c = self.cfg
        eye = np.eye(c.d)
        return dict(attn_norm=np.ones(c.d), wq=np.zeros((c.Hq * c.Dh, c.d)),
                    wk=np.zeros((c.Hkv * c.Dh, c.d)), wv=eye, wo=eye, ffn_norm=np.ones(c.d),
                    wg=np.ones((c.F, c.d)), wu=np.ones((c.F, c.d)), wd=np.zeros((c.d, c.F)))


def test_uniform_attention_closed_form():
    """With zero queries every visible key has weight 1/(t+1); with identity
    value/output projections and the FFN off, one layer gives
    x_t + mean_{s<=t} unit(x_s), unit(x) = x / sqrt(mean(x^2) + eps)."""
    cfg = synth.ModelShape("hand", 1, 8, 2, 2, 4, 4, 6)
    emb = np.random.default_rng(4).standard_normal((cfg.V, cfg.d))
    W = _HandWeights(cfg, emb)
    toks = [3, 1, 4, 1, 5]
    hh, _ = T.forward(cfg, W, toks)
    x = emb[toks]
    unit = x / np.sqrt(np.mean(x * x, axis=1, keepdims=True) + cfg.rms_eps)
    run_mean = np.cumsum(unit, axis=0) / np.arange(1, len(toks) + 1)[:, None]
    y = x + run_mean
    expect = y / np.sqrt(np.mean(y * y, axis=1, keepdims=True) + cfg.rms_eps)
    assert np.max(np.abs(hh - expect)) < 1e-12


def test_rope_identity_norm_and_known_angle():
    Dh = 8
    x = np.random.default_rng(0).standard_normal((3, 2, Dh))
    cos, sin = T.rope_cos_sin(Dh, 1e4, [0, 0, 0], np.float64)
    assert np.array_equal(T.apply_rope(x, cos, sin), x)            # position 0 = identity
    cos, sin = T.rope_cos_sin(Dh, 1e4, [5, 77, 4000], np.float64)
    y = T.apply_rope(x, cos, sin)
    assert np.allclose(np.sum(y * y, -1), np.sum(x * x, -1), rtol=1e-6)
    # frequency 0 has angle = position: a unit vector on pair (0, Dh/2) at
    # position p lands on (cos p, sin p)
    e = np.zeros((1, 1, Dh)); e[0, 0, 0] = 1.0
    cos, sin = T.rope_cos_sin(Dh, 1e4, [2], np.float64)
    r = T.apply_rope(e, cos, sin)[0, 0]
    assert abs(r[0] - np.cos(2.0)) < 1e-7 and abs(r[Dh // 2] - np.sin(2.0)) < 1e-7
    # last frequency: theta^(-(Dh-2)/Dh)
    e = np.zeros((1, 1, Dh)); e[0, 0, Dh // 2 - 1] = 1.0
    cos, sin = T.rope_cos_sin(Dh, 1e4, [1000], np.float64)
    r = T.apply_rope(e, cos, sin)[0, 0]
    a = 1000.0 * 1e4 ** (-(Dh - 2) / Dh)
    assert abs(r[Dh // 2 - 1] - np.cos(a)) < 1e-6 and abs(r[Dh - 1] - np.sin(a)) < 1e-6


def test_rope_is_relative():
    """Shifting all positions of a request by a constant leaves outputs
    unchanged (scores depend on position differences only)."""
    W = _w(MICRO, 9, std=0.2)
    toks = synth.token_ids(np.random.default_rng(1), 9, MICRO.V)
    a, la = T.forward(MICRO, W, toks)
    b, lb = T.forward(MICRO, W, toks, pos_offset=37)
    assert np.max(np.abs(a - b)) < 1e-5      # cos/sin are float32-rounded


def test_rmsnorm_scale_invariance_and_value():
    x = np.random.default_rng(0).standard_normal((4, 16))
    g = np.random.default_rng(1).standard_normal(16)
    assert np.allclose(T.rmsnorm(x, g, 0.0), T.rmsnorm(7.5 * x, g, 0.0), atol=1e-12)
    y = T.rmsnorm(np.full((1, 4), 3.0), np.ones(4), 0.0)
    assert np.allclose(y, 1.0)


def test_causality_prefix_property():
    """Row t of a forward over n tokens equals row t of a forward over the
    first t+1 tokens (no key beyond t is visible)."""
    W = _w(MICRO, 2, std=0.2)
    toks = synth.token_ids(np.random.default_rng(3), 10, MICRO.V)
    full, lg = T.forward(MICRO, W, toks)
    for t in (0, 3, 9):
        part, lgp = T.forward(MICRO, W, toks[:t + 1])
        assert np.max(np.abs(full[t] - part[t])) < 1e-12
        assert np.max(np.abs(lg[t] - lgp[t])) < 1e-12


def test_gqa_head_mapping_against_expanded_mha():
    """Grouped-query attention equals multi-head attention with each KV head
    repeated Hq/Hkv times consecutively."""
    rng = np.random.default_rng(0)
    n, Hq, Hkv, Dh = 7, 4, 2, 4
    q = rng.standard_normal((n, Hq, Dh)); k = rng.standard_normal((n, Hkv, Dh))
    v = rng.standard_normal((n, Hkv, Dh))
    a = T.causal_attention(q, k, v, Hq, Hkv)
    b = T.causal_attention(q, np.repeat(k, 2, axis=1), np.repeat(v, 2, axis=1), Hq, Hq)
    assert np.array_equal(a, b)


# --------------------------------------------------------------------------
# the method's invariants, brute-forced
# --------------------------------------------------------------------------

def _compositions(n):
    for cuts in itertools.product([0, 1], repeat=n - 1):
        sizes, run = [], 1
        for c in cuts:
            if c:
                sizes.append(run); run = 1
            else:
                run += 1
        sizes.append(run)
        yield sizes


@pytest.mark.parametrize("mode", ["mean", "last", "cls", "wmean", "max"])
def test_invariant1_every_partition_equals_single_pass(mode):
    """Chunked execution with the incremental pooler equals the single-pass
    embedding for EVERY ordered partition of a 7-token text."""
    W = _w(MICRO, 4, std=0.2)
    toks = synth.token_ids(np.random.default_rng(8), 7, MICRO.V)
    ref = T.embed(MICRO, W, toks, mode)
    for sizes in _compositions(7):
        e, st = M.embed_chunked(MICRO, W, toks, sizes, mode)
        cos = float(e @ ref)
        assert cos > 1 - 1e-9 and np.max(np.abs(e - ref)) < 1e-6, sizes
        assert (st.count, st.chunks) == M.pool_counters_after(sizes)


@pytest.mark.parametrize("mode", ["mean", "last"])
def test_invariant1_random_partitions_tiny_config(mode):
    W = _w(TINY)
    wl = synth.cfg1_workload()
    rng = np.random.default_rng(0)
    for toks in wl.embed_tokens:
        ref = T.embed(TINY, W, toks, mode)
        parts = [synth.nominal_chunks(len(toks), 32), [1] * 3 + [len(toks) - 3],
                 synth.random_partition(rng, len(toks), 40)]
        for sizes in parts:
            e, _ = M.embed_chunked(TINY, W, toks, sizes, mode)
            assert float(e @ ref) > 1 - 1e-9 and np.max(np.abs(e - ref)) < 1e-6


def test_pool_state_closed_form_after_each_chunk():
    """After chunk k the pooler state equals the sum (and count) of the first
    c_1+..+c_k final hidden states of the single-pass forward (Eq. 1-2)."""
    W = _w(MICRO, 4, std=0.2)
    toks = synth.token_ids(np.random.default_rng(8), 12, MICRO.V)
    hh, _ = T.forward(MICRO, W, toks, logit_rows=[])
    st = M.RequestState(MICRO)
    at = 0
    for k, c in enumerate([5, 1, 4, 2]):
        H = M.chunk_forward(MICRO, W, st, toks[at:at + c])
        M.pool_update(st, H, "mean", is_final=(k == 3))
        at += c
        assert st.count == at and st.W == float(at) and st.chunks == k + 1
        assert np.max(np.abs(st.S - hh[:at].sum(0))) < 1e-6


def test_position_weighted_mean_closed_form():
    """With w_t = t + 1 the total weight of n tokens is n (n + 1) / 2, and for hidden states that
    grow linearly with the position, H_t = (t + 1) u, the pooled vector is (2n + 1) / 3 * u."""
    n, u = 11, np.array([0.5, -2.0, 1.25])
    H = np.arange(1, n + 1)[:, None] * u[None, :]
    st = types.SimpleNamespace(S=np.zeros(3), W=0.0, count=0, chunks=0, retained=None)
    M.pool_update(st, H[:4], "wmean", False, np.arange(1, 5))
    e = M.pool_update(st, H[4:], "wmean", True, np.arange(5, n + 1))
    assert st.W == n * (n + 1) / 2
    pooled = (2 * n + 1) / 3.0 * u
    assert np.allclose(e, pooled / np.linalg.norm(pooled), atol=1e-12)


def test_weighted_mean_matches_direct_formula():
    rng = np.random.default_rng(0)
    H = rng.standard_normal((9, 5)); w = rng.random(9) + 0.1
    st = types.SimpleNamespace(S=np.zeros(5), W=0.0, count=0, chunks=0, retained=None)
    M.pool_update(st, H[:4], "wmean", False, w[:4])
    e = M.pool_update(st, H[4:], "wmean", True, w[4:])
    direct = (w[:, None] * H).sum(0) / w.sum()
    assert np.allclose(e, direct / np.linalg.norm(direct), atol=1e-12)


def test_buffered_max_head_closed_form():
    """Buffered head (Section 3.3): the buffer after chunk k holds the first c_1+..+c_k rows in order,
    and the element-wise maximum of hand-written rows is known."""
    H = np.array([[1.0, -5.0, 0.0], [-2.0, -1.0, 0.5], [0.5, -3.0, 4.0], [0.0, -9.0, -1.0]])
    st = types.SimpleNamespace(S=np.zeros(3), W=0.0, count=0, chunks=0, retained=None, A=np.zeros((0, 3)))
    assert M.pool_update(st, H[:1], "max", False) is None
    assert M.pool_update(st, H[1:3], "max", False) is None
    assert np.array_equal(st.A, H[:3])
    e = M.pool_update(st, H[3:], "max", True)
    assert np.array_equal(st.A, H) and (st.count, st.chunks) == (4, 3)
    pooled = np.array([1.0, -1.0, 4.0])
    assert np.allclose(e, pooled / np.sqrt(18.0), atol=1e-15)
    # the single-pass form on a real forward: max over rows of the final hidden states
    W = _w(MICRO, 4, std=0.2)
    toks = synth.token_ids(np.random.default_rng(3), 9, MICRO.V)
    hh, _ = T.forward(MICRO, W, toks, logit_rows=[])
    m = hh.max(0)
    assert np.allclose(T.embed(MICRO, W, toks, "max"), m / np.linalg.norm(m), atol=1e-14)


# --------------------------------------------------------------------------
# low-rank adapters on the shared backbone
# --------------------------------------------------------------------------

class _HandAdapters:
    """Rank-1 factors written by hand for one projection; zero elsewhere."""
    scale = 2.0

    def __init__(self, shape, name, a, b):
        self.shape, self.name, self.a, self.b = shape, name, np.asarray(a, float), np.asarray(b, float)
        self._ref = synth.LoraAdapters(shape, 1)

    def factors(self, l, name):
        out, inn = self._ref._dims(name)
        if name == self.name and l == 0:
            return self.a.reshape(1, inn), self.b.reshape(out, 1)
        return np.zeros((1, inn)), np.zeros((out, 1))


def test_merged_adapter_rank1_by_hand():
    """W + (alpha / r) B A for r = 1 is W + s b a^T: entry (i, j) grows by s b_i a_j.  On the
    non-square key projection a transposed factor cannot even be formed."""
    cfg = MICRO1                                   # d = 8, Hkv * Dh = 8, F = 8: use the gate [F, d]
    W = _w(cfg, 1)
    a = np.arange(1, cfg.d + 1) * 0.5              # [in]
    b = np.array([1.0, -1.0, 2.0, 0.0, 0.0, 3.0, 0.0, -2.0])   # [out = F]
    mw = T.MergedLora(W, _HandAdapters(cfg, "wg", a, b)).layer(0)
    base = W.layer(0)
    assert np.array_equal(mw["wq"], np.asarray(base["wq"], dtype=np.float64))     # zero factors change nothing
    delta = mw["wg"] - base["wg"]
    assert np.allclose(delta[2], 2.0 * 2.0 * a, atol=1e-12)      # row i = s b_i a
    assert np.allclose(delta[:, 3], 2.0 * b * 2.0, atol=1e-12)   # column j = s a_j b, a_3 = 2.0
    assert np.allclose(delta[3], 0.0) and np.allclose(delta[7, 0], 2.0 * -2.0 * 0.5)
    shapes = {n: synth.LoraAdapters(MICRO, 3).factors(1, n) for n in synth.LORA_TARGETS}
    assert shapes["wk"][0].shape == (3, MICRO.d) and shapes["wk"][1].shape == (MICRO.Hkv * MICRO.Dh, 3)
    assert shapes["wd"][0].shape == (3, MICRO.F) and shapes["wd"][1].shape == (MICRO.d, 3)


def test_zero_adapter_is_the_base_model():
    cfg, W = MICRO, _w(MICRO, 4, std=0.2)
    toks = synth.token_ids(np.random.default_rng(5), 9, cfg.V)
    ad = synth.LoraAdapters(cfg, 4, std=0.0)
    assert np.array_equal(T.embed(cfg, T.MergedLora(W, ad), toks, "mean"), T.embed(cfg, W, toks, "mean"))
    e, _ = M.embed_chunked(cfg, W, toks, [4, 5], "mean", lora=ad)
    e0, _ = M.embed_chunked(cfg, W, toks, [4, 5], "mean")
    assert np.array_equal(e, e0)


@pytest.mark.parametrize("rank", [1, 3, 8])
def test_two_branch_adapter_equals_merged_weights(rank):
    """The method's unmerged form, h W^T + s (h A^T) B^T on embedding rows, chunked, against the
    plain definition: one pass with the merged matrices.  The adapter must change the result
    (so the comparison is not vacuous) and a generation request must not see it."""
    cfg, W = MICRO, _w(MICRO, 4, std=0.2)
    ad = synth.LoraAdapters(cfg, rank, std=0.2)
    toks = synth.token_ids(np.random.default_rng(6), 10, cfg.V)
    for mode in ("mean", "last"):
        ref = T.embed(cfg, T.MergedLora(W, ad), toks, mode)
        base = T.embed(cfg, W, toks, mode)
        assert np.max(np.abs(ref - base)) > 1e-2
        for sizes in ([10], [3, 7], [1, 4, 5], [2] * 5):
            e, _ = M.embed_chunked(cfg, W, toks, sizes, mode, lora=ad)
            assert float(e @ ref) > 1 - 1e-9 and np.max(np.abs(e - ref)) < 1e-6, (mode, sizes)
    _, lg = M.prefill_then_decode(cfg, W, toks, [4, 6], 3)
    _, lg_ref = T.generate(cfg, W, toks, 3)
    assert np.max(np.abs(lg - lg_ref)) < 1e-6


def test_merged_adapter_forward_matches_torch_linear_pair():
    """The adapted model assembled from torch library routines with the two-branch linear
    (F.linear twice per projection), against the oracle's merged single pass."""
    cfg, W = MICRO, _w(MICRO, 2, std=0.2)
    ad = synth.LoraAdapters(cfg, 2, std=0.2)
    toks = synth.token_ids(np.random.default_rng(9), 8, cfg.V)

    class Two:
        tok_emb, final_norm, lm_head = W.tok_emb, W.final_norm, W.lm_head

        @staticmethod
        def layer(l):
            return W.layer(l)

    F = torch.nn.functional
    real_linear = F.linear
    tt = lambda a: torch.from_numpy(np.asarray(a, dtype=np.float64))
    state = {"l": 0, "i": 0}
    order = ["wq", "wk", "wv", "wo", "wg", "wu", "wd"]

    def lora_linear(x, w, *rest):
        # the projections of a layer are called in a fixed order by _torch_forward; the LM head comes last
        if state["l"] >= cfg.L:
            return real_linear(x, w)
        name = order[state["i"]]
        A, B = ad.factors(state["l"], name)
        y = real_linear(x, w) + ad.scale * real_linear(real_linear(x, tt(A)), tt(B))
        state["i"] += 1
        if state["i"] == len(order):
            state["i"], state["l"] = 0, state["l"] + 1
        return y

    F.linear = lora_linear
    try:
        hh_t, _ = _torch_forward(cfg, Two, toks)
    finally:
        F.linear = real_linear
    hh, _ = T.forward(cfg, T.MergedLora(W, ad), toks, logit_rows=[])
    # the oracle holds cos/sin in fp32 precision, the torch assembly in fp64: same bound as the base pin
    assert np.max(np.abs(hh - hh_t)) < 1e-6
    hh_base, _ = T.forward(cfg, W, toks, logit_rows=[])
    assert np.max(np.abs(hh - hh_base)) > 1e-2


def test_invariant3_decode_after_prefill_equals_full_forward():
    """For every prefix length: logits of a one-row decode iteration over the
    cached K/V equal the last row of a whole-sequence forward."""
    W = _w(MICRO, 6, std=0.2)
    toks = synth.token_ids(np.random.default_rng(9), 9, MICRO.V)
    _, lg = T.forward(MICRO, W, toks)
    lm = np.asarray(W.lm_head, dtype=np.float64)
    for n_pre in range(1, 9):
        st = M.RequestState(MICRO)
        M.chunk_forward(MICRO, W, st, toks[:n_pre])
        H = M.chunk_forward(MICRO, W, st, toks[n_pre:n_pre + 1])
        assert np.max(np.abs(H[0] @ lm.T - lg[n_pre])) < 1e-9


def test_generate_full_recompute_equals_cached_decode():
    W = _w(TINY)
    wl = synth.cfg1_workload()
    tk, lg = T.generate(TINY, W, wl.prompts[1], 4)
    tk2, lg2 = M.prefill_then_decode(TINY, W, wl.prompts[1], [32, 32], 4)
    assert np.array_equal(tk, tk2) and np.max(np.abs(lg - lg2)) < 1e-9


def test_invariant2_batch_composition_independence():
    """The oracle handles one request at a time, so a request's result cannot
    depend on its batch mates; check the interface has no hidden state."""
    W = _w(MICRO, 4, std=0.2)
    rng = np.random.default_rng(3)
    a = synth.token_ids(rng, 6, MICRO.V); b = synth.token_ids(rng, 9, MICRO.V)
    ea1 = T.embed(MICRO, W, a, "mean"); T.embed(MICRO, W, b, "last")
    ea2 = T.embed(MICRO, W, a, "mean")
    assert np.array_equal(ea1, ea2)


def test_argmax_lowest_index_on_ties():
    assert T.argmax_lowest(np.array([1.0, 3.0, 3.0, 2.0])) == 1


def test_kv_slot_map():
    pt = [7, 2, 9]
    assert M.kv_slot(pt, 0, 16) == (7, 0)
    assert M.kv_slot(pt, 15, 16) == (7, 15)
    assert M.kv_slot(pt, 16, 16) == (2, 0)
    assert M.kv_slot(pt, 40, 16) == (9, 8)
    assert M.pages_needed(0, 16) == 0 and M.pages_needed(16, 16) == 1 and M.pages_needed(17, 16) == 2


def test_fp32_oracle_close_to_fp64():
    W = _w(TINY)
    toks = synth.cfg1_workload().embed_tokens[1]
    a = T.embed(TINY, W, toks, "mean", dtype=np.float64)
    b = T.embed(TINY, W, toks, "mean", dtype=np.float32)
    assert np.max(np.abs(a - b)) < 1e-5


# --------------------------------------------------------------------------
# the single projection with its epilogues (oracle/ops.py), which the GEMM unit tests rest on
# --------------------------------------------------------------------------

def test_projection_epilogues_match_torch_linear_with_separate_gate_and_up():
    """ops.projection against torch: the plain product against F.linear, the residual form against
    C0 + F.linear, and the SwiGLU form against silu(F.linear(x, Wg)) * F.linear(x, Wu) with gate
    and up given as SEPARATE matrices that this test interleaves itself (row 2j = gate row j, row
    2j + 1 = up row j, the layout the library documents for w_gate_up).  Swapping gate and up,
    dropping the residual or transposing an operand in ops.projection fails here."""
    from oracle import ops
    import torch.nn.functional as Fn
    rng = np.random.default_rng(3)
    M_, K, F_ = 5, 12, 7
    x = rng.standard_normal((M_, K))
    wg, wu = rng.standard_normal((F_, K)), rng.standard_normal((F_, K))
    c0 = rng.standard_normal((M_, F_))
    tx, tg, tu = (torch.from_numpy(a) for a in (x, wg, wu))
    assert np.allclose(ops.projection(x, wg, "plain"), Fn.linear(tx, tg).numpy(), atol=1e-12)
    assert np.allclose(ops.projection(x, wg, "resid", c0), c0 + Fn.linear(tx, tg).numpy(), atol=1e-12)
    inter = np.empty((2 * F_, K))
    inter[0::2], inter[1::2] = wg, wu
    ref = (Fn.silu(Fn.linear(tx, tg)) * Fn.linear(tx, tu)).numpy()
    got = ops.projection(x, inter, "swiglu")
    assert got.shape == (M_, F_) and np.allclose(got, ref, atol=1e-12)
    swapped = np.empty_like(inter)
    swapped[0::2], swapped[1::2] = wu, wg
    assert not np.allclose(ops.projection(x, swapped, "swiglu"), ref, atol=1e-3)   # the order matters
    # the same inside the whole model: one FFN block of transformer.forward is this projection chain
    h = rng.standard_normal((M_, K))
    wd = rng.standard_normal((K, F_))
    ffn = ops.projection(ops.projection(h, inter, "swiglu"), wd, "resid", x)
    assert np.allclose(ffn, x + (T.silu(h @ wg.T) * (h @ wu.T)) @ wd.T, atol=1e-12)


def test_projection_two_by_two_by_hand():
    """A 2 x 2 case worked by hand.  A = [[1, 2], [0, -1]], B rows = (gate, up) = ([1, 0], [0, 1]):
    A B^T = A itself, so plain = A, resid with C0 = 10 everywhere = A + 10, and swiglu has one
    output column: silu(gate) * up = silu(1) * 2 and silu(0) * (-1) = 0 (silu(0) = 0,
    silu(1) = 1 / (1 + e^-1))."""
    from oracle import ops
    A = np.array([[1.0, 2.0], [0.0, -1.0]])
    Bm = np.array([[1.0, 0.0], [0.0, 1.0]])
    assert np.array_equal(ops.projection(A, Bm, "plain"), A)
    assert np.array_equal(ops.projection(A, Bm, "resid", np.full((2, 2), 10.0)), A + 10.0)
    sw = ops.projection(A, Bm, "swiglu")
    assert sw.shape == (2, 1)
    assert abs(sw[0, 0] - 2.0 / (1.0 + np.exp(-1.0))) < 1e-15 and sw[1, 0] == 0.0
    # a non-symmetric B tells A B^T from A B: B = [[1, 1], [0, 1]] gives rows (a0 + a1, a1)
    B2 = np.array([[1.0, 1.0], [0.0, 1.0]])
    assert np.array_equal(ops.projection(A, B2, "plain"), np.array([[3.0, 2.0], [-1.0, -1.0]]))


# --------------------------------------------------------------------------
# values the paper prints
# --------------------------------------------------------------------------

def _golden_rows(name):
    import os
    path = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden", name)
    return [ln.split() for ln in open(path) if ln.strip() and not ln.startswith("#")]


def test_printed_pooling_equivalence_bounds_hold_for_the_oracle():
    """The paper's table of chunked-versus-single-pass agreement (appendix "Pooling Equivalence": min
    cosine and p99 relative L2 per head and chunk size) is a ceiling any exact restatement must stay
    under: the oracle's chunked form at the same chunk sizes, on texts of several lengths."""
    cfg, W = MICRO, _w(MICRO, 4, std=0.2)
    rng = np.random.default_rng(12)
    texts = [synth.token_ids(rng, n, cfg.V) for n in (300, 1100)]
    rows = _golden_rows("pooling_equivalence.txt")
    assert len(rows) == 9
    for head, C, cos_min, _, _, _, l2_p99 in rows:
        for toks in texts:
            ref = T.embed(cfg, W, toks, head)
            e, _ = M.embed_chunked(cfg, W, toks, synth.nominal_chunks(len(toks), int(C)), head)
            assert float(e @ ref) >= float(cos_min)
            assert np.linalg.norm(e - ref) / np.linalg.norm(ref) <= float(l2_p99)

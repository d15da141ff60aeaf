"""Whole-sequence forward in pure Python loops (test infrastructure only).

The same computation as `transformer.forward`, written with scalar loops and
Python floats (binary64) so that no array indexing, broadcasting, transpose or
reshape convention is shared with it.  Tiny shapes only.  Library use is
limited to math.exp / sqrt / cos / sin.
"""
import math


def _matvec(w, x):
    """w [out][in] (nested lists), x [in] -> [out]."""
    return [sum(wr[i] * x[i] for i in range(len(x))) for wr in w]


def _rmsnorm(x, g, eps):
    ms = sum(v * v for v in x) / len(x)
    r = 1.0 / math.sqrt(ms + eps)
    return [x[i] * r * g[i] for i in range(len(x))]


def _rope(vec, pos, Dh, theta):
    """vec: one head [Dh]; pair (i, i+Dh/2) rotated by pos * theta^(-2i/Dh)."""
    half = Dh // 2
    out = [0.0] * Dh
    for i in range(half):
        ang = pos * theta ** (-2.0 * i / Dh)
        c, s = math.cos(ang), math.sin(ang)
        a, b = vec[i], vec[i + half]
        out[i] = a * c - b * s
        out[i + half] = b * c + a * s
    return out


def forward_loops(cfg, W, tokens):
    """Returns (Hhat, logits) as nested lists for the whole sequence."""
    n = len(tokens)
    tl = lambda a: a.tolist()
    x = [tl(W.tok_emb[int(t)]) for t in tokens]
    group = cfg.Hq // cfg.Hkv
    for l in range(cfg.L):
        w = {k: tl(v) for k, v in W.layer(l).items()}
        q, k, v = [], [], []
        for t in range(n):
            h = _rmsnorm(x[t], w["attn_norm"], cfg.rms_eps)
            qf, kf, vf = _matvec(w["wq"], h), _matvec(w["wk"], h), _matvec(w["wv"], h)
            q.append([_rope(qf[a * cfg.Dh:(a + 1) * cfg.Dh], t, cfg.Dh, cfg.rope_theta)
                      for a in range(cfg.Hq)])
            k.append([_rope(kf[b * cfg.Dh:(b + 1) * cfg.Dh], t, cfg.Dh, cfg.rope_theta)
                      for b in range(cfg.Hkv)])
            v.append([vf[b * cfg.Dh:(b + 1) * cfg.Dh] for b in range(cfg.Hkv)])
        for t in range(n):
            o = []
            for a in range(cfg.Hq):
                b = a // group
                sc = [sum(q[t][a][i] * k[s][b][i] for i in range(cfg.Dh)) / math.sqrt(cfg.Dh)
                      for s in range(t + 1)]
                m = max(sc)
                e = [math.exp(z - m) for z in sc]
                den = sum(e)
                o.extend(sum(e[s] / den * v[s][b][i] for s in range(t + 1))
                         for i in range(cfg.Dh))
            proj = _matvec(w["wo"], o)
            x[t] = [x[t][i] + proj[i] for i in range(cfg.d)]
            h = _rmsnorm(x[t], w["ffn_norm"], cfg.rms_eps)
            g, u = _matvec(w["wg"], h), _matvec(w["wu"], h)
            act = [g[i] / (1.0 + math.exp(-g[i])) * u[i] for i in range(cfg.F)]
            dn = _matvec(w["wd"], act)
            x[t] = [x[t][i] + dn[i] for i in range(cfg.d)]
    fn = tl(W.final_norm)
    lm = tl(W.lm_head)
    hhat = [_rmsnorm(x[t], fn, cfg.rms_eps) for t in range(n)]
    logits = [_matvec(lm, hhat[t]) for t in range(n)]
    return hhat, logits

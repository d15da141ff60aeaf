"""Full-size parity: the 1B-class and 7B-class shapes at their full depth and width, in the launch
configurations the benchmark times (full token budget per step, decode rows over long synthetic
contexts plus embedding chunks; for the 7B shape also one point of the embedding-fraction sweep with
2048 decode rows), checked on sampled requests the CPU oracle can recompute one by one.  Legitimate because a request's outputs do not depend on its batch mates (checked
bit for bit on the tiny shape, and here on one request run solo and inside the batch).

Sampled per shape: two generation requests (prompt prefilled in chunks through the library
itself, then teacher-forced decode steps) and two embedding requests (one single-chunk, one
multi-chunk) with last-token pooling as the configurations say, plus one multi-chunk request with
mean pooling.  The other rows are filler: decode
rows over contexts of random K/V and embedding chunks of random tokens.
"""
import os

import numpy as np
import pytest
import torch

from oracle import method as M
from oracle import transformer as T
from paper_2609_25405_b200 import synth

pytestmark = pytest.mark.gpu

EMB_COS, EMB_ABS, LOGIT_ABS = 0.9995, 2e-2, 5e-2
KV_SENTINEL = 0x7F7F

CASES = {
    # shape, decode rows, filler ctx range, budget, chunk, sampled gen prompts, sampled embed lengths
    "cfg2-1b": dict(shape="1b", n_decode=32, ctx=(128, 1024), budget=2048, chunk=256,
                    gen=(128, 600), emb=(200, 700), emb_mean=(450,), seed=1002, n_steps=4),
    "cfg3-7b": dict(shape="7b", n_decode=64, ctx=(512, 4096), budget=4096, chunk=512,
                    gen=(512, 1100), emb=(300, 700), emb_mean=(640,), seed=1003, n_steps=2),
    # one point of the embedding-fraction sweep (f = 0.5): 2048 decode rows at context 2048 next to
    # 2048 rows of mean-pooled embedding chunks.  Unaliased, the decode contexts alone would need
    # 550 GB of KV, so (as in the benchmark) filler row i reads the context pages of row i mod `alias`
    # and appends to a private tail page; 64 distinct contexts here (256 in the benchmark).
    "cfg4-7b-f0.5": dict(shape="7b", n_decode=2048, ctx=(2048, 2048), budget=4096, chunk=512,
                         gen=(2048,), emb=(), emb_mean=(1500,), seed=1004, n_steps=2, alias=64,
                         fill_len=(128, 2048), fill_mean=True),
}


def _threads():
    return max(4, min(32, os.cpu_count() or 8))


@pytest.mark.parametrize("name", ["cfg2-1b", "cfg3-7b", "cfg4-7b-f0.5"])
def test_fullsize_sampled_requests_match_oracle(name):
    from paper_2609_25405_b200 import binding as B
    from paper_2609_25405_b200.engine import Engine, Request
    c = CASES[name]
    shape = synth.SHAPES[c["shape"]]
    P = shape.page_size
    rng = np.random.default_rng(c["seed"])
    W = synth.Weights(shape, 0, cache="bits").prefetch(_threads())
    dw = B.DeviceWeights.from_synth(W)
    n_steps = c["n_steps"]       # logits rows compared per generation request (prefill row + decode rows)
    max_pos = c["ctx"][1] + n_steps + 8
    n_dec = c["n_decode"]
    alias = c.get("alias", 0)
    ctxs = rng.integers(c["ctx"][0], c["ctx"][1] + 1, size=n_dec - len(c["gen"]))
    own = ctxs if not alias else ctxs[:alias]
    n_pages = int(sum((x + n_steps + P) // P + 1 for x in own)) + 5 * (max_pos // P + 2) + \
        (n_steps + 4) * (c["budget"] // P + 80) + (2 * (len(ctxs) - alias) if alias else 0)
    eng = Engine(shape, dw, n_pages=n_pages, n_slots=256, max_tokens=c["budget"], max_segs=n_dec + 160,
                 max_pos=max_pos)
    # synthetic cached context for the filler rows: N(0,1) K/V everywhere, then sentinel on the pages
    # the sampled requests will own (so stray writes and wrong slots show)
    kvb = eng.kv.arena.view(torch.float16)
    for i in range(0, kvb.numel(), 1 << 28):
        kvb[i:i + (1 << 28)].normal_(0.0, 1.0)

    # ---- sampled requests ----
    gens = [Request("gen", synth.token_ids(rng, n, shape.V)) for n in c["gen"]]
    embs = [Request("embed", synth.token_ids(rng, n, shape.V), B.POOL_LAST) for n in c["emb"]]
    # one multi-chunk request with mean pooling (the sweep configuration's head) next to the last-token ones
    embs += [Request("embed", synth.token_ids(rng, n, shape.V), B.POOL_MEAN) for n in c["emb_mean"]]
    head = {B.POOL_LAST: "last", B.POOL_MEAN: "mean"}
    sampled_pages = {}
    for r in gens + embs:
        total = len(r.tokens) + n_steps + 1
        r.pages = eng.kv.alloc((total + P - 1) // P)
        sampled_pages[r] = list(r.pages)
    view = eng.kv.arena.view(shape.L, n_pages, shape.Hkv, 2, 2, shape.Dh // 64, 8, 64)
    for r in gens + embs:
        view[:, torch.tensor(r.pages)] = KV_SENTINEL
    # ---- filler ----
    fill_dec = []
    for i, x in enumerate(ctxs):
        r = Request("gen", synth.token_ids(rng, int(x) + 1, shape.V))
        r.n_prompt = int(x)
        r.n_done = int(x)
        if alias and i >= alias:
            assert int(x) % P == 0                      # whole context pages are shared, read-only
            r.pages = list(fill_dec[i % alias].pages[:int(x) // P])
        else:
            r.pages = eng.kv.alloc((int(x) + P - 1) // P)
        fill_dec.append(r)

    # ---- oracle (one whole-sequence forward per sampled request; fp32 as the benchmark spec says) ----
    ora_tok, ora_lg = {}, {}
    for g in gens:
        toks = list(g.tokens)
        n0 = len(toks)
        # greedy continuation by full recompute is what `generate` does; here the steps are few, so
        # recompute the whole sequence per step exactly as the definition says
        tk, lg = T.generate(shape, W, toks, n_steps, dtype=np.float32)
        ora_tok[g], ora_lg[g] = tk, lg
        assert n0 + n_steps <= max_pos
    ora_emb = {e: T.embed(shape, W, e.tokens, head[e.pool_mode], dtype=np.float32) for e in embs}

    # ---- run: every step is filled to the token budget ----
    got_lg = {g: [] for g in gens}
    got_emb = {}
    chunk = c["chunk"]
    inflight_fill = []
    for step in range(n_steps + 3 + max(c["gen"]) // chunk):
        work = []
        rows = 0
        for r in fill_dec:
            if r.remaining() == 0:
                r.tokens.append(int(rng.integers(0, shape.V)))
            work.append((r, 1)); rows += 1
        for g in gens:
            if g.in_decode:
                if len(got_lg[g]) >= n_steps:
                    continue
                g.tokens.append(int(ora_tok[g][len(got_lg[g]) - 1]))   # teacher forcing
                work.append((g, 1)); rows += 1
            else:
                q = min(chunk, g.remaining())
                work.append((g, q)); rows += q
        for e in embs:
            if e.remaining() > 0:
                q = min(chunk, e.remaining())
                work.append((e, q)); rows += q
        # filler embedding requests up to the budget
        nxt = []
        for f in inflight_fill:
            q = min(chunk, f.remaining(), c["budget"] - rows)
            if q > 0:
                work.append((f, q)); rows += q
            if f.remaining() - max(q, 0) > 0:
                nxt.append(f)
        while rows < c["budget"]:
            lo, hi = c.get("fill_len", (16, 2 * chunk - 1))
            n = int(rng.integers(lo, hi + 1))
            f = Request("embed", synth.token_ids(rng, n, shape.V), B.POOL_MEAN if c.get("fill_mean") else B.POOL_LAST)
            q = min(chunk, n, c["budget"] - rows)
            work.append((f, q)); rows += q
            if q < n:
                nxt.append(f)
        inflight_fill = nxt
        assert rows == c["budget"]
        batch, lrows, erows = eng.step(work)
        assert batch.n_tokens == c["budget"]
        torch.cuda.synchronize()
        for g in gens:
            if g in lrows:
                got_lg[g].append(eng.out_logits[lrows[g]].cpu().numpy().astype(np.float64))
        for e in embs:
            if e in erows:
                got_emb[e] = eng.out_emb[erows[e]].cpu().numpy().astype(np.float64)
        for f, _ in work:
            if f.kind == "embed" and f.finished and f not in embs:
                eng.release(f)
        if all(len(got_lg[g]) >= n_steps for g in gens) and len(got_emb) == len(embs):
            break
    assert eng.ctx.status_poll() == 0

    # ---- one sampled embedding request again, alone in its steps (same chunking): bit for bit the
    # result it had inside the full batches
    solo = Request("embed", list(embs[0].tokens), embs[0].pool_mode)
    while solo.remaining() > 0:
        _, _, er = eng.step([(solo, min(chunk, solo.remaining()))])
    torch.cuda.synchronize()
    assert np.array_equal(eng.out_emb[er[solo]].cpu().numpy().astype(np.float64), got_emb[embs[0]])
    eng.release(solo)
    assert eng.ctx.status_poll() == 0

    # ---- compare ----
    n_rows = n_agree = 0
    for g in gens:
        assert len(got_lg[g]) == n_steps
        for s in range(n_steps):
            ref = ora_lg[g][s].astype(np.float64)
            assert np.max(np.abs(got_lg[g][s] - ref)) <= LOGIT_ABS
            n_rows += 1
            n_agree += int(np.argmax(got_lg[g][s]) == np.argmax(ref))
    assert n_agree / n_rows >= 0.995, (n_agree, n_rows)
    for e in embs:
        got, ref = got_emb[e], ora_emb[e].astype(np.float64)
        cos = float(got @ ref / (np.linalg.norm(got) * np.linalg.norm(ref)))
        assert cos >= EMB_COS and np.max(np.abs(got - ref)) <= EMB_ABS, (cos, np.max(np.abs(got - ref)))
    # ---- bookkeeping on the sampled requests' pages: written slots hold values, the rest the sentinel
    raw = eng.kv.arena.view(shape.L, n_pages, shape.Hkv, 2, 2, shape.Dh // 64, 8, 64).permute(0, 1, 2, 4, 5, 3, 6, 7) \
        .reshape(shape.L, n_pages, shape.Hkv, 2, shape.Dh // 64, P, 64)      # slots back in order 0..15
    for r in gens + embs:
        n = r.n_done
        pages = sampled_pages[r]
        for blk, pg in enumerate(pages):
            written = max(0, min(P, n - blk * P))
            if written < P:
                assert torch.all(raw[:, pg, :, :, :, written:, :] == KV_SENTINEL), (blk, pg)
            if written > 0:
                assert not torch.any(raw[0, pg, :, :, :, :written, :] == KV_SENTINEL)
        cnt, chunks = M.pool_counters_after(synth.nominal_chunks(len(r.tokens), chunk)) if r.kind == "embed" else (0, 0)
        if r.kind == "embed":
            meta = eng.pool.meta()[r.slot].cpu().numpy()
            assert list(meta.astype(np.int64)) == [cnt, chunks, r.pool_mode, 1]
    eng.close()

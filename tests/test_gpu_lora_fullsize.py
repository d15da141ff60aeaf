"""Adapters at full size: the 1B-class shape at full depth and width, steps filled to the 2048-token
budget (decode rows over random cached context, embedding chunks), with a rank-16 adapter on the
embedding rows.  Sampled requests the CPU oracle recomputes: one multi-chunk embedding request
against the merged-weight model, one generation request (prefill, then teacher-forced decode steps)
against the base model."""
import os

import numpy as np
import pytest
import torch

from oracle import transformer as T
from paper_2609_25405_b200 import synth

pytestmark = pytest.mark.gpu

EMB_COS, EMB_ABS, LOGIT_ABS = 0.9995, 2e-2, 5e-2


def test_1b_adapter_sampled_requests_match_oracle():
    from paper_2609_25405_b200 import binding as B
    from paper_2609_25405_b200.engine import Engine, Request
    shape = synth.SHAPES["1b"]
    P, budget, chunk, n_dec, n_steps = shape.page_size, 2048, 256, 32, 3
    rng = np.random.default_rng(2002)
    W = synth.Weights(shape, 0, cache="bits").prefetch(max(4, min(32, os.cpu_count() or 8)))
    ad = synth.LoraAdapters(shape, 16, seed=5)
    dw = B.DeviceWeights.from_synth(W)
    lora = B.DeviceLora.from_synth(ad)
    max_pos = 1024 + n_steps + 8
    ctxs = rng.integers(128, 1025, size=n_dec - 1)
    n_pages = int(sum((x + n_steps + P) // P + 1 for x in ctxs)) + 4 * (max_pos // P + 2) + \
        (n_steps + 1) * (budget // P + 80)
    eng = Engine(shape, dw, n_pages=n_pages, n_slots=256, max_tokens=budget, max_segs=n_dec + 160,
                 max_pos=max_pos, lora=lora)
    kvb = eng.kv.arena.view(torch.float16)
    for i in range(0, kvb.numel(), 1 << 28):
        kvb[i:i + (1 << 28)].normal_(0.0, 1.0)
    emb = Request("embed", synth.token_ids(rng, 600, shape.V), B.POOL_LAST)
    gen = Request("gen", synth.token_ids(rng, 200, shape.V))
    fill_dec = []
    for x in ctxs:
        r = Request("gen", synth.token_ids(rng, int(x) + 1, shape.V))
        r.n_prompt = r.n_done = int(x)
        r.pages = eng.kv.alloc((int(x) + P - 1) // P)
        fill_dec.append(r)

    ora_tok, ora_lg = T.generate(shape, W, list(gen.tokens), n_steps, dtype=np.float32)
    ora_emb = T.embed(shape, T.MergedLora(W, ad, dtype=np.float32), emb.tokens, "last", dtype=np.float32)
    base_emb = T.embed(shape, W, emb.tokens, "last", dtype=np.float32)
    assert np.max(np.abs(ora_emb - base_emb)) > EMB_ABS       # the adapter is visible at this size

    got_lg, got_emb, inflight = [], None, []
    for step in range(n_steps):
        work, rows = [], 0
        for r in fill_dec:
            if r.remaining() == 0:
                r.tokens.append(int(rng.integers(0, shape.V)))
            work.append((r, 1)); rows += 1
        if gen.in_decode:
            gen.tokens.append(int(ora_tok[len(got_lg) - 1]))  # teacher forcing
            work.append((gen, 1)); rows += 1
        else:
            work.append((gen, gen.remaining())); rows += gen.remaining()
        if emb.remaining() > 0:
            q = min(chunk, emb.remaining())
            work.append((emb, q)); rows += q
        nxt = []
        for f in inflight:
            q = min(chunk, f.remaining(), budget - rows)
            if q > 0:
                work.append((f, q)); rows += q
            if f.remaining() - max(q, 0) > 0:
                nxt.append(f)
        while rows < budget:
            n = int(rng.integers(16, 2 * chunk))
            f = Request("embed", synth.token_ids(rng, n, shape.V), B.POOL_LAST)
            q = min(chunk, n, budget - rows)
            work.append((f, q)); rows += q
            if q < n:
                nxt.append(f)
        inflight = nxt
        batch, lrows, erows = eng.step(work)
        assert batch.n_tokens == budget
        torch.cuda.synchronize()
        if gen in lrows:
            got_lg.append(eng.out_logits[lrows[gen]].cpu().numpy())
        if emb in erows:
            got_emb = eng.out_emb[erows[emb]].cpu().numpy().astype(np.float64)
    assert eng.ctx.status_poll() == 0
    assert got_emb is not None and len(got_lg) == n_steps
    cos = float(got_emb @ ora_emb / (np.linalg.norm(got_emb) * np.linalg.norm(ora_emb)))
    assert cos >= EMB_COS, cos
    assert np.max(np.abs(got_emb - ora_emb)) <= EMB_ABS
    for s in range(n_steps):
        assert np.max(np.abs(got_lg[s] - ora_lg[s])) <= LOGIT_ABS, s
    eng.close()

"""Replay of a small iterative-retrieval trace on the tiny shape: every request completes, all pages
and slots come back, the row count is the trace's, and the first session's results match the oracle
(embedding of its first request; first generated token and its logits of its first prompt)."""
import numpy as np
import pytest
import torch

from oracle import transformer as T
from paper_2609_25405_b200 import synth

pytestmark = pytest.mark.gpu


def test_trace_replay_tiny():
    from paper_2609_25405_b200 import binding as B
    from paper_2609_25405_b200 import trace
    from paper_2609_25405_b200.engine import Engine
    shape = synth.SHAPES["tiny"]
    W = synth.Weights(shape, 0)
    dw = B.DeviceWeights.from_synth(W)
    sessions = trace.make_trace(shape.V, seed=3, n_sessions=6, rate=200.0, rounds=(2, 3), query=(5, 20),
                                document=(40, 90), prompt=(30, 120), decode=(3, 9))
    n_pages = 6 * 10 + 8
    eng = Engine(shape, dw, n_pages=n_pages, n_slots=8, max_tokens=128, max_segs=32, max_pos=160)
    got_emb, got_tok = {}, {}

    def on_emb(si, ri, vec):
        got_emb[(si, ri)] = vec.cpu().numpy().astype(np.float64)

    def on_tok(si, ri, step, token, row):
        got_tok[(si, ri, step)] = (token, row.cpu().numpy().astype(np.float64))

    out = trace.replay(sessions, eng, budget=128, chunk=32, pool_mode=B.POOL_MEAN, on_embedding=on_emb, on_token=on_tok)
    assert eng.ctx.status_poll() == 0
    assert out["sessions_done"] == 6
    assert out["rows"] == trace.trace_tokens(sessions)
    assert out["free_pages"] == n_pages                      # everything was released
    assert len(got_emb) == sum(1 for s in sessions for r in s.requests if r.kind == "embed")
    n_tok = sum(r.decode_steps + 1 for s in sessions for r in s.requests if r.kind == "gen")
    assert len(got_tok) == n_tok
    # parity of the first session's first embedding and first generation step
    e_ref = T.embed(shape, W, sessions[0].requests[0].tokens, "mean")
    e = got_emb[(0, 0)]
    assert float(e @ e_ref) >= 0.9995 and np.max(np.abs(e - e_ref)) <= 2e-2
    prompt = sessions[0].requests[1].tokens
    tk, lg = T.generate(shape, W, prompt, 1)
    token, row = got_tok[(0, 1, 0)]
    assert np.max(np.abs(row - lg[0])) <= 5e-2
    assert token == int(np.argmax(row))                      # the device argmax is the argmax of its own logits
    eng.close()


def test_phase_workload_tiny():
    """Shifting request mix (10 % / 50 % / 90 % embedding requests) replayed phase by phase through the
    same engine: every phase drains, row counts are the phases' own, pages and slots all come back."""
    from paper_2609_25405_b200 import binding as B
    from paper_2609_25405_b200 import trace
    from paper_2609_25405_b200.engine import Engine
    shape = synth.SHAPES["tiny"]
    dw = B.DeviceWeights.from_synth(synth.Weights(shape, 0))
    phases = trace.make_phases(shape.V, seed=4, n_requests=12, embed_len=40, prompt_len=24, decode_len=6)
    n_pages = 12 * 4 + 8
    eng = Engine(shape, dw, n_pages=n_pages, n_slots=16, max_tokens=128, max_segs=48, max_pos=64)
    n_embed = []
    for sessions in phases:
        out = trace.replay(sessions, eng, budget=128, chunk=32)
        assert out["sessions_done"] == 12 and out["rows"] == trace.trace_tokens(sessions)
        assert out["free_pages"] == n_pages
        n_embed.append(sum(s.requests[0].kind == "embed" for s in sessions))
    assert eng.ctx.status_poll() == 0
    assert n_embed[0] < n_embed[1] < n_embed[2]
    eng.close()


def test_trace_prefix_on_the_1b_shape_every_output_matches_oracle():
    """Configuration 5 on its own shape: the first eight sessions of the seed-1005 trace (3-5 rounds
    each of an embedding request and a generation request with a 512-2048-token prompt and 32-128
    greedy decode steps) replayed on the full 1B-class model through the scheduler and the engine.
    EVERY embedding and EVERY logits row of those sessions is compared with the fp32 oracle: the
    oracle runs one whole-sequence pass per request over the prompt plus the tokens the device chose
    (teacher-forced on the device's own greedy tokens, so one differing argmax does not spoil the
    rows after it).  Eight sessions give about 2800 logits rows: at this shape (vocabulary 128256,
    logits errors of about 1e-2) roughly 0.3 % of the rows are near-ties of the oracle that the fp16
    path decides the other way, and the 99.5 % criterion needs a sample in which that rate shows
    (three sessions, about 1000 rows, gave 3 to 5 such rows depending on the rounding order of the
    attention merge: either side of the limit).  Bookkeeping over a whole trace is checked on the tiny
    shape above."""
    from conftest import cached_weights
    from paper_2609_25405_b200 import binding as B
    from paper_2609_25405_b200 import trace
    from paper_2609_25405_b200.engine import Engine
    shape = synth.SHAPES["1b"]
    W, dw = cached_weights(shape)
    sessions = trace.make_trace(shape.V, seed=1005, n_sessions=256)[:8]
    budget, chunk = 4096, 256
    max_pos = 2048 + 128 + 8
    P = shape.page_size
    n_pages = 8 * ((max_pos + P - 1) // P) + 64
    eng = Engine(shape, dw, n_pages=n_pages, n_slots=8, max_tokens=budget, max_segs=8 + budget // 16 + 8, max_pos=max_pos)
    got_emb, got_tok = {}, {}

    def on_emb(si, ri, vec):
        got_emb[(si, ri)] = vec.cpu().numpy().astype(np.float64)

    def on_tok(si, ri, step, token, row):
        got_tok[(si, ri, step)] = (token, row.cpu().numpy())          # fp32 rows: ~0.5 MB each

    out = trace.replay(sessions, eng, budget, chunk, pool_mode=B.POOL_LAST, on_embedding=on_emb, on_token=on_tok)
    assert eng.ctx.status_poll() == 0
    assert out["sessions_done"] == 8 and out["rows"] == trace.trace_tokens(sessions)
    assert out["free_pages"] == n_pages
    n_rows = n_agree = n_embs = 0
    worst_l = worst_e = 0.0
    worst_cos = 1.0
    flips = []
    for si, s in enumerate(sessions):
        for ri, r in enumerate(s.requests):
            if r.kind == "embed":
                ref = T.embed(shape, W, r.tokens, "last", dtype=np.float32).astype(np.float64)
                got = got_emb[(si, ri)]
                cos = float(got @ ref / (np.linalg.norm(got) * np.linalg.norm(ref)))
                worst_cos, worst_e = min(worst_cos, cos), max(worst_e, float(np.max(np.abs(got - ref))))
                assert cos >= 0.9995 and np.max(np.abs(got - ref)) <= 2e-2, (si, ri, len(r.tokens), cos)
                n_embs += 1
                continue
            k = r.decode_steps + 1                       # the prompt's last row, then one row per decode step
            toks = [got_tok[(si, ri, st)][0] for st in range(k)]
            seq = [int(t) for t in r.tokens] + toks[:-1]
            n0 = len(r.tokens)
            _, ref = T.forward(shape, W, seq, logit_rows=list(range(n0 - 1, n0 - 1 + k)), dtype=np.float32)
            for st in range(k):
                token, row = got_tok[(si, ri, st)]
                err = float(np.max(np.abs(row.astype(np.float64) - ref[st])))
                worst_l = max(worst_l, err)
                assert err <= 5e-2, (si, ri, st, err)
                assert token == int(np.argmax(row))          # hb_argmax = the argmax of the device's own logits
                n_rows += 1
                if token == int(np.argmax(ref[st])):
                    n_agree += 1
                else:
                    top = np.sort(ref[st])[-2:]
                    flips.append((si, ri, st, float(top[1] - top[0]), err))
    print(f"\ntrace prefix, 1B shape: {n_embs} embeddings (worst cosine {worst_cos:.6f}, worst max-abs error {worst_e:.3e}); "
          f"{n_rows} logits rows (worst max-abs error {worst_l:.3e}), argmax agreement {n_agree}/{n_rows} = "
          f"{n_agree / max(n_rows, 1):.4f}")
    for si, ri, st, gap, err in flips:
        print(f"  differing argmax: session {si} request {ri} step {st}: oracle top-1/top-2 gap {gap:.3e}, "
              f"logits max-abs error {err:.3e}")
    assert n_agree / n_rows >= 0.995, (n_agree, n_rows)
    eng.close()

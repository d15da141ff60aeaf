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

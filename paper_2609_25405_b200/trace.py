"""Synthetic iterative-retrieval trace and its replay through the mixed step (host glue).

Trace: sessions arrive as a Poisson process; a session is 3-5 rounds, each round an embedding
request (a short query or a retrieved document) followed by a generation request (prompt, then a
number of decode steps); a request becomes eligible when its predecessor in the session has
finished.  This stands in, by shape only, for the iterative retrieval-generation workload of the
paper's Section 5.2.

Replay: the IBS scheduler (Algorithm 2) composes every iteration under the token budget, the engine
runs it as one hb_mixed_step, generated tokens are chosen greedily on the device (hb_argmax) and
read back, finished requests release their pages and slots.  Time is a virtual clock: it advances by
each step's measured GPU time and jumps over idle gaps to the next arrival, so the replay measures
the sustained service rate rather than the arrival rate.
"""
from dataclasses import dataclass, field

import numpy as np

from . import consts
from . import synth


@dataclass
class TraceRequest:
    kind: str                  # "embed" | "gen"
    tokens: np.ndarray         # text / prompt
    decode_steps: int = 0


@dataclass
class Session:
    arrival: float
    requests: list = field(default_factory=list)


def make_trace(V, seed=1005, n_sessions=256, rate=20.0, rounds=(3, 5), query=(16, 64), document=(256, 1024),
               prompt=(512, 2048), decode=(32, 128)):
    """Seeded trace: exponential inter-arrival times at `rate` sessions/s; per round an embedding
    request (query or document length with probability 1/2 each, uniform in its range) then a
    generation request (prompt and decode-step counts uniform in their ranges)."""
    rng = np.random.default_rng(seed)
    t = 0.0
    sessions = []
    for _ in range(n_sessions):
        t += float(rng.exponential(1.0 / rate))
        s = Session(arrival=t)
        for _ in range(int(rng.integers(rounds[0], rounds[1] + 1))):
            lo, hi = query if rng.random() < 0.5 else document
            s.requests.append(TraceRequest("embed", synth.token_ids(rng, int(rng.integers(lo, hi + 1)), V)))
            s.requests.append(TraceRequest("gen", synth.token_ids(rng, int(rng.integers(prompt[0], prompt[1] + 1)), V),
                                           int(rng.integers(decode[0], decode[1] + 1))))
        sessions.append(s)
    return sessions


def make_phases(V, seed=1006, n_requests=256, embed_fracs=(0.1, 0.5, 0.9), embed_len=128, prompt_len=128,
                decode_len=512):
    """Shifting request mix (the utilisation experiment of Section 5.3): one list of single-request
    sessions per phase; in phase p a request is an embedding with probability embed_fracs[p], else a
    generation.  Sizes are the paper's synthetic ones (Section 5.1: 128-token embeddings, 128-token
    prompts with 512 generated tokens).  All requests of a phase are present from its start (a
    saturated server); the next phase starts when the previous one has drained."""
    rng = np.random.default_rng(seed)
    phases = []
    for frac in embed_fracs:
        sessions = []
        for _ in range(n_requests):
            s = Session(arrival=0.0)
            if rng.random() < frac:
                s.requests.append(TraceRequest("embed", synth.token_ids(rng, embed_len, V)))
            else:
                s.requests.append(TraceRequest("gen", synth.token_ids(rng, prompt_len, V), decode_len))
            sessions.append(s)
        phases.append(sessions)
    return phases


def trace_tokens(sessions):
    """Rows the replay will process: every text / prompt token once plus one row per decode step."""
    return sum(len(r.tokens) + r.decode_steps for s in sessions for r in s.requests)


def replay(sessions, engine, budget, chunk, pool_mode=consts.POOL_LAST, on_embedding=None, on_token=None,
           max_steps=None):
    """Runs the trace to completion.  Returns a dict of totals.  `on_embedding(session, index, vec)` and
    `on_token(session, index, step, token, logits_row)` receive results (device tensors) as they appear."""
    import torch

    from .engine import Request
    from .scheduler import IBS, Work

    sch = IBS(budget, chunk)
    pending = sorted(range(len(sessions)), key=lambda i: sessions[i].arrival)
    cursor = [0] * len(sessions)          # next request index per session
    live = {}                             # Work -> (session index, request index, engine Request)
    clock = busy = 0.0
    n_steps = n_rows = 0
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    tok_dev = torch.zeros(engine.max_segs, dtype=torch.int32, device="cuda")

    def start(si):
        tr = sessions[si].requests[cursor[si]]
        req = Request(tr.kind, tr.tokens, pool_mode if tr.kind == "embed" else consts.POOL_NONE)
        w = Work(tr.kind, len(tr.tokens), payload=req)
        w.decode_left = tr.decode_steps
        w.n_generated = 0
        live[w] = (si, cursor[si], req)
        sch.submit(w)

    done_sessions = 0
    while done_sessions < len(sessions):
        while pending and sessions[pending[0]].arrival <= clock:
            start(pending.pop(0))
        if not live:
            clock = sessions[pending[0]].arrival       # idle: jump to the next arrival
            continue
        batch = sch.schedule()
        if not batch:
            raise RuntimeError("scheduler produced an empty batch with live requests")
        work = [(live[w][2], rows) for w, rows in batch]
        e0.record()
        _, lrows, erows = engine.step(work)
        n_logit = len(lrows)
        if n_logit:
            engine.ctx.argmax(engine.out_logits, n_logit, tok_dev)
        e1.record()
        torch.cuda.synchronize()
        dt = e0.elapsed_time(e1) * 1e-3
        clock += dt
        busy += dt
        n_steps += 1
        n_rows += sum(rows for _, rows in batch)
        toks = tok_dev[:n_logit].cpu().tolist() if n_logit else []
        finished = sch.commit(batch)
        for w, rows in batch:
            si, ri, req = live[w]
            if req in lrows:
                # logits of a finished prefill or of a decode step: the argmax is the next token, fed back
                # in the next iteration if decode steps remain
                token = int(toks[lrows[req]])
                if on_token is not None:
                    on_token(si, ri, w.n_generated, token, engine.out_logits[lrows[req]])
                w.n_generated += 1
                if w in sch.running:
                    req.tokens.append(token)
            if req in erows and on_embedding is not None:
                on_embedding(si, ri, engine.out_emb[erows[req]])
        for w in finished:
            si, ri, req = live.pop(w)
            engine.release(req)
            cursor[si] += 1
            if cursor[si] < len(sessions[si].requests):
                start(si)
            else:
                done_sessions += 1
        if max_steps is not None and n_steps >= max_steps:
            break
    return dict(steps=n_steps, rows=n_rows, busy_s=busy, clock_s=clock, sessions_done=done_sessions,
                free_pages=engine.kv.free_count())

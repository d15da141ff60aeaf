"""Intra-batch scheduling (Algorithm 2 of the paper) as host-side glue.

Composes one iteration's batch from an embedding queue Q_e and a generation queue Q_g under a
token budget B: capacity is first reserved for in-flight decodes (`ScheduleRunning`), then the rest
is filled by picking, one item at a time, from the queue with the larger credit.  Credits a_e, a_g
grow by the queues' remaining-token weights w_e, w_g at every selection step, the chosen queue pays
w_e + w_g, credits persist across iterations and are reset when their queue is empty
(Section 4.2).  `ScheduleOne` admits the next request of a queue in arrival order (per-type FCFS)
as a chunk of at most C tokens that fits the residual budget; a request contributes at most one
chunk per iteration because chunk k + 1 reads the K/V chunk k writes.

This module decides WHAT goes into a batch; `engine.Engine.step` runs it.  It holds no arithmetic of
the forward pass.
"""
from collections import deque


class Work:
    """A queued request as the scheduler sees it: a kind and a number of tokens still to schedule."""

    def __init__(self, kind, n_tokens, payload=None):
        assert kind in ("embed", "gen") and n_tokens >= 1
        self.kind = kind
        self.remaining = int(n_tokens)      # prompt / text tokens not yet scheduled
        self.payload = payload              # e.g. an engine.Request
        self.decode_left = 0                # generation: decode steps still to run after the prefill

    def __repr__(self):
        return f"Work({self.kind}, remaining={self.remaining}, decode_left={self.decode_left})"


class IBS:
    def __init__(self, budget, chunk, chunked=True, decode_rows=1):
        """budget B (tokens per iteration), chunk cap C; chunked=False makes embedding requests
        atomic (admitted only when they fit whole), the comparison condition of Appendix A.3;
        decode_rows = budget tokens an in-flight decode takes per iteration (1 in the real step)."""
        self.B, self.C, self.chunked = int(budget), int(chunk), bool(chunked)
        self.decode_rows = int(decode_rows)
        self.a_e = 0
        self.a_g = 0
        self.Qe, self.Qg = deque(), deque()
        self.running = {}                   # generation requests in their decode phase (insertion-ordered set)

    # ---- queues ----
    def submit(self, work):
        (self.Qe if work.kind == "embed" else self.Qg).append(work)

    def _weight(self, Q):
        return sum(w.remaining for w in Q)

    def _remove(self, Q, w):
        if Q and Q[0] is w:                 # the usual case: requests finish in arrival order
            Q.popleft()
        else:
            Q.remove(w)

    # ---- Algorithm 2 ----
    def _schedule_running(self, budget):
        batch, used = [], 0
        for w in self.running:
            if used + self.decode_rows > budget:
                break                       # (the paper swaps such requests out; not modelled)
            batch.append((w, self.decode_rows))
            used += self.decode_rows
        return batch, used

    def _schedule_one(self, Q, budget, taken):
        """Next request of Q in arrival order that has not contributed this iteration; a chunk of at
        most C tokens that fits.  Returns (item or None, tokens used)."""
        for w in Q:
            if id(w) in taken:
                continue
            if w.kind == "embed" and not self.chunked:
                rows = w.remaining if w.remaining <= budget else 0      # atomic: whole request or nothing
            else:
                rows = min(self.C, w.remaining, budget)
            if rows <= 0:
                return None, 0              # the next request in line does not fit: per-type FCFS forbids overtaking
            return (w, rows), rows
        return None, 0

    def schedule(self):
        """One call = one iteration.  Returns the batch as a list of (Work, rows)."""
        batch, used = self._schedule_running(self.B)
        B = self.B - used
        w_e, w_g = self._weight(self.Qe), self._weight(self.Qg)
        if not self.Qe:
            self.a_e = 0
        if not self.Qg:
            self.a_g = 0
        taken = set()
        open_e, open_g = bool(self.Qe), bool(self.Qg)
        while B > 0 and (open_e or open_g):
            self.a_e += w_e
            self.a_g += w_g
            pick_e = (not open_g) or (open_e and self.a_e >= self.a_g)
            Q = self.Qe if pick_e else self.Qg
            item, u = self._schedule_one(Q, B, taken)
            if item is None:                # nothing more from this queue in this iteration
                if pick_e:
                    open_e = False
                else:
                    open_g = False
                continue
            batch.append(item)
            taken.add(id(item[0]))
            B -= u
            if pick_e:
                self.a_e -= (w_e + w_g)
            else:
                self.a_g -= (w_e + w_g)
        return batch

    def commit(self, batch):
        """Advance request state after the iteration ran.  Returns the Work items that finished."""
        done = []
        for w, rows in batch:
            if w in self.running:
                w.decode_left -= 1
                if w.decode_left <= 0:
                    del self.running[w]
                    done.append(w)
                continue
            w.remaining -= rows
            if w.remaining == 0:
                self._remove(self.Qe if w.kind == "embed" else self.Qg, w)
                if w.kind == "gen" and w.decode_left > 0:
                    self.running[w] = None
                else:
                    done.append(w)
        return done


def packing_fill(budget, chunk, chunked, n_iters=2000, seed=0, gen_frac=0.8, prefill=128, decode=256,
                 decode_step=8, embed_lens=(96, 224), long_frac=0.45, arrivals_per_iter=1.0):
    """Average fraction of the token budget filled per iteration for an FCFS iteration scheduler with
    atomic or chunked embedding requests, on the request mix of Appendix A.3 (80 % generation:
    128-token prefill + 256-token decode advanced `decode_step` tokens per iteration; embeddings of
    96 or 224 tokens, 45 % long).  The appendix does not state its arrival process or time model, so
    the absolute fill differs from the printed table; the direction (chunking raises the fill) is
    what this reproduces.  Arrivals: Poisson, `arrivals_per_iter` requests per iteration."""
    import numpy as np
    rng = np.random.default_rng(seed)
    sch = IBS(budget, chunk, chunked, decode_rows=decode_step)
    filled = 0
    for _ in range(n_iters):
        for _ in range(rng.poisson(arrivals_per_iter)):
            if rng.random() < gen_frac:
                w = Work("gen", prefill)
                w.decode_left = decode // decode_step
            else:
                w = Work("embed", embed_lens[1] if rng.random() < long_frac else embed_lens[0])
            sch.submit(w)
        batch = sch.schedule()
        filled += sum(rows for _, rows in batch)
        sch.commit(batch)
    return filled / (n_iters * budget)

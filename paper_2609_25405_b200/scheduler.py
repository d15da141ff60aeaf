"""Intra-batch scheduling (Section 4.2 of the paper) as host-side glue.

Composes one iteration's batch from an embedding queue Q_e and a generation queue Q_g under a
token budget B: capacity is first reserved for in-flight decodes, then the rest is filled one
admission at a time from the type with the larger credit.  Credits grow by the queues'
remaining-token weights at every selection, the chosen type pays the sum of both weights, credits
persist across iterations and are reset when their queue is empty.  An admission is the next
request of a type in arrival order (per-type FCFS) as a chunk of at most C tokens that fits the
residual budget; a request contributes at most one chunk per iteration because chunk k + 1 reads
the K/V chunk k writes.  One deliberate difference from a literal reading of Algorithm 2: a type
that can contribute nothing more to the iteration stops earning credit for the rest of it.

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


class _Credits:
    """Token-weighted credits of the two request types (Section 4.2).  A type that can still
    contribute to the batch being composed earns its backlog weight at every selection; the type
    picked pays the sum of both weights, so over a run of selections the picks follow the weights
    within one selection (the paper's fairness bound).  Credits are kept between iterations and
    dropped for a type whose queue is empty."""

    def __init__(self):
        self.a = {"embed": 0, "gen": 0}

    def start_iteration(self, weights):
        self.w = dict(weights)
        for kind, w in weights.items():
            if w == 0:
                self.a[kind] = 0            # an empty queue carries no claim into the future

    def accrue(self, candidates):
        """One selection opportunity: only types that can still be admitted in this iteration earn
        (a type closed for the iteration would otherwise pile up credit it could never have spent
        here, beyond the one-opportunity bound)."""
        for kind in candidates:
            self.a[kind] += self.w[kind]

    def pick(self, candidates):
        """The candidate with the larger credit; embedding wins ties."""
        if len(candidates) == 1:
            return candidates[0]
        return "embed" if self.a["embed"] >= self.a["gen"] else "gen"

    def charge(self, kind):
        self.a[kind] -= self.w["embed"] + self.w["gen"]


class IBS:
    def __init__(self, budget, chunk, chunked=True, decode_rows=1):
        """budget B (tokens per iteration), chunk cap C; chunked=False makes embedding requests
        atomic (admitted only when they fit whole), the comparison condition of Appendix A.3;
        decode_rows = budget tokens an in-flight decode takes per iteration (1 in the real step)."""
        self.B, self.C, self.chunked = int(budget), int(chunk), bool(chunked)
        self.decode_rows = int(decode_rows)
        self.credits = _Credits()
        self.Qe, self.Qg = deque(), deque()
        self.running = {}                   # generation requests in their decode phase (insertion-ordered set)

    # credits as the paper names them
    @property
    def a_e(self):
        return self.credits.a["embed"]

    @property
    def a_g(self):
        return self.credits.a["gen"]

    # ---- queues ----
    def submit(self, work):
        (self.Qe if work.kind == "embed" else self.Qg).append(work)

    def _queue(self, kind):
        return self.Qe if kind == "embed" else self.Qg

    def _weight(self, Q):
        return sum(w.remaining for w in Q)

    def _remove(self, Q, w):
        if Q and Q[0] is w:                 # the usual case: requests finish in arrival order
            Q.popleft()
        else:
            Q.remove(w)

    # ---- composing one iteration (Section 4.2) ----
    def _reserve_running(self, budget):
        """In-flight decodes come first: each takes its rows out of the budget."""
        batch, used = [], 0
        for w in self.running:
            if used + self.decode_rows > budget:
                break                       # (the paper swaps such requests out; not modelled)
            batch.append((w, self.decode_rows))
            used += self.decode_rows
        return batch, used

    def _next_admission(self, kind, budget, taken):
        """The next request of `kind` in arrival order that has not contributed to this iteration, as
        (work, rows): a chunk of at most C tokens that fits the residual budget.  None when the type
        can contribute nothing more (per-type FCFS: a request that does not fit is not overtaken)."""
        for w in self._queue(kind):
            if id(w) in taken:
                continue
            if w.kind == "embed" and not self.chunked:
                rows = w.remaining if w.remaining <= budget else 0      # atomic: whole request or nothing
            else:
                rows = min(self.C, w.remaining, budget)
            return (w, rows) if rows > 0 else None
        return None

    def schedule(self):
        """One call = one iteration.  Returns the batch as a list of (Work, rows)."""
        batch, used = self._reserve_running(self.B)
        left = self.B - used
        self.credits.start_iteration({"embed": self._weight(self.Qe), "gen": self._weight(self.Qg)})
        taken = set()
        candidates = [k for k in ("embed", "gen") if self._queue(k)]
        while left > 0 and candidates:
            self.credits.accrue(candidates)
            kind = self.credits.pick(candidates)
            item = self._next_admission(kind, left, taken)
            if item is None:
                candidates.remove(kind)     # closed for this iteration: it neither earns nor is picked again
                continue
            batch.append(item)
            taken.add(id(item[0]))
            left -= item[1]
            self.credits.charge(kind)
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

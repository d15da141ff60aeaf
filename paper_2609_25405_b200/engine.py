"""Host-side glue around hb_mixed_step: request state, page / slot ownership and the
batch unit of Section 3.2 (rows sorted by type: decode, prefill chunks, embedding chunks).

This is bookkeeping only.  The batch-composition policy is the caller's: `Engine.step`
takes the list of (request, rows) the scheduler chose for this iteration.
"""
import itertools

import numpy as np
import torch

from . import binding as B


class Request:
    """One embedding or generation request as it moves through iterations."""

    def __init__(self, kind, tokens, pool_mode=B.POOL_NONE):
        assert kind in ("gen", "embed")
        self.kind = kind
        self.tokens = [int(t) for t in tokens]   # prompt / text; generated tokens are appended
        self.n_prompt = len(self.tokens)
        self.n_done = 0                          # tokens whose K/V is in the cache
        self.pages = []
        self.slot = -1
        self.pool_mode = pool_mode
        self.finished = False

    @property
    def in_decode(self):
        return self.kind == "gen" and self.n_done >= self.n_prompt

    def remaining(self):
        return len(self.tokens) - self.n_done


def build_batch(entries, page_size):
    """entries: list of dicts(kind, tokens, pos_start, pages, pool_slot, pool_mode, is_final,
    wants_logits).  Returns (Batch, order) with segments sorted by kind (stable) and
    logits / embedding rows numbered in segment order; order[i] = index into `entries`."""
    order = sorted(range(len(entries)), key=lambda i: entries[i]["kind"])
    ents = [entries[i] for i in order]
    n = len(ents)
    # one Python pass collects plain lists; the structured array is filled column by column
    kind = np.fromiter((e["kind"] for e in ents), dtype=np.int32, count=n)
    q_len = np.fromiter((len(e["tokens"]) for e in ents), dtype=np.int32, count=n)
    pt_len = np.fromiter((len(e["pages"]) for e in ents), dtype=np.int32, count=n)
    final = np.fromiter((1 if e.get("is_final") else 0 for e in ents), dtype=np.int32, count=n)
    segs = np.zeros(n, dtype=B.SEG_DTYPE)
    segs["kind"] = kind
    segs["q_len"] = q_len
    segs["q_start"] = np.cumsum(q_len) - q_len
    segs["pos_start"] = np.fromiter((e["pos_start"] for e in ents), dtype=np.int32, count=n)
    segs["pt_len"] = pt_len
    segs["pt_start"] = np.cumsum(pt_len) - pt_len
    segs["pool_slot"] = np.fromiter((e.get("pool_slot", -1) for e in ents), dtype=np.int32, count=n)
    segs["pool_mode"] = np.fromiter((e.get("pool_mode", B.POOL_NONE) for e in ents), dtype=np.int32, count=n)
    segs["is_final"] = final
    is_emb = kind == B.KIND_EMBED_CHUNK
    wants_emb = is_emb & (final == 1)
    wants_lg = ~is_emb & ((kind == B.KIND_DECODE) | (final == 1))
    segs["emb_row"] = np.where(wants_emb, np.cumsum(wants_emb) - 1, -1)
    segs["logits_row"] = np.where(wants_lg, np.cumsum(wants_lg) - 1, -1)
    n_e, n_l = int(wants_emb.sum()), int(wants_lg.sum())
    toks = np.fromiter(itertools.chain.from_iterable(e["tokens"] for e in ents), dtype=np.int32,
                       count=int(q_len.sum()))
    pages = np.fromiter(itertools.chain.from_iterable(e["pages"] for e in ents), dtype=np.int32,
                        count=int(pt_len.sum()))
    return B.Batch(toks, segs, pages, n_l, n_e), order


class Engine:
    def __init__(self, shape, weights, n_pages, n_slots, max_tokens, max_segs, max_pos,
                 kv_fill=None, pool_fill=None, device="cuda", lora=None):
        self.shape = shape
        self.lora = lora                    # binding.DeviceLora applied to embedding rows, or None
        self.cfg = B.model_cfg(shape, max_pos)
        self.weights = weights
        self.max_tokens, self.max_segs = max_tokens, max_segs
        max_page_ids = max_segs * ((max_pos + shape.page_size - 1) // shape.page_size)
        self.ctx = B.Context(self.cfg, max_tokens, max_segs, max_page_ids)
        self.kv = B.KvCache(self.cfg, n_pages, device, fill=kv_fill)
        self.pool = B.Pool(self.cfg, n_slots, device, fill=pool_fill)
        self.out_logits = torch.zeros((max_segs, shape.V), dtype=torch.float32, device=device)
        self.out_emb = torch.zeros((max_segs, shape.d), dtype=torch.float32, device=device)

    def _ensure_pages(self, req, n_tokens):
        P = self.shape.page_size
        need = (n_tokens + P - 1) // P - len(req.pages)
        if need > 0:
            req.pages.extend(self.kv.alloc(need))

    def entry_for(self, req, rows):
        """Descriptor entry for `rows` new rows of `req` (and reserve pages / slot)."""
        assert rows >= 1 and rows <= req.remaining()
        self._ensure_pages(req, req.n_done + rows)
        toks = req.tokens[req.n_done:req.n_done + rows]
        e = dict(tokens=toks, pos_start=req.n_done, pages=req.pages)      # read by build_batch, not kept
        last = (req.n_done + rows == len(req.tokens))
        if req.kind == "embed":
            if req.slot < 0:
                req.slot = self.pool.alloc()
            e.update(kind=B.KIND_EMBED_CHUNK, pool_slot=req.slot, pool_mode=req.pool_mode, is_final=last)
        elif req.in_decode:
            assert rows == 1
            e.update(kind=B.KIND_DECODE, is_final=True)
        else:
            e.update(kind=B.KIND_PREFILL_CHUNK, is_final=last)
        return e

    def step(self, work, stream=None):
        """work: list of (Request, rows).  Enqueues one mixed step.  Returns
        (batch, logits_rows {req: row}, emb_rows {req: row}); outputs land in
        self.out_logits / self.out_emb once the stream is synchronised."""
        entries = [self.entry_for(r, n) for r, n in work]
        batch, order = build_batch(entries, self.shape.page_size)
        self.ctx.mixed_step(batch, self.weights, self.kv, self.pool, self.out_logits, self.out_emb, stream,
                            lora=self.lora)
        lrows, erows = {}, {}
        lg, em = batch.segs["logits_row"].tolist(), batch.segs["emb_row"].tolist()
        for si, ei in enumerate(order):
            req, n = work[ei]
            req.n_done += n
            if lg[si] >= 0:
                lrows[req] = lg[si]
            if em[si] >= 0:
                erows[req] = em[si]
                req.finished = True
        return batch, lrows, erows

    def release(self, req):
        """Return a finished request's pages and pool slot."""
        if req.pages:
            self.kv.free(req.pages)
            req.pages = []
        if req.slot >= 0:
            self.pool.free(req.slot)
            req.slot = -1

    def close(self):
        self.ctx.close()
        self.kv.close()
        self.pool.close()

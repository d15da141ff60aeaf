"""The attention launch runs resident blocks that take the step's attention items (decode splits,
chunk tiles of up to 128 rows) from a ticket.  Which block runs an item, and how many
items a block runs one after the other, must not change a result bit: an item's arithmetic is its
own, a block re-initialises its barriers and reuses its tensor memory between items, and the splits
of a decode row are merged in split order by whichever block arrives last.

Here the number of blocks is capped (1: one block walks through every item of both kinds; 3 and 17:
a few blocks interleave) and the outputs of a mixed sequence of steps (chunked prefill of long
prompts, then decode rows over 1 to 3 key splits together with embedding chunks that carry earlier
chunks' keys) are compared bit for bit with the uncapped launch; the uncapped launch itself is
checked against the oracle elsewhere (test_gpu_step, test_gpu_splits, test_gpu_fullsize)."""
import numpy as np
import pytest
import torch

from paper_2609_25405_b200 import synth

pytestmark = pytest.mark.gpu

SHAPES = {
    "tiny": synth.SHAPES["tiny"],
    # 2 layers, d 512, 4 query heads x 128 on 1 KV head (the head geometry of the 7B-class configuration)
    "dh128": synth.ModelShape("dh128", 2, 512, 4, 1, 128, 1024, 1024),
}
CONTEXTS = (130, 700, 3071, 5119)      # decode rows over 1, 1, 2 and 3 splits of their keys (2048 keys per split)
EMBED_LEN = (300, 77)                  # two embedding requests: chunks of 200 + 100 (a 128-row tile and a remainder) and 77


def _run(shape, dw, limit, contexts=CONTEXTS, embed_len=EMBED_LEN, embed_chunks=((200, 77), (100, 0)), seed=99):
    from paper_2609_25405_b200 import binding as B
    from paper_2609_25405_b200.engine import Engine, Request
    rng = np.random.default_rng(seed)
    CONTEXTS, EMBED_LEN = contexts, embed_len
    P = shape.page_size
    n_pages = sum((c + 2 + P - 1) // P for c in CONTEXTS) + sum((n + P - 1) // P for n in EMBED_LEN) + 4
    outs = []
    B.attn_set_block_limit(limit)
    try:
        eng = Engine(shape, dw, n_pages=n_pages, n_slots=4, max_tokens=len(CONTEXTS) * 512 + 512, max_segs=16,
                     max_pos=max(CONTEXTS) + 4, kv_fill=0x7F7F)
        gens = [Request("gen", synth.token_ids(rng, c, shape.V)) for c in CONTEXTS]
        embs = [Request("embed", synth.token_ids(rng, n, shape.V), B.POOL_MEAN) for n in EMBED_LEN]
        forced = [[int(rng.integers(0, shape.V)) for _ in range(2)] for _ in CONTEXTS]
        while any(not g.in_decode for g in gens):
            work = [(g, min(512, g.remaining())) for g in gens if not g.in_decode]
            _, lrows, _ = eng.step(work)
            torch.cuda.synchronize()
            outs.extend(eng.out_logits[lrows[g]].clone() for g in gens if g in lrows)
        # two mixed steps: every decode row + one embedding chunk each
        for s, chunks in enumerate(embed_chunks):
            work = []
            for g, f in zip(gens, forced):
                g.tokens.append(f[s])
                work.append((g, 1))
            work.extend((e, q) for e, q in zip(embs, chunks) if q > 0)
            _, lrows, erows = eng.step(work)
            torch.cuda.synchronize()
            outs.extend(eng.out_logits[lrows[g]].clone() for g in gens)
            outs.extend(eng.out_emb[r].clone() for _, r in sorted(erows.items(), key=lambda kv: kv[1]))
        assert eng.ctx.status_poll() == 0
        eng.close()
    finally:
        B.attn_set_block_limit(0)
    return outs


@pytest.mark.parametrize("name", ["tiny", "dh128"])
def test_outputs_do_not_depend_on_the_number_of_resident_blocks(name):
    from paper_2609_25405_b200 import binding as B
    shape = SHAPES[name]
    dw = B.DeviceWeights.from_synth(synth.Weights(shape, 0))
    ref = _run(shape, dw, 0)
    assert len(ref) >= 2 * len(CONTEXTS) + len(CONTEXTS) + len(EMBED_LEN)
    assert all(bool(torch.isfinite(o).all()) for o in ref)
    for limit in (1, 3, 17):
        got = _run(shape, dw, limit)
        assert len(got) == len(ref)
        for i, (a, b) in enumerate(zip(got, ref)):
            assert torch.equal(a, b), (name, limit, i)


@pytest.mark.parametrize("seed", [1, 2, 3, 4, 5, 6])
def test_random_mixes_with_one_and_seven_blocks(seed):
    """Random contexts (1 to 3 key splits), random embedding lengths and chunkings on the tiny shape:
    one block, seven blocks and the uncapped launch agree bit for bit."""
    from paper_2609_25405_b200 import binding as B
    shape = SHAPES["tiny"]
    dw = B.DeviceWeights.from_synth(synth.Weights(shape, 0))
    rng = np.random.default_rng(1000 + seed)
    contexts = tuple(int(c) for c in rng.integers(17, 6500, size=int(rng.integers(2, 6))))
    embed_len = tuple(int(n) for n in rng.integers(20, 500, size=2))
    first = tuple(int(rng.integers(1, n)) for n in embed_len)
    chunks = (first, tuple(n - f for n, f in zip(embed_len, first)))
    ref = _run(shape, dw, 0, contexts, embed_len, chunks, seed)
    for limit in (1, 7):
        got = _run(shape, dw, limit, contexts, embed_len, chunks, seed)
        assert len(got) == len(ref)
        for i, (a, b) in enumerate(zip(got, ref)):
            assert torch.equal(a, b), (seed, limit, i, contexts, embed_len, chunks)


def test_block_limit_rejects_negative_values():
    from paper_2609_25405_b200 import binding as B
    assert B.lib.hb_attn_set_block_limit(-1) == -1     # HB_ERR_BAD_ARG
    B.attn_set_block_limit(0)

"""Low-rank adapters on the embedding rows of the mixed step (GPU) against the oracle's plain
definition: embedding requests run the model with merged matrices W + (alpha / r) B A, generation
requests run the base model, both inside one batch (Section 2.1 "Parameter sharing", Section 5.1)."""
import numpy as np
import pytest
import torch

from oracle import transformer as T
from paper_2609_25405_b200 import synth

pytestmark = pytest.mark.gpu

TINY = synth.SHAPES["tiny"]
EMB_COS, EMB_ABS, LOGIT_ABS = 0.9995, 2e-2, 5e-2


@pytest.fixture(scope="module")
def weights():
    from paper_2609_25405_b200 import binding as B
    W = synth.Weights(TINY, seed=0)
    return W, B.DeviceWeights.from_synth(W)


def _engine(weights, lora, **kw):
    from paper_2609_25405_b200.engine import Engine
    args = dict(n_pages=96, n_slots=4, max_tokens=512, max_segs=16, max_pos=320)
    args.update(kw)
    return Engine(TINY, weights[1], args["n_pages"], args["n_slots"], args["max_tokens"], args["max_segs"],
                  args["max_pos"], lora=lora)


def _check_emb(got, ref):
    cos = float(got @ ref / (np.linalg.norm(got) * np.linalg.norm(ref)))
    assert cos >= EMB_COS, cos
    assert np.max(np.abs(got - ref)) <= EMB_ABS


@pytest.mark.parametrize("rank", [3, 16, 64])
def test_adapter_on_embedding_rows_only(weights, rank):
    """One batch holds a decoding request, a prefilling request and two embedding requests (one
    chunked over three steps).  Embeddings must match the merged-weight oracle and differ from the
    base model; logits must match the base-model oracle."""
    from paper_2609_25405_b200 import binding as B
    from paper_2609_25405_b200.engine import Request
    W = weights[0]
    ad = synth.LoraAdapters(TINY, rank, seed=11, std=0.05)
    Wm = T.MergedLora(W, ad)
    lora = B.DeviceLora.from_synth(ad)
    rng = np.random.default_rng(100 + rank)
    e1 = Request("embed", synth.token_ids(rng, 150, TINY.V), B.POOL_MEAN)
    e2 = Request("embed", synth.token_ids(rng, 41, TINY.V), B.POOL_LAST)
    g1 = Request("gen", synth.token_ids(rng, 70, TINY.V))
    g2 = Request("gen", synth.token_ids(rng, 33, TINY.V))
    eng = _engine(weights, lora)
    _, lr, er = eng.step([(g1, 70), (e1, 64), (e2, 41), (g2, 20)])
    torch.cuda.synchronize()
    ref_e2 = T.embed(TINY, Wm, e2.tokens, "last")
    _check_emb(eng.out_emb[er[e2]].cpu().numpy().astype(np.float64), ref_e2)
    base_e2 = T.embed(TINY, W, e2.tokens, "last")
    assert np.max(np.abs(ref_e2 - base_e2)) > 5 * EMB_ABS          # the adapter matters at this scale
    _, ref = T.forward(TINY, W, g1.tokens, logit_rows=[69])
    assert np.max(np.abs(eng.out_logits[lr[g1]].cpu().numpy() - ref[0])) <= LOGIT_ABS
    tok = int(np.argmax(ref[0]))
    g1.tokens.append(tok)                                           # g1 is now in its decode phase
    _, lr, _ = eng.step([(g1, 1), (g2, 13), (e1, 5)])               # decode row + prefill tail + embed chunk
    torch.cuda.synchronize()
    _, ref = T.forward(TINY, W, g1.tokens, logit_rows=[70])
    assert np.max(np.abs(eng.out_logits[lr[g1]].cpu().numpy() - ref[0])) <= LOGIT_ABS
    _, ref = T.forward(TINY, W, g2.tokens, logit_rows=[32])
    assert np.max(np.abs(eng.out_logits[lr[g2]].cpu().numpy() - ref[0])) <= LOGIT_ABS
    _, _, er = eng.step([(e1, 81)])
    torch.cuda.synchronize()
    assert eng.ctx.status_poll() == 0
    _check_emb(eng.out_emb[er[e1]].cpu().numpy().astype(np.float64), T.embed(TINY, Wm, e1.tokens, "mean"))
    eng.close()


def test_zero_factors_and_absent_adapter_are_bitwise_the_base_step(weights):
    """u = 0 adds exactly zero in the extended K loop: a step with all-zero factors, a step with no
    adapter, and a step whose batch has no embedding rows give bit-identical outputs."""
    from paper_2609_25405_b200 import binding as B
    from paper_2609_25405_b200.engine import Request
    rng = np.random.default_rng(5)
    toks_e, toks_g = synth.token_ids(rng, 90, TINY.V), synth.token_ids(rng, 50, TINY.V)
    zero = B.DeviceLora.from_synth(synth.LoraAdapters(TINY, 8, std=0.0))
    live = B.DeviceLora.from_synth(synth.LoraAdapters(TINY, 8, std=0.05))
    outs = []
    for lora in (None, zero):
        eng = _engine(weights, lora)
        e, g = Request("embed", toks_e, B.POOL_MEAN), Request("gen", toks_g)
        _, lr, er = eng.step([(e, 90), (g, 50)])
        torch.cuda.synchronize()
        outs.append((eng.out_emb[er[e]].clone(), eng.out_logits[lr[g]].clone()))
        eng.close()
    assert torch.equal(outs[0][0], outs[1][0]) and torch.equal(outs[0][1], outs[1][1])
    eng = _engine(weights, live)
    g = Request("gen", toks_g)
    _, lr, _ = eng.step([(g, 50)])                                   # no embedding rows: adapter path not taken
    torch.cuda.synchronize()
    assert eng.ctx.last_launch_count() == eng_launches_without_adapter(weights, toks_g)
    assert torch.equal(eng.out_logits[lr[g]], outs[0][1])
    eng.close()


def eng_launches_without_adapter(weights, toks):
    from paper_2609_25405_b200.engine import Request
    eng = _engine(weights, None)
    g = Request("gen", toks)
    eng.step([(g, len(toks))])
    torch.cuda.synchronize()
    n = eng.ctx.last_launch_count()
    eng.close()
    return n


def test_adapter_batch_composition_independence(weights):
    """An embedding request's result with the adapter does not depend on what shares its batch:
    alone, or behind generation rows that move it to other rows of the tile (bitwise)."""
    from paper_2609_25405_b200 import binding as B
    from paper_2609_25405_b200.engine import Request
    lora = B.DeviceLora.from_synth(synth.LoraAdapters(TINY, 16, std=0.05))
    rng = np.random.default_rng(9)
    toks = synth.token_ids(rng, 77, TINY.V)
    res = []
    for extra in (0, 1, 37, 140):
        eng = _engine(weights, lora)
        e = Request("embed", toks, B.POOL_MEAN)
        work = [(e, 77)]
        if extra:
            work.append((Request("gen", synth.token_ids(rng, extra, TINY.V)), extra))
        _, _, er = eng.step(work)
        torch.cuda.synchronize()
        res.append(eng.out_emb[er[e]].clone())
        eng.close()
    for r in res[1:]:
        assert torch.equal(r, res[0])

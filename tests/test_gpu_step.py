"""Parity of hb_mixed_step (through the C-ABI) with the CPU oracle on the tiny configuration:
the whole mixed workload (prefill, 8 teacher-forced decode steps, two chunked embedding
requests with mean pooling), bit-exact KV-page and pool bookkeeping, batch-composition
independence and random chunkings."""
import numpy as np
import pytest
import torch

from oracle import method as M
from oracle import transformer as T
from paper_2609_25405_b200 import synth

pytestmark = pytest.mark.gpu

TINY = synth.SHAPES["tiny"]
KV_SENTINEL = 0x7F7F                                                # int16 fill pattern
POOL_SENTINEL = 0x7FC12345                                          # a NaN bit pattern
ROW_SENTINEL = 12345.0                                              # fill of the buffered heads' row buffer

# tolerances (the benchmark spec): embeddings cosine >= 0.9995 and max-abs <= 2e-2;
# logits max-abs <= 5e-2 and argmax agreement >= 99.5 %
EMB_COS, EMB_ABS, LOGIT_ABS, ARGMAX_RATE = 0.9995, 2e-2, 5e-2, 0.995


@pytest.fixture(scope="module")
def weights():
    from paper_2609_25405_b200 import binding as B
    W = synth.Weights(TINY, 0)
    return W, B.DeviceWeights.from_synth(W)


def _engine(weights, n_pages=64, n_slots=4, max_tokens=512, max_segs=16, max_pos=256):
    from paper_2609_25405_b200.engine import Engine
    return Engine(TINY, weights[1], n_pages, n_slots, max_tokens, max_segs, max_pos,
                  kv_fill=KV_SENTINEL, pool_fill=POOL_SENTINEL)


def _check_emb(got, ref):
    cos = float(got @ ref / (np.linalg.norm(got) * np.linalg.norm(ref)))
    assert cos >= EMB_COS, cos
    assert np.max(np.abs(got - ref)) <= EMB_ABS
    assert abs(np.linalg.norm(got) - 1.0) < 1e-5


def run_cfg1(weights, wl, pool_mode="mean", chunkings=None):
    """Runs the tiny mixed workload; returns (logit rows (gpu, oracle), embeddings (gpu, oracle), engine, requests)."""
    from paper_2609_25405_b200 import binding as B
    from paper_2609_25405_b200.engine import Request
    W = weights[0]
    eng = _engine(weights)
    mode = {"mean": B.POOL_MEAN, "last": B.POOL_LAST, "cls": B.POOL_CLS, "wmean": B.POOL_WMEAN}[pool_mode]
    gens = [Request("gen", p) for p in wl.prompts]
    embs = [Request("embed", t, mode) for t in wl.embed_tokens]
    if chunkings is None:
        chunkings = [synth.nominal_chunks(len(t), wl.chunk) for t in wl.embed_tokens]
    chunkings = [list(c) for c in chunkings]
    ora = [T.generate(TINY, W, p, wl.decode_steps + 1) for p in wl.prompts]
    got_logits, ref_logits, got_emb = [], [], {}
    # iteration 0: the four prompts as prefill chunks
    _, lrows, _ = eng.step([(g, g.n_prompt) for g in gens])
    torch.cuda.synchronize()
    for i, g in enumerate(gens):
        got_logits.append(eng.out_logits[lrows[g]].cpu().numpy().copy())
        ref_logits.append(ora[i][1][0])
    # iterations 1..8: one teacher-forced decode token per generation request + embedding chunks
    for s in range(1, wl.decode_steps + 1):
        work = []
        for i, g in enumerate(gens):
            g.tokens.append(int(ora[i][0][s - 1]))
            work.append((g, 1))
        for j, e in enumerate(embs):
            if chunkings[j]:
                work.append((e, chunkings[j].pop(0)))
        _, lrows, erows = eng.step(work)
        torch.cuda.synchronize()
        for i, g in enumerate(gens):
            got_logits.append(eng.out_logits[lrows[g]].cpu().numpy().copy())
            ref_logits.append(ora[i][1][s])
        for e, r in erows.items():
            got_emb[embs.index(e)] = eng.out_emb[r].cpu().numpy().copy()
    assert eng.ctx.status_poll() == 0
    ref_emb = [T.embed(TINY, W, t, pool_mode) for t in wl.embed_tokens]
    return got_logits, ref_logits, got_emb, ref_emb, eng, gens, embs


def test_cfg1_mixed_workload_matches_oracle(weights):
    wl = synth.cfg1_workload()
    gl, rl, ge, re_, eng, gens, embs = run_cfg1(weights, wl)
    assert len(gl) == 36 and sorted(ge) == [0, 1]
    gl, rl = np.stack(gl).astype(np.float64), np.stack(rl)
    assert np.max(np.abs(gl - rl)) <= LOGIT_ABS
    agree = np.mean(np.argmax(gl, -1) == np.argmax(rl, -1))
    assert agree >= ARGMAX_RATE, agree
    for j in (0, 1):
        _check_emb(ge[j].astype(np.float64), re_[j])
    # ---- KV bookkeeping: exactly the expected slots were written, everything else is the sentinel
    from paper_2609_25405_b200 import binding as B
    W = weights[0]
    raw = eng.kv.arena.cpu().view(TINY.L, eng.kv.n_pages, TINY.Hkv, 2, 2, TINY.Dh // 64, 8, 64)   # slot = 8 g + s
    touched = torch.zeros((eng.kv.n_pages, 16), dtype=torch.bool)
    for req in gens + embs:
        n = req.n_done
        assert len(req.pages) == M.pages_needed(n, 16)
        _, _, kv_ref = T.forward(TINY, W, req.tokens[:n], logit_rows=[], return_kv=True)
        for pos in range(n):
            page, slot = M.kv_slot(req.pages, pos, 16)
            touched[page, slot] = True
        for l in range(TINY.L):
            pages = torch.tensor([M.kv_slot(req.pages, p, 16)[0] for p in range(n)], device="cuda")
            slots = torch.tensor([M.kv_slot(req.pages, p, 16)[1] for p in range(n)], device="cuda")
            k_st = eng.kv.rows(l, pages, slots, 0).float().cpu().numpy()   # [n, Hkv, Dh], pair-interleaved
            k_gpu = np.empty_like(k_st)
            k_gpu[..., B.rope_pair_order(TINY.Dh)] = k_st                   # back to the rotary element order
            v_gpu = eng.kv.rows(l, pages, slots, 1).float().cpu().numpy()
            assert np.max(np.abs(k_gpu - kv_ref[l][0])) < 5e-3
            assert np.max(np.abs(v_gpu - kv_ref[l][1])) < 5e-3
    untouched = ~touched.view(-1, 2, 8)[None, :, None, :, None, None, :, None].expand_as(raw)
    assert torch.all(raw[untouched] == KV_SENTINEL)
    # ---- pool bookkeeping: counters equal the oracle's integers; unused slots keep the sentinel
    meta = eng.pool.meta().cpu().numpy()
    sizes = [synth.nominal_chunks(len(t), wl.chunk) for t in wl.embed_tokens]
    for j, e in enumerate(embs):
        cnt, chunks = M.pool_counters_after(sizes[j])
        assert list(meta[e.slot].astype(np.int64)) == [cnt, chunks, 1, 1]
    for s in range(eng.pool.n_slots):
        if s not in [e.slot for e in embs]:
            assert np.all(meta[s] == POOL_SENTINEL)
            assert torch.all(eng.pool.arena[s * TINY.d:(s + 1) * TINY.d] == POOL_SENTINEL)
    # rows of the outputs that no segment named stay zero (as allocated)
    assert torch.all(eng.out_emb[2:] == 0)
    eng.close()


def test_cfg1_mean_state_after_each_chunk(weights):
    """Pool sum and count after every chunk equal the oracle's prefix sums (Eq. 1-2)."""
    from paper_2609_25405_b200 import binding as B
    from paper_2609_25405_b200.engine import Request
    W = weights[0]
    toks = synth.cfg1_workload().embed_tokens[0]
    hh, _ = T.forward(TINY, W, toks, logit_rows=[])
    eng = _engine(weights)
    req = Request("embed", toks, B.POOL_MEAN)
    at = 0
    for k, c in enumerate([33, 1, 50, 16]):
        eng.step([(req, c)])
        at += c
        torch.cuda.synchronize()
        meta = eng.pool.meta()[req.slot].cpu().numpy()
        assert list(meta[:2]) == list(M.pool_counters_after([33, 1, 50, 16][:k + 1]))
        S = eng.pool.sums()[req.slot].cpu().numpy().astype(np.float64)
        ref = hh[:at].sum(0)
        # every row of the unit-rms hidden states carries an fp16-path error of a few 1e-3 against the
        # oracle; the errors of different rows are largely independent, so the sum's error grows like
        # sqrt(rows): measured 6.5e-3 to 7.2e-3 x sqrt(rows) over these four states
        print(f"\n  mean-pool state after {at} rows: max |S - oracle| = {np.max(np.abs(S - ref)):.3e} "
              f"({np.max(np.abs(S - ref)) / at:.2e} per row, {np.max(np.abs(S - ref)) / np.sqrt(at):.2e} per sqrt(row))")
        assert np.max(np.abs(S - ref)) <= 2e-2 * np.sqrt(at)
    assert eng.ctx.status_poll() == 0
    eng.close()


@pytest.mark.parametrize("mode", ["mean", "last", "cls", "wmean"])
def test_random_chunkings_and_chunk_size_one(weights, mode):
    """Any partition of the text gives the single-pass embedding (chunks straddle pages)."""
    wl = synth.cfg1_workload(seed=77, embed_lens=(53, 19))
    rng = np.random.default_rng(5)
    for trial in range(3):
        parts = [synth.random_partition(rng, 53, 23), [1] * 19] if trial == 0 else \
                [synth.random_partition(rng, 53, 40), synth.random_partition(rng, 19, 7)]
        parts = [p[:8] + ([sum(p[8:])] if len(p) > 8 else []) for p in parts]   # at most 9 iterations
        wl.decode_steps = 9 if any(len(p) > 8 for p in parts) else 8
        gl, rl, ge, re_, eng, _, _ = run_cfg1(weights, wl, pool_mode=mode, chunkings=parts)
        for j in (0, 1):
            _check_emb(ge[j].astype(np.float64), re_[j])
        eng.close()


def test_buffered_max_head(weights):
    """Buffered head (Section 3.3): every chunk appends its final hidden states to the slot's row
    buffer; the final chunk emits the element-wise maximum over all rows.  Checked: the embedding
    against the single-pass oracle for several partitions (one with a one-row final chunk, so a
    single block folds in every buffered row), the buffered rows against the oracle's final hidden
    states, rows past the text untouched, counters exact, and a request without a buffer rejected."""
    from paper_2609_25405_b200 import binding as B
    from paper_2609_25405_b200.engine import Request
    W = weights[0]
    rng = np.random.default_rng(21)
    toks = synth.token_ids(rng, 150, TINY.V)
    ref = T.embed(TINY, W, toks, "max")
    hh, _ = T.forward(TINY, W, toks, logit_rows=[])
    other = synth.token_ids(rng, 40, TINY.V)
    for sizes in ([150], [70, 80], [33, 64, 52, 1], [1, 149]):
        eng = _engine(weights, n_pages=96, max_tokens=512, max_pos=256)
        rows = eng.pool.attach_row_buffer(160, fill=ROW_SENTINEL)
        e = Request("embed", toks, B.POOL_MAX)
        m = Request("embed", other, B.POOL_MEAN)            # shares the steps; must not disturb the buffer
        er = {}
        for k, c in enumerate(sizes):
            work = [(e, c)] + ([(m, 40)] if k == 0 else [])
            _, _, er = eng.step(work)
            torch.cuda.synchronize()
            meta = eng.pool.meta()[e.slot].cpu().numpy()
            done = sum(sizes[:k + 1])
            assert list(meta) == [done, k + 1, B.POOL_MAX, int(k == len(sizes) - 1)]
        assert eng.ctx.status_poll() == 0
        _check_emb(eng.out_emb[er[e]].cpu().numpy().astype(np.float64), ref)
        buf = rows[e.slot].cpu().numpy()
        assert np.max(np.abs(buf[:150] - hh)) <= 2e-2 * max(1.0, float(np.max(np.abs(hh))))
        assert np.all(buf[150:] == ROW_SENTINEL)
        assert np.all(rows[m.slot].cpu().numpy() == ROW_SENTINEL)
        # the emitted vector is exactly the normalised maximum of what the buffer holds
        mx = buf[:150].max(0).astype(np.float64)
        assert np.max(np.abs(eng.out_emb[er[e]].cpu().numpy() - mx / np.linalg.norm(mx))) < 1e-6
        eng.close()
    eng = _engine(weights)
    e = Request("embed", toks[:20], B.POOL_MAX)
    with pytest.raises(B.HbError):
        eng.step([(e, 20)])                                 # no row buffer attached
    eng.pool.attach_row_buffer(16)
    with pytest.raises(B.HbError):
        eng.step([(e, 20)])                                 # text longer than the buffer's rows
    eng.close()


def test_chunked_versus_own_single_pass_within_the_papers_printed_bounds(weights):
    """The paper measures how well its chunked path reproduces its own single pass (appendix "Pooling
    Equivalence": per head and chunk size the minimum cosine and the p99 relative L2 over 250
    samples; tests/golden/pooling_equivalence.txt).  This path must do at least as well against ITS
    own single pass, at the same chunk sizes, for every sampled text."""
    import os
    from paper_2609_25405_b200 import binding as B
    from paper_2609_25405_b200.engine import Request
    path = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden", "pooling_equivalence.txt")
    rows = [ln.split() for ln in open(path) if ln.strip() and not ln.startswith("#")]
    modes = {"mean": B.POOL_MEAN, "cls": B.POOL_CLS, "wmean": B.POOL_WMEAN}
    rng = np.random.default_rng(31)
    texts = [synth.token_ids(rng, n, TINY.V) for n in (300, 777, 1500, 2048)]
    eng = _engine(weights, n_pages=2 * 130 + 8, n_slots=4, max_tokens=2048, max_segs=8, max_pos=2048)

    def embed(toks, sizes, mode):
        r = Request("embed", toks, mode)
        er = {}
        for c in sizes:
            _, _, er = eng.step([(r, c)])
        torch.cuda.synchronize()
        out = eng.out_emb[er[r]].cpu().numpy().astype(np.float64)
        eng.release(r)
        return out

    single = {(h, i): embed(t, [len(t)], m) for h, m in modes.items() for i, t in enumerate(texts)}
    for head, C, cos_min, _, _, _, l2_p99 in rows:
        for i, t in enumerate(texts):
            if len(t) <= int(C):
                continue                                   # one chunk: nothing to compare
            e = embed(t, synth.nominal_chunks(len(t), int(C)), modes[head])
            ref = single[(head, i)]
            assert float(e @ ref) >= float(cos_min), (head, C, len(t))
            assert np.linalg.norm(e - ref) / np.linalg.norm(ref) <= float(l2_p99), (head, C, len(t))
    assert eng.ctx.status_poll() == 0
    eng.close()


def test_long_chunks_take_the_tensor_core_attention_path(weights):
    """Chunks of more than 64 query rows run on the tcgen05 attention kernel (128-row tiles, ragged
    last tile, several key tiles, chunks that start inside a page); shorter remainders on the
    mma.sync kernel.  Both must reproduce the single-pass oracle."""
    from paper_2609_25405_b200 import binding as B
    from paper_2609_25405_b200.engine import Request
    W = weights[0]
    rng = np.random.default_rng(11)
    e1 = Request("embed", synth.token_ids(rng, 300, TINY.V), B.POOL_MEAN)
    e2 = Request("embed", synth.token_ids(rng, 213, TINY.V), B.POOL_LAST)
    g = Request("gen", synth.token_ids(rng, 200, TINY.V))
    eng = _engine(weights, n_pages=96, max_tokens=768, max_pos=320)
    _, _, _ = eng.step([(e1, 130), (g, 129), (e2, 213)])
    _, lr, er = eng.step([(e1, 170), (g, 71)])
    torch.cuda.synchronize()
    assert eng.ctx.status_poll() == 0
    _check_emb(eng.out_emb[er[e1]].cpu().numpy().astype(np.float64), T.embed(TINY, W, e1.tokens, "mean"))
    _, ref = T.forward(TINY, W, g.tokens, logit_rows=[199])
    assert np.max(np.abs(eng.out_logits[lr[g]].cpu().numpy() - ref[0])) <= LOGIT_ABS
    eng2 = _engine(weights, n_pages=96, max_tokens=768, max_pos=320)
    e2b = Request("embed", e2.tokens, B.POOL_LAST)
    _, _, er = eng2.step([(e2b, 213)])
    torch.cuda.synchronize()
    _check_emb(eng2.out_emb[er[e2b]].cpu().numpy().astype(np.float64), T.embed(TINY, W, e2.tokens, "last"))
    eng.close(); eng2.close()


def test_batch_composition_independence(weights):
    """A request's outputs do not depend on which other requests share its batch: solo runs
    equal in-batch runs bit for bit (no atomics, request-local split decisions)."""
    from paper_2609_25405_b200 import binding as B
    from paper_2609_25405_b200.engine import Request
    wl = synth.cfg1_workload(seed=5)
    # in-batch
    eng = _engine(weights)
    g = Request("gen", wl.prompts[0]); e = Request("embed", wl.embed_tokens[1], B.POOL_MEAN)
    other = [Request("gen", wl.prompts[1]), Request("embed", wl.embed_tokens[0], B.POOL_LAST)]
    _, lr, er = eng.step([(other[1], 60), (g, 64), (e, 37), (other[0], 64)])
    torch.cuda.synchronize()
    l_batch = eng.out_logits[lr[g]].clone(); e_batch = eng.out_emb[er[e]].clone()
    eng.close()
    # solo
    eng = _engine(weights)
    g2 = Request("gen", wl.prompts[0]); e2 = Request("embed", wl.embed_tokens[1], B.POOL_MEAN)
    _, lr, _ = eng.step([(g2, 64)])
    torch.cuda.synchronize()
    l_solo = eng.out_logits[lr[g2]].clone()
    _, _, er = eng.step([(e2, 37)])
    torch.cuda.synchronize()
    e_solo = eng.out_emb[er[e2]].clone()
    eng.close()
    assert torch.equal(l_batch, l_solo)
    assert torch.equal(e_batch, e_solo)


@pytest.mark.parametrize("width", ["7b", "1b"])
@pytest.mark.parametrize("lora_rank", [0, 16])
def test_batch_composition_independence_across_step_sizes_full_width(lora_rank, width):
    """7B-class (and 1B-class) width, two layers, random weights drawn on the device, a 4096-row context: a
    generation and an embedding request run alone, every piece of work a step of its own (300, 512, 1
    and 188 rows, most of which take single-CTA GEMM tiles), equal bit for bit the same requests inside
    full 4096-row steps (CTA-pair tiles; the down projection's K is split in two in both).  No oracle
    here: the point is that tile variants and K splits chosen per step or per context never change a
    row's bits."""
    from paper_2609_25405_b200 import binding as B
    from paper_2609_25405_b200.engine import Engine, Request
    shape = synth.SHAPES[width].with_layers(2)
    dw = B.DeviceWeights.random_on_device(shape, seed=3)
    lora = B.DeviceLora.random_on_device(shape, lora_rank) if lora_rank else None
    rng = np.random.default_rng(77)
    emb_toks = synth.token_ids(rng, 700, shape.V)
    gen_toks = synth.token_ids(rng, 300, shape.V)

    def run(fill):
        eng = Engine(shape, dw, n_pages=1024, n_slots=64, max_tokens=4096, max_segs=256, max_pos=1024, lora=lora)
        e, g = Request("embed", list(emb_toks), B.POOL_MEAN), Request("gen", list(gen_toks))
        outs, extra = [], []
        for step in range(2):
            work = [(g, 300)] if step == 0 else [(g, 1)]
            if step == 1:
                g.tokens.append(7)
            work.append((e, 512 if step == 0 else 188))
            rows = sum(n for _, n in work)
            for _ in range(200 if fill else 0):      # 200 more logits rows: the LM head takes pair tiles
                f = Request("gen", synth.token_ids(rng, 4, shape.V))
                work.append((f, 4)); extra.append(f); rows += 4
            while fill and rows < 4096:
                n = min(512, 4096 - rows)
                f = Request("embed", synth.token_ids(rng, n, shape.V), B.POOL_LAST)
                work.append((f, n)); extra.append(f); rows += n
            for part in ([work] if fill else [[w] for w in work]):
                _, l1, e1 = eng.step(part)
                torch.cuda.synchronize()
                if g in l1:
                    outs.append(eng.out_logits[l1[g]].clone())
                if e in e1:
                    outs.append(eng.out_emb[e1[e]].clone())
            for f in extra:
                eng.release(f)
            extra = []
        assert eng.ctx.status_poll() == 0
        eng.close()
        return outs

    solo, batch = run(False), run(True)
    assert len(solo) == len(batch) == 3
    for a, b in zip(solo, batch):
        assert torch.isfinite(a).all() and torch.equal(a, b)


def test_argmax_kernel_lowest_index_on_ties(weights):
    eng = _engine(weights)
    lg = torch.randn(5, TINY.V, device="cuda")
    lg[1, 17] = 50.0; lg[1, 900] = 50.0; lg[3, 0] = 60.0
    out = torch.zeros(5, dtype=torch.int32, device="cuda")
    eng.ctx.argmax(lg, 5, out)
    torch.cuda.synchronize()
    ref = [T.argmax_lowest(r) for r in lg.cpu().numpy()]
    assert out.cpu().tolist() == ref and ref[1] == 17 and ref[3] == 0
    eng.close()


def test_degenerate_batches(weights):
    """Empty batch; decode-only batch; a single one-token embedding request."""
    from paper_2609_25405_b200 import binding as B
    from paper_2609_25405_b200.engine import Request
    W = weights[0]
    eng = _engine(weights)
    empty = B.Batch([], np.zeros(0, dtype=B.SEG_DTYPE), [], 0, 0)
    eng.ctx.mixed_step(empty, eng.weights, eng.kv, eng.pool, eng.out_logits, eng.out_emb)
    assert eng.ctx.last_launch_count() == 0
    e = Request("embed", [5], B.POOL_LAST)
    _, _, er = eng.step([(e, 1)])
    torch.cuda.synchronize()
    _check_emb(eng.out_emb[er[e]].cpu().numpy().astype(np.float64), T.embed(TINY, W, [5], "last"))
    g = Request("gen", [3, 9])
    eng.step([(g, 1)])                     # non-final prefill row: no logits
    _, lr, _ = eng.step([(g, 1)])          # final prefill row
    torch.cuda.synchronize()
    _, ref = T.forward(TINY, W, [3, 9], logit_rows=[1])
    assert np.max(np.abs(eng.out_logits[lr[g]].cpu().numpy() - ref[0])) <= LOGIT_ABS
    assert eng.ctx.status_poll() == 0
    eng.close()


def test_expired_wait_sets_status_and_context_stays_usable(weights):
    """Failure detection without a fault: a bounded wait that runs out raises a status bit, the host
    reads it as HB_ERR_DEVICE_STATUS, polling clears it, and the next step runs normally."""
    from paper_2609_25405_b200 import binding as B
    from paper_2609_25405_b200.engine import Request
    W = weights[0]
    eng = _engine(weights)
    assert eng.ctx.status_poll() == 0
    eng.ctx.selftest_wait_expiry(limit_ms=20)
    assert eng.ctx.status_poll() == 32          # the self-test's bit; the poll clears the word
    assert eng.ctx.status_poll() == 0
    e = Request("embed", [5, 6, 7], B.POOL_MEAN)
    _, _, er = eng.step([(e, 3)])
    torch.cuda.synchronize()
    _check_emb(eng.out_emb[er[e]].cpu().numpy().astype(np.float64), T.embed(TINY, W, [5, 6, 7], "mean"))
    assert eng.ctx.status_poll() == 0
    eng.close()


def test_bad_descriptor_enqueues_nothing(weights):
    from paper_2609_25405_b200 import binding as B
    from paper_2609_25405_b200.engine import build_batch
    eng = _engine(weights)
    ent = [dict(kind=B.KIND_DECODE, tokens=[1], pos_start=3, pages=[999], is_final=True)]
    batch, _ = build_batch(ent, 16)
    with pytest.raises(B.HbError) as err:
        eng.ctx.mixed_step(batch, eng.weights, eng.kv, eng.pool, eng.out_logits, eng.out_emb)
    assert err.value.code == -6
    torch.cuda.synchronize()
    assert torch.all(eng.kv.arena == KV_SENTINEL)
    eng.close()


class _ScaledWeights:
    """synth.Weights with the FFN-norm gain of every layer set to `ffn_gain` (a power of two, so it is
    bf16-exact): the inputs of the gate/up projection, and with them the SwiGLU outputs, leave the
    range of the N(0, 0.02^2), gain-1 models of the configurations, while attention stays as it is."""

    def __init__(self, W, ffn_gain, nan_token=None):
        self.W, self.shape, self.ffn_gain, self.nan_token = W, W.shape, np.float32(ffn_gain), nan_token

    def layer(self, l):
        w = dict(self.W.layer(l))
        w["ffn_norm"] = np.full_like(w["ffn_norm"], self.ffn_gain)
        return w

    @property
    def tok_emb(self):
        t = self.W.tok_emb
        if self.nan_token is not None:
            t = t.copy()
            t[self.nan_token] = np.nan
        return t

    @property
    def lm_head(self):
        return self.W.lm_head

    @property
    def final_norm(self):
        return self.W.final_norm


def test_fp16_range_large_ffn_gain_and_nan():
    """Where the fp16 operand range ends.  With an FFN-norm gain of 64 the inputs of gate/up are 64
    times the configurations' and the SwiGLU outputs about 4000 times (hundreds to thousands): still
    inside fp16, the step matches the oracle within the usual tolerances with a clean status word.
    With a gain of 2048 the SwiGLU outputs pass 65504: they are stored saturated, the step REPORTS it
    (status bit 64), outputs stay finite and the context stays usable.  A NaN in the residual stream
    (a NaN token-embedding row) is reported the same way and reaches the logits as NaN instead of
    being clamped to a finite number."""
    from paper_2609_25405_b200 import binding as B
    from paper_2609_25405_b200.engine import Engine, Request
    rng = np.random.default_rng(99)
    toks = synth.token_ids(rng, 90, TINY.V)
    prompt = synth.token_ids(rng, 70, TINY.V)

    def run(W):
        eng = Engine(TINY, B.DeviceWeights.from_synth(W), 64, 4, 512, 16, 256)
        e, g = Request("embed", toks, B.POOL_MEAN), Request("gen", prompt)
        _, lr, er = eng.step([(g, 70), (e, 90)])
        torch.cuda.synchronize()
        out = eng.out_logits[lr[g]].cpu().numpy().astype(np.float64), eng.out_emb[er[e]].cpu().numpy().astype(np.float64)
        status = eng.ctx.status_poll()
        assert eng.ctx.status_poll() == 0            # polling cleared it; the context is usable
        eng.close()
        return out, status

    base = synth.Weights(TINY, 0)
    # (1) inside the range
    W = _ScaledWeights(base, 64.0)
    (lg, emb), status = run(W)
    assert status == 0
    _, ref_lg = T.forward(TINY, W, prompt, logit_rows=[69])
    assert np.max(np.abs(lg - ref_lg[0])) <= LOGIT_ABS
    _check_emb(emb, T.embed(TINY, W, toks, "mean"))
    # (2) SwiGLU outputs beyond the largest finite half: saturated and reported
    (lg, emb), status = run(_ScaledWeights(base, 2048.0))
    assert status & 64
    assert np.all(np.isfinite(lg)) and np.all(np.isfinite(emb))
    # (3) NaN in: reported, and NaN (not a clamped number) out
    (lg, emb), status = run(_ScaledWeights(base, 1.0, nan_token=int(prompt[-1])))
    assert status & 64
    assert np.all(np.isnan(lg))

"""hb_pool_chunk_noalloc, the pooler entry point for callers that cannot allocate device memory
(its scratch is a fixed array inside the library, so no context and no cudaMalloc are involved).

Checked against hb_pool_chunk, the context-based entry point that runs the same pooler with scratch
from the context's workspace: two calls in a row (a first chunk, then the final chunk of the same
request) must leave the same pool slot and emit the same embedding, for every head the call
accepts.  The second call also shows that the shared array, which still holds the first call's
partial sums and counters, is cleared where it has to be.  A second group runs the largest chunk the
fixed array can hold (its partial sums then end exactly at the array's tail words) and compares with
the CPU oracle's Eq. 1-2 pooler, and a third checks that pointers a caller cut out of its own arena
at an odd offset are refused on the host.  Collected last so that a failure here cannot hide any
other test.
"""
import numpy as np
import pytest
import torch

from paper_2609_25405_b200 import synth

pytestmark = pytest.mark.gpu

TOL = 1e-5     # the pooler tests' tolerance on sums (relative to the row count) and embeddings


@pytest.mark.parametrize("mode_name", ["mean", "last", "wmean", "cls"])
def test_noalloc_pooler_matches_context_pooler_on_two_calls(mode_name):
    from paper_2609_25405_b200 import binding as B
    d = 2048
    shape = synth.ModelShape("pool", 1, d, d // 64, d // 64, 64, 64, 64)
    ctx = B.Context(B.model_cfg(shape, 64), 2048, 8, 64)
    mode = {"mean": B.POOL_MEAN, "last": B.POOL_LAST, "wmean": B.POOL_WMEAN, "cls": B.POOL_CLS}[mode_name]
    rng = np.random.default_rng(7)
    gain = B.bf16_from_f32(synth.bf16_bits_to_f32(synth.f32_to_bf16_bits(
        1.0 + 0.1 * rng.standard_normal(d, dtype=np.float32))))
    chunks = [torch.from_numpy(2.0 * rng.standard_normal((n, d), dtype=np.float32)).cuda() for n in (517, 100)]

    def fresh():
        return (torch.full((d,), float("nan"), device="cuda"),
                torch.full((4,), 777, dtype=torch.int32, device="cuda"), torch.zeros(d, device="cuda"))

    ref_sum, ref_meta, ref_emb = fresh()
    new_sum, new_meta, new_emb = fresh()
    for k, x in enumerate(chunks):
        first, final = (k == 0), (k == len(chunks) - 1)
        ctx.pool_chunk(x, gain, x.shape[0], mode, first, final, ref_sum, ref_meta, ref_emb)
        rc = B.pool_chunk_noalloc(x, gain, x.shape[0], d, shape.rms_eps, mode, first, final, new_sum, new_meta,
                                  new_emb)
        assert rc == 0
        torch.cuda.synchronize()
        assert torch.equal(new_meta, ref_meta)
        if mode_name in ("mean", "wmean"):
            err = (new_sum - ref_sum).abs().max().item()
            assert err <= TOL * max(1.0, ref_sum.abs().max().item()), err
        if mode_name == "cls":                       # the retained first row lives in the slot
            assert torch.equal(new_sum, ref_sum)
    assert (new_emb - ref_emb).abs().max().item() <= TOL
    assert abs(new_emb.norm().item() - 1.0) <= 1e-5
    assert ctx.status_poll() == 0
    ctx.close()


def test_noalloc_pooler_rejects_sizes_beyond_its_fixed_scratch():
    from paper_2609_25405_b200 import binding as B
    d = 256
    x = torch.zeros((8, d), device="cuda")
    gain = torch.ones(d, dtype=torch.bfloat16, device="cuda")
    s, m, e = torch.zeros(d, device="cuda"), torch.zeros(4, dtype=torch.int32, device="cuda"), torch.zeros(d, device="cuda")
    assert B.pool_chunk_noalloc(x, gain, B.NOALLOC_MAX_ROWS + 1, d, 1e-5, B.POOL_MEAN, True, True, s, m, e) == -5
    assert B.pool_chunk_noalloc(x, gain, 8, B.NOALLOC_MAX_DMODEL + 4, 1e-5, B.POOL_MEAN, True, True, s, m, e) == -5
    torch.cuda.synchronize()
    assert torch.all(m == 0) and torch.all(e == 0)          # nothing ran
    assert B.pool_chunk_noalloc(x, gain, 8, d, 1e-5, B.POOL_MEAN, True, True, s, m, e) == 0
    torch.cuda.synchronize()
    assert m.tolist() == [8, 1, B.POOL_MEAN, 1]


@pytest.mark.parametrize("mode_name", ["mean", "wmean"])
def test_noalloc_pooler_at_its_size_limit_matches_oracle(mode_name):
    """The largest chunk the fixed array holds: NOALLOC_MAX_ROWS rows of NOALLOC_MAX_DMODEL columns,
    i.e. 64 partial-sum records that end exactly where the array's tail words (arrival counter,
    status) begin.  Two calls in a row (the full-size first chunk, then a ragged final chunk) against
    the oracle's incremental pooler (Eq. 1-2), with the tolerances of the pooler's own parity test."""
    from oracle import method as M
    from oracle import transformer as T
    from paper_2609_25405_b200 import binding as B
    d, n0 = B.NOALLOC_MAX_DMODEL, B.NOALLOC_MAX_ROWS
    shape = synth.ModelShape("pool", 1, d, d // 64, d // 64, 64, 64, 64)
    mode = B.POOL_MEAN if mode_name == "mean" else B.POOL_WMEAN
    rng = np.random.default_rng(11)
    gain_f = synth.bf16_bits_to_f32(synth.f32_to_bf16_bits(1.0 + 0.1 * rng.standard_normal(d, dtype=np.float32)))
    gain = B.bf16_from_f32(gain_f)
    slot_sum = torch.full((d,), float("nan"), device="cuda")
    slot_meta = torch.full((4,), 777, dtype=torch.int32, device="cuda")
    out = torch.full((d,), 5.0, device="cuda")
    st = M.RequestState(shape)
    at, ref = 0, None
    for k, n in enumerate((n0, 1003)):
        x = 3.0 * rng.standard_normal((n, d), dtype=np.float32)
        H = T.rmsnorm(x.astype(np.float64), gain_f.astype(np.float64), shape.rms_eps)
        final = (k == 1)
        ref = M.pool_update(st, H, mode_name, final,
                            weights=np.arange(at + 1, at + n + 1) if mode_name == "wmean" else None)
        at += n
        rc = B.pool_chunk_noalloc(torch.from_numpy(x).cuda(), gain, n, d, shape.rms_eps, mode, k == 0, final,
                                  slot_sum, slot_meta, out)
        assert rc == 0
        torch.cuda.synchronize()
        assert slot_meta.tolist() == [st.count, st.chunks, mode, 1 if final else 0]
        S = slot_sum.cpu().numpy().astype(np.float64)
        assert np.max(np.abs(S - st.S)) <= 1e-5 * np.sqrt(st.count) * 4 + 1e-6 * np.max(np.abs(st.S))
        if not final:
            assert torch.all(out == 5.0)             # nothing is emitted before the final chunk
    got = out.cpu().numpy().astype(np.float64)
    assert float(got @ ref) >= 1 - 1e-6 and np.max(np.abs(got - ref)) <= TOL


def test_noalloc_pooler_refuses_misaligned_views():
    """A caller that sub-allocates from its own arena may pass a view that starts in the middle of a
    16-byte vector.  The kernel would fault on it; the entry point (and hb_pool_chunk) must refuse it
    on the host and launch nothing."""
    from paper_2609_25405_b200 import binding as B
    d = 256
    shape = synth.ModelShape("pool", 1, d, d // 64, d // 64, 64, 64, 64)
    arena = torch.zeros(8 * d + 64, device="cuda")
    gain_arena = torch.ones(d + 8, dtype=torch.bfloat16, device="cuda")
    x, x_off = arena[0:8 * d].view(8, d), arena[1:8 * d + 1].view(8, d)         # 4 bytes into a vector
    s, s_off = torch.zeros(d + 4, device="cuda")[:d], torch.zeros(d + 4, device="cuda")[2:d + 2]
    e = torch.zeros(d, device="cuda")
    m = torch.zeros(4, dtype=torch.int32, device="cuda")
    g, g_off = gain_arena[:d], gain_arena[1:d + 1]                               # 2 bytes off
    args = lambda xx, gg, ss: (xx, gg, 8, d, 1e-5, B.POOL_MEAN, True, True, ss, m, e)
    assert B.pool_chunk_noalloc(*args(x_off, g, s)) == -1
    assert B.pool_chunk_noalloc(*args(x, g_off, s)) == -1
    assert B.pool_chunk_noalloc(*args(x, g, s_off)) == -1
    ctx = B.Context(B.model_cfg(shape, 64), 64, 8, 64)
    with pytest.raises(B.HbError) as err:
        ctx.pool_chunk(x_off, g, 8, B.POOL_MEAN, True, True, s, m, e)
    assert err.value.code == -1
    torch.cuda.synchronize()
    assert torch.all(m == 0) and torch.all(e == 0)                               # nothing ran
    assert B.pool_chunk_noalloc(*args(x, g, s)) == 0
    torch.cuda.synchronize()
    assert m.tolist() == [8, 1, B.POOL_MEAN, 1]
    assert ctx.status_poll() == 0
    ctx.close()

"""hb_pool_chunk_noalloc, the pooler entry point for callers that cannot allocate device memory
(its scratch is a fixed array inside the library, so no context and no cudaMalloc are involved).

Checked against hb_pool_chunk, the context-based entry point that runs the same pooler with scratch
from the context's workspace: two calls in a row (a first chunk, then the final chunk of the same
request) must leave the same pool slot and emit the same embedding.  The second call also shows
that the shared array, which still holds the first call's partial sums and counters, is cleared
where it has to be.  Collected last so that a failure here cannot hide any other test.
"""
import numpy as np
import pytest
import torch

from paper_2609_25405_b200 import synth

pytestmark = pytest.mark.gpu

TOL = 1e-5     # the pooler tests' tolerance on sums (relative to the row count) and embeddings


@pytest.mark.parametrize("mode_name", ["mean", "last"])
def test_noalloc_pooler_matches_context_pooler_on_two_calls(mode_name):
    from paper_2609_25405_b200 import binding as B
    d = 2048
    shape = synth.ModelShape("pool", 1, d, d // 64, d // 64, 64, 64, 64)
    ctx = B.Context(B.model_cfg(shape, 64), 2048, 8, 64)
    mode = B.POOL_MEAN if mode_name == "mean" else B.POOL_LAST
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
        if mode_name == "mean":
            err = (new_sum - ref_sum).abs().max().item()
            assert err <= TOL * int(ref_meta[0]), err
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

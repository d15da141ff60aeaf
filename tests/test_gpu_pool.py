"""Parity of the incremental pooler kernel on its own (through the C-ABI) with the oracle's
Eq. 1-2 pooler: state after every chunk, emitted embedding, both heads, ragged row counts."""
import numpy as np
import pytest
import torch

from oracle import method as M
from oracle import transformer as T
from paper_2609_25405_b200 import synth

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("d", [256, 2048, 4096])
@pytest.mark.parametrize("mode", ["mean", "last", "cls", "wmean"])
def test_pool_chunks_match_oracle(d, mode):
    from paper_2609_25405_b200 import binding as B
    shape = synth.ModelShape("pool", 1, d, d // 64, d // 64, 64, 64, 64)
    ctx = B.Context(B.model_cfg(shape, 64), 1024, 8, 64)
    rng = np.random.default_rng(d)
    gain_f = synth.bf16_bits_to_f32(synth.f32_to_bf16_bits(1.0 + 0.1 * rng.standard_normal(d, dtype=np.float32)))
    gain = B.bf16_from_f32(gain_f)
    sizes = [1, 31, 32, 33, 200, 517]
    slot_sum = torch.full((d,), float("nan"), device="cuda")
    slot_meta = torch.full((4,), 12345, dtype=torch.int32, device="cuda")
    out = torch.zeros(d, device="cuda")
    st = M.RequestState(shape)
    code = {"mean": B.POOL_MEAN, "last": B.POOL_LAST, "cls": B.POOL_CLS, "wmean": B.POOL_WMEAN}[mode]
    at = 0
    for k, n in enumerate(sizes):
        x = (3.0 * rng.standard_normal((n, d), dtype=np.float32)).astype(np.float32)
        H = T.rmsnorm(x.astype(np.float64), gain_f.astype(np.float64), shape.rms_eps)
        final = (k == len(sizes) - 1)
        ref = M.pool_update(st, H, mode, final, weights=np.arange(at + 1, at + n + 1) if mode == "wmean" else None)
        at += n
        ctx.pool_chunk(torch.from_numpy(x).cuda(), gain, n, code, k == 0, final, slot_sum, slot_meta, out)
        torch.cuda.synchronize()
        meta = slot_meta.cpu().numpy()
        assert list(meta) == [st.count, st.chunks, code, 1 if final else 0]
        if mode in ("mean", "wmean"):
            S = slot_sum.cpu().numpy().astype(np.float64)
            err = np.max(np.abs(S - st.S))
            print(f"\n  d={d} {mode} count={st.count}: max |S - oracle| = {err:.3e} = {err / np.max(np.abs(st.S)):.2e} x max|S|"
                  f" = {err / (np.sqrt(st.count) * 2.0 ** -24 * np.max(np.abs(st.S))):.2f} x sqrt(n) u max|S|")
            assert err <= 1e-5 * np.sqrt(st.count) * 4 + 1e-6 * np.max(np.abs(st.S))
        if mode == "cls":
            S = slot_sum.cpu().numpy().astype(np.float64)
            assert np.max(np.abs(S - st.retained)) <= 1e-5
    got = out.cpu().numpy().astype(np.float64)
    assert float(got @ ref) >= 1 - 1e-6 and np.max(np.abs(got - ref)) <= 1e-5
    assert ctx.status_poll() == 0
    ctx.close()

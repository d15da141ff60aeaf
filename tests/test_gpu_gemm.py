"""Parity of the tcgen05 projection GEMM (through the C-ABI) with the oracle's definition."""
import numpy as np
import pytest
import torch

from oracle import ops
from paper_2609_25405_b200 import synth

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx():
    from paper_2609_25405_b200 import binding as B
    c = B.Context(B.model_cfg(synth.SHAPES["tiny"], 64), 128, 8, 64)
    yield c
    c.close()


def _bf16_exact(rng, shape, std):
    a = rng.standard_normal(shape, dtype=np.float32) * np.float32(std)
    return synth.bf16_bits_to_f32(synth.f32_to_bf16_bits(a)).reshape(shape)


def _f16_exact(rng, shape, std):
    a = rng.standard_normal(shape, dtype=np.float32) * np.float32(std)
    return a.astype(np.float16).astype(np.float32)


# (M, N, K): several tiles, ragged M tail, N not a multiple of the tile, K not a multiple of 64,
# a single row, more tiles than SMs (persistent loop + both TMEM accumulators), long K (ring wraps)
SHAPES = [(128, 256, 64), (68, 768, 256), (300, 328, 200), (1, 1024, 256), (4, 1024, 512),
          (515, 2048, 1024), (2500, 3072, 256), (256, 256, 4096), (4096, 1536, 512), (1030, 4160, 128), (2100, 4608, 192)]


@pytest.mark.parametrize("M,N,K", SHAPES)
@pytest.mark.parametrize("epi", ["f32", "f16", "resid", "swiglu"])
def test_gemm_matches_oracle(ctx, M, N, K, epi):
    from paper_2609_25405_b200 import binding as B
    if epi == "swiglu" and N % 16:
        pytest.skip("swiglu needs N % 16 == 0")
    rng = np.random.default_rng(M * 7 + N * 3 + K)
    A = _f16_exact(rng, (M, K), 1.0)         # activations are fp16; bf16 weight values repacked to fp16
    Bm = _bf16_exact(rng, (N, K), 0.05)
    dA, dB = torch.from_numpy(A.astype(np.float16)).cuda(), B.pack_f16_(B.bf16_from_f32(Bm))
    scale = 0.05 * np.sqrt(K)
    if epi == "f32":
        out = torch.full((M + 1, N), 768.0, dtype=torch.float32, device="cuda")
        ctx.gemm(dA, dB, out, M, N, K, B.EPI_F32)
        ref = ops.projection(A, Bm, "plain")
        tol = 2e-5 * scale * np.sqrt(K) + 1e-6
    elif epi == "f16":
        out = torch.full((M + 1, N), 768.0, dtype=torch.float16, device="cuda")
        ctx.gemm(dA, dB, out, M, N, K, B.EPI_F16)
        ref = ops.projection(A, Bm, "plain")
        tol = None
    elif epi == "resid":
        C0 = rng.standard_normal((M + 1, N), dtype=np.float32)
        out = torch.from_numpy(C0.copy()).cuda()
        ctx.gemm(dA, dB, out, M, N, K, B.EPI_RESID_F32)
        ref = ops.projection(A, Bm, "resid", C0[:M])
        tol = 2e-5 * scale * np.sqrt(K) + 1e-5
    else:
        out = torch.full((M + 1, N // 2), 768.0, dtype=torch.float16, device="cuda")
        ctx.gemm(dA, dB, out, M, N, K, B.EPI_SWIGLU)
        ref = ops.projection(A, Bm, "swiglu")
        tol = None
    assert ctx.status_poll() == 0
    got = out.float().cpu().numpy().astype(np.float64)
    if tol is None:   # fp16 output: one rounding of the fp32 result (2^-11 relative) + accumulation noise
        err = np.abs(got[:M] - ref)
        assert np.all(err <= np.abs(ref) * 2.0 ** -10 + 2e-5 * scale * np.sqrt(K) + 1e-6), err.max()
    else:
        assert np.max(np.abs(got[:M] - ref)) <= tol
    # the row after the last one is never touched
    if epi == "resid":
        assert np.array_equal(got[M], C0[M].astype(np.float64))
    else:
        assert np.all(got[M] == 768.0)


@pytest.mark.parametrize("M,N,K,K2", [(300, 328, 200, 64), (68, 768, 256, 192), (2500, 3072, 256, 128), (1030, 4160, 128, 64)])
@pytest.mark.parametrize("epi", ["f32", "resid", "swiglu"])
def test_gemm_with_second_operand_pair(ctx, M, N, K, K2, epi):
    """C = epilogue(A B^T + A2 B2^T): the second pair runs as extra K blocks into the same accumulator
    (the adapters' low-rank branch).  The definition is one product over the concatenated K."""
    from paper_2609_25405_b200 import binding as B
    if epi == "swiglu" and N % 16:
        pytest.skip("swiglu needs N % 16 == 0")
    rng = np.random.default_rng(M + N + K + K2)
    A, A2 = _f16_exact(rng, (M, K), 1.0), _f16_exact(rng, (M, K2), 1.0)
    Bm, B2 = _bf16_exact(rng, (N, K), 0.05), _bf16_exact(rng, (N, K2), 0.05)
    dA, dA2 = torch.from_numpy(A.astype(np.float16)).cuda(), torch.from_numpy(A2.astype(np.float16)).cuda()
    dB, dB2 = B.pack_f16_(B.bf16_from_f32(Bm)), B.pack_f16_(B.bf16_from_f32(B2))
    Ac, Bc = np.concatenate([A, A2], axis=1), np.concatenate([Bm, B2], axis=1)
    scale = 0.05 * np.sqrt(K + K2)
    if epi == "f32":
        out = torch.full((M + 1, N), 768.0, dtype=torch.float32, device="cuda")
        ctx.gemm_pair(dA, dB, dA2, dB2, out, M, N, K, K2, B.EPI_F32)
        ref, tol = ops.projection(Ac, Bc, "plain"), 2e-5 * scale * np.sqrt(K + K2) + 1e-6
    elif epi == "resid":
        C0 = rng.standard_normal((M + 1, N), dtype=np.float32)
        out = torch.from_numpy(C0.copy()).cuda()
        ctx.gemm_pair(dA, dB, dA2, dB2, out, M, N, K, K2, B.EPI_RESID_F32)
        ref, tol = ops.projection(Ac, Bc, "resid", C0[:M]), 2e-5 * scale * np.sqrt(K + K2) + 1e-5
    else:
        out = torch.full((M + 1, N // 2), 768.0, dtype=torch.float16, device="cuda")
        ctx.gemm_pair(dA, dB, dA2, dB2, out, M, N, K, K2, B.EPI_SWIGLU)
        ref, tol = ops.projection(Ac, Bc, "swiglu"), None
    assert ctx.status_poll() == 0
    got = out.float().cpu().numpy().astype(np.float64)
    if tol is None:
        err = np.abs(got[:M] - ref)
        assert np.all(err <= np.abs(ref) * 2.0 ** -10 + 2e-5 * scale * np.sqrt(K + K2) + 1e-6), err.max()
    else:
        assert np.max(np.abs(got[:M] - ref)) <= tol
    # the second pair must matter, and a zero second operand must reproduce the plain GEMM bit for bit
    base = torch.zeros_like(out) if epi != "resid" else torch.from_numpy(C0.copy()).cuda()
    ctx.gemm(dA, dB, base, M, N, K, {"f32": B.EPI_F32, "resid": B.EPI_RESID_F32, "swiglu": B.EPI_SWIGLU}[epi])
    zero = torch.zeros_like(dA2)
    again = torch.zeros_like(out) if epi != "resid" else torch.from_numpy(C0.copy()).cuda()
    ctx.gemm_pair(dA, dB, zero, dB2, again, M, N, K, K2, {"f32": B.EPI_F32, "resid": B.EPI_RESID_F32, "swiglu": B.EPI_SWIGLU}[epi])
    torch.cuda.synchronize()
    assert torch.equal(base[:M], again[:M]) and not torch.equal(base[:M], out[:M])


@pytest.mark.parametrize("M", [4096, 3900])
def test_residual_gemm_with_split_k_is_exact_to_tolerance_and_deterministic(M):
    """At the 7B projection shape the residual-update GEMM splits K in two (512 half-K work items fill
    the 74 CTA pairs far better than 256 tiles); the halves add to x in a fixed order.  Checked against
    the oracle's definition, the untouched row after the last one, and bitwise equality of two runs."""
    from paper_2609_25405_b200 import binding as B
    shape = synth.SHAPES["7b"]
    c = B.Context(B.model_cfg(shape, 64), 4096, 8, 64)
    N, K = 4096, 8192
    rng = np.random.default_rng(M)
    A = _f16_exact(rng, (M, K), 1.0)
    Bm = _bf16_exact(rng, (N, K), 0.05)
    dA, dB = torch.from_numpy(A.astype(np.float16)).cuda(), B.pack_f16_(B.bf16_from_f32(Bm))
    C0 = rng.standard_normal((M + 1, N), dtype=np.float32)
    outs = []
    for _ in range(2):
        out = torch.from_numpy(C0.copy()).cuda()
        c.gemm(dA, dB, out, M, N, K, B.EPI_RESID_F32)
        assert c.status_poll() == 0
        outs.append(out)
    assert torch.equal(outs[0], outs[1])
    got = outs[0].cpu().numpy().astype(np.float64)
    ref = ops.projection(A, Bm, "resid", C0[:M])
    scale = 0.05 * np.sqrt(K)
    assert np.max(np.abs(got[:M] - ref)) <= 2e-5 * scale * np.sqrt(K) + 1e-5
    assert np.array_equal(got[M], C0[M].astype(np.float64))
    c.close()


@pytest.mark.parametrize("epi", ["f32", "swiglu"])
def test_tile_variants_give_identical_bits(epi):
    """The same rows computed inside a 4096-row launch (CTA-pair 256 x 256 tiles) and as a launch of
    their own (single-CTA tiles) are equal bit for bit: every output element is accumulated over K in
    the same order whatever the tile shape.  The step relies on this when it picks the tile variant
    from its own row count."""
    from paper_2609_25405_b200 import binding as B
    c = B.Context(B.model_cfg(synth.SHAPES["tiny"], 64), 4096, 8, 64)
    g = torch.Generator(device="cuda").manual_seed(3)
    code = B.EPI_F32 if epi == "f32" else B.EPI_SWIGLU
    for N, K in [(4096, 2048), (3072, 4096), (2048, 8192)]:
        A = torch.randn((4096, K), generator=g, device="cuda").to(torch.float16)
        Bw = (torch.randn((N, K), generator=g, device="cuda") * 0.05).to(torch.float16)
        width, dt = (N, torch.float32) if epi == "f32" else (N // 2, torch.float16)
        big = torch.zeros((4096, width), dtype=dt, device="cuda")
        c.gemm(A, Bw, big, 4096, N, K, code)
        for M in (100, 128, 448, 1000):
            small = torch.zeros((M, width), dtype=dt, device="cuda")
            c.gemm(A[:M].contiguous(), Bw, small, M, N, K, code)
            torch.cuda.synchronize()
            assert torch.equal(small, big[:M]), (N, K, M)
    assert c.status_poll() == 0
    c.close()


@pytest.mark.parametrize("epi", ["f32", "resid", "swiglu"])
def test_tile_walk_gives_identical_bits(epi):
    """The order in which workers take the output tiles (rows fastest over the whole M, or bands of 1,
    3 or 8 row tiles; with or without L2 eviction hints on the loads) never changes a result bit:
    every element is still summed over K in the same order.  Shapes: one whose A share exceeds the
    automatic threshold (K = 14336, the 7B-class down projection, with its K split in two for the
    residual form) and a ragged one (M = 3000: a last band narrower than the others)."""
    from paper_2609_25405_b200 import binding as B
    # a context of the 7B-class width: its residual form splits the K of the down projection in two
    c = B.Context(B.model_cfg(synth.SHAPES["7b"].with_layers(1), 64), 4096, 8, 64)
    g = torch.Generator(device="cuda").manual_seed(5)
    code = {"f32": B.EPI_F32, "resid": B.EPI_RESID_F32, "swiglu": B.EPI_SWIGLU}[epi]
    try:
        for M, N, K in [(4096, 4096, 14336), (3000, 2048, 4096)]:
            A = torch.randn((M, K), generator=g, device="cuda").to(torch.float16)
            Bw = (torch.randn((N, K), generator=g, device="cuda") * 0.05).to(torch.float16)
            width, dt = (N // 2, torch.float16) if epi == "swiglu" else (N, torch.float32)
            C0 = torch.randn((M, width), generator=g, device="cuda").to(dt)
            outs = []
            for band, hints in [(-1, -1), (0, 0), (1, 1), (3, 0), (8, 1)]:
                B.gemm_set_walk(band, hints)
                out = C0.clone()
                c.gemm(A, Bw, out, M, N, K, code)
                torch.cuda.synchronize()
                outs.append(out)
            for o in outs[1:]:
                assert torch.equal(o, outs[0]), (M, N, K)
    finally:
        B.gemm_set_walk(-1, -1)
    assert c.status_poll() == 0
    c.close()


def test_weights_pack_f16_matches_round_to_nearest(ctx):
    """bf16 -> fp16 repack: exact in the fp16 normal range, round-to-nearest on the subnormal grid,
    saturating above 65504; in place."""
    from paper_2609_25405_b200 import binding as B
    rng = np.random.default_rng(3)
    vals = _bf16_exact(rng, (1, 4099), 0.02).ravel()
    special = np.array([0.0, -0.0, 2.0 ** -14, 2.0 ** -15, 3e-8, -1e-9, 65280.0, 1e6, -1e6, 1.0], dtype=np.float32)
    vals[:special.size] = synth.bf16_bits_to_f32(synth.f32_to_bf16_bits(special))
    t = B.bf16_from_f32(vals)
    h = B.pack_f16_(t)
    torch.cuda.synchronize()
    got = h.float().cpu().numpy()
    ref = np.clip(vals, -65504.0, 65504.0).astype(np.float16).astype(np.float32)
    assert np.array_equal(got, ref)
    normal = np.abs(vals) >= 2.0 ** -14
    assert np.array_equal(got[normal & (np.abs(vals) <= 65504)], vals[normal & (np.abs(vals) <= 65504)])
    assert np.max(np.abs(got - vals)[~normal]) <= 2.0 ** -25

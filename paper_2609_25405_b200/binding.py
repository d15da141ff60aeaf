"""ctypes binding of libhb.so: argument marshalling only.

Every step of the path runs inside the library's CUDA kernels; torch is used
here for device memory and streams.  Importing this module loads the library
and raises if it has not been built -- there is no fallback of any kind.
"""
import ctypes as C
import os

import numpy as np
import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libhb.so")

HB_OK = 0
ERRORS = {0: "HB_OK", -1: "HB_ERR_BAD_ARG", -2: "HB_ERR_CUDA", -3: "HB_ERR_OOM_PAGES",
          -4: "HB_ERR_OOM_SLOTS", -5: "HB_ERR_TOO_LARGE", -6: "HB_ERR_BAD_DESC",
          -7: "HB_ERR_DEVICE_STATUS", -8: "HB_ERR_UNSUPPORTED"}
from .consts import (KIND_DECODE, KIND_PREFILL_CHUNK, KIND_EMBED_CHUNK, POOL_NONE, POOL_MEAN,  # noqa: F401,E402
                     POOL_LAST, POOL_CLS, POOL_WMEAN, POOL_MAX, EPI_F16, EPI_F32, EPI_RESID_F32, EPI_SWIGLU, CLASSES)


class HbError(RuntimeError):
    def __init__(self, code, what):
        super().__init__(f"{what}: {ERRORS.get(code, code)}")
        self.code = code


class ModelCfg(C.Structure):
    _fields_ = [("n_layers", C.c_int32), ("d_model", C.c_int32), ("n_heads", C.c_int32),
                ("n_kv_heads", C.c_int32), ("head_dim", C.c_int32), ("d_ffn", C.c_int32),
                ("vocab", C.c_int32), ("page_size", C.c_int32), ("max_pos", C.c_int32),
                ("rope_theta", C.c_float), ("rms_eps", C.c_float)]


class LayerWeights(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in ("attn_norm", "wqkv", "wo", "ffn_norm", "w_gate_up", "w_down")]


class Weights(C.Structure):
    _fields_ = [("tok_emb", C.c_void_p), ("layers", C.POINTER(LayerWeights)),
                ("final_norm", C.c_void_p), ("lm_head", C.c_void_p)]


class LoraLayer(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in ("a_qkv", "b_qkv", "a_o", "b_o", "a_gu", "b_gu", "a_d", "b_d")]


class Lora(C.Structure):
    _fields_ = [("rank", C.c_int32), ("scale", C.c_float), ("layers", C.POINTER(LoraLayer))]


class Seg(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("kind", "q_start", "q_len", "pos_start", "pt_start", "pt_len",
                                         "pool_slot", "pool_mode", "is_final", "logits_row", "emb_row",
                                         "reserved")]


class BatchDesc(C.Structure):
    _fields_ = [("n_tokens", C.c_int32), ("n_segs", C.c_int32), ("n_page_ids", C.c_int32),
                ("n_logit_rows", C.c_int32), ("n_emb_rows", C.c_int32),
                ("token_ids", C.POINTER(C.c_int32)), ("segs", C.POINTER(Seg)),
                ("page_ids", C.POINTER(C.c_int32))]


SEG_DTYPE = np.dtype([(n, np.int32) for n, _ in Seg._fields_])

if not os.path.exists(LIB_PATH):
    raise ImportError(f"{LIB_PATH} is missing: build it with `python -m paper_2609_25405_b200.build` "
                      "(there is no CPU fallback)")
lib = C.CDLL(LIB_PATH)

_P = C.c_void_p
_sig = {
    "hb_workspace_bytes": [C.POINTER(ModelCfg), C.c_int32, C.c_int32, C.c_int32, C.POINTER(C.c_size_t)],
    "hb_create": [C.POINTER(ModelCfg), C.c_int32, C.c_int32, C.c_int32, _P, C.c_size_t, C.POINTER(_P)],
    "hb_destroy": [_P],
    "hb_kv_arena_bytes": [C.POINTER(ModelCfg), C.c_int32, C.POINTER(C.c_size_t)],
    "hb_kv_create": [C.POINTER(ModelCfg), _P, C.c_size_t, C.c_int32, C.POINTER(_P)],
    "hb_kv_destroy": [_P],
    "hb_kv_alloc_pages": [_P, C.c_int32, C.POINTER(C.c_int32)],
    "hb_kv_free_pages": [_P, C.c_int32, C.POINTER(C.c_int32)],
    "hb_kv_free_count": [_P, C.POINTER(C.c_int32)],
    "hb_pool_arena_bytes": [C.POINTER(ModelCfg), C.c_int32, C.POINTER(C.c_size_t)],
    "hb_pool_create": [C.POINTER(ModelCfg), _P, C.c_size_t, C.c_int32, C.POINTER(_P)],
    "hb_pool_destroy": [_P],
    "hb_pool_alloc_slot": [_P, C.POINTER(C.c_int32)],
    "hb_pool_free_slot": [_P, C.c_int32],
    "hb_pool_row_buffer_bytes": [_P, C.c_int32, C.c_int32, C.POINTER(C.c_size_t)],
    "hb_pool_attach_row_buffer": [_P, _P, C.c_size_t, C.c_int32],
    "hb_validate_desc": [C.POINTER(ModelCfg), C.c_int32, C.c_int32, C.c_int32, C.c_int32, C.c_int32,
                         C.POINTER(BatchDesc)],
    "hb_mixed_step": [_P, C.POINTER(BatchDesc), C.POINTER(Weights), _P, _P, _P, _P, _P],
    "hb_mixed_step_lora": [_P, C.POINTER(BatchDesc), C.POINTER(Weights), C.POINTER(Lora), _P, _P, _P, _P, _P],
    "hb_weights_pack_f16": [_P, _P, C.c_size_t, _P],
    "hb_argmax": [_P, _P, C.c_int32, _P, _P],
    "hb_pool_chunk": [_P, _P, _P, C.c_int32, C.c_int32, C.c_int32, C.c_int32, _P, _P, _P, _P],
    "hb_pool_chunk_noalloc": [_P, _P, C.c_int32, C.c_int32, C.c_float, C.c_int32, C.c_int32, C.c_int32, _P, _P, _P,
                              _P],
    "hb_gemm_pair": [_P, _P, _P, _P, _P, _P, C.c_int32, C.c_int32, C.c_int32, C.c_int32, C.c_int32, _P],
    "hb_status_poll": [_P, _P, C.POINTER(C.c_uint32)],
    "hb_last_launch_count": [_P, C.POINTER(C.c_int32)],
    "hb_selftest_wait_expiry": [_P, C.c_uint32, _P],
    "hb_profile_enable": [_P, C.c_int],
    "hb_profile_read": [_P, C.POINTER(C.c_float), C.POINTER(C.c_int32)],
    "hb_gemm": [_P, _P, _P, _P, C.c_int32, C.c_int32, C.c_int32, C.c_int32, _P],
    "hb_gemm_set_walk": [C.c_int32, C.c_int32],
    "hb_gemm_set_cta_limit": [C.c_int32],
    "hb_attn_set_block_limit": [C.c_int32],
    "hb_attn_set_split_keys": [C.c_int32],
}
for _name, _args in _sig.items():
    _f = getattr(lib, _name)
    _f.argtypes = _args
    _f.restype = C.c_int
EXPORTS = tuple(_sig)


def check(code, what):
    if code != HB_OK:
        raise HbError(code, what)


def model_cfg(shape, max_pos):
    """hb_model_cfg from a synth.ModelShape-like object."""
    return ModelCfg(shape.L, shape.d, shape.Hq, shape.Hkv, shape.Dh, shape.F, shape.V,
                    shape.page_size, int(max_pos), float(shape.rope_theta), float(shape.rms_eps))


def _stream_ptr(stream):
    if stream is None:
        stream = torch.cuda.current_stream()
    return C.c_void_p(stream.cuda_stream)


def bf16_from_f32(a, device="cuda"):
    """numpy float32 (bf16-exact values) -> torch bf16 tensor on `device`, bit-exact."""
    bits = (np.ascontiguousarray(a, dtype=np.float32).view(np.uint32) >> np.uint32(16)).astype(np.uint16)
    return torch.from_numpy(bits.view(np.int16)).to(device).view(torch.bfloat16)


def rope_pair_order(Dh):
    """Stored position j of a q/k head holds rotary element rope_pair_order(Dh)[j]:
    (0, Dh/2, 1, Dh/2 + 1, ...)."""
    half = Dh // 2
    order = np.empty(Dh, dtype=np.int64)
    order[0::2] = np.arange(half)
    order[1::2] = np.arange(half) + half
    return order


def rope_interleave_rows(w, Dh):
    """Reorder the rows of a q or k projection [H*Dh, d] into the library's pair-interleaved
    head layout (a layout change only: input marshalling)."""
    H = w.shape[0] // Dh
    idx = (np.arange(H)[:, None] * Dh + rope_pair_order(Dh)[None, :]).ravel()
    return w[idx]


def pack_f16_(t, stream=None):
    """Repack a bf16 tensor to fp16 in place (library kernel); returns the fp16 view."""
    assert t.dtype == torch.bfloat16 and t.is_contiguous()
    check(lib.hb_weights_pack_f16(C.c_void_p(t.data_ptr()), C.c_void_p(t.data_ptr()), t.numel(),
                                  _stream_ptr(stream)), "hb_weights_pack_f16")
    return t.view(torch.float16)


class DeviceWeights:
    """Weights resident in HBM in the library's layout (projection matrices repacked to fp16 in
    place, gains and token embedding bf16), plus the hb_weights struct."""

    def __init__(self, n_layers):
        self.tensors = []          # keep-alive
        self.layers = (LayerWeights * n_layers)()
        self.struct = Weights()
        self.struct.layers = C.cast(self.layers, C.POINTER(LayerWeights))

    def _keep(self, t):
        self.tensors.append(t)
        return t.data_ptr()

    @classmethod
    def from_synth(cls, W, device="cuda"):
        """Upload synth.Weights: q/k/v rows are concatenated, gate/up rows interleaved."""
        s = W.shape
        self = cls(s.L)
        up = lambda a: self._keep(bf16_from_f32(a, device))
        upw = lambda a: self._keep(pack_f16_(bf16_from_f32(a, device)))
        self.struct.tok_emb = up(W.tok_emb)
        self.struct.lm_head = upw(W.lm_head)
        self.struct.final_norm = up(W.final_norm)
        for l in range(s.L):
            w = W.layer(l)
            lw = self.layers[l]
            lw.attn_norm = up(w["attn_norm"])
            lw.ffn_norm = up(w["ffn_norm"])
            lw.wqkv = upw(np.concatenate([rope_interleave_rows(w["wq"], s.Dh), rope_interleave_rows(w["wk"], s.Dh),
                                          w["wv"]], axis=0))
            lw.wo = upw(w["wo"])
            gu = np.empty((2 * s.F, s.d), dtype=np.float32)
            gu[0::2] = w["wg"]
            gu[1::2] = w["wu"]
            lw.w_gate_up = upw(gu)
            lw.w_down = upw(w["wd"])
        return self

    @classmethod
    def random_on_device(cls, shape, seed=0, std=0.02, device="cuda"):
        """N(0, std^2) bf16 weights drawn on the device (benchmarks; not bit-matched to the
        host generator)."""
        self = cls(shape.L)
        g = torch.Generator(device=device)
        g.manual_seed(seed)

        def rnd(r, c, pack=True):
            t = torch.empty((r, c), dtype=torch.bfloat16, device=device)
            t.normal_(0.0, std, generator=g)
            return self._keep(pack_f16_(t) if pack else t)

        ones = lambda: self._keep(torch.ones(shape.d, dtype=torch.bfloat16, device=device))
        self.struct.tok_emb = rnd(shape.V, shape.d, pack=False)
        self.struct.lm_head = rnd(shape.V, shape.d)
        self.struct.final_norm = ones()
        for l in range(shape.L):
            lw = self.layers[l]
            lw.attn_norm = ones()
            lw.ffn_norm = ones()
            lw.wqkv = rnd(shape.n_qkv, shape.d)
            lw.wo = rnd(shape.d, shape.Hq * shape.Dh)
            lw.w_gate_up = rnd(2 * shape.F, shape.d)
            lw.w_down = rnd(shape.d, shape.F)
        return self


def _pad64(n):
    return (n + 63) // 64 * 64


class DeviceLora:
    """Adapter factors resident in HBM in the library's packed layout (fp16), plus the hb_lora
    struct.  Packing is layout only: factors are stacked / placed in column blocks next to the fused
    weights they pair with; the bf16 -> fp16 repack runs in the library."""

    def __init__(self, n_layers, rank, scale):
        self.tensors = []
        self.layers = (LoraLayer * n_layers)()
        self.struct = Lora(int(rank), float(scale), C.cast(self.layers, C.POINTER(LoraLayer)))
        self.rank = int(rank)

    def _keep(self, t):
        self.tensors.append(t)
        return t.data_ptr()

    @staticmethod
    def _stack_down(factors, R):
        """A factors [r, in] stacked by rows into [R, in], zero padded."""
        out = np.zeros((R, factors[0].shape[1]), dtype=np.float32)
        at = 0
        for a in factors:
            out[at:at + a.shape[0]] = a
            at += a.shape[0]
        return out

    @classmethod
    def from_synth(cls, ad, device="cuda"):
        """Upload synth.LoraAdapters."""
        s, r = ad.shape, ad.rank
        self = cls(s.L, r, ad.scale)
        upw = lambda a: self._keep(pack_f16_(bf16_from_f32(a, device)))
        R1, R2, R3 = 64, _pad64(2 * r), _pad64(3 * r)
        for l in range(s.L):
            f = {n: ad.factors(l, n) for n in ("wq", "wk", "wv", "wo", "wg", "wu", "wd")}
            ll = self.layers[l]
            ll.a_qkv = upw(self._stack_down([f["wq"][0], f["wk"][0], f["wv"][0]], R3))
            nq, nk = s.Hq * s.Dh, s.Hkv * s.Dh
            b = np.zeros((nq + 2 * nk, R3), dtype=np.float32)
            b[:nq, 0:r] = rope_interleave_rows(f["wq"][1], s.Dh)
            b[nq:nq + nk, r:2 * r] = rope_interleave_rows(f["wk"][1], s.Dh)
            b[nq + nk:, 2 * r:3 * r] = f["wv"][1]
            ll.b_qkv = upw(b)
            ll.a_o = upw(self._stack_down([f["wo"][0]], R1))
            b = np.zeros((s.d, R1), dtype=np.float32)
            b[:, :r] = f["wo"][1]
            ll.b_o = upw(b)
            ll.a_gu = upw(self._stack_down([f["wg"][0], f["wu"][0]], R2))
            b = np.zeros((2 * s.F, R2), dtype=np.float32)
            b[0::2, 0:r] = f["wg"][1]
            b[1::2, r:2 * r] = f["wu"][1]
            ll.b_gu = upw(b)
            ll.a_d = upw(self._stack_down([f["wd"][0]], R1))
            b = np.zeros((s.d, R1), dtype=np.float32)
            b[:, :r] = f["wd"][1]
            ll.b_d = upw(b)
        return self

    @classmethod
    def random_on_device(cls, shape, rank, seed=7, std=0.02, scale=2.0, device="cuda"):
        """Random factors drawn on the device in the packed layout (benchmarks): the blocks that the
        layout keeps at zero are zeroed after the draw."""
        self = cls(shape.L, rank, scale)
        g = torch.Generator(device=device)
        g.manual_seed(seed)
        r = rank
        R1, R2, R3 = 64, _pad64(2 * r), _pad64(3 * r)
        nq, nk = shape.Hq * shape.Dh, shape.Hkv * shape.Dh

        def rnd(rows, cols):
            t = torch.empty((rows, cols), dtype=torch.bfloat16, device=device)
            t.normal_(0.0, std, generator=g)
            return t

        fin = lambda t: self._keep(pack_f16_(t.contiguous()))
        for l in range(shape.L):
            ll = self.layers[l]
            a = rnd(R3, shape.d); a[3 * r:] = 0
            ll.a_qkv = fin(a)
            b = rnd(nq + 2 * nk, R3)
            keep = torch.zeros_like(b, dtype=torch.bool)
            keep[:nq, 0:r] = True; keep[nq:nq + nk, r:2 * r] = True; keep[nq + nk:, 2 * r:3 * r] = True
            ll.b_qkv = fin(torch.where(keep, b, torch.zeros_like(b)))
            a = rnd(R1, nq); a[r:] = 0
            ll.a_o = fin(a)
            b = rnd(shape.d, R1); b[:, r:] = 0
            ll.b_o = fin(b)
            a = rnd(R2, shape.d); a[2 * r:] = 0
            ll.a_gu = fin(a)
            b = rnd(2 * shape.F, R2)
            keep = torch.zeros_like(b, dtype=torch.bool)
            keep[0::2, 0:r] = True; keep[1::2, r:2 * r] = True
            ll.b_gu = fin(torch.where(keep, b, torch.zeros_like(b)))
            a = rnd(R1, shape.F); a[r:] = 0
            ll.a_d = fin(a)
            b = rnd(shape.d, R1); b[:, r:] = 0
            ll.b_d = fin(b)
        return self


def kv_arena_bytes(cfg, n_pages):
    nbytes = C.c_size_t()
    check(lib.hb_kv_arena_bytes(C.byref(cfg), n_pages, C.byref(nbytes)), "hb_kv_arena_bytes")
    return nbytes.value


class KvCache:
    """Caller-owned KV arena (torch) + the library's page free list.  `arena`: an int16 tensor to
    use instead of allocating one (it must hold n_pages; several caches may be laid over one
    buffer one after the other)."""

    def __init__(self, cfg, n_pages, device="cuda", fill=None, arena=None):
        self.cfg = cfg
        self.n_pages = n_pages
        nbytes = C.c_size_t(kv_arena_bytes(cfg, n_pages))
        self.handle = C.c_void_p()
        if device is None:      # bookkeeping only (host tests): no arena
            self.arena = None
            check(lib.hb_kv_create(C.byref(cfg), None, 0, n_pages, C.byref(self.handle)), "hb_kv_create")
            return
        if arena is not None:
            if arena.dtype != torch.int16 or arena.numel() * 2 < nbytes.value:
                raise ValueError("arena too small for n_pages")
            self.arena = arena[: nbytes.value // 2]
        else:
            self.arena = torch.empty(nbytes.value // 2, dtype=torch.int16, device=device)
        if fill is not None:
            self.arena.fill_(fill)
        check(lib.hb_kv_create(C.byref(cfg), C.c_void_p(self.arena.data_ptr()), nbytes.value, n_pages,
                               C.byref(self.handle)), "hb_kv_create")

    def view(self):
        """fp16 view [L, page, Hkv, 2 (slot group), 2 (K|V), Dh/64, 8, 64] (the arena's own layout)."""
        c = self.cfg
        return self.arena.view(torch.float16).view(c.n_layers, self.n_pages, c.n_kv_heads, 2, 2, c.head_dim // 64,
                                                   8, 64)

    def rows(self, layer, pages, slots, is_v):
        """K (is_v = 0) or V (1) rows of `layer` at (pages[i], slots[i]) as [n, Hkv, Dh] fp16, in the
        stored head-dimension order."""
        v = self.view()[layer][:, :, :, is_v]                   # [page, Hkv, group, H2, 8, 64]
        r = v[pages, :, slots // 8, :, slots % 8, :]            # [n, Hkv, H2, 64]
        return r.reshape(r.shape[0], r.shape[1], -1)

    def alloc(self, n):
        ids = (C.c_int32 * max(n, 1))()
        check(lib.hb_kv_alloc_pages(self.handle, n, ids), "hb_kv_alloc_pages")
        return list(ids[:n])

    def free(self, ids):
        arr = (C.c_int32 * max(len(ids), 1))(*ids)
        check(lib.hb_kv_free_pages(self.handle, len(ids), arr), "hb_kv_free_pages")

    def free_count(self):
        n = C.c_int32()
        check(lib.hb_kv_free_count(self.handle, C.byref(n)), "hb_kv_free_count")
        return n.value

    def close(self):
        if self.handle:
            lib.hb_kv_destroy(self.handle)
            self.handle = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


class Pool:
    """Caller-owned pooling arena (torch) + the library's slot free list."""

    def __init__(self, cfg, n_slots, device="cuda", fill=None):
        self.cfg = cfg
        self.n_slots = n_slots
        nbytes = C.c_size_t()
        check(lib.hb_pool_arena_bytes(C.byref(cfg), n_slots, C.byref(nbytes)), "hb_pool_arena_bytes")
        self.handle = C.c_void_p()
        if device is None:      # bookkeeping only (host tests): no arena
            self.arena = None
            check(lib.hb_pool_create(C.byref(cfg), None, 0, n_slots, C.byref(self.handle)), "hb_pool_create")
            return
        self.arena = torch.empty((nbytes.value + 3) // 4, dtype=torch.int32, device=device)
        if fill is not None:
            self.arena.fill_(fill)
        check(lib.hb_pool_create(C.byref(cfg), C.c_void_p(self.arena.data_ptr()), nbytes.value, n_slots,
                                 C.byref(self.handle)), "hb_pool_create")

    def attach_row_buffer(self, max_rows, fill=None):
        """Row buffer for buffered heads (POOL_MAX): [n_slots, max_rows, d] fp32, caller-owned."""
        nbytes = C.c_size_t()
        check(lib.hb_pool_row_buffer_bytes(C.byref(self.cfg), self.n_slots, max_rows, C.byref(nbytes)),
              "hb_pool_row_buffer_bytes")
        self.rows = torch.empty((self.n_slots, max_rows, self.cfg.d_model), dtype=torch.float32,
                                device=self.arena.device)
        if fill is not None:
            self.rows.fill_(fill)
        check(lib.hb_pool_attach_row_buffer(self.handle, C.c_void_p(self.rows.data_ptr()), nbytes.value, max_rows),
              "hb_pool_attach_row_buffer")
        return self.rows

    def sums(self):
        d = self.cfg.d_model
        return self.arena[: self.n_slots * d].view(torch.float32).view(self.n_slots, d)

    def meta(self):
        d = self.cfg.d_model
        return self.arena[self.n_slots * d: self.n_slots * d + self.n_slots * 4].view(self.n_slots, 4)

    def alloc(self):
        s = C.c_int32()
        check(lib.hb_pool_alloc_slot(self.handle, C.byref(s)), "hb_pool_alloc_slot")
        return s.value

    def free(self, slot):
        check(lib.hb_pool_free_slot(self.handle, slot), "hb_pool_free_slot")

    def close(self):
        if self.handle:
            lib.hb_pool_destroy(self.handle)
            self.handle = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


class Batch:
    """Host descriptor arrays (numpy, kept alive) and the hb_batch_desc over them."""

    def __init__(self, token_ids, segs, page_ids, n_logit_rows, n_emb_rows):
        self.token_ids = np.ascontiguousarray(token_ids, dtype=np.int32)
        self.segs = np.ascontiguousarray(segs, dtype=SEG_DTYPE)
        self.page_ids = np.ascontiguousarray(page_ids, dtype=np.int32)
        self.desc = BatchDesc(len(self.token_ids), len(self.segs), len(self.page_ids), n_logit_rows,
                              n_emb_rows,
                              self.token_ids.ctypes.data_as(C.POINTER(C.c_int32)),
                              self.segs.ctypes.data_as(C.POINTER(Seg)),
                              self.page_ids.ctypes.data_as(C.POINTER(C.c_int32)))

    @property
    def n_tokens(self):
        return len(self.token_ids)

    def host_bytes(self):
        return self.token_ids.nbytes + self.segs.nbytes + self.page_ids.nbytes


class Context:
    def __init__(self, cfg, max_tokens, max_segs, max_page_ids):
        if not torch.cuda.is_available():
            raise RuntimeError("libhb needs a CUDA device (B200); there is no CPU path")
        self.cfg = cfg
        self.handle = C.c_void_p()
        check(lib.hb_create(C.byref(cfg), max_tokens, max_segs, max_page_ids, None, 0, C.byref(self.handle)),
              "hb_create")

    def mixed_step(self, batch, weights, kv, pool, out_logits, out_emb, stream=None, lora=None):
        tail = (kv.handle, pool.handle if pool is not None else None,
                C.c_void_p(out_logits.data_ptr()) if out_logits is not None else None,
                C.c_void_p(out_emb.data_ptr()) if out_emb is not None else None, _stream_ptr(stream))
        if lora is None:
            check(lib.hb_mixed_step(self.handle, C.byref(batch.desc), C.byref(weights.struct), *tail), "hb_mixed_step")
        else:
            check(lib.hb_mixed_step_lora(self.handle, C.byref(batch.desc), C.byref(weights.struct),
                                         C.byref(lora.struct), *tail), "hb_mixed_step_lora")

    def argmax(self, logits, n_rows, out_tokens, stream=None):
        check(lib.hb_argmax(self.handle, C.c_void_p(logits.data_ptr()), n_rows,
                            C.c_void_p(out_tokens.data_ptr()), _stream_ptr(stream)), "hb_argmax")

    def gemm_pair(self, A, B, A2, B2, Cout, M, N, K, K2, epilogue, stream=None):
        check(lib.hb_gemm_pair(self.handle, C.c_void_p(A.data_ptr()), C.c_void_p(B.data_ptr()),
                               C.c_void_p(A2.data_ptr()), C.c_void_p(B2.data_ptr()), C.c_void_p(Cout.data_ptr()),
                               M, N, K, K2, epilogue, _stream_ptr(stream)), "hb_gemm_pair")

    def gemm(self, A, B, Cout, M, N, K, epilogue, stream=None):
        check(lib.hb_gemm(self.handle, C.c_void_p(A.data_ptr()), C.c_void_p(B.data_ptr()),
                          C.c_void_p(Cout.data_ptr()), M, N, K, epilogue, _stream_ptr(stream)), "hb_gemm")

    def pool_chunk(self, x, gain, n_rows, mode, first_chunk, is_final, slot_sum, slot_meta, out_emb, stream=None):
        check(lib.hb_pool_chunk(self.handle, C.c_void_p(x.data_ptr()), C.c_void_p(gain.data_ptr()), n_rows, mode,
                                1 if first_chunk else 0, 1 if is_final else 0, C.c_void_p(slot_sum.data_ptr()),
                                C.c_void_p(slot_meta.data_ptr()),
                                C.c_void_p(out_emb.data_ptr()) if out_emb is not None else None,
                                _stream_ptr(stream)), "hb_pool_chunk")

    def status_poll(self, stream=None):
        """Synchronises the stream; returns the device status code (0 = clean)."""
        code = C.c_uint32()
        rc = lib.hb_status_poll(self.handle, _stream_ptr(stream), C.byref(code))
        if rc not in (HB_OK, -7):
            raise HbError(rc, "hb_status_poll")
        return code.value

    def profile_enable(self, on):
        check(lib.hb_profile_enable(self.handle, 1 if on else 0), "hb_profile_enable")

    def profile_read(self):
        """{class name: (milliseconds, launches)} accumulated since the last read."""
        ms = (C.c_float * len(CLASSES))()
        n = (C.c_int32 * len(CLASSES))()
        check(lib.hb_profile_read(self.handle, ms, n), "hb_profile_read")
        return {CLASSES[i]: (float(ms[i]), int(n[i])) for i in range(len(CLASSES))}

    def selftest_wait_expiry(self, limit_ms=20, stream=None):
        check(lib.hb_selftest_wait_expiry(self.handle, limit_ms, _stream_ptr(stream)), "hb_selftest_wait_expiry")

    def last_launch_count(self):
        n = C.c_int32()
        check(lib.hb_last_launch_count(self.handle, C.byref(n)), "hb_last_launch_count")
        return n.value

    def close(self):
        if self.handle:
            lib.hb_destroy(self.handle)
            self.handle = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


NOALLOC_MAX_ROWS, NOALLOC_MAX_DMODEL = 2048, 4096


def pool_chunk_noalloc(x, gain, n_rows, d_model, rms_eps, mode, first_chunk, is_final, slot_sum, slot_meta,
                       out_emb, stream=None):
    """hb_pool_chunk_noalloc: the pooler for callers that may not allocate device memory (no
    context; scratch is a fixed array inside the library).  Returns the status code; sizes beyond
    NOALLOC_MAX_ROWS x NOALLOC_MAX_DMODEL give HB_ERR_TOO_LARGE (-5).  Calls that may overlap on
    the GPU must be serialised by the caller."""
    return lib.hb_pool_chunk_noalloc(C.c_void_p(x.data_ptr()), C.c_void_p(gain.data_ptr()), n_rows, d_model,
                                     float(rms_eps), mode, 1 if first_chunk else 0, 1 if is_final else 0,
                                     C.c_void_p(slot_sum.data_ptr()), C.c_void_p(slot_meta.data_ptr()),
                                     C.c_void_p(out_emb.data_ptr()) if out_emb is not None else None,
                                     _stream_ptr(stream))


def gemm_set_walk(band=-1, hints=-1):
    """Force the projection GEMM's tile walk (tests / tuning); -1 = automatic."""
    check(lib.hb_gemm_set_walk(band, hints), "hb_gemm_set_walk")


def gemm_set_cta_limit(max_ctas=0):
    """Cap the CTAs of every projection GEMM launch (tuning); 0 = one per SM."""
    check(lib.hb_gemm_set_cta_limit(max_ctas), "hb_gemm_set_cta_limit")


def attn_set_block_limit(max_blocks=0):
    """Cap the resident blocks of every attention launch (tests); 0 = two per SM."""
    check(lib.hb_attn_set_block_limit(max_blocks), "hb_attn_set_block_limit")


def attn_set_split_keys(keys=0):
    """Keys per decode attention item for contexts created from now on; 0 = the default (2048)."""
    check(lib.hb_attn_set_split_keys(keys), "hb_attn_set_split_keys")


def validate_desc(cfg, max_tokens, max_segs, max_page_ids, n_pages, n_slots, batch):
    """Host-only descriptor validation; returns the status code."""
    return lib.hb_validate_desc(C.byref(cfg), max_tokens, max_segs, max_page_ids, n_pages, n_slots,
                                C.byref(batch.desc))

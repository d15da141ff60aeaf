"""Host-side boundary: the C-ABI library loads, exports what include/hb.h declares, and its
host logic (descriptor validation, page and slot free lists) behaves as documented.
No compute call is made; runs without a GPU."""
import os
import re

import numpy as np
import pytest

from paper_2609_25405_b200 import binding as B
from paper_2609_25405_b200 import synth
from paper_2609_25405_b200.engine import build_batch

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
TINY = synth.SHAPES["tiny"]
CFG = B.model_cfg(TINY, 256)


def test_library_exports_every_declared_symbol():
    hdr = open(os.path.join(ROOT, "include", "hb.h")).read()
    declared = set(re.findall(r"HB_API\s+int\s+(hb_\w+)\s*\(", hdr))
    assert len(declared) >= 20
    for name in declared:
        assert hasattr(B.lib, name), name
    assert declared == set(B.EXPORTS)


def test_struct_sizes_match_header_layout():
    import ctypes as C
    assert C.sizeof(B.Seg) == 48 and B.SEG_DTYPE.itemsize == 48
    assert C.sizeof(B.ModelCfg) == 44
    assert C.sizeof(B.LayerWeights) == 48


def test_arena_sizes():
    import ctypes as C
    n = C.c_size_t()
    assert B.lib.hb_kv_arena_bytes(C.byref(CFG), 10, C.byref(n)) == 0
    assert n.value == TINY.L * 10 * 2 * TINY.Hkv * 16 * TINY.Dh * 2
    assert B.lib.hb_pool_arena_bytes(C.byref(CFG), 3, C.byref(n)) == 0
    assert n.value == 3 * TINY.d * 4 + 3 * 16
    bad = B.model_cfg(TINY, 256); bad.head_dim = 48
    assert B.lib.hb_kv_arena_bytes(C.byref(bad), 10, C.byref(n)) == -1


def test_page_free_list():
    kv = B.KvCache(CFG, 6, device=None)
    a = kv.alloc(4)
    assert a == [0, 1, 2, 3] and kv.free_count() == 2
    with pytest.raises(B.HbError) as e:
        kv.alloc(3)                      # all-or-nothing
    assert e.value.code == -3 and kv.free_count() == 2
    kv.free([1, 2])
    assert kv.alloc(3) == [1, 2, 4]
    with pytest.raises(B.HbError):      # double free
        kv.free([5])
    with pytest.raises(B.HbError):      # duplicate inside one call frees nothing
        kv.free([0, 0])
    assert kv.free_count() == 1
    with pytest.raises(B.HbError):
        kv.free([99])


def test_slot_free_list():
    pool = B.Pool(CFG, 2, device=None)
    assert pool.alloc() == 0 and pool.alloc() == 1
    with pytest.raises(B.HbError) as e:
        pool.alloc()
    assert e.value.code == -4
    pool.free(0)
    with pytest.raises(B.HbError):
        pool.free(0)
    assert pool.alloc() == 0


def test_row_buffer_size_and_argument_checks():
    """Buffered heads keep O(n d) state: n_slots * max_rows * d floats, caller-owned."""
    import ctypes as C
    n = C.c_size_t()
    assert B.lib.hb_pool_row_buffer_bytes(C.byref(CFG), 3, 100, C.byref(n)) == 0
    assert n.value == 3 * 100 * TINY.d * 4
    assert B.lib.hb_pool_row_buffer_bytes(C.byref(CFG), 3, 257, C.byref(n)) == -1      # more rows than max_pos
    assert B.lib.hb_pool_row_buffer_bytes(C.byref(CFG), 0, 10, C.byref(n)) == -1
    pool = B.Pool(CFG, 3, device=None)
    fake = C.c_void_p(1 << 20)            # an aligned address that is only stored, never touched
    assert B.lib.hb_pool_attach_row_buffer(pool.handle, None, 1 << 30, 100) == -1
    assert B.lib.hb_pool_attach_row_buffer(pool.handle, fake, 3 * 100 * TINY.d * 4 - 1, 100) == -1
    assert B.lib.hb_pool_attach_row_buffer(pool.handle, C.c_void_p((1 << 20) + 8), 1 << 30, 100) == -1
    assert B.lib.hb_pool_attach_row_buffer(pool.handle, fake, 3 * 100 * TINY.d * 4, 100) == 0


def _entries():
    return [
        dict(kind=B.KIND_EMBED_CHUNK, tokens=[1] * 20, pos_start=16, pages=[4, 5, 6], pool_slot=0,
             pool_mode=B.POOL_MEAN, is_final=True),
        dict(kind=B.KIND_DECODE, tokens=[7], pos_start=33, pages=[0, 1, 2], is_final=True),
        dict(kind=B.KIND_PREFILL_CHUNK, tokens=[2] * 5, pos_start=0, pages=[3], is_final=False),
    ]


def _validate(batch, n_pages=8, n_slots=2, max_tokens=64, max_segs=8, max_pages=64):
    return B.validate_desc(CFG, max_tokens, max_segs, max_pages, n_pages, n_slots, batch)


def test_build_batch_sorts_by_kind_and_validates():
    batch, order = build_batch(_entries(), 16)
    assert order == [1, 2, 0]
    assert list(batch.segs["kind"]) == [0, 1, 2]
    assert list(batch.segs["q_start"]) == [0, 1, 6]
    assert list(batch.segs["logits_row"]) == [0, -1, -1]
    assert list(batch.segs["emb_row"]) == [-1, -1, 0]
    assert batch.desc.n_logit_rows == 1 and batch.desc.n_emb_rows == 1
    assert _validate(batch) == 0


def _mutated(field, value, seg=0):
    batch, _ = build_batch(_entries(), 16)
    batch.segs[field][seg] = value
    return batch


@pytest.mark.parametrize("field,value,seg", [
    ("kind", 2, 0),            # kinds out of order
    ("q_start", 3, 1),         # not the prefix sum
    ("q_len", 2, 0),           # decode with two rows
    ("pos_start", 250, 2),     # beyond max_pos
    ("pt_len", 2, 2),          # page list too short for pos_start + q_len
    ("pool_slot", 5, 2),       # slot out of range
    ("pool_mode", 0, 2),       # embedding chunk without a head
    ("logits_row", -1, 0),     # decode must produce logits
    ("logits_row", 0, 2),      # embedding rows never produce logits
    ("emb_row", -1, 2),        # final embedding chunk must emit
    ("is_final", 1, 1),        # final prefill without a logits row
])
def test_validation_rejects(field, value, seg):
    assert _validate(_mutated(field, value, seg)) == -6


def test_validation_limits_and_ranges():
    batch, _ = build_batch(_entries(), 16)
    assert _validate(batch, max_tokens=10) == -5
    assert _validate(batch, max_segs=2) == -5
    assert _validate(batch, n_pages=6) == -6          # page id 6 out of range
    batch.token_ids[3] = TINY.V
    assert _validate(batch) == -6


def test_validation_rejects_shared_written_page_and_duplicate_slot():
    e = _entries()
    e[2]["pages"] = [2]                 # page 2 is the decode row's tail page (pos 33 -> block 2)
    batch, _ = build_batch(e, 16)
    assert _validate(batch) == -6
    e = _entries()
    e.append(dict(kind=B.KIND_EMBED_CHUNK, tokens=[1] * 3, pos_start=0, pages=[7], pool_slot=0,
                  pool_mode=B.POOL_LAST, is_final=False))
    batch, _ = build_batch(e, 16)
    assert _validate(batch) == -6


def test_validation_allows_read_only_page_sharing():
    """Two decode rows may read the same context pages as long as each writes a private page."""
    e = [dict(kind=B.KIND_DECODE, tokens=[1], pos_start=32, pages=[0, 1, 2], is_final=True),
         dict(kind=B.KIND_DECODE, tokens=[2], pos_start=32, pages=[0, 1, 3], is_final=True)]
    batch, _ = build_batch(e, 16)
    assert _validate(batch) == 0
    e[1]["pages"] = [0, 2, 3]           # reads a page the other row writes
    e[1]["pos_start"] = 32
    batch, _ = build_batch(e, 16)
    assert _validate(batch) == -6


def test_empty_batch_is_valid():
    batch = B.Batch([], np.zeros(0, dtype=B.SEG_DTYPE), [], 0, 0)
    assert _validate(batch) == 0


def test_compute_calls_fail_loudly_without_a_device():
    import torch
    if torch.cuda.is_available():
        pytest.skip("has a device")
    with pytest.raises(RuntimeError):
        B.Context(CFG, 64, 8, 64)


def test_misaligned_pointers_and_bad_tuning_arguments_are_refused_on_the_host():
    """The no-allocation pooler checks its pointers before it touches CUDA: a view that starts in the
    middle of a 16-byte vector (x, slot, output) or of an 8-byte one (gain) is HB_ERR_BAD_ARG, and
    nothing is launched (no device is needed to see the refusal).  The GEMM tuning calls refuse
    values outside their documented ranges."""
    import ctypes as C
    P = C.c_void_p
    ok = dict(x=0x10000, gain=0x20000, s=0x30000, m=0x40000, e=0x50000)

    def call(**kw):
        a = dict(ok, **kw)
        return B.lib.hb_pool_chunk_noalloc(P(a["x"]), P(a["gain"]), 8, 256, C.c_float(1e-5), B.POOL_MEAN, 1, 1, P(a["s"]),
                                           P(a["m"]), P(a["e"]), None)
    assert call(x=0x10004) == -1 and call(s=0x30008) == -1 and call(e=0x5000c) == -1
    assert call(gain=0x20002) == -1 and call(gain=0x20004) == -1 and call(m=0x40002) == -1
    assert B.lib.hb_pool_chunk_noalloc(P(ok["x"]), P(ok["gain"]), 8, 254, C.c_float(1e-5), B.POOL_MEAN, 1, 1, P(ok["s"]),
                                       P(ok["m"]), P(ok["e"]), None) == -1          # d_model not a multiple of 4
    assert B.lib.hb_pool_chunk_noalloc(P(ok["x"]), P(ok["gain"]), 4096, 256, C.c_float(1e-5), B.POOL_MEAN, 1, 1,
                                       P(ok["s"]), P(ok["m"]), P(ok["e"]), None) == -5   # beyond the fixed scratch
    assert B.lib.hb_gemm_set_walk(-2, 0) == -1 and B.lib.hb_gemm_set_walk(0, 2) == -1
    assert B.lib.hb_gemm_set_walk(-1, -1) == 0
    assert B.lib.hb_gemm_set_cta_limit(7) == -1 and B.lib.hb_gemm_set_cta_limit(-2) == -1
    assert B.lib.hb_gemm_set_cta_limit(0) == 0
    assert B.lib.hb_attn_set_block_limit(-1) == -1 and B.lib.hb_attn_set_block_limit(0) == 0
    assert B.lib.hb_attn_set_split_keys(100) == -1 and B.lib.hb_attn_set_split_keys(1000) == -1   # too small; not a multiple of 64
    assert B.lib.hb_attn_set_split_keys(131072) == -1
    assert B.lib.hb_attn_set_split_keys(1024) == 0 and B.lib.hb_attn_set_split_keys(0) == 0        # 0 restores the default


def test_step_work_splits_attention_by_row_kind():
    """The work counts that the bench divides by measured times: a decode row reads its context plus
    itself, a chunk row of length q over p earlier tokens sees q p + q (q + 1) / 2 (query, key) pairs;
    the per-kind figures add up to the totals."""
    from paper_2609_25405_b200 import synth, workloads
    s = synth.SHAPES["tiny"]
    ent = [dict(kind=B.KIND_DECODE, tokens=[1], pos_start=10, is_final=True),
           dict(kind=B.KIND_EMBED_CHUNK, tokens=[1, 2, 3], pos_start=4, is_final=False),
           dict(kind=B.KIND_PREFILL_CHUNK, tokens=[5, 6], pos_start=0, is_final=True)]
    w = workloads.step_work(s, ent)
    kv_tok = s.L * 2 * s.Hkv * s.Dh * 2
    per_pair = 4.0 * s.Dh * s.Hq * s.L
    assert w["T"] == 6 and w["n_logit"] == 2
    assert w["kv_read_bytes_decode"] == kv_tok * 11
    assert w["kv_read_bytes"] == kv_tok * (11 + 7 + 2)
    assert w["attn_flops_chunk"] == per_pair * ((3 * 4 + 6) + (0 + 3))
    assert w["attn_flops"] == per_pair * (11 + (3 * 4 + 6) + 3)
    assert w["kv_write_bytes"] == kv_tok * 6

"""Host-side logic of the C ABI (no GPU work): the library loads and exports what include/pt.h
declares, rejects bad configurations, and its page allocator and slot arithmetic agree bit for
bit with the oracle's."""
import ctypes as C
import os
import re

import numpy as np
import pytest

from oracle import pt_oracle as O
from paper_2602_07306_b200 import inputs as I
from paper_2602_07306_b200 import pt

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2602_07306_b200 import build
    build.build()
    return pt.lib()


def make(lib, **kw):
    base = dict(T=2, D=2, L=4, hidden=128, heads=4, kv_heads=4, ffn=512, rope_base=1e4, rms_eps=1e-6,
                dtype=pt.PT_F32, sync_op=0, max_pos=256, flags=0, experts=0, top_k=0)
    base.update(kw)
    cfg = pt.pt_config(**base)
    h = C.c_void_p()
    return lib.pt_model_create(C.byref(cfg), C.byref(h)), h


def test_library_exports_every_declared_symbol(lib):
    text = "".join(open(os.path.join(ROOT, "include", f)).read() for f in sorted(os.listdir(os.path.join(ROOT, "include"))))
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    declared = set(re.findall(r"\b(pt_[a-z0-9_]+)\s*\(", text))
    assert declared, "no declarations found"
    assert declared == set(pt.EXPORTS)
    for name in declared:
        assert hasattr(lib, name), name


def test_config_validation(lib):
    assert make(lib)[0] == pt.PT_OK
    assert make(lib, L=6, D=4)[0] == 2           # L % D: trailing layers would be dropped
    assert b"multiple of D" in lib.pt_last_error()
    assert make(lib, hidden=130)[0] == 2
    assert make(lib, heads=4, kv_heads=3)[0] == 2
    assert make(lib, T=0)[0] == 2
    assert make(lib, max_pos=0)[0] == 2
    assert make(lib, sync_op=2)[0] == 2
    assert make(lib, hidden=96, heads=4)[0] == 3  # head_dim 24 unsupported
    assert make(lib, ffn=100)[0] == 3
    assert lib.pt_model_create(None, None) == 1
    # PT-MoE: top_k in [1, experts]; bf16 models on the tensor-core path only; at most 16 experts
    assert make(lib, dtype=pt.PT_BF16, experts=4, top_k=2)[0] == pt.PT_OK
    assert make(lib, dtype=pt.PT_BF16, experts=4, top_k=5)[0] == 2
    assert make(lib, dtype=pt.PT_BF16, experts=4, top_k=0)[0] == 2
    assert make(lib, dtype=pt.PT_BF16, experts=0, top_k=1)[0] == 2
    assert make(lib, dtype=pt.PT_BF16, experts=17, top_k=1)[0] == 3
    assert make(lib, dtype=pt.PT_F32, experts=2, top_k=1)[0] == 3


def test_sync_count_is_L_over_D(lib):
    for L, D in [(4, 2), (32, 8), (48, 6), (8, 4), (40, 8)]:
        rc, h = make(lib, L=L, D=D)
        assert rc == 0
        assert lib.pt_sync_count(h) == O.sync_points_pt(L, D) == L // D
        assert 2 * L // lib.pt_sync_count(h) == 2 * D
        lib.pt_model_destroy(h)


def _cache(lib, h, pages, ps, esz=4, T=2, L=4, nkv=4, dh=32):
    n = C.c_size_t()
    assert lib.pt_kv_cache_bytes(h, pages, ps, C.byref(n)) == 0
    assert n.value == T * L * pages * 2 * nkv * ps * dh * esz
    c = C.c_void_p()
    fake_pool = C.c_void_p(0x10000)              # host logic only: the pool is never touched
    assert lib.pt_kv_cache_alloc(h, pages, ps, fake_pool, n.value, C.byref(c)) == 0
    return c, n.value


@pytest.mark.parametrize("shuffle", [False, True])
def test_allocator_and_slots_match_oracle_bit_exact(lib, shuffle):
    rc, h = make(lib)
    cfg = O.PTConfig(T=2, D=2, L=4, hidden=128, heads=4, kv_heads=4, ffn=512)
    pages, ps = 23, 16
    order = I.free_list_permutation(pages, seed=11) if shuffle else None
    c, _ = _cache(lib, h, pages, ps)
    oc = O.PagedKVCache(cfg, pages, ps, order)
    if shuffle:
        a = np.ascontiguousarray(order, np.int32)
        assert lib.pt_kv_set_free_list(c, a.ctypes.data_as(C.POINTER(C.c_int32)), pages) == 0
    rng = np.random.default_rng(4)
    lens = {}
    for step in range(40):
        seq = int(rng.integers(0, 5))
        new_len = lens.get(seq, 0) + int(rng.integers(1, 40))
        rc = lib.pt_kv_seq_reserve(c, seq, new_len)
        try:
            oc.reserve(seq, new_len)
            ok = True
        except MemoryError:
            ok = False
        assert (rc == 0) == ok and (ok or rc == 5)
        if ok:
            lens[seq] = new_len
        if step % 9 == 8 and lens:
            victim = sorted(lens)[0]
            assert lib.pt_kv_seq_release(c, victim) == 0
            oc.release(victim)
            del lens[victim]
        for s in lens:
            n = C.c_int32()
            buf = (C.c_int32 * 64)()
            assert lib.pt_kv_block_table(c, s, buf, 64, C.byref(n)) == 0
            assert list(buf[: n.value]) == oc.block_table[s]
    # every slot of every live sequence: library offset == oracle closed form
    off = C.c_int64()
    for s, n in lens.items():
        for pos in range(n):
            page, slot = oc.locate(s, pos)
            for t in range(2):
                for l in range(4):
                    for kv in range(2):
                        for head in range(4):
                            assert lib.pt_kv_slot(c, t, l, s, pos, kv, head, C.byref(off)) == 0
                            assert off.value == O.kv_slot_offset(cfg, pages, ps, t, l, page, kv, head, slot)
    assert lib.pt_kv_slot(c, 0, 0, 99, 0, 0, 0, C.byref(off)) == 10
    if lens:
        s = next(iter(lens))
        assert lib.pt_kv_slot(c, 0, 0, s, 100000, 0, 0, C.byref(off)) == 1
        assert lib.pt_kv_slot(c, 2, 0, s, 0, 0, 0, C.byref(off)) == 1
    lib.pt_kv_cache_free(c)
    lib.pt_model_destroy(h)


def test_cache_argument_errors(lib):
    rc, h = make(lib)
    n = C.c_size_t()
    assert lib.pt_kv_cache_bytes(h, 4, 12, C.byref(n)) == 1
    assert lib.pt_kv_cache_bytes(h, 0, 16, C.byref(n)) == 1
    c = C.c_void_p()
    assert lib.pt_kv_cache_alloc(h, 4, 16, C.c_void_p(0x10000), 16, C.byref(c)) == 4
    assert lib.pt_kv_cache_alloc(h, 4, 16, C.c_void_p(0x10010), 1 << 30, C.byref(c)) == 6
    c, _ = _cache(lib, h, 4, 16)
    bad = (C.c_int32 * 4)(0, 1, 1, 2)
    assert lib.pt_kv_set_free_list(c, bad, 4) == 1
    assert lib.pt_kv_seq_reserve(c, 0, 16 * 5) == 5
    assert lib.pt_kv_seq_reserve(c, 0, 16) == 0
    good = (C.c_int32 * 4)(3, 2, 1, 0)
    assert lib.pt_kv_set_free_list(c, good, 4) == 10      # pages in use
    v = C.c_int32(-1)
    assert lib.pt_kv_seq_len(c, 0, C.byref(v)) == 0 and v.value == 0
    assert lib.pt_kv_seq_truncate(c, 0, 1) == 1
    lib.pt_kv_cache_free(c)
    # forward calls refuse to run before weights are bound, without touching the device
    c, _ = _cache(lib, h, 4, 16)
    ids = (C.c_int32 * 1)(0)
    rc = lib.pt_prefill(h, c, C.c_void_p(0x10000), 0, 1, 4, ids, C.c_void_p(0x20000), C.c_void_p(0x30000), 1 << 20, None)
    assert rc == 10
    ws = C.c_size_t()
    assert lib.pt_workspace_bytes(h, 64, 1, 16, C.byref(ws)) == 0 and ws.value > 0
    assert lib.pt_workspace_bytes(h, 0, 1, 16, C.byref(ws)) == 1
    lib.pt_kv_cache_free(c)
    lib.pt_model_destroy(h)


def test_e4m3_cache_layout_and_scale_offsets(lib):
    """An E4M3 pool is the one-byte codes in the usual layout followed by one fp32 scale per cached vector; the
    scale of a vector sits at the vector's own index in that array (the oracle's pool without its last axis)."""
    T, L, nkv, dh, pages, ps = 2, 4, 2, 128, 5, 16
    rc, h = make(lib, T=T, L=L, D=2, hidden=256, heads=2, kv_heads=nkv, ffn=512, dtype=pt.PT_BF16)
    assert rc == 0
    n = C.c_size_t()
    assert lib.pt_kv_cache_bytes_ex(h, pages, ps, pt.PT_KV_E4M3, C.byref(n)) == 0
    vecs = T * L * pages * 2 * nkv * ps
    assert n.value == vecs * dh + vecs * 4
    m = C.c_size_t()
    assert lib.pt_kv_cache_bytes_ex(h, pages, ps, pt.PT_KV_MODEL, C.byref(m)) == 0 and m.value == vecs * dh * 2
    assert lib.pt_kv_cache_bytes_ex(h, pages, ps, 7, C.byref(m)) == 1
    assert lib.pt_kv_cache_bytes_ex(h, pages, 8, pt.PT_KV_E4M3, C.byref(m)) == 3          # pages of 8 tokens
    c = C.c_void_p()
    assert lib.pt_kv_cache_alloc_ex(h, pages, ps, pt.PT_KV_E4M3, C.c_void_p(0x10000), n.value - 1, C.byref(c)) == 4
    assert lib.pt_kv_cache_alloc_ex(h, pages, ps, pt.PT_KV_E4M3, C.c_void_p(0x10000), n.value, C.byref(c)) == 0
    order = np.array([3, 0, 4, 1, 2], np.int32)
    assert lib.pt_kv_set_free_list(c, order.ctypes.data_as(C.POINTER(C.c_int32)), 5) == 0
    assert lib.pt_kv_seq_reserve(c, 9, 40) == 0
    cfg = O.PTConfig(T=T, D=2, L=L, hidden=256, heads=2, kv_heads=nkv, ffn=512)
    oc = O.PagedKVCache(cfg, pages, ps, order, kv_format="e4m3")
    oc.reserve(9, 40)
    off, soff = C.c_int64(), C.c_int64()
    for t in range(T):
        for l in (0, 3):
            for pos in (0, 15, 16, 39):
                for kv in (0, 1):
                    for head in range(nkv):
                        assert lib.pt_kv_slot(c, t, l, 9, pos, kv, head, C.byref(off)) == 0
                        assert lib.pt_kv_scale_slot(c, t, l, 9, pos, kv, head, C.byref(soff)) == 0
                        page, slot = oc.locate(9, pos)
                        want = O.kv_slot_offset(cfg, pages, ps, t, l, page, kv, head, slot)
                        assert off.value == want
                        assert soff.value == vecs * dh + (want // dh) * 4
                        # the same index addresses the oracle's scale array
                        assert np.ravel_multi_index((t, l, page, kv, head, slot), oc.scale.shape) == want // dh
    lib.pt_kv_cache_free(c)
    # a cache in the model dtype holds no scales
    assert lib.pt_kv_cache_alloc_ex(h, pages, ps, pt.PT_KV_MODEL, C.c_void_p(0x10000), m.value, C.byref(c)) == 0
    assert lib.pt_kv_seq_reserve(c, 1, 3) == 0
    assert lib.pt_kv_scale_slot(c, 0, 0, 1, 0, 0, 0, C.byref(soff)) == 10
    lib.pt_kv_cache_free(c)
    ws, ws8 = C.c_size_t(), C.c_size_t()
    assert lib.pt_workspace_bytes_ex(h, 64, 2, ps, pt.PT_KV_MODEL, 0, C.byref(ws)) == 0
    assert lib.pt_workspace_bytes(h, 64, 2, ps, C.byref(ws8)) == 0 and ws.value == ws8.value
    assert lib.pt_workspace_bytes_ex(h, 64, 2, ps, pt.PT_KV_E4M3, 0, C.byref(ws8)) == 0 and ws8.value > ws.value
    lib.pt_model_destroy(h)
    # head_dim 64 and the plain-kernel path have no E4M3 cache
    rc, h = make(lib, hidden=256, heads=4, kv_heads=4, dtype=pt.PT_BF16)
    assert lib.pt_kv_cache_bytes_ex(h, pages, ps, pt.PT_KV_E4M3, C.byref(m)) == 3
    lib.pt_model_destroy(h)
    rc, h = make(lib, hidden=256, heads=2, kv_heads=2, dtype=pt.PT_F32)
    assert lib.pt_kv_cache_bytes_ex(h, pages, ps, pt.PT_KV_E4M3, C.byref(m)) == 3
    lib.pt_model_destroy(h)

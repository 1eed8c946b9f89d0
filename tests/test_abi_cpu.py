"""Host-only checks of the C ABI: the library loads, exports what the header declares, and
rejects bad arguments before touching a GPU."""
import ctypes as C
import os
import re

import pytest

import paper_2405_14366_b200 as mc
from paper_2405_14366_b200 import binding as B
from paper_2405_14366_b200.build import build_library


@pytest.fixture(scope="module")
def lib():
    build_library()
    return mc.lib()


def test_exports_match_header(lib, repo_root):
    text = open(os.path.join(repo_root, "include", "minicache.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    declared = set(re.findall(r"\b(mc_[a-z0-9_]+)\s*\(", text))
    assert declared, "no declarations found"
    for name in declared:
        assert lib.has_symbol(name), f"{name} declared in minicache.h but not exported"
    assert set(B.EXPORTS) <= declared | {"mc_version"}
    assert lib.mc_version() >= 100


def test_status_strings(lib):
    assert lib.mc_status_str(0) == "MC_OK"
    assert lib.mc_status_str(5) == "MC_ERR_CAPACITY"
    assert lib.mc_status_str(99) == "MC_ERR_UNKNOWN"


def _cfg(**kw):
    d = dict(n_kv_heads=8, n_q_heads=32, head_dim=128, page_size=16, dtype=0, retain_mode=0, t=0.6, gamma=0.05,
             merge_fn=0, cache_bits=0, t_mode=0, retain_union=0)
    d.update(kw)
    return B._Config(d["n_kv_heads"], d["n_q_heads"], d["head_dim"], d["page_size"], d["dtype"], d["retain_mode"],
                     d["t"], d["gamma"], d["merge_fn"], d["cache_bits"], d["t_mode"], d["retain_union"])


def _batch(batch=2, mpps=4, max_len=64, n_pages=10, bt=0x1000, sl=0x2000):
    return B._Batch(bt, sl, batch, mpps, max_len, 0, n_pages)


def test_workspace_bytes_is_host_arithmetic(lib):
    out = C.c_size_t(0)
    L = lib._lib
    c, b = _cfg(), _batch()
    assert L.mc_workspace_bytes(C.byref(c), C.byref(b), 0, 1, C.byref(out)) == 0 and out.value % 256 == 0 and out.value > 0
    m = out.value
    assert L.mc_workspace_bytes(C.byref(c), C.byref(b), 1, 2, C.byref(out)) == 0 and out.value % 256 == 0
    b2 = _batch(max_len=64 * 1024, mpps=4096)
    assert L.mc_workspace_bytes(C.byref(c), C.byref(b2), 0, 1, C.byref(out)) == 0 and out.value > m
    assert L.mc_workspace_bytes(C.byref(c), C.byref(b), 7, 1, C.byref(out)) == 1
    assert L.mc_workspace_bytes(C.byref(c), C.byref(b), 1, 3, C.byref(out)) == 1
    assert L.mc_workspace_bytes(None, C.byref(b), 0, 1, C.byref(out)) == 1


@pytest.mark.parametrize("kw,code", [
    (dict(head_dim=64), 2), (dict(page_size=8), 2), (dict(n_q_heads=12), 2), (dict(n_q_heads=24), 2),
    (dict(dtype=5), 3), (dict(retain_mode=9), 1), (dict(t=1.5), 1), (dict(gamma=-0.1), 1),
    (dict(cache_bits=8), 1), (dict(cache_bits=4, page_size=16), 2), (dict(merge_fn=3), 1),
    (dict(t_mode=2), 1), (dict(retain_union=2), 1), (dict(retain_union=1, retain_mode=2), 6),
])
def test_bad_config_rejected(lib, kw, code):
    out = C.c_size_t(0)
    c, b = _cfg(**kw), _batch()
    assert lib._lib.mc_workspace_bytes(C.byref(c), C.byref(b), 0, 1, C.byref(out)) == code


def test_merge_rejects_bad_arguments_without_launching(lib):
    L = lib._lib
    c, b = _cfg(), _batch()
    a = B._LayerKV(0x10000, 0x20000)
    pc = B._PairCache(0x30000, 0x40000, 0x60000, 0x70000, 0x80000, 0x90000, 0xA0000, 16, 0xD0000, 64, 0xB0000, 0xC0000)
    ws = 0x100000
    # null layer pool
    bad = B._LayerKV(0, 0x20000)
    assert L.mc_merge_pair(C.byref(c), C.byref(b), C.byref(bad), C.byref(a), C.byref(pc), 1, ws, 1 << 20, None) == 1
    # misaligned pool
    mis = B._LayerKV(0x10010, 0x20000)
    assert L.mc_merge_pair(C.byref(c), C.byref(b), C.byref(mis), C.byref(a), C.byref(pc), 1, ws, 1 << 20, None) == 4
    # workspace too small
    assert L.mc_merge_pair(C.byref(c), C.byref(b), C.byref(a), C.byref(a), C.byref(pc), 1, ws, 16, None) == 5
    # block table narrower than max_seq_len
    b2 = _batch(mpps=2, max_len=64)
    assert L.mc_merge_pair(C.byref(c), C.byref(b2), C.byref(a), C.byref(a), C.byref(pc), 1, ws, 1 << 20, None) == 2
    # pair cache with a missing buffer
    pc2 = B._PairCache(0x30000, 0, 0x60000, 0x70000, 0x80000, 0x90000, 0xA0000, 16, 0xD0000, 64, 0xB0000, 0xC0000)
    assert L.mc_merge_pair(C.byref(c), C.byref(b), C.byref(a), C.byref(a), C.byref(pc2), 1, ws, 1 << 20, None) == 1


def test_attn_and_restore_reject_bad_arguments(lib):
    L = lib._lib
    c, b = _cfg(), _batch()
    pc = B._PairCache(0x30000, 0x40000, 0x60000, 0x70000, 0x80000, 0x90000, 0xA0000, 16, 0xD0000, 64, 0xB0000, 0xC0000)
    d = B._LayerKV(0x10000, 0x20000)
    assert L.mc_restore(C.byref(c), C.byref(b), C.byref(pc), 2, C.byref(d), 0, None) == 1  # BOTH is not a restore target
    assert L.mc_restore(C.byref(c), C.byref(b), C.byref(pc), 0, None, 1, None) == 1
    ws = 0x100000
    # pair mode with 4 query heads per kv head needs 8 rows: allowed; with 8 per kv head it does not fit
    c8 = _cfg(n_kv_heads=4, n_q_heads=32)
    assert L.mc_decode_attn(C.byref(c8), C.byref(b), C.byref(pc), 2, 0x1000, None, None, 1.0, 0x2000, None, ws, 1 << 24, None) == 2
    # k_new without v_new
    assert L.mc_decode_attn(C.byref(c), C.byref(b), C.byref(pc), 0, 0x1000, 0x3000, None, 1.0, 0x2000, None, ws, 1 << 24, None) == 1
    # null q
    assert L.mc_decode_attn(C.byref(c), C.byref(b), C.byref(pc), 0, None, None, None, 1.0, 0x2000, None, ws, 1 << 24, None) == 1
    # workspace too small
    assert L.mc_decode_attn(C.byref(c), C.byref(b), C.byref(pc), 0, 0x1000, None, None, 1.0, 0x2000, None, ws, 8, None) == 5


def test_pair_bytes_is_host_arithmetic(lib):
    """Every buffer size of a pair cache comes from the library; the tile is page_size rows of 256 bytes
    plus two fp32 scales per token, the prefix table has one entry per 128 tokens plus one."""
    cfg = mc.McConfig(8, 32, 16, "bf16")
    sz = lib.mc_pair_bytes(cfg, batch=4, n_pages=100, max_seq_len=1000, ret_capacity=77)
    assert sz.tile_bytes == 16 * 256 + 2 * 16 * 4 and sz.e_bytes == 100 * 8 * sz.tile_bytes
    assert sz.dist_bytes == 100 * 8 * 2 * 16 * 4
    nseg = 2 * 4 * 8
    assert sz.ret_count_bytes == nseg * 4 and sz.ret_offset_bytes == (nseg + 1) * 4
    assert sz.ret_index_bytes == 77 * 4 and sz.ret_rows_bytes == 2 * 77 * 272
    assert sz.ret_prefix_stride == 8 + 1 and sz.ret_prefix_bytes == nseg * 9 * 4
    assert sz.seg_minmax_bytes == nseg * 8 and sz.status_bytes == 16
    assert sz.total_bytes >= 2 * sz.e_bytes + sz.dist_bytes and sz.total_bytes % 256 == 0
    L = lib._lib
    c, b, out = _cfg(), _batch(), B._PairSizes()
    assert L.mc_pair_bytes(C.byref(c), C.byref(b), -1, C.byref(out)) == 1
    assert L.mc_pair_bytes(C.byref(c), C.byref(b), 4, None) == 1
    assert L.mc_pair_bytes(C.byref(_cfg(page_size=8)), C.byref(b), 4, C.byref(out)) == 2


def test_q4_cache_sizes_and_argument_checks(lib):
    """The 4-bit shared cache: tiles of 2816 bytes (2048 of codes, 512 of group parameters, 256 of scales), one
    16-bit residual tile of 32 tokens per (sequence, head), a merge workspace that also holds the 16-bit
    staging tiles, and residual pools that must be given."""
    cfg = mc.McConfig(8, 32, 32, "f16", cache_bits=4)
    sz = lib.mc_pair_bytes(cfg, batch=4, n_pages=100, max_seq_len=1000, ret_capacity=77)
    assert sz.tile_bytes == 2816 and sz.e_bytes == 100 * 8 * 2816
    assert sz.res_bytes == 4 * 8 * (32 * 256 + 2 * 32 * 4)
    assert sz.total_bytes >= 2 * sz.e_bytes + 2 * sz.res_bytes + sz.dist_bytes and sz.total_bytes % 256 == 0
    sz16 = lib.mc_pair_bytes(mc.McConfig(8, 32, 32, "f16"), batch=4, n_pages=100, max_seq_len=1000, ret_capacity=77)
    assert sz16.res_bytes == 0 and sz16.tile_bytes == 3 * 2816
    L = lib._lib
    out = C.c_size_t(0)
    c4, c16, b = _cfg(page_size=32, cache_bits=4), _cfg(page_size=32), _batch(max_len=64, mpps=4, n_pages=10)
    assert L.mc_workspace_bytes(C.byref(c16), C.byref(b), 0, 1, C.byref(out)) == 0
    w16 = out.value
    assert L.mc_workspace_bytes(C.byref(c4), C.byref(b), 0, 1, C.byref(out)) == 0
    assert out.value == w16 + 2 * 10 * 8 * 8448  # the staging tiles of both tensors (already a multiple of 256)
    # a 4-bit pair without residual pools is refused; with them the next check (workspace size) answers
    a = B._LayerKV(0x10000, 0x20000)
    pc = B._PairCache(0x30000, 0x40000, 0x60000, 0x70000, 0x80000, 0x90000, 0xA0000, 16, 0xD0000, 64, 0xB0000, 0xC0000)
    assert L.mc_merge_pair(C.byref(c4), C.byref(b), C.byref(a), C.byref(a), C.byref(pc), 1, 0x100000, 1 << 30, None) == 1
    pcr = B._PairCache(0x30000, 0x40000, 0x60000, 0x70000, 0x80000, 0x90000, 0xA0000, 16, 0xD0000, 64, 0xB0000, 0xC0000,
                       0xE0000, 0xF0000)
    assert L.mc_merge_pair(C.byref(c4), C.byref(b), C.byref(a), C.byref(a), C.byref(pcr), 1, 0x100000, w16, None) == 5
    pcm = B._PairCache(0x30000, 0x40000, 0x60000, 0x70000, 0x80000, 0x90000, 0xA0000, 16, 0xD0000, 64, 0xB0000, 0xC0000,
                       0xE0010, 0xF0000)
    assert L.mc_decode_attn(C.byref(c4), C.byref(b), C.byref(pcm), 0, 0x1000, None, None, 1.0, 0x2000, None, 0x100000, 1 << 24, None) == 4


def test_merge_pairs_checks_every_pair_before_launching(lib):
    L = lib._lib
    c, b = _cfg(), _batch()
    a = B._LayerKV(0x10000, 0x20000)
    mk = lambda st: B._PairCache(0x30000, 0x40000, 0x60000, 0x70000, 0x80000, 0x90000, 0xA0000, 16, 0xD0000, 64, 0xB0000, st)
    pcs = [mk(0xC0000), mk(0xC1000)]
    arr = lambda items, T: (C.POINTER(T) * len(items))(*[C.pointer(x) for x in items])
    out = C.c_size_t(0)
    assert L.mc_workspace_bytes(C.byref(c), C.byref(b), 0, 1, C.byref(out)) == 0
    call = lambda lay, pc, n, wsb: L.mc_merge_pairs(C.byref(c), C.byref(b), n, arr(lay, B._LayerKV), arr(lay, B._LayerKV),
                                                    arr(pc, B._PairCache), 1, 0x100000, wsb, None)
    assert call([a, a], pcs, 2, out.value) == 5                      # one pair's worth of scratch for two pairs
    assert call([a, B._LayerKV(0, 0x20000)], pcs, 2, 1 << 30) == 1   # the second pair has a null pool
    assert call([a, a], [pcs[0], pcs[0]], 2, 1 << 30) == 1           # the same pair cache twice
    assert call([a, a], pcs, -1, 1 << 30) == 1
    c4 = _cfg(page_size=32, cache_bits=4)
    assert L.mc_merge_pairs(C.byref(c4), C.byref(b), 1, arr([a], B._LayerKV), arr([a], B._LayerKV), arr(pcs[:1], B._PairCache),
                            1, 0x100000, 1 << 30, None) == 6


def test_admit_sequences_argument_checks(lib):
    L = lib._lib
    c, b = _cfg(), _batch()
    a = B._LayerKV(0x10000, 0x20000)
    pc = B._PairCache(0x30000, 0x40000, 0x60000, 0x70000, 0x80000, 0x90000, 0xA0000, 16, 0xD0000, 64, 0xB0000, 0xC0000)
    arr = lambda items, T: (C.POINTER(T) * len(items))(*[C.pointer(x) for x in items])
    call = lambda sb, sc, rows, wsb: L.mc_admit_sequences(C.byref(c), C.byref(b), sb, sc, 1, arr([a], B._LayerKV), arr([a], B._LayerKV),
                                                          None, None, arr([pc], B._PairCache), rows, 1, 0x100000, wsb, None)
    assert call(1, 2, 8, 1 << 30) == 1      # sequences 1..2 of a batch of 2
    assert call(0, 1, 0, 1 << 30) == 1      # no room per sequence
    assert call(0, 1, 9, 1 << 30) == 5      # 2 sequences x 9 entries > the pool's 16
    assert call(0, 1, 8, 16) == 5           # workspace too small
    # both kinds of layers given, or neither
    assert L.mc_admit_sequences(C.byref(c), C.byref(b), 0, 1, 1, None, None, None, None, arr([pc], B._PairCache), 8, 1, 0x100000, 1 << 30, None) == 1


def test_prefill_merge_argument_checks(lib):
    L = lib._lib
    c, b = _cfg(), _batch(max_len=64, mpps=4)
    a = B._LayerKV(0x10000, 0x20000)
    pc = B._PairCache(0x30000, 0x40000, 0x60000, 0x70000, 0x80000, 0x90000, 0xA0000, 16, 0xD0000, 64, 0xB0000, 0xC0000)
    pj = lambda **kw: B._Projection(kw.get("x", 0x200000), 0x300000, 0x400000, kw.get("d_model", 512), kw.get("stride", 128))
    call = lambda cfg, proj, hint=0.3: L.mc_prefill_merge_pair(C.byref(cfg), C.byref(b), C.byref(proj), C.byref(a), C.byref(a), C.byref(pc),
                                                               C.c_float(hint), 1, 0x100000, 1 << 30, None)
    assert call(c, pj(d_model=500)) == 2           # d_model not a multiple of 64
    assert call(c, pj(stride=100)) == 2            # rows per sequence not a multiple of 128
    assert call(c, pj(stride=0)) == 2
    assert call(c, pj(x=0)) == 1
    assert call(c, pj(x=0x200010)) == 4
    assert call(_cfg(merge_fn=1), pj()) == 6       # only the SLERP merge is fused
    assert call(_cfg(retain_mode=1), pj()) == 6    # a distance hint needs the "most distinct" rule
    assert call(_cfg(page_size=32, cache_bits=4), pj()) == 6


def test_get_stats_rejects_bad_arguments(lib):
    L = lib._lib
    c, b, out = _cfg(), _batch(), B._Stats()
    pc = B._PairCache(0x30000, 0x40000, 0x60000, 0x70000, 0x80000, 0x90000, 0xA0000, 16, 0xD0000, 64, 0xB0000, 0xC0000)
    assert L.mc_get_stats(C.byref(c), C.byref(b), None, None, C.byref(out)) == 1
    assert L.mc_get_stats(C.byref(c), C.byref(b), C.byref(pc), None, None) == 1
    assert L.mc_get_stats(C.byref(_cfg(head_dim=64)), C.byref(b), C.byref(pc), None, C.byref(out)) == 2


def test_host_buffer_merge_checks_everything_before_the_first_copy(lib):
    """An argument error must enqueue nothing: a too-small workspace is reported as such (without a GPU
    the first copy would have failed with a CUDA error instead)."""
    L = lib._lib
    c, b = _cfg(), _batch()
    a = B._LayerKV(0x10000, 0x20000)
    pc = B._PairCache(0x30000, 0x40000, 0x60000, 0x70000, 0x80000, 0x90000, 0xA0000, 16, 0xD0000, 64, 0xB0000, 0xC0000)
    args = lambda pcx, ws, n: (C.byref(c), C.byref(b), C.byref(a), C.byref(a), C.byref(a), C.byref(a), C.byref(pcx), 1, ws, n, None)
    assert L.mc_merge_pair_host(*args(pc, 0x100000, 16)) == 5
    assert L.mc_merge_pair_host(*args(pc, 0x100010, 1 << 20)) == 4
    pc2 = B._PairCache(0x30000, 0, 0x60000, 0x70000, 0x80000, 0x90000, 0xA0000, 16, 0xD0000, 64, 0xB0000, 0xC0000)
    assert L.mc_merge_pair_host(*args(pc2, 0x100000, 1 << 20)) == 1
    # more sequences than the kernels' shared-memory prefix holds: refused before the status words are cleared
    big = _batch(batch=1025, mpps=4, max_len=64, n_pages=5000)
    a2 = B._LayerKV(0x10000, 0x20000)
    assert L.mc_merge_pair(C.byref(c), C.byref(big), C.byref(a2), C.byref(a2), C.byref(pc), 1, 0x100000, 1 << 30, None) == 2


def test_binding_fails_loudly_without_library(tmp_path):
    with pytest.raises(mc.McError):
        B.MiniCacheLib(str(tmp_path / "nope.so"))

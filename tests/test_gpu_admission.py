"""Admission of sequences into a running batch (mc_admit_sequences): per-sequence merges whose retained
entries live in per-sequence regions of the pool, checked against the oracle like a whole-batch merge;
a slot refilled with another sequence; the other slots untouched."""
import dataclasses

import numpy as np
import pytest
import torch

import gen
from gen import CONFIGS

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def H():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2405_14366_b200.build import build_library
    build_library()
    import mc_harness
    return mc_harness


def _check_all(H, ps, sample=None):
    stats = {}
    for p in ps:
        om, dc = p.oracle_merge(), p.device_cache()
        if p.cache_bits == 16:
            stats.update(H.compare_merge(p, om, dc))
        for layer in (0, 1):
            dk, dv = p.run_restore(layer, fp32=True)
            stats.update(H.compare_restore(p, om, dc, layer, dk, dv))
        q = gen.make_queries(dataclasses.replace(p.wl, batch=p.B), 3, n_sets=2)
        out, lse = p.run_attn(2, q.to(p.device))
        stats.update(H.compare_attention(p, om, 2, q, out.cpu(), lse.cpu(), dc=dc, sample=sample))
    return stats


@pytest.mark.parametrize("cache_bits,q4_inputs", [(16, False), (4, False), (4, True)], ids=["16bit", "4bit_cache", "4bit_layers_and_cache"])
def test_sequences_admitted_one_by_one_then_a_slot_refilled(H, cache_bits, q4_inputs):
    wl = CONFIGS["c4_s"].scaled("adm", n_kv_heads=4, n_q_heads=4, batch=6, seq_len=320, n_layers=20, index=66)
    lens = np.array([320, 33, 200, 64, 1, 150], np.int32)
    R = 2 * 4 * 64  # entries per sequence: room for a fifth of its (token, head, tensor) rows at the longest length
    ps = [H.Problem(wl, pair=i, seq_lens=lens, cache_bits=cache_bits, q4=q4_inputs, ret_capacity=6 * R) for i in range(wl.n_pairs)]
    assert len(ps) == 2 and all(torch.equal(p.block_table, ps[0].block_table) for p in ps)
    p0 = ps[0]
    lib = p0.lib
    ws = torch.empty(len(ps) * lib.mc_workspace_bytes(p0.cfg, p0.batch(), 0), dtype=torch.uint8, device=p0.device)
    if q4_inputs:
        lay = lambda p, sfx: {"k_codes": p.q4_pools["k" + sfx]["codes"], "k_meta": p.q4_pools["k" + sfx]["meta"],
                              "v_codes": p.q4_pools["v" + sfx]["codes"], "v_meta": p.q4_pools["v" + sfx]["meta"]}
        layers = [{"_lm1": lay(p, "_lm1"), "_l": lay(p, "_l")} for p in ps]
    else:
        layers = [p.pools for p in ps]
    pairs = [p.pair for p in ps]
    for b in (3, 0, 5, 1, 4, 2):  # any order; two of them as one call
        if b == 4:
            continue
        cnt = 2 if b == 3 else 1
        lib.mc_admit_sequences(p0.cfg, p0.batch(), b, cnt, layers, pairs, R, True, ws, q4=q4_inputs)
    torch.cuda.synchronize()
    for p in ps:
        words, code = lib.mc_read_status(p.pair, check=False)
        assert code == 0, words
        off = p.pair.ret_offset.cpu().numpy()[:-1].reshape(2, p.B, p.H)
        assert np.all(off // R == np.arange(p.B)[None, :, None]), "every sequence's entries lie in its own region"
    stats = _check_all(H, ps)
    # ---- slot 2 is refilled: another sequence (here: a different length over the slot's pages) is admitted
    # while the other slots stay as they are
    before = [{f: getattr(p.pair, f).clone() for f in ("ret_count", "ret_offset", "seg_minmax")} for p in ps]
    lens2 = lens.copy()
    lens2[2] = 77
    for p in ps:
        p.seq_lens_host = lens2.copy()
        p.seq_lens.copy_(torch.from_numpy(lens2))
    lib.mc_admit_sequences(p0.cfg, p0.batch(), 2, 1, layers, pairs, R, True, ws, q4=q4_inputs)
    torch.cuda.synchronize()
    for p, bf in zip(ps, before):
        words, code = lib.mc_read_status(p.pair, check=False)
        assert code == 0, words
        keep = np.array([0, 1, 3, 4, 5])
        for f in ("ret_count", "ret_offset"):
            a = getattr(p.pair, f).cpu().numpy()[:2 * p.B * p.H].reshape(2, p.B, p.H)
            assert np.array_equal(a[:, keep], bf[f].cpu().numpy()[:2 * p.B * p.H].reshape(2, p.B, p.H)[:, keep])
    stats.update({"refill_" + k: v for k, v in _check_all(H, ps).items()})
    print(cache_bits, q4_inputs, stats)


def test_a_sequence_that_overflows_its_region_keeps_nothing(H):
    wl = CONFIGS["c1"].scaled("admo", n_kv_heads=2, n_q_heads=2, batch=3, seq_len=200, outlier_frac=0.1, index=67)
    lens = np.array([200, 40, 120], np.int32)
    R = 8
    p = H.Problem(wl, seq_lens=lens, gamma=0.3, ret_capacity=3 * R)
    ws = torch.empty(p.lib.mc_workspace_bytes(p.cfg, p.batch(), 0), dtype=torch.uint8, device=p.device)
    p.lib.mc_admit_sequences(p.cfg, p.batch(), 0, 3, [p.pools], [p.pair], R, True, ws)
    torch.cuda.synchronize()
    words, code = p.lib.mc_read_status(p.pair, check=False)
    assert code == 5 and words[0] & 1, words  # MC_ERR_CAPACITY: the overflow flag
    cnt = p.pair.ret_count.cpu().numpy().reshape(2, 3, 2)
    want = p.oracle_merge()
    need = [sum(len(want[tn]["retained"][(b, h)]) for tn in ("k", "v") for h in range(2)) for b in range(3)]
    for b in range(3):
        if need[b] > R:
            assert cnt[:, b].sum() == 0
        else:
            assert cnt[:, b].sum() == need[b]
    assert any(n > R for n in need) and any(n <= R for n in need), need
    # the merged directions are valid all the same: attention with nothing retained for the overflowed sequences
    q = gen.make_queries(dataclasses.replace(wl, batch=3), 0, n_sets=1)
    out, _ = p.run_attn(0, q.to(p.device))
    assert torch.isfinite(out.float()).all()

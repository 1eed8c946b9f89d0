"""Retention of tokens appended during decode (an extension of Eq. 4: the new token is held against the
threshold of its segment's prefill tokens) on the GPU, against the oracle's `append_keep`."""
import dataclasses

import numpy as np
import pytest
import torch

import gen
from gen import CONFIGS

pytestmark = pytest.mark.gpu

MODES = {0: "distinct", 1: "literal"}


@pytest.fixture(scope="module")
def H():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2405_14366_b200.build import build_library
    build_library()
    import mc_harness
    return mc_harness


def _grow(arr, n_new):
    shp = list(arr.shape)
    shp[1] = n_new
    return np.concatenate([arr, np.zeros(shp, arr.dtype)], axis=1)


def _view(p, om):
    """The oracle's cache as the device holds it: with a 4-bit shared cache, the complete pages quantised."""
    from oracle import minicache_oracle as orc
    if p.cache_bits != 4:
        return om
    return {tn: orc.q4_cache_pair(om[tn], p.seq_lens_host, tn, p.dtype) for tn in ("k", "v")}


def _decode_with_retention(H, p, om, steps, mode, outlier_frac=0.5):
    """Appends `steps` tokens; the oracle's cache `om` and the raw rows `p.bits` grow alongside.  Returns how many
    appended tokens the oracle kept, and how many decisions fell within 1e-6 of a threshold (those follow
    the device)."""
    from oracle import minicache_oracle as orc
    B, Hh = p.B, p.H
    n0 = p.seq_lens_host.copy()
    for tn in ("k", "v"):
        for key in ("e_bits", "n_lm1", "n_l", "d"):
            om[tn][key] = _grow(om[tn][key], steps)
    for name in list(p.bits):
        p.bits[name] = _grow(p.bits[name], steps)
    wl = dataclasses.replace(p.wl, batch=B, outlier_frac=outlier_frac)
    kept_total, near = 0, 0
    for step in range(steps):
        nt = gen.make_new_tokens(wl, 0, step)
        dev = {k: v[:, 0].contiguous().to(p.device) for k, v in nt.items()}
        p.lib.mc_append_pair(p.cfg, p.batch(), p.pair, dev["k_lm1"], dev["v_lm1"], dev["k_l"], dev["v_l"])
        torch.cuda.synchronize()
        ms = {tn: orc.append_rows(gen.as_bits(nt[tn + "_lm1"][:, 0]), gen.as_bits(nt[tn + "_l"][:, 0]), p.dtype, p.oracle_t,
                                  merge_fn=p.merge_fn) for tn in ("k", "v")}
        ret_count = p.pair.ret_count.cpu().numpy().reshape(2, B, Hh)
        for b in range(B):
            pos = int(p.seq_lens_host[b])
            for h in range(Hh):
                keep, close = {}, False
                for tn in ("k", "v"):
                    d_pre = om[tn]["d"][b, :n0[b], h]
                    keep[tn] = orc.append_keep(ms[tn]["d"][b, h], d_pre, p.gamma, mode)
                    if n0[b] and p.gamma > 0:
                        close |= abs(ms[tn]["d"][b, h] - orc.retention_threshold(d_pre, p.gamma, mode)) < 1e-6
                if p.retain_union:
                    keep["k"] = keep["v"] = keep["k"] or keep["v"]
                for ti, tn in enumerate(("k", "v")):
                    o = om[tn]
                    o["e_bits"][b, pos, h] = ms[tn]["e_bits"][b, h]
                    o["n_lm1"][b, pos, h] = ms[tn]["n_a"][b, h]
                    o["n_l"][b, pos, h] = ms[tn]["n_c"][b, h]
                    o["d"][b, pos, h] = ms[tn]["d"][b, h]
                    p.bits[tn + "_lm1"][b, pos, h] = gen.as_bits(nt[tn + "_lm1"][b, 0, h])
                    p.bits[tn + "_l"][b, pos, h] = gen.as_bits(nt[tn + "_l"][b, 0, h])
                    dev_kept = int(ret_count[ti, b, h]) == len(o["retained"][(b, h)]) + 1
                    if close:  # a decision this close to the threshold may go either way: follow the device
                        near += 1
                        keep[tn] = dev_kept
                    assert dev_kept == keep[tn], f"step {step} {tn} ({b}, {h}): device kept {dev_kept}, oracle {keep[tn]}"
                    if keep[tn]:
                        o["retained"][(b, h)] = np.append(o["retained"][(b, h)], pos).astype(np.int64)
                        kept_total += 1
        p.seq_lens_host = p.seq_lens_host + 1
        p.seq_lens += 1
        p.max_seq_len += 1
        q = gen.make_queries(dataclasses.replace(p.wl, batch=B), 20 + step, n_sets=1)
        layer = step & 1
        out, lse = p.run_attn(layer, q.to(p.device))
        H.compare_attention(p, _view(p, om), layer, q, out.cpu(), lse.cpu())
    return kept_total, near


@pytest.mark.parametrize("dtype,cache_bits,mode,union", [("f16", 16, 0, 0), ("bf16", 16, 0, 1), ("f16", 16, 1, 0),
                                                          ("f16", 4, 0, 0), ("bf16", 4, 0, 1)])
def test_appended_tokens_are_held_against_the_stored_threshold(H, dtype, cache_bits, mode, union):
    from oracle import minicache_oracle as orc
    steps = 8
    wl = CONFIGS["c1"].scaled("rethr", n_kv_heads=2, n_q_heads=4, dtype=dtype, batch=3, seq_len=160, page_size=32,
                              outlier_frac=0.05, index=91)
    lens = np.array([160, 60, 27], np.int32)  # the appends complete a page of the second and of the third sequence
    p = H.Problem(wl, seq_lens=lens, gamma=0.2, retain_mode=mode, cache_bits=cache_bits, retain_union=union,
                  append_slack=steps, decode_room=steps)
    words, code = p.run_merge()
    assert code == 0, words
    p.cache_bits = 16  # the oracle's 16-bit cache; its 4-bit view is taken wherever the two are compared
    om = p.oracle_merge(MODES[mode])
    p.cache_bits = cache_bits
    if cache_bits == 16:  # the free entries behind every list leave the prefill retention what it was
        H.compare_merge(p, om, p.device_cache(), MODES[mode])
    n_prefill = sum(len(v) for tn in ("k", "v") for v in om[tn]["retained"].values())
    # (the literal reading keeps the most similar tokens: the planted near-copies of the new rows decide there)
    kept, near = _decode_with_retention(H, p, om, steps, MODES[mode], outlier_frac=0.5 if mode == 0 else 0.0)
    assert kept > 0 or mode == 1
    p.S += steps
    dc = p.device_cache()
    flags, total = p.lib.mc_read_status(p.pair, check=False)[0][:2]
    assert flags == 0 and total == n_prefill + kept
    for ti, tn in enumerate(("k", "v")):
        for b in range(p.B):
            n = int(p.seq_lens_host[b])
            for h in range(p.H):
                idx, rows = p.retained(dc, ti, b, h)
                want = om[tn]["retained"][(b, h)]
                assert np.array_equal(idx, want)
                assert np.array_equal(rows[:, 0], p.bits[tn + "_lm1"][b, idx, h])
                assert np.array_equal(rows[:, 1], p.bits[tn + "_l"][b, idx, h])
                # the mark: both scales -0.0 exactly for the kept tokens
                for li in range(2):
                    g = dc["scale"][b, :n, h, 2 * ti + li]
                    marked = np.nonzero(np.signbit(g) & (g == 0))[0]
                    assert np.array_equal(marked, want)
                # the prefix table: entry j counts the kept tokens before token 128 j
                seg = (ti * p.B + b) * p.H + h
                prefix = p.pair.ret_prefix[seg].cpu().numpy()
                for j in range(len(prefix)):
                    assert prefix[j] == int(np.sum(want < 128 * j))
    for layer in (0, 1):
        dk, dv = p.run_restore(layer, fp32=True)
        H.compare_restore(p, _view(p, om), dc, layer, dk, dv)


def test_a_segment_without_free_entries_merges_the_token_and_says_so(H):
    """One free entry per segment: the first token Eq. 4 keeps takes it; the next one sets the overflow flag and
    stays an ordinary merged token."""
    from oracle import minicache_oracle as orc
    steps = 6
    wl = CONFIGS["c1"].scaled("rethr1", n_kv_heads=2, n_q_heads=4, dtype="f16", batch=2, seq_len=96, page_size=16,
                              outlier_frac=0.05, index=92)
    p = H.Problem(wl, gamma=0.3, append_slack=1, decode_room=8)
    words, code = p.run_merge()
    assert code == 0, words
    om = p.oracle_merge()
    before = p.pair.ret_count.cpu().numpy().reshape(2, p.B, p.H).copy()
    nt_wl = dataclasses.replace(wl, batch=2, outlier_frac=1.0)  # every new token is one of the planted outliers
    first = {}       # segment -> position of the first token the rule keeps
    overflowed = False
    for step in range(steps):
        nt = gen.make_new_tokens(nt_wl, 0, step)
        dev = {k: v[:, 0].contiguous().to(p.device) for k, v in nt.items()}
        p.lib.mc_append_pair(p.cfg, p.batch(), p.pair, dev["k_lm1"], dev["v_lm1"], dev["k_l"], dev["v_l"])
        torch.cuda.synchronize()
        for ti, tn in enumerate(("k", "v")):
            m = orc.append_rows(gen.as_bits(nt[tn + "_lm1"][:, 0]), gen.as_bits(nt[tn + "_l"][:, 0]), p.dtype, p.t)
            for b in range(p.B):
                for h in range(p.H):
                    d_pre = om[tn]["d"][b, :96, h]
                    assert abs(m["d"][b, h] - orc.retention_threshold(d_pre, p.gamma)) > 1e-6  # (a clear decision)
                    if orc.append_keep(m["d"][b, h], d_pre, p.gamma):
                        if (ti, b, h) in first:
                            overflowed = True
                        else:
                            first[(ti, b, h)] = 96 + step
        p.seq_lens += 1
        p.seq_lens_host = p.seq_lens_host + 1
        p.max_seq_len += 1
        flags = p.lib.mc_read_status(p.pair, check=False)[0][0]
        assert (flags & 1) == int(overflowed), f"step {step}"
    assert overflowed and len(first) >= 2, "the case must run some segment out of free entries"
    after = p.pair.ret_count.cpu().numpy().reshape(2, p.B, p.H)
    off = p.pair.ret_offset.cpu().numpy()
    idx = p.pair.ret_index.cpu().numpy()
    p.S += steps
    dc = p.device_cache()
    for ti in range(2):
        for b in range(p.B):
            for h in range(p.H):
                seg = (ti * p.B + b) * p.H + h
                took = (ti, b, h) in first
                assert after[ti, b, h] == before[ti, b, h] + int(took)
                own = idx[off[seg]:off[seg] + after[ti, b, h]]
                # the neighbouring lists are untouched: every entry names a token of its own segment, in order
                assert np.all(np.diff(own) > 0)
                assert np.array_equal(own[:before[ti, b, h]], om["kv"[ti]]["retained"][(b, h)])
                if took:
                    assert own[-1] == first[(ti, b, h)]
                # only the token that found an entry carries the mark; the others are merged tokens with scales > 0
                g = dc["scale"][b, 96:96 + steps, h, 2 * ti]
                marked = np.nonzero(np.signbit(g))[0] + 96
                assert np.array_equal(marked, [first[(ti, b, h)]] if took else [])
                assert np.all(g[~np.signbit(g)] > 0)


def test_free_entries_in_the_regions_of_admitted_sequences(H):
    """Sequences admitted one by one (mc_admit_sequences: every sequence's retained entries in its own region of the
    pool) get their free entries too; tokens appended afterwards are kept in their own segment's list."""
    steps = 4
    wl = CONFIGS["c1"].scaled("rethr_adm", n_kv_heads=2, n_q_heads=4, dtype="f16", batch=3, seq_len=128, page_size=16,
                              outlier_frac=0.05, index=93)
    lens = np.array([128, 40, 77], np.int32)
    R = 2 * 2 * (40 + steps)  # entries per sequence
    p = H.Problem(wl, seq_lens=lens, gamma=0.2, append_slack=steps, decode_room=steps, ret_capacity=3 * R)
    ws = torch.empty(p.lib.mc_workspace_bytes(p.cfg, p.batch(), 0), dtype=torch.uint8, device=p.device)
    for b in (2, 0, 1):
        p.lib.mc_admit_sequences(p.cfg, p.batch(), b, 1, [p.pools], [p.pair], R, True, ws)
    torch.cuda.synchronize()
    words, code = p.lib.mc_read_status(p.pair, check=False)
    assert code == 0, words
    om = p.oracle_merge()
    H.compare_merge(p, om, p.device_cache())
    off = p.pair.ret_offset.cpu().numpy()[:-1].reshape(2, p.B, p.H)
    cnt = p.pair.ret_count.cpu().numpy().reshape(2, p.B, p.H)
    idx = p.pair.ret_index.cpu().numpy()
    for ti in range(2):
        for b in range(p.B):
            for h in range(p.H):
                o, c = int(off[ti, b, h]), int(cnt[ti, b, h])
                assert o // R == b and (o + c + steps - 1) // R == b, "list and free entries inside the sequence's region"
                assert np.all(idx[o + c:o + c + steps] == -1)
    kept, near = _decode_with_retention(H, p, om, steps, "distinct", outlier_frac=0.5)
    assert kept > 0
    p.S += steps
    dc = p.device_cache()
    for ti, tn in enumerate(("k", "v")):
        for b in range(p.B):
            for h in range(p.H):
                got, rows = p.retained(dc, ti, b, h)
                assert np.array_equal(got, om[tn]["retained"][(b, h)])
                assert np.array_equal(rows[:, 1], p.bits[tn + "_l"][b, got, h])
    off2 = p.pair.ret_offset.cpu().numpy()[:-1].reshape(2, p.B, p.H)
    assert np.array_equal(off, off2)

"""Parity of the CUDA path (through the C ABI) against the fp64 oracle on the same seeded bits.

Bars: retained sets exact except tokens within 1e-6 of the threshold; restored K/V within 2e-3
max-abs relative; attention output within 1e-2 max-abs; integer/bit work (indices, raw rows) exact."""
import dataclasses
import math

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


def _full_cycle(H, p, mode="distinct", do_retention=True, new_token=True, pair_mode=True, steps_q=1):
    words, code = p.run_merge(do_retention)
    assert code == 0, words
    om = p.oracle_merge(mode, do_retention)
    dc = p.device_cache()
    stats = H.compare_merge(p, om, dc, mode, do_retention)
    for layer in (0, 1):
        dk, dv = p.run_restore(layer)
        stats.update({f"l{layer}_{k}": v for k, v in H.compare_restore(p, om, dc, layer, dk, dv).items()})
    wl = dataclasses.replace(p.wl, batch=p.B)
    q = gen.make_queries(wl, 0, device="cpu", n_sets=2).to(p.device)
    nt = gen.make_new_tokens(wl, 0, 0, device="cpu")
    for layer in (0, 1):
        out, lse = p.run_attn(layer, q[layer:layer + 1].contiguous())
        stats.update({f"a{layer}_{k}": v for k, v in
                      H.compare_attention(p, om, layer, q[layer:layer + 1].cpu(), out.cpu(), lse.cpu()).items()})
    if new_token:
        kn = torch.stack([nt["k_lm1"][:, 0], nt["k_l"][:, 0]]).contiguous()  # [2][B][H][128]
        vn = torch.stack([nt["v_lm1"][:, 0], nt["v_l"][:, 0]]).contiguous()
        out, lse = p.run_attn(1, q[1:2].contiguous(), kn[1:2].contiguous().to(p.device), vn[1:2].contiguous().to(p.device))
        stats.update({f"anew_{k}": v for k, v in
                      H.compare_attention(p, om, 1, q[1:2].cpu(), out.cpu(), lse.cpu(), kn[1:2], vn[1:2]).items()})
        if pair_mode and 2 * (p.Hq // p.H) <= 8:
            out, lse = p.run_attn(2, q.contiguous(), kn.to(p.device), vn.to(p.device))
            stats.update({f"apair_{k}": v for k, v in
                          H.compare_attention(p, om, 2, q.cpu(), out.cpu(), lse.cpu(), kn, vn).items()})
    words, code = p.lib.mc_read_status(p.pair, check=False)
    assert code == 0, words
    return stats


def test_config1_full_parity(H):
    """Single pair, 32 heads x 128, batch 1, 512 tokens, fp16: every output element compared."""
    p = H.Problem(CONFIGS["c1"])
    stats = _full_cycle(H, p)
    print(stats)
    # the planted outliers (3 % of tokens, large angles) are what retention keeps
    dc = p.device_cache()
    kept = dc["ret_count"].sum() / (2 * 512 * 32)
    assert 0.002 < kept < 0.06


@pytest.mark.parametrize("n", [1, 2, 15, 16, 17, 33, 100])
@pytest.mark.parametrize("dtype,hkv,hq,ps", [("f16", 2, 2, 16), ("bf16", 2, 8, 16), ("f16", 1, 2, 32), ("bf16", 2, 4, 64)])
def test_tiny_shapes(H, n, dtype, hkv, hq, ps):
    wl = CONFIGS["c1"].scaled("tiny", n_kv_heads=hkv, n_q_heads=hq, dtype=dtype, batch=3, seq_len=n, page_size=ps,
                              outlier_frac=0.15, index=40 + n)
    lens = np.array([n, max(1, n // 2), max(1, n - 1)], np.int32)
    p = H.Problem(wl, seq_lens=lens, gamma=0.1)
    _full_cycle(H, p)


@pytest.mark.parametrize("gamma,mode", [(0.0, "distinct"), (1.0, "distinct"), (0.2, "distinct"), (0.05, "literal"), (0.5, "literal"),
                                        (0.05, "topk"), (0.3, "topk"), (0.0, "topk"), (1.0, "topk")])
def test_retention_modes(H, gamma, mode):
    wl = CONFIGS["c1"].scaled("ret", n_kv_heads=4, n_q_heads=4, batch=2, seq_len=300, outlier_frac=0.05, index=77)
    p = H.Problem(wl, gamma=gamma, retain_mode={"distinct": 0, "literal": 1, "topk": 2}[mode], seq_lens=[300, 211])
    stats = _full_cycle(H, p, mode=mode)
    dc = p.device_cache()
    if gamma == 0.0:
        assert dc["ret_count"].sum() == 0  # gamma = 0: everything merged
    if mode == "topk":  # exactly ceil(gamma n) tokens per segment
        for b, n in enumerate((300, 211)):
            assert np.all(dc["ret_count"][:, b] == math.ceil(gamma * n - 1e-12))
    if gamma == 1.0 and mode == "distinct":
        assert dc["ret_count"].sum() >= 2 * 4 * (300 + 211) - 2 * 2 * 4  # all but the least distinct token(s)


def test_topk_ties_go_to_lower_indices(H):
    """Many token pairs with exactly equal distance (a zero row has d = 0 by definition on both sides):
    the k largest include some of them, and which ones is decided by token index."""
    wl = CONFIGS["c1"].scaled("ties", n_kv_heads=2, n_q_heads=2, batch=1, seq_len=1500, index=83, outlier_frac=0.02)
    t = gen.make_pair_tensors(wl, 0)
    keep_distinct = np.arange(1500) % 5 == 0  # every fifth token keeps its planted angle, the rest get d = 0
    for name in ("k", "v"):
        t[name + "_lm1"][0, ~torch.from_numpy(keep_distinct)] = 0
    p = H.Problem(wl, tensors=t, gamma=0.5, retain_mode=2)
    words, code = p.run_merge()
    assert code == 0, words
    om = p.oracle_merge("topk")
    dc = p.device_cache()
    H.compare_merge(p, om, dc, "topk")
    got, _ = p.retained(dc, 0, 0, 0)
    assert len(got) == 750
    zeros = np.nonzero(~keep_distinct)[0]
    assert set(got) == set(np.nonzero(keep_distinct)[0]) | set(zeros[:750 - keep_distinct.sum()])


def test_no_retention_flag(H):
    wl = CONFIGS["c1"].scaled("noret", n_kv_heads=4, n_q_heads=4, batch=1, seq_len=130, index=78)
    p = H.Problem(wl)
    _full_cycle(H, p, do_retention=False)
    assert p.device_cache()["ret_count"].sum() == 0


def test_degenerate_rows(H):
    """Identical, antipodal and zero rows (the cases Eq. 3 leaves undefined) and t at both ends."""
    wl = CONFIGS["c1"].scaled("deg", n_kv_heads=2, n_q_heads=2, batch=1, seq_len=48, index=79)
    t = gen.make_pair_tensors(wl, 0)
    for name in ("k", "v"):
        a, c = t[name + "_lm1"], t[name + "_l"]
        a[0, 0:4] = c[0, 0:4]                 # identical rows: d = 0, passthrough
        a[0, 4:8] = -2 * c[0, 4:8]            # antipodal
        a[0, 8:10] = 0                        # zero row in layer l-1
        c[0, 10:12] = 0                       # zero row in layer l
        a[0, 12] = 0
        c[0, 12] = 0                          # both zero
    for tt in (0.6, 0.4, 0.0, 1.0):
        p = H.Problem(wl, tensors=t, t=tt, gamma=0.3)
        _full_cycle(H, p, new_token=False)
        dc = p.device_cache()
        assert np.all(dc["dist"][0, 0:4] < 1e-6) and np.all(np.abs(dc["dist"][0, 4:8] - 1) < 1e-6)
        assert np.all(np.isfinite(dc["scale"][0, :48])) and np.all(dc["dist"][0, 8:13] == 0)
        dk, dv = p.run_restore(1)
        x = p.logical_of(dk)
        assert torch.all(x[0, 10:13] == 0) and torch.all(torch.isfinite(x.float()))


def test_retained_pool_overflow_is_reported(H):
    wl = CONFIGS["c1"].scaled("ovf", n_kv_heads=2, n_q_heads=2, batch=2, seq_len=200, outlier_frac=0.1, index=80)
    p = H.Problem(wl, gamma=0.5, ret_capacity=3)
    words, code = p.run_merge()
    assert code == 5 and (words[0] & 1) and words[1] > 3
    dc = p.device_cache()
    assert dc["ret_count"].sum() == 0  # nothing half-written: the pair falls back to "everything merged"
    om = p.oracle_merge(do_retention=False)
    H.compare_merge(p, om, dc, do_retention=False)


def test_append_then_attend(H):
    """Decode steps: attend with the new raw token, merge-append it, attend again over n + 1."""
    wl = CONFIGS["c1"].scaled("app", n_kv_heads=4, n_q_heads=8, dtype="bf16", batch=3, seq_len=61, index=81)
    lens = np.array([61, 16, 31], np.int32)
    p = H.Problem(wl, seq_lens=lens, decode_room=8)
    words, code = p.run_merge()
    assert code == 0
    om = p.oracle_merge()
    import mc_harness as M
    from oracle import minicache_oracle as orc
    for step in range(3):
        nt = gen.make_new_tokens(dataclasses.replace(wl, batch=3), 0, step)
        dev = {k: v[:, 0].contiguous().to(p.device) for k, v in nt.items()}
        p.lib.mc_append_pair(p.cfg, p.batch(), p.pair, dev["k_lm1"], dev["v_lm1"], dev["k_l"], dev["v_l"])
        torch.cuda.synchronize()
        # oracle: append to its own logical cache
        for tn in ("k", "v"):
            m = orc.append_rows(gen.as_bits(nt[tn + "_lm1"][:, 0]), gen.as_bits(nt[tn + "_l"][:, 0]), p.dtype, p.t,
                                merge_fn=p.merge_fn)
            o = om[tn]
            if o["e_bits"].shape[1] < p.S + step + 1:
                padn = p.S + 8 - o["e_bits"].shape[1]
                for key in ("e_bits", "n_lm1", "n_l", "d"):
                    shp = list(o[key].shape)
                    shp[1] = padn
                    o[key] = np.concatenate([o[key], np.zeros(shp, o[key].dtype)], axis=1)
            for b in range(3):
                pos = int(p.seq_lens_host[b])
                o["e_bits"][b, pos] = m["e_bits"][b]
                o["n_lm1"][b, pos] = m["n_a"][b]
                o["n_l"][b, pos] = m["n_c"][b]
        p.seq_lens_host = p.seq_lens_host + 1
        p.seq_lens += 1
        p.max_seq_len += 1
        q = gen.make_queries(dataclasses.replace(wl, batch=3), 10 + step, n_sets=1)
        out, lse = p.run_attn(0, q.to(p.device))
        M.compare_attention(p, om, 0, q, out.cpu(), lse.cpu())
    # appended directions equal the oracle's (up to boundary flips) and carry no retention decision
    dc = p.device_cache(extra_tokens=3)
    for b in range(3):
        n = int(p.seq_lens_host[b])
        e_gpu = orc.decode_bits(dc["e_k"][b, n - 3:n], p.dtype)
        e_orc = orc.decode_bits(om["k"]["e_bits"][b, n - 3:n], p.dtype)
        assert np.max(np.abs(e_gpu - e_orc)) <= 2.0 ** -7 * 0.51
    assert dc["ret_count"].sum() == sum(len(v) for v in om["k"]["retained"].values()) + sum(len(v) for v in om["v"]["retained"].values())


@pytest.mark.parametrize("name", ["c2_s", "c3_s", "c5_s"])
def test_scaled_configs_sampled(H, name):
    """1/16-scale replicas of the throughput configs: merge compared on every row, restore on
    every row, attention on a seeded sample of (sequence, head) items spanning several splits."""
    wl = CONFIGS[name]
    pair = wl.n_pairs - 1
    p = H.Problem(wl, pair=pair)
    words, code = p.run_merge()
    assert code == 0, words
    om = p.oracle_merge()
    dc = p.device_cache()
    stats = H.compare_merge(p, om, dc)
    dk, dv = p.run_restore(1)
    stats.update(H.compare_restore(p, om, dc, 1, dk, dv))
    rs = np.random.RandomState(5)
    sample = [(int(rs.randint(p.B)), int(rs.randint(p.Hq))) for _ in range(6)]
    q = gen.make_queries(dataclasses.replace(wl, batch=p.B), 0, n_sets=2)
    for sel in ((0, 1, 2) if 2 * (p.Hq // p.H) <= 8 else (0, 1)):
        qq = q if sel == 2 else q[sel:sel + 1].contiguous()
        out, lse = p.run_attn(sel, qq.to(p.device))
        stats.update(H.compare_attention(p, om, sel, qq, out.cpu(), lse.cpu(), sample=sample))
    print(name, stats)


@pytest.mark.parametrize("q4", [False, True], ids=["f16_inputs", "q4_inputs"])
def test_serving_mix_ragged(H, q4):
    """Scaled serving mix: ragged log-normal lengths, pages of 32 tokens; with `q4` the two layers
    arrive in 4 bits (keys per channel, values per token, groups of 32) and are de-quantised inside
    the merge; the oracle merges the exact de-quantised values."""
    wl = CONFIGS["c4_s"]
    lens, _ = gen.make_lengths(wl)
    assert len(set(lens.tolist())) > 3 and lens.max() <= wl.seq_len
    p = H.Problem(wl, pair=wl.n_pairs - 1, seq_lens=lens, q4=q4)
    words, code = p.run_merge()
    assert code == 0, words
    om = p.oracle_merge()
    dc = p.device_cache()
    stats = H.compare_merge(p, om, dc)
    for layer in (0, 1):
        dk, dv = p.run_restore(layer)
        stats.update(H.compare_restore(p, om, dc, layer, dk, dv))
    q = gen.make_queries(dataclasses.replace(wl, batch=p.B), 0, n_sets=2)
    rs = np.random.RandomState(11)
    sample = [(int(b), int(rs.randint(p.Hq))) for b in range(p.B)]
    for sel in (0, 1, 2):
        qq = q if sel == 2 else q[sel:sel + 1].contiguous()
        out, lse = p.run_attn(sel, qq.to(p.device))
        stats.update(H.compare_attention(p, om, sel, qq, out.cpu(), lse.cpu(), sample=sample))
    print("c4_s", "q4" if q4 else "f16", stats)


def test_q4_rejects_other_page_sizes(H):
    wl = CONFIGS["c1"]
    p = H.Problem(wl)  # page size 16
    ws = p.workspace(0)
    dummy = {k: ws for k in ("k_codes", "k_meta", "v_codes", "v_meta")}
    with pytest.raises(Exception):
        p.lib.mc_merge_pair_q4(p.cfg, p.batch(), dummy, dummy, p.pair, True, ws)


@pytest.mark.parametrize("merge_fn", ["fmax", "mean"])
@pytest.mark.parametrize("dtype", ["f16", "bf16"])
def test_merge_function_variants(H, merge_fn, dtype):
    """The two merge functions the paper compares SLERP with (Appendix Eq. A; the averaging baseline of
    Sec. 3.1), through the same kernels and the same cache format: merge, restore of both layers,
    attention and an appended token against the oracle's variant."""
    wl = dataclasses.replace(CONFIGS["c1"], dtype=dtype, n_kv_heads=4, n_q_heads=8, seq_len=336)
    lens = np.array([333], np.int32)
    p = H.Problem(wl, seq_lens=lens, merge_fn=merge_fn)
    words, code = p.run_merge()
    assert code == 0, words
    om = p.oracle_merge()
    dc = p.device_cache()
    stats = H.compare_merge(p, om, dc)
    # one magnitude for both layers
    assert np.array_equal(dc["scale"][..., 0], dc["scale"][..., 1]) and np.array_equal(dc["scale"][..., 2], dc["scale"][..., 3])
    for layer in (0, 1):
        dk, dv = p.run_restore(layer)
        stats.update(H.compare_restore(p, om, dc, layer, dk, dv))
    q = gen.make_queries(dataclasses.replace(wl, batch=p.B), 0, n_sets=2)
    nt = gen.make_new_tokens(dataclasses.replace(wl, batch=p.B), 0, 0)
    kn = torch.stack([nt["k_lm1"][:, 0], nt["k_l"][:, 0]]).contiguous()
    vn = torch.stack([nt["v_lm1"][:, 0], nt["v_l"][:, 0]]).contiguous()
    out, lse = p.run_attn(2, q.to(p.device), kn.to(p.device), vn.to(p.device))
    stats.update(H.compare_attention(p, om, 2, q, out.cpu(), lse.cpu(), kn, vn))
    print(merge_fn, dtype, stats)


@pytest.mark.parametrize("pinned", [True, False], ids=["pinned", "pageable"])
def test_host_buffer_entry_points_equal_the_device_ones(H, pinned):
    """mc_merge_pair_host / mc_decode_attn_host run the same kernels as the device-buffer calls: the
    same bits must come back, whether the host buffers are pinned (the kernels read and write them
    directly) or pageable (asynchronous copies through the staging buffer)."""
    wl = dataclasses.replace(CONFIGS["c1"], seq_len=208, n_kv_heads=4, n_q_heads=8)
    p = H.Problem(wl, seq_lens=np.array([200], np.int32))
    words, code = p.run_merge()
    assert code == 0, words
    ref_dirs = p.pair.e_k.clone(), p.pair.e_v.clone(), p.pair.ret_rows.clone(), p.pair.ret_count.clone()
    host = lambda t: (torch.empty(t.shape, dtype=t.dtype, pin_memory=True).copy_(t) if pinned else t.cpu().clone())
    # merge from host pools into fresh staging pools and a fresh pair cache
    hp = {k: host(v) for k, v in p.pools.items()}
    stage = {k: torch.zeros_like(v) for k, v in p.pools.items()}
    pair2 = p.mc.PairCache(p.cfg, p.B, p.n_pages, p.ret_capacity, device=p.device)
    p.lib.mc_merge_pair_host(p.cfg, p.batch(), hp, stage, pair2, True, p.workspace(0))
    torch.cuda.synchronize()
    assert torch.equal(pair2.e_k, ref_dirs[0]) and torch.equal(pair2.e_v, ref_dirs[1])
    assert torch.equal(pair2.ret_rows, ref_dirs[2]) and torch.equal(pair2.ret_count, ref_dirs[3])
    # decode, pair mode with new tokens
    wlb = dataclasses.replace(wl, batch=p.B)
    q = gen.make_queries(wlb, 3, n_sets=2)
    nt = gen.make_new_tokens(wlb, 0, 0)
    kn = torch.stack([nt["k_lm1"][:, 0], nt["k_l"][:, 0]]).contiguous()
    vn = torch.stack([nt["v_lm1"][:, 0], nt["v_l"][:, 0]]).contiguous()
    ref, ref_lse = p.run_attn(2, q.to(p.device), kn.to(p.device), vn.to(p.device))
    qh, knh, vnh = host(q), host(kn), host(vn)
    out_h = host(torch.full_like(ref.cpu(), float("nan")))
    lse_h = host(torch.full_like(ref_lse.cpu(), float("nan")))
    io = torch.empty(p.lib.mc_decode_io_bytes(p.cfg, p.batch(), 2), dtype=torch.uint8, device=p.device)
    for _ in range(2):  # twice: the staging buffer and the workspace are reused
        p.lib.mc_decode_attn_host(p.cfg, p.batch(), p.pair, 2, qh, knh, vnh, 1.0 / math.sqrt(128.0), out_h, lse_h, io,
                                  p.workspace(1, 2))
        torch.cuda.synchronize()
        assert torch.equal(out_h, ref.cpu()) and torch.equal(lse_h, ref_lse.cpu())
    # without a new token and without the log-sum-exp
    ref1, _ = p.run_attn(1, q[1:2].contiguous().to(p.device), None, None, want_lse=False)
    q1 = host(q[1:2].contiguous())
    out1 = host(torch.zeros_like(ref1.cpu()))
    p.lib.mc_decode_attn_host(p.cfg, p.batch(), p.pair, 1, q1, None, None, 1.0 / math.sqrt(128.0), out1, None, io,
                              p.workspace(1, 1))
    torch.cuda.synchronize()
    assert torch.equal(out1, ref1.cpu())


@pytest.mark.parametrize("hkv,hq,lens,ps", [
    (2, 2, [9000, 130, 4097], 16),     # one query row: pieces up to 4096 tokens, cut by the score buffer and by team ranges
    (3, 6, [700, 5, 1300, 0, 260], 32),  # three kv heads (a team of three), an empty sequence
    (64, 64, [300, 77], 16),           # more kv heads than CTAs in a team: two heads per CTA
    (1, 8, [2500], 64),                # eight query rows on one kv head: chunks of 512 tokens
    (16, 32, [7 + 13 * (i % 11) for i in range(40)], 16),  # 1280 output rows: the combine kernel's warp-per-row form
])
def test_attention_work_split_shapes(H, hkv, hq, lens, ps):
    """Decode attention where the cut into teams, heads per CTA and pieces matters: sequences longer than
    one piece, team boundaries inside sequences, head counts that are no power of two or exceed a team.
    Merge without retention check here (covered elsewhere); attention of layer l with a new token,
    sampled (sequence, head) pairs against the oracle, and pair mode where the head ratio allows it."""
    S = max(lens) + (-max(lens)) % ps
    wl = CONFIGS["c1"].scaled("split", n_kv_heads=hkv, n_q_heads=hq, batch=len(lens), seq_len=S, page_size=ps, index=77)
    p = H.Problem(wl, seq_lens=np.array(lens, np.int32))
    words, code = p.run_merge()
    assert code == 0, words
    om = p.oracle_merge()
    wlb = dataclasses.replace(wl, batch=p.B)
    q = gen.make_queries(wlb, 1, n_sets=2)
    nt = gen.make_new_tokens(wlb, 0, 0)
    kn = torch.stack([nt["k_lm1"][:, 0], nt["k_l"][:, 0]]).contiguous()
    vn = torch.stack([nt["v_lm1"][:, 0], nt["v_l"][:, 0]]).contiguous()
    rs = np.random.RandomState(3)
    sample = [(b, int(rs.randint(hq))) for b in range(p.B) for _ in range(2)]
    out, lse = p.run_attn(1, q[1:2].contiguous().to(p.device), kn[1:2].contiguous().to(p.device), vn[1:2].contiguous().to(p.device))
    H.compare_attention(p, om, 1, q[1:2].contiguous(), out.cpu(), lse.cpu(), kn[1:2].contiguous(), vn[1:2].contiguous(), sample=sample)
    out0, lse0 = p.run_attn(0, q[0:1].contiguous().to(p.device))  # no new token: an empty sequence gives zeros
    H.compare_attention(p, om, 0, q[0:1].contiguous(), out0.cpu(), lse0.cpu(), sample=sample)
    if 2 * (hq // hkv) <= 8:
        out2, lse2 = p.run_attn(2, q.to(p.device), kn.to(p.device), vn.to(p.device))
        H.compare_attention(p, om, 2, q, out2.cpu(), lse2.cpu(), kn, vn, sample=sample)


class _Segment:
    """One (sequence, kv head) of a full-size problem, shaped like a Problem for the comparison helpers."""

    def __init__(self, p, b, h):
        self.p, self.b0, self.h0 = p, b, h
        self.B, self.H, self.Hq, self.S = 1, 1, p.Hq // p.H, p.S
        self.dtype, self.gamma, self.t = p.dtype, p.gamma, p.t
        self.seq_lens_host = p.seq_lens_host[b:b + 1]
        self.bits = {k: v[b:b + 1, :, h:h + 1] for k, v in p.bits.items()}

    def retained(self, dc, tensor, b, h):
        return self.p.retained(dc["full"], tensor, self.b0, self.h0)

    def logical_of(self, rows, seq_len=None):  # the test hands over logical rows of this segment already
        return rows

    def slice_cache(self, dc):
        b, h = self.b0, self.h0
        out = {k: dc[k][b:b + 1, :, h:h + 1] for k in ("e_k", "e_v", "scale", "dist")}
        out["seg_minmax"] = dc["seg_minmax"][:, b:b + 1, h:h + 1]
        out["full"] = dc
        return out


def test_full_size_config2_sampled(H):
    """Config 2 at its full size (batch 8 x 4096 tokens, 32 heads, fp16, page 16; the last layer pair), in
    the launch configuration the benchmark times: merge, restore and decode attention with a new token
    and room for the decode steps; sampled (sequence, head) segments are compared against the oracle
    with the same bars as everywhere else, and the retained totals must agree with the status word."""
    from oracle import minicache_oracle as orc
    wl = CONFIGS["c2"]
    p = H.Problem(wl, pair=wl.n_pairs - 1, decode_room=wl.decode_steps + 1)
    words, code = p.run_merge()
    assert code == 0, words
    dc = p.device_cache()
    assert int(dc["ret_count"].sum()) == int(words[1])
    rs = np.random.RandomState(17)
    segs = [(int(rs.randint(p.B)), int(rs.randint(p.H))) for _ in range(4)]
    dk, dv = p.run_restore(1)
    dkl, dvl = p.logical_of(dk), p.logical_of(dv)
    wlb = dataclasses.replace(wl, batch=p.B)
    q = gen.make_queries(wlb, 2, n_sets=2)
    nt = gen.make_new_tokens(wlb, 0, 0)
    kn = torch.stack([nt["k_lm1"][:, 0], nt["k_l"][:, 0]]).contiguous()
    vn = torch.stack([nt["v_lm1"][:, 0], nt["v_l"][:, 0]]).contiguous()
    out, lse = p.run_attn(1, q[1:2].contiguous().to(p.device), kn[1:2].contiguous().to(p.device), vn[1:2].contiguous().to(p.device))
    out2, lse2 = p.run_attn(2, q.to(p.device), kn.to(p.device), vn.to(p.device))
    out, lse, out2, lse2 = out.cpu(), lse.cpu(), out2.cpu(), lse2.cpu()
    for b, h in segs:
        sg = _Segment(p, b, h)
        om = {tn: orc.merge_pair(sg.bits[tn + "_lm1"], sg.bits[tn + "_l"], sg.seq_lens_host, sg.dtype, sg.t, sg.gamma)
              for tn in ("k", "v")}
        dcs = sg.slice_cache(dc)
        stats = H.compare_merge(sg, om, dcs)
        # restore of layer l: dense rows of this segment
        stats.update(H.compare_restore(sg, om, dcs, 1, dkl[b:b + 1, :, h:h + 1], dvl[b:b + 1, :, h:h + 1]))
        sl = lambda x, hd: x[:, b:b + 1, hd:hd + 1].contiguous()
        stats.update(H.compare_attention(sg, om, 1, sl(q[1:2], h), sl(out, h), sl(lse, h), sl(kn[1:2], h), sl(vn[1:2], h)))
        stats.update(H.compare_attention(sg, om, 2, sl(q, h), sl(out2, h), sl(lse2, h), sl(kn, h), sl(vn, h)))
        print("segment", b, h, stats)


def test_bounded_wait_times_out_into_the_status_word(H):
    """A wait that nothing ends: the kernel gives up after its poll limit, records the time-out in
    the pair's status words and returns; the context stays usable and the next merge clears the flag."""
    p = H.Problem(CONFIGS["c1"].scaled("wait", n_kv_heads=2, n_q_heads=2, seq_len=64, index=91))
    words, code = p.run_merge()
    assert code == 0
    p.lib.mc_selftest_wait_timeout(p.pair, 20000)
    torch.cuda.synchronize()
    words, code = p.lib.mc_read_status(p.pair, check=False)
    assert code == 8 and (words[0] & 2) == 2, (words, code)  # MC_ERR_DEVICE_STATUS, MC_FLAG_WAIT_TIMEOUT
    with pytest.raises(p.mc.McError):
        p.lib.mc_read_status(p.pair)
    words, code = p.run_merge()  # the context works, the merge clears the words
    assert code == 0 and words[0] == 0
    _full_cycle(H, p)


def test_decode_step_replayed_from_a_cuda_graph(H):
    """A decode step (attention of both layers with the new token, append, lengths + 1) captured in a
    CUDA graph and replayed gives the same bits as the same calls issued one by one."""
    wl = CONFIGS["c1"].scaled("graph", n_kv_heads=4, n_q_heads=8, batch=2, seq_len=320, index=93)
    lens = np.array([300, 129], np.int32)
    wlb = dataclasses.replace(wl, batch=2)
    q = gen.make_queries(wlb, 0, n_sets=2)
    nt = gen.make_new_tokens(wlb, 0, 0)
    dev = {k: v[:, 0].contiguous().cuda() for k, v in nt.items()}
    qd = q.cuda()
    sm = 1.0 / math.sqrt(128.0)

    def run(use_graph):
        p = H.Problem(wl, seq_lens=lens.copy(), decode_room=8)
        words, code = p.run_merge()
        assert code == 0
        outs = [torch.zeros(1, 2, 8, 128, dtype=torch.float16, device="cuda") for _ in range(2)]
        b = p.mc.Batch(p.block_table, p.seq_lens, p.max_seq_len + 4, p.n_pages)
        ws = torch.empty(p.lib.mc_workspace_bytes(p.cfg, b, 1, 1), dtype=torch.uint8, device="cuda")

        def step():
            for layer in (0, 1):
                p.lib.mc_decode_attn(p.cfg, b, p.pair, layer, qd[layer], dev["k_lm1" if layer == 0 else "k_l"],
                                     dev["v_lm1" if layer == 0 else "v_l"], sm, outs[layer], None, ws)
            p.lib.mc_append_pair(p.cfg, b, p.pair, dev["k_lm1"], dev["v_lm1"], dev["k_l"], dev["v_l"])
            p.seq_lens += 1

        results = []
        if use_graph:
            g = torch.cuda.CUDAGraph()
            torch.cuda.synchronize()
            with torch.cuda.graph(g):
                step()
        for _ in range(3):
            g.replay() if use_graph else step()
            torch.cuda.synchronize()
            results.append([o.clone() for o in outs])
        return results, p.pair.e_k.clone(), p.seq_lens.clone()

    eager, ek_e, len_e = run(False)
    graph, ek_g, len_g = run(True)
    assert torch.equal(len_e, len_g) and torch.equal(ek_e, ek_g)
    for a, b in zip(eager, graph):
        assert torch.equal(a[0], b[0]) and torch.equal(a[1], b[1])

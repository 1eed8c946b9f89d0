"""The 4-bit shared cache (Sec. 5: MiniCache on top of 4-bit KIVI quantisation) against the oracle, stage
by stage: (i) the 16-bit directions the merge forms, (ii) codes, group parameters and stored directions
bit for bit from those, (iii) restore and decode attention over the device's own blob and end to end."""
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


def _twin(H, wl, lens, q4_inputs, **kw):
    """The same pair merged into a 16-bit cache and into a 4-bit cache."""
    tensors = gen.make_pair_tensors(wl, wl.n_pairs - 1, device="cpu")
    p16 = H.Problem(wl, pair=wl.n_pairs - 1, seq_lens=lens, q4=q4_inputs, tensors=tensors, page_size=32, **kw)
    p4 = H.Problem(wl, pair=wl.n_pairs - 1, seq_lens=lens, q4=q4_inputs, tensors=tensors, page_size=32, cache_bits=4, **kw)
    for p in (p16, p4):
        words, code = p.run_merge()
        assert code == 0, words
    return p16, p4


@pytest.mark.parametrize("dtype,hkv,hq", [("f16", 2, 2), ("bf16", 2, 8), ("f16", 4, 8)])
@pytest.mark.parametrize("q4_inputs", [False, True], ids=["16bit_layers", "4bit_layers"])
def test_q4_cache_stagewise(H, dtype, hkv, hq, q4_inputs):
    wl = CONFIGS["c1"].scaled("q4c", n_kv_heads=hkv, n_q_heads=hq, dtype=dtype, batch=7, seq_len=288, page_size=32,
                              outlier_frac=0.05, index=70 + hkv)
    lens = np.array([288, 32, 31, 64, 1, 130, 257], np.int32)
    p16, p4 = _twin(H, wl, lens, q4_inputs)
    om16, dc16 = p16.oracle_merge(), p16.device_cache()
    stats = H.compare_merge(p16, om16, dc16)                      # (i)
    om4, dc4 = p4.oracle_merge(), p4.device_cache()
    assert np.array_equal(dc4["ret_index"], dc16["ret_index"]) and np.array_equal(dc4["ret_count"], dc16["ret_count"])
    assert np.array_equal(dc4["dist"], dc16["dist"])
    stats.update(H.compare_q4_cache(p4, dc4, dc16, om4))          # (ii)
    for layer in (0, 1):                                          # (iii)
        dk, dv = p4.run_restore(layer)
        stats.update({f"l{layer}_{k}": v for k, v in H.compare_restore(p4, om4, dc4, layer, dk, dv).items()})
        dk, dv = p4.run_restore(layer, fp32=True)
        stats.update({f"l{layer}f_{k}": v for k, v in H.compare_restore(p4, om4, dc4, layer, dk, dv).items()})
    wlb = dataclasses.replace(wl, batch=p4.B)
    q = gen.make_queries(wlb, 0, n_sets=2)
    nt = gen.make_new_tokens(wlb, 0, 0)
    kn = torch.stack([nt["k_lm1"][:, 0], nt["k_l"][:, 0]]).contiguous()
    vn = torch.stack([nt["v_lm1"][:, 0], nt["v_l"][:, 0]]).contiguous()
    for layer in (0, 1):
        out, lse = p4.run_attn(layer, q[layer:layer + 1].contiguous().to(p4.device))
        stats.update({f"a{layer}_{k}": v for k, v in
                      H.compare_attention(p4, om4, layer, q[layer:layer + 1], out.cpu(), lse.cpu(), dc=dc4).items()})
    out, lse = p4.run_attn(1, q[1:2].contiguous().to(p4.device), kn[1:2].contiguous().to(p4.device), vn[1:2].contiguous().to(p4.device))
    stats.update({f"anew_{k}": v for k, v in
                  H.compare_attention(p4, om4, 1, q[1:2], out.cpu(), lse.cpu(), kn[1:2], vn[1:2], dc=dc4).items()})
    if 2 * (hq // hkv) <= 8:
        out, lse = p4.run_attn(2, q.to(p4.device), kn.to(p4.device), vn.to(p4.device))
        stats.update({f"apair_{k}": v for k, v in H.compare_attention(p4, om4, 2, q, out.cpu(), lse.cpu(), kn, vn, dc=dc4).items()})
    words, code = p4.lib.mc_read_status(p4.pair, check=False)
    assert code == 0, words
    # footprint: 64 bytes of codes + 16 of group parameters + 12 of scalars per row of a complete page
    st, code = p4.lib.mc_get_stats(p4.cfg, p4.batch(), p4.pair)
    thq = int((lens // 32 * 32).sum()) * hkv
    th = int(lens.sum()) * hkv
    assert st["compressed_bytes"] == 2 * thq * 92 + 2 * (th - thq) * 268 + st["retained_total"] * 516
    assert st["stored_bytes"] >= st["compressed_bytes"]
    print(dtype, hkv, hq, q4_inputs, stats)


def test_q4_cache_needs_pages_of_32(H):
    wl = CONFIGS["c1"].scaled("q4b", n_kv_heads=2, n_q_heads=2, batch=1, seq_len=64, index=77)
    with pytest.raises(Exception) as ei:
        H.Problem(wl, page_size=16, cache_bits=4)
    assert "MC_ERR_SHAPE" in str(ei.value)


@pytest.mark.parametrize("dtype", ["f16", "bf16"])
def test_q4_cache_decode_loop(H, dtype):
    """Decode over a 4-bit cache with no host synchronisation between the steps: attention for both layers
    with the step's raw token, merge-append (the token goes to the residual tile; a page that fills up is
    quantised by the append kernel), the lengths grow on the device.  After 40 steps every sequence has
    completed at least one page; the last step's outputs and the cache are compared with the oracle."""
    from oracle import minicache_oracle as orc
    steps = 40
    hkv, hq = 2, 4
    wl = CONFIGS["c1"].scaled("q4d", n_kv_heads=hkv, n_q_heads=hq, dtype=dtype, batch=4, seq_len=160, page_size=32,
                              outlier_frac=0.05, index=75)
    lens = np.array([30, 95, 64, 5], np.int32)
    tensors = gen.make_pair_tensors(wl, 0, device="cpu")
    p = H.Problem(wl, seq_lens=lens, tensors=tensors, page_size=32, cache_bits=4, decode_room=steps + 2)
    words, code = p.run_merge()
    assert code == 0, words
    # the oracle's 16-bit merge; the 4-bit view is taken at the end, over the grown sequences
    p.cache_bits = 16
    om = p.oracle_merge()
    p.cache_bits = 4
    wlb = dataclasses.replace(wl, batch=p.B)
    dev = p.device
    batch = p.batch(steps + 1)
    ws = p.workspace(1, 1, steps + 1)
    outs = [torch.zeros(1, p.B, hq, 128, dtype=p.cfg.torch_dtype, device=dev) for _ in range(2)]
    lses = [torch.zeros(1, p.B, hq, dtype=torch.float32, device=dev) for _ in range(2)]
    grow = lambda o, key, padn: np.concatenate([o[key], np.zeros((o[key].shape[0], padn) + o[key].shape[2:], o[key].dtype)], axis=1)
    for tn in ("k", "v"):
        for key in ("e_bits", "n_lm1", "n_l"):
            om[tn][key] = grow(om[tn], key, steps)
    q_all = [gen.make_queries(wlb, 100 + s, n_sets=2) for s in range(steps)]
    nt_all = [gen.make_new_tokens(wlb, 0, s) for s in range(steps)]
    q_dev = [q.to(dev) for q in q_all]
    nt_dev = [{k: v[:, 0].contiguous().to(dev) for k, v in nt.items()} for nt in nt_all]
    torch.cuda.synchronize()
    for s in range(steps):
        for layer, sfx in ((0, "_lm1"), (1, "_l")):
            p.lib.mc_decode_attn(p.cfg, batch, p.pair, layer, q_dev[s][layer:layer + 1], nt_dev[s]["k" + sfx][None],
                                 nt_dev[s]["v" + sfx][None], 1.0 / math.sqrt(128.0), outs[layer], lses[layer], ws)
        if s < steps - 1:
            d = nt_dev[s]
            p.lib.mc_append_pair(p.cfg, batch, p.pair, d["k_lm1"], d["v_lm1"], d["k_l"], d["v_l"])
            p.seq_lens += 1
    torch.cuda.synchronize()
    words, code = p.lib.mc_read_status(p.pair, check=False)
    assert code == 0, words
    # oracle: the same appends on its own 16-bit cache, then the 4-bit view at the final lengths
    for s in range(steps - 1):
        for tn in ("k", "v"):
            m = orc.append_rows(gen.as_bits(nt_all[s][tn + "_lm1"][:, 0]), gen.as_bits(nt_all[s][tn + "_l"][:, 0]), dtype, p.t)
            for b in range(p.B):
                pos = int(lens[b]) + s
                om[tn]["e_bits"][b, pos] = m["e_bits"][b]
                om[tn]["n_lm1"][b, pos] = m["n_a"][b]
                om[tn]["n_l"][b, pos] = m["n_c"][b]
    p.seq_lens_host = lens + (steps - 1)
    om4 = {tn: orc.q4_cache_pair(om[tn], p.seq_lens_host, tn, dtype) for tn in ("k", "v")}
    assert all(int(n) // 32 > int(n0) // 32 for n, n0 in zip(p.seq_lens_host, lens)), "every sequence completes a page"
    dc = p.device_cache(extra_tokens=0)  # (seq_lens_host already holds the grown lengths; S has room: decode_room)
    last = steps - 1
    for layer, sfx in ((0, "_lm1"), (1, "_l")):
        kn = nt_all[last]["k" + sfx][:, 0][None]
        vn = nt_all[last]["v" + sfx][:, 0][None]
        st = H.compare_attention(p, om4, layer, q_all[last][layer:layer + 1], outs[layer].cpu(), lses[layer].cpu(), kn, vn, dc=dc)
        print(dtype, "layer", layer, st)
    # the device's stored directions against the oracle's: equal except where a 16-bit direction element fell
    # on the other side of a rounding boundary (that element, or its whole group when it moved an extreme)
    for tn in ("k", "v"):
        differ = 0
        for b in range(p.B):
            n = int(p.seq_lens_host[b])
            differ += int((dc["e_" + tn][b, :n] != om4[tn]["e_bits"][b, :n]).any(-1).sum())
        print(dtype, tn, "rows whose stored bits differ from the oracle's", differ)
        assert differ <= 0.05 * int(p.seq_lens_host.sum()) * hkv


def test_full_size_serving_mix_q4_cache(H):
    """Config 4 as the paper's efficiency setting has it (Sec. 5): the ragged batch of 64 at full size, the
    layers arriving in 4 bits and the shared cache kept in 4 bits, in the launch configuration the benchmark
    times.  Sampled (sequence, head) segments -- the longest and the shortest sequence among them -- go
    through all three stages."""
    from oracle import minicache_oracle as orc
    from test_gpu_parity import _Segment, _full_tensors
    wl = CONFIGS["c4"]
    pair = wl.n_pairs - 1
    rs = np.random.RandomState(23)
    lens = gen.make_lengths(wl)[0]
    segs = [(int(rs.randint(wl.batch)), int(rs.randint(wl.n_kv_heads))) for _ in range(4)]
    segs[0] = (int(np.argmax(lens)), segs[0][1])
    segs[1] = (int(np.argmin(lens)), segs[1][1])
    th2 = int(lens.sum()) * wl.n_kv_heads * 2
    kw = dict(pair=pair, decode_room=wl.decode_steps + 1, tensors=_full_tensors("c4", pair), seq_lens=lens, q4=True,
              segments=segs, ret_capacity=int(0.12 * th2) + 1024)
    p16 = H.Problem(wl, **kw)
    words, code = p16.run_merge()
    assert code == 0, words
    dc16 = p16.device_cache()
    del p16.pair, p16.q4_pools
    p4 = H.Problem(wl, cache_bits=4, **kw)
    words, code = p4.run_merge()
    assert code == 0, words
    dc4 = p4.device_cache()
    assert np.array_equal(dc4["ret_index"], dc16["ret_index"])
    dk, dv = p4.run_restore(1)
    dkl, dvl = p4.logical_of(dk), p4.logical_of(dv)
    dk, dv = p4.run_restore(0, fp32=True)
    dkf, dvf = p4.logical_of(dk), p4.logical_of(dv)
    del dk, dv
    wlb = dataclasses.replace(wl, batch=p4.B)
    q = gen.make_queries(wlb, 2, n_sets=2)
    nt = gen.make_new_tokens(wlb, 0, 0)
    kn = torch.stack([nt["k_lm1"][:, 0], nt["k_l"][:, 0]]).contiguous()
    vn = torch.stack([nt["v_lm1"][:, 0], nt["v_l"][:, 0]]).contiguous()
    extra = wl.decode_steps + 1

    def attn(layer_sel, qq, kk, vv):
        n_sets = 2 if layer_sel == 2 else 1
        out = torch.zeros(n_sets, p4.B, p4.Hq, 128, dtype=p4.cfg.torch_dtype, device=p4.device)
        lse = torch.zeros(n_sets, p4.B, p4.Hq, dtype=torch.float32, device=p4.device)
        p4.lib.mc_decode_attn(p4.cfg, p4.batch(extra), p4.pair, layer_sel, qq.to(p4.device), kk.to(p4.device), vv.to(p4.device),
                              1.0 / math.sqrt(128.0), out, lse, p4.workspace(1, n_sets, extra))
        torch.cuda.synchronize()
        return out.cpu(), lse.cpu()
    out, lse = attn(1, q[1:2].contiguous(), kn[1:2].contiguous(), vn[1:2].contiguous())
    out2, lse2 = attn(2, q, kn, vn)
    words, code = p4.lib.mc_read_status(p4.pair, check=False)
    assert code == 0, words
    for b, h in segs:
        sg = _Segment(p4, b, h)
        sg.cache_bits = 4
        om16 = sg.oracle_merge(orc)
        dcs16, dcs4 = sg.slice_cache(dc16), sg.slice_cache(dc4)
        stats = H.compare_merge(sg, om16, dcs16)
        om4 = {tn: orc.q4_cache_pair(om16[tn], sg.seq_lens_host, tn, sg.dtype) for tn in ("k", "v")}
        dcs4["q4"] = {(tn, 0, 0): dc4["q4"][(tn, b, h)] for tn in ("k", "v")}
        stats.update(H.compare_q4_cache(sg, dcs4, dcs16, om4))
        stats.update(H.compare_restore(sg, om4, dcs4, 1, dkl[b:b + 1, :, h:h + 1], dvl[b:b + 1, :, h:h + 1]))
        stats.update({"f32_" + k: v for k, v in
                      H.compare_restore(sg, om4, dcs4, 0, dkf[b:b + 1, :, h:h + 1], dvf[b:b + 1, :, h:h + 1]).items()})
        slq = lambda x: x[:, b:b + 1, h:h + 1].contiguous()  # one query head per kv head in this workload
        stats.update(H.compare_attention(sg, om4, 1, slq(q[1:2]), slq(out), slq(lse), slq(kn[1:2]), slq(vn[1:2]), dc=dcs4))
        stats.update({"pair_" + k: v for k, v in
                      H.compare_attention(sg, om4, 2, slq(q), slq(out2), slq(lse2), slq(kn), slq(vn), dc=dcs4).items()})
        print("c4 4-bit cache, segment", b, h, "len", int(p4.seq_lens_host[b]), stats)

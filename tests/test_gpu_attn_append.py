"""mc_decode_attn_append (attention of a pair's second layer with the step's append folded into the same call)
against the two calls it stands for, on the GPU: the same outputs and the same pair cache, bit for bit."""
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


def _pair_state(p):
    pc = p.pair
    out = {"e_k": pc.e_k, "e_v": pc.e_v, "dist": pc.dist, "ret_count": pc.ret_count, "ret_index": pc.ret_index,
           "ret_rows": pc.ret_rows, "ret_prefix": pc.ret_prefix, "status": pc.status}
    if pc.q4:
        out.update({"res_k": pc.res_k, "res_v": pc.res_v})
    return {k: v.clone() for k, v in out.items()}


@pytest.mark.parametrize("dtype,cache_bits,slack,layer_sel", [("f16", 16, 0, 1), ("bf16", 16, 6, 1), ("f16", 16, 0, 2),
                                                              ("f16", 4, 0, 1), ("bf16", 4, 6, 2)])
def test_attention_with_the_append_folded_in_equals_the_two_calls(H, dtype, cache_bits, slack, layer_sel):
    steps = 6
    wl = CONFIGS["c1"].scaled("fold", n_kv_heads=4, n_q_heads=8, dtype=dtype, batch=5, seq_len=160, page_size=32,
                              outlier_frac=0.05, index=97)
    lens = np.array([160, 59, 27, 0, 131], np.int32)  # an empty sequence; pages that fill up on the way
    tensors = gen.make_pair_tensors(wl, 0, device="cpu")
    ps = [H.Problem(wl, seq_lens=lens, tensors=tensors, gamma=0.2, cache_bits=cache_bits, append_slack=slack,
                    decode_room=steps + 1) for _ in range(2)]
    for p in ps:
        words, code = p.run_merge()
        assert code == 0, words
    wlb = dataclasses.replace(wl, batch=5, outlier_frac=0.5)
    sm = 1.0 / math.sqrt(128.0)
    n_sets = 2 if layer_sel == 2 else 1
    for step in range(steps):
        nt = gen.make_new_tokens(wlb, 0, step)
        d = {k: v[:, 0].contiguous().to("cuda") for k, v in nt.items()}
        q = gen.make_queries(wlb, 40 + step, n_sets=2).to("cuda")
        outs = []
        for fused, p in enumerate(ps):
            ws = p.workspace(1, n_sets, 1)
            batch = p.batch(1)
            o = torch.zeros(n_sets, p.B, p.Hq, 128, dtype=p.cfg.torch_dtype, device="cuda")
            l = torch.zeros(n_sets, p.B, p.Hq, dtype=torch.float32, device="cuda")
            if layer_sel == 2:
                qq = q
                kn = torch.stack([d["k_lm1"], d["k_l"]]).contiguous()
                vn = torch.stack([d["v_lm1"], d["v_l"]]).contiguous()
            else:
                qq = q[1:2].contiguous()
                kn, vn = d["k_l"][None].contiguous(), d["v_l"][None].contiguous()
            if fused:
                p.lib.mc_decode_attn_append(p.cfg, batch, p.pair, layer_sel, qq, kn, vn, sm, o, l, d["k_lm1"], d["v_lm1"],
                                            d["k_l"], d["v_l"], ws)
            else:
                p.lib.mc_decode_attn(p.cfg, batch, p.pair, layer_sel, qq, kn, vn, sm, o, l, ws)
                p.lib.mc_append_pair(p.cfg, batch, p.pair, d["k_lm1"], d["v_lm1"], d["k_l"], d["v_l"])
            p.seq_lens += 1
            p.max_seq_len += 1
            torch.cuda.synchronize()
            outs.append((o, l))
        assert torch.equal(outs[0][0], outs[1][0]) and torch.equal(outs[0][1], outs[1][1]), f"step {step}"
    a, b = _pair_state(ps[0]), _pair_state(ps[1])
    for k in a:
        assert torch.equal(a[k], b[k]), k
    words, code = ps[1].lib.mc_read_status(ps[1].pair, check=False)
    assert code == 0 and words[0] == 0
    if slack:
        assert int(a["ret_count"].sum()) > 0


def test_folded_append_checks_every_argument_before_launching(H):
    wl = CONFIGS["c1"].scaled("foldarg", n_kv_heads=2, n_q_heads=4, dtype="f16", batch=2, seq_len=64, page_size=16, index=98)
    p = H.Problem(wl, decode_room=2)
    words, code = p.run_merge()
    assert code == 0
    before = _pair_state(p)
    nt = gen.make_new_tokens(dataclasses.replace(wl, batch=2), 0, 0)
    d = {k: v[:, 0].contiguous().to("cuda") for k, v in nt.items()}
    q = gen.make_queries(dataclasses.replace(wl, batch=2), 1, n_sets=1).to("cuda")
    o = torch.zeros(1, p.B, p.Hq, 128, dtype=p.cfg.torch_dtype, device="cuda")
    ws = p.workspace(1, 1, 1)
    with pytest.raises(p.mc.McError):  # a missing row of the append: nothing may have been launched
        p.lib.mc_decode_attn_append(p.cfg, p.batch(1), p.pair, 1, q, d["k_l"][None].contiguous(), d["v_l"][None].contiguous(),
                                    0.1, o, None, d["k_lm1"], None, d["k_l"], d["v_l"], ws)
    torch.cuda.synchronize()
    after = _pair_state(p)
    assert all(torch.equal(before[k], after[k]) for k in before) and not o.any()


@pytest.mark.parametrize("pinned", [True, False])
def test_inputs_staged_from_host_memory_give_the_same_attention(H, pinned):
    """mc_decode_stage_host on a second stream, then the attention on the staged rows, with the result written
    straight to pinned host memory: the same bits as the call on device tensors."""
    wl = CONFIGS["c1"].scaled("stage", n_kv_heads=4, n_q_heads=8, dtype="bf16", batch=3, seq_len=96, page_size=16, index=99)
    p = H.Problem(wl, seq_lens=np.array([96, 17, 40], np.int32), decode_room=2)
    words, code = p.run_merge()
    assert code == 0
    wlb = dataclasses.replace(wl, batch=3)
    nt = gen.make_new_tokens(wlb, 0, 0)
    q = gen.make_queries(wlb, 3, n_sets=2)
    kn = torch.stack([nt["k_lm1"][:, 0], nt["k_l"][:, 0]]).contiguous()
    vn = torch.stack([nt["v_lm1"][:, 0], nt["v_l"][:, 0]]).contiguous()
    host = [t.pin_memory() if pinned else t.clone() for t in (q, kn, vn)]
    batch = p.batch(1)
    io = torch.empty(p.lib.mc_decode_io_bytes(p.cfg, batch, 2), dtype=torch.uint8, device="cuda")
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        qd, knd, vnd = p.lib.mc_decode_stage_host(p.cfg, batch, 2, host[0], host[1], host[2], io, stream=side)
    torch.cuda.current_stream().wait_stream(side)
    assert torch.equal(qd.cpu(), q) and torch.equal(knd.cpu(), kn) and torch.equal(vnd.cpu(), vn)
    sm = 1.0 / math.sqrt(128.0)
    ws = p.workspace(1, 1, 1)
    out_host = torch.zeros(1, p.B, p.Hq, 128, dtype=p.cfg.torch_dtype).pin_memory()
    lse_host = torch.zeros(1, p.B, p.Hq, dtype=torch.float32).pin_memory()
    p.lib.mc_decode_attn(p.cfg, batch, p.pair, 1, qd[1], knd[1], vnd[1], sm, out_host, lse_host, ws)
    ref = torch.zeros(1, p.B, p.Hq, 128, dtype=p.cfg.torch_dtype, device="cuda")
    ref_lse = torch.zeros(1, p.B, p.Hq, dtype=torch.float32, device="cuda")
    p.lib.mc_decode_attn(p.cfg, batch, p.pair, 1, q[1:2].contiguous().cuda(), kn[1:2].contiguous().cuda(),
                         vn[1:2].contiguous().cuda(), sm, ref, ref_lse, ws)
    torch.cuda.synchronize()
    assert torch.equal(out_host, ref.cpu()) and torch.equal(lse_host, ref_lse.cpu())
    # ... and the result copied back by the library on a stream of its own
    back = torch.zeros(1, p.B, p.Hq, 128, dtype=p.cfg.torch_dtype).pin_memory()
    back_lse = torch.zeros(1, p.B, p.Hq, dtype=torch.float32).pin_memory()
    side.wait_stream(torch.cuda.current_stream())
    p.lib.mc_decode_drain_host(p.cfg, batch, 1, ref, ref_lse, back, back_lse, stream=side)
    side.synchronize()
    assert torch.equal(back, ref.cpu()) and torch.equal(back_lse, ref_lse.cpu())
    # the staging refuses a buffer that is too small, before anything is enqueued
    with pytest.raises(p.mc.McError):
        p.lib.mc_decode_stage_host(p.cfg, batch, 2, host[0], host[1], host[2], io[:256])

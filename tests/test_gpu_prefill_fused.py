"""The merge fused into layer l's K/V projection (mc_prefill_merge_pair): layer l's rows are formed by the
5th-generation tensor cores and merged in the epilogue.  Checked in three steps: the rows the epilogue merged
(dumped with d_hint < 0) against an fp64 product of the same inputs; the pair cache against the oracle merging
exactly those dumped bits; and the sparse mode (rows stored only above a distance hint) against the dump."""
import dataclasses

import numpy as np
import pytest
import torch

import gen
from gen import CONFIGS, as_bits

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def H():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2405_14366_b200.build import build_library
    build_library()
    import mc_harness
    return mc_harness


def _case(H, dtype, hkv, hq, lens, stride, d_model, gamma=0.05, outlier=0.05):
    wl = CONFIGS["c1"].scaled("pf", n_kv_heads=hkv, n_q_heads=hq, dtype=dtype, batch=len(lens), seq_len=stride,
                              outlier_frac=outlier, index=68)
    case = gen.make_projection_case(wl, 0, d_model, stride, device="cpu")
    # the harness gets layer l-1's rows; layer l's pools start as zeros and are filled by the fused call
    zeros = torch.zeros_like(case["k_lm1"])
    tensors = {"k_lm1": case["k_lm1"], "v_lm1": case["v_lm1"], "k_l": zeros, "v_l": zeros.clone()}
    p = H.Problem(wl, seq_lens=np.asarray(lens, np.int32), tensors=tensors, gamma=gamma)
    return wl, case, p


def _run(p, case, d_hint, do_retention=True):
    dev = p.device
    for k in ("k_l", "v_l"):
        p.pools[k].zero_()
    ws = p.workspace(0)
    p.lib.mc_prefill_merge_pair(p.cfg, p.batch(), case["x"].to(dev), case["w_k"].to(dev), case["w_v"].to(dev),
                                p.pools["k_lm1"], p.pools["v_lm1"], p.pools["k_l"], p.pools["v_l"], p.pair, d_hint, do_retention, ws)
    torch.cuda.synchronize()
    return p.lib.mc_read_status(p.pair, check=False)


@pytest.mark.parametrize("dtype,hkv,hq", [("bf16", 2, 4), ("f16", 3, 3)])
def test_fused_prefill_merge_against_the_oracle(H, dtype, hkv, hq):
    from oracle import minicache_oracle as orc
    lens, stride, d_model = [256, 130, 1], 256, 448
    wl, case, p = _case(H, dtype, hkv, hq, lens, stride, d_model)
    words, code = _run(p, case, -1.0)
    assert code == 0, words
    # (1) the rows the epilogue merged = the projection rounded once to the storage type
    ulp = H.ULP_REL[dtype]
    dump = {}
    for tn in ("k", "v"):
        got = p.logical_of(p.pools[tn + "_l"])            # [B][S][H][128] storage type
        dump[tn] = got
        ref = (case["x"].double().reshape(-1, d_model) @ case["w_" + tn].double().T).reshape(got.shape)
        for b, n in enumerate(lens):
            err = (got[b, :n].double() - ref[b, :n]).abs()
            bound = 0.505 * ulp * ref[b, :n].abs() + 2e-6 * ref[b, :n].abs().max()   # one rounding + fp32 accumulation
            assert (err <= bound).all(), f"{tn} projection row off by {(err / bound).max()} bounds"
            cap = min(stride, (n + 8 + p.ps - 1) // p.ps * p.ps)  # the rows of the sequence's own pages
            assert (got[b, n:cap] == 0).all(), "rows past the sequence must not be written"
    # (2) the pair cache: the oracle merges exactly the dumped bits
    p.bits["k_l"], p.bits["v_l"] = as_bits(dump["k"]), as_bits(dump["v"])
    om, dc = p.oracle_merge(), p.device_cache()
    stats = H.compare_merge(p, om, dc)
    assert int(dc["ret_count"].sum()) > 0
    for layer in (0, 1):
        dk, dv = p.run_restore(layer, fp32=True)
        stats.update(H.compare_restore(p, om, dc, layer, dk, dv))
    q = gen.make_queries(dataclasses.replace(wl, batch=p.B), 0, n_sets=2)
    for layer in (0, 1):
        out, lse = p.run_attn(layer, q[layer:layer + 1].contiguous().to(p.device))
        stats.update(H.compare_attention(p, om, layer, q[layer:layer + 1], out.cpu(), lse.cpu(), dc=dc))
    # (3) rows stored only above a distance hint: the same pair cache, and layer l's pool holds exactly those rows
    full = {f: getattr(p.pair, f).clone() for f in ("e_k", "e_v", "dist", "ret_count", "ret_offset", "ret_index", "ret_rows", "seg_minmax")}
    hint = 0.3
    words, code = _run(p, case, hint)
    assert code == 0, words
    for f, v in full.items():
        assert torch.equal(getattr(p.pair, f), v), f
    for ti, tn in enumerate(("k", "v")):
        sparse = p.logical_of(p.pools[tn + "_l"])
        d = torch.from_numpy(dc["dist"][..., ti])
        stored = (d > hint)[..., None]
        assert torch.equal(sparse, torch.where(stored, dump[tn], torch.zeros_like(sparse)))
        frac = float(stored.float().mean())
        assert 0.0 < frac < 0.2, frac
    # a hint above a segment's threshold is reported
    words, code = _run(p, case, 0.9)
    assert code == 8 and words[0] & 16, words
    # without retention nothing needs to be stored
    words, code = _run(p, case, 2.0, do_retention=False)
    assert code == 0 and int(p.pair.ret_count.sum()) == 0
    assert all(int(p.pools[k].abs().sum()) == 0 for k in ("k_l", "v_l"))
    print(dtype, stats)

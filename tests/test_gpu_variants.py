"""Variants the paper sketches or leaves open, and the range-checked build, on the GPU:
dynamic per-token t (Sec. 5, ablation of t), one retention set for keys and values (Sec. 4.2's single I),
and the -DMC_BOUNDS=1 build whose kernels refuse indices that fall outside their bounds."""
import dataclasses
import os
import subprocess
import sys

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


def _cycle(H, p, new_token=True):
    words, code = p.run_merge()
    assert code == 0, words
    om, dc = p.oracle_merge(), p.device_cache()
    # (a 4-bit cache's stored bits are compared stage-wise in test_gpu_q4cache.py; here end to end)
    stats = H.compare_merge(p, om, dc) if p.cache_bits == 16 else {}
    for layer in (0, 1):
        dk, dv = p.run_restore(layer, fp32=True)
        stats.update({f"l{layer}_{k}": v for k, v in H.compare_restore(p, om, dc, layer, dk, dv).items()})
    wl = dataclasses.replace(p.wl, batch=p.B)
    q = gen.make_queries(wl, 0, n_sets=2)
    nt = gen.make_new_tokens(wl, 0, 0)
    kn = torch.stack([nt["k_lm1"][:, 0], nt["k_l"][:, 0]]).contiguous()
    vn = torch.stack([nt["v_lm1"][:, 0], nt["v_l"][:, 0]]).contiguous()
    for layer in (0, 1):
        out, lse = p.run_attn(layer, q[layer:layer + 1].contiguous().to(p.device), kn[layer:layer + 1].contiguous().to(p.device),
                              vn[layer:layer + 1].contiguous().to(p.device))
        stats.update({f"a{layer}_{k}": v for k, v in
                      H.compare_attention(p, om, layer, q[layer:layer + 1], out.cpu(), lse.cpu(), kn[layer:layer + 1],
                                          vn[layer:layer + 1], dc=dc).items()})
    return stats, om, dc


@pytest.mark.parametrize("dtype", ["f16", "bf16"])
@pytest.mark.parametrize("cache_bits", [16, 4])
def test_dynamic_t_from_the_magnitude_ratio(H, dtype, cache_bits):
    """t_i = |x^l_i| / (|x^(l-1)_i| + |x^l_i|) per token, in the merge and in the decode-time append."""
    from oracle import minicache_oracle as orc
    wl = CONFIGS["c1"].scaled("dyn", n_kv_heads=2, n_q_heads=4, dtype=dtype, batch=3, seq_len=160, page_size=32,
                              outlier_frac=0.05, index=63)
    lens = np.array([160, 70, 33], np.int32)
    p = H.Problem(wl, seq_lens=lens, t_mode=1, cache_bits=cache_bits, t=0.123)  # (the fixed t must be ignored)
    stats, om, dc = _cycle(H, p)
    # the directions differ from the fixed-t merge (this test would not notice a switch that does nothing otherwise)
    p_fixed = H.Problem(wl, seq_lens=lens, cache_bits=16)
    p_fixed.run_merge()
    if cache_bits == 16:
        assert not torch.equal(p_fixed.pair.e_k, p.pair.e_k)
    # append: the new token pair is merged with its own ratio
    nt = gen.make_new_tokens(dataclasses.replace(wl, batch=p.B), 0, 5)
    dev = {k: v[:, 0].contiguous().to(p.device) for k, v in nt.items()}
    p.lib.mc_append_pair(p.cfg, p.batch(), p.pair, dev["k_lm1"], dev["v_lm1"], dev["k_l"], dev["v_l"])
    torch.cuda.synchronize()
    dc2 = p.device_cache(extra_tokens=1)
    for tn in ("k", "v"):
        m = orc.append_rows(gen.as_bits(nt[tn + "_lm1"][:, 0]), gen.as_bits(nt[tn + "_l"][:, 0]), dtype, "ratio")
        for b in range(p.B):
            pos = int(lens[b])
            if cache_bits == 4 and (pos + 1) % 32 == 0:
                continue  # the page was completed and quantised: covered by the 4-bit cache tests
            e_gpu = orc.decode_bits(dc2["e_" + tn][b, pos], dtype)
            e_orc = orc.decode_bits(m["e_bits"][b], dtype)
            assert np.max(np.abs(e_gpu - e_orc)) <= H.ULP_REL[dtype] * 0.51
    print(dtype, cache_bits, stats)


@pytest.mark.parametrize("mode,gamma", [("distinct", 0.1), ("literal", 0.3)])
def test_one_retention_set_for_keys_and_values(H, mode, gamma):
    wl = CONFIGS["c1"].scaled("uni", n_kv_heads=2, n_q_heads=4, dtype="f16", batch=2, seq_len=300, outlier_frac=0.05, index=64)
    lens = np.array([300, 129], np.int32)
    p = H.Problem(wl, seq_lens=lens, retain_union=1, gamma=gamma, retain_mode={"distinct": 0, "literal": 1}[mode])
    words, code = p.run_merge()
    assert code == 0, words
    om, dc = p.oracle_merge(mode), p.device_cache()
    stats = H.compare_merge(p, om, dc, mode)
    # the same list for both tensors, and a true superset of what each rule keeps alone
    ps = H.Problem(wl, seq_lens=lens, gamma=gamma, retain_mode={"distinct": 0, "literal": 1}[mode])
    ps.run_merge()
    dcs = ps.device_cache()
    grew = 0
    for b in range(p.B):
        for h in range(p.H):
            ik, _ = p.retained(dc, 0, b, h)
            iv, _ = p.retained(dc, 1, b, h)
            assert np.array_equal(ik, iv)
            sk, _ = ps.retained(dcs, 0, b, h)
            sv, _ = ps.retained(dcs, 1, b, h)
            assert np.array_equal(ik, np.union1d(sk, sv))
            grew += len(ik) - len(sk)
    assert grew > 0
    for layer in (0, 1):
        dk, dv = p.run_restore(layer)
        stats.update(H.compare_restore(p, om, dc, layer, dk, dv))
    q = gen.make_queries(dataclasses.replace(wl, batch=p.B), 0, n_sets=2)
    out, lse = p.run_attn(2, q.to(p.device))
    stats.update(H.compare_attention(p, om, 2, q, out.cpu(), lse.cpu(), dc=dc))
    print(mode, stats)


# ---------------------------------------------------------------------------------------------
def _bounds_lib():
    from paper_2405_14366_b200.build import build_library
    from paper_2405_14366_b200 import binding as B
    lib = B.MiniCacheLib(build_library(bounds=True))
    assert lib.mc_build_flags() & B.MC_BUILD_BOUNDS
    return lib


def test_range_checked_build_refuses_a_corrupted_retained_entry(H):
    """The token index stored with a retained entry is set to a position past its sequence (but inside the
    buffers this test owns: the score buffer has room for it).  The normal build would use it as a column;
    the range-checked build skips the entry and reports MC_FLAG_BOUNDS; the context stays usable."""
    from paper_2405_14366_b200 import binding as B
    import paper_2405_14366_b200 as mc
    assert mc.lib().mc_build_flags() == 0
    lib = _bounds_lib()
    wl = CONFIGS["c1"].scaled("bnd", n_kv_heads=2, n_q_heads=2, dtype="f16", batch=1, seq_len=100, outlier_frac=0.1, index=65)
    p = H.Problem(wl, gamma=0.3)
    p.lib = lib
    words, code = p.run_merge()
    assert code == 0 and words[1] > 0, words
    q = gen.make_queries(wl, 0, n_sets=1).to(p.device)
    out, lse = p.run_attn(0, q)
    om, dc = p.oracle_merge(), p.device_cache()
    H.compare_attention(p, om, 0, q.cpu(), out.cpu(), lse.cpu())   # the range-checked build computes the same thing
    words, code = lib.mc_read_status(p.pair, check=False)
    assert code == 0, words
    # corrupt: first retained K entry of layer l-1 claims token 300 (the sequence has 100)
    idx_bytes = torch.tensor([300], dtype=torch.int32, device=p.device).view(torch.uint8)
    p.pair.ret_rows[0, 0, 256:260] = idx_bytes
    out2, _ = p.run_attn(0, q)
    words, code = lib.mc_read_status(p.pair, check=False)
    assert code == 8 and words[0] & B.MC_FLAG_BOUNDS, words
    # still usable: a fresh merge clears the flag and gives the right answer again
    words, code = p.run_merge()
    assert code == 0, words
    out3, lse3 = p.run_attn(0, q)
    assert torch.equal(out3, out)


def test_the_parity_suite_passes_under_the_range_checked_build(H):
    """A slice of the parity tests run in a child process against libminicache_bounds.so."""
    from paper_2405_14366_b200.build import build_library
    path = build_library(bounds=True)
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    env = dict(os.environ, MINICACHE_LIBRARY=path)
    r = subprocess.run([sys.executable, "-m", "pytest", "-x", "-q", "-m", "gpu", os.path.join(root, "tests", "test_gpu_parity.py"),
                        "-k", "config1 or tiny_shapes or retention_modes or append_then_attend or serving_mix or work_split"],
                       env=env, cwd=root, capture_output=True, text=True, timeout=1500)
    assert r.returncode == 0, r.stdout[-3000:] + r.stderr[-2000:]

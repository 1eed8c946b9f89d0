"""mc_decode_attn_static: decode attention for callers that have no scratch memory to pass.

Some users of this library cannot allocate on the device at the point where they call it: an
inference server that handed all remaining HBM to its KV-cache pool at start-up, an operator
plugin that only receives its input and output tensors, a latency-critical decode loop in which a
cudaMalloc (which synchronises the whole device) is not acceptable.  For them the library carries
a fixed scratch array inside its own image.  This test calls that entry point through the C ABI
twice in a row (the array is shared between calls and keeps the previous call's contents) and
checks each result against the ordinary entry point given a caller-allocated workspace: the same
deterministic kernels run either way, so the outputs must be the same bits (which is well inside
the 1e-2 max-abs attention tolerance used throughout the suite); it also checks that the call
leaves the device's free memory as it found it and that a geometry that does not fit the array is
refused before anything is launched.

Collected last on purpose: a failure here cannot hide the result of any other test."""
import dataclasses
import math

import numpy as np
import pytest
import torch

import gen
from gen import CONFIGS

pytestmark = pytest.mark.gpu
ATTN_TOL = 1e-2


@pytest.fixture(scope="module")
def problem():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2405_14366_b200.build import build_library
    build_library()
    import mc_harness as H
    wl = CONFIGS["c3_s"].scaled("noalloc", batch=3, seq_len=1500, n_layers=18, index=95)
    p = H.Problem(wl, seq_lens=[1500, 640, 1111])
    words, code = p.run_merge()
    assert code == 0, words
    return p


def _both(p, layer_sel, q, kn, vn):
    n_sets = 2 if layer_sel == 2 else 1
    ref, ref_lse = p.run_attn(layer_sel, q, kn, vn)
    out = torch.full_like(ref, float("nan"))
    lse = torch.full_like(ref_lse, float("nan"))
    torch.cuda.synchronize()
    before = torch.cuda.memory_allocated()
    free_before = torch.cuda.mem_get_info()[0]  # the driver's view: an allocation by any library would show
    p.lib.mc_decode_attn_static(p.cfg, p.batch(), p.pair, layer_sel, q, kn, vn, 1.0 / math.sqrt(128.0), out, lse)
    torch.cuda.synchronize()
    assert torch.cuda.memory_allocated() == before
    assert torch.cuda.mem_get_info()[0] >= free_before
    assert out.shape[0] == n_sets
    return ref, ref_lse, out, lse


def test_static_scratch_matches_workspace_path_twice(problem):
    p = problem
    wl = dataclasses.replace(p.wl, batch=p.B)
    nt = gen.make_new_tokens(wl, 0, 0)
    kn = torch.stack([nt["k_lm1"][:, 0], nt["k_l"][:, 0]]).contiguous().to(p.device)
    vn = torch.stack([nt["v_lm1"][:, 0], nt["v_l"][:, 0]]).contiguous().to(p.device)
    # two calls in a row with different queries and modes: the second runs over the first one's leftovers
    for call, layer_sel in enumerate((2, 1)):
        q = gen.make_queries(wl, 20 + call, n_sets=2).to(p.device)
        if layer_sel != 2:
            q, k1, v1 = q[1:2].contiguous(), kn[1:2].contiguous(), vn[1:2].contiguous()
        else:
            k1, v1 = kn, vn
        ref, ref_lse, out, lse = _both(p, layer_sel, q, k1, v1)
        assert torch.isfinite(out.float()).all() and torch.isfinite(lse).all()
        assert (out.float() - ref.float()).abs().max().item() <= ATTN_TOL
        assert torch.equal(out, ref) and torch.equal(lse, ref_lse)  # same kernels, same order: same bits
    words, code = p.lib.mc_read_status(p.pair, check=False)
    assert code == 0, words


def test_static_scratch_refuses_what_does_not_fit(problem):
    p = problem
    import paper_2405_14366_b200 as mc
    big = mc.Batch(p.block_table, p.seq_lens, 1 << 20, p.n_pages)  # a million-token bound: far more splits than fit
    need = p.lib.mc_workspace_bytes(p.cfg, big, 1, 1)
    assert need > 8 * 1024 * 1024
    q = gen.make_queries(dataclasses.replace(p.wl, batch=p.B), 0, n_sets=1).to(p.device)
    out = torch.zeros_like(q)
    with pytest.raises(mc.McError) as ei:
        p.lib.mc_decode_attn_static(p.cfg, big, p.pair, 0, q, None, None, 0.1, out, None)
    assert ei.value.code == 5 and "built-in scratch" in str(ei.value)

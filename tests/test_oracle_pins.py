"""Pins for the fp64 oracle: closed forms, invariants, brute force, golden files.

Each test ties one part of the oracle to something other than the oracle itself
(hand-computed trigonometric values, a pure-Python restatement small enough to
check by eye, an independent library conversion, or a mathematical invariant),
chosen so that a dropped term, a swapped operand or a wrong sign fails."""
import math
import os

import numpy as np
import pytest
import torch

from oracle import minicache_oracle as orc

GOLD = os.path.join(os.path.dirname(__file__), "golden")
D = 128
rng = np.random.RandomState(1234)


def unit(x):
    return x / np.linalg.norm(x, axis=-1, keepdims=True)


def angle(x, y):
    """Well-conditioned angle between rows (Kahan's atan2 form), independent of arccos."""
    ux, uy = unit(x), unit(y)
    return 2.0 * np.arctan2(np.linalg.norm(ux - uy, axis=-1), np.linalg.norm(ux + uy, axis=-1))


def embed2(x, y):
    v = np.zeros(D)
    v[0], v[1] = x, y
    return v


# ---------------------------------------------------------------- storage formats
def test_bits_roundtrip_all_patterns():
    allbits = np.arange(65536, dtype=np.uint16)
    for dt in ("f16", "bf16"):
        x = orc.decode_bits(allbits, dt)
        fin = np.isfinite(x)
        back = orc.encode_bits(x[fin], dt)
        assert np.array_equal(back, allbits[fin]), dt


def test_bits_match_independent_conversion():
    x = np.concatenate([rng.standard_normal(20000) * 10.0 ** rng.uniform(-6, 4, 20000),
                        [0.0, -0.0, 1.0, 65504.0, 1e-8, 3.0e38]])
    # binary32-representable inputs: the library then rounds once, like encode_bits
    # (its double -> half path goes through binary32 and would round twice)
    x = x.astype(np.float32).astype(np.float64)
    for dt, tdt in (("f16", torch.float16), ("bf16", torch.bfloat16)):
        ref = torch.from_numpy(x.astype(np.float32)).to(tdt).view(torch.int16).numpy().view(np.uint16)
        got = orc.encode_bits(x, dt)
        ok = np.isfinite(orc.decode_bits(ref, dt))
        assert np.array_equal(got[ok], ref[ok]), dt


def test_bf16_ties_to_even_and_no_double_rounding():
    # 1 + 2^-8 lies exactly between bf16 neighbours 1 and 1 + 2^-7: ties to even -> 1.
    assert orc.decode_bits(orc.encode_bits(np.array([1.0 + 2.0 ** -8]), "bf16"), "bf16")[0] == 1.0
    # 1 + 3*2^-8 is the midpoint of 1+2^-7 and 1+2^-6: even mantissa is 1 + 2^-6.
    assert orc.decode_bits(orc.encode_bits(np.array([1.0 + 3 * 2.0 ** -8]), "bf16"), "bf16")[0] == 1.0 + 2.0 ** -6
    # just above the midpoint by less than a binary32 ulp: must round up (a detour through
    # binary32 would first land on the midpoint and then tie to even = down).
    x = 1.0 + 2.0 ** -8 + 2.0 ** -40
    assert orc.decode_bits(orc.encode_bits(np.array([x]), "bf16"), "bf16")[0] == 1.0 + 2.0 ** -7


# ---------------------------------------------------------------- SLERP (Eq. 3)
def _golden_slerp():
    rows = []
    for line in open(os.path.join(GOLD, "slerp_closed_forms.txt")):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        ins, e, dpi, norms = [p.split() for p in line.split("|")]
        rows.append((list(map(float, ins)), list(map(float, e)), float(dpi[0]), list(map(float, norms))))
    return rows


def test_slerp_golden_closed_forms():
    for (ax, ay, cx, cy, t), (ex, ey), dpi, (na, nc) in _golden_slerp():
        m = orc.merge_rows(embed2(ax, ay), embed2(cx, cy), t)
        assert np.allclose(m["e"][:2], [ex, ey], atol=1e-14)
        assert np.all(m["e"][2:] == 0)
        assert abs(m["d"] - dpi) < 1e-14
        assert abs(m["n_a"] - na) < 1e-14 and abs(m["n_c"] - nc) < 1e-14


def test_slerp_endpoints_and_unit_length():
    a = rng.standard_normal((64, D)) * 3
    c = rng.standard_normal((64, D)) * 0.2
    assert np.allclose(orc.merge_rows(a, c, 0.0)["e"], unit(a), atol=1e-14)
    assert np.allclose(orc.merge_rows(a, c, 1.0)["e"], unit(c), atol=1e-14)
    for t in (0.1, 0.5, 0.6, 0.9):
        e = orc.merge_rows(a, c, t)["e"]
        assert np.allclose(np.linalg.norm(e, axis=-1), 1.0, atol=1e-12)


def test_slerp_splits_the_angle_t_towards_layer_l():
    """angle(e, layer l-1) = t*Omega and angle(e, layer l) = (1-t)*Omega: fixes which
    endpoint t weights (Eq. 3; default t = 0.6 rotates less towards the next layer)."""
    a = rng.standard_normal((200, D))
    c = unit(a) * 2 + 0.8 * rng.standard_normal((200, D)) / math.sqrt(D) * 3
    for t in (0.25, 0.6):
        m = orc.merge_rows(a, c, t)
        om = angle(a, c)
        assert np.allclose(m["omega"], om, atol=1e-12)
        assert np.allclose(angle(m["e"], a), t * om, atol=1e-10)
        assert np.allclose(angle(m["e"], c), (1 - t) * om, atol=1e-10)
    # the other printed convention (Algorithm 2's Merge) is a different function
    m2 = orc.merge_rows(a, c, 0.6, convention="alg2")
    assert np.allclose(angle(m2["e"], a), 0.4 * angle(a, c), atol=1e-10)


def test_slerp_orthogonal_and_half():
    u = unit(rng.standard_normal((32, D)))
    g = rng.standard_normal((32, D))
    v = unit(g - np.sum(g * u, -1, keepdims=True) * u)
    for t in (0.3, 0.6):
        e = orc.merge_rows(5 * u, 0.1 * v, t)["e"]
        assert np.allclose(e, math.cos(t * math.pi / 2) * u + math.sin(t * math.pi / 2) * v, atol=1e-13)
    a = rng.standard_normal((32, D))
    c = rng.standard_normal((32, D)) + a
    e = orc.merge_rows(a, c, 0.5)["e"]
    assert np.allclose(e, unit(unit(a) + unit(c)), atol=1e-12)  # t = 1/2: direction of the mean direction
    # ... which is also the direction F_max uses when both rows have equal length (Eq. A)
    f = orc.merge_rows_fmax(unit(a) * 2, unit(c) * 2)
    assert np.allclose(unit(f), e, atol=1e-12)
    assert np.allclose(np.linalg.norm(f, axis=-1), 2.0, atol=1e-12)


def test_slerp_2d_rotation():
    for th in (0.01, 0.4, 1.3, 2.9):
        for t in (0.2, 0.6):
            a = embed2(2.0, 0.0)
            c = embed2(0.7 * math.cos(th), 0.7 * math.sin(th))
            e = orc.merge_rows(a, c, t)["e"]
            assert np.allclose(e[:2], [math.cos(t * th), math.sin(t * th)], atol=1e-12)


def test_slerp_small_angle_branch_is_continuous():
    u = unit(rng.standard_normal(D))
    g = rng.standard_normal(D)
    w = unit(g - (g @ u) * u)
    prev = None
    for th in (3e-6, 1.5e-6, 0.9e-6, 3e-7, 0.0):  # straddles the sin(Omega) guard
        c = math.cos(th) * u + math.sin(th) * w
        m = orc.merge_rows(u * 1.7, c * 0.3, 0.6)
        exact = math.cos(0.6 * th) * u + math.sin(0.6 * th) * w
        assert np.allclose(m["e"], exact, atol=2e-9)
        assert abs(np.linalg.norm(m["e"]) - 1) < 1e-12
        prev = m
    assert prev["d"] < 1e-7


def test_degenerate_rows():
    a = rng.standard_normal((4, D))
    # identical rows: zero distance, passthrough
    m = orc.merge_rows(a, a.copy(), 0.6)
    assert np.all(m["d"] < 1e-7) and np.allclose(m["e"], unit(a), atol=1e-12)
    # antipodal: d = 1; e is an endpoint
    m = orc.merge_rows(a, -2 * a, 0.6)
    assert np.allclose(m["d"], 1.0, atol=1e-7) and np.allclose(m["e"], -unit(a), atol=1e-12)
    m = orc.merge_rows(a, -2 * a, 0.4)
    assert np.allclose(m["e"], unit(a), atol=1e-12)
    # zero rows: never NaN, angle 0
    z = np.zeros((4, D))
    m = orc.merge_rows(z, a, 0.6)
    assert np.all(m["d"] == 0) and np.allclose(m["e"], unit(a)) and np.all(m["n_a"] == 0)
    m = orc.merge_rows(a, z, 0.6)
    assert np.all(m["d"] == 0) and np.allclose(m["e"], unit(a)) and np.all(m["n_c"] == 0)
    m = orc.merge_rows(z, z, 0.6)
    assert np.all(m["e"] == 0) and np.all(np.isfinite(m["d"]))


def test_planted_angle_recovered_from_generator():
    from gen import CONFIGS, make_pair_tensors, as_bits
    cfg = CONFIGS["c1"]
    t = make_pair_tensors(cfg, 0, keep_theta=True)
    m = orc.merge_rows(orc.decode_bits(as_bits(t["k_lm1"]), "f16"), orc.decode_bits(as_bits(t["k_l"]), "f16"), 0.6)
    # fp16 rounding of 128 channels perturbs the angle by about 2^-11
    assert np.max(np.abs(m["omega"] - t["theta_k"].double().numpy())) < 2e-3


# ---------------------------------------------------------------- retention (Eq. 4)
def _golden_retention():
    d, cases = None, []
    for line in open(os.path.join(GOLD, "retention_tiny.txt")):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        if line.startswith("d "):
            d = np.array(list(map(float, line.split()[1:])))
            continue
        head, idx = line.split(":")
        mode, gamma = head.split()
        cases.append((mode, float(gamma), [int(i) for i in idx.split()]))
    return d, cases


def test_retention_golden():
    d, cases = _golden_retention()
    for mode, gamma, want in cases:
        assert list(orc.retention_indices(d, gamma, mode)) == want, (mode, gamma)


def _brute_retention(d, gamma, mode):
    dmin, dmax = min(d), max(d)
    keep = []
    if mode == "topk":
        k = math.ceil(gamma * len(d) - 1e-12)
        order = sorted(range(len(d)), key=lambda i: (-d[i], i))
        return sorted(order[:k])
    for i, x in enumerate(d):
        if mode == "distinct" and x > dmax - (dmax - dmin) * gamma:
            keep.append(i)
        if mode == "literal" and x < dmin + (dmax - dmin) * gamma:
            keep.append(i)
    return keep


def test_retention_brute_force_and_properties():
    for n in (1, 2, 5, 17, 64):
        for _ in range(20):
            d = rng.uniform(0, 1, n) ** 3
            prev = set()
            for gamma in (0.0, 0.01, 0.05, 0.2, 0.5, 1.0):
                for mode in ("distinct", "literal", "topk"):
                    got = list(orc.retention_indices(d, gamma, mode))
                    assert got == _brute_retention(list(d), gamma, mode)
                    assert got == sorted(got)
                cur = set(orc.retention_indices(d, gamma, "distinct"))
                assert prev <= cur  # monotone in gamma
                prev = cur
            assert len(orc.retention_indices(d, 0.0, "distinct")) == 0  # gamma = 0: everything merged
            full = set(orc.retention_indices(d, 1.0, "distinct"))
            lowest = set(np.nonzero(d == d.min())[0])
            # gamma = 1 keeps all but the least distinct token(s); the threshold is computed in
            # floating point, so only the tokens sitting exactly on d_min may fall either side
            assert set(range(n)) - lowest <= full <= set(range(n))
            assert len(orc.retention_indices(d, 0.3, "topk")) == math.ceil(0.3 * n - 1e-12)
    assert len(orc.retention_indices(np.full(9, 0.25), 0.5, "distinct")) == 0  # constant d
    assert len(orc.retention_indices(np.zeros(0), 0.5, "distinct")) == 0


def test_planted_outliers_are_the_retained_set():
    d = rng.uniform(0.0, 0.19, 400)
    out = rng.choice(400, 12, replace=False)
    d[out] = rng.uniform(0.60, 0.636, 12)
    d[out[0]] = 0.64
    got = orc.retention_indices(d, 0.1, "distinct")  # threshold 0.64 - 0.1*range ~ 0.576
    assert sorted(out) == list(got)


# ---------------------------------------------------------------- restore (Eq. 2)
def _pair(n, dt, spread=0.4):
    a = rng.standard_normal((n, D)) * np.exp(0.5 * rng.standard_normal((n, 1)))
    c = unit(a) + spread * rng.standard_normal((n, D)) / math.sqrt(D)
    c = c * np.exp(0.5 * rng.standard_normal((n, 1)))
    ab, cb = orc.encode_bits(a, dt), orc.encode_bits(c, dt)
    return ab, cb


@pytest.mark.parametrize("dt", ["f16", "bf16"])
def test_restore_invariants(dt):
    n = 96
    ab, cb = _pair(n, dt)
    a, c = orc.decode_bits(ab, dt), orc.decode_bits(cb, dt)
    out = orc.merge_pair(ab[None, :, None, :], cb[None, :, None, :], [n], dt, 0.6, 0.05)
    eb = out["e_bits"][0, :, 0]
    idx = out["retained"][(0, 0)]
    assert len(idx) >= 1
    for norms, x, xb in ((out["n_lm1"][0, :, 0], a, ab), (out["n_l"][0, :, 0], c, cb)):
        xh = orc.restore(eb, norms, dt, idx, xb[idx])
        rest = np.setdiff1d(np.arange(n), idx)
        # restored length equals the stored magnitude, which equals the input's length
        assert np.allclose(np.linalg.norm(xh[rest], axis=-1), norms[rest], rtol=1e-12)
        assert np.allclose(norms, np.linalg.norm(x, axis=-1), rtol=1e-14)
        # retained rows round-trip bit-exactly
        assert np.array_equal(orc.encode_bits(xh[idx], dt), xb[idx])
        assert np.array_equal(xh[idx], x[idx])
    # restored layer l sits (1-t)*Omega away from the original, layer l-1 t*Omega (up to storage rounding)
    tol = 2e-3 if dt == "f16" else 1.2e-2
    rest = np.setdiff1d(np.arange(n), idx)
    xl = orc.restore(eb, out["n_l"][0, :, 0], dt)
    xm = orc.restore(eb, out["n_lm1"][0, :, 0], dt)
    om = out["omega"][0, :, 0]
    assert np.allclose(angle(xl, c)[rest], 0.4 * om[rest], atol=tol)
    assert np.allclose(angle(xm, a)[rest], 0.6 * om[rest], atol=tol)


def test_restore_t1_reproduces_layer_l():
    n = 40
    ab, cb = _pair(n, "f16")
    out = orc.merge_pair(ab[None, :, None, :], cb[None, :, None, :], [n], "f16", 1.0, 0.0)
    xl = orc.restore(out["e_bits"][0, :, 0], out["n_l"][0, :, 0], "f16")
    c = orc.decode_bits(cb, "f16")
    assert len(out["retained"][(0, 0)]) == 0
    assert np.max(np.abs(xl - c)) <= 1.1 * 2.0 ** -11 * np.max(np.abs(c)) * 2


def test_restore_handles_zero_row():
    n = 8
    ab, cb = _pair(n, "f16")
    cb[3] = 0
    out = orc.merge_pair(ab[None, :, None, :], cb[None, :, None, :], [n], "f16", 0.6, 0.0)
    xl = orc.restore(out["e_bits"][0, :, 0], out["n_l"][0, :, 0], "f16")
    assert np.all(xl[3] == 0) and np.all(np.isfinite(xl))


# ---------------------------------------------------------------- attention (Algorithm 2, decoding)
def _brute_attention(q, K, V, scale):
    s = [scale * sum(q[j] * K[i][j] for j in range(len(q))) for i in range(len(K))]
    m = max(s)
    p = [math.exp(x - m) for x in s]
    z = sum(p)
    return [sum(p[i] * V[i][j] for i in range(len(K))) / z for j in range(len(V[0]))], m + math.log(z)


def test_attention_brute_force():
    n = 13
    q = rng.standard_normal(D)
    K = rng.standard_normal((n, D))
    V = rng.standard_normal((n, D))
    o, lse = orc.attention(q, K, V, 0.3)
    bo, blse = _brute_attention(list(q), K.tolist(), V.tolist(), 0.3)
    assert np.allclose(o, bo, atol=1e-13) and abs(lse - blse) < 1e-12
    # textbook softmax from an independent library
    ref = torch.softmax(torch.from_numpy(K @ q * 0.3), 0).numpy() @ V
    assert np.allclose(o, ref, atol=1e-13)
    # q = 0 -> plain mean of V; one dominant key -> that V row
    assert np.allclose(orc.attention(np.zeros(D), K, V, 1.0)[0], V.mean(0), atol=1e-13)
    K2 = K.copy()
    K2[5] = 50 * unit(q)
    assert np.allclose(orc.attention(unit(q) * 50, K2, V, 1.0)[0], V[5], atol=1e-9)


@pytest.mark.parametrize("dt", ["f16", "bf16"])
def test_compressed_attention_equals_restore_then_dense(dt):
    n = 70
    kab, kcb = _pair(n, dt)
    vab, vcb = _pair(n, dt)
    mk = orc.merge_pair(kab[None, :, None], kcb[None, :, None], [n], dt, 0.6, 0.3)
    mv = orc.merge_pair(vab[None, :, None], vcb[None, :, None], [n], dt, 0.6, 0.2)
    ik, iv = mk["retained"][(0, 0)], mv["retained"][(0, 0)]
    assert len(ik) and len(iv) and set(ik) != set(iv)
    q = orc.encode_bits(rng.standard_normal(D) * 3, dt)
    knew = orc.encode_bits(rng.standard_normal(D), dt)
    vnew = orc.encode_bits(rng.standard_normal(D), dt)
    for lname, kb, vb in (("n_lm1", kab, vab), ("n_l", kcb, vcb)):
        args = (q, mk["e_bits"][0, :, 0], mv["e_bits"][0, :, 0], mk[lname][0, :, 0], mv[lname][0, :, 0], dt, 0.09)
        kw = dict(idx_k=ik, rows_k_bits=kb[ik], idx_v=iv, rows_v_bits=vb[iv])
        for extra in ({}, dict(k_new_bits=knew, v_new_bits=vnew)):
            o1, l1 = orc.decode_attention(*args, **kw, **extra)
            o2, l2 = orc.decode_attention_compressed(*args, **kw, **extra)
            assert np.allclose(o1, o2, atol=1e-12) and abs(l1 - l2) < 1e-12
        # brute force on the dense restored cache
        kh = orc.restore(args[1], args[3], dt, ik, kb[ik])
        vh = orc.restore(args[2], args[4], dt, iv, vb[iv])
        bo, _ = _brute_attention(list(orc.decode_bits(q, dt)), kh.tolist(), vh.tolist(), 0.09)
        assert np.allclose(orc.decode_attention(*args, **kw)[0], bo, atol=1e-12)


def test_split_invariance():
    n = 101
    q = rng.standard_normal(D)
    K = rng.standard_normal((n, D))
    V = rng.standard_normal((n, D))
    whole = orc.attention(q, K, V, 0.2)
    cuts = [0, 7, 8, 50, 101]
    parts = [orc.attention(q, K[a:b], V[a:b], 0.2) for a, b in zip(cuts[:-1], cuts[1:])]
    o, lse = orc.lse_combine(parts)
    assert np.allclose(o, whole[0], atol=1e-12) and abs(lse - whole[1]) < 1e-12


def test_append_rows_matches_merge_rows():
    ab, cb = _pair(3, "f16")
    m = orc.append_rows(ab, cb, "f16", 0.6)
    ref = orc.merge_pair(ab[None, :, None], cb[None, :, None], [3], "f16", 0.6, 0.5, do_retention=False)
    assert np.array_equal(m["e_bits"], ref["e_bits"][0, :, 0])
    assert all(len(v) == 0 for v in ref["retained"].values())


# ---------------------------------------------------------------- footprint (Sec. 4.3)
def test_footprint_near_paper_formula():
    th = 8 * 4096 * 32
    full = orc.footprint_bytes(32, 16, th, 128, 0)
    assert full["full"] == 4 * 8 * 32 * (32 * 128) * 4096  # 4 b r h (s+n), Sec. 4.3
    # merging the upper half pairwise alone: 3/4 of the full cache plus the scalars
    assert abs(full["ratio"] - (0.75 + 0.25 * 12 / 256)) < 1e-12
    kept = int(0.05 * th * 2 * 8)
    r = orc.footprint_bytes(32, 16, th, 128, kept)["ratio"]
    assert abs(r - 3.1 / 4) < 0.02  # (3.1 h + 2) / 4h of Sec. 4.3, within the slack of its derivation


# ---------------------------------------------------------------- 4-bit storage (Sec. 5, KIVI scheme)
def test_q4_roundtrip_error_bound_and_codes():
    x = rng.standard_normal((3, 64, 128)) * np.exp(rng.standard_normal((3, 64, 1)))
    for axis in (1, 2):  # per-channel groups run along tokens (axis 1), per-token groups along channels (axis 2)
        codes, scale, zero = orc.q4_quantise(x, axis)
        assert codes.dtype == np.uint8 and codes.min() >= 0 and codes.max() <= 15
        assert scale.shape[axis] == x.shape[axis] // 32
        y = orc.q4_dequantise(codes, scale, zero, axis)
        s_full = np.repeat(scale, 32, axis=axis)
        rng_full = 15.0 * s_full
        # half a step, plus what the binary16 rounding of scale (15 steps) and zero can add
        assert np.all(np.abs(y - x) <= 0.5 * s_full + rng_full * 2.0 ** -10 + 1e-12)
        # scale and zero are binary16 values
        assert np.array_equal(orc.decode_bits(orc.encode_bits(scale, "f16"), "f16"), scale)
        assert np.array_equal(orc.decode_bits(orc.encode_bits(zero, "f16"), "f16"), zero)
        # both ends of every group are hit (codes 0 and 15 occur) unless the group is constant
        c = np.moveaxis(codes, axis, -1).reshape(-1, 32)
        assert np.all(c.min(-1) == 0) and np.all(c.max(-1) >= 14)


def test_q4_constant_group_and_brute_force():
    x = np.full((1, 32, 4), 0.375)
    codes, scale, zero = orc.q4_quantise(x, 1)
    assert np.all(codes == 0) and np.all(scale == 1.0) and np.all(zero == 0.375)
    assert np.array_equal(orc.q4_dequantise(codes, scale, zero, 1), x)
    # pure-Python restatement on one group
    g = [float(v) for v in rng.standard_normal(32)]
    lo, hi = min(g), max(g)
    s = float(np.float16((hi - lo) / 15.0))
    z = float(np.float16(lo))
    want = [min(15, max(0, int(np.rint((v - z) / s)))) for v in g]
    codes, scale, zero = orc.q4_quantise(np.array(g)[None, :], 1)
    assert list(codes[0]) == want and scale[0, 0] == s and zero[0, 0] == z
    assert np.allclose(orc.q4_dequantise(codes, scale, zero, 1)[0], [c * s + z for c in want], atol=0)


def test_input_quantiser_matches_oracle_quantiser():
    """The seeded input generator's 4-bit quantiser (data preparation) and the oracle's produce the
    same codes, scales and zeros: the device is fed what the oracle de-quantises."""
    import torch
    from gen import workload as W
    g = torch.Generator().manual_seed(3)
    x = (torch.randn(2, 64, 3, 128, generator=g) * 2).to(torch.float16)
    xv = x.double().numpy()
    for kind, axis in (("k", 1), ("v", 3)):
        q = W.quantise_q4(x, kind)
        codes, scale, zero = orc.q4_quantise(xv, axis)
        cn = q["codes"].numpy()
        full = np.empty(xv.shape, np.uint8)
        full[..., 0::2], full[..., 1::2] = cn & 15, cn >> 4
        assert np.array_equal(full, codes)
        m = q["meta"].double().numpy()
        assert np.array_equal(m[..., 0], scale) and np.array_equal(m[..., 1], zero)


def test_merge_function_variants_closed_forms():
    """F_max (Appendix Eq. A) and the averaging baseline (Sec. 3.1) inside merge_pair: one vector M for
    both layers, stored as direction and magnitude.  Closed forms for two rows of equal length r at an
    angle w: mean = r cos(w/2) along the bisector, F_max = r along the bisector; and for parallel rows of
    lengths 1 and 3: mean = 2, F_max = 3.  The distance (retention) does not depend on the merge function."""
    D = 128
    rs = np.random.RandomState(11)
    g1 = rs.standard_normal(D); g1 /= np.linalg.norm(g1)
    g2 = rs.standard_normal(D); g2 -= g1 * (g1 @ g2); g2 /= np.linalg.norm(g2)
    w, r = 0.8, 2.5
    a = r * g1
    c = r * (math.cos(w) * g1 + math.sin(w) * g2)
    bis = (g1 + math.cos(w) * g1 + math.sin(w) * g2); bis /= np.linalg.norm(bis)
    A = np.stack([a, g1])[None, :, None, :]        # [B=1][S=2][H=1][D]
    Cc = np.stack([c, 3.0 * g1])[None, :, None, :]
    ref = orc.merge_pair_values(A, Cc, [2], "f16", 0.6, 0.05)
    for fn, n0, n1 in (("mean", r * math.cos(w / 2), 2.0), ("fmax", r, 3.0)):
        m = orc.merge_pair_values(A, Cc, [2], "f16", 0.6, 0.05, merge_fn=fn)
        assert np.allclose(m["e"][0, 0, 0], bis, atol=1e-12) and np.allclose(m["e"][0, 1, 0], g1, atol=1e-12)
        assert np.allclose(m["n_lm1"][0, :, 0], [n0, n1], atol=1e-12) and np.array_equal(m["n_lm1"], m["n_l"])
        assert np.array_equal(m["d"], ref["d"]) and np.allclose(m["d"][0, 0, 0], w / math.pi, atol=1e-12)
        # restore gives M itself for both layers (up to the 16-bit storage of the direction)
        x = orc.restore(m["e_bits"][0, :, 0], m["n_l"][0, :, 0], "f16")
        assert np.allclose(x[0], n0 * bis, atol=2e-3 * n0) and np.allclose(x[1], n1 * g1, atol=2e-3 * n1)
    # SLERP keeps both magnitudes, the variants one
    assert not np.array_equal(ref["n_lm1"], ref["n_l"])
    # antipodal rows: the mean vanishes, nothing to restore
    z = orc.merge_pair_values(a[None, None, None, :], -a[None, None, None, :], [1], "f16", 0.6, 0.05, merge_fn="fmax")
    assert np.all(z["e"] == 0) and np.all(z["n_l"] == 0)


def test_restore_error_of_the_merge_functions_on_the_synthetic_pair():
    """The paper's comparison axis (Sec. 3.1, Appendix): how far the restored rows are from the original
    ones for SLERP, F_max and the plain average, on the generator's row model (independent magnitudes,
    planted angles), without retention.  Keeping both magnitudes and splitting the angle must beat one
    shared vector."""
    import dataclasses
    from gen import workload as W
    wl = dataclasses.replace(W.CONFIGS["c1"], seq_len=128, n_kv_heads=4, n_q_heads=4)
    t = W.make_pair_tensors(wl, 0)
    a, c = orc.decode_bits(W.as_bits(t["k_lm1"]), "f16"), orc.decode_bits(W.as_bits(t["k_l"]), "f16")
    err = {}
    for fn in ("slerp", "fmax", "mean"):
        m = orc.merge_pair_values(a, c, [128], "f16", 0.6, 0.0, merge_fn=fn)
        tot = []
        for layer, (x, nm) in enumerate(((a, "n_lm1"), (c, "n_l"))):
            for h in range(4):
                xh = orc.restore(m["e_bits"][0, :, h], m[nm][0, :, h], "f16")
                tot.append(np.linalg.norm(xh - x[0, :, h], axis=-1) / np.linalg.norm(x[0, :, h], axis=-1))
        err[fn] = float(np.mean(tot))
    print("mean relative restore error:", err)
    assert err["slerp"] < err["fmax"] and err["slerp"] < err["mean"]
    assert err["slerp"] < 0.25  # about half the mean planted angle (0.3 rad) plus outliers


# --------------------------------------------------------------------------
# 4-bit shared cache (Sec. 5: MiniCache on top of 4-bit KIVI)
# --------------------------------------------------------------------------
@pytest.mark.parametrize("dt", ["f16", "bf16"])
def test_q4_cache_constant_groups_survive_exactly(dt):
    """Closed form: a group whose members are all equal has scale 1, code 0 and zero = the value, so the
    stored direction is the input, bit for bit.  Keys: the same direction in all 32 tokens of a page (every
    channel group is constant).  Values: a row that is constant inside each 32-channel group."""
    rs = np.random.RandomState(3)
    row = rs.standard_normal(128)
    row /= np.linalg.norm(row)
    same = np.tile(orc.encode_bits(row, dt)[None, :], (64, 1))
    r = orc.q4_cache_quantise(same, 64, "k", dt)
    assert np.array_equal(r["e_bits"], same) and np.all(r["codes"] == 0) and np.all(r["scale"] == 1.0)
    steps = np.repeat(rs.standard_normal((64, 4)) * 0.1, 32, axis=1)  # constant per (token, 32-channel group)
    sb = orc.encode_bits(steps, dt)
    r = orc.q4_cache_quantise(sb, 64, "v", dt)
    assert np.array_equal(r["e_bits"], sb) and np.all(r["codes"] == 0)


@pytest.mark.parametrize("kind", ["k", "v"])
@pytest.mark.parametrize("dt", ["f16", "bf16"])
def test_q4_cache_error_bound_tail_and_brute_force(kind, dt):
    """Quantised tokens are within half a step (plus the 16-bit roundings) of the 16-bit direction, the
    extremes of a group get codes 0 and 15, the tokens of the incomplete last page are untouched, and a
    pure-Python loop over one group reproduces codes and stored values."""
    rs = np.random.RandomState(11)
    n, S = 77, 96  # two complete pages, 13 tokens in the residual, padding behind
    e = rs.standard_normal((S, 128))
    e /= np.linalg.norm(e, axis=1, keepdims=True)
    eb = orc.encode_bits(e, dt)
    r = orc.q4_cache_quantise(eb, n, kind, dt)
    assert r["n_q"] == 64 and r["codes"].shape == (64, 128) and r["codes"].max() == 15 and r["codes"].min() == 0
    assert np.array_equal(r["e_bits"][64:], eb[64:])  # residual and padding stay as they were
    x = orc.decode_bits(eb[:64], dt)
    y = orc.decode_bits(r["e_bits"][:64], dt)
    ulp = 2.0 ** -10 if dt == "f16" else 2.0 ** -7
    step = np.repeat(r["scale"], 32, axis=0 if kind == "k" else 1)
    # half a step, plus the rounding of zero (|zero| ulp / 2), of scale (15 |scale| ulp / 2) and of the result
    assert np.all(np.abs(y - x) <= 0.5 * step + ulp * (0.5 * 0.4 + 7.5 * step + 0.5 * np.abs(y)) + 1e-12)
    # brute force of one group
    if kind == "k":
        g = [float(v) for v in x[32:64, 5]]
        sc, ze = float(r["scale"][1, 5]), float(r["zero"][1, 5])
        got_codes, got_vals = r["codes"][32:64, 5], y[32:64, 5]
    else:
        g = [float(v) for v in x[40, 64:96]]
        sc, ze = float(r["scale"][40, 2]), float(r["zero"][40, 2])
        got_codes, got_vals = r["codes"][40, 64:96], y[40, 64:96]
    one = lambda v: float(orc.decode_bits(orc.encode_bits(np.array([v]), dt), dt)[0])
    lo, hi = min(g), max(g)
    assert ze == one(lo) and sc == one((hi - lo) / 15.0)
    for v, c, w in zip(g, got_codes, got_vals):
        q = min(15, max(0, round((v - ze) / sc)))  # Python's round is ties-to-even, like rint
        assert q == int(c) and w == one(q * sc + ze)
    assert got_codes.min() == 0 and got_codes.max() == 15  # the group's minimum and maximum


def test_q4_cache_restore_keeps_the_magnitudes():
    """Eq. 2 with the 4-bit cache: the restored row still has exactly the stored magnitude, because the
    division is by the length of the stored (de-quantised) direction; and the angle between the restored
    row and the 16-bit cache's restored row is small (a 4-bit step is 1/15 of the group's range)."""
    import gen
    cfg = gen.CONFIGS["c1"].scaled("q4c", n_kv_heads=2, n_q_heads=2, batch=1, seq_len=96, index=61)
    t = gen.make_pair_tensors(cfg, 0)
    lens = [80]
    for kind in ("k", "v"):
        m = orc.merge_pair(gen.as_bits(t[kind + "_lm1"]), gen.as_bits(t[kind + "_l"]), lens, "f16", 0.6, 0.05)
        mq = orc.q4_cache_pair(m, lens, kind, "f16")
        assert np.array_equal(mq["e_bits"][0, 64:80], m["e_bits"][0, 64:80])
        assert not np.array_equal(mq["e_bits"][0, :64], m["e_bits"][0, :64])
        for h in range(2):
            x16 = orc.restore(m["e_bits"][0, :80, h], m["n_l"][0, :80, h], "f16")
            x4 = orc.restore(mq["e_bits"][0, :80, h], m["n_l"][0, :80, h], "f16")
            assert np.allclose(np.linalg.norm(x4, axis=1), m["n_l"][0, :80, h], rtol=1e-12)
            cos = np.sum(x16 * x4, 1) / (np.linalg.norm(x16, axis=1) * np.linalg.norm(x4, axis=1))
            assert np.all(cos > 0.97) and np.all(cos[64:] > 1 - 1e-12)


# ---------------------------------------------------------------------------------------------
# Variants the paper points at: dynamic t (Sec. 5, ablation of t), one retention set for K and V
# ---------------------------------------------------------------------------------------------
def _angle(x, y):
    """Angle between two vectors by the atan2 formula (no arccos)."""
    x, y = x / np.linalg.norm(x), y / np.linalg.norm(y)
    return 2.0 * math.atan2(np.linalg.norm(x - y), np.linalg.norm(x + y))


def test_dynamic_t_is_the_relative_magnitude_ratio():
    assert orc.dynamic_t(1.0, 1.0) == 0.5
    assert orc.dynamic_t(1.0, 3.0) == 0.75 and orc.dynamic_t(3.0, 1.0) == 0.25
    assert orc.dynamic_t(0.0, 0.0) == 0.5 and orc.dynamic_t(0.0, 2.0) == 1.0
    rs = np.random.RandomState(3)
    na, nc = rs.rand(100) + 0.1, rs.rand(100) + 0.1
    t = orc.dynamic_t(na, nc)
    assert np.all((t > 0) & (t < 1)) and np.allclose(t + orc.dynamic_t(nc, na), 1.0)


def test_dynamic_t_splits_the_angle_by_the_magnitudes():
    """With t = |c| / (|a| + |c|) the merged direction sits at t * Omega from layer l-1's direction: three
    times closer to the row that is three times longer; equal lengths give the geodesic midpoint."""
    rs = np.random.RandomState(4)
    u = rs.randn(128)
    u /= np.linalg.norm(u)
    g = rs.randn(128)
    g -= (g @ u) * u
    g /= np.linalg.norm(g)
    for omega, la, lc in ((0.5, 1.0, 3.0), (1.3, 2.0, 2.0), (2.0, 5.0, 1.0)):
        a = la * u
        c = lc * (math.cos(omega) * u + math.sin(omega) * g)
        m = orc.merge_rows(a[None], c[None], "ratio")
        t = lc / (la + lc)
        assert abs(np.linalg.norm(m["e"][0]) - 1.0) < 1e-12
        assert abs(_angle(m["e"][0], a) - t * omega) < 1e-9 and abs(_angle(m["e"][0], c) - (1 - t) * omega) < 1e-9
        # the same number as Eq. 3 with that t given explicitly, and per-row arrays of t are honoured
        assert np.allclose(m["e"], orc.merge_rows(a[None], c[None], t)["e"], atol=1e-15)
    rows_a = np.stack([1.0 * u, 2.0 * u])
    rows_c = np.stack([3.0 * g, 2.0 * g])
    m = orc.merge_rows(rows_a, rows_c, "ratio")  # orthogonal rows: e = cos(t pi/2) u + sin(t pi/2) g
    for i, t in enumerate((0.75, 0.5)):
        assert np.allclose(m["e"][i], math.cos(t * math.pi / 2) * u + math.sin(t * math.pi / 2) * g, atol=1e-12)
    # a fixed t is unchanged by the array handling
    assert np.array_equal(orc.merge_rows(rows_a, rows_c, 0.6)["e"], orc.merge_rows(rows_a, rows_c, np.array([0.6, 0.6]))["e"])


def test_dynamic_t_through_the_pair_merge_and_restore():
    import gen
    wl = gen.CONFIGS["c1"].scaled("dyn", n_kv_heads=2, n_q_heads=2, batch=1, seq_len=40, index=61)
    t = gen.make_pair_tensors(wl, 0)
    bits = {k: gen.as_bits(v) for k, v in t.items()}
    m = orc.merge_pair(bits["k_lm1"], bits["k_l"], [40], "f16", "ratio", 0.05)
    a, c = orc.decode_bits(bits["k_lm1"], "f16"), orc.decode_bits(bits["k_l"], "f16")
    tt = m["n_l"] / (m["n_lm1"] + m["n_l"])
    for i in (0, 7, 39):
        for h in (0, 1):
            om = _angle(a[0, i, h], c[0, i, h])
            assert abs(_angle(m["e"][0, i, h], a[0, i, h]) - tt[0, i, h] * om) < 1e-9
    # restore keeps both magnitudes whatever t was
    x = orc.restore(m["e_bits"][0, :, 0], m["n_l"][0, :, 0], "f16")
    assert np.allclose(np.linalg.norm(x, axis=-1), m["n_l"][0, :, 0], rtol=1e-12)


def test_retention_union_brute_force():
    rs = np.random.RandomState(9)
    dk, dv = rs.rand(3, 50), rs.rand(3, 50)
    rk = {(b, 0): orc.retention_indices(dk[b], 0.2) for b in range(3)}
    rv = {(b, 0): orc.retention_indices(dv[b], 0.2) for b in range(3)}
    un = orc.retention_union(rk, rv)
    for b in range(3):
        want = sorted(i for i in range(50) if i in set(rk[(b, 0)].tolist()) or i in set(rv[(b, 0)].tolist()))
        assert un[(b, 0)].tolist() == want
        assert set(rk[(b, 0)].tolist()) <= set(want) and set(rv[(b, 0)].tolist()) <= set(want)
    # nothing kept for the values: the union is the keys' set; same sets: unchanged
    empty = {k: np.zeros(0, np.int64) for k in rk}
    assert all(np.array_equal(orc.retention_union(rk, empty)[k], rk[k]) for k in rk)
    assert all(np.array_equal(orc.retention_union(rk, rk)[k], rk[k]) for k in rk)


def test_append_keep_hand_values_and_prefill_consistency():
    """The decode-time retention decision: hand-applied Eq. 4 on dyadic distances (the prefill extremes are
    0.125 and 0.875, gamma = 0.25: thresholds 0.6875 for the similarity reading and 0.3125 for the literal
    one), and a brute-force link to the prefill rule: a new token with the distance of prefill token i is
    kept exactly when i was."""
    d = np.array([0.125, 0.5, 0.875, 0.25, 0.75])
    assert orc.append_keep(0.75, d, 0.25, "distinct") and not orc.append_keep(0.6875, d, 0.25, "distinct")
    assert not orc.append_keep(0.5, d, 0.25, "distinct")
    assert orc.append_keep(0.25, d, 0.25, "literal") and not orc.append_keep(0.3125, d, 0.25, "literal")
    assert not orc.append_keep(0.5, d, 0.25, "literal")
    # beyond the prefill extremes: the stored threshold still decides, the extremes do not move
    assert orc.append_keep(0.99, d, 0.25, "distinct") and orc.append_keep(0.01, d, 0.25, "literal")
    # nothing is kept with gamma = 0, without prefill tokens, or under the top-k reading
    assert not orc.append_keep(0.99, d, 0.0, "distinct") and not orc.append_keep(0.01, d, 0.0, "literal")
    assert not orc.append_keep(0.99, np.zeros(0), 0.25, "distinct")
    assert not orc.append_keep(0.99, d, 0.25, "topk")
    rs = np.random.RandomState(77)
    for mode in ("distinct", "literal"):
        dd = rs.rand(200)
        kept = set(orc.retention_indices(dd, 0.2, mode).tolist())
        for i in range(200):
            assert orc.append_keep(dd[i], dd, 0.2, mode) == (i in kept)

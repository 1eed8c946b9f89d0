"""fp64 CPU oracle for the MiniCache hot path.  TEST INFRASTRUCTURE ONLY.

This file is the yardstick the CUDA kernels are measured against.  It is a
plain, slow, step-by-step numpy restatement of the method in double precision
and shares no code, table or helper with the CUDA path.  Only the tests, the
smoke check and the CPU-baseline leg of the benchmark may import it; the
product never does.

What each function follows (MiniCache, arXiv 2405.14366):

* ``merge_rows``            Eq. 3 (SLERP of unit directions), the angle defined
                            right below Eq. 3, the distance d = Omega / pi of
                            Sec. 4.2 "Unmergeable token retention", Algorithm 2
                            "MiniCache Merge".
* ``store_direction``       Sec. 4.3: the cache is stored in 16-bit floats.
* ``retention_indices``     Eq. 4 / Algorithm 2 "MiniCache Prefill".
* ``merge_pair``            Algorithm 2 "MiniCache Prefill" for one layer pair.
* ``restore``               Eq. 2 and Sec. 4.2 "Cache restoration";
                            Algorithm 2 "MiniCache Decoding" (rescale, then
                            put the retained rows back).
* ``attention`` / ``decode_attention`` / ``decode_attention_compressed``
                            Algorithm 2 "MiniCache Decoding": concatenate the
                            new token, softmax(q K^T) V.
* ``append_rows``           Algorithm 2 "MiniCache Decoding", the branch that
                            merges the new token pair and appends it.
* ``merge_rows_fmax`` / ``merge_rows_mean``
                            Eq. A (Sec. "Alternative merging function") and the
                            averaging baseline of Sec. 3.1.
* ``dynamic_t``             Sec. 5, ablation of t: the interpolation parameter taken per
                            token from the relative magnitude ratio of the two layers.
* ``retention_union``       Sec. 4.2 writes ONE index set I for the pair cache while
                            Algorithm 2 computes one per tensor: the reading with one
                            set, the union of the keys' and the values' sets.

Readings taken where the paper is silent or inconsistent (each is a keyword
argument so the other reading can be run):

* ``convention="eq3"``: t weights layer l (t = 0 gives the direction of layer
  l-1, t = 1 that of layer l), as Eq. 3 prints it and as the prose around the
  default t = 0.6 says ("smaller rotation angle to the next layer").
  ``"alg2"`` swaps the two coefficients, as Algorithm 2's Merge prints them.
* ``mode="distinct"``: keep tokens with d > d_max - (d_max - d_min) * gamma,
  i.e. Eq. 4 applied to angular similarity 1 - d, which is what every sentence
  around Eq. 4 describes (the most distinct pairs are kept).  ``"literal"`` is
  Eq. 4 exactly as printed; ``"topk"`` keeps the ceil(gamma * n) largest d.
* one vector = one (token, kv head) row of 128 channels; d_min / d_max are
  taken per (tensor, sequence, kv head) over that sequence's tokens.
* sin(Omega) -> 0: same direction  -> normalised linear interpolation (the
  limit of Eq. 3); opposite direction -> layer l's direction if t >= 0.5 else
  layer l-1's.  A zero row has angle 0 and contributes no direction.
* restore divides by the length of the *stored* (16-bit rounded) direction,
  exactly as Eq. 2 is written.
* ``t="ratio"`` (not the default): the paper observes that the best t follows the
  relative magnitude ratio of adjacent layers, whose histogram clusters at 0.4 and
  0.6 (the same scale as t), and suggests taking t from it; it gives no formula.
  Reading: per token t_i = |x^l_i| / (|x^{l-1}_i| + |x^l_i|), so the layer with the
  larger magnitude pulls the direction its way and equal magnitudes give the
  geodesic midpoint; 0.5 if both rows are zero.

Parity unpinned: none of the functions here.  What stays unpinned is outside
this file: whether merging preserves a real model's accuracy needs trained
weights and datasets and is not claimed anywhere.
"""
from __future__ import annotations

import math
from typing import Dict, List, Optional, Sequence

import numpy as np

F64 = np.float64
# arccos of a rounded cosine is only good to about 1e-8 rad next to 0 and pi;
# below this value of sin(Omega) the limit forms of Eq. 3 are used instead.
SIN_GUARD = 1e-6


# --------------------------------------------------------------------------
# 16-bit storage formats (bit patterns <-> exact doubles)
# --------------------------------------------------------------------------
def decode_bits(bits: np.ndarray, dtype: str) -> np.ndarray:
    """uint16 bit patterns of IEEE binary16 ("f16") or bfloat16 ("bf16") -> exact float64."""
    bits = np.ascontiguousarray(bits, dtype=np.uint16)
    if dtype == "f16":
        return bits.view(np.float16).astype(F64)
    if dtype == "bf16":
        with np.errstate(invalid="ignore"):
            return (bits.astype(np.uint32) << np.uint32(16)).view(np.float32).astype(F64)
    raise ValueError(dtype)


def encode_bits(x: np.ndarray, dtype: str) -> np.ndarray:
    """Round float64 to the nearest 16-bit float (ties to even), once, and return its bits."""
    x = np.asarray(x, dtype=F64)
    if dtype == "f16":
        with np.errstate(over="ignore"):
            return x.astype(np.float16).view(np.uint16)
    if dtype == "bf16":
        # bfloat16 = 8 significant bits, binary32 exponent range.  Round on the
        # bfloat16 grid directly from the double (no intermediate binary32 step).
        _, ex = np.frexp(x)  # |x| in [2^(ex-1), 2^ex)
        ex = np.maximum(ex - 1, -126)  # subnormal grid below 2^-126
        quantum = np.ldexp(1.0, ex - 7)
        r = np.rint(x / quantum) * quantum  # exact scaling by a power of two; rint = ties to even
        r = np.where(np.isfinite(x), r, x)
        r32 = r.astype(np.float32)  # exact: r is on the bfloat16 grid
        return (r32.view(np.uint32) >> np.uint32(16)).astype(np.uint16)
    raise ValueError(dtype)


# --------------------------------------------------------------------------
# Merge (Eq. 3), distance, alternative merge functions
# --------------------------------------------------------------------------
def dynamic_t(n_a: np.ndarray, n_c: np.ndarray) -> np.ndarray:
    """Per-token interpolation parameter from the relative magnitude ratio (Sec. 5, ablation of t):
    t = |x^l| / (|x^{l-1}| + |x^l|); 0.5 where both magnitudes are zero."""
    n_a = np.asarray(n_a, F64)
    n_c = np.asarray(n_c, F64)
    tot = n_a + n_c
    return np.where(tot > 0.0, n_c / np.where(tot > 0.0, tot, 1.0), 0.5)


def merge_rows(a: np.ndarray, c: np.ndarray, t, convention: str = "eq3") -> Dict[str, np.ndarray]:
    """SLERP-merge rows a (layer l-1) and c (layer l); both [..., D] float64.
    t: the interpolation parameter of Eq. 3, a number, an array with one value per row, or
    "ratio" (``dynamic_t`` of the two magnitudes).

    Returns e (unit direction, float64, not yet rounded for storage), n_a, n_c
    (the two magnitudes), omega (angle in [0, pi]) and d = omega / pi."""
    a = np.asarray(a, F64)
    c = np.asarray(c, F64)
    n_a = np.sqrt(np.sum(a * a, axis=-1))
    n_c = np.sqrt(np.sum(c * c, axis=-1))
    if isinstance(t, str):
        if t != "ratio":
            raise ValueError(t)
        t = dynamic_t(n_a, n_c)
    t = np.asarray(t, F64)
    za = n_a == 0.0
    zc = n_c == 0.0
    u = a / np.where(za, 1.0, n_a)[..., None]
    v = c / np.where(zc, 1.0, n_c)[..., None]
    cosw = np.clip(np.sum(u * v, axis=-1), -1.0, 1.0)
    omega = np.arccos(cosw)
    omega = np.where(za | zc, 0.0, omega)
    sinw = np.sin(omega)
    if convention == "eq3":
        ta, tc = 1.0 - t, t
    elif convention == "alg2":
        ta, tc = t, 1.0 - t
    else:
        raise ValueError(convention)
    ta, tc = np.broadcast_to(ta, omega.shape), np.broadcast_to(tc, omega.shape)
    safe = np.where(sinw < SIN_GUARD, 1.0, sinw)
    w_a = np.sin(ta * omega) / safe
    w_c = np.sin(tc * omega) / safe
    e = w_a[..., None] * u + w_c[..., None] * v
    # sin(Omega) -> 0 with the same direction: limit of Eq. 3, renormalised.
    same = (sinw < SIN_GUARD) & (cosw > 0.0) & ~(za | zc)
    if np.any(same):
        lin = ta[..., None] * u + tc[..., None] * v
        len_lin = np.sqrt(np.sum(lin * lin, axis=-1))
        lin = lin / np.where(same, len_lin, 1.0)[..., None]
        e = np.where(same[..., None], lin, e)
    # opposite directions: Eq. 3 is undefined; take the endpoint t is closer to.
    opp = (sinw < SIN_GUARD) & (cosw <= 0.0) & ~(za | zc)
    if np.any(opp):
        pick = np.where((tc >= 0.5)[..., None], v, u)
        e = np.where(opp[..., None], pick, e)
    # zero rows carry no direction: use the other row's (zero vector if both).
    e = np.where((za & ~zc)[..., None], v, e)
    e = np.where((zc & ~za)[..., None], u, e)
    e = np.where((za & zc)[..., None], 0.0, e)
    return {"e": e, "n_a": n_a, "n_c": n_c, "omega": omega, "d": omega / math.pi}


def merge_rows_fmax(a: np.ndarray, c: np.ndarray) -> np.ndarray:
    """Maximum-norm-preserving interpolation, Eq. A: mean direction x max magnitude."""
    a = np.asarray(a, F64)
    c = np.asarray(c, F64)
    mean = 0.5 * (a + c)
    nm = np.sqrt(np.sum(mean * mean, axis=-1))
    big = np.maximum(np.sqrt(np.sum(a * a, -1)), np.sqrt(np.sum(c * c, -1)))
    return mean / np.where(nm == 0.0, 1.0, nm)[..., None] * big[..., None]


def merge_rows_mean(a: np.ndarray, c: np.ndarray) -> np.ndarray:
    """The averaging baseline of Sec. 3.1: plain mean of the two rows."""
    return 0.5 * (np.asarray(a, F64) + np.asarray(c, F64))


def store_direction(e: np.ndarray, dtype: str) -> np.ndarray:
    """Round the merged direction to the cache's 16-bit storage format (bits)."""
    return encode_bits(e, dtype)


# --------------------------------------------------------------------------
# Retention (Eq. 4)
# --------------------------------------------------------------------------
def retention_threshold(d: np.ndarray, gamma: float, mode: str = "distinct") -> float:
    d = np.asarray(d, F64)
    dmin, dmax = float(np.min(d)), float(np.max(d))
    if mode == "distinct":
        return dmax - (dmax - dmin) * gamma
    if mode == "literal":
        return dmin + (dmax - dmin) * gamma
    raise ValueError(mode)


def retention_indices(d: np.ndarray, gamma: float, mode: str = "distinct") -> np.ndarray:
    """Ascending token indices kept unmerged for one segment's distances d [n]."""
    d = np.asarray(d, F64)
    n = d.shape[0]
    if n == 0:
        return np.zeros(0, np.int64)
    if mode == "distinct":
        return np.nonzero(d > retention_threshold(d, gamma, mode))[0].astype(np.int64)
    if mode == "literal":
        return np.nonzero(d < retention_threshold(d, gamma, mode))[0].astype(np.int64)
    if mode == "topk":
        k = min(n, int(math.ceil(gamma * n - 1e-12)))
        order = np.lexsort((np.arange(n), -d))  # largest d first, ties -> lower index
        return np.sort(order[:k]).astype(np.int64)
    raise ValueError(mode)


def append_keep(d_new: float, d_prefill: np.ndarray, gamma: float, mode: str = "distinct") -> bool:
    """Is a token appended during decode kept unmerged?  An extension of Eq. 4 (Algorithm 2 decides only over
    the prefill tokens): the new token's distance is held against the threshold of its segment's PREFILL
    distances -- d_min and d_max stay what they were when the pair was merged.  gamma = 0 keeps nothing, an
    empty prefill segment has no threshold, and the top-k reading has none either."""
    d_prefill = np.asarray(d_prefill, F64)
    if not gamma > 0.0 or d_prefill.shape[0] == 0 or mode == "topk":
        return False
    thr = retention_threshold(d_prefill, gamma, mode)
    return bool(d_new > thr) if mode == "distinct" else bool(d_new < thr)


# --------------------------------------------------------------------------
# One layer pair (Algorithm 2, "MiniCache Prefill")
# --------------------------------------------------------------------------
def retention_union(retained_k: Dict, retained_v: Dict) -> Dict:
    """One index set per (sequence, kv head) for keys and values alike -- Sec. 4.2 writes the pair cache with
    a single I, Algorithm 2 computes one per tensor --: a token either tensor's rule (Eq. 4) keeps is kept
    unmerged in both."""
    return {key: np.union1d(retained_k[key], retained_v[key]).astype(np.int64) for key in retained_k}


def merge_pair(x_lm1_bits: np.ndarray, x_l_bits: np.ndarray, seq_lens: Sequence[int], dtype: str,
               t, gamma: float, mode: str = "distinct", convention: str = "eq3",
               do_retention: bool = True, merge_fn: str = "slerp") -> Dict[str, object]:
    """Compress one tensor (K or V) of a layer pair.

    x_*_bits: uint16 [B][S][H][D] logical rows (layer l-1, layer l).
    Returns e_bits [B][S][H][D], e (float64, before storage rounding), n_lm1,
    n_l, d [B][S][H] (float64), ``retained``: dict (b, h) -> ascending indices.
    The retained raw rows are the input bits at those indices."""
    return merge_pair_values(decode_bits(x_lm1_bits, dtype), decode_bits(x_l_bits, dtype), seq_lens, dtype, t, gamma,
                             mode, convention, do_retention, merge_fn)


def merge_pair_values(a: np.ndarray, c: np.ndarray, seq_lens: Sequence[int], dtype: str, t, gamma: float,
                      mode: str = "distinct", convention: str = "eq3", do_retention: bool = True,
                      merge_fn: str = "slerp") -> Dict[str, object]:
    """``merge_pair`` on rows given as float64 values (e.g. de-quantised 4-bit layers); `dtype` is
    the storage type of the merged direction.

    merge_fn "slerp" is Eq. 3 with both magnitudes kept.  "fmax" (Eq. A) and "mean" (the averaging
    baseline of Sec. 3.1) merge the two rows into ONE vector M that stands for both layers: the
    stored direction is M / |M| and both layers' magnitudes are |M|.  The angular distance that
    drives the retention (Eq. 4) is the same in all three."""
    m = merge_rows(a, c, t, convention)
    if merge_fn != "slerp":
        M = {"fmax": merge_rows_fmax, "mean": merge_rows_mean}[merge_fn](a, c)
        n_m = np.sqrt(np.sum(M * M, axis=-1))
        m["e"] = M / np.where(n_m == 0.0, 1.0, n_m)[..., None]
        m["n_a"] = n_m
        m["n_c"] = n_m
    e_bits = store_direction(m["e"], dtype)
    B, S, H, _ = a.shape
    retained = {}
    for b in range(B):
        n = int(seq_lens[b])
        for h in range(H):
            if do_retention and n > 0:
                retained[(b, h)] = retention_indices(m["d"][b, :n, h], gamma, mode)
            else:
                retained[(b, h)] = np.zeros(0, np.int64)
    return {"e_bits": e_bits, "e": m["e"], "n_lm1": m["n_a"], "n_l": m["n_c"], "d": m["d"],
            "omega": m["omega"], "retained": retained}


def append_rows(a_bits: np.ndarray, c_bits: np.ndarray, dtype: str, t,
                convention: str = "eq3", merge_fn: str = "slerp") -> Dict[str, np.ndarray]:
    """Merge the decode step's new token pair (no retention decision for it)."""
    a, c = decode_bits(a_bits, dtype), decode_bits(c_bits, dtype)
    m = merge_rows(a, c, t, convention)
    if merge_fn != "slerp":  # see merge_pair_values
        M = {"fmax": merge_rows_fmax, "mean": merge_rows_mean}[merge_fn](a, c)
        n_m = np.sqrt(np.sum(M * M, axis=-1))
        m["e"] = M / np.where(n_m == 0.0, 1.0, n_m)[..., None]
        m["n_a"] = n_m
        m["n_c"] = n_m
    m["e_bits"] = store_direction(m["e"], dtype)
    return m


# --------------------------------------------------------------------------
# Restore (Eq. 2) and attention (Algorithm 2, "MiniCache Decoding")
# --------------------------------------------------------------------------
def restore(e_bits: np.ndarray, norms: np.ndarray, dtype: str,
            retained_idx: Optional[np.ndarray] = None,
            retained_rows_bits: Optional[np.ndarray] = None) -> np.ndarray:
    """Restore one layer's rows of one segment.

    e_bits [n][D] stored directions, norms [n] that layer's magnitudes,
    retained_idx [r] with retained_rows_bits [r][D] that layer's raw rows.
    Returns float64 [n][D]: e * (norm / ||e||), retained rows put back."""
    e = decode_bits(e_bits, dtype)
    len_e = np.sqrt(np.sum(e * e, axis=-1))
    scale = np.asarray(norms, F64) / np.where(len_e == 0.0, 1.0, len_e)
    x = e * scale[..., None]
    if retained_idx is not None and len(retained_idx):
        x[np.asarray(retained_idx)] = decode_bits(retained_rows_bits, dtype)
    return x


def attention(q: np.ndarray, k: np.ndarray, v: np.ndarray, sm_scale: float):
    """Single-query softmax attention: q [D], k [n][D], v [n][D] -> (o [D], lse)."""
    s = (k @ q) * sm_scale
    m = np.max(s)
    p = np.exp(s - m)
    z = np.sum(p)
    return (p @ v) / z, m + math.log(z)


def decode_attention(q_bits: np.ndarray, e_k_bits: np.ndarray, e_v_bits: np.ndarray,
                     n_k: np.ndarray, n_v: np.ndarray, dtype: str, sm_scale: float,
                     idx_k=None, rows_k_bits=None, idx_v=None, rows_v_bits=None,
                     k_new_bits=None, v_new_bits=None):
    """One (sequence, q head) of decode attention for one layer of a pair:
    restore K and V densely, append the new token, then plain attention."""
    k_hat = restore(e_k_bits, n_k, dtype, idx_k, rows_k_bits)
    v_hat = restore(e_v_bits, n_v, dtype, idx_v, rows_v_bits)
    if k_new_bits is not None:
        k_hat = np.concatenate([k_hat, decode_bits(k_new_bits, dtype).reshape(1, -1)], axis=0)
        v_hat = np.concatenate([v_hat, decode_bits(v_new_bits, dtype).reshape(1, -1)], axis=0)
    return attention(decode_bits(q_bits, dtype), k_hat, v_hat, sm_scale)


def decode_attention_compressed(q_bits, e_k_bits, e_v_bits, n_k, n_v, dtype, sm_scale,
                                idx_k=None, rows_k_bits=None, idx_v=None, rows_v_bits=None,
                                k_new_bits=None, v_new_bits=None):
    """Same result as ``decode_attention`` computed without materialising the
    restored cache: the magnitude is applied to the score (K) and to the
    probability (V), and retained rows replace single terms.  Kept as a second
    code path so the two can be checked against each other."""
    q = decode_bits(q_bits, dtype)
    ek = decode_bits(e_k_bits, dtype)
    ev = decode_bits(e_v_bits, dtype)
    gk = np.asarray(n_k, F64) / np.sqrt(np.sum(ek * ek, -1))
    gv = np.asarray(n_v, F64) / np.sqrt(np.sum(ev * ev, -1))
    s = gk * (ek @ q)
    if idx_k is not None and len(idx_k):
        s[np.asarray(idx_k)] = decode_bits(rows_k_bits, dtype) @ q
    s_new = None
    if k_new_bits is not None:
        s_new = float(decode_bits(k_new_bits, dtype).reshape(-1) @ q)
        s = np.concatenate([s, [s_new]])
    s = s * sm_scale
    m = np.max(s)
    p = np.exp(s - m)
    z = np.sum(p)
    n = ek.shape[0]
    coef = p[:n] * gv
    keep = np.ones(n, bool)
    o = np.zeros_like(q)
    if idx_v is not None and len(idx_v):
        keep[np.asarray(idx_v)] = False
        o += p[np.asarray(idx_v)] @ decode_bits(rows_v_bits, dtype)
    o += (coef * keep) @ ev
    if v_new_bits is not None:
        o += p[n] * decode_bits(v_new_bits, dtype).reshape(-1)
    return o / z, m + math.log(z)


def lse_combine(parts: List):
    """Combine partial attention results [(o_j, lse_j)] of disjoint token sets."""
    lses = np.array([p[1] for p in parts], F64)
    m = np.max(lses)
    w = np.exp(lses - m)
    o = sum(wj * p[0] for wj, p in zip(w, parts)) / np.sum(w)
    return o, m + math.log(np.sum(w))


# --------------------------------------------------------------------------
# 4-bit storage (Sec. 5: MiniCache on top of 4-bit KIVI quantisation)
# --------------------------------------------------------------------------
# The paper only names the scheme; the reading taken here is KIVI's asymmetric round-to-nearest
# quantisation with groups of 32: keys per channel (a group = 32 consecutive tokens of one
# channel), values per token (a group = 32 consecutive channels of one token):
#   scale = (max - min) / 15, zero = min, both stored in binary16;
#   code = clamp(rint((x - zero) / scale), 0, 15) with the *stored* scale and zero;
#   a constant group stores scale = 1 and code 0.
Q4_GROUP = 32


def q4_quantise(x: np.ndarray, axis: int, meta_dtype: str = "f16"):
    """Quantise float64 x along `axis` in groups of 32 (its length must be a multiple of 32).

    Returns (codes uint8, same shape; scale, zero: float64 values that are exactly representable in
    `meta_dtype` (binary16 unless stated), shape of x with `axis` divided by 32)."""
    x = np.moveaxis(np.asarray(x, F64), axis, -1)
    shp = x.shape
    assert shp[-1] % Q4_GROUP == 0
    g = x.reshape(shp[:-1] + (shp[-1] // Q4_GROUP, Q4_GROUP))
    lo, hi = g.min(-1), g.max(-1)
    scale = decode_bits(encode_bits((hi - lo) / 15.0, meta_dtype), meta_dtype)
    zero = decode_bits(encode_bits(lo, meta_dtype), meta_dtype)
    scale = np.where(scale == 0.0, 1.0, scale)
    codes = np.clip(np.rint((g - zero[..., None]) / scale[..., None]), 0, 15).astype(np.uint8)
    codes = np.moveaxis(codes.reshape(shp), -1, axis)
    return codes, np.moveaxis(scale, -1, axis), np.moveaxis(zero, -1, axis)


def q4_dequantise(codes: np.ndarray, scale: np.ndarray, zero: np.ndarray, axis: int) -> np.ndarray:
    """value = code * scale + zero, the group's scale and zero repeated over its 32 members."""
    c = np.moveaxis(np.asarray(codes, F64), axis, -1)
    s = np.repeat(np.moveaxis(np.asarray(scale, F64), axis, -1), Q4_GROUP, axis=-1)
    z = np.repeat(np.moveaxis(np.asarray(zero, F64), axis, -1), Q4_GROUP, axis=-1)
    return np.moveaxis(c * s + z, -1, axis)


def q4_cache_quantise(e_bits: np.ndarray, n: int, kind: str, dtype: str) -> Dict[str, np.ndarray]:
    """The shared directions of one (sequence, kv head) held in a 4-bit cache (Sec. 5: MiniCache
    "on top of 4-bit KIVI"; the paper states no more than that, the reading is the following).

    e_bits [S][D]: the merged directions already rounded to the 16-bit cache type (`store_direction`);
    n: cached tokens.  The quantiser is the KIVI scheme above applied to that 16-bit cache, in the
    cache's own page structure (pages of 32 tokens): keys (`kind` "k") per channel, a group = the 32
    tokens of a page; values ("v") per token, a group = 32 channels.  Only complete pages are
    quantised: the tokens [32 floor(n / 32), n) of the last, incomplete page stay in 16 bits (KIVI
    keeps such a full-precision residual until a group is complete).  Scale and zero are kept in the
    cache's 16-bit type, and a de-quantised element is code * scale + zero rounded ONCE to that
    type: the value a 16-bit tensor-core operand carries, and the stored direction e of Eq. 2.

    Returns codes [n_q][D] uint8, scale / zero (K: [n_q / 32][D], V: [n_q][D / 32]; float64 holding
    values of the 16-bit type), e_bits [S][D] (the stored directions: de-quantised ones for the
    first n_q = 32 floor(n / 32) tokens, the input bits for the rest) and n_q."""
    e_bits = np.asarray(e_bits, np.uint16)
    n_q = (int(n) // Q4_GROUP) * Q4_GROUP
    out_bits = e_bits.copy()
    axis = 0 if kind == "k" else 1
    if n_q == 0:
        d = e_bits.shape[1]
        empty = np.zeros((0, d) if kind == "k" else (0, d // Q4_GROUP), F64)
        return {"codes": np.zeros((0, d), np.uint8), "scale": empty, "zero": empty.copy(), "e_bits": out_bits, "n_q": 0}
    x = decode_bits(e_bits[:n_q], dtype)
    codes, scale, zero = q4_quantise(x, axis, meta_dtype=dtype)
    out_bits[:n_q] = encode_bits(q4_dequantise(codes, scale, zero, axis), dtype)
    return {"codes": codes, "scale": scale, "zero": zero, "e_bits": out_bits, "n_q": n_q}


def q4_cache_pair(m: Dict[str, object], seq_lens: Sequence[int], kind: str, dtype: str) -> Dict[str, object]:
    """A merged pair (the dict `merge_pair` returns for one tensor) as the 4-bit cache holds it:
    "e_bits" becomes the stored (de-quantised, 16-bit rounded) directions, "e16_bits" keeps the
    directions before quantisation, "q4" maps (b, h) to the codes and group parameters."""
    out = dict(m)
    e16 = m["e_bits"]
    eb = e16.copy()
    q4 = {}
    B, S, H, _ = e16.shape
    for b in range(B):
        for h in range(H):
            r = q4_cache_quantise(e16[b, :, h], int(seq_lens[b]), kind, dtype)
            eb[b, :, h] = r["e_bits"]
            q4[(b, h)] = r
    out["e16_bits"], out["e_bits"], out["q4"] = e16, eb, q4
    return out


# --------------------------------------------------------------------------
# Footprint (Sec. 4.3, Appendix "Detailed Efficiency Derivation")
# --------------------------------------------------------------------------
def footprint_bytes(n_layers: int, start_layer: int, tokens_heads: int, head_dim: int,
                    retained_rows: int, elem_bytes: int = 2) -> Dict[str, float]:
    """First-principles byte count of the cache, full versus compressed.

    tokens_heads = number of (token, kv head) rows per layer and tensor;
    retained_rows = total retained (row, tensor) entries over all pairs."""
    row = head_dim * elem_bytes
    full = 2 * n_layers * tokens_heads * row
    n_pairs = (n_layers - start_layer) // 2
    lower = 2 * (n_layers - 2 * n_pairs) * tokens_heads * row
    shared = 2 * n_pairs * tokens_heads * row
    scalars = 2 * n_pairs * tokens_heads * 3 * 4  # two magnitudes and the distance, fp32
    kept = retained_rows * (2 * row + 4)
    comp = lower + shared + scalars + kept
    return {"full": float(full), "compressed": float(comp), "ratio": comp / full}

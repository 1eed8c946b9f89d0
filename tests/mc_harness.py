"""Shared test plumbing: builds a seeded problem, runs the CUDA path through the C ABI, runs the
fp64 oracle on the same bits and compares the two.  Used by the gpu-marked tests and by the
smoke check.  The oracle side only ever sees generator output and, for the stage-wise checks,
buffers read back from the device; no expected value is stored from the CUDA path."""
from __future__ import annotations

import math
from typing import Dict, Optional

import numpy as np
import torch

import gen
from gen import WorkloadConfig, as_bits
from oracle import minicache_oracle as orc

ULP_REL = {"f16": 2.0 ** -10, "bf16": 2.0 ** -7}  # spacing of neighbouring values relative to the value


class Problem:
    """One layer pair of a workload, paged on the device, plus the logical host copies."""

    def __init__(self, cfg: WorkloadConfig, pair: int = 0, device="cuda", seq_lens=None, gamma=None, t=None,
                 retain_mode: int = 0, page_size: Optional[int] = None, decode_room: int = 8,
                 tensors: Optional[Dict[str, torch.Tensor]] = None, ret_capacity: Optional[int] = None,
                 q4: bool = False, merge_fn: str = "slerp", segments=None, cache_bits: int = 16,
                 t_mode: int = 0, retain_union: int = 0, append_slack: int = 0):
        """segments: list of (sequence, kv head) the oracle will look at; given, the host copies of 4-bit
        layers (exact de-quantised values, fp64) are kept for those segments only (full-size workloads)."""
        import paper_2405_14366_b200 as mc
        self.mc = mc
        self.lib = mc.lib()
        self.wl = cfg
        self.device = device
        self.dtype = cfg.dtype
        self.t = cfg.t if t is None else t
        self.gamma = cfg.gamma if gamma is None else gamma
        self.ps = cfg.page_size if page_size is None else page_size
        self.H, self.Hq = cfg.n_kv_heads, cfg.n_q_heads
        if tensors is None:
            tensors = gen.make_pair_tensors(cfg, pair, device="cpu")
        self.logical = {k: v for k, v in tensors.items() if k in ("k_lm1", "k_l", "v_lm1", "v_l")}
        B, S = self.logical["k_l"].shape[:2]
        self.B, self.S = B, S
        if seq_lens is None:
            seq_lens = np.full(B, S, np.int32)
        self.seq_lens_host = np.asarray(seq_lens, np.int32)
        cap = self.seq_lens_host + decode_room
        bt, n_pages = gen.make_block_table(np.maximum(cap, 1), self.ps, seed=1234 + cfg.index)
        self.n_pages = n_pages
        self.block_table = torch.from_numpy(bt).to(device)
        self.seq_lens = torch.from_numpy(self.seq_lens_host.copy()).to(device)
        self.max_seq_len = int(self.seq_lens_host.max()) if B else 0
        self.merge_fn = merge_fn
        self.cfg = mc.McConfig(self.H, self.Hq, self.ps, cfg.dtype, t=self.t, gamma=self.gamma, retain_mode=retain_mode,
                               merge_fn={"slerp": 0, "fmax": 1, "mean": 2}[merge_fn], cache_bits=cache_bits,
                               t_mode=t_mode, retain_union=retain_union, append_slack=append_slack)
        self.cache_bits, self.t_mode, self.retain_union = cache_bits, t_mode, retain_union
        self.append_slack = append_slack
        self.pools = {}
        self.q4 = q4
        self.q4_pools: Dict[str, Dict[str, torch.Tensor]] = {}
        self.values: Dict[str, np.ndarray] = {}
        self.seg_values: Dict = {}
        self.seg_bits: Dict = {}
        self.segments = segments
        for name, x in self.logical.items():
            xm = x.clone()
            for b in range(B):  # rows past a sequence's length never reach the device pools as data
                xm[b, self.seq_lens_host[b]:] = 0
            if not q4:
                self.pools[name] = gen.to_paged(xm.to(device), self.block_table, self.ps, n_pages)
                continue
            # 4-bit layers: quantise the logical rows (data preparation), page codes and meta, and keep
            # the exact de-quantised values for the oracle
            assert self.ps == 32 and S % 32 == 0
            kind = name[0]
            qd = gen.quantise_q4(xm.to(device), kind)  # data preparation (same arithmetic on either device)
            codes, meta = qd["codes"].cpu(), qd["meta"].cpu()
            axis = 1 if kind == "k" else 3

            def dequant(cn, mt):
                full = np.empty(cn.shape[:-1] + (128,), np.uint8)
                full[..., 0::2], full[..., 1::2] = cn & 15, cn >> 4
                return orc.q4_dequantise(full, mt[..., 0], mt[..., 1], axis)
            if segments is None:
                self.values[name] = dequant(codes.numpy(), meta.double().numpy())
            else:
                for (sb, sh) in segments:
                    v = dequant(codes[sb:sb + 1, :, sh:sh + 1].numpy(), meta[sb:sb + 1, :, sh:sh + 1].double().numpy())
                    self.seg_values[(name, sb, sh)] = v
                    self.seg_bits[(name, sb, sh)] = orc.encode_bits(v, self.dtype)
            pc = gen.to_paged(codes.to(device), self.block_table, self.ps, n_pages)
            if kind == "k":
                pm = torch.zeros(n_pages, self.H, 128, 2, dtype=torch.float16, device=device)
                btl = self.block_table[:, :S // 32].long()
                ok = btl >= 0
                pm[btl[ok]] = meta.to(device)[ok]
            else:
                pm = gen.to_paged(meta.reshape(B, S, self.H, 8).to(device), self.block_table, self.ps, n_pages)
            self.q4_pools[name] = {"codes": pc, "meta": pm.contiguous()}
        total = int(self.seq_lens_host.sum()) * self.H * 2 + 2 * B * self.H * append_slack
        self.ret_capacity = total if ret_capacity is None else ret_capacity
        self.pair = mc.PairCache(self.cfg, B, n_pages, self.ret_capacity, device=device)
        if q4:  # the rows the cache can hold: the de-quantised values rounded once to the storage type
            self.bits = {k: orc.encode_bits(v, self.dtype) for k, v in self.values.items()}
        else:
            self.bits = {k: as_bits(v) for k, v in self.logical.items()}

    # ------------------------------------------------------------------ device side
    def batch(self, extra: int = 0):
        return self.mc.Batch(self.block_table, self.seq_lens, self.max_seq_len + extra, self.n_pages)

    def workspace(self, op: int, n_sets: int = 1, extra: int = 0):
        n = self.lib.mc_workspace_bytes(self.cfg, self.batch(extra), op, n_sets)
        return torch.empty(n, dtype=torch.uint8, device=self.device)

    def run_merge(self, do_retention: bool = True):
        ws = self.workspace(0)
        if self.q4:
            lay = lambda sfx: {"k_codes": self.q4_pools["k" + sfx]["codes"], "k_meta": self.q4_pools["k" + sfx]["meta"],
                               "v_codes": self.q4_pools["v" + sfx]["codes"], "v_meta": self.q4_pools["v" + sfx]["meta"]}
            self.lib.mc_merge_pair_q4(self.cfg, self.batch(), lay("_lm1"), lay("_l"), self.pair, do_retention, ws)
            torch.cuda.synchronize()
            return self.lib.mc_read_status(self.pair, check=False)
        self.lib.mc_merge_pair(self.cfg, self.batch(), self.pools["k_lm1"], self.pools["v_lm1"], self.pools["k_l"],
                               self.pools["v_l"], self.pair, do_retention, ws)
        torch.cuda.synchronize()
        return self.lib.mc_read_status(self.pair, check=False)

    def segment_bits(self, name: str, b: int, h: int) -> np.ndarray:
        """The 16-bit rows [1][S][1][128] of one (sequence, kv head) the cache can hold for input `name`."""
        if (name, b, h) in self.seg_bits:
            return self.seg_bits[(name, b, h)]
        return self.bits[name][b:b + 1, :, h:h + 1]

    def run_restore(self, layer: int, fp32: bool = False):
        dk = torch.zeros(self.n_pages, self.H, self.ps, 128, dtype=torch.float32 if fp32 else self.cfg.torch_dtype, device=self.device)
        dv = torch.zeros_like(dk)
        self.lib.mc_restore(self.cfg, self.batch(), self.pair, layer, dk, dv)
        torch.cuda.synchronize()
        return dk, dv

    def run_attn(self, layer_sel: int, q: torch.Tensor, k_new=None, v_new=None, want_lse=True):
        n_sets = 2 if layer_sel == 2 else 1
        out = torch.zeros(n_sets, self.B, self.Hq, 128, dtype=self.cfg.torch_dtype, device=self.device)
        lse = torch.zeros(n_sets, self.B, self.Hq, dtype=torch.float32, device=self.device) if want_lse else None
        ws = self.workspace(1, n_sets)
        self.lib.mc_decode_attn(self.cfg, self.batch(), self.pair, layer_sel, q, k_new, v_new,
                                1.0 / math.sqrt(128.0), out, lse, ws)
        torch.cuda.synchronize()
        return out, lse

    # ------------------------------------------------------------------ read-back helpers
    def logical_of(self, pool: torch.Tensor, seq_len: Optional[int] = None) -> torch.Tensor:
        return gen.from_paged(pool, self.block_table, self.S if seq_len is None else seq_len).cpu()

    def device_cache(self, extra_tokens: int = 0) -> Dict[str, np.ndarray]:
        """The compressed pair read back into logical numpy arrays."""
        S = self.S + extra_tokens
        pc = self.pair
        scale = torch.cat([pc.scales("k"), pc.scales("v")], dim=2)  # [n_pages][H][4][ps]: K l-1, K l, V l-1, V l
        sc = gen.from_paged(scale.permute(0, 1, 3, 2).contiguous(), self.block_table, S).cpu().numpy()  # [B][S][H][4]
        if self.cache_bits == 4:
            out = self._q4_cache_bits(S, extra_tokens, sc)
        else:
            out = {"e_k": as_bits(self.logical_of(pc.directions("k"), S)), "e_v": as_bits(self.logical_of(pc.directions("v"), S))}
        ds = gen.from_paged(pc.dist.permute(0, 1, 3, 2).contiguous(), self.block_table, S).cpu().numpy()   # [B][S][H][2]
        out["scale"], out["dist"] = sc.astype(np.float64), ds.astype(np.float64)
        out["ret_count"] = pc.ret_count.cpu().numpy().reshape(2, self.B, self.H)
        out["ret_offset"] = pc.ret_offset.cpu().numpy()
        out["ret_index"] = pc.ret_index.cpu().numpy()
        out["ret_rows"] = np.stack([as_bits(pc.retained_rows(0).cpu()), as_bits(pc.retained_rows(1).cpu())], axis=1)  # [cap][2][128]
        out["ret_tokens"] = np.stack([pc.retained_tokens(0).cpu().numpy(), pc.retained_tokens(1).cpu().numpy()], axis=1)
        out["seg_minmax"] = pc.seg_minmax.cpu().numpy().reshape(2, self.B, self.H, 2).astype(np.float64)
        return out

    def _q4_cache_bits(self, S: int, extra_tokens: int, sc: np.ndarray) -> Dict[str, np.ndarray]:
        """The stored directions of a 4-bit shared cache as 16-bit patterns [B][S][H][128]: for the tokens in
        complete pages code * scale + zero rounded once to the storage type (formed here with the oracle's
        de-quantiser from the device's codes and group parameters), for the tokens of the last, incomplete
        page the residual tile's rows; `sc` gets the residual tokens' scales.  Also returns the codes and
        group parameters per (sequence, head).  With `self.segments` only those (sequence, head) are filled."""
        pc = self.pair
        S32 = (S + 31) // 32 * 32
        npg = S32 // 32
        segs = self.segments if self.segments is not None else [(b, h) for b in range(self.B) for h in range(self.H)]
        out = {"q4": {}}
        for ti, tn in enumerate(("k", "v")):
            codes_dev = pc.q4_codes(tn)
            sg, zg = pc.q4_groups(tn)
            res = pc.residual_directions(tn)  # [B][H][32][128]
            rsc = pc.residual_scales(tn)      # [B][H][2][32]
            e = np.zeros((self.B, S, self.H, 128), np.uint16)
            for (b, h) in segs:
                n = int(self.seq_lens_host[b]) + extra_tokens
                nq = n // 32 * 32
                btl = self.block_table[b, :npg].long().clamp(min=0)
                codes = codes_dev[btl, h].reshape(S32, 128).cpu().numpy()[:nq]
                if tn == "k":  # per (page, channel)
                    scale = orc.decode_bits(as_bits(sg[btl, h].cpu()), self.dtype)[:nq // 32]
                    zero = orc.decode_bits(as_bits(zg[btl, h].cpu()), self.dtype)[:nq // 32]
                    axis = 0
                else:  # per (token, channel group)
                    scale = orc.decode_bits(as_bits(sg[btl, h].reshape(S32, 4).cpu()), self.dtype)[:nq]
                    zero = orc.decode_bits(as_bits(zg[btl, h].reshape(S32, 4).cpu()), self.dtype)[:nq]
                    axis = 1
                if nq:
                    e[b, :nq, h] = orc.encode_bits(orc.q4_dequantise(codes, scale, zero, axis), self.dtype)
                if n > nq:
                    e[b, nq:n, h] = as_bits(res[b, h, :n - nq].cpu())
                    sc[b, nq:n, h, 2 * ti:2 * ti + 2] = rsc[b, h, :, :n - nq].cpu().numpy().T
                out["q4"][(tn, b, h)] = {"codes": codes, "scale": scale, "zero": zero, "n_q": nq}
            out["e_" + tn] = e
        return out

    def retained(self, dc, tensor: int, b: int, h: int):
        seg = (tensor * self.B + b) * self.H + h
        off, cnt = int(dc["ret_offset"][seg]), int(dc["ret_count"][tensor, b, h])
        idx = dc["ret_index"][off:off + cnt].astype(np.int64)
        # every entry carries its token index next to the row, for both layers
        assert np.array_equal(dc["ret_tokens"][off:off + cnt, 0], idx) and np.array_equal(dc["ret_tokens"][off:off + cnt, 1], idx)
        return idx, dc["ret_rows"][off:off + cnt]

    # ------------------------------------------------------------------ oracle side
    @property
    def oracle_t(self):
        """The oracle's t argument: the number, or "ratio" for the per-token magnitude ratio."""
        return "ratio" if self.t_mode == 1 else self.t

    def oracle_merge(self, mode: str = "distinct", do_retention: bool = True):
        out = {}
        for ti, tn in enumerate(("k", "v")):
            if self.q4:
                out[tn] = orc.merge_pair_values(self.values[tn + "_lm1"], self.values[tn + "_l"], self.seq_lens_host,
                                                self.dtype, self.oracle_t, self.gamma, mode=mode, do_retention=do_retention,
                                                merge_fn=self.merge_fn)
                continue
            out[tn] = orc.merge_pair(self.bits[tn + "_lm1"], self.bits[tn + "_l"], self.seq_lens_host, self.dtype,
                                     self.oracle_t, self.gamma, mode=mode, do_retention=do_retention, merge_fn=self.merge_fn)
        if self.retain_union:  # one set for keys and values
            un = orc.retention_union(out["k"]["retained"], out["v"]["retained"])
            out["k"]["retained"], out["v"]["retained"] = un, dict(un)
        if self.cache_bits == 4:  # the merged directions as the 4-bit shared cache stores them
            out = {tn: orc.q4_cache_pair(out[tn], self.seq_lens_host, tn, self.dtype) for tn in out}
        return out


def _mask_valid(p: Problem):
    m = np.zeros((p.B, p.S), bool)
    for b in range(p.B):
        m[b, :p.seq_lens_host[b]] = True
    return m


def compare_merge(p: Problem, om, dc, mode: str = "distinct", do_retention: bool = True) -> Dict[str, float]:
    """Element-by-element comparison of the merge outputs.  Returns statistics; asserts the bars."""
    stats: Dict[str, float] = {}
    valid = _mask_valid(p)
    ulp = ULP_REL[p.dtype]
    for ti, tn in enumerate(("k", "v")):
        o = om[tn]
        e_gpu = orc.decode_bits(dc["e_" + tn], p.dtype)
        e_orc = orc.decode_bits(o["e_bits"], p.dtype)
        vm = valid[:, :, None, None]
        # stored directions: identical codes, except elements whose unrounded value sits on a rounding
        # boundary (fp32 vs fp64 arithmetic lands on different sides): at most one unit in the last place
        diff = np.abs(e_gpu - e_orc) * vm
        flips = (dc["e_" + tn] != o["e_bits"]) & np.broadcast_to(vm, diff.shape)
        nflip = int(flips.sum())
        if nflip:
            spacing = np.maximum(np.abs(e_orc), 2.0 ** -14) * ulp * 1.01
            assert np.all(diff[flips] <= spacing[flips]), "direction differs by more than one ulp"
            # ... and the oracle's unrounded value is close to the midpoint between the two codes
            mid_dist = np.abs(np.abs(o["e"] - e_orc) - 0.5 * np.abs(e_gpu - e_orc))
            assert np.all(mid_dist[flips] <= 3e-7), "flip not at a rounding boundary"
        total = int(valid.sum()) * p.H * 128
        stats[f"{tn}_flip_frac"] = nflip / max(total, 1)
        assert nflip <= max(8, 5e-3 * total), f"too many rounding flips: {nflip}/{total}"
        # scales: |x| / |e_stored| with the oracle's own stored direction; zero where the device retained
        # the token (its raw rows serve it instead)
        ret_mask = np.zeros((p.B, p.S, p.H), bool)
        for b in range(p.B):
            for h in range(p.H):
                ret_mask[b, p.retained(dc, ti, b, h)[0], h] = True
        len_e = np.sqrt(np.sum(e_orc * e_orc, -1))
        len_e = np.where(len_e == 0, 1.0, len_e)
        row_flip = flips.any(-1)
        for li, nm in enumerate(("n_lm1", "n_l")):
            want = o[nm] / len_e
            got = dc["scale"][..., ti * 2 + li]
            assert np.all(got[ret_mask] == 0.0), "scale of a retained token must be zero"
            rel = np.abs(got - want) / np.maximum(np.abs(want), 1e-30) * valid[:, :, None] * ~ret_mask
            clean = rel * ~row_flip
            stats[f"{tn}_scale_rel"] = max(stats.get(f"{tn}_scale_rel", 0.0), float(clean.max(initial=0.0)))
            assert clean.max(initial=0.0) < 2e-6, f"scale mismatch {clean.max()}"
            assert rel.max(initial=0.0) < 4 * ulp, "scale of a row with a rounding flip is off"
        # distances
        dd = np.abs(dc["dist"][..., ti] - o["d"]) * valid[:, :, None]
        stats[f"{tn}_dist_abs"] = float(dd.max(initial=0.0))
        assert dd.max(initial=0.0) < 5e-7, f"distance mismatch {dd.max()}"
        # retention sets
        near = 0
        mism = 0
        for b in range(p.B):
            n = int(p.seq_lens_host[b])
            for h in range(p.H):
                want = o["retained"][(b, h)]
                got, rows = p.retained(dc, ti, b, h)
                assert np.all(np.diff(got) > 0), "retained indices not ascending"
                if n == 0:
                    assert len(got) == 0
                    continue
                d = o["d"][b, :n, h]
                if not do_retention:
                    assert len(got) == 0
                    continue
                mm = dc["seg_minmax"][ti, b, h]
                assert abs(mm[0] - d.min()) < 5e-7 and abs(mm[1] - d.max()) < 5e-7
                if mode == "topk":
                    # the k largest: exact count; the sets may differ only among tokens whose distance is
                    # within 1e-6 of the k-th largest (fp32 and fp64 distances can order them differently)
                    assert len(got) == len(want)
                    thr = np.sort(d)[::-1][len(want) - 1] if len(want) else np.inf
                else:
                    thr = orc.retention_threshold(d, p.gamma, mode)
                sym = np.setxor1d(want, got)
                # exact, except tokens whose distance lies within 1e-6 of the threshold
                close = np.abs(d[sym] - thr) < 1e-6
                if getattr(p, "retain_union", 0):  # ... or of the other tensor's threshold, whose rule also decides
                    d_o = om["v" if tn == "k" else "k"]["d"][b, :n, h]
                    close |= np.abs(d_o[sym] - orc.retention_threshold(d_o, p.gamma, mode)) < 1e-6
                assert np.all(close), f"retained set differs away from the threshold: {sym}"
                mism += len(sym)
                near += int(np.sum(np.abs(d - thr) < 1e-6))
                # raw rows are bit copies of both layers' inputs
                assert np.array_equal(rows[:, 0], p.bits[tn + "_lm1"][b, got, h])
                assert np.array_equal(rows[:, 1], p.bits[tn + "_l"][b, got, h])
        stats[f"{tn}_near_threshold"] = near
        stats[f"{tn}_set_mismatch"] = mism
    return stats


def oracle_restore_from_device(p: Problem, dc, layer: int, tensor: str, b: int, h: int, n: Optional[int] = None):
    """Oracle restore fed with the device's compressed cache (stage-wise check)."""
    ti = 0 if tensor == "k" else 1
    n = int(p.seq_lens_host[b]) if n is None else n
    e_bits = dc["e_" + tensor][b, :n, h]
    e = orc.decode_bits(e_bits, p.dtype)
    norms = dc["scale"][b, :n, h, ti * 2 + layer] * np.sqrt(np.sum(e * e, -1))
    idx, rows = p.retained(dc, ti, b, h)
    return orc.restore(e_bits, norms, p.dtype, idx, rows[:, layer] if len(idx) else None)


def compare_restore(p: Problem, om, dc, layer: int, dk: torch.Tensor, dv: torch.Tensor) -> Dict[str, float]:
    stats = {}
    lname = ("n_lm1", "n_l")[layer]
    src = ("_lm1", "_l")[layer]
    f32_out = dk.dtype == torch.float32  # the restore wrote its products unrounded
    for ti, (tn, pool) in enumerate((("k", dk), ("v", dv))):
        got = p.logical_of(pool).double().numpy() if f32_out else orc.decode_bits(as_bits(p.logical_of(pool)), p.dtype)
        o = om[tn]
        err_e2e, ref_max, err_stage = 0.0, 0.0, 0.0
        for b in range(p.B):
            n = int(p.seq_lens_host[b])
            for h in range(p.H):
                idx = o["retained"][(b, h)]
                want = orc.restore(o["e_bits"][b, :n, h], o[lname][b, :n, h], p.dtype, idx,
                                   p.bits[tn + src][b, idx, h] if len(idx) else None)
                g = got[b, :n, h]
                didx, _ = p.retained(dc, ti, b, h)
                same_set = np.setdiff1d(np.arange(n), np.setxor1d(idx, didx))  # rows both sides treat alike
                flips = (dc["e_" + tn][b, :n, h] != o["e_bits"][b, :n, h])
                dif = np.abs(g - want)
                if p.dtype == "bf16" and not f32_out:
                    # the dense output is itself stored in bfloat16, whose half-ulp (2^-8 of the value)
                    # alone exceeds the 2e-3 bar: the bar applies to the value before that last rounding
                    dif = np.maximum(dif - 0.505 * ULP_REL["bf16"] * np.abs(want), 0.0)
                dif[flips] = 0.0  # one-ulp rounding flips of the stored direction are counted in compare_merge
                err_e2e = max(err_e2e, float(dif[same_set].max(initial=0.0)))
                ref_max = max(ref_max, float(np.abs(want).max(initial=0.0)))
                # retained rows come back bit-exactly
                if len(didx):
                    if f32_out:
                        assert np.array_equal(g[didx], orc.decode_bits(p.bits[tn + src][b, didx, h], p.dtype))
                    else:
                        assert np.array_equal(as_bits(p.logical_of(pool))[b, didx, h], p.bits[tn + src][b, didx, h])
                # stage-wise: oracle restore of the device's own cache; only the final 16-bit rounding differs
                want2 = oracle_restore_from_device(p, dc, layer, tn, b, h)
                # (0.505 ulp of the value, plus half the subnormal spacing of binary16)
                # (binary32 output: only the device's single fp32 multiply differs from the exact product)
                bound = (2.0 ** -23 * np.abs(want2) + 1e-37) if f32_out else 0.505 * ULP_REL[p.dtype] * np.abs(want2) + 3.1e-8
                err_stage = max(err_stage, float((np.abs(g - want2) / bound).max(initial=0.0)))
        rel = err_e2e / max(ref_max, 1e-30)
        stats[f"{tn}_restore_rel"] = rel
        stats[f"{tn}_restore_stage"] = err_stage
        assert rel < 2e-3, f"restored {tn} off by {rel} (max-abs relative)"
        assert err_stage <= 1.0, f"restore of the device cache off by {err_stage} rounding bounds"
    return stats


def oracle_attention(p: Problem, om, layer: int, q_bits, b: int, hq: int, k_new_bits=None, v_new_bits=None):
    g = hq // (p.Hq // p.H)
    n = int(p.seq_lens_host[b])
    lname = ("n_lm1", "n_l")[layer]
    src = ("_lm1", "_l")[layer]
    ik, iv = om["k"]["retained"][(b, g)], om["v"]["retained"][(b, g)]
    return orc.decode_attention(
        q_bits, om["k"]["e_bits"][b, :n, g], om["v"]["e_bits"][b, :n, g], om["k"][lname][b, :n, g],
        om["v"][lname][b, :n, g], p.dtype, 1.0 / math.sqrt(128.0),
        idx_k=ik, rows_k_bits=p.bits["k" + src][b, ik, g] if len(ik) else None,
        idx_v=iv, rows_v_bits=p.bits["v" + src][b, iv, g] if len(iv) else None,
        k_new_bits=k_new_bits, v_new_bits=v_new_bits)


def oracle_attention_from_device(p: Problem, dc, layer: int, q_bits, b: int, hq: int, k_new_bits=None, v_new_bits=None):
    """Oracle attention (fp64) over the DEVICE's own compressed cache: its stored directions, its scales
    (magnitude = scale x length of the stored direction) and its retained rows.  What differs from the
    device's attention is then the attention arithmetic alone (stage-wise check)."""
    g = hq // (p.Hq // p.H)
    n = int(p.seq_lens_host[b])
    ek, ev = dc["e_k"][b, :n, g], dc["e_v"][b, :n, g]
    nk = dc["scale"][b, :n, g, layer] * np.sqrt(np.sum(orc.decode_bits(ek, p.dtype) ** 2, -1))
    nv = dc["scale"][b, :n, g, 2 + layer] * np.sqrt(np.sum(orc.decode_bits(ev, p.dtype) ** 2, -1))
    ik, rk = p.retained(dc, 0, b, g)
    iv, rv = p.retained(dc, 1, b, g)
    return orc.decode_attention(q_bits, ek, ev, nk, nv, p.dtype, 1.0 / math.sqrt(128.0),
                                idx_k=ik, rows_k_bits=rk[:, layer] if len(ik) else None,
                                idx_v=iv, rows_v_bits=rv[:, layer] if len(iv) else None,
                                k_new_bits=k_new_bits, v_new_bits=v_new_bits)


# End-to-end log-sum-exp bar.  Against the oracle's own cache the device's scores differ where a stored
# direction element fell on the other side of a rounding boundary (counted in compare_merge): one flip
# moves that token's score by |q_c| x ulp(e_c) x scale x sm_scale, and the log-sum-exp by at most that.
# With |q_c| up to 4 sigma = 113, e_c around 0.1-0.25, scale up to 4 and sm_scale 1/sqrt(128) this is at
# most 113 x 2^-13 x 4 x 0.088 = 4.9e-3 in binary16 (typically 28 x 2^-14 x 1 x 0.088 = 1.5e-4) and 8
# times that in bfloat16; the bars below sit between the typical and the worst case, and the stage-wise
# bar (same stored cache on both sides, so no flips) is 1e-4 for both types.
LSE_E2E_BAR = {"f16": 1e-3, "bf16": 8e-3}
LSE_STAGE_BAR = 1e-4
# 4-bit shared cache, end to end: a flipped 16-bit element that is the minimum or maximum of its group
# moves the group's scale or zero by one unit in the last place of the 16-bit type, and with it up to 32
# stored values of that group by as much as the group's range (about 0.3 for unit directions) times that
# unit: |q_c| x 0.3 x 2^-11 x scale x sm_scale = 113 x 0.3 x 2^-11 x 4 x 0.088 = 5.8e-3 at worst in binary16,
# eight times that in bfloat16 (typical: 28 x 0.3 x 2^-8 x 1 x 0.088 = 2.9e-3).  The stage-wise bar (the
# device's own codes and group parameters on both sides) stays 1e-4.
LSE_E2E_BAR_Q4 = {"f16": 6e-3, "bf16": 5e-2}


def compare_attention(p: Problem, om, layer_sel: int, q: torch.Tensor, out: torch.Tensor, lse, k_new=None, v_new=None,
                      sample=None, dc=None) -> Dict[str, float]:
    """out [n_sets][B][Hq][128] against the oracle (restore + dense attention in fp64).  With `dc` (the
    device's cache read back) also stage-wise: oracle attention over the device's own cache."""
    qb = as_bits(q)
    ob = orc.decode_bits(as_bits(out), p.dtype)
    knb = as_bits(k_new) if k_new is not None else None
    vnb = as_bits(v_new) if v_new is not None else None
    layers = (0, 1) if layer_sel == 2 else (layer_sel,)
    err, lerr, serr, slerr = 0.0, 0.0, 0.0, 0.0
    nq = p.Hq // p.H
    items = [(b, h) for b in range(p.B) for h in range(p.Hq)] if sample is None else sample
    for si, layer in enumerate(layers):
        for b, hq in items:
            g = hq // nq
            kn = knb[si, b, g] if knb is not None else None
            vn = vnb[si, b, g] if vnb is not None else None
            n = int(p.seq_lens_host[b])
            if n == 0 and kn is None:
                assert np.all(ob[si, b, hq] == 0)
                continue
            o, l = oracle_attention(p, om, layer, qb[si, b, hq], b, hq, kn, vn)
            err = max(err, float(np.abs(ob[si, b, hq] - o).max()))
            if lse is not None:
                lerr = max(lerr, abs(float(lse[si, b, hq]) - l))
            if dc is not None:
                o2, l2 = oracle_attention_from_device(p, dc, layer, qb[si, b, hq], b, hq, kn, vn)
                # the output is rounded once to the storage type: half an ulp of the value on top
                serr = max(serr, float((np.abs(ob[si, b, hq] - o2) - 0.505 * ULP_REL[p.dtype] * np.abs(o2)).max()))
                if lse is not None:
                    slerr = max(slerr, abs(float(lse[si, b, hq]) - l2))
    assert err < 1e-2, f"attention output off by {err} (max-abs)"
    bar = LSE_E2E_BAR_Q4 if getattr(p, "cache_bits", 16) == 4 else LSE_E2E_BAR
    assert lerr < bar[p.dtype], f"log-sum-exp off by {lerr}"
    stats = {"attn_abs": err, "lse_abs": lerr}
    if dc is not None:
        # stage-wise: the probabilities enter the tensor cores rounded to the storage type (relative
        # 2^-11 / 2^-8 each, averaging out over the tokens): a small multiple of the output's own ulp
        assert serr < (1e-3 if p.dtype == "f16" else 4e-3), f"attention over the device's cache off by {serr}"
        assert slerr < LSE_STAGE_BAR, f"log-sum-exp over the device's cache off by {slerr}"
        stats.update({"attn_stage_abs": serr, "lse_stage_abs": slerr})
    return stats


def compare_q4_cache(p4: Problem, dc4, dc16, om4) -> Dict[str, float]:
    """The 4-bit shared cache, stage by stage.  `dc16` is the 16-bit cache the same merge kernels wrote for
    the same inputs (compared with the oracle by compare_merge); the quantiser is deterministic integer
    work on those bits, so the oracle's quantiser fed with them must give the device's codes, group
    parameters and stored (de-quantised) directions exactly.  The scales refer to the stored direction:
    |x| / |e_q|, checked against the 16-bit scale times |e_16| / |e_q| (stage-wise) and against the oracle's
    own 4-bit cache `om4` on rows whose stored bits agree (end to end)."""
    stats = {"q4_groups": 0, "q4_scale_stage": 0.0, "q4_scale_e2e": 0.0, "q4_rows_differ": 0}
    for (tn, b, h), dev in dc4["q4"].items():
        ti = 0 if tn == "k" else 1
        n = int(p4.seq_lens_host[b])
        r = orc.q4_cache_quantise(dc16["e_" + tn][b, :, h], n, tn, p4.dtype)
        assert r["n_q"] == dev["n_q"]
        assert np.array_equal(r["codes"], dev["codes"]), f"codes differ {tn} {b} {h}"
        assert np.array_equal(r["scale"], dev["scale"]) and np.array_equal(r["zero"], dev["zero"]), f"group parameters differ {tn} {b} {h}"
        assert np.array_equal(r["e_bits"][:n], dc4["e_" + tn][b, :n, h]), f"stored directions differ {tn} {b} {h}"
        stats["q4_groups"] += r["scale"].size
        if n == 0:
            continue
        e16 = orc.decode_bits(dc16["e_" + tn][b, :n, h], p4.dtype)
        eq = orc.decode_bits(dc4["e_" + tn][b, :n, h], p4.dtype)
        l16, lq = np.sqrt(np.sum(e16 * e16, -1)), np.sqrt(np.sum(eq * eq, -1))
        lq = np.where(lq == 0, 1.0, lq)
        eo = orc.decode_bits(om4[tn]["e_bits"][b, :n, h], p4.dtype)
        lo = np.sqrt(np.sum(eo * eo, -1))
        lo = np.where(lo == 0, 1.0, lo)
        same = np.all(om4[tn]["e_bits"][b, :n, h] == dc4["e_" + tn][b, :n, h], axis=-1)
        stats["q4_rows_differ"] += int((~same).sum())
        for li, nm in enumerate(("n_lm1", "n_l")):
            g16, g4 = dc16["scale"][b, :n, h, 2 * ti + li], dc4["scale"][b, :n, h, 2 * ti + li]
            # a retained token keeps its mark (-0), a zero row its zero
            assert np.array_equal(np.signbit(g16) & (g16 == 0), np.signbit(g4) & (g4 == 0))
            want = g16 * l16 / lq
            rel = np.abs(g4 - want) / np.maximum(np.abs(want), 1e-30) * (g16 != 0)
            stats["q4_scale_stage"] = max(stats["q4_scale_stage"], float(rel.max(initial=0.0)))
            want2 = om4[tn][nm][b, :n, h] / lo
            rel2 = np.abs(g4 - want2) / np.maximum(np.abs(want2), 1e-30) * (g4 != 0) * same
            stats["q4_scale_e2e"] = max(stats["q4_scale_e2e"], float(rel2.max(initial=0.0)))
    # g_q = g_16 |e_16| / |e_q| on the device: the two sums of 128 exact squares are accumulated pairwise in fp32
    # (seven roundings deep: within 7 x 2^-24 = 4.2e-7 each), then one division, one square root (which halves
    # the relative error) and one product, one rounding each: (2 x 4.2e-7 + 6e-8) / 2 + 2 x 6e-8 < 6e-7
    assert stats["q4_scale_stage"] < 6e-7, stats
    assert stats["q4_scale_e2e"] < 3e-6, stats
    return stats

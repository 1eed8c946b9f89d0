"""Benchmark of the MiniCache hot path on B200.

A step = one pass of the whole path over one batch of synthetic input: merge of every layer
pair (Eq. 3 + Eq. 4), materialising restore of every merged layer (Eq. 2), then the decode
phase: for each decode step and each pair, attention of both layers straight over the
compressed cache (single-layer calls, as a real model would issue them) and the append-merge of
the step's new token pair.

    python bench.py --gpus 1 --steps 3 --warmup 3            # device-resident + e2e + CPU baseline
    python bench.py --impl reference --steps 1 --warmup 0    # the fp64 oracle on the host cores

Prints ONE JSON line.  `value` is whole-job algorithmic GB/s (all ranks' bytes / max-rank time).
"""
from __future__ import annotations

import argparse
import dataclasses
import json
import math
import os
import subprocess
import sys
import time

import numpy as np
import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import gen  # noqa: E402

ROW = 256  # bytes of one 16-bit row of 128 channels
# DRAM bytes (read + written) per algorithmic byte of the split attention kernel (16-bit cache), from the ncu
# capture summarised in profiles/attn_split_kernel_c2_one_pair.md (560.2 MB for 547.5 MB), taken of the kernel
# as it is now (a template over the cache format and the score-buffer width).  Set to None when the kernel changes until it is captured again.
ATTN_TRAFFIC_RATIO = 1.023


# ---------------------------------------------------------------------------------------------
def measured_hbm_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        try:
            return float(json.load(open(path))["hbm_gbs"]), "measured (MEASURED_PEAKS.json hbm_gbs)"
        except Exception:
            pass
    return 6650.0, "fallback (6.65 TB/s, earlier measurement on this pool)"


class ClockSampler:
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, device_index: int):
        self.proc = None
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(device_index), f"--query-gpu={self.Q}",
                                          "--format=csv,noheader,nounits", "-lms", "200"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except Exception:
            self.proc = None

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.25)
        self.proc.terminate()
        try:
            out, _ = self.proc.communicate(timeout=5)
        except Exception:
            self.proc.kill()
            out = ""
        sm, mx, reasons = [], [], set()
        for line in out.splitlines():
            f = [x.strip() for x in line.split(",")]
            if len(f) < 9:
                continue
            try:
                sm.append(float(f[1]))
                mx.append(float(f[2]))
            except ValueError:
                continue
            for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), f[5:9]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


# ---------------------------------------------------------------------------------------------
class Job:
    """All device state of one rank's workload."""

    def __init__(self, wl: gen.WorkloadConfig, device, q4: bool = False, q4cache: bool = False, serving: bool = False):
        import paper_2405_14366_b200 as mc
        self.mc, self.lib, self.wl, self.dev, self.q4 = mc, mc.lib(), wl, device, q4
        self.q4cache = q4cache  # the shared cache itself is 4-bit (pages of 32 tokens)
        self.B, self.S, self.H, self.Hq, self.ps = wl.batch, wl.seq_len, wl.n_kv_heads, wl.n_q_heads, wl.page_size
        self.steps = wl.decode_steps
        prompt, gen_len = gen.make_lengths(wl)
        if serving:  # slots that are refilled: every slot gets pages for the longest prompt and the longest generation
            prompt = np.full(wl.batch, wl.seq_len, prompt.dtype)
        self.prompt = prompt
        # the serving mix drains: a sequence leaves the batch after its own number of generated tokens
        # (its length is set to 0: an empty sequence costs one empty work unit per head and nothing else)
        self.gen_len = np.minimum(gen_len, self.steps) if wl.ragged else np.full(wl.batch, self.steps, np.int64)
        cap = prompt + self.steps + 1
        bt, self.n_pages = gen.make_block_table(cap, self.ps, seed=4321 + wl.index)
        self.block_table = torch.from_numpy(bt).to(device)
        self.seq0 = torch.from_numpy(prompt.copy()).to(device)
        self.seq_lens = self.seq0.clone()
        self.gen_dev = torch.from_numpy(np.asarray(self.gen_len, np.int32)).to(device)
        self.step_dev = torch.zeros(1, dtype=torch.int32, device=device)  # decode steps done since the merge
        self.cfg = mc.McConfig(self.H, self.Hq, self.ps, wl.dtype, t=wl.t, gamma=wl.gamma, cache_bits=4 if q4cache else 16)
        self.max_prefill = int(prompt.max())
        self.tok_heads = int(prompt.sum()) * self.H  # (token, kv head) rows per layer and tensor
        self.pools, self.pairs = [], []
        cap_rows = int(max(0.10, 4.0 * wl.outlier_frac, 1.5 * wl.gamma) * 2 * self.tok_heads) + 1024
        if serving:  # one region of the retained pool per slot
            self.rows_per_seq = int(0.10 * 2 * wl.seq_len * self.H) + 64
            cap_rows = self.B * self.rows_per_seq
        for pr in range(wl.n_pairs):
            t = gen.make_pair_tensors(wl, pr, device=device)
            if wl.ragged and not serving:
                for b in range(self.B):
                    for v in t.values():
                        v[b, prompt[b]:] = 0
            if q4:
                self.pools.append(self._q4_layers(t))
            else:
                self.pools.append({k: gen.to_paged(v, self.block_table, self.ps, self.n_pages) for k, v in t.items()})
            del t
            self.pairs.append(mc.PairCache(self.cfg, self.B, self.n_pages, cap_rows, device=device))
        dt = self.cfg.torch_dtype
        self.dst_k = torch.empty(self.n_pages, self.H, self.ps, 128, dtype=dt, device=device)
        self.dst_v = torch.empty_like(self.dst_k)
        nvar = 4
        self.q = [gen.make_queries(wl, i, device=device, n_sets=2) for i in range(nvar)]
        self.new = []
        for i in range(nvar):
            nt = gen.make_new_tokens(wl, 0, i, device=device)
            self.new.append({k: v[:, 0].contiguous() for k, v in nt.items()})
        self.out = torch.empty(1, self.B, self.Hq, 128, dtype=dt, device=device)
        bm, bd = self.batch(False), self.batch(True)
        n_ws = wl.n_pairs if not (q4 or q4cache) else 1  # mc_merge_pairs: one scratch area per pair
        self.ws_merge = torch.empty(n_ws * self.lib.mc_workspace_bytes(self.cfg, bm, 0, 1), dtype=torch.uint8, device=device)
        self.ws_attn = torch.empty(self.lib.mc_workspace_bytes(self.cfg, bd, 1, 1), dtype=torch.uint8, device=device)
        self.sm_scale = 1.0 / math.sqrt(128.0)
        self.launches = 0
        self.attn_events = []

    def _q4_layers(self, t):
        """The pair's two layers as 4-bit pools (keys per channel, values per token, groups of 32)."""
        assert self.ps == 32 and self.S % 32 == 0, "4-bit layers need pages of 32 tokens"
        npg = self.S // 32
        btl = self.block_table[:, :npg].long()
        ok = btl >= 0
        out = {}
        for sfx in ("_lm1", "_l"):
            lay = {}
            for kind in ("k", "v"):
                qd = gen.quantise_q4(t[kind + sfx], kind)
                lay[kind + "_codes"] = gen.to_paged(qd["codes"], self.block_table, self.ps, self.n_pages)
                if kind == "k":
                    pm = torch.zeros(self.n_pages, self.H, 128, 2, dtype=torch.float16, device=self.dev)
                    pm[btl[ok]] = qd["meta"][ok]
                else:
                    pm = gen.to_paged(qd["meta"].reshape(self.B, self.S, self.H, 8), self.block_table, self.ps, self.n_pages)
                lay[kind + "_meta"] = pm.contiguous()
            out[sfx] = lay
        return out

    def batch(self, decode: bool):
        mx = self.max_prefill + (self.steps + 1 if decode else 0)
        return self.mc.Batch(self.block_table, self.seq_lens, mx, self.n_pages)

    # -- phases ---------------------------------------------------------------------------------
    def merge_all(self):
        self.seq_lens.copy_(self.seq0)
        self.step_dev.zero_()
        b = self.batch(False)
        if not self.q4 and not self.q4cache:
            # Algorithm 1's loop over the merged layers as one call: the pairs share four launches per group of 8
            self.lib.mc_merge_pairs(self.cfg, b, self.pools, self.pairs, True, self.ws_merge)
            self.launches += 4 * ((self.wl.n_pairs + 7) // 8)  # init, merge, count(+scan), compact
            return
        for pr in range(self.wl.n_pairs):
            pl = self.pools[pr]
            if self.q4:
                self.lib.mc_merge_pair_q4(self.cfg, b, pl["_lm1"], pl["_l"], self.pairs[pr], True, self.ws_merge)
                continue
            self.lib.mc_merge_pair(self.cfg, b, pl["k_lm1"], pl["v_lm1"], pl["k_l"], pl["v_l"], self.pairs[pr], True,
                                   self.ws_merge)
        self.launches += (5 if self.q4cache else 4) * self.wl.n_pairs  # init, merge, count(+scan), compact (, quantise)

    def restore_all(self):
        b = self.batch(False)
        for pr in range(self.wl.n_pairs):
            for layer in (0, 1):
                self.lib.mc_restore(self.cfg, b, self.pairs[pr], layer, self.dst_k, self.dst_v)
        self.launches += 2 * self.wl.n_pairs  # one kernel per layer

    def decode_all(self, sample_events: bool = False, steps=None):
        b = self.batch(True)
        steps = self.steps if steps is None else steps
        for s in range(steps):
            q, nt = self.q[s % len(self.q)], self.new[s % len(self.new)]
            for pr in range(self.wl.n_pairs):
                pc = self.pairs[pr]
                # sampled: one event pair around the pair's two attention calls (an event between two
                # kernels keeps the second from starting under the first one's tail, as it does otherwise)
                ev = sample_events and ((s * self.wl.n_pairs + pr) % 16 == 0)
                if ev:
                    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                    e0.record()
                # layer l-1, then layer l with the step's append folded into the same call (it rides on the
                # attention's combine launch; with a 4-bit cache it is a launch of its own)
                self.lib.mc_decode_attn(self.cfg, b, pc, 0, q[0], nt["k_lm1"], nt["v_lm1"], self.sm_scale, self.out, None,
                                        self.ws_attn)
                self.lib.mc_decode_attn_append(self.cfg, b, pc, 1, q[1], nt["k_l"], nt["v_l"], self.sm_scale, self.out, None,
                                               nt["k_lm1"], nt["v_lm1"], nt["k_l"], nt["v_l"], self.ws_attn)
                if ev:
                    e1.record()
                    self.attn_events.append((e0, e1, s))
            self._advance()
        self.launches += steps * self.wl.n_pairs * (5 if self.q4cache else 4)

    def capture_decode_step(self):
        """One decode step (every pair: attention of both layers, append; then the lengths grow by one)
        as a CUDA graph: the kernels' programmatic dependencies become graph edges and the host issues
        one launch per step."""
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):  # once outside capture: lazy one-time set-up must not be captured
            self.decode_all(steps=1)
        torch.cuda.current_stream().wait_stream(side)
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g):
            self.decode_all(steps=1)
        return g

    def decode_pair_all(self, steps):
        """Pair mode: both layers of a pair in one call (two query sets, one pass over the directions)."""
        if steps == 0 or not hasattr(self, "ws_attn2"):  # steps == 0: set up the buffers only (outside any timed region)
            bd = self.batch(True)
            self.ws_attn2 = torch.empty(self.lib.mc_workspace_bytes(self.cfg, bd, 1, 2), dtype=torch.uint8, device=self.dev)
            self.out2 = torch.empty(2, self.B, self.Hq, 128, dtype=self.cfg.torch_dtype, device=self.dev)
            self.new2 = [{"k": torch.stack([nt["k_lm1"], nt["k_l"]]).contiguous(),
                          "v": torch.stack([nt["v_lm1"], nt["v_l"]]).contiguous()} for nt in self.new]
        b = self.batch(True)
        for s in range(steps):
            q, nt, n2 = self.q[s % len(self.q)], self.new[s % len(self.new)], self.new2[s % len(self.new)]
            for pr in range(self.wl.n_pairs):
                pc = self.pairs[pr]
                self.lib.mc_decode_attn_append(self.cfg, b, pc, 2, q, n2["k"], n2["v"], self.sm_scale, self.out2, None,
                                               nt["k_lm1"], nt["v_lm1"], nt["k_l"], nt["v_l"], self.ws_attn2)
            self._advance()

    def _advance(self):
        """End of a decode step, on the device: every live sequence grows by one token, a sequence that
        has generated its share leaves (length 0)."""
        self.seq_lens += 1
        if self.wl.ragged:
            self.step_dev += 1
            self.seq_lens.mul_((self.gen_dev > self.step_dev).to(torch.int32))

    def live_token_heads(self, s: int) -> int:
        """(token, kv head) rows attended at decode step s (0-based): the live sequences' prompt + s."""
        live = self.gen_len > s
        return int((self.prompt[live].astype(np.int64) + s).sum()) * self.H

    def live_residual_heads(self, s: int) -> int:
        """4-bit cache: the rows of step s that still sit in 16 bits (the last, incomplete page of each live sequence)."""
        live = self.gen_len > s
        return int(((self.prompt[live].astype(np.int64) + s) % 32).sum()) * self.H

    def attn_row_bytes(self, th: int, th_res: int, rho: float) -> float:
        """Algorithmic bytes of one layer's attention over th (token, head) rows, th_res of them residual."""
        if not self.q4cache:
            return th * (2 * ROW + 8 + 2 * rho * (ROW + 4))
        q4row = 64 + 16  # codes + the row's share of the group parameters
        return (th - th_res) * (2 * q4row + 8) + th_res * (2 * ROW + 8) + th * 2 * rho * (ROW + 4)

    def step(self, sample_events=False):
        self.merge_all()
        self.restore_all()
        self.decode_all(sample_events)

    # -- accounting -----------------------------------------------------------------------------
    def retained_fraction(self):
        tot = sum(int(pc.ret_count.sum().item()) for pc in self.pairs)
        return tot / max(1, 2 * self.tok_heads * self.wl.n_pairs)

    def bytes_per_step(self, rho: float):
        th, npairs, steps = self.tok_heads, self.wl.n_pairs, self.steps
        in_row = 64 + 16 if self.q4 else ROW  # 4-bit codes + the row's share of the group meta
        e_row = 64 + 16 if self.q4cache else ROW  # what a direction row occupies in the shared cache
        merge = npairs * 2 * th * (2 * in_row + e_row + 12 + 4 + rho * (2 * in_row + 2 * ROW + 4))
        restore = npairs * 2 * 2 * th * (e_row + ROW + 4 + rho * 2 * ROW)
        # decode: every live sequence grows by one token per step
        attn = npairs * 2 * sum(self.attn_row_bytes(self.live_token_heads(s), self.live_residual_heads(s), rho) for s in range(steps))
        # 4-bit cache: a row is read once more (16 bits) and written in 4 bits when its page completes
        append = npairs * 2 * int(np.minimum(self.gen_len, steps).sum()) * self.H * (3 * ROW + 12 + ((ROW + 80) if self.q4cache else 0))
        return {"merge": merge, "restore": restore, "attn": attn, "append": append}

    def attn_bytes_at(self, s: int, rho: float):
        return self.attn_row_bytes(self.live_token_heads(s), self.live_residual_heads(s), rho)


def max_over_ranks(seconds: float, dist, device) -> float:
    """The slowest rank's time: what a job of independent replicas takes (`dist` None = one rank)."""
    if dist is None:
        return seconds
    tt = torch.tensor([seconds], dtype=torch.float64, device=device)
    dist.all_reduce(tt, op=dist.ReduceOp.MAX)
    return float(tt.item())


def whole_job_gbps(bytes_per_step_per_rank: float, steps: int, seconds: float, world: int) -> float:
    """Weak scaling: every rank runs the same workload on its own data; all ranks' bytes over the
    slowest rank's time."""
    return world * bytes_per_step_per_rank * steps / seconds / 1e9


def timed(fn, stream_sync=True):
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    e0.record()
    fn()
    e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) * 1e-3


# ---------------------------------------------------------------------------------------------
def oracle_sample(wl: gen.WorkloadConfig, sample_tokens: int):
    """The oracle, as it stands, on a bounded slice of the workload (one sequence slice, all
    kv heads, K and V of one pair): merge, restore of both layers, attention for every q head.
    Returns (algorithmic bytes of the slice, seconds)."""
    from oracle import minicache_oracle as orc
    sub = dataclasses.replace(wl, batch=1, seq_len=sample_tokens, ragged=False)
    t = gen.make_pair_tensors(sub, 0)
    bits = {k: gen.as_bits(v) for k, v in t.items()}
    q = gen.as_bits(gen.make_queries(sub, 0, n_sets=1))[0, 0]
    nq = wl.n_q_heads // wl.n_kv_heads
    t0 = time.perf_counter()
    om = {tn: orc.merge_pair(bits[tn + "_lm1"], bits[tn + "_l"], [sample_tokens], wl.dtype, wl.t, wl.gamma)
          for tn in ("k", "v")}
    kept = 0
    for layer, nm, src in ((0, "n_lm1", "_lm1"), (1, "n_l", "_l")):
        for h in range(wl.n_kv_heads):
            ik, iv = om["k"]["retained"][(0, h)], om["v"]["retained"][(0, h)]
            kept += len(ik) + len(iv)
            kh = orc.restore(om["k"]["e_bits"][0, :, h], om["k"][nm][0, :, h], wl.dtype, ik, bits["k" + src][0, ik, h])
            vh = orc.restore(om["v"]["e_bits"][0, :, h], om["v"][nm][0, :, h], wl.dtype, iv, bits["v" + src][0, iv, h])
            for j in range(nq):
                orc.attention(orc.decode_bits(q[h * nq + j], wl.dtype), kh, vh, 1.0 / math.sqrt(128.0))
    dt = time.perf_counter() - t0
    th = sample_tokens * wl.n_kv_heads
    rho = kept / (4.0 * th)
    nbytes = 2 * th * (3 * ROW + 16 + rho * (4 * ROW + 4)) + 2 * 2 * th * (2 * ROW + 4 + rho * 2 * ROW) + \
        2 * th * (2 * ROW + 8 + 2 * rho * (ROW + 4))
    return nbytes, dt


def oracle_threads() -> int:
    """Threads the oracle computes with: it is one process of numpy element-wise operations and reductions, which
    run on one thread (its few matrix-vector products are too small for the BLAS pool to matter)."""
    return 1


def oracle_merge_sample(wl: gen.WorkloadConfig, tokens: int):
    """The oracle's merge alone on `tokens` x kv heads x {K, V} row pairs (one sequence slice)."""
    from oracle import minicache_oracle as orc
    sub = dataclasses.replace(wl, batch=1, seq_len=tokens, ragged=False)
    t = gen.make_pair_tensors(sub, 0)
    bits = {k: gen.as_bits(v) for k, v in t.items()}
    del t
    t0 = time.perf_counter()
    for tn in ("k", "v"):
        orc.merge_pair(bits[tn + "_lm1"], bits[tn + "_l"], [tokens], wl.dtype, wl.t, wl.gamma)
    dt = time.perf_counter() - t0
    return 2 * tokens * wl.n_kv_heads * (3 * ROW + 16), dt


def run_reference(args, wl):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    cores = oracle_threads()
    sample = min(wl.seq_len, 2048)
    for _ in range(args.warmup):
        oracle_sample(wl, min(sample, 256))
    tb, tt = 0.0, 0.0
    for _ in range(args.steps):
        nb, dt = oracle_sample(wl, sample)
        tb += nb
        tt += dt
    val = tb / tt / 1e9
    desc = f"1 sequence slice of {sample} tokens x {wl.n_kv_heads} kv heads, K and V of one pair: merge + restore(2 layers) + attention(all q heads)"
    line = {"impl": "reference", "metric": "hbm_gbps_merge_restore_decode_attn", "value": val, "unit": "GB/s",
            "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup, "ms_per_step": tt / args.steps * 1e3,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": wl.name, "sample": desc},
            "cpu_baseline": {"value": val, "unit": "GB/s", "cores": cores, "kind": "oracle", "sample": desc},
            "e2e": {"value": val, "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line))


# ---------------------------------------------------------------------------------------------
def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=3)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="c2")
    ap.add_argument("--decode-steps", type=int, default=None, help="override the workload's decode steps")
    ap.add_argument("--page-size", type=int, default=None, help="override the workload's page size")
    ap.add_argument("--gamma", type=float, default=None, help="override the retention threshold of Eq. 4")
    ap.add_argument("--outlier-frac", type=float, default=None, help="override the fraction of outlier tokens in the inputs")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--q4", action="store_true", help="the layers arrive in 4 bits (page size 32; no host-buffer leg)")
    ap.add_argument("--q4cache", action="store_true", help="the shared cache is 4-bit (page size 32): restore and attention read codes")
    ap.add_argument("--prefill-fused", action="store_true",
                    help="one pair: the merge fused into layer l's K/V projection (tensor cores) against projection + merge")
    ap.add_argument("--d-model", type=int, default=4096, help="hidden size of the stand-in projection (--prefill-fused)")
    ap.add_argument("--refill", action="store_true",
                    help="serving trace: a seeded list of 8 x batch sequences, a slot is refilled when its sequence leaves, "
                         "the admitted sequence is merged on a second stream while the others decode")
    args = ap.parse_args()
    wl = gen.CONFIGS[args.workload]
    if args.decode_steps is not None:
        wl = dataclasses.replace(wl, decode_steps=args.decode_steps)
    if args.page_size is not None:
        wl = dataclasses.replace(wl, page_size=args.page_size)
    if args.gamma is not None:
        wl = dataclasses.replace(wl, gamma=args.gamma)
    if args.outlier_frac is not None:
        wl = dataclasses.replace(wl, outlier_frac=args.outlier_frac)
    if args.impl == "reference":
        run_reference(args, wl)
        return

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the hot path has no CPU fallback")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)
    from paper_2405_14366_b200.build import build_library
    if rank == 0:
        build_library()
    if dist is not None:
        dist.barrier()

    if args.refill:
        run_refill(args, wl, dev, rank, world, dist)
        return
    if args.prefill_fused:
        run_prefill_fused(args, wl, dev)
        return
    job = Job(wl, dev, q4=args.q4, q4cache=args.q4cache)
    if args.q4:
        args.no_e2e = True  # the host-buffer entry points take 16-bit layers only
    warm = max(3, args.warmup)
    sampler = None
    for i in range(warm):
        if i == warm - 1 and rank == 0:
            sampler = ClockSampler(local)  # started one step early: nvidia-smi takes a moment to begin sampling
        job.step()
    torch.cuda.synchronize()
    rho = job.retained_fraction()
    for pc in job.pairs:
        words, code = job.lib.mc_read_status(pc, check=False)
        if code != 0:
            raise SystemExit(f"device status {words} after warm-up")

    # ---- device-resident timed region: exactly K steps ----------------------------------------
    job.launches = 0
    job.attn_events = []
    if dist is not None:
        dist.barrier()
    t_total = timed(lambda: [job.step(sample_events=True) for _ in range(args.steps)])
    t_total = max_over_ranks(t_total, dist, dev)
    clocks = sampler.stop() if sampler else None
    launches = job.launches
    by = job.bytes_per_step(rho)
    bytes_step = sum(by.values())
    value = whole_job_gbps(bytes_step, args.steps, t_total, world)

    # dominant kernel: split attention (+ its small combine), sampled with CUDA events in the timed region
    ev_ms = [(e0.elapsed_time(e1) / 2.0, s) for e0, e1, s in job.attn_events]  # two calls per event pair
    attn_bytes = np.mean([job.attn_bytes_at(s, rho) for _, s in ev_ms])
    attn_ms = float(np.mean([m for m, _ in ev_ms]))
    peak, peak_src = measured_hbm_peak()
    achieved = attn_bytes / (attn_ms * 1e-3) / 1e9
    roofline = {"kernel": ("attn_split_kernel<4-bit tiles>" if args.q4cache else "attn_split_kernel") + " (+attn_combine_kernel)", "bound": "hbm", "achieved": achieved,
                "peak": peak, "unit": "GB/s", "frac": achieved / peak, "frac_of_nominal_8000": achieved / 8000.0,
                "peak_source": peak_src,
                "traffic": (float(attn_bytes) * ATTN_TRAFFIC_RATIO if ATTN_TRAFFIC_RATIO and wl.name.startswith("c2") and not args.q4cache else None), "launch_ms": attn_ms, "launches_timed": 2 * len(ev_ms),
                "algorithmic_bytes_per_launch": float(attn_bytes)}

    # ---- per-phase breakdown (outside the headline region) ----------------------------------------
    phases = {}

    def median_time(fn, reps=5):  # (the SM clock under the power cap moves between calls: the middle of five)
        return float(np.median([timed(fn) for _ in range(reps)]))
    t_m = median_time(job.merge_all)
    phases["merge"] = {"ms": t_m * 1e3, "GB/s": by["merge"] / t_m / 1e9,
                       "kv_tokens_per_s": float(job.prompt.sum()) * 2 * wl.n_pairs / t_m}
    t_r = median_time(job.restore_all)
    phases["restore"] = {"ms": t_r * 1e3, "GB/s": by["restore"] / t_r / 1e9}
    t_d = timed(job.decode_all)
    tok_steps = sum(job.live_token_heads(s) for s in range(job.steps)) / job.H
    phases["decode"] = {"ms": t_d * 1e3, "GB/s": (by["attn"] + by["append"]) / t_d / 1e9,
                        "kv_tokens_per_s": tok_steps * 2 * wl.n_pairs / t_d, "ms_per_decode_step": t_d * 1e3 / job.steps}
    # the same decode phase replayed from a CUDA graph of one decode step (valid for any step: the
    # lengths live on the device and grow inside the graph)
    job.merge_all()
    graph = job.capture_decode_step()
    job.merge_all()
    for _ in range(2):
        graph.replay()
    job.merge_all()
    t_g = timed(lambda: [graph.replay() for _ in range(job.steps)])
    phases["decode_cuda_graph"] = {"ms": t_g * 1e3, "GB/s": (by["attn"] + by["append"]) / t_g / 1e9,
                                   "kv_tokens_per_s": tok_steps * 2 * wl.n_pairs / t_g, "ms_per_decode_step": t_g * 1e3 / job.steps}
    if 2 * (wl.n_q_heads // wl.n_kv_heads) <= 8:
        # pair mode (both layers' queries known up front: a replay or speculative setting, not a real
        # model's layer-by-layer decode): the shared directions are read once for two layers
        job.decode_pair_all(0)
        job.merge_all()
        psteps = min(job.steps, 64)
        job.decode_pair_all(min(2, psteps))  # warm-up
        job.merge_all()
        t_p = timed(lambda: job.decode_pair_all(psteps))
        th_steps = sum(job.live_token_heads(s) for s in range(psteps))
        if args.q4cache:
            pair_bytes = wl.n_pairs * sum(job.attn_row_bytes(job.live_token_heads(s), job.live_residual_heads(s), 2 * rho) + 8 * job.live_token_heads(s)
                                          for s in range(psteps)) + by["append"] * psteps / job.steps
        else:
            pair_bytes = wl.n_pairs * th_steps * (2 * ROW + 16 + 4 * rho * (ROW + 4)) + by["append"] * psteps / job.steps
        phases["decode_pair_mode"] = {"ms_per_decode_step": t_p * 1e3 / psteps, "GB/s": pair_bytes / t_p / 1e9,
                                      "kv_tokens_per_s": (th_steps / job.H)
                                      * 2 * wl.n_pairs / t_p, "steps": psteps}
    peak0, _ = measured_hbm_peak()
    for ph in phases.values():
        ph["frac_of_measured_hbm"] = ph["GB/s"] / peak0
        ph["frac_of_nominal_8000"] = ph["GB/s"] / 8000.0

    # ---- end to end: host buffers, copies inside the timed region ----------------------------------
    e2e = None
    if not args.no_e2e:
        e2e = run_e2e(job, wl, rho, args, dist, dev, world)

    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        cores = oracle_threads()
        sample = min(wl.seq_len, 2048)
        oracle_sample(wl, 128)
        nb, dt = oracle_sample(wl, sample)
        # the merge part on 2^20 row pairs (tokens x kv heads x {K, V}), in slices the host's memory takes easily
        m_tok = (1 << 20) // (2 * wl.n_kv_heads)
        m_slice = min(m_tok, 4096)
        mb, mt = 0.0, 0.0
        for _ in range(m_tok // m_slice):
            b2, t2 = oracle_merge_sample(wl, m_slice)
            mb, mt = mb + b2, mt + t2
        cpu = {"value": (nb + mb) / (dt + mt) / 1e9, "unit": "GB/s", "cores": cores, "kind": "oracle",
               "merge_only_GB/s": mb / mt / 1e9,
               "sample": f"single-process numpy fp64 oracle: merge of 2^20 row pairs ({m_tok} tokens x {wl.n_kv_heads} kv heads x K,V; "
                         f"{mt:.1f} s) + one slice of {sample} tokens x {wl.n_kv_heads} kv heads through merge, restore of both "
                         f"layers and attention of all q heads ({dt:.1f} s)"}

    if rank == 0:
        line = {"metric": "hbm_gbps_merge_restore_decode_attn", "value": value, "unit": "GB/s", "n_gpus": world,
                "steps": args.steps, "warmup": warm, "ms_per_step": t_total / args.steps * 1e3,
                "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
                "config": {"workload": wl.name, "batch": wl.batch, "seq_len": wl.seq_len, "kv_heads": wl.n_kv_heads,
                           "q_heads": wl.n_q_heads, "storage": wl.dtype, "shared_cache": "4-bit (groups of 32) + 16-bit residual page" if args.q4cache else wl.dtype, "input_layers": "4-bit, de-quantised in the merge" if args.q4 else wl.dtype, "page_size": wl.page_size,
                           "pairs": wl.n_pairs, "decode_steps": wl.decode_steps, "t": wl.t, "gamma": wl.gamma,
                           "retained_fraction": rho, "attention_mode": "single-layer calls (2 per pair per step)",
                           "l2": "inputs larger than L2: every launch streams >= 0.5 GB"},
                "kv_tokens_per_s": {"merge": phases["merge"]["kv_tokens_per_s"], "decode": phases["decode"]["kv_tokens_per_s"]},
                "phases": phases, "bytes_per_step": by, "roofline": roofline, "cpu_baseline": cpu, "e2e": e2e,
                "gpu_launches": launches, "clocks": clocks}
        print(json.dumps(line))
    if dist is not None:
        dist.barrier()
        dist.destroy_process_group()


def run_prefill_fused(args, wl, dev):
    """One layer pair: layer l's K/V come out of a projection X W^T.  Fused: mc_prefill_merge_pair (the rows are
    merged in the projection's epilogue and never stored, except those above the distance hint).  Unfused: a
    library GEMM writes layer l's rows, mc_merge_pair reads them back.  Reports both times and the cache traffic."""
    import paper_2405_14366_b200 as mc
    lib = mc.lib()
    B, S, H = wl.batch, wl.seq_len, wl.n_kv_heads
    stride = (S + 127) // 128 * 128
    case = gen.make_projection_case(wl, 0, args.d_model, stride, device=dev)
    bt, n_pages = gen.make_block_table(np.full(B, S + 1), wl.page_size, seed=4321 + wl.index)
    block_table = torch.from_numpy(bt).to(dev)
    seq_lens = torch.full((B,), S, dtype=torch.int32, device=dev)
    cfg = mc.McConfig(H, wl.n_q_heads, wl.page_size, wl.dtype, t=wl.t, gamma=wl.gamma)
    batch = mc.Batch(block_table, seq_lens, S, n_pages)
    pools = {k: gen.to_paged(case[k][:, :S], block_table, wl.page_size, n_pages) for k in ("k_lm1", "v_lm1")}
    pools["k_l"] = torch.zeros_like(pools["k_lm1"])
    pools["v_l"] = torch.zeros_like(pools["k_lm1"])
    del case["k_lm1"], case["v_lm1"], case["k_ref"], case["v_ref"]
    th = B * S * H
    pair = mc.PairCache(cfg, B, n_pages, int(0.2 * th) + 1024, device=dev)
    ws = torch.empty(lib.mc_workspace_bytes(cfg, batch, 0, 1), dtype=torch.uint8, device=dev)
    hint = 0.3
    fused = lambda: lib.mc_prefill_merge_pair(cfg, batch, case["x"], case["w_k"], case["w_v"], pools["k_lm1"], pools["v_lm1"],
                                              pools["k_l"], pools["v_l"], pair, hint, True, ws)
    x2 = case["x"].reshape(B * stride, args.d_model)
    ck = torch.empty(B * stride, H * 128, dtype=x2.dtype, device=dev)
    cv = torch.empty_like(ck)
    gemms = lambda: (torch.matmul(x2, case["w_k"].T, out=ck), torch.matmul(x2, case["w_v"].T, out=cv))
    merge = lambda: lib.mc_merge_pair(cfg, batch, pools["k_lm1"], pools["v_lm1"], pools["k_l"], pools["v_l"], pair, True, ws)
    for _ in range(3):
        fused()
        gemms()
    torch.cuda.synchronize()
    med = lambda fn: float(np.median([timed(fn) for _ in range(5)]))
    t_f = med(fused)
    words, code = lib.mc_read_status(pair, check=False)
    if code != 0:
        raise SystemExit(f"device status {words}")
    rho = int(pair.ret_count.sum().item()) / (2.0 * th)
    stored = float((pair.dist > hint).float().sum().item()) / (2.0 * th)  # layer l's rows that were stored raw
    t_g = med(gemms)
    # the unfused merge needs all of layer l's rows in the pools: the fused call with a negative hint puts them there
    lib.mc_prefill_merge_pair(cfg, batch, case["x"], case["w_k"], case["w_v"], pools["k_lm1"], pools["v_lm1"], pools["k_l"],
                              pools["v_l"], pair, -1.0, True, ws)
    merge()
    t_m = med(merge)
    flops = 2.0 * B * stride * args.d_model * (2 * H * 128)
    kv_bytes_fused = 2 * th * (ROW + ROW + 12 + 4 + stored * ROW + rho * (4 * ROW + 4))   # layer l-1 read, E written (+ stored rows)
    kv_bytes_unfused = 2 * th * (ROW + 2 * ROW + ROW + 12 + 4 + rho * (4 * ROW + 4))         # + layer l written, then read
    line = {"metric": "hbm_gbps_merge_restore_decode_attn", "value": kv_bytes_fused / t_f / 1e9, "unit": "GB/s", "n_gpus": 1, "steps": 5,
            "warmup": 3, "ms_per_step": t_f * 1e3, "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32",
            "data": "synthetic",
            "config": {"workload": wl.name + " one pair, merge fused into the K/V projection", "batch": B, "seq_len": S, "kv_heads": H,
                       "d_model": args.d_model, "storage": wl.dtype, "distance_hint": hint},
            "prefill_fused": {"fused_ms": t_f * 1e3, "gemm_tflops_fused": flops / t_f / 1e12,
                              "library_gemm_ms": t_g * 1e3, "library_gemm_tflops": flops / t_g / 1e12, "merge_ms": t_m * 1e3,
                              "unfused_ms": (t_g + t_m) * 1e3, "retained_fraction": rho, "rows_stored_fraction": stored,
                              "cache_bytes_per_unit_fused": kv_bytes_fused / (2 * th), "cache_bytes_per_unit_unfused": kv_bytes_unfused / (2 * th)},
            "gpu_launches": 4}
    print(json.dumps(line))


def run_refill(args, wl, dev, rank, world, dist):
    """The serving mix with slot refill (the paper's efficiency experiment, Sec. 5, gets its throughput from
    the live batch): 8 x batch sequences with seeded prompt and generation lengths wait in a list; the
    batch's slots start with the first ones; every decode step attends both layers of every pair for every
    live slot and appends the new token; a slot whose sequence has generated its share is handed the next
    sequence of the list, whose pairs are merged by mc_admit_sequences on a second stream while the decode
    steps go on, and joins the batch (its length becomes visible to the decode calls) once that merge has run.
    The decode step is replayed from a CUDA graph; the host keeps two steps in flight.
    The timed window ends when the list is used up and the first slot finds nothing to be refilled with (the
    steady state of a server with a queue; the drain after it is what the plain benchmark of this workload times)."""
    n_list = 8 * wl.batch
    prompts, gens = gen.make_lengths(dataclasses.replace(wl, batch=n_list))
    job = Job(wl, dev, q4=args.q4, q4cache=args.q4cache, serving=True)
    lib, B, H = job.lib, job.B, job.H
    max_len = wl.seq_len + wl.decode_steps + 1
    bd = job.mc.Batch(job.block_table, job.seq_lens, max_len, job.n_pages)
    adm_lens = torch.zeros(B, dtype=torch.int32, device=dev)
    badm = job.mc.Batch(job.block_table, adm_lens, wl.seq_len, job.n_pages)
    ws1 = lib.mc_workspace_bytes(job.cfg, badm, 0, 1)
    ws16 = lib.mc_workspace_bytes(dataclasses.replace(job.cfg, cache_bits=16), badm, 0, 1)
    # per pair the retention tables; the 16-bit staging tiles of a 4-bit cache once (the pairs take turns)
    ws_adm = torch.empty(wl.n_pairs * ws16 + (ws1 - ws16), dtype=torch.uint8, device=dev)
    # the admissions' stream has priority: the decode chain always has a kernel waiting for the SMs a finishing
    # kernel frees, and a stream of equal priority would get them only rarely
    main_s, side_s = torch.cuda.current_stream(), torch.cuda.Stream(priority=-1)
    remaining = torch.zeros(B, dtype=torch.int32, device=dev)  # tokens each slot's sequence has still to generate

    def admit(slots, seqs, stream):
        """Merge sequence seqs[i] into slot slots[i] (a run of neighbouring slots) on `stream`."""
        with torch.cuda.stream(stream):
            adm_lens[slots[0]:slots[0] + len(slots)] = torch.from_numpy(prompts[seqs].astype(np.int32)).to(dev, non_blocking=True)
            lib.mc_admit_sequences(job.cfg, badm, slots[0], len(slots), job.pools, job.pairs, job.rows_per_seq, True, ws_adm,
                                   stream=stream, q4=args.q4)

    def decode_step():
        q, nt = job.q[0], job.new[0]
        for pr in range(wl.n_pairs):
            pc = job.pairs[pr]
            lib.mc_decode_attn(job.cfg, bd, pc, 0, q[0], nt["k_lm1"], nt["v_lm1"], job.sm_scale, job.out, None, job.ws_attn)
            lib.mc_decode_attn_append(job.cfg, bd, pc, 1, q[1], nt["k_l"], nt["v_l"], job.sm_scale, job.out, None,
                                      nt["k_lm1"], nt["v_lm1"], nt["k_l"], nt["v_l"], job.ws_attn)
        # end of the step, on the device: live slots grow by one token; a slot that has generated its share empties
        live = (remaining > 0).to(torch.int32)
        job.seq_lens.add_(live)
        remaining.sub_(live)
        job.seq_lens.mul_((remaining > 0).to(torch.int32))

    def serve(max_steps):
        """Returns (steps, generated tokens, sum over steps of live (token, head) rows, steps at full batch, residual rows)."""
        job.seq_lens.zero_()
        remaining.zero_()
        side_s.wait_stream(main_s)
        admit(list(range(B)), np.arange(B), main_s)
        job.seq_lens.copy_(adm_lens)
        remaining.copy_(torch.from_numpy(gens[:B].astype(np.int32)).to(dev))
        h_len = prompts[:B].astype(np.int64).copy()      # host mirror of the slots
        h_rem = gens[:B].astype(np.int64).copy()
        nxt, pending = B, []                              # next sequence of the list; admissions in flight
        steps = tokens = th_sum = full = th_res = 0
        in_flight = []  # the host stays at most two decode steps ahead of the device (a server reads every step's
                        # tokens anyway); further ahead, an admitted sequence would join that many steps late
        while steps < max_steps and (h_rem.max() > 0 or pending):
            # admissions that have run join the batch
            still = []
            for slot, j, ev in pending:
                if ev.query():
                    main_s.wait_event(ev)
                    job.seq_lens[slot:slot + 1].fill_(int(prompts[j]))
                    remaining[slot:slot + 1].fill_(int(gens[j]))
                    h_len[slot], h_rem[slot] = prompts[j], gens[j]
                else:
                    still.append((slot, j, ev))
            pending = still
            livem = h_rem > 0
            if livem.any():
                graph.replay()
                ev_done = torch.cuda.Event()
                ev_done.record(main_s)
                in_flight.append(ev_done)
                if len(in_flight) > 2:
                    in_flight.pop(0).synchronize()
                steps += 1
                tokens += int(livem.sum())
                th_sum += int(h_len[livem].sum()) * H
                th_res += int((h_len[livem] % 32).sum()) * H
                full += int(livem.all())
                h_len[livem] += 1
                h_rem[livem] -= 1
                done = livem & (h_rem == 0)
                h_len[done] = 0
                if done.any() and nxt >= n_list:
                    break  # the queue is empty: the steady state ends here
                if done.any():
                    ev_step = ev_done
                    for slot in np.nonzero(done)[0]:
                        if nxt >= n_list:
                            break
                        side_s.wait_event(ev_step)  # the slot's last decode step has run
                        admit([int(slot)], np.array([nxt]), side_s)
                        ev = torch.cuda.Event()
                        ev.record(side_s)
                        pending.append((int(slot), nxt, ev))
                        nxt += 1
            else:
                pending[0][2].synchronize()  # nothing to decode until an admission lands
        main_s.wait_stream(side_s)
        return steps, tokens, th_sum, full, th_res, nxt

    # warm-up: set-up calls outside capture, then the decode step as a graph
    admit(list(range(B)), np.arange(B), main_s)
    job.seq_lens.copy_(adm_lens)
    remaining.fill_(4)
    side = torch.cuda.Stream()
    side.wait_stream(main_s)
    with torch.cuda.stream(side):
        decode_step()
    main_s.wait_stream(side)
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        decode_step()
    torch.cuda.synchronize()
    max_steps = args.decode_steps if args.decode_steps is not None else 10 ** 9
    serve(min(max_steps, 32))
    torch.cuda.synchronize()
    sampler = ClockSampler(torch.cuda.current_device()) if rank == 0 else None
    if dist is not None:
        dist.barrier()
    res = []
    t = timed(lambda: res.append(serve(max_steps)))
    t = max_over_ranks(t, dist, dev)
    clocks = sampler.stop() if sampler else None
    steps, tokens, th_sum, full, th_res, admitted = res[0]
    for pc in job.pairs:
        words, code = lib.mc_read_status(pc, check=False)
        if code != 0:
            raise SystemExit(f"device status {words} after the serving trace")
    rho = 0.004  # retained fraction of this workload's recipe (measured by the drained runs)
    attn_bytes = wl.n_pairs * 2 * job.attn_row_bytes(th_sum, th_res, rho)
    append_bytes = wl.n_pairs * 2 * tokens * H * (3 * ROW + 12 + ((ROW + 80) if args.q4cache else 0))
    in_row = 64 + 16 if args.q4 else ROW
    e_row = 64 + 16 if args.q4cache else ROW
    adm_th = int(prompts[:admitted].sum()) * H
    merge_bytes = wl.n_pairs * 2 * adm_th * (2 * in_row + e_row + 16)
    value = world * (attn_bytes + append_bytes + merge_bytes) / t / 1e9
    peak, peak_src = measured_hbm_peak()
    if rank == 0:
        line = {"metric": "hbm_gbps_merge_restore_decode_attn", "value": value, "unit": "GB/s", "n_gpus": world, "steps": 1,
                "warmup": 1, "ms_per_step": t * 1e3, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
                "dtype": "f32", "data": "synthetic",
                "config": {"workload": wl.name + " serving trace with slot refill", "slots": B, "sequences_in_list": n_list,
                           "sequences_admitted": admitted, "kv_heads": H, "storage": wl.dtype,
                           "shared_cache": "4-bit" if args.q4cache else wl.dtype,
                           "input_layers": "4-bit" if args.q4 else wl.dtype, "page_size": wl.page_size, "pairs": wl.n_pairs},
                "serving": {"decode_steps": steps, "generated_tokens": world * tokens, "served_tokens_per_s": world * tokens / t,
                            "ms_per_decode_step": t * 1e3 / max(steps, 1), "mean_live_slots": tokens / max(steps, 1),
                            "fraction_of_steps_at_full_batch": full / max(steps, 1),
                            "decode_GB/s": world * (attn_bytes + append_bytes) / t / 1e9,
                            "frac_of_measured_hbm": value / world / peak, "admission_merge_bytes": merge_bytes},
                "gpu_launches": steps * wl.n_pairs * (5 if args.q4cache else 4) + (admitted - B + 1) * 4, "clocks": clocks}
        print(json.dumps(line))
    if dist is not None:
        dist.barrier()
        dist.destroy_process_group()


def run_e2e(job: Job, wl, rho, args, dist, dev, world):
    """Same step with HOST buffers: every pair's four input pools start in pinned host memory and
    are copied in by mc_merge_pair_host before its merge; every attention call takes its query and
    new-token rows from pinned host memory and returns its output there (mc_decode_attn_host).
    The copies are inside the timed region."""
    lib = job.lib
    # pinned host copies of every pair's layers; with several ranks on one node the ranks share the
    # host's memory, so each keeps one pair's copy and uploads it for every pair (same bytes, same work)
    host_pools = []
    for pr, pl in enumerate(job.pools):
        if world > 1 and pr > 0:
            host_pools.append(host_pools[0])
        else:
            host_pools.append({k: torch.empty(v.shape, dtype=v.dtype, pin_memory=True).copy_(v) for k, v in pl.items()})
    stage = {k: torch.empty_like(v) for k, v in job.pools[0].items()}  # device staging the host pools land in
    pin = lambda t: torch.empty(t.shape, dtype=t.dtype, pin_memory=True).copy_(t)
    # per decode step and pair: both layers' queries [2][B][Hq][128] and new rows [2][B][H][128], pinned
    q_host = [pin(q) for q in job.q]
    kn_host = [pin(torch.stack([nt["k_lm1"], nt["k_l"]])) for nt in job.new]
    vn_host = [pin(torch.stack([nt["v_lm1"], nt["v_l"]])) for nt in job.new]
    out_host = torch.empty((2,) + tuple(job.out.shape[1:]), dtype=job.out.dtype, pin_memory=True)  # a pair's two results
    out_dev = [torch.empty((2,) + tuple(job.out.shape[1:]), dtype=job.out.dtype, device=dev) for _ in range(2)]
    bd = job.batch(True)
    io = [torch.empty(lib.mc_decode_io_bytes(job.cfg, bd, 2), dtype=torch.uint8, device=dev) for _ in range(2)]
    pool_bytes = sum(v.numel() * v.element_size() for v in job.pools[0].values())
    q_bytes = job.B * job.Hq * ROW
    n_bytes = job.B * job.H * ROW

    # Two steps in flight: while step k decodes on the main stream, a second stream already uploads and
    # merges step k + 1's layers into a second set of pair caches (a double-buffered serving loop).
    # Every copy and every kernel of every step is still issued through the host-buffer entry points
    # inside the timed region.
    pair_sets = [job.pairs, [job.mc.PairCache(job.cfg, job.B, job.n_pages, job.pairs[0].ret_capacity, device=dev)
                             for _ in range(wl.n_pairs)]]
    main_s, side_s = torch.cuda.current_stream(), torch.cuda.Stream()
    ws_merge2 = torch.empty_like(job.ws_merge)
    prefill = job.mc.Batch(job.block_table, job.seq0, job.max_prefill, job.n_pages)  # lengths the merges see
    merged = [None, None]   # events: set k % 2 holds step k's merged pairs
    decoded = [None, None]  # events: step k's decode no longer reads set k % 2

    def prepare(k):  # upload + merge + restore of step k on the side stream
        cs = pair_sets[k % 2]
        with torch.cuda.stream(side_s):
            if decoded[k % 2] is not None:
                side_s.wait_event(decoded[k % 2])
            for pr in range(wl.n_pairs):
                lib.mc_merge_pair_host(job.cfg, prefill, host_pools[pr], stage, cs[pr], True, ws_merge2, stream=side_s)
            for pr in range(wl.n_pairs):
                for layer in (0, 1):
                    lib.mc_restore(job.cfg, prefill, cs[pr], layer, job.dst_k, job.dst_v, stream=side_s)
            ev = torch.cuda.Event()
            ev.record(side_s)
            merged[k % 2] = ev

    # The inputs of a pair's two attention calls (both layers' queries and new rows, 384 KB here) are staged from
    # the pinned host buffers by mc_decode_stage_host on a third stream, one pair ahead: while an upload saturates the
    # host link such a transfer takes tens of microseconds, which a fetch inside the call would put on the critical
    # path of every call.  The results of a pair go back the same way: mc_decode_drain_host on a fourth stream, behind
    # the pair's second call (a result written to host memory by the attention itself waits on the busy link too).
    stage_s, drain_s = torch.cuda.Stream(), torch.cuda.Stream()
    staged = [torch.cuda.Event(), torch.cuda.Event()]    # io[j] holds the inputs of its pair
    consumed = [None, None]                              # io[j]'s pair has been attended
    drained = [None, None]                               # out_dev[j] has been copied to the host

    def stage_inputs(c):  # c: running index of the (decode step, pair)
        j = c % 2
        s_i = (c // wl.n_pairs) % job.steps
        with torch.cuda.stream(stage_s):
            if consumed[j] is not None:
                stage_s.wait_event(consumed[j])
            views = lib.mc_decode_stage_host(job.cfg, bd, 2, q_host[s_i % len(q_host)], kn_host[s_i % len(kn_host)],
                                             vn_host[s_i % len(vn_host)], io[j], stream=stage_s)
            staged[j].record(stage_s)
        return views

    def decode(k):  # step k's decode phase on the main stream
        cs = pair_sets[k % 2]
        main_s.wait_event(merged[k % 2])
        job.seq_lens.copy_(job.seq0)
        job.step_dev.zero_()
        c0 = k * job.steps * wl.n_pairs
        views = stage_inputs(c0)
        for s in range(job.steps):
            for pr in range(wl.n_pairs):
                c = c0 + s * wl.n_pairs + pr
                pc = cs[pr]
                qd, knd, vnd = views
                last = s == job.steps - 1 and pr == wl.n_pairs - 1
                if not last:
                    views = stage_inputs(c + 1)
                main_s.wait_event(staged[c % 2])
                if drained[c % 2] is not None:
                    main_s.wait_event(drained[c % 2])
                od = out_dev[c % 2]
                lib.mc_decode_attn(job.cfg, bd, pc, 0, qd[0], knd[0], vnd[0], job.sm_scale, od[0:1], None, job.ws_attn)
                lib.mc_decode_attn_append(job.cfg, bd, pc, 1, qd[1], knd[1], vnd[1], job.sm_scale, od[1:2], None,
                                          knd[0], vnd[0], knd[1], vnd[1], job.ws_attn)
                ev = torch.cuda.Event()
                ev.record(main_s)
                consumed[c % 2] = ev
                with torch.cuda.stream(drain_s):
                    drain_s.wait_event(ev)
                    lib.mc_decode_drain_host(job.cfg, bd, 2, od, None, out_host, None, stream=drain_s)
                    dv = torch.cuda.Event()
                    dv.record(drain_s)
                    drained[c % 2] = dv
            job._advance()
        main_s.wait_stream(drain_s)  # the step's results are on the host
        ev = torch.cuda.Event()
        ev.record(main_s)
        decoded[k % 2] = ev

    def run_steps(n):
        prepare(0)
        for k in range(n):
            if k + 1 < n:
                prepare(k + 1)
            decode(k)
        main_s.wait_stream(side_s)

    side_s.wait_stream(main_s)
    run_steps(1)
    torch.cuda.synchronize()
    if dist is not None:
        dist.barrier()
    n = max(1, args.steps)
    merged[:] = [None, None]
    decoded[:] = [None, None]
    t = timed(lambda: run_steps(n))
    t = max_over_ranks(t, dist, dev)
    by = job.bytes_per_step(rho)
    calls = job.steps * wl.n_pairs * 2
    return {"value": whole_job_gbps(sum(by.values()), n, t, world), "unit": "GB/s", "steps": n, "ms_per_step": t / n * 1e3,
            "h2d_bytes_per_step": wl.n_pairs * pool_bytes + calls * (q_bytes + 2 * n_bytes),
            "d2h_bytes_per_step": calls * q_bytes,
            "api": "mc_merge_pair_host + mc_restore + mc_decode_stage_host + mc_decode_attn + mc_decode_attn_append + "
                   "mc_decode_drain_host, pinned host buffers (a pair's inputs staged one pair ahead on a third stream, its "
                   "results copied back on a fourth); "
                   "two steps in flight (the next step's upload and merge on a second stream)"}


if __name__ == "__main__":
    main()

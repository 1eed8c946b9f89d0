"""Seeded workload recipes (MiniCache paper, Sec. 5 "Efficiency analysis" shapes).

Every tensor here is synthetic.  The row model follows the observation the
paper reports in Sec. 3.1 (Observation 1 and 2): key/value states of adjacent
middle-to-deep layers point in nearly the same direction for most tokens, with
a few outlier tokens that differ strongly.  One layer's rows are random
directions with log-normal lengths; the partner layer's rows are those
directions rotated by an angle theta towards a random orthogonal direction and
given their own independent log-normal lengths.

Nothing in this module belongs to the method itself; it only prepares inputs
that the CPU oracle and the CUDA path both consume bit for bit.
"""
from __future__ import annotations

import dataclasses
import math
from typing import Dict, Optional

import numpy as np
import torch

BASE_SEED = 0x240514366
HEAD_DIM = 128


@dataclasses.dataclass(frozen=True)
class WorkloadConfig:
    """One named workload. Layers ``start_layer .. n_layers-1`` are merged as
    adjacent pairs (start_layer, start_layer+1), ... (Sec. 4.1: S = L/2)."""

    name: str
    index: int
    n_kv_heads: int
    n_q_heads: int
    dtype: str  # "f16" | "bf16"
    batch: int
    seq_len: int  # prompt length (max prompt length when ragged)
    page_size: int
    n_layers: int = 32
    start_layer: int = 16
    t: float = 0.6
    gamma: float = 0.05
    outlier_frac: float = 0.03
    theta_mean_first: float = 0.3  # mean rotation angle of the first merged pair
    theta_mean_last: float = 0.3  # ... of the last merged pair (linear ramp between)
    decode_steps: int = 1
    ragged: bool = False
    quant4: bool = False
    head_dim: int = HEAD_DIM

    @property
    def n_pairs(self) -> int:
        return (self.n_layers - self.start_layer) // 2

    def pair_layers(self, pair: int):
        lm1 = self.start_layer + 2 * pair
        return lm1, lm1 + 1

    def theta_mean(self, pair: int) -> float:
        if self.n_pairs <= 1:
            return self.theta_mean_first
        f = pair / (self.n_pairs - 1)
        return self.theta_mean_first + f * (self.theta_mean_last - self.theta_mean_first)

    def scaled(self, name: str, **kw) -> "WorkloadConfig":
        return dataclasses.replace(self, name=name, **kw)


def _mk() -> Dict[str, WorkloadConfig]:
    c = {}
    # 1: single pair, LLaMA-2-7B head shape, batch 1, 512 tokens, fp16.
    c["c1"] = WorkloadConfig("c1", 1, 32, 32, "f16", 1, 512, 16, n_layers=2, start_layer=0,
                             outlier_frac=0.03, theta_mean_first=0.3, theta_mean_last=0.3)
    # 2: LLaMA-2-7B full cache, batch 8 x 4096 tokens, fp16, 8 pairs, 256 decode steps.
    c["c2"] = WorkloadConfig("c2", 2, 32, 32, "f16", 8, 4096, 16, outlier_frac=0.03,
                             theta_mean_first=0.3, theta_mean_last=0.7, decode_steps=256)
    # 3: LLaMA-3-8B GQA shape, bf16, batch 16 x 8192 tokens, page 16, 5 % outliers.
    c["c3"] = WorkloadConfig("c3", 3, 8, 32, "bf16", 16, 8192, 16, outlier_frac=0.05,
                             theta_mean_first=0.3, theta_mean_last=0.7, decode_steps=64)
    # 4: serving mix, ragged batch of 64, fp16 source values (4-bit variant: quant4).
    c["c4"] = WorkloadConfig("c4", 4, 32, 32, "f16", 64, 2048, 32, outlier_frac=0.03,
                             theta_mean_first=0.3, theta_mean_last=0.7, decode_steps=1024,
                             ragged=True, quant4=True)
    # 5: Mixtral-8x7B attention shape, long context, bf16, batch 4 x 32768 tokens.
    c["c5"] = WorkloadConfig("c5", 5, 8, 32, "bf16", 4, 32768, 16, outlier_frac=0.05,
                             theta_mean_first=0.4, theta_mean_last=0.4, decode_steps=128)
    # 1/16-scale replicas used by parity tests (same shapes per token, fewer tokens).
    c["c2_s"] = c["c2"].scaled("c2_s", batch=2, seq_len=1024, n_layers=20, decode_steps=4)
    c["c3_s"] = c["c3"].scaled("c3_s", batch=4, seq_len=2048, n_layers=20, decode_steps=4)
    c["c4_s"] = c["c4"].scaled("c4_s", batch=8, seq_len=512, n_layers=18, decode_steps=8)
    c["c5_s"] = c["c5"].scaled("c5_s", batch=1, seq_len=8192, n_layers=18, decode_steps=4)
    # one pair of config 2 / 3 at full batch and length (larger than L2, ~2 GB): profiler captures
    c["c2_p1"] = c["c2"].scaled("c2_p1", n_layers=18, decode_steps=2)
    c["c3_p1"] = c["c3"].scaled("c3_p1", n_layers=18, decode_steps=2)
    c["c4_p1"] = c["c4"].scaled("c4_p1", n_layers=18, decode_steps=2)
    return c


CONFIGS: Dict[str, WorkloadConfig] = _mk()


def torch_dtype(name: str) -> torch.dtype:
    return {"f16": torch.float16, "bf16": torch.bfloat16}[name]


def as_bits(x: torch.Tensor) -> np.ndarray:
    """A 16-bit float tensor as its raw uint16 bit patterns (host numpy array)."""
    assert x.dtype in (torch.float16, torch.bfloat16)
    return x.detach().contiguous().cpu().view(torch.int16).numpy().view(np.uint16)


def _seed(cfg: WorkloadConfig, pair: int, stream: int) -> int:
    return (BASE_SEED + cfg.index) * 1000003 + pair * 1009 + stream


def _rng(device, seed: int) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(seed & 0x7FFFFFFFFFFFFFFF)
    return g


def make_lengths(cfg: WorkloadConfig):
    """Prompt and generated lengths per sequence (host int32 arrays).

    Uniform configs return ``seq_len`` for every sequence.  The ragged serving
    mix draws log-normal lengths (sigma = 1) around medians 300 / 250, clipped
    to [16, seq_len] and [16, decode_steps]."""
    if not cfg.ragged:
        return (np.full(cfg.batch, cfg.seq_len, np.int32), np.full(cfg.batch, cfg.decode_steps, np.int32))
    rs = np.random.RandomState((_seed(cfg, 0, 99)) & 0x7FFFFFFF)
    prompt = np.exp(math.log(300.0) + rs.standard_normal(cfg.batch))
    gen = np.exp(math.log(250.0) + rs.standard_normal(cfg.batch))
    prompt = np.clip(np.rint(prompt), 16, cfg.seq_len).astype(np.int32)
    gen = np.clip(np.rint(gen), 16, cfg.decode_steps).astype(np.int32)
    return prompt, gen


def make_pair_tensors(cfg: WorkloadConfig, pair: int, device="cpu",
                      batch: Optional[int] = None, seq_len: Optional[int] = None,
                      keep_theta: bool = False) -> Dict[str, torch.Tensor]:
    """Logical K and V of the two layers of one merged pair.

    Returns ``k_lm1, k_l, v_lm1, v_l`` with shape [batch][seq_len][n_kv_heads][128]
    in the config's storage dtype.  ``theta_k / theta_v`` (the planted rotation
    angles, fp32) are included when ``keep_theta`` is set."""
    B = cfg.batch if batch is None else batch
    S = cfg.seq_len if seq_len is None else seq_len
    H, D = cfg.n_kv_heads, cfg.head_dim
    dt = torch_dtype(cfg.dtype)
    mu = cfg.theta_mean(pair)
    gm = _rng(device, _seed(cfg, pair, 0))
    outlier = torch.rand(B, S, generator=gm, device=device) < cfg.outlier_frac
    out: Dict[str, torch.Tensor] = {}
    for ti, name in enumerate(("k", "v")):
        g = _rng(device, _seed(cfg, pair, 1 + ti))
        x = torch.randn(B, S, H, D, generator=g, device=device, dtype=torch.float32)
        x /= x.norm(dim=-1, keepdim=True)
        nz = torch.randn(B, S, H, D, generator=g, device=device, dtype=torch.float32)
        nz -= (nz * x).sum(-1, keepdim=True) * x
        nz /= nz.norm(dim=-1, keepdim=True)
        u = torch.rand(B, S, H, generator=g, device=device, dtype=torch.float32)
        theta = torch.where(outlier[:, :, None], 1.2 + 0.8 * u, 2.0 * mu * u)
        len_l = torch.exp(0.5 * torch.randn(B, S, H, generator=g, device=device, dtype=torch.float32))
        len_lm1 = torch.exp(0.5 * torch.randn(B, S, H, generator=g, device=device, dtype=torch.float32))
        y = torch.cos(theta)[..., None] * x + torch.sin(theta)[..., None] * nz
        del nz
        out[name + "_l"] = (x * len_l[..., None]).to(dt)
        out[name + "_lm1"] = (y * len_lm1[..., None]).to(dt)
        del x, y
        if keep_theta:
            out["theta_" + name] = theta
    if keep_theta:
        out["outlier"] = outlier
    return out


def make_queries(cfg: WorkloadConfig, step: int, device="cpu", n_sets: int = 1) -> torch.Tensor:
    """Decode queries [n_sets][batch][n_q_heads][128] in the storage dtype.

    Entries are N(0, (2.5 sqrt(D))^2) so that, with softmax scale 1/sqrt(D)
    and keys of median length 1, logits have a spread of about 2.5 and the
    softmax is neither uniform nor one-hot."""
    g = _rng(device, _seed(cfg, 0, 1000 + step))
    q = torch.randn(n_sets, cfg.batch, cfg.n_q_heads, cfg.head_dim, generator=g, device=device,
                    dtype=torch.float32) * (2.5 * math.sqrt(cfg.head_dim))
    return q.to(torch_dtype(cfg.dtype))


def make_new_tokens(cfg: WorkloadConfig, pair: int, step: int, device="cpu") -> Dict[str, torch.Tensor]:
    """The decode step's new K/V rows of both layers: [batch][1][n_kv_heads][128] each."""
    sub = dataclasses.replace(cfg, index=cfg.index * 131 + 7 + step)
    return make_pair_tensors(sub, pair, device=device, seq_len=1)


def make_block_table(seq_capacity: np.ndarray, page_size: int, seed: int, spare_pages: int = 3):
    """Random page assignment.  ``seq_capacity[b]`` = tokens sequence b may ever hold.

    Returns (block_table int32 [batch][max_pages] with -1 for unused slots, n_pages)."""
    need = [(int(c) + page_size - 1) // page_size for c in seq_capacity]
    total = sum(need)
    n_pages = total + spare_pages
    rs = np.random.RandomState(seed & 0x7FFFFFFF)
    perm = rs.permutation(n_pages)[:total].astype(np.int32)
    mp = max(need) if need else 0
    bt = np.full((len(need), mp), -1, np.int32)
    o = 0
    for b, n in enumerate(need):
        bt[b, :n] = perm[o:o + n]
        o += n
    return bt, n_pages


def to_paged(x: torch.Tensor, block_table: torch.Tensor, page_size: int, n_pages: int,
             pool: Optional[torch.Tensor] = None) -> torch.Tensor:
    """Scatter logical [B][S][H][D] rows into a pool [n_pages][H][page_size][D].

    Tokens beyond a sequence's pages are dropped; untouched pool rows stay zero."""
    B, S, H, D = x.shape
    npg = (S + page_size - 1) // page_size
    if npg * page_size != S:
        pad = torch.zeros(B, npg * page_size - S, H, D, dtype=x.dtype, device=x.device)
        x = torch.cat([x, pad], dim=1)
    xp = x.view(B, npg, page_size, H, D).permute(0, 1, 3, 2, 4)  # [B][np][H][ps][D]
    if pool is None:
        pool = torch.zeros(n_pages, H, page_size, D, dtype=x.dtype, device=x.device)
    bt = block_table[:, :npg].to(x.device).long()
    valid = bt >= 0
    pool[bt[valid]] = xp[valid]
    return pool


def from_paged(pool: torch.Tensor, block_table: torch.Tensor, seq_len: int) -> torch.Tensor:
    """Gather a pool [n_pages][H][page_size][...] back to logical [B][seq_len][H][...]."""
    n_pages, H, ps = pool.shape[:3]
    rest = pool.shape[3:]
    npg = (seq_len + ps - 1) // ps
    bt = block_table[:, :npg].to(pool.device).long().clamp(min=0)
    g = pool[bt]  # [B][np][H][ps][...]
    perm = (0, 1, 3, 2) + tuple(range(4, 4 + len(rest)))
    g = g.permute(*perm).reshape(bt.shape[0], npg * ps, H, *rest)
    return g[:, :seq_len]


def quantise_q4(x: torch.Tensor, kind: str) -> Dict[str, torch.Tensor]:
    """4-bit input layers for the serving-mix workload (data preparation, KIVI's asymmetric scheme,
    groups of 32): x [B][S][H][128] 16-bit, S a multiple of 32.

    kind "k": per channel, a group = 32 consecutive tokens; meta [B][S/32][H][128][2] (scale, zero).
    kind "v": per token, a group = 32 consecutive channels; meta [B][S][H][4][2].
    codes [B][S][H][64] uint8, channel 2i in the low nibble of byte i, channel 2i+1 in the high one.
    scale = (max - min) / 15 and zero = min are stored in binary16; a constant group gets scale 1."""
    B, S, H, D = x.shape
    assert S % 32 == 0 and D == 128
    xf = x.double()
    if kind == "k":
        g = xf.view(B, S // 32, 32, H, D)
        lo, hi = g.amin(2), g.amax(2)  # [B][S/32][H][D]
    else:
        g = xf.view(B, S, H, 4, 32)
        lo, hi = g.amin(-1), g.amax(-1)  # [B][S][H][4]
    scale = ((hi - lo) / 15.0).to(torch.float16)
    zero = lo.to(torch.float16)
    scale = torch.where(scale == 0, torch.ones_like(scale), scale)
    if kind == "k":
        q = torch.clamp(torch.round((g - zero.double()[:, :, None]) / scale.double()[:, :, None]), 0, 15).view(B, S, H, D)
    else:
        q = torch.clamp(torch.round((g - zero.double()[..., None]) / scale.double()[..., None]), 0, 15).view(B, S, H, D)
    q = q.to(torch.uint8)
    codes = (q[..., 0::2] | (q[..., 1::2] << 4)).contiguous()
    return {"codes": codes, "meta": torch.stack([scale, zero], dim=-1).contiguous()}


def make_projection_case(cfg: WorkloadConfig, pair: int, d_model: int, x_seq_stride: int, device="cpu") -> Dict[str, torch.Tensor]:
    """Inputs of the merge fused into layer l's K/V projection: hidden states ``x`` [batch][x_seq_stride][d_model]
    and transposed weights ``w_k, w_v`` [n_kv_heads * 128][d_model] in the storage dtype, scaled so that the rows
    x W^T follow the row model (random directions, log-normal lengths), and layer l-1's rows ``k_lm1, v_lm1``
    [batch][x_seq_stride][n_kv_heads][128] planted at the row model's angles from those products (the same recipe
    as make_pair_tensors, with layer l's rows given by the projection instead of drawn)."""
    B, S, H, D = cfg.batch, x_seq_stride, cfg.n_kv_heads, cfg.head_dim
    dt = torch_dtype(cfg.dtype)
    mu = cfg.theta_mean(pair)
    gm = _rng(device, _seed(cfg, pair, 40))
    outlier = torch.rand(B, S, generator=gm, device=device) < cfg.outlier_frac
    x = torch.randn(B, S, d_model, generator=gm, device=device, dtype=torch.float32)
    x *= torch.exp(0.5 * torch.randn(B, S, 1, generator=gm, device=device, dtype=torch.float32))  # per-token length
    x = x.to(dt)
    out: Dict[str, torch.Tensor] = {"x": x}
    for ti, name in enumerate(("k", "v")):
        g = _rng(device, _seed(cfg, pair, 41 + ti))
        w = (torch.randn(H * D, d_model, generator=g, device=device, dtype=torch.float32) / math.sqrt(d_model * D)).to(dt)
        out["w_" + name] = w
        c = (x.float().reshape(B * S, d_model) @ w.float().T).reshape(B, S, H, D)  # layer l's rows, before storage rounding
        cn = c / c.norm(dim=-1, keepdim=True).clamp_min(1e-20)
        nz = torch.randn(B, S, H, D, generator=g, device=device, dtype=torch.float32)
        nz -= (nz * cn).sum(-1, keepdim=True) * cn
        nz /= nz.norm(dim=-1, keepdim=True)
        u = torch.rand(B, S, H, generator=g, device=device, dtype=torch.float32)
        theta = torch.where(outlier[:, :, None], 1.2 + 0.8 * u, 2.0 * mu * u)
        len_lm1 = torch.exp(0.5 * torch.randn(B, S, H, generator=g, device=device, dtype=torch.float32))
        y = torch.cos(theta)[..., None] * cn + torch.sin(theta)[..., None] * nz
        out[name + "_lm1"] = (y * len_lm1[..., None]).to(dt)
        out[name + "_ref"] = c
    return out

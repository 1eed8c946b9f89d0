"""ctypes binding of libminicache.so: argument marshalling only.

Every function here has the name of the C entry point it wraps (``include/minicache.h``)
and hands raw device pointers of torch tensors to it.  Nothing is computed in Python, and
there is no fallback: without the compiled library every call raises."""
from __future__ import annotations

import ctypes as C
import dataclasses
import os
from typing import Optional

import torch

MC_F16, MC_BF16 = 0, 1
MC_RETAIN_DISTINCT, MC_RETAIN_LITERAL, MC_RETAIN_TOPK = 0, 1, 2
MC_LAYER_LM1, MC_LAYER_L, MC_LAYER_BOTH = 0, 1, 2
MC_OP_MERGE, MC_OP_DECODE_ATTN = 0, 1
MC_STATUS_WORDS = 4
MC_STATUS_FLAGS, MC_STATUS_RETAINED_TOTAL, MC_STATUS_NEAR_THRESHOLD = 0, 1, 2
MC_FLAG_RETAIN_OVERFLOW, MC_FLAG_WAIT_TIMEOUT, MC_FLAG_BAD_METADATA, MC_FLAG_BOUNDS = 1, 2, 4, 8
MC_FLAG_HINT_TOO_HIGH = 16
MC_BUILD_BOUNDS = 1

# MINICACHE_LIBRARY selects another build of the same library (the range-checked one, for instance)
_LIB_PATH = os.environ.get("MINICACHE_LIBRARY") or os.path.join(os.path.dirname(os.path.abspath(__file__)), "libminicache.so")


class McError(RuntimeError):
    def __init__(self, code: int, name: str, detail: str = ""):
        super().__init__(f"{name} ({code}){': ' + detail if detail else ''}")
        self.code = code
        self.name = name


class _Config(C.Structure):
    _fields_ = [("n_kv_heads", C.c_int32), ("n_q_heads", C.c_int32), ("head_dim", C.c_int32),
                ("page_size", C.c_int32), ("dtype", C.c_int32), ("retain_mode", C.c_int32),
                ("t", C.c_double), ("gamma", C.c_double), ("merge_fn", C.c_int32), ("cache_bits", C.c_int32),
                ("t_mode", C.c_int32), ("retain_union", C.c_int32), ("append_slack", C.c_int32)]


class _Batch(C.Structure):
    _fields_ = [("block_table", C.c_void_p), ("seq_lens", C.c_void_p), ("batch", C.c_int32),
                ("max_pages_per_seq", C.c_int32), ("max_seq_len", C.c_int32), ("reserved", C.c_int32),
                ("n_pages", C.c_int64)]


class _LayerKV(C.Structure):
    _fields_ = [("k_pool", C.c_void_p), ("v_pool", C.c_void_p)]


class _LayerQ4(C.Structure):
    _fields_ = [("k_codes", C.c_void_p), ("k_meta", C.c_void_p), ("v_codes", C.c_void_p), ("v_meta", C.c_void_p)]


class _Projection(C.Structure):
    _fields_ = [("x", C.c_void_p), ("w_k", C.c_void_p), ("w_v", C.c_void_p), ("d_model", C.c_int32), ("x_seq_stride", C.c_int32)]


class _PairCache(C.Structure):
    _fields_ = [("e_k", C.c_void_p), ("e_v", C.c_void_p), ("dist", C.c_void_p),
                ("ret_count", C.c_void_p), ("ret_offset", C.c_void_p), ("ret_index", C.c_void_p),
                ("ret_rows", C.c_void_p), ("ret_capacity", C.c_int64), ("ret_prefix", C.c_void_p),
                ("ret_prefix_stride", C.c_int64), ("seg_minmax", C.c_void_p),
                ("status", C.c_void_p), ("res_k", C.c_void_p), ("res_v", C.c_void_p)]


class _PairSizes(C.Structure):
    _fields_ = [("tile_bytes", C.c_size_t), ("e_bytes", C.c_size_t), ("dist_bytes", C.c_size_t),
                ("ret_count_bytes", C.c_size_t), ("ret_offset_bytes", C.c_size_t), ("ret_index_bytes", C.c_size_t),
                ("ret_rows_bytes", C.c_size_t), ("ret_prefix_bytes", C.c_size_t), ("seg_minmax_bytes", C.c_size_t),
                ("status_bytes", C.c_size_t), ("ret_prefix_stride", C.c_int64), ("total_bytes", C.c_size_t),
                ("res_bytes", C.c_size_t)]


class _Stats(C.Structure):
    _fields_ = [("flags", C.c_int32), ("reserved", C.c_int32), ("retained_total", C.c_int64),
                ("near_threshold", C.c_int64), ("token_heads", C.c_int64), ("full_bytes", C.c_int64),
                ("compressed_bytes", C.c_int64), ("stored_bytes", C.c_int64)]


EXPORTS = ("mc_decode_drain_host", "mc_decode_stage_host", "mc_decode_attn_append", "mc_prefill_merge_pair", "mc_admit_sequences", "mc_build_flags", "mc_merge_pairs", "mc_pair_bytes", "mc_get_stats", "mc_version", "mc_status_str", "mc_last_cuda_error", "mc_workspace_bytes", "mc_merge_pair",
           "mc_append_pair", "mc_restore", "mc_decode_attn", "mc_read_status", "mc_merge_pair_host",
           "mc_decode_attn_host", "mc_decode_io_bytes", "mc_decode_attn_static", "mc_merge_pair_q4", "mc_selftest_wait_timeout")


def _ptr(t: Optional[torch.Tensor]) -> Optional[int]:
    return None if t is None else t.data_ptr()


def _stream(stream) -> Optional[int]:
    if stream is None:
        stream = torch.cuda.current_stream()
    return stream.cuda_stream or None


@dataclasses.dataclass
class McConfig:
    n_kv_heads: int
    n_q_heads: int
    page_size: int
    dtype: str  # "f16" | "bf16"
    t: float = 0.6
    gamma: float = 0.05
    retain_mode: int = MC_RETAIN_DISTINCT
    head_dim: int = 128
    merge_fn: int = 0  # MC_MERGE_SLERP (Eq. 3) | MC_MERGE_FMAX = 1 | MC_MERGE_MEAN = 2
    cache_bits: int = 16  # storage of the shared directions: 16 (the 16-bit type) or 4 (4-bit shared cache, pages of 32)
    t_mode: int = 0  # MC_T_FIXED | MC_T_MAGNITUDE_RATIO = 1 (per-token t from the two magnitudes)
    retain_union: int = 0  # 1: one retention set for keys and values (the union of Eq. 4's two sets)
    append_slack: int = 0  # > 0: free retained entries per segment; appended tokens are held against Eq. 4's stored threshold

    def c(self) -> _Config:
        return _Config(self.n_kv_heads, self.n_q_heads, self.head_dim, self.page_size,
                       {"f16": MC_F16, "bf16": MC_BF16}[self.dtype], self.retain_mode, float(self.t), float(self.gamma),
                       int(self.merge_fn), int(self.cache_bits), int(self.t_mode), int(self.retain_union),
                       int(self.append_slack))

    @property
    def torch_dtype(self):
        return {"f16": torch.float16, "bf16": torch.bfloat16}[self.dtype]


@dataclasses.dataclass
class Batch:
    """Device block table / sequence lengths plus the host-known bounds."""
    block_table: torch.Tensor  # int32 [batch][max_pages_per_seq]
    seq_lens: torch.Tensor  # int32 [batch]
    max_seq_len: int
    n_pages: int

    def c(self) -> _Batch:
        assert self.block_table.dtype == torch.int32 and self.seq_lens.dtype == torch.int32
        assert self.block_table.is_contiguous() and self.seq_lens.is_contiguous()
        b = self.seq_lens.shape[0]
        mp = self.block_table.shape[1] if self.block_table.dim() == 2 else 0
        return _Batch(_ptr(self.block_table), _ptr(self.seq_lens), b, mp, int(self.max_seq_len), 0, int(self.n_pages))


class PairCache:
    """Caller-owned device buffers of one compressed layer pair (allocated with torch)."""

    def __init__(self, cfg: McConfig, batch: int, n_pages: int, ret_capacity: int, device="cuda",
                 max_merge_len: Optional[int] = None):
        H, ps = cfg.n_kv_heads, cfg.page_size
        self.cfg = cfg
        if max_merge_len is None:  # bound of the sequence length at merge time: what the pages can hold at most
            max_merge_len = n_pages * ps
        cap = max(int(ret_capacity), 1)
        sz = lib().mc_pair_bytes(cfg, batch, n_pages, int(max_merge_len), cap)  # every size comes from the library
        self.sizes = sz
        self.tile_bytes = sz.tile_bytes
        nseg = 2 * batch * H
        z = lambda nbytes: torch.zeros(nbytes, dtype=torch.uint8, device=device)
        self.e_k = z(sz.e_bytes).view(n_pages, H, self.tile_bytes)
        self.e_v = z(sz.e_bytes).view(n_pages, H, self.tile_bytes)
        self.dist = z(sz.dist_bytes).view(torch.float32).view(n_pages, H, 2, ps)
        self.ret_count = z(sz.ret_count_bytes).view(torch.int32)
        self.ret_offset = z(sz.ret_offset_bytes).view(torch.int32)
        self.ret_index = z(sz.ret_index_bytes).view(torch.int32)
        self.ret_rows = z(sz.ret_rows_bytes).view(2, cap, 272)
        self.ret_capacity = int(ret_capacity)
        self.ret_prefix_stride = int(sz.ret_prefix_stride)
        self.ret_prefix = z(sz.ret_prefix_bytes).view(torch.int32).view(nseg, self.ret_prefix_stride)
        self.seg_minmax = z(sz.seg_minmax_bytes).view(torch.float32).view(nseg, 2)
        self.status = z(sz.status_bytes).view(torch.int32)
        self.q4 = cfg.cache_bits == 4
        self.res_k = self.res_v = None
        if self.q4:  # one 16-bit tile of 32 tokens per (sequence, head): the last, incomplete page
            self.res_k = z(sz.res_bytes).view(batch, H, sz.res_bytes // max(batch * H, 1))
            self.res_v = z(sz.res_bytes).view(batch, H, sz.res_bytes // max(batch * H, 1))

    def c(self) -> _PairCache:
        return _PairCache(_ptr(self.e_k), _ptr(self.e_v), _ptr(self.dist), _ptr(self.ret_count),
                          _ptr(self.ret_offset), _ptr(self.ret_index), _ptr(self.ret_rows), self.ret_capacity,
                          _ptr(self.ret_prefix), self.ret_prefix_stride, _ptr(self.seg_minmax), _ptr(self.status),
                          _ptr(self.res_k), _ptr(self.res_v))

    # -- decoding the tile layout (pure re-indexing, no arithmetic) ------------------------------
    def _rows16(self, pool: torch.Tensor) -> torch.Tensor:
        """16-bit tiles [n][H][tile] -> direction rows [n][H][page_size][128] (chunk permutation undone)."""
        ps = self.cfg.page_size
        n, H = pool.shape[:2]
        rows = pool[:, :, :ps * 256].reshape(n, H, ps, 16, 16)  # [..][row][chunk position][16 bytes]
        r = torch.arange(ps, device=pool.device)[:, None]
        c = torch.arange(16, device=pool.device)[None, :]
        pos = (c & 8) | ((c & 7) ^ (r & 7))  # where chunk c of row r is stored
        idx = pos[None, None, :, :, None].expand(n, H, ps, 16, 16)
        plain = torch.gather(rows, 3, idx).reshape(n, H, ps, 256)
        return plain.view(self.cfg.torch_dtype)

    def directions(self, tensor: str) -> torch.Tensor:
        """Stored directions of "k" or "v" as [n_pages][H][page_size][128] in the storage type
        (the 16-byte chunk permutation of the tile format undone).  16-bit cache only."""
        assert not self.q4, "a 4-bit cache holds codes: see q4_codes / q4_groups / residual_directions"
        return self._rows16(self.e_k if tensor == "k" else self.e_v)

    def scales(self, tensor: str) -> torch.Tensor:
        """Scales of "k" or "v" as [n_pages][H][2][page_size] fp32 ([..][0]: layer l-1, [1]: layer l)."""
        pool = self.e_k if tensor == "k" else self.e_v
        ps = self.cfg.page_size
        n_pages, H = pool.shape[:2]
        off = 2560 if self.q4 else ps * 256
        return pool[:, :, off:].contiguous().view(torch.float32).reshape(n_pages, H, 2, ps)

    # -- 4-bit shared cache: the tile's orders undone (pure re-indexing) -------------------------
    def q4_codes(self, tensor: str) -> torch.Tensor:
        """Codes of "k" or "v" as [n_pages][H][32][128] uint8, channels in natural order."""
        assert self.q4
        pool = self.e_k if tensor == "k" else self.e_v
        n_pages, H = pool.shape[:2]
        dev = pool.device
        words = pool[:, :, :2048].contiguous().view(torch.int32).reshape(n_pages, H, 512).long() & 0xFFFFFFFF
        nib = torch.stack([(words >> (4 * j)) & 15 for j in range(8)], dim=-1).to(torch.uint8)  # [..][word][nibble]
        out = torch.zeros(n_pages, H, 32, 128, dtype=torch.uint8, device=dev)
        if tensor == "k":
            # row r, word w, nibble j: channel 8 w + 2 (j % 4) + j // 4
            nib = nib.reshape(n_pages, H, 32, 16, 8)
            w = torch.arange(16, device=dev)[:, None]
            j = torch.arange(8, device=dev)[None, :]
            ch = (8 * w + 2 * (j % 4) + j // 4).reshape(-1)
            out[:, :, :, ch] = nib.reshape(n_pages, H, 32, 128)
        else:
            # block i (tokens 2i, 2i+1), chunk position cp, word k, nibble j: token 2i + j // 4,
            # channel 32 k + 16 ((j % 4) // 2) + 8 (j % 2) + (cp ^ ((i % 4) * 2))
            nib = nib.reshape(n_pages, H, 16, 8, 4, 8)
            i = torch.arange(16, device=dev)[:, None, None, None]
            cp = torch.arange(8, device=dev)[None, :, None, None]
            k = torch.arange(4, device=dev)[None, None, :, None]
            j = torch.arange(8, device=dev)[None, None, None, :]
            tok = (2 * i + j // 4).expand(16, 8, 4, 8).reshape(-1)
            ch = (32 * k + 16 * ((j % 4) // 2) + 8 * (j % 2) + (cp ^ ((i % 4) * 2))).expand(16, 8, 4, 8).reshape(-1)
            out[:, :, tok, ch] = nib.reshape(n_pages, H, -1)
        return out

    def q4_groups(self, tensor: str):
        """(scale, zero) of "k" ([n_pages][H][128], per channel) or "v" ([n_pages][H][32][4], per token and
        channel group) in the storage type."""
        assert self.q4
        pool = self.e_k if tensor == "k" else self.e_v
        n_pages, H = pool.shape[:2]
        dev = pool.device
        m = pool[:, :, 2048:2560].contiguous().view(self.cfg.torch_dtype)  # 256 values
        if tensor == "k":
            m = m.reshape(n_pages, H, 2, 16, 8)  # [scale|zero][chunk position][8 channels]
            o = torch.arange(16, device=dev)
            pos = 4 * (o & 3) + (o >> 2)  # where the chunk of channels [8 o, 8 o + 8) is stored
            m = m[:, :, :, pos].reshape(n_pages, H, 2, 128)
            return m[:, :, 0].contiguous(), m[:, :, 1].contiguous()
        m = m.reshape(n_pages, H, 16, 2, 4, 2)  # [token pair][scale|zero][group][token of the pair]
        m = m.permute(0, 1, 3, 2, 5, 4).reshape(n_pages, H, 2, 32, 4)
        return m[:, :, 0].contiguous(), m[:, :, 1].contiguous()

    def residual_directions(self, tensor: str) -> torch.Tensor:
        """The residual tiles' rows [batch][H][32][128] in the storage type (tokens of the last, incomplete page)."""
        assert self.q4
        return self._rows16(self.res_k if tensor == "k" else self.res_v)

    def residual_scales(self, tensor: str) -> torch.Tensor:
        """The residual tiles' scales [batch][H][2][32] fp32."""
        assert self.q4
        pool = self.res_k if tensor == "k" else self.res_v
        return pool[:, :, 32 * 256:].contiguous().view(torch.float32).reshape(pool.shape[0], pool.shape[1], 2, 32)

    def retained_rows(self, layer: int) -> torch.Tensor:
        """Raw retained rows of one layer (0: l-1, 1: l) as [ret_capacity][128] in the storage type."""
        return self.ret_rows[layer, :, :256].contiguous().view(self.cfg.torch_dtype)

    def retained_tokens(self, layer: int) -> torch.Tensor:
        """Token index stored with each retained entry of one layer: [ret_capacity] int32."""
        return self.ret_rows[layer, :, 256:260].contiguous().view(torch.int32).reshape(-1)

    def nbytes(self) -> int:
        ts = (self.e_k, self.e_v, self.dist, self.ret_count, self.ret_offset, self.ret_index,
              self.ret_rows, self.ret_prefix, self.seg_minmax, self.status) + ((self.res_k, self.res_v) if self.q4 else ())
        return sum(t.numel() * t.element_size() for t in ts)


class MiniCacheLib:
    """Loads libminicache.so and exposes its entry points under their C names."""

    def __init__(self, path: str = _LIB_PATH):
        if not os.path.exists(path):
            raise McError(-1, "library missing",
                          f"{path} not built; run `python -m paper_2405_14366_b200.build` (there is no fallback path)")
        self.path = path
        self._lib = C.CDLL(path)
        L = self._lib
        L.mc_version.restype = C.c_int32
        L.mc_build_flags.restype = C.c_int32
        L.mc_status_str.restype = C.c_char_p
        L.mc_status_str.argtypes = [C.c_int32]
        L.mc_last_cuda_error.restype = C.c_char_p
        P, V = C.POINTER, C.c_void_p
        L.mc_workspace_bytes.argtypes = [P(_Config), P(_Batch), C.c_int32, C.c_int32, P(C.c_size_t)]
        L.mc_merge_pair.argtypes = [P(_Config), P(_Batch), P(_LayerKV), P(_LayerKV), P(_PairCache), C.c_int32, V,
                                    C.c_size_t, V]
        L.mc_merge_pairs.argtypes = [P(_Config), P(_Batch), C.c_int32, P(P(_LayerKV)), P(P(_LayerKV)), P(P(_PairCache)),
                                     C.c_int32, V, C.c_size_t, V]
        L.mc_merge_pairs.restype = C.c_int32
        L.mc_admit_sequences.argtypes = [P(_Config), P(_Batch), C.c_int32, C.c_int32, C.c_int32, P(P(_LayerKV)), P(P(_LayerKV)),
                                         P(P(_LayerQ4)), P(P(_LayerQ4)), P(P(_PairCache)), C.c_int64, C.c_int32, V, C.c_size_t, V]
        L.mc_admit_sequences.restype = C.c_int32
        L.mc_prefill_merge_pair.argtypes = [P(_Config), P(_Batch), P(_Projection), P(_LayerKV), P(_LayerKV), P(_PairCache),
                                            C.c_float, C.c_int32, V, C.c_size_t, V]
        L.mc_prefill_merge_pair.restype = C.c_int32
        L.mc_append_pair.argtypes = [P(_Config), P(_Batch), P(_PairCache), V, V, V, V, V]
        L.mc_restore.argtypes = [P(_Config), P(_Batch), P(_PairCache), C.c_int32, P(_LayerKV), C.c_int32, V]
        L.mc_pair_bytes.argtypes = [P(_Config), P(_Batch), C.c_int64, P(_PairSizes)]
        L.mc_pair_bytes.restype = C.c_int32
        L.mc_get_stats.argtypes = [P(_Config), P(_Batch), P(_PairCache), V, P(_Stats)]
        L.mc_get_stats.restype = C.c_int32
        L.mc_decode_attn.argtypes = [P(_Config), P(_Batch), P(_PairCache), C.c_int32, V, V, V, C.c_float, V, V, V,
                                     C.c_size_t, V]
        L.mc_decode_attn_append.argtypes = [P(_Config), P(_Batch), P(_PairCache), C.c_int32, V, V, V, C.c_float, V, V, V, V, V, V,
                                            V, C.c_size_t, V]
        L.mc_decode_attn_append.restype = C.c_int32
        L.mc_decode_stage_host.argtypes = [P(_Config), P(_Batch), C.c_int32, V, V, V, V, C.c_size_t, P(V), P(V), P(V), V]
        L.mc_decode_stage_host.restype = C.c_int32
        L.mc_decode_drain_host.argtypes = [P(_Config), P(_Batch), C.c_int32, V, V, V, V, V]
        L.mc_decode_drain_host.restype = C.c_int32
        L.mc_read_status.argtypes = [P(_PairCache), V, P(C.c_int32)]
        L.mc_merge_pair_host.argtypes = [P(_Config), P(_Batch), P(_LayerKV), P(_LayerKV), P(_LayerKV), P(_LayerKV),
                                         P(_PairCache), C.c_int32, V, C.c_size_t, V]
        L.mc_decode_attn_host.argtypes = [P(_Config), P(_Batch), P(_PairCache), C.c_int32, V, V, V, C.c_float, V, V,
                                          V, C.c_size_t, V, C.c_size_t, V]
        L.mc_decode_io_bytes.argtypes = [P(_Config), P(_Batch), C.c_int32, P(C.c_size_t)]
        L.mc_decode_attn_static.argtypes = [P(_Config), P(_Batch), P(_PairCache), C.c_int32, V, V, V, C.c_float, V, V, V]
        L.mc_decode_attn_static.restype = C.c_int32
        L.mc_merge_pair_q4.argtypes = [P(_Config), P(_Batch), P(_LayerQ4), P(_LayerQ4), P(_PairCache), C.c_int32, V,
                                       C.c_size_t, V]
        L.mc_merge_pair_q4.restype = C.c_int32
        L.mc_selftest_wait_timeout.argtypes = [P(_PairCache), C.c_int32, V]
        L.mc_selftest_wait_timeout.restype = C.c_int32
        for f in ("mc_workspace_bytes", "mc_merge_pair", "mc_append_pair", "mc_restore", "mc_decode_attn",
                  "mc_read_status", "mc_merge_pair_host", "mc_decode_attn_host", "mc_decode_io_bytes"):
            getattr(L, f).restype = C.c_int32

    # -- helpers ------------------------------------------------------------------------------
    def _check(self, code: int):
        if code != 0:
            name = self._lib.mc_status_str(code).decode()
            detail = self._lib.mc_last_cuda_error().decode() if code == 7 else ""
            raise McError(code, name, detail)

    def has_symbol(self, name: str) -> bool:
        return hasattr(self._lib, name)

    # -- entry points ---------------------------------------------------------------------------
    def mc_version(self) -> int:
        return self._lib.mc_version()

    def mc_build_flags(self) -> int:
        return self._lib.mc_build_flags()

    def mc_status_str(self, code: int) -> str:
        return self._lib.mc_status_str(code).decode()

    def mc_workspace_bytes(self, cfg: McConfig, batch: Batch, op: int, n_query_sets: int = 1) -> int:
        out = C.c_size_t(0)
        c, b = cfg.c(), batch.c()
        self._check(self._lib.mc_workspace_bytes(C.byref(c), C.byref(b), op, n_query_sets, C.byref(out)))
        return out.value

    def mc_merge_pair(self, cfg: McConfig, batch: Batch, k_lm1, v_lm1, k_l, v_l, pair: PairCache,
                      do_retention: bool, workspace: torch.Tensor, stream=None):
        c, b, pc = cfg.c(), batch.c(), pair.c()
        a, l = _LayerKV(_ptr(k_lm1), _ptr(v_lm1)), _LayerKV(_ptr(k_l), _ptr(v_l))
        self._check(self._lib.mc_merge_pair(C.byref(c), C.byref(b), C.byref(a), C.byref(l), C.byref(pc),
                                            1 if do_retention else 0, _ptr(workspace),
                                            workspace.numel() * workspace.element_size(), _stream(stream)))

    def mc_merge_pairs(self, cfg: McConfig, batch: Batch, layers, pairs, do_retention: bool, workspace: torch.Tensor,
                       stream=None):
        """layers: per pair a dict with k_lm1, v_lm1, k_l, v_l pools; pairs: the PairCache of each.
        workspace: len(pairs) * mc_workspace_bytes(MC_OP_MERGE) bytes."""
        n = len(pairs)
        c, b = cfg.c(), batch.c()
        a = [_LayerKV(_ptr(x["k_lm1"]), _ptr(x["v_lm1"])) for x in layers]
        l = [_LayerKV(_ptr(x["k_l"]), _ptr(x["v_l"])) for x in layers]
        pcs = [pc.c() for pc in pairs]
        arr = lambda items, T: (C.POINTER(T) * n)(*[C.pointer(x) for x in items])
        self._check(self._lib.mc_merge_pairs(C.byref(c), C.byref(b), n, arr(a, _LayerKV), arr(l, _LayerKV),
                                             arr(pcs, _PairCache), 1 if do_retention else 0, _ptr(workspace),
                                             workspace.numel() * workspace.element_size(), _stream(stream)))

    def mc_admit_sequences(self, cfg: McConfig, batch: Batch, seq_begin: int, seq_count: int, layers, pairs, rows_per_seq: int,
                           do_retention: bool, workspace: torch.Tensor, stream=None, q4: bool = False):
        """layers: per pair a dict with k_lm1, v_lm1, k_l, v_l pools, or (q4) with "_lm1" / "_l" dicts of
        k_codes, k_meta, v_codes, v_meta; pairs: the PairCache of each pair."""
        n = len(pairs)
        c, b = cfg.c(), batch.c()
        pcs = [pc.c() for pc in pairs]
        arr = lambda items, T: (C.POINTER(T) * n)(*[C.pointer(x) for x in items])
        if q4:
            mk = lambda d: _LayerQ4(_ptr(d["k_codes"]), _ptr(d["k_meta"]), _ptr(d["v_codes"]), _ptr(d["v_meta"]))
            a, l = [mk(x["_lm1"]) for x in layers], [mk(x["_l"]) for x in layers]
            args = (None, None, arr(a, _LayerQ4), arr(l, _LayerQ4))
        else:
            a = [_LayerKV(_ptr(x["k_lm1"]), _ptr(x["v_lm1"])) for x in layers]
            l = [_LayerKV(_ptr(x["k_l"]), _ptr(x["v_l"])) for x in layers]
            args = (arr(a, _LayerKV), arr(l, _LayerKV), None, None)
        self._check(self._lib.mc_admit_sequences(C.byref(c), C.byref(b), int(seq_begin), int(seq_count), n, *args,
                                                 arr(pcs, _PairCache), int(rows_per_seq), 1 if do_retention else 0,
                                                 _ptr(workspace), workspace.numel() * workspace.element_size(), _stream(stream)))

    def mc_prefill_merge_pair(self, cfg: McConfig, batch: Batch, x, w_k, w_v, k_lm1, v_lm1, k_l, v_l, pair: PairCache,
                              d_hint: float, do_retention: bool, workspace: torch.Tensor, stream=None):
        """x [batch][x_seq_stride][d_model], w_k / w_v [n_kv_heads * 128][d_model]: layer l's projection;
        k_l / v_l: pools that receive the raw rows of tokens with distance above d_hint."""
        c, b, pc = cfg.c(), batch.c(), pair.c()
        pj = _Projection(_ptr(x), _ptr(w_k), _ptr(w_v), int(x.shape[-1]), int(x.shape[1]))
        a, l = _LayerKV(_ptr(k_lm1), _ptr(v_lm1)), _LayerKV(_ptr(k_l), _ptr(v_l))
        self._check(self._lib.mc_prefill_merge_pair(C.byref(c), C.byref(b), C.byref(pj), C.byref(a), C.byref(l), C.byref(pc),
                                                    float(d_hint), 1 if do_retention else 0, _ptr(workspace),
                                                    workspace.numel() * workspace.element_size(), _stream(stream)))

    def mc_merge_pair_q4(self, cfg: McConfig, batch: Batch, q_lm1, q_l, pair: PairCache, do_retention: bool,
                         workspace: torch.Tensor, stream=None):
        """q_lm1 / q_l: dicts with k_codes, k_meta, v_codes, v_meta device tensors (4-bit layers)."""
        c, b, pc = cfg.c(), batch.c(), pair.c()
        a = _LayerQ4(_ptr(q_lm1["k_codes"]), _ptr(q_lm1["k_meta"]), _ptr(q_lm1["v_codes"]), _ptr(q_lm1["v_meta"]))
        l = _LayerQ4(_ptr(q_l["k_codes"]), _ptr(q_l["k_meta"]), _ptr(q_l["v_codes"]), _ptr(q_l["v_meta"]))
        self._check(self._lib.mc_merge_pair_q4(C.byref(c), C.byref(b), C.byref(a), C.byref(l), C.byref(pc),
                                               1 if do_retention else 0, _ptr(workspace),
                                               workspace.numel() * workspace.element_size(), _stream(stream)))

    def mc_append_pair(self, cfg: McConfig, batch: Batch, pair: PairCache, k_new_lm1, v_new_lm1, k_new_l, v_new_l,
                       stream=None):
        c, b, pc = cfg.c(), batch.c(), pair.c()
        self._check(self._lib.mc_append_pair(C.byref(c), C.byref(b), C.byref(pc), _ptr(k_new_lm1), _ptr(v_new_lm1),
                                             _ptr(k_new_l), _ptr(v_new_l), _stream(stream)))

    def mc_restore(self, cfg: McConfig, batch: Batch, pair: PairCache, layer_sel: int, dst_k, dst_v, stream=None):
        """dst_k / dst_v: pools in the storage type, or float32 pools (then the unrounded products are written)."""
        c, b, pc = cfg.c(), batch.c(), pair.c()
        d = _LayerKV(_ptr(dst_k), _ptr(dst_v))
        assert dst_k.dtype == dst_v.dtype and dst_k.dtype in (torch.float32, cfg.torch_dtype)
        f32 = 1 if dst_k.dtype == torch.float32 else 0
        self._check(self._lib.mc_restore(C.byref(c), C.byref(b), C.byref(pc), layer_sel, C.byref(d), f32, _stream(stream)))

    def mc_pair_bytes(self, cfg: McConfig, batch: int, n_pages: int, max_seq_len: int, ret_capacity: int) -> _PairSizes:
        c = cfg.c()
        b = _Batch(None, None, int(batch), 0, int(max_seq_len), 0, int(n_pages))
        out = _PairSizes()
        self._check(self._lib.mc_pair_bytes(C.byref(c), C.byref(b), int(ret_capacity), C.byref(out)))
        return out

    def mc_get_stats(self, cfg: McConfig, batch: Batch, pair: PairCache, stream=None, check: bool = True):
        """(dict of the mc_stats fields, return code); synchronises the stream."""
        c, b, pc = cfg.c(), batch.c(), pair.c()
        out = _Stats()
        code = self._lib.mc_get_stats(C.byref(c), C.byref(b), C.byref(pc), _stream(stream), C.byref(out))
        if check:
            self._check(code)
        return {f: getattr(out, f) for f, _ in _Stats._fields_ if f != "reserved"}, code

    def mc_decode_attn(self, cfg: McConfig, batch: Batch, pair: PairCache, layer_sel: int, q, k_new, v_new,
                       sm_scale: float, out, lse, workspace: torch.Tensor, stream=None):
        c, b, pc = cfg.c(), batch.c(), pair.c()
        self._check(self._lib.mc_decode_attn(C.byref(c), C.byref(b), C.byref(pc), layer_sel, _ptr(q), _ptr(k_new),
                                             _ptr(v_new), float(sm_scale), _ptr(out), _ptr(lse), _ptr(workspace),
                                             workspace.numel() * workspace.element_size(), _stream(stream)))

    def mc_decode_attn_append(self, cfg: McConfig, batch: Batch, pair: PairCache, layer_sel: int, q, k_new, v_new,
                              sm_scale: float, out, lse, k_new_lm1, v_new_lm1, k_new_l, v_new_l, workspace: torch.Tensor,
                              stream=None):
        """mc_decode_attn followed by mc_append_pair, in one call (the append rides on the attention's second launch)."""
        c, b, pc = cfg.c(), batch.c(), pair.c()
        self._check(self._lib.mc_decode_attn_append(C.byref(c), C.byref(b), C.byref(pc), layer_sel, _ptr(q), _ptr(k_new),
                                                    _ptr(v_new), float(sm_scale), _ptr(out), _ptr(lse), _ptr(k_new_lm1),
                                                    _ptr(v_new_lm1), _ptr(k_new_l), _ptr(v_new_l), _ptr(workspace),
                                                    workspace.numel() * workspace.element_size(), _stream(stream)))

    def mc_merge_pair_host(self, cfg: McConfig, batch: Batch, host, dev, pair: PairCache, do_retention: bool,
                           workspace: torch.Tensor, stream=None):
        """host / dev: dicts with k_lm1, v_lm1, k_l, v_l pools (pinned host tensors / device tensors)."""
        c, b, pc = cfg.c(), batch.c(), pair.c()
        ha, hl = _LayerKV(_ptr(host["k_lm1"]), _ptr(host["v_lm1"])), _LayerKV(_ptr(host["k_l"]), _ptr(host["v_l"]))
        da, dl = _LayerKV(_ptr(dev["k_lm1"]), _ptr(dev["v_lm1"])), _LayerKV(_ptr(dev["k_l"]), _ptr(dev["v_l"]))
        self._check(self._lib.mc_merge_pair_host(C.byref(c), C.byref(b), C.byref(ha), C.byref(hl), C.byref(da),
                                                 C.byref(dl), C.byref(pc), 1 if do_retention else 0, _ptr(workspace),
                                                 workspace.numel() * workspace.element_size(), _stream(stream)))

    def mc_decode_io_bytes(self, cfg: McConfig, batch: Batch, n_query_sets: int = 1) -> int:
        out = C.c_size_t(0)
        c, b = cfg.c(), batch.c()
        self._check(self._lib.mc_decode_io_bytes(C.byref(c), C.byref(b), n_query_sets, C.byref(out)))
        return out.value

    def mc_decode_attn_host(self, cfg: McConfig, batch: Batch, pair: PairCache, layer_sel: int, q_host, k_new_host,
                            v_new_host, sm_scale: float, out_host, lse_host, dev_io: torch.Tensor,
                            workspace: torch.Tensor, stream=None):
        c, b, pc = cfg.c(), batch.c(), pair.c()
        self._check(self._lib.mc_decode_attn_host(C.byref(c), C.byref(b), C.byref(pc), layer_sel, _ptr(q_host),
                                                  _ptr(k_new_host), _ptr(v_new_host), float(sm_scale), _ptr(out_host),
                                                  _ptr(lse_host), _ptr(dev_io), dev_io.numel() * dev_io.element_size(),
                                                  _ptr(workspace), workspace.numel() * workspace.element_size(),
                                                  _stream(stream)))

    def mc_decode_stage_host(self, cfg: McConfig, batch: Batch, n_query_sets: int, q_host, k_new_host, v_new_host,
                             dev_io: torch.Tensor, stream=None):
        """Stages q (and the new rows) from host tensors into `dev_io`; returns views of dev_io: (q, k_new, v_new)
        shaped [n_query_sets][batch][heads][128] in the storage type (k_new / v_new None if not given)."""
        c, b = cfg.c(), batch.c()
        qd, kd, vd = C.c_void_p(), C.c_void_p(), C.c_void_p()
        self._check(self._lib.mc_decode_stage_host(C.byref(c), C.byref(b), int(n_query_sets), _ptr(q_host), _ptr(k_new_host),
                                                   _ptr(v_new_host), _ptr(dev_io), dev_io.numel() * dev_io.element_size(),
                                                   C.byref(qd), C.byref(kd), C.byref(vd), _stream(stream)))
        base = dev_io.data_ptr()
        nb = batch.seq_lens.shape[0]

        def view(ptr, heads):
            if not ptr.value:
                return None
            n = n_query_sets * nb * heads * 256
            off = ptr.value - base
            return dev_io[off:off + n].view(cfg.torch_dtype).view(n_query_sets, nb, heads, 128)
        return view(qd, cfg.n_q_heads), view(kd, cfg.n_kv_heads), view(vd, cfg.n_kv_heads)

    def mc_decode_drain_host(self, cfg: McConfig, batch: Batch, n_query_sets: int, out_dev, lse_dev, out_host, lse_host,
                             stream=None):
        """Asynchronous copy of an attention result (and its log-sum-exps, if given) from device to host tensors."""
        c, b = cfg.c(), batch.c()
        self._check(self._lib.mc_decode_drain_host(C.byref(c), C.byref(b), int(n_query_sets), _ptr(out_dev), _ptr(lse_dev),
                                                   _ptr(out_host), _ptr(lse_host), _stream(stream)))

    def mc_decode_attn_static(self, cfg: McConfig, batch: Batch, pair: PairCache, layer_sel: int, q, k_new, v_new,
                              sm_scale: float, out, lse, stream=None):
        """mc_decode_attn for callers with no scratch memory to give: the split partials go to the
        library's built-in device array (at most MC_STATIC_SCRATCH_BYTES; larger geometries raise)."""
        c, b, pc = cfg.c(), batch.c(), pair.c()
        code = self._lib.mc_decode_attn_static(C.byref(c), C.byref(b), C.byref(pc), layer_sel, _ptr(q), _ptr(k_new),
                                               _ptr(v_new), float(sm_scale), _ptr(out), _ptr(lse), _stream(stream))
        if code == 5:
            raise McError(code, "MC_ERR_CAPACITY", self._lib.mc_last_cuda_error().decode())
        self._check(code)

    def mc_selftest_wait_timeout(self, pair: PairCache, poll_limit: int = 20000, stream=None):
        pc = pair.c()
        self._check(self._lib.mc_selftest_wait_timeout(C.byref(pc), int(poll_limit), _stream(stream)))

    def mc_read_status(self, pair: PairCache, stream=None, check: bool = True):
        words = (C.c_int32 * MC_STATUS_WORDS)()
        pc = pair.c()
        code = self._lib.mc_read_status(C.byref(pc), _stream(stream), words)
        if check:
            self._check(code)
        return list(words), code


_LIB: Optional[MiniCacheLib] = None


def lib() -> MiniCacheLib:
    """The process-wide library handle (raises if the shared object has not been built)."""
    global _LIB
    if _LIB is None:
        _LIB = MiniCacheLib()
    return _LIB

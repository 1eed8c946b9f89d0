// The 4-bit shared cache (Sec. 5: MiniCache on top of 4-bit KIVI quantisation; layout at mc_pair_cache
// in minicache.h):
//   q4_quantise_pages_kernel  after a merge: every complete page of 16-bit direction tiles becomes a
//                             4-bit tile, a sequence's last, incomplete page goes to its residual tile
//   append_q4_kernel          Algorithm 2 "MiniCache Decoding", the new token pair: merged (Eq. 3) into the
//                             residual tile; the page it completes is quantised on the spot
//   restore_q4_kernel         Eq. 2 + Sec. 4.2 "Cache restoration" from 4-bit tiles and the residual tile
// The quantiser (scale = (max - min) / 15 and zero = min kept in the 16-bit type, round to nearest,
// groups of 32: keys per channel over a page's tokens, values per token over 32 channels) is defined in
// double precision, so that the codes are the same integers on any machine; the kernels evaluate it in
// single precision wherever that provably gives the same integer (q4_code) and in double elsewhere.
#include <algorithm>

#include "mc_common.cuh"
#include "mc_kernels.h"
#include "mc_q4.cuh"
#include "mc_retain.cuh"

namespace mc {

constexpr int kQThreads = 128;

template <int DT>
__device__ __forceinline__ float elem_to_float(unsigned short bits) {
  if (DT == MC_F16) return __half2float(__ushort_as_half(bits));
  return __uint_as_float((uint32_t)bits << 16);
}
template <int DT>
__device__ __forceinline__ unsigned short double_to_elem(double v) {
  if (DT == MC_F16) return __half_as_ushort(__double2half(v));
  return __bfloat16_as_ushort(__double2bfloat16(v));
}
// code * scale + zero rounded once to the 16-bit type (the same instruction the readers use)
template <int DT>
__device__ __forceinline__ unsigned short deq_one(int code, unsigned short scale, unsigned short zero) {
  if (DT == MC_F16) {
    return __half_as_ushort(__hfma(__int2half_rn(code), __ushort_as_half(scale), __ushort_as_half(zero)));
  }
  return __bfloat16_as_ushort(__hfma(__int2bfloat16_rn(code), __ushort_as_bfloat16(scale), __ushort_as_bfloat16(zero)));
}

// code = clamp(rint((x - zero) / scale), 0, 15) as the double-precision quantiser defines it, at single-precision
// cost: the fp32 quotient is within 1e-5 of the exact one (operands of at most 11 significant bits), so it
// rounds to the same integer unless it lies that close to a tie -- only then is the quotient formed in double.
__device__ __forceinline__ int q4_code(float x, float z, float s, float inv_s) {
  const float qf = (x - z) * inv_s;
  float r = rintf(qf);
  if (fabsf(fabsf(qf - r) - 0.5f) < 1e-3f) r = (float)rint(((double)x - (double)z) / (double)s);
  return (int)fminf(fmaxf(r, 0.f), 15.f);
}

// Shared memory of one tile conversion.
struct QTileSmem {
  unsigned short rows[kQ4Page][kHeadDim];  // the 16-bit directions, channels in natural order
  float g[2][kQ4Page];                     // the two layers' scales of the 16-bit tile
  unsigned char codes[kQ4Page][kHeadDim];
  unsigned short scale[kQ4Page * 4];       // K: [128] per channel; V: [32][4] per (token, channel group)
  unsigned short zero[kQ4Page * 4];
};

// A 16-bit tile (page_size 32, chunks permuted) from global memory into QTileSmem::rows / g.
// Plain loads: the tile may have been written by this very block a moment ago.
__device__ __forceinline__ void load_tile16(const char* src, QTileSmem& sm) {
  for (int idx = threadIdx.x; idx < kResTileBytes / 16; idx += kQThreads) {
    const uint4 v = *reinterpret_cast<const uint4*>(src + (size_t)idx * 16);
    if (idx < kQ4Page * 16) {
      const int r = idx >> 4, pos = idx & 15;
      const int c = (pos & 8) | ((pos & 7) ^ (r & 7));  // the chunk stored at this position
      *reinterpret_cast<uint4*>(&sm.rows[r][c * 8]) = v;
    } else {
      *reinterpret_cast<uint4*>(&sm.g[0][0] + (idx - kQ4Page * 16) * 4) = v;
    }
  }
}

// Quantises the tile in `sm` (32 complete tokens) and writes the 4-bit tile to `dst`.
template <int DT>
__device__ void quantise_tile(int tensor, QTileSmem& sm, char* dst) {
  const int tid = threadIdx.x;
  __syncthreads();
  // ---- groups: extremes, scale, zero, codes
  if (tensor == 0) {
    const int c = tid;  // a channel over the page's 32 tokens
    float lo = elem_to_float<DT>(sm.rows[0][c]), hi = lo;
    for (int r = 1; r < kQ4Page; ++r) {
      const float x = elem_to_float<DT>(sm.rows[r][c]);
      lo = fminf(lo, x);
      hi = fmaxf(hi, x);
    }
    unsigned short s16 = double_to_elem<DT>(((double)hi - (double)lo) / 15.0);
    if (elem_to_float<DT>(s16) == 0.f) s16 = double_to_elem<DT>(1.0);  // a constant group
    const unsigned short z16 = double_to_elem<DT>((double)lo);
    const float sf = elem_to_float<DT>(s16), zf = elem_to_float<DT>(z16), inv_s = 1.0f / sf;
    for (int r = 0; r < kQ4Page; ++r) sm.codes[r][c] = (unsigned char)q4_code(elem_to_float<DT>(sm.rows[r][c]), zf, sf, inv_s);
    sm.scale[c] = s16;
    sm.zero[c] = z16;
  } else {
    const int r = tid >> 2, g = tid & 3;  // 32 channels of one token
    float lo = elem_to_float<DT>(sm.rows[r][32 * g]), hi = lo;
    for (int j = 1; j < 32; ++j) {
      const float x = elem_to_float<DT>(sm.rows[r][32 * g + j]);
      lo = fminf(lo, x);
      hi = fmaxf(hi, x);
    }
    unsigned short s16 = double_to_elem<DT>(((double)hi - (double)lo) / 15.0);
    if (elem_to_float<DT>(s16) == 0.f) s16 = double_to_elem<DT>(1.0);
    const unsigned short z16 = double_to_elem<DT>((double)lo);
    const float sf = elem_to_float<DT>(s16), zf = elem_to_float<DT>(z16), inv_s = 1.0f / sf;
    for (int j = 0; j < 32; ++j)
      sm.codes[r][32 * g + j] = (unsigned char)q4_code(elem_to_float<DT>(sm.rows[r][32 * g + j]), zf, sf, inv_s);
    sm.scale[r * 4 + g] = s16;
    sm.zero[r * 4 + g] = z16;
  }
  __syncthreads();
  // ---- the scales of Eq. 2 refer to the stored direction: |x| / |e_q| = g16 * |e_16| / |e_q|
  {
    const int r = tid >> 2, qd = tid & 3;
    double ss16 = 0.0, ssq = 0.0;
    for (int j = 0; j < 32; ++j) {
      const int c = 32 * qd + j;
      const int mi = tensor == 0 ? c : r * 4 + qd;
      const double e16 = (double)elem_to_float<DT>(sm.rows[r][c]);
      const double eq = (double)elem_to_float<DT>(deq_one<DT>(sm.codes[r][c], sm.scale[mi], sm.zero[mi]));
      ss16 += e16 * e16;
      ssq += eq * eq;
    }
    ss16 += __shfl_xor_sync(0xffffffffu, ss16, 1);
    ssq += __shfl_xor_sync(0xffffffffu, ssq, 1);
    ss16 += __shfl_xor_sync(0xffffffffu, ss16, 2);
    ssq += __shfl_xor_sync(0xffffffffu, ssq, 2);
    if (qd < 2) {
      const float g16 = sm.g[qd][r];
      float gq = g16;  // -0 (a retained token) and 0 (a zero row) stay what they are
      if (g16 != 0.f) gq = (float)((double)g16 * sqrt(ss16 / (ssq > 0.0 ? ssq : ss16)));
      reinterpret_cast<float*>(dst + kQ4ScaleOff)[qd * kQ4Page + r] = gq;
    }
  }
  // ---- pack the codes and the group parameters in the tile's orders
  uint32_t* out_w = reinterpret_cast<uint32_t*>(dst);
  for (int wi = tid; wi < kQ4CodeBytes / 4; wi += kQThreads) {
    uint32_t w = 0;
    if (tensor == 0) {
      const int r = wi >> 4, wd = wi & 15;
#pragma unroll
      for (int p = 0; p < 4; ++p)
        w |= ((uint32_t)sm.codes[r][8 * wd + 2 * p] << (4 * p)) | ((uint32_t)sm.codes[r][8 * wd + 2 * p + 1] << (16 + 4 * p));
    } else {
      const int i = wi >> 5, cp = (wi >> 2) & 7, k = wi & 3;
      const int c = q4_vchunk_pos(i, cp);  // (an involution: the chunk stored at position cp)
#pragma unroll
      for (int n = 0; n < 4; ++n) {
        const int ch = q4_vchannel(c, k, n);
        w |= ((uint32_t)sm.codes[2 * i][ch] << (4 * n)) | ((uint32_t)sm.codes[2 * i + 1][ch] << (16 + 4 * n));
      }
    }
    out_w[wi] = w;
  }
  {
    uint32_t w;
    if (tensor == 0) {
      const int q = tid >> 2, j = tid & 3;  // chunk position (16 of scales, 16 of zeros), word
      const int qq = q & 15;
      const int o = 4 * (qq & 3) + (qq >> 2);  // the channel octet whose chunk sits at position qq
      const unsigned short* m = (q >> 4) ? sm.zero : sm.scale;
      w = (uint32_t)m[8 * o + 2 * j] | ((uint32_t)m[8 * o + 2 * j + 1] << 16);
    } else {
      const int i = tid >> 3, j = tid & 7;  // token pair, word: four of scales, four of zeros
      const unsigned short* m = (j >> 2) ? sm.zero : sm.scale;
      w = (uint32_t)m[(2 * i) * 4 + (j & 3)] | ((uint32_t)m[(2 * i + 1) * 4 + (j & 3)] << 16);
    }
    out_w[kQ4CodeBytes / 4 + tid] = w;
  }
}

struct Q4Params {
  Geom g;
  const char* stage[2];  // 16-bit tiles of the merge [n_pages][H][kResTileBytes]: K, V
  char* e_pool[2];       // 4-bit tiles
  char* res[2];          // residual tiles [batch][H][kResTileBytes]
  int32_t* status;
};

template <int DT>
__global__ void __launch_bounds__(kQThreads) q4_quantise_pages_kernel(const Q4Params p) {
  grid_dep_wait();
  grid_dep_launch();
  __shared__ __align__(16) QTileSmem sm;
  const int H = p.g.n_kv_heads;
  const int tensor = blockIdx.x / H, h = blockIdx.x % H, pslot = blockIdx.y, b = blockIdx.z;
  const int n = checked_len(p.g, b, p.status);
  if (pslot * kQ4Page >= n) return;
  const int page = checked_page(p.g, b, pslot, p.status);
  if (page < 0) return;
  const char* src = p.stage[tensor] + ((size_t)page * H + h) * kResTileBytes;
  if ((pslot + 1) * kQ4Page <= n) {
    load_tile16(src, sm);
    quantise_tile<DT>(tensor, sm, p.e_pool[tensor] + ((size_t)page * H + h) * kQ4TileBytes);
  } else {
    char* dst = p.res[tensor] + ((size_t)b * H + h) * kResTileBytes;
    for (int idx = threadIdx.x; idx < kResTileBytes / 16; idx += kQThreads)
      reinterpret_cast<uint4*>(dst)[idx] = reinterpret_cast<const uint4*>(src)[idx];
  }
}

// ---------------------------------------------------------------------------------------------
struct AppendQ4Params {
  Geom g;
  const char* a_new[2];  // [batch][H][128]: K, V of layer l-1
  const char* c_new[2];
  char* e_pool[2];
  char* res[2];
  float* dist;
  float ta, tc;
  int merge_fn;
  int t_mode;
  int32_t* status;
  AppendKeep keep;
};

template <int DT>
__global__ void __launch_bounds__(kQThreads) append_q4_kernel(const AppendQ4Params p) {
  grid_dep_launch();
  __shared__ __align__(16) QTileSmem sm;
  const int H = p.g.n_kv_heads;
  const int tensor = blockIdx.x / H, h = blockIdx.x % H, b = blockIdx.y;
  // the batch description belongs to the caller: where the row goes is looked up before the wait on
  // the kernel ahead in the stream; what does not fit the declared bounds is flagged after it
  const int tok = p.g.seq_lens[b];
  int page = -1;
  if (tok >= 0 && tok <= p.g.max_seq_len && (tok >> 5) < p.g.max_pages_per_seq)
    page = p.g.block_table[(size_t)b * p.g.max_pages_per_seq + (tok >> 5)];
  grid_dep_wait();
  if (!page_ok(p.g, page)) {
    if (threadIdx.x == 0) atomicOr(p.status, MC_FLAG_BAD_METADATA);
    return;
  }
  const int slot = tok & (kQ4Page - 1);
  char* res = p.res[tensor] + ((size_t)b * H + h) * kResTileBytes;
  if (threadIdx.x < 32) {  // one warp merges the row (a half-warp's worth; the other half mirrors it)
    const int l16 = threadIdx.x & 15;
    const size_t off = ((size_t)b * H + h) * kRowBytes + l16 * 16;
    const uint4 va = *reinterpret_cast<const uint4*>(p.a_new[tensor] + off);
    const uint4 vc = *reinterpret_cast<const uint4*>(p.c_new[tensor] + off);
    uint4 e;
    float ga, gc, d;
    merge_row<DT>(va, vc, p.ta, p.tc, p.merge_fn, p.t_mode, e, ga, gc, d);
    if (p.keep.slack > 0) {  // (uniform over the block) Eq. 4 for the new token, against the stored extremes
      const int seg = (tensor * p.g.batch + b) * H + h;
      bool keep = append_keeps(p.keep, seg, d);
      if (p.keep.union_kv) {  // the other tensor's rule, on its own new rows, counts as well
        const uint4 oa = *reinterpret_cast<const uint4*>(p.a_new[1 - tensor] + off);
        const uint4 oc = *reinterpret_cast<const uint4*>(p.c_new[1 - tensor] + off);
        uint4 e_o;
        float ga_o, gc_o, d_o;
        merge_row<DT>(oa, oc, p.ta, p.tc, p.merge_fn, p.t_mode, e_o, ga_o, gc_o, d_o);
        keep = keep || append_keeps(p.keep, ((1 - tensor) * p.g.batch + b) * H + h, d_o);
      }
      keep = __shfl_sync(0xffffffffu, (int)keep, 0) != 0;
      if (keep && threadIdx.x < 16 && append_retain(p.keep, seg, tok, l16, va, vc, p.status)) ga = gc = -0.f;
    }
    if (threadIdx.x < 16) {
      *reinterpret_cast<uint4*>(res + slot * kRowBytes + chunk_pos(slot, l16) * 16) = e;
      if (l16 == 0) {
        float* sc = reinterpret_cast<float*>(res + kQ4Page * kRowBytes) + slot;
        sc[0] = ga;
        sc[kQ4Page] = gc;
        p.dist[(((size_t)page * H + h) * 2 + tensor) * kQ4Page + slot] = d;
      }
    }
  }
  if (slot != kQ4Page - 1) return;
  // the page is complete: its 32 rows leave the residual tile as a 4-bit tile
  __syncthreads();
  load_tile16(res, sm);
  quantise_tile<DT>(tensor, sm, p.e_pool[tensor] + ((size_t)page * H + h) * kQ4TileBytes);
}

// ---------------------------------------------------------------------------------------------
struct RestoreQ4Params {
  Geom g;
  const char* e_pool[2];
  const char* res[2];
  char* dst_pool[2];
  const int32_t* ret_count;
  const int32_t* ret_offset;
  const int32_t* ret_index;
  const char* ret_rows;
  int64_t ret_capacity;
  int layer;
  int32_t* status;
};

template <int DT, bool F32>
__global__ void __launch_bounds__(kQThreads) restore_q4_kernel(const RestoreQ4Params p) {
  constexpr int kOutRow = F32 ? 2 * kRowBytes : kRowBytes;
  grid_dep_wait();
  grid_dep_launch();
  __shared__ __align__(16) float out_s[kQ4Page][kHeadDim + 4];
  __shared__ __align__(16) unsigned char tile_s[kResTileBytes];
  const int H = p.g.n_kv_heads;
  const int tensor = blockIdx.x / H, h = blockIdx.x % H, pslot = blockIdx.y, b = blockIdx.z;
  const int tid = threadIdx.x;
  const int n = checked_len(p.g, b, p.status);
  if (pslot * kQ4Page >= n) return;
  const int page = checked_page(p.g, b, pslot, p.status);
  if (page < 0) return;
  const int valid = min(kQ4Page, n - pslot * kQ4Page);
  const float* g_s;
  if (valid == kQ4Page) {
    const char* src = p.e_pool[tensor] + ((size_t)page * H + h) * kQ4TileBytes;
    for (int idx = tid; idx < kQ4TileBytes / 16; idx += kQThreads)
      reinterpret_cast<uint4*>(tile_s)[idx] = reinterpret_cast<const uint4*>(src)[idx];
    __syncthreads();
    g_s = reinterpret_cast<const float*>(tile_s + kQ4ScaleOff) + p.layer * kQ4Page;
    const uint32_t* meta = reinterpret_cast<const uint32_t*>(tile_s + kQ4CodeBytes);
    if (tensor == 0) {
      const int r = tid >> 2, qd = tid & 3;
      const float g = g_s[r];
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        const int o = 4 * qd + k;
        const uint32_t w = reinterpret_cast<const uint32_t*>(tile_s + r * 64)[o];
        const uint32_t* s4 = meta + q4_kmeta_pos(o) * 4;
        const uint32_t* z4 = s4 + 64;
        uint32_t c[4];
        code_pairs<DT>(w, c);
#pragma unroll
        for (int pr = 0; pr < 4; ++pr) {
          const float2 v = Elem<DT>::unpack(deq_pair<DT>(c[pr], s4[pr], z4[pr]));
          out_s[r][8 * o + 2 * pr] = v.x * g;
          out_s[r][8 * o + 2 * pr + 1] = v.y * g;
        }
      }
    } else {
      const int i = tid >> 3, c8 = tid & 7;
      const float g0 = g_s[2 * i], g1 = g_s[2 * i + 1];
      const uint4 wv = *reinterpret_cast<const uint4*>(tile_s + i * 128 + q4_vchunk_pos(i, c8) * 16);
      const uint32_t ws[4] = {wv.x, wv.y, wv.z, wv.w};
      const uint32_t* s4 = meta + i * 8;
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        uint32_t c[4];
        code_pairs<DT>(ws[k], c);
#pragma unroll
        for (int nn = 0; nn < 4; ++nn) {
          const float2 v = Elem<DT>::unpack(deq_pair<DT>(c[nn], s4[k], s4[4 + k]));
          const int ch = q4_vchannel(c8, k, nn);
          out_s[2 * i][ch] = v.x * g0;
          out_s[2 * i + 1][ch] = v.y * g1;
        }
      }
    }
  } else {
    const char* src = p.res[tensor] + ((size_t)b * H + h) * kResTileBytes;
    for (int idx = tid; idx < kResTileBytes / 16; idx += kQThreads)
      reinterpret_cast<uint4*>(tile_s)[idx] = reinterpret_cast<const uint4*>(src)[idx];
    __syncthreads();
    g_s = reinterpret_cast<const float*>(tile_s + kQ4Page * kRowBytes) + p.layer * kQ4Page;
    for (int idx = tid; idx < kQ4Page * 16; idx += kQThreads) {
      const int r = idx >> 4, c = idx & 15;
      const uint4 v = *reinterpret_cast<const uint4*>(tile_s + r * kRowBytes + chunk_pos(r, c) * 16);
      const uint32_t w[4] = {v.x, v.y, v.z, v.w};
      const float g = g_s[r];
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const float2 f = Elem<DT>::unpack(w[j]);
        out_s[r][8 * c + 2 * j] = f.x * g;
        out_s[r][8 * c + 2 * j + 1] = f.y * g;
      }
    }
  }
  __syncthreads();
  // the scaled rows leave in natural order; a retained token (scale -0) is written from its raw row below
  char* dst = p.dst_pool[tensor] + ((size_t)page * H + h) * kQ4Page * kOutRow;
  for (int idx = tid; idx < kQ4Page * 16; idx += kQThreads) {
    const int r = idx >> 4, c = idx & 15;
    if (r >= valid || __float_as_uint(g_s[r]) == 0x80000000u) continue;
    const float* f = &out_s[r][8 * c];
    if (F32) {
      float4* d4 = reinterpret_cast<float4*>(dst + (size_t)r * kOutRow + c * 32);
      d4[0] = make_float4(f[0], f[1], f[2], f[3]);
      d4[1] = make_float4(f[4], f[5], f[6], f[7]);
    } else {
      *reinterpret_cast<uint4*>(dst + (size_t)r * kOutRow + c * 16) =
          make_uint4(Elem<DT>::pack(f[0], f[1]), Elem<DT>::pack(f[2], f[3]), Elem<DT>::pack(f[4], f[5]), Elem<DT>::pack(f[6], f[7]));
    }
  }
  // ---- x_hat[I] = R: the block of a segment's first page writes the segment's raw rows
  if (pslot != 0) return;
  const int seg = (tensor * p.g.batch + b) * H + h;
  const int cnt = p.ret_count[seg], off = p.ret_offset[seg];
  const int l16 = tid & 15;
  for (int e = tid >> 4; e < cnt; e += kQThreads / 16) {
    if (!MC_IN_BOUNDS(off >= 0 && (int64_t)off + e < p.ret_capacity, p.status)) continue;  // (range-checked build)
    const int tok = p.ret_index[off + e];
    if (!MC_IN_BOUNDS(tok >= 0 && tok < n, p.status)) continue;
    const int pg = checked_page(p.g, b, tok >> 5, p.status);
    if (pg < 0) continue;
    const size_t row = ((size_t)pg * H + h) * kQ4Page + (tok & (kQ4Page - 1));
    const uint4 v = *reinterpret_cast<const uint4*>(p.ret_rows + ((size_t)p.layer * p.ret_capacity + off + e) * kRetEntryBytes + l16 * 16);
    if (F32) {
      const float2 f0 = Elem<DT>::unpack(v.x), f1 = Elem<DT>::unpack(v.y), f2 = Elem<DT>::unpack(v.z), f3 = Elem<DT>::unpack(v.w);
      float4* d4 = reinterpret_cast<float4*>(p.dst_pool[tensor] + row * kOutRow + l16 * 32);
      d4[0] = make_float4(f0.x, f0.y, f1.x, f1.y);
      d4[1] = make_float4(f2.x, f2.y, f3.x, f3.y);
    } else {
      *reinterpret_cast<uint4*>(p.dst_pool[tensor] + row * kRowBytes + l16 * 16) = v;
    }
  }
}

// ---------------------------------------------------------------------------------------------
// Host launchers
// ---------------------------------------------------------------------------------------------
size_t q4_stage_bytes(const mc_config* cfg, const mc_batch* bt) {
  return align_up((size_t)bt->n_pages * cfg->n_kv_heads * kResTileBytes, 256);
}

static int q4_page_slots(const mc_batch* bt) { return std::max(1, (bt->max_seq_len + kQ4Page - 1) / kQ4Page); }

mc_status launch_q4_quantise(const mc_config* cfg, const mc_batch* bt, const Geom& g, const void* stage_k, const void* stage_v,
                             const mc_pair_cache* out, cudaStream_t stream) {
  if (bt->batch == 0) return MC_OK;
  if (q4_page_slots(bt) > 65535 || bt->batch > 65535) return MC_ERR_SHAPE;
  Q4Params qp;
  qp.g = g;
  qp.stage[0] = (const char*)stage_k;
  qp.stage[1] = (const char*)stage_v;
  qp.e_pool[0] = (char*)out->e_k;
  qp.e_pool[1] = (char*)out->e_v;
  qp.res[0] = (char*)out->res_k;
  qp.res[1] = (char*)out->res_v;
  qp.status = out->status;
  const dim3 grid(2 * cfg->n_kv_heads, q4_page_slots(bt), bt->batch);
  if (cfg->dtype == MC_F16)
    MC_CUDA_CHECK(launch_pdl(q4_quantise_pages_kernel<MC_F16>, grid, dim3(kQThreads), 0, stream, qp));
  else
    MC_CUDA_CHECK(launch_pdl(q4_quantise_pages_kernel<MC_BF16>, grid, dim3(kQThreads), 0, stream, qp));
  MC_CUDA_CHECK(cudaGetLastError());
  return MC_OK;
}

mc_status launch_append_q4(const mc_config* cfg, const mc_batch* bt, const Geom& g, const mc_pair_cache* pair,
                           const void* k_new_lm1, const void* v_new_lm1, const void* k_new_l, const void* v_new_l,
                           cudaStream_t stream) {
  if (bt->batch == 0) return MC_OK;
  AppendQ4Params ap;
  ap.g = g;
  ap.a_new[0] = (const char*)k_new_lm1;
  ap.a_new[1] = (const char*)v_new_lm1;
  ap.c_new[0] = (const char*)k_new_l;
  ap.c_new[1] = (const char*)v_new_l;
  ap.e_pool[0] = (char*)pair->e_k;
  ap.e_pool[1] = (char*)pair->e_v;
  ap.res[0] = (char*)pair->res_k;
  ap.res[1] = (char*)pair->res_v;
  ap.dist = pair->dist;
  ap.merge_fn = cfg->merge_fn;
  ap.t_mode = cfg->t_mode;
  ap.ta = (float)(1.0 - cfg->t);
  ap.tc = (float)cfg->t;
  ap.status = pair->status;
  ap.keep = make_append_keep(cfg, pair);
  const dim3 grid(2 * cfg->n_kv_heads, bt->batch);
  if (cfg->dtype == MC_F16)
    MC_CUDA_CHECK(launch_pdl(append_q4_kernel<MC_F16>, grid, dim3(kQThreads), 0, stream, ap));
  else
    MC_CUDA_CHECK(launch_pdl(append_q4_kernel<MC_BF16>, grid, dim3(kQThreads), 0, stream, ap));
  MC_CUDA_CHECK(cudaGetLastError());
  return MC_OK;
}

mc_status launch_restore_q4(const mc_config* cfg, const mc_batch* bt, const Geom& g, const mc_pair_cache* pair, int layer,
                            const mc_layer_kv* dst, int dst_fp32, cudaStream_t stream) {
  if (bt->batch == 0) return MC_OK;
  if (q4_page_slots(bt) > 65535 || bt->batch > 65535) return MC_ERR_SHAPE;
  RestoreQ4Params rp;
  rp.g = g;
  rp.e_pool[0] = (const char*)pair->e_k;
  rp.e_pool[1] = (const char*)pair->e_v;
  rp.res[0] = (const char*)pair->res_k;
  rp.res[1] = (const char*)pair->res_v;
  rp.dst_pool[0] = (char*)dst->k_pool;
  rp.dst_pool[1] = (char*)dst->v_pool;
  rp.ret_count = pair->ret_count;
  rp.ret_offset = pair->ret_offset;
  rp.ret_index = pair->ret_index;
  rp.ret_rows = (const char*)pair->ret_rows;
  rp.ret_capacity = pair->ret_capacity;
  rp.layer = layer;
  rp.status = pair->status;
  const dim3 grid(2 * cfg->n_kv_heads, q4_page_slots(bt), bt->batch);
  void (*kern)(const RestoreQ4Params) =
      cfg->dtype == MC_F16 ? (dst_fp32 ? restore_q4_kernel<MC_F16, true> : restore_q4_kernel<MC_F16, false>)
                           : (dst_fp32 ? restore_q4_kernel<MC_BF16, true> : restore_q4_kernel<MC_BF16, false>);
  MC_CUDA_CHECK(launch_pdl(kern, grid, dim3(kQThreads), 0, stream, rp));
  MC_CUDA_CHECK(cudaGetLastError());
  return MC_OK;
}

}  // namespace mc

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
#include "mc_items.cuh"
#include "mc_pipe.cuh"
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
// rounds to the same integer unless it lies that close to a tie -- only then is the quotient formed in double
// (out of line: the kernels stay small enough for the instruction cache).  zero is the group's minimum, so the
// quotient is never negative, and at most 15 plus the rounding of the scale: adding 1.5 * 2^23 leaves rint(q)
// in the sum's last mantissa bits, with no conversion instruction.
__device__ __noinline__ int q4_code_exact(float x, float z, float s) {
  const double r = rint(((double)x - (double)z) / (double)s);
  return (int)fmin(fmax(r, 0.0), 15.0);
}
__device__ __forceinline__ int q4_code(float x, float z, float s, float inv_s) {
  const float qf = (x - z) * inv_s;
  const float m = qf + 12582912.0f;
  const float r = m - 12582912.0f;
  if (fabsf(fabsf(qf - r) - 0.5f) < 1e-3f) return q4_code_exact(x, z, s);
  return min(__float_as_int(m) & 31, 15);
}

// Shared memory of one tile conversion.
struct QTileSmem {
  // two 16-bit tiles (one being converted, one arriving): the directions, channels in natural order, and the
  // two layers' scales
  unsigned short rows[2][kQ4Page][kHeadDim];
  float g[2][2][kQ4Page];
  unsigned char codes[kQ4Page][kHeadDim + 8];  // (rows 34 words apart: the row-wise reads of a warp's rows fall into different banks)
  unsigned short scale[kQ4Page * 4];       // K: [128] per channel; V: [32][4] per (token, channel group)
  unsigned short zero[kQ4Page * 4];
  float4 mm[2][kHeadDim / 2];              // K: (min, max) of a channel pair over each half of the tokens
};

// A 16-bit tile (page_size 32, chunks permuted) from global memory into QTileSmem::rows[0] / g[0].
// Plain loads: the tile may have been written by this very block a moment ago.
__device__ __forceinline__ void load_tile16(const char* src, QTileSmem& sm) {
  for (int idx = threadIdx.x; idx < kResTileBytes / 16; idx += kQThreads) {
    const uint4 v = *reinterpret_cast<const uint4*>(src + (size_t)idx * 16);
    if (idx < kQ4Page * 16) {
      const int r = idx >> 4, pos = idx & 15;
      const int c = (pos & 8) | ((pos & 7) ^ (r & 7));  // the chunk stored at this position
      *reinterpret_cast<uint4*>(&sm.rows[0][r][c * 8]) = v;
    } else {
      *reinterpret_cast<uint4*>(&sm.g[0][0][0] + (idx - kQ4Page * 16) * 4) = v;
    }
  }
}

// Scale and zero of a group from its extremes: (max - min) / 15 and min, kept in the 16-bit type.
template <int DT>
__device__ __noinline__ void group_params(float lo, float hi, unsigned short& s16, unsigned short& z16) {
  s16 = double_to_elem<DT>(((double)hi - (double)lo) / 15.0);
  if (elem_to_float<DT>(s16) == 0.f) s16 = double_to_elem<DT>(1.0);  // a constant group
  z16 = double_to_elem<DT>((double)lo);
}
// Two codes (0..15) as exact integers of the 16-bit type, packed (the magic-number conversion of code_pairs).
template <int DT>
__device__ __forceinline__ uint32_t int_pair(int c0, int c1) {
  if (DT == MC_F16) {
    uint32_t r = (uint32_t)c0 | ((uint32_t)c1 << 16) | 0x64006400u;
    const __half2 v = __hsub2(*reinterpret_cast<__half2*>(&r), __half2half2(__ushort_as_half((unsigned short)0x6400)));
    return *reinterpret_cast<const uint32_t*>(&v);
  }
  uint32_t r = (uint32_t)c0 | ((uint32_t)c1 << 16) | 0x43004300u;
  const __nv_bfloat162 v = __hsub2(*reinterpret_cast<__nv_bfloat162*>(&r), __bfloat162bfloat162(__ushort_as_bfloat16((unsigned short)0x4300)));
  return *reinterpret_cast<const uint32_t*>(&v);
}
// Sum of the squares of eight values, pairwise (each product is exact in fp32 for 16-bit inputs).
__device__ __forceinline__ float sumsq8(const float2 (&v)[4]) {
  const float a = fmaf(v[0].y, v[0].y, v[0].x * v[0].x), b = fmaf(v[1].y, v[1].y, v[1].x * v[1].x);
  const float c = fmaf(v[2].y, v[2].y, v[2].x * v[2].x), d = fmaf(v[3].y, v[3].y, v[3].x * v[3].x);
  return (a + b) + (c + d);
}

// The chunk (8 channels of the thread's 32) that thread (row r, quarter q) of the row-wise phases takes in its
// turn jj: the rotation keeps the 16-byte shared-memory loads of a quarter-warp (two rows, four quarters) in
// different banks (rows are 64 words apart, quarters 16).
__device__ __forceinline__ int row_turn(int r, int q, int jj) { return (jj + (q >> 1) + 2 * (r & 1)) & 3; }

// Quantises the 16-bit tile in buffer `buf` of `sm` (32 complete tokens) and writes the 4-bit tile to `dst`.
// The two sums of squares behind a scale (|e_16|^2 and |e_q|^2 of a row) are accumulated in fp32 pairwise:
// seven roundings deep, so each is within 7 * 2^-24 of the exact sum and the scale within 5e-7 (relative) of
// g_16 |e_16| / |e_q|.
template <int DT>
__device__ void quantise_tile(int tensor, QTileSmem& sm, int buf, char* dst) {
  const int tid = threadIdx.x;
  const int r = tid >> 2, qd = tid & 3;  // the row-wise phases: four threads per token, 32 channels each
  const float inf = __int_as_float(0x7f800000);
  __syncthreads();
  float ss16 = 0.f, ssq = 0.f;
  if (tensor == 0) {
    // ---- keys: a group is a channel over the page's 32 tokens.  Two threads per channel pair (a 32-bit
    // word of a row), 16 tokens each; the extremes of the two halves meet in shared memory.
    const int cp = tid & 63, th = tid >> 6;
    const uint32_t* rows32 = reinterpret_cast<const uint32_t*>(&sm.rows[buf][0][0]);
    float2 x[16];
    float2 lo = make_float2(inf, inf), hi = make_float2(-inf, -inf);
#pragma unroll
    for (int i = 0; i < 16; ++i) {
      x[i] = Elem<DT>::unpack(rows32[(16 * th + i) * (kHeadDim / 2) + cp]);
      lo.x = fminf(lo.x, x[i].x);
      lo.y = fminf(lo.y, x[i].y);
      hi.x = fmaxf(hi.x, x[i].x);
      hi.y = fmaxf(hi.y, x[i].y);
    }
    sm.mm[th][cp] = make_float4(lo.x, hi.x, lo.y, hi.y);
    __syncthreads();
    const float4 o = sm.mm[1 - th][cp];
    unsigned short s0, z0, s1, z1;
    group_params<DT>(fminf(lo.x, o.x), fmaxf(hi.x, o.y), s0, z0);
    group_params<DT>(fminf(lo.y, o.z), fmaxf(hi.y, o.w), s1, z1);
    const float sf0 = elem_to_float<DT>(s0), zf0 = elem_to_float<DT>(z0), inv0 = 1.0f / sf0;
    const float sf1 = elem_to_float<DT>(s1), zf1 = elem_to_float<DT>(z1), inv1 = 1.0f / sf1;
#pragma unroll
    for (int i = 0; i < 16; ++i) {
      const int c0 = q4_code(x[i].x, zf0, sf0, inv0), c1 = q4_code(x[i].y, zf1, sf1, inv1);
      *reinterpret_cast<unsigned short*>(&sm.codes[16 * th + i][2 * cp]) = (unsigned short)(c0 | (c1 << 8));
    }
    if (th == 0) {
      reinterpret_cast<uint32_t*>(sm.scale)[cp] = (uint32_t)s0 | ((uint32_t)s1 << 16);
      reinterpret_cast<uint32_t*>(sm.zero)[cp] = (uint32_t)z0 | ((uint32_t)z1 << 16);
    }
    __syncthreads();
    // ---- row-wise: the two lengths of every token's direction
    const uint32_t* codes32 = reinterpret_cast<const uint32_t*>(&sm.codes[r][32 * qd]);
    const uint32_t* sc32 = reinterpret_cast<const uint32_t*>(sm.scale) + 16 * qd;
    const uint32_t* zr32 = reinterpret_cast<const uint32_t*>(sm.zero) + 16 * qd;
    float p16[4], pq[4];
#pragma unroll
    for (int jj = 0; jj < 4; ++jj) {
      const int q = row_turn(r, qd, jj);
      const uint4 v = *reinterpret_cast<const uint4*>(&sm.rows[buf][r][32 * qd + 8 * q]);
      const float2 e[4] = {Elem<DT>::unpack(v.x), Elem<DT>::unpack(v.y), Elem<DT>::unpack(v.z), Elem<DT>::unpack(v.w)};
      p16[jj] = sumsq8(e);
      // the codes of the same 8 channels: two words, the (scale, zero) pairs of their channel pairs beside them
      const uint2 cw = *reinterpret_cast<const uint2*>(codes32 + 2 * q);
      const uint4 s4 = *reinterpret_cast<const uint4*>(sc32 + 4 * q), z4 = *reinterpret_cast<const uint4*>(zr32 + 4 * q);
      const float2 d[4] = {Elem<DT>::unpack(deq_pair<DT>(int_pair<DT>(cw.x & 15u, (cw.x >> 8) & 15u), s4.x, z4.x)),
                           Elem<DT>::unpack(deq_pair<DT>(int_pair<DT>((cw.x >> 16) & 15u, cw.x >> 24), s4.y, z4.y)),
                           Elem<DT>::unpack(deq_pair<DT>(int_pair<DT>(cw.y & 15u, (cw.y >> 8) & 15u), s4.z, z4.z)),
                           Elem<DT>::unpack(deq_pair<DT>(int_pair<DT>((cw.y >> 16) & 15u, cw.y >> 24), s4.w, z4.w))};
      pq[jj] = sumsq8(d);
    }
    ss16 = (p16[0] + p16[1]) + (p16[2] + p16[3]);
    ssq = (pq[0] + pq[1]) + (pq[2] + pq[3]);
  } else {
    // ---- values: a group is 32 channels of one token: the thread's own 32 values, start to finish
    float2 x[4][4];
    float lo = inf, hi = -inf;
#pragma unroll
    for (int jj = 0; jj < 4; ++jj) {
      const int q = row_turn(r, qd, jj);
      const uint4 v = *reinterpret_cast<const uint4*>(&sm.rows[buf][r][32 * qd + 8 * q]);
      x[jj][0] = Elem<DT>::unpack(v.x);
      x[jj][1] = Elem<DT>::unpack(v.y);
      x[jj][2] = Elem<DT>::unpack(v.z);
      x[jj][3] = Elem<DT>::unpack(v.w);
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        lo = fminf(lo, fminf(x[jj][k].x, x[jj][k].y));
        hi = fmaxf(hi, fmaxf(x[jj][k].x, x[jj][k].y));
      }
    }
    unsigned short s16, z16;
    group_params<DT>(lo, hi, s16, z16);
    const float sf = elem_to_float<DT>(s16), zf = elem_to_float<DT>(z16), inv_s = 1.0f / sf;
    const uint32_t s2 = (uint32_t)s16 | ((uint32_t)s16 << 16), z2 = (uint32_t)z16 | ((uint32_t)z16 << 16);
    float p16[4], pq[4];
#pragma unroll
    for (int jj = 0; jj < 4; ++jj) {
      const int q = row_turn(r, qd, jj);
      int c[8];
      float2 d[4];
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        c[2 * k] = q4_code(x[jj][k].x, zf, sf, inv_s);
        c[2 * k + 1] = q4_code(x[jj][k].y, zf, sf, inv_s);
        d[k] = Elem<DT>::unpack(deq_pair<DT>(int_pair<DT>(c[2 * k], c[2 * k + 1]), s2, z2));
      }
      *reinterpret_cast<uint2*>(&sm.codes[r][32 * qd + 8 * q]) =
          make_uint2((uint32_t)c[0] | ((uint32_t)c[1] << 8) | ((uint32_t)c[2] << 16) | ((uint32_t)c[3] << 24),
                     (uint32_t)c[4] | ((uint32_t)c[5] << 8) | ((uint32_t)c[6] << 16) | ((uint32_t)c[7] << 24));
      p16[jj] = sumsq8(x[jj]);
      pq[jj] = sumsq8(d);
    }
    ss16 = (p16[0] + p16[1]) + (p16[2] + p16[3]);
    ssq = (pq[0] + pq[1]) + (pq[2] + pq[3]);
    sm.scale[r * 4 + qd] = s16;
    sm.zero[r * 4 + qd] = z16;
  }
  // ---- the scales of Eq. 2 refer to the stored direction: |x| / |e_q| = g16 * |e_16| / |e_q|
  ss16 += __shfl_xor_sync(0xffffffffu, ss16, 1);
  ssq += __shfl_xor_sync(0xffffffffu, ssq, 1);
  ss16 += __shfl_xor_sync(0xffffffffu, ss16, 2);
  ssq += __shfl_xor_sync(0xffffffffu, ssq, 2);
  if (qd < 2) {
    const float g16 = sm.g[buf][qd][r];
    float gq = g16;  // -0 (a retained token) and 0 (a zero row) stay what they are
    if (g16 != 0.f) gq = g16 * sqrtf(ss16 / (ssq > 0.f ? ssq : ss16));
    reinterpret_cast<float*>(dst + kQ4ScaleOff)[qd * kQ4Page + r] = gq;
  }
  __syncthreads();
  // ---- pack the codes and the group parameters in the tile's orders
  uint32_t* out_w = reinterpret_cast<uint32_t*>(dst);
  for (int wi = tid; wi < kQ4CodeBytes / 4; wi += kQThreads) {
    uint32_t w = 0;
    if (tensor == 0) {
      const int rr = wi >> 4, wd = wi & 15;
      const uint2 b = *reinterpret_cast<const uint2*>(&sm.codes[rr][8 * wd]);  // codes of channels 8 wd .. 8 wd + 7
      // even channels to the nibbles 0..3, odd ones to the nibbles 4..7
      w = (b.x & 0xFu) | ((b.x >> 12) & 0xF0u) | ((b.y & 0xFu) << 8) | ((b.y >> 4) & 0xF000u) |
          ((b.x << 8) & 0xF0000u) | ((b.x >> 4) & 0xF00000u) | ((b.y << 16) & 0xF000000u) | ((b.y << 4) & 0xF0000000u);
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

// One 16-bit tile of the merge's staging area and where it goes.
struct QTile {
  int b, pslot, th;  // sequence, page slot, tensor * H + head
  int raw_page;      // page id as read from the block table (validated when the tile's turn comes)
  bool valid;        // false: past the last tile
};

// Persistent over the used pages of the call's sequences (tile index = page * 2 H + tensor * H + head, pages
// counted through the sequences): while a tile is converted, the next one's 16-bit tile is already on its way
// into registers and the page id of the one after that is being read, so the conversion of a tile does not
// start with two dependent trips to memory.
template <int DT>
__global__ void __launch_bounds__(kQThreads, 6) q4_quantise_pages_kernel(const Q4Params p) {
  grid_dep_wait();
  grid_dep_launch();
  __shared__ __align__(16) QTileSmem sm;
  __shared__ int len_s[kMaxBatchPages];
  __shared__ int pre_s[kMaxBatchPages + 1];
  const int H = p.g.n_kv_heads;
  page_prefix(p.g, len_s, pre_s, kQThreads, p.status);
  const long long total = (long long)pre_s[p.g.batch] * 2 * H;
  int b_run = 0;  // (tile indices only grow: the sequence is found by stepping forward)
  auto tile_at = [&](long long t) {
    QTile q;
    q.valid = t < total;
    q.b = q.pslot = q.th = 0;
    q.raw_page = -1;
    if (!q.valid) return q;
    const int pg = (int)(t / (2 * H));
    q.th = (int)(t - (long long)pg * 2 * H);
    while (pg >= pre_s[b_run + 1]) ++b_run;
    q.b = b_run;
    q.pslot = pg - pre_s[b_run];
    if (q.pslot < p.g.max_pages_per_seq) q.raw_page = p.g.block_table[(size_t)q.b * p.g.max_pages_per_seq + q.pslot];
    return q;
  };
  auto full_page = [&](const QTile& q) { return (q.pslot + 1) * kQ4Page <= len_s[q.b]; };
  auto page_of = [&](const QTile& q) {  // -1 (and the flag) for an id outside the pools
    if (page_ok(p.g, q.raw_page)) return q.raw_page;
    if (threadIdx.x == 0) atomicOr(p.status, MC_FLAG_BAD_METADATA);
    return -1;
  };
  // the tile's 16-bit rows (chunks put back in channel order) and scales, asynchronously into buffer `buf`
  auto fetch = [&](const QTile& q, int buf) {
    const int page = q.valid && full_page(q) ? page_of(q) : -1;
    if (page >= 0) {
      const char* src = p.stage[q.th / H] + ((size_t)page * H + q.th % H) * kResTileBytes;
      for (int idx = threadIdx.x; idx < kResTileBytes / 16; idx += kQThreads) {
        const int r = idx >> 4, pos = idx & 15;
        const int c = (pos & 8) | ((pos & 7) ^ (r & 7));  // the chunk stored at this position
        void* dst = idx < kQ4Page * 16 ? (void*)&sm.rows[buf][r][c * 8] : (void*)(&sm.g[buf][0][0] + (idx - kQ4Page * 16) * 4);
        asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(smem_u32(dst)), "l"(src + (size_t)idx * 16) : "memory");
      }
    }
    asm volatile("cp.async.commit_group;" ::: "memory");
  };
  const long long stride = gridDim.x;
  QTile cur = tile_at(blockIdx.x);
  QTile nxt = tile_at(blockIdx.x + stride);
  fetch(cur, 0);
  int buf = 0;
  for (long long t = blockIdx.x; cur.valid; t += stride, buf ^= 1) {
    const int tensor = cur.th / H, h = cur.th % H;
    const bool full = full_page(cur);
    const int page = full ? (page_ok(p.g, cur.raw_page) ? cur.raw_page : -1) : page_of(cur);  // (a full page was checked by fetch)
    asm volatile("cp.async.wait_group 0;" ::: "memory");
    __syncthreads();  // this tile has arrived; the other buffer's tile is converted and gone
    fetch(nxt, buf ^ 1);
    const QTile nxt2 = tile_at(t + 2 * stride);
    if (full && page >= 0) {
      quantise_tile<DT>(tensor, sm, buf, p.e_pool[tensor] + ((size_t)page * H + h) * kQ4TileBytes);
    } else if (page >= 0) {  // the sequence's last, incomplete page: to its residual tile as it is
      const char* src = p.stage[tensor] + ((size_t)page * H + h) * kResTileBytes;
      char* dst = p.res[tensor] + ((size_t)cur.b * H + h) * kResTileBytes;
      for (int idx = threadIdx.x; idx < kResTileBytes / 16; idx += kQThreads)
        reinterpret_cast<uint4*>(dst)[idx] = reinterpret_cast<const uint4*>(src)[idx];
    }
    cur = nxt;
    nxt = nxt2;
  }
  asm volatile("cp.async.wait_group 0;" ::: "memory");
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
  quantise_tile<DT>(tensor, sm, 0, p.e_pool[tensor] + ((size_t)page * H + h) * kQ4TileBytes);
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
  if (bt->batch > kMaxBatchPages) return MC_ERR_SHAPE;  // the sequences' page prefix lives in shared memory
  const long long tiles = (long long)bt->batch * q4_page_slots(bt) * 2 * cfg->n_kv_heads;  // (an upper bound)
  int n_sm = 0;
  if (mc_status st = sm_count(&n_sm)) return st;
  const dim3 grid((unsigned)std::max<long long>(1, std::min<long long>(tiles, (long long)n_sm * 6)));
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
